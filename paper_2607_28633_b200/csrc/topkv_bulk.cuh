// Bulk-async page copy for sm_100a: a persistent grid whose warps each run a private
// multi-stage ring in shared memory. Global -> shared copies are cp.async.bulk completing on
// an mbarrier; shared -> global copies are cp.async.bulk bulk-groups. No thread ever touches
// the payload: the warp only computes addresses and issues copies, one lane per copy.
//
// Work item = a run of up to `tpc` tokens of one page. Its image in shared memory is laid
// out in WIRE order, so the wire side is one copy (F copies for the PLANAR order) and the
// pool side is one copy per unit (one per plane when tokens are contiguous on both sides).
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "topkv_common.cuh"

namespace topkv {

constexpr int kBulkWarps = 2;       // independent pipelines per CTA
constexpr int kBulkThreads = kBulkWarps * 32;
constexpr int kBulkMaxStages = 8;
constexpr int kBulkMaxR = TOPKV_MAX_INLINE_R;
constexpr uint32_t kWaitPollLimit = 1u << 22;  // bounded mbarrier wait (each poll may suspend)

struct BulkParams {
  KParams k;
  int tpc;          // tokens per work item
  int cpp;          // work items per page = ceil(P / tpc)
  int stage_bytes;  // bytes of one ring stage (>= tpc * F * U * unit_bytes), multiple of 128
  int nstages;      // ring depth per warp
  int merged;       // pool side: one copy per plane
};

struct ItemDesc {
  uint8_t* pool_page;
  int64_t n_first;  // global index of the item's first token
  int t0, nt;       // first token inside the page, number of tokens
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

template <int F, bool PACK>
__global__ void __launch_bounds__(kBulkThreads, 1) topkv_bulk_kernel(const BulkParams bp) {
  extern __shared__ __align__(128) uint8_t smem[];
  const KParams& p = bp.k;
  pdl_prologue(p.overlap);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int S = bp.nstages;

  // shared memory map: [kBulkWarps * S stages][mbarriers][item descriptors][cu int32][pc int32]
  uint8_t* stage_base = smem + (size_t)warp * S * bp.stage_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)kBulkWarps * S * bp.stage_bytes);
  ItemDesc* descs = reinterpret_cast<ItemDesc*>(bars + kBulkWarps * kBulkMaxStages);
  int32_t* s_cu = reinterpret_cast<int32_t*>(descs + kBulkWarps * kBulkMaxStages);  // [R+1] tokens
  int32_t* s_pc = s_cu + (p.R + 1);                                                 // [R+1] pages
  uint64_t* my_bars = bars + warp * kBulkMaxStages;
  ItemDesc* my_descs = descs + warp * kBulkMaxStages;

  // ---- per-CTA plan: token and page prefix sums in shared memory (R <= kBulkMaxR) ----------
  for (int q = threadIdx.x; q < p.R; q += kBulkThreads) {
    int s = p.sl[q];
    const int64_t row_tokens = (int64_t)p.maxp * p.P;  // what one block-table row can describe
    if (s < 0 || s > row_tokens) {
      raise_error(kErrTable);
      s = s < 0 ? 0 : (int)row_tokens;
    }
    s_cu[q + 1] = s;
    s_pc[q + 1] = (s + p.P - 1) / p.P;
  }
  if (threadIdx.x == 0) {
    s_cu[0] = 0;
    s_pc[0] = 0;
  }
  if (lane == 0)
    for (int s = 0; s < S; ++s) mbar_init(smem_addr(&my_bars[s]), 1);
  __syncthreads();
  if (warp == 0) {  // inclusive scans, 32 entries per round
    int carry_c = 0, carry_p = 0;
    for (int base = 1; base <= p.R; base += 32) {
      const int q = base + lane;
      int c = q <= p.R ? s_cu[q] : 0, g = q <= p.R ? s_pc[q] : 0;
      for (int o = 1; o < 32; o <<= 1) {
        const int c2 = __shfl_up_sync(0xffffffffu, c, o), g2 = __shfl_up_sync(0xffffffffu, g, o);
        if (lane >= o) {
          c += c2;
          g += g2;
        }
      }
      if (q <= p.R) {
        s_cu[q] = c + carry_c;
        s_pc[q] = g + carry_p;
      }
      carry_c += __shfl_sync(0xffffffffu, c, 31);
      carry_p += __shfl_sync(0xffffffffu, g, 31);
    }
  }
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  __syncthreads();

  // rows from the K plane to the V plane of a PLANAR slab
  const int64_t T = p.plane_rows >= 0 ? p.plane_rows : ((p.T >= 0) ? p.T : (int64_t)s_cu[p.R]);
  {
    const int64_t row = (int64_t)p.U * p.unit_chunks * 16, S = s_cu[p.R];  // uniform over the grid
    const bool fits = p.planar ? ((F - 1) * T + S) * row <= p.wire_limit : S * F * row <= p.wire_limit;
    if (!fits) {
      if (threadIdx.x == 0) raise_error(kErrWire);
      pdl_epilogue(p.overlap);
      return;
    }
  }
  const int64_t unit_bytes = (int64_t)p.unit_chunks * 16;
  const int64_t total_items = (int64_t)s_pc[p.R] * bp.cpp;
  const int64_t gw = (int64_t)blockIdx.x * kBulkWarps + warp;
  const int64_t GW = (int64_t)gridDim.x * kBulkWarps;
  int64_t next_item = gw;

  // Advances to this warp's next non-empty item; fills d. Uniform across the warp.
  auto fetch = [&](ItemDesc& d) -> bool {
    while (next_item < total_items) {
      const int64_t it = next_item;
      next_item += GW;
      const int m = (int)(it / bp.cpp);
      const int k = (int)(it - (int64_t)m * bp.cpp);
      int lo = 0, hi = p.R;  // largest r with s_pc[r] <= m
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (s_pc[mid] <= m) lo = mid;
        else hi = mid;
      }
      const int r = lo, j = m - s_pc[r];
      const int s_r = s_cu[r + 1] - s_cu[r];
      const int first = j * p.P + k * bp.tpc;
      if (first >= s_r) continue;  // chunk past the end of a partial page
      d.t0 = k * bp.tpc;
      d.nt = min(min(bp.tpc, p.P - d.t0), s_r - first);
      d.n_first = (int64_t)s_cu[r] + first;
      const int64_t page = p.bt[(int64_t)r * p.maxp + j];
      if (page < 0 || page >= p.num_pages) {
        raise_error(kErrTable);
        continue;
      }
      d.pool_page = p.pool + page * p.S_page;
      return true;
    }
    return false;
  };

  // pool side of an item: copies between the pool and the stage image (wire order)
  auto pool_side = [&](const ItemDesc& d, uint32_t stage, uint32_t bar) {
    if (bp.merged) {
      if (lane < F) {
        const int c = lane;
        const uint32_t bytes = (uint32_t)(d.nt * unit_bytes);
        uint8_t* g = d.pool_page + c * p.S_kv + (int64_t)d.t0 * p.S_tok;
        const uint32_t s = stage + (uint32_t)c * bytes;
        if (PACK) bulk_g2s(s, g, bytes, bar);
        else bulk_s2g(g, s, bytes);
      }
      return;
    }
    const int units = d.nt * F * p.U;
    for (int q = lane; q < units; q += 32) {
      int h = 0, tc = q;
      if (p.U > 1) {
        tc = q / p.U;
        h = q - tc * p.U;
      }
      int c, t;
      if (p.planar) {
        c = tc / d.nt;
        t = tc - c * d.nt;
      } else {
        t = tc / F;
        c = tc - t * F;
      }
      uint8_t* g = d.pool_page + c * p.S_kv + (int64_t)(d.t0 + t) * p.S_tok + h * p.S_unit;
      const uint32_t s = stage + (uint32_t)(q * unit_bytes);
      if (PACK) bulk_g2s(s, g, (uint32_t)unit_bytes, bar);
      else bulk_s2g(g, s, (uint32_t)unit_bytes);
    }
  };

  // wire side of an item: one run, or one run per plane for the PLANAR order
  auto wire_side = [&](const ItemDesc& d, uint32_t stage, uint32_t bar) {
    const int64_t row = unit_bytes * p.U;
    if (!p.planar || F == 1) {
      if (lane == 0) {
        const uint32_t bytes = (uint32_t)(d.nt * F * row);
        uint8_t* g = p.wire + d.n_first * F * row;
        if (PACK) bulk_s2g(g, stage, bytes);
        else bulk_g2s(stage, g, bytes, bar);
      }
    } else if (lane < F) {
      const int c = lane;
      const uint32_t bytes = (uint32_t)(d.nt * row);
      uint8_t* g = p.wire + ((int64_t)c * T + d.n_first) * row;
      const uint32_t s = stage + (uint32_t)c * bytes;
      if (PACK) bulk_s2g(g, s, bytes);
      else bulk_g2s(s, g, bytes, bar);
    }
  };

  auto issue_loads = [&](int slot, const ItemDesc& d) {
    const uint32_t bar = smem_addr(&my_bars[slot]);
    const uint32_t stage = smem_addr(stage_base + (size_t)slot * bp.stage_bytes);
    if (lane == 0) {
      my_descs[slot] = d;
      mbar_expect_tx(bar, (uint32_t)(d.nt * F * p.U * unit_bytes));
    }
    __syncwarp();
    if (PACK) pool_side(d, stage, bar);
    else wire_side(d, stage, bar);
  };

  int issued = 0, consumed = 0;
  ItemDesc d;
  while (issued < S - 1 && fetch(d)) {
    issue_loads(issued % S, d);
    ++issued;
  }
  bool failed = false;
  while (consumed < issued) {
    const int slot = consumed % S;
    const uint32_t bar = smem_addr(&my_bars[slot]);
    const uint32_t parity = (uint32_t)(consumed / S) & 1u;
    uint32_t polls = 0;
    while (!mbar_try_wait(bar, parity)) {
      if (++polls > kWaitPollLimit) {
        failed = true;
        break;
      }
    }
    if (failed) break;
    const ItemDesc cur = my_descs[slot];
    const uint32_t stage = smem_addr(stage_base + (size_t)slot * bp.stage_bytes);
    if (PACK) wire_side(cur, stage, 0);
    else pool_side(cur, stage, 0);
    bulk_commit();
    ++consumed;
    if (fetch(d)) {
      bulk_wait_read<1>();  // the stage being refilled was drained one item ago
      __syncwarp();
      issue_loads(issued % S, d);
      ++issued;
    }
  }
  if (failed && lane == 0) raise_error(kErrWait);
  bulk_wait_all();
  pdl_epilogue(p.overlap);
}

}  // namespace topkv
