// Vectorised page copy (kernel family 0) and the plan kernel.
//
// pack / unpack with plain 16- or 32-byte global loads and stores: one CTA of 256 threads per
// span (one page, or up to 64 small pages of one request), every warp-wide access a fully
// coalesced 512 B or 1 KiB segment, 128 bytes per thread in flight before the first store.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "topkv_common.cuh"

namespace topkv {

constexpr int kThreads = 256;
constexpr int kMinCtasPerSm = 3;  // register cap: 3 x 256 threads resident per SM
constexpr int kMaxPagesPerCta = 64;
constexpr int64_t kSpanTargetBytes = 64 * 1024;  // bytes one CTA of the vectorised family moves
constexpr int kUnroll16 = 8;  // vectors in flight per thread, 16-byte vectors
constexpr int kUnroll32 = 4;  // and 32-byte vectors

// Sum of sl[0..n) over the CTA, result broadcast to all threads. n <= TOPKV_MAX_INLINE_R.
__device__ __forceinline__ int64_t block_prefix(const int32_t* __restrict__ sl, int n, int r_split,
                                                int window, int64_t* total_out) {
  // returns sum_{q < r_split} sl[q]; *total_out = sum_{q < n} sl[q]
  __shared__ int64_t s_part[2][kThreads / 32];
  int64_t below = 0, all = 0;
  for (int q = threadIdx.x; q < n; q += kThreads) {
    int64_t v = sl[q];
    if (window > 0 && v > window) v = window;  // a windowed layer keeps min(s, W) tokens
    all += v;
    if (q < r_split) below += v;
  }
  for (int o = 16; o > 0; o >>= 1) {
    below += __shfl_xor_sync(0xffffffffu, below, o);
    all += __shfl_xor_sync(0xffffffffu, all, o);
  }
  if ((threadIdx.x & 31) == 0) {
    s_part[0][threadIdx.x >> 5] = below;
    s_part[1][threadIdx.x >> 5] = all;
  }
  __syncthreads();
  below = 0;
  all = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) {
    below += s_part[0][w];
    all += s_part[1][w];
  }
  *total_out = all;
  return below;
}

// One CTA per (request, page column). F: planes per token; PACK: pool -> wire, else
// wire -> pool; MERGED: the valid tokens of a page form one contiguous run per plane on
// both sides (MLA rows, or PLANAR wire with a token-contiguous pool).
// Returns (uniformly over the CTA) -1 when the span holds no token this layer keeps, else the
// span's number r * spr + (span of request r), whichever CTA of whichever grid form took it:
// that number indexes the flags of a span link.
template <int F, bool PACK, bool MERGED, int VEC, bool MULTI>
__device__ __forceinline__ int copy_span_work(const KParams& p, const int slot) {
  // A span = `ppc` consecutive page columns of one request (one page when pages are large;
  // several small pages, so that every CTA moves a few tens of KiB).
  __shared__ int32_t s_pages[kMaxPagesPerCta];
  __shared__ int s_link_failed;
  // blockIdx.y = layer of a multi-layer launch (0 and zero strides for a single layer)
  uint8_t* const pool = p.pool + (int64_t)blockIdx.y * p.S_layer;
  uint8_t* const wire = p.wire + (int64_t)blockIdx.y * p.W_layer;
  const int gspr = p.wspr > 0 ? p.wspr : p.spr;  // spans per request that have a CTA
  int r = slot / gspr;
  int sidx = slot - r * gspr;  // span of request r
  if (p.compact && !find_span<kThreads>(p.sl, p.R, p.maxp * p.P, p.ppc * p.P, slot, &r, &sidx)) return -1;
  const int s_r = p.const_len > 0 ? p.const_len : p.sl[r];
  // first token this layer keeps: 0, or s_r - window for a windowed layer (§2.2)
  const int b_r = (p.window > 0 && s_r > p.window) ? s_r - p.window : 0;
  // a length longer than its block-table row: reported by every CTA of the request (a windowed
  // layer may run none for its first spans), and only what the row holds is copied
  const bool over_long = s_r > p.maxp * p.P;
  if (over_long && threadIdx.x == 0) raise_error(kErrTable);
  if (p.wspr > 0) {            // counted from the span that holds the first kept token
    sidx += b_r / (p.ppc * p.P);
    if (sidx >= p.spr) return -1;
  }
  // The span: `ppc` whole page columns from column j0 on, or, when pages are far larger than a
  // CTA's share, `tps` tokens of page column j0 (`cpp` CTAs per page).
  int j0, first, span_tokens;
  if (p.cpp > 1) {
    j0 = sidx / p.cpp;
    first = j0 * p.P + (sidx - j0 * p.cpp) * p.tps;
    span_tokens = min(p.tps, (j0 + 1) * p.P - first);
  } else {
    j0 = sidx * p.ppc;
    first = j0 * p.P;  // first token of the span's page columns
    span_tokens = p.ppc * p.P;
  }
  const int tid = threadIdx.x;
  int hi = min(first + span_tokens, s_r);
  if (over_long) hi = min(hi, p.maxp * p.P);
  const int lo = max(first, b_r);
  if (lo >= hi) return -1;
  const int span_id = r * p.spr + sidx;
  // linked launch: ask for this span's flag now, so that the answer travels while the rest of
  // the tables is read; it is looked at (and asked for again, if need be) just before data is
  // touched
  const int32_t* const link_flag =
      p.link_await != nullptr ? p.link_await + ((int64_t)blockIdx.y * p.R * p.spr + span_id) : nullptr;
  int link_seen = 0;
  if (link_flag != nullptr && tid == 0) link_seen = ld_acquire_gpu(link_flag);
  const int v = hi - lo;                // kept tokens in this span
  const int ts0 = lo - j0 * p.P;        // where they start, counted from the start of page column j0
  const int jlo = ts0 / p.P, jhi = (ts0 + v - 1) / p.P;  // page columns (relative to j0) they touch

  int64_t cu_r, T = p.T;
  if (p.const_len > 0) {
    cu_r = (int64_t)r * p.const_len;
    if (T < 0) T = (int64_t)p.R * p.const_len;
  } else if (p.cu != nullptr) {
    cu_r = p.cu[r];
    if (p.planar && p.plane_rows < 0 && T < 0) T = p.cu[p.R];
  } else {
    int64_t total;
    const bool need_T = p.planar && p.plane_rows < 0 && T < 0;
    cu_r = block_prefix(p.sl, need_T ? p.R : r, r, p.window, &total);
    if (need_T) T = total;
  }
  const int64_t PR = p.plane_rows >= 0 ? p.plane_rows : T;  // rows from the K to the V plane
  if (tid >= jlo && tid <= jhi) {
    int pg = p.bt[(int64_t)r * p.maxp + j0 + tid];
    if (pg < 0 || pg >= p.num_pages) {  // unusable entry: the page is skipped, nothing is touched
      pg = -1;
      raise_error(kErrTable);
    }
    s_pages[tid] = pg;
  }
  __syncthreads();
  const int64_t n0 = cu_r + (lo - b_r);  // wire index of the span's first kept token
  const int64_t unit_bytes = (int64_t)p.unit_chunks * VEC;
  {  // the span must lie inside the wire slab, whatever lengths the device tables hold
    const int64_t row = unit_bytes * p.U;
    const bool fits = p.planar ? (n0 >= 0 && ((F - 1) * PR + n0 + v) * row <= p.wire_limit)
                               : (n0 >= 0 && (n0 + v) * F * row <= p.wire_limit);
    if (!fits) {
      if (tid == 0) raise_error(kErrWire);
      return span_id;
    }
  }
  // tables read, addresses known: from here on the pool and the wire are touched
  if (p.late_wait) pdl_wait_prior_grid();
  if (p.link_await != nullptr) {  // wait for this span's flag, not for the whole kernel before
    if (tid == 0) {
      uint32_t polls = 0;
      int failed = 0;
      while (link_seen != p.await_epoch) {
        if (++polls > kLinkPollLimit) {
          failed = 1;
          break;
        }
        __nanosleep(100);
        link_seen = ld_acquire_gpu(link_flag);
      }
      s_link_failed = failed;
    }
    __syncthreads();
    if (s_link_failed) {  // the span is skipped and reported; nothing was touched
      if (tid == 0) raise_error(kErrWait);
      return span_id;
    }
  }
  constexpr int kUnroll = VEC == 32 ? kUnroll32 : kUnroll16;

  if (MERGED) {
    // per page, F runs of (valid tokens) * row bytes each (U == 1 here)
    for (int jj = jlo; jj <= jhi; ++jj) {
      if (s_pages[jj] < 0) continue;
      const int t_lo = max(0, ts0 - jj * p.P), t_hi = min(p.P, ts0 + v - jj * p.P);
      const int n = (t_hi - t_lo) * p.unit_chunks;
      uint8_t* pool_page = pool + (int64_t)s_pages[jj] * p.S_page + (int64_t)t_lo * p.S_tok;
#pragma unroll
      for (int c = 0; c < F; ++c) {
        uint8_t* a = pool_page + c * p.S_kv;
        // not planar => F == 1
        uint8_t* b = wire +
                     ((p.planar ? c * PR : 0) + n0 + (int64_t)(jj * p.P + t_lo - ts0)) * unit_bytes;
        const uint8_t* src = PACK ? a : b;
        uint8_t* dst = PACK ? b : a;
        for (int w0 = tid; w0 < n; w0 += kThreads * kUnroll) {
          Vec<VEC> buf[kUnroll];
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            const int w = w0 + u * kThreads;
            if (w < n) buf[u].load(src + (int64_t)w * VEC);
          }
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            const int w = w0 + u * kThreads;
            if (w < n) buf[u].store(dst + (int64_t)w * VEC);
          }
        }
      }
    }
    return span_id;
  }

  // Units of the span in wire order: q = (ts*F + c)*U + h (TOKEN_KV) or q = (c*v + ts)*U + h
  // (PLANAR), ts = token index inside the span. `tpu` threads cooperate on one unit.
  const int nunits = v * F * p.U;
  const int tpu = min(p.unit_chunks, kThreads);
  const int groups = kThreads / tpu;
  const int my_g = tid / tpu;
  const int my_w = tid - my_g * tpu;
  if (my_g >= groups) return span_id;
  uint8_t* wire_span = wire + n0 * F * p.U * unit_bytes;  // TOKEN_KV: the span is one run
  if (!MULTI && s_pages[0] < 0) return span_id;                // single page, unusable: skip it
  uint8_t* page0 = pool + (int64_t)s_pages[0] * p.S_page + (int64_t)ts0 * p.S_tok;

  for (int q0 = my_g; q0 < nunits; q0 += groups * kUnroll) {
    for (int w = my_w; w < p.unit_chunks; w += tpu) {
      Vec<VEC> buf[kUnroll];
      uint8_t* dstp[kUnroll];  // only the store side is kept across the batch of loads
      bool ok[kUnroll];
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const int q = min(q0 + u * groups, nunits - 1);  // clamped: addresses stay valid
        int h = 0, tc = q;
        if (p.U > 1) {
          tc = q / p.U;
          h = q - tc * p.U;
        }
        int c, ts;
        uint8_t *a, *b;
        if (p.planar) {
          c = (F > 1 && tc >= v) ? 1 : 0;
          ts = tc - c * v;
          b = wire + (((int64_t)c * PR + n0 + ts) * p.U + h) * unit_bytes + (int64_t)w * VEC;
        } else {
          ts = tc / F;
          c = tc - ts * F;
          b = wire_span + (int64_t)q * unit_bytes + (int64_t)w * VEC;
        }
        if (MULTI) {  // several pages per span: look the token's page up
          const int jj = (ts0 + ts) / p.P;
          const int t = ts0 + ts - jj * p.P;
          const int pg = s_pages[jj];
          a = pool + (int64_t)pg * p.S_page + c * p.S_kv + t * p.S_tok + h * p.S_unit +
              (int64_t)w * VEC;
          ok[u] = q0 + u * groups < nunits && pg >= 0;
        } else {
          a = page0 + c * p.S_kv + ts * p.S_tok + h * p.S_unit + (int64_t)w * VEC;
          ok[u] = q0 + u * groups < nunits;
        }
        dstp[u] = PACK ? b : a;
        if (ok[u]) buf[u].load(PACK ? a : b);
      }
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        if (ok[u]) buf[u].store(dstp[u]);
      }
    }
  }
  return span_id;
}

// One span, and, for a linked launch, the publication of its flag once every thread of the CTA
// has issued its stores (spans without kept tokens publish nothing: their consumers, which see
// the same lengths, do not wait for them either).
template <int F, bool PACK, bool MERGED, int VEC, bool MULTI>
__device__ __forceinline__ void copy_span(const KParams& p, const int slot) {
  const int span_id = copy_span_work<F, PACK, MERGED, VEC, MULTI>(p, slot);
  if (p.link_signal != nullptr && span_id >= 0) {
    __syncthreads();  // every thread's stores are ordered before thread 0's release below
    if (threadIdx.x == 0)
      st_release_gpu(p.link_signal + ((int64_t)blockIdx.y * p.R * p.spr + span_id), p.signal_epoch);
  }
}

template <int F, bool PACK, bool MERGED, int VEC, bool MULTI>
__global__ void __launch_bounds__(kThreads, kMinCtasPerSm)
topkv_page_copy_kernel(const KParams p) {
  pdl_prologue(p.overlap | p.late_wait);  // late_wait: copy_span waits once the tables are read
  copy_span<F, PACK, MERGED, VEC, MULTI>(p, blockIdx.x);
  pdl_epilogue(p.overlap | p.late_wait);  // CTAs without work never reached the wait
}

// The same copy with a bounded grid: gridDim.x CTAs walk all R * spr spans, CTA b taking spans
// b, b + gridDim.x, ... Used when the wire is pinned host memory reached over PCIe (the direct
// host leg): the link, not the SMs, sets the pace there, a few CTAs keep it full, and the rest
// of the GPU stays with whatever else is running (the prefill). Neighbouring CTAs work on
// neighbouring spans, so the host side is written (read) in roughly ascending order.
template <int F, bool PACK, bool MERGED, int VEC, bool MULTI>
__global__ void __launch_bounds__(kThreads, kMinCtasPerSm)
topkv_page_copy_walk_kernel(const KParams p) {
  pdl_prologue(p.overlap | p.late_wait);
  const int nslots = p.R * (p.wspr > 0 ? p.wspr : p.spr);
  for (int slot = blockIdx.x; slot < nslots; slot += gridDim.x) {
    copy_span<F, PACK, MERGED, VEC, MULTI>(p, slot);
    __syncthreads();  // the span's page ids in shared memory are re-used by the next span
  }
  pdl_epilogue(p.overlap | p.late_wait);
}

// Exclusive prefix sum of seq_lens into int64 [R+1]; one CTA, any R.
__global__ void __launch_bounds__(kThreads)
topkv_plan_kernel(const int32_t* __restrict__ sl, int R, int window, int64_t* __restrict__ cu) {
  __shared__ int64_t s_warp[kThreads / 32];
  __shared__ int64_t s_carry;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (tid == 0) s_carry = 0;
  __syncthreads();
  for (int base = 0; base < R; base += kThreads) {
    const int q = base + tid;
    int64_t x = q < R ? (int64_t)sl[q] : 0;
    if (window > 0 && x > window) x = window;
    int64_t inc = x;  // inclusive scan inside the warp
    for (int o = 1; o < 32; o <<= 1) {
      const int64_t y = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += y;
    }
    if (lane == 31) s_warp[wid] = inc;
    __syncthreads();
    int64_t before = s_carry;
    for (int w = 0; w < wid; ++w) before += s_warp[w];
    if (q < R) cu[q] = before + inc - x;
    __syncthreads();
    if (tid == kThreads - 1) s_carry = before + inc;
    __syncthreads();
  }
  if (tid == 0) cu[R] = s_carry;
}

}  // namespace topkv
