// Types shared by the TopKV kernels (device side) and their host launchers.
#pragma once
#include <cstdint>

#include <cuda_runtime.h>

#include "topkv.h"

namespace topkv {

// ------------------------------------------------------------------------------------------
// Kernel parameters (plain data, passed by value).
// A "unit" is the largest run of bytes that is contiguous on both sides for one
// (token, plane): the whole [head][dim] row when heads are contiguous in the pool,
// otherwise one head (U = H units per row).
// ------------------------------------------------------------------------------------------
struct KParams {
  uint8_t* pool;          // base of this layer's pool slab
  uint8_t* wire;          // base of this layer's wire slab (device, or mapped pinned host)
  const int32_t* bt;      // [R][maxp]
  const int32_t* sl;      // [R]
  const int64_t* cu;      // [R+1] or nullptr
  int64_t T;              // total tokens or -1
  int64_t S_page, S_kv, S_tok, S_unit;  // pool strides, bytes
  int R, maxp, P;
  int U;                  // units per (token, plane)
  int unit_chunks;        // VEC-byte chunks per unit
  int planar;             // wire order
  int64_t plane_rows;     // PLANAR: rows between the planes of a slab, or -1 = total tokens T
  int window;             // 0, or the layer keeps only the last min(s, window) tokens
  int ppc, spr;           // vectorised family: page columns per CTA, CTAs per request
  int wspr;               // windowed layer: only the `wspr` spans per request that the window can touch get
                          // a CTA, counted from the span of the first kept token (0 = all `spr` spans)
  int compact;            // 1: the grid holds one CTA per span that CAN hold tokens (total_tokens / span + R of
                          // them) instead of one per block-table column; each CTA finds its request and
                          // span from the lengths (ragged batches: nearly half the columns are empty)
  int cpp, tps;           // pages far larger than a CTA's span are split: CTAs per page (1 = whole
                          // pages), tokens per CTA of a split page
  int const_len;          // > 0: every request has exactly this many tokens; sl and cu are not read
                          // (the fixed-size state of a linear-attention layer, cut into rows)
  int64_t num_pages;      // pages per pool slab: every page id is checked against it
  int64_t wire_limit;     // bytes that may be touched behind `wire` (this layer's slab)
  int overlap;            // 1: caller declared this launch independent of the kernels before it
  int late_wait;          // 1: tables are settled, wait for the previous kernel only before touching data
  int64_t S_layer, W_layer;  // multi-layer launch: bytes from one layer's slab to the next (pool, wire)
  // span links: ordering against an earlier kernel span by span instead of grid by grid
  const int32_t* link_await;  // flags this launch waits for, one per span, or nullptr
  int32_t* link_signal;       // flags this launch publishes, one per span, or nullptr
  int await_epoch, signal_epoch;
};

// Error bits raised by kernels (never a trap): read back with topkv_device_error_flags().
//   1  a bounded wait inside a kernel ran out
//   2  a table entry was unusable (page id outside the pool, or a length longer than its
//      block-table row): the affected pages were skipped
//   4  the lengths found on the device do not fit the wire slab: the affected work was skipped
__device__ int g_device_error_flags = 0;
constexpr int kErrWait = 1, kErrTable = 2, kErrWire = 4;
__device__ __forceinline__ void raise_error(int bit) {
  if ((*(volatile int*)&g_device_error_flags & bit) == 0) atomicOr(&g_device_error_flags, bit);
}

// Programmatic dependent launch. Every copy kernel is launched with programmatic stream
// serialisation, so its CTAs may become resident while the previous kernel of the stream
// drains. By default a kernel waits for that previous kernel to finish (and its writes to be
// visible) before it reads anything; a launch the caller declared independent skips the wait
// and only holds one thread back at its end, so that kernels still COMPLETE in stream order.
__device__ __forceinline__ void pdl_wait_prior_grid() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void pdl_release_next_grid() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_prologue(int overlap) {
  if (!overlap) pdl_wait_prior_grid();
  pdl_release_next_grid();
}
__device__ __forceinline__ void pdl_epilogue(int overlap) {
  if (overlap && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) pdl_wait_prior_grid();
}

// Span links. A linked launch does not wait for the kernel before it as a whole: every CTA waits
// (bounded) until the flag of ITS span holds the epoch it expects, and publishes its own span's
// flag once its stores are issued. Programmatic dependent launch makes this safe: a kernel's
// CTAs are only scheduled once every CTA of all earlier kernels of the stream has started, so
// the CTA that a waiter depends on is resident or finished and never waits for the waiter.
constexpr uint32_t kLinkPollLimit = 1u << 19;  // a poll is a 100 ns pause and one load: gives up after about half a second
__device__ __forceinline__ int ld_acquire_gpu(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_gpu(int32_t* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// The compact grid of a ragged batch: CTA `slot` takes the slot-th span that holds tokens,
// counted request by request (request q has ceil(min(s_q, row_tokens) / span_tokens) of them).
// An inclusive scan of those counts over the CTA (R <= THREADS), then the one thread whose
// request contains that span says so. Returns false (uniformly) when `slot` lies past the last
// span. If there are more spans than CTAs, the lengths on the device exceed the total the grid
// was sized from: CTA 0 raises the wire bit.
template <int THREADS>
__device__ __forceinline__ bool find_span(const int32_t* __restrict__ sl, int R, int row_tokens,
                                          int span_tokens, int slot, int* r_out, int* sidx_out) {
  __shared__ int s_scan[THREADS / 32];
  __shared__ int s_hit[2];
  const int t = threadIdx.x, lane = t & 31, wid = t >> 5;
  int n_q = 0;
  if (t < R) n_q = (min(max(sl[t], 0), row_tokens) + span_tokens - 1) / span_tokens;
  int incl = n_q;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += up;
  }
  if (lane == 31) s_scan[wid] = incl;
  if (t == 0) s_hit[0] = -1;
  __syncthreads();
  int total = 0;
#pragma unroll
  for (int w = 0; w < THREADS / 32; ++w) {
    if (w < wid) incl += s_scan[w];
    total += s_scan[w];
  }
  if (n_q > 0 && slot >= incl - n_q && slot < incl) {
    s_hit[0] = t;
    s_hit[1] = slot - (incl - n_q);
  }
  if (t == 0 && slot == 0 && total > (int)gridDim.x) raise_error(kErrWire);
  __syncthreads();
  *r_out = s_hit[0];
  *sidx_out = s_hit[1];
  return s_hit[0] >= 0;
}

// Streaming vector accesses: every byte is touched exactly once, so neither side should
// displace anything useful from L1 / L2. Vec<32> uses the 256-bit global accesses of sm_100.
template <int VEC>
struct Vec;
template <>
struct Vec<16> {
  uint32_t v[4];
  __device__ __forceinline__ void load(const uint8_t* p) {
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3])
                 : "l"(p));
  }
  __device__ __forceinline__ void store(uint8_t* p) const {
    asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v[0]),
                 "r"(v[1]), "r"(v[2]), "r"(v[3])
                 : "memory");
  }
};
template <>
struct Vec<32> {
  uint32_t v[8];
  __device__ __forceinline__ void load(const uint8_t* p) {
    asm volatile(
        "ld.global.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7])
        : "l"(p));
  }
  __device__ __forceinline__ void store(uint8_t* p) const {
    asm volatile(
        "st.global.L1::no_allocate.L2::evict_first.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p),
        "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
        : "memory");
  }
};

// Launch with programmatic stream serialisation allowed (see pdl_prologue above).
template <typename P>
cudaError_t launch_pdl(void (*kernel)(const P), dim3 grid, dim3 block, size_t smem,
                       cudaStream_t stream, const P& params) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, params);
}

}  // namespace topkv
