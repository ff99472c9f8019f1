// TopKV data plane for B200 (sm_100a): per-layer pack / unpack of a paged KV cache to and
// from a contiguous wire slab (§3.4 layout, sent layer by layer as in §5.2), and the
// pinned-host PCIe leg (§3.3). Pure byte movement: no arithmetic on the elements.
//
// This file holds the host side: argument checks, launch geometry and the extern "C" entry
// points declared and documented in include/topkv.h. The kernels live in the .cuh files next
// to it (topkv_vec: vectorised page copy and plan; topkv_bulk: bulk-async ring; topkv_repage:
// pool to pool; topkv_crc: checksummed copy); topkv_host.cpp holds the CUDA-free helpers.
// Nothing here ever calls the CPU oracle.
#include "topkv.h"

#include <cuda_runtime.h>

#include "topkv_bulk.cuh"
#include "topkv_common.cuh"
#include "topkv_crc.cuh"
#include "topkv_repage.cuh"
#include "topkv_vec.cuh"

#include <algorithm>
#include <atomic>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <utility>
#include <vector>

namespace {

using namespace topkv;

// ------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------
thread_local int g_last_cuda_error = 0;
std::atomic<int64_t> g_launches{0};
std::atomic<int> g_variant{0};
// Direct host leg: 0 = one CTA per span, n = at most n CTAs walk the spans. 6 CTAs already keep
// the link full in both directions; 16 leaves slack and still costs a concurrent GEMM nothing
// measurable, where one CTA per span slowed it by 30 %.
std::atomic<int> g_host_leg_ctas{TOPKV_DEFAULT_HOST_LEG_CTAS};

inline bool mult16(int64_t x) { return (x & 15) == 0; }
inline bool mult16p(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int cuda_fail(cudaError_t e) {
  g_last_cuda_error = static_cast<int>(e);
  return TOPKV_ERR_CUDA;
}

struct Resolved {
  int64_t row_bytes;   // H*D*E
  int64_t unit_bytes;  // contiguous unit
  int U;
  bool merged;
};

int check_layout(const topkv_layout* lo, Resolved* out) {
  if (lo == nullptr || lo->struct_size != sizeof(topkv_layout)) return TOPKV_ERR_INVALID_ARG;
  if (lo->reserved != 0) return TOPKV_ERR_INVALID_ARG;
  if (lo->num_layers == 0 || lo->num_kv_heads == 0 || lo->head_dim == 0 || lo->elem_bytes == 0 ||
      lo->page_tokens == 0 || lo->num_pool_pages <= 0)
    return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  if (lo->kv_factor != 1 && lo->kv_factor != 2) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  if (lo->wire_order != TOPKV_WIRE_TOKEN_KV && lo->wire_order != TOPKV_WIRE_PLANAR)
    return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  if (lo->kind != TOPKV_KIND_GQA && lo->kind != TOPKV_KIND_MLA) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  if (lo->kind == TOPKV_KIND_MLA && lo->kv_factor != 1) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  const int64_t head_bytes = (int64_t)lo->head_dim * lo->elem_bytes;
  const int64_t row_bytes = head_bytes * lo->num_kv_heads;
  if (row_bytes > (1ll << 30)) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  const bool heads_contig = lo->num_kv_heads == 1 || lo->pool_head_stride == head_bytes;
  const int64_t unit = heads_contig ? row_bytes : head_bytes;
  if (lo->pool_page_stride <= 0 || lo->pool_layer_stride <= 0 ||
      (lo->page_tokens > 1 && lo->pool_token_stride < unit) ||
      (lo->kv_factor > 1 && lo->pool_kv_stride <= 0) ||
      (!heads_contig && lo->pool_head_stride < head_bytes) || lo->wire_layer_stride < 0 ||
      lo->wire_plane_stride < 0 || lo->wire_plane_stride % row_bytes != 0 ||
      (lo->wire_plane_stride != 0 && lo->wire_order != TOPKV_WIRE_PLANAR))
    return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  if (!mult16(unit) || !mult16(lo->pool_page_stride) || !mult16(lo->pool_token_stride) ||
      !mult16(lo->pool_layer_stride) || (lo->kv_factor > 1 && !mult16(lo->pool_kv_stride)) ||
      (!heads_contig && !mult16(lo->pool_head_stride)) || !mult16(lo->wire_layer_stride))
    return TOPKV_ERR_ALIGNMENT;
  out->row_bytes = row_bytes;
  out->unit_bytes = unit;
  out->U = heads_contig ? 1 : (int)lo->num_kv_heads;
  out->merged = heads_contig && (lo->page_tokens == 1 || lo->pool_token_stride == row_bytes) &&
                (lo->kv_factor == 1 || lo->wire_order == TOPKV_WIRE_PLANAR);
  return TOPKV_OK;
}

int check_batch(const topkv_layout* lo, const topkv_batch* b) {
  if (b == nullptr || b->struct_size != sizeof(topkv_batch) ||
      (b->flags & ~(uint32_t)(TOPKV_FLAG_OVERLAP_PREVIOUS | TOPKV_FLAG_TABLES_SETTLED)) != 0)
    return TOPKV_ERR_INVALID_ARG;
  if (b->num_requests < 0 || b->max_pages_per_req < 0 || b->total_tokens < -1 ||
      b->window_tokens < 0 || b->reserved != 0)
    return TOPKV_ERR_INVALID_ARG;
  if (b->num_requests > 0 && b->max_pages_per_req > 0) {
    if (b->block_table == nullptr || b->seq_lens == nullptr) return TOPKV_ERR_INVALID_ARG;
    if (b->cu_seq_lens == nullptr && b->num_requests > TOPKV_MAX_INLINE_R)
      return TOPKV_ERR_INVALID_ARG;
    if ((int64_t)b->num_requests * b->max_pages_per_req > 0x7fffffffll) return TOPKV_ERR_INVALID_ARG;
    // a block-table row must not describe more tokens than an int32 length can hold
    if ((int64_t)b->max_pages_per_req * lo->page_tokens > 0x7fffffffll) return TOPKV_ERR_INVALID_ARG;
    if (b->total_tokens > (int64_t)b->num_requests * b->max_pages_per_req * lo->page_tokens)
      return TOPKV_ERR_INVALID_ARG;
  }
  return TOPKV_OK;
}

// Validates everything and fills the kernel parameters for one layer. `wire_base` is the base
// of the whole wire buffer (layer 0's slab) of `capacity` bytes.
int prepare(int layer, const void* pool, const topkv_layout* lo, const topkv_batch* b,
            const void* wire_base, int64_t capacity, int64_t wire_layer_stride, KParams* kp,
            Resolved* rs, int64_t* n_layer_out) {
  int st = check_layout(lo, rs);
  if (st != TOPKV_OK) return st;
  st = check_batch(lo, b);
  if (st != TOPKV_OK) return st;
  if (layer < 0 || (uint32_t)layer >= lo->num_layers) return TOPKV_ERR_LAYER_RANGE;
  if (pool == nullptr || wire_base == nullptr || capacity < 0) return TOPKV_ERR_INVALID_ARG;
  if (!mult16p(pool) || !mult16p(wire_base)) return TOPKV_ERR_ALIGNMENT;
  int64_t n_layer = -1;
  const bool spread = lo->wire_plane_stride > 0;  // planes of a slab are not adjacent
  if (b->total_tokens >= 0) {
    n_layer = b->total_tokens * lo->kv_factor * rs->row_bytes;
    const int64_t extent = spread ? (lo->kv_factor - 1) * lo->wire_plane_stride + b->total_tokens * rs->row_bytes
                                  : n_layer;  // bytes from the slab's base to its last byte
    if ((int64_t)layer * wire_layer_stride + extent > capacity) return TOPKV_ERR_CAPACITY;
  }
  *n_layer_out = n_layer;
  kp->pool = const_cast<uint8_t*>(static_cast<const uint8_t*>(pool)) + (int64_t)layer * lo->pool_layer_stride;
  kp->wire = const_cast<uint8_t*>(static_cast<const uint8_t*>(wire_base)) + (int64_t)layer * wire_layer_stride;
  kp->bt = b->block_table;
  kp->sl = b->seq_lens;
  kp->cu = b->cu_seq_lens;
  kp->T = b->total_tokens;
  kp->S_page = lo->pool_page_stride;
  kp->S_kv = lo->kv_factor > 1 ? lo->pool_kv_stride : 0;
  kp->S_tok = lo->pool_token_stride;
  kp->S_unit = rs->U > 1 ? lo->pool_head_stride : 0;
  kp->R = b->num_requests;
  kp->maxp = b->max_pages_per_req;
  kp->P = (int)lo->page_tokens;
  kp->U = rs->U;
  kp->unit_chunks = (int)(rs->unit_bytes / 16);
  kp->planar = lo->wire_order == TOPKV_WIRE_PLANAR;
  kp->overlap = (b->flags & TOPKV_FLAG_OVERLAP_PREVIOUS) ? 1 : 0;
  kp->late_wait = (!kp->overlap && (b->flags & TOPKV_FLAG_TABLES_SETTLED)) ? 1 : 0;
  kp->ppc = 1;
  kp->spr = kp->maxp;
  kp->cpp = 1;
  kp->tps = 0;
  kp->const_len = 0;
  kp->window = b->window_tokens;
  kp->num_pages = lo->num_pool_pages;
  kp->wire_limit = (n_layer >= 0 && !spread) ? n_layer : capacity - (int64_t)layer * wire_layer_stride;
  kp->plane_rows = spread ? lo->wire_plane_stride / rs->row_bytes : -1;
  kp->S_layer = 0;
  kp->W_layer = 0;
  kp->link_await = nullptr;
  kp->link_signal = nullptr;
  kp->await_epoch = 0;
  kp->signal_epoch = 0;
  return TOPKV_OK;
}

template <bool PACK, int VEC, bool MULTI>
cudaError_t launch_vec2(const KParams& kp, bool merged, int F, dim3 grid, cudaStream_t stream, bool walk) {
  const dim3 block(kThreads);
  if (walk) {  // bounded grid, every CTA walks several spans
    if (merged) {
      if (F == 1) return launch_pdl(topkv_page_copy_walk_kernel<1, PACK, true, VEC, MULTI>, grid, block, 0, stream, kp);
      return launch_pdl(topkv_page_copy_walk_kernel<2, PACK, true, VEC, MULTI>, grid, block, 0, stream, kp);
    }
    if (F == 1) return launch_pdl(topkv_page_copy_walk_kernel<1, PACK, false, VEC, MULTI>, grid, block, 0, stream, kp);
    return launch_pdl(topkv_page_copy_walk_kernel<2, PACK, false, VEC, MULTI>, grid, block, 0, stream, kp);
  }
  if (merged) {
    if (F == 1) return launch_pdl(topkv_page_copy_kernel<1, PACK, true, VEC, MULTI>, grid, block, 0, stream, kp);
    return launch_pdl(topkv_page_copy_kernel<2, PACK, true, VEC, MULTI>, grid, block, 0, stream, kp);
  }
  if (F == 1) return launch_pdl(topkv_page_copy_kernel<1, PACK, false, VEC, MULTI>, grid, block, 0, stream, kp);
  return launch_pdl(topkv_page_copy_kernel<2, PACK, false, VEC, MULTI>, grid, block, 0, stream, kp);
}

template <bool PACK, int VEC>
cudaError_t launch_vec(const KParams& kp, bool merged, int F, dim3 grid, cudaStream_t stream, bool walk) {
  if (kp.ppc > 1) return launch_vec2<PACK, VEC, true>(kp, merged, F, grid, stream, walk);
  return launch_vec2<PACK, VEC, false>(kp, merged, F, grid, stream, walk);
}

// ---- bulk-async family -------------------------------------------------------------------
constexpr int kSmemBudget = 227 * 1024;   // opt-in dynamic shared memory per CTA on sm_100
constexpr int kStageTarget = 36 * 1024;   // bytes of payload per ring stage

struct DeviceInfo {
  int sms = 0;
  bool attr_set[4] = {false, false, false, false};
};
std::mutex g_devinfo_mutex;
DeviceInfo g_devinfo[64];

template <int F, bool PACK>
int bulk_prepare_device(int* sms_out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return TOPKV_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_devinfo_mutex);
  DeviceInfo& di = g_devinfo[dev];
  if (di.sms == 0) {
    e = cudaDeviceGetAttribute(&di.sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  const int idx = (F - 1) * 2 + (PACK ? 1 : 0);
  if (!di.attr_set[idx]) {
    e = cudaFuncSetAttribute(topkv_bulk_kernel<F, PACK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kSmemBudget);
    if (e != cudaSuccess) return cuda_fail(e);
    di.attr_set[idx] = true;
  }
  *sms_out = di.sms;
  return TOPKV_OK;
}

// Launches the bulk-async kernel when the shape fits its shared-memory ring; *handled tells
// the caller whether it did (otherwise the vectorised family takes over).
template <bool PACK>
int launch_bulk(const KParams& kp0, const Resolved& rs, int F, cudaStream_t stream, bool* handled) {
  *handled = false;
  if (kp0.R > kBulkMaxR || kp0.window > 0 || kp0.const_len > 0) return TOPKV_OK;
  if ((int64_t)kp0.R * kp0.maxp * kp0.P > 0x7fffffffll) return TOPKV_OK;  // its prefix sums are int32
  const int64_t tok_bytes = (int64_t)F * rs.row_bytes;
  if (tok_bytes > kStageTarget || rs.unit_bytes > 0x7fffffff) return TOPKV_OK;
  if (!rs.merged && rs.unit_bytes < 1024) return TOPKV_OK;  // per-copy cost dominates small units
  BulkParams bp;
  bp.k = kp0;
  bp.k.unit_chunks = (int)(rs.unit_bytes / 16);
  bp.tpc = (int)std::min<int64_t>(kp0.P, kStageTarget / tok_bytes);
  bp.cpp = (kp0.P + bp.tpc - 1) / bp.tpc;
  bp.tpc = (kp0.P + bp.cpp - 1) / bp.cpp;  // even split of the page
  bp.stage_bytes = (int)((bp.tpc * tok_bytes + 127) / 128 * 128);
  bp.merged = rs.merged ? 1 : 0;
  const int fixed = kBulkWarps * kBulkMaxStages * (int)(sizeof(uint64_t) + sizeof(ItemDesc)) +
                    2 * (kp0.R + 1) * (int)sizeof(int32_t);
  bp.nstages = std::min(kBulkMaxStages, (kSmemBudget - fixed) / (kBulkWarps * bp.stage_bytes));
  if (bp.nstages < 2) return TOPKV_OK;
  const size_t smem = (size_t)kBulkWarps * bp.nstages * bp.stage_bytes + fixed;
  int sms = 0;
  int st = (F == 1) ? bulk_prepare_device<1, PACK>(&sms) : bulk_prepare_device<2, PACK>(&sms);
  if (st != TOPKV_OK) return st;
  const dim3 grid((unsigned)sms), block(kBulkThreads);
  const cudaError_t e = (F == 1) ? launch_pdl(topkv_bulk_kernel<1, PACK>, grid, block, smem, stream, bp)
                                 : launch_pdl(topkv_bulk_kernel<2, PACK>, grid, block, smem, stream, bp);
  if (e != cudaSuccess) return cuda_fail(e);
  *handled = true;
  return TOPKV_OK;
}

// Bytes per access of the vectorised family: 32 only when every address the kernel can form
// is 32-byte aligned. A launch over several layers also adds multiples of the two layer
// strides inside the kernel (blockIdx.y), which the ABI only requires to be multiples of 16.
int copy_vector_bytes(const KParams& kp, int64_t unit_bytes, int layers) {
  uintptr_t m = reinterpret_cast<uintptr_t>(kp.pool) | reinterpret_cast<uintptr_t>(kp.wire) |
                (uintptr_t)kp.S_page | (uintptr_t)kp.S_kv | (uintptr_t)kp.S_tok | (uintptr_t)kp.S_unit |
                (uintptr_t)unit_bytes;
  if (layers > 1) m |= (uintptr_t)kp.S_layer | (uintptr_t)kp.W_layer;
  return (m & 31) == 0 ? 32 : 16;
}

// How the vectorised family cuts a block-table row into spans (one CTA each): `ppc` whole page
// columns per span when pages are small, `cpp` CTAs per page when pages are far larger than a
// CTA's share, one page otherwise. Fills ppc, spr, cpp, tps.
void span_geometry(KParams* kp, int F, int64_t row_bytes) {
  const int64_t page_bytes = (int64_t)kp->P * F * row_bytes;
  kp->ppc = (int)std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(kMaxPagesPerCta, kp->maxp),
                                                       kSpanTargetBytes / page_bytes));
  kp->spr = (kp->maxp + kp->ppc - 1) / kp->ppc;
  kp->cpp = 1;
  kp->tps = 0;
  if (page_bytes >= 2 * kSpanTargetBytes && kp->P > 1) {  // huge pages: several CTAs per page
    const int64_t tok_bytes = (int64_t)F * row_bytes;
    kp->tps = (int)std::max<int64_t>(1, std::min<int64_t>(kp->P, kSpanTargetBytes / tok_bytes));
    kp->cpp = (kp->P + kp->tps - 1) / kp->tps;
    if ((int64_t)kp->maxp * kp->cpp > 0x7fffffffll / std::max(1, kp->R)) {  // keep R * spr an int
      kp->cpp = 1;
      kp->tps = 0;
    } else if (kp->cpp > 1) {
      kp->spr = kp->maxp * kp->cpp;
    }
  }
}

// A windowed layer keeps at most `window` tokens per request, wherever they lie in its row: the
// window touches at most ceil(window / span) + 1 spans, so only that many CTAs per request are
// launched and each finds its span from the request's length (a 128-token window of a
// 4,096-token row: 5 CTAs instead of 128, of which 123 would find nothing to do).
void window_spans(KParams* kp) {
  kp->wspr = 0;
  if (kp->window <= 0 || kp->cpp != 1 || kp->const_len > 0) return;
  const int64_t span_tokens = (int64_t)kp->ppc * kp->P;
  const int64_t need = (kp->window + span_tokens - 1) / span_tokens + 1;
  if (need < kp->spr) kp->wspr = (int)need;
}

// Cuts the batch into spans and decides how many CTAs per layer the vectorised family launches
// (fills ppc, spr, cpp, tps, wspr, compact). *walk: the grid is bounded by max_ctas and every CTA
// walks several spans.
int64_t grid_spans(KParams* kp, int F, int64_t row_bytes, int max_ctas, bool* walk) {
  span_geometry(kp, F, row_bytes);
  window_spans(kp);
  int64_t spans = (int64_t)kp->R * (kp->wspr > 0 ? kp->wspr : kp->spr);
  *walk = max_ctas > 0 && spans > max_ctas;
  // A ragged batch fills far fewer block-table columns than R * max_pages_per_req: when the
  // caller has stated the total, total / span + R CTAs are enough for every span that can hold
  // tokens (request q has ceil(s_q / span) <= s_q / span + 1 of them), and each finds its place
  // from the lengths (worth it from 10 % fewer CTAs on). The search runs before the kernel's
  // wait for its predecessor where the flags allow that; a launch that must wait first would
  // only lengthen its start by it, and keeps the plain grid.
  kp->compact = 0;
  if (!*walk && (kp->overlap || kp->late_wait) && kp->T >= 0 && kp->window == 0 && kp->cpp == 1 &&
      kp->const_len == 0 && kp->R <= kThreads) {
    const int64_t bound = kp->T / ((int64_t)kp->ppc * kp->P) + kp->R;
    if (bound * 10 < spans * 9) {
      kp->compact = 1;
      spans = bound;
    }
  }
  return spans;
}

// max_ctas > 0: the wire is host memory behind PCIe; at most that many CTAs walk the spans.
// layers > 1: one launch covers that many consecutive layers (kp describes the first one and
// carries the layer strides); the vectorised family only.
template <bool PACK>
int launch_copy(KParams kp, const Resolved& rs, int F, cudaStream_t stream, int max_ctas = 0,
                int layers = 1) {
  const int64_t slots = (int64_t)kp.R * kp.maxp;
  if (slots == 0 || layers == 0) return TOPKV_OK;
  bool handled = false;
  const bool linked = kp.link_await != nullptr || kp.link_signal != nullptr;
  if (max_ctas <= 0 && layers == 1 && !linked && g_variant.load(std::memory_order_relaxed) == 1) {
    const int st = launch_bulk<PACK>(kp, rs, F, stream, &handled);
    if (st != TOPKV_OK) return st;
  }
  if (!handled) {
    bool walk = false;
    const int64_t spans = grid_spans(&kp, F, rs.row_bytes, max_ctas, &walk);
    const dim3 grid((unsigned)(walk ? max_ctas : spans), (unsigned)layers);
    cudaError_t le;
    if (copy_vector_bytes(kp, rs.unit_bytes, layers) == 32) {
      kp.unit_chunks = (int)(rs.unit_bytes / 32);
      le = launch_vec<PACK, 32>(kp, rs.merged, F, grid, stream, walk);
    } else {
      kp.unit_chunks = (int)(rs.unit_bytes / 16);
      le = launch_vec<PACK, 16>(kp, rs.merged, F, grid, stream, walk);
    }
    if (le != cudaSuccess) {
      cudaGetLastError();
      return cuda_fail(le);
    }
  }
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return TOPKV_OK;
}

// Device-visible address of a pinned host buffer (identity under unified addressing, but
// asked for explicitly so that pageable memory is refused instead of faulting).
int mapped_device_pointer(const void* h, void** d) {
  cudaPointerAttributes attr;
  cudaError_t e = cudaPointerGetAttributes(&attr, h);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return cuda_fail(e);
  }
  if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) return TOPKV_ERR_INVALID_ARG;
  *d = attr.devicePointer;
  return TOPKV_OK;
}

// ---- built-in staging slab of topkv_pack_layer_to_host_noalloc ---------------------------
// Lives in the library's device image: present on every GPU that loads the library, shared by
// all calls. In host code the name below is only a handle; the device address comes from
// cudaGetSymbolAddress, looked up once per device.
static __device__ __align__(256) unsigned char g_noalloc_staging[TOPKV_NOALLOC_STAGING_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void* g_noalloc_addr[kMaxDevices] = {};

int noalloc_staging_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= kMaxDevices) return TOPKV_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  if (g_noalloc_addr[dev] == nullptr) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_staging);  // address on the CURRENT device
    if (e != cudaSuccess) {
      cudaGetLastError();
      return cuda_fail(e);
    }
    if (ptr == nullptr) return TOPKV_ERR_CUDA;
    g_noalloc_addr[dev] = ptr;
  }
  *out = g_noalloc_addr[dev];
  return TOPKV_OK;
}

// ---- CRC-64 fused into pack / unpack ------------------------------------------------------------
// Cuts the contiguous unit (a token row, or one head of a head-split pool) into runs of at most
// kCrcRunMax bytes, one per lane; fails when no such cut exists or the tables would not fit.
int crc_geometry(const topkv_layout* lo, const Resolved& rs, int maxp, CrcGeom* g) {
  int rpu = 0;
  for (int k = 1; k <= 65536; ++k) {
    if (rs.unit_bytes % k) continue;
    const int64_t run = rs.unit_bytes / k;
    if (run % 16) continue;
    if (run <= kCrcRunMax) {
      rpu = k;
      break;
    }
  }
  if (rpu == 0) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  g->rpu = rpu;
  g->run_bytes = (int)(rs.unit_bytes / rpu);
  g->rpr = rs.U * rpu;
  const int run16 = g->run_bytes / 16;
  g->pitch = (run16 | 1) * 16;  // odd number of 16-byte slots: lanes' rows start in distinct banks
  const int64_t runs = (int64_t)maxp * lo->page_tokens * g->rpr;  // of one block-table row
  if (runs > 0x7fffff00ll) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  g->kmax = (int)std::max<int64_t>(1, (runs + kCrcRunsPerItem - 1) / kCrcRunsPerItem);
  return TOPKV_OK;
}

constexpr int kCrcMaxR = 8192;  // the per-CTA plan (12 bytes per request) lives in shared memory

// Warps per CTA and dynamic shared memory of the checksummed copy for this shape.
// Two CTAs share an SM (half of its shared memory each), so that a CTA of the next launch can
// move in as soon as one of this launch's two has finished (measured: 47.2 -> 45.4 us per layer).
constexpr int kCrcCtasPerSm = 2;
int crc_launch_shape(const CrcGeom& g, int R, int stages, int* warps, size_t* smem) {
  const size_t fixed = kCrcMaxWarps * kCrcMaxStages * sizeof(uint64_t) + (size_t)(R + 1) * 12 + 16;
  const size_t per_warp = (size_t)stages * ((size_t)kCrcRunsPerItem * g.pitch + 32 * 8 + 8);
  if (fixed + per_warp > (size_t)kSmemBudget) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  // shared memory one CTA may take when several share an SM (1 KiB per CTA is the system's)
  size_t budget = (size_t)(233472 / kCrcCtasPerSm) - 1024;
  if (budget > (size_t)kSmemBudget) budget = kSmemBudget;
  if (fixed + per_warp > budget) budget = kSmemBudget;
  *warps = (int)std::min<size_t>(kCrcMaxWarps, (budget - fixed) / per_warp);
  *smem = (size_t)*warps * per_warp + fixed;
  return TOPKV_OK;
}

std::mutex g_crc_mutex;
bool g_crc_attr_set[64][4] = {};

template <int F, bool PACK>
int crc_prepare_device(int* sms_out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= 64) return TOPKV_ERR_INVALID_ARG;
  {
    std::lock_guard<std::mutex> lock(g_devinfo_mutex);
    DeviceInfo& di = g_devinfo[dev];
    if (di.sms == 0) {
      e = cudaDeviceGetAttribute(&di.sms, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return cuda_fail(e);
    }
    *sms_out = di.sms;
  }
  std::lock_guard<std::mutex> lock(g_crc_mutex);
  const int idx = (F - 1) * 2 + (PACK ? 1 : 0);
  if (!g_crc_attr_set[dev][idx]) {
    e = cudaFuncSetAttribute(topkv_crc_copy_kernel<F, PACK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kSmemBudget);
    if (e != cudaSuccess) return cuda_fail(e);
    g_crc_attr_set[dev][idx] = true;
  }
  return TOPKV_OK;
}

// A checksummed copy, validated and ready to launch: everything that can be refused is refused
// by crc_plan, so that a caller with work of its own to enqueue (the host leg's copies) only
// starts once the whole call is known to be acceptable.
struct CrcLaunch {
  CrcCopyParams cp;
  dim3 grid, block;
  size_t smem = 0;
  int F = 0;
  int64_t n_layer = -1;  // bytes of the layer's slab when total_tokens is known
  bool empty = true;     // nothing to launch (no requests, or no table columns)
};

// slab_override: device address to use for this layer's wire slab instead of wire + layer*stride
// (a staging slab, or the device view of a pinned host slab); max_ctas > 0: the wire is host
// memory behind PCIe, at most that many CTAs run.
// staging_capacity >= 0: slab_override is the staging slab of the staged host leg, which needs the
// slab's size on the host, adjacent planes (one contiguous copy) and room for the slab.
template <bool PACK>
int crc_plan(int layer, const void* pool, const topkv_layout* lo, const topkv_batch* b, const void* wire,
             int64_t cap, void* ws, int64_t ws_bytes, void* slab_override, int max_ctas, CrcLaunch* out,
             int64_t staging_capacity = -1) {
  CrcCopyParams& cp = out->cp;
  Resolved rs;
  int st = prepare(layer, pool, lo, b, wire, cap, lo ? lo->wire_layer_stride : 0, &cp.k, &rs, &out->n_layer);
  if (st != TOPKV_OK) return st;
  if (staging_capacity >= 0) {
    if (out->n_layer < 0) return TOPKV_ERR_INVALID_ARG;
    if (lo->wire_plane_stride != 0) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
    if (!mult16p(slab_override)) return TOPKV_ERR_ALIGNMENT;
    if (staging_capacity < out->n_layer) return TOPKV_ERR_CAPACITY;
  }
  if (slab_override != nullptr) cp.k.wire = static_cast<uint8_t*>(slab_override);
  if (ws == nullptr || !mult16p(ws)) return TOPKV_ERR_INVALID_ARG;
  const int F = (int)lo->kv_factor, R = b->num_requests, maxp = b->max_pages_per_req;
  const int L = (int)lo->num_layers;
  if (R > kCrcMaxR) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  st = crc_geometry(lo, rs, maxp, &cp.g);
  if (st != TOPKV_OK) return st;
  if (ws_bytes < 8 * crc_workspace_words(cp.g.kmax, L, R, F)) return TOPKV_ERR_CAPACITY;
  out->F = F;
  out->empty = R == 0 || maxp == 0;
  if (out->empty) return TOPKV_OK;
  if ((int64_t)R * cp.g.kmax * F > 0x7fffffffll) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  cp.w = crc_carve(ws, cp.g.kmax, L, R, F);
  cp.layer = layer;
  cp.stages = TOPKV_CRC_STAGES;
  int warps = 0, sms = 0;
  st = crc_launch_shape(cp.g, R, cp.stages, &warps, &out->smem);
  if (st != TOPKV_OK) return st;
  st = (F == 1) ? crc_prepare_device<1, PACK>(&sms) : crc_prepare_device<2, PACK>(&sms);
  if (st != TOPKV_OK) return st;
  // persistent grid: kCrcCtasPerSm CTAs per SM, fewer when there is less work or the wire is behind PCIe
  const int64_t items = (int64_t)R * cp.g.kmax * F;  // upper bound
  int64_t ctas = std::min<int64_t>((int64_t)sms * kCrcCtasPerSm, (items + warps - 1) / warps);
  if (max_ctas > 0) ctas = std::min<int64_t>(ctas, max_ctas);
  out->grid = dim3((unsigned)std::max<int64_t>(1, ctas));
  out->block = dim3((unsigned)(warps * 32));
  return TOPKV_OK;
}

template <bool PACK>
int crc_launch(const CrcLaunch& cl, cudaStream_t stream) {
  if (cl.empty) return TOPKV_OK;
  cudaError_t e;
  if (cl.F == 1) e = launch_pdl(topkv_crc_copy_kernel<1, PACK>, cl.grid, cl.block, cl.smem, stream, cl.cp);
  else e = launch_pdl(topkv_crc_copy_kernel<2, PACK>, cl.grid, cl.block, cl.smem, stream, cl.cp);
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return TOPKV_OK;
}

template <bool PACK>
int crc_copy(int layer, const void* pool, const topkv_layout* lo, const topkv_batch* b,
             const void* wire, int64_t cap, void* ws, int64_t ws_bytes, cudaStream_t stream) {
  CrcLaunch cl;
  const int st = crc_plan<PACK>(layer, pool, lo, b, wire, cap, ws, ws_bytes, nullptr, 0, &cl);
  return st != TOPKV_OK ? st : crc_launch<PACK>(cl, stream);
}

// Host leg with checksums: the same two forms as the plain host-leg calls. Every argument is
// checked before the first copy or kernel is enqueued.
template <bool PACK>
int crc_host_leg(int layer, const void* pool, const topkv_layout* layout,
                        const topkv_batch* batch, const void* h_pinned, int64_t host_bytes,
                        void* d_staging, int64_t staging_capacity_bytes, void* ws, int64_t ws_bytes,
                        cudaStream_t s) {
  if (layout == nullptr || batch == nullptr || h_pinned == nullptr) return TOPKV_ERR_INVALID_ARG;
  CrcLaunch cl;
  if (d_staging == nullptr) {  // direct: the kernel works on the mapped pinned slab
    // validate with the host address first (layer range, capacity, workspace), then map it
    int st = crc_plan<PACK>(layer, pool, layout, batch, h_pinned, host_bytes, ws, ws_bytes, nullptr,
                            g_host_leg_ctas.load(std::memory_order_relaxed), &cl);
    if (st != TOPKV_OK) return st;
    void* dev = nullptr;
    st = mapped_device_pointer(h_pinned, &dev);
    if (st != TOPKV_OK) return st;
    cl.cp.k.wire = static_cast<uint8_t*>(dev) + (int64_t)layer * layout->wire_layer_stride;
    return crc_launch<PACK>(cl, s);
  }
  if (staging_capacity_bytes < 0) return TOPKV_ERR_INVALID_ARG;
  int st = crc_plan<PACK>(layer, pool, layout, batch, h_pinned, host_bytes, ws, ws_bytes, d_staging, 0, &cl,
                          staging_capacity_bytes);
  if (st != TOPKV_OK) return st;
  const int64_t n_layer = cl.n_layer;  // known: total_tokens >= 0
  // the layer index and the host capacity have been checked: the slab lies inside h_pinned
  const uint8_t* host_slab = static_cast<const uint8_t*>(h_pinned) + (int64_t)layer * layout->wire_layer_stride;
  if (!PACK && n_layer > 0) {  // bring the slab in first
    const cudaError_t e = cudaMemcpyAsync(d_staging, host_slab, (size_t)n_layer, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  st = crc_launch<PACK>(cl, s);
  if (st != TOPKV_OK) return st;
  if (PACK && n_layer > 0) {
    const cudaError_t e = cudaMemcpyAsync(const_cast<uint8_t*>(host_slab), d_staging, (size_t)n_layer,
                                          cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return TOPKV_OK;
}

// ---- ranges of layers --------------------------------------------------------------------------
// Checks that every layer of the range would be accepted before the first one is enqueued.
int check_layer_range(int first_layer, int num_layers, const void* pool, const topkv_layout* layout,
                      const topkv_batch* batch, const void* h_pinned, int64_t host_bytes,
                      const void* d_staging, int64_t staging_capacity_bytes) {
  if (num_layers < 0 || first_layer < 0) return TOPKV_ERR_LAYER_RANGE;
  if (layout == nullptr || batch == nullptr || h_pinned == nullptr) return TOPKV_ERR_INVALID_ARG;
  KParams kp;
  Resolved rs;
  int64_t n_layer;
  for (int i = 0; i < num_layers; ++i) {
    const int st = prepare(first_layer + i, pool, layout, batch, h_pinned, host_bytes,
                           layout->wire_layer_stride, &kp, &rs, &n_layer);
    if (st != TOPKV_OK) return st;
  }
  if (d_staging != nullptr) {
    if (batch->total_tokens < 0) return TOPKV_ERR_INVALID_ARG;
    if (layout->wire_plane_stride != 0) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
    if (!mult16p(d_staging)) return TOPKV_ERR_ALIGNMENT;
    if (staging_capacity_bytes < topkv_wire_layer_bytes(layout, batch->total_tokens)) return TOPKV_ERR_CAPACITY;
  } else if (num_layers > 0) {
    void* dev = nullptr;
    const int st = mapped_device_pointer(h_pinned, &dev);  // refuses pageable memory up front
    if (st != TOPKV_OK) return st;
  }
  return TOPKV_OK;
}

// lanes = 1: every layer on streams[0] with stagings[0]. lanes = 2: layer i of the range on
// streams[i % 2] with stagings[i % 2] (staged form only), so that the copy engine moves one
// layer while the kernel of the next one runs.
template <bool PACK>
int issue_layers(int first_layer, int num_layers, const void* pool, const topkv_layout* layout,
                 const topkv_batch* batch, const void* h_pinned, int64_t host_bytes, void* const* stagings,
                 int64_t staging_capacity_bytes, const topkv_event_t* layer_ready,
                 const topkv_event_t* layer_done, const topkv_stream_t* streams, int lanes) {
  if (stagings == nullptr || streams == nullptr) return TOPKV_ERR_INVALID_ARG;
  for (int q = 0; q < lanes; ++q) {
    if (lanes > 1 && stagings[q] == nullptr) return TOPKV_ERR_INVALID_ARG;  // two lanes: staged form only
    const int st = check_layer_range(first_layer, num_layers, pool, layout, batch, h_pinned, host_bytes,
                                     stagings[q], staging_capacity_bytes);
    if (st != TOPKV_OK) return st;
  }
  if (lanes > 1 && (stagings[0] == stagings[1] || streams[0] == streams[1])) return TOPKV_ERR_INVALID_ARG;
  for (int i = 0; i < num_layers; ++i) {
    const int q = i % lanes;
    cudaStream_t s = reinterpret_cast<cudaStream_t>(streams[q]);
    if (layer_ready != nullptr && layer_ready[i] != nullptr) {
      const cudaError_t e = cudaStreamWaitEvent(s, reinterpret_cast<cudaEvent_t>(layer_ready[i]), 0);
      if (e != cudaSuccess) return cuda_fail(e);
    }
    const int st =
        PACK ? topkv_pack_layer_to_host(first_layer + i, pool, layout, batch, const_cast<void*>(h_pinned),
                                        host_bytes, stagings[q], staging_capacity_bytes, streams[q])
             : topkv_unpack_layer_from_host(first_layer + i, const_cast<void*>(pool), layout, batch, h_pinned,
                                            host_bytes, stagings[q], staging_capacity_bytes, streams[q]);
    if (st != TOPKV_OK) return st;
    if (layer_done != nullptr && layer_done[i] != nullptr) {
      const cudaError_t e = cudaEventRecord(reinterpret_cast<cudaEvent_t>(layer_done[i]), s);
      if (e != cudaSuccess) return cuda_fail(e);
    }
  }
  return TOPKV_OK;
}

namespace multi {

// Validates a range of layers and fills the parameters of ONE launch that covers it.
// *launch is false when there is nothing to launch (an empty range).
int plan_layers(int first_layer, int num_layers, const void* pool, const topkv_layout* layout,
                const topkv_batch* batch, const void* d_wire, int64_t wire_bytes, KParams* kp,
                Resolved* rs, bool* launch) {
  *launch = false;
  if (num_layers < 0 || first_layer < 0) return TOPKV_ERR_LAYER_RANGE;
  if (num_layers > 65535) return TOPKV_ERR_INVALID_ARG;  // grid.y
  KParams kp_last;
  int64_t n_layer;
  if (num_layers == 0) {  // still validate the descriptors
    if (layout == nullptr) return TOPKV_ERR_INVALID_ARG;
    const int st = check_layout(layout, rs);
    return st != TOPKV_OK ? st : check_batch(layout, batch);
  }
  int st = prepare(first_layer, pool, layout, batch, d_wire, wire_bytes,
                   layout ? layout->wire_layer_stride : 0, kp, rs, &n_layer);
  if (st != TOPKV_OK) return st;
  st = prepare(first_layer + num_layers - 1, pool, layout, batch, d_wire, wire_bytes,
               layout->wire_layer_stride, &kp_last, rs, &n_layer);  // range and capacity of the last
  if (st != TOPKV_OK) return st;
  if (num_layers > 1) {
    if (layout->wire_layer_stride <= 0) return TOPKV_ERR_INVALID_ARG;  // all layers on one slab
    kp->S_layer = layout->pool_layer_stride;
    kp->W_layer = layout->wire_layer_stride;
    kp->wire_limit = std::min(kp->wire_limit, kp_last.wire_limit);  // the tightest slab bounds them all
  }
  *launch = true;
  return TOPKV_OK;
}

// One launch for the layers [first_layer, first_layer + num_layers).
template <bool PACK>
int copy_layers(int first_layer, int num_layers, const void* pool, const topkv_layout* layout,
                const topkv_batch* batch, const void* d_wire, int64_t wire_bytes, cudaStream_t s) {
  KParams kp;
  Resolved rs;
  bool launch = false;
  const int st = plan_layers(first_layer, num_layers, pool, layout, batch, d_wire, wire_bytes, &kp, &rs, &launch);
  if (st != TOPKV_OK || !launch) return st;
  return launch_copy<PACK>(kp, rs, (int)layout->kv_factor, s, 0, num_layers);
}

}  // namespace multi

// ---- a model whose layers differ in kind (§2.2) -------------------------------------------------
namespace model {

struct LayerPlan {
  KParams kp;
  Resolved rs;
  int F = 0;
  int64_t offset = 0;   // where the layer's slab starts in the wire buffer
  int64_t n_slab = 0;   // its size in bytes
  bool empty = false;   // nothing to launch
};

// The tokens of the batch that a layer of a given kind keeps come from the host copy of the
// lengths. Scratch of the call in progress on this thread (cleared at every entry point): the
// sums are remembered per distinct window (a model has a handful), so a call costs one pass
// over the lengths per window, not one per layer.
thread_local struct {
  const int32_t* lens = nullptr;
  int R = -1;
  std::vector<std::pair<int64_t, int64_t>> sums;  // (window or -1 for all tokens, tokens kept)
} g_token_sums;

void reset_token_sums(const topkv_layer_table* t, int R) {
  g_token_sums.lens = t->h_seq_lens;
  g_token_sums.R = R;
  g_token_sums.sums.clear();
}

int check_table(const topkv_layout* lo, const topkv_batch* b, const topkv_layer_table* t) {
  if (t == nullptr || t->struct_size != sizeof(topkv_layer_table) || t->specs == nullptr)
    return TOPKV_ERR_INVALID_ARG;
  if (lo == nullptr || b == nullptr) return TOPKV_ERR_INVALID_ARG;
  if (lo->struct_size != sizeof(topkv_layout)) return TOPKV_ERR_INVALID_ARG;  // fields are read below
  if (b->struct_size != sizeof(topkv_batch) || b->window_tokens != 0) return TOPKV_ERR_INVALID_ARG;
  if (b->num_requests < 0) return TOPKV_ERR_INVALID_ARG;
  if (b->num_requests > 0 && t->h_seq_lens == nullptr) return TOPKV_ERR_INVALID_ARG;
  for (int r = 0; r < b->num_requests; ++r)
    if (t->h_seq_lens[r] < 0) return TOPKV_ERR_INVALID_ARG;
  if (lo->wire_plane_stride != 0) return TOPKV_ERR_UNSUPPORTED_LAYOUT;  // slabs lie back to back
  reset_token_sums(t, b->num_requests);  // the lengths may have changed in place since the last call
  return TOPKV_OK;
}

// Tokens of the batch that a layer of this kind keeps (see g_token_sums).
int64_t kept_tokens(const topkv_layer_table* t, int R, const topkv_layer_spec& sp) {
  const int64_t key = sp.kind == TOPKV_LAYER_WINDOW ? sp.param : -1;
  if (g_token_sums.lens != t->h_seq_lens || g_token_sums.R != R) reset_token_sums(t, R);
  for (const auto& kv : g_token_sums.sums)
    if (kv.first == key) return kv.second;
  int64_t total = 0;
  for (int r = 0; r < R; ++r) {
    const int64_t s = t->h_seq_lens[r];
    total += (key >= 0 && key < s) ? key : s;
  }
  g_token_sums.sums.emplace_back(key, total);
  return total;
}

int slab_bytes(const topkv_layout* lo, const topkv_layer_table* t, int R, uint32_t l, int64_t* out) {
  const topkv_layer_spec& sp = t->specs[l];
  if (sp.reserved != 0 || sp.param < 0) return TOPKV_ERR_INVALID_ARG;
  const int64_t tok_bytes = (int64_t)lo->kv_factor * lo->num_kv_heads * lo->head_dim * lo->elem_bytes;
  switch (sp.kind) {
    case TOPKV_LAYER_FULL:
    case TOPKV_LAYER_WINDOW: *out = tok_bytes * kept_tokens(t, R, sp); return TOPKV_OK;
    case TOPKV_LAYER_STATE: *out = (int64_t)R * sp.param; return TOPKV_OK;
    default: return TOPKV_ERR_INVALID_ARG;
  }
}

// Plans model layer l: validates it and fills the kernel parameters, exactly as the per-layer
// calls would for the view this layer has of the pools. `wire_base` / `capacity` describe the
// whole wire buffer (device, or pinned host); `offset` is the layer's place in it.
int plan_layer(uint32_t l, const void* pool, const topkv_layout* lo, const topkv_batch* b,
               const topkv_layer_table* t, const void* wire_base, int64_t capacity, int64_t offset,
               uint32_t flags, LayerPlan* out) {
  const int R = b->num_requests;
  const topkv_layer_spec& sp = t->specs[l];
  int st = slab_bytes(lo, t, R, l, &out->n_slab);
  if (st != TOPKV_OK) return st;
  out->offset = offset;
  if (wire_base == nullptr || capacity < 0) return TOPKV_ERR_INVALID_ARG;
  if (offset + out->n_slab > capacity) return TOPKV_ERR_CAPACITY;
  uint32_t ord = 0;  // this layer's number among the layers of its own pool
  for (uint32_t q = 0; q < l; ++q)
    ord += (t->specs[q].kind == TOPKV_LAYER_STATE) == (sp.kind == TOPKV_LAYER_STATE) ? 1u : 0u;
  const uint8_t* slab = static_cast<const uint8_t*>(wire_base) + offset;
  if (sp.kind != TOPKV_LAYER_STATE) {
    topkv_layout lo2 = *lo;
    lo2.wire_layer_stride = 0;  // the slab is addressed directly
    topkv_batch b2 = *b;
    b2.flags = flags;
    b2.window_tokens = sp.kind == TOPKV_LAYER_WINDOW ? (int32_t)std::min<int64_t>(sp.param, 0x7fffffff) : 0;
    if (sp.kind == TOPKV_LAYER_WINDOW && sp.param == 0) return TOPKV_ERR_INVALID_ARG;  // a window of no tokens
    b2.total_tokens = R > 0 ? kept_tokens(t, R, sp) : 0;
    if (b2.window_tokens != 0) b2.cu_seq_lens = nullptr;  // the plan's prefix sums count whole sequences
    if (b->total_tokens >= 0 && R > 0) {                  // the two descriptions of the batch must agree
      topkv_layer_spec full = {TOPKV_LAYER_FULL, 0, 0};
      if (kept_tokens(t, R, full) != b->total_tokens) return TOPKV_ERR_INVALID_ARG;
    }
    int64_t n_layer = 0;
    st = prepare((int)ord, pool, &lo2, &b2, slab, capacity - offset, 0, &out->kp, &out->rs, &n_layer);
    if (st != TOPKV_OK) return st;
    out->F = (int)lo->kv_factor;
    out->empty = (int64_t)out->kp.R * out->kp.maxp == 0;
    return TOPKV_OK;
  }
  // a constant-state layer: R states of sp.param bytes, one slot each, shipped in request order.
  // The copy kernel sees the slot as one page of `k` rows, every request having exactly k tokens.
  const int64_t B = sp.param;
  out->F = 1;
  out->empty = R == 0 || B == 0;
  if (out->empty) return TOPKV_OK;
  if (t->state_pool == nullptr || t->state_slots == nullptr || t->num_state_slots <= 0)
    return TOPKV_ERR_INVALID_ARG;
  if (t->state_slot_stride < B || t->state_layer_stride <= 0) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  if (!mult16(B) || !mult16(t->state_slot_stride) || !mult16(t->state_layer_stride) ||
      !mult16p(t->state_pool) || !mult16p(slab))
    return TOPKV_ERR_ALIGNMENT;
  int64_t row = 4096;  // the largest power of two up to 4 KiB that divides the state
  while (B % row) row >>= 1;
  const int64_t k = B / row;
  if (k * (int64_t)R > 0x7fffffffll) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  KParams& kp = out->kp;
  kp = KParams{};
  kp.pool = static_cast<uint8_t*>(t->state_pool) + (int64_t)ord * t->state_layer_stride;
  kp.wire = const_cast<uint8_t*>(slab);
  kp.bt = t->state_slots;  // [R][1]: the slot is the request's only "page"
  kp.sl = nullptr;
  kp.cu = nullptr;
  kp.T = (int64_t)R * k;
  kp.S_page = t->state_slot_stride;
  kp.S_kv = 0;
  kp.S_tok = row;
  kp.S_unit = 0;
  kp.R = R;
  kp.maxp = 1;
  kp.P = (int)k;
  kp.U = 1;
  kp.unit_chunks = (int)(row / 16);
  kp.planar = 0;
  kp.plane_rows = -1;
  kp.window = 0;
  kp.ppc = 1;
  kp.spr = 1;
  kp.cpp = 1;
  kp.tps = 0;
  kp.const_len = (int)k;
  kp.num_pages = t->num_state_slots;
  kp.wire_limit = out->n_slab;
  kp.overlap = (flags & TOPKV_FLAG_OVERLAP_PREVIOUS) ? 1 : 0;
  kp.late_wait = (!kp.overlap && (flags & TOPKV_FLAG_TABLES_SETTLED)) ? 1 : 0;
  kp.S_layer = 0;
  kp.W_layer = 0;
  out->rs.row_bytes = row;
  out->rs.unit_bytes = row;
  out->rs.U = 1;
  out->rs.merged = true;
  return TOPKV_OK;
}

int check_range(const topkv_layer_table* t, int first_layer, int num_layers) {
  if (first_layer < 0 || num_layers < 0 || (int64_t)first_layer + num_layers > (int64_t)t->num_layers)
    return TOPKV_ERR_LAYER_RANGE;
  return TOPKV_OK;
}

// Offset of layer `first` and, through `visit`, every layer of the range with its offset.
template <typename Visit>
int for_layers(int first_layer, int num_layers, const topkv_layout* lo, const topkv_batch* b,
               const topkv_layer_table* t, Visit visit) {
  int64_t off = 0;
  for (uint32_t l = 0; l < (uint32_t)(first_layer + num_layers); ++l) {
    int64_t n = 0;
    const int st = slab_bytes(lo, t, b->num_requests, l, &n);
    if (st != TOPKV_OK) return st;
    if (l >= (uint32_t)first_layer) {
      const int sv = visit(l, off);
      if (sv != TOPKV_OK) return sv;
    }
    off += n;
  }
  return TOPKV_OK;
}

// Device to device. The layers of one call touch different slabs and different pool layers, so
// every launch after the first may overlap its predecessor, and layers of the same kind and
// parameter whose places in their pool and in the wire form an arithmetic progression (every
// other layer of a model that alternates windowed and full layers; the state layers between the
// full ones) are equal slabs at a constant stride on both sides: they go into ONE launch, the
// layer being blockIdx.y, instead of one launch-bound kernel each.
template <bool PACK>
int copy_layers(int first_layer, int num_layers, const void* pool, const topkv_layout* lo,
                const topkv_batch* b, const topkv_layer_table* t, const void* d_wire, int64_t wire_bytes,
                cudaStream_t s) {
  int st = check_table(lo, b, t);
  if (st != TOPKV_OK) return st;
  st = check_range(t, first_layer, num_layers);
  if (st != TOPKV_OK) return st;
  struct Info {
    int64_t off;
    uint32_t ord;
    bool done;
  };
  std::vector<Info> info((size_t)num_layers);
  LayerPlan lp;
  st = for_layers(first_layer, num_layers, lo, b, t, [&](uint32_t l, int64_t off) {  // validate all first
    uint32_t ord = 0;
    for (uint32_t q = 0; q < l; ++q)
      ord += (t->specs[q].kind == TOPKV_LAYER_STATE) == (t->specs[l].kind == TOPKV_LAYER_STATE) ? 1u : 0u;
    info[l - first_layer] = {off, ord, false};
    return plan_layer(l, pool, lo, b, t, d_wire, wire_bytes, off, b->flags, &lp);
  });
  if (st != TOPKV_OK) return st;
  // the runs: same kind and parameter, constant stride in pool and wire
  struct Run {
    int first, count;
    int64_t d_off, d_ord, bytes;
  };
  std::vector<Run> runs;
  for (int i = 0; i < num_layers; ++i) {
    if (info[i].done) continue;
    const topkv_layer_spec& sp = t->specs[first_layer + i];
    int count = 1, last = i;
    int64_t d_off = 0, d_ord = 0;
    for (int j = i + 1; j < num_layers && count < 65535; ++j) {
      const topkv_layer_spec& sq = t->specs[first_layer + j];
      if (info[j].done || sq.kind != sp.kind || sq.param != sp.param) continue;
      const int64_t o = info[j].off - info[last].off, r = (int64_t)info[j].ord - info[last].ord;
      if (count == 1) {
        d_off = o;
        d_ord = r;
      } else if (o != d_off || r != d_ord) {
        continue;
      }
      info[j].done = true;
      last = j;
      ++count;
    }
    info[i].done = true;
    int64_t n = 0;
    st = slab_bytes(lo, t, b->num_requests, (uint32_t)(first_layer + i), &n);
    if (st != TOPKV_OK) return st;
    runs.push_back({i, count, d_off, d_ord, n * count});
  }
  // The launches of one call are independent of each other, so their order is free: the largest
  // run goes first and the small ones (the 4 MiB slabs of windowed layers) run under its tail
  // instead of standing alone, launch-bound, between two large ones.
  std::stable_sort(runs.begin(), runs.end(), [](const Run& a, const Run& c) { return a.bytes > c.bytes; });
  bool launched = false;
  for (const Run& run : runs) {
    const bool is_state = t->specs[first_layer + run.first].kind == TOPKV_LAYER_STATE;
    const uint32_t flags = launched ? (b->flags | TOPKV_FLAG_OVERLAP_PREVIOUS) : b->flags;
    st = plan_layer((uint32_t)(first_layer + run.first), pool, lo, b, t, d_wire, wire_bytes, info[run.first].off,
                    flags, &lp);
    if (st != TOPKV_OK) return st;
    if (lp.empty) continue;
    if (run.count > 1) {
      lp.kp.S_layer = run.d_ord * (is_state ? t->state_layer_stride : lo->pool_layer_stride);
      lp.kp.W_layer = run.d_off;
    }
    st = launch_copy<PACK>(lp.kp, lp.rs, lp.F, s, 0, run.count);
    if (st != TOPKV_OK) return st;
    launched = true;
  }
  return TOPKV_OK;
}

// The side-stream schedule of §5.2 for such a model: per layer wait, ship over PCIe, record.
template <bool PACK>
int issue_layers(int first_layer, int num_layers, const void* pool, const topkv_layout* lo,
                 const topkv_batch* b, const topkv_layer_table* t, const void* h_pinned, int64_t host_bytes,
                 void* d_staging, int64_t staging_capacity_bytes, const topkv_event_t* layer_ready,
                 const topkv_event_t* layer_done, cudaStream_t s) {
  int st = check_table(lo, b, t);
  if (st != TOPKV_OK) return st;
  st = check_range(t, first_layer, num_layers);
  if (st != TOPKV_OK) return st;
  if (h_pinned == nullptr) return TOPKV_ERR_INVALID_ARG;
  if (d_staging != nullptr && !mult16p(d_staging)) return TOPKV_ERR_ALIGNMENT;
  LayerPlan lp;
  st = for_layers(first_layer, num_layers, lo, b, t, [&](uint32_t l, int64_t off) {  // validate all first
    const int sv = plan_layer(l, pool, lo, b, t, h_pinned, host_bytes, off, b->flags, &lp);
    if (sv != TOPKV_OK) return sv;
    if (d_staging != nullptr && staging_capacity_bytes < lp.n_slab) return (int)TOPKV_ERR_CAPACITY;
    return (int)TOPKV_OK;
  });
  if (st != TOPKV_OK) return st;
  uint8_t* dev_view = nullptr;  // the pinned buffer as the GPU sees it (direct form)
  if (d_staging == nullptr && num_layers > 0) {
    void* dev = nullptr;
    st = mapped_device_pointer(h_pinned, &dev);  // refuses pageable memory before anything is enqueued
    if (st != TOPKV_OK) return st;
    dev_view = static_cast<uint8_t*>(dev);
  }
  const int host_ctas = g_host_leg_ctas.load(std::memory_order_relaxed);
  return for_layers(first_layer, num_layers, lo, b, t, [&](uint32_t l, int64_t off) {
    const int i = (int)l - first_layer;
    if (layer_ready != nullptr && layer_ready[i] != nullptr) {
      const cudaError_t e = cudaStreamWaitEvent(s, reinterpret_cast<cudaEvent_t>(layer_ready[i]), 0);
      if (e != cudaSuccess) return cuda_fail(e);
    }
    int sv = plan_layer(l, pool, lo, b, t, h_pinned, host_bytes, off, b->flags, &lp);
    if (sv != TOPKV_OK) return sv;
    uint8_t* host_slab = const_cast<uint8_t*>(static_cast<const uint8_t*>(h_pinned)) + off;
    if (!lp.empty && lp.n_slab > 0) {
      if (d_staging == nullptr) {  // direct: mapped stores / loads from a bounded grid
        lp.kp.wire = dev_view + off;
        sv = launch_copy<PACK>(lp.kp, lp.rs, lp.F, s, host_ctas);
        if (sv != TOPKV_OK) return sv;
      } else {
        lp.kp.wire = static_cast<uint8_t*>(d_staging);
        if (!PACK) {
          const cudaError_t e = cudaMemcpyAsync(d_staging, host_slab, (size_t)lp.n_slab, cudaMemcpyHostToDevice, s);
          if (e != cudaSuccess) return cuda_fail(e);
        }
        sv = launch_copy<PACK>(lp.kp, lp.rs, lp.F, s);
        if (sv != TOPKV_OK) return sv;
        if (PACK) {
          const cudaError_t e = cudaMemcpyAsync(host_slab, d_staging, (size_t)lp.n_slab, cudaMemcpyDeviceToHost, s);
          if (e != cudaSuccess) return cuda_fail(e);
        }
      }
    }
    if (layer_done != nullptr && layer_done[i] != nullptr) {
      const cudaError_t e = cudaEventRecord(reinterpret_cast<cudaEvent_t>(layer_done[i]), s);
      if (e != cudaSuccess) return cuda_fail(e);
    }
    return (int)TOPKV_OK;
  });
}

}  // namespace model
}  // namespace

extern "C" {

int topkv_pack_layer(int layer, const void* src_pool, const topkv_layout* layout,
                     const topkv_batch* batch, void* d_wire, int64_t wire_capacity_bytes,
                     topkv_stream_t stream) {
  KParams kp;
  Resolved rs;
  int64_t n_layer;
  const int st = prepare(layer, src_pool, layout, batch, d_wire, wire_capacity_bytes,
                         layout ? layout->wire_layer_stride : 0, &kp, &rs, &n_layer);
  if (st != TOPKV_OK) return st;
  return launch_copy<true>(kp, rs, (int)layout->kv_factor, reinterpret_cast<cudaStream_t>(stream));
}

int topkv_unpack_layer(int layer, void* dst_pool, const topkv_layout* layout,
                       const topkv_batch* batch, const void* d_wire, int64_t wire_bytes,
                       topkv_stream_t stream) {
  KParams kp;
  Resolved rs;
  int64_t n_layer;
  const int st = prepare(layer, dst_pool, layout, batch, d_wire, wire_bytes,
                         layout ? layout->wire_layer_stride : 0, &kp, &rs, &n_layer);
  if (st != TOPKV_OK) return st;
  return launch_copy<false>(kp, rs, (int)layout->kv_factor, reinterpret_cast<cudaStream_t>(stream));
}


namespace {
// Checks a span link and puts it into the kernel parameters: a linked launch orders itself
// span by span, so it never waits for the previous kernel as a whole (kp->overlap) unless the
// link asks for that too; then it waits before it reads anything and releases the next kernel
// only afterwards, which orders every later linked launch behind the previous kernel as well.
int apply_link(const topkv_span_link* link, KParams* kp) {
  if (link == nullptr || link->struct_size != sizeof(topkv_span_link) ||
      (link->flags & ~TOPKV_LINK_WAIT_PREVIOUS) != 0)
    return TOPKV_ERR_INVALID_ARG;
  if (link->d_await == nullptr && link->d_signal == nullptr) return TOPKV_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(link->d_await) | reinterpret_cast<uintptr_t>(link->d_signal)) & 3)
    return TOPKV_ERR_ALIGNMENT;
  kp->link_await = link->d_await;
  kp->link_signal = link->d_signal;
  kp->await_epoch = (int)link->await_epoch;
  kp->signal_epoch = (int)link->signal_epoch;
  kp->overlap = (link->flags & TOPKV_LINK_WAIT_PREVIOUS) ? 0 : 1;
  kp->late_wait = 0;
  return TOPKV_OK;
}
}  // namespace

int64_t topkv_span_link_words(const topkv_layout* layout, const topkv_batch* batch) {
  Resolved rs;
  int st = check_layout(layout, &rs);
  if (st != TOPKV_OK) return st;
  st = check_batch(layout, batch);
  if (st != TOPKV_OK) return st;
  KParams kp = {};
  kp.R = batch->num_requests;
  kp.maxp = batch->max_pages_per_req;
  kp.P = (int)layout->page_tokens;
  if ((int64_t)kp.R * kp.maxp == 0) return 0;
  span_geometry(&kp, (int)layout->kv_factor, rs.row_bytes);
  return (int64_t)kp.R * kp.spr;
}

int topkv_pack_layer_linked(int layer, const void* src_pool, const topkv_layout* layout,
                            const topkv_batch* batch, void* d_wire, int64_t wire_capacity_bytes,
                            const topkv_span_link* link, topkv_stream_t stream) {
  KParams kp;
  Resolved rs;
  int64_t n_layer;
  int st = prepare(layer, src_pool, layout, batch, d_wire, wire_capacity_bytes,
                   layout ? layout->wire_layer_stride : 0, &kp, &rs, &n_layer);
  if (st != TOPKV_OK) return st;
  st = apply_link(link, &kp);
  if (st != TOPKV_OK) return st;
  return launch_copy<true>(kp, rs, (int)layout->kv_factor, reinterpret_cast<cudaStream_t>(stream));
}

int topkv_unpack_layer_linked(int layer, void* dst_pool, const topkv_layout* layout,
                              const topkv_batch* batch, const void* d_wire, int64_t wire_bytes,
                              const topkv_span_link* link, topkv_stream_t stream) {
  KParams kp;
  Resolved rs;
  int64_t n_layer;
  int st = prepare(layer, dst_pool, layout, batch, d_wire, wire_bytes,
                   layout ? layout->wire_layer_stride : 0, &kp, &rs, &n_layer);
  if (st != TOPKV_OK) return st;
  st = apply_link(link, &kp);
  if (st != TOPKV_OK) return st;
  return launch_copy<false>(kp, rs, (int)layout->kv_factor, reinterpret_cast<cudaStream_t>(stream));
}

int topkv_relay_layers_linked(int first_layer, int num_layers, const void* src_pool,
                              const topkv_layout* src_layout, const topkv_batch* src_batch, void* dst_pool,
                              const topkv_layout* dst_layout, const topkv_batch* dst_batch, void* d_slab,
                              int64_t slab_bytes, int32_t* d_flags, int64_t flags_words,
                              uint32_t first_epoch, topkv_stream_t stream) {
  if (first_layer < 0 || num_layers < 0) return TOPKV_ERR_LAYER_RANGE;
  if (src_layout == nullptr || dst_layout == nullptr || src_layout->struct_size != sizeof(topkv_layout) ||
      dst_layout->struct_size != sizeof(topkv_layout))
    return TOPKV_ERR_INVALID_ARG;
  const int64_t ws = topkv_span_link_words(src_layout, src_batch);
  const int64_t wd = topkv_span_link_words(dst_layout, dst_batch);
  if (ws < 0) return (int)ws;
  if (wd < 0) return (int)wd;
  // both sides must cut the batch into the same spans and agree on what a wire row is
  if (ws != wd || src_layout->page_tokens != dst_layout->page_tokens ||
      src_batch->num_requests != dst_batch->num_requests ||
      src_batch->max_pages_per_req != dst_batch->max_pages_per_req ||
      src_batch->window_tokens != dst_batch->window_tokens ||
      src_layout->kv_factor != dst_layout->kv_factor || src_layout->num_kv_heads != dst_layout->num_kv_heads ||
      src_layout->head_dim != dst_layout->head_dim || src_layout->elem_bytes != dst_layout->elem_bytes ||
      src_layout->wire_order != dst_layout->wire_order ||
      src_layout->wire_plane_stride != dst_layout->wire_plane_stride)
    return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  if (ws > 0 && (d_flags == nullptr || flags_words < 2 * ws)) return d_flags == nullptr ? TOPKV_ERR_INVALID_ARG
                                                                                        : TOPKV_ERR_CAPACITY;
  if ((uint64_t)first_epoch + (uint64_t)num_layers > 0x7fffffffull) return TOPKV_ERR_INVALID_ARG;
  topkv_layout ls = *src_layout, ld = *dst_layout;
  ls.wire_layer_stride = 0;  // every layer goes through the one slab
  ld.wire_layer_stride = 0;
  // validate every layer on both sides before the first launch
  KParams kp;
  Resolved rs;
  int64_t n_layer;
  for (int i = 0; i < num_layers; ++i) {
    int st = prepare(first_layer + i, src_pool, &ls, src_batch, d_slab, slab_bytes, 0, &kp, &rs, &n_layer);
    if (st != TOPKV_OK) return st;
    st = prepare(first_layer + i, dst_pool, &ld, dst_batch, d_slab, slab_bytes, 0, &kp, &rs, &n_layer);
    if (st != TOPKV_OK) return st;
  }
  int32_t* packed = d_flags;         // span s of the slab holds the layer of epoch e
  int32_t* consumed = d_flags + ws;  // span s of the slab has been read for the layer of epoch e
  for (int i = 0; i < num_layers; ++i) {
    const uint32_t e = first_epoch + (uint32_t)i;
    const uint32_t lf = (i == 0 && !(src_batch->flags & TOPKV_FLAG_OVERLAP_PREVIOUS)) ? TOPKV_LINK_WAIT_PREVIOUS : 0u;
    topkv_span_link lp = {sizeof(topkv_span_link), e, e + 1, lf, e ? consumed : nullptr, packed};
    int st = topkv_pack_layer_linked(first_layer + i, src_pool, &ls, src_batch, d_slab, slab_bytes, &lp, stream);
    if (st != TOPKV_OK) return st;
    topkv_span_link lu = {sizeof(topkv_span_link), e + 1, e + 1, 0, packed, consumed};
    st = topkv_unpack_layer_linked(first_layer + i, dst_pool, &ld, dst_batch, d_slab, slab_bytes, &lu, stream);
    if (st != TOPKV_OK) return st;
  }
  return TOPKV_OK;
}

int topkv_pack_layers(int first_layer, int num_layers, const void* src_pool, const topkv_layout* layout,
                      const topkv_batch* batch, void* d_wire, int64_t wire_capacity_bytes,
                      topkv_stream_t stream) {
  return multi::copy_layers<true>(first_layer, num_layers, src_pool, layout, batch, d_wire, wire_capacity_bytes,
                                  reinterpret_cast<cudaStream_t>(stream));
}

int topkv_unpack_layers(int first_layer, int num_layers, void* dst_pool, const topkv_layout* layout,
                        const topkv_batch* batch, const void* d_wire, int64_t wire_bytes,
                        topkv_stream_t stream) {
  return multi::copy_layers<false>(first_layer, num_layers, dst_pool, layout, batch, d_wire, wire_bytes,
                                   reinterpret_cast<cudaStream_t>(stream));
}

int topkv_pack_layer_to_host(int layer, const void* src_pool, const topkv_layout* layout,
                             const topkv_batch* batch, void* h_pinned, int64_t host_capacity_bytes,
                             void* d_staging, int64_t staging_capacity_bytes,
                             topkv_stream_t stream) {
  KParams kp;
  Resolved rs;
  int64_t n_layer;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (d_staging == nullptr) {  // direct stores into the mapped pinned buffer
    int st = prepare(layer, src_pool, layout, batch, h_pinned, host_capacity_bytes,
                     layout ? layout->wire_layer_stride : 0, &kp, &rs, &n_layer);
    if (st != TOPKV_OK) return st;
    void* dev = nullptr;
    st = mapped_device_pointer(h_pinned, &dev);
    if (st != TOPKV_OK) return st;
    kp.wire = static_cast<uint8_t*>(dev) + (int64_t)layer * layout->wire_layer_stride;
    return launch_copy<true>(kp, rs, (int)layout->kv_factor, s,
                             g_host_leg_ctas.load(std::memory_order_relaxed));
  }
  // staged: pack this layer into the staging slab, then one copy-engine transfer
  if (batch != nullptr && batch->struct_size == sizeof(topkv_batch) && batch->total_tokens < 0)
    return TOPKV_ERR_INVALID_ARG;
  int st = prepare(layer, src_pool, layout, batch, h_pinned, host_capacity_bytes,
                   layout ? layout->wire_layer_stride : 0, &kp, &rs, &n_layer);
  if (st != TOPKV_OK) return st;
  if (layout->wire_plane_stride != 0) return TOPKV_ERR_UNSUPPORTED_LAYOUT;  // one contiguous copy
  if (!mult16p(d_staging)) return TOPKV_ERR_ALIGNMENT;
  if (staging_capacity_bytes < n_layer) return TOPKV_ERR_CAPACITY;
  uint8_t* host_slab = kp.wire;
  kp.wire = static_cast<uint8_t*>(d_staging);
  st = launch_copy<true>(kp, rs, (int)layout->kv_factor, s);
  if (st != TOPKV_OK) return st;
  if (n_layer > 0) {
    const cudaError_t e = cudaMemcpyAsync(host_slab, d_staging, (size_t)n_layer, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return TOPKV_OK;
}

int topkv_unpack_layer_from_host(int layer, void* dst_pool, const topkv_layout* layout,
                                 const topkv_batch* batch, const void* h_pinned, int64_t host_bytes,
                                 void* d_staging, int64_t staging_capacity_bytes,
                                 topkv_stream_t stream) {
  KParams kp;
  Resolved rs;
  int64_t n_layer;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (d_staging == nullptr) {  // direct loads from the mapped pinned buffer
    int st = prepare(layer, dst_pool, layout, batch, h_pinned, host_bytes,
                     layout ? layout->wire_layer_stride : 0, &kp, &rs, &n_layer);
    if (st != TOPKV_OK) return st;
    void* dev = nullptr;
    st = mapped_device_pointer(h_pinned, &dev);
    if (st != TOPKV_OK) return st;
    kp.wire = static_cast<uint8_t*>(dev) + (int64_t)layer * layout->wire_layer_stride;
    return launch_copy<false>(kp, rs, (int)layout->kv_factor, s,
                              g_host_leg_ctas.load(std::memory_order_relaxed));
  }
  if (batch != nullptr && batch->struct_size == sizeof(topkv_batch) && batch->total_tokens < 0)
    return TOPKV_ERR_INVALID_ARG;
  int st = prepare(layer, dst_pool, layout, batch, h_pinned, host_bytes,
                   layout ? layout->wire_layer_stride : 0, &kp, &rs, &n_layer);
  if (st != TOPKV_OK) return st;
  if (layout->wire_plane_stride != 0) return TOPKV_ERR_UNSUPPORTED_LAYOUT;  // one contiguous copy
  if (!mult16p(d_staging)) return TOPKV_ERR_ALIGNMENT;
  if (staging_capacity_bytes < n_layer) return TOPKV_ERR_CAPACITY;
  if (n_layer > 0) {
    const cudaError_t e = cudaMemcpyAsync(d_staging, kp.wire, (size_t)n_layer, cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  kp.wire = static_cast<uint8_t*>(d_staging);
  return launch_copy<false>(kp, rs, (int)layout->kv_factor, s);
}

int topkv_pack_layers_to_host_pipelined(int first_layer, int num_layers, const void* src_pool,
                                        const topkv_layout* layout, const topkv_batch* batch,
                                        void* h_pinned, int64_t host_capacity_bytes, void* d_staging,
                                        int64_t staging_capacity_bytes,
                                        const topkv_event_t* layer_ready,
                                        const topkv_event_t* layer_done, topkv_stream_t side_stream) {
  return issue_layers<true>(first_layer, num_layers, src_pool, layout, batch, h_pinned, host_capacity_bytes,
                            &d_staging, staging_capacity_bytes, layer_ready, layer_done, &side_stream, 1);
}

int topkv_pack_layers_to_host_two_lanes(int first_layer, int num_layers, const void* src_pool,
                                        const topkv_layout* layout, const topkv_batch* batch,
                                        void* h_pinned, int64_t host_capacity_bytes, void* const* d_stagings,
                                        int64_t staging_capacity_bytes, const topkv_event_t* layer_ready,
                                        const topkv_event_t* layer_done, const topkv_stream_t* side_streams) {
  return issue_layers<true>(first_layer, num_layers, src_pool, layout, batch, h_pinned, host_capacity_bytes,
                            d_stagings, staging_capacity_bytes, layer_ready, layer_done, side_streams, 2);
}

int topkv_unpack_layers_from_host_two_lanes(int first_layer, int num_layers, void* dst_pool,
                                            const topkv_layout* layout, const topkv_batch* batch,
                                            const void* h_pinned, int64_t host_bytes, void* const* d_stagings,
                                            int64_t staging_capacity_bytes, const topkv_event_t* layer_ready,
                                            const topkv_event_t* layer_done,
                                            const topkv_stream_t* side_streams) {
  return issue_layers<false>(first_layer, num_layers, dst_pool, layout, batch, h_pinned, host_bytes, d_stagings,
                             staging_capacity_bytes, layer_ready, layer_done, side_streams, 2);
}

int topkv_unpack_layers_from_host_pipelined(int first_layer, int num_layers, void* dst_pool,
                                            const topkv_layout* layout, const topkv_batch* batch,
                                            const void* h_pinned, int64_t host_bytes, void* d_staging,
                                            int64_t staging_capacity_bytes,
                                            const topkv_event_t* layer_ready,
                                            const topkv_event_t* layer_done,
                                            topkv_stream_t side_stream) {
  return issue_layers<false>(first_layer, num_layers, dst_pool, layout, batch, h_pinned, host_bytes,
                             &d_staging, staging_capacity_bytes, layer_ready, layer_done, &side_stream, 1);
}

int topkv_layer_table_offsets(const topkv_layout* layout, const topkv_layer_table* table,
                              int32_t num_requests, int64_t* h_offsets) {
  if (layout == nullptr || layout->struct_size != sizeof(topkv_layout) || table == nullptr ||
      table->struct_size != sizeof(topkv_layer_table) || table->specs == nullptr || h_offsets == nullptr ||
      num_requests < 0 || (num_requests > 0 && table->h_seq_lens == nullptr))
    return TOPKV_ERR_INVALID_ARG;
  for (int32_t r = 0; r < num_requests; ++r)
    if (table->h_seq_lens[r] < 0) return TOPKV_ERR_INVALID_ARG;
  model::reset_token_sums(table, num_requests);
  int64_t off = 0;
  for (uint32_t l = 0; l < table->num_layers; ++l) {
    h_offsets[l] = off;
    int64_t n = 0;
    const int st = model::slab_bytes(layout, table, num_requests, l, &n);
    if (st != TOPKV_OK) return st;
    off += n;
  }
  h_offsets[table->num_layers] = off;
  return TOPKV_OK;
}

int topkv_pack_model_layers(int first_layer, int num_layers, const void* src_pool, const topkv_layout* layout,
                            const topkv_batch* batch, const topkv_layer_table* table, void* d_wire,
                            int64_t wire_capacity_bytes, topkv_stream_t stream) {
  return model::copy_layers<true>(first_layer, num_layers, src_pool, layout, batch, table, d_wire,
                                  wire_capacity_bytes, reinterpret_cast<cudaStream_t>(stream));
}

int topkv_unpack_model_layers(int first_layer, int num_layers, void* dst_pool, const topkv_layout* layout,
                              const topkv_batch* batch, const topkv_layer_table* table, const void* d_wire,
                              int64_t wire_bytes, topkv_stream_t stream) {
  return model::copy_layers<false>(first_layer, num_layers, dst_pool, layout, batch, table, d_wire, wire_bytes,
                                   reinterpret_cast<cudaStream_t>(stream));
}

int topkv_pack_model_layers_to_host_pipelined(int first_layer, int num_layers, const void* src_pool,
                                              const topkv_layout* layout, const topkv_batch* batch,
                                              const topkv_layer_table* table, void* h_pinned,
                                              int64_t host_capacity_bytes, void* d_staging,
                                              int64_t staging_capacity_bytes, const topkv_event_t* layer_ready,
                                              const topkv_event_t* layer_done, topkv_stream_t side_stream) {
  return model::issue_layers<true>(first_layer, num_layers, src_pool, layout, batch, table, h_pinned,
                                   host_capacity_bytes, d_staging, staging_capacity_bytes, layer_ready,
                                   layer_done, reinterpret_cast<cudaStream_t>(side_stream));
}

int topkv_unpack_model_layers_from_host_pipelined(int first_layer, int num_layers, void* dst_pool,
                                                  const topkv_layout* layout, const topkv_batch* batch,
                                                  const topkv_layer_table* table, const void* h_pinned,
                                                  int64_t host_bytes, void* d_staging,
                                                  int64_t staging_capacity_bytes,
                                                  const topkv_event_t* layer_ready,
                                                  const topkv_event_t* layer_done, topkv_stream_t side_stream) {
  return model::issue_layers<false>(first_layer, num_layers, dst_pool, layout, batch, table, h_pinned, host_bytes,
                                    d_staging, staging_capacity_bytes, layer_ready, layer_done,
                                    reinterpret_cast<cudaStream_t>(side_stream));
}

int topkv_pack_layer_to_host_noalloc(int layer, const void* src_pool, const topkv_layout* layout,
                                     const topkv_batch* batch, void* h_pinned,
                                     int64_t host_capacity_bytes, topkv_stream_t stream) {
  KParams kp;
  Resolved rs;
  int64_t n_layer;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (batch != nullptr && batch->struct_size == sizeof(topkv_batch) && batch->total_tokens < 0)
    return TOPKV_ERR_INVALID_ARG;
  int st = prepare(layer, src_pool, layout, batch, h_pinned, host_capacity_bytes,
                   layout ? layout->wire_layer_stride : 0, &kp, &rs, &n_layer);
  if (st != TOPKV_OK) return st;
  if (layout->wire_plane_stride != 0) return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  if (n_layer > (int64_t)TOPKV_NOALLOC_STAGING_BYTES) return TOPKV_ERR_CAPACITY;
  void* staging = nullptr;
  st = noalloc_staging_address(&staging);  // first call on this device: symbol lookup
  if (st != TOPKV_OK) return st;
  uint8_t* host_slab = kp.wire;
  kp.wire = static_cast<uint8_t*>(staging);  // the device address, never the host-side handle
  st = launch_copy<true>(kp, rs, (int)layout->kv_factor, s);
  if (st != TOPKV_OK) return st;
  if (n_layer > 0) {
    const cudaError_t e = cudaMemcpyAsync(host_slab, staging, (size_t)n_layer, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return TOPKV_OK;
}

int topkv_repage_layer(int layer, const void* src_pool, const topkv_layout* src_layout,
                       const topkv_batch* src_batch, void* dst_pool,
                       const topkv_layout* dst_layout, const topkv_batch* dst_batch,
                       topkv_stream_t stream) {
  Resolved rs_s, rs_d;
  int st = check_layout(src_layout, &rs_s);
  if (st != TOPKV_OK) return st;
  st = check_layout(dst_layout, &rs_d);
  if (st != TOPKV_OK) return st;
  st = check_batch(src_layout, src_batch);
  if (st != TOPKV_OK) return st;
  st = check_batch(dst_layout, dst_batch);
  if (st != TOPKV_OK) return st;
  const topkv_layout *ls = src_layout, *ld = dst_layout;
  if (ls->kv_factor != ld->kv_factor || ls->num_kv_heads != ld->num_kv_heads ||
      ls->head_dim != ld->head_dim || ls->elem_bytes != ld->elem_bytes)
    return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  if (src_batch->num_requests != dst_batch->num_requests) return TOPKV_ERR_INVALID_ARG;
  if (src_batch->window_tokens != 0 || dst_batch->window_tokens != 0) return TOPKV_ERR_INVALID_ARG;
  if (layer < 0 || (uint32_t)layer >= ls->num_layers || (uint32_t)layer >= ld->num_layers)
    return TOPKV_ERR_LAYER_RANGE;
  if (src_pool == nullptr || dst_pool == nullptr) return TOPKV_ERR_INVALID_ARG;
  if (!mult16p(src_pool) || !mult16p(dst_pool)) return TOPKV_ERR_ALIGNMENT;
  if (src_batch->num_requests == 0 || src_batch->max_pages_per_req == 0 ||
      dst_batch->max_pages_per_req == 0)
    return TOPKV_OK;
  const int F = (int)ls->kv_factor;
  const int64_t head_bytes = (int64_t)ls->head_dim * ls->elem_bytes;
  const bool rows = rs_s.U == 1 && rs_d.U == 1;  // whole rows contiguous in both pools
  RepageParams p;
  p.src = const_cast<uint8_t*>(static_cast<const uint8_t*>(src_pool)) + (int64_t)layer * ls->pool_layer_stride;
  p.dst = static_cast<uint8_t*>(dst_pool) + (int64_t)layer * ld->pool_layer_stride;
  p.bt_s = src_batch->block_table;
  p.bt_d = dst_batch->block_table;
  p.sl = src_batch->seq_lens;
  p.Ss_page = ls->pool_page_stride;
  p.Ss_kv = F > 1 ? ls->pool_kv_stride : 0;
  p.Ss_tok = ls->pool_token_stride;
  p.Ss_unit = rows ? 0 : (rs_s.U == 1 ? head_bytes : ls->pool_head_stride);
  p.Sd_page = ld->pool_page_stride;
  p.Sd_kv = F > 1 ? ld->pool_kv_stride : 0;
  p.Sd_tok = ld->pool_token_stride;
  p.Sd_unit = rows ? 0 : (rs_d.U == 1 ? head_bytes : ld->pool_head_stride);
  p.ns_pages = ls->num_pool_pages;
  p.nd_pages = ld->num_pool_pages;
  p.R = src_batch->num_requests;
  p.maxp_s = src_batch->max_pages_per_req;
  p.maxp_d = dst_batch->max_pages_per_req;
  p.Ps = (int)ls->page_tokens;
  p.Pd = (int)ld->page_tokens;
  p.U = rows ? 1 : (int)ls->num_kv_heads;
  const int64_t unit_bytes = rows ? rs_s.row_bytes : head_bytes;
  const int64_t tok_bytes = (int64_t)F * rs_s.row_bytes;
  const int pmin = std::min(p.Ps, p.Pd);
  p.span_tokens = (int)std::max<int64_t>(
      1, std::min<int64_t>(kSpanTargetBytes / tok_bytes, (int64_t)(kRepageMaxPages - 1) * pmin));
  const int64_t row_tokens = std::min((int64_t)p.maxp_s * p.Ps, (int64_t)p.maxp_d * p.Pd);
  p.spr = (int)((row_tokens + p.span_tokens - 1) / p.span_tokens);
  if ((int64_t)p.R * p.spr > 0x7fffffffll) return TOPKV_ERR_INVALID_ARG;
  p.overlap = ((src_batch->flags & dst_batch->flags) & TOPKV_FLAG_OVERLAP_PREVIOUS) ? 1 : 0;
  const bool wide = ((reinterpret_cast<uintptr_t>(p.src) | reinterpret_cast<uintptr_t>(p.dst) |
                      (uintptr_t)p.Ss_page | (uintptr_t)p.Ss_kv | (uintptr_t)p.Ss_tok |
                      (uintptr_t)p.Ss_unit | (uintptr_t)p.Sd_page | (uintptr_t)p.Sd_kv |
                      (uintptr_t)p.Sd_tok | (uintptr_t)p.Sd_unit | (uintptr_t)unit_bytes) & 31) == 0;
  // a ragged batch whose total the caller has stated: one CTA per span that can hold tokens
  int64_t spans = (int64_t)p.R * p.spr;
  p.compact = 0;
  if (p.overlap && src_batch->total_tokens >= 0 && p.R <= kRepageThreads) {
    const int64_t bound = src_batch->total_tokens / p.span_tokens + p.R;
    if (bound * 10 < spans * 9) {
      p.compact = 1;
      spans = bound;
    }
  }
  const dim3 grid((unsigned)spans), block(kRepageThreads);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  cudaError_t le;
  if (wide) {
    p.unit_chunks = (int)(unit_bytes / 32);
    le = (F == 1) ? launch_pdl(topkv_repage_kernel<1, 32>, grid, block, 0, s, p)
                  : launch_pdl(topkv_repage_kernel<2, 32>, grid, block, 0, s, p);
  } else {
    p.unit_chunks = (int)(unit_bytes / 16);
    le = (F == 1) ? launch_pdl(topkv_repage_kernel<1, 16>, grid, block, 0, s, p)
                  : launch_pdl(topkv_repage_kernel<2, 16>, grid, block, 0, s, p);
  }
  if (le != cudaSuccess) {
    cudaGetLastError();
    return cuda_fail(le);
  }
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return TOPKV_OK;
}

int topkv_pack_layer_to_host_crc(int layer, const void* src_pool, const topkv_layout* layout,
                                 const topkv_batch* batch, void* h_pinned, int64_t host_capacity_bytes,
                                 void* d_staging, int64_t staging_capacity_bytes, void* d_workspace,
                                 int64_t workspace_bytes, topkv_stream_t stream) {
  return crc_host_leg<true>(layer, src_pool, layout, batch, h_pinned, host_capacity_bytes, d_staging,
                            staging_capacity_bytes, d_workspace, workspace_bytes,
                            reinterpret_cast<cudaStream_t>(stream));
}

int topkv_unpack_layer_from_host_crc(int layer, void* dst_pool, const topkv_layout* layout,
                                     const topkv_batch* batch, const void* h_pinned, int64_t host_bytes,
                                     void* d_staging, int64_t staging_capacity_bytes,
                                     void* d_workspace, int64_t workspace_bytes,
                                     topkv_stream_t stream) {
  return crc_host_leg<false>(layer, dst_pool, layout, batch, h_pinned, host_bytes, d_staging,
                             staging_capacity_bytes, d_workspace, workspace_bytes,
                             reinterpret_cast<cudaStream_t>(stream));
}

int64_t topkv_crc_workspace_bytes(const topkv_layout* layout, int32_t num_requests,
                                  int32_t max_pages_per_req) {
  Resolved rs;
  int st = check_layout(layout, &rs);
  if (st != TOPKV_OK) return st;
  if (num_requests < 0 || max_pages_per_req < 0) return TOPKV_ERR_INVALID_ARG;
  CrcGeom g;
  st = crc_geometry(layout, rs, max_pages_per_req, &g);
  if (st != TOPKV_OK) return st;
  return 8 * crc_workspace_words(g.kmax, (int)layout->num_layers, num_requests, (int)layout->kv_factor);
}

int topkv_crc_begin(const topkv_layout* layout, const topkv_batch* batch, void* d_workspace,
                    int64_t workspace_bytes, topkv_stream_t stream) {
  Resolved rs;
  int st = check_layout(layout, &rs);
  if (st != TOPKV_OK) return st;
  st = check_batch(layout, batch);
  if (st != TOPKV_OK) return st;
  if (d_workspace == nullptr || !mult16p(d_workspace)) return TOPKV_ERR_INVALID_ARG;
  const int F = (int)layout->kv_factor, R = batch->num_requests, maxp = batch->max_pages_per_req;
  const int L = (int)layout->num_layers;
  CrcGeom g;
  st = crc_geometry(layout, rs, maxp, &g);
  if (st != TOPKV_OK) return st;
  if (workspace_bytes < 8 * crc_workspace_words(g.kmax, L, R, F)) return TOPKV_ERR_CAPACITY;
  if (R == 0) return TOPKV_OK;
  const CrcWorkspace w = crc_carve(d_workspace, g.kmax, L, R, F);
  const int64_t total = std::max<int64_t>(32 + (int64_t)g.kmax + 1 + R + (int64_t)L * R * g.kmax * F, L);
  const unsigned blocks = (unsigned)std::min<int64_t>((total + 255) / 256, 1024);
  topkv_crc_begin_kernel<<<blocks, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      w, g, batch->seq_lens, L, R, maxp, (int)layout->page_tokens, rs.row_bytes, F);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return TOPKV_OK;
}

int topkv_pack_layer_crc(int layer, const void* src_pool, const topkv_layout* layout,
                         const topkv_batch* batch, void* d_wire, int64_t wire_capacity_bytes,
                         void* d_workspace, int64_t workspace_bytes, topkv_stream_t stream) {
  return crc_copy<true>(layer, src_pool, layout, batch, d_wire, wire_capacity_bytes, d_workspace,
                        workspace_bytes, reinterpret_cast<cudaStream_t>(stream));
}

int topkv_unpack_layer_crc(int layer, void* dst_pool, const topkv_layout* layout,
                           const topkv_batch* batch, const void* d_wire, int64_t wire_bytes,
                           void* d_workspace, int64_t workspace_bytes, topkv_stream_t stream) {
  return crc_copy<false>(layer, dst_pool, layout, batch, d_wire, wire_bytes, d_workspace,
                         workspace_bytes, reinterpret_cast<cudaStream_t>(stream));
}

int topkv_crc_finish(const topkv_layout* layout, const topkv_batch* batch, void* d_workspace,
                     int64_t workspace_bytes, uint64_t* d_crc_out, topkv_stream_t stream) {
  Resolved rs;
  int st = check_layout(layout, &rs);
  if (st != TOPKV_OK) return st;
  st = check_batch(layout, batch);
  if (st != TOPKV_OK) return st;
  if (d_workspace == nullptr || !mult16p(d_workspace) || d_crc_out == nullptr)
    return TOPKV_ERR_INVALID_ARG;
  const int F = (int)layout->kv_factor, R = batch->num_requests, maxp = batch->max_pages_per_req;
  const int L = (int)layout->num_layers;
  CrcGeom g;
  st = crc_geometry(layout, rs, maxp, &g);
  if (st != TOPKV_OK) return st;
  if (workspace_bytes < 8 * crc_workspace_words(g.kmax, L, R, F)) return TOPKV_ERR_CAPACITY;
  if (R == 0) return TOPKV_OK;
  const CrcWorkspace w = crc_carve(d_workspace, g.kmax, L, R, F);
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const int64_t warps = (int64_t)L * R * F;  // one per (layer, request, plane)
  if ((warps + 3) / 4 > 0x7fffffffll) return TOPKV_ERR_INVALID_ARG;
  topkv_crc_layer_kernel<<<(unsigned)((warps + 3) / 4), 128, 0, s>>>(w, g, batch->seq_lens, L, R, F, maxp,
                                                                     (int)layout->page_tokens);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  topkv_crc_finish_kernel<<<(R * F + 3) / 4, 128, 0, s>>>(w, batch->seq_lens, L, R, F, maxp,  // a warp each
                                                                (int)layout->page_tokens, rs.row_bytes, d_crc_out);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(2, std::memory_order_relaxed);
  return TOPKV_OK;
}

int topkv_build_plan(const topkv_batch* batch, int64_t* d_cu_seq_lens, topkv_stream_t stream) {
  if (batch == nullptr || batch->struct_size != sizeof(topkv_batch) || d_cu_seq_lens == nullptr)
    return TOPKV_ERR_INVALID_ARG;
  if (batch->num_requests < 0 || (batch->num_requests > 0 && batch->seq_lens == nullptr) ||
      batch->window_tokens < 0)
    return TOPKV_ERR_INVALID_ARG;
  topkv_plan_kernel<<<1, kThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      batch->seq_lens, batch->num_requests, batch->window_tokens, d_cu_seq_lens);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e);
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return TOPKV_OK;
}

int topkv_last_cuda_error(void) { return g_last_cuda_error; }

int topkv_reset_device_error_flags(void) {
  const int zero = 0;
  cudaError_t e = cudaDeviceSynchronize();  // no kernel may still raise a bit behind the reset
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaMemcpyToSymbol(g_device_error_flags, &zero, sizeof(int));
  if (e != cudaSuccess) return cuda_fail(e);
  return TOPKV_OK;
}

int topkv_device_error_flags(void) {
  int flags = 0;
  // every stream of the device, the non-blocking ones included, has to be done: the copy below
  // runs on the legacy default stream, which orders against blocking streams only
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e);
  e = cudaMemcpyFromSymbol(&flags, g_device_error_flags, sizeof(int));
  if (e != cudaSuccess) return cuda_fail(e);
  return flags;
}
int64_t topkv_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int topkv_copy_vector_bytes(int first_layer, int num_layers, const void* pool, const topkv_layout* layout,
                            const topkv_batch* batch, const void* d_wire, int64_t wire_bytes) {
  KParams kp;
  Resolved rs;
  bool launch = false;
  const int st = multi::plan_layers(first_layer, num_layers, pool, layout, batch, d_wire, wire_bytes, &kp, &rs,
                                    &launch);
  if (st != TOPKV_OK) return st;
  return launch ? copy_vector_bytes(kp, rs.unit_bytes, num_layers) : 0;
}

int64_t topkv_copy_grid_ctas(int layer, const void* pool, const topkv_layout* layout, const topkv_batch* batch,
                             const void* d_wire, int64_t wire_bytes, int32_t* compact) {
  KParams kp;
  Resolved rs;
  int64_t n_layer;
  const int st = prepare(layer, pool, layout, batch, d_wire, wire_bytes, layout ? layout->wire_layer_stride : 0,
                         &kp, &rs, &n_layer);
  if (st != TOPKV_OK) return st;
  if (compact != nullptr) *compact = 0;
  if ((int64_t)kp.R * kp.maxp == 0) return 0;
  bool walk = false;
  const int64_t spans = grid_spans(&kp, (int)layout->kv_factor, rs.row_bytes, 0, &walk);
  if (compact != nullptr) *compact = kp.compact;
  return spans;
}

int topkv_set_host_leg_ctas(int ctas) {
  if (ctas < 0 || ctas > 65535) return TOPKV_ERR_INVALID_ARG;
  return g_host_leg_ctas.exchange(ctas);
}

int topkv_set_kernel_variant(int variant) {
  if (variant < 0 || variant > 1) return TOPKV_ERR_INVALID_ARG;
  return g_variant.exchange(variant);
}

}  // extern "C"
