// Direct re-paging: paged pool -> paged pool through two block tables, without a wire slab.
// Same result as unpack(pack(.)) of the same layer, at half the memory traffic. The two pools
// may differ in page size and in every stride; they share F, H, D and E.
#pragma once
#include <cuda_runtime.h>

#include <cstdint>

#include "topkv_common.cuh"

namespace topkv {

constexpr int kRepageThreads = 256;
constexpr int kRepageMaxPages = 64;  // page ids staged per side per CTA

struct RepageParams {
  uint8_t* src;  // this layer's slab of the source pool
  uint8_t* dst;  // this layer's slab of the destination pool
  const int32_t* bt_s;
  const int32_t* bt_d;
  const int32_t* sl;
  int64_t Ss_page, Ss_kv, Ss_tok, Ss_unit;
  int64_t Sd_page, Sd_kv, Sd_tok, Sd_unit;
  int64_t ns_pages, nd_pages;
  int R, maxp_s, maxp_d, Ps, Pd;
  int U;            // units per (token, plane): 1, or H when either pool splits heads
  int unit_chunks;  // VEC-byte chunks per unit
  int span_tokens;  // tokens per CTA
  int spr;          // CTAs per request
  int compact;      // 1: one CTA per span that can hold tokens (see find_span), not per (request, span) slot
  int overlap;
};

template <int F, int VEC>
__global__ void __launch_bounds__(kRepageThreads, 3) topkv_repage_kernel(const RepageParams p) {
  __shared__ int32_t s_pg_s[kRepageMaxPages];
  __shared__ int32_t s_pg_d[kRepageMaxPages];
  pdl_prologue(p.overlap);
  constexpr int kUnroll = VEC == 32 ? 4 : 8;
  const int tid = threadIdx.x;
  const int slot = blockIdx.x;
  const int64_t row_tokens = min((int64_t)p.maxp_s * p.Ps, (int64_t)p.maxp_d * p.Pd);
  int r = slot / p.spr;
  int sidx = slot - r * p.spr;
  if (p.compact &&
      !find_span<kRepageThreads>(p.sl, p.R, (int)min(row_tokens, (int64_t)0x7fffffff), p.span_tokens, slot, &r, &sidx)) {
    pdl_epilogue(p.overlap);
    return;
  }
  const int first = sidx * p.span_tokens;
  int s_r = p.sl[r];
  if (s_r > row_tokens) {  // longer than a block-table row: copy what both rows describe
    s_r = (int)row_tokens;
    if (tid == 0 && first == 0) raise_error(kErrTable);
  }
  if (first < s_r) {
    const int v = min(p.span_tokens, s_r - first);
    const int js0 = first / p.Ps, jd0 = first / p.Pd;
    const int ns = (first + v - 1) / p.Ps - js0 + 1, nd = (first + v - 1) / p.Pd - jd0 + 1;
    if (tid < ns) {
      int pg = p.bt_s[(int64_t)r * p.maxp_s + js0 + tid];
      if (pg < 0 || pg >= p.ns_pages) {
        pg = -1;
        raise_error(kErrTable);
      }
      s_pg_s[tid] = pg;
    }
    if (tid >= 64 && tid - 64 < nd) {
      int pg = p.bt_d[(int64_t)r * p.maxp_d + jd0 + tid - 64];
      if (pg < 0 || pg >= p.nd_pages) {
        pg = -1;
        raise_error(kErrTable);
      }
      s_pg_d[tid - 64] = pg;
    }
    __syncthreads();

    const int nunits = v * F * p.U;
    const int tpu = min(p.unit_chunks, kRepageThreads);
    const int groups = kRepageThreads / tpu;
    const int my_g = tid / tpu;
    const int my_w = tid - my_g * tpu;
    if (my_g < groups) {
      for (int q0 = my_g; q0 < nunits; q0 += groups * kUnroll) {
        for (int w = my_w; w < p.unit_chunks; w += tpu) {
          Vec<VEC> buf[kUnroll];
          uint8_t* dstp[kUnroll];
          bool ok[kUnroll];
#pragma unroll
          for (int u = 0; u < kUnroll; ++u) {
            const int q = min(q0 + u * groups, nunits - 1);
            int h = 0, tc = q;
            if (p.U > 1) {
              tc = q / p.U;
              h = q - tc * p.U;
            }
            const int ts = tc / F, c = tc - ts * F;
            const int i = first + ts;
            const int js = i / p.Ps, jd = i / p.Pd;
            const int pgs = s_pg_s[js - js0], pgd = s_pg_d[jd - jd0];
            const uint8_t* a = p.src + (int64_t)pgs * p.Ss_page + c * p.Ss_kv +
                               (int64_t)(i - js * p.Ps) * p.Ss_tok + h * p.Ss_unit + (int64_t)w * VEC;
            dstp[u] = p.dst + (int64_t)pgd * p.Sd_page + c * p.Sd_kv +
                      (int64_t)(i - jd * p.Pd) * p.Sd_tok + h * p.Sd_unit + (int64_t)w * VEC;
            ok[u] = q0 + u * groups < nunits && pgs >= 0 && pgd >= 0;
            if (ok[u]) buf[u].load(a);
          }
#pragma unroll
          for (int u = 0; u < kUnroll; ++u)
            if (ok[u]) buf[u].store(dstp[u]);
        }
      }
    }
  }
  pdl_epilogue(p.overlap);
}

}  // namespace topkv
