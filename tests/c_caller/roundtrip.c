/* A caller written in C against the CUDA runtime: no Python and no torch anywhere near the path.
 * Builds a small ragged paged batch from a counter-based generator, packs every layer with the
 * library, unpacks it into a second pool with its own block table, and compares wire and
 * destination byte for byte with the CPU oracle (test infrastructure, linked only here).
 * Exit status 0 = identical. */
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "topkv.h"
#include "topkv_oracle.h"

#define CK(x)                                                                  \
  do {                                                                         \
    cudaError_t e_ = (x);                                                      \
    if (e_ != cudaSuccess) {                                                   \
      printf("CUDA error %s at line %d\n", cudaGetErrorString(e_), __LINE__);  \
      return 2;                                                                \
    }                                                                          \
  } while (0)

static uint64_t mix(uint64_t x) { /* splitmix64 */
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}

int main(void) {
  enum { L = 3, F = 2, H = 8, D = 128, E = 2, P = 16, R = 5, MAXP = 40 };
  const int32_t lens[R] = {600, 0, 17, 333, 64};
  int64_t T = 0, need = 0;
  int32_t sl[R], bt_s[R][MAXP], bt_d[R][MAXP];
  for (int r = 0; r < R; ++r) {
    sl[r] = lens[r];
    T += sl[r];
    need += (sl[r] + P - 1) / P;
  }
  const int64_t pages = need + 7;
  /* two different page orders: source pages ascending from 3 with a stride, destination descending */
  int64_t next = 0;
  for (int r = 0; r < R; ++r)
    for (int j = 0; j < MAXP; ++j) {
      const int used = j < (sl[r] + P - 1) / P;
      bt_s[r][j] = used ? (int32_t)((next * 5 + 3) % pages) : -1; /* 5 and `pages` are coprime below */
      bt_d[r][j] = used ? (int32_t)(pages - 1 - next) : -1;
      next += used;
    }
  if (pages % 5 == 0) { printf("pick another page count\n"); return 2; }

  topkv_layout lo;
  memset(&lo, 0, sizeof lo);
  lo.struct_size = sizeof lo;
  lo.kind = TOPKV_KIND_GQA;
  lo.num_layers = L; lo.kv_factor = F; lo.num_kv_heads = H; lo.head_dim = D; lo.elem_bytes = E;
  lo.page_tokens = P; lo.num_pool_pages = pages; lo.wire_order = TOPKV_WIRE_TOKEN_KV;
  if (topkv_layout_default_strides(&lo) != TOPKV_OK) return 3;
  const int64_t n_layer = topkv_wire_layer_bytes(&lo, T);
  lo.wire_layer_stride = n_layer;
  const int64_t pool_bytes = (int64_t)L * lo.pool_layer_stride, wire_bytes = (int64_t)L * n_layer;

  uint8_t* h_src = (uint8_t*)malloc(pool_bytes);
  uint8_t* h_dst = (uint8_t*)malloc(pool_bytes);
  uint8_t* h_dst_got = (uint8_t*)malloc(pool_bytes);
  uint8_t* h_wire = (uint8_t*)calloc(wire_bytes, 1);
  uint8_t* h_wire_got = (uint8_t*)malloc(wire_bytes);
  for (int64_t i = 0; i < pool_bytes / 8; ++i) {
    ((uint64_t*)h_src)[i] = mix((uint64_t)i);
    ((uint64_t*)h_dst)[i] = mix((uint64_t)i + (1ull << 40));
  }

  uint8_t *d_src, *d_dst, *d_wire;
  int32_t *d_bts, *d_btd, *d_sl;
  int64_t* d_cu;
  cudaStream_t stream;
  CK(cudaStreamCreateWithFlags(&stream, cudaStreamNonBlocking));
  CK(cudaMalloc((void**)&d_src, pool_bytes));
  CK(cudaMalloc((void**)&d_dst, pool_bytes));
  CK(cudaMalloc((void**)&d_wire, wire_bytes));
  CK(cudaMalloc((void**)&d_bts, sizeof bt_s));
  CK(cudaMalloc((void**)&d_btd, sizeof bt_d));
  CK(cudaMalloc((void**)&d_sl, sizeof sl));
  CK(cudaMalloc((void**)&d_cu, (R + 1) * sizeof(int64_t)));
  CK(cudaMemcpy(d_src, h_src, pool_bytes, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_dst, h_dst, pool_bytes, cudaMemcpyHostToDevice));
  CK(cudaMemset(d_wire, 0, wire_bytes));
  CK(cudaMemcpy(d_bts, bt_s, sizeof bt_s, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_btd, bt_d, sizeof bt_d, cudaMemcpyHostToDevice));
  CK(cudaMemcpy(d_sl, sl, sizeof sl, cudaMemcpyHostToDevice));

  topkv_batch bs, bd;
  memset(&bs, 0, sizeof bs);
  bs.struct_size = sizeof bs;
  bs.num_requests = R; bs.max_pages_per_req = MAXP;
  bs.block_table = d_bts; bs.seq_lens = d_sl; bs.cu_seq_lens = d_cu; bs.total_tokens = T;
  bd = bs;
  bd.block_table = d_btd;
  int st = topkv_build_plan(&bs, d_cu, (topkv_stream_t)stream);
  for (int l = 0; l < L && st == TOPKV_OK; ++l) {
    /* every layer has its own slab of the wire and of the pools: independent launches */
    bs.flags = l ? TOPKV_FLAG_OVERLAP_PREVIOUS : 0;
    st = topkv_pack_layer(l, d_src, &lo, &bs, d_wire, wire_bytes, (topkv_stream_t)stream);
  }
  for (int l = 0; l < L && st == TOPKV_OK; ++l) {
    bd.flags = l ? TOPKV_FLAG_OVERLAP_PREVIOUS : 0;
    st = topkv_unpack_layer(l, d_dst, &lo, &bd, d_wire, wire_bytes, (topkv_stream_t)stream);
  }
  if (st != TOPKV_OK) { printf("library status %d (%s)\n", st, topkv_strerror(st)); return 4; }
  CK(cudaStreamSynchronize(stream));
  if (topkv_device_error_flags() != 0) { printf("device error flags\n"); return 5; }
  CK(cudaMemcpy(h_wire_got, d_wire, wire_bytes, cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(h_dst_got, d_dst, pool_bytes, cudaMemcpyDeviceToHost));

  oracle_geom g;
  memset(&g, 0, sizeof g);
  g.L = L; g.F = F; g.h_kv = H; g.d_h = D; g.b_p = E; g.P = P;
  g.S_head = (int64_t)D * E; g.S_tok = (int64_t)H * D * E; g.S_kv = (int64_t)P * g.S_tok;
  g.S_page = (int64_t)F * g.S_kv; g.S_layer = pages * g.S_page;
  g.W_layer = n_layer; g.wire_order = ORACLE_WIRE_TOKEN_KV;
  for (int l = 0; l < L; ++l) {
    oracle_pack_ref(&g, l, h_src, R, MAXP, &bt_s[0][0], sl, h_wire);
    oracle_unpack_ref(&g, l, h_dst, R, MAXP, &bt_d[0][0], sl, h_wire);
  }
  const int wire_ok = memcmp(h_wire, h_wire_got, wire_bytes) == 0;
  const int dst_ok = memcmp(h_dst, h_dst_got, pool_bytes) == 0;
  printf("T=%lld n_layer=%lld launches=%lld wire %s, destination pool %s\n", (long long)T, (long long)n_layer,
         (long long)topkv_kernel_launch_count(), wire_ok ? "identical" : "DIFFERS", dst_ok ? "identical" : "DIFFERS");
  return (wire_ok && dst_ok) ? 0 : 1;
}
