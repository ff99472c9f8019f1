/* Drives the CUDA-free part of the library (size bookkeeping, validator, header, host CRC-64,
 * retry policy, analytic helpers) under AddressSanitizer / UndefinedBehaviorSanitizer: built by
 * tests/test_oracle_sanitizers.py from paper_2607_28633_b200/csrc/topkv_host.cpp, no GPU. */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "topkv.h"

static unsigned long long rng_state = 88172645463325252ULL;
static unsigned rnd(unsigned n) {
  rng_state ^= rng_state << 13;
  rng_state ^= rng_state >> 7;
  rng_state ^= rng_state << 17;
  return (unsigned)(rng_state % n);
}

static int attempts_left;
static int attempt(void* ctx) {
  (void)ctx;
  return --attempts_left > 0 ? TOPKV_ERR_CHECKSUM : TOPKV_OK;
}

int main(void) {
  for (int it = 0; it < 200; ++it) {
    topkv_layout lo;
    memset(&lo, 0, sizeof lo);
    lo.struct_size = (uint32_t)sizeof lo;
    lo.kv_factor = 1 + rnd(2);
    lo.kind = TOPKV_KIND_GQA;
    lo.num_layers = 1 + rnd(6);
    lo.num_kv_heads = 1 + rnd(8);
    lo.head_dim = 8 * (1 + rnd(16));
    lo.elem_bytes = 2;
    lo.page_tokens = 1 + rnd(32);
    lo.wire_order = rnd(2) ? TOPKV_WIRE_PLANAR : TOPKV_WIRE_TOKEN_KV;
    lo.num_pool_pages = 4 + rnd(60);
    if (topkv_layout_default_strides(&lo) != TOPKV_OK) return 1;
    const int R = (int)rnd(6), maxp = 1 + (int)rnd(5);
    int32_t* bt = (int32_t*)malloc(sizeof(int32_t) * (size_t)(R * maxp + 1));
    int32_t* sl = (int32_t*)malloc(sizeof(int32_t) * (size_t)(R + 1));
    int64_t used = 0;
    for (int r = 0; r < R; ++r) {
      sl[r] = (int32_t)rnd((unsigned)(maxp * (int)lo.page_tokens + 1));
      for (int j = 0; j < maxp; ++j) {
        const int needed = j * (int)lo.page_tokens < sl[r];
        bt[r * maxp + j] = needed ? (int32_t)(used++ % lo.num_pool_pages) : -1;
      }
    }
    /* any verdict is fine here (pages may repeat once the pool is exhausted): the point is that
     * the validator reads nothing outside the two tables */
    (void)topkv_validate_batch_host(&lo, R, maxp, bt, sl, 1);
    (void)topkv_validate_batch_host(&lo, R, maxp, bt, sl, 0);
    if (R > 0 && maxp > 0) {
      bt[0] = (int32_t)lo.num_pool_pages + 3; /* out of range: must be reported, not followed */
      if (sl[0] > 0 && topkv_validate_batch_host(&lo, R, maxp, bt, sl, 0) == TOPKV_OK) return 2;
    }
    const int64_t T = 1 + rnd(5000);
    if (topkv_wire_layer_bytes(&lo, T) != T * lo.kv_factor * lo.num_kv_heads * lo.head_dim * lo.elem_bytes)
      return 3;
    if (topkv_kv_bytes(&lo, T) != topkv_wire_layer_bytes(&lo, T) * lo.num_layers) return 4;
    topkv_layer_spec specs[8];
    for (unsigned l = 0; l < lo.num_layers; ++l) {
      specs[l].kind = l % 2;
      specs[l].reserved = 0;
      specs[l].param = l % 2 ? 1 + rnd(64) : 0;
    }
    if (topkv_kv_bytes_layered(&lo, specs, T) > topkv_kv_bytes(&lo, T)) return 5;
    /* header round trip and a corrupted header */
    unsigned char data[300];
    for (unsigned i = 0; i < sizeof data; ++i) data[i] = (unsigned char)rnd(256);
    const uint64_t ck = topkv_crc64(data, (int64_t)rnd(300)), cv = topkv_crc64(data + 1, 17);
    topkv_wire_header h;
    if (topkv_header_fill(&h, 7 + it, 99, &lo, T, ck, cv) != TOPKV_OK) return 6;
    if (topkv_header_check(&h, &lo, T, ck, lo.kv_factor == 2 ? cv : 0) != TOPKV_OK) return 7;
    if (topkv_header_check(&h, &lo, T, ck ^ 1, lo.kv_factor == 2 ? cv : 0) != TOPKV_ERR_CHECKSUM) return 8;
    free(bt);
    free(sl);
  }
  if (topkv_crc64("123456789", 9) != 0xB90956C775A41001ULL) return 9; /* catalogue check value */
  attempts_left = 3;
  if (topkv_retry(attempt, NULL, 2, 1) != TOPKV_OK) return 10;
  attempts_left = 10;
  if (topkv_retry(attempt, NULL, 2, 1) != TOPKV_ERR_CHECKSUM) return 11;
  if (topkv_model_hidden_fraction(80, 0.5e-3, 52e-3) < 0.75) return 12;
  {
    topkv_endpoint a, b;
    memset(&a, 0, sizeof a);
    memset(&b, 0, sizeof b);
    a.struct_size = b.struct_size = (uint32_t)sizeof(topkv_endpoint);
    a.has_nvlink = b.has_nvlink = 1;
    a.nvlink_domain = "node-a"; a.node_ip = "10.0.0.1";
    b.nvlink_domain = "node-a"; b.node_ip = "10.0.0.1";
    if (topkv_select_transport(&a, &b, 0, 0) != TOPKV_TRANSPORT_NVLINK) return 14;
    b.nvlink_domain = "node-b"; b.node_ip = "10.0.0.2";
    if (topkv_select_transport(&a, &b, 1, 0) != TOPKV_TRANSPORT_RDMA) return 15;
    if (topkv_select_transport(&a, &b, 0, 0) != TOPKV_TRANSPORT_TCP) return 16;
    if (topkv_select_transport(&a, &b, 0, TOPKV_TRANSPORT_PCIE) != TOPKV_TRANSPORT_PCIE) return 17;
    if (topkv_planning_rate(TOPKV_TRANSPORT_NVLINK) != 450e9 || topkv_planning_rate(9) != 0.0) return 18;
    if (strcmp(topkv_transport_name(TOPKV_TRANSPORT_TCP), "tcp") != 0) return 19;
  }
  for (int s = -12; s <= 1; ++s)
    if (topkv_strerror(s) == NULL) return 13;
  printf("sanitized host shims ok\n");
  return 0;
}
