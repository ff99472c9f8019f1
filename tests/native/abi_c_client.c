/* A plain C99 client of the C ABI: includes the public header, links against the library and
 * calls the entry points that need no GPU. Built and run by tests/test_abi_host.py. */
#include <stdio.h>
#include <string.h>

#include "topkv.h"

static int fail(const char* what) {
  fprintf(stderr, "abi_c_client: %s\n", what);
  return 1;
}

int main(void) {
  topkv_layout lo;
  memset(&lo, 0, sizeof lo);
  lo.struct_size = (uint32_t)sizeof lo;
  lo.kind = TOPKV_KIND_GQA;
  lo.num_layers = 80; /* Llama-3-70B: Table 1 */
  lo.kv_factor = 2;
  lo.num_kv_heads = 8;
  lo.head_dim = 128;
  lo.elem_bytes = 2;
  lo.page_tokens = 16;
  lo.wire_order = TOPKV_WIRE_TOKEN_KV;
  lo.num_pool_pages = 4096;
  if (topkv_layout_default_strides(&lo) != TOPKV_OK) return fail("default strides");
  if (lo.pool_page_stride != 65536) return fail("page stride");
  if (topkv_kv_bytes(&lo, 4096) != 1342177280LL) return fail("Eq. 1 for 4096 tokens");
  if (topkv_wire_layer_bytes(&lo, 4096) * 80 != 1342177280LL) return fail("slab bytes");
  if (topkv_version() < 100) return fail("version");
  if (topkv_strerror(TOPKV_ERR_CAPACITY) == NULL) return fail("strerror");
  /* Table 4: 1.3 GB over PCIe at 50 GB/s = 26 ms */
  {
    const double t = topkv_model_transfer_s(1.3e9, 50e9, 0.0);
    if (t < 0.0259 || t > 0.0261) return fail("Eq. 2");
  }
  /* argument errors are reported before anything touches a GPU */
  if (topkv_pack_layer(0, NULL, &lo, NULL, NULL, 0, NULL) != TOPKV_ERR_INVALID_ARG) return fail("null batch");
  if (topkv_set_host_leg_ctas(-1) != TOPKV_ERR_INVALID_ARG) return fail("cta bound");
  printf("abi_c_client ok\n");
  return 0;
}
