/* Runs the CPU oracle on small problems under AddressSanitizer / UBSan (built and started by
 * tests/test_oracle_sanitizers.py). Exits 0 when nothing is reported and the results agree
 * with a byte-wise recomputation made here. */
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "topkv_oracle.h"

static unsigned lcg(unsigned* s) { return *s = *s * 1664525u + 1013904223u; }

int main(void) {
  unsigned seed = 12345;
  for (int trial = 0; trial < 40; ++trial) {
    oracle_geom g;
    memset(&g, 0, sizeof g);
    g.L = 2; g.F = 1 + trial % 2; g.h_kv = 1 + lcg(&seed) % 3; g.d_h = 8 * (1 + lcg(&seed) % 3);
    g.b_p = 2; g.P = 1 + lcg(&seed) % 5; g.wire_order = trial % 3 == 0; g.window = trial % 4 == 1 ? 3 : 0;
    int64_t R = 1 + lcg(&seed) % 4, maxp = 4;
    int32_t sl[4], bt[16];
    int64_t npages = 0, T = 0;
    for (int64_t r = 0; r < R; ++r) {
      sl[r] = (int32_t)(lcg(&seed) % (unsigned)(maxp * g.P + 1));
      int64_t keep = g.window > 0 && sl[r] > g.window ? g.window : sl[r];
      T += keep;
      for (int64_t j = 0; j < maxp; ++j) bt[r * maxp + j] = (int32_t)npages++;
    }
    g.S_head = g.d_h * g.b_p; g.S_tok = g.h_kv * g.S_head; g.S_kv = g.P * g.S_tok;
    g.S_page = g.F * g.S_kv; g.S_layer = npages * g.S_page;
    int64_t row = g.h_kv * g.d_h * g.b_p, n_layer = T * g.F * row;
    g.W_layer = n_layer;
    uint8_t* pool = malloc((size_t)(g.L * g.S_layer));
    uint8_t* back = malloc((size_t)(g.L * g.S_layer));
    uint8_t* wire_a = calloc((size_t)(g.L * n_layer + 1), 1);
    uint8_t* wire_b = calloc((size_t)(g.L * n_layer + 1), 1);
    for (int64_t k = 0; k < g.L * g.S_layer; ++k) pool[k] = (uint8_t)(lcg(&seed) >> 24);
    memset(back, 0x5A, (size_t)(g.L * g.S_layer));
    for (int64_t l = 0; l < g.L; ++l) {
      oracle_pack_ref(&g, l, pool, R, maxp, bt, sl, wire_a);
      oracle_pack_rows(&g, l, pool, R, maxp, bt, sl, wire_b, 3);
      oracle_unpack_ref(&g, l, back, R, maxp, bt, sl, wire_a);
    }
    if (memcmp(wire_a, wire_b, (size_t)(g.L * n_layer)) != 0) { puts("ref and rows differ"); return 1; }
    /* unpacking through the same table restores exactly the kept rows */
    for (int64_t l = 0; l < g.L; ++l) {
      oracle_pack_rows(&g, l, back, R, maxp, bt, sl, wire_b, 2);
    }
    if (memcmp(wire_a, wire_b, (size_t)(g.L * n_layer)) != 0) { puts("round trip differs"); return 1; }
    for (int64_t r = 0; r < R; ++r)
      for (int64_t c = 0; c < g.F; ++c)
        if (oracle_kv_plane_crc(&g, pool, R, maxp, bt, sl, r, c) !=
            oracle_kv_plane_crc(&g, back, R, maxp, bt, sl, r, c)) { puts("crc differs"); return 1; }
    /* the same batch as a model whose layers differ in kind: windowed, state, full, state */
    {
      int64_t kind[4] = {1, 2, 0, 2}, param[4] = {2, 48, 0, 16}, off[5];
      int64_t S_slot = 64, S_state_layer = (R + 1) * S_slot + 16;
      int32_t slot[4];
      for (int64_t r = 0; r < R; ++r) slot[r] = (int32_t)(R - r); /* slots 1..R of R + 1 */
      oracle_geom gm = g;
      gm.window = 0;
      oracle_layered_offsets(&gm, 4, kind, param, R, sl, off);
      uint8_t* sp = malloc((size_t)(2 * S_state_layer));
      uint8_t* sp_back = malloc((size_t)(2 * S_state_layer));
      for (int64_t k = 0; k < 2 * S_state_layer; ++k) sp[k] = (uint8_t)(lcg(&seed) >> 24);
      memset(sp_back, 0x33, (size_t)(2 * S_state_layer));
      uint8_t* lw = calloc((size_t)(off[4] + 1), 1);
      uint8_t* lw2 = calloc((size_t)(off[4] + 1), 1);
      memset(back, 0x5A, (size_t)(g.L * g.S_layer));
      oracle_pack_layered(&gm, 4, kind, param, pool, R, maxp, bt, sl, sp, S_state_layer, S_slot, slot, lw);
      oracle_unpack_layered(&gm, 4, kind, param, back, R, maxp, bt, sl, sp_back, S_state_layer, S_slot, slot, lw);
      oracle_pack_layered(&gm, 4, kind, param, back, R, maxp, bt, sl, sp_back, S_state_layer, S_slot, slot, lw2);
      if (memcmp(lw, lw2, (size_t)off[4]) != 0) { puts("layered round trip differs"); return 1; }
      free(sp); free(sp_back); free(lw); free(lw2);
    }
    free(pool); free(back); free(wire_a); free(wire_b);
  }
  if (oracle_select_transport(0, "a", 1, "1.1.1.1", "a", 1, "1.1.1.1", 0) != ORACLE_MODE_NVLINK ||
      oracle_select_transport(0, "a", 1, "1.1.1.1", "b", 1, "1.1.1.2", 0) != ORACLE_MODE_TCP ||
      oracle_planning_rate(ORACLE_MODE_PCIE) != 50e9) { puts("selector"); return 1; }
  if (oracle_crc64_iso((const uint8_t*)"123456789", 9) != 0xB90956C775A41001ull) { puts("check value"); return 1; }
  puts("sanitized oracle ok");
  return 0;
}
