/*
 * CPU oracle (see topkv_oracle.h). TEST INFRASTRUCTURE ONLY.
 *
 * Pinned by tests/test_oracle_*.py against: the values of Table 1 and Table 4, the §5.2
 * worked example, a hand-derived miniature, an independently derived inverse index map,
 * memcpy / row-gather special cases, and round-trip and permutation invariants.
 * The layered pack / unpack (layers of different kinds, §2.2) is pinned against numpy slices of
 * the full pack and a fancy-index gather of the state slots, and its size against Eq. 1 per
 * layer kind; the transport selector against every branch of Alg. 1 and, with Eq. 2, Table 4.
 * The CRC routine is pinned against liblzma (ECMA-182 polynomial), both catalogue check values
 * and a polynomial-remainder derivation.
 * parity unpinned: WHICH CRC-64 the paper means (it names no polynomial; the ISO 3309 one is
 * this build's reading) and the header's field order and widths (the paper lists the fields
 * and the 128-byte size only). Everything else in this file is pinned.
 */
#include "topkv_oracle.h"

#include <pthread.h>
#include <stdlib.h>
#include <string.h>

int64_t oracle_kv_bytes(int64_t F, int64_t L, int64_t h_kv, int64_t d_h, int64_t s, int64_t b_p) {
  return F * L * h_kv * d_h * s * b_p; /* Eq. 1 with the leading 2 generalised to F (§5.3) */
}

int64_t oracle_kv_bytes_layered(int64_t F, int64_t h_kv, int64_t d_h, int64_t s, int64_t b_p,
                                int64_t L, const int64_t* kind, const int64_t* param) {
  int64_t total = 0;
  for (int64_t l = 0; l < L; ++l) {
    if (kind[l] == 2) {
      total += param[l]; /* fixed state, independent of s */
    } else {
      int64_t tokens = s;
      if (kind[l] == 1 && param[l] < s) tokens = param[l]; /* capped at the window */
      total += F * h_kv * d_h * tokens * b_p;
    }
  }
  return total;
}

double oracle_transfer_s(double S_bytes, double B, double L_m) { return S_bytes / B + L_m; } /* Eq. 2 */

double oracle_t_eff(double T_last, double T_xfer, double T_rem) { /* Eq. 3 */
  double d = T_xfer - T_rem;
  return T_last > d ? T_last : d;
}

double oracle_hidden_fraction(int64_t L, double t_layer, double T_xfer) {
  double T_rem = (double)(L - 1) * t_layer; /* compute left once the first layer is done */
  double f = T_rem / T_xfer;
  return f > 1.0 ? 1.0 : f;
}

/* Pool byte offset of element (l, page, c, t, h, d), byte b. */
static int64_t poff(const oracle_geom* g, int64_t l, int64_t page, int64_t c, int64_t t,
                    int64_t h, int64_t d, int64_t b) {
  return l * g->S_layer + page * g->S_page + c * g->S_kv + t * g->S_tok + h * g->S_head +
         d * g->b_p + b;
}

/* Wire byte offset of element (l, global token n = cu_r + i, c, h, d), byte b; T = total tokens. */
static int64_t woff(const oracle_geom* g, int64_t l, int64_t n, int64_t T, int64_t c, int64_t h,
                    int64_t d, int64_t b) {
  int64_t row_bytes = g->h_kv * g->d_h * g->b_p;
  /* PLANAR: plane c starts c*T rows into the slab, or c*W_plane bytes when the caller spreads
   * the planes (e.g. K of all layers, then V of all layers, as in the paper's payload, §3.4) */
  int64_t plane_rows = g->W_plane > 0 ? g->W_plane / row_bytes : T;
  int64_t row = (g->wire_order == ORACLE_WIRE_PLANAR) ? (c * plane_rows + n) : (n * g->F + c);
  return l * g->W_layer + row * row_bytes + (h * g->d_h + d) * g->b_p + b;
}

/* First token a layer keeps for a sequence of s tokens: 0, or s - window for a windowed layer. */
static int64_t first_kept(const oracle_geom* g, int64_t s) {
  return (g->window > 0 && s > g->window) ? s - g->window : 0;
}

static int64_t total_tokens(const oracle_geom* g, int64_t R, const int32_t* sl) {
  int64_t T = 0;
  for (int64_t r = 0; r < R; ++r) T += sl[r] - first_kept(g, sl[r]);
  return T;
}

void oracle_pack_ref(const oracle_geom* g, int64_t layer, const uint8_t* pool, int64_t R,
                     int64_t maxp, const int32_t* bt, const int32_t* sl, uint8_t* wire) {
  int64_t T = total_tokens(g, R, sl);
  int64_t cu = 0;
  for (int64_t r = 0; r < R; ++r) {
    int64_t i0 = first_kept(g, sl[r]);
    for (int64_t i = i0; i < sl[r]; ++i) {
      int64_t page = bt[r * maxp + i / g->P];
      int64_t t = i % g->P;
      for (int64_t c = 0; c < g->F; ++c)
        for (int64_t h = 0; h < g->h_kv; ++h)
          for (int64_t d = 0; d < g->d_h; ++d)
            for (int64_t b = 0; b < g->b_p; ++b)
              wire[woff(g, layer, cu + i - i0, T, c, h, d, b)] = pool[poff(g, layer, page, c, t, h, d, b)];
    }
    cu += sl[r] - i0;
  }
}

void oracle_unpack_ref(const oracle_geom* g, int64_t layer, uint8_t* pool, int64_t R,
                       int64_t maxp, const int32_t* bt, const int32_t* sl, const uint8_t* wire) {
  int64_t T = total_tokens(g, R, sl);
  int64_t cu = 0;
  for (int64_t r = 0; r < R; ++r) {
    int64_t i0 = first_kept(g, sl[r]);
    for (int64_t i = i0; i < sl[r]; ++i) {
      int64_t page = bt[r * maxp + i / g->P];
      int64_t t = i % g->P;
      for (int64_t c = 0; c < g->F; ++c)
        for (int64_t h = 0; h < g->h_kv; ++h)
          for (int64_t d = 0; d < g->d_h; ++d)
            for (int64_t b = 0; b < g->b_p; ++b)
              pool[poff(g, layer, page, c, t, h, d, b)] = wire[woff(g, layer, cu + i - i0, T, c, h, d, b)];
    }
    cu += sl[r] - i0;
  }
}

/* ---- row-memcpy form, threaded over requests ---------------------------------------- */

typedef struct job {
  const oracle_geom* g;
  int64_t layer, R, maxp, T;
  const int32_t *bt, *sl;
  const int64_t* cu;
  uint8_t* pool; /* written by unpack only */
  uint8_t* wire; /* written by pack only   */
  int pack;
  int64_t r_begin, r_end;
} job;

static void* run_job(void* arg) {
  job* j = (job*)arg;
  const oracle_geom* g = j->g;
  size_t head_bytes = (size_t)(g->d_h * g->b_p);
  for (int64_t r = j->r_begin; r < j->r_end; ++r) {
    int64_t i0 = first_kept(g, j->sl[r]);
    for (int64_t i = i0; i < j->sl[r]; ++i) {
      int64_t page = j->bt[r * j->maxp + i / g->P];
      int64_t t = i % g->P;
      for (int64_t c = 0; c < g->F; ++c)
        for (int64_t h = 0; h < g->h_kv; ++h) {
          uint8_t* p = j->pool + poff(g, j->layer, page, c, t, h, 0, 0);
          uint8_t* w = j->wire + woff(g, j->layer, j->cu[r] + i - i0, j->T, c, h, 0, 0);
          if (j->pack) memcpy(w, p, head_bytes);
          else memcpy(p, w, head_bytes);
        }
    }
  }
  return NULL;
}

static void run_rows(const oracle_geom* g, int64_t layer, uint8_t* pool, int64_t R, int64_t maxp,
                     const int32_t* bt, const int32_t* sl, uint8_t* wire, int threads, int pack) {
  if (threads < 1) threads = 1;
  if (threads > 256) threads = 256;
  if (R < threads) threads = R > 0 ? (int)R : 1;
  int64_t* cu = (int64_t*)malloc(sizeof(int64_t) * (size_t)(R + 1));
  cu[0] = 0;
  for (int64_t r = 0; r < R; ++r) cu[r + 1] = cu[r] + sl[r] - first_kept(g, sl[r]);
  job jobs[256];
  pthread_t tid[256];
  for (int k = 0; k < threads; ++k) {
    job* j = &jobs[k];
    j->g = g; j->layer = layer; j->R = R; j->maxp = maxp; j->T = cu[R];
    j->bt = bt; j->sl = sl; j->cu = cu; j->pool = pool; j->wire = wire; j->pack = pack;
    j->r_begin = R * k / threads;
    j->r_end = R * (k + 1) / threads;
  }
  for (int k = 1; k < threads; ++k) pthread_create(&tid[k], NULL, run_job, &jobs[k]);
  run_job(&jobs[0]);
  for (int k = 1; k < threads; ++k) pthread_join(tid[k], NULL);
  free(cu);
}

void oracle_pack_rows(const oracle_geom* g, int64_t layer, const uint8_t* pool, int64_t R,
                      int64_t maxp, const int32_t* bt, const int32_t* sl, uint8_t* wire,
                      int threads) {
  run_rows(g, layer, (uint8_t*)pool, R, maxp, bt, sl, wire, threads, 1);
}

void oracle_unpack_rows(const oracle_geom* g, int64_t layer, uint8_t* pool, int64_t R,
                        int64_t maxp, const int32_t* bt, const int32_t* sl, const uint8_t* wire,
                        int threads) {
  run_rows(g, layer, pool, R, maxp, bt, sl, (uint8_t*)wire, threads, 0);
}

/* ---- layers of different kinds on the data path (§2.2) ---------------------------------- */

static int64_t kept_by_kind(int64_t kind, int64_t param, int64_t s) {
  return (kind == 1 && param < s) ? param : s; /* a windowed layer is capped at its window */
}

void oracle_layered_offsets(const oracle_geom* g, int64_t n_layers, const int64_t* kind,
                            const int64_t* param, int64_t R, const int32_t* sl, int64_t* offsets) {
  int64_t tok_bytes = g->F * g->h_kv * g->d_h * g->b_p;
  int64_t off = 0;
  for (int64_t l = 0; l < n_layers; ++l) {
    offsets[l] = off;
    for (int64_t r = 0; r < R; ++r)
      off += (kind[l] == 2) ? param[l] : tok_bytes * kept_by_kind(kind[l], param[l], sl[r]);
  }
  offsets[n_layers] = off;
}

static void layered(const oracle_geom* g, int64_t n_layers, const int64_t* kind, const int64_t* param,
                    uint8_t* pool, int64_t R, int64_t maxp, const int32_t* bt, const int32_t* sl,
                    uint8_t* state_pool, int64_t S_state_layer, int64_t S_slot, const int32_t* slot,
                    uint8_t* wire, int pack) {
  int64_t* off = (int64_t*)malloc(sizeof(int64_t) * (size_t)(n_layers + 1));
  oracle_layered_offsets(g, n_layers, kind, param, R, sl, off);
  int64_t a = 0, j = 0; /* attention layers and state layers seen so far */
  for (int64_t l = 0; l < n_layers; ++l) {
    uint8_t* slab = wire + off[l];
    if (kind[l] == 2) {
      for (int64_t r = 0; r < R; ++r)
        for (int64_t b = 0; b < param[l]; ++b) {
          uint8_t* st = state_pool + j * S_state_layer + (int64_t)slot[r] * S_slot + b;
          if (pack) slab[r * param[l] + b] = *st;
          else *st = slab[r * param[l] + b];
        }
      ++j;
    } else {
      oracle_geom gl = *g; /* this layer's view: its window, its slab as the whole wire */
      gl.window = (kind[l] == 1) ? param[l] : 0;
      gl.W_layer = 0;
      gl.W_plane = 0;
      if (pack) oracle_pack_ref(&gl, a, pool, R, maxp, bt, sl, slab);
      else oracle_unpack_ref(&gl, a, pool, R, maxp, bt, sl, slab);
      ++a;
    }
  }
  free(off);
}

void oracle_pack_layered(const oracle_geom* g, int64_t n_layers, const int64_t* kind,
                         const int64_t* param, const uint8_t* pool, int64_t R, int64_t maxp,
                         const int32_t* bt, const int32_t* sl, const uint8_t* state_pool,
                         int64_t S_state_layer, int64_t S_slot, const int32_t* slot, uint8_t* wire) {
  layered(g, n_layers, kind, param, (uint8_t*)pool, R, maxp, bt, sl, (uint8_t*)state_pool, S_state_layer,
          S_slot, slot, wire, 1);
}

void oracle_unpack_layered(const oracle_geom* g, int64_t n_layers, const int64_t* kind,
                           const int64_t* param, uint8_t* pool, int64_t R, int64_t maxp,
                           const int32_t* bt, const int32_t* sl, uint8_t* state_pool,
                           int64_t S_state_layer, int64_t S_slot, const int32_t* slot,
                           const uint8_t* wire) {
  layered(g, n_layers, kind, param, pool, R, maxp, bt, sl, state_pool, S_state_layer, S_slot, slot,
          (uint8_t*)wire, 0);
}

/* ---- transport selection (Alg. 1), planning rates (§3.3) ---------------------------------- */

int oracle_select_transport(int override_mode, const char* s_domain, int s_has_nvlink,
                            const char* s_ip, const char* t_domain, int t_has_nvlink,
                            const char* t_ip, int cluster_has_rdma) {
  if (override_mode != 0) return override_mode;                 /* manual override configured   */
  int has_nvlink = s_has_nvlink && t_has_nvlink && strcmp(s_domain, t_domain) == 0;
  if (has_nvlink) return ORACLE_MODE_NVLINK;                    /* same NVLink domain           */
  if (strcmp(s_ip, t_ip) == 0) return ORACLE_MODE_PCIE;         /* same node, cross-domain      */
  if (cluster_has_rdma) return ORACLE_MODE_RDMA;                /* cross-node, RDMA available   */
  return ORACLE_MODE_TCP;                                       /* fallback                     */
}

double oracle_planning_rate(int mode) {
  switch (mode) {
    case ORACLE_MODE_NVLINK: return 450e9; /* NVLink 4.0, 18 links, unidirectional       */
    case ORACLE_MODE_PCIE: return 50e9;    /* Gen5 x16 practical throughput              */
    case ORACLE_MODE_RDMA: return 25e9;    /* 400 Gbps InfiniBand NDR less protocol cost */
    case ORACLE_MODE_TCP: return 10e9;     /* 100 Gbps Ethernet with gRPC framing        */
    default: return 0.0;
  }
}

/* ---- CRC-64 (§3.4) -------------------------------------------------------------------- */

/* One step of the reflected shift register: feed the byte, then shift eight times. */
static uint64_t crc64_byte(uint64_t crc, uint8_t b, uint64_t poly_reflected) {
  crc ^= b;
  for (int k = 0; k < 8; ++k) crc = (crc & 1) ? (crc >> 1) ^ poly_reflected : (crc >> 1);
  return crc;
}

uint64_t oracle_crc64(const uint8_t* data, int64_t n, uint64_t poly_reflected) {
  uint64_t crc = ~(uint64_t)0; /* initial value: all ones */
  for (int64_t i = 0; i < n; ++i) crc = crc64_byte(crc, data[i], poly_reflected);
  return ~crc; /* final inversion */
}

#define ORACLE_POLY_ISO_REFLECTED 0xD800000000000000ull /* x^64 + x^4 + x^3 + x + 1 */

uint64_t oracle_crc64_iso(const uint8_t* data, int64_t n) {
  return oracle_crc64(data, n, ORACLE_POLY_ISO_REFLECTED);
}

uint64_t oracle_kv_plane_crc(const oracle_geom* g, const uint8_t* pool, int64_t R, int64_t maxp,
                             const int32_t* bt, const int32_t* sl, int64_t r, int64_t c) {
  (void)R;
  uint64_t crc = ~(uint64_t)0;
  for (int64_t l = 0; l < g->L; ++l)
    for (int64_t i = first_kept(g, sl[r]); i < sl[r]; ++i) {
      int64_t page = bt[r * maxp + i / g->P];
      int64_t t = i % g->P;
      for (int64_t h = 0; h < g->h_kv; ++h)
        for (int64_t d = 0; d < g->d_h; ++d)
          for (int64_t b = 0; b < g->b_p; ++b)
            crc = crc64_byte(crc, pool[poff(g, l, page, c, t, h, d, b)], ORACLE_POLY_ISO_REFLECTED);
    }
  return ~crc;
}

uint64_t oracle_kv_plane_crc_layered(const oracle_geom* g, const uint8_t* pool, int64_t R,
                                     int64_t maxp, const int32_t* bt, const int32_t* sl, int64_t r,
                                     int64_t c, const int64_t* layer_window) {
  (void)R;
  uint64_t crc = ~(uint64_t)0;
  for (int64_t l = 0; l < g->L; ++l) {
    int64_t W = layer_window[l];
    int64_t i0 = (W > 0 && sl[r] > W) ? sl[r] - W : 0; /* a windowed layer keeps the last W */
    for (int64_t i = i0; i < sl[r]; ++i) {
      int64_t page = bt[r * maxp + i / g->P];
      int64_t t = i % g->P;
      for (int64_t h = 0; h < g->h_kv; ++h)
        for (int64_t d = 0; d < g->d_h; ++d)
          for (int64_t b = 0; b < g->b_p; ++b)
            crc = crc64_byte(crc, pool[poff(g, l, page, c, t, h, d, b)], ORACLE_POLY_ISO_REFLECTED);
    }
  }
  return ~crc;
}
