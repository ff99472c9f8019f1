/*
 * CPU oracle for the paged-KV pack / unpack path. TEST INFRASTRUCTURE ONLY: it is
 * called by the tests, by the smoke check and by the benchmark's CPU-baseline leg,
 * never by the product library, with which it shares no code and no header.
 *
 * Everything here is the plain definition written out (the result of pack/unpack is
 * exactly defined, bit for bit), in the paper's notation:
 *   L layers, h_kv KV heads, d_h head dim, b_p bytes per element (Eq. 1),
 *   F = 2 for separate K and V tensors, 1 for a single MLA latent (§5.3).
 * Serialised layout: per layer, rows of [kv_heads][head_dim] elements, contiguous (§3.4).
 */
#ifndef TOPKV_ORACLE_H_
#define TOPKV_ORACLE_H_
#include <stdint.h>

enum { ORACLE_WIRE_TOKEN_KV = 0, ORACLE_WIRE_PLANAR = 1 };

typedef struct oracle_geom {
  int64_t L, F, h_kv, d_h, b_p; /* Eq. 1 symbols (+ F)                            */
  int64_t P;                    /* tokens per page                                */
  int64_t S_layer, S_page, S_kv, S_tok, S_head; /* pool strides, bytes            */
  int64_t W_layer;              /* bytes between wire slabs of consecutive layers */
  int64_t wire_order;           /* ORACLE_WIRE_*                                  */
  int64_t W_plane;              /* PLANAR only: bytes between the K and the V     */
                                /* plane of a slab; 0 = they are adjacent (T rows) */
  int64_t window;               /* 0: all tokens; W > 0: a windowed layer keeps   */
                                /* (and sends) only the last min(s, W) tokens     */
} oracle_geom;

/* Eq. 1 (F = 2) and its MLA form (F = 1, §5.3): F * L * h_kv * d_h * s * b_p. */
int64_t oracle_kv_bytes(int64_t F, int64_t L, int64_t h_kv, int64_t d_h, int64_t s, int64_t b_p);

/* Eq. 1 extended per layer kind (§2.2): a full layer counts s tokens, a windowed layer
 * min(s, window) tokens, a constant-state layer a fixed number of bytes. kind[l] is
 * 0 = full, 1 = windowed (param = window in tokens), 2 = constant state (param = bytes). */
int64_t oracle_kv_bytes_layered(int64_t F, int64_t h_kv, int64_t d_h, int64_t s, int64_t b_p,
                                int64_t L, const int64_t* kind, const int64_t* param);

/* Eq. 2. */
double oracle_transfer_s(double S_bytes, double B_bytes_per_s, double L_m_s);
/* Eq. 3. */
double oracle_t_eff(double T_last, double T_xfer, double T_rem);
/* §5.2 worked example: share of T_xfer covered by the (L-1) layers still computing. */
double oracle_hidden_fraction(int64_t L, double t_layer, double T_xfer);

/* Byte-by-byte definition, one thread. `pool` is the base of layer 0, `wire` the base of
 * the wire slab of layer 0; bt is int32 [R][maxp] (host), sl is int32 [R] (host). */
void oracle_pack_ref(const oracle_geom* g, int64_t layer, const uint8_t* pool, int64_t R,
                     int64_t maxp, const int32_t* bt, const int32_t* sl, uint8_t* wire);
void oracle_unpack_ref(const oracle_geom* g, int64_t layer, uint8_t* pool, int64_t R,
                       int64_t maxp, const int32_t* bt, const int32_t* sl, const uint8_t* wire);

/* Same definition, one memcpy per (request, token, plane, head) row of d_h*b_p bytes,
 * requests split over `threads` POSIX threads. */
void oracle_pack_rows(const oracle_geom* g, int64_t layer, const uint8_t* pool, int64_t R,
                      int64_t maxp, const int32_t* bt, const int32_t* sl, uint8_t* wire,
                      int threads);
void oracle_unpack_rows(const oracle_geom* g, int64_t layer, uint8_t* pool, int64_t R,
                        int64_t maxp, const int32_t* bt, const int32_t* sl, const uint8_t* wire,
                        int threads);

/* ---- a model whose layers differ in kind, on the data path (§2.2) ---------------------------
 * kind[l] / param[l] as for oracle_kv_bytes_layered. Attention layers (full, windowed) live in
 * the paged pool and are numbered among themselves in model order: the a-th attention layer is
 * layer a of the pool (g->L of them). Constant-state layers keep one fixed-size state per
 * request in a pool of slots and are numbered among themselves too: byte b of the state of
 * request r in the j-th state layer is state_pool[j*S_state_layer + slot[r]*S_slot + b].
 * The wire holds the layers' slabs back to back in model order (the order in which the
 * pipelined transfer sends them, §5.2): an attention layer's slab is the pack of the tokens it
 * keeps (all, or the last min(s, window)), a state layer's slab the R states in request order.
 * offsets[l] is where slab l starts, offsets[n_layers] the total: the sum over the requests of
 * Eq. 1 per layer kind. g->window, g->W_layer and g->W_plane are not used. */
void oracle_layered_offsets(const oracle_geom* g, int64_t n_layers, const int64_t* kind,
                            const int64_t* param, int64_t R, const int32_t* sl, int64_t* offsets);
void oracle_pack_layered(const oracle_geom* g, int64_t n_layers, const int64_t* kind,
                         const int64_t* param, const uint8_t* pool, int64_t R, int64_t maxp,
                         const int32_t* bt, const int32_t* sl, const uint8_t* state_pool,
                         int64_t S_state_layer, int64_t S_slot, const int32_t* slot, uint8_t* wire);
void oracle_unpack_layered(const oracle_geom* g, int64_t n_layers, const int64_t* kind,
                           const int64_t* param, uint8_t* pool, int64_t R, int64_t maxp,
                           const int32_t* bt, const int32_t* sl, uint8_t* state_pool,
                           int64_t S_state_layer, int64_t S_slot, const int32_t* slot,
                           const uint8_t* wire);

/* ---- transport selection (Alg. 1) and the planning rates of §3.3 -------------------------
 * Modes in the order Alg. 1 tries them. override_mode 0 = no manual override configured.
 * HasNVLink(s, t): both instances report NVLink and are registered in the same NVLink domain
 * (the paper compares node names: an 8-GPU domain is a node); IsSameNode(s, t): equal node IP
 * addresses; HasRDMA(): a cluster-level flag. */
enum { ORACLE_MODE_NVLINK = 1, ORACLE_MODE_PCIE = 2, ORACLE_MODE_RDMA = 3, ORACLE_MODE_TCP = 4 };
int oracle_select_transport(int override_mode, const char* s_domain, int s_has_nvlink,
                            const char* s_ip, const char* t_domain, int t_has_nvlink,
                            const char* t_ip, int cluster_has_rdma);
/* Achievable rate the orchestrator plans with, bytes per second (§3.3); 0 for an unknown mode. */
double oracle_planning_rate(int mode);

/* ---- integrity check of the serialised tensors (§3.4) -----------------------------------
 * The paper's header carries "CRC-64 checksums for both key and value tensors" and does not
 * name the polynomial. Reading taken: the reflected CRC-64 with all-ones initial value and
 * final inversion, on the ISO 3309 polynomial x^64 + x^4 + x^3 + x + 1 (catalogue name
 * CRC-64/GO-ISO). oracle_crc64 is the textbook bit-by-bit shift register for any reflected
 * polynomial, so that the same routine can be checked against a library on the ECMA-182
 * polynomial; oracle_crc64_iso fixes the ISO one. */
uint64_t oracle_crc64(const uint8_t* data, int64_t n, uint64_t poly_reflected);
uint64_t oracle_crc64_iso(const uint8_t* data, int64_t n);

/* CRC of plane c (0 = K, 1 = V) of request r, over the tensor in the paper's order
 * [layers][seq_len][kv_heads][head_dim] (§3.4), read from the paged pool through the block
 * table. A windowed geometry contributes only the tokens it keeps. */
uint64_t oracle_kv_plane_crc(const oracle_geom* g, const uint8_t* pool, int64_t R, int64_t maxp,
                             const int32_t* bt, const int32_t* sl, int64_t r, int64_t c);
/* The same for a model whose layers differ in kind (§2.2): layer l keeps all tokens when
 * layer_window[l] == 0, else the last min(s, layer_window[l]); the tensor that is checksummed
 * is the concatenation, layer by layer, of what each layer keeps. g->window is not used. */
uint64_t oracle_kv_plane_crc_layered(const oracle_geom* g, const uint8_t* pool, int64_t R,
                                     int64_t maxp, const int32_t* bt, const int32_t* sl, int64_t r,
                                     int64_t c, const int64_t* layer_window);
#endif
