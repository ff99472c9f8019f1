/*
 * topkv.h — C ABI of the TopKV data plane for one B200 (sm_100a).
 *
 * The library moves ONE LAYER of a batch's paged KV cache between a paged block
 * pool and a contiguous "wire" buffer, the unit that the paper's pipelined
 * layer-by-layer transfer sends while later layers still compute (§5.2), in the
 * contiguous serialised layout that lets a link move it as one DMA (§3.4).
 *
 *   pack    : paged pool  -> contiguous wire      (prefill side)
 *   unpack  : contiguous wire -> paged pool       (decode side, own block table)
 *   *_host  : the same with the wire in pinned host memory (the PCIe leg, §3.3)
 *
 * Elements are opaque `elem_bytes`-wide words (FP16 in the paper, §2.2; bf16 in
 * the benchmark shapes): bytes are moved, never interpreted, so every result is
 * bit-exact by construction.
 *
 * Notation (follows the paper's Eq. 1 where it has a symbol):
 *   L layers, h_kv = num_kv_heads (H), d_h = head_dim (D), b_p = elem_bytes (E),
 *   F = kv_factor (2: separate K and V planes; 1: a single MLA latent row, §5.3),
 *   P = page_tokens, R = requests, s_r = seq_lens[r], cu_r = sum_{q<r} s_q,
 *   T = cu_R, row_bytes = H*D*E, N_layer = T*F*row_bytes.
 *
 * Pool addressing (bytes):
 *   poff(l,p,c,t,h,d) = l*pool_layer_stride + p*pool_page_stride + c*pool_kv_stride
 *                     + t*pool_token_stride + h*pool_head_stride + d*E
 * Wire addressing (bytes), per layer slab:
 *   TOKEN_KV : woff(r,i,c,h,d) = ((cu_r + i)*F + c)*row_bytes + (h*D + d)*E
 *   PLANAR   : woff(r,i,c,h,d) = (c*T + cu_r + i)*row_bytes   + (h*D + d)*E
 * TOKEN_KV is the batched order [request][token][K|V][head][dim]; PLANAR is the
 * paper's "K tensor then V tensor, each [seq_len][kv_heads][head_dim]" (§3.4).
 * The wire slab of layer l starts at wire + l*wire_layer_stride.
 *
 * pack   : for r<R, i<s_r, c<F, h<H, d<D : wire[woff(r,i,c,h,d)] = pool[poff(l, bt[r][i/P], c, i%P, h, d)]
 * unpack : for the same index set        : pool[poff(l, bt[r][i/P], c, i%P, h, d)] = wire[woff(r,i,c,h,d)]
 *          and every other pool byte keeps its value.
 *
 * Ownership: the caller owns every buffer. The entry points below allocate
 * nothing, free nothing and only enqueue work on `stream`; results are valid
 * once the caller has synchronised with the stream. All `const void*`/`void*`
 * arguments are DEVICE pointers unless their name starts with `h_`.
 *
 * Stream capture: topkv_pack_layer, topkv_unpack_layer, the two host-leg calls,
 * topkv_repage_layer, topkv_build_plan and the checksummed copies only enqueue kernels and
 * copies, so they may be issued while `stream` is being captured into a CUDA graph (the
 * descriptors are read at call time; the buffers they point to at replay time). The first
 * checksummed copy on a device (and the first call of kernel family 1) also raises that
 * kernel's shared-memory limit, once per device: make that first call outside a capture.
 *
 * Errors: every int-returning function returns TOPKV_OK (0) or a negative
 * topkv_status. Every argument is checked before anything is enqueued, so when an error is
 * returned nothing has been launched. The one exception is TOPKV_ERR_CUDA reported by the CUDA
 * runtime itself in the middle of a call that enqueues more than one operation (the staged
 * host-leg calls: a kernel and a copy; the pipelined calls: one of each per layer): what was
 * enqueued before the failing operation stays enqueued.
 */
#ifndef TOPKV_H_
#define TOPKV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* A CUDA stream handle (cudaStream_t). Declared opaquely so that this header
 * compiles without the CUDA toolkit. */
typedef struct CUstream_st* topkv_stream_t;
typedef struct CUevent_st* topkv_event_t;   /* opaque cudaEvent_t */

typedef enum topkv_status {
  TOPKV_OK = 0,
  TOPKV_ERR_INVALID_ARG = -1,        /* NULL pointer, negative count, struct_size mismatch   */
  TOPKV_ERR_LAYER_RANGE = -2,        /* layer not in [0, num_layers)                          */
  TOPKV_ERR_ALIGNMENT = -3,          /* a base, stride or row_bytes is not a multiple of 16 B */
  TOPKV_ERR_CAPACITY = -4,           /* wire / host / staging buffer smaller than N_layer     */
  TOPKV_ERR_UNSUPPORTED_LAYOUT = -5, /* descriptor is self-inconsistent or not supported      */
  TOPKV_ERR_CUDA = -6,               /* a CUDA call failed; see topkv_last_cuda_error()       */
  TOPKV_ERR_CHECKSUM = -7            /* header magic, dimensions or a CRC-64 do not match      */
} topkv_status;

enum { TOPKV_KIND_GQA = 0, TOPKV_KIND_MLA = 1 };
enum { TOPKV_WIRE_TOKEN_KV = 0, TOPKV_WIRE_PLANAR = 1 };

/* Describes one paged pool and the wire format. All strides are in bytes; the
 * head_dim axis is always contiguous. */
typedef struct topkv_layout {
  uint32_t struct_size;     /* = sizeof(topkv_layout); guards against ABI drift          */
  uint32_t kind;            /* TOPKV_KIND_GQA or TOPKV_KIND_MLA (informational; F rules)  */
  uint32_t num_layers;      /* L                                                          */
  uint32_t kv_factor;       /* F: 2 = K and V planes, 1 = one latent row per token (§5.3) */
  uint32_t num_kv_heads;    /* H (1 for MLA)                                              */
  uint32_t head_dim;        /* D (576 = 512 + 64 for the DeepSeek-V3 latent, §5.3)        */
  uint32_t elem_bytes;      /* E = b_p of Eq. 1 (2 for FP16 / bf16)                       */
  uint32_t page_tokens;     /* P                                                          */
  uint32_t wire_order;      /* TOPKV_WIRE_TOKEN_KV or TOPKV_WIRE_PLANAR                   */
  uint32_t reserved;        /* must be 0                                                  */
  int64_t num_pool_pages;   /* pages per layer slab                                       */
  int64_t pool_layer_stride;
  int64_t pool_page_stride;
  int64_t pool_kv_stride;   /* ignored when F == 1                                        */
  int64_t pool_token_stride;
  int64_t pool_head_stride; /* ignored when H == 1                                        */
  int64_t wire_layer_stride;/* bytes between wire slabs; 0 = caller passes layer's slab   */
  int64_t wire_plane_stride;/* PLANAR only: bytes from the K plane to the V plane of a    */
                            /* slab; 0 = adjacent (T*row_bytes). With one request, a      */
                            /* layer stride of s*row_bytes and a plane stride of          */
                            /* L*s*row_bytes the layers assemble the paper's payload: the */
                            /* K tensor [layers][seq_len][heads][dim], then the V tensor  */
                            /* (§3.4). Must be a multiple of row_bytes; not accepted by   */
                            /* the staged host-leg calls (they copy one contiguous slab). */
} topkv_layout;

/* One batch of requests. block_table and seq_lens do not depend on the layer
 * (a page id addresses the same page slot in every layer slab). */
typedef struct topkv_batch {
  uint32_t struct_size;          /* = sizeof(topkv_batch)                                   */
  int32_t num_requests;          /* R >= 0                                                  */
  int32_t max_pages_per_req;     /* block-table row width (columns)                         */
  uint32_t flags;                /* 0 or TOPKV_FLAG_* bits (below)                          */
  const int32_t* block_table;    /* DEVICE int32 [R][max_pages_per_req]; columns at or past */
                                 /* ceil(s_r/P) are ignored (conventionally -1)             */
  const int32_t* seq_lens;       /* DEVICE int32 [R], each in [0, max_pages_per_req*P]      */
  const int64_t* cu_seq_lens;    /* DEVICE int64 [R+1] from topkv_build_plan, or NULL: then */
                                 /* each CTA derives it (allowed for R <= TOPKV_MAX_INLINE_R)*/
  int64_t total_tokens;          /* T if the host knows it, else -1. When -1 the capacity   */
                                 /* checks are skipped and the caller guarantees them. A    */
                                 /* stated total must equal the sum of seq_lens: it bounds  */
                                 /* the slab and, for a ragged batch, the number of CTAs    */
                                 /* (T / span + R instead of one per block-table column); a */
                                 /* total below the device lengths raises error bit 4.      */
  int32_t window_tokens;         /* 0 = every token. W > 0 = a windowed layer (§2.2): only  */
                                 /* the last min(s_r, W) tokens of each request are kept,   */
                                 /* so only they are packed / unpacked; T, cu_seq_lens and  */
                                 /* N_layer then count min(s_r, W) per request, and table   */
                                 /* columns before the window are ignored.                  */
  int32_t reserved;              /* must be 0                                               */
} topkv_batch;

/* topkv_batch.flags. Every copy kernel is launched so that it may become resident while the
 * previous kernel of the stream drains, but by default it touches memory only after that
 * kernel has finished. With TOPKV_FLAG_OVERLAP_PREVIOUS the caller declares that this call
 * reads nothing and overwrites nothing that the kernels enqueued before it on `stream` write
 * or read, back to the most recent call made WITHOUT the flag (or the most recent non-kernel
 * operation, e.g. a copy or an event wait, which is always honoured). The call's kernel may
 * then move data while those kernels finish their tails, e.g. pack of layer l+1 behind pack
 * of layer l. Completion stays in stream order: whatever is enqueued after the call starts
 * only after all of them are done. */
#define TOPKV_FLAG_OVERLAP_PREVIOUS 1u
/* TOPKV_FLAG_TABLES_SETTLED: the caller declares that block_table, seq_lens and cu_seq_lens
 * were NOT written by the kernels enqueued just before this call on `stream` (they were
 * uploaded or built earlier and something has been waited for since: a copy, an event, a
 * synchronisation). The kernel then reads its tables and works out its addresses while the
 * previous kernel still drains and waits for that kernel only before it touches the pool or
 * the wire, so the data it depends on may still come from that kernel (unpack of layer l right
 * behind pack of layer l). Honoured by topkv_pack_layer(s) / topkv_unpack_layer(s) and the
 * host-leg calls in the vectorised kernel family; ignored elsewhere. */
#define TOPKV_FLAG_TABLES_SETTLED 2u

/* Largest R for which cu_seq_lens may be NULL. */
#define TOPKV_MAX_INLINE_R 1024

/* ---- the four hot-path calls (§3.4 layout, issued per layer as in §5.2) -------------- */

/* Gathers layer `layer` of the batch from the paged pool `src_pool` (base of layer 0) into
 * the wire slab at d_wire + layer*wire_layer_stride. wire_capacity_bytes is the size of the
 * whole buffer behind d_wire. Enqueues one kernel on `stream`. */
int topkv_pack_layer(int layer, const void* src_pool, const topkv_layout* layout,
                     const topkv_batch* batch, void* d_wire, int64_t wire_capacity_bytes,
                     topkv_stream_t stream);

/* Inverse of topkv_pack_layer: scatters the wire slab into `dst_pool` through the batch's
 * (destination) block table. Pool bytes that no valid token addresses are not written.
 * Precondition (unchecked on the device): no two requests share a destination page. */
int topkv_unpack_layer(int layer, void* dst_pool, const topkv_layout* layout,
                       const topkv_batch* batch, const void* d_wire, int64_t wire_bytes,
                       topkv_stream_t stream);

/* pack with the wire slab landing in caller-owned PINNED host memory `h_pinned`
 * (slab of layer l at h_pinned + l*wire_layer_stride), the PCIe leg of §3.3.
 *   d_staging != NULL : kernel packs into d_staging (>= N_layer bytes, device), then one
 *                       cudaMemcpyAsync device->host on the same stream (copy engine).
 *   d_staging == NULL : the kernel stores straight into the mapped pinned buffer; h_pinned
 *                       must be device-accessible at the same address (cudaHostAlloc under
 *                       unified addressing). Requires batch->total_tokens >= 0 only for the
 *                       staged form (the copy size must be known on the host).
 * Measured on a B200 (PCIe Gen5 x16, 128 MiB slabs): staged 0.98 of a pinned cudaMemcpyAsync of
 * the same size, direct 0.92. Layers that are ready together reach 1.00 when they alternate
 * between two streams with a staging slab each (the copy engine moves layer l while the
 * kernel of layer l+1 runs); calls on one stream follow each other, kernel, copy, kernel, ... */
int topkv_pack_layer_to_host(int layer, const void* src_pool, const topkv_layout* layout,
                             const topkv_batch* batch, void* h_pinned,
                             int64_t host_capacity_bytes, void* d_staging,
                             int64_t staging_capacity_bytes, topkv_stream_t stream);

/* unpack with the wire slab read from pinned host memory; same two forms as above
 * (host->device copy into d_staging then unpack, or direct mapped loads). */
int topkv_unpack_layer_from_host(int layer, void* dst_pool, const topkv_layout* layout,
                                 const topkv_batch* batch, const void* h_pinned,
                                 int64_t host_bytes, void* d_staging,
                                 int64_t staging_capacity_bytes, topkv_stream_t stream);

/* ---- span links: dependent launches that do not wait for each other as a whole (§5.2) -------
 * In a relay, the unpack of layer l reads what the pack of layer l has just written (§5.2 sends
 * a layer as soon as it exists), so that launch can never be declared independent, and as an
 * ordinary launch it waits for the LAST CTA of the pack before its first CTA may touch memory.
 * A span link orders the two kernels span by span instead: both cut the batch into the same
 * spans (one CTA each; the same lengths, page_tokens, row size and max_pages_per_req on both
 * sides, whatever the block tables), every CTA of the first kernel publishes its span's flag
 * when its stores are issued, and every CTA of the second waits for the flag of ITS span only,
 * so the second kernel runs under the first one's tail like an independent launch.
 *   d_signal : flags this call publishes (value signal_epoch), or NULL
 *   d_await  : flags this call waits for (until they hold await_epoch), or NULL
 * Both are DEVICE int32 arrays of topkv_span_link_words() entries, owned by the caller, that
 * must not already hold the epochs of the calls about to use them (zero them once and use
 * epochs 1, 2, 3, ...: an array is reused by giving every pair of calls its own epoch).
 * A linked call never waits for the previous kernel as a whole and reads its tables at once,
 * as if TOPKV_FLAG_OVERLAP_PREVIOUS were set: the caller promises that the tables were not
 * written by kernels still running and that EVERY conflict with kernels enqueued before it on
 * `stream` is covered by the link. The FIRST call of a chain usually cannot promise that (the
 * kernel before it wrote the pool, or the plan): give it TOPKV_LINK_WAIT_PREVIOUS, which makes
 * it an ordinary launch towards everything before it (it waits for the previous kernel to
 * finish before it reads anything, and only then lets the next linked kernel in, so that the
 * calls after it are ordered behind that kernel too) and a linked one towards what follows.
 * For pack(l) -> unpack(l) -> pack(l+1) -> ... through one slab:
 * pack(l+1) awaits the flags unpack(l) publishes (the slab has been read) and publishes the
 * flags unpack(l+1) awaits. Kernels still complete in stream order. Waits are bounded (about
 * half a second): a flag that never arrives raises bit 1 of topkv_device_error_flags() and skips the
 * span. Linked launches are safe because a kernel's CTAs are scheduled only after every CTA of
 * the earlier kernels of the stream has started: enqueue the linked calls on ONE stream, in
 * producer-before-consumer order, with no other work between them. The epochs are plain
 * arguments: a CUDA graph that captured linked calls replays the epochs of the capture, so such
 * a graph must clear the flag arrays (a memset node) ahead of the linked calls of every replay.
 * Vectorised kernel family, one layer per call. */
#define TOPKV_LINK_WAIT_PREVIOUS 1u /* also wait for the previous kernel of the stream as a whole */
typedef struct topkv_span_link {
  uint32_t struct_size;   /* = sizeof(topkv_span_link)               */
  uint32_t await_epoch;   /* value the awaited flags must reach      */
  uint32_t signal_epoch;  /* value written into the published flags  */
  uint32_t flags;         /* 0 or TOPKV_LINK_WAIT_PREVIOUS           */
  const int32_t* d_await; /* DEVICE int32 [words] or NULL            */
  int32_t* d_signal;      /* DEVICE int32 [words] or NULL            */
} topkv_span_link;
/* Number of flags (spans) of one layer of this batch, or a negative topkv_status. */
int64_t topkv_span_link_words(const topkv_layout* layout, const topkv_batch* batch);
int topkv_pack_layer_linked(int layer, const void* src_pool, const topkv_layout* layout,
                            const topkv_batch* batch, void* d_wire, int64_t wire_capacity_bytes,
                            const topkv_span_link* link, topkv_stream_t stream);
int topkv_unpack_layer_linked(int layer, void* dst_pool, const topkv_layout* layout,
                              const topkv_batch* batch, const void* d_wire, int64_t wire_bytes,
                              const topkv_span_link* link, topkv_stream_t stream);

/* The whole relay of a range of layers through ONE wire slab as one call: for every layer,
 * pack (source pool -> slab) and unpack (slab -> destination pool), all 2 * num_layers launches
 * span-linked: unpack(l) follows pack(l) span by span, pack(l+1) overwrites a span of the slab as
 * soon as unpack(l) has read it. This is the shape a transfer to another GPU has (pack into the
 * receiver's slab, unpack there, §5.2) run on one GPU; where both pools are on this GPU and no
 * wire is wanted, topkv_repage_layer moves half the bytes.
 * The two sides must describe the same requests and cut them into the same spans: equal
 * num_requests, max_pages_per_req, window_tokens, page_tokens, kv_factor, heads, head_dim,
 * elem_bytes and wire order (else TOPKV_ERR_UNSUPPORTED_LAYOUT); block tables, strides and pool
 * sizes may differ. wire_layer_stride of both layouts is ignored: d_slab (slab_bytes >= N_layer)
 * is the slab of every layer. d_flags: DEVICE int32 [2 * topkv_span_link_words()], zeroed once by
 * the caller; first_epoch = the number of layers already relayed through these flags since they
 * were zeroed (0 the first time; the call uses epochs first_epoch + 1 .. first_epoch +
 * num_layers). The first pack of the call waits for the kernel enqueued before the call as a
 * whole (TOPKV_LINK_WAIT_PREVIOUS), unless src_batch carries TOPKV_FLAG_OVERLAP_PREVIOUS; all
 * later launches are ordered behind it through their links. Everything is validated for every
 * layer before the first launch. */
int topkv_relay_layers_linked(int first_layer, int num_layers, const void* src_pool,
                              const topkv_layout* src_layout, const topkv_batch* src_batch,
                              void* dst_pool, const topkv_layout* dst_layout,
                              const topkv_batch* dst_batch, void* d_slab, int64_t slab_bytes,
                              int32_t* d_flags, int64_t flags_words, uint32_t first_epoch,
                              topkv_stream_t stream);

/* ---- direct re-paging (no wire slab) -------------------------------------------------------- */

/* Moves layer `layer` of the batch from one paged pool straight into another paged pool with
 * its own block table, page size and strides: the same bytes end up in `dst_pool` as after
 * topkv_pack_layer followed by topkv_unpack_layer, at half the memory traffic and with no
 * wire buffer. This is the same-GPU case of handing a cache over, e.g. when a worker changes
 * role (§3.5) and the cache must move into the other role's pool.
 * The two layouts must agree in kv_factor, num_kv_heads, head_dim and elem_bytes; everything
 * else may differ. Lengths are read from src_batch->seq_lens (dst_batch->seq_lens must hold
 * the same values); cu_seq_lens is not used; src_batch->total_tokens, when stated (>= 0), must
 * be the sum of the lengths and lets a ragged batch launch one CTA per span that can hold
 * tokens (a total below the device lengths raises error bit 4). The launch overlaps the
 * previous kernel only if BOTH batches carry TOPKV_FLAG_OVERLAP_PREVIOUS. Preconditions as for
 * unpack: no two requests share a destination page; the pools do not overlap. */
int topkv_repage_layer(int layer, const void* src_pool, const topkv_layout* src_layout,
                       const topkv_batch* src_batch, void* dst_pool,
                       const topkv_layout* dst_layout, const topkv_batch* dst_batch,
                       topkv_stream_t stream);

/* ---- integrity: wire header and CRC-64 (§3.4) ------------------------------------------------ */

/* The fixed 128-byte header of §3.4, one per request: magic, request ID, model ID, tensor
 * dimensions (sequence length, layers, KV heads, head dimension), tensor sizes, CRC-64 of the
 * key tensor and of the value tensor. The paper fixes the content and the size; field order
 * and widths below are this library's reading (the order in which the paper lists them,
 * little-endian, zero padded). For an MLA cache (kv_factor 1) v_bytes and crc_v are 0. */
typedef struct topkv_wire_header {
  char magic[8];          /* "KVCACHE1"                                                    */
  uint64_t request_id;
  uint64_t model_id;
  uint32_t seq_len, num_layers, num_kv_heads, head_dim, elem_bytes, kv_factor;
  uint64_t k_bytes, v_bytes; /* L * seq_len * H * D * E each                                */
  uint64_t crc_k, crc_v;
  uint8_t reserved[48];   /* zero                                                           */
} topkv_wire_header;

int topkv_header_fill(topkv_wire_header* header, uint64_t request_id, uint64_t model_id,
                      const topkv_layout* layout, int64_t seq_len, uint64_t crc_k, uint64_t crc_v);
/* TOPKV_OK, or TOPKV_ERR_CHECKSUM when the magic, a dimension, a size or a checksum differs
 * from what the receiver expects / has computed. */
int topkv_header_check(const topkv_wire_header* header, const topkv_layout* layout,
                       int64_t seq_len, uint64_t crc_k, uint64_t crc_v);

/* The checksum: reflected CRC-64, all-ones initial value, final inversion, ISO 3309
 * polynomial x^64 + x^4 + x^3 + x + 1 (the paper names no polynomial: this is the
 * generator of Go's crc64.ISO table, catalogue name CRC-64/GO-ISO, check value of "123456789"
 * 0xB90956C775A41001). The K (V) checksum of a request covers its K (V) tensor in the order
 * [layers][seq_len][kv_heads][head_dim]. topkv_crc64 is the plain HOST routine. */
uint64_t topkv_crc64(const void* h_data, int64_t nbytes);

/* Device-side checksumming, fused into pack / unpack. Usage, per batch:
 *   topkv_crc_begin(...)                 once: constant tables, clears the remainders (on `stream`)
 *   topkv_pack_layer_crc(l, ...)         every layer l of the layout, in any order
 *                                        (topkv_unpack_layer_crc on the receiving side); doing a
 *                                        layer again (a re-send) rewrites its remainders
 *   topkv_crc_finish(...)                d_crc_out[r*F + c] = checksum of request r, plane c;
 *                                        may be called again, changes nothing in the workspace
 * d_workspace: DEVICE scratch of at least topkv_crc_workspace_bytes(...) bytes, 16-byte
 * aligned, owned by the caller and reserved for this batch from begin to finish. It holds one
 * 8-byte remainder per 32 runs (of at most 1 KiB) of every request, plane and layer, i.e.
 * about N_layer * L / 4096 bytes (Llama-3-70B shape, 8 x 4096 tokens: 2.6 MB). d_crc_out:
 * DEVICE uint64 [R*F]. batch->cu_seq_lens and total_tokens are optional (the kernel rebuilds
 * the prefix sums from seq_lens), head-split pools are supported; num_requests at most 8192
 * (else TOPKV_ERR_UNSUPPORTED_LAYOUT). Layers may differ in kind (§2.2): a layer copied with
 * batch->window_tokens = W contributes the last min(s, W) tokens of every request to the
 * checksum, exactly the rows it ships; the workspace remembers each layer's window for
 * topkv_crc_finish, whose own batch argument only supplies the tables (its window_tokens is
 * ignored). TOPKV_FLAG_OVERLAP_PREVIOUS may be set as for the plain calls, with one rule that
 * follows from its definition: the first checksummed copy enqueued after topkv_crc_begin reads
 * and writes what begin wrote, so that copy must NOT carry the flag (begin's own batch argument
 * may carry any flags; begin ignores them and never lets a later kernel start early). The bytes
 * moved are identical to topkv_pack_layer / topkv_unpack_layer. */
int64_t topkv_crc_workspace_bytes(const topkv_layout* layout, int32_t num_requests,
                                  int32_t max_pages_per_req);
int topkv_crc_begin(const topkv_layout* layout, const topkv_batch* batch, void* d_workspace,
                    int64_t workspace_bytes, topkv_stream_t stream);
int topkv_pack_layer_crc(int layer, const void* src_pool, const topkv_layout* layout,
                         const topkv_batch* batch, void* d_wire, int64_t wire_capacity_bytes,
                         void* d_workspace, int64_t workspace_bytes, topkv_stream_t stream);
int topkv_unpack_layer_crc(int layer, void* dst_pool, const topkv_layout* layout,
                           const topkv_batch* batch, const void* d_wire, int64_t wire_bytes,
                           void* d_workspace, int64_t workspace_bytes, topkv_stream_t stream);
int topkv_crc_finish(const topkv_layout* layout, const topkv_batch* batch, void* d_workspace,
                     int64_t workspace_bytes, uint64_t* d_crc_out, topkv_stream_t stream);
/* The host leg with checksums: topkv_pack_layer_to_host / topkv_unpack_layer_from_host with the
 * checksummed copy as their kernel (same staged and direct forms, same rules), so that the
 * sender checksums while it ships a layer and the receiver while it places it. */
int topkv_pack_layer_to_host_crc(int layer, const void* src_pool, const topkv_layout* layout,
                                 const topkv_batch* batch, void* h_pinned, int64_t host_capacity_bytes,
                                 void* d_staging, int64_t staging_capacity_bytes, void* d_workspace,
                                 int64_t workspace_bytes, topkv_stream_t stream);
int topkv_unpack_layer_from_host_crc(int layer, void* dst_pool, const topkv_layout* layout,
                                     const topkv_batch* batch, const void* h_pinned, int64_t host_bytes,
                                     void* d_staging, int64_t staging_capacity_bytes,
                                     void* d_workspace, int64_t workspace_bytes,
                                     topkv_stream_t stream);

/* Several layers in ONE launch: the layers first_layer .. first_layer + num_layers - 1 of the
 * same batch, exactly as num_layers calls of topkv_pack_layer / topkv_unpack_layer would move
 * them (layer l between pool + l*pool_layer_stride and wire + l*wire_layer_stride). For the side
 * that is not pipelined layer by layer (§5.2 sends per layer; a receiver that gets a whole
 * payload, a re-send after a failed check, §3.1, small decode-side batches), where the launch
 * and the ramp of one kernel per layer would dominate. layout->wire_layer_stride must be > 0
 * when num_layers > 1 (TOPKV_ERR_INVALID_ARG); num_layers <= 65535; num_layers == 0 validates
 * and launches nothing. Other arguments, flags and errors as for the per-layer calls. */
int topkv_pack_layers(int first_layer, int num_layers, const void* src_pool,
                      const topkv_layout* layout, const topkv_batch* batch, void* d_wire,
                      int64_t wire_capacity_bytes, topkv_stream_t stream);
int topkv_unpack_layers(int first_layer, int num_layers, void* dst_pool, const topkv_layout* layout,
                        const topkv_batch* batch, const void* d_wire, int64_t wire_bytes,
                        topkv_stream_t stream);

/* ---- layer-by-layer issue on a side stream (§5.2, Eq. 3) -------------------------------------
 * The pipelined transfer as one call per side: for l = first_layer .. first_layer+num_layers-1,
 * in order, on `side_stream`:
 *     wait for layer_ready[l - first_layer]     (skipped when layer_ready == NULL or the entry is)
 *     topkv_pack_layer_to_host(l, ...)          (topkv_unpack_layer_from_host for the receiver)
 *     record layer_done[l - first_layer]        (skipped when layer_done == NULL or the entry is)
 * so that the transfer of layer l runs while the caller's main stream computes layers l+1..,
 * which recorded layer_ready[l] after layer l's K/V were written. A receiver passes the
 * sender's layer_done events as its layer_ready. Only enqueues; returns after the last layer
 * has been enqueued. Arguments, forms (d_staging NULL = direct) and errors as for the per-layer
 * calls; the events are the caller's, created on the stream's device. Everything is validated
 * for every layer before anything is enqueued, so on an error status nothing was launched,
 * except TOPKV_ERR_CUDA from the runtime in the middle of the loop (layers before it stay
 * enqueued). One staging slab serves all layers: they follow each other on one stream. */
int topkv_pack_layers_to_host_pipelined(int first_layer, int num_layers, const void* src_pool,
                                        const topkv_layout* layout, const topkv_batch* batch,
                                        void* h_pinned, int64_t host_capacity_bytes, void* d_staging,
                                        int64_t staging_capacity_bytes,
                                        const topkv_event_t* layer_ready,
                                        const topkv_event_t* layer_done, topkv_stream_t side_stream);
int topkv_unpack_layers_from_host_pipelined(int first_layer, int num_layers, void* dst_pool,
                                            const topkv_layout* layout, const topkv_batch* batch,
                                            const void* h_pinned, int64_t host_bytes, void* d_staging,
                                            int64_t staging_capacity_bytes,
                                            const topkv_event_t* layer_ready,
                                            const topkv_event_t* layer_done,
                                            topkv_stream_t side_stream);

/* The same schedule on TWO lanes (staged form only): layer i of the range goes to
 * side_streams[i % 2] with d_stagings[i % 2] (HOST arrays of two entries each; the two streams and
 * the two slabs must differ, each slab holds one layer), so that the copy engine moves one layer
 * while the kernel of the next one runs: measured 1.000 / 0.997 of a pinned cudaMemcpyAsync where
 * one lane reaches 0.98. layer_ready[i] is waited for and layer_done[i] recorded on the lane that
 * ships layer i; order between the two lanes is the caller's (e.g. by waiting for the last two
 * layer_done events). Errors as for the one-lane calls. */
int topkv_pack_layers_to_host_two_lanes(int first_layer, int num_layers, const void* src_pool,
                                        const topkv_layout* layout, const topkv_batch* batch,
                                        void* h_pinned, int64_t host_capacity_bytes,
                                        void* const* d_stagings, int64_t staging_capacity_bytes,
                                        const topkv_event_t* layer_ready,
                                        const topkv_event_t* layer_done,
                                        const topkv_stream_t* side_streams);
int topkv_unpack_layers_from_host_two_lanes(int first_layer, int num_layers, void* dst_pool,
                                            const topkv_layout* layout, const topkv_batch* batch,
                                            const void* h_pinned, int64_t host_bytes,
                                            void* const* d_stagings, int64_t staging_capacity_bytes,
                                            const topkv_event_t* layer_ready,
                                            const topkv_event_t* layer_done,
                                            const topkv_stream_t* side_streams);

/* Host-side retry policy of the transfer orchestrator (§3.1: 2 retries, 100 ms exponential
 * backoff): calls attempt(ctx) until it returns TOPKV_OK, at most 1 + retries times, sleeping
 * backoff_ms, 2*backoff_ms, ... between attempts. Returns the last status. */
int topkv_retry(int (*attempt)(void* ctx), void* ctx, int retries, int backoff_ms);

/* ---- allocation-free host leg -------------------------------------------------------------- */

/* Size of the library's built-in staging slab (bytes). Every GPU that loads the library
 * reserves this much device memory until the process exits. */
#define TOPKV_NOALLOC_STAGING_BYTES (8 * 1024 * 1024)

/* (No counterpart in the paper: this exists for callers, not for the method.)
 *
 * Staged form of topkv_pack_layer_to_host for callers that cannot provide a staging slab
 * because they are not allowed to allocate device memory: code running inside another
 * framework's memory pool with a fixed budget, plug-ins loaded after that pool has claimed
 * the GPU, and paths where a cudaMalloc would stall the device (it synchronises) in the
 * middle of serving. The staging slab is a fixed array inside the library's own device image,
 * so this call performs no cudaMalloc / cudaFree and calls no allocating routine.
 *
 * Same result as topkv_pack_layer_to_host with a caller staging slab: layer `layer` is packed
 * into the built-in slab, then copied to h_pinned + layer*wire_layer_stride by the copy
 * engine, all on `stream`. batch->total_tokens must be known (>= 0).
 *
 * Limits and rules:
 *  - N_layer must not exceed TOPKV_NOALLOC_STAGING_BYTES, else TOPKV_ERR_CAPACITY is returned
 *    and nothing is launched.
 *  - The first call on each device looks up the slab's device address (once per device, with
 *    that device current). Make that first call outside any stream capture.
 *  - There is ONE slab per device, shared by every call and every stream, and it keeps the
 *    previous call's bytes. Nothing in it needs to start at zero (each call overwrites the
 *    N_layer bytes it then copies out), but two calls whose GPU work may overlap (different
 *    streams, no ordering between them) race on it: order them on one stream or with events. */
int topkv_pack_layer_to_host_noalloc(int layer, const void* src_pool, const topkv_layout* layout,
                                     const topkv_batch* batch, void* h_pinned,
                                     int64_t host_capacity_bytes, topkv_stream_t stream);

/* ---- plan (layer-invariant, once per batch) ------------------------------------------ */

/* Writes the exclusive prefix sum of seq_lens to d_cu_seq_lens (DEVICE int64 [R+1]). */
int topkv_build_plan(const topkv_batch* batch, int64_t* d_cu_seq_lens, topkv_stream_t stream);

/* Host-side validator for tests and debugging: h_block_table [R][max_pages] and
 * h_seq_lens [R] are HOST copies. Checks seq_len range, that every used page id lies in
 * [0, num_pool_pages) and, when require_disjoint != 0, that no page id is used twice
 * (the unpack precondition). Returns TOPKV_OK or TOPKV_ERR_INVALID_ARG. */
int topkv_validate_batch_host(const topkv_layout* layout, int32_t num_requests,
                              int32_t max_pages_per_req, const int32_t* h_block_table,
                              const int32_t* h_seq_lens, int require_disjoint);

/* ---- size bookkeeping ------------------------------------------------------------------ */

/* Fills the stride fields of *layout for the default page-major pool
 * pool[l][page][c][t][h][d] from its shape fields; wire_layer_stride is left untouched. */
int topkv_layout_default_strides(topkv_layout* layout);

/* N_layer = total_tokens * F * H * D * E, or a negative topkv_status. */
int64_t topkv_wire_layer_bytes(const topkv_layout* layout, int64_t total_tokens);

/* Eq. 1 with the §5.3 MLA rule: F * L * H * D * seq_len * E bytes for one sequence. */
int64_t topkv_kv_bytes(const topkv_layout* layout, int64_t seq_len);

/* Eq. 1 extended per layer kind (§2.2): a full layer counts seq_len tokens, a windowed layer
 * min(seq_len, window) tokens, a constant-state layer (linear attention) a fixed byte count. */
enum { TOPKV_LAYER_FULL = 0, TOPKV_LAYER_WINDOW = 1, TOPKV_LAYER_STATE = 2 };
typedef struct topkv_layer_spec {
  uint32_t kind;     /* TOPKV_LAYER_*                                               */
  uint32_t reserved; /* must be 0                                                   */
  int64_t param;     /* WINDOW: window in tokens; STATE: bytes; FULL: ignored       */
} topkv_layer_spec;
/* specs: HOST array [layout->num_layers]. Returns bytes or a negative topkv_status. */
int64_t topkv_kv_bytes_layered(const topkv_layout* layout, const topkv_layer_spec* specs,
                               int64_t seq_len);

/* ---- a model whose layers differ in kind, on the data path (§2.2) ---------------------------
 * Hybrid models mix layer kinds: full-attention layers cache every token, windowed layers only
 * the last W, linear-attention layers a fixed-size state per request. A layer table describes
 * such a model to the data path, one topkv_layer_spec per MODEL layer, so that the range calls
 * and the side-stream schedule of §5.2 can run it:
 *   FULL, WINDOW  live in the paged pool and share the batch's block table. They are numbered
 *                 among themselves in model order: the a-th attention layer of the model is
 *                 layer a of the pool (layout->num_layers counts attention layers only). A
 *                 WINDOW layer ships the last min(s_r, param) tokens of every request.
 *   STATE         one state of `param` bytes per request, in a pool of slots: the state of
 *                 request r in the j-th STATE layer of the model (numbered among themselves)
 *                 starts at state_pool + j*state_layer_stride + state_slots[r]*state_slot_stride.
 *                 param, both strides and the pool base must be multiples of 16 bytes.
 * The wire holds the layers' slabs back to back in model order (the order in which they are
 * sent): an attention layer's slab is exactly what topkv_pack_layer produces for that layer
 * with that window (wire order as in the layout), a STATE layer's slab the R states in request
 * order. Slab l starts at h_offsets[l] of topkv_layer_table_offsets; the total,
 * h_offsets[num_layers], is Eq. 1 per layer kind summed over the requests.
 * Rules: batch->window_tokens must be 0 (the table decides per layer); batch->cu_seq_lens, when
 * given, serves the FULL layers, WINDOW layers derive their prefix sums in the kernel, so a
 * model with WINDOW layers needs num_requests <= TOPKV_MAX_INLINE_R; h_seq_lens must hold the
 * values of batch->seq_lens (if batch->total_tokens is given it must equal their sum). */
typedef struct topkv_layer_table {
  uint32_t struct_size;           /* = sizeof(topkv_layer_table)                                */
  uint32_t num_layers;            /* layers of the model, every kind                            */
  const topkv_layer_spec* specs;  /* HOST [num_layers]                                          */
  const int32_t* h_seq_lens;      /* HOST int32 [R]: the lengths, to size every slab on the host */
  void* state_pool;               /* DEVICE: slots of the STATE layers; NULL if there are none  */
  const int32_t* state_slots;     /* DEVICE int32 [R]: slot of request r                        */
  int64_t state_layer_stride;     /* bytes from one STATE layer's slots to the next one's       */
  int64_t state_slot_stride;      /* bytes between two slots (>= the largest state)             */
  int64_t num_state_slots;        /* every slot id is checked against it on the device          */
} topkv_layer_table;

/* h_offsets: HOST int64 [table->num_layers + 1]. */
int topkv_layer_table_offsets(const topkv_layout* layout, const topkv_layer_table* table,
                              int32_t num_requests, int64_t* h_offsets);

/* Model layers first_layer .. first_layer + num_layers - 1 between the pools and the wire buffer
 * behind d_wire (slab l at d_wire + h_offsets[l]), device to device, on `stream`. Layers of the
 * same kind and parameter that lie at a constant stride in their pool and in the wire (every
 * other layer of a model that alternates windowed and full layers, the state layers between
 * the full ones) share one launch; otherwise one kernel per layer. The layers of one call touch
 * different slabs and different pool layers, so every launch after the first is allowed to
 * overlap its predecessor (and the layers are moved in no particular order); batch->flags
 * applies to the first. Everything is validated for every layer before anything is launched. For unpack,
 * `dst_pool` and table->state_pool are the destination pools, batch->block_table and
 * table->state_slots the destination's tables. */
int topkv_pack_model_layers(int first_layer, int num_layers, const void* src_pool,
                            const topkv_layout* layout, const topkv_batch* batch,
                            const topkv_layer_table* table, void* d_wire,
                            int64_t wire_capacity_bytes, topkv_stream_t stream);
int topkv_unpack_model_layers(int first_layer, int num_layers, void* dst_pool,
                              const topkv_layout* layout, const topkv_batch* batch,
                              const topkv_layer_table* table, const void* d_wire,
                              int64_t wire_bytes, topkv_stream_t stream);

/* The layer-by-layer side-stream schedule (see topkv_pack_layers_to_host_pipelined) for such a
 * model: per model layer, wait for layer_ready[i], ship the layer's slab to (from) h_pinned +
 * h_offsets[l] over PCIe, record layer_done[i]. d_staging != NULL: staged form, the slab must
 * hold the largest slab of the range; NULL: direct form. Errors as for the plain pipelined
 * calls. */
int topkv_pack_model_layers_to_host_pipelined(int first_layer, int num_layers, const void* src_pool,
                                              const topkv_layout* layout, const topkv_batch* batch,
                                              const topkv_layer_table* table, void* h_pinned,
                                              int64_t host_capacity_bytes, void* d_staging,
                                              int64_t staging_capacity_bytes,
                                              const topkv_event_t* layer_ready,
                                              const topkv_event_t* layer_done,
                                              topkv_stream_t side_stream);
int topkv_unpack_model_layers_from_host_pipelined(int first_layer, int num_layers, void* dst_pool,
                                                  const topkv_layout* layout, const topkv_batch* batch,
                                                  const topkv_layer_table* table, const void* h_pinned,
                                                  int64_t host_bytes, void* d_staging,
                                                  int64_t staging_capacity_bytes,
                                                  const topkv_event_t* layer_ready,
                                                  const topkv_event_t* layer_done,
                                                  topkv_stream_t side_stream);

/* ---- CPU-side analytic helpers (context only; no GPU work) ------------------------------- */

/* Eq. 2: bytes / bandwidth + setup latency, in seconds. */
double topkv_model_transfer_s(double bytes, double bandwidth_bytes_per_s, double setup_s);

/* Eq. 3: T_eff = max(t_last, t_xfer - t_rem). */
double topkv_model_t_eff_s(double t_last_s, double t_xfer_s, double t_rem_s);

/* Fraction of t_xfer hidden behind the (layers-1) layers still computing after the first
 * layer's cache is ready (§5.2 worked example): min(1, (layers-1)*t_layer / t_xfer). */
double topkv_model_hidden_fraction(int layers, double t_layer_compute_s, double t_xfer_total_s);

/* ---- transport selection (Alg. 1) and planning rates (§3.3): host only, context -------------
 * What the transfer manager decides BEFORE any byte moves: which transport carries the cache
 * from the source instance to the target instance. This library implements one of those
 * transports on one GPU (the pinned-host PCIe leg); the selector is here so that a caller can
 * apply the paper's rule and its latency model (Eq. 2) to size a transfer. It moves no data
 * and opens no connection. */
enum {
  TOPKV_TRANSPORT_NVLINK = 1, /* same NVLink domain: 450 GB/s unidirectional (NVLink 4.0, 18 links) */
  TOPKV_TRANSPORT_PCIE = 2,   /* same node, cross-domain: 50 GB/s (Gen5 x16, practical)             */
  TOPKV_TRANSPORT_RDMA = 3,   /* cross-node, RDMA available: 25 GB/s (InfiniBand NDR)               */
  TOPKV_TRANSPORT_TCP = 4     /* fallback: 10 GB/s (100 GbE with gRPC framing)                      */
};
/* What a worker instance reports when it registers (§3.2). Strings are NUL-terminated, HOST. */
typedef struct topkv_endpoint {
  uint32_t struct_size;      /* = sizeof(topkv_endpoint)                                          */
  uint32_t has_nvlink;       /* the instance reports HasNVLink = true                             */
  const char* nvlink_domain; /* the NVLink domain it is registered in; the paper compares node    */
                             /* names (an 8-GPU domain is a node); may be NULL when has_nvlink = 0 */
  const char* node_ip;       /* IsSameNode compares node IP addresses                             */
} topkv_endpoint;
/* Alg. 1, in its order: a configured override (override_mode != 0) wins; else NVLINK when both
 * instances report NVLink and sit in the same domain; else PCIE on the same node; else RDMA when
 * the cluster has it (cluster_has_rdma != 0); else TCP. Returns a TOPKV_TRANSPORT_* value, or
 * TOPKV_ERR_INVALID_ARG (NULL, struct_size mismatch, unknown override, missing node_ip). */
int topkv_select_transport(const topkv_endpoint* source, const topkv_endpoint* target,
                           int cluster_has_rdma, int override_mode);
/* The achievable rate the orchestrator plans with for a mode, bytes per second (§3.3: 450, 50,
 * 25, 10 GB/s); 0.0 for an unknown mode. Table 4 = topkv_model_transfer_s(1.3e9, rate, 0). */
double topkv_planning_rate(int mode);
/* "nvlink", "pcie", "rdma", "tcp", or "unknown". */
const char* topkv_transport_name(int mode);

/* ---- diagnostics ------------------------------------------------------------------------ */

const char* topkv_strerror(int status);
int topkv_version(void);
/* cudaError_t of the most recent failing CUDA call made by this library on this thread. */
int topkv_last_cuda_error(void);
/* Device-side checks. Kernels never trap; when a device table is unusable they skip the
 * affected work and raise a bit in a per-device status word:
 *   1  a bounded wait inside a kernel ran out (output incomplete)
 *   2  a page id lay outside [0, num_pool_pages) or a length exceeded its block-table row:
 *      those pages were skipped, nothing outside the pool was touched
 *   4  the lengths found on the device did not fit the wire slab (N_layer when total_tokens is
 *      known, else the capacity passed): that work was skipped, nothing outside was touched
 * topkv_device_error_flags() waits for ALL work on the current device (cudaDeviceSynchronize:
 * every stream, non-blocking ones included; not a hot-path call) and returns the bits raised on
 * it since the library was loaded or the flags were last reset (0 = none), or a negative
 * topkv_status; topkv_reset_device_error_flags() waits the same way, then clears them. */
int topkv_device_error_flags(void);
int topkv_reset_device_error_flags(void);
/* Width in bytes (16 or 32) of the global loads and stores that topkv_pack_layers /
 * topkv_unpack_layers would use for these arguments in the vectorised kernel family (same
 * arguments, same checks, nothing is launched; 0 for an empty range; a negative topkv_status
 * when the arguments would be refused). 32 requires every base and every stride the kernel adds,
 * the two layer strides included when num_layers > 1, to be a multiple of 32 bytes. */
int topkv_copy_vector_bytes(int first_layer, int num_layers, const void* pool,
                            const topkv_layout* layout, const topkv_batch* batch,
                            const void* d_wire, int64_t wire_bytes);
/* Number of CTAs per layer that topkv_pack_layer / topkv_unpack_layer would launch for these
 * arguments in the vectorised kernel family (same arguments, same checks, nothing is launched;
 * a negative topkv_status when they would be refused). One CTA per span of a block-table row
 * (R * spans per row), or, for a ragged batch whose total is stated and whose launch may read
 * its tables before it waits for its predecessor (either flag), total_tokens / span_tokens + R
 * CTAs: *compact (may be NULL) says which. Whatever the lengths, as long as they add up to
 * total_tokens, that many CTAs cover every span that holds tokens. */
int64_t topkv_copy_grid_ctas(int layer, const void* pool, const topkv_layout* layout,
                             const topkv_batch* batch, const void* d_wire, int64_t wire_bytes,
                             int32_t* compact);
/* Number of kernels this library has launched in this process (all threads). */
int64_t topkv_kernel_launch_count(void);
/* Selects the kernel family used by the four hot calls: 0 = vectorised load/store,
 * 1 = bulk-async copies staged through shared memory. Returns the previous value, or
 * TOPKV_ERR_INVALID_ARG. Process-wide; intended for benchmarking, not for the hot path. */
int topkv_set_kernel_variant(int variant);
/* Grid of the DIRECT host leg (topkv_pack_layer_to_host / topkv_unpack_layer_from_host with
 * d_staging == NULL), the PCIe transport of §3.3 / Table 4: n > 0 = at most n CTAs walk all
 * spans of pages (default TOPKV_DEFAULT_HOST_LEG_CTAS); 0 = one CTA per span, as for a device
 * wire. The PCIe link sets the pace of that leg, so a few CTAs keep it full while the rest of
 * the GPU stays with the prefill that runs beside the transfer (§5.2): on a B200 4 CTAs fill the
 * link with stores and 6 with loads, and when the link is busy all the time every CTA beyond
 * that holds an SM that a GEMM beside it cannot use (8 CTAs: 7 % slower prefill, 16: 40 %).
 * Returns the previous
 * value, or TOPKV_ERR_INVALID_ARG for n < 0 or n > 65535. Process-wide; takes effect for calls
 * made after it returns. The bytes moved are the same for every setting. */
#define TOPKV_DEFAULT_HOST_LEG_CTAS 8
int topkv_set_host_leg_ctas(int ctas);

#ifdef __cplusplus
}
#endif
#endif /* TOPKV_H_ */
