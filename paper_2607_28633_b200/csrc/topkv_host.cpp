// Host-only part of the TopKV library: size bookkeeping (Eq. 1), the analytic helpers
// (Eq. 2, Eq. 3), the host-side batch validator and diagnostics. No CUDA calls here.
#include "topkv.h"

#include <chrono>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <thread>
#include <vector>

namespace {
bool layout_header_ok(const topkv_layout* lo) {
  return lo != nullptr && lo->struct_size == sizeof(topkv_layout);
}
}  // namespace

extern "C" {

int topkv_layout_default_strides(topkv_layout* lo) {
  if (!layout_header_ok(lo)) return TOPKV_ERR_INVALID_ARG;
  if (lo->kv_factor == 0 || lo->num_kv_heads == 0 || lo->head_dim == 0 || lo->elem_bytes == 0 ||
      lo->page_tokens == 0 || lo->num_pool_pages <= 0)
    return TOPKV_ERR_UNSUPPORTED_LAYOUT;
  // pool[l][page][c][t][h][d], innermost contiguous
  lo->pool_head_stride = (int64_t)lo->head_dim * lo->elem_bytes;
  lo->pool_token_stride = lo->pool_head_stride * lo->num_kv_heads;
  lo->pool_kv_stride = lo->pool_token_stride * lo->page_tokens;
  lo->pool_page_stride = lo->pool_kv_stride * lo->kv_factor;
  lo->pool_layer_stride = lo->pool_page_stride * lo->num_pool_pages;
  return TOPKV_OK;
}

int64_t topkv_wire_layer_bytes(const topkv_layout* lo, int64_t total_tokens) {
  if (!layout_header_ok(lo) || total_tokens < 0) return TOPKV_ERR_INVALID_ARG;
  return total_tokens * lo->kv_factor * lo->num_kv_heads * lo->head_dim * lo->elem_bytes;
}

int64_t topkv_kv_bytes(const topkv_layout* lo, int64_t seq_len) {
  if (!layout_header_ok(lo) || seq_len < 0) return TOPKV_ERR_INVALID_ARG;
  // Eq. 1: 2 * L * h_kv * d_h * s * b_p; the leading 2 becomes 1 for an MLA latent (§5.3).
  return (int64_t)lo->kv_factor * lo->num_layers * lo->num_kv_heads * lo->head_dim * seq_len *
         lo->elem_bytes;
}

int64_t topkv_kv_bytes_layered(const topkv_layout* lo, const topkv_layer_spec* specs,
                               int64_t seq_len) {
  if (!layout_header_ok(lo) || specs == nullptr || seq_len < 0) return TOPKV_ERR_INVALID_ARG;
  const int64_t tok_bytes = (int64_t)lo->kv_factor * lo->num_kv_heads * lo->head_dim * lo->elem_bytes;
  int64_t total = 0;
  for (uint32_t l = 0; l < lo->num_layers; ++l) {
    const topkv_layer_spec& sp = specs[l];
    if (sp.reserved != 0 || sp.param < 0) return TOPKV_ERR_INVALID_ARG;
    switch (sp.kind) {
      case TOPKV_LAYER_FULL: total += tok_bytes * seq_len; break;
      case TOPKV_LAYER_WINDOW: total += tok_bytes * (sp.param < seq_len ? sp.param : seq_len); break;
      case TOPKV_LAYER_STATE: total += sp.param; break;
      default: return TOPKV_ERR_INVALID_ARG;
    }
  }
  return total;
}

double topkv_model_transfer_s(double bytes, double bandwidth_bytes_per_s, double setup_s) {
  return bytes / bandwidth_bytes_per_s + setup_s;
}

double topkv_model_t_eff_s(double t_last_s, double t_xfer_s, double t_rem_s) {
  const double exposed = t_xfer_s - t_rem_s;
  return exposed > t_last_s ? exposed : t_last_s;
}

double topkv_model_hidden_fraction(int layers, double t_layer_compute_s, double t_xfer_total_s) {
  if (t_xfer_total_s <= 0.0) return 1.0;
  const double covered = (layers - 1) * t_layer_compute_s / t_xfer_total_s;
  return covered < 1.0 ? covered : 1.0;
}

// ---- transport selection (Alg. 1), planning rates (§3.3) ----------------------------------------
int topkv_select_transport(const topkv_endpoint* s, const topkv_endpoint* t, int cluster_has_rdma,
                           int override_mode) {
  if (s == nullptr || t == nullptr || s->struct_size != sizeof(topkv_endpoint) ||
      t->struct_size != sizeof(topkv_endpoint))
    return TOPKV_ERR_INVALID_ARG;
  if (override_mode != 0) {  // a manual override is returned as configured
    if (override_mode < TOPKV_TRANSPORT_NVLINK || override_mode > TOPKV_TRANSPORT_TCP)
      return TOPKV_ERR_INVALID_ARG;
    return override_mode;
  }
  if (s->node_ip == nullptr || t->node_ip == nullptr) return TOPKV_ERR_INVALID_ARG;
  const bool both_report = s->has_nvlink != 0 && t->has_nvlink != 0;
  if (both_report && (s->nvlink_domain == nullptr || t->nvlink_domain == nullptr))
    return TOPKV_ERR_INVALID_ARG;
  if (both_report && std::strcmp(s->nvlink_domain, t->nvlink_domain) == 0) return TOPKV_TRANSPORT_NVLINK;
  if (std::strcmp(s->node_ip, t->node_ip) == 0) return TOPKV_TRANSPORT_PCIE;
  return cluster_has_rdma != 0 ? TOPKV_TRANSPORT_RDMA : TOPKV_TRANSPORT_TCP;
}

double topkv_planning_rate(int mode) {
  static const double kGBps[5] = {0.0, 450.0, 50.0, 25.0, 10.0};
  if (mode < TOPKV_TRANSPORT_NVLINK || mode > TOPKV_TRANSPORT_TCP) return 0.0;
  return kGBps[mode] * 1e9;
}

const char* topkv_transport_name(int mode) {
  static const char* const kNames[5] = {"unknown", "nvlink", "pcie", "rdma", "tcp"};
  return (mode >= TOPKV_TRANSPORT_NVLINK && mode <= TOPKV_TRANSPORT_TCP) ? kNames[mode] : kNames[0];
}

int topkv_validate_batch_host(const topkv_layout* lo, int32_t R, int32_t maxp,
                              const int32_t* h_bt, const int32_t* h_sl, int require_disjoint) {
  if (!layout_header_ok(lo) || R < 0 || maxp < 0) return TOPKV_ERR_INVALID_ARG;
  if (R > 0 && (h_sl == nullptr || (maxp > 0 && h_bt == nullptr))) return TOPKV_ERR_INVALID_ARG;
  if (lo->page_tokens == 0 || lo->num_pool_pages <= 0) return TOPKV_ERR_INVALID_ARG;
  std::vector<uint8_t> seen;
  if (require_disjoint) seen.assign((size_t)lo->num_pool_pages, 0);
  const int64_t P = lo->page_tokens;
  for (int32_t r = 0; r < R; ++r) {
    const int64_t s = h_sl[r];
    if (s < 0 || s > (int64_t)maxp * P) return TOPKV_ERR_INVALID_ARG;
    const int64_t n = (s + P - 1) / P;
    for (int64_t j = 0; j < n; ++j) {
      const int64_t page = h_bt[(int64_t)r * maxp + j];
      if (page < 0 || page >= lo->num_pool_pages) return TOPKV_ERR_INVALID_ARG;
      if (require_disjoint) {
        if (seen[(size_t)page]) return TOPKV_ERR_INVALID_ARG;
        seen[(size_t)page] = 1;
      }
    }
  }
  return TOPKV_OK;
}

// ---- CRC-64 (host), header, retry --------------------------------------------------------------
namespace {
uint64_t g_crc_table[256];
std::once_flag g_crc_once;
void build_crc_table() {
  const uint64_t poly = 0xD800000000000000ull;  // x^64 + x^4 + x^3 + x + 1, reflected
  for (int b = 0; b < 256; ++b) {
    uint64_t v = (uint64_t)b;
    for (int k = 0; k < 8; ++k) v = (v & 1) ? (v >> 1) ^ poly : (v >> 1);
    g_crc_table[b] = v;
  }
}
}  // namespace

uint64_t topkv_crc64(const void* h_data, int64_t nbytes) {
  std::call_once(g_crc_once, build_crc_table);
  const uint8_t* p = static_cast<const uint8_t*>(h_data);
  uint64_t crc = ~0ull;
  for (int64_t i = 0; i < nbytes; ++i) crc = g_crc_table[(crc ^ p[i]) & 0xff] ^ (crc >> 8);
  return ~crc;
}

int topkv_header_fill(topkv_wire_header* h, uint64_t request_id, uint64_t model_id,
                      const topkv_layout* lo, int64_t seq_len, uint64_t crc_k, uint64_t crc_v) {
  if (h == nullptr || !layout_header_ok(lo) || seq_len < 0 || seq_len > 0xffffffffll)
    return TOPKV_ERR_INVALID_ARG;
  static_assert(sizeof(topkv_wire_header) == 128, "the header is 128 bytes");
  std::memset(h, 0, sizeof(*h));
  std::memcpy(h->magic, "KVCACHE1", 8);
  h->request_id = request_id;
  h->model_id = model_id;
  h->seq_len = (uint32_t)seq_len;
  h->num_layers = lo->num_layers;
  h->num_kv_heads = lo->num_kv_heads;
  h->head_dim = lo->head_dim;
  h->elem_bytes = lo->elem_bytes;
  h->kv_factor = lo->kv_factor;
  const uint64_t plane = (uint64_t)lo->num_layers * (uint64_t)seq_len * lo->num_kv_heads *
                         lo->head_dim * lo->elem_bytes;
  h->k_bytes = plane;
  h->v_bytes = lo->kv_factor == 2 ? plane : 0;
  h->crc_k = crc_k;
  h->crc_v = lo->kv_factor == 2 ? crc_v : 0;
  return TOPKV_OK;
}

int topkv_header_check(const topkv_wire_header* h, const topkv_layout* lo, int64_t seq_len,
                       uint64_t crc_k, uint64_t crc_v) {
  if (h == nullptr || !layout_header_ok(lo) || seq_len < 0) return TOPKV_ERR_INVALID_ARG;
  topkv_wire_header want;
  const int st = topkv_header_fill(&want, h->request_id, h->model_id, lo, seq_len, crc_k, crc_v);
  if (st != TOPKV_OK) return st;
  return std::memcmp(&want, h, sizeof(want)) == 0 ? TOPKV_OK : TOPKV_ERR_CHECKSUM;
}

int topkv_retry(int (*attempt)(void* ctx), void* ctx, int retries, int backoff_ms) {
  if (attempt == nullptr || retries < 0 || backoff_ms < 0) return TOPKV_ERR_INVALID_ARG;
  int status = attempt(ctx);
  int64_t wait_ms = backoff_ms;
  for (int k = 0; k < retries && status != TOPKV_OK; ++k) {
    std::this_thread::sleep_for(std::chrono::milliseconds(wait_ms));
    wait_ms *= 2;
    status = attempt(ctx);
  }
  return status;
}

const char* topkv_strerror(int status) {
  switch (status) {
    case TOPKV_OK: return "ok";
    case TOPKV_ERR_INVALID_ARG: return "invalid argument";
    case TOPKV_ERR_LAYER_RANGE: return "layer index out of range";
    case TOPKV_ERR_ALIGNMENT: return "pointer, stride or row size not a multiple of 16 bytes";
    case TOPKV_ERR_CAPACITY: return "buffer too small for this layer's wire slab";
    case TOPKV_ERR_UNSUPPORTED_LAYOUT: return "unsupported or inconsistent layout descriptor";
    case TOPKV_ERR_CUDA: return "CUDA call failed (see topkv_last_cuda_error)";
    case TOPKV_ERR_CHECKSUM: return "header or CRC-64 mismatch";
    default: return "unknown status";
  }
}

int topkv_version(void) { return 120; }

}  // extern "C"
