// Host-only part of the TopKV library: size bookkeeping (Eq. 1), the analytic helpers
// (Eq. 2, Eq. 3), the host-side batch validator and diagnostics. No CUDA calls here.
#include "topkv.h"

#include <cstdint>
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

const char* topkv_strerror(int status) {
  switch (status) {
    case TOPKV_OK: return "ok";
    case TOPKV_ERR_INVALID_ARG: return "invalid argument";
    case TOPKV_ERR_LAYER_RANGE: return "layer index out of range";
    case TOPKV_ERR_ALIGNMENT: return "pointer, stride or row size not a multiple of 16 bytes";
    case TOPKV_ERR_CAPACITY: return "buffer too small for this layer's wire slab";
    case TOPKV_ERR_UNSUPPORTED_LAYOUT: return "unsupported or inconsistent layout descriptor";
    case TOPKV_ERR_CUDA: return "CUDA call failed (see topkv_last_cuda_error)";
    default: return "unknown status";
  }
}

int topkv_version(void) { return 100; }

}  // extern "C"
