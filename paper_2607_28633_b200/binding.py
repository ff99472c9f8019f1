"""ctypes binding of the TopKV C-ABI library (``include/topkv.h``).

Argument marshalling only: every function below has the name and the argument order of the
C entry point it calls, accepts torch tensors (their ``data_ptr()`` is passed) or raw integer
addresses, and returns the C status code unchanged. ``check()`` turns a negative status into
an exception. The library is loaded on first use; if it has not been built this module
raises — there is no fallback implementation.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_double, c_int, c_int32, c_int64, c_uint32, c_void_p

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtopkv.so")

TOPKV_OK = 0
TOPKV_ERR_INVALID_ARG = -1
TOPKV_ERR_LAYER_RANGE = -2
TOPKV_ERR_ALIGNMENT = -3
TOPKV_ERR_CAPACITY = -4
TOPKV_ERR_UNSUPPORTED_LAYOUT = -5
TOPKV_ERR_CUDA = -6
TOPKV_ERR_CHECKSUM = -7

TOPKV_KIND_GQA, TOPKV_KIND_MLA = 0, 1
TOPKV_WIRE_TOKEN_KV, TOPKV_WIRE_PLANAR = 0, 1
TOPKV_MAX_INLINE_R = 1024
TOPKV_FLAG_OVERLAP_PREVIOUS = 1
TOPKV_FLAG_TABLES_SETTLED = 2
TOPKV_LINK_WAIT_PREVIOUS = 1
TOPKV_NOALLOC_STAGING_BYTES = 8 * 1024 * 1024

# every symbol include/topkv.h declares
EXPORTS = (
    "topkv_pack_layer", "topkv_unpack_layer", "topkv_pack_layer_to_host",
    "topkv_unpack_layer_from_host", "topkv_build_plan", "topkv_validate_batch_host",
    "topkv_layout_default_strides", "topkv_wire_layer_bytes", "topkv_kv_bytes",
    "topkv_model_transfer_s", "topkv_model_t_eff_s", "topkv_model_hidden_fraction",
    "topkv_strerror", "topkv_version", "topkv_last_cuda_error", "topkv_kernel_launch_count",
    "topkv_set_kernel_variant", "topkv_pack_layer_to_host_noalloc", "topkv_device_error_flags",
    "topkv_reset_device_error_flags", "topkv_repage_layer", "topkv_kv_bytes_layered",
    "topkv_header_fill", "topkv_header_check", "topkv_crc64", "topkv_crc_workspace_bytes",
    "topkv_crc_begin", "topkv_pack_layer_crc", "topkv_unpack_layer_crc", "topkv_crc_finish",
    "topkv_retry", "topkv_pack_layer_to_host_crc", "topkv_unpack_layer_from_host_crc",
    "topkv_set_host_leg_ctas", "topkv_pack_layers_to_host_pipelined",
    "topkv_unpack_layers_from_host_pipelined", "topkv_pack_layers", "topkv_unpack_layers",
    "topkv_copy_vector_bytes", "topkv_copy_grid_ctas", "topkv_select_transport", "topkv_planning_rate",
    "topkv_transport_name", "topkv_layer_table_offsets", "topkv_pack_model_layers",
    "topkv_unpack_model_layers", "topkv_pack_model_layers_to_host_pipelined",
    "topkv_unpack_model_layers_from_host_pipelined", "topkv_span_link_words",
    "topkv_pack_layer_linked", "topkv_unpack_layer_linked",
    "topkv_pack_layers_to_host_two_lanes", "topkv_unpack_layers_from_host_two_lanes",
    "topkv_relay_layers_linked",
)


class topkv_layout(ctypes.Structure):
    _fields_ = [
        ("struct_size", c_uint32), ("kind", c_uint32), ("num_layers", c_uint32),
        ("kv_factor", c_uint32), ("num_kv_heads", c_uint32), ("head_dim", c_uint32),
        ("elem_bytes", c_uint32), ("page_tokens", c_uint32), ("wire_order", c_uint32),
        ("reserved", c_uint32), ("num_pool_pages", c_int64), ("pool_layer_stride", c_int64),
        ("pool_page_stride", c_int64), ("pool_kv_stride", c_int64),
        ("pool_token_stride", c_int64), ("pool_head_stride", c_int64),
        ("wire_layer_stride", c_int64), ("wire_plane_stride", c_int64),
    ]


class topkv_batch(ctypes.Structure):
    _fields_ = [
        ("struct_size", c_uint32), ("num_requests", c_int32), ("max_pages_per_req", c_int32),
        ("flags", c_uint32), ("block_table", c_void_p), ("seq_lens", c_void_p),
        ("cu_seq_lens", c_void_p), ("total_tokens", c_int64), ("window_tokens", c_int32),
        ("reserved", c_int32),
    ]


class topkv_layer_spec(ctypes.Structure):
    _fields_ = [("kind", c_uint32), ("reserved", c_uint32), ("param", c_int64)]


TOPKV_LAYER_FULL, TOPKV_LAYER_WINDOW, TOPKV_LAYER_STATE = 0, 1, 2


class topkv_span_link(ctypes.Structure):
    _fields_ = [("struct_size", c_uint32), ("await_epoch", c_uint32), ("signal_epoch", c_uint32),
                ("flags", c_uint32), ("d_await", c_void_p), ("d_signal", c_void_p)]


def make_span_link(d_await=None, await_epoch=0, d_signal=None, signal_epoch=0,
                   flags: int = 0) -> topkv_span_link:
    k = topkv_span_link()
    k.struct_size = ctypes.sizeof(topkv_span_link)
    k.await_epoch, k.signal_epoch, k.flags = await_epoch, signal_epoch, flags
    k.d_await, k.d_signal = _ptr(d_await), _ptr(d_signal)
    k._keepalive = (d_await, d_signal)
    return k


class topkv_layer_table(ctypes.Structure):
    _fields_ = [("struct_size", c_uint32), ("num_layers", c_uint32), ("specs", c_void_p),
                ("h_seq_lens", c_void_p), ("state_pool", c_void_p), ("state_slots", c_void_p),
                ("state_layer_stride", c_int64), ("state_slot_stride", c_int64),
                ("num_state_slots", c_int64)]


def make_layer_table(specs, h_seq_lens, state_pool=None, state_slots=None, state_layer_stride=0,
                     state_slot_stride=0, num_state_slots=0) -> topkv_layer_table:
    """specs: sequence of (kind, param) per model layer; h_seq_lens: numpy int32 [R] on the host;
    state_pool / state_slots: device tensors (or None). The table keeps what it points to alive."""
    import numpy as np
    arr = (topkv_layer_spec * len(specs))()
    for i, (kind, param) in enumerate(specs):
        arr[i].kind, arr[i].param = kind, param
    lens = np.ascontiguousarray(h_seq_lens, dtype=np.int32)
    t = topkv_layer_table()
    t.struct_size = ctypes.sizeof(topkv_layer_table)
    t.num_layers = len(specs)
    t.specs = ctypes.addressof(arr)
    t.h_seq_lens = lens.ctypes.data
    t.state_pool = _ptr(state_pool)
    t.state_slots = _ptr(state_slots)
    t.state_layer_stride, t.state_slot_stride = state_layer_stride, state_slot_stride
    t.num_state_slots = num_state_slots
    t._keepalive = (arr, lens, state_pool, state_slots)
    return t
TOPKV_TRANSPORT_NVLINK, TOPKV_TRANSPORT_PCIE, TOPKV_TRANSPORT_RDMA, TOPKV_TRANSPORT_TCP = 1, 2, 3, 4


class topkv_endpoint(ctypes.Structure):
    _fields_ = [("struct_size", c_uint32), ("has_nvlink", c_uint32),
                ("nvlink_domain", ctypes.c_char_p), ("node_ip", ctypes.c_char_p)]


def make_endpoint(nvlink_domain, has_nvlink, node_ip) -> topkv_endpoint:
    e = topkv_endpoint()
    e.struct_size = ctypes.sizeof(topkv_endpoint)
    e.has_nvlink = 1 if has_nvlink else 0
    e.nvlink_domain = None if nvlink_domain is None else nvlink_domain.encode()
    e.node_ip = None if node_ip is None else node_ip.encode()
    return e


class topkv_wire_header(ctypes.Structure):
    _fields_ = [
        ("magic", ctypes.c_char * 8), ("request_id", ctypes.c_uint64), ("model_id", ctypes.c_uint64),
        ("seq_len", c_uint32), ("num_layers", c_uint32), ("num_kv_heads", c_uint32),
        ("head_dim", c_uint32), ("elem_bytes", c_uint32), ("kv_factor", c_uint32),
        ("k_bytes", ctypes.c_uint64), ("v_bytes", ctypes.c_uint64), ("crc_k", ctypes.c_uint64),
        ("crc_v", ctypes.c_uint64), ("reserved", ctypes.c_uint8 * 48),
    ]


RETRY_ATTEMPT = ctypes.CFUNCTYPE(c_int, c_void_p)


class TopkvError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        super().__init__(f"topkv status {status}: {topkv_strerror(status)}")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libtopkv.so (built by ``__graft_entry__.build()``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} not found: build the CUDA library first "
                "(python -c 'import __graft_entry__ as g; g.build()'); there is no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        lp, bp = ctypes.POINTER(topkv_layout), ctypes.POINTER(topkv_batch)
        L.topkv_pack_layer.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64, c_void_p]
        L.topkv_unpack_layer.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64, c_void_p]
        L.topkv_pack_layer_to_host.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64,
                                               c_void_p, c_int64, c_void_p]
        L.topkv_unpack_layer_from_host.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64,
                                                   c_void_p, c_int64, c_void_p]
        L.topkv_build_plan.argtypes = [bp, c_void_p, c_void_p]
        u64 = ctypes.c_uint64
        hp = ctypes.POINTER(topkv_wire_header)
        L.topkv_header_fill.argtypes = [hp, u64, u64, lp, c_int64, u64, u64]
        L.topkv_header_check.argtypes = [hp, lp, c_int64, u64, u64]
        L.topkv_crc64.argtypes = [c_void_p, c_int64]
        L.topkv_crc64.restype = u64
        L.topkv_crc_workspace_bytes.argtypes = [lp, c_int32, c_int32]
        L.topkv_crc_workspace_bytes.restype = c_int64
        L.topkv_crc_begin.argtypes = [lp, bp, c_void_p, c_int64, c_void_p]
        L.topkv_pack_layer_crc.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64, c_void_p,
                                           c_int64, c_void_p]
        L.topkv_unpack_layer_crc.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64, c_void_p,
                                             c_int64, c_void_p]
        L.topkv_crc_finish.argtypes = [lp, bp, c_void_p, c_int64, c_void_p, c_void_p]
        for fn in (L.topkv_pack_layer_to_host_crc, L.topkv_unpack_layer_from_host_crc):
            fn.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64, c_void_p, c_int64, c_void_p,
                           c_int64, c_void_p]
        L.topkv_retry.argtypes = [RETRY_ATTEMPT, c_void_p, c_int, c_int]
        L.topkv_repage_layer.argtypes = [c_int, c_void_p, lp, bp, c_void_p, lp, bp, c_void_p]
        L.topkv_pack_layer_to_host_noalloc.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64,
                                                       c_void_p]
        L.topkv_validate_batch_host.argtypes = [lp, c_int32, c_int32, c_void_p, c_void_p, c_int]
        L.topkv_layout_default_strides.argtypes = [lp]
        L.topkv_wire_layer_bytes.argtypes = [lp, c_int64]
        L.topkv_wire_layer_bytes.restype = c_int64
        L.topkv_kv_bytes.argtypes = [lp, c_int64]
        L.topkv_kv_bytes.restype = c_int64
        L.topkv_kv_bytes_layered.argtypes = [lp, c_void_p, c_int64]
        L.topkv_kv_bytes_layered.restype = c_int64
        L.topkv_model_transfer_s.argtypes = [c_double] * 3
        L.topkv_model_transfer_s.restype = c_double
        L.topkv_model_t_eff_s.argtypes = [c_double] * 3
        L.topkv_model_t_eff_s.restype = c_double
        L.topkv_model_hidden_fraction.argtypes = [c_int, c_double, c_double]
        L.topkv_model_hidden_fraction.restype = c_double
        L.topkv_strerror.argtypes = [c_int]
        L.topkv_strerror.restype = ctypes.c_char_p
        L.topkv_kernel_launch_count.restype = c_int64
        L.topkv_set_kernel_variant.argtypes = [c_int]
        L.topkv_set_host_leg_ctas.argtypes = [c_int]
        L.topkv_pack_layers.argtypes = [c_int, c_int, c_void_p, lp, bp, c_void_p, c_int64, c_void_p]
        L.topkv_unpack_layers.argtypes = [c_int, c_int, c_void_p, lp, bp, c_void_p, c_int64, c_void_p]
        for fn in (L.topkv_pack_layers_to_host_two_lanes, L.topkv_unpack_layers_from_host_two_lanes):
            fn.argtypes = [c_int, c_int, c_void_p, lp, bp, c_void_p, c_int64, c_void_p, c_int64,
                           c_void_p, c_void_p, c_void_p]
        kp_ = ctypes.POINTER(topkv_span_link)
        L.topkv_span_link_words.argtypes = [lp, bp]
        L.topkv_span_link_words.restype = c_int64
        L.topkv_pack_layer_linked.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64, kp_, c_void_p]
        L.topkv_unpack_layer_linked.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64, kp_, c_void_p]
        L.topkv_relay_layers_linked.argtypes = [c_int, c_int, c_void_p, lp, bp, c_void_p, lp, bp, c_void_p,
                                                c_int64, c_void_p, c_int64, c_uint32, c_void_p]
        tp = ctypes.POINTER(topkv_layer_table)
        L.topkv_layer_table_offsets.argtypes = [lp, tp, c_int32, c_void_p]
        L.topkv_pack_model_layers.argtypes = [c_int, c_int, c_void_p, lp, bp, tp, c_void_p, c_int64, c_void_p]
        L.topkv_unpack_model_layers.argtypes = [c_int, c_int, c_void_p, lp, bp, tp, c_void_p, c_int64, c_void_p]
        for fn in (L.topkv_pack_model_layers_to_host_pipelined,
                   L.topkv_unpack_model_layers_from_host_pipelined):
            fn.argtypes = [c_int, c_int, c_void_p, lp, bp, tp, c_void_p, c_int64, c_void_p, c_int64,
                           c_void_p, c_void_p, c_void_p]
        ep = ctypes.POINTER(topkv_endpoint)
        L.topkv_select_transport.argtypes = [ep, ep, c_int, c_int]
        L.topkv_planning_rate.argtypes = [c_int]
        L.topkv_planning_rate.restype = c_double
        L.topkv_transport_name.argtypes = [c_int]
        L.topkv_transport_name.restype = ctypes.c_char_p
        L.topkv_copy_vector_bytes.argtypes = [c_int, c_int, c_void_p, lp, bp, c_void_p, c_int64]
        L.topkv_copy_grid_ctas.restype = c_int64
        L.topkv_copy_grid_ctas.argtypes = [c_int, c_void_p, lp, bp, c_void_p, c_int64, ctypes.POINTER(c_int32)]
        for fn in (L.topkv_pack_layers_to_host_pipelined, L.topkv_unpack_layers_from_host_pipelined):
            fn.argtypes = [c_int, c_int, c_void_p, lp, bp, c_void_p, c_int64, c_void_p, c_int64,
                           c_void_p, c_void_p, c_void_p]
        _lib = L
    return _lib


def _ptr(x) -> int | None:
    """torch tensor / numpy array / int / None -> address."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(type(x))


def _stream(s) -> int | None:
    if s is None:
        return None
    if isinstance(s, int):
        return s or None
    return s.cuda_stream or None  # torch.cuda.Stream


def check(status: int) -> int:
    if status < 0:
        raise TopkvError(status)
    return status


# ---- constructors for the two descriptors -------------------------------------------------

def make_layout(L: int, F: int, H: int, D: int, E: int, P: int, num_pool_pages: int,
                wire_order: int = TOPKV_WIRE_TOKEN_KV, wire_layer_stride: int = 0,
                kind: int | None = None) -> topkv_layout:
    """Layout of the default page-major pool pool[l][page][c][t][h][d]."""
    lo = topkv_layout()
    lo.struct_size = ctypes.sizeof(topkv_layout)
    lo.kind = (TOPKV_KIND_MLA if F == 1 and H == 1 else TOPKV_KIND_GQA) if kind is None else kind
    lo.num_layers, lo.kv_factor, lo.num_kv_heads, lo.head_dim = L, F, H, D
    lo.elem_bytes, lo.page_tokens, lo.wire_order = E, P, wire_order
    lo.num_pool_pages = num_pool_pages
    lo.wire_layer_stride = wire_layer_stride
    check(topkv_layout_default_strides(lo))
    return lo


def make_batch(block_table, seq_lens, total_tokens: int = -1, cu_seq_lens=None,
               flags: int = 0, window_tokens: int = 0) -> topkv_batch:
    """block_table: device int32 [R][maxp]; seq_lens: device int32 [R]. The descriptor keeps a
    reference to the tensors it was built from."""
    b = topkv_batch()
    b.struct_size = ctypes.sizeof(topkv_batch)
    b.num_requests = int(block_table.shape[0])
    b.max_pages_per_req = int(block_table.shape[1]) if block_table.ndim == 2 else 0
    b.block_table = _ptr(block_table)
    b.seq_lens = _ptr(seq_lens)
    b.cu_seq_lens = _ptr(cu_seq_lens)
    b.total_tokens = total_tokens
    b.flags = flags
    b.window_tokens = window_tokens
    # The struct only holds addresses: keep the tensors alive with it, so that a temporary
    # passed here cannot be freed (and its memory reused) while the descriptor is in use.
    b._keepalive = (block_table, seq_lens, cu_seq_lens)
    return b


# ---- the C entry points, same names, same order ---------------------------------------------

def topkv_pack_layer(layer, src_pool, layout, batch, d_wire, wire_capacity_bytes, stream=None):
    return lib().topkv_pack_layer(layer, _ptr(src_pool), ctypes.byref(layout), ctypes.byref(batch),
                                  _ptr(d_wire), wire_capacity_bytes, _stream(stream))


def topkv_unpack_layer(layer, dst_pool, layout, batch, d_wire, wire_bytes, stream=None):
    return lib().topkv_unpack_layer(layer, _ptr(dst_pool), ctypes.byref(layout),
                                    ctypes.byref(batch), _ptr(d_wire), wire_bytes, _stream(stream))


def topkv_pack_layers(first_layer, num_layers, src_pool, layout, batch, d_wire, wire_capacity_bytes,
                      stream=None):
    return lib().topkv_pack_layers(first_layer, num_layers, _ptr(src_pool), ctypes.byref(layout),
                                   ctypes.byref(batch), _ptr(d_wire), wire_capacity_bytes,
                                   _stream(stream))


def topkv_unpack_layers(first_layer, num_layers, dst_pool, layout, batch, d_wire, wire_bytes,
                        stream=None):
    return lib().topkv_unpack_layers(first_layer, num_layers, _ptr(dst_pool), ctypes.byref(layout),
                                     ctypes.byref(batch), _ptr(d_wire), wire_bytes, _stream(stream))


def topkv_copy_grid_ctas(layer, pool, layout, batch, d_wire, wire_bytes):
    """(CTAs per layer or a negative status, compact grid or not)."""
    compact = c_int32(0)
    n = lib().topkv_copy_grid_ctas(layer, _ptr(pool), ctypes.byref(layout), ctypes.byref(batch), _ptr(d_wire),
                                   wire_bytes, ctypes.byref(compact))
    return int(n), bool(compact.value)


def topkv_copy_vector_bytes(first_layer, num_layers, pool, layout, batch, d_wire, wire_bytes):
    return lib().topkv_copy_vector_bytes(first_layer, num_layers, _ptr(pool), ctypes.byref(layout),
                                         ctypes.byref(batch), _ptr(d_wire), wire_bytes)


def topkv_pack_layer_to_host(layer, src_pool, layout, batch, h_pinned, host_capacity_bytes,
                             d_staging, staging_capacity_bytes, stream=None):
    return lib().topkv_pack_layer_to_host(layer, _ptr(src_pool), ctypes.byref(layout),
                                          ctypes.byref(batch), _ptr(h_pinned), host_capacity_bytes,
                                          _ptr(d_staging), staging_capacity_bytes, _stream(stream))


def topkv_unpack_layer_from_host(layer, dst_pool, layout, batch, h_pinned, host_bytes, d_staging,
                                 staging_capacity_bytes, stream=None):
    return lib().topkv_unpack_layer_from_host(layer, _ptr(dst_pool), ctypes.byref(layout),
                                              ctypes.byref(batch), _ptr(h_pinned), host_bytes,
                                              _ptr(d_staging), staging_capacity_bytes,
                                              _stream(stream))


def _events(events, n):
    """torch.cuda.Event list (entries may be None) -> C array of cudaEvent_t, or None."""
    if events is None:
        return None
    assert len(events) == n
    arr = (c_void_p * n)()
    for i, e in enumerate(events):
        if e is None:
            continue
        if not e.cuda_event:
            # torch creates the CUDA event only at its first record(): give it a handle now
            # (recording on the current stream; the library's own record replaces it)
            e.record()
        arr[i] = e.cuda_event
    return arr


def topkv_pack_layers_to_host_pipelined(first_layer, num_layers, src_pool, layout, batch, h_pinned,
                                        host_capacity_bytes, d_staging, staging_capacity_bytes,
                                        layer_ready=None, layer_done=None, side_stream=None):
    return lib().topkv_pack_layers_to_host_pipelined(
        first_layer, num_layers, _ptr(src_pool), ctypes.byref(layout), ctypes.byref(batch),
        _ptr(h_pinned), host_capacity_bytes, _ptr(d_staging), staging_capacity_bytes,
        _events(layer_ready, num_layers), _events(layer_done, num_layers), _stream(side_stream))


def topkv_unpack_layers_from_host_pipelined(first_layer, num_layers, dst_pool, layout, batch, h_pinned,
                                            host_bytes, d_staging, staging_capacity_bytes,
                                            layer_ready=None, layer_done=None, side_stream=None):
    return lib().topkv_unpack_layers_from_host_pipelined(
        first_layer, num_layers, _ptr(dst_pool), ctypes.byref(layout), ctypes.byref(batch),
        _ptr(h_pinned), host_bytes, _ptr(d_staging), staging_capacity_bytes,
        _events(layer_ready, num_layers), _events(layer_done, num_layers), _stream(side_stream))


def topkv_span_link_words(layout, batch):
    return lib().topkv_span_link_words(ctypes.byref(layout), ctypes.byref(batch))


def topkv_pack_layer_linked(layer, src_pool, layout, batch, d_wire, wire_capacity_bytes, link,
                            stream=None):
    return lib().topkv_pack_layer_linked(layer, _ptr(src_pool), ctypes.byref(layout),
                                         ctypes.byref(batch), _ptr(d_wire), wire_capacity_bytes,
                                         ctypes.byref(link), _stream(stream))


def topkv_unpack_layer_linked(layer, dst_pool, layout, batch, d_wire, wire_bytes, link, stream=None):
    return lib().topkv_unpack_layer_linked(layer, _ptr(dst_pool), ctypes.byref(layout),
                                           ctypes.byref(batch), _ptr(d_wire), wire_bytes,
                                           ctypes.byref(link), _stream(stream))


def topkv_relay_layers_linked(first_layer, num_layers, src_pool, src_layout, src_batch, dst_pool,
                              dst_layout, dst_batch, d_slab, slab_bytes, d_flags, flags_words,
                              first_epoch, stream=None):
    return lib().topkv_relay_layers_linked(
        first_layer, num_layers, _ptr(src_pool), ctypes.byref(src_layout), ctypes.byref(src_batch),
        _ptr(dst_pool), ctypes.byref(dst_layout), ctypes.byref(dst_batch), _ptr(d_slab), slab_bytes,
        _ptr(d_flags), flags_words, first_epoch, _stream(stream))


def topkv_layer_table_offsets(layout, table, num_requests):
    """Returns (status, offsets) with offsets a numpy int64 [num_layers + 1]."""
    import numpy as np
    off = np.zeros(table.num_layers + 1, dtype=np.int64)
    st = lib().topkv_layer_table_offsets(ctypes.byref(layout), ctypes.byref(table), num_requests,
                                         off.ctypes.data)
    return st, off


def topkv_pack_model_layers(first_layer, num_layers, src_pool, layout, batch, table, d_wire,
                            wire_capacity_bytes, stream=None):
    return lib().topkv_pack_model_layers(first_layer, num_layers, _ptr(src_pool), ctypes.byref(layout),
                                         ctypes.byref(batch), ctypes.byref(table), _ptr(d_wire),
                                         wire_capacity_bytes, _stream(stream))


def topkv_unpack_model_layers(first_layer, num_layers, dst_pool, layout, batch, table, d_wire,
                              wire_bytes, stream=None):
    return lib().topkv_unpack_model_layers(first_layer, num_layers, _ptr(dst_pool), ctypes.byref(layout),
                                           ctypes.byref(batch), ctypes.byref(table), _ptr(d_wire),
                                           wire_bytes, _stream(stream))


def topkv_pack_model_layers_to_host_pipelined(first_layer, num_layers, src_pool, layout, batch, table,
                                              h_pinned, host_capacity_bytes, d_staging,
                                              staging_capacity_bytes, layer_ready=None, layer_done=None,
                                              side_stream=None):
    return lib().topkv_pack_model_layers_to_host_pipelined(
        first_layer, num_layers, _ptr(src_pool), ctypes.byref(layout), ctypes.byref(batch),
        ctypes.byref(table), _ptr(h_pinned), host_capacity_bytes, _ptr(d_staging), staging_capacity_bytes,
        _events(layer_ready, num_layers), _events(layer_done, num_layers), _stream(side_stream))


def topkv_unpack_model_layers_from_host_pipelined(first_layer, num_layers, dst_pool, layout, batch, table,
                                                  h_pinned, host_bytes, d_staging,
                                                  staging_capacity_bytes, layer_ready=None,
                                                  layer_done=None, side_stream=None):
    return lib().topkv_unpack_model_layers_from_host_pipelined(
        first_layer, num_layers, _ptr(dst_pool), ctypes.byref(layout), ctypes.byref(batch),
        ctypes.byref(table), _ptr(h_pinned), host_bytes, _ptr(d_staging), staging_capacity_bytes,
        _events(layer_ready, num_layers), _events(layer_done, num_layers), _stream(side_stream))


def _two(ptrs, conv):
    arr = (c_void_p * 2)()
    arr[0], arr[1] = conv(ptrs[0]), conv(ptrs[1])
    return arr


def topkv_pack_layers_to_host_two_lanes(first_layer, num_layers, src_pool, layout, batch, h_pinned,
                                        host_capacity_bytes, d_stagings, staging_capacity_bytes,
                                        layer_ready=None, layer_done=None, side_streams=None):
    """d_stagings and side_streams: sequences of two device slabs / two streams."""
    return lib().topkv_pack_layers_to_host_two_lanes(
        first_layer, num_layers, _ptr(src_pool), ctypes.byref(layout), ctypes.byref(batch),
        _ptr(h_pinned), host_capacity_bytes, _two(d_stagings, _ptr), staging_capacity_bytes,
        _events(layer_ready, num_layers), _events(layer_done, num_layers), _two(side_streams, _stream))


def topkv_unpack_layers_from_host_two_lanes(first_layer, num_layers, dst_pool, layout, batch, h_pinned,
                                            host_bytes, d_stagings, staging_capacity_bytes,
                                            layer_ready=None, layer_done=None, side_streams=None):
    return lib().topkv_unpack_layers_from_host_two_lanes(
        first_layer, num_layers, _ptr(dst_pool), ctypes.byref(layout), ctypes.byref(batch),
        _ptr(h_pinned), host_bytes, _two(d_stagings, _ptr), staging_capacity_bytes,
        _events(layer_ready, num_layers), _events(layer_done, num_layers), _two(side_streams, _stream))


def topkv_pack_layer_to_host_noalloc(layer, src_pool, layout, batch, h_pinned,
                                     host_capacity_bytes, stream=None):
    """Staged pack-to-host for callers that may not allocate device memory: the staging slab
    is the library's built-in TOPKV_NOALLOC_STAGING_BYTES array. One slab per device, shared by
    all calls; make the first call on a device outside stream capture."""
    return lib().topkv_pack_layer_to_host_noalloc(
        layer, _ptr(src_pool), ctypes.byref(layout), ctypes.byref(batch), _ptr(h_pinned),
        host_capacity_bytes, _stream(stream))


def topkv_repage_layer(layer, src_pool, src_layout, src_batch, dst_pool, dst_layout, dst_batch,
                       stream=None):
    return lib().topkv_repage_layer(layer, _ptr(src_pool), ctypes.byref(src_layout),
                                    ctypes.byref(src_batch), _ptr(dst_pool),
                                    ctypes.byref(dst_layout), ctypes.byref(dst_batch),
                                    _stream(stream))


def topkv_header_fill(header, request_id, model_id, layout, seq_len, crc_k, crc_v):
    return lib().topkv_header_fill(ctypes.byref(header), request_id, model_id, ctypes.byref(layout),
                                   seq_len, crc_k, crc_v)


def topkv_header_check(header, layout, seq_len, crc_k, crc_v):
    return lib().topkv_header_check(ctypes.byref(header), ctypes.byref(layout), seq_len, crc_k,
                                    crc_v)


def topkv_crc64(h_data, nbytes=None):
    """Host CRC-64 of a bytes object or a numpy array."""
    if isinstance(h_data, (bytes, bytearray)):
        buf = (ctypes.c_char * len(h_data)).from_buffer_copy(h_data)
        return lib().topkv_crc64(ctypes.addressof(buf), len(h_data))
    return lib().topkv_crc64(_ptr(h_data), h_data.nbytes if nbytes is None else nbytes)


def topkv_crc_workspace_bytes(layout, num_requests, max_pages_per_req):
    return lib().topkv_crc_workspace_bytes(ctypes.byref(layout), num_requests, max_pages_per_req)


def topkv_crc_begin(layout, batch, d_workspace, workspace_bytes, stream=None):
    return lib().topkv_crc_begin(ctypes.byref(layout), ctypes.byref(batch), _ptr(d_workspace),
                                 workspace_bytes, _stream(stream))


def topkv_pack_layer_crc(layer, src_pool, layout, batch, d_wire, wire_capacity_bytes, d_workspace,
                         workspace_bytes, stream=None):
    return lib().topkv_pack_layer_crc(layer, _ptr(src_pool), ctypes.byref(layout),
                                      ctypes.byref(batch), _ptr(d_wire), wire_capacity_bytes,
                                      _ptr(d_workspace), workspace_bytes, _stream(stream))


def topkv_unpack_layer_crc(layer, dst_pool, layout, batch, d_wire, wire_bytes, d_workspace,
                           workspace_bytes, stream=None):
    return lib().topkv_unpack_layer_crc(layer, _ptr(dst_pool), ctypes.byref(layout),
                                        ctypes.byref(batch), _ptr(d_wire), wire_bytes,
                                        _ptr(d_workspace), workspace_bytes, _stream(stream))


def topkv_crc_finish(layout, batch, d_workspace, workspace_bytes, d_crc_out, stream=None):
    return lib().topkv_crc_finish(ctypes.byref(layout), ctypes.byref(batch), _ptr(d_workspace),
                                  workspace_bytes, _ptr(d_crc_out), _stream(stream))


def topkv_pack_layer_to_host_crc(layer, src_pool, layout, batch, h_pinned, host_capacity_bytes,
                                 d_staging, staging_capacity_bytes, d_workspace, workspace_bytes,
                                 stream=None):
    return lib().topkv_pack_layer_to_host_crc(
        layer, _ptr(src_pool), ctypes.byref(layout), ctypes.byref(batch), _ptr(h_pinned),
        host_capacity_bytes, _ptr(d_staging), staging_capacity_bytes, _ptr(d_workspace),
        workspace_bytes, _stream(stream))


def topkv_unpack_layer_from_host_crc(layer, dst_pool, layout, batch, h_pinned, host_bytes,
                                     d_staging, staging_capacity_bytes, d_workspace,
                                     workspace_bytes, stream=None):
    return lib().topkv_unpack_layer_from_host_crc(
        layer, _ptr(dst_pool), ctypes.byref(layout), ctypes.byref(batch), _ptr(h_pinned), host_bytes,
        _ptr(d_staging), staging_capacity_bytes, _ptr(d_workspace), workspace_bytes, _stream(stream))


def topkv_retry(attempt, retries=2, backoff_ms=100):
    """attempt: a Python callable returning a topkv status; §3.1's policy by default."""
    cb = RETRY_ATTEMPT(lambda _ctx: int(attempt()))
    return lib().topkv_retry(cb, None, retries, backoff_ms)


def topkv_build_plan(batch, d_cu_seq_lens, stream=None):
    return lib().topkv_build_plan(ctypes.byref(batch), _ptr(d_cu_seq_lens), _stream(stream))


def topkv_validate_batch_host(layout, num_requests, max_pages_per_req, h_block_table, h_seq_lens,
                              require_disjoint):
    return lib().topkv_validate_batch_host(ctypes.byref(layout), num_requests, max_pages_per_req,
                                           _ptr(h_block_table), _ptr(h_seq_lens),
                                           int(require_disjoint))


def topkv_layout_default_strides(layout):
    return lib().topkv_layout_default_strides(ctypes.byref(layout))


def topkv_wire_layer_bytes(layout, total_tokens):
    return lib().topkv_wire_layer_bytes(ctypes.byref(layout), total_tokens)


def topkv_kv_bytes(layout, seq_len):
    return lib().topkv_kv_bytes(ctypes.byref(layout), seq_len)


def topkv_kv_bytes_layered(layout, specs, seq_len):
    """specs: sequence of (kind, param) pairs, one per layer, or a ctypes array of
    topkv_layer_spec."""
    if not isinstance(specs, ctypes.Array):
        arr = (topkv_layer_spec * len(specs))()
        for i, (kind, param) in enumerate(specs):
            arr[i].kind, arr[i].param = kind, param
        specs = arr
    return lib().topkv_kv_bytes_layered(ctypes.byref(layout), ctypes.addressof(specs), seq_len)


def topkv_model_transfer_s(nbytes, bandwidth_bytes_per_s, setup_s=0.0):
    return lib().topkv_model_transfer_s(nbytes, bandwidth_bytes_per_s, setup_s)


def topkv_model_t_eff_s(t_last_s, t_xfer_s, t_rem_s):
    return lib().topkv_model_t_eff_s(t_last_s, t_xfer_s, t_rem_s)


def topkv_model_hidden_fraction(layers, t_layer_compute_s, t_xfer_total_s):
    return lib().topkv_model_hidden_fraction(layers, t_layer_compute_s, t_xfer_total_s)


def topkv_select_transport(source, target, cluster_has_rdma, override_mode=0):
    return lib().topkv_select_transport(ctypes.byref(source), ctypes.byref(target),
                                        int(bool(cluster_has_rdma)), override_mode)


def topkv_planning_rate(mode):
    return lib().topkv_planning_rate(mode)


def topkv_transport_name(mode):
    return lib().topkv_transport_name(mode).decode()


def topkv_strerror(status):
    return lib().topkv_strerror(status).decode()


def topkv_version():
    return lib().topkv_version()


def topkv_last_cuda_error():
    return lib().topkv_last_cuda_error()


def topkv_device_error_flags():
    return lib().topkv_device_error_flags()


def topkv_reset_device_error_flags():
    return lib().topkv_reset_device_error_flags()


def topkv_kernel_launch_count():
    return lib().topkv_kernel_launch_count()


def topkv_set_host_leg_ctas(ctas):
    return lib().topkv_set_host_leg_ctas(ctas)


def topkv_set_kernel_variant(variant):
    return lib().topkv_set_kernel_variant(variant)
