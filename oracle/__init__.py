"""CPU oracle for the paged-KV pack / unpack path — TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the product library never does, and this package never imports the product.

The arithmetic lives in ``topkv_oracle.c`` (plain C, the definition written out); this
module compiles it with gcc on first use and wraps it for numpy arrays. Symbols follow the
paper: ``L`` layers, ``h_kv`` KV heads, ``d_h`` head dim, ``b_p`` bytes per element (Eq. 1),
``F`` = 2 for separate K and V tensors and 1 for a single MLA latent (§5.3).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

WIRE_TOKEN_KV = 0
WIRE_PLANAR = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "topkv_oracle.c")
_HDR = os.path.join(_HERE, "topkv_oracle.h")
_SO = os.path.join(_HERE, "libtopkv_oracle.so")


def build(force: bool = False) -> str:
    """Compiles the C oracle with gcc (no CUDA involved) and returns the path of the .so."""
    stale = (not os.path.exists(_SO)) or any(
        os.path.getmtime(p) > os.path.getmtime(_SO) for p in (_SRC, _HDR))
    if force or stale:
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-Wall", "-Wextra", "-shared", "-fPIC", "-o", tmp,
                               _SRC, "-lpthread"])
        os.replace(tmp, _SO)
    return _SO


class _Geom(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in (
        "L", "F", "h_kv", "d_h", "b_p", "P", "S_layer", "S_page", "S_kv", "S_tok", "S_head",
        "W_layer", "wire_order", "W_plane", "window")]


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, f64, vp = ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.oracle_kv_bytes.restype = i64
        lib.oracle_kv_bytes.argtypes = [i64] * 6
        lib.oracle_kv_bytes_layered.restype = i64
        lib.oracle_kv_bytes_layered.argtypes = [i64] * 6 + [vp, vp]
        lib.oracle_transfer_s.restype = f64
        lib.oracle_transfer_s.argtypes = [f64] * 3
        lib.oracle_t_eff.restype = f64
        lib.oracle_t_eff.argtypes = [f64] * 3
        lib.oracle_hidden_fraction.restype = f64
        lib.oracle_hidden_fraction.argtypes = [i64, f64, f64]
        gp = ctypes.POINTER(_Geom)
        for name in ("oracle_pack_ref", "oracle_unpack_ref"):
            fn = getattr(lib, name)
            fn.restype = None
            fn.argtypes = [gp, i64, vp, i64, i64, vp, vp, vp]
        for name in ("oracle_pack_rows", "oracle_unpack_rows"):
            fn = getattr(lib, name)
            fn.restype = None
            fn.argtypes = [gp, i64, vp, i64, i64, vp, vp, vp, ctypes.c_int]
        u64 = ctypes.c_uint64
        lib.oracle_crc64.restype = u64
        lib.oracle_crc64.argtypes = [vp, i64, u64]
        lib.oracle_crc64_iso.restype = u64
        lib.oracle_crc64_iso.argtypes = [vp, i64]
        lib.oracle_kv_plane_crc.restype = u64
        lib.oracle_kv_plane_crc.argtypes = [gp, vp, i64, i64, vp, vp, i64, i64]
        lib.oracle_kv_plane_crc_layered.restype = u64
        lib.oracle_kv_plane_crc_layered.argtypes = [gp, vp, i64, i64, vp, vp, i64, i64, vp]
        for name in ("oracle_pack_layered", "oracle_unpack_layered"):
            fn = getattr(lib, name)
            fn.restype = None
            fn.argtypes = [gp, i64, vp, vp, vp, i64, i64, vp, vp, vp, i64, i64, vp, vp]
        lib.oracle_layered_offsets.restype = None
        lib.oracle_layered_offsets.argtypes = [gp, i64, vp, vp, i64, vp, vp]
        cp, ci = ctypes.c_char_p, ctypes.c_int
        lib.oracle_select_transport.restype = ci
        lib.oracle_select_transport.argtypes = [ci, cp, ci, cp, cp, ci, cp, ci]
        lib.oracle_planning_rate.restype = f64
        lib.oracle_planning_rate.argtypes = [ci]
        _lib = lib
    return _lib


@dataclass
class Geom:
    """Shape of one paged pool and of the wire format. Strides are in bytes."""
    L: int
    F: int
    h_kv: int
    d_h: int
    b_p: int
    P: int
    num_pages: int
    wire_order: int = WIRE_TOKEN_KV
    S_layer: int = 0
    S_page: int = 0
    S_kv: int = 0
    S_tok: int = 0
    S_head: int = 0
    W_layer: int = 0
    W_plane: int = 0         # PLANAR: bytes between the planes of a slab (0 = adjacent)
    window: int = 0          # 0: every token; W > 0: the layer keeps only the last min(s, W)

    def __post_init__(self):
        if self.S_page == 0:  # default pool: pool[l][page][c][t][h][d], dim contiguous
            self.S_head = self.d_h * self.b_p
            self.S_tok = self.h_kv * self.S_head
            self.S_kv = self.P * self.S_tok
            self.S_page = self.F * self.S_kv
            self.S_layer = self.num_pages * self.S_page

    @property
    def row_bytes(self) -> int:
        return self.h_kv * self.d_h * self.b_p

    def wire_layer_bytes(self, T: int) -> int:
        """Bytes of one layer's wire slab for T tokens: every token carries F rows (§3.4)."""
        return T * self.F * self.row_bytes

    def pool_bytes(self) -> int:
        return self.L * self.S_layer

    def _c(self) -> _Geom:
        return _Geom(self.L, self.F, self.h_kv, self.d_h, self.b_p, self.P, self.S_layer,
                     self.S_page, self.S_kv, self.S_tok, self.S_head, self.W_layer,
                     self.wire_order, self.W_plane, self.window)

    def kept_tokens(self, sl) -> int:
        """Tokens of a batch that this layer keeps: sum of min(s, window) (all, if no window)."""
        sl = np.asarray(sl, dtype=np.int64)
        return int(sl.sum() if self.window <= 0 else np.minimum(sl, self.window).sum())


def kv_bytes(L: int, h_kv: int, d_h: int, s: int, b_p: int = 2, F: int = 2) -> int:
    """Eq. 1 (F = 2), or the MLA form without the K/V factor (F = 1, §5.3)."""
    return int(_load().oracle_kv_bytes(F, L, h_kv, d_h, s, b_p))


def kv_bytes_layered(h_kv: int, d_h: int, s: int, kinds, b_p: int = 2, F: int = 2) -> int:
    """Eq. 1 extended per layer kind (§2.2). ``kinds`` is one entry per layer: ("full",),
    ("window", W) or ("state", nbytes)."""
    code = {"full": 0, "window": 1, "state": 2}
    k = np.array([code[x[0]] for x in kinds], dtype=np.int64)
    prm = np.array([x[1] if len(x) > 1 else 0 for x in kinds], dtype=np.int64)
    lib = _load()
    return int(lib.oracle_kv_bytes_layered(F, h_kv, d_h, s, b_p, len(kinds), k.ctypes.data,
                                           prm.ctypes.data))


def transfer_s(S_bytes: float, B_bytes_per_s: float, L_m_s: float = 0.0) -> float:
    """Eq. 2."""
    return float(_load().oracle_transfer_s(S_bytes, B_bytes_per_s, L_m_s))


def t_eff(T_last: float, T_xfer: float, T_rem: float) -> float:
    """Eq. 3."""
    return float(_load().oracle_t_eff(T_last, T_xfer, T_rem))


def hidden_fraction(L: int, t_layer: float, T_xfer: float) -> float:
    """§5.2 worked example: min(1, (L-1)*t_layer / T_xfer)."""
    return float(_load().oracle_hidden_fraction(L, t_layer, T_xfer))


def _u8(a: np.ndarray, writable: bool) -> np.ndarray:
    assert a.dtype == np.uint8 and a.ndim == 1 and a.flags.c_contiguous
    if writable:
        assert a.flags.writeable
    return a


def _tables(bt: np.ndarray, sl: np.ndarray):
    bt = np.ascontiguousarray(bt, dtype=np.int32)
    sl = np.ascontiguousarray(sl, dtype=np.int32)
    assert bt.ndim == 2 and sl.ndim == 1 and bt.shape[0] == sl.shape[0]
    return bt, sl


def _check_extent(g: Geom, layer: int, pool: np.ndarray, bt, sl, wire: np.ndarray):
    """Guards the C loops: every offset they will form must lie inside the arrays."""
    T = g.kept_tokens(sl)
    need_wire = layer * g.W_layer + g.wire_layer_bytes(T)
    if g.W_plane > 0 and g.wire_order == WIRE_PLANAR:
        need_wire = layer * g.W_layer + (g.F - 1) * g.W_plane + T * g.row_bytes
    assert wire.size >= need_wire, (wire.size, need_wire)
    assert 0 <= layer < g.L
    for r in range(sl.shape[0]):
        n = -(-int(sl[r]) // g.P)
        assert n <= bt.shape[1]
        lo = 0 if g.window <= 0 or sl[r] <= g.window else (int(sl[r]) - g.window) // g.P
        if n:
            used = bt[r, lo:n]              # pages before the window are never touched
            assert used.min() >= 0
            last = (layer * g.S_layer + int(used.max()) * g.S_page + (g.F - 1) * g.S_kv
                    + (g.P - 1) * g.S_tok + (g.h_kv - 1) * g.S_head + g.d_h * g.b_p)
            assert pool.size >= last, (pool.size, last)


def pack(g: Geom, layer: int, pool: np.ndarray, bt: np.ndarray, sl: np.ndarray,
         wire: np.ndarray | None = None, impl: str = "ref", threads: int = 1) -> np.ndarray:
    """wire <- pool through the block table. ``pool`` is the uint8 view from layer 0's base,
    ``wire`` the uint8 view from layer 0's slab (allocated, zero-filled, if None)."""
    bt, sl = _tables(bt, sl)
    T = g.kept_tokens(sl)
    if wire is None:
        assert g.W_plane == 0, "spread planes need a caller-sized wire"
        wire = np.zeros(layer * g.W_layer + g.wire_layer_bytes(T), dtype=np.uint8)
    _u8(pool, False), _u8(wire, True)
    _check_extent(g, layer, pool, bt, sl, wire)
    cg = g._c()
    args = (ctypes.byref(cg), layer, pool.ctypes.data, sl.shape[0], bt.shape[1],
            bt.ctypes.data, sl.ctypes.data, wire.ctypes.data)
    if impl == "ref":
        _load().oracle_pack_ref(*args)
    elif impl == "rows":
        _load().oracle_pack_rows(*args, threads)
    else:
        raise ValueError(impl)
    return wire


def unpack(g: Geom, layer: int, pool: np.ndarray, bt: np.ndarray, sl: np.ndarray,
           wire: np.ndarray, impl: str = "ref", threads: int = 1) -> np.ndarray:
    """pool <- wire through the block table, in place; untouched pool bytes keep their value."""
    bt, sl = _tables(bt, sl)
    _u8(pool, True), _u8(wire, False)
    _check_extent(g, layer, pool, bt, sl, wire)
    cg = g._c()
    args = (ctypes.byref(cg), layer, pool.ctypes.data, sl.shape[0], bt.shape[1],
            bt.ctypes.data, sl.ctypes.data, wire.ctypes.data)
    if impl == "ref":
        _load().oracle_unpack_ref(*args)
    elif impl == "rows":
        _load().oracle_unpack_rows(*args, threads)
    else:
        raise ValueError(impl)
    return pool


# ---- layers of different kinds on the data path (§2.2) ----------------------------------------

_KIND = {"full": 0, "window": 1, "state": 2}


def _kinds(kinds):
    k = np.array([_KIND[x[0]] for x in kinds], dtype=np.int64)
    prm = np.array([x[1] if len(x) > 1 else 0 for x in kinds], dtype=np.int64)
    return k, prm


def layered_offsets(g: Geom, kinds, sl) -> np.ndarray:
    """Where every layer's slab starts on the wire of a model whose layers differ in kind
    (``kinds`` as for kv_bytes_layered, one entry per model layer); the last entry is the total,
    the sum over the requests of Eq. 1 per layer kind."""
    k, prm = _kinds(kinds)
    sl = np.ascontiguousarray(sl, dtype=np.int32)
    off = np.zeros(len(kinds) + 1, dtype=np.int64)
    cg = g._c()
    _load().oracle_layered_offsets(ctypes.byref(cg), len(kinds), k.ctypes.data, prm.ctypes.data,
                                   sl.shape[0], sl.ctypes.data, off.ctypes.data)
    return off


def _layered_args(g, kinds, pool, bt, sl, state_pool, S_state_layer, S_slot, slots, wire):
    k, prm = _kinds(kinds)
    bt, sl = _tables(bt, sl)
    n_att = int((k != 2).sum())
    assert n_att <= g.L, "the paged pool holds one layer per attention layer of the model"
    off = layered_offsets(g, kinds, sl)
    assert wire.size >= int(off[-1]), (wire.size, int(off[-1]))
    # extent guards for the C loops: every attention layer like a per-layer call
    for a, l in enumerate(np.flatnonzero(k != 2)):
        gl = Geom(**{**g.__dict__, "window": int(prm[l]) if k[l] == 1 else 0, "W_layer": 0, "W_plane": 0})
        _check_extent(gl, a, pool, bt, sl, wire[int(off[l]):])
    n_state = int((k == 2).sum())
    if n_state:
        slots = np.ascontiguousarray(slots, dtype=np.int32)
        assert slots.shape == sl.shape and slots.min() >= 0
        need = (n_state - 1) * S_state_layer + int(slots.max()) * S_slot + int(prm[k == 2].max())
        assert state_pool is not None and state_pool.size >= need, (need,)
        assert int(prm[k == 2].max()) <= S_slot
    else:
        slots = np.zeros(sl.shape, dtype=np.int32)
        state_pool = np.zeros(1, dtype=np.uint8) if state_pool is None else state_pool
    cg = g._c()
    return (cg, k, prm, bt, sl, slots, state_pool, off,
            (ctypes.byref(cg), len(kinds), k.ctypes.data, prm.ctypes.data, pool.ctypes.data,
             sl.shape[0], bt.shape[1], bt.ctypes.data, sl.ctypes.data, state_pool.ctypes.data,
             S_state_layer, S_slot, slots.ctypes.data, wire.ctypes.data))


def pack_layered(g: Geom, kinds, pool, bt, sl, state_pool=None, S_state_layer: int = 0,
                 S_slot: int = 0, slots=None, wire=None):
    """All layers of a model whose layers differ in kind onto one wire, slab after slab in model
    order. Returns (wire, offsets)."""
    off = layered_offsets(g, kinds, sl)
    if wire is None:
        wire = np.zeros(max(int(off[-1]), 1), dtype=np.uint8)
    _u8(pool, False), _u8(wire, True)
    keep = _layered_args(g, kinds, pool, bt, sl, state_pool, S_state_layer, S_slot, slots, wire)
    _load().oracle_pack_layered(*keep[-1])
    return wire, off


def unpack_layered(g: Geom, kinds, pool, bt, sl, wire, state_pool=None, S_state_layer: int = 0,
                   S_slot: int = 0, slots=None):
    """The inverse, in place: pool (and state_pool) <- wire; untouched bytes keep their value."""
    _u8(pool, True), _u8(wire, False)
    if state_pool is not None:
        _u8(state_pool, True)
    keep = _layered_args(g, kinds, pool, bt, sl, state_pool, S_state_layer, S_slot, slots, wire)
    _load().oracle_unpack_layered(*keep[-1])
    return pool


# ---- transport selection (Alg. 1) and planning rates (§3.3) -----------------------------------

MODES = {"nvlink": 1, "pcie": 2, "rdma": 3, "tcp": 4}
MODE_NAMES = {v: k for k, v in MODES.items()}


def select_transport(s, t, cluster_has_rdma: bool, override: str | None = None) -> str:
    """Alg. 1. ``s`` and ``t`` are (nvlink_domain, has_nvlink, node_ip) of the source and the
    target instance. Returns "nvlink", "pcie", "rdma" or "tcp"."""
    m = _load().oracle_select_transport(
        MODES[override] if override else 0, s[0].encode(), int(bool(s[1])), s[2].encode(),
        t[0].encode(), int(bool(t[1])), t[2].encode(), int(bool(cluster_has_rdma)))
    return MODE_NAMES[m]


def planning_rate(mode: str) -> float:
    """Bytes per second the orchestrator plans with for a mode (§3.3)."""
    return float(_load().oracle_planning_rate(MODES[mode]))


# ---- integrity check and header of the serialised cache (§3.4) --------------------------------

POLY_ISO_REFLECTED = 0xD800000000000000    # x^64 + x^4 + x^3 + x + 1 (CRC-64/GO-ISO), the reading taken
POLY_ECMA_REFLECTED = 0xC96C5795D7870F42   # ECMA-182 (CRC-64/XZ), used only to check the routine
HEADER_BYTES = 128
HEADER_MAGIC = b"KVCACHE1"


def crc64(data, poly_reflected: int = POLY_ISO_REFLECTED) -> int:
    """Reflected CRC-64, all-ones initial value, final inversion, bit by bit."""
    a = np.frombuffer(bytes(data), dtype=np.uint8) if not isinstance(data, np.ndarray) else data
    a = np.ascontiguousarray(a, dtype=np.uint8)
    return int(_load().oracle_crc64(a.ctypes.data, a.size, poly_reflected))


def kv_plane_crc(g: Geom, pool: np.ndarray, bt: np.ndarray, sl: np.ndarray, r: int, c: int,
                 layer_windows=None) -> int:
    """CRC-64 of the K (c = 0) or V (c = 1) tensor of request r in the order
    [layers][seq_len][kv_heads][head_dim], gathered from the paged pool. ``layer_windows``
    (one entry per layer, 0 = full) describes a model with windowed layers (§2.2): every layer
    contributes the tokens it keeps."""
    bt, sl = _tables(bt, sl)
    _u8(pool, False)
    cg = g._c()
    if layer_windows is not None:
        lw = np.ascontiguousarray(layer_windows, dtype=np.int64)
        assert lw.shape == (g.L,)
        return int(_load().oracle_kv_plane_crc_layered(
            ctypes.byref(cg), pool.ctypes.data, sl.shape[0], bt.shape[1], bt.ctypes.data,
            sl.ctypes.data, r, c, lw.ctypes.data))
    return int(_load().oracle_kv_plane_crc(ctypes.byref(cg), pool.ctypes.data, sl.shape[0],
                                           bt.shape[1], bt.ctypes.data, sl.ctypes.data, r, c))


def build_header(request_id: int, model_id: int, seq_len: int, g: Geom, crc_k: int, crc_v: int) -> bytes:
    """The fixed 128-byte header of §3.4: magic, request ID, model ID, tensor dimensions
    (sequence length, layers, KV heads, head dimension), tensor sizes, the two checksums.
    The paper fixes the content and the total size, not the field order or widths; the order
    below follows the order in which §3.4 lists the fields, little-endian, zero padded."""
    import struct
    plane = g.L * seq_len * g.h_kv * g.d_h * g.b_p
    body = struct.pack("<8sQQIIIIIIQQQQ", HEADER_MAGIC, request_id, model_id, seq_len, g.L, g.h_kv,
                       g.d_h, g.b_p, g.F, plane, plane if g.F == 2 else 0, crc_k,
                       crc_v if g.F == 2 else 0)
    assert len(body) == 80
    return body + bytes(HEADER_BYTES - len(body))
