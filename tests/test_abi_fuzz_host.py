"""Host-side fuzz of the C-ABI entry points on a GPU-less box: random (mostly malformed)
layouts, batches, layer tables and links with fake addresses. Every call must come back with
a status from the documented set, and nothing may be launched: whatever is acceptable ends in
TOPKV_ERR_CUDA (there is no device here), everything else in its validation status."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import __graft_entry__ as entry
from paper_2607_28633_b200 import binding as tk

KNOWN = {tk.TOPKV_OK, tk.TOPKV_ERR_INVALID_ARG, tk.TOPKV_ERR_LAYER_RANGE, tk.TOPKV_ERR_ALIGNMENT,
         tk.TOPKV_ERR_CAPACITY, tk.TOPKV_ERR_UNSUPPORTED_LAYOUT, tk.TOPKV_ERR_CUDA}


class _Fake:
    def __init__(self, addr, shape):
        self._a, self.shape, self.ndim = addr, shape, len(shape)

    def data_ptr(self):
        return self._a


@pytest.fixture(scope="module", autouse=True)
def _built():
    entry.build()
    if torch.cuda.is_available():
        pytest.skip("fake addresses must never reach a real device")


def _draw(rng):
    """A valid descriptor pair (one of a few shapes) with zero, one or two random defects."""
    pick = lambda xs: xs[int(rng.integers(0, len(xs)))]
    L, F, H, D, E, P, pages = pick([(2, 2, 8, 128, 2, 16, 64), (5, 1, 1, 576, 2, 64, 40),
                                    (80, 2, 8, 128, 1, 16, 4096), (3, 2, 2, 64, 2, 256, 8),
                                    (4, 2, 1, 128, 2, 1, 100)])
    lo = tk.make_layout(L, F, H, D, E, P, pages, wire_order=pick([0, 0, 1]))
    R, maxp = pick([(4, 16), (1, 1), (16, 256), (1024, 2), (0, 4)])
    T = pick([-1, min(436, R * maxp * P), R * maxp * P])
    lo.wire_layer_stride = pick([0, T * F * H * D * E if T > 0 else 0])
    b = tk.make_batch(_Fake(0x10000, (R, maxp)), _Fake(0x20000, (R,)), T,
                      _Fake(0x30000, (R + 1,)) if rng.random() < 0.5 else None,
                      pick([0, 0, 1, 2, 3]), pick([0, 0, 0, 128]))
    for _ in range(int(pick([0, 0, 1, 1, 2]))):
        k = int(rng.integers(0, 16))
        if k == 0: lo.struct_size = 8
        elif k == 1: lo.kind = 5
        elif k == 2: lo.kv_factor = 3
        elif k == 3: lo.num_kv_heads = 0
        elif k == 4: lo.head_dim = 7
        elif k == 5: lo.page_tokens = 0
        elif k == 6: lo.wire_order = 9
        elif k == 7: lo.num_pool_pages = pick([0, -3])
        elif k == 8: lo.pool_token_stride += pick([8, 16, -16])
        elif k == 9: lo.pool_layer_stride += 16
        elif k == 10: lo.wire_layer_stride = pick([24, -16, (1 << 20) + 16])
        elif k == 11: lo.wire_plane_stride = pick([4096, 100])
        elif k == 12: b.num_requests = pick([-1, 1025, 9000])
        elif k == 13: b.max_pages_per_req = pick([-2, 0, 1 << 30])
        elif k == 14: b.struct_size = 12
        elif k == 15: b.total_tokens, b.flags, b.block_table = pick([(-5, 0, 0x10000), (1 << 40, 0, 0x10000),
                                                                  (T, 8, 0x10000), (T, 0, None)])
    return lo, b


@pytest.mark.parametrize("seed", range(6))
def test_entry_points_survive_random_descriptors(seed):
    rng = np.random.default_rng(seed)
    before = tk.topkv_kernel_launch_count()
    pool, wire, host, st, ws = 0x7000000, 0x9000000, 0xB000000, 0xC000000, 0xD000000
    seen = set()
    for it in range(250):
        lo, b = _draw(rng)
        layer = int(rng.integers(-1, 6))
        cap = int(rng.choice([0, 1 << 20, 1 << 40, -1]))
        off = int(rng.choice([0, 0, 0, 8, 16]))
        calls = [
            lambda: tk.topkv_pack_layer(layer, pool + off, lo, b, wire, cap),
            lambda: tk.topkv_unpack_layer(layer, pool, lo, b, wire + off, cap),
            lambda: tk.topkv_pack_layers(layer, int(rng.integers(0, 4)), pool, lo, b, wire, cap),
            lambda: tk.topkv_unpack_layers(layer, 2, pool, lo, b, wire, cap),
            lambda: tk.topkv_copy_vector_bytes(layer, 2, pool, lo, b, wire, cap),
            lambda: tk.topkv_pack_layer_to_host(layer, pool, lo, b, host, cap, st + off, cap),
            lambda: tk.topkv_unpack_layer_from_host(layer, pool, lo, b, host, cap, st, cap),
            lambda: tk.topkv_pack_layers_to_host_pipelined(layer, 2, pool, lo, b, host, cap, st, cap),
            lambda: tk.topkv_pack_layers_to_host_two_lanes(layer, 2, pool, lo, b, host, cap, [st, st + 4096],
                                                           cap, None, None, [0x100, 0x200]),
            lambda: tk.topkv_repage_layer(layer, pool, lo, b, wire, lo, b),
            lambda: tk.topkv_pack_layer_crc(layer, pool, lo, b, wire, cap, ws + off, cap),
            lambda: tk.topkv_unpack_layer_from_host_crc(layer, pool, lo, b, host, cap, st, cap, ws, cap),
            lambda: tk.topkv_crc_begin(lo, b, ws, cap),
            lambda: tk.topkv_pack_layer_linked(layer, pool, lo, b, wire, cap,
                                               tk.make_span_link(0xE000000, 1, 0xE100000 + off, 2)),
            lambda: tk.topkv_pack_layer_to_host_noalloc(layer, pool, lo, b, host, cap),
            lambda: tk.topkv_unpack_layer_linked(layer, pool, lo, b, wire, cap,
                                                 tk.make_span_link(0xE000000, 1, None, 0, int(rng.integers(0, 3)))),
            lambda: tk.topkv_relay_layers_linked(layer, int(rng.integers(0, 4)), pool, lo, b, pool + (1 << 30), lo,
                                                 b, wire, cap, 0xE000000, int(rng.choice([0, 64, 1 << 30])),
                                                 int(rng.integers(0, 5)), None),
            lambda: tk.topkv_unpack_layers_from_host_two_lanes(layer, 3, pool, lo, b, host, cap, [st, st + 4096],
                                                               cap, None, None, [0x100, 0x200]),
        ]
        for fn in calls:
            st_code = fn()
            assert st_code in KNOWN or st_code in (16, 32), st_code      # vector width is a value
            seen.add(st_code)
        # size helpers never crash either
        tk.topkv_wire_layer_bytes(lo, int(rng.integers(-2, 1 << 20)))
        tk.topkv_crc_workspace_bytes(lo, b.num_requests, b.max_pages_per_req)
        tk.topkv_span_link_words(lo, b)
        n, compact = tk.topkv_copy_grid_ctas(layer, pool, lo, b, wire, cap)
        assert n >= 0 or n in KNOWN, n
        kinds = [(int(rng.integers(0, 4)), int(rng.choice([0, 16, 128, 24, -1]))) for _ in range(4)]
        lens = np.asarray(rng.integers(0, 300, size=max(b.num_requests, 1)), dtype=np.int32)
        t = tk.make_layer_table(kinds, lens, 0xF000000, 0xF100000, 1 << 20, 4096, 64)
        code = tk.topkv_pack_model_layers(0, int(rng.integers(0, 6)), pool, lo, b, t, wire, cap)
        assert code in KNOWN, code
        code = tk.topkv_unpack_model_layers_from_host_pipelined(0, 4, pool, lo, b, t, host, cap, st, cap)
        assert code in KNOWN, code
    assert tk.topkv_kernel_launch_count() == before
    assert tk.TOPKV_ERR_CUDA in seen and tk.TOPKV_ERR_INVALID_ARG in seen      # both sides were reached
