"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle, byte for byte
(pure byte movement: the bar is bit-exact everywhere)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import oracle
from oracle import Geom
from paper_2607_28633_b200 import binding as tk
from paper_2607_28633_b200 import harness
from paper_2607_28633_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import __graft_entry__ as entry
    entry.build()
    return torch.device("cuda:0")


@pytest.fixture(autouse=True, params=[0, 1], ids=["vec", "bulk"])
def variant(request, dev):
    """Every test runs once per kernel family (vectorised load/store, bulk-async ring)."""
    prev = tk.topkv_set_kernel_variant(request.param)
    tk.check(tk.topkv_reset_device_error_flags())
    yield request.param
    tk.topkv_set_kernel_variant(prev)
    assert tk.topkv_device_error_flags() == 0


def _geom(spec, npages, L, wire_order, W_layer):
    return Geom(L=L, F=spec.F, h_kv=spec.H, d_h=spec.D, b_p=spec.E, P=spec.P, num_pages=npages,
                wire_order=wire_order, W_layer=W_layer)


# -------------------------------------------------------------------- cfg1, every option

@pytest.mark.parametrize("wire_order", [tk.TOPKV_WIRE_TOKEN_KV, tk.TOPKV_WIRE_PLANAR])
@pytest.mark.parametrize("use_plan", [True, False])
@pytest.mark.parametrize("know_T", [True, False])
def test_cfg1_pack_unpack(dev, wire_order, use_plan, know_T):
    w = harness.setup(wl.CFG1, dev, wire_order=wire_order, use_plan=use_plan)
    b, s = w.batch, w.batch.spec
    if not know_T:
        w.src_batch.total_tokens = -1
        w.dst_batch.total_tokens = -1
    g = _geom(s, b.num_pool_pages, s.L, wire_order, w.n_layer)
    src_h = w.src_pool.cpu().numpy()
    dst_h = w.dst_pool.cpu().numpy()
    stream = torch.cuda.Stream(dev)
    for layer in range(s.L):
        w.pack(layer, stream)
        w.unpack(layer, stream)
    stream.synchronize()
    want_wire = np.zeros(s.L * w.n_layer, dtype=np.uint8)
    for layer in range(s.L):
        oracle.pack(g, layer, src_h, b.src_block_table, b.seq_lens, wire=want_wire)
        oracle.unpack(g, layer, dst_h, b.dst_block_table, b.seq_lens, want_wire)
    assert np.array_equal(w.wire.cpu().numpy(), want_wire)
    assert np.array_equal(w.dst_pool.cpu().numpy(), dst_h)
    assert np.array_equal(w.src_pool.cpu().numpy(), src_h)          # source untouched


def test_build_plan(dev):
    for R in (1, 5, 255, 256, 257, 1000, 3000):
        sl = np.random.default_rng(R).integers(0, 9000, size=R).astype(np.int32)
        d_sl = torch.from_numpy(sl).to(dev)
        cu = torch.full((R + 1,), -7, dtype=torch.int64, device=dev)
        b = tk.make_batch(torch.zeros((R, 1), dtype=torch.int32, device=dev), d_sl)
        tk.check(tk.topkv_build_plan(b, cu))
        torch.cuda.synchronize()
        want = np.concatenate([[0], np.cumsum(sl.astype(np.int64))])
        assert np.array_equal(cu.cpu().numpy(), want)


# -------------------------------------------------------------------- random small cases

def _case(seed):
    """Random geometry, including strided pools, head-split rows, 16-byte-only alignment,
    1-byte and 2-byte elements, empty requests, full last pages and single tokens."""
    rng = np.random.default_rng(seed)
    F = int(rng.integers(1, 3))
    H = int(rng.choice([1, 2, 4, 8]))
    D = int(rng.choice([8, 24, 64, 72, 128, 576]))
    P = int(rng.choice([1, 3, 16, 64]))
    # element width b_p: 2 bytes (FP16 / bf16) or 1 byte (FP8), every pool style with both;
    # a 1-byte head must still be a multiple of 16 bytes
    E = 1 if (seed // 4) % 2 == 1 else 2
    if E == 1 and D % 16:
        D *= 2
    L = 2
    R = int(rng.integers(1, 7))
    sl = rng.integers(0, 4 * P + 2, size=R).astype(np.int32)
    if seed % 5 == 0:
        sl[rng.integers(0, R)] = 0
    if seed % 5 == 1:
        sl[rng.integers(0, R)] = P * int(rng.integers(1, 4))
    if seed % 7 == 2:
        sl[:] = 0
    pages = (sl + P - 1) // P
    maxp = max(int(pages.max()), 1) + int(rng.integers(0, 3))
    npages = int(pages.sum()) + int(rng.integers(1, 5))
    g = Geom(L=L, F=F, h_kv=H, d_h=D, b_p=E, P=P, num_pages=npages)
    style = seed % 4
    if style == 1:      # padded token stride (keeps heads contiguous)
        g.S_tok = H * D * E + 16 * int(rng.integers(1, 3))
        g.S_kv = P * g.S_tok
        g.S_page = F * g.S_kv + 32
        g.S_layer = npages * g.S_page
    elif style == 2:    # head-major inside the page: pool[l][page][c][h][t][d]
        g.S_tok = D * E
        g.S_head = P * g.S_tok
        g.S_kv = H * g.S_head
        g.S_page = F * g.S_kv
        g.S_layer = npages * g.S_page
    elif style == 3:    # plane-major pool: pool[l][c][page][t][h][d]
        g.S_page = P * g.S_tok
        g.S_kv = npages * g.S_page
        g.S_layer = F * g.S_kv + 16
    g.wire_order = int(rng.integers(0, 2))
    T = int(sl.sum())
    g.W_layer = g.wire_layer_bytes(T) + 16 * int(rng.integers(0, 3))
    bt_s = np.full((R, maxp), -1, dtype=np.int32)
    bt_d = np.full((R, maxp), -1, dtype=np.int32)
    ps, pd, pos = rng.permutation(npages), rng.permutation(npages), 0
    for r in range(R):
        bt_s[r, :pages[r]] = ps[pos:pos + pages[r]]
        bt_d[r, :pages[r]] = pd[pos:pos + pages[r]]
        pos += pages[r]
    return g, sl, bt_s, bt_d, rng


def _layout_from_geom(g: Geom):
    lo = tk.make_layout(g.L, g.F, g.h_kv, g.d_h, g.b_p, g.P, g.num_pages, wire_order=g.wire_order,
                        wire_layer_stride=g.W_layer,
                        kind=tk.TOPKV_KIND_GQA)
    lo.pool_layer_stride, lo.pool_page_stride, lo.pool_kv_stride = g.S_layer, g.S_page, g.S_kv
    lo.pool_token_stride, lo.pool_head_stride = g.S_tok, g.S_head
    lo.wire_plane_stride = g.W_plane
    return lo


@pytest.mark.parametrize("seed", range(40))
def test_random_geometries(dev, seed):
    g, sl, bt_s, bt_d, rng = _case(seed)
    lo = _layout_from_geom(g)
    T = int(sl.sum())
    guard = 64
    skew = 16 * (seed % 2)                     # odd seeds: 16-byte (not 32-byte) aligned bases
    src_h = rng.integers(0, 256, g.L * g.S_layer, dtype=np.uint8)
    fill_h = rng.integers(0, 256, g.L * g.S_layer, dtype=np.uint8)
    wire_len = g.L * g.W_layer + 32            # slack for the last layer's padding
    src_buf = torch.zeros(src_h.size + skew, dtype=torch.uint8, device=dev)
    src = src_buf[skew:]
    src.copy_(torch.from_numpy(src_h))
    dst_buf = torch.zeros(fill_h.size + skew, dtype=torch.uint8, device=dev)
    dst = dst_buf[skew:]
    dst.copy_(torch.from_numpy(fill_h))
    wire_buf = torch.full((guard + wire_len + guard + skew,), 0xA5, dtype=torch.uint8, device=dev)
    wire = wire_buf[guard + skew:guard + skew + wire_len]
    d_sl = torch.from_numpy(sl).to(dev)
    d_bs, d_bd = torch.from_numpy(bt_s).to(dev), torch.from_numpy(bt_d).to(dev)
    know_T = seed % 3 != 0
    bs = tk.make_batch(d_bs, d_sl, T if know_T else -1)
    bd = tk.make_batch(d_bd, d_sl, T if know_T else -1)
    assert tk.topkv_validate_batch_host(lo, len(sl), bt_s.shape[1], bt_s, sl, 0) == tk.TOPKV_OK
    assert tk.topkv_validate_batch_host(lo, len(sl), bt_d.shape[1], bt_d, sl, 1) == tk.TOPKV_OK
    for layer in range(g.L):
        tk.check(tk.topkv_pack_layer(layer, src, lo, bs, wire, wire.numel()))
        tk.check(tk.topkv_unpack_layer(layer, dst, lo, bd, wire, wire.numel()))
    torch.cuda.synchronize()
    want_wire = np.full(wire_len, 0xA5, dtype=np.uint8)
    want_dst = fill_h.copy()
    for layer in range(g.L):
        oracle.pack(g, layer, src_h, bt_s, sl, wire=want_wire)
        oracle.unpack(g, layer, want_dst, bt_d, sl, want_wire)
    got = wire_buf.cpu().numpy()
    assert (got[:guard + skew] == 0xA5).all() and (got[guard + skew + wire_len:] == 0xA5).all()
    assert np.array_equal(got[guard + skew:guard + skew + wire_len], want_wire)
    assert np.array_equal(dst.cpu().numpy(), want_dst)


def test_many_short_requests_inline_and_planned(dev):
    """R at the inline limit (each CTA derives the prefix sum) and beyond it (plan required)."""
    for R, planned in ((tk.TOPKV_MAX_INLINE_R, False), (tk.TOPKV_MAX_INLINE_R, True), (2500, True)):
        rng = np.random.default_rng(R + planned)
        g = Geom(L=1, F=2, h_kv=2, d_h=64, b_p=2, P=16, num_pages=2 * R + 5)
        sl = rng.integers(0, 33, size=R).astype(np.int32)
        pages = (sl + 15) // 16
        bt = np.full((R, 3), -1, dtype=np.int32)
        perm, pos = rng.permutation(g.num_pages), 0
        for r in range(R):
            bt[r, :pages[r]] = perm[pos:pos + pages[r]]
            pos += pages[r]
        T = int(sl.sum())
        for order in (0, 1):
            g.wire_order = order
            lo = _layout_from_geom(g)
            src_h = rng.integers(0, 256, g.S_layer, dtype=np.uint8)
            src = torch.from_numpy(src_h).to(dev)
            wire = torch.zeros(g.wire_layer_bytes(T), dtype=torch.uint8, device=dev)
            d_sl, d_bt = torch.from_numpy(sl).to(dev), torch.from_numpy(bt).to(dev)
            cu = None
            if planned:
                cu = torch.zeros(R + 1, dtype=torch.int64, device=dev)
                tk.check(tk.topkv_build_plan(tk.make_batch(d_bt, d_sl), cu))
            b = tk.make_batch(d_bt, d_sl, -1, cu)
            tk.check(tk.topkv_pack_layer(0, src, lo, b, wire, wire.numel()))
            torch.cuda.synchronize()
            want = oracle.pack(g, 0, src_h, bt, sl, impl="rows", threads=4)
            assert np.array_equal(wire.cpu().numpy(), want)
    # without a plan a batch beyond the inline limit is refused, nothing is launched
    b = tk.make_batch(d_bt, d_sl, -1, None)
    assert tk.topkv_pack_layer(0, src, lo, b, wire, wire.numel()) == tk.TOPKV_ERR_INVALID_ARG


@pytest.mark.parametrize("P,H,D", [(1, 1, 8), (2, 1, 64), (4, 2, 128), (16, 1, 128)])
def test_small_pages_many_per_cta(dev, P, H, D):
    """Pages far smaller than a CTA's span: long block-table rows are cut into several spans
    of up to 64 pages, with ragged ends in the middle of a span and of a page."""
    rng = np.random.default_rng(P * 1000 + D)
    R = 5
    sl = np.array([300 * P + 1, 0, 64 * P, 129 * P - 1, 7], dtype=np.int32)
    pages = (sl + P - 1) // P
    maxp = int(pages.max()) + 2
    npages = int(pages.sum()) + 9
    for order in (0, 1):
        for F in (1, 2):
            g = Geom(L=2, F=F, h_kv=H, d_h=D, b_p=2, P=P, num_pages=npages, wire_order=order)
            T = int(sl.sum())
            g.W_layer = g.wire_layer_bytes(T)
            bt_s = np.full((R, maxp), -1, dtype=np.int32)
            bt_d = np.full((R, maxp), -1, dtype=np.int32)
            ps, pd, pos = rng.permutation(npages), rng.permutation(npages), 0
            for r in range(R):
                bt_s[r, :pages[r]] = ps[pos:pos + pages[r]]
                bt_d[r, :pages[r]] = pd[pos:pos + pages[r]]
                pos += pages[r]
            lo = _layout_from_geom(g)
            src_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
            dst_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
            src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h).to(dev)
            wire = torch.zeros(2 * g.W_layer, dtype=torch.uint8, device=dev)
            d_sl = torch.from_numpy(sl).to(dev)
            d_bs, d_bd = torch.from_numpy(bt_s).to(dev), torch.from_numpy(bt_d).to(dev)
            bs = tk.make_batch(d_bs, d_sl, T)
            bd = tk.make_batch(d_bd, d_sl, T)
            want_wire = np.zeros(2 * g.W_layer, dtype=np.uint8)
            for layer in range(2):
                tk.check(tk.topkv_pack_layer(layer, src, lo, bs, wire, wire.numel()))
                tk.check(tk.topkv_unpack_layer(layer, dst, lo, bd, wire, wire.numel()))
                oracle.pack(g, layer, src_h, bt_s, sl, wire=want_wire, impl="rows")
                oracle.unpack(g, layer, dst_h, bt_d, sl, want_wire, impl="rows")
            torch.cuda.synchronize()
            assert np.array_equal(wire.cpu().numpy(), want_wire), (order, F)
            assert np.array_equal(dst.cpu().numpy(), dst_h), (order, F)


@pytest.mark.parametrize("path", ["per_layer", "layer_range", "checksummed"])
def test_unusable_tables_are_skipped_not_followed(dev, path, variant):
    """Device-side checks: a page id outside the pool, a length longer than its table row and
    lengths that overflow the wire slab raise status bits; the affected work is skipped, the
    rest is copied, and nothing outside the buffers is touched (guard bands, untouched pool)."""
    rng = np.random.default_rng(77)
    g = Geom(L=1, F=2, h_kv=2, d_h=64, b_p=2, P=16, num_pages=40)
    sl = np.array([40, 16, 33], dtype=np.int32)
    bt = np.array([[3, 9, 12, -1], [7, -1, -1, -1], [1, 2, 5, -1]], dtype=np.int32)
    T = int(sl.sum())
    lo = _layout_from_geom(g)
    src_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
    src = torch.from_numpy(src_h).to(dev)
    guard = 4096
    n = g.wire_layer_bytes(T)

    def run(bt_dev, sl_dev, total, cap):
        buf = torch.full((guard + n + guard,), 0xC3, dtype=torch.uint8, device=dev)
        d_bt, d_sl = torch.from_numpy(bt_dev).to(dev), torch.from_numpy(sl_dev).to(dev)
        b = tk.make_batch(d_bt, d_sl, total)
        tk.check(tk.topkv_reset_device_error_flags())
        if path == "per_layer":
            tk.check(tk.topkv_pack_layer(0, src, lo, b, buf[guard:], cap))
        elif path == "layer_range":
            tk.check(tk.topkv_pack_layers(0, 1, src, lo, b, buf[guard:], cap))
        else:
            nws = tk.topkv_crc_workspace_bytes(lo, len(sl_dev), bt_dev.shape[1])
            ws = torch.zeros(nws, dtype=torch.uint8, device=dev)
            tk.check(tk.topkv_crc_begin(lo, b, ws, nws))
            tk.check(tk.topkv_pack_layer_crc(0, src, lo, b, buf[guard:], cap, ws, nws))
        flags = tk.topkv_device_error_flags()
        out = buf.cpu().numpy()
        assert (out[:guard] == 0xC3).all() and (out[guard + n:] == 0xC3).all()
        return flags, out[guard:guard + n]

    if path == "checksummed" and variant == 1:
        pytest.skip("the checksumming copy has one kernel family")
    want = oracle.pack(g, 0, src_h, bt, sl)
    flags, got = run(bt, sl, T, n)
    assert flags == 0 and np.array_equal(got, want)
    # (a) a page id outside the pool: that page's 16 tokens are skipped, all others copied
    bad = bt.copy(); bad[0, 1] = 40
    flags, got = run(bad, sl, T, n)
    assert flags == 2
    lo_b, hi_b = 16 * g.F * g.row_bytes, 32 * g.F * g.row_bytes     # tokens 16..31 of request 0
    assert np.array_equal(got[:lo_b], want[:lo_b]) and np.array_equal(got[hi_b:], want[hi_b:])
    assert (got[lo_b:hi_b] == 0xC3).all()
    bad = bt.copy(); bad[2, 0] = -5
    flags, _ = run(bad, sl, T, n)
    assert flags == 2
    # (b) a length longer than its block-table row (4 columns = 64 tokens)
    long = sl.copy(); long[1] = 65
    flags, _ = run(bt, long, T, n)
    assert flags & 2
    if path != "checksummed":                # the same under a window, however far past the row the length is
        for s_long in (65, 200):
            long[1] = s_long
            d_bt, d_sl = torch.from_numpy(bt).to(dev), torch.from_numpy(long).to(dev)
            buf = torch.full((n + 4096,), 0xC3, dtype=torch.uint8, device=dev)
            tk.check(tk.topkv_reset_device_error_flags())
            tk.check(tk.topkv_pack_layer(0, src, lo, tk.make_batch(d_bt, d_sl, -1, None, 0, 16), buf, n))
            assert tk.topkv_device_error_flags() & 2, s_long
    # (c) device lengths that need more wire than the slab has
    more = sl.copy(); more[2] = 48
    bt48 = bt.copy(); bt48[2, 2] = 5
    flags, _ = run(bt48, more, T, n)
    assert flags & 4
    flags, _ = run(bt48, more, -1, n)                               # unknown T: capacity rules
    assert flags & 4
    tk.check(tk.topkv_reset_device_error_flags())


@pytest.mark.parametrize("R", [1, 7, 33, 256, 257])
def test_compact_grid_for_ragged_batches(dev, R, variant):
    """One long request among many short and empty ones: the block-table row is long, most of
    its columns are empty for most requests, and with the total stated the grid holds one CTA
    per span that can hold tokens (total / span + R) instead of one per column, each CTA finding
    its request from the lengths (up to 256 requests; beyond that, and with an unknown total,
    one CTA per column as before). Pack and unpack against the oracle for every form; a stated
    total below what the device lengths add up to raises the wire bit and touches nothing
    outside the slab."""
    rng = np.random.default_rng(1000 + R)
    for P, H, D in ((16, 8, 128), (4, 1, 64)):
        F, E = 2, 2
        sl = rng.integers(0, 3 * P + 2, size=R).astype(np.int32)
        if R > 2:
            sl[rng.integers(0, R, size=max(1, R // 5))] = 0
        sl[rng.integers(0, R)] = 645                               # one long request: a long row
        pages = (sl + P - 1) // P
        maxp = int(pages.max()) + 2
        npages = int(pages.sum()) + 3
        g = Geom(L=2, F=F, h_kv=H, d_h=D, b_p=E, P=P, num_pages=npages)
        T = int(sl.sum())
        g.W_layer = g.wire_layer_bytes(T) + 32
        bt_s = np.full((R, maxp), -1, dtype=np.int32)
        bt_d = np.full((R, maxp), -1, dtype=np.int32)
        ps, pd, pos = rng.permutation(npages), rng.permutation(npages), 0
        for r in range(R):
            bt_s[r, :pages[r]] = ps[pos:pos + pages[r]]
            bt_d[r, :pages[r]] = pd[pos:pos + pages[r]]
            pos += pages[r]
        lo = _layout_from_geom(g)
        src_h = rng.integers(0, 256, g.L * g.S_layer, dtype=np.uint8)
        dst_h0 = rng.integers(0, 256, g.L * g.S_layer, dtype=np.uint8)
        src = torch.from_numpy(src_h).to(dev)
        d_sl = torch.from_numpy(sl).to(dev)
        d_bs, d_bd = torch.from_numpy(bt_s).to(dev), torch.from_numpy(bt_d).to(dev)
        want = np.full(g.L * g.W_layer + 64, 0x3C, dtype=np.uint8)
        want_dst = dst_h0.copy()
        for layer in range(g.L):
            oracle.pack(g, layer, src_h, bt_s, sl, wire=want)
            oracle.unpack(g, layer, want_dst, bt_d, sl, want)
        for total in (T, -1):
            cu = None
            wire = torch.full((g.L * g.W_layer + 64,), 0x3C, dtype=torch.uint8, device=dev)
            dst = torch.from_numpy(dst_h0).to(dev)
            # the compact grid is taken by launches that may read their tables before they wait
            # for the kernel before them; the tables here were uploaded long before
            ts = tk.TOPKV_FLAG_TABLES_SETTLED
            bs, bd = tk.make_batch(d_bs, d_sl, total, cu, ts), tk.make_batch(d_bd, d_sl, total, cu, ts)
            for layer in range(g.L):
                tk.check(tk.topkv_pack_layer(layer, src, lo, bs, wire, wire.numel()))
                tk.check(tk.topkv_unpack_layer(layer, dst, lo, bd, wire, wire.numel()))
            torch.cuda.synchronize()
            assert tk.topkv_device_error_flags() == 0
            assert np.array_equal(wire.cpu().numpy(), want), (P, total)
            assert np.array_equal(dst.cpu().numpy(), want_dst), (P, total)
            # both layers in one launch
            wire.fill_(0x3C)
            tk.check(tk.topkv_pack_layers(0, g.L, src, lo, bs, wire, wire.numel()))
            torch.cuda.synchronize()
            assert np.array_equal(wire.cpu().numpy(), want), (P, total, "range")
        # a total that understates the device lengths: reported, nothing outside the slab touched
        if T > 4 * P:
            short = T - 3 * P
            n_short = g.wire_layer_bytes(short)
            guard = 4096
            buf = torch.full((guard + n_short + guard,), 0xC3, dtype=torch.uint8, device=dev)
            lo1 = _layout_from_geom(g)
            lo1.wire_layer_stride = 0
            tk.check(tk.topkv_reset_device_error_flags())
            tk.check(tk.topkv_pack_layer(0, src, lo1, tk.make_batch(d_bs, d_sl, short, None,
                                                                    tk.TOPKV_FLAG_TABLES_SETTLED),
                                         buf[guard:], n_short))
            assert tk.topkv_device_error_flags() & 4
            out = buf.cpu().numpy()
            assert (out[:guard] == 0xC3).all() and (out[guard + n_short:] == 0xC3).all()
            tk.check(tk.topkv_reset_device_error_flags())


# -------------------------------------------------------------------- benchmark shapes

def _check_layers(w, layers, dev, threads=8):
    """pack + unpack the given layers and compare each slab with the oracle."""
    b, s = w.batch, w.batch.spec
    g = _geom(s, b.num_pool_pages, 1, w.layout.wire_order, 0)      # one-slab view
    slab = w.slab_bytes
    for layer in layers:
        src_h = harness.layer_slab_to_numpy(w.src_pool, slab, layer)
        dst_h = harness.layer_slab_to_numpy(w.dst_pool, slab, layer)
        w.pack(layer)
        w.unpack(layer)
        torch.cuda.synchronize()
        want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=threads)
        got = w.wire[layer * w.n_layer:(layer + 1) * w.n_layer].cpu().numpy()
        assert np.array_equal(got, want), f"pack layer {layer}"
        oracle.unpack(g, 0, dst_h, b.dst_block_table, b.seq_lens, want, impl="rows", threads=threads)
        assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, slab, layer), dst_h), \
            f"unpack layer {layer}"


@pytest.mark.parametrize("name", ["cfg2", "cfg4"])
def test_bench_shapes_reduced_layers(dev, name):
    spec = wl.ALL[name]
    w = harness.setup(spec, dev, layers=3)
    assert w.batch.spec.R == spec.R
    _check_layers(w, range(3), dev)
    del w
    torch.cuda.empty_cache()


def _oracle_token(spec, page_host, t):
    """The wire bytes of token t of one page, computed by the oracle on a one-page problem."""
    g = Geom(L=1, F=spec.F, h_kv=spec.H, d_h=spec.D, b_p=spec.E, P=spec.P, num_pages=1)
    wire = oracle.pack(g, 0, page_host, np.zeros((1, 1), dtype=np.int32),
                       np.array([t + 1], dtype=np.int32))
    return wire[t * spec.tok_bytes:(t + 1) * spec.tok_bytes]


@pytest.mark.parametrize("name", ["cfg2", "cfg3", "cfg4"])
def test_full_size_in_the_bench_launch_configuration(dev, name, variant):
    """The workloads at full size, all layers resident, issued as bench.py issues them (one
    stream, TOPKV_FLAG_OVERLAP_PREVIOUS after the first layer of each phase). EVERY layer's wire
    slab and EVERY layer's destination slab (untouched bytes included) is compared in full with
    the oracle; a few sampled tokens are also checked one by one through a one-page oracle
    problem, which ties the batch-level comparison to the per-token definition.
    Once per shape the checksummed chain runs beside it, again as bench.py issues it (begin, one
    checksummed copy per layer with the flag after the first, finish; pack, then unpack, into a
    second wire and a second destination pool): its slabs are compared with the same oracle
    slabs, and the CRC-64 of every request's K and V tensor over ALL layers, from both
    directions, with the oracle's bit-by-bit CRC of the tensor gathered from the source pool."""
    from concurrent.futures import ThreadPoolExecutor
    spec = wl.ALL[name]
    w = harness.setup(spec, dev)
    b, s = w.batch, spec
    stream = torch.cuda.Stream(dev)
    g1 = _geom(s, b.num_pool_pages, 1, 0, 0)
    dst_before = w.dst_pool.clone()                       # on the device: a host copy is 20 GiB
    for layer in range(s.L):
        w.pack(layer, stream, overlap=layer > 0)
    for layer in range(s.L):
        w.unpack(layer, stream, overlap=layer > 0)
    stream.synchronize()
    assert tk.topkv_device_error_flags() == 0
    with_crc = variant == 0
    if with_crc:
        wire2 = torch.zeros_like(w.wire)
        dst2 = dst_before.clone()
        nws = tk.topkv_crc_workspace_bytes(w.layout, s.R, b.max_pages_per_req)
        ws = torch.empty(nws, dtype=torch.uint8, device=dev)
        crcs = {}
        for what, fn, pool, batch in (("pack", tk.topkv_pack_layer_crc, w.src_pool, w.src_batch),
                                      ("unpack", tk.topkv_unpack_layer_crc, dst2, w.dst_batch)):
            crc = torch.zeros(s.R * s.F, dtype=torch.int64, device=dev)
            tk.check(tk.topkv_crc_begin(w.layout, batch, ws, nws, stream))
            for layer in range(s.L):
                tk.check(fn(layer, pool, w.layout, w._flagged(batch, layer > 0), wire2, wire2.numel(), ws,
                            nws, stream))
            tk.check(tk.topkv_crc_finish(w.layout, batch, ws, nws, crc, stream))
            stream.synchronize()
            crcs[what] = crc.cpu().numpy().view(np.uint64).reshape(s.R, s.F)
        assert tk.topkv_device_error_flags() == 0
        pool_h = np.empty(s.L * w.slab_bytes, dtype=np.uint8)      # the whole source pool, for the CRCs
    for layer in range(s.L):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
        want = oracle.pack(g1, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=16)
        got = w.wire[layer * w.n_layer:(layer + 1) * w.n_layer].cpu().numpy()
        assert np.array_equal(got, want), f"pack layer {layer}"
        dst_h = harness.layer_slab_to_numpy(dst_before, w.slab_bytes, layer)
        oracle.unpack(g1, 0, dst_h, b.dst_block_table, b.seq_lens, want, impl="rows", threads=16)
        assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer), dst_h), \
            f"unpack layer {layer}"
        if with_crc:
            got2 = wire2[layer * w.n_layer:(layer + 1) * w.n_layer].cpu().numpy()
            assert np.array_equal(got2, want), f"checksummed pack, layer {layer}"
            assert np.array_equal(harness.layer_slab_to_numpy(dst2, w.slab_bytes, layer), dst_h), \
                f"checksummed unpack, layer {layer}"
            pool_h[layer * w.slab_bytes:(layer + 1) * w.slab_bytes] = src_h
    if with_crc:
        gL = _geom(s, b.num_pool_pages, s.L, 0, 0)
        pairs = [(r, c) for r in range(s.R) for c in range(s.F)]
        with ThreadPoolExecutor(max_workers=16) as ex:     # the C routine runs without the GIL
            want_crc = list(ex.map(lambda rc: oracle.kv_plane_crc(gL, pool_h, b.src_block_table, b.seq_lens,
                                                                  rc[0], rc[1]), pairs))
        for (r, c), v in zip(pairs, want_crc):
            assert int(crcs["pack"][r, c]) == v, ("pack", r, c)
            assert int(crcs["unpack"][r, c]) == v, ("unpack", r, c)
        del wire2, dst2, ws, pool_h
    rng = np.random.default_rng(7)
    cu = np.concatenate([[0], np.cumsum(b.seq_lens.astype(np.int64))])
    for layer in rng.choice(s.L, size=min(8, s.L), replace=False):
        layer = int(layer)
        r = int(rng.integers(0, s.R))
        i = int(rng.integers(0, b.seq_lens[r]))
        wo = layer * w.n_layer + (int(cu[r]) + i) * s.tok_bytes
        got_wire = w.wire[wo:wo + s.tok_bytes].cpu().numpy()
        for pool, table in ((w.src_pool, b.src_block_table), (w.dst_pool, b.dst_block_table)):
            po = layer * w.slab_bytes + int(table[r, i // s.P]) * s.page_bytes
            page_h = pool[po:po + s.page_bytes].cpu().numpy()
            assert np.array_equal(_oracle_token(s, page_h, i % s.P), got_wire), (layer, r, i)
    del w, dst_before
    torch.cuda.empty_cache()


def test_cfg3_host_leg_full_size(dev, variant):
    """Configuration 3 as stated: all 80 layers of the 70B-shaped cache packed to pinned host
    memory over PCIe (staged form, one 128 MiB slab per layer, 10 GiB in all), then unpacked from
    the host into the destination pool. Every pinned slab and every destination slab is
    compared in full with the oracle. In the vectorised family the same layers then go through
    the form bench.py times as its end-to-end number: the pipelined relay of the two two-lane
    calls (each direction alternating between two streams and two staging slabs, the receiver's
    layer_ready events being the sender's layer_done), compared with the same oracle slabs."""
    spec = wl.CFG3
    w = harness.setup(spec, dev, need_wire=False)
    b, s = w.batch, spec
    g1 = _geom(s, b.num_pool_pages, 1, 0, 0)
    n = w.n_layer
    try:
        pinned = torch.empty(s.L * n, dtype=torch.uint8).pin_memory()
    except RuntimeError:
        pytest.skip("this box refuses 10 GiB of pinned memory")
    pinned.fill_(0x6B)
    dst_before = w.dst_pool.clone()
    staging = torch.empty(n, dtype=torch.uint8, device=dev)
    stream = torch.cuda.Stream(dev)
    stream.wait_stream(torch.cuda.current_stream(dev))
    for layer in range(s.L):
        w.pack_to_host(layer, pinned, staging, stream)
    for layer in range(s.L):
        w.unpack_from_host(layer, pinned, staging, stream)
    stream.synchronize()
    assert tk.topkv_device_error_flags() == 0
    relay = variant == 0
    if relay:   # keep the first form's results aside and run the relay into the same buffers
        host_seq = pinned.clone()                       # pageable copy
        dst_seq = w.dst_pool.clone()
        w.dst_pool.copy_(dst_before)
        pinned.fill_(0x6B)
        tx = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
        rx = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
        st_tx = [staging, torch.empty_like(staging)]
        st_rx = [torch.empty_like(staging), torch.empty_like(staging)]
        sent = [torch.cuda.Event() for _ in range(s.L)]
        torch.cuda.synchronize()
        tk.check(tk.topkv_pack_layers_to_host_two_lanes(
            0, s.L, w.src_pool, w.layout, w.src_batch, pinned, s.L * n, st_tx, n, None, sent, tx))
        tk.check(tk.topkv_unpack_layers_from_host_two_lanes(
            0, s.L, w.dst_pool, w.layout, w.dst_batch, pinned, s.L * n, st_rx, n, sent, None, rx))
        torch.cuda.synchronize()
        assert tk.topkv_device_error_flags() == 0
    else:
        host_seq, dst_seq = pinned, w.dst_pool
    host, host1 = pinned.numpy(), host_seq.numpy()
    for layer in range(s.L):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
        want = oracle.pack(g1, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=16)
        assert np.array_equal(host1[layer * n:(layer + 1) * n], want), f"to host, layer {layer}"
        dst_h = harness.layer_slab_to_numpy(dst_before, w.slab_bytes, layer)
        oracle.unpack(g1, 0, dst_h, b.dst_block_table, b.seq_lens, want, impl="rows", threads=16)
        assert np.array_equal(harness.layer_slab_to_numpy(dst_seq, w.slab_bytes, layer), dst_h), \
            f"from host, layer {layer}"
        if relay:
            assert np.array_equal(host[layer * n:(layer + 1) * n], want), f"relay to host, layer {layer}"
            assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer), dst_h), \
                f"relay from host, layer {layer}"
    del w, dst_before, pinned, staging, host_seq, dst_seq
    torch.cuda.empty_cache()


def test_fp8_elements_bench_shape(dev):
    """1-byte elements (b_p = 1 in Eq. 1) on the 70B batch: 8 x 128 x 1 = 1 KiB rows, 32 KiB
    pages, two layers, compared in full with the oracle built with b_p = 1."""
    from dataclasses import replace
    spec = replace(wl.with_layers(wl.CFG3, 2), E=1, name="cfg3_fp8")
    w = harness.setup(spec, dev, fill_dst=True)
    assert w.layout.elem_bytes == 1 and w.n_layer == 8 * 4096 * 2 * 1024
    stream = torch.cuda.Stream(dev)
    stream.wait_stream(torch.cuda.current_stream(dev))
    dst_before = [harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l) for l in range(2)]
    for layer in range(2):
        w.pack(layer, stream, overlap=layer > 0)
    for layer in range(2):
        w.unpack(layer, stream, overlap=layer > 0)
    stream.synchronize()
    b = w.batch
    g1 = _geom(spec, b.num_pool_pages, 1, 0, 0)
    assert g1.b_p == 1 and g1.row_bytes == 1024
    for layer in range(2):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
        want = oracle.pack(g1, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=16)
        assert np.array_equal(w.wire[layer * w.n_layer:(layer + 1) * w.n_layer].cpu().numpy(), want)
        oracle.unpack(g1, 0, dst_before[layer], b.dst_block_table, b.seq_lens, want, impl="rows", threads=16)
        assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer), dst_before[layer])
    del w
    torch.cuda.empty_cache()


@pytest.mark.parametrize("pieces", [1, 16])
def test_constant_state_layer_as_a_one_row_layout(dev, pieces):
    """A linear-attention layer carries a fixed-size state per request instead of per-token
    rows (§2.2). It goes through the same calls as a one-plane layout with one-token pages:
    F = 1, H = 1, P = 1, and either the whole state slot as ONE page of `state` bytes
    (pieces = 1) or the slot described as `pieces` consecutive pages of state / pieces bytes
    (table row = slot * pieces + 0 .. pieces - 1), so that `pieces` CTAs share a large state.
    The bytes shipped per request and layer are exactly the ("state", n) term of Eq. 1 per layer
    kind, and they equal the oracle's pack of that geometry."""
    rng = np.random.default_rng(31 + pieces)
    state = 32 * 128 * 128 * 2                            # 32 heads of 128 x 128 bf16 = 1 MiB
    L, R, slots = 3, 5, 9                                 # state layers, requests, pool slots
    assert oracle.kv_bytes_layered(1, 1, 4096, [("state", state)] * L) == L * state
    E = 2
    g = Geom(L=L, F=1, h_kv=1, d_h=state // pieces // E, b_p=E, P=1, num_pages=slots * pieces)
    assert g.S_page * pieces == state and g.S_layer == slots * state
    sl = np.full(R, pieces, dtype=np.int32)               # every request has exactly one state
    sub = np.arange(pieces, dtype=np.int32)[None, :]
    slot_s = rng.permutation(slots)[:R].astype(np.int32).reshape(R, 1) * pieces + sub
    slot_d = rng.permutation(slots)[:R].astype(np.int32).reshape(R, 1) * pieces + sub
    T = int(sl.sum())
    g.W_layer = g.wire_layer_bytes(T)
    assert g.W_layer == R * state                         # R states per layer on the wire
    lo = _layout_from_geom(g)
    assert tk.topkv_kv_bytes_layered(lo, [(tk.TOPKV_LAYER_STATE, state)] * L, 4096) == L * state
    assert tk.topkv_wire_layer_bytes(lo, T) == R * state
    src_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
    dst_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
    src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h).to(dev)
    wire = torch.zeros(L * g.W_layer, dtype=torch.uint8, device=dev)
    d_sl = torch.from_numpy(sl).to(dev)
    bs = tk.make_batch(torch.from_numpy(slot_s).to(dev), d_sl, T)
    bd = tk.make_batch(torch.from_numpy(slot_d).to(dev), d_sl, T)
    want = np.zeros(L * g.W_layer, dtype=np.uint8)
    for layer in range(L):
        tk.check(tk.topkv_pack_layer(layer, src, lo, bs, wire, wire.numel()))
        tk.check(tk.topkv_unpack_layer(layer, dst, lo, bd, wire, wire.numel()))
        oracle.pack(g, layer, src_h, slot_s, sl, wire=want, impl="rows")
        oracle.unpack(g, layer, dst_h, slot_d, sl, want, impl="rows")
    torch.cuda.synchronize()
    assert np.array_equal(wire.cpu().numpy(), want)
    assert np.array_equal(dst.cpu().numpy(), dst_h)
    # the wire is the requests' states in request order: the plain definition, written out
    for layer in range(L):
        for r in range(R):
            a = layer * g.S_layer + int(slot_s[r, 0]) * g.S_page
            assert np.array_equal(want[layer * g.W_layer + r * state:][:state], src_h[a:a + state])


def test_overlapped_launches_keep_results_and_order(dev):
    """TOPKV_FLAG_OVERLAP_PREVIOUS on every layer after the first: results are unchanged, and
    work enqueued after the chain (a copy on the same stream) sees all of it."""
    spec = wl.with_layers(wl.CFG2, 6)
    w = harness.setup(spec, dev)
    b, s = w.batch, spec
    g = _geom(s, b.num_pool_pages, 1, 0, 0)
    stream = torch.cuda.Stream(dev)
    host_wire = torch.empty(w.wire.numel(), dtype=torch.uint8).pin_memory()
    host_dst = torch.empty(w.dst_pool.numel(), dtype=torch.uint8).pin_memory()
    dst_before = [harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l) for l in range(s.L)]
    with torch.cuda.stream(stream):
        for l in range(s.L):
            w.pack(l, stream, overlap=l > 0)
        host_wire.copy_(w.wire, non_blocking=True)          # right behind the chain
        for l in range(s.L):
            w.unpack(l, stream, overlap=l > 0)              # unpack(0) waits for the packs
        host_dst.copy_(w.dst_pool, non_blocking=True)
    stream.synchronize()
    for l in range(s.L):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, l)
        want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
        assert np.array_equal(host_wire[l * w.n_layer:(l + 1) * w.n_layer].numpy(), want), l
        oracle.unpack(g, 0, dst_before[l], b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
        assert np.array_equal(host_dst[l * w.slab_bytes:(l + 1) * w.slab_bytes].numpy(),
                              dst_before[l]), l
    del w
    torch.cuda.empty_cache()


def test_settled_tables_flag_keeps_data_dependences(dev):
    """TOPKV_FLAG_TABLES_SETTLED: the kernel reads its tables while its predecessor drains but
    touches data only after it. A chain in which every kernel depends on the DATA of the one
    just before it (pack of layer l into ONE shared wire slab, then unpack of that slab, for
    every layer, then a copy right behind) gives the oracle's result; empty batches and a
    following kernel without the flag keep stream order too."""
    spec = wl.with_layers(wl.CFG2, 6)
    w = harness.setup(spec, dev, need_wire=False)
    b, s = w.batch, spec
    g = _geom(s, b.num_pool_pages, 1, 0, 0)
    stream = torch.cuda.Stream(dev)
    flag = tk.TOPKV_FLAG_TABLES_SETTLED
    bs = tk.make_batch(w.src_bt, w.seq_lens, b.total_tokens, w.cu, flag)
    bd = tk.make_batch(w.dst_bt, w.seq_lens, b.total_tokens, w.cu, flag)
    lo1 = tk.make_layout(s.L, s.F, s.H, s.D, s.E, s.P, b.num_pool_pages)   # wire_layer_stride 0
    slab = torch.zeros(w.n_layer, dtype=torch.uint8, device=dev)            # one slab for all layers
    host_dst = torch.empty(w.dst_pool.numel(), dtype=torch.uint8).pin_memory()
    dst_before = [harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l) for l in range(s.L)]
    zeros = torch.zeros(s.R, dtype=torch.int32, device=dev)
    empty = tk.make_batch(w.src_bt, zeros, 0, None, flag)
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for l in range(s.L):
            tk.check(tk.topkv_pack_layer(l, w.src_pool, lo1, bs, slab, slab.numel(), stream))
            tk.check(tk.topkv_pack_layer(l, w.src_pool, lo1, empty, slab, slab.numel(), stream))
            tk.check(tk.topkv_unpack_layer(l, w.dst_pool, lo1, bd, slab, slab.numel(), stream))
        host_dst.copy_(w.dst_pool, non_blocking=True)
    stream.synchronize()
    for l in range(s.L):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, l)
        want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
        oracle.unpack(g, 0, dst_before[l], b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
        assert np.array_equal(host_dst[l * w.slab_bytes:(l + 1) * w.slab_bytes].numpy(),
                              dst_before[l]), l
    assert tk.topkv_device_error_flags() == 0
    del w
    torch.cuda.empty_cache()


def test_cuda_graph_capture_and_replay(dev):
    """The hot calls only enqueue work, so a whole layer loop can be captured in a CUDA graph
    and replayed (the launch-bound tiny case is where that pays)."""
    w = harness.setup(wl.CFG1, dev)
    b, s = w.batch, wl.CFG1
    g = _geom(s, b.num_pool_pages, s.L, 0, w.n_layer)
    src_h, dst_h = w.src_pool.cpu().numpy(), w.dst_pool.cpu().numpy()
    stream = torch.cuda.Stream(dev)
    with torch.cuda.stream(stream):                      # warm up outside the capture
        for layer in range(s.L):
            w.pack(layer, stream)
            w.unpack(layer, stream)
    stream.synchronize()
    w.wire.zero_()
    w.dst_pool.copy_(torch.from_numpy(dst_h))
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for layer in range(s.L):
            w.pack(layer, stream, overlap=layer > 0)
        for layer in range(s.L):
            w.unpack(layer, stream, overlap=layer > 0)
    assert not w.wire.any()                              # capturing executed nothing
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    want_wire = np.zeros(s.L * w.n_layer, dtype=np.uint8)
    for layer in range(s.L):
        oracle.pack(g, layer, src_h, b.src_block_table, b.seq_lens, wire=want_wire)
        oracle.unpack(g, layer, dst_h, b.dst_block_table, b.seq_lens, want_wire)
    assert np.array_equal(w.wire.cpu().numpy(), want_wire)
    assert np.array_equal(w.dst_pool.cpu().numpy(), dst_h)


def test_cuda_graph_capture_of_the_checksummed_path_and_layer_ranges(dev, variant):
    """begin, the checksummed pack of every layer, finish, and a multi-layer unpack captured
    in one CUDA graph: nothing runs during the capture, and after replays the wire, the pool
    and the checksums are the oracle's (the remainders are stored, so replays do not add up)."""
    if variant == 1:
        pytest.skip("the checksumming copy has one kernel family")
    w = harness.setup(wl.CFG1, dev)
    b, s = w.batch, wl.CFG1
    g = _geom(s, b.num_pool_pages, s.L, 0, w.n_layer)
    src_h, dst_h = w.src_pool.cpu().numpy(), w.dst_pool.cpu().numpy()
    nws = tk.topkv_crc_workspace_bytes(w.layout, s.R, b.max_pages_per_req)
    ws = torch.zeros(nws, dtype=torch.uint8, device=dev)
    crc = torch.zeros(s.R * s.F, dtype=torch.int64, device=dev)
    stream = torch.cuda.Stream(dev)

    def enqueue():
        tk.check(tk.topkv_crc_begin(w.layout, w.src_batch, ws, nws, stream))
        for layer in range(s.L):
            tk.check(tk.topkv_pack_layer_crc(layer, w.src_pool, w.layout, w.src_batch, w.wire,
                                             w.wire.numel(), ws, nws, stream))
        tk.check(tk.topkv_crc_finish(w.layout, w.src_batch, ws, nws, crc, stream))
        tk.check(tk.topkv_unpack_layers(0, s.L, w.dst_pool, w.layout, w.dst_batch, w.wire,
                                        w.wire.numel(), stream))

    with torch.cuda.stream(stream):                      # first use on this device: outside capture
        enqueue()
    stream.synchronize()
    w.wire.zero_()
    crc.zero_()
    w.dst_pool.copy_(torch.from_numpy(dst_h))
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        enqueue()
    assert not w.wire.any() and not crc.any()            # capturing executed nothing
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    want_wire = np.zeros(s.L * w.n_layer, dtype=np.uint8)
    for layer in range(s.L):
        oracle.pack(g, layer, src_h, b.src_block_table, b.seq_lens, wire=want_wire)
        oracle.unpack(g, layer, dst_h, b.dst_block_table, b.seq_lens, want_wire)
    assert np.array_equal(w.wire.cpu().numpy(), want_wire)
    assert np.array_equal(w.dst_pool.cpu().numpy(), dst_h)
    got = crc.cpu().numpy().view(np.uint64).reshape(s.R, s.F)
    for r in range(s.R):
        for c in range(s.F):
            assert int(got[r, c]) == oracle.kv_plane_crc(g, src_h, b.src_block_table, b.seq_lens, r, c)


def test_two_batches_on_two_streams(dev):
    """Independent batches issued concurrently on two streams do not disturb each other (the
    library keeps no per-call state)."""
    specs = [wl.with_layers(wl.CFG2, 3), wl.with_layers(wl.CFG4, 3)]
    ws = [harness.setup(sp, dev) for sp in specs]
    streams = [torch.cuda.Stream(dev) for _ in ws]
    before = [[harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l) for l in range(3)] for w in ws]
    for layer in range(3):
        for w, st in zip(ws, streams):
            w.pack(layer, st, overlap=layer > 0)
    for layer in range(3):
        for w, st in zip(ws, streams):
            w.unpack(layer, st, overlap=layer > 0)
    torch.cuda.synchronize()
    for w, sp, dst0 in zip(ws, specs, before):
        g = _geom(sp, w.batch.num_pool_pages, 1, 0, 0)
        for layer in range(3):
            src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
            want = oracle.pack(g, 0, src_h, w.batch.src_block_table, w.batch.seq_lens, impl="rows", threads=8)
            assert np.array_equal(w.wire[layer * w.n_layer:(layer + 1) * w.n_layer].cpu().numpy(), want)
            oracle.unpack(g, 0, dst0[layer], w.batch.dst_block_table, w.batch.seq_lens, want,
                          impl="rows", threads=8)
            assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer), dst0[layer])
    del ws
    torch.cuda.empty_cache()


# -------------------------------------------------------------------- windowed layers (§2.2)

@pytest.mark.parametrize("seed", range(16))
def test_windowed_layers(dev, seed):
    """A windowed layer keeps (and ships) only the last min(s, W) tokens of each request;
    block-table columns before the window are stale (-1 here) and must never be followed."""
    g, sl, bt_s, bt_d, rng = _case(seed)
    W = int(rng.choice([1, 2, g.P, g.P + 1, 3 * g.P - 1, 1000]))
    g.window = W
    for bt in (bt_s, bt_d):                               # free the pages before the window
        for r in range(len(sl)):
            bt[r, :max(0, int(sl[r]) - W) // g.P] = -1
    T = g.kept_tokens(sl)
    g.W_layer = g.wire_layer_bytes(T) + 32
    lo = _layout_from_geom(g)
    src_h = rng.integers(0, 256, g.L * g.S_layer, dtype=np.uint8)
    dst_h = rng.integers(0, 256, g.L * g.S_layer, dtype=np.uint8)
    src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h).to(dev)
    wire = torch.full((g.L * g.W_layer + 64,), 0x3C, dtype=torch.uint8, device=dev)
    d_sl = torch.from_numpy(sl).to(dev)
    d_bs, d_bd = torch.from_numpy(bt_s).to(dev), torch.from_numpy(bt_d).to(dev)
    cu = None
    if seed % 2:
        cu = torch.zeros(len(sl) + 1, dtype=torch.int64, device=dev)
        tk.check(tk.topkv_build_plan(tk.make_batch(d_bs, d_sl, window_tokens=W), cu))
        want_cu = np.concatenate([[0], np.cumsum(np.minimum(sl, W).astype(np.int64))])
        assert np.array_equal(cu.cpu().numpy(), want_cu)
    bs = tk.make_batch(d_bs, d_sl, T if seed % 3 else -1, cu, window_tokens=W)
    bd = tk.make_batch(d_bd, d_sl, T if seed % 3 else -1, cu, window_tokens=W)
    want_wire = np.full(g.L * g.W_layer + 64, 0x3C, dtype=np.uint8)
    for layer in range(g.L):
        tk.check(tk.topkv_pack_layer(layer, src, lo, bs, wire, wire.numel()))
        tk.check(tk.topkv_unpack_layer(layer, dst, lo, bd, wire, wire.numel()))
        oracle.pack(g, layer, src_h, bt_s, sl, wire=want_wire)
        oracle.unpack(g, layer, dst_h, bt_d, sl, want_wire)
    torch.cuda.synchronize()
    assert np.array_equal(wire.cpu().numpy(), want_wire)
    assert np.array_equal(dst.cpu().numpy(), dst_h)


@pytest.mark.parametrize("P,H,D", [(4, 1, 64), (16, 8, 128), (1, 2, 64)])
def test_window_spans_counted_from_the_first_kept_token(dev, variant, P, H, D):
    """Long rows with a short window: only the few spans a window can touch get a CTA, each
    placed from the request's own length. Lengths and windows sit on and around span borders
    (a span = 64 KiB worth of page columns: 64 pages of 4 tokens here, one page of 16, 64 pages
    of one token), with empty requests, requests shorter than the window and stale (-1)
    columns before every window. Pack, unpack and a linked pack -> unpack pair."""
    rng = np.random.default_rng(900 + P)
    E, F = 2, 2
    page_bytes = P * F * H * D * E
    ppc = max(1, min(64, 65536 // page_bytes))
    span = ppc * P
    maxp = (12 * span) // P + 3
    for W in (1, span - 1, span, span + 1, 2 * span + 1, 3 * span):
        if W <= 0:
            continue
        lens = [0, 1, max(1, W - 1), W, W + 1, 5 * span, 5 * span + 1, 5 * span - 1, 7 * span + W // 2,
                12 * span, 12 * span - W + 1, int(rng.integers(1, 12 * span))]
        sl = np.array(lens, dtype=np.int32)
        R = len(sl)
        pages = (sl + P - 1) // P
        npages = int(pages.sum()) + 3
        g = Geom(L=1, F=F, h_kv=H, d_h=D, b_p=E, P=P, num_pages=npages)
        g.window = W
        T = g.kept_tokens(sl)
        g.W_layer = g.wire_layer_bytes(T)
        bt_s = np.full((R, maxp), -1, dtype=np.int32)
        bt_d = np.full((R, maxp), -1, dtype=np.int32)
        ps, pd, pos = rng.permutation(npages), rng.permutation(npages), 0
        for r in range(R):
            bt_s[r, :pages[r]] = ps[pos:pos + pages[r]]
            bt_d[r, :pages[r]] = pd[pos:pos + pages[r]]
            pos += pages[r]
            stale = max(0, int(sl[r]) - W) // P                 # columns wholly before the window
            bt_s[r, :stale] = -1
            bt_d[r, :stale] = -1
        lo = _layout_from_geom(g)
        src_h = rng.integers(0, 256, g.S_layer, dtype=np.uint8)
        dst_h = rng.integers(0, 256, g.S_layer, dtype=np.uint8)
        src = torch.from_numpy(src_h).to(dev)
        dst, dst2 = torch.from_numpy(dst_h).to(dev), torch.from_numpy(dst_h).to(dev)
        wire = torch.full((g.W_layer + 64,), 0x3C, dtype=torch.uint8, device=dev)
        wire2 = torch.full((g.W_layer + 64,), 0x3C, dtype=torch.uint8, device=dev)
        d_sl = torch.from_numpy(sl).to(dev)
        bs = tk.make_batch(torch.from_numpy(bt_s).to(dev), d_sl, T, None, 0, W)
        bd = tk.make_batch(torch.from_numpy(bt_d).to(dev), d_sl, T, None, 0, W)
        tk.check(tk.topkv_pack_layer(0, src, lo, bs, wire, wire.numel()))
        tk.check(tk.topkv_unpack_layer(0, dst, lo, bd, wire, wire.numel()))
        want = np.full(g.W_layer + 64, 0x3C, dtype=np.uint8)
        oracle.pack(g, 0, src_h, bt_s, sl, wire=want)
        oracle.unpack(g, 0, dst_h, bt_d, sl, want)
        torch.cuda.synchronize()
        assert tk.topkv_device_error_flags() == 0
        assert np.array_equal(wire.cpu().numpy(), want), W
        assert np.array_equal(dst.cpu().numpy(), dst_h), W
        if variant == 0:
            words = tk.topkv_span_link_words(lo, bs)
            flags = torch.zeros(max(1, words), dtype=torch.int32, device=dev)
            stream = torch.cuda.Stream(dev)
            stream.wait_stream(torch.cuda.current_stream(dev))
            tk.check(tk.topkv_pack_layer_linked(0, src, lo, bs, wire2, wire2.numel(),
                                                tk.make_span_link(None, 0, flags, 3), stream))
            tk.check(tk.topkv_unpack_layer_linked(0, dst2, lo, bd, wire2, wire2.numel(),
                                                  tk.make_span_link(flags, 3, None, 0), stream))
            stream.synchronize()
            assert tk.topkv_device_error_flags() == 0
            assert np.array_equal(wire2.cpu().numpy(), want), W
            assert np.array_equal(dst2.cpu().numpy(), dst_h), W


def test_windowed_layer_bench_shape(dev):
    """gpt-oss-like windowed layer on the 8B batch: window 128 of up to 4096 tokens."""
    w = harness.setup(wl.CFG2, dev, layers=2)
    b, s = w.batch, wl.CFG2
    W = 128
    g = _geom(s, b.num_pool_pages, 1, 0, 0)
    g.window = W
    T = g.kept_tokens(b.seq_lens)
    assert T == 16 * 128
    bs = tk.make_batch(w.src_bt, w.seq_lens, T, None, window_tokens=W)
    bd = tk.make_batch(w.dst_bt, w.seq_lens, T, None, window_tokens=W)
    n = g.wire_layer_bytes(T)
    wire = torch.zeros(n, dtype=torch.uint8, device=dev)
    lo = tk.make_layout(2, s.F, s.H, s.D, s.E, s.P, b.num_pool_pages, wire_layer_stride=0)
    for layer in range(2):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
        dst_h = harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer)
        tk.check(tk.topkv_pack_layer(layer, w.src_pool, lo, bs, wire, n))
        tk.check(tk.topkv_unpack_layer(layer, w.dst_pool, lo, bd, wire, n))
        torch.cuda.synchronize()
        want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
        assert np.array_equal(wire.cpu().numpy(), want)
        oracle.unpack(g, 0, dst_h, b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
        assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer), dst_h)
    del w
    torch.cuda.empty_cache()


# -------------------------------------------------------------------- header + CRC-64 (§3.4)

def _crc_run(dev, g, sl, bt_s, bt_d, src_h, dst_h, corrupt=None, use_plan=True, repeat_layer=None):
    """Sender: pack every layer with checksums. Receiver: unpack with checksums from the
    (optionally corrupted) wire. Returns wire, destination pool and both checksum arrays."""
    lo = _layout_from_geom(g)
    R, F = len(sl), g.F
    T = int(sl.sum())
    src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h.copy()).to(dev)
    wire = torch.zeros(max(g.L * g.W_layer, 16), dtype=torch.uint8, device=dev)
    d_sl = torch.from_numpy(sl).to(dev)
    d_bs, d_bd = torch.from_numpy(bt_s).to(dev), torch.from_numpy(bt_d).to(dev)
    cu = None
    if use_plan:
        cu = torch.zeros(R + 1, dtype=torch.int64, device=dev)
        tk.check(tk.topkv_build_plan(tk.make_batch(d_bs, d_sl), cu))
    Tk = T if use_plan else -1                          # without a plan: total unknown as well
    bs, bd = tk.make_batch(d_bs, d_sl, Tk, cu), tk.make_batch(d_bd, d_sl, Tk, cu)
    ov = tk.TOPKV_FLAG_OVERLAP_PREVIOUS                 # layers after the first may overlap
    bs_ov, bd_ov = tk.make_batch(d_bs, d_sl, Tk, cu, ov), tk.make_batch(d_bd, d_sl, Tk, cu, ov)
    nws = tk.topkv_crc_workspace_bytes(lo, R, bt_s.shape[1])
    assert nws > 0
    out = []
    for side, (pool, batch, batch_ov, fn) in enumerate(((src, bs, bs_ov, tk.topkv_pack_layer_crc),
                                                        (dst, bd, bd_ov, tk.topkv_unpack_layer_crc))):
        ws = torch.full((nws,), 0xEE, dtype=torch.uint8, device=dev)   # scratch starts dirty
        crc = torch.zeros(R * F, dtype=torch.int64, device=dev)
        tk.check(tk.topkv_crc_begin(lo, batch, ws, nws))
        order = list(range(g.L)) if side == 0 else list(reversed(range(g.L)))  # any layer order
        for k, layer in enumerate(order):
            tk.check(fn(layer, pool, lo, batch_ov if k else batch, wire, wire.numel(), ws, nws))
        if repeat_layer is not None:                    # doing a layer again changes nothing
            tk.check(fn(repeat_layer, pool, lo, batch, wire, wire.numel(), ws, nws))
        tk.check(tk.topkv_crc_finish(lo, batch, ws, nws, crc))
        tk.check(tk.topkv_crc_finish(lo, batch, ws, nws, crc))   # and so does finishing twice
        torch.cuda.synchronize()
        out.append(crc.cpu().numpy().view(np.uint64).reshape(R, F))
        if side == 0 and corrupt is not None:
            wire[corrupt] ^= 0x10                      # one flipped bit on the way
    return wire.cpu().numpy(), dst.cpu().numpy(), out[0], out[1]


@pytest.mark.parametrize("seed", range(24))
def test_crc_fused_pack_unpack(dev, seed, variant):
    if variant == 1:
        pytest.skip("the checksumming copy has one kernel family")
    rng = np.random.default_rng(500 + seed)
    F = int(rng.integers(1, 3))
    H, D = [(8, 128), (1, 576), (1, 128), (2, 8), (4, 64), (8, 256)][seed % 6]
    P = int(rng.choice([1, 4, 16]))
    R = int(rng.integers(1, 5))
    sl = rng.integers(0, 4 * P + 2, size=R).astype(np.int32)
    if seed >= 12:                                     # long requests: many items per plane
        sl = rng.integers(0, 40 * P + 2, size=R).astype(np.int32)
    if seed % 4 == 1:
        sl[rng.integers(0, R)] = 0
    pages = (sl + P - 1) // P
    maxp = max(int(pages.max()), 1) + 1
    npages = int(pages.sum()) + 2
    g = Geom(L=3, F=F, h_kv=H, d_h=D, b_p=2, P=P, num_pages=npages,
             wire_order=int(rng.integers(0, 2)))
    if seed % 3 == 2:                                  # plane-major pool with padded tokens
        g.S_tok = H * D * 2 + 32
        g.S_page = P * g.S_tok
        g.S_kv = npages * g.S_page
        g.S_layer = F * g.S_kv
    elif seed % 3 == 1 and H > 1:                      # head-major inside the page
        g.S_tok = D * 2
        g.S_head = P * g.S_tok
        g.S_kv = H * g.S_head
        g.S_page = F * g.S_kv
        g.S_layer = npages * g.S_page
    T = int(sl.sum())
    g.W_layer = g.wire_layer_bytes(T)
    bt_s = np.full((R, maxp), -1, dtype=np.int32)
    bt_d = np.full((R, maxp), -1, dtype=np.int32)
    ps, pd, pos = rng.permutation(npages), rng.permutation(npages), 0
    for r in range(R):
        bt_s[r, :pages[r]] = ps[pos:pos + pages[r]]
        bt_d[r, :pages[r]] = pd[pos:pos + pages[r]]
        pos += pages[r]
    src_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
    dst_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
    wire, dst, crc_tx, crc_rx = _crc_run(dev, g, sl, bt_s, bt_d, src_h, dst_h,
                                         use_plan=seed % 2 == 0, repeat_layer=seed % g.L)
    want_wire = np.zeros(max(g.L * g.W_layer, 16), dtype=np.uint8)
    want_dst = dst_h.copy()
    for layer in range(g.L):
        oracle.pack(g, layer, src_h, bt_s, sl, wire=want_wire)
        oracle.unpack(g, layer, want_dst, bt_d, sl, want_wire)
    assert np.array_equal(wire, want_wire) and np.array_equal(dst, want_dst)
    for r in range(R):
        for c in range(F):
            want = oracle.kv_plane_crc(g, src_h, bt_s, sl, r, c)
            assert int(crc_tx[r, c]) == want, (r, c, hex(int(crc_tx[r, c])), hex(want))
            assert int(crc_rx[r, c]) == want


@pytest.mark.parametrize("seed", range(8))
def test_crc_with_windowed_layers(dev, seed, variant):
    """A model whose layers differ in kind (§2.2): full layers and windowed layers with two
    different windows. Every layer is packed / unpacked with its own window; the checksums
    equal the oracle's CRC over what every layer keeps, the bytes the oracle's windowed pack."""
    if variant == 1:
        pytest.skip("the checksumming copy has one kernel family")
    import copy
    rng = np.random.default_rng(900 + seed)
    F = int(rng.integers(1, 3))
    H, D = [(8, 128), (1, 576), (2, 64), (4, 32)][seed % 4]
    P = int(rng.choice([1, 4, 16]))
    R = int(rng.integers(1, 5))
    sl = rng.integers(0, 12 * P + 2, size=R).astype(np.int32)
    if seed % 3 == 0:
        sl[rng.integers(0, R)] = 0
    L = 5
    windows = [0, 2 * P + 1, 0, 3, 2 * P + 1]
    pages = (sl + P - 1) // P
    maxp = max(int(pages.max()), 1) + 1
    npages = int(pages.sum()) + 2
    g = Geom(L=L, F=F, h_kv=H, d_h=D, b_p=2, P=P, num_pages=npages, wire_order=seed % 2)
    g.W_layer = g.wire_layer_bytes(int(sl.sum()))      # slabs sized for a full layer
    bt_s = np.full((R, maxp), -1, dtype=np.int32)
    bt_d = np.full((R, maxp), -1, dtype=np.int32)
    ps, pd, pos = rng.permutation(npages), rng.permutation(npages), 0
    for r in range(R):
        bt_s[r, :pages[r]] = ps[pos:pos + pages[r]]
        bt_d[r, :pages[r]] = pd[pos:pos + pages[r]]
        pos += pages[r]
    src_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
    dst_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
    lo = _layout_from_geom(g)
    src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h.copy()).to(dev)
    wire = torch.zeros(max(L * g.W_layer, 16), dtype=torch.uint8, device=dev)
    d_sl = torch.from_numpy(sl).to(dev)
    d_bs, d_bd = torch.from_numpy(bt_s).to(dev), torch.from_numpy(bt_d).to(dev)
    nws = tk.topkv_crc_workspace_bytes(lo, R, maxp)
    got = []
    want_wire = np.zeros(max(L * g.W_layer, 16), dtype=np.uint8)
    want_dst = dst_h.copy()
    for side, (pool, d_bt, fn) in enumerate(((src, d_bs, tk.topkv_pack_layer_crc),
                                             (dst, d_bd, tk.topkv_unpack_layer_crc))):
        ws = torch.full((nws,), 0x77, dtype=torch.uint8, device=dev)
        crc = torch.zeros(R * F, dtype=torch.int64, device=dev)
        tk.check(tk.topkv_crc_begin(lo, tk.make_batch(d_bt, d_sl), ws, nws))
        for layer in range(L):
            W = windows[layer]
            kept = int(sl.sum()) if W == 0 else int(np.minimum(sl, W).sum())
            batch = tk.make_batch(d_bt, d_sl, kept if seed % 2 else -1, None, 0, W)
            tk.check(fn(layer, pool, lo, batch, wire, wire.numel(), ws, nws))
        tk.check(tk.topkv_crc_finish(lo, tk.make_batch(d_bt, d_sl), ws, nws, crc))
        torch.cuda.synchronize()
        got.append(crc.cpu().numpy().view(np.uint64).reshape(R, F))
    for layer in range(L):
        gl = copy.copy(g)
        gl.window = windows[layer]
        oracle.pack(gl, layer, src_h, bt_s, sl, wire=want_wire)
        oracle.unpack(gl, layer, want_dst, bt_d, sl, want_wire)
    assert np.array_equal(wire.cpu().numpy(), want_wire)
    assert np.array_equal(dst.cpu().numpy(), want_dst)
    for r in range(R):
        for c in range(F):
            want = oracle.kv_plane_crc(g, src_h, bt_s, sl, r, c, layer_windows=windows)
            assert int(got[0][r, c]) == want, (r, c)
            assert int(got[1][r, c]) == want


def test_crc_cfg1_header_round_trip_and_corruption(dev, variant):
    """cfg1 end to end: the sender's headers verify on the receiver; one flipped wire bit makes
    exactly the affected request fail with TOPKV_ERR_CHECKSUM, and the retry policy of §3.1
    (re-send, then verify again) recovers."""
    if variant == 1:
        pytest.skip("the checksumming copy has one kernel family")
    b = wl.make_batch(wl.CFG1)
    s = b.spec
    g = _geom(s, b.num_pool_pages, s.L, 0, b.total_tokens * s.tok_bytes)
    src_h = wl.fill_numpy(g.pool_bytes(), b.seeds["data"])
    dst_h = wl.fill_numpy(g.pool_bytes(), b.seeds["dst_fill"])
    lo = _layout_from_geom(g)
    _, _, tx, rx = _crc_run(dev, g, b.seq_lens, b.src_block_table, b.dst_block_table, src_h, dst_h)
    headers = []
    for r in range(s.R):
        assert int(tx[r, 0]) == oracle.kv_plane_crc(g, src_h, b.src_block_table, b.seq_lens, r, 0)
        assert int(tx[r, 1]) == oracle.kv_plane_crc(g, src_h, b.src_block_table, b.seq_lens, r, 1)
        h = tk.topkv_wire_header()
        tk.check(tk.topkv_header_fill(h, 1000 + r, 42, lo, int(b.seq_lens[r]), int(tx[r, 0]), int(tx[r, 1])))
        headers.append(h)
        assert tk.topkv_header_check(h, lo, int(b.seq_lens[r]), int(rx[r, 0]), int(rx[r, 1])) == 0
    # flip one bit inside request 2's V row of token 5, layer 1
    cu = np.concatenate([[0], np.cumsum(b.seq_lens)])
    off = 1 * g.W_layer + ((int(cu[2]) + 5) * 2 + 1) * g.row_bytes + 77
    attempts = []

    def transfer():
        bad = off if not attempts else None           # the first attempt is corrupted in flight
        attempts.append(1)
        _, _, _, rx2 = _crc_run(dev, g, b.seq_lens, b.src_block_table, b.dst_block_table, src_h,
                                dst_h, corrupt=bad)
        status = [tk.topkv_header_check(headers[r], lo, int(b.seq_lens[r]), int(rx2[r, 0]),
                                        int(rx2[r, 1])) for r in range(s.R)]
        if len(attempts) == 1:
            assert status == [0, 0, tk.TOPKV_ERR_CHECKSUM, 0]
        return min(status)

    assert tk.topkv_retry(transfer, retries=2, backoff_ms=1) == tk.TOPKV_OK
    assert len(attempts) == 2


def test_paper_payload_one_request_end_to_end(dev, variant):
    """§3.4 end to end for one request: 128-byte header, then the K tensor
    [layers][seq_len][kv_heads][head_dim], then the V tensor, assembled by per-layer PLANAR
    packs (layer stride = one plane, plane stride = L planes); the header's checksums come from
    the checksummed copy and equal the host CRC-64 of the payload's two halves."""
    rng = np.random.default_rng(91)
    L, H, D, P, s_len = 5, 8, 128, 16, 333
    npages = 40
    g = Geom(L=L, F=2, h_kv=H, d_h=D, b_p=2, P=P, num_pages=npages, wire_order=1)
    plane = s_len * g.row_bytes
    g.W_layer, g.W_plane = plane, L * plane
    sl = np.array([s_len], dtype=np.int32)
    bt = rng.permutation(npages)[:21].astype(np.int32).reshape(1, 21)
    lo = _layout_from_geom(g)
    src_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
    src = torch.from_numpy(src_h).to(dev)
    d_sl, d_bt = torch.from_numpy(sl).to(dev), torch.from_numpy(bt).to(dev)
    cu = torch.zeros(2, dtype=torch.int64, device=dev)
    tk.check(tk.topkv_build_plan(tk.make_batch(d_bt, d_sl), cu))
    batch = tk.make_batch(d_bt, d_sl, s_len, cu)
    message = torch.zeros(128 + 2 * L * plane, dtype=torch.uint8, device=dev)
    payload = message[128:]
    want = np.zeros(2 * L * plane, dtype=np.uint8)
    for layer in range(L):
        oracle.pack(g, layer, src_h, bt, sl, wire=want)
    # plain pack (both kernel families)
    for layer in range(L):
        tk.check(tk.topkv_pack_layer(layer, src, lo, batch, payload, payload.numel()))
    torch.cuda.synchronize()
    assert np.array_equal(payload.cpu().numpy(), want)
    # checksummed pack into a fresh message, header built from the device checksums
    payload.zero_()
    nws = tk.topkv_crc_workspace_bytes(lo, 1, 21)
    ws = torch.zeros(nws, dtype=torch.uint8, device=dev)
    crc = torch.zeros(2, dtype=torch.int64, device=dev)
    tk.check(tk.topkv_crc_begin(lo, batch, ws, nws))
    for layer in range(L):
        tk.check(tk.topkv_pack_layer_crc(layer, src, lo, batch, payload, payload.numel(), ws, nws))
    tk.check(tk.topkv_crc_finish(lo, batch, ws, nws, crc))
    torch.cuda.synchronize()
    crc_k, crc_v = (int(x) for x in crc.cpu().numpy().view(np.uint64))
    h = tk.topkv_wire_header()
    tk.check(tk.topkv_header_fill(h, 77, 5, lo, s_len, crc_k, crc_v))
    message[:128] = torch.frombuffer(bytearray(bytes(h)), dtype=torch.uint8).to(dev)
    msg = message.cpu().numpy()
    assert bytes(msg[:8]) == b"KVCACHE1" and np.array_equal(msg[128:], want)
    k_bytes = L * plane
    assert tk.topkv_crc64(np.ascontiguousarray(msg[128:128 + k_bytes])) == crc_k
    assert tk.topkv_crc64(np.ascontiguousarray(msg[128 + k_bytes:])) == crc_v
    assert crc_k == oracle.kv_plane_crc(g, src_h, bt, sl, 0, 0) == oracle.crc64(want[:k_bytes])
    assert crc_v == oracle.kv_plane_crc(g, src_h, bt, sl, 0, 1) == oracle.crc64(want[k_bytes:])
    assert bytes(msg[:128]) == oracle.build_header(77, 5, s_len, g, crc_k, crc_v)
    assert h.k_bytes == k_bytes


@pytest.mark.parametrize("staged", [True, False])
def test_host_leg_with_checksums(dev, staged, variant):
    """Sender: pack to pinned host memory with checksums; receiver: unpack from it with
    checksums. Bytes and both sets of checksums equal the oracle's."""
    if variant == 1:
        pytest.skip("the checksumming copy has one kernel family")
    w = harness.setup(wl.CFG1, dev)
    b, s = w.batch, wl.CFG1
    g = _geom(s, b.num_pool_pages, s.L, 0, w.n_layer)
    src_h, dst_h = w.src_pool.cpu().numpy(), w.dst_pool.cpu().numpy()
    pinned = torch.zeros(s.L * w.n_layer, dtype=torch.uint8).pin_memory()
    staging = torch.zeros(w.n_layer, dtype=torch.uint8, device=dev) if staged else None
    cap = w.n_layer if staged else 0
    nws = tk.topkv_crc_workspace_bytes(w.layout, s.R, b.max_pages_per_req)
    got = []
    for fn, pool, batch in ((tk.topkv_pack_layer_to_host_crc, w.src_pool, w.src_batch),
                            (tk.topkv_unpack_layer_from_host_crc, w.dst_pool, w.dst_batch)):
        ws = torch.zeros(nws, dtype=torch.uint8, device=dev)
        crc = torch.zeros(s.R * s.F, dtype=torch.int64, device=dev)
        tk.check(tk.topkv_crc_begin(w.layout, batch, ws, nws))
        for layer in range(s.L):
            tk.check(fn(layer, pool, w.layout, batch, pinned, pinned.numel(), staging, cap, ws, nws))
        tk.check(tk.topkv_crc_finish(w.layout, batch, ws, nws, crc))
        torch.cuda.synchronize()
        got.append(crc.cpu().numpy().view(np.uint64).reshape(s.R, s.F))
    want_wire = np.zeros(s.L * w.n_layer, dtype=np.uint8)
    for layer in range(s.L):
        oracle.pack(g, layer, src_h, b.src_block_table, b.seq_lens, wire=want_wire)
        oracle.unpack(g, layer, dst_h, b.dst_block_table, b.seq_lens, want_wire)
    assert np.array_equal(pinned.numpy(), want_wire)
    assert np.array_equal(w.dst_pool.cpu().numpy(), dst_h)
    for r in range(s.R):
        for c in range(s.F):
            want = oracle.kv_plane_crc(g, src_h, b.src_block_table, b.seq_lens, r, c)
            assert int(got[0][r, c]) == want and int(got[1][r, c]) == want


# -------------------------------------------------------------------- direct re-paging

def _repage_case(seed):
    """Two pools with different page sizes and strides, the same requests."""
    rng = np.random.default_rng(1000 + seed)
    F = int(rng.integers(1, 3))
    H = int(rng.choice([1, 2, 8]))
    D = int(rng.choice([8, 64, 128]))
    Ps, Pd = int(rng.choice([1, 3, 16, 64])), int(rng.choice([1, 4, 16, 32]))
    R = int(rng.integers(1, 6))
    sl = rng.integers(0, 5 * max(Ps, Pd) + 3, size=R).astype(np.int32)
    if seed % 4 == 0:
        sl[rng.integers(0, R)] = 0
    geoms, tables = [], []
    for P, style in ((Ps, seed % 3), (Pd, (seed // 3) % 3)):
        pages = (sl + P - 1) // P
        npages = int(pages.sum()) + 3
        g = Geom(L=2, F=F, h_kv=H, d_h=D, b_p=2, P=P, num_pages=npages)
        if style == 1:      # head-major inside the page
            g.S_tok = D * 2
            g.S_head = P * g.S_tok
            g.S_kv = H * g.S_head
            g.S_page = F * g.S_kv
            g.S_layer = npages * g.S_page
        elif style == 2:    # padded tokens, plane-major pool
            g.S_tok = H * D * 2 + 16
            g.S_page = P * g.S_tok
            g.S_kv = npages * g.S_page
            g.S_layer = F * g.S_kv + 48
        maxp = max(int(pages.max()), 1) + int(rng.integers(0, 2))
        bt = np.full((R, maxp), -1, dtype=np.int32)
        perm, pos = rng.permutation(npages), 0
        for r in range(R):
            bt[r, :pages[r]] = perm[pos:pos + pages[r]]
            pos += pages[r]
        geoms.append(g)
        tables.append(bt)
    return geoms, tables, sl, rng


@pytest.mark.parametrize("seed", range(24))
def test_repage_equals_unpack_of_pack(dev, seed, variant):
    if variant == 1:
        pytest.skip("re-paging has one kernel family")
    (gs, gd), (bt_s, bt_d), sl, rng = _repage_case(seed)
    T = int(sl.sum())
    src_h = rng.integers(0, 256, gs.pool_bytes(), dtype=np.uint8)
    dst_h = rng.integers(0, 256, gd.pool_bytes(), dtype=np.uint8)
    src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h).to(dev)
    d_sl = torch.from_numpy(sl).to(dev)
    d_bs, d_bd = torch.from_numpy(bt_s).to(dev), torch.from_numpy(bt_d).to(dev)
    los, lod = _layout_from_geom(gs), _layout_from_geom(gd)
    for layer in range(2):
        tk.check(tk.topkv_repage_layer(layer, src, los, tk.make_batch(d_bs, d_sl, T), dst, lod,
                                       tk.make_batch(d_bd, d_sl, T)))
        wire = oracle.pack(gs, layer, src_h, bt_s, sl)
        gd.W_layer = gs.W_layer
        oracle.unpack(gd, layer, dst_h, bt_d, sl, wire)
    torch.cuda.synchronize()
    assert np.array_equal(dst.cpu().numpy(), dst_h)
    assert np.array_equal(src.cpu().numpy(), src_h)


def test_repage_bench_shape(dev, variant):
    if variant == 1:
        pytest.skip("re-paging has one kernel family")
    w = harness.setup(wl.CFG2, dev, layers=2)
    b, s = w.batch, wl.CFG2
    g = _geom(s, b.num_pool_pages, 1, 0, 0)
    for layer in range(2):
        dst_h = harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer)
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
        tk.check(tk.topkv_repage_layer(layer, w.src_pool, w.layout, w.src_batch, w.dst_pool,
                                       w.layout, w.dst_batch))
        torch.cuda.synchronize()
        wire = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
        oracle.unpack(g, 0, dst_h, b.dst_block_table, b.seq_lens, wire, impl="rows", threads=8)
        assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer), dst_h)
    del w
    torch.cuda.empty_cache()


@pytest.mark.parametrize("R", [3, 40, 256, 300])
def test_repage_compact_grid_for_ragged_batches(dev, R, variant):
    """Re-paging a ragged batch (one long request, many short and empty ones) between pools of
    different page size with the total stated and the launches declared independent: the grid
    holds one CTA per span that can hold tokens (up to 256 requests; the full grid beyond).
    Both layers, against the oracle's unpack of the oracle's pack; a total below the device
    lengths is reported."""
    if variant == 1:
        pytest.skip("re-paging has one kernel family")
    rng = np.random.default_rng(2000 + R)
    F, H, D, E = 2, 2, 64, 2
    Ps, Pd = 16, 4
    sl = rng.integers(0, 40, size=R).astype(np.int32)
    sl[rng.integers(0, R, size=max(1, R // 4))] = 0
    sl[rng.integers(0, R)] = 3000
    T = int(sl.sum())

    def side(P, seed):
        pages = (sl + P - 1) // P
        npages = int(pages.sum()) + 5
        g = Geom(L=2, F=F, h_kv=H, d_h=D, b_p=E, P=P, num_pages=npages)
        g.W_layer = g.wire_layer_bytes(T)
        bt = np.full((R, int(pages.max()) + 1), -1, dtype=np.int32)
        perm, pos = np.random.default_rng(seed).permutation(npages), 0
        for r in range(R):
            bt[r, :pages[r]] = perm[pos:pos + pages[r]]
            pos += pages[r]
        return g, bt
    (gs, bt_s), (gd, bt_d) = side(Ps, 1), side(Pd, 2)
    src_h = rng.integers(0, 256, gs.pool_bytes(), dtype=np.uint8)
    dst_h = rng.integers(0, 256, gd.pool_bytes(), dtype=np.uint8)
    src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h).to(dev)
    d_sl = torch.from_numpy(sl).to(dev)
    d_bs, d_bd = torch.from_numpy(bt_s).to(dev), torch.from_numpy(bt_d).to(dev)
    los, lod = _layout_from_geom(gs), _layout_from_geom(gd)
    ov = tk.TOPKV_FLAG_OVERLAP_PREVIOUS
    torch.cuda.synchronize()
    for layer in range(2):      # the two layers touch different slabs: independent launches
        tk.check(tk.topkv_repage_layer(layer, src, los, tk.make_batch(d_bs, d_sl, T, None, ov), dst, lod,
                                       tk.make_batch(d_bd, d_sl, T, None, ov)))
        wire = oracle.pack(gs, layer, src_h, bt_s, sl)
        oracle.unpack(gd, layer, dst_h, bt_d, sl, wire)
    torch.cuda.synchronize()
    assert tk.topkv_device_error_flags() == 0
    assert np.array_equal(dst.cpu().numpy(), dst_h)
    assert np.array_equal(src.cpu().numpy(), src_h)
    span = min(65536 // (F * H * D * E), 63 * min(Ps, Pd))     # tokens per CTA of the re-paging kernel
    spans = int(((sl + span - 1) // span).sum())
    if R <= 256 and (T - 2000) // span + R < spans:
        # an understated total leaves spans without a CTA: reported, nothing else touched
        tk.check(tk.topkv_repage_layer(0, src, los, tk.make_batch(d_bs, d_sl, T - 2000, None, ov), dst, lod,
                                       tk.make_batch(d_bd, d_sl, T - 2000, None, ov)))
        assert tk.topkv_device_error_flags() & 4
        assert np.array_equal(dst.cpu().numpy(), dst_h)      # what was copied was copied to the same places
        tk.check(tk.topkv_reset_device_error_flags())


# -------------------------------------------------------------------- host leg

@pytest.fixture
def host_leg_ctas(request):
    prev = tk.topkv_set_host_leg_ctas(request.param)
    assert prev >= 0
    yield request.param
    tk.topkv_set_host_leg_ctas(prev)


def test_host_leg_cta_bound_setter(dev):
    assert tk.topkv_set_host_leg_ctas(-1) == tk.TOPKV_ERR_INVALID_ARG
    assert tk.topkv_set_host_leg_ctas(1 << 16) == tk.TOPKV_ERR_INVALID_ARG
    prev = tk.topkv_set_host_leg_ctas(5)
    assert prev == 8                                   # the documented default
    assert tk.topkv_set_host_leg_ctas(prev) == 5


@pytest.mark.parametrize("host_leg_ctas", [0, 1, 3, 16, 1000], indirect=True)
@pytest.mark.parametrize("seed", range(6))
def test_direct_host_leg_walking_grid_random_geometries(dev, seed, host_leg_ctas, variant):
    """The direct host leg with a bounded grid (every CTA walks several spans): pinned bytes
    and destination pool equal the oracle's for strided pools, both wire orders, empty and
    ragged requests, small pages grouped per CTA, more CTAs than spans."""
    if variant == 1:
        pytest.skip("the bounded grid belongs to the vectorised family")
    rng = np.random.default_rng(7000 + seed)
    F = int(rng.integers(1, 3))
    H, D = [(8, 128), (1, 576), (2, 64), (4, 8), (8, 64), (1, 128)][seed]
    P = int(rng.choice([1, 4, 16, 64]))
    R = int(rng.integers(1, 7))
    sl = rng.integers(0, 6 * P + 3, size=R).astype(np.int32)
    if seed % 2:
        sl[rng.integers(0, R)] = 0
    pages = (sl + P - 1) // P
    maxp = max(int(pages.max()), 1) + 1
    npages = int(pages.sum()) + 3
    g = Geom(L=2, F=F, h_kv=H, d_h=D, b_p=2, P=P, num_pages=npages, wire_order=seed % 2)
    if seed % 3 == 1:                                  # head-major inside the page
        g.S_tok = D * 2
        g.S_head = P * g.S_tok
        g.S_kv = H * g.S_head
        g.S_page = F * g.S_kv
        g.S_layer = npages * g.S_page
    T = int(sl.sum())
    g.W_layer = g.wire_layer_bytes(T) + 32
    bt_s = np.full((R, maxp), -1, dtype=np.int32)
    bt_d = np.full((R, maxp), -1, dtype=np.int32)
    ps, pd, pos = rng.permutation(npages), rng.permutation(npages), 0
    for r in range(R):
        bt_s[r, :pages[r]] = ps[pos:pos + pages[r]]
        bt_d[r, :pages[r]] = pd[pos:pos + pages[r]]
        pos += pages[r]
    src_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
    dst_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
    lo = _layout_from_geom(g)
    src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h.copy()).to(dev)
    d_sl = torch.from_numpy(sl).to(dev)
    d_bs, d_bd = torch.from_numpy(bt_s).to(dev), torch.from_numpy(bt_d).to(dev)
    bs, bd = tk.make_batch(d_bs, d_sl, T), tk.make_batch(d_bd, d_sl, T)
    pinned = torch.full((2 * g.W_layer,), 0xA5, dtype=torch.uint8).pin_memory()
    want = np.full(2 * g.W_layer, 0xA5, dtype=np.uint8)
    for layer in (1, 0):
        tk.check(tk.topkv_pack_layer_to_host(layer, src, lo, bs, pinned, pinned.numel(), None, 0))
        oracle.pack(g, layer, src_h, bt_s, sl, wire=want)
    torch.cuda.synchronize()
    assert np.array_equal(pinned.numpy(), want)       # gaps between slabs untouched as well
    for layer in (0, 1):
        tk.check(tk.topkv_unpack_layer_from_host(layer, dst, lo, bd, pinned, pinned.numel(), None, 0))
        oracle.unpack(g, layer, dst_h, bt_d, sl, want)
    torch.cuda.synchronize()
    assert np.array_equal(dst.cpu().numpy(), dst_h)
    assert np.array_equal(src.cpu().numpy(), src_h)


@pytest.mark.parametrize("staged", [True, False])
def test_host_leg_cfg1(dev, staged):
    w = harness.setup(wl.CFG1, dev)
    b, s = w.batch, w.batch.spec
    g = _geom(s, b.num_pool_pages, s.L, 0, w.n_layer)
    src_h, dst_h = w.src_pool.cpu().numpy(), w.dst_pool.cpu().numpy()
    pinned = torch.full((s.L * w.n_layer,), 0x5A, dtype=torch.uint8).pin_memory()
    staging = torch.zeros(w.n_layer, dtype=torch.uint8, device=dev) if staged else None
    stream = torch.cuda.Stream(dev)
    for layer in range(s.L):
        w.pack_to_host(layer, pinned, staging, stream)
    stream.synchronize()
    want_wire = np.zeros(s.L * w.n_layer, dtype=np.uint8)
    for layer in range(s.L):
        oracle.pack(g, layer, src_h, b.src_block_table, b.seq_lens, wire=want_wire)
    assert np.array_equal(pinned.numpy(), want_wire)
    for layer in range(s.L):
        w.unpack_from_host(layer, pinned, staging, stream)
    stream.synchronize()
    for layer in range(s.L):
        oracle.unpack(g, layer, dst_h, b.dst_block_table, b.seq_lens, want_wire)
    assert np.array_equal(w.dst_pool.cpu().numpy(), dst_h)


def test_host_leg_refuses_pageable_memory(dev):
    w = harness.setup(wl.CFG1, dev)
    pageable = torch.zeros(w.batch.spec.L * w.n_layer, dtype=torch.uint8)
    st = tk.topkv_pack_layer_to_host(0, w.src_pool, w.layout, w.src_batch, pageable,
                                     pageable.numel(), None, 0)
    assert st in (tk.TOPKV_ERR_INVALID_ARG, tk.TOPKV_ERR_CUDA)
    torch.cuda.synchronize()


def test_host_leg_cfg3_shape_two_layers(dev):
    """The 70B shape's per-layer slab (128 MiB) through pinned memory, both forms."""
    w = harness.setup(wl.CFG3, dev, layers=2)
    b, s = w.batch, w.batch.spec
    g = _geom(s, b.num_pool_pages, 1, 0, 0)
    pinned = torch.zeros(2 * w.n_layer, dtype=torch.uint8).pin_memory()
    staging = torch.zeros(w.n_layer, dtype=torch.uint8, device=dev)
    for staged, layer in ((True, 0), (False, 1)):
        w.pack_to_host(layer, pinned, staging if staged else None)
        torch.cuda.synchronize()
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
        want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
        assert np.array_equal(pinned[layer * w.n_layer:(layer + 1) * w.n_layer].numpy(), want)
        dst_h = harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer)
        w.unpack_from_host(layer, pinned, None if staged else staging)   # the other form back
        torch.cuda.synchronize()
        oracle.unpack(g, 0, dst_h, b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
        assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer), dst_h)
    del w
    torch.cuda.empty_cache()


def test_side_stream_overlap_run_is_bit_exact(dev, variant):
    """The layer-by-layer side-stream issue under the GEMM stand-in (reduced: 6 layers, ring of
    4 pinned slots): what lands in pinned memory is the oracle's wire slab of that layer."""
    if variant == 1:
        pytest.skip("the overlap driver is kernel-family agnostic; run once")
    from paper_2607_28633_b200 import overlap
    spec = wl.with_layers(wl.CFG5, 6)
    w = harness.setup(spec, dev, need_dst=False, need_wire=False)
    b, s = w.batch, spec
    g = _geom(s, b.num_pool_pages, 1, 0, 0)
    slots = 4
    pre = overlap.PrefillStandIn(dev, 7, tokens=1024, hidden=2048, ffn=4096)
    staging = torch.zeros(w.n_layer, dtype=torch.uint8, device=dev)
    for st in (staging, None):
        pinned = torch.zeros(slots * w.n_layer, dtype=torch.uint8).pin_memory()
        r = overlap.run_overlap(w, pinned, st, pre, slots=slots, warmup_layers=1)
        # timing figures are only sanity-checked: on a cold box the overlapped pass can be slower
        # than the serial one, so the hidden fraction of this tiny case may even be negative
        assert r.layers == 6 and r.t_xfer_serial_ms > 0 and r.exposed_ms >= 0 and r.hidden <= 1.0
        assert r.hidden_upper_bound == pytest.approx(1 - 1 / 6)
        # the ring holds the last `slots` layers: 2, 3 in slots 2, 3 and 4, 5 in slots 0, 1
        for layer in (2, 3, 4, 5):
            src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
            want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
            slot = layer % slots
            assert np.array_equal(pinned[slot * w.n_layer:(slot + 1) * w.n_layer].numpy(), want)
    del w
    torch.cuda.empty_cache()


def test_cfg5_full_size_overlap_run(dev, variant):
    """The overlap workload at full size as bench.py runs it: 80 layers, 4 x 4096 tokens, the
    full-size GEMM stand-in on the main stream, every layer shipped to its own pinned slab by
    the side stream (staged form, issued with topkv_pack_layers_to_host_pipelined). Every
    layer's pinned slab is compared in full with the oracle's wire slab, and a few sampled
    tokens with what the oracle computes for them one by one."""
    if variant == 1:
        pytest.skip("the overlap driver is kernel-family agnostic; run once")
    from paper_2607_28633_b200 import overlap
    spec = wl.CFG5
    w = harness.setup(spec, dev, need_dst=False, need_wire=False)
    b, s = w.batch, spec
    g = _geom(s, b.num_pool_pages, 1, 0, 0)
    try:
        pinned = torch.zeros(s.L * w.n_layer, dtype=torch.uint8).pin_memory()
    except RuntimeError:
        pytest.skip("this box refuses 5 GiB of pinned memory")
    staging = torch.zeros(w.n_layer, dtype=torch.uint8, device=dev)
    pre = overlap.PrefillStandIn(dev, 11)
    r = overlap.run_overlap(w, pinned, staging, pre)
    assert r.layers == 80 and r.hidden_upper_bound == pytest.approx(1 - 1 / 80)
    assert 0.0 <= r.exposed_ms and r.hidden <= 1.0
    host = pinned.numpy()
    for layer in range(s.L):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
        want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=16)
        assert np.array_equal(host[layer * w.n_layer:(layer + 1) * w.n_layer], want), layer
    rng = np.random.default_rng(8)
    cu = np.concatenate([[0], np.cumsum(b.seq_lens.astype(np.int64))])
    for layer in (0, 37, 79):
        for _ in range(3):
            q = int(rng.integers(0, s.R))
            i = int(rng.integers(0, b.seq_lens[q]))
            wo = layer * w.n_layer + (int(cu[q]) + i) * s.tok_bytes
            po = layer * w.slab_bytes + int(b.src_block_table[q, i // s.P]) * s.page_bytes
            page_h = w.src_pool[po:po + s.page_bytes].cpu().numpy()
            assert np.array_equal(_oracle_token(s, page_h, i % s.P), host[wo:wo + s.tok_bytes]), \
                (layer, q, i)
    del w, pinned, staging, pre
    torch.cuda.empty_cache()


@pytest.mark.parametrize("streams_per_direction", [1, 2])
def test_relay_through_host_on_two_streams(dev, streams_per_direction):
    """pack_to_host on one set of streams, unpack_from_host on another, gated per layer by an
    event (with two streams per direction, each with its own staging slab, the copy engine moves
    layer l while the kernel of layer l + 1 runs: the configuration bench.py times as e2e): the
    destination pool ends up as the oracle's unpack of the oracle's pack."""
    L, k = 5, streams_per_direction
    spec = wl.with_layers(wl.CFG2, L)
    w = harness.setup(spec, dev)
    b = w.batch
    g = _geom(spec, b.num_pool_pages, 1, 0, 0)
    tx = [torch.cuda.Stream(dev) for _ in range(k)]
    rx = [torch.cuda.Stream(dev) for _ in range(k)]
    pinned = torch.zeros(L * w.n_layer, dtype=torch.uint8).pin_memory()
    st_tx = [torch.zeros(w.n_layer, dtype=torch.uint8, device=dev) for _ in range(k)]
    st_rx = [torch.zeros(w.n_layer, dtype=torch.uint8, device=dev) for _ in range(k)]
    before = [harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l) for l in range(L)]
    for layer in range(L):
        q = layer % k
        w.pack_to_host(layer, pinned, st_tx[q], tx[q])
        ev = torch.cuda.Event()
        ev.record(tx[q])
        rx[q].wait_event(ev)
        w.unpack_from_host(layer, pinned, st_rx[q], rx[q])
    torch.cuda.synchronize()
    for layer in range(L):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
        want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
        assert np.array_equal(pinned[layer * w.n_layer:(layer + 1) * w.n_layer].numpy(), want)
        oracle.unpack(g, 0, before[layer], b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
        assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer), before[layer])
    del w
    torch.cuda.empty_cache()


@pytest.mark.parametrize("staged", [True, False])
def test_pipelined_layer_range_calls(dev, staged):
    """topkv_pack_layers_to_host_pipelined / topkv_unpack_layers_from_host_pipelined: one call
    per side enqueues the whole layer-by-layer transfer, gated by per-layer events. Sender and
    receiver run on two streams; the receiver's layer_ready are the sender's layer_done."""
    spec = wl.with_layers(wl.CFG2, 4)
    w = harness.setup(spec, dev, need_wire=False)
    b = w.batch
    g = _geom(spec, b.num_pool_pages, 1, 0, 0)
    L, n = 4, w.n_layer
    pinned = torch.zeros(L * n, dtype=torch.uint8).pin_memory()
    st_tx = torch.zeros(n, dtype=torch.uint8, device=dev) if staged else None
    st_rx = torch.zeros(n, dtype=torch.uint8, device=dev) if staged else None
    cap = n if staged else 0
    before = [harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l) for l in range(L)]
    main = torch.cuda.current_stream(dev)
    tx, rx = torch.cuda.Stream(dev, priority=-1), torch.cuda.Stream(dev)
    x = torch.randn(2048, 2048, device=dev)
    ready = []
    for layer in range(L):                               # stands for the prefill of layer l
        x = (x @ x.T) * 1e-3
        ev = torch.cuda.Event()
        ev.record(main)
        ready.append(ev if layer != 2 else None)         # a missing entry means "no wait"
    main.synchronize()                                   # layer 2 has no event: it must be ready
    sent = [torch.cuda.Event() for _ in range(L)]
    # layers 1..3 first, then layer 0 alone: ranges are independent calls
    tk.check(tk.topkv_pack_layers_to_host_pipelined(1, 3, w.src_pool, w.layout, w.src_batch, pinned,
                                                    pinned.numel(), st_tx, cap, ready[1:], sent[1:], tx))
    tk.check(tk.topkv_pack_layers_to_host_pipelined(0, 1, w.src_pool, w.layout, w.src_batch, pinned,
                                                    pinned.numel(), st_tx, cap, ready[:1], sent[:1], tx))
    tk.check(tk.topkv_unpack_layers_from_host_pipelined(0, L, w.dst_pool, w.layout, w.dst_batch, pinned,
                                                        pinned.numel(), st_rx, cap, sent, None, rx))
    torch.cuda.synchronize()
    for layer in range(L):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
        want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
        assert np.array_equal(pinned[layer * n:(layer + 1) * n].numpy(), want)
        oracle.unpack(g, 0, before[layer], b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
        assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer), before[layer])
    # errors are found for the whole range before anything is enqueued
    launches = tk.topkv_kernel_launch_count()
    assert tk.topkv_pack_layers_to_host_pipelined(2, 3, w.src_pool, w.layout, w.src_batch, pinned,
                                                  pinned.numel(), st_tx, cap, None, None, tx) \
        == tk.TOPKV_ERR_LAYER_RANGE
    assert tk.topkv_pack_layers_to_host_pipelined(0, L, w.src_pool, w.layout, w.src_batch, pinned,
                                                  pinned.numel() - 16, st_tx, cap, None, None, tx) \
        == tk.TOPKV_ERR_CAPACITY
    assert tk.topkv_kernel_launch_count() == launches
    assert tk.topkv_pack_layers_to_host_pipelined(0, 0, w.src_pool, w.layout, w.src_batch, pinned,
                                                  pinned.numel(), st_tx, cap, None, None, tx) == tk.TOPKV_OK
    del w
    torch.cuda.empty_cache()


@pytest.mark.parametrize("seed", range(10))
def test_many_layers_in_one_launch(dev, seed, variant):
    """topkv_pack_layers / topkv_unpack_layers equal the oracle's per-layer pack / unpack for a
    range of layers of the layout (random geometries: strided and head-split pools, both wire
    orders, padded wire slabs, empty batches); the layer outside the range is untouched."""
    g, sl, bt_s, bt_d, rng = _case(seed)
    g.L = 3
    g.W_layer = max(g.W_layer, 16)                     # several layers need distinct slabs
    if seed % 2:                                       # slab strides that are 16 mod 32: layer 1's
        g.W_layer += 16 if g.W_layer % 32 == 0 else 0  # slabs are then only 16-byte aligned
    lo = _layout_from_geom(g)
    T = int(sl.sum())
    src_h = rng.integers(0, 256, g.L * g.S_layer, dtype=np.uint8)
    fill_h = rng.integers(0, 256, g.L * g.S_layer, dtype=np.uint8)
    wire_len = g.L * g.W_layer + 32
    src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(fill_h.copy()).to(dev)
    wire = torch.full((wire_len,), 0x3C, dtype=torch.uint8, device=dev)
    d_sl = torch.from_numpy(sl).to(dev)
    d_bs, d_bd = torch.from_numpy(bt_s).to(dev), torch.from_numpy(bt_d).to(dev)
    know_T = seed % 2 == 0
    bs = tk.make_batch(d_bs, d_sl, T if know_T else -1)
    bd = tk.make_batch(d_bd, d_sl, T if know_T else -1)
    first, count = (1, g.L - 1) if seed % 3 else (0, g.L)
    if count > 1 and (g.W_layer % 32 or g.S_layer % 32):
        assert tk.topkv_copy_vector_bytes(first, count, src, lo, bs, wire, wire.numel()) == 16
    tk.check(tk.topkv_pack_layers(first, count, src, lo, bs, wire, wire.numel()))
    want_wire = np.full(wire_len, 0x3C, dtype=np.uint8)
    want_dst = fill_h.copy()
    for layer in range(first, first + count):
        oracle.pack(g, layer, src_h, bt_s, sl, wire=want_wire)
        oracle.unpack(g, layer, want_dst, bt_d, sl, want_wire)
    torch.cuda.synchronize()
    assert np.array_equal(wire.cpu().numpy(), want_wire)
    tk.check(tk.topkv_unpack_layers(first, count, dst, lo, bd, wire, wire.numel()))
    torch.cuda.synchronize()
    assert np.array_equal(dst.cpu().numpy(), want_dst)
    assert np.array_equal(src.cpu().numpy(), src_h)
    assert tk.topkv_pack_layers(1, g.L, src, lo, bs, wire, wire.numel()) == tk.TOPKV_ERR_LAYER_RANGE
    assert tk.topkv_pack_layers(0, 0, src, lo, bs, wire, wire.numel()) == tk.TOPKV_OK


def test_many_layers_in_one_launch_with_padded_slabs(dev, variant):
    """32-byte aligned buffers and a first layer of 0, but layer strides that are 16 mod 32 (a
    padded wire slab, a padded pool slab): every later layer's slab is only 16-byte aligned, so
    the launch must use 16-byte accesses; bytes equal the oracle's."""
    rng = np.random.default_rng(4242)
    L, R, P = 4, 3, 16
    sl = np.array([40, 16, 33], dtype=np.int32)
    pages = (sl + P - 1) // P
    npages = int(pages.sum()) + 2
    for pad_wire, pad_pool in ((16, 0), (0, 16), (16, 16), (48, 80)):
        g = Geom(L=L, F=2, h_kv=2, d_h=64, b_p=2, P=P, num_pages=npages)
        g.S_layer += pad_pool
        T = int(sl.sum())
        g.W_layer = g.wire_layer_bytes(T) + pad_wire
        assert g.wire_layer_bytes(T) % 32 == 0
        bt_s = np.full((R, 3), -1, dtype=np.int32)
        bt_d = np.full((R, 3), -1, dtype=np.int32)
        ps, pd, pos = rng.permutation(npages), rng.permutation(npages), 0
        for r in range(R):
            bt_s[r, :pages[r]] = ps[pos:pos + pages[r]]
            bt_d[r, :pages[r]] = pd[pos:pos + pages[r]]
            pos += pages[r]
        lo = _layout_from_geom(g)
        src_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
        dst_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
        src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h).to(dev)
        wire = torch.full((L * g.W_layer,), 0x5C, dtype=torch.uint8, device=dev)
        assert src.data_ptr() % 32 == 0 and dst.data_ptr() % 32 == 0 and wire.data_ptr() % 32 == 0
        d_sl = torch.from_numpy(sl).to(dev)
        bs = tk.make_batch(torch.from_numpy(bt_s).to(dev), d_sl, T)
        bd = tk.make_batch(torch.from_numpy(bt_d).to(dev), d_sl, T)
        assert tk.topkv_copy_vector_bytes(0, L, src, lo, bs, wire, wire.numel()) == 16
        assert tk.topkv_copy_vector_bytes(0, 1, src, lo, bs, wire, wire.numel()) == 32
        tk.check(tk.topkv_pack_layers(0, L, src, lo, bs, wire, wire.numel()))
        tk.check(tk.topkv_unpack_layers(0, L, dst, lo, bd, wire, wire.numel()))
        torch.cuda.synchronize()
        want = np.full(L * g.W_layer, 0x5C, dtype=np.uint8)
        for layer in range(L):
            oracle.pack(g, layer, src_h, bt_s, sl, wire=want)
            oracle.unpack(g, layer, dst_h, bt_d, sl, want)
        assert np.array_equal(wire.cpu().numpy(), want), (pad_wire, pad_pool)
        assert np.array_equal(dst.cpu().numpy(), dst_h), (pad_wire, pad_pool)


def test_many_layers_in_one_launch_cfg1(dev, variant):
    w = harness.setup(wl.CFG1, dev)
    b, s = w.batch, wl.CFG1
    g = _geom(s, b.num_pool_pages, s.L, 0, w.n_layer)
    src_h, dst_h = w.src_pool.cpu().numpy(), w.dst_pool.cpu().numpy()
    tk.check(tk.topkv_pack_layers(0, s.L, w.src_pool, w.layout, w.src_batch, w.wire, w.wire.numel()))
    tk.check(tk.topkv_unpack_layers(0, s.L, w.dst_pool, w.layout, w.dst_batch, w.wire, w.wire.numel()))
    torch.cuda.synchronize()
    want = np.zeros(s.L * w.n_layer, dtype=np.uint8)
    for layer in range(s.L):
        oracle.pack(g, layer, src_h, b.src_block_table, b.seq_lens, wire=want)
        oracle.unpack(g, layer, dst_h, b.dst_block_table, b.seq_lens, want)
    assert np.array_equal(w.wire.cpu().numpy(), want)
    assert np.array_equal(w.dst_pool.cpu().numpy(), dst_h)


def test_smoke_entry(dev):
    import __graft_entry__ as entry
    entry.smoke()


# -------------------------------------------------------------------- huge pages, hybrid models (§2.2)

@pytest.mark.parametrize("F,H,D,P", [(2, 8, 128, 256), (1, 1, 576, 512), (2, 2, 64, 300), (2, 8, 128, 64)])
def test_pages_far_larger_than_a_span_are_split_between_ctas(dev, F, H, D, P):
    """Pages of 256 KiB to 1 MiB: several CTAs share a page, each taking a run of its tokens;
    ragged lengths end in the middle of a CTA's run, windows start in the middle of one."""
    rng = np.random.default_rng(P + D)
    sl = np.array([P + 37, 0, 3 * P, 1, 2 * P - 1], dtype=np.int32)
    R = len(sl)
    pages = (sl + P - 1) // P
    maxp = int(pages.max()) + 1
    npages = int(pages.sum()) + 2
    for order in (0, 1):
        for window in (0, P // 2 + 5):
            g = Geom(L=2, F=F, h_kv=H, d_h=D, b_p=2, P=P, num_pages=npages, wire_order=order,
                     window=window)
            T = g.kept_tokens(sl)
            g.W_layer = g.wire_layer_bytes(T)
            bt_s = np.full((R, maxp), -1, dtype=np.int32)
            bt_d = np.full((R, maxp), -1, dtype=np.int32)
            ps, pd, pos = rng.permutation(npages), rng.permutation(npages), 0
            for r in range(R):
                bt_s[r, :pages[r]] = ps[pos:pos + pages[r]]
                bt_d[r, :pages[r]] = pd[pos:pos + pages[r]]
                pos += pages[r]
            lo = _layout_from_geom(g)
            src_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
            dst_h = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
            src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h).to(dev)
            wire = torch.zeros(2 * g.W_layer, dtype=torch.uint8, device=dev)
            d_sl = torch.from_numpy(sl).to(dev)
            bs = tk.make_batch(torch.from_numpy(bt_s).to(dev), d_sl, T, None, 0, window)
            bd = tk.make_batch(torch.from_numpy(bt_d).to(dev), d_sl, T, None, 0, window)
            want = np.zeros(2 * g.W_layer, dtype=np.uint8)
            for layer in range(2):
                tk.check(tk.topkv_pack_layer(layer, src, lo, bs, wire, wire.numel()))
                tk.check(tk.topkv_unpack_layer(layer, dst, lo, bd, wire, wire.numel()))
                oracle.pack(g, layer, src_h, bt_s, sl, wire=want, impl="rows")
                oracle.unpack(g, layer, dst_h, bt_d, sl, want, impl="rows")
            torch.cuda.synchronize()
            assert np.array_equal(wire.cpu().numpy(), want), (order, window)
            assert np.array_equal(dst.cpu().numpy(), dst_h), (order, window)


def _hybrid(dev, kinds, H, D, P, sl, state_slot_stride, rng, F=2, wire_order=0):
    """Device and host side of a hybrid model: paged pools for the attention layers, slot pools
    for the state layers, source and destination each with their own tables and slots."""
    R = len(sl)
    n_att = sum(k[0] != "state" for k in kinds)
    n_state = len(kinds) - n_att
    pages = (sl + P - 1) // P
    maxp = max(int(pages.max()), 1)
    npages = int(pages.sum()) + 3
    g = Geom(L=max(n_att, 1), F=F, h_kv=H, d_h=D, b_p=2, P=P, num_pages=npages, wire_order=wire_order)
    n_slots = R + 2
    S_sl = n_slots * state_slot_stride + 32
    side = {}
    for name in ("src", "dst"):
        bt = np.full((R, maxp), -1, dtype=np.int32)
        perm, pos = rng.permutation(npages), 0
        for r in range(R):
            bt[r, :pages[r]] = perm[pos:pos + pages[r]]
            pos += pages[r]
        pool = rng.integers(0, 256, g.pool_bytes(), dtype=np.uint8)
        sp = rng.integers(0, 256, max(n_state * S_sl, 16), dtype=np.uint8)
        slots = rng.permutation(n_slots)[:R].astype(np.int32)
        side[name] = dict(bt=bt, pool=pool, sp=sp, slots=slots,
                          d_bt=torch.from_numpy(bt).to(dev), d_pool=torch.from_numpy(pool).to(dev),
                          d_sp=torch.from_numpy(sp).to(dev), d_slots=torch.from_numpy(slots).to(dev))
    code = {"full": tk.TOPKV_LAYER_FULL, "window": tk.TOPKV_LAYER_WINDOW, "state": tk.TOPKV_LAYER_STATE}
    specs = [(code[k[0]], k[1] if len(k) > 1 else 0) for k in kinds]
    lo = _layout_from_geom(g)
    d_sl = torch.from_numpy(sl).to(dev)
    T = int(sl.sum())
    for name in ("src", "dst"):
        s = side[name]
        s["batch"] = tk.make_batch(s["d_bt"], d_sl, T)
        s["table"] = tk.make_layer_table(specs, sl, s["d_sp"] if n_state else None,
                                         s["d_slots"] if n_state else None, S_sl, state_slot_stride,
                                         n_slots)
    return g, lo, side, S_sl


@pytest.mark.parametrize("seed", range(6))
def test_hybrid_model_layers_device_to_device(dev, seed):
    """Full, windowed and constant-state layers in mixed order through topkv_pack_model_layers /
    topkv_unpack_model_layers: the wire is the oracle's layered pack (slabs back to back in model
    order, offsets equal), the destination pools the oracle's layered unpack, untouched bytes
    included; ranges of layers leave the other slabs alone."""
    rng = np.random.default_rng(3100 + seed)
    H, D, P = [(8, 64, 16), (1, 128, 4), (2, 64, 1)][seed % 3]
    F = 1 if seed == 4 else 2
    state_a, state_b = 48 * 1024 + 16 * (seed % 3), 300 * 1024      # one below, one above a CTA's span
    kinds = [("full",), ("window", 5), ("state", state_a), ("window", 1), ("state", state_b),
             ("full",), ("window", 1000)]
    if seed % 2:
        kinds = kinds[::-1]
    R = int(rng.integers(1, 6))
    sl = rng.integers(0, 5 * P + 3, size=R).astype(np.int32)
    if seed % 3 == 0:
        sl[int(rng.integers(0, R))] = 0
    slot_stride = 304 * 1024
    g, lo, side, S_sl = _hybrid(dev, kinds, H, D, P, sl, slot_stride, rng, F=F, wire_order=seed % 2)
    s, d = side["src"], side["dst"]
    want, off = oracle.pack_layered(g, kinds, s["pool"], s["bt"], sl, s["sp"], S_sl, slot_stride, s["slots"])
    st, got_off = tk.topkv_layer_table_offsets(lo, s["table"], R)
    assert st == tk.TOPKV_OK and np.array_equal(got_off, off)
    assert int(off[-1]) == sum(oracle.kv_bytes_layered(H, D, int(x), kinds, F=F) for x in sl)
    L = len(kinds)
    total = int(off[-1])
    wire = torch.full((total + 64,), 0x3C, dtype=torch.uint8, device=dev)
    # in two ranges, the later one first
    tk.check(tk.topkv_pack_model_layers(3, L - 3, s["d_pool"], lo, s["batch"], s["table"], wire, total))
    torch.cuda.synchronize()
    assert (wire[:int(off[3])] == 0x3C).all()
    tk.check(tk.topkv_pack_model_layers(0, 3, s["d_pool"], lo, s["batch"], s["table"], wire, total))
    torch.cuda.synchronize()
    got = wire.cpu().numpy()
    assert np.array_equal(got[:total], want[:total]) and (got[total:] == 0x3C).all()
    tk.check(tk.topkv_unpack_model_layers(0, L, d["d_pool"], lo, d["batch"], d["table"], wire, total))
    torch.cuda.synchronize()
    oracle.unpack_layered(g, kinds, d["pool"], d["bt"], sl, want, d["sp"], S_sl, slot_stride, d["slots"])
    assert np.array_equal(d["d_pool"].cpu().numpy(), d["pool"])
    assert np.array_equal(d["d_sp"].cpu().numpy(), d["sp"])
    assert np.array_equal(s["d_pool"].cpu().numpy(), s["pool"])          # sources untouched
    assert np.array_equal(s["d_sp"].cpu().numpy(), s["sp"])
    # errors are found for the whole range before anything is launched
    before = tk.topkv_kernel_launch_count()
    assert tk.topkv_pack_model_layers(0, L + 1, s["d_pool"], lo, s["batch"], s["table"], wire, total) \
        == tk.TOPKV_ERR_LAYER_RANGE
    assert tk.topkv_pack_model_layers(0, L, s["d_pool"], lo, s["batch"], s["table"], wire, total - 16) \
        == tk.TOPKV_ERR_CAPACITY
    assert tk.topkv_kernel_launch_count() == before


@pytest.mark.parametrize("staged", [True, False])
def test_gpt_oss_shaped_hybrid_through_the_side_stream_schedule(dev, staged, golden):
    """A gpt-oss-shaped model (§2.2: 36 layers, every other one windowed at 128 tokens, 8 KV
    heads of 64) through the pipelined side-stream calls: the sender ships model layer l after
    its event, the receiver places it after the sender's done-event. What lands in pinned memory
    is the oracle's layered wire, its size Eq. 1 per layer kind (0.15 binary GB per 4K-token
    request), and the destination pool the oracle's layered unpack."""
    rng = np.random.default_rng(77)
    gd = golden("paper_values.txt")
    L, nw = int(gd["layered.gpt_oss_120b.layers"]), int(gd["layered.gpt_oss_120b.windowed"])
    kinds = [("window", 128) if l % 2 == 0 else ("full",) for l in range(L)]
    assert sum(k[0] == "window" for k in kinds) == nw
    sl = np.array([4096, 700, 128, 129, 2049], dtype=np.int32)
    R = len(sl)
    g, lo, side, _ = _hybrid(dev, kinds, 8, 64, 16, sl, 16, rng)
    s, d = side["src"], side["dst"]
    want, off = oracle.pack_layered(g, kinds, s["pool"], s["bt"], sl)
    total = int(off[-1])
    per_request = [oracle.kv_bytes_layered(8, 64, int(x), kinds) for x in sl]
    assert total == sum(per_request)
    assert round(per_request[0] / 2**30, 2) == float(gd["layered.gpt_oss_120b.gb"])
    st, got_off = tk.topkv_layer_table_offsets(lo, s["table"], R)
    assert st == tk.TOPKV_OK and np.array_equal(got_off, off)
    pinned = torch.full((total,), 0x99, dtype=torch.uint8).pin_memory()
    biggest = int(np.diff(off).max())
    st_tx = torch.empty(biggest, dtype=torch.uint8, device=dev) if staged else None
    st_rx = torch.empty(biggest, dtype=torch.uint8, device=dev) if staged else None
    cap = biggest if staged else 0
    main = torch.cuda.current_stream(dev)
    tx, rx = torch.cuda.Stream(dev, priority=-1), torch.cuda.Stream(dev)
    x = torch.randn(1024, 1024, device=dev)
    ready = []
    for layer in range(L):                               # stands for the prefill of layer l
        x = (x @ x.T) * 1e-3
        ev = torch.cuda.Event()
        ev.record(main)
        ready.append(ev)
    sent = [torch.cuda.Event() for _ in range(L)]
    tk.check(tk.topkv_pack_model_layers_to_host_pipelined(
        0, L, s["d_pool"], lo, s["batch"], s["table"], pinned, total, st_tx, cap, ready, sent, tx))
    tk.check(tk.topkv_unpack_model_layers_from_host_pipelined(
        0, L, d["d_pool"], lo, d["batch"], d["table"], pinned, total, st_rx, cap, sent, None, rx))
    torch.cuda.synchronize()
    assert np.array_equal(pinned.numpy(), want[:total])
    oracle.unpack_layered(g, kinds, d["pool"], d["bt"], sl, want)
    assert np.array_equal(d["d_pool"].cpu().numpy(), d["pool"])
    # a staging slab smaller than the largest slab of the range is refused before any launch
    if staged:
        before = tk.topkv_kernel_launch_count()
        assert tk.topkv_pack_model_layers_to_host_pipelined(
            0, L, s["d_pool"], lo, s["batch"], s["table"], pinned, total, st_tx, biggest - 16, None,
            None, tx) == tk.TOPKV_ERR_CAPACITY
        assert tk.topkv_kernel_launch_count() == before


def test_qwen_shaped_hybrid_with_state_layers_through_the_host(dev):
    """Three of every four layers carry a constant state (§2.2's 45-of-60 split, shortened to 12
    layers): staged side-stream transfer of attention and state slabs alike."""
    rng = np.random.default_rng(78)
    state = 512 * 1024
    kinds = [("full",) if l % 4 == 3 else ("state", state) for l in range(12)]
    sl = np.array([333, 64, 1000], dtype=np.int32)
    g, lo, side, S_sl = _hybrid(dev, kinds, 2, 256, 16, sl, state, rng)
    s, d = side["src"], side["dst"]
    want, off = oracle.pack_layered(g, kinds, s["pool"], s["bt"], sl, s["sp"], S_sl, state, s["slots"])
    total = int(off[-1])
    assert total == sum(oracle.kv_bytes_layered(2, 256, int(x), kinds) for x in sl)
    assert off[1] - off[0] == len(sl) * state
    pinned = torch.zeros(total, dtype=torch.uint8).pin_memory()
    biggest = int(np.diff(off).max())
    staging = torch.empty(biggest, dtype=torch.uint8, device=dev)
    stream = torch.cuda.Stream(dev)
    stream.wait_stream(torch.cuda.current_stream(dev))
    L = len(kinds)
    tk.check(tk.topkv_pack_model_layers_to_host_pipelined(
        0, L, s["d_pool"], lo, s["batch"], s["table"], pinned, total, staging, biggest, None, None, stream))
    tk.check(tk.topkv_unpack_model_layers_from_host_pipelined(
        0, L, d["d_pool"], lo, d["batch"], d["table"], pinned, total, None, 0, None, None, stream))
    stream.synchronize()
    assert np.array_equal(pinned.numpy(), want[:total])
    oracle.unpack_layered(g, kinds, d["pool"], d["bt"], sl, want, d["sp"], S_sl, state, d["slots"])
    assert np.array_equal(d["d_pool"].cpu().numpy(), d["pool"])
    assert np.array_equal(d["d_sp"].cpu().numpy(), d["sp"])


# -------------------------------------------------------------------- span links

def _linked_chain(w, lo1, slab, stream, flags_p, flags_u, epoch0, layers):
    """pack(l) -> unpack(l) -> pack(l+1) -> ... through ONE slab, every launch linked span by span
    to the one it depends on: unpack(l) awaits pack(l); pack(l+1) awaits unpack(l)."""
    b = w.batch
    bs = tk.make_batch(w.src_bt, w.seq_lens, b.total_tokens, w.cu)
    bd = tk.make_batch(w.dst_bt, w.seq_lens, b.total_tokens, w.cu)
    e = epoch0
    for k, l in enumerate(layers):
        lp = tk.make_span_link(flags_u if e else None, e, flags_p, e + 1)   # e = 0: nothing before it
        tk.check(tk.topkv_pack_layer_linked(l, w.src_pool, lo1, bs, slab, slab.numel(), lp, stream))
        lu = tk.make_span_link(flags_p, e + 1, flags_u, e + 1)
        tk.check(tk.topkv_unpack_layer_linked(l, w.dst_pool, lo1, bd, slab, slab.numel(), lu, stream))
        e += 1
    return e


def test_span_linked_chain_through_one_slab(dev, variant):
    """Every kernel of the chain depends on the DATA of the kernel just before it (one shared
    wire slab), none waits for its predecessor as a whole: they are ordered span by span. The
    destination pool is the oracle's unpack of the oracle's pack for every layer, twice over
    (the flag arrays are reused with increasing epochs), with a copy right behind the chain."""
    if variant == 1:
        pytest.skip("span links belong to the vectorised family")
    spec = wl.with_layers(wl.CFG2, 6)
    w = harness.setup(spec, dev, need_wire=False)
    b, s = w.batch, spec
    g = _geom(s, b.num_pool_pages, 1, 0, 0)
    stream = torch.cuda.Stream(dev)
    lo1 = tk.make_layout(s.L, s.F, s.H, s.D, s.E, s.P, b.num_pool_pages)   # wire_layer_stride 0
    slab = torch.zeros(w.n_layer, dtype=torch.uint8, device=dev)
    words = tk.topkv_span_link_words(lo1, w.src_batch)
    assert words == s.R * b.max_pages_per_req                            # one 64 KiB page per span
    flags_p = torch.zeros(words, dtype=torch.int32, device=dev)
    flags_u = torch.zeros(words, dtype=torch.int32, device=dev)
    host_dst = torch.empty(w.dst_pool.numel(), dtype=torch.uint8).pin_memory()
    dst_before = [harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l) for l in range(s.L)]
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        e = _linked_chain(w, lo1, slab, stream, flags_p, flags_u, 0, range(s.L))
        e = _linked_chain(w, lo1, slab, stream, flags_p, flags_u, e, reversed(range(s.L)))
        host_dst.copy_(w.dst_pool, non_blocking=True)
    stream.synchronize()
    assert tk.topkv_device_error_flags() == 0
    assert int(flags_p.max()) == e and int(flags_u.max()) == e
    for l in range(s.L):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, l)
        want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
        oracle.unpack(g, 0, dst_before[l], b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
        assert np.array_equal(host_dst[l * w.slab_bytes:(l + 1) * w.slab_bytes].numpy(), dst_before[l]), l
    del w
    torch.cuda.empty_cache()


@pytest.mark.parametrize("seed", range(8))
def test_span_linked_pairs_random_geometries(dev, seed, variant):
    """Linked pack -> unpack pairs on small random geometries (empty requests and empty spans
    publish and await nothing, windows, strided pools, grouped small pages, both wire orders)."""
    if variant == 1:
        pytest.skip("span links belong to the vectorised family")
    g, sl, bt_s, bt_d, rng = _case(seed)
    if seed % 2:
        g.window = int(rng.choice([1, g.P, 2 * g.P + 1]))
    T = g.kept_tokens(sl)
    g.W_layer = g.wire_layer_bytes(T) + 16
    lo = _layout_from_geom(g)
    src_h = rng.integers(0, 256, g.L * g.S_layer, dtype=np.uint8)
    dst_h = rng.integers(0, 256, g.L * g.S_layer, dtype=np.uint8)
    src, dst = torch.from_numpy(src_h).to(dev), torch.from_numpy(dst_h).to(dev)
    wire = torch.full((g.L * g.W_layer + 32,), 0x3C, dtype=torch.uint8, device=dev)
    d_sl = torch.from_numpy(sl).to(dev)
    bs = tk.make_batch(torch.from_numpy(bt_s).to(dev), d_sl, T, None, 0, g.window)
    bd = tk.make_batch(torch.from_numpy(bt_d).to(dev), d_sl, T, None, 0, g.window)
    words = tk.topkv_span_link_words(lo, bs)
    assert words >= 0
    flags = torch.zeros(max(words, 1) * g.L, dtype=torch.int32, device=dev)
    stream = torch.cuda.Stream(dev)
    stream.wait_stream(torch.cuda.current_stream(dev))
    want = np.full(g.L * g.W_layer + 32, 0x3C, dtype=np.uint8)
    for layer in range(g.L):
        f = flags[layer * max(words, 1):(layer + 1) * max(words, 1)]
        tk.check(tk.topkv_pack_layer_linked(layer, src, lo, bs, wire, wire.numel(),
                                            tk.make_span_link(None, 0, f, 7), stream))
        tk.check(tk.topkv_unpack_layer_linked(layer, dst, lo, bd, wire, wire.numel(),
                                              tk.make_span_link(f, 7, None, 0), stream))
        oracle.pack(g, layer, src_h, bt_s, sl, wire=want)
        oracle.unpack(g, layer, dst_h, bt_d, sl, want)
    stream.synchronize()
    assert np.array_equal(wire.cpu().numpy(), want)
    assert np.array_equal(dst.cpu().numpy(), dst_h)


def test_span_link_that_never_arrives_gives_up_and_reports(dev, variant):
    """An unpack linked to flags that nothing publishes: every CTA's bounded wait runs out (about
    half a second), the spans are skipped, bit 1 of the device status word is raised, the destination
    pool is untouched and the context stays usable."""
    if variant == 1:
        pytest.skip("span links belong to the vectorised family")
    w = harness.setup(wl.CFG1, dev)
    before = w.dst_pool.cpu().numpy()
    words = tk.topkv_span_link_words(w.layout, w.dst_batch)
    flags = torch.zeros(words, dtype=torch.int32, device=dev)
    torch.cuda.synchronize()
    tk.check(tk.topkv_unpack_layer_linked(0, w.dst_pool, w.layout, w.dst_batch, w.wire, w.wire.numel(),
                                          tk.make_span_link(flags, 5, None, 0)))
    assert tk.topkv_device_error_flags() == 1
    assert np.array_equal(w.dst_pool.cpu().numpy(), before)
    tk.check(tk.topkv_reset_device_error_flags())
    # the same call with the flags in place goes through
    flags.fill_(5)
    torch.cuda.synchronize()
    tk.check(tk.topkv_pack_layer(0, w.src_pool, w.layout, w.src_batch, w.wire, w.wire.numel()))
    tk.check(tk.topkv_unpack_layer_linked(0, w.dst_pool, w.layout, w.dst_batch, w.wire, w.wire.numel(),
                                          tk.make_span_link(flags, 5, None, 0)))
    assert tk.topkv_device_error_flags() == 0
    assert not np.array_equal(w.dst_pool.cpu().numpy(), before)


def test_two_lane_host_leg_relay(dev):
    """topkv_pack_layers_to_host_two_lanes / topkv_unpack_layers_from_host_two_lanes: the whole
    relay through pinned memory as two calls, each direction alternating between two streams and
    two staging slabs, the receiver gated by the sender's per-layer events. Pinned slabs and
    destination pool equal the oracle's, for an odd number of layers and for a sub-range."""
    L = 5
    spec = wl.with_layers(wl.CFG2, L)
    w = harness.setup(spec, dev, need_wire=False)
    b = w.batch
    g = _geom(spec, b.num_pool_pages, 1, 0, 0)
    n = w.n_layer
    pinned = torch.zeros(L * n, dtype=torch.uint8).pin_memory()
    tx = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    rx = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    st_tx = [torch.empty(n, dtype=torch.uint8, device=dev) for _ in range(2)]
    st_rx = [torch.empty(n, dtype=torch.uint8, device=dev) for _ in range(2)]
    before = [harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l) for l in range(L)]
    torch.cuda.synchronize()
    sent = [torch.cuda.Event() for _ in range(L)]
    # layers 1..4 first, then layer 0 on its own
    tk.check(tk.topkv_pack_layers_to_host_two_lanes(1, L - 1, w.src_pool, w.layout, w.src_batch, pinned,
                                                    pinned.numel(), st_tx, n, None, sent[1:], tx))
    tk.check(tk.topkv_pack_layers_to_host_two_lanes(0, 1, w.src_pool, w.layout, w.src_batch, pinned,
                                                    pinned.numel(), st_tx, n, None, sent[:1], tx))
    tk.check(tk.topkv_unpack_layers_from_host_two_lanes(0, L, w.dst_pool, w.layout, w.dst_batch, pinned,
                                                        pinned.numel(), st_rx, n, sent, None, rx))
    torch.cuda.synchronize()
    assert tk.topkv_device_error_flags() == 0
    for layer in range(L):
        src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
        want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
        assert np.array_equal(pinned[layer * n:(layer + 1) * n].numpy(), want), layer
        oracle.unpack(g, 0, before[layer], b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
        assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, layer), before[layer])
    # refused before anything is enqueued: one slab or one stream given twice, a missing slab
    launches = tk.topkv_kernel_launch_count()
    P2 = tk.topkv_pack_layers_to_host_two_lanes
    args = (0, L, w.src_pool, w.layout, w.src_batch, pinned, pinned.numel())
    assert P2(*args, [st_tx[0], st_tx[0]], n, None, None, tx) == tk.TOPKV_ERR_INVALID_ARG
    assert P2(*args, st_tx, n, None, None, [tx[0], tx[0]]) == tk.TOPKV_ERR_INVALID_ARG
    assert P2(*args, [st_tx[0], None], n, None, None, tx) == tk.TOPKV_ERR_INVALID_ARG
    assert P2(*args, st_tx, n - 16, None, None, tx) == tk.TOPKV_ERR_CAPACITY
    assert P2(2, L, w.src_pool, w.layout, w.src_batch, pinned, pinned.numel(), st_tx, n, None, None, tx) \
        == tk.TOPKV_ERR_LAYER_RANGE
    assert tk.topkv_kernel_launch_count() == launches
    del w
    torch.cuda.empty_cache()


def test_relay_layers_linked_one_call(dev, variant):
    """topkv_relay_layers_linked: a range of layers from one paged pool into another through ONE
    slab as a single call (2 launches per layer, all span-linked), twice with continuing epochs;
    the destination is the oracle's unpack of the oracle's pack, the source is untouched."""
    if variant == 1:
        pytest.skip("span links belong to the vectorised family")
    for name, L in (("cfg2", 5), ("cfg4", 3)):
        spec = wl.with_layers(wl.ALL[name], L)
        w = harness.setup(spec, dev, need_wire=False)
        b = w.batch
        g = _geom(spec, b.num_pool_pages, 1, 0, 0)
        slab = torch.zeros(w.n_layer, dtype=torch.uint8, device=dev)
        words = tk.topkv_span_link_words(w.layout, w.src_batch)
        flags = torch.zeros(2 * words, dtype=torch.int32, device=dev)
        before = [harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l) for l in range(L)]
        stream = torch.cuda.Stream(dev)
        stream.wait_stream(torch.cuda.current_stream(dev))
        args = (w.src_pool, w.layout, w.src_batch, w.dst_pool, w.layout, w.dst_batch, slab, slab.numel(),
                flags, flags.numel())
        tk.check(tk.topkv_relay_layers_linked(0, 2, *args, 0, stream))
        tk.check(tk.topkv_relay_layers_linked(2, L - 2, *args, 2, stream))      # epochs continue
        stream.synchronize()
        assert tk.topkv_device_error_flags() == 0 and int(flags.max()) == L
        for l in range(L):
            src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, l)
            want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
            oracle.unpack(g, 0, before[l], b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
            assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l), before[l]), (name, l)
        # refused before anything is launched
        launches = tk.topkv_kernel_launch_count()
        assert tk.topkv_relay_layers_linked(0, L + 1, *args, 0, stream) == tk.TOPKV_ERR_LAYER_RANGE
        assert tk.topkv_relay_layers_linked(0, L, *args[:8], flags, words, 0, stream) == tk.TOPKV_ERR_CAPACITY
        other = tk.make_layout(L, spec.F, spec.H, spec.D, spec.E, spec.P * 2, b.num_pool_pages)
        assert tk.topkv_relay_layers_linked(0, L, w.src_pool, w.layout, w.src_batch, w.dst_pool, other,
                                            w.dst_batch, slab, slab.numel(), flags, flags.numel(), 0,
                                            stream) == tk.TOPKV_ERR_UNSUPPORTED_LAYOUT
        assert tk.topkv_kernel_launch_count() == launches
        del w
        torch.cuda.empty_cache()


def test_linked_relay_captured_in_a_cuda_graph(dev, variant):
    """The linked relay of several layers through one slab captured in a CUDA graph together
    with the clearing of its flag array (the epochs are plain arguments, so every replay starts
    from cleared flags): nothing runs during the capture; after every replay, with new source
    contents each time, the destination is the oracle's unpack of the oracle's pack."""
    if variant == 1:
        pytest.skip("span links belong to the vectorised family")
    L = 4
    spec = wl.with_layers(wl.CFG2, L)
    w = harness.setup(spec, dev, need_wire=False)
    b = w.batch
    g = _geom(spec, b.num_pool_pages, 1, 0, 0)
    n = w.n_layer
    slab = torch.zeros(n, dtype=torch.uint8, device=dev)
    words = tk.topkv_span_link_words(w.layout, w.src_batch)
    flags = torch.zeros(2 * words, dtype=torch.int32, device=dev)
    stream = torch.cuda.Stream(dev)
    args = (w.src_pool, w.layout, w.src_batch, w.dst_pool, w.layout, w.dst_batch, slab, n, flags, flags.numel())
    with torch.cuda.stream(stream):                      # warm up outside the capture
        tk.check(tk.topkv_relay_layers_linked(0, 1, *args, 0, stream))
    stream.synchronize()
    dst0 = w.dst_pool.clone()
    flags.zero_()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        flags.zero_()
        tk.check(tk.topkv_relay_layers_linked(0, L, *args, 0, stream))
    assert not flags.any()                               # capturing executed nothing
    fresh = wl.fill_torch(2 * L * w.slab_bytes, 99, dev, raw_bits=True)
    for rep in range(2):
        w.src_pool.copy_(fresh[rep * L * w.slab_bytes:(rep + 1) * L * w.slab_bytes])
        w.dst_pool.copy_(dst0)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert tk.topkv_device_error_flags() == 0 and int(flags.max()) == L
        for l in range(L):
            src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, l)
            want = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
            dst_h = harness.layer_slab_to_numpy(dst0, w.slab_bytes, l)
            oracle.unpack(g, 0, dst_h, b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
            assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l), dst_h), (rep, l)
    del w, graph
    torch.cuda.empty_cache()


def test_linked_relay_many_calls_alternating_sources(dev, variant):
    """The linked relay called 120 times in a row through the same slab and the same flag arrays
    (epochs continuing), the source alternating at random between two pools with different
    contents: a span read before it was rewritten, or rewritten before it was read, would leave
    bytes of the other source in the destination. Checked against the oracle's result for the
    source of the last call, every few calls."""
    if variant == 1:
        pytest.skip("span links belong to the vectorised family")
    L = 3
    spec = wl.with_layers(wl.CFG2, L)
    w = harness.setup(spec, dev, need_wire=False)
    b = w.batch
    g = _geom(spec, b.num_pool_pages, 1, 0, 0)
    n = w.n_layer
    srcs = [w.src_pool, wl.fill_torch(w.src_pool.numel(), 4321, dev, raw_bits=True)]
    want = []                                             # the oracle's destination pool per source
    for src in srcs:
        pool = w.dst_pool.cpu().numpy().copy()
        for l in range(L):
            src_h = harness.layer_slab_to_numpy(src, w.slab_bytes, l)
            wire = oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens, impl="rows", threads=8)
            oracle.unpack(g, 0, pool[l * w.slab_bytes:(l + 1) * w.slab_bytes], b.dst_block_table, b.seq_lens,
                          wire, impl="rows", threads=8)
        want.append(torch.from_numpy(pool).to(dev))
    assert not torch.equal(want[0], want[1])
    slab = torch.zeros(n, dtype=torch.uint8, device=dev)
    words = tk.topkv_span_link_words(w.layout, w.src_batch)
    flags = torch.zeros(2 * words, dtype=torch.int32, device=dev)
    stream = torch.cuda.Stream(dev)
    stream.wait_stream(torch.cuda.current_stream(dev))
    rng = np.random.default_rng(3)
    epoch = 0
    for it in range(120):
        k = int(rng.integers(0, 2))
        tk.check(tk.topkv_relay_layers_linked(0, L, srcs[k], w.layout, w.src_batch, w.dst_pool, w.layout,
                                              w.dst_batch, slab, n, flags, flags.numel(), epoch, stream))
        epoch += L
        if it % 7 == 6 or it == 119:
            stream.synchronize()
            assert torch.equal(w.dst_pool, want[k]), it
    assert tk.topkv_device_error_flags() == 0 and int(flags.max()) == epoch
    del w, srcs, want
    torch.cuda.empty_cache()


def test_relay_call_right_behind_a_kernel_that_writes_its_source(dev, variant):
    """The first launch of topkv_relay_layers_linked is an ordinary launch towards what precedes
    the call (TOPKV_LINK_WAIT_PREVIOUS): kernels that rewrite the source pool and the plan are
    enqueued on the same stream right before it, with nothing in between, and the destination
    must hold the NEW source contents. The same with hand-made links whose first one carries
    the flag."""
    if variant == 1:
        pytest.skip("span links belong to the vectorised family")
    L = 3
    spec = wl.with_layers(wl.CFG2, L)
    w = harness.setup(spec, dev, need_wire=False)
    b = w.batch
    g = _geom(spec, b.num_pool_pages, 1, 0, 0)
    n = w.n_layer
    fresh = wl.fill_torch(2 * L * n, 4242, dev, raw_bits=True)          # two new contents for the source
    slab = torch.zeros(n, dtype=torch.uint8, device=dev)
    words = tk.topkv_span_link_words(w.layout, w.src_batch)
    cu = torch.zeros_like(w.cu)
    T = b.total_tokens
    bs = tk.make_batch(w.src_bt, w.seq_lens, T, cu)
    bd = tk.make_batch(w.dst_bt, w.seq_lens, T, cu)
    stream = torch.cuda.Stream(dev)
    lo1 = tk.make_layout(spec.L, spec.F, spec.H, spec.D, spec.E, spec.P, b.num_pool_pages)
    for round_, by_hand in enumerate((False, True)):
        flags = torch.zeros(2 * words, dtype=torch.int32, device=dev)
        cu.zero_()
        src_h = [harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, l) for l in range(L)]
        dst_h = [harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l) for l in range(L)]
        wire_in = fresh[round_ * L * n:(round_ + 1) * L * n]
        torch.cuda.synchronize()
        # the producers: the plan both sides read, and new contents for every source layer
        tk.check(tk.topkv_build_plan(tk.make_batch(w.src_bt, w.seq_lens), cu, stream))
        for l in range(L):
            tk.check(tk.topkv_unpack_layer(l, w.src_pool, w.layout, w.src_batch, wire_in, wire_in.numel(), stream))
        if not by_hand:
            tk.check(tk.topkv_relay_layers_linked(0, L, w.src_pool, w.layout, bs, w.dst_pool, w.layout, bd, slab,
                                                  n, flags, flags.numel(), 0, stream))
        else:
            fp, fu = flags[:words], flags[words:]
            for l in range(L):
                lp = tk.make_span_link(fu if l else None, l, fp, l + 1,
                                       tk.TOPKV_LINK_WAIT_PREVIOUS if l == 0 else 0)
                tk.check(tk.topkv_pack_layer_linked(l, w.src_pool, lo1, bs, slab, n, lp, stream))
                tk.check(tk.topkv_unpack_layer_linked(l, w.dst_pool, lo1, bd, slab, n,
                                                      tk.make_span_link(fp, l + 1, fu, l + 1), stream))
        stream.synchronize()
        assert tk.topkv_device_error_flags() == 0
        win = wire_in.cpu().numpy()
        for l in range(L):
            oracle.unpack(g, 0, src_h[l], b.src_block_table, b.seq_lens, win[l * n:(l + 1) * n],
                          impl="rows", threads=8)
            assert np.array_equal(harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, l), src_h[l]), l
            want = oracle.pack(g, 0, src_h[l], b.src_block_table, b.seq_lens, impl="rows", threads=8)
            oracle.unpack(g, 0, dst_h[l], b.dst_block_table, b.seq_lens, want, impl="rows", threads=8)
            assert np.array_equal(harness.layer_slab_to_numpy(w.dst_pool, w.slab_bytes, l), dst_h[l]), (by_hand, l)
    del w
    torch.cuda.empty_cache()


# -------------------------------------------------------------------- random call sequences

@pytest.mark.parametrize("seed", range(24))
def test_random_call_sequences_against_an_oracle_model(dev, seed, variant):
    """A random sequence of calls on one stream (pack, unpack, layer ranges, re-paging, linked
    pairs, staged and direct host legs; lengths from a plan or not, total stated or not, a
    window or not) with the flags a caller may legitimately set: TOPKV_FLAG_OVERLAP_PREVIOUS only
    when the call touches nothing that the calls since the last unflagged one touch,
    TOPKV_FLAG_TABLES_SETTLED always (the tables are never written by a kernel here). The same
    sequence is applied to numpy copies with the oracle; every buffer must agree at the end."""
    g, sl, bt_s, bt_d, rng = _case(seed)
    rng = np.random.default_rng(7000 + seed)
    W = int(rng.choice([0, 0, 1, g.P + 1, 3 * g.P]))
    g.window = W
    T = g.kept_tokens(sl)
    g.W_layer = g.wire_layer_bytes(T) + 16 * int(rng.integers(0, 3))
    lo = _layout_from_geom(g)
    nbytes = g.L * g.S_layer
    wire_len = g.L * g.W_layer + 32
    h = {"src": rng.integers(0, 256, nbytes, dtype=np.uint8), "dst": rng.integers(0, 256, nbytes, dtype=np.uint8),
         "wire": rng.integers(0, 256, wire_len, dtype=np.uint8), "host": rng.integers(0, 256, wire_len, dtype=np.uint8)}
    d = {k: torch.from_numpy(v.copy()).to(dev) for k, v in h.items() if k != "host"}
    pinned = torch.from_numpy(h["host"].copy()).pin_memory()
    staging = torch.zeros(max(g.W_layer, 16), dtype=torch.uint8, device=dev)
    d_sl = torch.from_numpy(sl).to(dev)
    d_bt = {"src": torch.from_numpy(bt_s).to(dev), "dst": torch.from_numpy(bt_d).to(dev)}
    h_bt = {"src": bt_s, "dst": bt_d}
    R = len(sl)
    cu = torch.zeros(R + 1, dtype=torch.int64, device=dev)
    tk.check(tk.topkv_build_plan(tk.make_batch(d_bt["src"], d_sl, window_tokens=W), cu))
    words = max(1, tk.topkv_span_link_words(lo, tk.make_batch(d_bt["src"], d_sl, T, None, 0, W)))
    link_flags = torch.zeros(words, dtype=torch.int32, device=dev)
    epoch = 0
    torch.cuda.synchronize()
    stream = torch.cuda.Stream(dev)
    since_unflagged = []          # (reads, writes) of the kernels since the last call without the flag

    def batch(side, flags):
        total = T if rng.integers(0, 2) else -1
        plan = cu if rng.integers(0, 2) else None
        return tk.make_batch(d_bt[side], d_sl, total, plan, flags, W)

    def flags_for(reads, writes, may_overlap=True):
        free = all(not (writes & (r2 | w2)) and not (reads & w2) for r2, w2 in since_unflagged)
        if may_overlap and since_unflagged and free and rng.integers(0, 2):
            since_unflagged.append((reads, writes))
            return tk.TOPKV_FLAG_OVERLAP_PREVIOUS
        since_unflagged[:] = [(reads, writes)]
        return tk.TOPKV_FLAG_TABLES_SETTLED if rng.integers(0, 2) else 0

    kinds = ["pack", "unpack", "pack_range", "unpack_range", "to_host", "from_host"]
    if W == 0:
        kinds.append("repage")
    if variant == 0:
        kinds.append("linked")
    for step in range(14):
        kind = str(rng.choice(kinds))
        layer = int(rng.integers(0, g.L))
        pool = str(rng.choice(["src", "dst"]))
        if kind == "pack":
            f = flags_for({(pool, layer)}, {("wire", layer)})
            tk.check(tk.topkv_pack_layer(layer, d[pool], lo, batch(pool, f), d["wire"], wire_len, stream))
            oracle.pack(g, layer, h[pool], h_bt[pool], sl, wire=h["wire"])
        elif kind == "unpack":
            f = flags_for({("wire", layer)}, {(pool, layer)})
            tk.check(tk.topkv_unpack_layer(layer, d[pool], lo, batch(pool, f), d["wire"], wire_len, stream))
            oracle.unpack(g, layer, h[pool], h_bt[pool], sl, h["wire"])
        elif kind in ("pack_range", "unpack_range"):
            first = int(rng.integers(0, g.L))
            n = int(rng.integers(1, g.L - first + 1))
            pools, wires = {(pool, l) for l in range(first, first + n)}, {("wire", l) for l in range(first, first + n)}
            if kind == "pack_range":
                f = flags_for(pools, wires)
                tk.check(tk.topkv_pack_layers(first, n, d[pool], lo, batch(pool, f), d["wire"], wire_len, stream))
                for l in range(first, first + n):
                    oracle.pack(g, l, h[pool], h_bt[pool], sl, wire=h["wire"])
            else:
                f = flags_for(wires, pools)
                tk.check(tk.topkv_unpack_layers(first, n, d[pool], lo, batch(pool, f), d["wire"], wire_len, stream))
                for l in range(first, first + n):
                    oracle.unpack(g, l, h[pool], h_bt[pool], sl, h["wire"])
        elif kind == "repage":
            other = "dst" if pool == "src" else "src"
            f = flags_for({(pool, layer)}, {(other, layer)})
            tk.check(tk.topkv_repage_layer(layer, d[pool], lo, batch(pool, f), d[other], lo, batch(other, f), stream))
            tmp = np.zeros(wire_len, dtype=np.uint8)
            oracle.pack(g, layer, h[pool], h_bt[pool], sl, wire=tmp)
            oracle.unpack(g, layer, h[other], h_bt[other], sl, tmp)
        elif kind == "linked":
            other = "dst" if pool == "src" else "src"
            since_unflagged[:] = []       # the first linked call waits for everything before it
            lp = tk.make_span_link(None, 0, link_flags, epoch + 1, tk.TOPKV_LINK_WAIT_PREVIOUS)
            tk.check(tk.topkv_pack_layer_linked(layer, d[pool], lo, batch(pool, 0), d["wire"], wire_len, lp, stream))
            lu = tk.make_span_link(link_flags, epoch + 1, None, 0)
            tk.check(tk.topkv_unpack_layer_linked(layer, d[other], lo, batch(other, 0), d["wire"], wire_len, lu,
                                                  stream))
            epoch += 1
            oracle.pack(g, layer, h[pool], h_bt[pool], sl, wire=h["wire"])
            oracle.unpack(g, layer, h[other], h_bt[other], sl, h["wire"])
            # the next call must not carry the overlap flag: make it see both kernels as unflagged work
            since_unflagged[:] = [({(pool, layer), ("wire", layer)}, {("wire", layer), (other, layer)})]
        else:
            staged = bool(rng.integers(0, 2))
            st, cap = (staging, staging.numel()) if staged else (None, 0)
            b = tk.make_batch(d_bt[pool], d_sl, T, cu if rng.integers(0, 2) else None, 0, W)
            since_unflagged[:] = []       # a copy, or a kernel without the flag
            if kind == "to_host":
                tk.check(tk.topkv_pack_layer_to_host(layer, d[pool], lo, b, pinned, wire_len, st, cap, stream))
                oracle.pack(g, layer, h[pool], h_bt[pool], sl, wire=h["host"])
                since_unflagged[:] = [({(pool, layer)}, {("host", layer)})]
            else:
                tk.check(tk.topkv_unpack_layer_from_host(layer, d[pool], lo, b, pinned, wire_len, st, cap, stream))
                oracle.unpack(g, layer, h[pool], h_bt[pool], sl, h["host"])
                since_unflagged[:] = [({("host", layer)}, {(pool, layer)})]
    stream.synchronize()
    assert tk.topkv_device_error_flags() == 0
    for k in ("src", "dst", "wire"):
        assert np.array_equal(d[k].cpu().numpy(), h[k]), k
    assert np.array_equal(pinned.numpy(), h["host"])
