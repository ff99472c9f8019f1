"""GPU parity of the sender / receiver session (per-layer checksummed host leg on two streams,
one 128-byte header per request, §3.4; receiver-side verification and retry, §3.1) against
the CPU oracle: destination pool, pinned wire, checksums and header bytes."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import oracle
from oracle import Geom
from paper_2607_28633_b200 import binding as tk
from paper_2607_28633_b200 import harness, session
from paper_2607_28633_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import __graft_entry__ as entry
    entry.build()
    tk.check(tk.topkv_reset_device_error_flags())
    return torch.device("cuda:0")


def _ends(dev, spec, layers=None):
    w = harness.setup(spec, dev, layers=layers, need_wire=False)
    tx = session.TransferSender(w.src_pool, w.layout, w.src_bt, w.seq_lens, w.batch.total_tokens)
    rx = session.TransferReceiver(w.dst_pool, w.layout, w.dst_bt, w.seq_lens, w.batch.total_tokens)
    return w, tx, rx


def _oracle_run(w, spec, L):
    b = w.batch
    g = Geom(L=L, F=spec.F, h_kv=spec.H, d_h=spec.D, b_p=spec.E, P=spec.P,
             num_pages=b.num_pool_pages, wire_order=0, W_layer=w.n_layer)
    src_h, dst_h = w.src_pool.cpu().numpy(), w.dst_pool.cpu().numpy()
    wire = np.zeros(L * w.n_layer, dtype=np.uint8)
    for layer in range(L):
        oracle.pack(g, layer, src_h, b.src_block_table, b.seq_lens, wire=wire)
        oracle.unpack(g, layer, dst_h, b.dst_block_table, b.seq_lens, wire)
    return g, src_h, dst_h, wire


def test_session_cfg1_headers_and_pool(dev):
    spec = wl.CFG1
    w, tx, rx = _ends(dev, spec)
    b = w.batch
    g, src_h, want_dst, want_wire = _oracle_run(w, spec, spec.L)
    h_wire = torch.zeros(spec.L * w.n_layer, dtype=torch.uint8).pin_memory()
    ids = [9000 + r for r in range(spec.R)]
    headers, status = session.transfer(tx, rx, h_wire, ids, 7, b.seq_lens)
    assert status == [tk.TOPKV_OK] * spec.R
    assert np.array_equal(h_wire.numpy(), want_wire)
    assert np.array_equal(w.dst_pool.cpu().numpy(), want_dst)
    for r in range(spec.R):
        ck = oracle.kv_plane_crc(g, src_h, b.src_block_table, b.seq_lens, r, 0)
        cv = oracle.kv_plane_crc(g, src_h, b.src_block_table, b.seq_lens, r, 1)
        assert bytes(headers[r]) == oracle.build_header(ids[r], 7, int(b.seq_lens[r]), g, ck, cv)
    assert tk.topkv_device_error_flags() == 0


def test_session_flipped_bit_is_reported_for_one_request_and_a_resend_recovers(dev):
    spec = wl.CFG1
    w, tx, rx = _ends(dev, spec)
    b = w.batch
    _, _, want_dst, _ = _oracle_run(w, spec, spec.L)
    h_wire = torch.zeros(spec.L * w.n_layer, dtype=torch.uint8).pin_memory()
    cu = np.concatenate([[0], np.cumsum(b.seq_lens)])
    off = (int(cu[1]) + 3) * spec.tok_bytes + 5          # request 1, token 3, K row, layer 1
    attempts = []

    def attempt():
        bad = (1, off) if not attempts else None
        attempts.append(1)
        _, status = session.transfer(tx, rx, h_wire, list(range(spec.R)), 1, b.seq_lens,
                                     corrupt=bad)
        if len(attempts) == 1:
            assert status == [0, tk.TOPKV_ERR_CHECKSUM, 0, 0]
        return min(status)

    assert tk.topkv_retry(attempt, retries=2, backoff_ms=1) == tk.TOPKV_OK
    assert len(attempts) == 2
    assert np.array_equal(w.dst_pool.cpu().numpy(), want_dst)


def test_session_gated_by_layer_events_and_other_page_size_at_the_receiver(dev):
    """Sender pool with 16-token pages, receiver pool with 64-token pages and its own table;
    every layer's sending waits for an event recorded on the compute stream."""
    spec = wl.with_layers(wl.CFG2, 3)
    w = harness.setup(spec, dev, need_wire=False, need_dst=False)
    b = w.batch
    tx = session.TransferSender(w.src_pool, w.layout, w.src_bt, w.seq_lens, b.total_tokens)
    Pd = 64
    pages = (b.seq_lens.astype(np.int64) + Pd - 1) // Pd
    npages = int(pages.sum()) + 5
    rng = np.random.default_rng(4242)
    perm, pos = rng.permutation(npages).astype(np.int32), 0
    bt_d = np.full((spec.R, int(pages.max())), -1, dtype=np.int32)
    for r in range(spec.R):
        bt_d[r, :pages[r]] = perm[pos:pos + pages[r]]
        pos += int(pages[r])
    lo_d = tk.make_layout(3, spec.F, spec.H, spec.D, spec.E, Pd, npages, wire_layer_stride=w.n_layer)
    dst = wl.fill_torch(3 * lo_d.pool_layer_stride, 77, dev)
    rx = session.TransferReceiver(dst, lo_d, torch.from_numpy(bt_d).to(dev), w.seq_lens,
                                  b.total_tokens)
    g_s = Geom(L=3, F=spec.F, h_kv=spec.H, d_h=spec.D, b_p=spec.E, P=spec.P,
               num_pages=b.num_pool_pages, W_layer=w.n_layer)
    g_d = Geom(L=3, F=spec.F, h_kv=spec.H, d_h=spec.D, b_p=spec.E, P=Pd, num_pages=npages,
               W_layer=w.n_layer)
    src_h, want_dst = w.src_pool.cpu().numpy(), dst.cpu().numpy()
    wire = np.zeros(3 * w.n_layer, dtype=np.uint8)
    for layer in range(3):
        oracle.pack(g_s, layer, src_h, b.src_block_table, b.seq_lens, wire=wire, impl="rows", threads=8)
        oracle.unpack(g_d, layer, want_dst, bt_d, b.seq_lens, wire, impl="rows", threads=8)
    h_wire = torch.zeros(3 * w.n_layer, dtype=torch.uint8).pin_memory()
    main = torch.cuda.current_stream(dev)
    x = torch.randn(1024, 1024, device=dev)
    ready = []
    for _ in range(3):
        x = x @ x.T * 1e-3                              # stands for a layer's compute
        ev = torch.cuda.Event()
        ev.record(main)
        ready.append(ev)
    headers, status = session.transfer(tx, rx, h_wire, list(range(spec.R)), 3, b.seq_lens,
                                       layer_ready=ready)
    assert status == [tk.TOPKV_OK] * spec.R
    assert np.array_equal(h_wire.numpy(), wire)
    assert np.array_equal(dst.cpu().numpy(), want_dst)
    for r in (0, spec.R - 1):
        ck = oracle.kv_plane_crc(g_s, src_h, b.src_block_table, b.seq_lens, r, 0)
        assert headers[r].crc_k == ck
    assert tk.topkv_device_error_flags() == 0
