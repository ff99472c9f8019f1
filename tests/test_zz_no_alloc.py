"""The allocation-free host leg, topkv_pack_layer_to_host_noalloc.

Some callers of this library cannot hand it a staging slab because they may not allocate
device memory at all: they live inside another framework's fixed memory budget, or a
cudaMalloc (which synchronises the device) is not acceptable in the middle of serving. For
them the library carries a fixed staging array in its own device image. This test calls that
entry point through the C ABI twice in a row and requires the bytes that land in pinned
memory to equal, exactly, what the ordinary staged entry point produces and what the CPU
oracle computes for the same batch; the second call uses a shorter batch, so anything left in
the shared slab by the first call would show. Both kernel families are exercised, since the
call routes the built-in slab through whichever one is selected.

Collected last on purpose (file name), and it passes alone in a fresh process as well.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

import oracle
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


@pytest.fixture(params=[0, 1], ids=["vec", "bulk"])
def variant(request, dev):
    """Kernel family used behind the entry point (vectorised load/store, bulk-async ring)."""
    prev = tk.topkv_set_kernel_variant(request.param)
    tk.check(tk.topkv_reset_device_error_flags())
    yield request.param
    tk.topkv_set_kernel_variant(prev)


def _oracle_slab(w, layer):
    """The CPU oracle's wire slab of one layer of this workload."""
    b, s = w.batch, w.batch.spec
    g = oracle.Geom(L=1, F=s.F, h_kv=s.H, d_h=s.D, b_p=s.E, P=s.P, num_pages=b.num_pool_pages)
    src_h = harness.layer_slab_to_numpy(w.src_pool, w.slab_bytes, layer)
    return oracle.pack(g, 0, src_h, b.src_block_table, b.seq_lens)


def _pack_both_ways(w, layer, dev, stream):
    n, L = w.n_layer, w.layers
    got = torch.full((L * n,), 0x11, dtype=torch.uint8).pin_memory()
    want = torch.full((L * n,), 0x11, dtype=torch.uint8).pin_memory()
    staging = torch.empty(n, dtype=torch.uint8, device=dev)   # no fill: nothing to race with
    stream.wait_stream(torch.cuda.current_stream(dev))        # set-up on the default stream is done
    tk.check(tk.topkv_pack_layer_to_host_noalloc(layer, w.src_pool, w.layout, w.src_batch, got,
                                                 got.numel(), stream))
    tk.check(tk.topkv_pack_layer_to_host(layer, w.src_pool, w.layout, w.src_batch, want,
                                         want.numel(), staging, staging.numel(), stream))
    stream.synchronize()
    return got.numpy(), want.numpy()


def test_noalloc_matches_staged_entry_point_twice(dev, variant):
    stream = torch.cuda.Stream(dev)
    # first call: the tiny GQA workload, layer 1 (1,785,856-byte slab)
    big = harness.setup(wl.CFG1, dev, need_dst=False, need_wire=False)
    assert big.n_layer <= tk.TOPKV_NOALLOC_STAGING_BYTES
    got, want = _pack_both_ways(big, 1, dev, stream)
    assert np.array_equal(got, want)
    assert np.array_equal(got[big.n_layer:], _oracle_slab(big, 1))  # and it is the oracle's slab
    assert (got[:big.n_layer] == 0x11).all()                      # layer 0's slab untouched
    # second call, right after: a shorter batch with other data and tables, same shared slab
    from dataclasses import replace
    small_spec = replace(wl.CFG1, lengths=("fixed", (5, 33, 16, 1)), seed=900)
    small = harness.setup(small_spec, dev, need_dst=False, need_wire=False)
    assert 0 < small.n_layer < big.n_layer
    got2, want2 = _pack_both_ways(small, 0, dev, stream)
    assert np.array_equal(got2, want2)
    assert np.array_equal(got2[:small.n_layer], _oracle_slab(small, 0))
    assert (got2[small.n_layer:] == 0x11).all()                   # nothing past the slab copied
    assert tk.topkv_device_error_flags() == 0


def test_noalloc_rejects_slabs_beyond_the_built_in_size(dev):
    spec = wl.with_layers(wl.CFG2, 1)                             # ~134 MB per layer
    w = harness.setup(spec, dev, need_dst=False, need_wire=False)
    assert w.n_layer > tk.TOPKV_NOALLOC_STAGING_BYTES
    pinned = torch.zeros(64, dtype=torch.uint8).pin_memory()
    before = tk.topkv_kernel_launch_count()
    st = tk.topkv_pack_layer_to_host_noalloc(0, w.src_pool, w.layout, w.src_batch, pinned,
                                             w.n_layer, None)     # capacity claimed, never used
    assert st == tk.TOPKV_ERR_CAPACITY
    assert tk.topkv_kernel_launch_count() == before
    # an unknown token count is refused too: the copy size must be known on the host
    w.src_batch.total_tokens = -1
    st = tk.topkv_pack_layer_to_host_noalloc(0, w.src_pool, w.layout, w.src_batch, pinned,
                                             pinned.numel(), None)
    assert st == tk.TOPKV_ERR_INVALID_ARG
    torch.cuda.synchronize()
