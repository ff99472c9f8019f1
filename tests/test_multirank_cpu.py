"""The N > 1 path on CPU: two gloo ranks draw rank-seeded batches (weak scaling: same shape,
different data and tables), and the timing scalars are reduced as bench.py does it (max of the
times, sum of the bytes). No GPU and no collective on the data path."""
import os
import socket
import subprocess
import sys
import textwrap

import numpy as np

from paper_2607_28633_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, {root!r})
    import numpy as np
    import torch
    from paper_2607_28633_b200 import dist_util, workloads as wl
    rank, world, _ = dist_util.env_rank_world()
    dist = dist_util.init("gloo")
    assert dist is not None and dist.get_world_size() == world == 2
    b = wl.make_batch(wl.CFG2, rank=rank)
    bytes_rank = 4.0 * b.total_tokens * wl.CFG2.tok_bytes * wl.CFG2.L
    ms_rank = 2.0 + rank                      # rank 1 is the slower one
    gbs, ms = dist_util.aggregate_throughput(dist, bytes_rank, ms_rank)
    # every rank must also see the other's token count through the reduction
    tot_tokens = dist_util.sum_over_ranks(dist, float(b.total_tokens))
    # bench.py's ranks agree on the smallest number of pinned slabs any of them obtained
    slots = int(round(-dist_util.max_over_ranks(dist, -float(80 if rank == 0 else 4))))
    assert slots == 4
    dist.barrier()
    print(json.dumps({{"rank": rank, "tokens": b.total_tokens, "gbs": gbs, "ms": ms,
                      "tot_tokens": tot_tokens,
                      "table_sum": int(b.src_block_table[b.src_block_table >= 0].sum())}}))
    dist.destroy_process_group()
""")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_weak_scaling(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(__import__("json").loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    b0, b1 = wl.make_batch(wl.CFG2, rank=0), wl.make_batch(wl.CFG2, rank=1)
    assert outs[0]["tokens"] == b0.total_tokens and outs[1]["tokens"] == b1.total_tokens
    assert outs[0]["tot_tokens"] == outs[1]["tot_tokens"] == b0.total_tokens + b1.total_tokens
    assert outs[0]["ms"] == outs[1]["ms"] == 3.0                       # max over ranks
    want = 4.0 * (b0.total_tokens + b1.total_tokens) * wl.CFG2.tok_bytes * wl.CFG2.L / 3e-3 / 1e9
    assert abs(outs[0]["gbs"] - want) < 1e-6 * want and outs[0]["gbs"] == outs[1]["gbs"]


def test_rank_seeding_gives_independent_batches_of_the_same_shape():
    b0, b1 = wl.make_batch(wl.CFG2, rank=0), wl.make_batch(wl.CFG2, rank=1)
    assert b0.spec == b1.spec and b0.seq_lens.shape == b1.seq_lens.shape
    assert not np.array_equal(b0.seq_lens, b1.seq_lens)
    assert b0.seeds["data"] != b1.seeds["data"]
    assert wl.make_batch(wl.CFG2, rank=1).seq_lens.tolist() == b1.seq_lens.tolist()   # reproducible
    for b in (b0, b1):
        used = b.src_block_table[b.src_block_table >= 0]
        assert len(np.unique(used)) == used.size == b.pages_needed       # a permutation prefix
        assert used.max() < b.num_pool_pages
        assert ((b.seq_lens >= 512) & (b.seq_lens <= 4096)).all()
        assert b.num_pool_pages == int(np.ceil(1.5 * b.pages_needed))


def test_workload_shapes_match_the_configurations():
    b3 = wl.make_batch(wl.CFG3)
    assert b3.total_tokens == 8 * 4096 and b3.total_tokens * wl.CFG3.tok_bytes == 134_217_728
    assert b3.num_pool_pages == 4096 and wl.CFG3.page_bytes == 65_536
    assert 80 * b3.total_tokens * wl.CFG3.tok_bytes == 10 * 2**30
    b4 = wl.make_batch(wl.CFG4)
    assert wl.CFG4.page_bytes == 73_728 and wl.CFG4.tok_bytes == 1152
    assert ((b4.seq_lens >= 1024) & (b4.seq_lens <= 8192)).all()
    b5 = wl.make_batch(wl.CFG5)
    assert b5.total_tokens * wl.CFG5.tok_bytes == 67_108_864 and b5.num_pool_pages == 2048
    b1 = wl.make_batch(wl.CFG1)
    assert b1.seq_lens.tolist() == [17, 64, 100, 255] and b1.max_pages_per_req == 16
    assert b1.num_pool_pages == 64 and b1.pages_needed == 29
