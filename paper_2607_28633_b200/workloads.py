"""Seeded synthetic inputs for the five benchmark configurations.

This module only draws shapes, lengths, block tables and cache contents. It contains none
of the pack / unpack arithmetic and imports neither the CUDA binding nor the CPU oracle, so
both sides can be fed the very same inputs.

The paper evaluates on no dataset; it uses public model *shapes* (Table 1, §5.3). The
workloads below take those shapes (Llama-3-8B / 70B GQA, DeepSeek-V3 MLA) and stand in for
serving traffic: prompt lengths uniform in a range, pages scattered over an over-provisioned
block pool by a random permutation, cache values N(0,1) bf16 (raw 16-bit patterns for the
tiny case so that NaN / Inf / denormal encodings are covered).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace

import numpy as np


@dataclass(frozen=True)
class WorkloadSpec:
    name: str
    L: int                 # layers
    F: int                 # 2 = K and V planes, 1 = one MLA latent row per token
    H: int                 # KV heads
    D: int                 # head dim
    E: int                 # bytes per element
    P: int                 # tokens per page
    R: int                 # requests
    lengths: tuple         # ("fixed", (..)) | ("uniform", lo, hi) inclusive | ("const", n)
    pool_factor: float     # pool pages = ceil(pool_factor * needed), or
    pool_pages: int = 0    # an explicit page count when > 0
    seed: int = 0          # base seed; streams are seed+1 .. seed+5
    raw_bits: bool = False # True: uniform random 16-bit patterns instead of N(0,1) bf16
    legs: tuple = ("pack", "unpack")
    note: str = ""

    @property
    def row_bytes(self) -> int:
        return self.H * self.D * self.E

    @property
    def tok_bytes(self) -> int:
        return self.F * self.row_bytes

    @property
    def page_bytes(self) -> int:
        return self.P * self.tok_bytes


CFG1 = WorkloadSpec("cfg1_tiny_gqa", L=2, F=2, H=8, D=128, E=2, P=16, R=4,
                    lengths=("fixed", (17, 64, 100, 255)), pool_factor=0.0, pool_pages=64,
                    seed=100, raw_bits=True, note="tiny GQA, raw 16-bit patterns")
CFG2 = WorkloadSpec("cfg2_llama3_8b", L=32, F=2, H=8, D=128, E=2, P=16, R=16,
                    lengths=("uniform", 512, 4096), pool_factor=1.5, seed=200,
                    note="Llama-3-8B-shaped GQA, per-layer pack then unpack, device to device")
CFG3 = WorkloadSpec("cfg3_llama3_70b", L=80, F=2, H=8, D=128, E=2, P=16, R=8,
                    lengths=("const", 4096), pool_factor=2.0, seed=300,
                    legs=("pack", "pack_to_host", "unpack_from_host"),
                    note="Llama-3-70B-shaped GQA, 8 x 4096 tokens, host leg")
CFG4 = WorkloadSpec("cfg4_dsv3_mla", L=61, F=1, H=1, D=576, E=2, P=64, R=32,
                    lengths=("uniform", 1024, 8192), pool_factor=1.5, seed=400,
                    note="DeepSeek-V3-shaped MLA latent rows")
CFG5 = WorkloadSpec("cfg5_overlap_70b", L=80, F=2, H=8, D=128, E=2, P=16, R=4,
                    lengths=("const", 4096), pool_factor=2.0, seed=500,
                    legs=("overlap",),
                    note="Llama-3-70B-shaped, 4 x 4096 tokens, side-stream pack to host under GEMMs")

ALL = {c.name.split("_")[0]: c for c in (CFG1, CFG2, CFG3, CFG4, CFG5)}

# The prefill stand-in of the overlap run: X[4096 x 8192] @ W1[8192 x 28672] @ W2[28672 x 8192].
GEMM_TOKENS, GEMM_HIDDEN, GEMM_FFN, GEMM_W_STD = 4096, 8192, 28672, 0.02


def with_layers(spec: WorkloadSpec, L: int) -> WorkloadSpec:
    """Same workload on fewer (or more) layers; everything else, tables included, unchanged."""
    return replace(spec, L=L)


@dataclass
class Batch:
    spec: WorkloadSpec
    seq_lens: np.ndarray        # int32 [R]
    src_block_table: np.ndarray # int32 [R][maxp], -1 padded
    dst_block_table: np.ndarray # int32 [R][maxp], -1 padded
    num_pool_pages: int
    max_pages_per_req: int
    total_tokens: int
    pages_needed: int
    seeds: dict = field(default_factory=dict)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def draw_seq_lens(spec: WorkloadSpec, seed: int) -> np.ndarray:
    kind = spec.lengths[0]
    if kind == "fixed":
        out = np.array(spec.lengths[1], dtype=np.int32)
        assert out.shape[0] == spec.R
    elif kind == "const":
        out = np.full(spec.R, spec.lengths[1], dtype=np.int32)
    elif kind == "uniform":
        lo, hi = spec.lengths[1], spec.lengths[2]
        out = _rng(seed).integers(lo, hi + 1, size=spec.R).astype(np.int32)
    else:
        raise ValueError(kind)
    return out


def _cut_table(perm: np.ndarray, pages_per_req: np.ndarray, maxp: int) -> np.ndarray:
    bt = np.full((pages_per_req.shape[0], maxp), -1, dtype=np.int32)
    pos = 0
    for r, n in enumerate(pages_per_req):
        bt[r, :n] = perm[pos:pos + n]
        pos += n
    return bt


def make_batch(spec: WorkloadSpec, rank: int = 0, max_pages_per_req: int | None = None) -> Batch:
    """Draws lengths and two independent block tables (source and destination pool).

    ``rank`` offsets every seed so that data-parallel replicas work on different batches.
    """
    base = spec.seed + 100000 * rank
    seeds = {"lens": base + 5, "data": base + 1, "src_perm": base + 2, "dst_perm": base + 3,
             "dst_fill": base + 4}
    sl = draw_seq_lens(spec, seeds["lens"])
    pages = (sl.astype(np.int64) + spec.P - 1) // spec.P
    needed = int(pages.sum())
    npool = spec.pool_pages if spec.pool_pages > 0 else int(np.ceil(spec.pool_factor * needed))
    assert npool >= needed
    maxp = int(pages.max()) if max_pages_per_req is None else max_pages_per_req
    maxp = max(maxp, 1)
    src = _cut_table(_rng(seeds["src_perm"]).permutation(npool)[:needed].astype(np.int32), pages, maxp)
    dst = _cut_table(_rng(seeds["dst_perm"]).permutation(npool)[:needed].astype(np.int32), pages, maxp)
    return Batch(spec, sl, src, dst, npool, maxp, int(sl.sum()), needed, seeds)


def pool_bytes(spec: WorkloadSpec, num_pool_pages: int, layers: int | None = None) -> int:
    L = spec.L if layers is None else layers
    return L * num_pool_pages * spec.page_bytes


def fill_numpy(nbytes: int, seed: int, raw_bits: bool = True) -> np.ndarray:
    """uint8 array of nbytes: uniform random 16-bit patterns, or N(0,1) rounded to bf16."""
    assert nbytes % 2 == 0
    g = _rng(seed)
    if raw_bits:
        return g.integers(0, 1 << 16, size=nbytes // 2, dtype=np.uint16).view(np.uint8)
    x = g.standard_normal(nbytes // 2, dtype=np.float32)
    u = x.view(np.uint32)
    # round-to-nearest-even truncation of fp32 to its top 16 bits (bf16)
    bf = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16).astype(np.uint16)
    return bf.view(np.uint8)


def fill_torch(nbytes: int, seed: int, device, raw_bits: bool = False, chunk_bytes: int = 1 << 30):
    """uint8 torch tensor of nbytes on ``device``, filled chunk by chunk from one seeded
    generator: N(0,1) bf16, or uniform random 16-bit patterns."""
    import torch
    assert nbytes % 2 == 0
    out = torch.empty(nbytes, dtype=torch.uint8, device=device)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    for off in range(0, nbytes, chunk_bytes):
        n = min(chunk_bytes, nbytes - off)
        view = out[off:off + n]
        if raw_bits:
            view.view(torch.int16).random_(-32768, 32768, generator=g)
        else:
            view.view(torch.bfloat16).normal_(0.0, 1.0, generator=g)
    return out
