"""Layer-by-layer issue on a side stream (§5.2 made real on one GPU).

The main stream runs a per-layer prefill stand-in (two bf16 GEMMs through torch; it carries
no correctness claim) and records an event after each layer. A high-priority side stream
waits for layer l's event and then runs ``topkv_pack_layer_to_host`` for that layer, so that
the transfer of layer l overlaps the compute of layers l+1 .. L-1. The two streams meet only
through events; the host enqueues everything ahead of time.

Measured quantities (all from CUDA events):
  t_xfer_serial  sum over layers of the transfer's duration with no compute running
  exposed        how long the last transfer ends after the last layer's compute
  hidden         1 - exposed / t_xfer_serial     (Eq. 3 with T_last := the last slab's transfer)
  slowdown       T_main(with transfer) / T_main(alone) - 1
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from . import workloads as wl
from .harness import DeviceWorkload


@dataclass
class OverlapResult:
    layers: int
    t_main_alone_ms: float
    t_main_overlap_ms: float
    t_layer_compute_ms: float
    t_xfer_serial_ms: float
    t_xfer_overlapped_ms: float | None
    exposed_ms: float
    hidden: float
    hidden_upper_bound: float
    slowdown: float
    bytes_per_layer: int
    xfer_gbs_serial: float

    def as_dict(self):
        return {k: (round(v, 6) if isinstance(v, float) else v) for k, v in self.__dict__.items()}


class PrefillStandIn:
    """X[4096 x 8192] @ W1[8192 x 28672] then @ W2[28672 x 8192], bf16, one seeded weight pair
    reused by every layer, every layer starting from the same X (no chaining)."""

    def __init__(self, device, seed: int, tokens=wl.GEMM_TOKENS, hidden=wl.GEMM_HIDDEN,
                 ffn=wl.GEMM_FFN, std=wl.GEMM_W_STD):
        g = torch.Generator(device=device)
        g.manual_seed(seed)
        bf = torch.bfloat16
        self.x = torch.empty(tokens, hidden, dtype=bf, device=device).normal_(0, 1, generator=g)
        self.w1 = torch.empty(hidden, ffn, dtype=bf, device=device).normal_(0, std, generator=g)
        self.w2 = torch.empty(ffn, hidden, dtype=bf, device=device).normal_(0, std, generator=g)
        self.y = torch.empty(tokens, ffn, dtype=bf, device=device)
        self.z = torch.empty(tokens, hidden, dtype=bf, device=device)
        self.flop_per_layer = 2 * 2 * tokens * hidden * ffn

    def layer(self):
        torch.matmul(self.x, self.w1, out=self.y)
        torch.matmul(self.y, self.w2, out=self.z)


def run_overlap(w: DeviceWorkload, h_pinned: torch.Tensor, staging, prefill: PrefillStandIn,
                layers: int | None = None, slots: int | None = None,
                warmup_layers: int = 3, crc_workspace=None) -> OverlapResult:
    """h_pinned holds ``slots`` wire slabs (a ring when slots < layers); w.layout must have
    wire_layer_stride == n_layer. With ``crc_workspace`` (a device buffer prepared by
    topkv_crc_begin) every transfer also checksums the layer (topkv_pack_layer_to_host_crc).
    Returns the event-timed overlap figures."""
    dev = w.src_pool.device
    L = w.layers if layers is None else layers
    n = w.n_layer
    slots = h_pinned.numel() // n if slots is None else slots
    assert slots >= 1 and h_pinned.numel() >= slots * n
    main = torch.cuda.Stream(dev)
    side = torch.cuda.Stream(dev, priority=-1)  # higher priority than the compute stream

    # Each layer's slab goes to ring slot l % slots: pass the slot's base as the buffer of
    # "layer 0" by giving the library a per-call view (stride-free addressing).
    lo = type(w.layout)()
    import ctypes
    ctypes.memmove(ctypes.byref(lo), ctypes.byref(w.layout), ctypes.sizeof(lo))
    lo.wire_layer_stride = 0
    from . import binding as tk

    def xfer(l, stream):
        slab = h_pinned[(l % slots) * n:(l % slots + 1) * n]
        cap = 0 if staging is None else staging.numel()
        if crc_workspace is None:
            tk.check(tk.topkv_pack_layer_to_host(l, w.src_pool, lo, w.src_batch, slab, n, staging,
                                                 cap, stream))
        else:
            tk.check(tk.topkv_pack_layer_to_host_crc(l, w.src_pool, lo, w.src_batch, slab, n, staging,
                                                     cap, crc_workspace, crc_workspace.numel(),
                                                     stream))

    def ev():
        return torch.cuda.Event(enable_timing=True)

    # warm-up: GEMM heuristics, transfer path
    with torch.cuda.stream(main):
        for _ in range(warmup_layers):
            prefill.layer()
    for l in range(min(warmup_layers, L)):
        xfer(l, side)
    torch.cuda.synchronize(dev)

    # (1) compute alone
    m0, m1 = ev(), ev()
    with torch.cuda.stream(main):
        m0.record(main)
        for _ in range(L):
            prefill.layer()
        m1.record(main)
    torch.cuda.synchronize(dev)
    t_main_alone = m0.elapsed_time(m1)

    # (2) transfers alone, serial, each timed
    bs, es = [ev() for _ in range(L)], [ev() for _ in range(L)]
    for l in range(L):
        bs[l].record(side)
        xfer(l, side)
        es[l].record(side)
    torch.cuda.synchronize(dev)
    t_xfer_serial = sum(bs[l].elapsed_time(es[l]) for l in range(L))

    # (3) overlapped
    done = [torch.cuda.Event() for _ in range(L)]
    bo, eo = [ev() for _ in range(L)], [ev() for _ in range(L)]
    s0, s1 = ev(), ev()
    with torch.cuda.stream(main):
        s0.record(main)
        for l in range(L):
            prefill.layer()
            done[l].record(main)
        s1.record(main)
    if slots >= L and crc_workspace is None:
        # the whole side-stream schedule as one library call: wait done[l], ship layer l,
        # record eo[l] (topkv_pack_layers_to_host_pipelined); bo[l] is not needed for `hidden`
        cap = 0 if staging is None else staging.numel()
        tk.check(tk.topkv_pack_layers_to_host_pipelined(
            0, L, w.src_pool, w.layout, w.src_batch, h_pinned, h_pinned.numel(), staging, cap,
            done, eo, side))
        bo = None
    else:
        for l in range(L):
            side.wait_event(done[l])
            bo[l].record(side)
            xfer(l, side)
            eo[l].record(side)
    torch.cuda.synchronize(dev)
    t_main_overlap = s0.elapsed_time(s1)
    exposed = max(0.0, s1.elapsed_time(eo[L - 1]))
    # sum of the per-layer spans in the overlapped pass (not observable when the schedule was
    # issued as one library call: no event sits between a layer's wait and its transfer)
    t_xfer_overlapped = (sum(bo[l].elapsed_time(eo[l]) for l in range(L)) if bo is not None
                         else None)
    hidden = 1.0 - exposed / t_xfer_serial if t_xfer_serial > 0 else 1.0
    return OverlapResult(
        layers=L, t_main_alone_ms=t_main_alone, t_main_overlap_ms=t_main_overlap,
        t_layer_compute_ms=t_main_alone / L, t_xfer_serial_ms=t_xfer_serial,
        t_xfer_overlapped_ms=t_xfer_overlapped, exposed_ms=exposed, hidden=hidden,
        hidden_upper_bound=1.0 - 1.0 / L, slowdown=t_main_overlap / t_main_alone - 1.0,
        bytes_per_layer=n, xfer_gbs_serial=n * L / (t_xfer_serial * 1e-3) / 1e9)
