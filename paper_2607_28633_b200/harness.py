"""Device-side set-up shared by the GPU tests and bench.py: allocates the pools, tables and
wire buffers of one workload with torch (device memory and streams only) and issues the
per-layer calls through the C-ABI binding. No pack / unpack arithmetic happens here, and
the CPU oracle is never imported."""
from __future__ import annotations

import ctypes
from dataclasses import dataclass, field

import numpy as np
import torch

from . import binding as tk
from . import workloads as wl


@dataclass
class DeviceWorkload:
    batch: wl.Batch
    layers: int                 # layers actually allocated (may be fewer than spec.L)
    layout: tk.topkv_layout
    n_layer: int                # bytes of one wire slab
    src_pool: torch.Tensor      # uint8 [layers * slab]
    dst_pool: torch.Tensor | None
    wire: torch.Tensor | None   # uint8 [layers * n_layer]
    seq_lens: torch.Tensor
    src_bt: torch.Tensor
    dst_bt: torch.Tensor
    cu: torch.Tensor            # int64 [R+1], filled by topkv_build_plan
    src_batch: tk.topkv_batch
    dst_batch: tk.topkv_batch
    _overlap_batches: dict = field(default_factory=dict)

    @property
    def slab_bytes(self) -> int:
        return self.layout.pool_layer_stride

    def _flagged(self, batch: tk.topkv_batch, overlap: bool) -> tk.topkv_batch:
        if not overlap:
            return batch
        key = id(batch)
        if key not in self._overlap_batches:
            b = tk.topkv_batch()
            ctypes.memmove(ctypes.byref(b), ctypes.byref(batch), ctypes.sizeof(b))
            b._keepalive = getattr(batch, "_keepalive", None)
            b.flags = tk.TOPKV_FLAG_OVERLAP_PREVIOUS
            self._overlap_batches[key] = b
        return self._overlap_batches[key]

    def pack(self, layer: int, stream=None, wire=None, overlap: bool = False):
        """overlap=True declares the call independent of the kernels enqueued just before it
        (TOPKV_FLAG_OVERLAP_PREVIOUS): true for pack(l+1) after pack(l)."""
        w = self.wire if wire is None else wire
        return tk.check(tk.topkv_pack_layer(layer, self.src_pool, self.layout,
                                            self._flagged(self.src_batch, overlap), w, w.numel(),
                                            stream))

    def unpack(self, layer: int, stream=None, wire=None, overlap: bool = False):
        w = self.wire if wire is None else wire
        return tk.check(tk.topkv_unpack_layer(layer, self.dst_pool, self.layout,
                                              self._flagged(self.dst_batch, overlap), w, w.numel(),
                                              stream))

    def pack_to_host(self, layer: int, h_pinned, staging=None, stream=None):
        return tk.check(tk.topkv_pack_layer_to_host(
            layer, self.src_pool, self.layout, self.src_batch, h_pinned, h_pinned.numel(), staging,
            0 if staging is None else staging.numel(), stream))

    def unpack_from_host(self, layer: int, h_pinned, staging=None, stream=None):
        return tk.check(tk.topkv_unpack_layer_from_host(
            layer, self.dst_pool, self.layout, self.dst_batch, h_pinned, h_pinned.numel(), staging,
            0 if staging is None else staging.numel(), stream))


def setup(spec: wl.WorkloadSpec, device, layers: int | None = None, rank: int = 0,
          wire_order: int = tk.TOPKV_WIRE_TOKEN_KV, need_dst: bool = True, need_wire: bool = True,
          use_plan: bool = True, fill_dst: bool = True) -> DeviceWorkload:
    """Draws the batch, fills the source pool (and the destination pool with a different
    seeded pattern, so that untouched bytes are part of any comparison) and builds the plan."""
    batch = wl.make_batch(spec, rank=rank)
    L = spec.L if layers is None else layers
    lo = tk.make_layout(L, spec.F, spec.H, spec.D, spec.E, spec.P, batch.num_pool_pages,
                        wire_order=wire_order)
    n_layer = tk.check(tk.topkv_wire_layer_bytes(lo, batch.total_tokens))   # N_layer, from the library
    lo.wire_layer_stride = n_layer
    nbytes = L * lo.pool_layer_stride
    src = wl.fill_torch(nbytes, batch.seeds["data"], device, raw_bits=spec.raw_bits)
    dst = None
    if need_dst:
        if fill_dst:
            dst = wl.fill_torch(nbytes, batch.seeds["dst_fill"], device, raw_bits=spec.raw_bits)
        else:
            dst = torch.zeros(nbytes, dtype=torch.uint8, device=device)
    wire = torch.zeros(L * n_layer, dtype=torch.uint8, device=device) if need_wire else None
    sl = torch.from_numpy(batch.seq_lens).to(device)
    bt_s = torch.from_numpy(batch.src_block_table).to(device)
    bt_d = torch.from_numpy(batch.dst_block_table).to(device)
    cu = torch.zeros(spec.R + 1, dtype=torch.int64, device=device)
    if use_plan:
        tk.check(tk.topkv_build_plan(tk.make_batch(bt_s, sl), cu, torch.cuda.current_stream(device)))
        torch.cuda.current_stream(device).synchronize()
    cu_arg = cu if use_plan else None
    return DeviceWorkload(batch, L, lo, n_layer, src, dst, wire, sl, bt_s, bt_d, cu,
                          tk.make_batch(bt_s, sl, batch.total_tokens, cu_arg),
                          tk.make_batch(bt_d, sl, batch.total_tokens, cu_arg))


def layer_slab_to_numpy(pool: torch.Tensor, slab_bytes: int, layer: int) -> np.ndarray:
    return pool[layer * slab_bytes:(layer + 1) * slab_bytes].cpu().numpy()
