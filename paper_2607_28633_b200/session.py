"""One request batch's pipelined transfer, both ends, on top of the C-ABI calls.

``TransferSender`` is what a prefill worker runs: after every layer's event it ships that
layer's slab to pinned host memory with the checksummed host leg, and at the end it emits one
128-byte header per request (§3.4). ``TransferReceiver`` is the decode side: it places every
layer from the host slab into its own paged pool, checksumming as it goes, and checks the
headers when the last layer is in; a mismatch is reported per request so that the caller can
retry (§3.1). Both only issue library calls on the streams they are given: no pack / unpack
arithmetic happens in Python, and nothing here touches the CPU oracle.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import numpy as np
import torch

from . import binding as tk


@dataclass
class Endpoint:
    """Device-side description of one end: pool, layout, tables (device tensors)."""
    pool: torch.Tensor
    layout: tk.topkv_layout
    block_table: torch.Tensor
    seq_lens: torch.Tensor
    total_tokens: int

    def __post_init__(self):
        dev = self.pool.device
        R = int(self.seq_lens.shape[0])
        self.cu = torch.zeros(R + 1, dtype=torch.int64, device=dev)
        tk.check(tk.topkv_build_plan(tk.make_batch(self.block_table, self.seq_lens), self.cu,
                                     torch.cuda.current_stream(dev)))
        self.batch = tk.make_batch(self.block_table, self.seq_lens, self.total_tokens, self.cu)
        self.n_layer = tk.topkv_wire_layer_bytes(self.layout, self.total_tokens)
        self.ws_bytes = tk.check(tk.topkv_crc_workspace_bytes(
            self.layout, R, int(self.block_table.shape[1])))
        self.workspace = torch.empty(self.ws_bytes, dtype=torch.uint8, device=dev)
        # two staging slabs: consecutive layers alternate between two streams, so that the copy
        # engine moves layer l while the kernel of layer l + 1 runs
        self.stagings = [torch.empty(max(self.n_layer, 16), dtype=torch.uint8, device=dev)
                         for _ in range(2)]
        self.crc = torch.zeros(R * self.layout.kv_factor, dtype=torch.int64, device=dev)
        torch.cuda.current_stream(dev).synchronize()

    @property
    def num_requests(self) -> int:
        return int(self.seq_lens.shape[0])

    def _checksums(self, stream) -> np.ndarray:
        tk.check(tk.topkv_crc_finish(self.layout, self.batch, self.workspace, self.ws_bytes,
                                     self.crc, stream))
        stream.synchronize()
        return self.crc.cpu().numpy().view(np.uint64).reshape(self.num_requests,
                                                              self.layout.kv_factor)


class TransferSender(Endpoint):
    """Ships layers to ``h_wire`` (pinned, ``L`` slabs of ``n_layer`` bytes, layer-major)."""

    def begin(self, stream):
        tk.check(tk.topkv_crc_begin(self.layout, self.batch, self.workspace, self.ws_bytes, stream))

    def send_layer(self, layer: int, h_wire: torch.Tensor, stream, slot: int = 0):
        st = self.stagings[slot]
        tk.check(tk.topkv_pack_layer_to_host_crc(
            layer, self.pool, self.layout, self.batch, h_wire, h_wire.numel(), st, st.numel(),
            self.workspace, self.ws_bytes, stream))

    def finish(self, stream, request_ids, model_id: int, h_seq_lens) -> list[tk.topkv_wire_header]:
        crc = self._checksums(stream)
        headers = []
        for r, rid in enumerate(request_ids):
            h = tk.topkv_wire_header()
            crc_v = int(crc[r, 1]) if self.layout.kv_factor == 2 else 0
            tk.check(tk.topkv_header_fill(h, int(rid), model_id, self.layout, int(h_seq_lens[r]),
                                          int(crc[r, 0]), crc_v))
            headers.append(h)
        return headers


class TransferReceiver(Endpoint):
    """Places layers from ``h_wire`` into its own pool and verifies the headers."""

    def begin(self, stream):
        tk.check(tk.topkv_crc_begin(self.layout, self.batch, self.workspace, self.ws_bytes, stream))

    def recv_layer(self, layer: int, h_wire: torch.Tensor, stream, slot: int = 0):
        st = self.stagings[slot]
        tk.check(tk.topkv_unpack_layer_from_host_crc(
            layer, self.pool, self.layout, self.batch, h_wire, h_wire.numel(), st, st.numel(),
            self.workspace, self.ws_bytes, stream))

    def finish(self, stream, headers, h_seq_lens) -> list[int]:
        """Status per request: TOPKV_OK or TOPKV_ERR_CHECKSUM."""
        crc = self._checksums(stream)
        out = []
        for r, h in enumerate(headers):
            crc_v = int(crc[r, 1]) if self.layout.kv_factor == 2 else 0
            out.append(tk.topkv_header_check(h, self.layout, int(h_seq_lens[r]), int(crc[r, 0]), crc_v))
        return out


def transfer(sender: TransferSender, receiver: TransferReceiver, h_wire: torch.Tensor,
             request_ids, model_id: int, h_seq_lens, layer_ready=None, corrupt=None):
    """Runs one whole transfer through pinned host memory, pipelined per layer (the receiver
    starts on layer l as soon as it has arrived); each side alternates between two streams. ``layer_ready[l]`` is an
    optional event (e.g. recorded by the prefill) that gates the sending of layer l.
    ``corrupt`` (layer, byte offset) flips one bit of that layer's slab in flight: a test hook
    standing in for a faulty link. Returns (headers, per-request status)."""
    dev = sender.pool.device
    tx = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    rx = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    L = sender.layout.num_layers

    def after(first, second):
        """second starts (continues) only after what first holds so far."""
        ev = torch.cuda.Event()
        ev.record(first)
        second.wait_event(ev)

    sender.begin(tx[0])
    receiver.begin(rx[0])
    after(tx[0], tx[1])
    after(rx[0], rx[1])
    for layer in range(L):
        q = layer & 1
        if layer_ready is not None:
            tx[q].wait_event(layer_ready[layer])
        sender.send_layer(layer, h_wire, tx[q], q)
        arrived = torch.cuda.Event()
        arrived.record(tx[q])
        if corrupt is not None and corrupt[0] == layer:
            arrived.synchronize()
            h_wire[layer * sender.layout.wire_layer_stride + corrupt[1]] ^= 0x04
        rx[q].wait_event(arrived)
        receiver.recv_layer(layer, h_wire, rx[q], q)
    after(tx[1], tx[0])
    after(rx[1], rx[0])
    headers = sender.finish(tx[0], request_ids, model_id, h_seq_lens)
    status = receiver.finish(rx[0], headers, h_seq_lens)
    return headers, status
