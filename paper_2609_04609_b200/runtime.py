"""Device-side state of one table of units (e.g. one MoE layer) and the per-iteration step.

Plumbing only: torch allocates the buffers and provides streams / events; every data-path
operation is a call into the C-ABI library (``ciera.encode``, ``ciera.transport``,
``ciera.decode``).  One ``LayerCodec`` plays both roles of the paper's Algorithm 1 on a single
GPU: the sender with its cache, and one receiver with its own cache; the device-to-device
``transport`` stands where the Allgather of the messages would be.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np
import torch

from . import ciera
from .workloads import VALUE_BYTES, layout_units


class LayerCodec:
    def __init__(self, units: np.ndarray, dtype: str, block: int, weights_bytes: int, cache_bytes: int,
                 msg_bytes: int, device="cuda:0", with_output: bool = True, slack: int = 0):
        """``slack``: extra bytes (entries, for the per-unit arrays) allocated behind every buffer; the
        library is never told about them, so whatever a caller puts there must survive every call."""
        self.dtype_name = dtype
        self.dtype = ciera.DTYPE_CODES[dtype]
        self.block = block
        self.device = torch.device(device)
        self.plan = ciera.Plan(units, self.dtype, block, self.device)
        self.units = self.plan.units
        dev = self.device
        self.weights_bytes, self.cache_bytes, self.msg_bytes = weights_bytes, cache_bytes, msg_bytes
        # every buffer is a view of an allocation that is `slack` bytes (entries) longer
        self.slack = slack
        self.allocations = {}

        def alloc(name, size, dt=torch.uint8):
            full = torch.zeros(size + slack, dtype=dt, device=dev)
            self.allocations[name] = full
            return full[:size]

        self.sender_cache = alloc("sender_cache", max(cache_bytes, 16))
        self.receiver_cache = alloc("receiver_cache", max(cache_bytes, 16))
        self.msg_send = alloc("msg_send", max(msg_bytes, 16))
        self.msg_recv = alloc("msg_recv", max(msg_bytes, 16))
        self.weights_out = alloc("weights_out", max(weights_bytes, 16)) if with_output else None
        n = max(self.plan.n_units, 1)
        self.wire_bytes = alloc("wire_bytes", n, torch.int64)
        self.changed_blocks = alloc("changed_blocks", n, torch.int32)
        self.workspace = self.plan.new_workspace()
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)

    @classmethod
    def from_tensors(cls, tensor_numels: Sequence[int], n_shards: int, dtype: str, block: int, device="cuda:0",
                     **kw) -> "LayerCodec":
        code = ciera.DTYPE_CODES[dtype]
        units, wb, cb, mb = layout_units(tensor_numels, n_shards, VALUE_BYTES[dtype],
                                         lambda n: ciera.message_capacity(n, code, block))
        return cls(units, dtype, block, wb, cb, mb, device, **kw)

    # -- Algorithm 1 state --------------------------------------------------------------------
    def init_caches(self, weights: Optional[torch.Tensor], stream=None) -> None:
        """Both caches := exponents(weights) (or zero when ``weights`` is None)."""
        ciera.cache_init(self.plan, self.sender_cache, weights, stream)
        ciera.cache_init(self.plan, self.receiver_cache, weights, stream)

    # -- sender with a hash per block instead of the exponent cache -------------------------------
    def init_hash_cache(self, weights: Optional[torch.Tensor], stream=None) -> None:
        """Allocates (once) and fills the sender's HashCache and the scratch of the hashed encode."""
        if getattr(self, "hash_cache", None) is None:
            self.hash_cache = torch.zeros(max(self.plan.hash_cache_bytes, 16), dtype=torch.uint8, device=self.device)
            self.hashed_workspace = self.plan.new_workspace()
        ciera.hash_cache_init(self.plan, self.hash_cache, weights, stream)

    def encode_hashed(self, weights: torch.Tensor, stream=None) -> None:
        ciera.encode_hashed(self.plan, weights, self.hash_cache, self.msg_send, self.wire_bytes, self.changed_blocks,
                            self.hashed_workspace, self.status, stream)

    # -- entropy stage around the transport --------------------------------------------------------
    def _entropy_scratch(self) -> torch.Tensor:
        if getattr(self, "entropy_scratch", None) is None:
            self.entropy_scratch = torch.empty(max(self.plan.entropy_scratch_bytes, 16), dtype=torch.uint8,
                                               device=self.device)
        return self.entropy_scratch

    def entropy_encode(self, stream=None) -> None:
        """After encode: code the payloads of the messages to send (wire_bytes shrink)."""
        ciera.entropy_encode(self.plan, self.msg_send, self.wire_bytes, self._entropy_scratch(), stream)

    def entropy_decode(self, stream=None) -> None:
        """After transport: restore the raw payloads of the received messages (wire_bytes grow back)."""
        ciera.entropy_decode(self.plan, self.msg_recv, self.wire_bytes, self._entropy_scratch(), self.status, stream)

    # -- the three stages -----------------------------------------------------------------------
    def encode(self, weights: torch.Tensor, stream=None) -> None:
        ciera.encode(self.plan, weights, self.sender_cache, self.msg_send, self.wire_bytes, self.changed_blocks,
                     self.workspace, self.status, stream)

    def transport(self, stream=None) -> None:
        ciera.transport(self.plan, self.msg_send, self.msg_recv, self.wire_bytes, self.workspace, self.status, stream)

    def decode(self, weights_out: Optional[torch.Tensor] = None, stream=None, check_length: bool = True) -> None:
        out = self.weights_out if weights_out is None else weights_out
        ciera.decode(self.plan, self.msg_recv, self.receiver_cache, out,
                     self.wire_bytes if check_length else None, self.workspace, self.status, stream)

    def step(self, weights: torch.Tensor, weights_out: Optional[torch.Tensor] = None, stream=None) -> None:
        self.encode(weights, stream)
        self.transport(stream)
        self.decode(weights_out, stream)

    def device_buffers(self, weights_dev: torch.Tensor) -> "ciera.DeviceBuffers":
        b = ciera.DeviceBuffers()
        b.weights_dev = weights_dev.data_ptr()
        b.sender_cache_dev = self.sender_cache.data_ptr()
        b.msg_send_dev = self.msg_send.data_ptr()
        b.msg_recv_dev = self.msg_recv.data_ptr()
        b.receiver_cache_dev = self.receiver_cache.data_ptr()
        b.weights_out_dev = self.weights_out.data_ptr()
        b.wire_bytes_dev = self.wire_bytes.data_ptr()
        b.changed_blocks_dev = self.changed_blocks.data_ptr()
        b.workspace_dev = self.workspace.data_ptr()
        b.status_dev = self.status.data_ptr()
        return b

    def step_host(self, weights_host: torch.Tensor, weights_out_host: torch.Tensor, staging: torch.Tensor,
                  wire_host: Optional[torch.Tensor] = None, stream=None) -> None:
        """Whole step on host-resident weights through ``ciera_roundtrip_host``."""
        ciera.roundtrip_host(self.plan, weights_host, weights_out_host, wire_host, self.device_buffers(staging), stream)

    def check_status(self) -> None:
        s = int(self.status.item())
        if s != 0:
            # a kernel that gave up leaves its scratch in an unspecified state: make it usable again
            ciera.workspace_init(self.plan, self.workspace)
            if getattr(self, "hashed_workspace", None) is not None:
                ciera.workspace_init(self.plan, self.hashed_workspace)
            raise ciera.CieraError("device status", s)

    # -- accounting -------------------------------------------------------------------------------
    def paper_bytes(self) -> int:
        """Transmitted bytes of the last encode by the paper's count (no pads)."""
        wire = self.wire_bytes.cpu().numpy()
        total = 0
        for u, w in zip(self.units, wire):
            n = int(u["n_values"])
            if n == 0:
                continue
            payload = int(w) - ciera.payload_offset(n, self.dtype, self.block)
            total += ciera.message_bytes(n, self.dtype, self.block, payload)
        return total

    def n_blocks(self) -> int:
        n = self.units["n_values"].astype(np.int64)
        return int(((n + self.block - 1) // self.block).sum())


def pipelined_step(layers: List[LayerCodec], weights: List[torch.Tensor], outs: List[Optional[torch.Tensor]],
                   s_enc: torch.cuda.Stream, s_dec: torch.cuda.Stream, events=None) -> None:
    """One iteration over a stack of layers on two streams: the sender-side work of layer l+1
    (encode, then the transport of its message) runs on ``s_enc`` while the receiver-side
    decode of layer l runs on ``s_dec`` -- the shape of the paper's computation-communication
    pipelining, where only the decompression of layer l stays on the critical path.  A caller that
    runs several iterations back to back must make the next iteration's sender side of a layer wait
    for this iteration's decode of that layer (they share the layer's message buffers)."""
    n = len(layers)
    if events is None:
        events = [torch.cuda.Event() for _ in range(n)]
    for l in range(n):
        layers[l].encode(weights[l], s_enc)
        layers[l].transport(s_enc)
        events[l].record(s_enc)
        s_dec.wait_event(events[l])
        layers[l].decode(outs[l], s_dec)


class LayerPipeline:
    """A stack of layers stepped repeatedly on two streams (see ``pipelined_step``).

    Across iterations it keeps the dependency that the layers' buffers impose: the sender side of
    layer l in iteration i+1 (it overwrites the layer's messages, lengths and scratch) starts only
    after the decode of layer l in iteration i has finished.  ``timers``, if given, collects six CUDA
    events per layer and step: around encode, transport (both on the sender stream) and decode; with
    ``entropy`` the changed exponents are rANS-coded before the transport and restored after it, and
    four more events are collected around those two stages."""

    def __init__(self, layers: List[LayerCodec], s_enc: Optional[torch.cuda.Stream] = None,
                 s_dec: Optional[torch.cuda.Stream] = None, entropy: bool = False):
        self.layers = layers
        self.entropy = entropy
        self.s_enc = s_enc if s_enc is not None else torch.cuda.Stream()
        self.s_dec = s_dec if s_dec is not None else torch.cuda.Stream()
        self.serial = self.s_enc == self.s_dec
        self.sent = [torch.cuda.Event() for _ in layers]
        self.decoded = [torch.cuda.Event() for _ in layers]
        cur = torch.cuda.current_stream()
        for ev in self.decoded:
            ev.record(cur)

    def step(self, weights: List[torch.Tensor], outs: Optional[List[Optional[torch.Tensor]]] = None,
             timers: Optional[list] = None) -> None:
        s_enc, s_dec = self.s_enc, self.s_dec
        for l, (codec, w) in enumerate(zip(self.layers, weights)):
            if not self.serial:
                s_enc.wait_event(self.decoded[l])
            t = [torch.cuda.Event(enable_timing=True) for _ in range(10)] if timers is not None else None
            if t:
                t[0].record(s_enc)
            if getattr(codec, "hash_cache", None) is not None:
                codec.encode_hashed(w, s_enc)
            else:
                codec.encode(w, s_enc)
            if t:
                t[1].record(s_enc)
            if self.entropy:
                if t:
                    t[6].record(s_enc)
                codec.entropy_encode(s_enc)
                if t:
                    t[7].record(s_enc)
            if t:
                t[2].record(s_enc)
            codec.transport(s_enc)
            if t:
                t[3].record(s_enc)
            if not self.serial:
                self.sent[l].record(s_enc)
                s_dec.wait_event(self.sent[l])
            if self.entropy:
                if t:
                    t[8].record(s_dec)
                codec.entropy_decode(s_dec)
                if t:
                    t[9].record(s_dec)
            if t:
                t[4].record(s_dec)
            codec.decode(None if outs is None else outs[l], s_dec)
            if not self.serial:
                self.decoded[l].record(s_dec)
            if t:
                t[5].record(s_dec)
                timers.append(t)

    def wait(self) -> None:
        """Makes the current stream wait for everything queued so far."""
        cur = torch.cuda.current_stream()
        cur.wait_stream(self.s_enc)
        cur.wait_stream(self.s_dec)
