"""Seeded synthetic inputs: weight trajectories and unit layouts.

This module serves both the CPU oracle's tests and the CUDA path's tests/benchmark.  It
holds none of the codec's arithmetic (no split, no merge, no message format): the
message-capacity rule is passed in by the caller, so each side supplies its own.

The paper measures on real training runs of OLMoE-1B-7B and other MoE models; neither
the models nor the corpora are available here, so these trajectories take the paper's
tensor shapes and the change rates it reports (Section 2.2-2.4) and stand in for them:

* ``step_gaussian``   W <- cast(W + 1e-4 * N(0,1))                      (tiny config)
* ``step_adam_like``  W <- cast(W + lr * sign(N(0,1)) * U(0.5,1.5))    (i.i.d. over values)
* ``step_clustered``  the Adam-like step applied only to a seeded fraction ``f`` of
  aligned segments, the rest bit-identical: reproduces a low block change rate at a
  sub-percent element change rate, the structure the paper reports for expert FFN shards
* ``inject_exponent_changes``  exact-rate exponent flips (+-1 on the exponent field),
  mantissas redrawn everywhere, for the change-rate sweep
"""
from __future__ import annotations

from typing import Callable, Iterable, List, Sequence, Tuple

import numpy as np
import torch

UNIT_DTYPE = np.dtype(
    [
        ("n_values", "<u8"),
        ("weights_off", "<u8"),
        ("cache_off", "<u8"),
        ("msg_off", "<u8"),
        ("msg_capacity", "<u8"),
    ]
)

TORCH_DTYPES = {"bf16": torch.bfloat16, "fp32": torch.float32, "fp16": torch.float16}
VALUE_BYTES = {"bf16": 2, "fp32": 4, "fp16": 2}


def _align(x: int, a: int) -> int:
    return (x + a - 1) // a * a


# ----------------------------------------------------------------------------- shapes


def olmoe_layer_shapes(n_experts: int = 64, d_model: int = 2048, d_ff: int = 1024) -> List[Tuple[int, int]]:
    """Expert FFN matrices of one OLMoE-shaped MoE layer: gate, up (d_model x d_ff), down."""
    shapes: List[Tuple[int, int]] = []
    for _ in range(n_experts):
        shapes += [(d_model, d_ff), (d_model, d_ff), (d_ff, d_model)]
    return shapes


def fine_grained_layer_shapes(n_experts: int = 256, d_model: int = 2048, d_ff: int = 512):
    return olmoe_layer_shapes(n_experts, d_model, d_ff)


def dense_tensor_sizes() -> List[int]:
    """Small dense tensors of the mixed-shape sweep, 4 KB ... 256 MB of bf16 in x4 steps."""
    out = []
    nbytes = 4 * 1024
    while nbytes <= 256 * 1024 * 1024:
        out.append(nbytes // 2)
        nbytes *= 4
    return out


# ----------------------------------------------------------------------------- layout


def layout_units(
    tensor_numels: Sequence[int],
    n_shards: int,
    value_bytes: int,
    capacity_fn: Callable[[int], int],
    align: int = 256,
):
    """Split every tensor into ``n_shards`` consecutive shards (a flat 1/W split) and lay
    the resulting units out in three flat buffers.

    Returns ``(units, weights_bytes, cache_bytes, msg_bytes)`` where ``units`` is a numpy
    array of UNIT_DTYPE.  Every offset is a multiple of ``align`` bytes.  ``capacity_fn(n)``
    gives the message-slot size of a unit of ``n`` values.
    """
    units = []
    w_off = c_off = m_off = 0
    for numel in tensor_numels:
        per = -(-numel // n_shards)
        for p in range(n_shards):
            lo = min(p * per, numel)
            hi = min(lo + per, numel)
            n = hi - lo
            cap = int(capacity_fn(n))
            units.append((n, w_off, c_off, m_off, cap))
            w_off += _align(n * value_bytes, align)
            c_off += _align(n, align)
            m_off += _align(cap, align)
    arr = np.array(units, dtype=UNIT_DTYPE)
    return arr, w_off, c_off, m_off


def unit_value_index(units: np.ndarray, value_bytes: int) -> np.ndarray:
    """For a flat weight buffer laid out by ``layout_units``: index (in values) of each
    unit's first value."""
    return (units["weights_off"] // value_bytes).astype(np.int64)


# ----------------------------------------------------------------------------- weights


def make_generator(seed: int, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def init_weights(n: int, dtype: str, gen: torch.Generator, std: float = 0.02) -> torch.Tensor:
    """W0 ~ N(0, std), drawn in fp32 and cast."""
    w = torch.randn(n, generator=gen, device=gen.device, dtype=torch.float32) * std
    return w.to(TORCH_DTYPES[dtype])


def step_gaussian(w: torch.Tensor, gen: torch.Generator, sigma: float = 1e-4) -> torch.Tensor:
    d = torch.randn(w.numel(), generator=gen, device=w.device, dtype=torch.float32) * sigma
    return (w.float() + d).to(w.dtype)


def _adam_like_delta(n: int, gen: torch.Generator, device, lr: float) -> torch.Tensor:
    s = torch.randn(n, generator=gen, device=device, dtype=torch.float32).sign_()
    u = torch.rand(n, generator=gen, device=device, dtype=torch.float32) + 0.5
    return s.mul_(u).mul_(lr)


def step_adam_like(w: torch.Tensor, gen: torch.Generator, lr: float = 1e-4) -> torch.Tensor:
    return (w.float() + _adam_like_delta(w.numel(), gen, w.device, lr)).to(w.dtype)


def step_clustered(w: torch.Tensor, gen: torch.Generator, f: float = 0.22, seg: int = 512,
                   lr: float = 1e-4) -> torch.Tensor:
    """Adam-like step on a Bernoulli(f) subset of ``seg``-aligned segments only."""
    n = w.numel()
    nseg = -(-n // seg)
    hit = torch.rand(nseg, generator=gen, device=w.device, dtype=torch.float32) < f
    mask = hit.repeat_interleave(seg)[:n]
    d = _adam_like_delta(n, gen, w.device, lr)
    d.mul_(mask)
    return (w.float() + d).to(w.dtype)


def as_bits(w: torch.Tensor) -> np.ndarray:
    """Raw bit patterns on the host: uint16 for bf16, uint32 for fp32."""
    if w.dtype in (torch.bfloat16, torch.float16):
        return w.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
    if w.dtype == torch.float32:
        return w.detach().cpu().contiguous().view(torch.int32).numpy().view(np.uint32)
    raise TypeError(w.dtype)


def from_bits(bits: np.ndarray) -> torch.Tensor:
    if bits.dtype == np.uint16:
        return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)
    if bits.dtype == np.uint32:
        return torch.from_numpy(bits.view(np.int32).copy()).view(torch.float32)
    raise TypeError(bits.dtype)


def inject_exponent_changes(w: torch.Tensor, gen: torch.Generator, c: float, seg: int = 0) -> torch.Tensor:
    """Next iterate with an exact-rate exponent change.

    A Bernoulli(c) mask over values (``seg == 0``) or over ``seg``-aligned segments
    (``seg > 0``, every value of a hit segment changes) selects the values whose exponent
    field moves by +-1 (kept inside 1..254, or 1..30 for fp16, and always moving); every value gets
    a fresh random mantissa; signs are kept.
    """
    n = w.numel()
    dev = w.device
    if w.dtype in (torch.bfloat16, torch.float16):
        bits = w.view(torch.int16).to(torch.int32) & 0xFFFF
        mant_bits, total = (7, 16) if w.dtype == torch.bfloat16 else (10, 16)
    else:
        bits = w.view(torch.int32).to(torch.int64) & 0xFFFFFFFF
        mant_bits, total = 23, 32
    emax = (1 << (total - 1 - mant_bits)) - 1  # all-ones exponent field: 255, or 31 for fp16
    if seg > 0:
        nseg = -(-n // seg)
        hit = torch.rand(nseg, generator=gen, device=dev) < c
        mask = hit.repeat_interleave(seg)[:n]
    else:
        mask = torch.rand(n, generator=gen, device=dev) < c
    e = (bits >> mant_bits) & emax
    up = torch.rand(n, generator=gen, device=dev) < 0.5
    up = (up | (e <= 1)) & ~(e >= emax - 1)
    e_new = torch.where(mask, torch.where(up, e + 1, e - 1), e)
    mant = torch.randint(0, 1 << mant_bits, (n,), generator=gen, device=dev, dtype=bits.dtype)
    sign = (bits >> (total - 1)) & 1
    out = (sign << (total - 1)) | (e_new << mant_bits) | mant
    if total == 16:
        out = torch.where(out >= 0x8000, out - 0x10000, out).to(torch.int16)
        return out.view(w.dtype)
    out = torch.where(out >= 0x80000000, out - 0x100000000, out).to(torch.int32)
    return out.view(torch.float32)


# ----------------------------------------------------------------------------- trajectories


def trajectory(n: int, dtype: str, seed: int, n_iters: int, model: str, device="cpu",
               **kw) -> Iterable[torch.Tensor]:
    """Yield W_0, W_1, ..., W_{n_iters} (flat tensors of ``n`` values)."""
    gen = make_generator(seed, device)
    w = init_weights(n, dtype, gen)
    yield w
    for _ in range(n_iters):
        if model == "gaussian":
            w = step_gaussian(w, gen, **kw)
        elif model == "adam":
            w = step_adam_like(w, gen, **kw)
        elif model == "clustered":
            w = step_clustered(w, gen, **kw)
        elif model == "inject":
            w = inject_exponent_changes(w, gen, **kw)
        else:
            raise ValueError(model)
        yield w
