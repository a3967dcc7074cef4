"""Seeded synthetic inputs and workload shapes for the Distributed-Lion step.

This module holds NO optimizer arithmetic: it only describes parameter sets
(segment tables) and produces gradients / initial parameters.  It serves the
CUDA library's tests and benchmark and, separately, the CPU checker's tests, so
that both sides consume the same bytes.

Every value is a pure function of ``(seed, step, stream, arena index)`` built
from a 64-bit integer hash, a quantile table made once on the CPU, and single
IEEE float32 multiplies / adds issued as separate tensor ops.  Integer ops and
single float ops give the same bits on a CPU and on a GPU, so a slab generated
on either device is byte-identical, and any coordinate range can be generated
without generating the rest.

The shapes follow the workloads the paper trains (Section 5: ViT-B/16 on
ImageNet-1K, GPT-2-family decoders on OpenWebText); the values stand in for
those runs' gradients, which need the datasets: correlated Gaussians across
workers, g_i = a * shared + b * private_i.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

ALIGN = 128            # segment starts are multiples of this many elements
MAJORITY = 0
AVERAGE = 1
MAJORITY_TERNARY = 2      # Majority Vote with Delta = 0 on an even-N tie
_MASK64 = (1 << 64) - 1
_TABLE_BITS = 16
_CHUNK = 1 << 24       # elements generated per pass (bounds temporaries)


# --------------------------------------------------------------------------
# layout
# --------------------------------------------------------------------------
def layout(numels: Sequence[int], align: int = ALIGN) -> Tuple[List[Tuple[int, int]], int]:
    """Place tensors of the given sizes back to back, each start rounded up to ``align``.

    Returns ``(segments, d_pad)`` with ``segments[k] = (elem_offset, numel)``.
    """
    segs, off = [], 0
    for n in numels:
        segs.append((off, int(n)))
        off += (int(n) + align - 1) // align * align
    return segs, max(off, align)


@dataclass
class Workload:
    name: str
    numels: List[int]
    n_workers: int
    mode: int
    grad_dtype: str                  # "f32" | "bf16"
    a_shared: float                  # g_i = scale * (a_shared * s + a_private * e_i)
    a_private: float
    scale: float
    zero_frac: float = 0.0           # exact zeros: half shared by all workers, half per worker
    beta1: float = 0.9
    beta2: float = 0.99
    lr: float = 1e-4
    weight_decay: float = 0.1
    x_std: float = 0.02
    seed: int = 42
    segments: List[Tuple[int, int]] = field(default_factory=list)
    d_pad: int = 0

    def __post_init__(self):
        self.segments, self.d_pad = layout(self.numels)

    @property
    def d(self) -> int:
        return int(sum(self.numels))

    @property
    def grad_bytes(self) -> int:
        return 4 if self.grad_dtype == "f32" else 2


def _gpt_shapes(vocab: int, n_pos: int, hidden: int, layers: int, ffn: int) -> List[int]:
    s = [vocab * hidden]
    if n_pos:
        s.append(n_pos * hidden)
    for _ in range(layers):
        s += [hidden * 3 * hidden, hidden * hidden, hidden * ffn, ffn * hidden,
              hidden, hidden, hidden, hidden]
    s += [hidden, hidden]
    return s


def _vit_b16_shapes() -> List[int]:
    s = [16 * 16 * 3 * 768]
    for _ in range(12):
        s += [768 * 2304, 768 * 768, 768 * 3072, 3072 * 768]
    s.append(768 * 1000)
    return s


def workload(name: str, n_workers: Optional[int] = None, mode: Optional[int] = None) -> Workload:
    """The five benchmark configurations (``c1`` .. ``c5``); ``n_workers`` / ``mode`` override."""
    inv = 1.0 / math.sqrt(1.25)
    if name == "c1":      # flat 1 Mi fp32, N=4, majority vote, 1 % exact zeros
        w = Workload("c1", [1 << 20], 4, MAJORITY, "f32", 1.0, 0.5, 1.0, zero_frac=0.01,
                     lr=1e-4, weight_decay=0.1)
    elif name == "c2":    # GPT-2-small-shaped table, N=8, averaging, bf16 grads of std 1e-3
        w = Workload("c2", _gpt_shapes(50257, 1024, 768, 12, 3072), 8, AVERAGE, "bf16",
                     inv, 0.5 * inv, 1e-3, lr=9e-5, weight_decay=1.0)
    elif name == "c3":    # ViT-B/16-shaped table, N=32, majority vote (even-N ties), bf16
        r = 1.0 / math.sqrt(2.0)
        w = Workload("c3", _vit_b16_shapes(), 32, MAJORITY, "bf16", r, r, 1e-3,
                     lr=1e-4, weight_decay=10.0)
    elif name == "c4":    # flat 100 M fp32, N swept 2..128, 0.3 shared / 0.7 private variance
        w = Workload("c4", [100_000_000], 128, MAJORITY, "f32", math.sqrt(0.3), math.sqrt(0.7),
                     1.0, lr=1e-4, weight_decay=0.1)
    elif name == "c5":    # 1.3B decoder-shaped table, N=16, bf16 grads, fp32 m per worker
        w = Workload("c5", _gpt_shapes(50257, 0, 2048, 24, 8192), 16, MAJORITY, "bf16",
                     inv, 0.5 * inv, 1e-3, lr=9e-5, weight_decay=1.0)
    else:
        raise KeyError(name)
    if n_workers is not None:
        w.n_workers = int(n_workers)
    if mode is not None:
        w.mode = int(mode)
    return w


def custom(numels: Sequence[int], n_workers: int, mode: int, grad_dtype: str = "f32",
           **kw) -> Workload:
    """A small ad-hoc workload for tests (defaults: c1's value model)."""
    args = dict(a_shared=1.0, a_private=0.5, scale=1.0)
    args.update(kw)
    return Workload("custom", list(numels), n_workers, mode, grad_dtype, **args)


# --------------------------------------------------------------------------
# counter-based generator
# --------------------------------------------------------------------------
def _mix_py(z: int) -> int:
    """64-bit finaliser (xor-shift-multiply), Python-int version for keys."""
    z &= _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def _key(seed: int, step: int, stream: int) -> int:
    k = _mix_py(seed + 0x9E3779B97F4A7C15)
    k = _mix_py(k ^ ((step + 1) * 0xD1B54A32D192ED03 & _MASK64))
    k = _mix_py(k ^ ((stream + 1) * 0x8CB92BA72F3D8DD7 & _MASK64))
    return k


def _signed(c: int) -> int:
    c &= _MASK64
    return c - (1 << 64) if c >= (1 << 63) else c


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _hash(idx: torch.Tensor, key: int) -> torch.Tensor:
    """The same finaliser on an int64 tensor of counters (wrapping multiply)."""
    z = idx + _signed(key)
    z = (z ^ _lsr(z, 30)) * _signed(0xBF58476D1CE4E5B9)
    z = (z ^ _lsr(z, 27)) * _signed(0x94D049BB133111EB)
    return z ^ _lsr(z, 31)


_tables_cpu: Optional[Tuple[torch.Tensor, torch.Tensor]] = None
_tables_dev = {}


def _tables(device: torch.device) -> Tuple[torch.Tensor, torch.Tensor]:
    """Standard-normal quantile table: bin lower edge and bin width, float32.

    Always computed on the CPU (double precision, then rounded once) and copied,
    so every device sees the same bytes.
    """
    global _tables_cpu
    if _tables_cpu is None:
        from scipy.special import ndtri
        n = 1 << _TABLE_BITS
        p = np.arange(n + 1, dtype=np.float64) / n
        p[0], p[-1] = 0.25 / n, 1.0 - 0.25 / n
        e = ndtri(p)
        lo = torch.from_numpy(e[:-1].astype(np.float32))
        width = torch.from_numpy((e[1:] - e[:-1]).astype(np.float32))
        _tables_cpu = (lo, width)
    key = str(device)
    if key not in _tables_dev:
        _tables_dev[key] = tuple(t.to(device) for t in _tables_cpu)
    return _tables_dev[key]


def _normal_and_bits(key: int, lo: int, hi: int, device: torch.device):
    """Approximately N(0,1) float32 values for counters [lo, hi), plus 16 spare hash bits."""
    idx = torch.arange(lo, hi, dtype=torch.int64, device=device)
    h = _hash(idx, key)
    t_lo, t_w = _tables(device)
    u = h & 0xFFFF
    frac = (_lsr(h, 16) & 0xFFFF).to(torch.float32) * (1.0 / 65536.0)
    val = t_lo[u] + frac * t_w[u]          # two ops, two roundings: same bits on every device
    spare = _lsr(h, 32) & 0xFFFF
    return val, spare


def _scalar(v: float, device) -> torch.Tensor:
    return torch.tensor(v, dtype=torch.float32, device=device)


def fill_grads(w: Workload, step: int, out: torch.Tensor, lo: int = 0,
               hi: Optional[int] = None, workers: Optional[Sequence[int]] = None) -> torch.Tensor:
    """Write g_{i,step}[lo:hi] for every worker into ``out`` ([N, hi-lo], f32 or bf16).

    ``lo``/``hi`` are arena indices (padding included); padding lanes get 0.
    ``workers`` restricts the rows to those workers (``out`` is [len(workers), hi-lo]);
    a worker's values do not depend on which other workers are generated with it.
    """
    hi = w.d_pad if hi is None else hi
    dev = out.device
    ids = list(range(w.n_workers)) if workers is None else [int(i) for i in workers]
    assert out.shape == (len(ids), hi - lo)
    a_s, a_p, sc = (_scalar(v, dev) for v in (w.a_shared, w.a_private, w.scale))
    zthr = int(round(w.zero_frac * 0.5 * 65536))
    for c0 in range(lo, hi, _CHUNK):
        c1 = min(hi, c0 + _CHUNK)
        s, s_bits = _normal_and_bits(_key(w.seed, step, 0), c0, c1, dev)
        s = s * a_s
        for row, i in enumerate(ids):
            e, e_bits = _normal_and_bits(_key(w.seed, step, 1 + i), c0, c1, dev)
            g = e * a_p
            g = g + s
            if w.scale != 1.0:
                g = g * sc
            if zthr:
                g = torch.where((s_bits < zthr) | (e_bits < zthr), torch.zeros_like(g), g)
            out[row, c0 - lo:c1 - lo] = g.to(out.dtype)
    _zero_padding(w, out, lo, hi)
    return out


def fill_x0(w: Workload, out: torch.Tensor, lo: int = 0, hi: Optional[int] = None) -> torch.Tensor:
    """Initial parameters x_0[lo:hi] ~ N(0, x_std), float32; padding lanes 0."""
    hi = w.d_pad if hi is None else hi
    dev = out.device
    assert out.shape == (hi - lo,)
    std = _scalar(w.x_std, dev)
    for c0 in range(lo, hi, _CHUNK):
        c1 = min(hi, c0 + _CHUNK)
        v, _ = _normal_and_bits(_key(w.seed, -1, 0), c0, c1, dev)
        out[c0 - lo:c1 - lo] = v * std
    _zero_padding(w, out.unsqueeze(0), lo, hi)
    return out


def _zero_padding(w: Workload, out2d: torch.Tensor, lo: int, hi: int) -> None:
    prev_end = 0
    for off, n in list(w.segments) + [(w.d_pad, 0)]:
        a, b = max(prev_end, lo), min(off, hi)
        if a < b:
            out2d[:, a - lo:b - lo] = 0
        prev_end = off + n


def grad_torch_dtype(w: Workload) -> torch.dtype:
    return torch.float32 if w.grad_dtype == "f32" else torch.bfloat16


def as_numpy_grads(g: torch.Tensor) -> np.ndarray:
    """Host view of a gradient tensor: float32, or the uint16 bit patterns of bf16."""
    g = g.detach().cpu().contiguous()
    if g.dtype == torch.bfloat16:
        return g.view(torch.int16).numpy().view(np.uint16)
    return g.numpy()
