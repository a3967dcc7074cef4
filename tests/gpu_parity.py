"""Helpers for the GPU-vs-oracle parity tests: run the CUDA library (through the
C ABI binding) and the CPU oracle on the same seeded inputs and compare element
by element.  The oracle never sees a value produced by the CUDA path.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

from oracle import dlion_oracle as orc
from paper_2404_00438_b200 import inputs

# Tolerance on fp32 state (momentum, parameters): 2 units in the last place, the
# bound the workload statement gives; signs, counts and Delta bits are exact.
TOL_ULP = 2


def ulp_diff(a: np.ndarray, b: np.ndarray) -> int:
    """Largest distance in units in the last place between two float32 arrays."""
    if a.size == 0:
        return 0
    assert a.dtype == np.float32 and b.dtype == np.float32 and a.shape == b.shape
    nan_a, nan_b = np.isnan(a), np.isnan(b)
    assert np.array_equal(nan_a, nan_b), "NaN pattern differs"
    ia = a.view(np.int32).astype(np.int64)
    ib = b.view(np.int32).astype(np.int64)
    ia = np.where(ia < 0, -(ia & 0x7FFFFFFF), ia)
    ib = np.where(ib < 0, -(ib & 0x7FFFFFFF), ib)
    d = np.abs(ia - ib)
    d[nan_a] = 0
    return int(d.max())


def gdtype_of(w: inputs.Workload) -> int:
    return 0 if w.grad_dtype == "f32" else 1


def clip_segments(segments: Sequence[Tuple[int, int]], lo: int, hi: int) -> List[Tuple[int, int]]:
    """Segments restricted to the arena range [lo, hi), offsets relative to lo."""
    out = []
    for off, n in segments:
        a, b = max(off, lo), min(off + n, hi)
        if a < b:
            out.append((a - lo, b - a))
    return out or [(0, 0)]


def make_ctx(dl, w: inputs.Workload, mode: Optional[int] = None):
    return dl.Dlion(w.segments, w.d_pad, w.n_workers, w.beta1, w.beta2, w.lr, w.weight_decay,
                    w.mode if mode is None else mode, gdtype_of(w))


class OracleState:
    """Oracle run on a coordinate slab [lo, hi) (coordinates are independent)."""

    def __init__(self, w: inputs.Workload, lo: int, hi: int, m0: np.ndarray, x0: np.ndarray,
                 modes: Sequence[int]):
        self.w, self.lo, self.hi = w, lo, hi
        self.n = hi - lo
        self.segs = clip_segments(w.segments, lo, hi)
        self.m = np.ascontiguousarray(m0, dtype=np.float32).copy()
        self.x = {md: np.ascontiguousarray(x0, dtype=np.float32).copy() for md in modes}
        self.packed = np.zeros((w.n_workers, self.n // 32), np.uint32)
        self.dbits = {md: np.zeros(self.n // 32, np.uint32) for md in modes}
        self.count = {md: (np.zeros(self.n, np.uint8) if w.n_workers <= 255 else None) for md in modes}

    def step(self, g: np.ndarray, nthreads: int = 8) -> None:
        w = self.w
        orc.worker_step(self.segs, self.n, w.n_workers, np.ascontiguousarray(g), self.m, self.packed,
                        w.beta1, w.beta2, nthreads=nthreads)
        for md in self.x:
            orc.aggregate_apply(self.segs, self.n, w.n_workers, md, self.packed, self.x[md], w.lr,
                                w.weight_decay, delta_bits=self.dbits[md], count=self.count[md],
                                nthreads=nthreads)


def compare(tag: str, got: np.ndarray, want: np.ndarray, exact: bool) -> int:
    if exact:
        if not np.array_equal(got, want):
            bad = np.flatnonzero(got.reshape(-1) != want.reshape(-1))
            raise AssertionError(f"{tag}: {bad.size} mismatches, first at flat index {bad[0]}: "
                                 f"got {got.reshape(-1)[bad[0]]!r} want {want.reshape(-1)[bad[0]]!r}")
        return 0
    u = ulp_diff(got, want)
    assert u <= TOL_ULP, f"{tag}: {u} ulp > {TOL_ULP}"
    return u


def run_small(dl, w: inputs.Workload, steps: int, path: str = "two_stage",
              modes: Sequence[int] = (0, 1), m0: Optional[torch.Tensor] = None,
              x0: Optional[torch.Tensor] = None, grads: Optional[List[torch.Tensor]] = None) -> int:
    """Whole-arena comparison on a case the oracle finishes quickly.

    path: "two_stage" (worker_step(-1) + aggregate_apply), "per_worker"
    (worker_step(i) for each i), or "fused".  Returns the largest ulp distance seen.
    """
    dev = torch.device("cuda:0")
    N, D, W = w.n_workers, w.d_pad, w.d_pad // 32
    gdt = inputs.grad_torch_dtype(w)
    if x0 is None:
        x0 = inputs.fill_x0(w, torch.empty(D))
    if m0 is None:
        m0 = torch.zeros(N, D)
    ora = OracleState(w, 0, D, m0.numpy(), x0.numpy(), modes)
    ctx = {md: make_ctx(dl, w, md) for md in modes}
    m = m0.to(dev)
    xs = {md: x0.to(dev) for md in modes}
    packed = torch.zeros(N, W, dtype=torch.int32, device=dev)
    dbits = torch.zeros(W, dtype=torch.int32, device=dev)
    count = torch.full((D,), 0, dtype=torch.uint8, device=dev) if N <= 255 else None   # byte counts: N <= 255
    worst = 0
    for t in range(steps):
        g_cpu = grads[t] if grads is not None else inputs.fill_grads(w, t, torch.empty(N, D, dtype=gdt))
        g = g_cpu.to(dev)
        ora.step(inputs.as_numpy_grads(g_cpu))
        m_before = m.clone()
        for k, md in enumerate(modes):
            if k > 0:
                m.copy_(m_before)               # every mode starts the step from the same momentum
            packed.zero_()
            if path == "fused":
                ctx[md].step_fused(g, m, xs[md], packed)
            else:
                if path == "per_worker":
                    for i in range(N):
                        ctx[md].worker_step(i, g[i], m[i], packed[i])
                else:
                    ctx[md].worker_step(-1, g, m, packed)
                dbits.zero_()
                if count is not None:
                    count.zero_()
                ctx[md].aggregate_apply(packed, xs[md], dbits, count)
            torch.cuda.synchronize()
            tag = f"step {t} mode {md} {path}"
            compare(tag + " packed", packed.cpu().numpy().view(np.uint32), ora.packed, True)
            worst = max(worst, compare(tag + " m", m.cpu().numpy(), ora.m, False))
            worst = max(worst, compare(tag + " x", xs[md].cpu().numpy(), ora.x[md], False))
            if path != "fused":
                compare(tag + " delta_bits", dbits.cpu().numpy().view(np.uint32), ora.dbits[md], True)
                if count is not None:
                    compare(tag + " count", count.cpu().numpy(), ora.count[md], True)
    for c in ctx.values():
        c.destroy()
    return worst


def pick_slabs(w: inputs.Workload, n_random: int = 3, width: int = 1 << 14, seed: int = 7):
    """Arena ranges to check at full size: both ends, a few segment joints, random interiors."""
    D = w.d_pad
    width = min(width, D)
    slabs = {(0, width), (D - width, D)}
    joints = [off for off, _ in w.segments[1:]]
    rng = np.random.default_rng(seed)
    for j in ([joints[0], joints[len(joints) // 2], joints[-1]] if joints else []):
        lo = max(0, min(D - width, (j - width // 2) // 128 * 128))
        slabs.add((lo, lo + width))
    for _ in range(n_random):
        lo = int(rng.integers(0, max(1, (D - width) // 128))) * 128
        slabs.add((lo, lo + width))
    return sorted(slabs)


def run_full(dl, w: inputs.Workload, steps: int, path: str = "two_stage",
             modes: Sequence[int] = (0, 1), slabs=None) -> int:
    """Full-size run in the launch configuration the benchmark times; the oracle
    recomputes sampled coordinate slabs from the same gradient bytes."""
    dev = torch.device("cuda:0")
    N, D, W = w.n_workers, w.d_pad, w.d_pad // 32
    gdt = inputs.grad_torch_dtype(w)
    slabs = slabs or pick_slabs(w)
    g = torch.empty(N, D, dtype=gdt, device=dev)
    m = torch.zeros(N, D, device=dev)
    x0 = inputs.fill_x0(w, torch.empty(D, device=dev))
    xs = {md: x0.clone() for md in modes}
    del x0
    packed = torch.zeros(N, W, dtype=torch.int32, device=dev)
    ctx = {md: make_ctx(dl, w, md) for md in modes}
    oras = [OracleState(w, lo, hi, np.zeros((N, hi - lo), np.float32),
                        xs[modes[0]][lo:hi].cpu().numpy(), modes) for lo, hi in slabs]
    worst = 0
    for t in range(steps):
        inputs.fill_grads(w, t, g)
        for o in oras:
            o.step(inputs.as_numpy_grads(g[:, o.lo:o.hi]))
        if path == "fused":
            assert len(modes) == 1
            ctx[modes[0]].step_fused(g, m, xs[modes[0]], packed)
        else:
            ctx[modes[0]].worker_step(-1, g, m, packed)
            for md in modes:
                ctx[md].aggregate_apply(packed, xs[md])
        torch.cuda.synchronize()
        for o in oras:
            tag = f"{w.name} N={N} step {t} slab [{o.lo},{o.hi}) {path}"
            compare(tag + " packed", packed[:, o.lo // 32:o.hi // 32].cpu().numpy().view(np.uint32),
                    o.packed, True)
            worst = max(worst, compare(tag + " m", m[:, o.lo:o.hi].cpu().numpy(), o.m, False))
            for md in modes:
                worst = max(worst, compare(tag + f" x mode {md}", xs[md][o.lo:o.hi].cpu().numpy(),
                                           o.x[md], False))
    for c in ctx.values():
        c.destroy()
    return worst
