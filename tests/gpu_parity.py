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


# --------------------------------------------------------------------------
# full-size runs: the oracle works slab by slab (coordinates are independent, so a
# slab is a complete problem); what it produces is uploaded and compared on the GPU
# --------------------------------------------------------------------------
def ulp_diff_dev(a: torch.Tensor, b: torch.Tensor) -> int:
    """ulp_diff for two float32 tensors on the same device (bounded temporaries)."""
    assert a.dtype == torch.float32 and b.dtype == torch.float32 and a.shape == b.shape
    ia, ib = a.reshape(-1).view(torch.int32), b.reshape(-1).view(torch.int32)
    if torch.equal(ia, ib):
        return 0
    worst = 0
    for c0 in range(0, ia.numel(), 1 << 26):
        fa, fb = a.reshape(-1)[c0:c0 + (1 << 26)], b.reshape(-1)[c0:c0 + (1 << 26)]
        nan_a, nan_b = torch.isnan(fa), torch.isnan(fb)
        assert torch.equal(nan_a, nan_b), "NaN pattern differs"
        ka, kb = (v.view(torch.int32).to(torch.int64) for v in (fa, fb))
        ka = torch.where(ka < 0, -(ka & 0x7FFFFFFF), ka)
        kb = torch.where(kb < 0, -(kb & 0x7FFFFFFF), kb)
        d = (ka - kb).abs()
        d[nan_a] = 0
        worst = max(worst, int(d.max().item()))
    return worst


def bf16_ulp_diff_dev(a: torch.Tensor, b: torch.Tensor) -> int:
    """Largest distance in bf16 units in the last place between two int16 tensors of bf16 bits."""
    if a.numel() == 0 or torch.equal(a, b):
        return 0
    ka, kb = a.to(torch.int32), b.to(torch.int32)
    ka = torch.where(ka < 0, -(ka & 0x7FFF), ka)
    kb = torch.where(kb < 0, -(kb & 0x7FFF), kb)
    return int((ka - kb).abs().max().item())


def compare_dev(tag: str, got: torch.Tensor, want: torch.Tensor, exact: bool) -> int:
    """got: the CUDA library's result (device); want: the oracle's, uploaded.  Integer and
    byte data are compared bit for bit, float32 state within TOL_ULP."""
    assert got.shape == want.shape and got.dtype == want.dtype, f"{tag}: shape or dtype differs"
    if exact:
        if not torch.equal(got, want):
            bad = torch.nonzero(got.reshape(-1) != want.reshape(-1))
            k = int(bad[0].item())
            raise AssertionError(f"{tag}: {bad.numel()} mismatches, first at flat index {k}: "
                                 f"got {got.reshape(-1)[k].item()!r} want {want.reshape(-1)[k].item()!r}")
        return 0
    u = ulp_diff_dev(got, want)
    assert u <= TOL_ULP, f"{tag}: {u} ulp > {TOL_ULP}"
    return u


def _pinned(shape, dtype) -> torch.Tensor:
    return torch.zeros(shape, dtype=dtype, pin_memory=True)


class SlabOracle:
    """The oracle's state of one arena range [lo, hi), in pinned host memory so that the
    per-step uploads run at PCIe speed.  state = "bf16" keeps the momentum as bf16 bits."""

    def __init__(self, w: inputs.Workload, lo: int, hi: int, modes: Sequence[int], state: str = "f32",
                 counts: bool = True):
        self.w, self.lo, self.hi, self.n, self.state = w, lo, hi, hi - lo, state
        self.segs = clip_segments(w.segments, lo, hi)
        N, n = w.n_workers, self.n
        self.m = _pinned((N, n), torch.float32 if state == "f32" else torch.int16)
        self.packed = _pinned((N, n // 32), torch.int32)
        self.x = {md: _pinned((n,), torch.float32) for md in modes}
        self.dbits = {md: _pinned((n // 32,), torch.int32) for md in modes}
        self.count = {md: (_pinned((n,), torch.uint8) if counts and N <= 255 else None) for md in modes}

    def reset(self, x0: torch.Tensor) -> None:
        self.m.zero_()
        for md in self.x:
            self.x[md].copy_(x0)

    def step(self, g: np.ndarray, nthreads: int) -> None:
        w = self.w
        m = self.m.numpy() if self.state == "f32" else self.m.numpy().view(np.uint16)
        packed = self.packed.numpy().view(np.uint32)
        if self.state == "f32":
            orc.worker_step(self.segs, self.n, w.n_workers, g, m, packed, w.beta1, w.beta2, nthreads=nthreads)
        else:
            orc.worker_step_ex(self.segs, self.n, w.n_workers, g, m, packed, [w.beta1] * w.n_workers,
                               [w.beta2] * w.n_workers, nthreads=nthreads)
        for md in self.x:
            orc.aggregate_apply(self.segs, self.n, w.n_workers, md, packed, self.x[md].numpy(), w.lr,
                                w.weight_decay, delta_bits=self.dbits[md].numpy().view(np.uint32),
                                count=None if self.count[md] is None else self.count[md].numpy(),
                                nthreads=nthreads)


def partition(d_pad: int, width: int):
    """[0, d_pad) cut into consecutive ranges of at most `width` coordinates (a multiple of 128)."""
    assert width % 128 == 0
    return [(lo, min(lo + width, d_pad)) for lo in range(0, d_pad, width)]


def pick_slabs(w: inputs.Workload, frac: float = 0.0, n_random: int = 3, width: int = 1 << 14,
               interior: int = 1 << 20, seed: int = 7):
    """Arena ranges to follow over many steps at full size: both ends, EVERY joint between two
    tensors (a window of `width` coordinates around it), and random interior ranges -- n_random
    of them, or as many ranges of `interior` coordinates as it takes to cover `frac` of the
    arena.  Overlapping ranges are merged."""
    D = w.d_pad
    width = min(width, D)
    want = [(0, width), (D - width, D)]
    for off, _ in w.segments[1:]:
        lo = max(0, min(D - width, (off - width // 2) // 128 * 128))
        want.append((lo, lo + width))
    rng = np.random.default_rng(seed)
    if frac > 0:
        interior = min(interior, D)
        for _ in range(int(np.ceil(frac * D / interior))):
            lo = int(rng.integers(0, max(1, (D - interior) // 128 + 1))) * 128
            want.append((lo, lo + interior))
    else:
        for _ in range(n_random):
            lo = int(rng.integers(0, max(1, (D - width) // 128))) * 128
            want.append((lo, lo + width))
    merged = []
    for lo, hi in sorted(want):
        if merged and lo <= merged[-1][1]:
            merged[-1] = (merged[-1][0], max(merged[-1][1], hi))
        else:
            merged.append((lo, hi))
    return merged


def run_full(dl, w: inputs.Workload, steps: int, path: str = "two_stage",
             modes: Sequence[int] = (0, 1), slabs=None, persist: bool = True, state: str = "f32",
             width: int = 1 << 22) -> int:
    """Full-size run in the launch configuration the benchmark times, checked against the
    oracle on the arena ranges `slabs` (default: the whole arena, cut into ranges of `width`
    coordinates) after EVERY step: packed signs, Delta bits and vote counts bit for bit,
    momentum and parameters within TOL_ULP.  The oracle is fed the gradient bytes the
    kernels read (copied out of the device arena).

    persist = True keeps the oracle's state of every range on the host from step to step
    (N * 4 bytes per covered coordinate).  persist = False holds one range at a time: after
    step t the oracle replays steps 0..t of the range from m = 0 and x_0, the earlier steps'
    gradients regenerated from the seed -- for arenas whose momentum does not fit host
    memory.  Returns the largest ulp distance seen.
    """
    import os
    dev = torch.device("cuda:0")
    N, D, W = w.n_workers, w.d_pad, w.d_pad // 32
    gdt = inputs.grad_torch_dtype(w)
    nthreads = os.cpu_count() or 1
    slabs = partition(D, width) if slabs is None else slabs
    widest = max(hi - lo for lo, hi in slabs)
    fused = path == "fused"
    if fused:
        assert len(modes) == 1
    sdt = torch.float32 if state == "f32" else torch.bfloat16
    g = torch.empty(N, D, dtype=gdt, device=dev)
    m = torch.zeros(N, D, dtype=sdt, device=dev)
    x0 = inputs.fill_x0(w, torch.empty(D, device=dev))
    xs = {md: x0.clone() for md in modes}
    if persist:
        x0 = None
    packed = torch.zeros(N, W, dtype=torch.int32, device=dev)
    dbits = {md: None if fused else torch.zeros(W, dtype=torch.int32, device=dev) for md in modes}
    count = {md: (torch.zeros(D, dtype=torch.uint8, device=dev) if not fused and N <= 255 else None)
             for md in modes}
    ctx = {md: make_ctx(dl, w, md) for md in modes}
    if state == "bf16":
        for c in ctx.values():
            c.set_momentum_dtype(dl.STATE_BF16)
    g_stage = _pinned((N * widest,), torch.int16 if gdt == torch.bfloat16 else torch.float32)
    if persist:
        oras = [SlabOracle(w, lo, hi, modes, state, counts=not fused) for lo, hi in slabs]
        for o in oras:
            o.reset(xs[modes[0]][o.lo:o.hi])
    else:
        one = {}                                    # one oracle state per distinct range length
        g_tmp = torch.empty(N, widest, dtype=gdt, device=dev)

    def stage_grads(src: torch.Tensor, n: int) -> np.ndarray:
        dst = g_stage[:N * n].view(N, n)
        dst.copy_(src.view(torch.int16) if gdt == torch.bfloat16 else src)
        a = dst.numpy()
        return a.view(np.uint16) if gdt == torch.bfloat16 else a

    worst = 0
    for t in range(steps):
        inputs.fill_grads(w, t, g)
        if fused:
            ctx[modes[0]].step_fused(g, m, xs[modes[0]], packed)
        else:
            ctx[modes[0]].worker_step(-1, g, m, packed)
            for md in modes:
                ctx[md].aggregate_apply(packed, xs[md], dbits[md], count[md])
        torch.cuda.synchronize()
        for k, (lo, hi) in enumerate(slabs):
            n = hi - lo
            if persist:
                o = oras[k]
                o.step(stage_grads(g[:, lo:hi], n), nthreads)
            else:
                if n not in one:
                    one[n] = SlabOracle(w, 0, n, modes, state, counts=not fused)
                o = one[n]
                o.lo, o.hi, o.segs = lo, hi, clip_segments(w.segments, lo, hi)
                o.reset(x0[lo:hi])
                for s in range(t):
                    o.step(stage_grads(inputs.fill_grads(w, s, g_tmp[:, :n], lo, hi), n), nthreads)
                o.step(stage_grads(g[:, lo:hi], n), nthreads)
            tag = f"{w.name} N={N} step {t} range [{lo},{hi}) {path} {state}"
            compare_dev(tag + " packed", packed[:, lo // 32:hi // 32], o.packed.to(dev), True)
            if state == "f32":
                worst = max(worst, compare_dev(tag + " m", m[:, lo:hi], o.m.to(dev), False))
            else:                                  # bf16 state: the tolerance is one bf16 ulp
                u = bf16_ulp_diff_dev(m[:, lo:hi].view(torch.int16), o.m.to(dev))
                assert u <= 1, f"{tag} m: {u} bf16 ulp"
                worst = max(worst, u)
            for md in modes:
                worst = max(worst, compare_dev(tag + f" x mode {md}", xs[md][lo:hi], o.x[md].to(dev), False))
                if not fused:
                    compare_dev(tag + f" delta_bits mode {md}", dbits[md][lo // 32:hi // 32], o.dbits[md].to(dev), True)
                    if count[md] is not None:
                        compare_dev(tag + f" count mode {md}", count[md][lo:hi], o.count[md].to(dev), True)
    for c in ctx.values():
        c.destroy()
    return worst


def cross_check_paths(dl, w: inputs.Workload, steps: int, mode: int) -> None:
    """Whole arenas, no CPU work: the product paths that promise identical bits -- the
    two-stage step; per-worker calls followed by dlion_aggregate + dlion_apply_delta; the
    one-launch step; the per-tensor mode (every tensor bound as its own pointer); and the
    scatter mode (sign words stored into four per-slice receive buffers, then voted on slice
    by slice and applied from the gathered message) -- are run side by side on the same
    gradients and must leave identical momentum, parameters and sign words everywhere,
    padding included.  (The oracle anchors the two-stage path; this extends that anchor to
    every coordinate of the other paths.)"""
    dev = torch.device("cuda:0")
    N, D, W = w.n_workers, w.d_pad, w.d_pad // 32
    gdt = inputs.grad_torch_dtype(w)
    ctx = make_ctx(dl, w, mode)
    g = torch.empty(N, D, dtype=gdt, device=dev)
    x0 = inputs.fill_x0(w, torch.empty(D, device=dev))
    P = 5
    ms = [torch.zeros(N, D, device=dev) for _ in range(P)]
    xs = [x0.clone() for _ in range(P)]
    ps = [torch.zeros(N, W, dtype=torch.int32, device=dev) for _ in range(4)]
    K = ctx.delta_planes()
    wire = torch.zeros(K * W, dtype=torch.int32, device=dev)
    # per-tensor mode: its own context; every tensor is a view into arenas 3
    tctx = make_ctx(dl, w, mode)
    tctx.bind_tensors(grads=[[g[i, o:o + k] for o, k in w.segments] for i in range(N)],
                      m=[[ms[3][i, o:o + k] for o, k in w.segments] for i in range(N)],
                      x=[xs[3][o:o + k] for o, k in w.segments])
    # scatter mode: four slices when the arena splits evenly, else two or one
    S = next(k for k in (4, 2, 1) if W % (4 * k) == 0)     # every slice a whole number of 128-coordinate groups
    SW = W // S
    sctx = make_ctx(dl, w, mode)
    server = dl.Dlion([(0, D // S)], D // S, N, w.beta1, w.beta2, w.lr, w.weight_decay, mode, gdtype_of(w))
    recv = [torch.zeros(N, SW, dtype=torch.int32, device=dev) for _ in range(S)]
    gathered = torch.zeros(S, K, SW, dtype=torch.int32, device=dev)
    for t in range(steps):
        inputs.fill_grads(w, t, g)
        ctx.worker_step(-1, g, ms[0], ps[0])
        ctx.aggregate_apply(ps[0], xs[0])
        for i in range(N):
            ctx.worker_step(i, g[i], ms[1][i], ps[1][i])
        ctx.aggregate(ps[1], wire)
        ctx.apply_delta(wire, xs[1])
        ctx.step_fused(g, ms[2], xs[2], ps[2])
        tctx.worker_step_tensors(-1, ps[3])
        tctx.aggregate_apply_tensors(ps[3])
        for i in range(N):
            sctx.bind_scatter(recv, SW, slot=i, rows=N)
            sctx.worker_step_scatter(i, g[i], ms[4][i])
        for q in range(S):
            server.aggregate(recv[q], gathered[q])
        ctx.apply_delta_sliced(gathered, SW, xs[4])
        torch.cuda.synchronize()
        names = ("two-stage", "per-worker + wire", "fused", "per-tensor", "scatter")
        for k in range(1, P):
            assert torch.equal(ms[k], ms[0]), f"{w.name} step {t}: momentum of the {names[k]} path differs"
            assert torch.equal(xs[k], xs[0]), f"{w.name} step {t}: parameters of the {names[k]} path differ"
        for k in range(1, 4):
            assert torch.equal(ps[k], ps[0]), f"{w.name} step {t}: sign words of the {names[k]} path differ"
        for q in range(S):
            assert torch.equal(recv[q], ps[0][:, q * SW:(q + 1) * SW]), f"{w.name} step {t}: receive buffer {q} differs"
    for c in (ctx, tctx, sctx, server):
        c.destroy()
