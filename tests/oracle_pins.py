"""Pins for the CPU oracle: each check ties it to something the paper or the
mathematics fixes, independent of the oracle's own code.

Every check takes ``lib`` (a loaded build of the oracle) so that the same checks
can be pointed at deliberately broken builds (see test_oracle_mutants.py).
All arithmetic here is numpy float64 / exact integers; nothing is copied from
the oracle.
"""
from __future__ import annotations

import os

import numpy as np

from oracle import dlion_oracle as orc

MAJ, AVG = orc.MAJORITY, orc.AVERAGE
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def unpack(packed: np.ndarray, d_pad: int) -> np.ndarray:
    """[N, W] uint32 -> [N, d_pad] of 0/1; bit b of word w is coordinate 32w+b."""
    n = packed.shape[0]
    return np.unpackbits(packed.view(np.uint8).reshape(n, -1), axis=1, bitorder="little")[:, :d_pad]


def f32(a):
    return np.asarray(a, dtype=np.float32)


def run_steps(lib, segs, d_pad, N, mode, grads, m0, x0, b1, b2, lr, wd, want_counts=False):
    """Run len(grads) full steps through the oracle; returns per-step records."""
    m = m0.copy()
    x = x0.copy()
    recs = []
    for g in grads:
        packed = np.zeros((N, d_pad // 32), np.uint32)
        orc.worker_step(segs, d_pad, N, np.ascontiguousarray(g), m, packed, b1, b2, lib=lib)
        dbits = np.zeros(d_pad // 32, np.uint32)
        cnt = np.zeros(d_pad, np.uint8) if (want_counts and N <= 255) else None
        orc.aggregate_apply(segs, d_pad, N, mode, packed, x, lr, wd, delta_bits=dbits, count=cnt,
                            lib=lib)
        recs.append(dict(packed=packed, m=m.copy(), x=x.copy(), delta_bits=dbits, count=cnt))
    return recs


def _flat(d):
    d_pad = (d + 127) // 128 * 128
    return [(0, d)], d_pad


def _rand_grads(rng, steps, N, d_pad, scale=1.0):
    return [f32(rng.standard_normal((N, d_pad)) * scale) for _ in range(steps)]


# ---------------------------------------------------------------- worked example
def check_hand_case(lib):
    hp, rows = {}, []
    for line in open(os.path.join(GOLDEN, "hand_case.txt")):
        line = line.split("#")[0].split()
        if not line:
            continue
        if len(line) == 2:
            hp[line[0]] = float(line[1])
        else:
            rows.append([float(v) for v in line])
    segs, d_pad = _flat(1)
    for mode, col in ((MAJ, 8), (AVG, 9)):
        m = np.zeros((2, d_pad), np.float32)
        x = np.zeros(d_pad, np.float32)
        x[0] = hp["x0"]
        for r in rows:
            g = np.zeros((2, d_pad), np.float32)
            g[0, 0], g[1, 0] = r[1], r[2]
            packed = np.zeros((2, d_pad // 32), np.uint32)
            cnt = np.zeros(d_pad, np.uint8)
            orc.worker_step(segs, d_pad, 2, g, m, packed, hp["beta1"], hp["beta2"], lib=lib)
            orc.aggregate_apply(segs, d_pad, 2, mode, packed, x, hp["eps"], hp["lambda"], count=cnt,
                                lib=lib)
            assert (int(packed[0, 0]) & 1, int(packed[1, 0]) & 1) == (int(r[3]), int(r[4]))
            assert int(cnt[0]) == int(r[5])
            assert (m[0, 0], m[1, 0]) == (np.float32(r[6]), np.float32(r[7]))
            assert x[0] == np.float32(r[col]), (mode, x[0], r[col])


# ---------------------------------------------------------------- sign conventions
def check_sign_of_zero_and_tie(lib):
    """Reading fixed for the 1-bit wire: sgn(+-0) = +1, and an even-N tie gives Delta = +1."""
    segs, d_pad = _flat(4)
    g = np.zeros((2, d_pad), np.float32)
    g[0, :4] = [0.0, -0.0, 1.0, -1.0]
    g[1, :4] = [0.0, -0.0, -1.0, -1.0]
    m = np.zeros((2, d_pad), np.float32)
    packed = np.zeros((2, d_pad // 32), np.uint32)
    orc.worker_step(segs, d_pad, 2, g, m, packed, 0.9, 0.99, lib=lib)
    assert packed[0, 0] == 0b0111 and packed[1, 0] == 0b0011
    x = np.zeros(d_pad, np.float32)
    dbits = np.zeros(d_pad // 32, np.uint32)
    orc.aggregate_apply(segs, d_pad, 2, MAJ, packed, x, 1.0, 0.0, delta_bits=dbits, lib=lib)
    # votes: (+,+) (+,+) (+,-)=tie (-,-)  ->  Delta = + + + -, x = -Delta
    assert dbits[0] == 0b0111
    assert list(x[:4]) == [-1.0, -1.0, -1.0, 1.0]


# ---------------------------------------------------------------- delta vs textbook sign
def check_delta_is_sign_of_blend(lib):
    """delta in {+-1} and equals the textbook sign of beta1*m + (1-beta1)*g (old m) wherever
    that value is clearly non-zero; the momentum follows its own closed form."""
    rng = np.random.default_rng(1)
    segs, d_pad = _flat(1000)
    N, T, b1, b2 = 3, 6, 0.9, 0.99
    grads = _rand_grads(rng, T, N, d_pad)
    recs = run_steps(lib, segs, d_pad, N, MAJ, grads, np.zeros((N, d_pad), np.float32),
                     np.zeros(d_pad, np.float32), b1, b2, 1e-3, 0.1)
    B1, B2 = float(np.float32(b1)), float(np.float32(b2))
    m64 = np.zeros((N, d_pad))
    for t, (g, r) in enumerate(zip(grads, recs)):
        c = B1 * m64 + (1.0 - B1) * g.astype(np.float64)
        bits = unpack(r["packed"], d_pad)[:, :1000]
        clear = np.abs(c[:, :1000]) > 1e-5
        assert clear.mean() > 0.99
        assert np.array_equal(bits[clear], (c[:, :1000] > 0)[clear].astype(np.uint8))
        m64 = B2 * m64 + (1.0 - B2) * g.astype(np.float64)
        # m_t = (1-beta2) sum_k beta2^(t-1-k) g_k   (momentum lemma in the appendix)
        closed = sum((1.0 - B2) * B2 ** (t - k) * grads[k].astype(np.float64) for k in range(t + 1))
        tol = (t + 2) * np.spacing(np.float32(np.abs(closed).max()))
        assert np.abs(r["m"][:, :1000] - closed[:, :1000]).max() <= tol
        assert np.abs(m64 - closed).max() < 1e-12


# ---------------------------------------------------------------- N = 1 is Lion (eq. 1)
def check_single_worker_is_lion(lib):
    rng = np.random.default_rng(2)
    segs, d_pad = _flat(777)
    T, b1, b2, lr, wd = 8, 0.9, 0.99, 1e-2, 0.5
    grads = _rand_grads(rng, T, 1, d_pad)
    x0 = f32(rng.standard_normal(d_pad))
    out = {}
    for mode in (MAJ, AVG):
        out[mode] = run_steps(lib, segs, d_pad, 1, mode, grads, np.zeros((1, d_pad), np.float32),
                              x0, b1, b2, lr, wd)
    B1, B2, LR, WD = (float(np.float32(v)) for v in (b1, b2, lr, wd))
    m = np.zeros(d_pad)
    x = x0.astype(np.float64)
    for t in range(T):
        g = grads[t][0].astype(np.float64)
        c = B1 * m + (1 - B1) * g
        delta = np.where(c >= 0, 1.0, -1.0)
        m = B2 * m + (1 - B2) * g
        x = x - LR * (delta + WD * x)
        for mode in (MAJ, AVG):
            got = out[mode][t]["x"][:777].astype(np.float64)
            assert np.abs(got - x[:777]).max() <= (t + 1) * 2 * np.spacing(np.float32(4.0))
        assert np.array_equal(out[MAJ][t]["x"], out[AVG][t]["x"])


# ---------------------------------------------------------------- identical workers
def check_identical_workers(lib):
    rng = np.random.default_rng(3)
    segs, d_pad = _flat(500)
    T, b1, b2, lr, wd = 5, 0.9, 0.99, 3e-3, 1.0
    g1 = _rand_grads(rng, T, 1, d_pad)
    x0 = f32(rng.standard_normal(d_pad) * 0.1)
    ref = run_steps(lib, segs, d_pad, 1, MAJ, g1, np.zeros((1, d_pad), np.float32), x0, b1, b2, lr, wd)
    for N in (2, 5, 8):
        gN = [np.repeat(g, N, axis=0) for g in g1]
        for mode in (MAJ, AVG):
            got = run_steps(lib, segs, d_pad, N, mode, gN, np.zeros((N, d_pad), np.float32), x0,
                            b1, b2, lr, wd)
            for t in range(T):
                assert np.array_equal(got[t]["x"], ref[t]["x"])
                for i in range(N):
                    assert np.array_equal(got[t]["m"][i], ref[t]["m"][0])
                    assert np.array_equal(got[t]["packed"][i], ref[t]["packed"][0])


# ---------------------------------------------------------------- beta = 0: signSGD + weight decay
def check_beta_zero_is_signsgd(lib):
    rng = np.random.default_rng(4)
    segs, d_pad = _flat(640)
    g = _rand_grads(rng, 3, 2, d_pad)
    x0 = f32(rng.standard_normal(d_pad))
    lr, wd = 0.01, 0.25
    recs = run_steps(lib, segs, d_pad, 2, AVG, g, f32(rng.standard_normal((2, d_pad))), x0, 0.0, 0.0,
                     lr, wd)
    x = x0.astype(np.float64)
    for t in range(3):
        assert np.array_equal(recs[t]["m"][:, :640], g[t][:, :640])        # m' = g exactly
        bits = unpack(recs[t]["packed"], d_pad)[:, :640]
        assert np.array_equal(bits, (g[t][:, :640] >= 0).astype(np.uint8))  # delta = sgn(g)
        delta = np.where(g[t] >= 0, 1.0, -1.0).mean(axis=0)
        x = x - float(np.float32(lr)) * (delta + float(np.float32(wd)) * x)
        assert np.abs(recs[t]["x"][:640] - x[:640]).max() <= (t + 1) * 2 * np.spacing(np.float32(4.0))


# ---------------------------------------------------------------- beta1 = beta2: Signum
def check_equal_betas_is_signum(lib):
    rng = np.random.default_rng(5)
    segs, d_pad = _flat(512)
    g = _rand_grads(rng, 4, 2, d_pad)
    recs = run_steps(lib, segs, d_pad, 2, MAJ, g, np.zeros((2, d_pad), np.float32),
                     np.zeros(d_pad, np.float32), 0.95, 0.95, 1e-3, 0.0)
    for r in recs:
        assert np.array_equal(unpack(r["packed"], d_pad), (r["m"] >= 0).astype(np.uint8))


# ---------------------------------------------------------------- votes by brute force
def check_counts_bruteforce(lib):
    rng = np.random.default_rng(6)
    segs = [(0, 70), (128, 1), (256, 33)]
    d_pad = 384
    valid = np.zeros(d_pad, bool)
    for o, n in segs:
        valid[o:o + n] = True
    for N in (1, 2, 3, 4, 7, 8, 33, 64, 255):
        bits = (rng.random((N, d_pad)) < rng.random(d_pad)[None, :]) & valid[None, :]
        packed = np.packbits(bits, axis=1, bitorder="little").view(np.uint32).reshape(N, -1).copy()
        P = bits.sum(axis=0)
        S = 2 * P.astype(np.int64) - N
        for mode in (MAJ, AVG):
            x0 = f32(rng.standard_normal(d_pad))
            x = x0.copy()
            dbits = np.zeros(d_pad // 32, np.uint32)
            cnt = np.full(d_pad, 7, np.uint8)
            lr, wd = 0.125, 0.5
            orc.aggregate_apply(segs, d_pad, N, mode, packed, x, lr, wd, delta_bits=dbits, count=cnt,
                                lib=lib)
            assert np.array_equal(cnt[valid], P[valid].astype(np.uint8))
            assert np.all(cnt[~valid] == 7) and np.array_equal(x[~valid], x0[~valid])
            got = unpack(dbits[None, :], d_pad)[0]
            assert np.array_equal(got[valid], (S >= 0)[valid].astype(np.uint8))
            assert not got[~valid].any()
            Delta = S / N if mode == AVG else np.where(S >= 0, 1.0, -1.0)
            want = x0.astype(np.float64) - lr * (Delta + wd * x0.astype(np.float64))
            assert np.abs(x[valid] - want[valid]).max() <= 2 * np.spacing(np.float32(4.0))
        # Delta read back exactly: x0 = 0, lr = 1, lambda = 0  ->  x' = -Delta
        for mode in (MAJ, AVG):
            x = np.zeros(d_pad, np.float32)
            orc.aggregate_apply(segs, d_pad, N, mode, packed, x, 1.0, 0.0, lib=lib)
            D = -x[valid].astype(np.float64)
            if mode == MAJ:
                assert np.array_equal(D, np.where(S[valid] >= 0, 1.0, -1.0))
            else:
                assert np.abs(D).max() <= 1.0
                k = np.rint(D * N)
                assert np.abs(D * N - k).max() < 1e-4 and np.array_equal(k, S[valid])
                assert np.all((k.astype(np.int64) - N) % 2 == 0)
                assert np.array_equal(x[valid], f32(-(S[valid] / N)))      # correctly rounded quotient


# ---------------------------------------------------------------- x closed form for constant Delta
def check_x_closed_form(lib):
    """x_{t+1} = (1-eps*lambda) x_t - eps*Delta unrolled (proof of the Phase-I theorem)."""
    segs, d_pad = _flat(256)
    rng = np.random.default_rng(7)
    x0 = f32(rng.standard_normal(d_pad) * 3)
    N, K = 3, 60
    for sgn in (1.0, -1.0):
        for lr, wd in ((0.01, 0.5), (0.003, 0.0), (0.1, 2.0)):
            for mode in (MAJ, AVG):
                grads = [np.full((N, d_pad), sgn, np.float32)] * K       # every vote is sgn
                recs = run_steps(lib, segs, d_pad, N, mode, grads, np.zeros((N, d_pad), np.float32),
                                 x0, 0.9, 0.99, lr, wd)
                LR, WD = float(np.float32(lr)), float(np.float32(wd))
                for k in (1, 2, 10, K):
                    w = (1 - LR * WD) ** k
                    if wd == 0.0:
                        want = x0.astype(np.float64) - k * LR * sgn
                    else:
                        want = w * x0.astype(np.float64) - (sgn / WD) * (1 - w)
                    err = np.abs(recs[k - 1]["x"][:256] - want[:256]).max()
                    assert err <= (k + 1) * np.spacing(np.float32(16.0)), (sgn, lr, wd, mode, k, err)


# ---------------------------------------------------------------- Phase-I contraction
def check_phase_one_contraction(lib):
    """dist(x_t, F) <= (1-eps*lambda)^(t-s) dist(x_s, F), F = {|lambda x| <= 1} (Phase-I theorem),
    coordinate-wise, for arbitrary votes; and F is invariant."""
    rng = np.random.default_rng(8)
    segs, d_pad = _flat(2048)
    N, T, lr, wd = 4, 40, 0.02, 4.0
    x0 = f32(rng.uniform(-3, 3, d_pad))
    grads = _rand_grads(rng, T, N, d_pad)
    for mode in (MAJ, AVG):
        recs = run_steps(lib, segs, d_pad, N, mode, grads, np.zeros((N, d_pad), np.float32), x0,
                         0.9, 0.99, lr, wd)
        dist = lambda v: np.maximum(np.abs(v.astype(np.float64)) - 1.0 / wd, 0.0)
        prev = dist(x0)
        rho = 1 - float(np.float32(lr)) * float(np.float32(wd))
        moved = 0
        for r in recs:
            cur = dist(r["x"])
            assert np.all(cur[:2048] <= rho * prev[:2048] + 1e-6)
            moved += int((cur[:2048] < prev[:2048]).sum())
            prev = cur
        assert moved > 1000
        assert dist(x0)[:2048].max() > 1.0 and prev[:2048].max() < dist(x0)[:2048].max() * rho ** T + 1e-5


# ---------------------------------------------------------------- padding
def check_padding_untouched(lib):
    rng = np.random.default_rng(9)
    segs = [(0, 5), (128, 200), (384, 31), (512, 32), (640, 1)]
    d_pad = 768
    valid = np.zeros(d_pad, bool)
    for o, n in segs:
        valid[o:o + n] = True
    N = 3
    for gdt in (np.float32, np.uint16):
        if gdt == np.float32:
            g = f32(rng.standard_normal((N, d_pad)))
        else:
            g = (f32(rng.standard_normal((N, d_pad))).view(np.uint32) >> 16).astype(np.uint16)
        m0 = f32(rng.standard_normal((N, d_pad)))
        m = m0.copy()
        packed = np.zeros((N, d_pad // 32), np.uint32)
        orc.worker_step(segs, d_pad, N, g, m, packed, 0.9, 0.99, lib=lib)
        assert np.array_equal(m[:, ~valid], m0[:, ~valid])
        assert np.all(m[:, valid] != m0[:, valid])
        assert not unpack(packed, d_pad)[:, ~valid].any()
        if gdt == np.uint16:      # bf16 widening is exact: same result as the widened fp32 gradient
            gw = (g.astype(np.uint32) << 16).view(np.float32)
            m2 = m0.copy()
            p2 = np.zeros_like(packed)
            orc.worker_step(segs, d_pad, N, gw, m2, p2, 0.9, 0.99, lib=lib)
            assert np.array_equal(m2, m) and np.array_equal(p2, packed)


# ---------------------------------------------------------------- Table 1
def check_wire_bits(lib):
    d = 1_000_000
    for n in (1, 2, 3, 4, 7, 8, 16, 32, 255, 256):
        assert orc.wire_bits(d, n, MAJ, 0, lib=lib) == n * d          # one bit per worker per parameter
        assert orc.wire_bits(d, n, AVG, 0, lib=lib) == n * d
        assert orc.wire_bits(d, n, MAJ, 1, lib=lib) == d
        bits = int(np.ceil(np.log2(n + 1)))                            # N+1 values {0..N}
        assert orc.wire_bits(d, n, AVG, 1, lib=lib) == bits * d
    # Table 1: full-precision methods move 32 d each way -> 32x more than Majority Vote
    assert 32 * d // orc.wire_bits(d, 1, MAJ, 1, lib=lib) == 32


# ---------------------------------------------------------------- server->worker wire format
def check_delta_wire_roundtrip(lib):
    """aggregate() writes Delta as broadcast (bits, or ceil(log2(N+1)) count bit planes: Section 3.2
    "Communication Cost"); apply_delta() decodes it.  Planes must decode to the brute-force counts,
    and the two halves together must equal the one-call server step."""
    rng = np.random.default_rng(10)
    segs = [(0, 70), (128, 1), (256, 33), (384, 64)]
    d_pad = 512
    W = d_pad // 32
    valid = np.zeros(d_pad, bool)
    for o, n in segs:
        valid[o:o + n] = True
    d = int(valid.sum())
    for N in (1, 2, 3, 4, 7, 8, 16, 33, 255, 256, 1000):
        bits = (rng.random((N, d_pad)) < rng.random(d_pad)[None, :]) & valid[None, :]
        packed = np.packbits(bits, axis=1, bitorder="little").view(np.uint32).reshape(N, -1).copy()
        P = bits.sum(axis=0).astype(np.int64)
        for mode in (MAJ, AVG):
            K = orc.delta_planes(N, mode, lib=lib)
            assert K == (1 if mode == MAJ else int(np.ceil(np.log2(N + 1))))
            assert K * d == orc.wire_bits(d, N, mode, 1, lib=lib)
            wire = np.full(K * W, 0xFFFFFFFF, np.uint32)          # garbage: must be overwritten or left alone
            orc.aggregate(segs, d_pad, N, mode, packed, wire, lib=lib)
            planes = unpack(wire.reshape(K, W), d_pad).astype(np.int64)
            if mode == MAJ:
                assert np.array_equal(planes[0][valid], (2 * P >= N)[valid].astype(np.int64))
            else:
                decoded = sum(planes[p] << p for p in range(K))
                assert np.array_equal(decoded[valid], P[valid])
            touched = np.zeros(W, bool)
            for o, n in segs:
                touched[o // 32:(o + n + 31) // 32] = True
            assert np.all(wire.reshape(K, W)[:, ~touched] == 0xFFFFFFFF)
            pad_in_touched = ~valid & np.repeat(touched, 32)
            assert not planes[:, pad_in_touched].any()
            x0 = f32(rng.standard_normal(d_pad))
            lr, wd = 0.125, 0.5
            xa, xb = x0.copy(), x0.copy()
            orc.apply_delta(segs, d_pad, N, mode, wire, xa, lr, wd, lib=lib)
            orc.aggregate_apply(segs, d_pad, N, mode, packed, xb, lr, wd, lib=lib)
            assert np.array_equal(xa, xb)
            S = 2 * P - N
            Delta = S / N if mode == AVG else np.where(S >= 0, 1.0, -1.0)
            want = x0.astype(np.float64) - lr * (Delta + wd * x0.astype(np.float64))
            assert np.abs(xa[valid] - want[valid]).max() <= 2 * np.spacing(np.float32(4.0))
            assert np.array_equal(xa[~valid], x0[~valid])


# ---------------------------------------------------------------- per-worker betas, bf16 momentum
def check_per_worker_betas(lib):
    """Algorithm 1 lets each worker set its own beta1, beta2: worker i of a mixed run must be
    the single-worker run with (beta1_i, beta2_i), bit for bit."""
    rng = np.random.default_rng(12)
    segs, d_pad = _flat(700)
    N, T = 4, 4
    b1s = [0.9, 0.5, 0.0, 0.95]
    b2s = [0.99, 0.75, 0.0, 0.95]
    grads = _rand_grads(rng, T, N, d_pad)
    m = np.zeros((N, d_pad), np.float32)
    solo = [np.zeros((1, d_pad), np.float32) for _ in range(N)]
    for g in grads:
        packed = np.zeros((N, d_pad // 32), np.uint32)
        orc.worker_step_ex(segs, d_pad, N, g, m, packed, b1s, b2s, lib=lib)
        for i in range(N):
            p1 = np.zeros((1, d_pad // 32), np.uint32)
            orc.worker_step(segs, d_pad, 1, np.ascontiguousarray(g[i:i + 1]), solo[i], p1, b1s[i], b2s[i],
                            lib=lib)
            assert np.array_equal(p1[0], packed[i]) and np.array_equal(solo[i][0], m[i])
    assert not np.array_equal(m[0], m[1])


def check_bf16_momentum_store(lib):
    """bf16 momentum: arithmetic in binary32, the stored value is the binary32 result rounded to
    nearest-even bf16 (checked against torch's float32 -> bfloat16 conversion, an independent
    routine), and the signs are those of the widened state."""
    import torch
    rng = np.random.default_rng(13)
    segs, d_pad = _flat(4096)
    N = 2

    def to_bits(a32):
        return torch.from_numpy(a32.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)

    def widen(b16):
        return (b16.astype(np.uint32) << 16).view(np.float32)

    m16 = to_bits(f32(rng.standard_normal((N, d_pad))))
    g = f32(rng.standard_normal((N, d_pad)))
    # exact ties: beta2 = 0 makes m' = g; these g sit halfway between two bf16 values
    g[0, :4] = [1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8), 3.4e38]
    for b1, b2 in ((0.9, 0.99), (0.5, 0.0)):
        m32 = widen(m16)
        p32 = np.zeros((N, d_pad // 32), np.uint32)
        orc.worker_step(segs, d_pad, N, g, m32, p32, b1, b2, lib=lib)            # fp32-state run from the same start
        mb = m16.copy()
        pb = np.zeros((N, d_pad // 32), np.uint32)
        orc.worker_step_ex(segs, d_pad, N, g, mb, pb, [b1] * N, [b2] * N, lib=lib)
        assert np.array_equal(pb, p32)                                           # same old m, same signs
        assert np.array_equal(mb[:, :4096], to_bits(m32)[:, :4096])              # RNE of the fp32 result
    assert widen(mb)[0, 0] == 1.0 and widen(mb)[0, 1] == 1.0 + 2.0 ** -6 and widen(mb)[0, 2] == -1.0
    assert np.isinf(widen(mb)[0, 3])                                              # rounds up past the largest bf16
    nan_state = np.full((1, 128), 0x7FC1, np.uint16)
    orc.worker_step_ex([(0, 128)], 128, 1, np.zeros((1, 128), np.float32), nan_state,
                       np.zeros((1, 4), np.uint32), [0.9], [0.99], lib=lib)
    assert np.isnan(widen(nan_state)).all()


# ---------------------------------------------------------------- Global Lion (comparison scheme)
def _hand_rows(name):
    hp, rows = {}, []
    for line in open(os.path.join(GOLDEN, name)):
        line = line.split("#")[0].split()
        if not line:
            continue
        if len(line) == 2:
            hp[line[0]] = float(line[1])
        else:
            rows.append([float(v) for v in line])
    return hp, rows


def check_global_lion_hand_case(lib):
    """The hand-derived example where the sign of the mean and the majority of the signs differ."""
    hp, rows = _hand_rows("global_lion_hand_case.txt")
    segs, d_pad = _flat(1)
    m = np.zeros((3, d_pad), np.float32)
    x = np.zeros(d_pad, np.float32)
    x[0] = hp["x0"]
    for r in rows:
        g = np.zeros((3, d_pad), np.float32)
        g[:, 0] = r[1:4]
        # the same blends through Distributed Lion's vote (from the same momentum), for the contrast
        m_d, x_d = m.copy(), x.copy()
        packed = np.zeros((3, d_pad // 32), np.uint32)
        dbits_d = np.zeros(d_pad // 32, np.uint32)
        orc.worker_step(segs, d_pad, 3, g, m_d, packed, hp["beta1"], hp["beta2"], lib=lib)
        orc.aggregate_apply(segs, d_pad, 3, MAJ, packed, x_d, hp["eps"], hp["lambda"], delta_bits=dbits_d, lib=lib)
        dbits = np.zeros(d_pad // 32, np.uint32)
        orc.global_step(segs, d_pad, 3, g, m, x, hp["beta1"], hp["beta2"], hp["eps"], hp["lambda"],
                        delta_bits=dbits, lib=lib)
        assert (1 if dbits[0] & 1 else -1) == int(r[4])
        assert x[0] == np.float32(r[5])
        assert tuple(m[:, 0]) == tuple(np.float32(v) for v in r[6:9])
        assert np.array_equal(m, m_d)                              # same momentum rule
        assert (1 if dbits_d[0] & 1 else -1) == int(r[9]) == -int(r[4])   # the two schemes disagree here
        assert dbits[0] >> 1 == 0 and not x[1:].any()              # padding untouched


def check_global_lion_definition(lib):
    """Sign of the float64 mean of the float64 blends wherever that mean is clearly non-zero;
    x from the float64 update within an ulp per operation; momentum equal to the worker step's;
    N = 1 is Lion (Eq. 1) = Distributed Lion under either rule; N identical workers = one worker."""
    rng = np.random.default_rng(11)
    b1, b2, lr, wd = 0.9, 0.99, 1e-2, 0.3
    for N, d in ((1, 700), (2, 515), (3, 700), (8, 333), (33, 129)):
        segs, d_pad = _flat(d)
        m = f32(rng.standard_normal((N, d_pad)) * 0.1)
        x = f32(rng.standard_normal(d_pad))
        for t in range(3):
            g = f32(rng.standard_normal((N, d_pad)))
            m_old, x_old = m.copy(), x.copy()
            dbits = np.zeros(d_pad // 32, np.uint32)
            orc.global_step(segs, d_pad, N, g, m, x, b1, b2, lr, wd, delta_bits=dbits, lib=lib)
            mt = np.float64(np.float32(b1)) * m_old.astype(np.float64) + (1.0 - np.float64(np.float32(b1))) * g
            mean = mt.mean(axis=0)
            clear = np.abs(mean[:d]) > 1e-5
            assert clear.mean() > 0.9
            got = unpack(dbits[None, :], d_pad)[0, :d].astype(bool)
            assert np.array_equal(got[clear], (mean[:d] > 0)[clear])
            delta = np.where(got, 1.0, -1.0)
            x64 = x_old[:d].astype(np.float64) - np.float64(np.float32(lr)) * (
                delta + np.float64(np.float32(wd)) * x_old[:d].astype(np.float64))
            assert np.abs(x[:d] - x64).max() <= 4 * np.spacing(np.float32(np.abs(x64).max() + 1))
            m_w = m_old.copy()
            orc.worker_step(segs, d_pad, N, g, m_w, np.zeros((N, d_pad // 32), np.uint32), b1, b2, lib=lib)
            assert np.array_equal(m, m_w)
            assert np.array_equal(x[d:], x_old[d:]) and np.array_equal(m[:, d:], m_old[:, d:])
            if N == 1:                                             # Lion, Eq. (1)
                for mode in (MAJ, AVG):
                    m1, x1 = m_old.copy(), x_old.copy()
                    pk = np.zeros((1, d_pad // 32), np.uint32)
                    orc.worker_step(segs, d_pad, 1, g, m1, pk, b1, b2, lib=lib)
                    orc.aggregate_apply(segs, d_pad, 1, mode, pk, x1, lr, wd, lib=lib)
                    assert np.array_equal(x, x1) and np.array_equal(dbits, pk[0])
    # N identical workers reproduce one worker (the sum of N equal values has that value's sign)
    segs, d_pad = _flat(300)
    for N in (2, 5, 16):
        g1 = f32(rng.standard_normal((1, d_pad)))
        g1[0, :7] = 0.0                                            # exact zeros: sign(0) = +1 either way
        m1 = f32(rng.standard_normal((1, d_pad)) * 0.1)
        m1[0, :7] = 0.0
        x1 = f32(rng.standard_normal(d_pad))
        mN, xN = np.repeat(m1, N, axis=0), x1.copy()
        orc.global_step(segs, d_pad, 1, g1, m1, x1, b1, b2, lr, wd, lib=lib)
        orc.global_step(segs, d_pad, N, np.repeat(g1, N, axis=0), mN, xN, b1, b2, lr, wd, lib=lib)
        assert np.array_equal(xN, x1) and all(np.array_equal(mN[i], m1[0]) for i in range(N))
    # bf16 gradients are widened exactly
    gb = (f32(rng.standard_normal((3, d_pad))).view(np.uint32) >> 16).astype(np.uint16)
    gf = (gb.astype(np.uint32) << 16).view(np.float32)
    ma, xa = np.zeros((3, d_pad), np.float32), np.ones(d_pad, np.float32)
    mb, xb = ma.copy(), xa.copy()
    orc.global_step(segs, d_pad, 3, gb, ma, xa, b1, b2, lr, wd, lib=lib)
    orc.global_step(segs, d_pad, 3, gf, mb, xb, b1, b2, lr, wd, lib=lib)
    assert np.array_equal(xa, xb) and np.array_equal(ma, mb)


def check_vote_counts16(lib):
    """16-bit vote counts against a brute-force column sum of the unpacked bits, for worker
    counts on both sides of one byte; they also agree with the byte counts where those exist
    and with the count planes of the Averaging message."""
    rng = np.random.default_rng(16)
    segs = [(0, 70), (128, 1), (256, 33)]
    d_pad = 384
    valid = np.zeros(d_pad, bool)
    for o, n in segs:
        valid[o:o + n] = True
    for N in (1, 3, 255, 256, 257, 1000, 4099):
        bits = (rng.random((N, d_pad)) < rng.random(d_pad)[None, :]) & valid[None, :]
        bits[:, 5] = True                      # every worker votes +1: the count is N itself
        bits[:, 6] = False
        packed = np.packbits(bits, axis=1, bitorder="little").view(np.uint32).reshape(N, -1).copy()
        cnt = np.full(d_pad, 0xABCD, np.uint16)
        orc.vote_counts16(segs, d_pad, N, packed, cnt, lib=lib)
        P = bits.sum(axis=0)
        assert np.array_equal(cnt[valid], P[valid].astype(np.uint16)) and cnt[5] == N and cnt[6] == 0
        assert np.all(cnt[~valid] == 0xABCD)
        K = orc.delta_planes(N, AVG, lib=lib)
        wire = np.zeros(K * d_pad // 32, np.uint32)
        orc.aggregate(segs, d_pad, N, AVG, packed, wire, lib=lib)
        planes = unpack(wire.reshape(K, -1), d_pad).astype(np.int64)
        assert np.array_equal((planes << np.arange(K)[:, None]).sum(axis=0)[valid], cnt[valid].astype(np.int64))
        if N <= 255:
            c8 = np.zeros(d_pad, np.uint8)
            orc.aggregate_apply(segs, d_pad, N, MAJ, packed, np.zeros(d_pad, np.float32), 0.1, 0.0, count=c8, lib=lib)
            assert np.array_equal(c8[valid], cnt[valid].astype(np.uint8))


def check_ternary_majority(lib):
    """The optional three-valued reading of the tie (mode MAJORITY_TERNARY): Delta is the
    textbook sign of S, zero included; with an odd N it is the binary Majority Vote; with N = 2
    it is Averaging; its two-plane message carries Delta + 1."""
    TER = orc.MAJORITY_TERNARY
    rng = np.random.default_rng(23)
    segs = [(0, 70), (128, 1), (256, 33)]
    d_pad = 384
    valid = np.zeros(d_pad, bool)
    for o, n in segs:
        valid[o:o + n] = True
    # hand case: N = 2, one vote each way (a tie), eps = 1/4, lambda = 1/2, x_0 = 2: pure decay, twice
    one = np.array([[1], [0]], np.uint32)
    x = np.zeros(32, np.float32)
    x[0] = 2.0
    orc.aggregate_apply([(0, 1)], 32, 2, TER, np.ascontiguousarray(one), x, 0.25, 0.5, lib=lib)
    assert x[0] == 1.75
    orc.aggregate_apply([(0, 1)], 32, 2, TER, np.ascontiguousarray(one), x, 0.25, 0.5, lib=lib)
    assert x[0] == 1.53125 and not x[1:].any()
    for N in (1, 2, 3, 4, 7, 8, 33, 64, 255, 256):
        bits = (rng.random((N, d_pad)) < rng.random(d_pad)[None, :]) & valid[None, :]
        if N % 2 == 0:                                   # exact ties on a few coordinates
            for j in (3, 40, 128, 260):
                bits[:, j] = np.arange(N) < N // 2
        packed = np.packbits(bits, axis=1, bitorder="little").view(np.uint32).reshape(N, -1).copy()
        S = 2 * bits.sum(axis=0).astype(np.int64) - N
        # Delta read back exactly: x_0 = 0, lr = 1, lambda = 0  ->  x' = -Delta
        x = np.zeros(d_pad, np.float32)
        dbits = np.zeros(d_pad // 32, np.uint32)
        orc.aggregate_apply(segs, d_pad, N, TER, packed, x, 1.0, 0.0, delta_bits=dbits, lib=lib)
        assert np.array_equal(-x[valid].astype(np.float64), np.sign(S[valid]).astype(np.float64))
        assert not x[~valid].any()
        assert np.array_equal(unpack(dbits[None, :], d_pad)[0][valid], (S >= 0)[valid].astype(np.uint8))
        if N % 2 == 0:
            assert (x[[3, 40, 128, 260]] == 0).all()
        x0 = f32(rng.standard_normal(d_pad))
        xt, xb, xa = x0.copy(), x0.copy(), x0.copy()
        orc.aggregate_apply(segs, d_pad, N, TER, packed, xt, 0.125, 0.5, lib=lib)
        orc.aggregate_apply(segs, d_pad, N, MAJ, packed, xb, 0.125, 0.5, lib=lib)
        orc.aggregate_apply(segs, d_pad, N, AVG, packed, xa, 0.125, 0.5, lib=lib)
        if N % 2 == 1:
            assert np.array_equal(xt, xb)                # no ties: the binary rule
        else:
            tie = (S == 0) & valid
            assert np.array_equal(xt[~tie], xb[~tie]) and not np.array_equal(xt[tie], xb[tie])
        if N == 2:
            assert np.array_equal(xt, xa)                # S/2 is -1, 0 or +1
        # the message: two planes holding Delta + 1; vote then apply equals the one-call step
        assert orc.delta_planes(N, TER, lib=lib) == 2 and orc.wire_bits(1000, N, TER, 1, lib=lib) == 2000
        wire = np.zeros(2 * d_pad // 32, np.uint32)
        wire[3] = 0xDEADBEEF                             # word 3 = coordinates 96..127: padding, must stay untouched
        orc.aggregate(segs, d_pad, N, TER, packed, wire, lib=lib)
        assert wire[3] == 0xDEADBEEF
        wire[3] = 0
        planes = unpack(wire.reshape(2, -1), d_pad).astype(np.int64)
        code = planes[0] + 2 * planes[1]
        assert np.array_equal(code[valid], np.sign(S[valid]) + 1) and not code[~valid].any()
        xw = x0.copy()
        orc.apply_delta(segs, d_pad, N, TER, wire, xw, 0.125, 0.5, lib=lib)
        assert np.array_equal(xw, xt)
    # a tie at every step: x_k = (1 - eps*lambda)^k x_0 (the closed form with Delta = 0)
    x = np.zeros(32, np.float32)
    x[0] = 3.0
    for _ in range(10):
        orc.aggregate_apply([(0, 1)], 32, 2, TER, np.ascontiguousarray(one), x, 0.01, 0.3, lib=lib)
    want = 3.0 * (1 - 0.01 * 0.3) ** 10
    assert abs(float(x[0]) - want) <= 10 * np.spacing(np.float32(3.0))


ALL_CHECKS = [check_hand_case, check_sign_of_zero_and_tie, check_delta_is_sign_of_blend,
              check_single_worker_is_lion, check_identical_workers, check_beta_zero_is_signsgd,
              check_equal_betas_is_signum, check_counts_bruteforce, check_x_closed_form,
              check_phase_one_contraction, check_padding_untouched, check_wire_bits,
              check_delta_wire_roundtrip, check_per_worker_betas, check_bf16_momentum_store,
              check_global_lion_hand_case, check_global_lion_definition, check_vote_counts16,
              check_ternary_majority]
