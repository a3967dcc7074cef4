"""CUDA library vs CPU oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

from paper_2404_00438_b200 import inputs
from tests import gpu_parity as gp

pytestmark = pytest.mark.gpu

MAJ, AVG = inputs.MAJORITY, inputs.AVERAGE
RAGGED = [5, 200, 31, 32, 1, 4096, 4097, 8191, 12289, 0, 33, 128, 127]


@pytest.fixture(scope="module")
def dl():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2404_00438_b200 import build
    build.build()
    from paper_2404_00438_b200 import dlion
    return dlion


# ---------------------------------------------------------------- config 1, ten steps
@pytest.mark.parametrize("path", ["two_stage", "per_worker", "fused"])
def test_c1_ten_steps(dl, path):
    w = inputs.workload("c1")
    worst = gp.run_small(dl, w, 10, path)
    assert worst == 0, "pinned evaluation order should reproduce the oracle's fp32 state bit for bit"


# ---------------------------------------------------------------- ragged tables, every N class
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5, 7, 8, 15, 16, 33, 64, 127, 128, 255])
@pytest.mark.parametrize("gd", ["f32", "bf16"])
def test_ragged_segments(dl, n, gd):
    scale = 1.0 if gd == "f32" else 1e-3
    w = inputs.custom(RAGGED, n, MAJ, gd, scale=scale, lr=1e-3, weight_decay=0.5, zero_frac=0.02)
    for path in ("two_stage", "fused"):
        gp.run_small(dl, w, 3, path)
    if n <= 8:
        gp.run_small(dl, w, 2, "per_worker")


def test_tiny_and_empty(dl):
    for numels in ([1], [31], [32], [33], [1000], [0, 0, 7], [0]):
        for n in (1, 2, 5):
            w = inputs.custom(numels, n, MAJ, "f32")
            for path in ("two_stage", "fused", "per_worker"):
                gp.run_small(dl, w, 2, path)


def test_multi_tile_with_ragged_tail(dl):
    w = inputs.custom([3 * 4096 * 160 + 1234, 777], 4, AVG, "bf16", scale=1e-3, lr=1e-3, weight_decay=1.0)
    for path in ("two_stage", "fused"):
        assert gp.run_small(dl, w, 3, path) == 0


# ---------------------------------------------------------------- degenerate values
def test_special_values(dl):
    """+-0, exact cancellation beta1*m = -(1-beta1)*g, NaN, +-Inf, denormals, |x| > 1/lambda."""
    n, d = 4, 4096 + 640
    w = inputs.custom([d], n, MAJ, "f32", beta1=0.5, beta2=0.75, lr=0.25, weight_decay=0.5)
    rng = np.random.default_rng(11)
    specials = np.array([0.0, -0.0, 1.0, -1.0, np.nan, np.inf, -np.inf, 1e-42, -1e-42, 3e38, -3e38,
                         1.1754944e-38], np.float32)
    m0 = rng.choice(specials, size=(n, w.d_pad)).astype(np.float32)
    g0 = rng.choice(specials, size=(n, w.d_pad)).astype(np.float32)
    g0[:, :512] = -m0[:, :512]                       # beta1 = 1/2: c = 0.5 m - 0.5 m = +-0 -> +1
    x0 = (rng.standard_normal(w.d_pad) * 5).astype(np.float32)
    g1 = rng.standard_normal((n, w.d_pad)).astype(np.float32)
    for a in (m0, g0, g1):
        a[:, d:] = 0
    x0[d:] = 0
    grads = [torch.from_numpy(g0), torch.from_numpy(g1)]
    for path in ("two_stage", "fused"):
        gp.run_small(dl, w, 2, path, m0=torch.from_numpy(m0), x0=torch.from_numpy(x0), grads=grads)


def test_even_n_ties_are_positive(dl):
    n, d = 6, 4096
    w = inputs.custom([d], n, MAJ, "f32", beta1=0.0, beta2=0.0, lr=1.0, weight_decay=0.0)
    g = torch.ones(n, w.d_pad)
    g[: n // 2] = -1.0                               # exact tie on every coordinate
    dev = torch.device("cuda:0")
    ctx = gp.make_ctx(dl, w)
    m = torch.zeros(n, w.d_pad, device=dev)
    x = torch.zeros(w.d_pad, device=dev)
    packed = torch.zeros(n, w.d_pad // 32, dtype=torch.int32, device=dev)
    dbits = torch.zeros(w.d_pad // 32, dtype=torch.int32, device=dev)
    ctx.worker_step(-1, g.to(dev), m, packed)
    ctx.aggregate_apply(packed, x, dbits)
    torch.cuda.synchronize()
    assert bool((x == -1.0).all()) and bool((dbits == -1).all())
    gp.run_small(dl, w, 1, "two_stage", grads=[g])
    ctx.destroy()


def test_set_lr_and_launch_count(dl):
    w = inputs.custom([5000], 3, AVG, "f32", lr=0.5, weight_decay=0.0)
    dev = torch.device("cuda:0")
    ctx = gp.make_ctx(dl, w)
    g = inputs.fill_grads(w, 0, torch.empty(3, w.d_pad)).to(dev)
    m = torch.zeros(3, w.d_pad, device=dev)
    packed = torch.zeros(3, w.d_pad // 32, dtype=torch.int32, device=dev)
    x1 = torch.zeros(w.d_pad, device=dev)
    x2 = torch.zeros(w.d_pad, device=dev)
    assert ctx.launch_count() == 0
    ctx.worker_step(-1, g, m, packed)
    ctx.aggregate_apply(packed, x1)
    ctx.set_lr(0.25)
    ctx.aggregate_apply(packed, x2)
    torch.cuda.synchronize()
    assert ctx.launch_count() == 3
    assert torch.equal(x1, 2 * x2)                   # lambda = 0: x' = -lr * Delta
    d = w.d
    assert ctx.wire_bytes(0) == (3 * d + 7) // 8 and ctx.wire_bytes(1) == (2 * d + 7) // 8
    assert ctx.wire_bytes(2) == 4 * d and ctx.wire_bytes(3) == 0
    ctx.destroy()


def test_argument_errors_with_a_context(dl):
    w = inputs.custom([5000], 2, MAJ, "f32")
    dev = torch.device("cuda:0")
    ctx = gp.make_ctx(dl, w)
    g = torch.zeros(2, w.d_pad, device=dev)
    m = torch.zeros(2, w.d_pad, device=dev)
    x = torch.zeros(w.d_pad + 4, device=dev)
    packed = torch.zeros(2, w.d_pad // 32, dtype=torch.int32, device=dev)
    for bad_worker in (-2, 2):
        with pytest.raises(dl.DlionError) as e:
            ctx.worker_step(bad_worker, g, m, packed)
        assert e.value.status == dl.EINVAL
    with pytest.raises(dl.DlionError) as e:
        ctx.aggregate_apply(packed, x[1:])           # 4-byte aligned only
    assert e.value.status == dl.EALIGN
    g_big = torch.zeros(2 * w.d_pad + 4, device=dev)
    with pytest.raises(dl.DlionError) as e:
        ctx.worker_step(-1, g_big[1:], m, packed)     # long enough and contiguous, but 4-byte aligned only
    assert e.value.status == dl.EALIGN
    with pytest.raises(ValueError):                  # too short: refused by the binding, nothing launched
        ctx.worker_step(-1, g.view(-1)[1:], m, packed)
    with pytest.raises(ValueError):                  # one worker's slice passed for all workers
        ctx.worker_step(-1, g[0], m, packed)
    with pytest.raises(ValueError):                  # strided view
        ctx.aggregate_apply(packed[:, 8:40], x)
    raw = dl.lib()
    assert raw.dlion_worker_step(ctx._ctx, -1, None, m.data_ptr(), packed.data_ptr(), None) == dl.EINVAL
    assert raw.dlion_step_host(ctx._ctx, g.data_ptr(), m.data_ptr(), x.data_ptr(), packed.data_ptr(),
                               g.data_ptr(), None, g.data_ptr(), None) == dl.EINVAL
    ctx.worker_step(-1, g, m, packed)                # the context is still usable
    torch.cuda.synchronize()
    ctx.destroy()


# ---------------------------------------------------------------- host-gradient step
@pytest.mark.parametrize("mode", [MAJ, AVG])
@pytest.mark.parametrize("n", [5, 300])
def test_step_host_matches_oracle(dl, mode, n):
    from oracle import dlion_oracle as orc
    w = inputs.custom([70000, 333] if n < 256 else [9000, 333], n, mode, "bf16", scale=1e-3, lr=1e-3, weight_decay=1.0)
    dev = torch.device("cuda:0")
    N, D, W = w.n_workers, w.d_pad, w.d_pad // 32
    ctx = gp.make_ctx(dl, w)
    x0 = inputs.fill_x0(w, torch.empty(D))
    ora = gp.OracleState(w, 0, D, np.zeros((N, D), np.float32), x0.numpy(), [mode])
    m = torch.zeros(N, D, device=dev)
    x = x0.to(dev)
    packed = torch.zeros(N, W, dtype=torch.int32, device=dev)
    staging = torch.empty(2, D, dtype=torch.bfloat16, device=dev)
    K = ctx.delta_planes()
    wire = torch.zeros(K * W, dtype=torch.int32, device=dev)
    host_wire = torch.zeros(K * W, dtype=torch.int32).pin_memory()
    host_g = torch.empty(N, D, dtype=torch.bfloat16).pin_memory()
    for t in range(4):
        inputs.fill_grads(w, t, host_g)
        ora.step(inputs.as_numpy_grads(host_g))
        ctx.step_host(host_g, m, x, packed, staging, wire, host_wire)
        torch.cuda.synchronize()
        gp.compare("packed", packed.cpu().numpy().view(np.uint32), ora.packed, True)
        gp.compare("m", m.cpu().numpy(), ora.m, False)
        gp.compare("x", x.cpu().numpy(), ora.x[mode], False)
        want = np.zeros(K * W, np.uint32)               # the broadcast message, from the oracle's own votes
        orc.aggregate(w.segments, D, N, mode, ora.packed, want)
        gp.compare("wire", host_wire.numpy().view(np.uint32), want, True)
    ctx.destroy()


# ---------------------------------------------------------------- server-only aggregate + worker-side apply
@pytest.mark.parametrize("n", [1, 2, 3, 4, 7, 8, 16, 33, 64, 255, 256, 300, 1000, 4097])
@pytest.mark.parametrize("mode", [MAJ, AVG])
def test_aggregate_then_apply_delta(dl, n, mode):
    from oracle import dlion_oracle as orc
    w = inputs.custom(RAGGED + [3 * 4096 + 5], n, mode, "f32", lr=1e-2, weight_decay=0.5)
    dev = torch.device("cuda:0")
    D, W = w.d_pad, w.d_pad // 32
    rng = np.random.default_rng(n * 2 + mode)
    valid = np.zeros(D, bool)
    for off, cnt in w.segments:
        valid[off:off + cnt] = True
    bits = (rng.random((n, D)) < rng.random(D)[None, :]) & valid[None, :]
    packed_np = np.packbits(bits, axis=1, bitorder="little").view(np.uint32).reshape(n, -1).copy()
    x0 = inputs.fill_x0(w, torch.empty(D))
    ctx = gp.make_ctx(dl, w)
    K = ctx.delta_planes()
    assert K == orc.delta_planes(n, mode)
    # oracle
    wire_ref = np.zeros(K * W, np.uint32)
    orc.aggregate(w.segments, D, n, mode, packed_np, wire_ref)
    x_ref = x0.numpy().copy()
    orc.apply_delta(w.segments, D, n, mode, wire_ref, x_ref, w.lr, w.weight_decay)
    # CUDA library
    packed = torch.from_numpy(packed_np.view(np.int32)).to(dev)
    wire = torch.zeros(K * W, dtype=torch.int32, device=dev)
    x = x0.to(dev)
    x_one = x0.to(dev)
    ctx.aggregate(packed, wire)
    ctx.apply_delta(wire, x)
    ctx.aggregate_apply(packed, x_one)
    torch.cuda.synchronize()
    gp.compare("delta wire", wire.cpu().numpy().view(np.uint32), wire_ref, True)
    gp.compare("x after apply_delta", x.cpu().numpy(), x_ref, True)
    assert torch.equal(x, x_one)
    ctx.destroy()


# ---------------------------------------------------------------- per-worker betas, bf16 momentum
def _bf16_ulp_diff(a: np.ndarray, b: np.ndarray) -> int:
    """Distance in bf16 units in the last place between two arrays of bf16 bit patterns."""
    def key(u):
        i = u.astype(np.int64)
        return np.where(i & 0x8000, -(i & 0x7FFF), i)
    return int(np.abs(key(a) - key(b)).max()) if a.size else 0


@pytest.mark.parametrize("state", ["f32", "bf16"])
@pytest.mark.parametrize("path", ["two_stage", "per_worker", "fused"])
@pytest.mark.parametrize("gd", ["f32", "bf16"])
def test_per_worker_betas_and_momentum_dtype(dl, state, path, gd):
    """Each worker with its own (beta1, beta2) -- including a Signum and a signSGD worker --
    and the momentum kept in fp32 or bf16.  Tolerance: signs, counts and Delta exact; fp32
    state 2 ulp; bf16 state 1 bf16 ulp (observed: identical bits)."""
    from oracle import dlion_oracle as orc
    n = 5
    b1s = [0.9, 0.5, 0.95, 0.0, 0.8]
    b2s = [0.99, 0.75, 0.95, 0.0, 0.999]
    w = inputs.custom(RAGGED + [2 * 4096 + 77], n, AVG, gd, scale=1.0 if gd == "f32" else 1e-3,
                      lr=1e-3, weight_decay=0.5, zero_frac=0.02)
    dev = torch.device("cuda:0")
    D, W = w.d_pad, w.d_pad // 32
    ctx = gp.make_ctx(dl, w)
    for i in range(n):
        ctx.set_worker_betas(i, b1s[i], b2s[i])
    if state == "bf16":
        ctx.set_momentum_dtype(dl.STATE_BF16)
    mt = torch.bfloat16 if state == "bf16" else torch.float32
    x0 = inputs.fill_x0(w, torch.empty(D))
    m_ref = np.zeros((n, D), np.uint16 if state == "bf16" else np.float32)
    x_ref = x0.numpy().copy()
    m = torch.zeros(n, D, dtype=mt, device=dev)
    x = x0.to(dev)
    packed = torch.zeros(n, W, dtype=torch.int32, device=dev)
    for t in range(4):
        g_cpu = inputs.fill_grads(w, t, torch.empty(n, D, dtype=inputs.grad_torch_dtype(w)))
        p_ref = np.zeros((n, W), np.uint32)
        orc.worker_step_ex(w.segments, D, n, inputs.as_numpy_grads(g_cpu), m_ref, p_ref, b1s, b2s)
        orc.aggregate_apply(w.segments, D, n, AVG, p_ref, x_ref, w.lr, w.weight_decay)
        g = g_cpu.to(dev)
        packed.zero_()
        if path == "fused":
            ctx.step_fused(g, m, x, packed)
        else:
            if path == "per_worker":
                for i in range(n):
                    ctx.worker_step(i, g[i], m[i], packed[i])
            else:
                ctx.worker_step(-1, g, m, packed)
            ctx.aggregate_apply(packed, x)
        torch.cuda.synchronize()
        gp.compare(f"step {t} packed", packed.cpu().numpy().view(np.uint32), p_ref, True)
        if state == "bf16":
            got = m.cpu().view(torch.int16).numpy().view(np.uint16)
            assert _bf16_ulp_diff(got, m_ref) <= 1
            assert np.array_equal(got, m_ref)
        else:
            assert gp.compare(f"step {t} m", m.cpu().numpy(), m_ref, False) == 0
        assert gp.compare(f"step {t} x", x.cpu().numpy(), x_ref, False) == 0
    ctx.destroy()


def test_new_setters_reject_bad_arguments(dl):
    w = inputs.custom([5000], 2, MAJ, "f32")
    ctx = gp.make_ctx(dl, w)
    for args in ((-1, 0.9, 0.99), (2, 0.9, 0.99), (0, 1.5, 0.99), (0, 0.9, float("nan"))):
        with pytest.raises(dl.DlionError) as e:
            ctx.set_worker_betas(*args)
        assert e.value.status == dl.EINVAL
    with pytest.raises(dl.DlionError) as e:
        ctx.set_momentum_dtype(7)
    assert e.value.status == dl.EINVAL
    ctx.destroy()


# ---------------------------------------------------------------- seeded random configurations
@pytest.mark.parametrize("seed", range(24))
def test_random_configurations(dl, seed):
    """Random segment tables (empty, tiny, ragged, multi-tile tensors), N, aggregation rule,
    gradient type and hyper-parameters; every path against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    nseg = int(rng.integers(1, 9))
    numels = [int(rng.choice([0, 1, 31, 33, 127, 129, 4095, 4096, 4097,
                              int(rng.integers(1, 20000)), int(rng.integers(1, 3 * 4096 * 4))]))
              for _ in range(nseg)]
    n = int(rng.choice([1, 2, 3, 4, 6, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64, 65, 100, 200, 255]))
    mode = int(rng.integers(0, 2))
    gd = str(rng.choice(["f32", "bf16"]))
    w = inputs.custom(numels, n, mode, gd, scale=1.0 if gd == "f32" else 1e-3,
                      a_private=float(rng.choice([0.25, 0.5, 1.0, 2.0])),
                      beta1=float(rng.choice([0.0, 0.5, 0.9, 0.95, 1.0])),
                      beta2=float(rng.choice([0.0, 0.75, 0.99, 0.999, 1.0])),
                      lr=float(rng.choice([1e-4, 1e-2, 0.25])), weight_decay=float(rng.choice([0.0, 0.1, 1.0, 10.0])),
                      zero_frac=float(rng.choice([0.0, 0.05])), seed=int(rng.integers(0, 1 << 30)))
    for path in ("two_stage", "fused") + (("per_worker",) if n <= 9 else ()):
        assert gp.run_small(dl, w, 3, path, modes=(mode,)) == 0


@pytest.mark.parametrize("seed", range(12))
def test_random_configurations_three_valued_tie_rule(dl, seed):
    """The same kind of random configuration under the three-valued tie rule; even worker counts
    are favoured so that ties occur."""
    rng = np.random.default_rng(5000 + seed)
    numels = [int(rng.choice([0, 1, 33, 129, 4096, 4097, int(rng.integers(1, 20000)), int(rng.integers(1, 3 * 4096 * 4))]))
              for _ in range(int(rng.integers(1, 7)))]
    n = int(rng.choice([1, 2, 2, 4, 4, 6, 8, 9, 16, 32, 64, 100, 254, 255]))
    gd = str(rng.choice(["f32", "bf16"]))
    w = inputs.custom(numels, n, inputs.MAJORITY_TERNARY, gd, scale=1.0 if gd == "f32" else 1e-3,
                      a_private=float(rng.choice([0.5, 1.0, 2.0])), beta1=float(rng.choice([0.0, 0.9, 0.95])),
                      beta2=float(rng.choice([0.0, 0.99, 0.999])), lr=float(rng.choice([1e-4, 1e-2, 0.25])),
                      weight_decay=float(rng.choice([0.0, 0.1, 1.0])), zero_frac=float(rng.choice([0.0, 0.05])),
                      seed=int(rng.integers(0, 1 << 30)))
    for path in ("two_stage", "fused"):
        assert gp.run_small(dl, w, 3, path, modes=(inputs.MAJORITY_TERNARY,)) == 0


# ---------------------------------------------------------------- guard bands
@pytest.mark.parametrize("gd,state", [("f32", "f32"), ("bf16", "f32"), ("bf16", "bf16")])
def test_nothing_is_written_outside_the_arenas(dl, gd, state):
    """Every buffer sits between two sentinel bands; after all kernels have run (full tiles that
    end exactly at the arena's end, ragged tails, both aggregation rules) the bands are intact."""
    n = 3
    w = inputs.custom([4097, 33, 2 * 4096], n, AVG, gd, scale=1.0 if gd == "f32" else 1e-3)
    dev = torch.device("cuda:0")
    D, W, G = w.d_pad, w.d_pad // 32, 256                       # G: guard elements on each side
    gdt = inputs.grad_torch_dtype(w)
    mdt = torch.bfloat16 if state == "bf16" else torch.float32

    def guarded(numel, dtype, fill):
        buf = torch.full((numel + 2 * G,), fill, dtype=dtype, device=dev)
        return buf, buf[G:G + numel]

    gbuf, g = guarded(n * D, gdt, 7.0)
    mbuf, m = guarded(n * D, mdt, 7.0)
    xbuf, x = guarded(D, torch.float32, 7.0)
    pbuf, packed = guarded(n * W, torch.int32, 0x5A5A5A5A)
    dbuf, dbits = guarded(W, torch.int32, 0x5A5A5A5A)
    cbuf, count = guarded(D, torch.uint8, 0x5A)
    g.view(n, D).copy_(inputs.fill_grads(w, 0, torch.empty(n, D, dtype=gdt)))
    m.zero_(); x.zero_(); packed.zero_(); dbits.zero_(); count.zero_()
    for mode in (MAJ, AVG):
        ctx = gp.make_ctx(dl, w, mode)
        if state == "bf16":
            ctx.set_momentum_dtype(dl.STATE_BF16)
        K = ctx.delta_planes()
        wbuf, wire = guarded(K * W, torch.int32, 0x5A5A5A5A)
        wire.zero_()
        ctx.worker_step(-1, g.view(n, D), m.view(n, D), packed.view(n, W))
        for i in range(n):
            ctx.worker_step(i, g.view(n, D)[i], m.view(n, D)[i], packed.view(n, W)[i])
        ctx.aggregate_apply(packed, x, dbits, count)
        ctx.step_fused(g, m, x, packed)
        ctx.aggregate(packed, wire)
        ctx.apply_delta(wire, x)
        torch.cuda.synchronize()
        for name, buf, fill in (("g", gbuf, 7.0), ("m", mbuf, 7.0), ("x", xbuf, 7.0), ("packed", pbuf, 0x5A5A5A5A),
                                ("delta_bits", dbuf, 0x5A5A5A5A), ("count", cbuf, 0x5A), ("wire", wbuf, 0x5A5A5A5A)):
            lo, hi = buf[:G], buf[-G:]
            assert bool((lo == fill).all()) and bool((hi == fill).all()), f"{name}: guard band overwritten"
        ctx.destroy()


def test_bf16_momentum_special_values(dl):
    """bf16 momentum with +-0, +-Inf, NaN, values that round up to Inf and bf16 denormals: same
    signs as the oracle, same stored bits wherever the result is a number, NaN where it is NaN."""
    from oracle import dlion_oracle as orc
    n, d = 2, 4096 + 200
    w = inputs.custom([d], n, MAJ, "f32", beta1=0.5, beta2=0.75)
    D, W = w.d_pad, w.d_pad // 32
    rng = np.random.default_rng(21)
    sp16 = np.array([0x0000, 0x8000, 0x3F80, 0xBF80, 0x7F80, 0xFF80, 0x7FC0, 0x0001, 0x8001, 0x7F7F, 0xFF7F, 0x0080],
                    np.uint16)
    m0 = rng.choice(sp16, size=(n, D)).astype(np.uint16)
    sp32 = np.array([0.0, -0.0, 1.0, -1.0, np.nan, np.inf, -np.inf, 1e-42, 3.4e38, -3.4e38, 1.0 + 2.0 ** -8], np.float32)
    g0 = rng.choice(sp32, size=(n, D)).astype(np.float32)
    m0[:, d:] = 0
    g0[:, d:] = 0
    m_ref, p_ref = m0.copy(), np.zeros((n, W), np.uint32)
    orc.worker_step_ex(w.segments, D, n, g0, m_ref, p_ref, [0.5] * n, [0.75] * n)
    dev = torch.device("cuda:0")
    ctx = gp.make_ctx(dl, w)
    ctx.set_momentum_dtype(dl.STATE_BF16)
    m = torch.from_numpy(m0.view(np.int16)).to(dev).view(torch.bfloat16)
    packed = torch.zeros(n, W, dtype=torch.int32, device=dev)
    ctx.worker_step(-1, torch.from_numpy(g0).to(dev), m, packed)
    torch.cuda.synchronize()
    gp.compare("packed", packed.cpu().numpy().view(np.uint32), p_ref, True)
    got = m.cpu().view(torch.int16).numpy().view(np.uint16)
    nan_ref = (m_ref & 0x7FFF) > 0x7F80
    nan_got = (got & 0x7FFF) > 0x7F80
    assert np.array_equal(nan_ref, nan_got)
    assert nan_ref.any() and np.array_equal(got[~nan_ref], m_ref[~nan_ref])
    ctx.destroy()


# ---------------------------------------------------------------- more than 255 workers
@pytest.mark.parametrize("n", [256, 511, 1000])
@pytest.mark.parametrize("mode", [MAJ, AVG])
def test_more_than_255_workers(dl, n, mode):
    """Vote counts beyond one byte: 9 and 10 bit planes; the byte-count outputs and the fused
    step say so instead of overflowing."""
    w = inputs.custom([4096 + 77, 33], n, mode, "bf16", scale=1e-3, lr=1e-3, weight_decay=0.5)
    assert gp.run_small(dl, w, 2, "two_stage", modes=(mode,)) == 0
    dev = torch.device("cuda:0")
    ctx = gp.make_ctx(dl, w)
    t = torch.zeros(n * w.d_pad, dtype=torch.int32, device=dev)
    with pytest.raises(dl.DlionError) as e:
        ctx.step_fused(t.view(torch.bfloat16)[:n * w.d_pad], t.view(torch.float32), t.view(torch.float32)[:w.d_pad], None)
    assert e.value.status == dl.EINVAL
    with pytest.raises(dl.DlionError) as e:
        ctx.aggregate_apply(t, t.view(torch.float32)[:w.d_pad], None, t.view(torch.uint8)[:w.d_pad])
    assert e.value.status == dl.EINVAL
    ctx.destroy()


@pytest.mark.parametrize("n", [3, 200, 255, 256, 300, 1000, 4097])
@pytest.mark.parametrize("mode", [MAJ, AVG])
def test_sixteen_bit_counts(dl, n, mode):
    """dlion_aggregate_apply_counts16 on a ragged table with several tiles: counts equal the
    oracle's, padding of the count buffer untouched, x as from the plain call."""
    from oracle import dlion_oracle as orc
    w = inputs.custom(RAGGED + [2 * 4096 + 5], n, mode, "f32", lr=1e-2, weight_decay=0.5)
    dev = torch.device("cuda:0")
    D = w.d_pad
    rng = np.random.default_rng(n * 2 + mode)
    valid = np.zeros(D, bool)
    for off, cnt in w.segments:
        valid[off:off + cnt] = True
    bits = (rng.integers(0, 256, (n, D), dtype=np.uint8) < rng.integers(0, 257, D)[None, :]) & valid[None, :]
    packed_np = np.packbits(bits, axis=1, bitorder="little").view(np.uint32).reshape(n, -1).copy()
    cnt_ref = np.full(D, 0x5A5A, np.uint16)
    orc.vote_counts16(w.segments, D, n, packed_np, cnt_ref)
    x_ref = inputs.fill_x0(w, torch.empty(D)).numpy().copy()
    orc.aggregate_apply(w.segments, D, n, mode, packed_np, x_ref, w.lr, w.weight_decay)
    ctx = gp.make_ctx(dl, w)
    packed = torch.from_numpy(packed_np.view(np.int32)).to(dev)
    x = inputs.fill_x0(w, torch.empty(D)).to(dev)
    cnt = torch.full((D,), 0x5A5A, dtype=torch.int16, device=dev)
    ctx.aggregate_apply_counts16(packed, x, None, cnt)
    torch.cuda.synchronize()
    gp.compare("16-bit counts", cnt.cpu().numpy().view(np.uint16), cnt_ref, True)
    gp.compare("x", x.cpu().numpy(), x_ref, True)
    ctx.destroy()


@pytest.mark.parametrize("n", [8191, 8192, 16383, 16384, 32768, 65535])
@pytest.mark.parametrize("mode", [MAJ, AVG])
def test_thirteen_to_sixteen_bit_planes(dl, n, mode):
    """The largest worker counts the library accepts (13 to 16 bit planes of votes, 65535 =
    DLION_MAX_WORKERS): the one-call server step, the server-only vote and the worker-side
    apply against the oracle on a ragged table.  The sign words are drawn directly (the vote
    does not care where they came from) with a different probability of +1 per coordinate, and
    a few coordinates are forced to the extremes: all +1, all -1, an exact tie (even N) and one
    vote short of it."""
    from oracle import dlion_oracle as orc
    w = inputs.custom([4096 + 77, 33, 1000], n, mode, "f32", lr=1e-2, weight_decay=0.5)
    dev = torch.device("cuda:0")
    D, W = w.d_pad, w.d_pad // 32
    rng = np.random.default_rng(n + mode)
    valid = np.zeros(D, bool)
    for off, cnt in w.segments:
        valid[off:off + cnt] = True
    bits = rng.integers(0, 256, (n, D), dtype=np.uint8) < rng.integers(0, 257, D)[None, :]
    half = (n + 1) // 2                                  # smallest count with Delta = +1
    for seg_off in (w.segments[0][0], w.segments[2][0]):
        bits[:, seg_off + 0] = True
        bits[:, seg_off + 1] = False
        bits[:, seg_off + 2] = np.arange(n) < half
        bits[:, seg_off + 3] = np.arange(n) < half - 1
        bits[:, seg_off + 4] = np.arange(n) >= n - half   # the same count held by the LAST workers
    bits &= valid[None, :]
    packed_np = np.packbits(bits, axis=1, bitorder="little").view(np.uint32).reshape(n, -1).copy()
    x0 = inputs.fill_x0(w, torch.empty(D))
    ctx = gp.make_ctx(dl, w)
    K = ctx.delta_planes()
    assert K == orc.delta_planes(n, mode) == (1 if mode == MAJ else int(n).bit_length())
    wire_ref = np.zeros(K * W, np.uint32)
    orc.aggregate(w.segments, D, n, mode, packed_np, wire_ref)
    x_ref = x0.numpy().copy()
    orc.apply_delta(w.segments, D, n, mode, wire_ref, x_ref, w.lr, w.weight_decay)
    x_ref1, dbits_ref = x0.numpy().copy(), np.zeros(W, np.uint32)
    orc.aggregate_apply(w.segments, D, n, mode, packed_np, x_ref1, w.lr, w.weight_decay, delta_bits=dbits_ref)
    packed = torch.from_numpy(packed_np.view(np.int32)).to(dev)
    wire = torch.zeros(K * W, dtype=torch.int32, device=dev)
    dbits = torch.zeros(W, dtype=torch.int32, device=dev)
    x, x_one = x0.to(dev), x0.to(dev)
    ctx.aggregate(packed, wire)
    ctx.apply_delta(wire, x)
    ctx.aggregate_apply(packed, x_one, dbits)
    torch.cuda.synchronize()
    gp.compare("delta wire", wire.cpu().numpy().view(np.uint32), wire_ref, True)
    gp.compare("x after apply_delta", x.cpu().numpy(), x_ref, True)
    gp.compare("x after aggregate_apply", x_one.cpu().numpy(), x_ref1, True)
    gp.compare("delta bits", dbits.cpu().numpy().view(np.uint32), dbits_ref, True)
    # the same call with the vote counts written out, 16 bits each
    cnt_ref = np.full(D, 0x5A5A, np.uint16)
    orc.vote_counts16(w.segments, D, n, packed_np, cnt_ref)
    cnt = torch.full((D,), 0x5A5A, dtype=torch.int16, device=dev)
    x_cnt = x0.to(dev)
    ctx.aggregate_apply_counts16(packed, x_cnt, None, cnt)
    torch.cuda.synchronize()
    gp.compare("16-bit counts", cnt.cpu().numpy().view(np.uint16), cnt_ref, True)
    assert torch.equal(x_cnt, x_one)
    ctx.destroy()


def test_step_host_with_bf16_momentum_and_worker_betas(dl):
    """The host-gradient step slices the momentum arena by its storage type and passes each
    worker's own betas."""
    from oracle import dlion_oracle as orc
    n = 3
    b1s, b2s = [0.9, 0.5, 0.0], [0.99, 0.75, 0.0]
    w = inputs.custom([9000, 77], n, MAJ, "bf16", scale=1e-3, lr=1e-3, weight_decay=1.0)
    dev = torch.device("cuda:0")
    D, W = w.d_pad, w.d_pad // 32
    ctx = gp.make_ctx(dl, w)
    ctx.set_momentum_dtype(dl.STATE_BF16)
    for i in range(n):
        ctx.set_worker_betas(i, b1s[i], b2s[i])
    x0 = inputs.fill_x0(w, torch.empty(D))
    m_ref, x_ref = np.zeros((n, D), np.uint16), x0.numpy().copy()
    m = torch.zeros(n, D, dtype=torch.bfloat16, device=dev)
    x = x0.to(dev)
    packed = torch.zeros(n, W, dtype=torch.int32, device=dev)
    staging = torch.empty(2, D, dtype=torch.bfloat16, device=dev)
    host_g = torch.empty(n, D, dtype=torch.bfloat16).pin_memory()
    for t in range(3):
        inputs.fill_grads(w, t, host_g)
        p_ref = np.zeros((n, W), np.uint32)
        orc.worker_step_ex(w.segments, D, n, inputs.as_numpy_grads(host_g), m_ref, p_ref, b1s, b2s)
        orc.aggregate_apply(w.segments, D, n, MAJ, p_ref, x_ref, w.lr, w.weight_decay)
        ctx.step_host(host_g, m, x, packed, staging)
        torch.cuda.synchronize()
        gp.compare("packed", packed.cpu().numpy().view(np.uint32), p_ref, True)
        assert np.array_equal(m.cpu().view(torch.int16).numpy().view(np.uint16), m_ref)
        assert gp.compare("x", x.cpu().numpy(), x_ref, False) == 0
    ctx.destroy()


def test_calls_can_be_captured_in_a_cuda_graph(dl):
    """worker_step, aggregate_apply and step_fused neither synchronise nor allocate, so a
    multi-step loop can be captured once and replayed; the replay must equal the eager steps."""
    w = inputs.custom([3 * 4096 + 5, 77], 4, MAJ, "f32", lr=1e-2, weight_decay=0.5)
    dev = torch.device("cuda:0")
    N, D, W = w.n_workers, w.d_pad, w.d_pad // 32
    ctx = gp.make_ctx(dl, w)
    g = inputs.fill_grads(w, 0, torch.empty(N, D)).to(dev)
    x0 = inputs.fill_x0(w, torch.empty(D)).to(dev)

    def run(eager: bool, fused: bool):
        m = torch.zeros(N, D, device=dev)
        x = x0.clone()
        packed = torch.zeros(N, W, dtype=torch.int32, device=dev)

        def steps():
            for _ in range(3):
                if fused:
                    ctx.step_fused(g, m, x, packed)
                else:
                    ctx.worker_step(-1, g, m, packed)
                    ctx.aggregate_apply(packed, x)
        if eager:
            steps()
        else:
            side = torch.cuda.Stream()
            gph = torch.cuda.CUDAGraph()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.graph(gph, stream=side):
                steps()
            gph.replay()
        torch.cuda.synchronize()
        return m, x, packed

    for fused in (False, True):
        a, b = run(True, fused), run(False, fused)
        assert all(torch.equal(u, v) for u, v in zip(a, b))
    ctx.destroy()


def test_checkpoint_and_resume_is_bit_identical(dl):
    """The library keeps no optimizer state of its own: saving m and x to the host after two
    steps, destroying the context, and resuming in a new context from the saved copies gives the
    same bits as four uninterrupted steps (per-worker betas and bf16 momentum included)."""
    dev = torch.device("cuda:0")
    n = 5
    w = inputs.custom(RAGGED, n, AVG, "bf16", scale=1e-3, lr=1e-3, weight_decay=0.5)
    D, W = w.d_pad, w.d_pad // 32

    def new_ctx():
        c = gp.make_ctx(dl, w)
        c.set_momentum_dtype(dl.STATE_BF16)
        c.set_worker_betas(3, 0.5, 0.5)
        return c

    grads = [inputs.fill_grads(w, t, torch.empty(n, D, dtype=torch.bfloat16)).to(dev) for t in range(4)]
    x0 = inputs.fill_x0(w, torch.empty(D))
    packed = torch.zeros(n, W, dtype=torch.int32, device=dev)
    ctx = new_ctx()
    m_a, x_a = torch.zeros(n, D, dtype=torch.bfloat16, device=dev), x0.to(dev)
    for t in range(4):
        ctx.worker_step(-1, grads[t], m_a, packed)
        ctx.aggregate_apply(packed, x_a)
    ctx.destroy()
    ctx = new_ctx()
    m_b, x_b = torch.zeros(n, D, dtype=torch.bfloat16, device=dev), x0.to(dev)
    for t in range(2):
        ctx.worker_step(-1, grads[t], m_b, packed)
        ctx.aggregate_apply(packed, x_b)
    torch.cuda.synchronize()
    saved_m, saved_x = m_b.cpu().clone(), x_b.cpu().clone()            # the checkpoint
    ctx.destroy()
    del m_b, x_b
    ctx = new_ctx()
    m_c, x_c = saved_m.to(dev), saved_x.to(dev)
    for t in range(2, 4):
        ctx.step_fused(grads[t], m_c, x_c, None)                       # resumed on another path, too
    torch.cuda.synchronize()
    assert torch.equal(m_c.view(torch.int16), m_a.view(torch.int16)) and torch.equal(x_c, x_a)
    ctx.destroy()
