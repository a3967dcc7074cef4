"""The optional three-valued tie rule (DLION_MAJORITY_TERNARY: Delta = 0 on an even-N tie)
through every path that takes an aggregation rule, against the oracle: the one-call server
step, the one-launch step, the vote into the two-plane message and the apply from it (also
from the all-gather layout), the host-gradient step and the fixed-scratch step.  Gradients
are built so that exact ties really occur."""
import numpy as np
import pytest
import torch

from paper_2404_00438_b200 import inputs
from tests import gpu_parity as gp

pytestmark = pytest.mark.gpu
TER = inputs.MAJORITY_TERNARY
RAGGED = [5, 200, 31, 4096, 4097, 12289, 0, 33, 127]


@pytest.fixture(scope="module")
def dl():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2404_00438_b200 import build
    build.build()
    from paper_2404_00438_b200 import dlion
    return dlion


def _packed_with_ties(w, n, rng):
    D = w.d_pad
    valid = np.zeros(D, bool)
    for off, cnt in w.segments:
        valid[off:off + cnt] = True
    bits = rng.integers(0, 256, (n, D), dtype=np.uint8) < rng.integers(0, 257, D)[None, :]
    if n % 2 == 0:                                       # every seventh coordinate is an exact tie
        order = rng.permuted(np.tile(np.arange(n) < n // 2, (D, 1)), axis=1).T
        tie = (np.arange(D) % 7 == 0)
        bits[:, tie] = order[:, tie]
    bits &= valid[None, :]
    return np.packbits(bits, axis=1, bitorder="little").view(np.uint32).reshape(n, -1).copy(), valid


@pytest.mark.parametrize("n", [1, 2, 3, 4, 8, 16, 33, 64, 254, 255, 256, 1000, 4098])
def test_server_side_with_ties(dl, n):
    from oracle import dlion_oracle as orc
    dev = torch.device("cuda:0")
    w = inputs.custom(RAGGED, n, TER, "f32", lr=1e-2, weight_decay=0.5)
    D, W = w.d_pad, w.d_pad // 32
    packed_np, valid = _packed_with_ties(w, n, np.random.default_rng(n))
    x0 = inputs.fill_x0(w, torch.empty(D))
    ctx = gp.make_ctx(dl, w)
    assert ctx.delta_planes() == 2 == orc.delta_planes(n, TER)
    assert ctx.wire_bytes(1) == (2 * w.d + 7) // 8
    x_ref, dbits_ref = x0.numpy().copy(), np.zeros(W, np.uint32)
    orc.aggregate_apply(w.segments, D, n, TER, packed_np, x_ref, w.lr, w.weight_decay, delta_bits=dbits_ref)
    wire_ref = np.zeros(2 * W, np.uint32)
    orc.aggregate(w.segments, D, n, TER, packed_np, wire_ref)
    if n % 2 == 0:
        assert wire_ref[:W].any()                        # ties are really there
    packed = torch.from_numpy(packed_np.view(np.int32)).to(dev)
    x_one, x_two, x_sl = x0.to(dev), x0.to(dev), x0.to(dev)
    dbits = torch.zeros(W, dtype=torch.int32, device=dev)
    wire = torch.zeros(2 * W, dtype=torch.int32, device=dev)
    ctx.aggregate_apply(packed, x_one, dbits)
    ctx.aggregate(packed, wire)
    ctx.apply_delta(wire, x_two)
    if W % 4 == 0:                                       # the same message in all-gather order, four slices
        sw = W // 4
        sliced = wire.view(2, 4, sw).permute(1, 0, 2).contiguous()
        ctx.apply_delta_sliced(sliced, sw, x_sl)
    else:
        x_sl = x_two
    torch.cuda.synchronize()
    gp.compare("x, one call", x_one.cpu().numpy(), x_ref, True)
    gp.compare("delta bits", dbits.cpu().numpy().view(np.uint32), dbits_ref, True)
    gp.compare("two-plane message", wire.cpu().numpy().view(np.uint32), wire_ref, True)
    gp.compare("x, vote then apply", x_two.cpu().numpy(), x_ref, True)
    gp.compare("x, apply from slices", x_sl.cpu().numpy(), x_ref, True)
    ctx.destroy()


@pytest.mark.parametrize("n,gd", [(2, "f32"), (4, "bf16"), (16, "bf16"), (7, "f32")])
def test_whole_steps_with_ties(dl, n, gd):
    """Whole steps on gradients that produce ties: workers come in +g / -g pairs on every
    third coordinate.  Two-stage, fused, host-gradient and fixed-scratch steps."""
    from oracle import dlion_oracle as orc
    dev = torch.device("cuda:0")
    w = inputs.custom([4096 * 2 + 77, 33, 5000], n, TER, gd, scale=1.0 if gd == "f32" else 1e-3, lr=1e-2, weight_decay=0.5)
    D, W = w.d_pad, w.d_pad // 32
    gdt = inputs.grad_torch_dtype(w)
    ctx = gp.make_ctx(dl, w)
    x0 = inputs.fill_x0(w, torch.empty(D))
    x_ref, m_ref, p_ref = x0.numpy().copy(), np.zeros((n, D), np.float32), np.zeros((n, W), np.uint32)
    xs = [x0.to(dev) for _ in range(3)]
    ms = [torch.zeros(n, D, device=dev) for _ in range(3)]
    packed = torch.zeros(n, W, dtype=torch.int32, device=dev)
    staging = torch.empty(2, D, dtype=gdt, device=dev)
    wire = torch.zeros(2 * W, dtype=torch.int32, device=dev)
    host_wire = torch.zeros(2 * W, dtype=torch.int32).pin_memory()
    ties_seen = 0
    for t in range(3):
        g_cpu = inputs.fill_grads(w, t, torch.empty(n, D, dtype=gdt))
        for i in range(0, n - 1, 2):                     # pairs of opposite workers on every third coordinate
            g_cpu[i + 1, ::3] = -g_cpu[i, ::3]
        if n % 2 == 1:
            g_cpu[n - 1, ::3] = g_cpu[0, ::3]
        g = g_cpu.to(dev)
        orc.worker_step(w.segments, D, n, inputs.as_numpy_grads(g_cpu), m_ref, p_ref, w.beta1, w.beta2)
        wire_ref = np.zeros(2 * W, np.uint32)
        orc.aggregate(w.segments, D, n, TER, p_ref, wire_ref)
        ties_seen += int(wire_ref[:W].any())
        orc.aggregate_apply(w.segments, D, n, TER, p_ref, x_ref, w.lr, w.weight_decay)
        ctx.worker_step(-1, g, ms[0], packed)
        ctx.aggregate_apply(packed, xs[0])
        ctx.step_fused(g, ms[1], xs[1], None)
        ctx.step_host(g_cpu.pin_memory(), ms[2], xs[2], packed, staging, wire, host_wire)
        torch.cuda.synchronize()
        for k, name in enumerate(("two-stage", "fused", "host-gradient")):
            gp.compare(f"step {t} {name} m", ms[k].cpu().numpy(), m_ref, True)
            gp.compare(f"step {t} {name} x", xs[k].cpu().numpy(), x_ref, True)
        gp.compare(f"step {t} message copied to the host", host_wire.numpy().view(np.uint32), wire_ref, True)
    assert ties_seen == (3 if n % 2 == 0 else 0)
    ctx.destroy()
    # the fixed-scratch step on a flat vector
    d = 100_003
    wf = inputs.custom([d], n, TER, gd, scale=1.0 if gd == "f32" else 1e-3, lr=1e-2, weight_decay=0.5)
    Df = wf.d_pad
    g_cpu = inputs.fill_grads(wf, 0, torch.empty(n, Df, dtype=gdt))
    for i in range(0, n - 1, 2):
        g_cpu[i + 1, ::3] = -g_cpu[i, ::3]
    x0 = inputs.fill_x0(wf, torch.empty(Df))
    x_ref, m_ref, p_ref = x0.numpy().copy(), np.zeros((n, Df), np.float32), np.zeros((n, Df // 32), np.uint32)
    orc.worker_step(wf.segments, Df, n, inputs.as_numpy_grads(g_cpu), m_ref, p_ref, wf.beta1, wf.beta2)
    orc.aggregate_apply(wf.segments, Df, n, TER, p_ref, x_ref, wf.lr, wf.weight_decay)
    x, m = x0.to(dev), torch.zeros(n, Df, device=dev)
    dl.step_static(d, n, wf.beta1, wf.beta2, wf.lr, wf.weight_decay, TER, gp.gdtype_of(wf), g_cpu.to(dev), m, x)
    torch.cuda.synchronize()
    gp.compare("fixed-scratch x", x.cpu().numpy(), x_ref, True)
    gp.compare("fixed-scratch m", m.cpu().numpy(), m_ref, True)
