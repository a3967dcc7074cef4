"""dlion_step_global (the Global-Lion comparison step: fp32 mean of the workers' blends, one
sign) against the CPU oracle's plain loop, element by element.  The sum order is fixed on
both sides (worker 0 first), so every bit must agree: the sign bits exactly, and the fp32
state within the 2-ulp tolerance of the other parity tests (0 observed)."""
import numpy as np
import pytest
import torch

from paper_2404_00438_b200 import inputs
from tests import gpu_parity as gp

pytestmark = pytest.mark.gpu
RAGGED = [5, 200, 31, 32, 1, 4096, 4097, 8191, 12289, 0, 33, 128, 127, 3 * 4096 + 5]


@pytest.fixture(scope="module")
def dl():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2404_00438_b200 import build
    build.build()
    from paper_2404_00438_b200 import dlion
    return dlion


def run_global(dl, w, steps, with_bits=True, m0=None, grads=None):
    from oracle import dlion_oracle as orc
    dev = torch.device("cuda:0")
    N, D, W = w.n_workers, w.d_pad, w.d_pad // 32
    gdt = inputs.grad_torch_dtype(w)
    ctx = gp.make_ctx(dl, w)
    x0 = inputs.fill_x0(w, torch.empty(D))
    m_cpu = torch.zeros(N, D) if m0 is None else m0
    m_ref, x_ref = m_cpu.numpy().copy(), x0.numpy().copy()
    m, x = m_cpu.to(dev), x0.to(dev)
    bits = torch.full((W,), 0x5A5A5A5A, dtype=torch.int32, device=dev) if with_bits else None
    bits_ref = np.full(W, 0x5A5A5A5A, np.uint32)            # words that hold no parameter stay as they were
    worst = 0
    for t in range(steps):
        g_cpu = grads[t] if grads is not None else inputs.fill_grads(w, t, torch.empty(N, D, dtype=gdt))
        orc.global_step(w.segments, D, N, inputs.as_numpy_grads(g_cpu), m_ref, x_ref, w.beta1, w.beta2,
                        w.lr, w.weight_decay, delta_bits=bits_ref)
        ctx.step_global(g_cpu.to(dev), m, x, bits)
        torch.cuda.synchronize()
        tag = f"N={N} step {t}"
        worst = max(worst, gp.compare(tag + " m", m.cpu().numpy(), m_ref, False))
        worst = max(worst, gp.compare(tag + " x", x.cpu().numpy(), x_ref, False))
        if with_bits:
            gp.compare(tag + " sign bits", bits.cpu().numpy().view(np.uint32), bits_ref, True)
    ctx.destroy()
    return worst


@pytest.mark.parametrize("n", [1, 2, 3, 4, 7, 8, 16, 33, 64])
@pytest.mark.parametrize("gd", ["f32", "bf16"])
def test_ragged_table(dl, n, gd):
    w = inputs.custom(RAGGED, n, inputs.MAJORITY, gd, scale=1.0 if gd == "f32" else 1e-3, lr=1e-2,
                      weight_decay=0.5, zero_frac=0.02)
    assert run_global(dl, w, 4) == 0
    assert run_global(dl, w, 2, with_bits=False) == 0


def test_c1_shape_ten_steps(dl):
    w = inputs.workload("c1")
    assert run_global(dl, w, 10) == 0


def test_cancelling_and_special_values(dl):
    """Blends that cancel exactly (mean +0 or -0 -> +1), a negative sum too small to survive the
    division (-denormal / N rounds to -0 -> +1), NaN (-> -1), infinities."""
    n, d = 4, 4096 + 64
    w = inputs.custom([d], n, inputs.MAJORITY, "f32", lr=1e-2, weight_decay=0.5)
    g = torch.zeros(n, w.d_pad)
    g[0, 0], g[1, 0] = 3.0, -3.0                           # cancels to +0
    g[0, 1], g[1, 1] = -3.0, 3.0
    g[:, 2] = torch.tensor([-1e-45, 0.0, 0.0, 0.0])        # -denormal: (1-beta1)*g underflows or stays tiny
    g[:, 3] = torch.tensor([float("nan"), 1.0, 1.0, 1.0])
    g[:, 4] = torch.tensor([float("inf"), -1.0, -1.0, -1.0])
    g[:, 5] = torch.tensor([float("inf"), float("-inf"), 0.0, 0.0])   # inf - inf = NaN -> -1
    g[:, 6] = torch.tensor([-0.0, -0.0, -0.0, -0.0])
    g[:, 4100] = torch.tensor([1e-38, -2e-38, 0.0, 0.0])   # ragged tile; tiny negative sum
    m0 = torch.zeros(n, w.d_pad)
    m0[0, 7], g[0, 7] = -1.4e-44, 0.0                      # beta1 * denormal; sum / 4 rounds to -0
    assert run_global(dl, w, 2, m0=m0, grads=[g, g]) == 0


def test_rejected_configurations(dl):
    w = inputs.custom([5000], 2, inputs.MAJORITY, "f32")
    dev = torch.device("cuda:0")
    g = torch.zeros(2, w.d_pad, device=dev)
    m = torch.zeros(2, w.d_pad, device=dev)
    x = torch.zeros(w.d_pad, device=dev)
    ctx = gp.make_ctx(dl, w)
    ctx.set_worker_betas(0, 0.5, 0.5)                      # per-worker betas are not part of the scheme
    with pytest.raises(dl.DlionError) as e:
        ctx.step_global(g, m, x)
    assert e.value.status == dl.EINVAL
    ctx.destroy()
    ctx = gp.make_ctx(dl, w)
    ctx.set_momentum_dtype(dl.STATE_BF16)
    assert dl.lib().dlion_step_global(ctx._ctx, g.data_ptr(), m.data_ptr(), x.data_ptr(), None, None) == dl.EINVAL
    ctx.destroy()
