"""dlion_step_static, the entry point for callers that cannot allocate device memory
(its segment table and wire buffer are a fixed array inside the library): it must give
what the regular two-stage calls give, call after call, although every call reuses the
same scratch.  Collected last on purpose, so that a run that stops at the first failure
has already run every other test."""
import numpy as np
import pytest
import torch

from paper_2404_00438_b200 import inputs
from tests import gpu_parity as gp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dl():
    assert torch.cuda.is_available(), "this test needs a CUDA device"
    from paper_2404_00438_b200 import build
    build.build()
    from paper_2404_00438_b200 import dlion
    return dlion


@pytest.mark.parametrize("mode", [inputs.MAJORITY, inputs.AVERAGE])
@pytest.mark.parametrize("gd,d,n", [("f32", 1_000_003, 4), ("bf16", 300_001, 16)])
def test_two_calls_in_a_row_match_the_regular_path(dl, mode, gd, d, n):
    dev = torch.device("cuda:0")
    w = inputs.custom([d], n, mode, gd, scale=1.0 if gd == "f32" else 1e-3, lr=1e-3, weight_decay=0.5)
    gdt = inputs.grad_torch_dtype(w)
    ctx = gp.make_ctx(dl, w)
    x0 = inputs.fill_x0(w, torch.empty(w.d_pad)).to(dev)
    m_ref, x_ref = torch.zeros(n, w.d_pad, device=dev), x0.clone()
    m_new, x_new = torch.zeros(n, w.d_pad, device=dev), x0.clone()
    packed = torch.zeros(n, w.d_pad // 32, dtype=torch.int32, device=dev)
    for t in range(2):                                   # the second call sees the first call's scratch
        g = inputs.fill_grads(w, t, torch.empty(n, w.d_pad, dtype=gdt)).to(dev)
        ctx.worker_step(-1, g, m_ref, packed)
        ctx.aggregate_apply(packed, x_ref)
        dl.step_static(d, n, w.beta1, w.beta2, w.lr, w.weight_decay, mode, gp.gdtype_of(w), g, m_new, x_new)
        torch.cuda.synchronize()
        assert gp.ulp_diff(m_new.cpu().numpy(), m_ref.cpu().numpy()) <= gp.TOL_ULP
        assert gp.ulp_diff(x_new.cpu().numpy(), x_ref.cpu().numpy()) <= gp.TOL_ULP
        assert torch.equal(m_new, m_ref) and torch.equal(x_new, x_ref)   # same kernels: same bits
    ctx.destroy()


def test_sizes_beyond_the_fixed_scratch_are_rejected(dl):
    dev = torch.device("cuda:0")
    t = torch.zeros(1024, device=dev)
    too_many = dl.STATIC_MAX_COORD_WORKERS // 4 + 128
    for d, n in ((too_many, 4), (dl.STATIC_MAX_COORD_WORKERS + 1, 1)):
        with pytest.raises(dl.DlionError) as e:
            dl.step_static(d, n, 0.9, 0.99, 1e-4, 0.0, 0, 0, t, t, t)
        assert e.value.status == dl.EINVAL
    longer = torch.zeros(1028, device=dev)
    with pytest.raises(dl.DlionError) as e:
        dl.step_static(1024, 1, 0.9, 0.99, 1e-4, 0.0, 0, 0, longer[1:], t, t)     # 4-byte aligned only
    assert e.value.status == dl.EALIGN
    with pytest.raises(ValueError):                          # shorter than the call's extent: nothing is launched
        dl.step_static(1024, 1, 0.9, 0.99, 1e-4, 0.0, 0, 0, t[1:], t, t)


def test_against_the_oracle_big_then_small_and_nothing_allocated(dl):
    """The entry point against the CPU oracle itself (not only against the regular CUDA path),
    a large problem followed by a smaller one with another worker count on the same scratch
    (the small one must not see the large one's stale sign bits), and the device's free memory
    unchanged across the calls after the first one (which is the set-up call)."""
    from oracle import dlion_oracle as orc
    dev = torch.device("cuda:0")
    warm = torch.zeros(128, device=dev)
    dl.step_static(128, 1, 0.9, 0.99, 1e-4, 0.0, 0, 0, warm, warm.clone(), warm.clone())   # set-up call
    torch.cuda.synchronize()
    cases = [(2_000_003, 33, inputs.AVERAGE, "bf16"), (70_001, 5, inputs.MAJORITY, "f32"),
             (4096 * 3 + 17, 300, inputs.AVERAGE, "f32")]
    prepared = []
    for d, n, mode, gd in cases:
        w = inputs.custom([d], n, mode, gd, scale=1.0 if gd == "f32" else 1e-3, lr=1e-3, weight_decay=0.5)
        gdt = inputs.grad_torch_dtype(w)
        g = [inputs.fill_grads(w, t, torch.empty(n, w.d_pad, dtype=gdt)) for t in range(2)]
        x0 = inputs.fill_x0(w, torch.empty(w.d_pad))
        prepared.append((w, g, [t.to(dev) for t in g], x0, x0.to(dev), torch.zeros(n, w.d_pad, device=dev)))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for w, g_cpu, g_dev, x0, x, m in prepared:
        for t in range(2):
            dl.step_static(w.d, w.n_workers, w.beta1, w.beta2, w.lr, w.weight_decay, w.mode, gp.gdtype_of(w),
                           g_dev[t], m, x)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before       # six steps, not a byte taken from the device
    for w, g_cpu, g_dev, x0, x, m in prepared:
        n, D = w.n_workers, w.d_pad
        m_ref, x_ref = np.zeros((n, D), np.float32), x0.numpy().copy()
        for t in range(2):
            packed = np.zeros((n, D // 32), np.uint32)
            orc.worker_step(w.segments, D, n, inputs.as_numpy_grads(g_cpu[t]), m_ref, packed, w.beta1, w.beta2, nthreads=8)
            orc.aggregate_apply(w.segments, D, n, w.mode, packed, x_ref, w.lr, w.weight_decay, nthreads=8)
        assert gp.compare(f"d={w.d} N={n} m", m.cpu().numpy(), m_ref, False) == 0
        assert gp.compare(f"d={w.d} N={n} x", x.cpu().numpy(), x_ref, False) == 0
