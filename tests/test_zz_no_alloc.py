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
    with pytest.raises(dl.DlionError) as e:
        dl.step_static(1024, 1, 0.9, 0.99, 1e-4, 0.0, 0, 0, t[1:], t, t)
    assert e.value.status == dl.EALIGN
