"""Per-tensor mode: a parameter LIST of separately allocated tensors (with their gradient and
momentum tensors) is stepped in place through pointer tables and must end, tensor by tensor,
with what the oracle computes on the same values laid out as one arena.  Every tensor sits
inside a larger allocation with guard values on both sides, so a write outside a tensor
shows."""
import numpy as np
import pytest
import torch

from paper_2404_00438_b200 import inputs
from tests import gpu_parity as gp

pytestmark = pytest.mark.gpu
MAJ, AVG = inputs.MAJORITY, inputs.AVERAGE
NUMELS = [5000, 77, 0, 3 * 4096, 12289, 1, 4096, 40001]
GUARD = 64                     # elements on each side; keeps the tensor 16-byte aligned


@pytest.fixture(scope="module")
def dl():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2404_00438_b200 import build
    build.build()
    from paper_2404_00438_b200 import dlion
    return dlion


class Guarded:
    """A tensor of n elements inside its own allocation, with guard values around it."""

    def __init__(self, values: torch.Tensor, dev):
        n = values.numel()
        self.fill = 7 if values.dtype in (torch.int16, torch.int32) else 7.0
        self.buf = torch.full((n + 2 * GUARD,), self.fill, dtype=values.dtype, device=dev)
        self.t = self.buf[GUARD:GUARD + n]
        self.t.copy_(values)

    def intact(self) -> bool:
        n = self.t.numel()
        return bool((self.buf[:GUARD] == self.fill).all() and (self.buf[GUARD + n:] == self.fill).all())


@pytest.mark.parametrize("n,gd,state,mode", [(1, "f32", "f32", MAJ), (3, "bf16", "f32", AVG), (16, "bf16", "bf16", MAJ),
                                             (4, "f32", "bf16", AVG), (300, "bf16", "f32", AVG)])
def test_tensor_list_equals_oracle(dl, n, gd, state, mode):
    from oracle import dlion_oracle as orc
    dev = torch.device("cuda:0")
    w = inputs.custom(NUMELS, n, mode, gd, scale=1.0 if gd == "f32" else 1e-3, lr=1e-2, weight_decay=0.5)
    D, W = w.d_pad, w.d_pad // 32
    gdt = inputs.grad_torch_dtype(w)
    sdt = torch.float32 if state == "f32" else torch.bfloat16
    ctx = gp.make_ctx(dl, w)
    if state == "bf16":
        ctx.set_momentum_dtype(dl.STATE_BF16)
    x0 = inputs.fill_x0(w, torch.empty(D))
    xs = [Guarded(x0[o:o + k], dev) for o, k in w.segments]
    xs2 = [Guarded(x0[o:o + k], dev) for o, k in w.segments]
    ms = [[Guarded(torch.zeros(k, dtype=sdt), dev) for o, k in w.segments] for _ in range(n)]
    packed = torch.zeros(n, W, dtype=torch.int32, device=dev)
    dbits = torch.zeros(W, dtype=torch.int32, device=dev)
    wire = torch.zeros(ctx.delta_planes() * W, dtype=torch.int32, device=dev)
    with pytest.raises(dl.DlionError) as e:                        # nothing bound yet
        ctx.worker_step_tensors(-1, packed)
    assert e.value.status == dl.ESTATE
    ctx.bind_tensors(m=[[t.t for t in row] for row in ms], x=[t.t for t in xs])
    # the oracle, on the same values as one arena
    x_ref = x0.numpy().copy()
    m_ref = np.zeros((n, D), np.float32 if state == "f32" else np.uint16)
    p_ref = np.zeros((n, W), np.uint32)
    d_ref = np.zeros(W, np.uint32)
    for t in range(3):
        g_cpu = inputs.fill_grads(w, t, torch.empty(n, D, dtype=gdt))
        gs = [[Guarded(g_cpu[i, o:o + k], dev) for o, k in w.segments] for i in range(n)]   # new tensors every step
        ctx.bind_tensors(grads=[[t_.t for t_ in row] for row in gs])
        if t % 2 == 0:
            ctx.worker_step_tensors(-1, packed)
        else:
            for i in range(n):
                ctx.worker_step_tensors(i, packed[i])
        ctx.aggregate_apply_tensors(packed, dbits)
        # the second copy of x takes the server-only vote and the worker-side apply
        ctx.bind_tensors(x=[t_.t for t_ in xs2])
        ctx.aggregate(packed, wire)
        ctx.apply_delta_tensors(wire)
        ctx.bind_tensors(x=[t_.t for t_ in xs])
        torch.cuda.synchronize()
        orc.worker_step_ex(w.segments, D, n, inputs.as_numpy_grads(g_cpu), m_ref, p_ref, [w.beta1] * n, [w.beta2] * n)
        orc.aggregate_apply(w.segments, D, n, mode, p_ref, x_ref, w.lr, w.weight_decay, delta_bits=d_ref)
        gp.compare(f"step {t} packed", packed.cpu().numpy().view(np.uint32), p_ref, True)
        gp.compare(f"step {t} delta bits", dbits.cpu().numpy().view(np.uint32), d_ref, True)
        for k, (o, cnt) in enumerate(w.segments):
            gp.compare(f"step {t} x[{k}]", xs[k].t.cpu().numpy(), x_ref[o:o + cnt], True)
            gp.compare(f"step {t} x2[{k}]", xs2[k].t.cpu().numpy(), x_ref[o:o + cnt], True)
            for i in range(n):
                got = ms[i][k].t.cpu()
                got = got.numpy() if state == "f32" else got.view(torch.int16).numpy().view(np.uint16)
                gp.compare(f"step {t} m[{i}][{k}]", got, m_ref[i, o:o + cnt], True)
        assert all(t_.intact() for row in gs for t_ in row)
    assert all(t_.intact() for t_ in xs + xs2) and all(t_.intact() for row in ms for t_ in row)
    ctx.destroy()


def test_bind_rejects_bad_tables(dl):
    dev = torch.device("cuda:0")
    w = inputs.custom([100, 0, 50], 2, MAJ, "f32")
    ctx = gp.make_ctx(dl, w)
    good = [torch.zeros(100, device=dev), None, torch.zeros(50, device=dev)]
    ctx.bind_tensors(x=good)
    with pytest.raises(ValueError):
        ctx.bind_tensors(x=[torch.zeros(99, device=dev), None, torch.zeros(50, device=dev)])     # too short
    with pytest.raises(ValueError):
        ctx.bind_tensors(x=good[:2])                                                              # a tensor missing
    with pytest.raises(ValueError):
        ctx.bind_tensors(grads=[good])                                                            # one worker of two
    off = torch.zeros(104, device=dev)[1:101]                                                     # 4-byte aligned only
    with pytest.raises(dl.DlionError) as e:
        ctx.bind_tensors(x=[off, None, good[2]])
    assert e.value.status == dl.EALIGN
    with pytest.raises(dl.DlionError) as e:
        ctx.bind_tensors()
    assert e.value.status == dl.EINVAL
    packed = torch.zeros(2, w.d_pad // 32, dtype=torch.int32, device=dev)
    with pytest.raises(dl.DlionError) as e:                        # parameters bound, gradients and momenta not
        ctx.worker_step_tensors(-1, packed)
    assert e.value.status == dl.ESTATE
    ctx.destroy()
