"""Scatter mode: the worker-side kernel stores its sign words straight into one receive buffer
per coordinate slice (the all-to-all of the worker = GPU exchange fused into the kernel).  The
S ranks are emulated on one GPU as S sets of buffers -- no kernel waits on another, the launches
simply run one after the other -- and the whole exchange (scatter, vote on each slice, apply
from the gathered message) must reproduce the oracle's S-worker step bit for bit."""
import numpy as np
import pytest
import torch

from paper_2404_00438_b200 import exchange, inputs
from tests import gpu_parity as gp

pytestmark = pytest.mark.gpu
MAJ, AVG = inputs.MAJORITY, inputs.AVERAGE


@pytest.fixture(scope="module")
def dl():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2404_00438_b200 import build
    build.build()
    from paper_2404_00438_b200 import dlion
    return dlion


@pytest.mark.parametrize("world,mode,gd,state", [(2, MAJ, "f32", "f32"), (3, AVG, "bf16", "f32"), (4, MAJ, "bf16", "bf16"),
                                                 (8, AVG, "f32", "f32"), (5, MAJ, "f32", "bf16")])
def test_scattered_signs_complete_the_exchange(dl, world, mode, gd, state):
    from oracle import dlion_oracle as orc
    dev = torch.device("cuda:0")
    w = inputs.custom([5000, 77, 3 * 4096, 12289, 1, 40000, 8 * 4096 + 3], world, mode, gd,
                      scale=1.0 if gd == "f32" else 1e-3, lr=1e-2, weight_decay=0.5)
    D = exchange.padded_length(w.d_pad, world)
    W, SW = D // 32, D // 32 // world
    gdt = inputs.grad_torch_dtype(w)
    sdt = torch.float32 if state == "f32" else torch.bfloat16
    model = dl.Dlion(w.segments, D, world, w.beta1, w.beta2, w.lr, w.weight_decay, mode, gp.gdtype_of(w))
    server = dl.Dlion([(0, D // world)], D // world, world, w.beta1, w.beta2, w.lr, w.weight_decay, mode, gp.gdtype_of(w))
    if state == "bf16":
        model.set_momentum_dtype(dl.STATE_BF16)
    K = model.delta_planes()
    # rank q's receive buffer, each inside its own allocation between two bands of a sentinel value
    GUARD, SENTINEL = 256, 0x5A5A5A5A
    backing = [torch.full((world * SW + 2 * GUARD,), SENTINEL, dtype=torch.int32, device=dev) for _ in range(world)]
    recv = [b[GUARD:GUARD + world * SW].view(world, SW) for b in backing]
    for r_ in recv:
        r_.zero_()
    gathered = torch.zeros(world, K, SW, dtype=torch.int32, device=dev)
    x0 = torch.zeros(D)
    x0[:w.d_pad] = inputs.fill_x0(w, torch.empty(w.d_pad))
    x = x0.to(dev)
    m = torch.zeros(world, D, dtype=sdt, device=dev)
    x_ref = x0.numpy().copy()
    m_ref = np.zeros((world, D), np.float32 if state == "f32" else np.uint16)
    p_ref = np.zeros((world, W), np.uint32)
    for t in range(3):
        g_cpu = torch.zeros(world, D, dtype=gdt)
        g_cpu[:, :w.d_pad] = inputs.fill_grads(w, t, torch.empty(world, w.d_pad, dtype=gdt))
        g = g_cpu.to(dev)
        for r in range(world):                        # "rank" r: its own worker, its own slot in every buffer
            model.bind_scatter(recv, SW, slot=r, rows=world)
            model.worker_step_scatter(r, g[r], m[r])
        for q in range(world):                        # "rank" q votes on its slice
            server.aggregate(recv[q], gathered[q])
        model.apply_delta_sliced(gathered, SW, x)
        torch.cuda.synchronize()
        orc.worker_step_ex(w.segments, D, world, inputs.as_numpy_grads(g_cpu), m_ref, p_ref,
                           [w.beta1] * world, [w.beta2] * world)
        orc.aggregate_apply(w.segments, D, world, mode, p_ref, x_ref, w.lr, w.weight_decay)
        for q in range(world):
            gp.compare(f"step {t} receive buffer {q}", recv[q].cpu().numpy().view(np.uint32),
                       p_ref[:, q * SW:(q + 1) * SW], True)
        got_m = m.cpu()
        got_m = got_m.numpy() if state == "f32" else got_m.view(torch.int16).numpy().view(np.uint16)
        gp.compare(f"step {t} m", got_m, m_ref, True)
        gp.compare(f"step {t} x", x.cpu().numpy(), x_ref, True)
    for b in backing:                                   # nothing was stored outside a receive buffer
        assert bool((b[:GUARD] == SENTINEL).all()) and bool((b[GUARD + world * SW:] == SENTINEL).all())
    # argument checks
    with pytest.raises(dl.DlionError) as e:
        model.bind_scatter(recv[:-1], SW, 0, world)                    # slices do not cover the arena
    assert e.value.status == dl.EINVAL
    with pytest.raises(dl.DlionError) as e:
        model.bind_scatter(recv, SW, world, world)                     # slot out of range
    assert e.value.status == dl.EINVAL
    fresh = dl.Dlion(w.segments, D, world, w.beta1, w.beta2, w.lr, w.weight_decay, mode, gp.gdtype_of(w))
    with pytest.raises(dl.DlionError) as e:
        fresh.worker_step_scatter(0, g[0], torch.zeros(D, device=dev))
    assert e.value.status == dl.ESTATE
    for c in (model, server, fresh):
        c.destroy()
