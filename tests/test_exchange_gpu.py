"""The exchange path on one GPU: a one-rank NCCL group drives DlionKernels (the three C-ABI
calls) and the two collectives end to end; the result must equal the single-process step and
the oracle.  (More than one GPU is not available to these tests; the multi-rank layout is
covered on CPU ranks in test_exchange_gloo.py.)"""
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

from paper_2404_00438_b200 import exchange, inputs
from tests import gpu_parity as gp

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", [inputs.MAJORITY, inputs.AVERAGE])
def test_single_rank_exchange_matches_oracle(mode):
    assert torch.cuda.is_available()
    from paper_2404_00438_b200 import build
    build.build()
    from oracle import dlion_oracle as orc
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1, device_id=dev)
    try:
        w = inputs.custom([70000, 333, 4097], 1, mode, "bf16", scale=1e-3, lr=1e-3, weight_decay=1.0)
        opt = exchange.DistributedLion(w.segments, w.d_pad, mode, beta1=w.beta1, beta2=w.beta2, lr=w.lr,
                                       weight_decay=w.weight_decay, gdtype=1)
        D = opt.d_pad_x
        assert D == w.d_pad
        x0 = inputs.fill_x0(w, torch.empty(D))
        x, m = x0.to(dev), torch.zeros(D, device=dev)
        x_ref, m_ref = x0.numpy().copy(), np.zeros((1, D), np.float32)
        for t in range(3):
            g = inputs.fill_grads(w, t, torch.empty(1, D, dtype=torch.bfloat16))
            opt.step(g[0].to(dev), m, x)
            torch.cuda.synchronize()
            packed = np.zeros((1, D // 32), np.uint32)
            orc.worker_step(w.segments, D, 1, inputs.as_numpy_grads(g), m_ref, packed, w.beta1, w.beta2)
            orc.aggregate_apply(w.segments, D, 1, mode, packed, x_ref, w.lr, w.weight_decay)
            gp.compare("packed", opt.packed.cpu().numpy().view(np.uint32), packed[0], True)
            assert gp.compare("m", m.cpu().numpy(), m_ref[0], False) == 0
            assert gp.compare("x", x.cpu().numpy(), x_ref, False) == 0
    finally:
        dist.destroy_process_group()


def test_optimizer_wrapper_trains_a_small_model_like_the_oracle():
    """Parameters re-pointed at the flat arena, gradients accumulated by autograd straight into
    the gradient arena, three steps; the arena must equal the oracle's x on the same gradients."""
    from paper_2404_00438_b200 import build
    build.build()
    from oracle import dlion_oracle as orc
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1, device_id=dev)
    try:
        torch.manual_seed(0)
        model = torch.nn.Sequential(torch.nn.Linear(37, 64), torch.nn.Tanh(), torch.nn.Linear(64, 5)).to(dev)
        opt = exchange.LionOptimizer(model.parameters(), lr=1e-2, betas=(0.9, 0.99), weight_decay=0.1, mode=0)
        D = opt.core.d_pad_x
        x_ref = opt.x.cpu().numpy().copy()
        m_ref = np.zeros((1, D), np.float32)
        data = torch.randn(16, 37, device=dev)
        target = torch.randn(16, 5, device=dev)
        for t in range(3):
            opt.zero_grad()
            loss = torch.nn.functional.mse_loss(model(data), target)
            loss.backward()
            g = opt.g.cpu().numpy().reshape(1, D).copy()
            assert np.abs(g).max() > 0
            opt.step()
            torch.cuda.synchronize()
            packed = np.zeros((1, D // 32), np.uint32)
            orc.worker_step(opt.segments, D, 1, g, m_ref, packed, 0.9, 0.99)
            orc.aggregate_apply(opt.segments, D, 1, 0, packed, x_ref, 1e-2, 0.1)
            assert gp.compare("x", opt.x.cpu().numpy(), x_ref, False) == 0
            flat = torch.cat([p.detach().reshape(-1) for p in model.parameters()]).cpu().numpy()
            want = np.concatenate([x_ref[o:o + k] for o, k in opt.segments])
            assert np.array_equal(flat, want)                   # the model really sees the arena
    finally:
        dist.destroy_process_group()


def test_in_place_optimizer_steps_the_models_own_tensors():
    """in_place=True: parameters and gradients stay where torch allocated them (gradients are
    even re-allocated every step) and are stepped through the per-tensor pointer tables; the
    parameters must equal the oracle's x on the same gradients, tensor by tensor."""
    from paper_2404_00438_b200 import build
    build.build()
    from oracle import dlion_oracle as orc
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1, device_id=dev)
    try:
        torch.manual_seed(1)
        model = torch.nn.Sequential(torch.nn.Linear(37, 64), torch.nn.Tanh(), torch.nn.Linear(64, 5000),
                                    torch.nn.Tanh(), torch.nn.Linear(5000, 3)).to(dev)
        params = list(model.parameters())
        ptrs = [p.data_ptr() for p in params]
        opt = exchange.LionOptimizer(params, lr=1e-2, betas=(0.9, 0.99), weight_decay=0.1, mode=1, in_place=True)
        D = opt.core.d_pad_x
        x_ref = np.zeros(D, np.float32)
        for p, (o, k) in zip(params, opt.segments):
            x_ref[o:o + k] = p.detach().reshape(-1).cpu().numpy()
        m_ref = np.zeros((1, D), np.float32)
        data = torch.randn(16, 37, device=dev)
        target = torch.randn(16, 3, device=dev)
        for t in range(3):
            opt.zero_grad(set_to_none=True)
            torch.nn.functional.mse_loss(model(data), target).backward()
            g = np.zeros((1, D), np.float32)
            for p, (o, k) in zip(params, opt.segments):
                g[0, o:o + k] = p.grad.reshape(-1).cpu().numpy()
            opt.step()
            torch.cuda.synchronize()
            packed = np.zeros((1, D // 32), np.uint32)
            orc.worker_step(opt.segments, D, 1, g, m_ref, packed, 0.9, 0.99)
            orc.aggregate_apply(opt.segments, D, 1, 1, packed, x_ref, 1e-2, 0.1)
            for p, (o, k) in zip(params, opt.segments):
                assert np.array_equal(p.detach().reshape(-1).cpu().numpy(), x_ref[o:o + k])
            assert gp.compare("m", opt.m.cpu().numpy(), m_ref[0], False) == 0
        assert [p.data_ptr() for p in params] == ptrs            # nothing was moved
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("mode", [inputs.MAJORITY, inputs.AVERAGE])
def test_fused_send_with_one_rank_matches_oracle(mode):
    """fused_send=True (receive buffer in symmetric memory, sign words stored by the
    worker-side kernel, barrier instead of the all-to-all) through a one-rank NCCL group.
    Skipped where this torch build cannot set up symmetric memory on the box."""
    from paper_2404_00438_b200 import build
    build.build()
    from oracle import dlion_oracle as orc
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1, device_id=dev)
    try:
        w = inputs.custom([70000, 333, 4097], 1, mode, "bf16", scale=1e-3, lr=1e-3, weight_decay=1.0)
        try:
            opt = exchange.DistributedLion(w.segments, w.d_pad, mode, beta1=w.beta1, beta2=w.beta2, lr=w.lr,
                                           weight_decay=w.weight_decay, gdtype=1, fused_send=True)
        except (ImportError, RuntimeError, AttributeError) as e:
            pytest.skip(f"symmetric memory is not available here: {e}")
        D = opt.d_pad_x
        x0 = inputs.fill_x0(w, torch.empty(D))
        x, m = x0.to(dev), torch.zeros(D, device=dev)
        x_ref, m_ref = x0.numpy().copy(), np.zeros((1, D), np.float32)
        for t in range(3):
            g = inputs.fill_grads(w, t, torch.empty(1, D, dtype=torch.bfloat16))
            opt.step(g[0].to(dev), m, x)
            torch.cuda.synchronize()
            packed = np.zeros((1, D // 32), np.uint32)
            orc.worker_step(w.segments, D, 1, inputs.as_numpy_grads(g), m_ref, packed, w.beta1, w.beta2)
            orc.aggregate_apply(w.segments, D, 1, mode, packed, x_ref, w.lr, w.weight_decay)
            gp.compare("receive buffer", opt.recv.cpu().numpy().view(np.uint32), packed, True)
            assert gp.compare("m", m.cpu().numpy(), m_ref[0], False) == 0
            assert gp.compare("x", x.cpu().numpy(), x_ref, False) == 0
    finally:
        dist.destroy_process_group()
