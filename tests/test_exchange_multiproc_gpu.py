"""The worker = process exchange with the CUDA kernels at world > 1: 2, 3 and 4 processes
share cuda:0, each is one worker (its own momentum, its own gradients), the three local
steps run through the C ABI on the GPU, and the two collectives run over gloo through
pinned host buffers (NCCL does not accept two ranks on one device).  No kernel waits on
another process: the ranks meet only in the host-side collectives.  Every rank must end
each step with the x, its own momentum and its own sign words of the oracle's
single-process N-worker step, bit for bit."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2404_00438_b200 import exchange, inputs

pytestmark = pytest.mark.gpu


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, mode, gd, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    torch.cuda.set_device(0)
    dev = torch.device("cuda:0")
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import dlion_oracle as orc
        w = inputs.custom([5000, 77, 3 * 4096, 12289, 1, 40000], world, mode, gd,
                          scale=1.0 if gd == "f32" else 1e-3, lr=1e-2, weight_decay=0.5)
        gdt = inputs.grad_torch_dtype(w)
        opt = exchange.DistributedLion(w.segments, w.d_pad, mode, beta1=w.beta1, beta2=w.beta2, lr=w.lr,
                                       weight_decay=w.weight_decay, gdtype=0 if gd == "f32" else 1,
                                       device=dev, host_staged=True)
        d_x = opt.d_pad_x
        assert opt.k == orc.delta_planes(world, mode)
        x0 = torch.zeros(d_x)
        x0[:w.d_pad] = inputs.fill_x0(w, torch.empty(w.d_pad))
        x, m = x0.to(dev), torch.zeros(d_x, device=dev)
        x_ref, m_ref = x0.numpy().copy(), np.zeros((world, d_x), np.float32)
        for t in range(4):
            g_all = torch.zeros(world, d_x, dtype=gdt)
            g_all[:, :w.d_pad] = inputs.fill_grads(w, t, torch.empty(world, w.d_pad, dtype=gdt))
            opt.step(g_all[rank].to(dev), m, x)
            torch.cuda.synchronize()
            packed = np.zeros((world, d_x // 32), np.uint32)          # the single-process N-worker step
            orc.worker_step(w.segments, d_x, world, inputs.as_numpy_grads(g_all), m_ref, packed, w.beta1, w.beta2)
            orc.aggregate_apply(w.segments, d_x, world, mode, packed, x_ref, w.lr, w.weight_decay)
            assert np.array_equal(opt.packed.cpu().numpy().view(np.uint32), packed[rank]), f"rank {rank} step {t}: signs"
            assert np.array_equal(m.cpu().numpy(), m_ref[rank]), f"rank {rank} step {t}: momentum"
            assert np.array_equal(x.cpu().numpy(), x_ref), f"rank {rank} step {t}: x"
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,mode,gd", [(2, 0, "f32"), (2, 1, "bf16"), (3, 1, "f32"), (4, 0, "bf16"), (4, 1, "f32"), (2, 2, "f32")])
def test_processes_sharing_one_gpu_equal_the_oracle(world, mode, gd, tmp_path):
    assert torch.cuda.is_available()
    from paper_2404_00438_b200 import build
    from oracle import dlion_oracle
    build.build()
    dlion_oracle.build()
    mp.spawn(_rank, args=(world, _free_port(), mode, gd, str(tmp_path)), nprocs=world, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))
