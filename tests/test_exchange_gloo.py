"""The one-worker-per-process exchange (all-to-all of bit shards, vote on the local slice,
all-gather of the broadcast message, apply) on 2, 3 and 4 CPU ranks over gloo.  The three
local steps are played by the CPU checker, so this tests the orchestration: shard layout,
plane reordering, and that every rank ends with the x of the single-process N-worker step."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2404_00438_b200 import exchange, inputs


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class OracleKernels:
    """Stand-in for the CUDA library on CPU ranks (test infrastructure)."""

    def __init__(self, segments, d_pad_x, world, w, mode):
        from oracle import dlion_oracle as orc
        self.orc, self.segments, self.d, self.world, self.w, self.mode = orc, segments, d_pad_x, world, w, mode
        self.slice_len = d_pad_x // world

    def worker_step(self, g, m, packed):
        p = np.zeros((1, self.d // 32), np.uint32)
        mm = m.numpy().reshape(1, -1)
        self.orc.worker_step(self.segments, self.d, 1, g.numpy().reshape(1, -1), mm, p, self.w.beta1, self.w.beta2)
        packed.copy_(torch.from_numpy(p[0].view(np.int32)))

    def aggregate(self, packed_slices, wire_slice):
        k = wire_slice.shape[0]
        wire = np.zeros(k * self.slice_len // 32, np.uint32)
        self.orc.aggregate([(0, self.slice_len)], self.slice_len, self.world, self.mode,
                           np.ascontiguousarray(packed_slices.numpy().view(np.uint32)), wire)
        wire_slice.copy_(torch.from_numpy(wire.view(np.int32)).view(k, -1))

    def delta_planes(self):
        return self.orc.delta_planes(self.world, self.mode)

    def apply_delta_sliced(self, gathered, slice_words, x):
        # [slice][plane][word] -> the plane-major message of the oracle's apply
        wire = np.ascontiguousarray(gathered.numpy().view(np.uint32).transpose(1, 0, 2)).reshape(-1)
        self.orc.apply_delta(self.segments, self.d, self.world, self.mode, wire, x.numpy(),
                             self.w.lr, self.w.weight_decay)


def _worker(rank, world, port, mode, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import dlion_oracle as orc
        w = inputs.custom([5000, 77, 4096, 12289, 1], world, mode, "f32", lr=1e-2, weight_decay=0.5)
        d_x = exchange.padded_length(w.d_pad, world)
        opt = exchange.DistributedLion(w.segments, w.d_pad, mode, kernels=OracleKernels(w.segments, d_x, world, w, mode),
                                       device=torch.device("cpu"))
        assert opt.d_pad_x == d_x and opt.k == orc.delta_planes(world, mode)
        x = torch.zeros(d_x)
        x[:w.d_pad] = inputs.fill_x0(w, torch.empty(w.d_pad))
        x_ref = x.numpy().copy()
        m = torch.zeros(d_x)
        m_ref = np.zeros((world, d_x), np.float32)
        for t in range(3):
            g_all = torch.zeros(world, d_x)
            g_all[:, :w.d_pad] = inputs.fill_grads(w, t, torch.empty(world, w.d_pad))
            opt.step(g_all[rank].clone(), m, x)
            # the single-process N-worker step on the same inputs
            packed = np.zeros((world, d_x // 32), np.uint32)
            orc.worker_step(w.segments, d_x, world, g_all.numpy(), m_ref, packed, w.beta1, w.beta2)
            orc.aggregate_apply(w.segments, d_x, world, mode, packed, x_ref, w.lr, w.weight_decay)
            assert np.array_equal(x.numpy(), x_ref), f"rank {rank} step {t}: x differs"
            assert np.array_equal(m.numpy(), m_ref[rank])
            assert np.array_equal(opt.packed.numpy().view(np.uint32), packed[rank])
        sent, received = opt.wire_bytes_per_step()
        assert sent == (world - 1) * d_x // world // 8 and received == opt.k * sent
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,mode", [(2, 0), (2, 1), (3, 0), (4, 1), (2, 2), (4, 2)])
def test_exchange_equals_single_process_step(world, mode, tmp_path, oracle):
    mp.spawn(_worker, args=(world, _free_port(), mode, str(tmp_path)), nprocs=world, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))
