"""Multi-process (gloo, world_size 2 and 3, CPU) check of the coordinate sharding:
every rank steps only its slab -- here with the CPU checker standing in for a GPU --
and the gathered slabs must equal the unsharded run bit for bit; the benchmark's
max-over-ranks timing reduction is exercised on the same process group."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2404_00438_b200 import inputs, shard


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _run_oracle(segs, d_pad, w, g_list, x0, mode):
    from oracle import dlion_oracle as orc
    m = np.zeros((w.n_workers, d_pad), np.float32)
    x = x0.copy()
    for g in g_list:
        packed = np.zeros((w.n_workers, d_pad // 32), np.uint32)
        orc.worker_step(segs, d_pad, w.n_workers, np.ascontiguousarray(g), m, packed, w.beta1, w.beta2)
        orc.aggregate_apply(segs, d_pad, w.n_workers, mode, packed, x, w.lr, w.weight_decay)
    return m, x


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = inputs.custom([5000, 77, 4096, 12289, 1], 3, inputs.AVERAGE, "f32", lr=1e-2, weight_decay=0.5)
        steps = 3
        full_g = [inputs.fill_grads(w, t, torch.empty(w.n_workers, w.d_pad)).numpy() for t in range(steps)]
        full_x0 = inputs.fill_x0(w, torch.empty(w.d_pad)).numpy()
        sh = shard.shard_segments(w.segments, rank, world)
        # gather this rank's slab of every arena
        g_loc = [np.zeros((w.n_workers, sh.d_pad), np.float32) for _ in range(steps)]
        x_loc = np.zeros(sh.d_pad, np.float32)
        for p in sh.pieces:
            for t in range(steps):
                g_loc[t][:, p.local_offset:p.local_offset + p.numel] = \
                    full_g[t][:, p.global_offset:p.global_offset + p.numel]
            x_loc[p.local_offset:p.local_offset + p.numel] = full_x0[p.global_offset:p.global_offset + p.numel]
        m_loc, x_new = _run_oracle(sh.segments, sh.d_pad, w, g_loc, x_loc, w.mode)
        # no data-path collective: the only exchange is this test's own gather of results
        mine = [(p.global_offset, p.numel, x_new[p.local_offset:p.local_offset + p.numel].copy(),
                 m_loc[:, p.local_offset:p.local_offset + p.numel].copy()) for p in sh.pieces]
        gathered = [None] * world
        dist.all_gather_object(gathered, mine)
        sizes = [None] * world
        dist.all_gather_object(sizes, sh.d)
        # the benchmark's timing reduction: max over ranks
        t = torch.tensor([float(rank + 1)], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert t.item() == float(world)
        if rank == 0:
            assert sum(sizes) == w.d
            assert max(sizes) - min(sizes) <= 2 * shard.ALIGN + max(n for n in w.numels if n < shard.ALIGN)
            m_ref, x_ref = _run_oracle(w.segments, w.d_pad, w, full_g, full_x0, w.mode)
            x_got = full_x0.copy()
            m_got = np.zeros_like(m_ref)
            covered = np.zeros(w.d_pad, np.int32)
            for pieces in gathered:
                for off, n, xs, ms in pieces:
                    assert off % shard.ALIGN == 0
                    x_got[off:off + n] = xs
                    m_got[:, off:off + n] = ms
                    covered[off:off + n] += 1
            valid = np.zeros(w.d_pad, bool)
            for off, n in w.segments:
                valid[off:off + n] = True
            assert np.array_equal(covered[valid], np.ones(valid.sum(), np.int32)) and not covered[~valid].any()
            assert np.array_equal(x_got, x_ref) and np.array_equal(m_got, m_ref)
            open(os.path.join(out_dir, "ok"), "w").write("ok")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_step_equals_unsharded(world, tmp_path, oracle):
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    assert (tmp_path / "ok").exists()


def test_shards_partition_the_model():
    for name in ("c2", "c3", "c5"):
        w = inputs.workload(name)
        for world in (1, 2, 4, 8):
            shards = [shard.shard_segments(w.segments, r, world) for r in range(world)]
            assert sum(s.d for s in shards) == w.d
            ideal = w.d / world
            assert all(abs(s.d - ideal) <= shard.ALIGN for s in shards)
            ends = 0
            for s in shards:
                for p in s.pieces:
                    assert p.global_offset % shard.ALIGN == 0 and p.local_offset % shard.ALIGN == 0
                    assert p.global_offset >= ends
                    ends = p.global_offset + p.numel
