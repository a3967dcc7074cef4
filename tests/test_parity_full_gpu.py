"""Full-size parity: the five workload configurations in the launch configuration
the benchmark times.  The oracle recomputes sampled coordinate slabs (both ends,
segment joints, random interiors) from the same gradient bytes; coordinates are
independent, so a slab is a complete problem."""
import pytest
import torch

from paper_2404_00438_b200 import inputs
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


def _free():
    torch.cuda.synchronize()
    torch.cuda.empty_cache()


def test_c2_gpt2_small_table(dl):
    assert gp.run_full(dl, inputs.workload("c2"), 10) == 0
    _free()
    assert gp.run_full(dl, inputs.workload("c2"), 3, "fused", modes=(AVG,)) == 0
    _free()


def test_c3_vit_b16_table(dl):
    assert gp.run_full(dl, inputs.workload("c3"), 10) == 0
    _free()
    assert gp.run_full(dl, inputs.workload("c3"), 3, "fused", modes=(MAJ,)) == 0
    _free()


@pytest.mark.parametrize("n", [2, 4, 8, 16, 32, 64, 128])
def test_c4_worker_sweep(dl, n):
    steps = 10 if n <= 8 else 3
    assert gp.run_full(dl, inputs.workload("c4", n_workers=n), steps) == 0
    _free()


def test_c5_decoder_1p3b(dl):
    assert gp.run_full(dl, inputs.workload("c5"), 10) == 0
    _free()
    assert gp.run_full(dl, inputs.workload("c5"), 2, "fused", modes=(MAJ,)) == 0
    _free()
