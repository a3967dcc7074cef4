"""Host-side checks of the C ABI that need no GPU: the library loads, exports
every symbol the header declares, and rejects malformed arguments before it
touches CUDA."""
import ctypes
import os
import re

import pytest
import torch

from paper_2404_00438_b200 import build as dl_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def dl():
    dl_build.build()
    from paper_2404_00438_b200 import dlion
    return dlion


def test_exports_match_header(dl):
    header = open(os.path.join(ROOT, "include", "dlion.h")).read()
    declared = set(re.findall(r"\b(dlion_[a-z0-9_]+)\s*\(", header))
    assert declared == set(dl.EXPORTS)
    raw = ctypes.CDLL(dl_build.LIB)
    for name in declared:
        assert hasattr(raw, name), f"{name} is declared in dlion.h but not exported"


def test_header_constants_match_binding(dl):
    header = open(os.path.join(ROOT, "include", "dlion.h")).read()
    assert int(re.search(r"#define DLION_ALIGN (\d+)u", header).group(1)) == dl.ALIGN
    assert int(re.search(r"#define DLION_MAX_WORKERS (\d+)u", header).group(1)) == dl.MAX_WORKERS


def test_check_layout(dl):
    assert dl.check_layout([(0, 100)], 128) == dl.OK
    assert dl.check_layout([(0, 128), (128, 5), (256, 0), (256, 256)], 512) == dl.OK
    assert dl.check_layout([], 128) == dl.EINVAL
    assert dl.check_layout([(0, 100)], 0) == dl.EINVAL
    assert dl.check_layout([(0, 100)], 100) == dl.EALIGN            # d_pad not a multiple of 128
    assert dl.check_layout([(64, 10)], 128) == dl.EALIGN            # offset not a multiple of 128
    assert dl.check_layout([(0, 200), (128, 10)], 512) == dl.EINVAL  # overlap
    assert dl.check_layout([(256, 10), (0, 10)], 512) == dl.EINVAL   # not ascending
    assert dl.check_layout([(0, 129)], 128) == dl.EINVAL            # runs past d_pad
    assert dl.check_layout([(128, 2 ** 64 - 1)], 256) == dl.EINVAL  # no wrap-around
    assert dl.lib().dlion_check_layout(None, 1, 128) == dl.EINVAL


@pytest.mark.parametrize("kw", [
    dict(n_workers=0), dict(n_workers=65536), dict(beta1=-0.1), dict(beta1=1.5), dict(beta2=float("nan")),
    dict(lr=-1.0), dict(lr=float("inf")), dict(weight_decay=-0.5), dict(mode=3), dict(gdtype=7),
])
def test_init_rejects_bad_arguments_before_cuda(dl, kw):
    args = dict(n_workers=4, beta1=0.9, beta2=0.99, lr=1e-4, weight_decay=0.1, mode=0, gdtype=0)
    args.update(kw)
    with pytest.raises(dl.DlionError) as e:
        dl.Dlion([(0, 100)], 128, **args)
    assert e.value.status == dl.EINVAL


def test_init_null_out_and_null_context_calls(dl):
    raw = dl.lib()
    seg = (dl.Segment * 1)()
    seg[0].numel = 10
    assert raw.dlion_init(None, seg, 1, 128, 1, 0.9, 0.99, 1e-4, 0.0, 0, 0) == dl.EINVAL
    assert raw.dlion_set_lr(None, 0.1) == dl.EINVAL
    assert raw.dlion_worker_step(None, 0, None, None, None, None) == dl.EINVAL
    assert raw.dlion_aggregate_apply(None, None, None, None, None, None) == dl.EINVAL
    assert raw.dlion_step_fused(None, None, None, None, None, None) == dl.EINVAL
    assert raw.dlion_step_host(None, None, None, None, None, None, None, None, None) == dl.EINVAL
    assert raw.dlion_wire_bytes(None, 0) == 0
    assert raw.dlion_launch_count(None) == 0
    raw.dlion_destroy(None)
    assert dl.status_str(dl.OK) == "ok" and "unknown" in dl.status_str(99)


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful on a machine without a GPU")
def test_no_gpu_means_an_error_not_a_fallback(dl):
    with pytest.raises(dl.DlionError) as e:
        dl.Dlion([(0, 100)], 128, 4)
    assert e.value.status == dl.ECUDA


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    import importlib
    import sys
    monkeypatch.setattr(dl_build, "LIB", str(tmp_path / "libdlion.so"))
    saved = sys.modules.pop("paper_2404_00438_b200.dlion", None)
    try:
        with pytest.raises(ImportError):
            importlib.import_module("paper_2404_00438_b200.dlion")
    finally:
        sys.modules.pop("paper_2404_00438_b200.dlion", None)
        if saved is not None:
            sys.modules["paper_2404_00438_b200.dlion"] = saved
