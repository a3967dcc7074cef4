"""The Python binding turns tensors into raw addresses, and the C ABI can only check
alignment; so the binding itself must refuse, before any launch, whatever would make a
kernel read or write out of bounds: tensors that are not on the GPU, strided views, wrong
element types, buffers shorter than the call's extent.  These checks need no GPU."""
import pytest
import torch

from paper_2404_00438_b200 import dlion


def test_host_tensor_is_refused_where_a_device_tensor_is_needed():
    with pytest.raises(ValueError, match="CUDA tensor"):
        dlion.check_tensor(torch.zeros(256), "x", (torch.float32,), 256, 0)


def test_host_memory_is_accepted_for_host_arguments():
    dlion.check_tensor(torch.zeros(4), "host_grads", (torch.float32,), 4, None, host=True)


def test_short_strided_and_mistyped_tensors_are_refused():
    ok = torch.zeros(8, 256)
    with pytest.raises(ValueError, match="elements"):
        dlion.check_tensor(ok, "g", (torch.float32,), 8 * 256 + 1, None, host=True)
    with pytest.raises(ValueError, match="contiguous"):
        dlion.check_tensor(ok[:, 10:138], "packed", (torch.float32,), 8, None, host=True)
    with pytest.raises(ValueError, match="dtype"):
        dlion.check_tensor(ok, "g", (torch.bfloat16,), 8, None, host=True)
    with pytest.raises(ValueError, match="required"):
        dlion.check_tensor(None, "x", (torch.float32,), 8, None, host=True)
    with pytest.raises(ValueError, match="torch.Tensor"):
        dlion.check_tensor([1.0, 2.0], "x", (torch.float32,), 2, None, host=True)
    dlion.check_tensor(None, "count_out", (torch.uint8,), 8, None, optional=True)   # nullable outputs may be absent
    dlion.check_tensor(ok, "g", (torch.float32,), 8 * 256, None, host=True)


def test_step_static_validates_before_calling_the_library():
    cpu = torch.zeros(1024)
    with pytest.raises(ValueError):                        # host tensors never reach the C call
        dlion.step_static(1024, 1, 0.9, 0.99, 1e-4, 0.0, dlion.MAJORITY, dlion.GRAD_F32, cpu, cpu, cpu)
    with pytest.raises(ValueError):
        dlion.step_static(1024, 1, 0.9, 0.99, 1e-4, 0.0, dlion.MAJORITY, dlion.GRAD_F32, None, cpu, cpu)


class _FakeCtx(dlion.Dlion):
    """A Dlion whose C context is never created: only the Python-side checks run."""

    def __init__(self, d_pad, n, gdtype=dlion.GRAD_F32, device_index=0):
        import ctypes
        self._ctx = ctypes.c_void_p()
        self.d_pad, self.n_workers, self.mode, self.gdtype = d_pad, n, dlion.MAJORITY, gdtype
        self.sdtype, self.words, self.device_index = dlion.STATE_F32, d_pad // 32, device_index

    def delta_planes(self):
        return 1


@pytest.mark.parametrize("call", ["worker_all", "worker_one", "aggregate_apply", "aggregate", "apply_delta",
                                  "step_fused", "step_host"])
def test_every_launching_method_checks_its_tensors_first(call):
    """With host tensors every launching method must raise ValueError (the null context
    would otherwise be handed to the library)."""
    n, d = 4, 1024
    c = _FakeCtx(d, n)
    g, m, x = torch.zeros(n, d), torch.zeros(n, d), torch.zeros(d)
    packed, wire = torch.zeros(n, d // 32, dtype=torch.int32), torch.zeros(d // 32, dtype=torch.int32)
    with pytest.raises(ValueError):
        {"worker_all": lambda: c.worker_step(-1, g, m, packed),
         "worker_one": lambda: c.worker_step(1, g[1], m[1], packed[1]),
         "aggregate_apply": lambda: c.aggregate_apply(packed, x),
         "aggregate": lambda: c.aggregate(packed, wire),
         "apply_delta": lambda: c.apply_delta(wire, x),
         "step_fused": lambda: c.step_fused(g, m, x),
         "step_host": lambda: c.step_host(g, m, x, packed, torch.zeros(2, d))}[call]()
