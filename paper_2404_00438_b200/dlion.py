"""Thin binding over the C ABI declared in ``include/dlion.h`` (same names).

Argument marshalling only: tensors become device pointers, the current torch
stream becomes the ``cudaStream_t``; every step of the optimizer runs in the CUDA
library.  Importing this module loads ``libdlion.so`` and raises if it is
missing: there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import torch

from . import build as _build

MAJORITY, AVERAGE, MAJORITY_TERNARY = 0, 1, 2
GRAD_F32, GRAD_BF16 = 0, 1
STATE_F32, STATE_BF16 = 0, 1
ALIGN = 128
MAX_WORKERS = 65535
OK, EINVAL, EALIGN, ENOMEM, ECUDA, ESTATE = range(6)

EXPORTS = ("dlion_check_layout", "dlion_init", "dlion_set_lr", "dlion_set_momentum_dtype",
           "dlion_set_worker_betas", "dlion_worker_step",
           "dlion_aggregate_apply", "dlion_aggregate_apply_counts16", "dlion_aggregate", "dlion_apply_delta", "dlion_apply_delta_sliced",
           "dlion_delta_planes",
           "dlion_bind_tensors", "dlion_worker_step_tensors", "dlion_aggregate_apply_tensors",
           "dlion_apply_delta_tensors", "dlion_bind_scatter", "dlion_worker_step_scatter", "dlion_step_fused", "dlion_step_global", "dlion_step_host", "dlion_step_static",
           "dlion_wire_bytes",
           "dlion_launch_count", "dlion_status_str", "dlion_destroy")


class Segment(ctypes.Structure):
    _fields_ = [("elem_offset", ctypes.c_uint64), ("numel", ctypes.c_uint64)]


class DlionError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_str(status)} (status {status})")


def _load() -> ctypes.CDLL:
    if not os.path.exists(_build.LIB):
        raise ImportError(
            f"{_build.LIB} is missing: build it with `python -m paper_2404_00438_b200.build` "
            "(nvcc, sm_100a). This package has no CPU fallback.")
    lib = ctypes.CDLL(_build.LIB)
    vp, u32, u64, f32, i32 = (ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_float,
                              ctypes.c_int)
    seg_p = ctypes.POINTER(Segment)
    lib.dlion_check_layout.argtypes = [seg_p, u32, u64]
    lib.dlion_check_layout.restype = i32
    lib.dlion_init.argtypes = [ctypes.POINTER(vp), seg_p, u32, u64, u32, f32, f32, f32, f32, i32, i32]
    lib.dlion_init.restype = i32
    lib.dlion_set_lr.argtypes = [vp, f32]
    lib.dlion_set_lr.restype = i32
    lib.dlion_set_momentum_dtype.argtypes = [vp, i32]
    lib.dlion_set_momentum_dtype.restype = i32
    lib.dlion_set_worker_betas.argtypes = [vp, i32, f32, f32]
    lib.dlion_set_worker_betas.restype = i32
    lib.dlion_worker_step.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.dlion_worker_step.restype = i32
    lib.dlion_aggregate_apply.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.dlion_aggregate_apply.restype = i32
    lib.dlion_aggregate_apply_counts16.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.dlion_aggregate_apply_counts16.restype = i32
    lib.dlion_aggregate.argtypes = [vp, vp, vp, vp]
    lib.dlion_aggregate.restype = i32
    lib.dlion_apply_delta.argtypes = [vp, vp, vp, vp]
    lib.dlion_apply_delta.restype = i32
    lib.dlion_apply_delta_sliced.argtypes = [vp, vp, u64, vp, vp]
    lib.dlion_apply_delta_sliced.restype = i32
    lib.dlion_delta_planes.argtypes = [vp]
    lib.dlion_delta_planes.restype = u32
    lib.dlion_bind_tensors.argtypes = [vp, vp, vp, vp, vp]
    lib.dlion_bind_tensors.restype = i32
    lib.dlion_worker_step_tensors.argtypes = [vp, i32, vp, vp]
    lib.dlion_worker_step_tensors.restype = i32
    lib.dlion_aggregate_apply_tensors.argtypes = [vp, vp, vp, vp]
    lib.dlion_aggregate_apply_tensors.restype = i32
    lib.dlion_apply_delta_tensors.argtypes = [vp, vp, u64, vp]
    lib.dlion_apply_delta_tensors.restype = i32
    lib.dlion_bind_scatter.argtypes = [vp, vp, u32, u64, u32, u32]
    lib.dlion_bind_scatter.restype = i32
    lib.dlion_worker_step_scatter.argtypes = [vp, i32, vp, vp, vp]
    lib.dlion_worker_step_scatter.restype = i32
    lib.dlion_step_fused.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.dlion_step_fused.restype = i32
    lib.dlion_step_global.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.dlion_step_global.restype = i32
    lib.dlion_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.dlion_step_host.restype = i32
    lib.dlion_step_static.argtypes = [u64, u32, f32, f32, f32, f32, i32, i32, vp, vp, vp, vp]
    lib.dlion_step_static.restype = i32
    lib.dlion_wire_bytes.argtypes = [vp, i32]
    lib.dlion_wire_bytes.restype = u64
    lib.dlion_launch_count.argtypes = [vp]
    lib.dlion_launch_count.restype = u64
    lib.dlion_status_str.argtypes = [i32]
    lib.dlion_status_str.restype = ctypes.c_char_p
    lib.dlion_destroy.argtypes = [vp]
    lib.dlion_destroy.restype = None
    return lib


_lib = _load()


def lib() -> ctypes.CDLL:
    """The loaded C library (for callers that want the raw ABI)."""
    return _lib


def status_str(status: int) -> str:
    return _lib.dlion_status_str(int(status)).decode()


def _seg_array(segments: Sequence[Tuple[int, int]]):
    arr = (Segment * max(len(segments), 1))()
    for k, (off, n) in enumerate(segments):
        arr[k].elem_offset = int(off)
        arr[k].numel = int(n)
    return arr


def check_layout(segments: Sequence[Tuple[int, int]], d_pad: int) -> int:
    """``dlion_check_layout``: returns the status code (no exception)."""
    return int(_lib.dlion_check_layout(_seg_array(segments), len(segments), int(d_pad)))


STATIC_MAX_COORD_WORKERS = 134217728


def step_static(d: int, n_workers: int, beta1: float, beta2: float, lr: float, weight_decay: float,
                mode: int, gdtype: int, grads: torch.Tensor, m: torch.Tensor, x: torch.Tensor) -> None:
    """``dlion_step_static``: one two-stage step on a flat vector for callers that cannot
    allocate device memory (no context, no wire buffer: both live in a fixed array inside the
    library, shared by all calls on the device).  Raises DlionError when N * d_pad exceeds
    STATIC_MAX_COORD_WORKERS."""
    d_pad = (int(d) + ALIGN - 1) // ALIGN * ALIGN
    dev = torch.cuda.current_device() if torch.cuda.is_available() else None
    fits = 0 < int(n_workers) * d_pad <= STATIC_MAX_COORD_WORKERS      # else the library rejects the size itself
    check_tensor(grads, "grads", _GRAD_DTYPES.get(int(gdtype)), int(n_workers) * d_pad if fits else 0, dev)
    check_tensor(m, "m", (torch.float32,), int(n_workers) * d_pad if fits else 0, dev)
    check_tensor(x, "x", (torch.float32,), d_pad if fits else 0, dev)
    st = _lib.dlion_step_static(int(d), int(n_workers), beta1, beta2, lr, weight_decay, int(mode),
                                int(gdtype), _ptr(grads), _ptr(m), _ptr(x), _stream())
    if st != OK:
        raise DlionError(st, "dlion_step_static")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


_WORD_DTYPES = tuple(t for t in (torch.int32, getattr(torch, "uint32", None)) if t is not None)
_HALFWORD_DTYPES = tuple(t for t in (torch.int16, getattr(torch, "uint16", None)) if t is not None)
_GRAD_DTYPES = {GRAD_F32: (torch.float32,), GRAD_BF16: (torch.bfloat16,)}
_STATE_DTYPES = {STATE_F32: (torch.float32,), STATE_BF16: (torch.bfloat16,)}


def check_tensor(t: Optional[torch.Tensor], name: str, dtypes, min_numel: int,
                 device_index: Optional[int], optional: bool = False, host: bool = False) -> None:
    """Raises ValueError unless ``t`` can be handed to the C ABI as a raw pointer: on the
    context's GPU (or, with ``host``, in host memory), contiguous, of one of ``dtypes`` and
    holding at least ``min_numel`` elements.  The C side sees only an address, so a wrong
    size, a strided view or a tensor on another device would otherwise become an
    out-of-bounds access inside a kernel.  Nothing is launched when this raises."""
    if t is None:
        if optional:
            return
        raise ValueError(f"{name}: a tensor is required")
    if not isinstance(t, torch.Tensor):
        raise ValueError(f"{name}: expected a torch.Tensor, got {type(t).__name__}")
    if host:
        if t.is_cuda:
            raise ValueError(f"{name}: must be in host memory")
    else:
        if not t.is_cuda:
            raise ValueError(f"{name}: must be a CUDA tensor (the library has no CPU path)")
        if device_index is not None and t.device.index != device_index:
            raise ValueError(f"{name}: is on cuda:{t.device.index}, the context lives on cuda:{device_index}")
    if dtypes is not None and t.dtype not in dtypes:
        raise ValueError(f"{name}: dtype {t.dtype}, expected one of {tuple(dtypes)}")
    if not t.is_contiguous():
        raise ValueError(f"{name}: must be contiguous (got strides {tuple(t.stride())})")
    if t.numel() < min_numel:
        raise ValueError(f"{name}: {t.numel()} elements, the call reads or writes {min_numel}")


class Dlion:
    """Owner of one ``dlion_ctx``.  Methods mirror the C calls one to one."""

    def __init__(self, segments: Sequence[Tuple[int, int]], d_pad: int, n_workers: int,
                 beta1: float = 0.9, beta2: float = 0.99, lr: float = 1e-4,
                 weight_decay: float = 0.0, mode: int = MAJORITY, gdtype: int = GRAD_F32):
        self._ctx = ctypes.c_void_p()
        st = _lib.dlion_init(ctypes.byref(self._ctx), _seg_array(segments), len(segments), int(d_pad),
                             int(n_workers), beta1, beta2, lr, weight_decay, int(mode), int(gdtype))
        if st != OK:
            self._ctx = ctypes.c_void_p()
            raise DlionError(st, "dlion_init")
        self.d_pad, self.n_workers, self.mode, self.gdtype = int(d_pad), int(n_workers), int(mode), int(gdtype)
        self.sdtype = STATE_F32
        self.words = self.d_pad // 32
        self.numels = [int(n) for _, n in segments]
        self.device_index = torch.cuda.current_device()

    def _check(self, st: int, where: str) -> None:
        if st != OK:
            raise DlionError(st, where)

    def _t(self, t, name, dtypes, min_numel, optional=False, host=False) -> None:
        check_tensor(t, name, dtypes, min_numel, self.device_index, optional=optional, host=host)

    def set_lr(self, lr: float) -> None:
        self._check(_lib.dlion_set_lr(self._ctx, lr), "dlion_set_lr")

    def set_momentum_dtype(self, sdtype: int) -> None:
        self._check(_lib.dlion_set_momentum_dtype(self._ctx, int(sdtype)), "dlion_set_momentum_dtype")
        self.sdtype = int(sdtype)

    def set_worker_betas(self, worker: int, beta1: float, beta2: float) -> None:
        self._check(_lib.dlion_set_worker_betas(self._ctx, int(worker), beta1, beta2),
                    "dlion_set_worker_betas")

    def worker_step(self, worker: int, grads: torch.Tensor, m: torch.Tensor,
                    packed: torch.Tensor) -> None:
        k = self.n_workers if int(worker) < 0 else 1
        self._t(grads, "grads", _GRAD_DTYPES[self.gdtype], k * self.d_pad)
        self._t(m, "m", _STATE_DTYPES[self.sdtype], k * self.d_pad)
        self._t(packed, "packed", _WORD_DTYPES, k * self.words)
        self._check(_lib.dlion_worker_step(self._ctx, int(worker), _ptr(grads), _ptr(m), _ptr(packed),
                                           _stream()), "dlion_worker_step")

    def aggregate_apply(self, packed: torch.Tensor, x: torch.Tensor,
                        delta_bits_out: Optional[torch.Tensor] = None,
                        count_out: Optional[torch.Tensor] = None) -> None:
        self._t(packed, "packed", _WORD_DTYPES, self.n_workers * self.words)
        self._t(x, "x", (torch.float32,), self.d_pad)
        self._t(delta_bits_out, "delta_bits_out", _WORD_DTYPES, self.words, optional=True)
        self._t(count_out, "count_out", (torch.uint8,), self.d_pad, optional=True)
        self._check(_lib.dlion_aggregate_apply(self._ctx, _ptr(packed), _ptr(x), _ptr(delta_bits_out),
                                               _ptr(count_out), _stream()), "dlion_aggregate_apply")

    def aggregate_apply_counts16(self, packed: torch.Tensor, x: torch.Tensor,
                                 delta_bits_out: Optional[torch.Tensor], count16_out: torch.Tensor) -> None:
        self._t(packed, "packed", _WORD_DTYPES, self.n_workers * self.words)
        self._t(x, "x", (torch.float32,), self.d_pad)
        self._t(delta_bits_out, "delta_bits_out", _WORD_DTYPES, self.words, optional=True)
        self._t(count16_out, "count16_out", _HALFWORD_DTYPES, self.d_pad)
        self._check(_lib.dlion_aggregate_apply_counts16(self._ctx, _ptr(packed), _ptr(x), _ptr(delta_bits_out),
                                                        _ptr(count16_out), _stream()),
                    "dlion_aggregate_apply_counts16")

    def aggregate(self, packed: torch.Tensor, delta_wire: torch.Tensor) -> None:
        self._t(packed, "packed", _WORD_DTYPES, self.n_workers * self.words)
        self._t(delta_wire, "delta_wire", _WORD_DTYPES, self.delta_planes() * self.words)
        self._check(_lib.dlion_aggregate(self._ctx, _ptr(packed), _ptr(delta_wire), _stream()),
                    "dlion_aggregate")

    def apply_delta(self, delta_wire: torch.Tensor, x: torch.Tensor) -> None:
        self._t(delta_wire, "delta_wire", _WORD_DTYPES, self.delta_planes() * self.words)
        self._t(x, "x", (torch.float32,), self.d_pad)
        self._check(_lib.dlion_apply_delta(self._ctx, _ptr(delta_wire), _ptr(x), _stream()),
                    "dlion_apply_delta")

    def apply_delta_sliced(self, delta_wire: torch.Tensor, slice_words: int, x: torch.Tensor) -> None:
        self._t(delta_wire, "delta_wire", _WORD_DTYPES, self.delta_planes() * self.words)
        self._t(x, "x", (torch.float32,), self.d_pad)
        self._check(_lib.dlion_apply_delta_sliced(self._ctx, _ptr(delta_wire), int(slice_words), _ptr(x),
                                                  _stream()), "dlion_apply_delta_sliced")

    def delta_planes(self) -> int:
        return int(_lib.dlion_delta_planes(self._ctx))

    # ---- per-tensor mode: separately allocated tensors stepped in place
    def _ptr_table(self, rows, name: str, dtypes):
        """ctypes array of device pointers from a list (or list of lists) of tensors, each
        checked against its segment's size; the tensors are kept alive by the caller."""
        flat = [t for row in rows for t in row] if rows and isinstance(rows[0], (list, tuple)) else list(rows)
        nseg = len(self.numels)
        if len(flat) % nseg != 0:
            raise ValueError(f"{name}: {len(flat)} tensors for {nseg} segments")
        arr = (ctypes.c_void_p * len(flat))()
        for j, t in enumerate(flat):
            need = self.numels[j % nseg]
            if t is None and need == 0:
                arr[j] = None
                continue
            check_tensor(t, f"{name}[{j}]", dtypes, need, self.device_index)
            arr[j] = t.data_ptr()
        return arr, len(flat) // nseg

    def bind_tensors(self, grads=None, m=None, x=None) -> None:
        """``dlion_bind_tensors``: grads and m are [N][nseg] lists of tensors (or flat lists in
        that order), x an [nseg] list; None keeps the previous binding of that table."""
        arrs = []
        for rows, name, dtypes, want in ((grads, "grads", _GRAD_DTYPES[self.gdtype], self.n_workers),
                                         (m, "m", _STATE_DTYPES[self.sdtype], self.n_workers),
                                         (x, "x", (torch.float32,), 1)):
            if rows is None:
                arrs.append(None)
                continue
            arr, got = self._ptr_table(rows, name, dtypes)
            if got != want:
                raise ValueError(f"{name}: tensors for {got} workers, expected {want}")
            arrs.append(arr)
        self._check(_lib.dlion_bind_tensors(self._ctx, arrs[0], arrs[1], arrs[2], _stream()), "dlion_bind_tensors")

    def worker_step_tensors(self, worker: int, packed: torch.Tensor) -> None:
        k = self.n_workers if int(worker) < 0 else 1
        self._t(packed, "packed", _WORD_DTYPES, k * self.words)
        self._check(_lib.dlion_worker_step_tensors(self._ctx, int(worker), _ptr(packed), _stream()),
                    "dlion_worker_step_tensors")

    def aggregate_apply_tensors(self, packed: torch.Tensor, delta_bits_out: Optional[torch.Tensor] = None) -> None:
        self._t(packed, "packed", _WORD_DTYPES, self.n_workers * self.words)
        self._t(delta_bits_out, "delta_bits_out", _WORD_DTYPES, self.words, optional=True)
        self._check(_lib.dlion_aggregate_apply_tensors(self._ctx, _ptr(packed), _ptr(delta_bits_out), _stream()),
                    "dlion_aggregate_apply_tensors")

    def apply_delta_tensors(self, delta_wire: torch.Tensor, slice_words: int = 0) -> None:
        self._t(delta_wire, "delta_wire", _WORD_DTYPES, self.delta_planes() * self.words)
        self._check(_lib.dlion_apply_delta_tensors(self._ctx, _ptr(delta_wire), int(slice_words), _stream()),
                    "dlion_apply_delta_tensors")

    # ---- scatter mode: sign words stored straight into per-slice receive buffers
    def bind_scatter(self, dst, slice_words: int, slot: int, rows: int) -> None:
        """``dlion_bind_scatter``: ``dst`` is a list with one entry per coordinate slice, each a
        tensor [rows, slice_words] of int32 on this device, or an integer device address (a
        peer's buffer mapped into this process; its extent cannot be checked here)."""
        arr = (ctypes.c_void_p * len(dst))()
        for r, t in enumerate(dst):
            if isinstance(t, int):
                arr[r] = t
            else:
                check_tensor(t, f"dst[{r}]", _WORD_DTYPES, int(rows) * int(slice_words), self.device_index)
                arr[r] = t.data_ptr()
        self._scatter_keepalive = [t for t in dst if not isinstance(t, int)]
        self._check(_lib.dlion_bind_scatter(self._ctx, arr, len(dst), int(slice_words), int(slot), int(rows)),
                    "dlion_bind_scatter")

    def worker_step_scatter(self, worker: int, grads: torch.Tensor, m: torch.Tensor) -> None:
        self._t(grads, "grads", _GRAD_DTYPES[self.gdtype], self.d_pad)
        self._t(m, "m", _STATE_DTYPES[self.sdtype], self.d_pad)
        self._check(_lib.dlion_worker_step_scatter(self._ctx, int(worker), _ptr(grads), _ptr(m), _stream()),
                    "dlion_worker_step_scatter")

    def step_fused(self, grads: torch.Tensor, m: torch.Tensor, x: torch.Tensor,
                   packed_out: Optional[torch.Tensor] = None) -> None:
        self._t(grads, "grads", _GRAD_DTYPES[self.gdtype], self.n_workers * self.d_pad)
        self._t(m, "m", _STATE_DTYPES[self.sdtype], self.n_workers * self.d_pad)
        self._t(x, "x", (torch.float32,), self.d_pad)
        self._t(packed_out, "packed_out", _WORD_DTYPES, self.n_workers * self.words, optional=True)
        self._check(_lib.dlion_step_fused(self._ctx, _ptr(grads), _ptr(m), _ptr(x), _ptr(packed_out),
                                          _stream()), "dlion_step_fused")

    def step_global(self, grads: torch.Tensor, m: torch.Tensor, x: torch.Tensor,
                    delta_bits_out: Optional[torch.Tensor] = None) -> None:
        self._t(grads, "grads", _GRAD_DTYPES[self.gdtype], self.n_workers * self.d_pad)
        self._t(m, "m", (torch.float32,), self.n_workers * self.d_pad)
        self._t(x, "x", (torch.float32,), self.d_pad)
        self._t(delta_bits_out, "delta_bits_out", _WORD_DTYPES, self.words, optional=True)
        self._check(_lib.dlion_step_global(self._ctx, _ptr(grads), _ptr(m), _ptr(x), _ptr(delta_bits_out),
                                           _stream()), "dlion_step_global")

    def step_host(self, host_grads: torch.Tensor, m: torch.Tensor, x: torch.Tensor,
                  packed: torch.Tensor, staging: torch.Tensor,
                  delta_wire_dev: Optional[torch.Tensor] = None,
                  host_delta_out: Optional[torch.Tensor] = None) -> None:
        wire_bytes = self.delta_planes() * self.words * 4
        self._t(host_grads, "host_grads", _GRAD_DTYPES[self.gdtype], self.n_workers * self.d_pad, host=True)
        self._t(m, "m", _STATE_DTYPES[self.sdtype], self.n_workers * self.d_pad)
        self._t(x, "x", (torch.float32,), self.d_pad)
        self._t(packed, "packed", _WORD_DTYPES, self.n_workers * self.words)
        self._t(staging, "staging", _GRAD_DTYPES[self.gdtype], 2 * self.d_pad)
        for t, name, host in ((delta_wire_dev, "delta_wire_dev", False), (host_delta_out, "host_delta_out", True)):
            self._t(t, name, None, 0, optional=True, host=host)
            if t is not None and t.numel() * t.element_size() < wire_bytes:
                raise ValueError(f"{name}: {t.numel() * t.element_size()} bytes, the message has {wire_bytes}")
        self._check(_lib.dlion_step_host(self._ctx, _ptr(host_grads), _ptr(m), _ptr(x), _ptr(packed),
                                         _ptr(staging), _ptr(delta_wire_dev), _ptr(host_delta_out),
                                         _stream()), "dlion_step_host")

    def wire_bytes(self, direction: int) -> int:
        return int(_lib.dlion_wire_bytes(self._ctx, int(direction)))

    def launch_count(self) -> int:
        return int(_lib.dlion_launch_count(self._ctx))

    def destroy(self) -> None:
        if self._ctx:
            _lib.dlion_destroy(self._ctx)
            self._ctx = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
