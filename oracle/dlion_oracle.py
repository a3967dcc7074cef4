"""ctypes loader for the CPU oracle (``dlion_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
CPU-baseline / reference legs of ``bench.py``.  The product package never
imports this module, and this module never imports the product package.

The wrapper only marshals numpy arrays; every arithmetic step is in the C++
file, which follows Algorithm 1 and Section 3.2 of arXiv 2404.00438.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dlion_oracle.cpp")
_LIB = os.path.join(_HERE, "libdlion_oracle.so")

MAJORITY = 0
AVERAGE = 1
MAJORITY_TERNARY = 2      # Majority Vote with Delta = 0 on an even-N tie (three-valued sign)
GRAD_F32 = 0
GRAD_BF16 = 1
STATE_F32 = 0
STATE_BF16 = 1

CXXFLAGS = ["-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
            "-fPIC", "-shared"]


class _Segment(ctypes.Structure):
    _fields_ = [("elem_offset", ctypes.c_uint64), ("numel", ctypes.c_uint64)]


def build(force: bool = False, src: str = _SRC, out: str = _LIB) -> str:
    """Compile the oracle with g++ (no contraction, no fast-math)."""
    if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(src):
        subprocess.run(["g++", *CXXFLAGS, "-o", out, src], check=True)
    return out


def load(path: Optional[str] = None) -> ctypes.CDLL:
    lib = ctypes.CDLL(path or build())
    lib.dlion_oracle_worker_step.restype = ctypes.c_int
    lib.dlion_oracle_worker_step.argtypes = [
        ctypes.POINTER(_Segment), ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint32,
        ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
        ctypes.c_float, ctypes.c_float, ctypes.c_int]
    lib.dlion_oracle_worker_step_ex.restype = ctypes.c_int
    lib.dlion_oracle_worker_step_ex.argtypes = [
        ctypes.POINTER(_Segment), ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint32,
        ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
    lib.dlion_oracle_aggregate_apply.restype = ctypes.c_int
    lib.dlion_oracle_aggregate_apply.argtypes = [
        ctypes.POINTER(_Segment), ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint32,
        ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
        ctypes.c_float, ctypes.c_float, ctypes.c_int]
    lib.dlion_oracle_wire_bits.restype = ctypes.c_uint64
    lib.dlion_oracle_wire_bits.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int,
                                           ctypes.c_int]
    lib.dlion_oracle_has_openmp.restype = ctypes.c_int
    lib.dlion_oracle_delta_planes.restype = ctypes.c_uint32
    lib.dlion_oracle_delta_planes.argtypes = [ctypes.c_uint32, ctypes.c_int]
    lib.dlion_oracle_aggregate.restype = ctypes.c_int
    lib.dlion_oracle_aggregate.argtypes = [
        ctypes.POINTER(_Segment), ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int,
        ctypes.c_void_p, ctypes.c_void_p]
    lib.dlion_oracle_apply_delta.restype = ctypes.c_int
    lib.dlion_oracle_apply_delta.argtypes = [
        ctypes.POINTER(_Segment), ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int,
        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float, ctypes.c_float]
    lib.dlion_oracle_vote_counts16.restype = ctypes.c_int
    lib.dlion_oracle_vote_counts16.argtypes = [
        ctypes.POINTER(_Segment), ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint32,
        ctypes.c_void_p, ctypes.c_void_p]
    lib.dlion_oracle_global_step.restype = ctypes.c_int
    lib.dlion_oracle_global_step.argtypes = [
        ctypes.POINTER(_Segment), ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int,
        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
        ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_float]
    return lib


_lib: Optional[ctypes.CDLL] = None


def _get() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = load()
    return _lib


def _segs(segments: Sequence[Tuple[int, int]]):
    arr = (_Segment * len(segments))()
    for k, (off, n) in enumerate(segments):
        arr[k].elem_offset = int(off)
        arr[k].numel = int(n)
    return arr


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(a: np.ndarray, dtype, size: int, name: str) -> None:
    if a.dtype != dtype or not a.flags.c_contiguous or a.size != size:
        raise ValueError(f"{name}: need C-contiguous {np.dtype(dtype)} with {size} elements, "
                         f"got {a.dtype} with {a.size}")


def worker_step(segments, d_pad: int, n_workers: int, g: np.ndarray, m: np.ndarray,
                packed: np.ndarray, beta1: float, beta2: float, nthreads: int = 1,
                lib: Optional[ctypes.CDLL] = None) -> None:
    """Alg. 1 worker side for all workers: updates ``m`` in place, writes ``packed``.

    ``g`` is float32 (fp32 gradients) or uint16 (bf16 bit patterns), shape [N, d_pad].
    """
    if g.dtype == np.float32:
        gdt = GRAD_F32
    elif g.dtype == np.uint16:
        gdt = GRAD_BF16
    else:
        raise ValueError("g must be float32 or uint16 (bf16 bits)")
    _check(g, g.dtype, n_workers * d_pad, "g")
    _check(m, np.float32, n_workers * d_pad, "m")
    _check(packed, np.uint32, n_workers * d_pad // 32, "packed")
    rc = (lib or _get()).dlion_oracle_worker_step(
        _segs(segments), len(segments), d_pad, n_workers, gdt, _ptr(g), _ptr(m), _ptr(packed),
        beta1, beta2, nthreads)
    if rc != 0:
        raise ValueError("dlion_oracle_worker_step rejected its arguments")


def worker_step_ex(segments, d_pad: int, n_workers: int, g: np.ndarray, m: np.ndarray,
                   packed: np.ndarray, beta1s, beta2s, nthreads: int = 1,
                   lib: Optional[ctypes.CDLL] = None) -> None:
    """General worker side: per-worker betas (Alg. 1, footnote to the inputs) and fp32 or
    bf16 momentum (``m`` float32, or uint16 holding bf16 bit patterns)."""
    gdt = {np.dtype(np.float32): GRAD_F32, np.dtype(np.uint16): GRAD_BF16}[g.dtype]
    mdt = {np.dtype(np.float32): STATE_F32, np.dtype(np.uint16): STATE_BF16}[m.dtype]
    b1 = np.ascontiguousarray(beta1s, dtype=np.float32)
    b2 = np.ascontiguousarray(beta2s, dtype=np.float32)
    _check(g, g.dtype, n_workers * d_pad, "g")
    _check(m, m.dtype, n_workers * d_pad, "m")
    _check(packed, np.uint32, n_workers * d_pad // 32, "packed")
    _check(b1, np.float32, n_workers, "beta1s")
    _check(b2, np.float32, n_workers, "beta2s")
    rc = (lib or _get()).dlion_oracle_worker_step_ex(
        _segs(segments), len(segments), d_pad, n_workers, gdt, mdt, _ptr(g), _ptr(m), _ptr(packed),
        _ptr(b1), _ptr(b2), nthreads)
    if rc != 0:
        raise ValueError("dlion_oracle_worker_step_ex rejected its arguments")


def aggregate_apply(segments, d_pad: int, n_workers: int, mode: int, packed: np.ndarray,
                    x: np.ndarray, lr: float, weight_decay: float,
                    delta_bits: Optional[np.ndarray] = None,
                    count: Optional[np.ndarray] = None, nthreads: int = 1,
                    lib: Optional[ctypes.CDLL] = None) -> None:
    """Alg. 1 server side + the x update of Section 3.2: updates ``x`` in place."""
    _check(packed, np.uint32, n_workers * d_pad // 32, "packed")
    _check(x, np.float32, d_pad, "x")
    if delta_bits is not None:
        _check(delta_bits, np.uint32, d_pad // 32, "delta_bits")
    if count is not None:
        _check(count, np.uint8, d_pad, "count")
    rc = (lib or _get()).dlion_oracle_aggregate_apply(
        _segs(segments), len(segments), d_pad, n_workers, mode, _ptr(packed), _ptr(x),
        _ptr(delta_bits), _ptr(count), lr, weight_decay, nthreads)
    if rc != 0:
        raise ValueError("dlion_oracle_aggregate_apply rejected its arguments")


def wire_bits(d: int, n_workers: int, mode: int, direction: int,
              lib: Optional[ctypes.CDLL] = None) -> int:
    """Table 1: bits per step, worker->server (0) or server->worker (1)."""
    return int((lib or _get()).dlion_oracle_wire_bits(d, n_workers, mode, direction))


def delta_planes(n_workers: int, mode: int, lib: Optional[ctypes.CDLL] = None) -> int:
    """Bit planes of the server->worker message: 1 (Majority Vote) or ceil(log2(N+1))."""
    return int((lib or _get()).dlion_oracle_delta_planes(n_workers, mode))


def aggregate(segments, d_pad: int, n_workers: int, mode: int, packed: np.ndarray,
              delta_wire: np.ndarray, lib: Optional[ctypes.CDLL] = None) -> None:
    """Alg. 1 server side alone: writes the broadcast message (bits, or count bit planes)."""
    _check(packed, np.uint32, n_workers * d_pad // 32, "packed")
    _check(delta_wire, np.uint32, delta_planes(n_workers, mode, lib) * d_pad // 32, "delta_wire")
    rc = (lib or _get()).dlion_oracle_aggregate(_segs(segments), len(segments), d_pad, n_workers, mode,
                                                _ptr(packed), _ptr(delta_wire))
    if rc != 0:
        raise ValueError("dlion_oracle_aggregate rejected its arguments")


def apply_delta(segments, d_pad: int, n_workers: int, mode: int, delta_wire: np.ndarray,
                x: np.ndarray, lr: float, weight_decay: float,
                lib: Optional[ctypes.CDLL] = None) -> None:
    """Alg. 1 worker side, first line: x <- x - eps (Delta + lambda x) from the wire format."""
    _check(delta_wire, np.uint32, delta_planes(n_workers, mode, lib) * d_pad // 32, "delta_wire")
    _check(x, np.float32, d_pad, "x")
    rc = (lib or _get()).dlion_oracle_apply_delta(_segs(segments), len(segments), d_pad, n_workers, mode,
                                                  _ptr(delta_wire), _ptr(x), lr, weight_decay)
    if rc != 0:
        raise ValueError("dlion_oracle_apply_delta rejected its arguments")


def vote_counts16(segments, d_pad: int, n_workers: int, packed: np.ndarray, count16: np.ndarray,
                  lib: Optional[ctypes.CDLL] = None) -> None:
    """The number of +1 votes of every parameter as uint16 (any N up to 65535)."""
    _check(packed, np.uint32, n_workers * d_pad // 32, "packed")
    _check(count16, np.uint16, d_pad, "count16")
    rc = (lib or _get()).dlion_oracle_vote_counts16(_segs(segments), len(segments), d_pad, n_workers,
                                                    _ptr(packed), _ptr(count16))
    if rc != 0:
        raise ValueError("dlion_oracle_vote_counts16 rejected its arguments")


def global_step(segments, d_pad: int, n_workers: int, g: np.ndarray, m: np.ndarray, x: np.ndarray,
                beta1: float, beta2: float, lr: float, weight_decay: float,
                delta_bits: Optional[np.ndarray] = None, lib: Optional[ctypes.CDLL] = None) -> None:
    """One step of Global Lion (appendix scheme): fp32 mean of the workers' blends, one sign,
    the x update; every worker's momentum updated in place."""
    gdt = {np.dtype(np.float32): GRAD_F32, np.dtype(np.uint16): GRAD_BF16}[g.dtype]
    _check(g, g.dtype, n_workers * d_pad, "g")
    _check(m, np.float32, n_workers * d_pad, "m")
    _check(x, np.float32, d_pad, "x")
    if delta_bits is not None:
        _check(delta_bits, np.uint32, d_pad // 32, "delta_bits")
    rc = (lib or _get()).dlion_oracle_global_step(_segs(segments), len(segments), d_pad, n_workers, gdt,
                                                  _ptr(g), _ptr(m), _ptr(x), _ptr(delta_bits),
                                                  beta1, beta2, lr, weight_decay)
    if rc != 0:
        raise ValueError("dlion_oracle_global_step rejected its arguments")


def has_openmp() -> bool:
    return bool(_get().dlion_oracle_has_openmp())
