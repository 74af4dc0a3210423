"""ctypes front end of the C oracle (loco_oracle.c).  Test infrastructure only.

Every function here only marshals numpy arrays into the C routines; the
arithmetic is all in the C file, which cites the passages of the paper
(arXiv 2407.04480) that it follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "loco_oracle.c")
_LIB = os.path.join(_HERE, "libloco_oracle.so")

F32, BF16 = 0, 1
SCALE_FIXED, SCALE_BLOCK_ABSMAX = 0, 1
STATE_INT8, STATE_FP32, STATE_NONE, STATE_FP32_Q8COMP = 0, 1, 2, 3
FLAG_NONFINITE = 1

# One rounding per written operation: no contraction into FMA, no fast-math.
CFLAGS = ["-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [("bits", C.c_int32), ("scale_mode", C.c_int32), ("block_size", C.c_int32),
                ("s", C.c_float), ("s_e", C.c_float), ("beta", C.c_float),
                ("reset_period", C.c_int32), ("state_fmt", C.c_int32),
                ("grad_dtype", C.c_int32), ("out_dtype", C.c_int32), ("num_partitions", C.c_int32),
                ("clip", C.c_float), ("rounding", C.c_int32), ("seed_lo", C.c_uint32), ("seed_hi", C.c_uint32)]


class _Adam(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("delta", C.c_float)]


class _Trace(C.Structure):
    _fields_ = [("c", C.c_void_p), ("h", C.c_void_p), ("q", C.c_void_p),
                ("d", C.c_void_p), ("delta", C.c_void_p), ("e_new", C.c_void_p)]


@dataclass
class OracleConfig:
    """Algorithm 1's inputs (s, s_e, T_c, beta) and the storage choices."""
    bits: int = 4
    scale_mode: int = SCALE_FIXED
    block_size: int = 256
    s: float = 2.0 ** 19
    s_e: float = 2.0 ** 21
    beta: float = 0.5
    reset_period: int = 512
    state_fmt: int = STATE_INT8
    grad_dtype: int = F32
    out_dtype: int = F32
    num_partitions: int = 1
    clip: float = 0.0
    rounding: int = 0
    seed: int = 0

    def c(self) -> _Cfg:
        return _Cfg(self.bits, self.scale_mode, self.block_size, self.s, self.s_e, self.beta,
                    self.reset_period, self.state_fmt, self.grad_dtype, self.out_dtype,
                    self.num_partitions, self.clip, self.rounding, self.seed & 0xFFFFFFFF, (self.seed >> 32) & 0xFFFFFFFF)


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u64, i32, i64, vp = C.c_uint64, C.c_int32, C.c_int64, C.c_void_p
        cp = C.POINTER(_Cfg)
        for name in ("orc_partition_capacity", "orc_partition_bytes", "orc_packed_bytes", "orc_state_bytes"):
            getattr(L, name).restype = u64
            getattr(L, name).argtypes = [cp, u64]
        L.orc_partition_elems.restype = u64
        L.orc_partition_elems.argtypes = [cp, u64, i32]
        L.orc_compressor.restype = None
        L.orc_compressor.argtypes = [vp, u64, C.c_float, i32, vp]
        L.orc_decompressor.restype = None
        L.orc_decompressor.argtypes = [vp, u64, C.c_float, vp]
        L.orc_pack_codes.restype = None
        L.orc_pack_codes.argtypes = [vp, u64, i32, vp]
        L.orc_unpack_codes.restype = None
        L.orc_unpack_codes.argtypes = [vp, u64, i32, vp]
        L.orc_send_step.restype = C.c_int
        L.orc_send_step.argtypes = [cp, u64, vp, vp, vp, i64, C.POINTER(_Trace), vp]
        L.orc_reduce.restype = C.c_int
        L.orc_reduce.argtypes = [cp, u64, C.POINTER(vp), i32, i32, i32, vp]
        L.orc_reduce_adam.restype = C.c_int
        L.orc_reduce_adam.argtypes = [cp, u64, C.POINTER(vp), i32, i32, i32, C.POINTER(_Adam), vp, vp, vp, vp]
        L.orc_philox4x32_10.restype = None
        L.orc_philox4x32_10.argtypes = [vp, vp, vp]
        L.orc_sr_uniform.restype = C.c_float
        L.orc_sr_uniform.argtypes = [cp, u64, i64]
        L.orc_pairwise_sum.restype = C.c_float
        L.orc_pairwise_sum.argtypes = [vp, u64]
        L.orc_f32_to_bf16.restype = C.c_uint16
        L.orc_f32_to_bf16.argtypes = [C.c_float]
        L.orc_bf16_to_f32.restype = C.c_float
        L.orc_bf16_to_f32.argtypes = [C.c_uint16]
        L.orc_f32_to_bf16_array.restype = None
        L.orc_f32_to_bf16_array.argtypes = [vp, u64, vp]
        L.orc_bf16_to_f32_array.restype = None
        L.orc_bf16_to_f32_array.argtypes = [vp, u64, vp]
        _lib = L
    return _lib


def _ptr(a: np.ndarray) -> int:
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def partition_capacity(cfg, n): return int(lib().orc_partition_capacity(C.byref(cfg.c()), n))
def partition_elems(cfg, n, j): return int(lib().orc_partition_elems(C.byref(cfg.c()), n, j))
def partition_bytes(cfg, n): return int(lib().orc_partition_bytes(C.byref(cfg.c()), n))
def packed_bytes(cfg, n): return int(lib().orc_packed_bytes(C.byref(cfg.c()), n))
def state_bytes(cfg, n): return int(lib().orc_state_bytes(C.byref(cfg.c()), n))


def compressor(h: np.ndarray, s: float, p: int) -> np.ndarray:
    """Eq. 1, first line."""
    h = np.ascontiguousarray(h, dtype=np.float32)
    q = np.empty(h.shape, dtype=np.int32)
    lib().orc_compressor(_ptr(h), h.size, s, p, _ptr(q))
    return q


def decompressor(q: np.ndarray, s: float) -> np.ndarray:
    """Eq. 1, second line."""
    q = np.ascontiguousarray(q, dtype=np.int32)
    out = np.empty(q.shape, dtype=np.float32)
    lib().orc_decompressor(_ptr(q), q.size, s, _ptr(out))
    return out


def pack_codes(q: np.ndarray, p: int) -> np.ndarray:
    q = np.ascontiguousarray(q, dtype=np.int32)
    out = np.zeros((q.size * p + 7) // 8, dtype=np.uint8)
    lib().orc_pack_codes(_ptr(q), q.size, p, _ptr(out))
    return out


def unpack_codes(b: np.ndarray, n: int, p: int) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint8)
    q = np.empty(n, dtype=np.int32)
    lib().orc_unpack_codes(_ptr(b), n, p, _ptr(q))
    return q


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """The oracle's fp32 -> bf16 conversion (round to nearest, ties to even), elementwise, as bit patterns."""
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float32).ravel())
    out = np.empty(x.size, dtype=np.uint16)
    lib().orc_f32_to_bf16_array(_ptr(x), x.size, _ptr(out))
    return out


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """The oracle's bf16 -> fp32 widening, elementwise."""
    b = np.ascontiguousarray(np.asarray(b, dtype=np.uint16).ravel())
    out = np.empty(b.size, dtype=np.float32)
    lib().orc_bf16_to_f32_array(_ptr(b), b.size, _ptr(out))
    return out


def new_state(cfg: OracleConfig, n: int) -> np.ndarray:
    """Zero error state (e~_0 = 0, Eq. 5's initialisation) as raw bytes."""
    return np.zeros(state_bytes(cfg, n), dtype=np.uint8)


def new_comm(cfg: OracleConfig, n: int, fill: int = 0) -> np.ndarray:
    return np.full(packed_bytes(cfg, n), fill, dtype=np.uint8)


def send_step(cfg: OracleConfig, grad: np.ndarray, state: np.ndarray, comm: np.ndarray, k: int,
              trace: bool = False, full_status: bool = False):
    """Algorithm 1 steps 1-2 for one worker; updates state and comm in place.

    grad is float32, or uint16 holding bf16 bit patterns.  Returns (flags, n_saturated) -- with full_status
    (flags, n_saturated, n_saturated_state) -- and, when trace is set, a dict of the per-element intermediates.
    """
    n = grad.size
    if cfg.grad_dtype == BF16:
        assert grad.dtype == np.uint16
    else:
        assert grad.dtype == np.float32
    assert state.dtype == np.uint8 and state.size >= state_bytes(cfg, n)
    assert comm.dtype == np.uint8 and comm.size >= packed_bytes(cfg, n)
    status = np.zeros(3, dtype=np.uint64)
    tr = None
    rec = None
    if trace:
        rec = {"c": np.zeros(n, np.float32), "h": np.zeros(n, np.float32), "q": np.zeros(n, np.int32),
               "d": np.zeros(n, np.float32), "delta": np.zeros(n, np.float32),
               "e_new": np.zeros(n, np.float32)}
        tr = _Trace(*[_ptr(rec[k_]) for k_ in ("c", "h", "q", "d", "delta", "e_new")])
    rc = lib().orc_send_step(C.byref(cfg.c()), n, _ptr(grad), _ptr(state) if state.size else None,
                             _ptr(comm) if comm.size else None, k,
                             C.byref(tr) if tr is not None else None, _ptr(status))
    if rc != 0:
        raise ValueError("oracle: bad configuration")
    out = (int(status[0]), int(status[1]), int(status[2])) if full_status else (int(status[0]), int(status[1]))
    return (out, rec) if trace else out


def reduce(cfg: OracleConfig, n: int, comms, first: int = 0, count: int | None = None) -> np.ndarray:
    """Eq. 8 over partitions [first, first+count) of the workers' communication buffers.

    comms: one full communication buffer (uint8 array) per worker.  Returns float32, or
    uint16 bf16 bit patterns when cfg.out_dtype is BF16.
    """
    if count is None:
        count = cfg.num_partitions - first
    stride = partition_bytes(cfg, n)
    n_out = sum(partition_elems(cfg, n, j) for j in range(first, first + count))
    out = np.zeros(n_out, dtype=np.uint16 if cfg.out_dtype == BF16 else np.float32)
    ptrs = (C.c_void_p * len(comms))(*[_ptr(c) + first * stride for c in comms])
    rc = lib().orc_reduce(C.byref(cfg.c()), n, ptrs, len(comms), first, count, _ptr(out) if n_out else None)
    if rc != 0:
        raise ValueError("oracle: bad configuration")
    return out


def reduce_adam(cfg: OracleConfig, n: int, comms, m: np.ndarray, v: np.ndarray, theta: np.ndarray, *, lr: float,
                beta1: float, beta2: float, delta: float, first: int = 0, count: int | None = None,
                want_grad: bool = False):
    """Eq. 8 followed by the paper's Adam-family step on the same elements; m, v, theta (float32) are updated in
    place.  Returns the averaged gradient (out_dtype) when want_grad is set."""
    if count is None:
        count = cfg.num_partitions - first
    stride = partition_bytes(cfg, n)
    n_out = sum(partition_elems(cfg, n, j) for j in range(first, first + count))
    for a in (m, v, theta):
        assert a.dtype == np.float32 and a.size >= n_out and a.flags["C_CONTIGUOUS"]
    out = np.zeros(n_out, dtype=np.uint16 if cfg.out_dtype == BF16 else np.float32) if want_grad else None
    ptrs = (C.c_void_p * len(comms))(*[_ptr(c) + first * stride for c in comms])
    ad = _Adam(lr, beta1, beta2, delta)
    rc = lib().orc_reduce_adam(C.byref(cfg.c()), n, ptrs, len(comms), first, count, C.byref(ad),
                               _ptr(m) if n_out else None, _ptr(v) if n_out else None, _ptr(theta) if n_out else None,
                               _ptr(out) if (want_grad and n_out) else None)
    if rc != 0:
        raise ValueError("oracle: bad configuration")
    return out


def philox4x32_10(ctr, key) -> np.ndarray:
    """The four output words of Philox4x32-10 for a 4-word counter and a 2-word key."""
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def pairwise_sum(a: np.ndarray) -> float:
    """fp32 pairwise (balanced binary tree) sum of a power-of-two number of values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    assert a.size > 0 and a.size & (a.size - 1) == 0
    return float(lib().orc_pairwise_sum(_ptr(a), a.size))


def sr_uniform(cfg: OracleConfig, i: int, k: int) -> float:
    return float(lib().orc_sr_uniform(C.byref(cfg.c()), i, k))


def state_views(cfg: OracleConfig, n: int, state: np.ndarray):
    """Split raw state bytes into (codes or fp32 values, block scales or None)."""
    if cfg.state_fmt == STATE_NONE:
        return None, None
    if cfg.state_fmt == STATE_INT8:
        codes = state[:n].view(np.int8)
        scales = None
        if cfg.scale_mode == SCALE_BLOCK_ABSMAX:
            off = (n + 255) // 256 * 256
            nb = (n + cfg.block_size - 1) // cfg.block_size
            scales = state[off:off + 4 * nb].view(np.float32)
        return codes, scales
    return state[:4 * n].view(np.float32), None


def comm_views(cfg: OracleConfig, n: int, comm: np.ndarray):
    """Per partition: (code bytes, scales or None) of the defined areas of a communication buffer."""
    lp = partition_capacity(cfg, n)
    stride = partition_bytes(cfg, n)
    cb = lp * cfg.bits // 8
    out = []
    for j in range(cfg.num_partitions):
        base = j * stride
        codes = comm[base:base + cb]
        scales = None
        if cfg.scale_mode == SCALE_BLOCK_ABSMAX:
            scales = comm[base + cb: base + cb + 4 * (lp // cfg.block_size)].view(np.float32)
        out.append((codes, scales))
    return out
