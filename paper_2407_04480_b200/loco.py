"""Thin Python binding of the LoCo C ABI (include/loco.h): argument marshalling only.

Every function has the name of the C entry point it calls and does nothing else than turn
torch tensors into raw device pointers.  All arithmetic of the method (Algorithm 1 and
Eq. 1-8 of arXiv 2407.04480) runs in the CUDA kernels of libloco_b200.so.  There is no CPU
fallback: if the library cannot be loaded, the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libloco_b200.so")

OK, ERR_ARG, ERR_ALIGN, ERR_SIZE, ERR_CUDA, ERR_UNSUPPORTED = 0, -1, -2, -3, -4, -5
F32, BF16 = 0, 1
SCALE_FIXED, SCALE_BLOCK_ABSMAX = 0, 1
STATE_INT8, STATE_FP32, STATE_NONE, STATE_FP32_Q8COMP = 0, 1, 2, 3
ROUND_NEAREST, ROUND_STOCHASTIC = 0, 1
FLAG_NONFINITE = 1

EXPORTS = ("loco_state_bytes", "loco_packed_bytes", "loco_partition_bytes", "loco_partition_capacity",
           "loco_partition_elems", "loco_config_check", "loco_state_init", "loco_state_reset",
           "loco_state_destroy", "loco_compensate_quantize_pack", "loco_unpack_dequant_reduce",
           "loco_last_status", "loco_status_string", "loco_launch_count",
           "loco_send_host_workspace_bytes", "loco_reduce_host_workspace_bytes",
           "loco_compensate_quantize_pack_host", "loco_unpack_dequant_reduce_host",
           "loco_unpack_dequant_reduce_host_noalloc", "loco_selfcheck_block_division",
           "loco_unpack_dequant_reduce_adam", "loco_compensate_quantize_pack_scatter",
           "loco_compensate_quantize_pack_multi", "loco_unpack_dequant_reduce_multi", "loco_status_counters")
NOALLOC_SCRATCH_BYTES = 4 * 1024 * 1024


class LocoError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s failed: %s (%d)" % (where, status_string(code), code))


class loco_config_t(C.Structure):
    _fields_ = [("bits", C.c_int32), ("scale_mode", C.c_int32), ("block_size", C.c_int32),
                ("s", C.c_float), ("s_e", C.c_float), ("beta", C.c_float),
                ("reset_period", C.c_int32), ("state_fmt", C.c_int32), ("grad_dtype", C.c_int32),
                ("out_dtype", C.c_int32), ("num_partitions", C.c_int32), ("collect_stats", C.c_int32),
                ("clip", C.c_float), ("rounding", C.c_int32), ("seed_lo", C.c_uint32), ("seed_hi", C.c_uint32)]


class loco_adam_t(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("delta", C.c_float)]


@dataclass
class Config:
    """Mirror of loco_config_t: Algorithm 1's inputs (s, s_e, T_c, beta), Eq. 1's p, storage choices."""
    bits: int = 4
    scale_mode: int = SCALE_FIXED
    block_size: int = 256
    s: float = 2.0 ** 19
    s_e: float = 2.0 ** 21
    beta: float = 0.5
    reset_period: int = 512
    state_fmt: int = STATE_INT8
    grad_dtype: int = BF16
    out_dtype: int = BF16
    num_partitions: int = 1
    collect_stats: int = 0
    clip: float = 0.0
    rounding: int = 0
    seed: int = 0

    def c(self) -> loco_config_t:
        return loco_config_t(self.bits, self.scale_mode, self.block_size, self.s, self.s_e, self.beta,
                             self.reset_period, self.state_fmt, self.grad_dtype, self.out_dtype,
                             self.num_partitions, self.collect_stats, self.clip, self.rounding,
                             self.seed & 0xFFFFFFFF, (self.seed >> 32) & 0xFFFFFFFF)


_lib = None


def lib() -> C.CDLL:
    """Load libloco_b200.so (built by paper_2407_04480_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("LoCo CUDA library missing: %s (run python -m paper_2407_04480_b200.build); "
                               "there is no CPU fallback" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        u64, i32, i64, vp = C.c_uint64, C.c_int32, C.c_int64, C.c_void_p
        cp = C.POINTER(loco_config_t)
        for name in ("loco_state_bytes", "loco_packed_bytes", "loco_partition_bytes", "loco_partition_capacity"):
            getattr(L, name).restype = u64
            getattr(L, name).argtypes = [cp, u64]
        L.loco_partition_elems.restype = u64
        L.loco_partition_elems.argtypes = [cp, u64, i32]
        L.loco_config_check.restype = C.c_int
        L.loco_config_check.argtypes = [cp]
        L.loco_state_init.restype = C.c_int
        L.loco_state_init.argtypes = [C.POINTER(vp), cp, u64, vp, u64, vp]
        L.loco_state_reset.restype = C.c_int
        L.loco_state_reset.argtypes = [vp, vp]
        L.loco_state_destroy.restype = C.c_int
        L.loco_state_destroy.argtypes = [vp]
        L.loco_compensate_quantize_pack.restype = C.c_int
        L.loco_compensate_quantize_pack.argtypes = [vp, vp, vp, i64, vp]
        L.loco_unpack_dequant_reduce.restype = C.c_int
        L.loco_unpack_dequant_reduce.argtypes = [cp, C.POINTER(vp), i32, u64, i32, i32, vp, vp]
        L.loco_send_host_workspace_bytes.restype = u64
        L.loco_send_host_workspace_bytes.argtypes = [cp, u64]
        L.loco_reduce_host_workspace_bytes.restype = u64
        L.loco_reduce_host_workspace_bytes.argtypes = [cp, u64, i32, i32]
        L.loco_compensate_quantize_pack_scatter.restype = C.c_int
        L.loco_compensate_quantize_pack_scatter.argtypes = [vp, vp, vp, i64, vp]
        L.loco_compensate_quantize_pack_multi.restype = C.c_int
        L.loco_compensate_quantize_pack_multi.argtypes = [vp, vp, vp, C.c_int32, i64, vp]
        L.loco_unpack_dequant_reduce_multi.restype = C.c_int
        L.loco_unpack_dequant_reduce_multi.argtypes = [vp, vp, C.c_int32, vp, vp, C.c_int32, vp]
        L.loco_compensate_quantize_pack_host.restype = C.c_int
        L.loco_compensate_quantize_pack_host.argtypes = [vp, vp, vp, vp, u64, i64, vp]
        L.loco_unpack_dequant_reduce_host.restype = C.c_int
        L.loco_unpack_dequant_reduce_host.argtypes = [cp, C.POINTER(vp), i32, u64, i32, i32, vp, vp, u64, vp]
        L.loco_unpack_dequant_reduce_host_noalloc.restype = C.c_int
        L.loco_unpack_dequant_reduce_host_noalloc.argtypes = [cp, C.POINTER(vp), i32, u64, i32, i32, vp, vp]
        L.loco_unpack_dequant_reduce_adam.restype = C.c_int
        L.loco_unpack_dequant_reduce_adam.argtypes = [cp, C.POINTER(vp), i32, u64, i32, i32, C.POINTER(loco_adam_t), vp, vp, vp, vp, vp]
        L.loco_selfcheck_block_division.restype = C.c_int
        L.loco_selfcheck_block_division.argtypes = [C.POINTER(u64)]
        L.loco_last_status.restype = C.c_int
        L.loco_last_status.argtypes = [vp, C.POINTER(C.c_uint32), C.POINTER(u64), vp]
        L.loco_status_counters.restype = C.c_int
        L.loco_status_counters.argtypes = [vp, C.POINTER(C.c_uint32), C.POINTER(u64), C.POINTER(u64), vp]
        L.loco_status_string.restype = C.c_char_p
        L.loco_status_string.argtypes = [C.c_int]
        L.loco_launch_count.restype = u64
        L.loco_launch_count.argtypes = []
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().loco_status_string(code).decode()


def _check(code: int, where: str) -> None:
    if code != OK:
        raise LocoError(code, where)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _dev_ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


# ---- sizes -----------------------------------------------------------------------------------

def loco_state_bytes(cfg: Config, n: int) -> int: return int(lib().loco_state_bytes(C.byref(cfg.c()), n))
def loco_packed_bytes(cfg: Config, n: int) -> int: return int(lib().loco_packed_bytes(C.byref(cfg.c()), n))
def loco_partition_bytes(cfg: Config, n: int) -> int: return int(lib().loco_partition_bytes(C.byref(cfg.c()), n))
def loco_partition_capacity(cfg: Config, n: int) -> int: return int(lib().loco_partition_capacity(C.byref(cfg.c()), n))
def loco_partition_elems(cfg: Config, n: int, j: int) -> int: return int(lib().loco_partition_elems(C.byref(cfg.c()), n, j))
def loco_config_check(cfg: Config) -> int: return int(lib().loco_config_check(C.byref(cfg.c())))
def loco_launch_count() -> int: return int(lib().loco_launch_count())


# ---- state -----------------------------------------------------------------------------------

class State:
    """Owner of a loco_state_t handle and of the torch tensor that holds the error state."""

    def __init__(self, cfg: Config, n: int, device="cuda", stream: Optional[torch.cuda.Stream] = None,
                 buffer: Optional[torch.Tensor] = None):
        self.cfg, self.n = cfg, n
        nbytes = loco_state_bytes(cfg, n)
        if buffer is None:
            buffer = torch.empty(max(nbytes, 16), dtype=torch.uint8, device=device)
        self.buffer = buffer
        self._h = C.c_void_p()
        _check(loco_state_init_raw(C.byref(self._h), cfg, n, _dev_ptr(buffer) if nbytes else None,
                                   buffer.numel() if nbytes else 0, _stream_ptr(stream)), "loco_state_init")

    @property
    def handle(self) -> C.c_void_p:
        if not self._h:
            raise RuntimeError("state already destroyed")
        return self._h

    def close(self) -> None:
        if self._h:
            code = lib().loco_state_destroy(self._h)
            self._h = C.c_void_p()
            _check(code, "loco_state_destroy")

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def loco_state_init_raw(out_handle, cfg: Config, n: int, d_state: Optional[int], d_state_bytes: int,
                        stream_ptr: Optional[int]) -> int:
    """loco_state_init with raw pointers; returns the status code."""
    return int(lib().loco_state_init(out_handle, C.byref(cfg.c()), n, d_state, d_state_bytes, stream_ptr))


def loco_state_init(cfg: Config, n: int, device="cuda", stream=None, buffer=None) -> State:
    return State(cfg, n, device=device, stream=stream, buffer=buffer)


def loco_state_reset(st: State, stream=None) -> None:
    _check(lib().loco_state_reset(st.handle, _stream_ptr(stream)), "loco_state_reset")


def loco_state_destroy(st: State) -> None:
    st.close()


# ---- the two passes --------------------------------------------------------------------------

def loco_compensate_quantize_pack(st: State, grad: torch.Tensor, comm: torch.Tensor, step_k: int,
                                  stream=None) -> None:
    """Send pass (Algorithm 1 steps 1-2) for iteration step_k: updates st's buffer and comm in place."""
    want = torch.bfloat16 if st.cfg.grad_dtype == BF16 else torch.float32
    if grad.dtype != want or grad.numel() != st.n:
        raise ValueError("gradient must be %s with %d elements" % (want, st.n))
    if comm.dtype != torch.uint8 or comm.numel() < loco_packed_bytes(st.cfg, st.n):
        raise ValueError("communication buffer too small or not uint8")
    _check(lib().loco_compensate_quantize_pack(st.handle, _dev_ptr(grad), _dev_ptr(comm), step_k,
                                               _stream_ptr(stream)), "loco_compensate_quantize_pack")


def loco_compensate_quantize_pack_scatter(st: State, grad: torch.Tensor, part_dst: Sequence, step_k: int,
                                          stream=None) -> None:
    """Send pass whose part j goes to part_dst[j] (a uint8 CUDA tensor of at least loco_partition_bytes(), or an
    int device address -- this GPU's memory or a peer's mapped here) instead of one contiguous buffer."""
    want = torch.bfloat16 if st.cfg.grad_dtype == BF16 else torch.float32
    if grad.dtype != want or grad.numel() != st.n:
        raise ValueError("gradient must be %s with %d elements" % (want, st.n))
    if len(part_dst) != st.cfg.num_partitions:
        raise ValueError("one destination per partition is needed (%d)" % st.cfg.num_partitions)
    need = loco_partition_bytes(st.cfg, st.n)
    for d in part_dst:
        if not isinstance(d, int) and (d.dtype != torch.uint8 or d.numel() < need):
            raise ValueError("a destination is too small or not uint8")
    ptrs = (C.c_void_p * len(part_dst))(*[d if isinstance(d, int) else _dev_ptr(d) for d in part_dst])
    _check(lib().loco_compensate_quantize_pack_scatter(st.handle, _dev_ptr(grad), ptrs, step_k, _stream_ptr(stream)),
           "loco_compensate_quantize_pack_scatter")


def loco_unpack_dequant_reduce(cfg: Config, packed: Sequence, n: int, out: torch.Tensor,
                               first_partition: int = 0, partition_count: Optional[int] = None,
                               stream=None) -> None:
    """Receive pass (Eq. 8).  packed: per worker, a uint8 CUDA tensor starting at partition
    `first_partition` of that worker's buffer, or an int device address of the same."""
    if partition_count is None:
        partition_count = cfg.num_partitions - first_partition
    ptrs = (C.c_void_p * len(packed))(*[p if isinstance(p, int) else _dev_ptr(p) for p in packed])
    want = torch.bfloat16 if cfg.out_dtype == BF16 else torch.float32
    if out.dtype != want:
        raise ValueError("output must be %s" % want)
    need = sum(loco_partition_elems(cfg, n, j) for j in range(first_partition, first_partition + partition_count))
    if out.numel() < need:
        raise ValueError("output holds %d elements, %d needed" % (out.numel(), need))
    _check(lib().loco_unpack_dequant_reduce(C.byref(cfg.c()), ptrs, len(packed), n, first_partition,
                                            partition_count, _dev_ptr(out), _stream_ptr(stream)),
           "loco_unpack_dequant_reduce")


class MultiSend:
    """Argument tables of loco_compensate_quantize_pack_multi, marshalled once for a fixed set of buckets."""

    def __init__(self, states: Sequence[State], grads: Sequence[torch.Tensor], comms: Sequence[torch.Tensor]):
        if not (len(states) == len(grads) == len(comms)):
            raise ValueError("one gradient and one communication buffer per state are needed")
        for st, g, c in zip(states, grads, comms):
            want = torch.bfloat16 if st.cfg.grad_dtype == BF16 else torch.float32
            if g.dtype != want or g.numel() != st.n:
                raise ValueError("gradient must be %s with %d elements" % (want, st.n))
            if c.dtype != torch.uint8 or c.numel() < loco_packed_bytes(st.cfg, st.n):
                raise ValueError("communication buffer too small or not uint8")
        self.keep = (list(states), list(grads), list(comms))
        self.count = len(states)
        self.h = (C.c_void_p * self.count)(*[st.handle.value for st in states])
        self.g = (C.c_void_p * self.count)(*[_dev_ptr(g) for g in grads])
        self.c = (C.c_void_p * self.count)(*[_dev_ptr(c) for c in comms])


def loco_compensate_quantize_pack_multi(ms: MultiSend, step_k: int, stream=None) -> None:
    """The send pass for all buckets of ms, their launches overlapped on the library's own streams."""
    _check(lib().loco_compensate_quantize_pack_multi(ms.h, ms.g, ms.c, ms.count, step_k, _stream_ptr(stream)),
           "loco_compensate_quantize_pack_multi")


class MultiReduce:
    """Argument tables of loco_unpack_dequant_reduce_multi for a fixed set of buckets (whole buckets, all parts)."""

    def __init__(self, cfg: Config, packed: Sequence[Sequence], ns: Sequence[int], outs: Sequence[torch.Tensor]):
        if not (len(packed) == len(ns) == len(outs)) or any(len(p) != len(packed[0]) for p in packed):
            raise ValueError("one list of worker buffers, one length and one output per bucket are needed")
        want = torch.bfloat16 if cfg.out_dtype == BF16 else torch.float32
        for n, o in zip(ns, outs):
            if o.dtype != want or o.numel() < n:
                raise ValueError("output must be %s with at least %d elements" % (want, n))
        self.cfg, self.count, self.workers = cfg, len(ns), len(packed[0]) if packed else 0
        self.keep = (list(packed), list(outs))
        self.rows = [(C.c_void_p * self.workers)(*[p if isinstance(p, int) else _dev_ptr(p) for p in row]) for row in packed]
        self.p = (C.c_void_p * self.count)(*[C.cast(r, C.c_void_p).value for r in self.rows])
        self.n = (C.c_uint64 * self.count)(*ns)
        self.o = (C.c_void_p * self.count)(*[_dev_ptr(o) for o in outs])


def loco_unpack_dequant_reduce_multi(mr: MultiReduce, stream=None) -> None:
    """The receive pass for all buckets of mr, their launches overlapped on the library's own streams."""
    _check(lib().loco_unpack_dequant_reduce_multi(C.byref(mr.cfg.c()), mr.p, mr.workers, mr.n, mr.o, mr.count,
                                                  _stream_ptr(stream)), "loco_unpack_dequant_reduce_multi")


def loco_last_status(st: State, stream=None):
    """(flags, n_saturated) accumulated since init/reset; synchronises the stream."""
    flags, sat = C.c_uint32(0), C.c_uint64(0)
    _check(lib().loco_last_status(st.handle, C.byref(flags), C.byref(sat), _stream_ptr(stream)), "loco_last_status")
    return int(flags.value), int(sat.value)


def loco_status_counters(st: State, stream=None):
    """(flags, saturated gradient codes, saturated 8-bit error codes) accumulated since init/reset; synchronises the stream."""
    flags, sat, ssat = C.c_uint32(0), C.c_uint64(0), C.c_uint64(0)
    _check(lib().loco_status_counters(st.handle, C.byref(flags), C.byref(sat), C.byref(ssat), _stream_ptr(stream)),
           "loco_status_counters")
    return int(flags.value), int(sat.value), int(ssat.value)


# ---- host-buffer variants --------------------------------------------------------------------

def loco_send_host_workspace_bytes(cfg: Config, n: int) -> int:
    return int(lib().loco_send_host_workspace_bytes(C.byref(cfg.c()), n))


def loco_reduce_host_workspace_bytes(cfg: Config, n: int, num_workers: int, partition_count: int) -> int:
    return int(lib().loco_reduce_host_workspace_bytes(C.byref(cfg.c()), n, num_workers, partition_count))


def _host_ptr(t: torch.Tensor) -> int:
    if t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous host tensor")
    return t.data_ptr()


def loco_compensate_quantize_pack_host(st: State, h_grad: torch.Tensor, h_comm: torch.Tensor, d_work: torch.Tensor,
                                       step_k: int, stream=None) -> None:
    """Send pass with gradient and communication buffer in host memory (pinned for asynchronous copies)."""
    _check(lib().loco_compensate_quantize_pack_host(st.handle, _host_ptr(h_grad), _host_ptr(h_comm), _dev_ptr(d_work),
                                                    d_work.numel() * d_work.element_size(), step_k,
                                                    _stream_ptr(stream)), "loco_compensate_quantize_pack_host")


def loco_unpack_dequant_reduce_host(cfg: Config, h_packed: Sequence[torch.Tensor], n: int, h_out: torch.Tensor,
                                    d_work: torch.Tensor, first_partition: int = 0,
                                    partition_count: Optional[int] = None, stream=None) -> None:
    """Receive pass with the workers' packed parts and the output in host memory."""
    if partition_count is None:
        partition_count = cfg.num_partitions - first_partition
    ptrs = (C.c_void_p * len(h_packed))(*[_host_ptr(p) for p in h_packed])
    _check(lib().loco_unpack_dequant_reduce_host(C.byref(cfg.c()), ptrs, len(h_packed), n, first_partition,
                                                 partition_count, _host_ptr(h_out), _dev_ptr(d_work),
                                                 d_work.numel() * d_work.element_size(), _stream_ptr(stream)),
           "loco_unpack_dequant_reduce_host")


def loco_unpack_dequant_reduce_host_noalloc(cfg: Config, h_packed: Sequence[torch.Tensor], n: int, h_out: torch.Tensor,
                                            first_partition: int = 0, partition_count: Optional[int] = None,
                                            stream=None) -> None:
    """Receive pass on host buffers for callers that cannot hand over device memory (the framework's allocator
    holds it all, or allocation is banned where the call is made): the library stages through its own fixed
    array of NOALLOC_SCRATCH_BYTES instead of a workspace.  Larger requests raise LocoError(ERR_SIZE).  Calls on
    one device share that array, so keep them on one stream; make the first call outside stream capture."""
    if partition_count is None:
        partition_count = cfg.num_partitions - first_partition
    ptrs = (C.c_void_p * len(h_packed))(*[_host_ptr(p) for p in h_packed])
    _check(lib().loco_unpack_dequant_reduce_host_noalloc(C.byref(cfg.c()), ptrs, len(h_packed), n, first_partition,
                                                         partition_count, _host_ptr(h_out), _stream_ptr(stream)),
           "loco_unpack_dequant_reduce_host_noalloc")


def loco_selfcheck_block_division():
    """(mismatches of amax/qmax, mismatches of qmax/amax) of the kernels' short division sequences against the IEEE
    division over every positive finite fp32 amax; both must be 0.  Synchronous, about a second."""
    out = (C.c_uint64 * 2)(0, 0)
    _check(lib().loco_selfcheck_block_division(out), "loco_selfcheck_block_division")
    return int(out[0]), int(out[1])


def loco_unpack_dequant_reduce_adam(cfg: Config, packed: Sequence, n: int, m: torch.Tensor, v: torch.Tensor, theta: torch.Tensor,
                                    *, lr: float, beta1: float, beta2: float, delta: float, grad_out: Optional[torch.Tensor] = None,
                                    first_partition: int = 0, partition_count: Optional[int] = None, stream=None) -> None:
    """Receive pass (Eq. 8) fused with the paper's Adam-family step: m, v, theta (fp32 CUDA tensors covering the valid
    elements of the parts) are updated in place; grad_out, if given, also receives the averaged gradient."""
    if partition_count is None:
        partition_count = cfg.num_partitions - first_partition
    ptrs = (C.c_void_p * len(packed))(*[p if isinstance(p, int) else _dev_ptr(p) for p in packed])
    need = sum(loco_partition_elems(cfg, n, j) for j in range(first_partition, first_partition + partition_count))
    for t in (m, v, theta):
        if t.dtype != torch.float32 or t.numel() < need:
            raise ValueError("m, v, theta must be float32 with at least %d elements" % need)
    if grad_out is not None:
        want = torch.bfloat16 if cfg.out_dtype == BF16 else torch.float32
        if grad_out.dtype != want or grad_out.numel() < need:
            raise ValueError("grad_out must be %s with at least %d elements" % (want, need))
    ad = loco_adam_t(lr, beta1, beta2, delta)
    _check(lib().loco_unpack_dequant_reduce_adam(C.byref(cfg.c()), ptrs, len(packed), n, first_partition, partition_count,
                                                 C.byref(ad), _dev_ptr(m), _dev_ptr(v), _dev_ptr(theta), _dev_ptr(grad_out),
                                                 _stream_ptr(stream)), "loco_unpack_dequant_reduce_adam")
