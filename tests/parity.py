"""Helpers for the GPU-versus-oracle parity tests.

The CUDA library and the oracle are driven side by side on the same input bytes; nothing
here computes any part of the method.  Comparison rules: codes, scales, 8-bit state and
their layout are compared bit for bit; fp32 state and the averaged gradient within
1e-5 relative / 1e-7 absolute (they are expected to be bit-identical as well, and the
number of differing words is reported).
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import loco_oracle as orc
from paper_2407_04480_b200 import loco

CANARY = 0xA5
RTOL, ATOL = 1e-5, 1e-7


def both_configs(**kw):
    """Build the library's and the oracle's configuration from one set of keyword arguments."""
    stats = kw.pop("collect_stats", 1)
    g = loco.Config(collect_stats=stats, **kw)
    o = orc.OracleConfig(**kw)
    return g, o


def to_device(arr: np.ndarray, bf16: bool) -> torch.Tensor:
    t = torch.from_numpy(arr.view(np.int16) if bf16 else arr).cuda()
    return t.view(torch.bfloat16) if bf16 else t


def guarded(nbytes: int, fill: int = CANARY, guard: int = 512):
    """A uint8 CUDA tensor of nbytes with `guard` canary bytes on both sides; returns (whole, view)."""
    whole = torch.full((nbytes + 2 * guard,), fill, dtype=torch.uint8, device="cuda")
    return whole, whole[guard:guard + nbytes]


def check_guards(whole: torch.Tensor, nbytes: int, fill: int = CANARY, guard: int = 512):
    w = whole.cpu().numpy()
    assert (w[:guard] == fill).all(), "write before the start of a buffer"
    assert (w[guard + nbytes:] == fill).all(), "write past the end of a buffer"


class Worker:
    """One simulated worker: library state + oracle state for one bucket of n elements."""

    def __init__(self, gcfg, ocfg, n):
        self.gcfg, self.ocfg, self.n = gcfg, ocfg, n
        self.state_bytes = loco.loco_state_bytes(gcfg, n)
        self.packed_bytes = loco.loco_packed_bytes(gcfg, n)
        assert self.state_bytes == orc.state_bytes(ocfg, n)
        assert self.packed_bytes == orc.packed_bytes(ocfg, n)
        self.state_whole, state_view = guarded(max(self.state_bytes, 16))
        self.gstate = loco.State(gcfg, n, buffer=state_view)
        self.comm_whole, self.gcomm = guarded(max(self.packed_bytes, 16))
        # a twin with the statistics switched the other way: the kernels take a different branch for it
        import dataclasses
        self.tcfg = dataclasses.replace(gcfg, collect_stats=0 if gcfg.collect_stats else 1)
        self.tstate_whole, tstate_view = guarded(max(self.state_bytes, 16))
        self.tstate = loco.State(self.tcfg, n, buffer=tstate_view)
        self.tcomm_whole, self.tcomm = guarded(max(self.packed_bytes, 16))
        self.ostate = orc.new_state(ocfg, n)
        self.ocomm = orc.new_comm(ocfg, n, fill=CANARY)
        self.osat = 0
        self.ossat = 0
        self.oflags = 0

    def step(self, grad_np: np.ndarray, k: int):
        bf16 = self.gcfg.grad_dtype == loco.BF16
        g = to_device(grad_np, bf16)
        loco.loco_compensate_quantize_pack(self.gstate, g, self.gcomm, k)
        loco.loco_compensate_quantize_pack(self.tstate, g, self.tcomm, k)
        torch.cuda.synchronize()
        flags, sat, ssat = orc.send_step(self.ocfg, grad_np, self.ostate, self.ocomm, k, full_status=True)
        self.oflags |= flags
        self.osat += sat
        self.ossat += ssat

    def compare(self, where=""):
        self._compare(self.gcfg, self.gstate, self.gcomm, self.state_whole, self.comm_whole, where)
        self._compare(self.tcfg, self.tstate, self.tcomm, self.tstate_whole, self.tcomm_whole, where + " (twin)")

    def _compare(self, gcfg, gstate_obj, gcomm_t, state_whole, comm_whole, where):
        n, ocfg = self.n, self.ocfg
        gcomm = gcomm_t.cpu().numpy()
        gstate = gstate_obj.buffer.cpu().numpy()
        for j, ((gc, gs), (oc, os_)) in enumerate(zip(orc.comm_views(ocfg, n, gcomm), orc.comm_views(ocfg, n, self.ocomm))):
            bad = int((gc != oc).sum())
            assert bad == 0, "%s partition %d: %d code bytes differ (first at %d)" % (where, j, bad, int(np.argmax(gc != oc)))
            if gs is not None:
                assert np.array_equal(gs.view(np.uint32), os_.view(np.uint32)), "%s partition %d: scales differ" % (where, j)
        # bytes of a stride past the code and scale areas are never written
        lp = orc.partition_capacity(ocfg, n)
        stride = orc.partition_bytes(ocfg, n)
        used = lp * ocfg.bits // 8 + (4 * (lp // ocfg.block_size) if ocfg.scale_mode == orc.SCALE_BLOCK_ABSMAX else 0)
        for j in range(ocfg.num_partitions):
            assert (gcomm[j * stride + used:(j + 1) * stride] == CANARY).all(), "%s pad bytes written" % where
        gv, gsc = orc.state_views(ocfg, n, gstate)
        ov, osc = orc.state_views(ocfg, n, self.ostate)
        if ocfg.state_fmt == orc.STATE_INT8:
            bad = int((gv != ov).sum())
            assert bad == 0, "%s: %d int8 state codes differ (first at %d)" % (where, bad, int(np.argmax(gv != ov)))
            if gsc is not None:
                assert np.array_equal(gsc.view(np.uint32), osc.view(np.uint32)), "%s: state scales differ" % where
        elif gv is not None:
            assert np.allclose(gv, ov, rtol=RTOL, atol=ATOL, equal_nan=True), "%s: fp32 state out of tolerance" % where
            nbad = int((gv.view(np.uint32) != ov.view(np.uint32)).sum())
            assert nbad == 0, "%s: %d fp32 state words are not bit-identical" % (where, nbad)
        check_guards(state_whole, max(self.state_bytes, 16))
        check_guards(comm_whole, max(self.packed_bytes, 16))
        flags, sat, ssat = loco.loco_status_counters(gstate_obj)
        assert (flags, sat) == loco.loco_last_status(gstate_obj)
        assert flags == self.oflags, "%s: flags %d vs %d" % (where, flags, self.oflags)
        if gcfg.collect_stats:
            assert sat == self.osat, "%s: saturated %d vs %d" % (where, sat, self.osat)
            assert ssat == self.ossat, "%s: saturated error codes %d vs %d" % (where, ssat, self.ossat)
        else:
            assert sat == 0 and ssat == 0


def reduce_both(gcfg, ocfg, n, workers, first=0, count=None):
    """Run the receive pass on the workers' library buffers and the oracle on the oracle's buffers."""
    if count is None:
        count = gcfg.num_partitions - first
    stride = loco.loco_partition_bytes(gcfg, n)
    n_out = sum(loco.loco_partition_elems(gcfg, n, j) for j in range(first, first + count))
    esize = 2 if gcfg.out_dtype == loco.BF16 else 4
    whole, view = guarded(max(n_out * esize, 16))
    out = view[:n_out * esize].view(torch.bfloat16 if esize == 2 else torch.float32)
    packed = [w.gcomm[first * stride:] for w in workers]
    loco.loco_unpack_dequant_reduce(gcfg, packed, n, out, first_partition=first, partition_count=count)
    torch.cuda.synchronize()
    check_guards(whole, max(n_out * esize, 16))
    got = out.view(torch.int16).cpu().numpy().view(np.uint16) if esize == 2 else out.cpu().numpy()
    want = orc.reduce(ocfg, n, [w.ocomm for w in workers], first=first, count=count)
    return got, want


def assert_reduced_equal(got, want, bf16, where=""):
    if bf16:
        bad = int((got != want).sum())
        assert bad == 0, "%s: %d bf16 outputs differ" % (where, bad)
    else:
        assert np.allclose(got, want, rtol=RTOL, atol=ATOL), "%s: averaged gradient out of tolerance" % where
        nbad = int((got.view(np.uint32) != want.view(np.uint32)).sum())
        assert nbad == 0, "%s: %d fp32 outputs are not bit-identical" % (where, nbad)
