"""GPU parity at the full sizes of the workload configurations, on windows of the buffers.

The oracle cannot walk 10^9..10^10 elements in a test, but with a global scale every element, and with block
scales every block, is computed independently of the rest of the bucket.  So the library processes the whole
buffer in the launch configuration the benchmark uses (one launch per bucket / flat buffer, all parts), and the
oracle recomputes seeded windows of it (the head, the ragged tail, both sides of part boundaries, random places)
as small buckets of their own; codes, scales and 8-bit state of each window are compared bit for bit, the
averaged gradient bit for bit as well.  Where a window sits inside the wire layout is restated here from the
layout's written definition (include/loco.h)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import loco_oracle as orc
from paper_2407_04480_b200 import inputs, loco

pytestmark = pytest.mark.gpu


def _free_gb():
    free, _ = torch.cuda.mem_get_info()
    return free / 2 ** 30


def _windows(n, lp, parts, length, extra, seed):
    """Window starts (multiples of 256, each window inside one part): head, tail, around part boundaries, random."""
    starts = {0}
    last = max(0, (n - 1) // 256 * 256 - length + 256)
    starts.add(max(0, min(last, (n // 256) * 256)))            # the ragged tail (may be shorter than `length`)
    starts.add(max(0, last - 256 * 3))
    for j in range(1, parts):
        b = j * lp
        if b < n:
            starts.add(b)
            if b >= length:
                starts.add(b - length)
    rng = np.random.default_rng(seed)
    for _ in range(extra):
        starts.add(int(rng.integers(0, max(1, n // 256))) * 256)
    out = []
    for s in sorted(starts):
        if s >= n:
            continue
        j = s // lp
        end = min(s + length, n, (j + 1) * lp)
        if end > s:
            out.append((s, end - s))
    return out


class WindowedBucket:
    """The library on the whole buffer, the oracle on windows of it."""

    def __init__(self, gcfg, n, windows):
        self.gcfg, self.n, self.windows = gcfg, n, windows
        kw = dataclasses.asdict(gcfg)
        kw.pop("collect_stats")
        kw["num_partitions"] = 1
        self.ocfg = orc.OracleConfig(**kw)
        self.state = loco.State(gcfg, n)
        self.comm = torch.empty(loco.loco_packed_bytes(gcfg, n), dtype=torch.uint8, device="cuda")
        self.lp = loco.loco_partition_capacity(gcfg, n)
        self.stride = loco.loco_partition_bytes(gcfg, n)
        self.ostate = [orc.new_state(self.ocfg, ln) for _, ln in windows]
        self.ocomm = [orc.new_comm(self.ocfg, ln) for _, ln in windows]

    def step(self, grad: torch.Tensor, k: int):
        loco.loco_compensate_quantize_pack(self.state, grad, self.comm, k)
        for (s, ln), ost, ocm in zip(self.windows, self.ostate, self.ocomm):
            orc.send_step(self.ocfg, inputs.as_numpy_bits(grad[s:s + ln]), ost, ocm, k)
        torch.cuda.synchronize()

    def window_bytes(self, comm: torch.Tensor, s: int, ln: int):
        """(code bytes, block scales or None) of bucket elements [s, s+ln) inside a packed buffer."""
        cfg = self.gcfg
        j, o = s // self.lp, s % self.lp
        base = j * self.stride
        c0 = base + o * cfg.bits // 8
        codes = comm[c0:c0 + (ln * cfg.bits + 7) // 8].cpu().numpy()
        scales = None
        if cfg.scale_mode == loco.SCALE_BLOCK_ABSMAX:
            B = cfg.block_size
            s0 = base + self.lp * cfg.bits // 8 + (o // B) * 4
            scales = comm[s0:s0 + 4 * ((ln + B - 1) // B)].cpu().numpy().view(np.float32)
        return codes, scales

    def compare(self, where=""):
        cfg = self.gcfg
        self.compared = getattr(self, "compared", 0)
        for (s, ln), ost, ocm in zip(self.windows, self.ostate, self.ocomm):
            self.compared += ln
            tag = "%s window [%d, +%d)" % (where, s, ln)
            codes, scales = self.window_bytes(self.comm, s, ln)
            (oc, osc), = orc.comm_views(self.ocfg, ln, ocm)
            nb = (ln * cfg.bits + 7) // 8
            assert np.array_equal(codes, oc[:nb]), "%s: code bytes differ" % tag
            if scales is not None:
                assert np.array_equal(scales.view(np.uint32), osc[:scales.size].view(np.uint32)), "%s: scales differ" % tag
            if cfg.state_fmt == loco.STATE_INT8:
                got = self.state.buffer[s:s + ln].cpu().numpy().view(np.int8)
                ov, oss = orc.state_views(self.ocfg, ln, ost)
                assert np.array_equal(got, ov), "%s: 8-bit state differs" % tag
                if oss is not None:
                    B = cfg.block_size
                    off = (self.n + 255) // 256 * 256 + (s // B) * 4
                    gs = self.state.buffer[off:off + 4 * oss.size].cpu().numpy().view(np.float32)
                    assert np.array_equal(gs.view(np.uint32), oss.view(np.uint32)), "%s: state scales differ" % tag
            elif cfg.state_fmt in (loco.STATE_FP32, loco.STATE_FP32_Q8COMP):
                got = self.state.buffer[4 * s:4 * (s + ln)].cpu().numpy().view(np.uint32)
                ov, _ = orc.state_views(self.ocfg, ln, ost)
                assert np.array_equal(got, ov.view(np.uint32)), "%s: fp32 state differs" % tag

    def compare_reduce(self, comms, out: torch.Tensor, where=""):
        """comms: every worker's whole packed buffer on the GPU; out: the library's averaged gradient (n elements)."""
        cfg = self.gcfg
        ocfg = dataclasses.replace(self.ocfg, out_dtype=cfg.out_dtype)
        for (s, ln) in self.windows:
            minis = []
            for cm in comms:
                codes, scales = self.window_bytes(cm, s, ln)
                mini = orc.new_comm(ocfg, ln)
                mini[:codes.size] = codes
                if scales is not None:
                    cap = orc.partition_capacity(ocfg, ln)
                    mini[cap * cfg.bits // 8: cap * cfg.bits // 8 + 4 * scales.size] = scales.view(np.uint8)
                minis.append(mini)
            want = orc.reduce(ocfg, ln, minis)
            got = out[s:s + ln]
            got = got.view(torch.int16).cpu().numpy().view(np.uint16) if cfg.out_dtype == loco.BF16 else got.cpu().numpy().view(np.uint32)
            want = want if cfg.out_dtype == loco.BF16 else want.view(np.uint32)
            assert np.array_equal(got, want), "%s window [%d, +%d): averaged gradient differs" % (where, s, ln)


def _fill_gaussian_bf16(dst: torch.Tensor, sigma: float, seed: int, worker: int, step: int):
    chunk = 1 << 28
    for off in range(0, dst.numel(), chunk):
        m = min(chunk, dst.numel() - off)
        dst[off:off + m] = inputs.gaussian(m, sigma, seed=seed, worker=worker, step=step, tag=off >> 8, dtype=torch.bfloat16, device="cuda")


def _random_codes(nbytes: int, seed: int) -> torch.Tensor:
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    out = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    chunk = 1 << 30
    for off in range(0, nbytes, chunk):
        m = min(chunk, nbytes - off)
        out[off:off + m] = torch.randint(0, 256, (m,), dtype=torch.uint8, device="cuda", generator=g)
    return out


# ---------------------------------------------------------------- config 3: 13B flat buffer, 8 parts, reset at 512

def test_config3_dense_13b_flat_buffer():
    """One flat bf16 buffer of 13,015,864,320 elements (more than 2^32: 64-bit indexing), reduce-scatter layout of 8
    parts, 4-bit codes, T_c = 512: iterations 511, 512 (reset fires), 513; then the 8-worker reduce of all parts."""
    if _free_gb() < 110:
        pytest.skip("needs ~105 GB of free device memory")
    layout = inputs.dense_13b()
    n = layout.numel
    assert n == 13_015_864_320
    gcfg = loco.Config(bits=4, s=2.0 ** 14, s_e=2.0 ** 16, beta=0.5, reset_period=512, state_fmt=loco.STATE_INT8,
                       grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=8)
    lp = loco.loco_partition_capacity(gcfg, n)
    assert lp * 8 >= n and loco.loco_partition_elems(gcfg, n, 7) == n - 7 * lp
    wb = WindowedBucket(gcfg, n, _windows(n, lp, 8, 1 << 18, 10, seed=3))
    grad = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    for k in (511, 512, 513):
        _fill_gaussian_bf16(grad, 1e-4, seed=2, worker=0, step=k)
        wb.step(grad, k)
        wb.compare("k=%d" % k)
        if k == 512:
            assert not bool(wb.state.buffer[:1 << 20].any()), "reset must zero the state"
    assert len(wb.windows) >= 20 and wb.compared >= 3 * 20 * (1 << 17)
    assert bool(wb.comm[:1 << 20].any()) and bool(wb.state.buffer[:1 << 20].any())
    del grad
    pb = loco.loco_packed_bytes(gcfg, n)
    comms = [wb.comm] + [_random_codes(pb, 100 + w) for w in range(7)]
    out = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    loco.loco_unpack_dequant_reduce(gcfg, comms, n, out)
    torch.cuda.synchronize()
    wb.compare_reduce(comms, out, "reduce")
    # one part at a time, as the owner rank of that part would do it
    for j in (0, 7):
        first = j * lp
        cnt = loco.loco_partition_elems(gcfg, n, j)
        part = torch.empty(cnt, dtype=torch.bfloat16, device="cuda")
        loco.loco_unpack_dequant_reduce(gcfg, [c[j * wb.stride:] for c in comms], n, part, first_partition=j, partition_count=1)
        torch.cuda.synchronize()
        assert torch.equal(part.view(torch.int16), out[first:first + cnt].view(torch.int16))


# ---------------------------------------------------------------- config 4: one Mixtral-8x7B layer, heavy tails, dead experts

@pytest.mark.parametrize("mode", [loco.SCALE_FIXED, loco.SCALE_BLOCK_ABSMAX])
def test_config4_mixtral_layer(mode):
    """One decoder layer (1,451,270,144 elements incl. 8 experts of 176,160,768), Student-t(3) x 1e-4 values, 2 of 8 experts
    all-zero; 8 workers each compress their own gradient for 3 iterations; then the 8-worker reduce."""
    if _free_gb() < 40:
        pytest.skip("needs ~35 GB of free device memory")
    layout = inputs.mixtral_layer()
    n = layout.numel
    assert n == 1_451_270_144
    scales = inputs.zero_expert_scales(3, layer=0)
    assert scales.count(0.0) == 2
    gcfg = loco.Config(bits=4, scale_mode=mode, block_size=256, s=2.0 ** 14, s_e=2.0 ** 16, beta=0.5, reset_period=0,
                       state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=8)
    lp = loco.loco_partition_capacity(gcfg, n)
    wins = _windows(n, lp, 8, 1 << 17, 6, seed=4)
    # make sure a dead expert is looked at: the first element of every expert
    pos = 0
    for numel, grp in layout.segments:
        if grp >= 1 and scales[grp] == 0.0:
            s0 = (pos + 255) // 256 * 256
            j = s0 // lp
            wins.append((s0, min(1 << 16, (j + 1) * lp - s0)))
        pos += numel
    workers = [WindowedBucket(gcfg, n, wins if w in (0, 7) else []) for w in range(8)]
    grad = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    chunk = 1 << 27
    for k in (1, 2, 3):
        for w, wb in enumerate(workers):
            for off in range(0, n, chunk):
                hi = min(off + chunk, n)
                grad[off:hi] = inputs.layout_slice(layout, off, hi, scales, 1e-4, seed=3, worker=w, step=k, dist="student_t", device="cuda")
            wb.step(grad, k)
        workers[0].compare("worker 0 k=%d" % k)
        workers[7].compare("worker 7 k=%d" % k)
    del grad
    comms = [wb.comm for wb in workers]
    out = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    loco.loco_unpack_dequant_reduce(gcfg, comms, n, out)
    torch.cuda.synchronize()
    workers[0].compare_reduce(comms, out, "reduce")


# ---------------------------------------------------------------- config 5: size / width / worker-count sweep

@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("gd", [loco.F32, loco.BF16])
def test_config5_sweep_small_sizes_full(bits, gd):
    """n = 2^16 .. 2^22: every byte against the oracle, 2 iterations, then reduces over 1..16 workers."""
    for log2n in (16, 18, 20, 22):
        n = 1 << log2n
        gcfg = loco.Config(bits=bits, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=loco.STATE_INT8,
                           grad_dtype=gd, out_dtype=gd, num_partitions=1)
        dt = torch.bfloat16 if gd == loco.BF16 else torch.float32
        workers = [WindowedBucket(gcfg, n, [(0, n)]) for _ in range(2)]
        for k in (1, 2):
            for w, wb in enumerate(workers):
                wb.step(inputs.gaussian(n, 1e-3, seed=4, worker=w, step=k, dtype=dt, device="cuda"), k)
        for wb in workers:
            wb.compare("n=2^%d" % log2n)
        pb = loco.loco_packed_bytes(gcfg, n)
        comms = [wb.comm for wb in workers] + [_random_codes(pb, 200 + w) for w in range(14)]
        for N in (1, 2, 4, 8, 16):
            out = torch.empty(n, dtype=dt, device="cuda")
            loco.loco_unpack_dequant_reduce(gcfg, comms[:N], n, out)
            torch.cuda.synchronize()
            workers[0].compare_reduce(comms[:N], out, "n=2^%d N=%d" % (log2n, N))


@pytest.mark.parametrize("bits,gd,log2n", [(4, loco.BF16, 30), (4, loco.F32, 27), (2, loco.BF16, 27), (8, loco.F32, 30), (8, loco.BF16, 27)])
def test_config5_sweep_large_sizes_windows(bits, gd, log2n):
    """n = 2^27 and 2^30 (1 Gi elements): windows of the buffer, 2 iterations, 16-worker reduce."""
    n = 1 << log2n
    esize = 2 if gd == loco.BF16 else 4
    need = n * (esize + 1 + bits / 8 * 16 + esize) / 2 ** 30 + 4
    if _free_gb() < need:
        pytest.skip("needs ~%d GB of free device memory" % need)
    gcfg = loco.Config(bits=bits, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=loco.STATE_INT8,
                       grad_dtype=gd, out_dtype=gd, num_partitions=4)
    dt = torch.bfloat16 if gd == loco.BF16 else torch.float32
    lp = loco.loco_partition_capacity(gcfg, n)
    wb = WindowedBucket(gcfg, n, _windows(n, lp, 4, 1 << 18, 8, seed=5))
    grad = torch.empty(n, dtype=dt, device="cuda")
    chunk = 1 << 27
    for k in (1, 2):
        for off in range(0, n, chunk):
            grad[off:off + chunk] = inputs.gaussian(min(chunk, n - off), 1e-3, seed=4, step=k, tag=off >> 8, dtype=dt, device="cuda")
        wb.step(grad, k)
        wb.compare("k=%d" % k)
    del grad
    pb = loco.loco_packed_bytes(gcfg, n)
    comms = [wb.comm] + [_random_codes(pb, 300 + w) for w in range(15)]
    out = torch.empty(n, dtype=dt, device="cuda")
    loco.loco_unpack_dequant_reduce(gcfg, comms, n, out)
    torch.cuda.synchronize()
    wb.compare_reduce(comms, out, "N=16")
