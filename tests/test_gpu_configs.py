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
    parts, 4-bit codes, T_c = 512: eight ordinary iterations, then iterations 510 ... 515 and 1022 ... 1026 (the reset
    fires at 512 and 1024); then the 8-worker reduce of all parts."""
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
    ks = list(range(1, 9)) + list(range(510, 516)) + list(range(1022, 1027))
    for k in ks:
        _fill_gaussian_bf16(grad, 1e-4, seed=2, worker=0, step=k)
        wb.step(grad, k)
        wb.compare("k=%d" % k)
        if k in (512, 1024):
            assert not bool(wb.state.buffer[:1 << 20].any()), "reset must zero the state"
            assert not bool(wb.state.buffer[n - (1 << 20):n].any()), "reset must zero the state"
    assert len(wb.windows) >= 20 and wb.compared >= len(ks) * 20 * (1 << 17)
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
    all-zero; 8 workers each compress their own gradient for 8 iterations; then the 8-worker reduce."""
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
    for k in range(1, 9):
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
    """n = 2^16 .. 2^24: every byte against the oracle, 2 iterations, then reduces over 1..16 workers."""
    for log2n in (16, 18, 20, 22, 24):
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
        for N in ((1, 2, 4, 8, 16) if log2n < 24 else (1, 8, 16)):
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


# ---------------------------------------------------------------- config 4, the view of one rank under expert parallelism 8

def test_config4_mixtral_per_rank_view():
    """Expert parallelism 8: a rank holds one expert of each of the 32 layers (32 x 176,160,768 elements) and the shared
    parameters (1,605,636,096): one flat bf16 buffer of 7,242,780,672 elements, heavy-tailed values, every fourth
    expert all-zero (an expert no token was routed to), 8 parts, fixed and block scales, 2 iterations."""
    if _free_gb() < 60:
        pytest.skip("needs ~45 GB of free device memory")
    expert, shared = 3 * 4096 * 14336, 1_605_636_096
    n = 32 * expert + shared
    assert n == 7_242_780_672
    grad = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    for mode in (loco.SCALE_FIXED, loco.SCALE_BLOCK_ABSMAX):
        gcfg = loco.Config(bits=4, scale_mode=mode, block_size=256, s=2.0 ** 14, s_e=2.0 ** 16, beta=0.5, reset_period=0,
                           state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=8)
        lp = loco.loco_partition_capacity(gcfg, n)
        wins = _windows(n, lp, 8, 1 << 17, 6, seed=6)
        for e in (3, 4, 31):                       # the start of a dead expert, of a live one, of the last one
            s0 = (e * expert + 255) // 256 * 256
            wins.append((s0, min(1 << 16, (s0 // lp + 1) * lp - s0)))
        wb = WindowedBucket(gcfg, n, wins)
        chunk = 1 << 27
        for k in (1, 2):
            for off in range(0, n, chunk):
                m = min(chunk, n - off)
                grad[off:off + m] = inputs.student_t(m, 3.0, 1e-4, seed=3, worker=0, step=k, tag=off >> 8, dtype=torch.bfloat16, device="cuda")
            for e in range(3, 32, 4):
                grad[e * expert:(e + 1) * expert] = 0
            wb.step(grad, k)
            wb.compare("mode %d k=%d" % (mode, k))
        del wb
    del grad


# ---------------------------------------------------------------- config 2: Llama-2-7B buckets over 100 iterations

def test_config2_llama_buckets_100_iterations():
    """Twelve 25M-element buckets of the Llama-2-7B layout -- the first, the partial last one, buckets that straddle
    tensors, the buckets of the layer groups with the largest and the smallest gradient scale -- each with 8 workers over
    100 iterations with T_c = 32 (three resets); the oracle follows windows of every bucket and worker (head, ragged tail,
    a part boundary, a random place); the 8-worker average is compared at iterations around a reset and at the end."""
    if _free_gb() < 12:
        pytest.skip("needs ~8 GB of free device memory")
    layout = inputs.llama2_7b()
    scales = inputs.group_scales(1, layout.n_groups)
    buckets = inputs.bucket_ranges(layout.numel, 25_000_000)
    assert len(buckets) == 270 and buckets[-1][1] - buckets[-1][0] == 13_415_616
    # first element of every layer group, to find the buckets of the extreme scales
    starts, pos = {}, 0
    for numel, grp in layout.segments:
        starts.setdefault(grp, pos)
        pos += numel
    big = max(range(1, 33), key=lambda g: scales[g])
    small = min(range(1, 33), key=lambda g: scales[g])
    picked = {0, 269, 5, starts[big] // 25_000_000 + 1, starts[small] // 25_000_000 + 1}
    rng = np.random.default_rng(12)
    while len(picked) < 12:
        picked.add(int(rng.integers(1, 269)))
    gcfg = loco.Config(bits=4, s=2.0 ** 14, s_e=2.0 ** 16, beta=0.5, reset_period=32, state_fmt=loco.STATE_INT8,
                       grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=8)
    workers = 8
    cells = []
    for b in sorted(picked):
        lo, hi = buckets[b]
        n = hi - lo
        lp = loco.loco_partition_capacity(gcfg, n)
        tail = max(0, (n - 1) // 256 * 256 - 4096)
        wins = [(0, 8192), (tail, n - tail), (3 * lp - 4096, 4096), (3 * lp, 4096)]
        s0 = int(rng.integers(0, n // 256 - 64)) * 256
        wins.append((s0, min(8192, (s0 // lp + 1) * lp - s0)))
        cells.append((b, lo, hi, [WindowedBucket(gcfg, n, wins) for _ in range(workers)]))
    check_reduce_at = {0, 31, 32, 33, 64, 99}
    for k in range(100):
        for b, lo, hi, wbs in cells:
            for w, wb in enumerate(wbs):
                g = inputs.layout_slice(layout, lo, hi, scales, 1e-4, seed=1, worker=w, step=k, device="cuda")
                wb.step(g, k)
            if k in check_reduce_at or k % 10 == 0:
                for wb in wbs:
                    wb.compare("bucket %d k=%d" % (b, k))
            if k in check_reduce_at:
                n = hi - lo
                out = torch.empty(n, dtype=torch.bfloat16, device="cuda")
                comms = [wb.comm for wb in wbs]
                loco.loco_unpack_dequant_reduce(gcfg, comms, n, out)
                torch.cuda.synchronize()
                wbs[0].compare_reduce(comms, out, "bucket %d k=%d" % (b, k))
    for b, lo, hi, wbs in cells:
        for wb in wbs:
            wb.compare("bucket %d end" % b)


# ---------------------------------------------------------------- more than 2^32 elements in ONE part

def test_block_scales_with_more_than_2_to_32_elements_in_one_part():
    """4,400,000,512 bf16 elements in a single part (num_partitions = 1), one scale per 256 elements: partition-local
    element indices and scale indices beyond 2^32.  Windows on both sides of the 2^32-nd element and at the ragged end;
    then the 2-worker average of the whole part."""
    if _free_gb() < 40:
        pytest.skip("needs ~30 GB of free device memory")
    n = 4_400_000_512 + 77
    gcfg = loco.Config(bits=4, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=256, beta=0.5, reset_period=0,
                       state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=1)
    lp = loco.loco_partition_capacity(gcfg, n)
    assert lp >= n > 1 << 32
    wins = _windows(n, lp, 1, 1 << 17, 4, seed=7) + [((1 << 32) - (1 << 16), 1 << 17), ((1 << 32) + 512 * 7, 1 << 16)]
    wb = WindowedBucket(gcfg, n, wins)
    grad = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    for k in (1, 2):
        _fill_gaussian_bf16(grad, 1e-3, seed=8, worker=0, step=k)
        wb.step(grad, k)
        wb.compare("k=%d" % k)
    del grad
    out = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    other = wb.comm.clone()
    loco.loco_unpack_dequant_reduce(gcfg, [wb.comm, other], n, out)
    torch.cuda.synchronize()
    wb.compare_reduce([wb.comm, other], out, "reduce")


def test_adam_fused_part_with_more_than_4_gib_of_codes():
    """The receive pass fused with the Adam-family step on one part whose 8-bit codes fill more than 4 GiB (4,300,000,256
    elements, 1 worker, non-power-of-two s so that the generic path runs): moments and weights of windows on both sides of
    the 4-GiB offset against the oracle."""
    if _free_gb() < 70:
        pytest.skip("needs ~60 GB of free device memory")
    n = 4_300_000_256 + 33
    kw = dict(bits=8, s=3000.0, s_e=12000.0, beta=0.5, reset_period=0, state_fmt=loco.STATE_NONE, grad_dtype=loco.BF16,
              out_dtype=loco.F32, num_partitions=1)
    gcfg = loco.Config(**kw)
    pb = loco.loco_packed_bytes(gcfg, n)
    assert pb > 1 << 32
    comm = _random_codes(pb, 900)
    m = torch.zeros(n, dtype=torch.float32, device="cuda")
    v = torch.zeros(n, dtype=torch.float32, device="cuda")
    theta = torch.ones(n, dtype=torch.float32, device="cuda")
    ad = dict(lr=1e-3, beta1=0.1, beta2=0.001, delta=1e-16)
    loco.loco_unpack_dequant_reduce_adam(gcfg, [comm], n, m, v, theta, **ad)
    torch.cuda.synchronize()
    ocfg = orc.OracleConfig(**kw)
    for s0 in (0, (1 << 32) - (1 << 15), (1 << 32) + 4096, n - 5000):
        ln = min(1 << 16, n - s0)
        mini = orc.new_comm(ocfg, ln)
        mini[:ln] = comm[s0:s0 + ln].cpu().numpy()
        om, ov, ot = np.zeros(ln, np.float32), np.zeros(ln, np.float32), np.ones(ln, np.float32)
        orc.reduce_adam(ocfg, ln, [mini], om, ov, ot, **ad)
        for got, want, name in ((m, om, "m"), (v, ov, "v"), (theta, ot, "theta")):
            g = got[s0:s0 + ln].cpu().numpy()
            assert np.array_equal(g.view(np.uint32), want.view(np.uint32)), "%s differs in window at %d" % (name, s0)
