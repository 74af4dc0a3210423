"""GPU parity for what sits around the paper's 4-bit path: the sign code ("1-bit LoCo"), blocks wider than a warp's row
(512 ... 4096 elements), the counter of clamped 8-bit error codes, and the table-driven multi-bucket send kernel.
Everything is compared with the CPU oracle on the same bytes: codes, scales and the 8-bit state bit for bit."""
import numpy as np
import pytest
import torch

from oracle import loco_oracle as orc
from paper_2407_04480_b200 import inputs, loco
from tests.parity import Worker, assert_reduced_equal, both_configs, reduce_both

pytestmark = pytest.mark.gpu


def run_steps(gcfg, ocfg, n, steps, sigma, seed, worker=0, k0=1, plant=None):
    w = Worker(gcfg, ocfg, n)
    dt = torch.bfloat16 if gcfg.grad_dtype == loco.BF16 else torch.float32
    for i in range(steps):
        g = inputs.gaussian(n, sigma, seed=seed, worker=worker, step=i, dtype=dt, device="cuda")
        if plant is not None:
            plant(g, i)
        w.step(inputs.as_numpy_bits(g), k0 + i)
        w.compare("step %d" % (k0 + i))
    return w


# ---------------------------------------------------------------- sign code

@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32, loco.STATE_NONE, loco.STATE_FP32_Q8COMP])
@pytest.mark.parametrize("gd", [loco.F32, loco.BF16])
def test_sign_code_global_scale(fmt, gd):
    n = (1 << 20) + 777
    gcfg, ocfg = both_configs(bits=1, s=2.0 ** 10, s_e=2.0 ** 13, beta=0.5, reset_period=3, state_fmt=fmt, grad_dtype=gd,
                              out_dtype=gd, num_partitions=3)
    ws = [run_steps(gcfg, ocfg, n, 4, 1e-3, seed=21, worker=w) for w in range(3)]
    got, want = reduce_both(gcfg, ocfg, n, ws)
    assert_reduced_equal(got, want, gd == loco.BF16)


@pytest.mark.parametrize("B", [32, 64, 256, 512, 2048])
@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32])
def test_sign_code_block_scale(B, fmt):
    n = 700_001
    gcfg, ocfg = both_configs(bits=1, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=B, beta=0.25, reset_period=3,
                              state_fmt=fmt, grad_dtype=loco.BF16, out_dtype=loco.F32, num_partitions=2)
    ws = [run_steps(gcfg, ocfg, n, 4, 1e-3, seed=22, worker=w) for w in range(2)]
    got, want = reduce_both(gcfg, ocfg, n, ws)
    assert_reduced_equal(got, want, False)


@pytest.mark.parametrize("mode", [loco.SCALE_FIXED, loco.SCALE_BLOCK_ABSMAX])
def test_sign_code_ragged_and_special_values(mode):
    def plant(g, i):
        if g.numel() >= 64:
            vals = torch.tensor([0.0, -0.0, float("nan"), float("inf"), -float("inf"), 1e-30, -1e-30, 3e38], device=g.device)
            g[5:5 + vals.numel()] = vals.to(g.dtype)
    for n in (1, 7, 15, 16, 17, 255, 256, 513, 4097, 65537):
        for gd in (loco.F32, loco.BF16):
            gcfg, ocfg = both_configs(bits=1, scale_mode=mode, block_size=64, s=2.0 ** 9, s_e=2.0 ** 12, beta=0.5,
                                      reset_period=0, state_fmt=loco.STATE_FP32, grad_dtype=gd, out_dtype=gd, num_partitions=3)
            ws = [run_steps(gcfg, ocfg, n, 2, 2e-3, seed=23, worker=w, plant=plant) for w in range(2)]
            got, want = reduce_both(gcfg, ocfg, n, ws)          # non-finite elements do not enter a block's mean
            assert_reduced_equal(got, want, gd == loco.BF16, "n=%d" % n)


@pytest.mark.parametrize("N", [1, 2, 3, 5, 8, 13, 16, 17])
@pytest.mark.parametrize("s", [3000.0, 2.0 ** 10])
def test_sign_code_reduce_workers(N, s):
    """Non-power-of-two s: +-fl(1/s) summed in worker order; power-of-two s and at most 16 workers: the negative
    workers of every element are counted and the sum is exact."""
    n = 300_003
    gcfg, ocfg = both_configs(bits=1, s=s, s_e=4 * s, beta=0.5, reset_period=0, state_fmt=loco.STATE_NONE,
                              grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=4)
    ws = [run_steps(gcfg, ocfg, n, 1, 1e-3, seed=24, worker=w) for w in range(N)]
    got, want = reduce_both(gcfg, ocfg, n, ws)
    assert_reduced_equal(got, want, True)
    got, want = reduce_both(gcfg, ocfg, n, ws, first=1, count=2)
    assert_reduced_equal(got, want, True)


@pytest.mark.parametrize("s", [3000.0, 2.0 ** 10])
@pytest.mark.parametrize("mode", [loco.SCALE_FIXED, loco.SCALE_BLOCK_ABSMAX])
def test_sign_code_receive_fused_with_the_adam_family_step(s, mode):
    from tests.test_gpu_adam import _check
    gcfg, _ = both_configs(bits=1, scale_mode=mode, block_size=128, s=s, s_e=4 * s, beta=0.5, reset_period=0,
                           state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, out_dtype=loco.F32, num_partitions=2)
    for workers in (3, 8):
        _check(gcfg, 200_003, workers, seed=25)


def test_sign_code_rejects_stochastic_rounding():
    cfg = loco.Config(bits=1, rounding=loco.ROUND_STOCHASTIC)
    assert loco.loco_config_check(cfg) == loco.ERR_ARG


# ---------------------------------------------------------------- blocks wider than a wide row

@pytest.mark.parametrize("B", [512, 1024, 4096])
@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32, loco.STATE_NONE])
def test_wide_blocks(B, bits, fmt):
    assert loco.loco_config_check(loco.Config(scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=B)) == loco.OK
    n = 600_000 + B // 2 + 3                       # a ragged last block
    gcfg, ocfg = both_configs(bits=bits, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=B, beta=0.5, reset_period=3,
                              state_fmt=fmt, grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=3)

    def plant(g, i):                               # one all-zero block, one block with an Inf, one with a NaN
        g[2 * B:3 * B] = 0
        if i == 1:
            g[5 * B + 7] = float("inf")
            g[9 * B + B - 1] = float("nan")

    ws = [run_steps(gcfg, ocfg, n, 4, 1e-3, seed=31, worker=w, plant=plant if w == 0 else None) for w in range(2)]
    got, want = reduce_both(gcfg, ocfg, n, ws[1:])            # worker 0's scales include a non-finite one
    assert_reduced_equal(got, want, True)


@pytest.mark.parametrize("B", [512, 2048])
def test_wide_blocks_small_and_ragged(B):
    for n in (1, 100, B - 1, B, B + 1, 3 * B + 17, 10 * B):
        gcfg, ocfg = both_configs(bits=4, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=B, beta=0.5, reset_period=0,
                                  state_fmt=loco.STATE_INT8, grad_dtype=loco.F32, out_dtype=loco.F32, num_partitions=2)
        ws = [run_steps(gcfg, ocfg, n, 3, 1e-3, seed=32, worker=w) for w in range(3)]
        got, want = reduce_both(gcfg, ocfg, n, ws)
        assert_reduced_equal(got, want, False, "n=%d" % n)


@pytest.mark.parametrize("B", [64, 256, 512, 1024, 4096])
def test_block_whose_error_maximum_is_below_the_fast_range(B):
    """The fast routine gives a row up at two points: the block maximum of h outside [2^-100, 2^100], and the block maximum of
    the new error outside it.  Here the second one alone fires: |h| <= 2^-90, every h one ulp beside a multiple of the block's
    scale, so the error is ~2^-115 everywhere in the block.  With blocks wider than a row all warps of the block must give up
    together, and the block is redone by one of them."""
    n = 40 * 4096 + 1234
    gcfg, ocfg = both_configs(bits=4, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=B, beta=0.5, reset_period=0,
                              state_fmt=loco.STATE_INT8, grad_dtype=loco.F32, out_dtype=loco.F32, num_partitions=2)
    rng = np.random.default_rng(77)
    amax = np.float32(2.0 ** -90)
    scale = np.float32(amax / np.float32(7.0))

    def plant(g, i):
        if i != 0:
            return
        for blk in (3, 17):                                      # two blocks of the first partition
            kq = rng.integers(-6, 7, B).astype(np.float32)
            h = (kq * scale).astype(np.float32)
            h = np.nextafter(h, np.float32(np.inf)).astype(np.float32)     # one ulp off the code's value (0 becomes the smallest denormal)
            h[0] = amax
            g[blk * B:(blk + 1) * B] = torch.from_numpy(h).to(g.device)

    ws = [run_steps(gcfg, ocfg, n, 3, 1e-3, seed=41, worker=w, plant=plant) for w in range(2)]
    got, want = reduce_both(gcfg, ocfg, n, ws)
    assert_reduced_equal(got, want, False)


# ---------------------------------------------------------------- clamped 8-bit error codes are counted

@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32_Q8COMP])
@pytest.mark.parametrize("s_e_factor", [4.0, 6.0])
def test_state_saturation_counter(fmt, s_e_factor):
    """The paper's s = 2^19 with gradients of size 1e-3: every gradient code and nearly every error code is clamped."""
    n = 500_001
    s = 2.0 ** 19
    gcfg, ocfg = both_configs(bits=4, s=s, s_e=s_e_factor * s, beta=0.5, reset_period=0, state_fmt=fmt, grad_dtype=loco.BF16,
                              out_dtype=loco.BF16)
    w = run_steps(gcfg, ocfg, n, 3, 1e-3, seed=41)
    assert w.ossat > n                              # the case is exercised (Worker.compare checks the equality)


# ---------------------------------------------------------------- multi-bucket send: one launch walking a table of buckets

def _multi_case(kw, sizes, steps=3, sigma=1e-3, plant=None, collect_stats=1):
    gcfg, ocfg = both_configs(collect_stats=collect_stats, **kw)
    dt = torch.bfloat16 if gcfg.grad_dtype == loco.BF16 else torch.float32
    states = [loco.State(gcfg, n) for n in sizes]
    comms = [torch.full((max(loco.loco_packed_bytes(gcfg, n), 16),), 0xA5, dtype=torch.uint8, device="cuda") for n in sizes]
    ostates = [orc.new_state(ocfg, n) for n in sizes]
    ocomms = [orc.new_comm(ocfg, n, fill=0xA5) for n in sizes]
    ostat = [[0, 0, 0] for _ in sizes]
    before = loco.loco_launch_count()
    for k in range(1, steps + 1):
        grads = [inputs.gaussian(n, sigma, seed=61, worker=i, step=k, dtype=dt, device="cuda") for i, n in enumerate(sizes)]
        if plant is not None:
            plant(grads, k)
        ms = loco.MultiSend(states, grads, comms)
        loco.loco_compensate_quantize_pack_multi(ms, k)
        torch.cuda.synchronize()
        for i, n in enumerate(sizes):
            if n == 0:
                continue
            f, a, b = orc.send_step(ocfg, inputs.as_numpy_bits(grads[i]), ostates[i], ocomms[i], k, full_status=True)
            ostat[i][0] |= f
            ostat[i][1] += a
            ostat[i][2] += b
    launches = loco.loco_launch_count() - before
    for i, n in enumerate(sizes):
        if n == 0:
            continue
        assert np.array_equal(comms[i].cpu().numpy()[:ocomms[i].size], ocomms[i]), "bucket %d (n = %d): communication buffer differs" % (i, n)
        sb = loco.loco_state_bytes(gcfg, n)
        gs, os_ = orc.state_views(ocfg, n, states[i].buffer.cpu().numpy()[:sb]), orc.state_views(ocfg, n, ostates[i])
        for a, b in zip(gs, os_):
            if a is not None:
                assert np.array_equal(a.view(np.uint8), b.view(np.uint8)), "bucket %d (n = %d): error state differs" % (i, n)
        f, a, b = loco.loco_status_counters(states[i])
        assert f == ostat[i][0], "bucket %d: flags" % i
        if collect_stats:
            assert (a, b) == (ostat[i][1], ostat[i][2]), "bucket %d: counters" % i
    return launches


def test_multi_send_table_kernel_mixed_sizes():
    sizes = [300_007, 1, 0, 255, 256, 257, 512, 1_000_000, 4096, 77, 2_500_123, 511, 65_537]
    kw = dict(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=2, state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16,
              out_dtype=loco.BF16, num_partitions=4)

    def plant(grads, k):
        if k == 2:
            grads[0][12345] = float("nan")
            grads[7][999_999] = float("inf")

    launches = _multi_case(kw, sizes, plant=plant)
    assert launches == 3                            # one launch per call, whatever the number of buckets


@pytest.mark.parametrize("kw", [
    dict(bits=4, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=64, state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, num_partitions=3),
    dict(bits=8, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=512, state_fmt=loco.STATE_INT8, grad_dtype=loco.F32, num_partitions=2),
    dict(bits=4, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=2048, state_fmt=loco.STATE_FP32, grad_dtype=loco.BF16, num_partitions=5),
    dict(bits=2, s=2.0 ** 9, s_e=6 * 2.0 ** 9, state_fmt=loco.STATE_FP32_Q8COMP, grad_dtype=loco.F32, num_partitions=1),
    dict(bits=1, s=2.0 ** 9, s_e=2.0 ** 12, state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, num_partitions=8),
    dict(bits=4, s=3000.0, s_e=12000.0, state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, num_partitions=8, rounding=1, seed=99),
    dict(bits=4, s=2.0 ** 19, s_e=2.0 ** 21, state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, num_partitions=8, clip=5e-4),
])
def test_multi_send_table_kernel_variants(kw):
    sizes = [100_003, 40_000, 1_300_000, 513, 9]
    base = dict(beta=0.5, reset_period=3, out_dtype=loco.BF16)
    base.update(kw)
    _multi_case(base, sizes)


def test_multi_send_more_buckets_than_one_table_holds():
    sizes = [1000 + 37 * i for i in range(1000)]
    kw = dict(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16,
              out_dtype=loco.BF16, num_partitions=2)
    launches = _multi_case(kw, sizes, steps=2, collect_stats=0)
    assert launches == 2 * 3                        # 1000 buckets, 448 per table


def test_multi_send_mixed_configurations_fall_into_runs():
    """Buckets of different configurations in one call: consecutive ones of the same configuration share a launch."""
    cfg_a = dict(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=0, grad_dtype=1, out_dtype=1, num_partitions=4)
    cfg_b = dict(cfg_a, bits=8)
    sizes = [50_000, 60_001, 70_002, 80_003]
    cfgs = [cfg_a, cfg_a, cfg_b, cfg_a]
    pairs = [both_configs(**c) for c in cfgs]
    states = [loco.State(g, n) for (g, _), n in zip(pairs, sizes)]
    comms = [torch.zeros(loco.loco_packed_bytes(g, n), dtype=torch.uint8, device="cuda") for (g, _), n in zip(pairs, sizes)]
    grads = [inputs.gaussian(n, 1e-3, seed=62, worker=i, dtype=torch.bfloat16, device="cuda") for i, n in enumerate(sizes)]
    before = loco.loco_launch_count()
    loco.loco_compensate_quantize_pack_multi(loco.MultiSend(states, grads, comms), 1)
    torch.cuda.synchronize()
    assert loco.loco_launch_count() - before == 3
    for i, ((_, o), n) in enumerate(zip(pairs, sizes)):
        ostate, ocomm = orc.new_state(o, n), orc.new_comm(o, n)
        orc.send_step(o, inputs.as_numpy_bits(grads[i]), ostate, ocomm, 1)
        assert np.array_equal(comms[i].cpu().numpy()[:ocomm.size], ocomm)
        assert np.array_equal(states[i].buffer.cpu().numpy()[:n], ostate[:n])


@pytest.mark.parametrize("kw", [
    dict(bits=4, s=2.0 ** 14, s_e=2.0 ** 16, state_fmt=loco.STATE_INT8, num_partitions=8),
    dict(bits=4, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=256, state_fmt=loco.STATE_INT8, num_partitions=8),
])
def test_multi_send_large_buckets(kw):
    """Seven buckets of about 25M elements in one launch (the size of the benchmark's buckets, ragged lengths among them).
    Bit-identical to the single-bucket calls, whose results the other tests hold against the oracle; one bucket's head
    and ragged tail also directly against the oracle."""
    sizes = [25_000_000, 24_999_999, 25_000_000, 13_415_616, 25_000_001, 25_000_000, 20_000_123]
    base = dict(beta=0.5, reset_period=0, grad_dtype=loco.BF16, out_dtype=loco.BF16)
    base.update(kw)
    gcfg, ocfg = both_configs(collect_stats=1, **base)
    grads = [inputs.gaussian(n, 1e-4, seed=71, worker=i, dtype=torch.bfloat16, device="cuda") for i, n in enumerate(sizes)]
    grads[3][777_777] = float("nan")
    multi = [loco.State(gcfg, n) for n in sizes]
    single = [loco.State(gcfg, n) for n in sizes]
    c_multi = [torch.zeros(loco.loco_packed_bytes(gcfg, n), dtype=torch.uint8, device="cuda") for n in sizes]
    c_single = [torch.zeros_like(c) for c in c_multi]
    ms = loco.MultiSend(multi, grads, c_multi)
    before = loco.loco_launch_count()
    for k in (1, 2):
        loco.loco_compensate_quantize_pack_multi(ms, k)
    torch.cuda.synchronize()
    assert loco.loco_launch_count() - before == 2
    for k in (1, 2):
        for st, g, c in zip(single, grads, c_single):
            loco.loco_compensate_quantize_pack(st, g, c, k)
    torch.cuda.synchronize()
    for i in range(len(sizes)):
        assert torch.equal(c_multi[i], c_single[i]), "bucket %d: codes differ" % i
        assert torch.equal(multi[i].buffer, single[i].buffer), "bucket %d: state differs" % i
        assert loco.loco_status_counters(multi[i]) == loco.loco_status_counters(single[i])
    assert loco.loco_status_counters(multi[3])[0] & loco.FLAG_NONFINITE
    # the head of the last bucket against the oracle (every element or block is computed independently of the rest)
    i, n, ln = len(sizes) - 1, sizes[-1], 1 << 18
    o1 = orc.OracleConfig(**{**base, "num_partitions": 1})
    ostate, ocomm = orc.new_state(o1, ln), orc.new_comm(o1, ln)
    for k in (1, 2):
        orc.send_step(o1, inputs.as_numpy_bits(grads[i][:ln]), ostate, ocomm, k)
    (oc, osc), = orc.comm_views(o1, ln, ocomm)
    got = c_multi[i].cpu().numpy()
    assert np.array_equal(got[:ln * 4 // 8], oc[:ln * 4 // 8])
    assert np.array_equal(multi[i].buffer[:ln].cpu().numpy(), ostate[:ln])
