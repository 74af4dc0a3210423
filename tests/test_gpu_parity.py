"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same bytes."""
import numpy as np
import pytest
import torch

from oracle import loco_oracle as orc
from paper_2407_04480_b200 import inputs, loco
from tests.parity import Worker, assert_reduced_equal, both_configs, reduce_both

pytestmark = pytest.mark.gpu


def grad_bits(t):
    return inputs.as_numpy_bits(t)


def run_steps(gcfg, ocfg, n, steps, sigma, seed, k0=0, worker=0, device="cuda"):
    w = Worker(gcfg, ocfg, n)
    dt = torch.bfloat16 if gcfg.grad_dtype == loco.BF16 else torch.float32
    for i in range(steps):
        g = inputs.gaussian(n, sigma, seed=seed, worker=worker, step=i, dtype=dt, device=device)
        w.step(grad_bits(g), k0 + i)
        w.compare("step %d" % (k0 + i))
    return w


# ---------------------------------------------------------------- config 1: 2^20 fp32, 4 steps

@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32, loco.STATE_FP32_Q8COMP, loco.STATE_NONE])
@pytest.mark.parametrize("beta", [0.5, 0.25, 1.0, 0.1, 0.0])
def test_config1_fixed_scale(fmt, beta):
    gcfg, ocfg = both_configs(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=beta, reset_period=512, state_fmt=fmt,
                              grad_dtype=loco.F32, out_dtype=loco.F32)
    w = run_steps(gcfg, ocfg, 1 << 20, 4, 1e-3, seed=0)
    got, want = reduce_both(gcfg, ocfg, 1 << 20, [w])
    assert_reduced_equal(got, want, False)


@pytest.mark.parametrize("T_c", [0, 2, 3])
@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32])
def test_config1_reset_periods(T_c, fmt):
    gcfg, ocfg = both_configs(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=T_c, state_fmt=fmt,
                              grad_dtype=loco.F32, out_dtype=loco.F32)
    run_steps(gcfg, ocfg, 1 << 20, 5, 1e-3, seed=0)


@pytest.mark.parametrize("s,s_e", [(2.0 ** 19, 6 * 2.0 ** 19), (2.0 ** 17, 4 * 2.0 ** 17), (3000.0, 12000.0),
                                   (2.0 ** 11, 6 * 2.0 ** 11)])
@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32_Q8COMP])
def test_config1_paper_scales(s, s_e, fmt):
    """The paper's own s = 2^19 / 2^17 with s_e = 4s or 6s (everything saturates at sigma = 1e-3),
    and scales whose reciprocal is not exact (division path)."""
    gcfg, ocfg = both_configs(bits=4, s=s, s_e=s_e, beta=0.5, reset_period=512, state_fmt=fmt,
                              grad_dtype=loco.F32, out_dtype=loco.F32)
    w = run_steps(gcfg, ocfg, 1 << 20, 4, 1e-3, seed=0)
    got, want = reduce_both(gcfg, ocfg, 1 << 20, [w])
    assert_reduced_equal(got, want, False)


@pytest.mark.parametrize("B", [32, 64, 128, 256])
@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32, loco.STATE_NONE])
def test_config1_block_absmax(B, fmt):
    gcfg, ocfg = both_configs(bits=4, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=B, beta=0.5, reset_period=3,
                              state_fmt=fmt, grad_dtype=loco.F32, out_dtype=loco.F32)
    w = run_steps(gcfg, ocfg, 1 << 20, 4, 1e-3, seed=0)
    got, want = reduce_both(gcfg, ocfg, 1 << 20, [w])
    assert_reduced_equal(got, want, False)


# ---------------------------------------------------------------- ragged sizes, partitions, widths

SIZES = [1, 7, 8, 9, 31, 255, 256, 257, 1000, 4097, 65537, 300001]


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("P", [1, 3, 8])
@pytest.mark.parametrize("mode", [loco.SCALE_FIXED, loco.SCALE_BLOCK_ABSMAX])
def test_ragged_sizes(bits, P, mode):
    for n in SIZES:
        for gd in (loco.F32, loco.BF16):
            gcfg, ocfg = both_configs(bits=bits, scale_mode=mode, block_size=64, s=2.0 ** 10, s_e=2.0 ** 12, beta=0.5,
                                      reset_period=0, state_fmt=loco.STATE_INT8, grad_dtype=gd, out_dtype=gd,
                                      num_partitions=P)
            ws = [run_steps(gcfg, ocfg, n, 3, 2e-3, seed=11, worker=w) for w in range(3)]
            got, want = reduce_both(gcfg, ocfg, n, ws)
            assert_reduced_equal(got, want, gd == loco.BF16, "n=%d" % n)
            for j in range(P):
                got, want = reduce_both(gcfg, ocfg, n, ws, first=j, count=1)
                assert got.size == loco.loco_partition_elems(gcfg, n, j)
                assert_reduced_equal(got, want, gd == loco.BF16, "n=%d part %d" % (n, j))


def test_empty_bucket():
    gcfg, _ = both_configs(bits=4, s=2.0 ** 10, s_e=2.0 ** 12)
    assert loco.loco_state_bytes(gcfg, 0) == 0 and loco.loco_packed_bytes(gcfg, 0) == 0
    st = loco.State(gcfg, 0)
    g = torch.empty(0, dtype=torch.bfloat16, device="cuda")
    comm = torch.empty(16, dtype=torch.uint8, device="cuda")
    loco.loco_compensate_quantize_pack(st, g, comm, 0)
    out = torch.empty(0, dtype=torch.bfloat16, device="cuda")
    loco.loco_unpack_dequant_reduce(gcfg, [comm], 0, out)
    torch.cuda.synchronize()


# ---------------------------------------------------------------- adversarial values

def special_values(n, s):
    """Exact ties (m + 1/2)/s, signed zeros, denormals, the ends of the range, huge and non-finite values."""
    rng = np.random.default_rng(5)
    x = rng.normal(0, 4.0 / s, n).astype(np.float32)
    ties = ((np.arange(-12, 12) + 0.5) / s).astype(np.float32)
    specials = np.concatenate([ties, [0.0, -0.0, 1e-45, -1e-45, 1e-39, 7.0 / s, -8.0 / s, 7.5 / s, -8.5 / s,
                                      3e38, -3e38, np.inf, -np.inf, np.nan]]).astype(np.float32)
    reps = n // (4 * specials.size)
    pos = rng.choice(n, specials.size * reps, replace=False)
    x[pos] = np.tile(specials, reps)
    return x


@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32])
@pytest.mark.parametrize("mode,s", [(loco.SCALE_FIXED, 2.0 ** 9), (loco.SCALE_FIXED, 1000.0),
                                    (loco.SCALE_BLOCK_ABSMAX, 1.0)])
def test_adversarial_values(fmt, mode, s):
    n = 50000
    for gd in (loco.F32, loco.BF16):
        gcfg, ocfg = both_configs(bits=4, scale_mode=mode, block_size=128, s=s, s_e=4 * s, beta=0.5, reset_period=0,
                                  state_fmt=fmt, grad_dtype=gd, out_dtype=loco.F32, num_partitions=2)
        w = Worker(gcfg, ocfg, n)
        for k in range(3):
            x = special_values(n, s if mode == loco.SCALE_FIXED else 512.0)
            if gd == loco.BF16:
                x = grad_bits(torch.from_numpy(x).to(torch.bfloat16))
            w.step(x, k + 1)
            w.compare("step %d" % k)
        assert w.oflags & orc.FLAG_NONFINITE
        got, want = reduce_both(gcfg, ocfg, n, [w])
        assert_reduced_equal(got, want, False)


def test_all_zero_blocks():
    n = 8192
    gcfg, ocfg = both_configs(bits=4, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=256, beta=0.5, reset_period=0,
                              state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, out_dtype=loco.BF16)
    w = Worker(gcfg, ocfg, n)
    for k in range(3):
        g = inputs.gaussian(n, 1e-4, seed=3, step=k, dtype=torch.bfloat16, device="cuda")
        g[1024:3072] = 0
        w.step(grad_bits(g), k + 1)
        w.compare()
    got, want = reduce_both(gcfg, ocfg, n, [w, w])
    assert_reduced_equal(got, want, True)


# ---------------------------------------------------------------- receive side

@pytest.mark.parametrize("N", [1, 2, 3, 5, 8, 16])
@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("mode,s", [(loco.SCALE_FIXED, 2.0 ** 12), (loco.SCALE_FIXED, 3000.0),
                                    (loco.SCALE_BLOCK_ABSMAX, 1.0)])
def test_reduce_workers(N, bits, mode, s):
    n = 200_003
    for od in (loco.F32, loco.BF16):
        gcfg, ocfg = both_configs(bits=bits, scale_mode=mode, block_size=256, s=s, s_e=4 * s, beta=0.5,
                                  reset_period=0, state_fmt=loco.STATE_NONE, grad_dtype=loco.BF16, out_dtype=od,
                                  num_partitions=4)
        ws = [run_steps(gcfg, ocfg, n, 1, 5e-4, seed=21, worker=w) for w in range(N)]
        got, want = reduce_both(gcfg, ocfg, n, ws)
        assert_reduced_equal(got, want, od == loco.BF16)
        got, want = reduce_both(gcfg, ocfg, n, ws, first=1, count=2)
        assert_reduced_equal(got, want, od == loco.BF16)


@pytest.mark.parametrize("N", [4, 6, 7, 9, 17, 33, 64])
@pytest.mark.parametrize("mode,s,B", [(loco.SCALE_FIXED, 2.0 ** 12, 256), (loco.SCALE_FIXED, 3000.0, 256),
                                      (loco.SCALE_BLOCK_ABSMAX, 1.0, 32), (loco.SCALE_BLOCK_ABSMAX, 1.0, 128)])
def test_reduce_group_shapes(N, mode, s, B):
    """Worker counts around the receive kernel's groups of four (one full group, a short last group, many groups, the
    maximum; 17+ workers leave the integer path) and bucket sizes from less than one wide row to a few rows per warp."""
    for n, bits in ((300, 4), (513, 8), (40_000, 2), (150_001, 4)):
        gcfg, ocfg = both_configs(bits=bits, scale_mode=mode, block_size=B, s=s, s_e=4 * s, beta=0.5,
                                  reset_period=0, state_fmt=loco.STATE_NONE, grad_dtype=loco.BF16, out_dtype=loco.BF16,
                                  num_partitions=2)
        base = [run_steps(gcfg, ocfg, n, 1, 5e-4, seed=33, worker=w) for w in range(min(N, 5))]
        ws = [base[w % len(base)] for w in range(N)]
        got, want = reduce_both(gcfg, ocfg, n, ws)
        assert_reduced_equal(got, want, True, "n=%d bits=%d N=%d" % (n, bits, N))


# ---------------------------------------------------------------- Llama-2-7B-shaped buckets, 8 workers

def test_llama_buckets_sampled():
    """25M-element bf16 buckets of the Llama-2-7B layout with per-layer scales: the first bucket, one
    that straddles tensors, and the partial last bucket; 8 workers, 3 iterations around a reset, then
    the 8-partition reduce."""
    layout = inputs.llama2_7b()
    scales = inputs.group_scales(1, layout.n_groups)
    buckets = inputs.bucket_ranges(layout.numel, 25_000_000)
    assert len(buckets) == 270 and buckets[-1][1] - buckets[-1][0] == 13_415_616
    for b in (0, 5, 269):
        lo, hi = buckets[b]
        n = hi - lo
        gcfg, ocfg = both_configs(bits=4, s=2.0 ** 14, s_e=2.0 ** 16, beta=0.5, reset_period=32,
                                  state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, out_dtype=loco.BF16,
                                  num_partitions=8)
        ws = [Worker(gcfg, ocfg, n) for _ in range(8 if b == 0 else 2)]
        for k in (31, 32, 33):
            for wi, w in enumerate(ws):
                g = inputs.layout_slice(layout, lo, hi, scales, 1e-4, seed=1, worker=wi, step=k, device="cuda")
                w.step(grad_bits(g), k)
            ws[0].compare("bucket %d step %d" % (b, k))
            ws[-1].compare("bucket %d step %d" % (b, k))
        got, want = reduce_both(gcfg, ocfg, n, ws)
        assert_reduced_equal(got, want, True, "bucket %d" % b)


# ---------------------------------------------------------------- argument checking

def test_argument_errors():
    gcfg, _ = both_configs(bits=4, s=2.0 ** 10, s_e=2.0 ** 12)
    n = 4096
    import ctypes as C
    buf = torch.zeros(n + 64, dtype=torch.uint8, device="cuda")
    h = C.c_void_p()
    assert loco.loco_state_init_raw(C.byref(h), gcfg, n, buf.data_ptr() + 1, n, None) == loco.ERR_ALIGN
    assert loco.loco_state_init_raw(C.byref(h), gcfg, n, buf.data_ptr(), n - 1, None) == loco.ERR_SIZE
    assert loco.loco_state_init_raw(C.byref(h), gcfg, n, None, n, None) == loco.ERR_ARG
    bad = loco.Config(bits=3)
    assert loco.loco_state_init_raw(C.byref(h), bad, n, buf.data_ptr(), n, None) == loco.ERR_ARG
    st = loco.State(gcfg, n)
    g = torch.zeros(n + 8, dtype=torch.bfloat16, device="cuda")
    comm = torch.zeros(loco.loco_packed_bytes(gcfg, n) + 16, dtype=torch.uint8, device="cuda")
    L = loco.lib()
    assert L.loco_compensate_quantize_pack(st.handle, g.data_ptr() + 2, comm.data_ptr(), 0, None) == loco.ERR_ALIGN
    assert L.loco_compensate_quantize_pack(st.handle, g.data_ptr(), comm.data_ptr() + 4, 0, None) == loco.ERR_ALIGN
    assert L.loco_compensate_quantize_pack(st.handle, g.data_ptr(), comm.data_ptr(), -1, None) == loco.ERR_ARG
    assert L.loco_compensate_quantize_pack(st.handle, None, comm.data_ptr(), 0, None) == loco.ERR_ARG
    out = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    ptrs = (C.c_void_p * 1)(comm.data_ptr())
    cfg_c = gcfg.c()
    assert L.loco_unpack_dequant_reduce(C.byref(cfg_c), ptrs, 0, n, 0, 1, out.data_ptr(), None) == loco.ERR_ARG
    assert L.loco_unpack_dequant_reduce(C.byref(cfg_c), ptrs, 1, n, 0, 2, out.data_ptr(), None) == loco.ERR_ARG
    assert L.loco_unpack_dequant_reduce(C.byref(cfg_c), ptrs, 1, n, 0, 1, out.data_ptr() + 2, None) == loco.ERR_ALIGN
    assert L.loco_unpack_dequant_reduce(C.byref(cfg_c), ptrs, 65, n, 0, 1, out.data_ptr(), None) == loco.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    st.close()


def test_state_reset_and_checkpoint_resume():
    """Explicit reset zeroes the state; saving the state tensor and k and restoring them resumes
    bit-identically (2K steps in one go versus K + restore + K)."""
    n = 100_000
    gcfg, ocfg = both_configs(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=loco.STATE_INT8,
                              grad_dtype=loco.BF16, out_dtype=loco.BF16)
    grads = [inputs.gaussian(n, 1e-3, seed=9, step=k, dtype=torch.bfloat16, device="cuda") for k in range(6)]
    comm_a = torch.zeros(loco.loco_packed_bytes(gcfg, n), dtype=torch.uint8, device="cuda")
    comm_b = torch.zeros_like(comm_a)
    a = loco.State(gcfg, n)
    for k in range(6):
        loco.loco_compensate_quantize_pack(a, grads[k], comm_a, k + 1)
    b = loco.State(gcfg, n)
    for k in range(3):
        loco.loco_compensate_quantize_pack(b, grads[k], comm_b, k + 1)
    saved = b.buffer.clone()
    c = loco.State(gcfg, n)
    c.buffer.copy_(saved)
    for k in range(3, 6):
        loco.loco_compensate_quantize_pack(c, grads[k], comm_b, k + 1)
    torch.cuda.synchronize()
    assert torch.equal(a.buffer, c.buffer) and torch.equal(comm_a, comm_b)
    assert a.buffer.any()
    loco.loco_state_reset(a)
    torch.cuda.synchronize()
    assert not a.buffer.any()


# ---------------------------------------------------------------- host-buffer entry points

@pytest.mark.parametrize("mode", [loco.SCALE_FIXED, loco.SCALE_BLOCK_ABSMAX])
def test_host_buffer_variants(mode):
    """The *_host entry points (gradient, packed parts and result in pinned host memory, staged through a
    caller-provided device workspace) give the oracle's bytes."""
    n, P, N = 300_001, 4, 3
    gcfg, ocfg = both_configs(bits=4, scale_mode=mode, block_size=128, s=2.0 ** 12, s_e=2.0 ** 14, beta=0.5,
                              reset_period=0, state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, out_dtype=loco.BF16,
                              num_partitions=P)
    stride = loco.loco_partition_bytes(gcfg, n)
    w_send = torch.empty(loco.loco_send_host_workspace_bytes(gcfg, n), dtype=torch.uint8, device="cuda")
    h_comms, o_comms = [], []
    for w in range(N):
        st = loco.State(gcfg, n)
        ostate, ocomm = orc.new_state(ocfg, n), orc.new_comm(ocfg, n)
        h_comm = torch.zeros(loco.loco_packed_bytes(gcfg, n), dtype=torch.uint8).pin_memory()
        for k in range(2):
            g = inputs.gaussian(n, 1e-3, seed=31, worker=w, step=k, dtype=torch.bfloat16)
            h_grad = g.pin_memory()
            loco.loco_compensate_quantize_pack_host(st, h_grad, h_comm, w_send, k + 1)
            torch.cuda.synchronize()
            orc.send_step(ocfg, grad_bits(g), ostate, ocomm, k + 1)
        for (gc, gs), (oc, os_) in zip(orc.comm_views(ocfg, n, h_comm.numpy()), orc.comm_views(ocfg, n, ocomm)):
            assert np.array_equal(gc, oc)
            if gs is not None:
                assert np.array_equal(gs.view(np.uint32), os_.view(np.uint32))
        assert np.array_equal(orc.state_views(ocfg, n, st.buffer.cpu().numpy())[0], orc.state_views(ocfg, n, ostate)[0])
        h_comms.append(h_comm)
        o_comms.append(ocomm)
    first, count = 1, 2
    w_red = torch.empty(loco.loco_reduce_host_workspace_bytes(gcfg, n, N, count), dtype=torch.uint8, device="cuda")
    n_out = sum(loco.loco_partition_elems(gcfg, n, j) for j in range(first, first + count))
    h_out = torch.zeros(n_out, dtype=torch.bfloat16).pin_memory()
    loco.loco_unpack_dequant_reduce_host(gcfg, [c[first * stride:] for c in h_comms], n, h_out, w_red,
                                         first_partition=first, partition_count=count)
    torch.cuda.synchronize()
    want = orc.reduce(ocfg, n, o_comms, first=first, count=count)
    assert_reduced_equal(h_out.view(torch.int16).numpy().view(np.uint16), want, True)
    # a workspace one byte short is refused before anything is enqueued
    with pytest.raises(loco.LocoError) as ei:
        loco.loco_unpack_dequant_reduce_host(gcfg, [c[first * stride:] for c in h_comms], n, h_out, w_red[:-1],
                                             first_partition=first, partition_count=count)
    assert ei.value.code == loco.ERR_SIZE


def test_block_scale_divisions_are_ieee_for_every_amax():
    """The block-scaled send path divides with short multiply-add sequences; the library checks them against the IEEE
    division for every positive finite fp32 amax and qmax in {1, 7, 127}."""
    assert loco.loco_selfcheck_block_division() == (0, 0)


# ---------------------------------------------------------------- element-wise clipping of the local gradient

@pytest.mark.parametrize("mode", [loco.SCALE_FIXED, loco.SCALE_BLOCK_ABSMAX])
@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32, loco.STATE_NONE])
def test_gradient_clipping(mode, fmt):
    """clip > 0: every gradient element is clamped to [-clip, clip] before Algorithm 1 (heavy-tailed values, so that many
    are clamped; a few +-Inf, which become +-clip, and NaN, which stay NaN)."""
    n = 200_003
    for gd in (loco.BF16, loco.F32):
        gcfg, ocfg = both_configs(bits=4, scale_mode=mode, block_size=128, s=2.0 ** 12, s_e=2.0 ** 14, beta=0.5, reset_period=0,
                                  state_fmt=fmt, grad_dtype=gd, out_dtype=loco.F32, num_partitions=3, clip=3e-4)
        w = Worker(gcfg, ocfg, n)
        dt = torch.bfloat16 if gd == loco.BF16 else torch.float32
        for k in range(3):
            g = inputs.student_t(n, 3.0, 1e-4, seed=15, step=k, dtype=torch.float32, device="cuda")
            g[1000 + k] = float("inf")
            g[70_000 + k] = float("-inf")
            if k == 1:
                g[150_000] = float("nan")
            assert int((g.abs() > 3e-4).sum()) > n // 20
            w.step(grad_bits(g.to(dt)), k + 1)
            w.compare("step %d" % k)
        assert w.oflags & orc.FLAG_NONFINITE
        got, want = reduce_both(gcfg, ocfg, n, [w])
        assert_reduced_equal(got, want, False)


def test_zero_plus_plus_style_weight_payload():
    """The 8-bit block-quantised weight payload of the LoCo-Zero++ variant is the send pass without error state (8-bit codes,
    one scale per block) and the receive pass with a single worker: round trip within half a quantisation step of the block."""
    n, B = 1_000_003, 256
    gcfg, ocfg = both_configs(bits=8, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=B, state_fmt=loco.STATE_NONE,
                              grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=8)
    wgt = inputs.gaussian(n, 0.02, seed=16, dtype=torch.bfloat16, device="cuda")
    w = Worker(gcfg, ocfg, n)
    w.step(grad_bits(wgt), 0)
    w.compare("weights")
    got, want = reduce_both(gcfg, ocfg, n, [w])
    assert_reduced_equal(got, want, True)
    back = torch.from_numpy(got.view(np.int16)).view(torch.bfloat16).float()
    x = wgt.float().cpu()
    pad = (-n) % B
    amax = torch.nn.functional.pad(x.abs(), (0, pad)).view(-1, B).max(dim=1).values
    step = (amax / 127.0).repeat_interleave(B)[:n]
    # half a step from the rounding to a code plus half a bf16 ulp of the result
    assert bool(((back - x).abs() <= 0.5 * step * 1.001 + x.abs() * 2.0 ** -8).all())


# ---------------------------------------------------------------- a long horizon: 100 iterations, several resets

@pytest.mark.parametrize("mode,fmt,rounding", [(loco.SCALE_FIXED, loco.STATE_INT8, 0), (loco.SCALE_FIXED, loco.STATE_FP32, 0),
                                               (loco.SCALE_BLOCK_ABSMAX, loco.STATE_INT8, 0), (loco.SCALE_FIXED, loco.STATE_INT8, 1)])
def test_hundred_iterations(mode, fmt, rounding):
    """100 consecutive iterations on one bucket (the iteration count the Llama-2-7B configuration names), error state carried
    from step to step on both sides, reset every 32 iterations: codes, scales and state compared around the resets and at the
    end -- a single differing state code anywhere on the way would show in what follows."""
    n = 400_003
    gcfg, ocfg = both_configs(bits=4, scale_mode=mode, block_size=128, s=2.0 ** 13, s_e=2.0 ** 15, beta=0.5, reset_period=32,
                              state_fmt=fmt, grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=8, rounding=rounding,
                              seed=7)
    w = Worker(gcfg, ocfg, n)
    check_at = {0, 1, 2, 31, 32, 33, 63, 64, 65, 98, 99}
    for k in range(100):
        g = inputs.gaussian(n, 1e-4, seed=41, worker=0, step=k, dtype=torch.bfloat16, device="cuda")
        w.step(grad_bits(g), k)
        if k in check_at:
            w.compare("iteration %d" % k)
    got, want = reduce_both(gcfg, ocfg, n, [w, w, w])
    assert_reduced_equal(got, want, True)


# ---------------------------------------------------------------- stochastic rounding on the shared Philox stream

@pytest.mark.parametrize("mode", [loco.SCALE_FIXED, loco.SCALE_BLOCK_ABSMAX])
@pytest.mark.parametrize("fmt", [loco.STATE_INT8, loco.STATE_FP32, loco.STATE_NONE])
@pytest.mark.parametrize("bits", [2, 4, 8])
def test_stochastic_rounding(mode, fmt, bits):
    """rounding = stochastic: the library and the oracle draw the same Philox4x32-10 numbers for (element, iteration, seed)
    and must produce the same codes, state and statistics bit for bit; ragged size, several parts, both gradient types."""
    n = 150_001
    for gd in (loco.BF16, loco.F32):
        gcfg, ocfg = both_configs(bits=bits, scale_mode=mode, block_size=64, s=2.0 ** 9, s_e=2.0 ** 11, beta=0.5, reset_period=0,
                                  state_fmt=fmt, grad_dtype=gd, out_dtype=loco.F32, num_partitions=3, rounding=1,
                                  seed=0x1234567890ABCDEF)
        w = run_steps(gcfg, ocfg, n, 3, 2e-3, seed=17, k0=5)
        got, want = reduce_both(gcfg, ocfg, n, [w])
        assert_reduced_equal(got, want, False)


@pytest.mark.parametrize("s,s_e", [(2.0 ** 9, 6 * 2.0 ** 9), (3000.0, 12000.0)])
def test_stochastic_rounding_other_decompressor_forms(s, s_e):
    """Scales for which the state decompressor is the Newton-Raphson form or the division itself: stochastic rounding then
    runs in the kernel variant that chooses the forms per call."""
    n = 90_007
    for fmt in (loco.STATE_INT8, loco.STATE_FP32_Q8COMP):
        gcfg, ocfg = both_configs(bits=4, s=s, s_e=s_e, beta=0.5, reset_period=0, state_fmt=fmt, grad_dtype=loco.BF16,
                                  out_dtype=loco.F32, num_partitions=2, rounding=1, seed=99)
        run_steps(gcfg, ocfg, n, 3, 2e-3, seed=19, k0=2)


def test_stochastic_rounding_differs_from_nearest_and_between_seeds():
    n = 1 << 16
    g = inputs.gaussian(n, 2e-3, seed=18, dtype=torch.bfloat16, device="cuda")
    codes = []
    for kw in (dict(rounding=0), dict(rounding=1, seed=1), dict(rounding=1, seed=2)):
        cfg = loco.Config(bits=4, s=2.0 ** 9, s_e=2.0 ** 11, state_fmt=loco.STATE_NONE, grad_dtype=loco.BF16, **kw)
        comm = torch.zeros(loco.loco_packed_bytes(cfg, n), dtype=torch.uint8, device="cuda")
        loco.loco_compensate_quantize_pack(loco.State(cfg, n), g, comm, 3)
        torch.cuda.synchronize()
        codes.append(comm.cpu().numpy())
    assert (codes[0] != codes[1]).mean() > 0.2 and (codes[1] != codes[2]).mean() > 0.2
