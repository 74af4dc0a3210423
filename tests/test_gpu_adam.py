"""GPU parity of the receive pass fused with the paper's Adam-family step (loco_unpack_dequant_reduce_adam) against the
oracle: moments and weights bit for bit (every fp32 operation, the square root and the division are IEEE on both sides),
the optional averaged gradient bit for bit as well."""
import numpy as np
import pytest
import torch

from oracle import loco_oracle as orc
from paper_2407_04480_b200 import inputs, loco

pytestmark = pytest.mark.gpu

ADAM = dict(lr=1e-3, beta1=0.1, beta2=0.001, delta=1e-16)


def _packed_buffers(gcfg, n, workers, seed, steps=2):
    """Every worker's packed buffer after `steps` send passes on its own gradient (CUDA tensors)."""
    comms = []
    dt = torch.bfloat16 if gcfg.grad_dtype == loco.BF16 else torch.float32
    for w in range(workers):
        st = loco.State(gcfg, n)
        comm = torch.zeros(max(16, loco.loco_packed_bytes(gcfg, n)), dtype=torch.uint8, device="cuda")
        for k in range(steps):
            g = inputs.gaussian(n, 1e-3, seed=seed, worker=w, step=k, dtype=dt, device="cuda")
            loco.loco_compensate_quantize_pack(st, g, comm, k + 1)
        comms.append(comm)
    torch.cuda.synchronize()
    return comms


def _check(gcfg, n, workers, seed, first=0, count=None, with_grad=True, rounds=2):
    kw = {k: getattr(gcfg, k) for k in ("bits", "scale_mode", "block_size", "s", "s_e", "beta", "reset_period", "state_fmt",
                                        "grad_dtype", "out_dtype", "num_partitions")}
    ocfg = orc.OracleConfig(**kw)
    if count is None:
        count = gcfg.num_partitions - first
    comms = _packed_buffers(gcfg, n, workers, seed)
    ocomms = [c.cpu().numpy() for c in comms]
    stride = loco.loco_partition_bytes(gcfg, n)
    n_out = sum(loco.loco_partition_elems(gcfg, n, j) for j in range(first, first + count))
    rng = np.random.default_rng(seed)
    m0 = rng.normal(0, 1e-3, n_out).astype(np.float32)
    v0 = (rng.random(n_out) * 1e-6).astype(np.float32)
    t0 = rng.normal(0, 1.0, n_out).astype(np.float32)
    guard = 64
    def dev(a):
        whole = torch.full((a.size + 2 * guard,), 12345.0, dtype=torch.float32, device="cuda")
        whole[guard:guard + a.size] = torch.from_numpy(a).cuda()
        return whole, whole[guard:guard + a.size]
    (mw, m), (vw, v), (tw, t) = dev(m0), dev(v0), dev(t0)
    om, ov, ot = m0.copy(), v0.copy(), t0.copy()
    gdt = torch.bfloat16 if gcfg.out_dtype == loco.BF16 else torch.float32
    for r in range(rounds):
        gout = torch.zeros(n_out, dtype=gdt, device="cuda") if with_grad else None
        loco.loco_unpack_dequant_reduce_adam(gcfg, [c[first * stride:] for c in comms], n, m, v, t, grad_out=gout,
                                             first_partition=first, partition_count=count, **ADAM)
        torch.cuda.synchronize()
        og = orc.reduce_adam(ocfg, n, ocomms, om, ov, ot, first=first, count=count, want_grad=with_grad, **ADAM)
        for name, got, want in (("m", m, om), ("v", v, ov), ("theta", t, ot)):
            g_ = got.cpu().numpy()
            bad = int((g_.view(np.uint32) != want.view(np.uint32)).sum())
            assert bad == 0, "round %d: %d words of %s differ (max abs %g)" % (r, bad, name, float(np.abs(g_ - want).max()))
        if with_grad:
            gg = gout.view(torch.int16).cpu().numpy().view(np.uint16) if gdt == torch.bfloat16 else gout.cpu().numpy().view(np.uint32)
            assert np.array_equal(gg, og if gdt == torch.bfloat16 else og.view(np.uint32))
    for whole in (mw, vw, tw):
        w = whole.cpu().numpy()
        assert (w[:guard] == 12345.0).all() and (w[guard + n_out:] == 12345.0).all(), "write outside the moment / weight arrays"
    assert np.abs(ot - t0).max() > 0


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("workers", [1, 3, 8])
def test_adam_fused_integer_path(bits, workers):
    gcfg = loco.Config(bits=bits, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=loco.STATE_INT8,
                       grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=4)
    _check(gcfg, 300_001, workers, seed=50 + bits)


@pytest.mark.parametrize("s", [3000.0, 2.0 ** 11])
@pytest.mark.parametrize("od", [loco.F32, loco.BF16])
def test_adam_fused_generic_and_output_types(s, od):
    gcfg = loco.Config(bits=4, s=s, s_e=4 * s, beta=0.5, reset_period=0, state_fmt=loco.STATE_INT8,
                       grad_dtype=loco.F32, out_dtype=od, num_partitions=3)
    _check(gcfg, 100_003, 5, seed=61, with_grad=(od == loco.F32))
    _check(gcfg, 100_003, 5, seed=62, first=1, count=1)


@pytest.mark.parametrize("B", [32, 256])
def test_adam_fused_block_scales(B):
    gcfg = loco.Config(bits=4, scale_mode=loco.SCALE_BLOCK_ABSMAX, block_size=B, beta=0.5, reset_period=0,
                       state_fmt=loco.STATE_INT8, grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=2)
    _check(gcfg, 70_001, 4, seed=70 + B)


@pytest.mark.parametrize("n", [1, 15, 16, 17, 511, 513, 4097])
def test_adam_fused_ragged_sizes(n):
    gcfg = loco.Config(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=loco.STATE_INT8,
                       grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=2)
    _check(gcfg, n, 2, seed=80 + n)


def test_adam_fused_argument_errors():
    import ctypes as C
    gcfg = loco.Config(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, state_fmt=loco.STATE_NONE)
    n = 4096
    comm = torch.zeros(loco.loco_packed_bytes(gcfg, n), dtype=torch.uint8, device="cuda")
    m = torch.zeros(n + 4, dtype=torch.float32, device="cuda")
    v, t = torch.zeros_like(m), torch.zeros_like(m)
    L = loco.lib()
    ptrs = (C.c_void_p * 1)(comm.data_ptr())
    cfg_c = gcfg.c()
    ok = loco.loco_adam_t(1e-3, 0.1, 0.01, 1e-8)
    call = lambda ad, pm, pv, pt: L.loco_unpack_dequant_reduce_adam(C.byref(cfg_c), ptrs, 1, n, 0, 1, ad, pm, pv, pt, None, None)
    assert call(None, m.data_ptr(), v.data_ptr(), t.data_ptr()) == loco.ERR_ARG
    assert call(C.byref(ok), None, v.data_ptr(), t.data_ptr()) == loco.ERR_ARG
    assert call(C.byref(ok), m.data_ptr() + 4, v.data_ptr(), t.data_ptr()) == loco.ERR_ALIGN
    assert call(C.byref(loco.loco_adam_t(1e-3, 1.5, 0.01, 1e-8)), m.data_ptr(), v.data_ptr(), t.data_ptr()) == loco.ERR_ARG
    assert call(C.byref(loco.loco_adam_t(1e-3, 0.1, 0.01, -1.0)), m.data_ptr(), v.data_ptr(), t.data_ptr()) == loco.ERR_ARG
    assert call(C.byref(ok), m.data_ptr(), v.data_ptr(), t.data_ptr()) == loco.OK
    torch.cuda.synchronize()
