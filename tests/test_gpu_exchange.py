"""The all-to-all of Sec. 3.3 folded into the send pass's stores, on one GPU.

N workers live on the one device.  Worker r's send pass writes part j of its communication buffer straight into
slot r of worker j's receive area (loco_compensate_quantize_pack_scatter); worker j then reduces its N slots with
the ordinary receive pass.  Stream order stands in for the barrier between the two passes; with several GPUs the
same pointers would name peers' memory.  Every slot must hold, bit for bit, the part the oracle's contiguous
buffer holds, the state must match the oracle's, and the concatenated results must equal the oracle's reduction
over all workers' whole buffers.
"""
import numpy as np
import pytest
import torch

from oracle import loco_oracle as orc
from paper_2407_04480_b200 import inputs, loco
from tests import parity

pytestmark = pytest.mark.gpu

CASES = [
    # (n, workers, config)
    (300_007, 4, dict(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=0, grad_dtype=1, out_dtype=1)),
    (1_000_003, 8, dict(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=4, state_fmt=0, grad_dtype=1, out_dtype=1)),
    (200_001, 3, dict(bits=8, s=2.0 ** 12, s_e=6 * 2.0 ** 12, beta=0.25, reset_period=0, state_fmt=1, grad_dtype=0, out_dtype=0)),
    (262_144, 2, dict(bits=2, s=2.0 ** 9, s_e=2.0 ** 11, beta=0.5, reset_period=0, state_fmt=2, grad_dtype=1, out_dtype=0)),
    (500_000, 4, dict(bits=4, scale_mode=1, block_size=64, s=1.0, s_e=1.0, beta=0.5, reset_period=0, state_fmt=0,
                      grad_dtype=1, out_dtype=1)),
    (777, 8, dict(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=0, grad_dtype=1, out_dtype=1)),
]


@pytest.mark.parametrize("n,workers,kw", CASES)
def test_scatter_send_then_local_reduce(n, workers, kw):
    gcfg, ocfg = parity.both_configs(num_partitions=workers, collect_stats=0, **kw)
    stride = loco.loco_partition_bytes(gcfg, n)
    lp = orc.partition_capacity(ocfg, n)
    used = lp * ocfg.bits // 8 + (4 * (lp // ocfg.block_size) if ocfg.scale_mode == orc.SCALE_BLOCK_ABSMAX else 0)
    bf16 = gcfg.grad_dtype == loco.BF16
    # receive area of worker j: N slots of one part each, canaries around the whole area
    areas = [parity.guarded(workers * stride) for _ in range(workers)]
    states = [loco.State(gcfg, n) for _ in range(workers)]
    ostates = [orc.new_state(ocfg, n) for _ in range(workers)]
    ocomms = [orc.new_comm(ocfg, n, fill=parity.CANARY) for _ in range(workers)]
    for k in range(3):
        for r in range(workers):
            g = inputs.gaussian(n, 1e-3, seed=31, worker=r, step=k, dtype=torch.bfloat16 if bf16 else torch.float32)
            gnp = inputs.as_numpy_bits(g)
            dst = [areas[j][1][r * stride:(r + 1) * stride] for j in range(workers)]
            loco.loco_compensate_quantize_pack_scatter(states[r], parity.to_device(gnp, bf16), dst, k)
            orc.send_step(ocfg, gnp, ostates[r], ocomms[r], k)
        torch.cuda.synchronize()
        # slot r of worker j == part j of worker r's contiguous buffer (pad bytes stay untouched)
        for j in range(workers):
            area = areas[j][1].cpu().numpy()
            for r in range(workers):
                got = area[r * stride:r * stride + used]
                want = ocomms[r][j * stride:j * stride + used]
                assert np.array_equal(got, want), "step %d: slot %d of worker %d differs" % (k, r, j)
                assert (area[r * stride + used:(r + 1) * stride] == parity.CANARY).all(), "pad bytes written"
            parity.check_guards(areas[j][0], workers * stride)
        for r in range(workers):
            gv, gsc = orc.state_views(ocfg, n, states[r].buffer.cpu().numpy())
            ov, osc = orc.state_views(ocfg, n, ostates[r])
            if gv is not None:
                assert np.array_equal(gv.view(np.uint8), ov.view(np.uint8)), "step %d: state of worker %d differs" % (k, r)
            if gsc is not None:
                assert np.array_equal(gsc.view(np.uint32), osc.view(np.uint32))
    # every worker reduces what it received, from its own area only
    esize = 2 if gcfg.out_dtype == loco.BF16 else 4
    pieces = []
    for j in range(workers):
        n_out = loco.loco_partition_elems(gcfg, n, j)
        whole, view = parity.guarded(max(n_out * esize, 16))
        out = view[:n_out * esize].view(torch.bfloat16 if esize == 2 else torch.float32)
        slots = [areas[j][1][r * stride:(r + 1) * stride] for r in range(workers)]
        loco.loco_unpack_dequant_reduce(gcfg, slots, n, out, first_partition=j, partition_count=1)
        torch.cuda.synchronize()
        parity.check_guards(whole, max(n_out * esize, 16))
        pieces.append(out.view(torch.int16).cpu().numpy().view(np.uint16) if esize == 2 else out.cpu().numpy())
    got = np.concatenate(pieces)
    want = orc.reduce(ocfg, n, ocomms)
    assert got.size == n
    parity.assert_reduced_equal(got, want, esize == 2, "scatter exchange")


def test_scatter_matches_contiguous_send_bytes():
    """The scattering pass and the contiguous pass write the same bytes from the same state."""
    n, workers = 3_000_000, 8
    kw = dict(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=0, grad_dtype=1, out_dtype=1)
    gcfg = loco.Config(num_partitions=workers, **kw)
    stride = loco.loco_partition_bytes(gcfg, n)
    a, b = loco.State(gcfg, n), loco.State(gcfg, n)
    comm = torch.zeros(workers * stride, dtype=torch.uint8, device="cuda")
    # destinations in shuffled order inside one arena, so that no part lands where the contiguous pass puts it
    arena = torch.zeros(workers * stride, dtype=torch.uint8, device="cuda")
    order = [5, 2, 7, 0, 3, 6, 1, 4]
    dst = [arena[order[j] * stride:(order[j] + 1) * stride] for j in range(workers)]
    for k in range(2):
        g = inputs.gaussian(n, 1e-3, seed=5, worker=0, step=k, dtype=torch.bfloat16, device="cuda")
        loco.loco_compensate_quantize_pack(a, g, comm, k)
        loco.loco_compensate_quantize_pack_scatter(b, g, dst, k)
    torch.cuda.synchronize()
    for j in range(workers):
        assert torch.equal(comm[j * stride:(j + 1) * stride], dst[j])
    assert torch.equal(a.buffer, b.buffer)


def test_scatter_argument_errors():
    gcfg = loco.Config(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=0, grad_dtype=1, out_dtype=1,
                       num_partitions=2)
    n = 4096
    st = loco.State(gcfg, n)
    g = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    stride = loco.loco_partition_bytes(gcfg, n)
    buf = torch.zeros(2 * stride + 64, dtype=torch.uint8, device="cuda")
    with pytest.raises(ValueError):
        loco.loco_compensate_quantize_pack_scatter(st, g, [buf[:stride]], 0)
    with pytest.raises(loco.LocoError) as e:
        loco.loco_compensate_quantize_pack_scatter(st, g, [buf.data_ptr(), buf.data_ptr() + stride + 4], 0)
    assert e.value.code == loco.ERR_ALIGN
    with pytest.raises(loco.LocoError) as e:
        loco.loco_compensate_quantize_pack_scatter(st, g, [buf.data_ptr(), 0], 0)
    assert e.value.code == loco.ERR_ARG
    big = loco.Config(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=0, grad_dtype=1, out_dtype=1,
                      num_partitions=65)
    n2 = 65 * 256
    st2 = loco.State(big, n2)
    g2 = torch.zeros(n2, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(loco.LocoError) as e:
        loco.loco_compensate_quantize_pack_scatter(st2, g2, [buf.data_ptr()] * 65, 0)
    assert e.value.code == loco.ERR_UNSUPPORTED
    torch.cuda.synchronize()


# ---- the torch.distributed plumbing, on the one GPU there is: a group of one rank ----------------------------------

def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.fixture(scope="module")
def one_rank_group():
    import os
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(_free_port())
    try:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    except Exception as err:                       # no usable NCCL transport on this machine: nothing of the library is at fault
        pytest.skip("torch.distributed (nccl) could not be initialised here: %s" % str(err).splitlines()[0])
    yield dist.group.WORLD
    torch.cuda.synchronize()
    dist.destroy_process_group()


@pytest.mark.parametrize("transport", ["collective", "peer_store"])
def test_bucket_exchange_group_of_one(one_rank_group, transport):
    """With one rank the exchange is the send pass, a transfer to itself and a one-worker average: the result is
    dec(q) of the oracle's codes, and the state is the oracle's, over several iterations (both areas get used)."""
    from paper_2407_04480_b200 import exchange
    n = 700_001
    kw = dict(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=0, grad_dtype=1, out_dtype=0)
    gcfg, ocfg = parity.both_configs(num_partitions=1, collect_stats=0, **kw)
    try:
        ex = exchange.BucketExchange(gcfg, n, group=one_rank_group, transport=transport)
    except (RuntimeError, ImportError, AttributeError) as err:
        if transport == "peer_store":
            pytest.skip("symmetric memory is not available here: %s" % str(err).splitlines()[0])
        raise
    assert ex.shard_elems() == n
    ostate, ocomm = orc.new_state(ocfg, n), orc.new_comm(ocfg, n)
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    for k in range(3):
        g = inputs.gaussian(n, 1e-3, seed=9, worker=0, step=k, dtype=torch.bfloat16)
        gnp = inputs.as_numpy_bits(g)
        ex.step(parity.to_device(gnp, True), k, out)
        torch.cuda.synchronize()
        orc.send_step(ocfg, gnp, ostate, ocomm, k)
        want = orc.reduce(ocfg, n, [ocomm])
        got = out.cpu().numpy()
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), "step %d" % k
        gv, _ = orc.state_views(ocfg, n, ex.state.buffer.cpu().numpy())
        ov, _ = orc.state_views(ocfg, n, ostate)
        assert np.array_equal(gv, ov)
