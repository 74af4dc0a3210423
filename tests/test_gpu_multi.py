"""Several buckets per call: loco_compensate_quantize_pack_multi / loco_unpack_dequant_reduce_multi must do exactly what the
single-bucket calls do (bit for bit, against the library's own single calls and against the oracle), keep the order of
the caller's stream on both sides of the call, and be capturable into a CUDA graph."""
import numpy as np
import pytest
import torch

from oracle import loco_oracle as orc
from paper_2407_04480_b200 import inputs, loco
from tests import parity

pytestmark = pytest.mark.gpu

SIZES = [300_007, 1_000_000, 4096, 77, 2_500_123]
KW = dict(bits=4, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=0, state_fmt=0, grad_dtype=1, out_dtype=1, num_partitions=4)


def _setup(collect_stats=0):
    gcfg, ocfg = parity.both_configs(collect_stats=collect_stats, **KW)
    grads = [inputs.gaussian(n, 1e-3, seed=51, worker=i, dtype=torch.bfloat16, device="cuda") for i, n in enumerate(SIZES)]
    return gcfg, ocfg, grads


def test_multi_send_equals_single_calls_and_oracle():
    gcfg, ocfg, grads = _setup()
    single = [loco.State(gcfg, n) for n in SIZES]
    multi = [loco.State(gcfg, n) for n in SIZES]
    c_single = [torch.zeros(loco.loco_packed_bytes(gcfg, n), dtype=torch.uint8, device="cuda") for n in SIZES]
    c_multi = [torch.zeros_like(c) for c in c_single]
    ms = loco.MultiSend(multi, grads, c_multi)
    for k in range(3):
        for st, g, c in zip(single, grads, c_single):
            loco.loco_compensate_quantize_pack(st, g, c, k)
        loco.loco_compensate_quantize_pack_multi(ms, k)
    torch.cuda.synchronize()
    for i in range(len(SIZES)):
        assert torch.equal(c_single[i], c_multi[i]), "bucket %d: codes differ" % i
        assert torch.equal(single[i].buffer, multi[i].buffer), "bucket %d: state differs" % i
    # and one bucket against the oracle
    i, n = 0, SIZES[0]
    ostate, ocomm = orc.new_state(ocfg, n), orc.new_comm(ocfg, n)
    for k in range(3):
        orc.send_step(ocfg, inputs.as_numpy_bits(grads[i].cpu()), ostate, ocomm, k)
    got = c_multi[i].cpu().numpy()
    for (gc, _), (oc, _) in zip(orc.comm_views(ocfg, n, got), orc.comm_views(ocfg, n, ocomm)):
        assert np.array_equal(gc, oc)


def test_multi_reduce_equals_single_calls():
    gcfg, ocfg, grads = _setup()
    workers = 3
    packed, outs_s, outs_m = [], [], []
    for i, n in enumerate(SIZES):
        bufs = []
        for w in range(workers):
            st = loco.State(gcfg, n)
            c = torch.zeros(loco.loco_packed_bytes(gcfg, n), dtype=torch.uint8, device="cuda")
            loco.loco_compensate_quantize_pack(st, inputs.gaussian(n, 1e-3, seed=52, worker=w, step=i, dtype=torch.bfloat16, device="cuda"), c, 1)
            bufs.append(c)
        packed.append(bufs)
        outs_s.append(torch.zeros(n, dtype=torch.bfloat16, device="cuda"))
        outs_m.append(torch.zeros(n, dtype=torch.bfloat16, device="cuda"))
    for bufs, n, o in zip(packed, SIZES, outs_s):
        loco.loco_unpack_dequant_reduce(gcfg, bufs, n, o)
    mr = loco.MultiReduce(gcfg, packed, SIZES, outs_m)
    loco.loco_unpack_dequant_reduce_multi(mr)
    torch.cuda.synchronize()
    for i in range(len(SIZES)):
        assert torch.equal(outs_s[i].view(torch.int16), outs_m[i].view(torch.int16)), "bucket %d" % i
    want = orc.reduce(ocfg, SIZES[2], [b.cpu().numpy() for b in packed[2]])
    assert np.array_equal(outs_m[2].view(torch.int16).cpu().numpy().view(np.uint16), want)


def test_multi_calls_keep_the_order_of_the_callers_stream():
    """Work enqueued on the stream before the call is seen by it, work enqueued after it sees its results."""
    gcfg, _, grads = _setup()
    states = [loco.State(gcfg, n) for n in SIZES]
    ref_states = [loco.State(gcfg, n) for n in SIZES]
    comms = [torch.zeros(loco.loco_packed_bytes(gcfg, n), dtype=torch.uint8, device="cuda") for n in SIZES]
    ref = [torch.zeros_like(c) for c in comms]
    staged = [torch.zeros_like(g) for g in grads]
    copies = []
    s = torch.cuda.Stream()
    torch.cuda.synchronize()
    ms = loco.MultiSend(states, staged, comms)
    with torch.cuda.stream(s):
        for k in range(4):
            for dst, g in zip(staged, grads):
                dst.copy_(g * (k + 1))                      # producers of the inputs, on the caller's stream
            loco.loco_compensate_quantize_pack_multi(ms, k, stream=s)
            copies.append([c.clone() for c in comms])      # consumers of the outputs, on the caller's stream
    torch.cuda.synchronize()
    for k in range(4):
        for i, (st, g, c) in enumerate(zip(ref_states, grads, ref)):
            loco.loco_compensate_quantize_pack(st, g * (k + 1), c, k)
        torch.cuda.synchronize()
        for i in range(len(SIZES)):
            assert torch.equal(copies[k][i], ref[i]), "iteration %d bucket %d" % (k, i)


def test_multi_calls_in_a_cuda_graph():
    gcfg, _, grads = _setup()
    states = [loco.State(gcfg, n) for n in SIZES]
    ref_states = [loco.State(gcfg, n) for n in SIZES]
    comms = [torch.zeros(loco.loco_packed_bytes(gcfg, n), dtype=torch.uint8, device="cuda") for n in SIZES]
    outs = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for n in SIZES]
    ms = loco.MultiSend(states, grads, comms)
    mr = loco.MultiReduce(gcfg, [[c, c] for c in comms], SIZES, outs)
    loco.loco_compensate_quantize_pack_multi(ms, 5)        # first call outside capture: creates the library's streams
    loco.loco_unpack_dequant_reduce_multi(mr)
    torch.cuda.synchronize()
    for st in states:
        loco.loco_state_reset(st)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        loco.loco_compensate_quantize_pack_multi(ms, 5)
        loco.loco_unpack_dequant_reduce_multi(mr)
    for _ in range(2):                                      # two replays = two iterations with the same k
        graph.replay()
    torch.cuda.synchronize()
    ref_c = [torch.zeros_like(c) for c in comms]
    ref_o = [torch.zeros_like(o) for o in outs]
    for _ in range(2):
        for st, g, c, n, o in zip(ref_states, grads, ref_c, SIZES, ref_o):
            loco.loco_compensate_quantize_pack(st, g, c, 5)
            loco.loco_unpack_dequant_reduce(gcfg, [c, c], n, o)
    torch.cuda.synchronize()
    for i in range(len(SIZES)):
        assert torch.equal(comms[i], ref_c[i]) and torch.equal(states[i].buffer, ref_states[i].buffer)
        assert torch.equal(outs[i].view(torch.int16), ref_o[i].view(torch.int16))


def test_multi_argument_errors():
    gcfg, _, grads = _setup()
    states = [loco.State(gcfg, n) for n in SIZES]
    comms = [torch.zeros(loco.loco_packed_bytes(gcfg, n), dtype=torch.uint8, device="cuda") for n in SIZES]
    with pytest.raises(ValueError):
        loco.MultiSend(states, grads[:-1], comms)
    ms = loco.MultiSend(states, grads, comms)
    with pytest.raises(loco.LocoError) as e:
        loco.loco_compensate_quantize_pack_multi(ms, -1)
    assert e.value.code == loco.ERR_ARG
    empty = loco.MultiSend([], [], [])
    loco.loco_compensate_quantize_pack_multi(empty, 0)     # nothing to do, no error
    torch.cuda.synchronize()
