#!/usr/bin/env python
"""Benchmark of the LoCo hot path (arXiv 2407.04480) on B200.

Workload (default): what ONE data-parallel rank of an 8-worker job does per training
iteration on a Llama-2-7B-shaped gradient -- 6,738,415,616 bf16 elements cut into 270
buckets of 25,000,000 (last one partial):
    phase A  for every bucket: send pass (Algorithm 1 steps 1-2: compensate, 4-bit codes,
             moving-average error into the 8-bit state, pack into the 8-part buffer);
    phase B  for every bucket: receive pass (Eq. 8) over all 8 parts of the bucket, averaging this
             worker's packed buffer with the buffers of the 7 other simulated workers (resident in
             the same HBM), into the bf16 gradient handed to the optimizer.
All inputs are synthetic and resident in HBM before the timed region; every bucket is read
once per step and the step touches ~70 GB, far more than the 126 MB L2.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  With --impl reference the CPU oracle is timed instead, on a
bounded sample of the same workload (it is a deliberately plain program: the ratio to it is
context, parity and the roofline fraction are the results).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

METRIC = "compensate+quantize and dequant-reduce GB/s of gradient per bucket pass (send, then 8-worker reduce)"
BUCKET = 25_000_000
WORKERS = 8
L2_BYTES = 126 * 1024 * 1024
# Paper-faithful settings (Eq. 1 global scale; Eq. 7 T_c; s_e = 4 s); beta is not printed in the paper.
CFG = dict(bits=4, scale_mode=0, block_size=256, s=2.0 ** 14, s_e=2.0 ** 16, beta=0.5, reset_period=512,
           state_fmt=0, grad_dtype=1, out_dtype=1, num_partitions=WORKERS)
# Algorithmic HBM bytes per element (bf16 gradient read, int8 state read + written, 4-bit code written).
SEND_BYTES_PER_ELEM = 2 + 1 + 1 + 0.5
# dram__bytes_read.sum + dram__bytes_write.sum per launch (one 25M-element bucket) from the ncu captures summarised under
# profiles/.  Reads equal the algorithmic reads; most written lines are still in the 126 MB L2 when a lone launch ends,
# so the DRAM write counter of a single captured launch is far below the algorithmic 37.5 / 50 MB.
SEND_DRAM_BYTES_PER_LAUNCH = 75.03e6 + 2.53e6
REDUCE_DRAM_BYTES_PER_LAUNCH = 100.03e6 + 14.24e6


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle samples taken every 200 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.dev = device_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.dev), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, reasons, smax = [], set(), None
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    smax = float(f[2])
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=smax, reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------------------------------------ our arm

class RankWorkload:
    """Buffers of one rank: its gradient, error state, own packed buffers, the 7 received parts, the output."""

    def __init__(self, rank: int, device: torch.device, max_buckets: int = 0):
        from paper_2407_04480_b200 import inputs, loco
        self.loco = loco
        self.cfg = loco.Config(**CFG)
        self.part = rank % WORKERS
        layout = inputs.llama2_7b()
        scales = inputs.group_scales(1, layout.n_groups)
        self.buckets = inputs.bucket_ranges(layout.numel, BUCKET)
        if max_buckets > 0:
            self.buckets = self.buckets[:max_buckets]
        self.total = self.buckets[-1][1]
        self.grad = torch.empty(self.total, dtype=torch.bfloat16, device=device)
        for lo, hi in self.buckets:
            self.grad[lo:hi] = inputs.layout_slice(layout, lo, hi, scales, 1e-4, seed=1, worker=rank, step=0,
                                                   device=device)
        cfg = self.cfg
        sb = [loco.loco_state_bytes(cfg, hi - lo) for lo, hi in self.buckets]
        pb = [loco.loco_packed_bytes(cfg, hi - lo) for lo, hi in self.buckets]
        self.state_buf = torch.empty(sum(sb), dtype=torch.uint8, device=device)
        self.comm_buf = torch.empty(sum(pb), dtype=torch.uint8, device=device)
        # packed buffers of the 7 other workers as they would sit after the exchange: any byte is two valid codes
        gen = torch.Generator(device=device)
        gen.manual_seed(1234 + rank)
        self.recv_buf = torch.empty(sum(pb) * (WORKERS - 1), dtype=torch.uint8, device=device)
        chunk = 1 << 30
        for off in range(0, self.recv_buf.numel(), chunk):
            m = min(chunk, self.recv_buf.numel() - off)
            self.recv_buf[off:off + m] = torch.randint(0, 256, (m,), dtype=torch.uint8, device=device, generator=gen)
        self.out_buf = torch.empty(self.total, dtype=torch.bfloat16, device=device)
        self.states, self.grads, self.comms, self.packed, self.outs = [], [], [], [], []
        so = co = ro = 0
        for i, (lo, hi) in enumerate(self.buckets):
            n = hi - lo
            self.states.append(loco.State(cfg, n, buffer=self.state_buf[so:so + sb[i]]))
            self.grads.append(self.grad[lo:hi])
            comm = self.comm_buf[co:co + pb[i]]
            self.comms.append(comm)
            ptrs = []
            for w in range(WORKERS):
                if w == self.part:
                    ptrs.append(comm.data_ptr())
                else:
                    ptrs.append(self.recv_buf.data_ptr() + ro)
                    ro += pb[i]
            self.packed.append(ptrs)
            self.outs.append(self.out_buf[lo:hi])
            so += sb[i]
            co += pb[i]
        self.send_bytes = SEND_BYTES_PER_ELEM * self.total
        self.recv_bytes = self.total * (WORKERS * 0.5 + 2)
        self.grad_bytes = 2 * self.total

    def _fan_out(self, launch, n_items: int, streams):
        """Issue item i on streams[i % len]: buckets are independent, so consecutive launches may overlap
        (the next kernel's CTAs fill the SMs that the previous kernel's tail leaves idle)."""
        if not streams:
            for i in range(n_items):
                launch(i, None)
            return
        cur = torch.cuda.current_stream()
        for s in streams:
            s.wait_stream(cur)
        for i in range(n_items):
            s = streams[i % len(streams)]
            with torch.cuda.stream(s):
                launch(i, s)
        for s in streams:
            cur.wait_stream(s)

    def send_phase(self, k: int, streams=None):
        f = self.loco.loco_compensate_quantize_pack
        self._fan_out(lambda i, s: f(self.states[i], self.grads[i], self.comms[i], k, stream=s), len(self.buckets), streams)

    def reduce_phase(self, streams=None):
        f = self.loco.loco_unpack_dequant_reduce
        self._fan_out(lambda i, s: f(self.cfg, self.packed[i], self.buckets[i][1] - self.buckets[i][0], self.outs[i], stream=s),
                      len(self.buckets), streams)


def run_e2e(wl: RankWorkload, steps: int, warmup: int):
    """Same step through the host-buffer entry points: every bucket's gradient and the 8 workers' packed
    buffers are copied from pinned host memory, the packed codes and the averaged gradient are copied back."""
    loco, cfg = wl.loco, wl.cfg
    ring = 3
    nmax = BUCKET
    pbytes = loco.loco_packed_bytes(cfg, nmax)
    h_grad = [torch.empty(nmax, dtype=torch.bfloat16).pin_memory() for _ in range(ring)]
    h_comm = [torch.empty(pbytes, dtype=torch.uint8).pin_memory() for _ in range(ring)]
    h_parts = [[torch.randint(0, 256, (pbytes,), dtype=torch.uint8).pin_memory() for _ in range(WORKERS)] for _ in range(ring)]
    h_out = [torch.empty(nmax, dtype=torch.bfloat16).pin_memory() for _ in range(ring)]
    for r in range(ring):
        h_grad[r].copy_(wl.grads[r].cpu())
    dev = wl.grad.device
    w_send = torch.empty(loco.loco_send_host_workspace_bytes(cfg, nmax), dtype=torch.uint8, device=dev)
    w_red = torch.empty(loco.loco_reduce_host_workspace_bytes(cfg, nmax, WORKERS, cfg.num_partitions), dtype=torch.uint8, device=dev)
    h2d = d2h = 0
    for i, (lo, hi) in enumerate(wl.buckets):
        n = hi - lo
        h2d += 2 * n + WORKERS * loco.loco_packed_bytes(cfg, n)
        d2h += loco.loco_packed_bytes(cfg, n) + 2 * n

    # Two streams: the send pass of bucket i+1 (gradient in, codes out) runs while the receive pass of bucket i (8 packed
    # buffers in, averaged gradient out) is still copying, so that both directions of the host link are busy; the receive
    # pass of a bucket starts only after its send pass has finished.
    s_send, s_recv = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    done = [torch.cuda.Event() for _ in wl.buckets]

    def step(k):
        cur = torch.cuda.current_stream()
        s_send.wait_stream(cur)
        s_recv.wait_stream(cur)
        for i, (lo, hi) in enumerate(wl.buckets):
            n = hi - lo
            r = i % ring
            loco.loco_compensate_quantize_pack_host(wl.states[i], h_grad[r][:n], h_comm[r], w_send, k, stream=s_send)
            done[i].record(s_send)
            s_recv.wait_event(done[i])
            loco.loco_unpack_dequant_reduce_host(cfg, h_parts[r], n, h_out[r], w_red, stream=s_recv)
        cur.wait_stream(s_send)
        cur.wait_stream(s_recv)

    for k in range(warmup):
        step(1000 + k)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for k in range(steps):
        step(2000 + k)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    return ms, h2d, d2h


def oracle_sample(threads: int, buckets_per_thread: int):
    """The oracle as it stands on `threads` host threads, each doing whole 25M-element buckets of the
    workload (send pass, then the receive pass over the whole bucket with 8 workers)."""
    import numpy as np
    from oracle import loco_oracle as orc
    ocfg = orc.OracleConfig(**CFG)
    n = BUCKET
    rng = np.random.default_rng(1)
    g = (rng.normal(0, 1e-4, n).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    others = [rng.integers(0, 256, orc.packed_bytes(ocfg, n), dtype=np.uint8) for _ in range(2)]
    states = [orc.new_state(ocfg, n) for _ in range(threads)]
    comms = [orc.new_comm(ocfg, n) for _ in range(threads)]
    orc.lib()

    def work(t):
        for b in range(buckets_per_thread):
            orc.send_step(ocfg, g, states[t], comms[t], 1 + b)
            orc.reduce(ocfg, n, [comms[t]] + [others[w % 2] for w in range(WORKERS - 1)])

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(work, range(threads)))
    dt = time.perf_counter() - t0
    elems = threads * buckets_per_thread * n
    return 2.0 * elems / dt / 1e9, dt, elems


# ------------------------------------------------------------------------------------------------ real exchange

def run_exchange(args, rank: int, world: int, device, config):
    """The same buckets with the exchange of Sec. 3.3 between the ranks: every rank compresses its own gradient into
    `world` parts, the parts travel (NCCL all-to-all, or the send kernel's own stores into the peers' receive slots),
    every rank averages the `world` copies of its part.  One stream per rank, bucket after bucket; no CUDA graph, since
    the collective sits between the two kernels.  value = gradient bytes entering the path on all ranks per second."""
    import torch.distributed as dist
    from paper_2407_04480_b200 import exchange, inputs, loco
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29531")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=device)
    cfg = loco.Config(**{**CFG, "num_partitions": world})
    layout = inputs.llama2_7b()
    scales = inputs.group_scales(1, layout.n_groups)
    buckets = inputs.bucket_ranges(layout.numel, BUCKET)
    if args.buckets > 0:
        buckets = buckets[:args.buckets]
    total = buckets[-1][1]
    grad = torch.empty(total, dtype=torch.bfloat16, device=device)
    for lo, hi in buckets:
        grad[lo:hi] = inputs.layout_slice(layout, lo, hi, scales, 1e-4, seed=1, worker=rank, step=0, device=device)
    if args.exchange == "reduce_scatter_bf16":
        # the uncompressed baseline: every bucket padded to a multiple of the group size and reduce-scattered as it is
        padded = [-(-(hi - lo) // world) * world for lo, hi in buckets]
        stage = torch.zeros(max(padded), dtype=torch.bfloat16, device=device)
        shard = torch.empty(max(padded) // world, dtype=torch.bfloat16, device=device)

        def step(k):
            for (lo, hi), m in zip(buckets, padded):
                stage[:hi - lo].copy_(grad[lo:hi])
                dist.reduce_scatter_tensor(shard[:m // world], stage[:m], op=dist.ReduceOp.AVG)
    else:
        transport = exchange.Transport(cfg, BUCKET, kind=args.exchange, device=device)
        exs = [exchange.BucketExchange(cfg, hi - lo, shared=transport) for lo, hi in buckets]
        shard = torch.empty(max(e.shard_elems() for e in exs), dtype=torch.bfloat16, device=device)

        def step(k):
            for e, (lo, hi) in zip(exs, buckets):
                e.step(grad[lo:hi], k, shard)

    for k in range(max(3, args.warmup)):
        step(k)
    dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(device.index)
    sampler.start()
    before = loco.loco_launch_count()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for k in range(args.steps):
        step(100 + k)
    end.record()
    dist.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    t = torch.tensor([start.elapsed_time(end) / args.steps], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    lt = torch.tensor([loco.loco_launch_count() - before], device=device, dtype=torch.int64)
    dist.all_reduce(lt)
    step_ms = float(t.item())
    if rank == 0:
        config = dict(config, exchange=args.exchange, streams=1, workers_on_reduce_side=world,
                      workload=config["workload"].split(":")[0] + ": %d bf16 buckets per rank; per bucket: send pass, exchange "
                      "of %d parts between the ranks, average of this rank's part" % (len(buckets), world))
        suffix = (" -- uncompressed bf16 NCCL reduce-scatter of the same buckets (what the method replaces; none of this "
                  "library's kernels)") if args.exchange == "reduce_scatter_bf16" else " -- with the real exchange"
        print(json.dumps({"metric": METRIC + suffix, "value": world * 2 * total / (step_ms * 1e-3) / 1e9,
                          "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
                          "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                          "dtype": "f32", "data": "synthetic", "config": config, "clocks": clocks, "e2e": None,
                          "gpu_launches": int(lt.item()), "roofline": None, "cpu_baseline": None}))
    dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------ sweep (config 5)

def _time_launches(launch, n_sets: int, launches: int, streams):
    """Average device time of `launch(set_index, stream)` over `launches` launches that walk round-robin over n_sets
    independent working sets and alternate between the streams (CUDA events on the current stream around all)."""
    def run(count):
        cur = torch.cuda.current_stream()
        for st in streams:
            st.wait_stream(cur)
        for i in range(count):
            st = streams[i % len(streams)]
            with torch.cuda.stream(st):
                launch(i % n_sets, st)
        for st in streams:
            cur.wait_stream(st)

    run(min(launches, 2 * n_sets))
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()                       # replayed, so that the host's launch cost is not what is timed
    with torch.cuda.graph(graph):
        run(launches)
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / launches          # microseconds


def sweep(args, device):
    """Throughput table over bucket size, gradient type, state format, code width, scale rule and worker count
    (Gaussian gradients, seed 4).  Every launch touches a working set that the previous launches did not leave in L2
    unless the row says so."""
    from paper_2407_04480_b200 import inputs, loco
    peak, peak_kind = measured_peak()
    # launches alternate between three streams, as the library's multi-bucket calls issue them (one stream with --streams 1)
    streams = [torch.cuda.Stream(device=device) for _ in range(3 if args.streams > 1 else 1)]
    rows = []
    budget = 6 << 30                    # device bytes per case

    def sets_for(bytes_per_set):
        want = max(3, -(-(1 << 30) // bytes_per_set))
        return int(max(1, min(want, 256, budget // max(1, bytes_per_set))))

    def send_case(label, n, **kw):
        if args.sweep_filter and args.sweep_filter not in "send: " + label:
            return
        base = dict(bits=4, scale_mode=0, block_size=256, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=512, state_fmt=0,
                    grad_dtype=1, out_dtype=1, num_partitions=8)
        scatter = kw.pop("scatter", False)
        base.update(kw)
        cfg = loco.Config(**base)
        gsz = 2 if cfg.grad_dtype == loco.BF16 else 4
        sb, pb = loco.loco_state_bytes(cfg, n), loco.loco_packed_bytes(cfg, n)
        nsets = sets_for(n * gsz + sb + pb)
        dt = torch.bfloat16 if gsz == 2 else torch.float32
        grads = [inputs.gaussian(n, 1e-3, seed=4, worker=i, dtype=dt, device=device) for i in range(nsets)]
        states = [loco.State(cfg, n) for _ in range(nsets)]
        comms = [torch.empty(max(pb, 16), dtype=torch.uint8, device=device) for _ in range(nsets)]
        if scatter:                                 # part j of every set goes to a buffer of its own ("worker j's receive slot")
            part = loco.loco_partition_bytes(cfg, n)
            dsts = [[torch.empty(max(part, 16), dtype=torch.uint8, device=device) for _ in range(cfg.num_partitions)]
                    for _ in range(nsets)]
            send = lambda i, k, st=None: loco.loco_compensate_quantize_pack_scatter(states[i], grads[i], dsts[i], k, stream=st)
        else:
            send = lambda i, k, st=None: loco.loco_compensate_quantize_pack(states[i], grads[i], comms[i], k, stream=st)
        for i in range(nsets):                      # a first iteration, so that the timed ones meet a non-zero state
            send(i, 1)
        torch.cuda.synchronize()
        us = _time_launches(lambda i, st: send(i, 2, st), nsets, max(12, min(200, 4 * nsets)), streams)
        state_rw = {0: 2, 1: 8, 2: 0, 3: 8}[cfg.state_fmt]
        scale_b = (4.0 / cfg.block_size) * (3 if cfg.state_fmt == 0 else 1) if cfg.scale_mode == 1 else 0.0
        bpe = gsz + state_rw + cfg.bits / 8 + scale_b
        gbs = bpe * n / us / 1e3
        rows.append(dict(kernel="send", case=label, n=n, bytes_per_elem=round(bpe, 3), us=round(us, 2), hbm_gbs=round(gbs, 1),
                         frac=round(gbs / peak, 3), grad_gbs=round(gsz * n / us / 1e3, 1),
                         l2_resident=bool(nsets * (n * gsz + sb + pb) < L2_BYTES)))
        print(json.dumps(rows[-1]), flush=True)

    def reduce_case(label, n, workers, **kw):
        if args.sweep_filter and args.sweep_filter not in "reduce: " + label:
            return
        base = dict(bits=4, scale_mode=0, block_size=256, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=512, state_fmt=2,
                    grad_dtype=1, out_dtype=1, num_partitions=8)
        one_part = kw.pop("one_part", False)            # only part 3 of 8: what one rank averages after the exchange
        base.update(kw)
        cfg = loco.Config(**base)
        osz = 2 if cfg.out_dtype == loco.BF16 else 4
        pb = loco.loco_packed_bytes(cfg, n)
        nsets = sets_for(workers * pb + n * osz)
        gen = torch.Generator(device=device)
        gen.manual_seed(4)
        packed = []
        for i in range(nsets):
            if cfg.scale_mode == 1:                 # block scales must be real numbers: compress real gradients
                bufs = []
                for w in range(workers):
                    st = loco.State(cfg, n)
                    c = torch.empty(max(pb, 16), dtype=torch.uint8, device=device)
                    loco.loco_compensate_quantize_pack(st, inputs.gaussian(n, 1e-3, seed=4, worker=w, step=i, dtype=torch.bfloat16, device=device), c, 1)
                    bufs.append(c)
                packed.append(bufs)
            else:
                packed.append([torch.randint(0, 256, (max(pb, 16),), dtype=torch.uint8, device=device, generator=gen) for _ in range(workers)])
        outs = [torch.empty(n, dtype=torch.bfloat16 if osz == 2 else torch.float32, device=device) for _ in range(nsets)]
        torch.cuda.synchronize()
        if one_part:
            stride = loco.loco_partition_bytes(cfg, n)
            slots = [[b[3 * stride:4 * stride] for b in bufs] for bufs in packed]
            us = _time_launches(lambda i, st: loco.loco_unpack_dequant_reduce(cfg, slots[i], n, outs[i], first_partition=3,
                                                                                partition_count=1, stream=st),
                                nsets, max(12, min(200, 4 * nsets)), streams)
            n = loco.loco_partition_elems(cfg, n, 3)        # elements this launch produces
        else:
            us = _time_launches(lambda i, st: loco.loco_unpack_dequant_reduce(cfg, packed[i], n, outs[i], stream=st),
                                nsets, max(12, min(200, 4 * nsets)), streams)
        bpe = workers * cfg.bits / 8 + osz + (workers * 4.0 / cfg.block_size if cfg.scale_mode == 1 else 0.0)
        gbs = bpe * n / us / 1e3
        rows.append(dict(kernel="reduce", case=label, n=n, workers=workers, bytes_per_elem=round(bpe, 3), us=round(us, 2),
                         hbm_gbs=round(gbs, 1), frac=round(gbs / peak, 3), grad_gbs=round(osz * n / us / 1e3, 1),
                         l2_resident=bool(nsets * (workers * pb + n * osz) < L2_BYTES)))
        print(json.dumps(rows[-1]), flush=True)

    def adam_case(label, n, workers, **kw):
        if args.sweep_filter and args.sweep_filter not in "reduce+adam: " + label:
            return
        base = dict(bits=4, scale_mode=0, block_size=256, s=2.0 ** 11, s_e=2.0 ** 13, beta=0.5, reset_period=512, state_fmt=2,
                    grad_dtype=1, out_dtype=1, num_partitions=8)
        base.update(kw)
        cfg = loco.Config(**base)
        pb = loco.loco_packed_bytes(cfg, n)
        nsets = sets_for(workers * pb + n * 12)
        gen = torch.Generator(device=device)
        gen.manual_seed(4)
        packed = [[torch.randint(0, 256, (max(pb, 16),), dtype=torch.uint8, device=device, generator=gen) for _ in range(workers)]
                  for _ in range(nsets)]
        ms = [torch.zeros(n, dtype=torch.float32, device=device) for _ in range(nsets)]
        vs = [torch.zeros(n, dtype=torch.float32, device=device) for _ in range(nsets)]
        ths = [torch.ones(n, dtype=torch.float32, device=device) for _ in range(nsets)]
        torch.cuda.synchronize()
        us = _time_launches(lambda i, st: loco.loco_unpack_dequant_reduce_adam(cfg, packed[i], n, ms[i], vs[i], ths[i], lr=1e-3, beta1=0.1,
                                                                                 beta2=0.001, delta=1e-16, stream=st),
                            nsets, max(12, min(200, 4 * nsets)), streams)
        bpe = workers * cfg.bits / 8 + 24
        gbs = bpe * n / us / 1e3
        rows.append(dict(kernel="reduce+adam", case=label, n=n, workers=workers, bytes_per_elem=round(bpe, 3), us=round(us, 2),
                         hbm_gbs=round(gbs, 1), frac=round(gbs / peak, 3), grad_gbs=round(4 * n / us / 1e3, 1),
                         l2_resident=bool(nsets * (workers * pb + n * 12) < L2_BYTES)))
        print(json.dumps(rows[-1]), flush=True)

    M = 25_000_000
    for log2n in (16, 18, 20, 22, 24, 27, 30):
        send_case("bf16 g, int8 state, 4 bit, fixed", 1 << log2n)
    for log2n in (16, 20, 24, 27, 30):
        send_case("fp32 g, int8 state, 4 bit, fixed", 1 << log2n, grad_dtype=0)
    for bits in (2, 4, 8):
        send_case("bf16 g, int8 state, %d bit, fixed" % bits, M, bits=bits)
        send_case("fp32 g, int8 state, %d bit, fixed" % bits, M, bits=bits, grad_dtype=0)
    send_case("bf16 g, int8 state, 4 bit, fixed, s_e = 6 s (Newton-Raphson decompressor)", M, s_e=6 * 2.0 ** 11)
    send_case("bf16 g, int8 state, 4 bit, fixed, statistics on", M, collect_stats=1)
    send_case("bf16 g, int8 state, 4 bit, fixed, element-wise clipping at 2 sigma", M, clip=2e-3)
    send_case("bf16 weights, no state, 8 bit, block-256 absmax (Zero++-style weight payload)", M, bits=8, scale_mode=1, state_fmt=2)
    send_case("bf16 g, int8 state, 4 bit, fixed, stochastic rounding (Philox4x32-10)", M, rounding=1, seed=7)
    send_case("bf16 g, int8 state, 4 bit, fixed, parts scattered to 8 receive slots (all-to-all in the stores)", M, scatter=True)
    send_case("bf16 g, fp32 state, 4 bit, fixed", M, state_fmt=1)
    send_case("bf16 g, fp32 state + 8-bit compensation, 4 bit, fixed", M, state_fmt=3)
    send_case("bf16 g, no state, 4 bit, fixed", M, state_fmt=2)
    for B in (256, 64, 32):
        send_case("bf16 g, int8 state, 4 bit, block-%d absmax" % B, M, scale_mode=1, block_size=B)
    send_case("fp32 g, int8 state, 4 bit, block-256 absmax", M, scale_mode=1, grad_dtype=0)
    for log2n in (16, 20, 24, 27, 30):
        reduce_case("4 bit, bf16 out, fixed", 1 << log2n, 8)
    for bits in (2, 4, 8):
        for od in (1, 0):
            for N in (1, 2, 4, 8, 16):
                reduce_case("%d bit, %s out, fixed" % (bits, "bf16" if od else "fp32"), M, N, bits=bits, out_dtype=od)
    reduce_case("4 bit, bf16 out, fixed, s = 3000 (generic path)", M, 8, s=3000.0)
    reduce_case("4 bit, bf16 out, fixed, 3 workers (division by 3)", M, 3)
    reduce_case("4 bit, bf16 out, fixed, one part of 8 of a 25M-element bucket (a rank's share after the exchange)", M, 8, one_part=True)
    reduce_case("4 bit, bf16 out, fixed, one part of 8 of a 200M-element bucket", 8 * M, 8, one_part=True)
    reduce_case("4 bit, bf16 out, block-256 absmax", M, 8, scale_mode=1)
    reduce_case("4 bit, bf16 out, block-32 absmax", M, 8, scale_mode=1, block_size=32)
    reduce_case("8 bit, bf16 out, block-256 absmax, 1 worker (Zero++-style weight payload)", M, 1, bits=8, scale_mode=1)
    for N in (1, 8, 16):
        adam_case("4 bit, fixed, Adam-family step fused, no gradient output", M, N)
    adam_case("8 bit, fixed, Adam-family step fused, no gradient output", M, 8, bits=8)
    adam_case("4 bit, fixed, Adam-family step fused, no gradient output", 1 << 27, 8)
    print("| kernel | case | n | workers | B/elem | us/launch | HBM GB/s | of %s peak %.0f | gradient GB/s | L2-resident |" % (peak_kind, peak))
    print("|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        print("| %s | %s | %d | %s | %s | %s | %s | %.3f | %s | %s |" % (r["kernel"], r["case"], r["n"], r.get("workers", "-"), r["bytes_per_elem"],
                                                                      r["us"], r["hbm_gbs"], r["frac"], r["grad_gbs"], "yes" if r["l2_resident"] else ""))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--buckets", type=int, default=0,
                    help="profiling aid: only the first K buckets of the workload (0 = all 270); not a bench line")
    ap.add_argument("--no-graph", action="store_true", help="profiling aid: launch every kernel directly")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the bench line: the size / type / width / worker-count table (one JSON line per case, then markdown)")
    ap.add_argument("--sweep-filter", default="", help="with --sweep: only the cases whose 'kernel: label' contains this text")
    ap.add_argument("--exchange", choices=("none", "collective", "peer_store", "reduce_scatter_bf16"), default="none",
                    help="none (default): every rank runs the two passes on its own buckets, no data-path collective; "
                         "collective / peer_store: the real exchange of Sec. 3.3 between the ranks (NCCL all-to-all, or the "
                         "send kernel storing into the peers' receive slots), each rank reducing its own shard; "
                         "reduce_scatter_bf16: what the method replaces -- NCCL reduce-scatter (average) of the uncompressed bf16 "
                         "buckets, none of this library's kernels, for comparison on the same buckets")
    ap.add_argument("--streams", type=int, default=2,
                    help="2 or more (default): each phase is one multi-bucket call of the library on one stream (the library overlaps "
                         "consecutive launches on streams of its own); 1: single-bucket calls strictly one after the other")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cores = os.cpu_count() or 1
    config = {"workload": "llama2-7b: 270 bf16 buckets of 25M elements (6,738,415,616): one worker's send pass per bucket, then the 8-worker reduce of the bucket",
              "bits": 4, "scale": "fixed s=2^14, s_e=4s (Eq. 1)", "beta": 0.5, "T_c": 512, "state": "int8",
              "workers_on_reduce_side": WORKERS, "out": "bf16",
              "streams": ("1 caller stream; loco_*_multi calls overlap consecutive buckets on the library's 3 streams"
                          if args.streams > 1 and not args.no_graph else "1, single-bucket calls one after the other"),
              "l2": "inputs larger than L2: each step streams ~70 GB once, no reuse between launches"}

    if args.impl == "reference":
        if rank != 0:
            return
        steps = max(1, args.steps)
        for _ in range(min(args.warmup, 1)):
            oracle_sample(cores, 1)
        t0 = time.perf_counter()
        elems = 0
        for _ in range(steps):
            _, _, e = oracle_sample(cores, 1)
            elems += e
        dt = time.perf_counter() - t0
        val = 2.0 * elems / dt / 1e9
        sample = "%d buckets of 25M elements per step (one per host thread), send + 8-worker reduce" % cores
        print(json.dumps({"impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus,
                          "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": dt / steps * 1e3,
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                          "data": "synthetic", "config": config,
                          "cpu_baseline": {"value": val, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
                          "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                          "gpu_launches": 0}))
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    from paper_2407_04480_b200 import loco
    loco.lib()
    if args.sweep:
        if rank == 0:
            sweep(args, device)
        return
    if args.exchange != "none":
        run_exchange(args, rank, world, device, config)
        return
    wl = RankWorkload(rank, device, args.buckets)
    nb = len(wl.buckets)
    if args.buckets > 0:
        config["workload"] += " -- REDUCED to the first %d buckets (profiling aid, not the bench workload)" % nb
    # The 540 launches of a step are captured once into two CUDA graphs (one per phase) and replayed,
    # so that the host's launch cost does not sit between kernels of a few microseconds each.
    wl.send_phase(1)
    wl.reduce_phase()
    torch.cuda.synchronize()
    if args.no_graph:
        class _Direct:
            def __init__(self, fn): self.replay = fn
        g_send, g_reduce = _Direct(lambda: wl.send_phase(100)), _Direct(wl.reduce_phase)
    else:
        side = [torch.cuda.Stream(device=device) for _ in range(args.streams)] if args.streams > 1 else None
        g_send, g_reduce = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        if args.streams > 1:
            # the library's multi-bucket calls, issued on this one stream: they take three streams of
            # the library's own and join them back, so that a bucket's tail overlaps the next bucket's start-up
            ms = loco.MultiSend(wl.states, wl.grads, wl.comms)
            mr = loco.MultiReduce(wl.cfg, wl.packed, [hi - lo for lo, hi in wl.buckets], wl.outs)
            loco.loco_compensate_quantize_pack_multi(ms, 100)       # first call outside capture: creates the library's streams
            loco.loco_unpack_dequant_reduce_multi(mr)
            torch.cuda.synchronize()
            with torch.cuda.graph(g_send):
                loco.loco_compensate_quantize_pack_multi(ms, 100)
            with torch.cuda.graph(g_reduce):
                loco.loco_unpack_dequant_reduce_multi(mr)
        else:
            with torch.cuda.graph(g_send):
                wl.send_phase(100, None)
            with torch.cuda.graph(g_reduce):
                wl.reduce_phase(None)
    for k in range(max(3, args.warmup)):
        g_send.replay()
        g_reduce.replay()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    barrier()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for k in range(K):
        ev[k][0].record()
        g_send.replay()
        ev[k][1].record()
        g_reduce.replay()
        ev[k][2].record()
    end.record()
    barrier()
    launches = 2 * nb * K          # one send and one receive kernel per bucket and step, replayed from the graphs
    clocks = sampler.stop()
    # outside the timed region: the same two phases with every launch strictly after the previous one (one stream),
    # which shows what a launch costs when nothing overlaps its start-up and its tail
    serial_us = None
    if not args.no_graph and args.streams > 1:
        s_send, s_reduce = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(s_send):
            wl.send_phase(100, None)
        with torch.cuda.graph(s_reduce):
            wl.reduce_phase(None)
        s_send.replay(); s_reduce.replay()
        sev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        torch.cuda.synchronize()
        sev[0].record(); s_send.replay(); s_send.replay(); sev[1].record(); s_reduce.replay(); s_reduce.replay(); sev[2].record()
        torch.cuda.synchronize()
        serial_us = (sev[0].elapsed_time(sev[1]) * 1e3 / (2 * nb), sev[1].elapsed_time(sev[2]) * 1e3 / (2 * nb))
    # also outside the timed region, for scale: a plain device-to-device copy (the driver's cudaMemcpyAsync, issued by
    # torch) that moves as many bytes per launch as the send kernel does, one launch per bucket over memory not in L2
    copy_us = None
    if not args.no_graph:
        half = int(SEND_BYTES_PER_ELEM * BUCKET / 2) // 256 * 256          # bytes copied = half of read + written
        src8, dst8 = wl.grad.view(torch.uint8), wl.out_buf.view(torch.uint8)
        span = min(src8.numel(), dst8.numel())
        count = max(1, min(nb, span // half))

        def copies(streams):
            wl._fan_out(lambda i, st: dst8[i * half:(i + 1) * half].copy_(src8[i * half:(i + 1) * half]), count, streams)

        res = []
        for strs in (None, side if args.streams > 1 else None):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                copies(strs)
            g.replay()
            ce = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            torch.cuda.synchronize()
            ce[0].record(); g.replay(); g.replay(); ce[1].record()
            torch.cuda.synchronize()
            res.append(ce[0].elapsed_time(ce[1]) * 1e3 / (2 * count))
        copy_us = {"bytes_moved_per_launch": 2 * half, "one_stream_launch_us": res[0], "one_stream_gbs": 2 * half / res[0] / 1e3,
                   "two_stream_launch_us": res[1], "two_stream_gbs": 2 * half / res[1] / 1e3}
    total_ms = start.elapsed_time(end)
    send_ms = sum(e[0].elapsed_time(e[1]) for e in ev) / K
    recv_ms = sum(e[1].elapsed_time(e[2]) for e in ev) / K
    step_ms = total_ms / K
    if dist is not None:
        t = torch.tensor([step_ms, send_ms, recv_ms], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        step_ms, send_ms, recv_ms = [float(x) for x in t]
        lt = torch.tensor([launches], device=device, dtype=torch.int64)
        dist.all_reduce(lt)
        launches = int(lt.item())

    e2e = None
    if not args.no_e2e:
        e_ms, h2d, d2h = run_e2e(wl, args.e2e_steps, 1)
        if dist is not None:
            t = torch.tensor([e_ms], device=device, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e_ms = float(t.item())
        e2e = {"value": world * wl.grad_bytes / (e_ms * 1e-3) / 1e9, "unit": "GB/s", "h2d_bytes_per_step": h2d * world,
               "d2h_bytes_per_step": d2h * world, "ms_per_step": e_ms, "steps": args.e2e_steps,
               "how": "loco_*_host entry points, pinned host buffers, copies inside the timed region; send and receive passes "
                      "on two streams so that host-to-device and device-to-host copies overlap"}
    if dist is not None:
        dist.barrier()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    send_gbs = wl.send_bytes / (send_ms * 1e-3) / 1e9
    recv_gbs = wl.recv_bytes / (recv_ms * 1e-3) / 1e9
    how = ("CUDA events around this kernel's phase of every timed step / launches in it; " +
           ("a phase is one multi-bucket call of the library on one stream, which spreads the launches over three streams of "
            "its own, so a kernel's start-up and tail overlap its neighbour" if args.streams > 1 and not args.no_graph else
            "every launch strictly after the previous one"))
    roof_send = {"kernel": "loco_send_kernel<bf16 g, int8 state, 4 bit, fixed scale>", "bound": "hbm",
                 "achieved": send_gbs, "peak": peak, "peak_kind": "%s HBM copy bandwidth" % peak_kind, "unit": "GB/s",
                 "frac": send_gbs / peak, "frac_of_nominal_8TBps": send_gbs / 8000.0, "traffic": SEND_DRAM_BYTES_PER_LAUNCH,
                 "algorithmic_bytes_per_launch": SEND_BYTES_PER_ELEM * BUCKET, "avg_launch_us": send_ms * 1e3 / nb,
                 "launches_per_step": nb, "how": how}
    roof_reduce = {"kernel": "loco_reduce_kernel<bf16 out, 4 bit, fixed scale>, 8 workers", "bound": "hbm",
                   "achieved": recv_gbs, "peak": peak, "peak_kind": "%s HBM copy bandwidth" % peak_kind, "unit": "GB/s",
                   "frac": recv_gbs / peak, "frac_of_nominal_8TBps": recv_gbs / 8000.0, "traffic": REDUCE_DRAM_BYTES_PER_LAUNCH,
                   "algorithmic_bytes_per_launch": (WORKERS * 0.5 + 2) * BUCKET, "avg_launch_us": recv_ms * 1e3 / nb,
                   "launches_per_step": nb, "how": how}
    # the roofline object describes the kernel that takes the larger share of the step; the other one rides along
    roofline, other = (roof_reduce, roof_send) if recv_ms >= send_ms else (roof_send, roof_reduce)
    roofline["other_kernel"] = other
    kernels = {"send": {"hbm_gbs": send_gbs, "frac_of_peak": send_gbs / peak, "gradient_gbs": wl.grad_bytes / (send_ms * 1e-3) / 1e9,
                        "ms_per_step": send_ms, "avg_launch_us": send_ms * 1e3 / nb, "bytes_per_elem": SEND_BYTES_PER_ELEM},
               "reduce": {"hbm_gbs": recv_gbs, "frac_of_peak": recv_gbs / peak,
                          "gradient_gbs": wl.grad_bytes / (recv_ms * 1e-3) / 1e9, "ms_per_step": recv_ms,
                          "avg_launch_us": recv_ms * 1e3 / nb, "bytes_per_out_elem": WORKERS * 0.5 + 2}}
    if serial_us is not None:
        kernels["send"]["one_stream_launch_us"] = serial_us[0]
        kernels["send"]["one_stream_hbm_gbs"] = wl.send_bytes / nb / (serial_us[0] * 1e-6) / 1e9
        kernels["reduce"]["one_stream_launch_us"] = serial_us[1]
        kernels["reduce"]["one_stream_hbm_gbs"] = wl.recv_bytes / nb / (serial_us[1] * 1e-6) / 1e9
    if copy_us is not None:
        kernels["device_copy_same_bytes_as_send"] = copy_us
    cpu = None
    if not args.no_cpu_baseline:
        v, dt, elems = oracle_sample(cores, 2)
        cpu = {"value": v, "unit": "GB/s", "cores": cores, "kind": "oracle",
               "sample": "%d buckets of 25M elements (2 per host thread), send + 8-worker reduce, %.1f s wall" % (2 * cores, dt)}
    line = {"metric": METRIC, "value": world * wl.grad_bytes / (step_ms * 1e-3) / 1e9, "unit": "GB/s", "n_gpus": world,
            "steps": K, "warmup": max(3, args.warmup), "ms_per_step": step_ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu,
            "kernels": kernels}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
