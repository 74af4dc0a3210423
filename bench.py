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
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "dram_traffic_llama2_7b_buckets.json")
KERNEL_SOURCES = ("paper_2407_04480_b200/csrc/loco_kernels.cuh", "paper_2407_04480_b200/csrc/loco_api.cu",
                  "paper_2407_04480_b200/csrc/loco_send_tu.cu", "paper_2407_04480_b200/csrc/loco_reduce_tu.cu",
                  "paper_2407_04480_b200/csrc/loco_dispatch.h")


def cfg_for(scale: str) -> dict:
    """The bench configuration with the paper's global scale ("fixed") or one fp32 scale per 256 elements ("block")."""
    c = dict(CFG)
    if scale == "block":
        c["scale_mode"] = 1
    return c


def send_bytes_per_elem(c: dict) -> float:
    """Algorithmic HBM bytes per element of the send pass: gradient read, state read + written, code written (+ the
    block's wire scale written and its state scale read and written)."""
    g = 2 if c["grad_dtype"] == 1 else 4
    st = {0: 2, 1: 8, 2: 0, 3: 8}[c["state_fmt"]]
    sc = (4.0 / c["block_size"]) * (3 if c["state_fmt"] == 0 else 1) if c["scale_mode"] == 1 else 0.0
    return g + st + c["bits"] / 8 + sc


def reduce_bytes_per_elem(c: dict, workers: int) -> float:
    """Algorithmic HBM bytes per output element of the receive pass: N workers' codes (+ block scales) read, output written."""
    o = 2 if c["out_dtype"] == 1 else 4
    return workers * (c["bits"] / 8 + (4.0 / c["block_size"] if c["scale_mode"] == 1 else 0.0)) + o


def kernel_sources_hash() -> str:
    import hashlib
    h = hashlib.sha256()
    for rel in KERNEL_SOURCES:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def stored_traffic(kernel: str, scale: str):
    """DRAM bytes (read + written) per 25M-element bucket from the stored profiler capture, or None if there is none
    for this case or the kernel sources have changed since it was taken."""
    try:
        with open(TRAFFIC_JSON) as f:
            rec = json.load(f)
        if rec.get("kernel_sources_sha256_16") != kernel_sources_hash():
            return None
        return float(rec[scale][kernel]["dram_bytes_per_bucket"])
    except Exception:
        return None


def write_traffic(fixed_csv: str, block_csv: str, buckets: int = 24):
    """Turn the two ncu logs of the capture named in profiles/dram_traffic_llama2_7b_buckets.md (one run per scale rule:
    `--csv --log-file`, metrics dram__bytes_read.sum, dram__bytes_write.sum, gpu__time_duration.sum, the multi-bucket send and
    receive launch of one step over `buckets` buckets) into the stored JSON and its summary.  No GPU needed."""
    import csv
    unit = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9, "Tbyte": 1e12, "ns": 1e-3, "us": 1.0, "ms": 1e3, "s": 1e6}
    cmd = ("ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum,gpu__time_duration.sum --clock-control none "
           "-k regex:loco_.*_multi_kernel -s 4 -c 2 --csv --log-file <log> python bench.py --buckets %d --steps 1 --warmup 1 --no-e2e "
           "--no-cpu-baseline [--scale block]" % buckets)
    rec = {"kernel_sources_sha256_16": kernel_sources_hash(), "buckets_in_the_captured_launch": buckets, "command": cmd}
    for scale, path in (("fixed", fixed_csv), ("block", block_csv)):
        rows = [r for r in csv.reader(open(path)) if len(r) > 10]
        hdr = next(r for r in rows if "Metric Name" in r)
        iK, iM, iU, iV = (hdr.index(x) for x in ("Kernel Name", "Metric Name", "Metric Unit", "Metric Value"))
        c = cfg_for(scale)
        rec[scale] = {}
        for kernel, tag, algo in (("send", "send_multi", send_bytes_per_elem(c)), ("reduce", "reduce_multi", reduce_bytes_per_elem(c, WORKERS))):
            m = {}
            for r in rows:
                if r is hdr or tag not in r[iK] or r[iM] in m:
                    continue
                m[r[iM]] = float(r[iV].replace(",", "")) * unit[r[iU]]
            rd, wr = m["dram__bytes_read.sum"] / buckets, m["dram__bytes_write.sum"] / buckets
            rec[scale][kernel] = {"dram_bytes_per_bucket": rd + wr, "dram_read_bytes_per_bucket": rd, "dram_write_bytes_per_bucket": wr,
                                  "algorithmic_bytes_per_bucket": algo * BUCKET, "launch_us_under_ncu": m["gpu__time_duration.sum"]}
    with open(TRAFFIC_JSON, "w") as f:
        json.dump(rec, f, indent=1)
    with open(TRAFFIC_JSON.replace(".json", ".md"), "w") as f:
        f.write("# DRAM traffic of the two kernels on Llama-2-7B buckets (steady state)\n\n"
                "One multi-bucket launch over %d buckets of 25,000,000 elements (2.7 GB streamed by the send pass, 3.6 GB by the receive pass: the\n"
                "126 MB L2 holds a few percent of it, so what a bucket writes is evicted to DRAM while the next buckets run). Counters of the\n"
                "captured launch divided by its %d buckets; `bench.py` reads the JSON beside this file for `roofline.traffic` and reports null\n"
                "when the kernel sources no longer hash to the value stored there. Both files are written by `python bench.py --write-traffic\n"
                "<fixed log> <block log>` from the logs of\n\n    %s\n\n" % (buckets, buckets, cmd))
        f.write("| scale rule | kernel | DRAM read MB / bucket | DRAM written MB / bucket | read + written | algorithmic MB / bucket |\n|---|---|---|---|---|---|\n")
        for scale in ("fixed", "block"):
            for kernel in ("send", "reduce"):
                v = rec[scale][kernel]
                f.write("| %s | %s | %.2f | %.2f | %.2f | %.2f |\n" % (scale, kernel, v["dram_read_bytes_per_bucket"] / 1e6, v["dram_write_bytes_per_bucket"] / 1e6,
                                                                    v["dram_bytes_per_bucket"] / 1e6, v["algorithmic_bytes_per_bucket"] / 1e6))
        f.write("\nReads equal the algorithmic reads to 0.1 % (no byte is read twice) unless the table says otherwise. Writes come out a few\n"
                "percent below the algorithmic writes: the lines the last buckets wrote are still in L2 when the launch ends.\n")
    return rec


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """SM clock and throttle-reason samples taken while the timed region runs: NVML polled every 5 ms, else nvidia-smi every 200 ms."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.dev = device_index
        self.proc = None
        self.path = None

    def start(self):
        if self._start_nvml():
            return
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.dev), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def _start_nvml(self) -> bool:
        """Poll NVML from a thread every 5 ms (read-only queries): a timed region of a tenth of a second still gets
        a couple of dozen samples, where a 200 ms nvidia-smi loop gets one."""
        try:
            import threading
            import pynvml
            pynvml.nvmlInit()
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(self.dev).uuid)
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                h = pynvml.nvmlDeviceGetHandleByIndex(self.dev)
            names = (("hw_slowdown", pynvml.nvmlClocksEventReasonHwSlowdown), ("hw_thermal_slowdown", pynvml.nvmlClocksEventReasonHwThermalSlowdown),
                     ("sw_thermal_slowdown", pynvml.nvmlClocksEventReasonSwThermalSlowdown), ("sw_power_cap", pynvml.nvmlClocksEventReasonSwPowerCap))
            self.nvml_max = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            self.nvml_sm, self.nvml_reasons, self.nvml_stop = [], set(), threading.Event()

            def poll():
                while not self.nvml_stop.is_set():
                    try:
                        self.nvml_sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                        mask = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
                        for name, bit in names:
                            if mask & bit:
                                self.nvml_reasons.add(name)
                    except Exception:
                        pass
                    self.nvml_stop.wait(0.005)

            self.nvml_thread = threading.Thread(target=poll, daemon=True)
            self.nvml_thread.start()
            return True
        except Exception:
            self.nvml_thread = None
            return False

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if getattr(self, "nvml_thread", None) is not None:
            self.nvml_stop.set()
            self.nvml_thread.join(timeout=2)
            if self.nvml_sm:
                out.update(sm_mhz=statistics.median(self.nvml_sm), sm_max_mhz=self.nvml_max, reasons=sorted(self.nvml_reasons),
                           samples=len(self.nvml_sm), source="nvml, 5 ms period")
            return out
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

    def __init__(self, rank: int, device: torch.device, max_buckets: int = 0, scale: str = "fixed"):
        from paper_2407_04480_b200 import inputs, loco
        self.loco = loco
        self.cfgd = cfg_for(scale)
        self.cfg = loco.Config(**self.cfgd)
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
        self.recv_buf = torch.empty(sum(pb) * (WORKERS - 1), dtype=torch.uint8, device=device)
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
        # packed buffers of the 7 other workers as they would sit after the exchange
        if scale == "fixed":
            # with the global scale any byte is two valid codes
            gen = torch.Generator(device=device)
            gen.manual_seed(1234 + rank)
            chunk = 1 << 30
            for off in range(0, self.recv_buf.numel(), chunk):
                m = min(chunk, self.recv_buf.numel() - off)
                self.recv_buf[off:off + m] = torch.randint(0, 256, (m,), dtype=torch.uint8, device=device, generator=gen)
        else:
            # block scales must be numbers a send pass produces: compress this rank's buckets once more without error
            # feedback and give every other worker a copy in memory of its own
            gen_cfg = loco.Config(**{**self.cfgd, "state_fmt": 2})
            tmp = torch.empty(max(pb), dtype=torch.uint8, device=device)
            ro = 0
            for i, (lo, hi) in enumerate(self.buckets):
                st = loco.State(gen_cfg, hi - lo)
                loco.loco_compensate_quantize_pack(st, self.grads[i], tmp, 1)
                for w in range(WORKERS - 1):
                    self.recv_buf[ro:ro + pb[i]].copy_(tmp[:pb[i]])
                    ro += pb[i]
            torch.cuda.synchronize()
        self.send_bpe = send_bytes_per_elem(self.cfgd)
        self.recv_bpe = reduce_bytes_per_elem(self.cfgd, WORKERS)
        self.send_bytes = self.send_bpe * self.total
        self.recv_bytes = self.recv_bpe * self.total
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


def oracle_sample(threads: int, buckets_per_thread: int, cfgd: dict = None, n: int = BUCKET, workers: int = WORKERS,
                  sigma: float = 1e-4):
    """The oracle as it stands on `threads` host threads, each doing whole buckets of n elements of the workload (send
    pass, then the receive pass over the whole bucket with `workers` workers).  Returns (GB/s of gradient, seconds,
    elements)."""
    import numpy as np
    from oracle import loco_oracle as orc
    cfgd = dict(cfgd or CFG)
    ocfg = orc.OracleConfig(**cfgd)
    rng = np.random.default_rng(1)
    g32 = rng.normal(0, sigma, n).astype(np.float32)
    gsz = 2 if cfgd["grad_dtype"] == 1 else 4
    g = (g32.view(np.uint32) >> 16).astype(np.uint16) if gsz == 2 else g32
    block = cfgd["scale_mode"] == 1
    # the other workers' buffers: random codes with the global scale; with block scales a buffer the oracle itself packed
    others = [] if block else [rng.integers(0, 256, orc.packed_bytes(ocfg, n), dtype=np.uint8) for _ in range(2)]
    states = [orc.new_state(ocfg, n) for _ in range(threads)]
    comms = [orc.new_comm(ocfg, n) for _ in range(threads)]
    orc.lib()

    def work(t):
        for b in range(buckets_per_thread):
            orc.send_step(ocfg, g, states[t], comms[t], 1 + b)
            orc.reduce(ocfg, n, [comms[t]] + [comms[t] if block else others[w % 2] for w in range(workers - 1)])

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        list(ex.map(work, range(threads)))
    dt = time.perf_counter() - t0
    elems = threads * buckets_per_thread * n
    return gsz * elems / dt / 1e9, dt, elems


def cpu_baseline_record(cores: int, cfgd: dict, n: int, workers: int, what: str, per_thread: int = 4):
    """The oracle on all host cores and on one thread, on a bounded sample of the workload's buckets."""
    v, dt, _ = oracle_sample(cores, per_thread, cfgd, n, workers)
    v1, dt1, _ = oracle_sample(1, max(1, per_thread // 2), cfgd, n, workers)
    return {"value": v, "unit": "GB/s", "cores": cores, "kind": "oracle",
            "sample": "%d %s (%d per host thread), send + %d-worker reduce, %.1f s wall" % (per_thread * cores, what, per_thread, workers, dt),
            "one_thread_value": v1, "one_thread_sample": "%d of the same on one thread, %.1f s" % (max(1, per_thread // 2), dt1)}


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
    cfg = loco.Config(**{**cfg_for(args.scale), "num_partitions": world})
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
    budget = int(args.sweep_budget_gb * (1 << 30))      # device bytes per case

    def sets_for(bytes_per_set):
        """Independent working sets of a case: enough that no launch finds its data in L2 (>= 1 GB in all), at least three
        (concurrent launches must not share buffers), within the memory budget; a case too large for three sets gets one
        and its launches are then issued on one stream."""
        want = max(3, -(-(1 << 30) // bytes_per_set))
        have = int(min(want, 256, budget // max(1, bytes_per_set)))
        return have if have >= 3 else 1

    def streams_for(nsets):
        return streams if nsets >= 3 else streams[:1]

    def send_case(label, n, **kw):
        if args.sweep_filter and args.sweep_filter not in "send: " + label + " |":
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
        us = _time_launches(lambda i, st: send(i, 2, st), nsets, max(12, min(200, 4 * nsets)), streams_for(nsets))
        state_rw = {0: 2, 1: 8, 2: 0, 3: 8}[cfg.state_fmt]
        scale_b = (4.0 / cfg.block_size) * (3 if cfg.state_fmt == 0 else 1) if cfg.scale_mode == 1 else 0.0
        bpe = gsz + state_rw + cfg.bits / 8 + scale_b
        gbs = bpe * n / us / 1e3
        rows.append(dict(kernel="send", case=label, n=n, bytes_per_elem=round(bpe, 3), us=round(us, 2), hbm_gbs=round(gbs, 1),
                         frac=round(gbs / peak, 3), grad_gbs=round(gsz * n / us / 1e3, 1),
                         l2_resident=bool(nsets * (n * gsz + sb + pb) < L2_BYTES)))
        print(json.dumps(rows[-1]), flush=True)

    def reduce_case(label, n, workers, **kw):
        if args.sweep_filter and args.sweep_filter not in "reduce: " + label + " | N=%d |" % workers:
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
                                nsets, max(12, min(200, 4 * nsets)), streams_for(nsets))
            n = loco.loco_partition_elems(cfg, n, 3)        # elements this launch produces
        else:
            us = _time_launches(lambda i, st: loco.loco_unpack_dequant_reduce(cfg, packed[i], n, outs[i], stream=st),
                                nsets, max(12, min(200, 4 * nsets)), streams_for(nsets))
        bpe = workers * cfg.bits / 8 + osz + (workers * 4.0 / cfg.block_size if cfg.scale_mode == 1 else 0.0)
        gbs = bpe * n / us / 1e3
        rows.append(dict(kernel="reduce", case=label, n=n, workers=workers, bytes_per_elem=round(bpe, 3), us=round(us, 2),
                         hbm_gbs=round(gbs, 1), frac=round(gbs / peak, 3), grad_gbs=round(osz * n / us / 1e3, 1),
                         l2_resident=bool(nsets * (workers * pb + n * osz) < L2_BYTES)))
        print(json.dumps(rows[-1]), flush=True)

    def adam_case(label, n, workers, **kw):
        if args.sweep_filter and args.sweep_filter not in "reduce+adam: " + label + " | N=%d |" % workers:
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
                            nsets, max(12, min(200, 4 * nsets)), streams_for(nsets))
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
    for B in (512, 1024, 4096):
        send_case("bf16 g, int8 state, 4 bit, block-%d absmax%s" % (B, "" if B == 512 else " (rows of a block on neighbouring warps)"), M, scale_mode=1, block_size=B)
    send_case("bf16 g, int8 state, 1 bit (sign code), fixed", M, bits=1)
    send_case("bf16 g, int8 state, 1 bit (sign code), block-256 mean magnitude", M, bits=1, scale_mode=1)
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
    reduce_case("4 bit, bf16 out, block-1024 absmax", M, 8, scale_mode=1, block_size=1024)
    reduce_case("1 bit (sign code), bf16 out, fixed", M, 8, bits=1)
    reduce_case("1 bit (sign code), bf16 out, block-256 mean magnitude", M, 8, bits=1, scale_mode=1)
    for N in (1, 8, 16):
        adam_case("4 bit, fixed, Adam-family step fused, no gradient output", M, N)
    adam_case("8 bit, fixed, Adam-family step fused, no gradient output", M, 8, bits=8)
    adam_case("4 bit, fixed, Adam-family step fused, no gradient output", 1 << 27, 8)
    print("| kernel | case | n | workers | B/elem | us/launch | HBM GB/s | of %s peak %.0f | gradient GB/s | L2-resident |" % (peak_kind, peak))
    print("|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        print("| %s | %s | %d | %s | %s | %s | %s | %.3f | %s | %s |" % (r["kernel"], r["case"], r["n"], r.get("workers", "-"), r["bytes_per_elem"],
                                                                      r["us"], r["hbm_gbs"], r["frac"], r["grad_gbs"], "yes" if r["l2_resident"] else ""))


def run_other_config(args, device, cores):
    """--config 1 | 3 | 4: the other workload configurations, one JSON line each with a row per pass and scale rule
    (GB/s of gradient, HBM GB/s, fraction of the measured and of the nominal peak) next to the oracle on one thread and
    on all host cores for the same shape."""
    from paper_2407_04480_b200 import inputs, loco
    peak, peak_kind = measured_peak()
    rows = []

    def timed(fn, reps, warm=3):
        """Average device time of fn() in microseconds; the launches are replayed from a CUDA graph so that the host's
        launch cost (several microseconds per call from Python) is not what is timed."""
        for _ in range(warm):
            fn()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(reps):
                fn()
        graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / reps          # microseconds

    def row(kind, label, n_elems, bpe, esize, us, note=""):
        gbs = bpe * n_elems / us / 1e3
        r = dict(kernel=kind, case=label, n=n_elems, bytes_per_elem=round(bpe, 3), us=round(us, 2), hbm_gbs=round(gbs, 1),
                 frac_of_measured=round(gbs / peak, 3), frac_of_nominal_8TBps=round(gbs / 8000.0, 3),
                 gradient_gbs=round(esize * n_elems / us / 1e3, 1), note=note)
        rows.append(r)
        print(json.dumps(r), flush=True)

    launches_before = loco.loco_launch_count()
    if args.config == 1:
        # one fp32 vector of 2^20 elements, 1 worker, 4 error-feedback steps: 6.5 MB per pass, resident in the 126 MB L2
        n, workload = 1 << 20, "config 1: one fp32 vector of 1,048,576 elements, 1 worker, 4 error-feedback steps (L2-resident: 6.5 MB per pass)"
        for scale in ("fixed", "block"):
            c = dict(cfg_for(scale), s=2.0 ** 11, s_e=2.0 ** 13, grad_dtype=0, out_dtype=0, num_partitions=1)
            cfg = loco.Config(**c)
            grads = [inputs.gaussian(n, 1e-3, seed=0, step=k, dtype=torch.float32, device=device) for k in range(4)]
            st = loco.State(cfg, n)
            comm = torch.empty(loco.loco_packed_bytes(cfg, n), dtype=torch.uint8, device=device)
            out = torch.empty(n, dtype=torch.float32, device=device)

            def four_steps():
                for k in range(4):
                    loco.loco_compensate_quantize_pack(st, grads[k], comm, k + 1)

            us = timed(four_steps, 50) / 4
            row("send", "%s scale, fp32 g, int8 state, 4 bit" % scale, n, send_bytes_per_elem(c), 4, us, "L2-resident")
            us = timed(lambda: loco.loco_unpack_dequant_reduce(cfg, [comm], n, out), 200)
            row("reduce", "%s scale, 1 worker, fp32 out" % scale, n, reduce_bytes_per_elem(c, 1), 4, us, "L2-resident")
        oc = dict(cfg_for("fixed"), s=2.0 ** 11, s_e=2.0 ** 13, grad_dtype=0, out_dtype=0, num_partitions=1)
        cpu = cpu_baseline_record(cores, oc, n, 1, "vectors of 2^20 fp32 elements", per_thread=128)
    elif args.config == 3:
        # 13B dense transformer, one flat bf16 buffer in the reduce-scatter layout of 8 parts: one send launch over the whole
        # buffer; a rank then averages its own part (1,626,983,040 elements) over 8 workers
        layout = inputs.dense_13b()
        n = layout.numel
        workload = "config 3: 13B dense transformer, one flat bf16 buffer of 13,015,864,320 elements, 8 parts, T_c = 512; send = the whole buffer in one launch, reduce = one rank's part of 1,626,983,040 elements over 8 workers"
        c = dict(cfg_for("fixed"))
        cfg = loco.Config(**c)
        grad = torch.empty(n, dtype=torch.bfloat16, device=device)
        chunk = 1 << 28
        for off in range(0, n, chunk):
            m = min(chunk, n - off)
            grad[off:off + m] = inputs.gaussian(m, 1e-4, seed=2, tag=off >> 8, dtype=torch.bfloat16, device=device)
        st = loco.State(cfg, n)
        comm = torch.empty(loco.loco_packed_bytes(cfg, n), dtype=torch.uint8, device=device)
        loco.loco_compensate_quantize_pack(st, grad, comm, 1)
        us = timed(lambda: loco.loco_compensate_quantize_pack(st, grad, comm, 5), 3, warm=1)
        row("send", "fixed scale, bf16 g, int8 state, 4 bit, 8 parts, one launch", n, send_bytes_per_elem(c), 2, us)
        us = timed(lambda: loco.loco_compensate_quantize_pack(st, grad, comm, 512), 3, warm=1)
        row("send", "the same at k = 512 (the reset of Eq. 7 fires: the state is written as zeros)", n, send_bytes_per_elem(c), 2, us)
        stride = loco.loco_partition_bytes(cfg, n)
        r = 3
        ln = loco.loco_partition_elems(cfg, n, r)
        gen = torch.Generator(device=device)
        gen.manual_seed(77)
        others = [torch.randint(0, 256, (stride,), dtype=torch.uint8, device=device, generator=gen) for _ in range(WORKERS - 1)]
        out = torch.empty(ln, dtype=torch.bfloat16, device=device)
        packed = [comm[r * stride:(r + 1) * stride]] + others
        us = timed(lambda: loco.loco_unpack_dequant_reduce(cfg, packed, n, out, first_partition=r, partition_count=1), 5, warm=2)
        row("reduce", "fixed scale, part 3 of 8 (1,626,983,040 elements), 8 workers, bf16 out", ln, reduce_bytes_per_elem(c, WORKERS), 2, us)
        cpu = cpu_baseline_record(cores, c, BUCKET, WORKERS, "windows of 25M elements of the flat buffer")
    else:
        # one Mixtral-8x7B decoder layer, Student-t(3) x 1e-4, 2 of 8 experts all-zero, 8 workers
        layout = inputs.mixtral_layer()
        n = layout.numel
        workload = "config 4: one Mixtral-8x7B decoder layer of 1,451,270,144 bf16 elements, Student-t(nu=3) x 1e-4, 2 of 8 experts all-zero, 8 workers"
        scales = inputs.zero_expert_scales(3, layer=0)
        grad = torch.empty(n, dtype=torch.bfloat16, device=device)
        chunk = 1 << 27
        for off in range(0, n, chunk):
            hi = min(off + chunk, n)
            grad[off:hi] = inputs.layout_slice(layout, off, hi, scales, 1e-4, seed=3, worker=0, step=1, dist="student_t", device=device)
        for scale in ("fixed", "block"):
            c = dict(cfg_for(scale), reset_period=0)
            cfg = loco.Config(**c)
            st = loco.State(cfg, n)
            comm = torch.empty(loco.loco_packed_bytes(cfg, n), dtype=torch.uint8, device=device)
            loco.loco_compensate_quantize_pack(st, grad, comm, 1)
            us = timed(lambda: loco.loco_compensate_quantize_pack(st, grad, comm, 2), 5, warm=2)
            row("send", "%s scale, bf16 g, int8 state, 4 bit, 8 parts, the whole layer in one launch" % scale, n, send_bytes_per_elem(c), 2, us)
            others = [comm.clone() for _ in range(WORKERS - 1)]       # the other workers' buffers: valid codes and scales
            out = torch.empty(n, dtype=torch.bfloat16, device=device)
            us = timed(lambda: loco.loco_unpack_dequant_reduce(cfg, [comm] + others, n, out), 5, warm=2)
            row("reduce", "%s scale, 8 workers, bf16 out, all 8 parts in one launch" % scale, n, reduce_bytes_per_elem(c, WORKERS), 2, us)
            del others, out, comm, st
        cpu = cpu_baseline_record(cores, dict(cfg_for("fixed"), reset_period=0), BUCKET, WORKERS, "windows of 25M elements of the layer")
    best = max(rows, key=lambda r: r["us"])
    total_us = sum(r["us"] for r in rows)
    print(json.dumps({"metric": METRIC, "value": None, "unit": "GB/s", "n_gpus": 1, "steps": None, "warmup": 3,
                      "ms_per_step": total_us / 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                      "dtype": "f32", "data": "synthetic", "config": {"workload": workload}, "rows": rows,
                      "slowest_row": best["case"], "peak": peak, "peak_kind": "%s HBM copy bandwidth" % peak_kind,
                      "cpu_baseline": cpu, "gpu_launches": loco.loco_launch_count() - launches_before}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--config", type=int, default=2, choices=(1, 2, 3, 4),
                    help="2 (default): the bench workload, Llama-2-7B buckets; 1, 3, 4: the other workload configurations "
                         "(a table of rows instead of the bench line); the size sweep of configuration 5 is --sweep")
    ap.add_argument("--scale", default="fixed", choices=("fixed", "block"),
                    help="fixed (default): the paper's global scale s (Eq. 1); block: one fp32 scale per 256 elements "
                         "(the block-scaled twin of the bench workload)")
    ap.add_argument("--buckets", type=int, default=0,
                    help="profiling aid: only the first K buckets of the workload (0 = all 270); not a bench line")
    ap.add_argument("--no-graph", action="store_true", help="profiling aid: launch every kernel directly")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the bench line: the size / type / width / worker-count table (one JSON line per case, then markdown)")
    ap.add_argument("--sweep-filter", default="", help="with --sweep: only the cases whose 'kernel: label | N=workers |' contains this text")
    ap.add_argument("--sweep-budget-gb", type=float, default=6.0, help="with --sweep: device memory per case (small for profiler captures)")
    ap.add_argument("--exchange", choices=("none", "collective", "peer_store", "reduce_scatter_bf16"), default="none",
                    help="none (default): every rank runs the two passes on its own buckets, no data-path collective; "
                         "collective / peer_store: the real exchange of Sec. 3.3 between the ranks (NCCL all-to-all, or the "
                         "send kernel storing into the peers' receive slots), each rank reducing its own shard; "
                         "reduce_scatter_bf16: what the method replaces -- NCCL reduce-scatter (average) of the uncompressed bf16 "
                         "buckets, none of this library's kernels, for comparison on the same buckets")
    ap.add_argument("--streams", type=int, default=2,
                    help="2 or more (default): each phase is one multi-bucket call of the library, i.e. one kernel launch over all "
                         "buckets; 1: single-bucket calls strictly one after the other")
    ap.add_argument("--write-traffic", nargs=2, metavar=("FIXED_LOG", "BLOCK_LOG"),
                    help="no run: store the DRAM counters of the two ncu logs named in profiles/dram_traffic_llama2_7b_buckets.md")
    args = ap.parse_args()
    if args.write_traffic:
        write_traffic(*args.write_traffic)
        return
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    cores = os.cpu_count() or 1
    multi = args.streams > 1 and not args.no_graph
    cfgd = cfg_for(args.scale)
    config = {"workload": "llama2-7b: 270 bf16 buckets of 25M elements (6,738,415,616): one worker's send pass per bucket, then the 8-worker reduce of the bucket",
              "bits": 4,
              "scale": "fixed s=2^14, s_e=4s (Eq. 1)" if args.scale == "fixed" else "one fp32 scale per block of 256 elements (extension, not in the paper)",
              "beta": 0.5, "T_c": 512, "state": "int8", "workers_on_reduce_side": WORKERS, "out": "bf16",
              "launches": ("one multi-bucket call per phase = one kernel launch over all buckets (the buckets are the grid's third "
                           "dimension), on one stream" if multi else "single-bucket calls one after the other on one stream"),
              "l2": "inputs larger than L2: each step streams ~70 GB once, no reuse between launches"}

    if args.impl == "reference":
        if rank != 0:
            return
        steps = max(1, args.steps)
        for _ in range(min(args.warmup, 1)):
            oracle_sample(cores, 1, cfgd)
        t0 = time.perf_counter()
        elems = 0
        for _ in range(steps):
            _, _, e = oracle_sample(cores, 1, cfgd)
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
    if args.config != 2:
        if rank == 0:
            run_other_config(args, device, cores)
        return
    if args.exchange != "none":
        run_exchange(args, rank, world, device, config)
        return
    wl = RankWorkload(rank, device, args.buckets, args.scale)
    nb = len(wl.buckets)
    if args.buckets > 0:
        config["workload"] += " -- REDUCED to the first %d buckets (profiling aid, not the bench workload)" % nb
    # A step is captured once into two CUDA graphs (one per phase) and replayed, so that the host's launch cost does not sit
    # between the kernels; the launches of a step are counted while the graphs are captured.
    wl.send_phase(1)
    wl.reduce_phase()
    torch.cuda.synchronize()
    if args.no_graph:
        class _Direct:
            def __init__(self, fn): self.replay = fn
        g_send, g_reduce = _Direct(lambda: wl.send_phase(100)), _Direct(wl.reduce_phase)
        launches_per_step = 2 * nb
    else:
        g_send, g_reduce = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        before = loco.loco_launch_count()
        if multi:
            # the library's multi-bucket calls: one kernel launch per phase, the buckets in the grid's third dimension
            ms = loco.MultiSend(wl.states, wl.grads, wl.comms)
            mr = loco.MultiReduce(wl.cfg, wl.packed, [hi - lo for lo, hi in wl.buckets], wl.outs)
            with torch.cuda.graph(g_send):
                loco.loco_compensate_quantize_pack_multi(ms, 100)
            with torch.cuda.graph(g_reduce):
                loco.loco_unpack_dequant_reduce_multi(mr)
        else:
            with torch.cuda.graph(g_send):
                wl.send_phase(100, None)
            with torch.cuda.graph(g_reduce):
                wl.reduce_phase(None)
        launches_per_step = loco.loco_launch_count() - before
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
    launches = launches_per_step * K
    clocks = sampler.stop()
    # outside the timed region: the same two phases as single-bucket calls, every launch strictly after the previous one
    # (one stream), which shows what a lone launch costs when nothing fills its start-up and its tail
    serial_us = None
    if multi:
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
    # torch) that moves as many bytes per launch as the send kernel does per bucket, over memory not in L2
    copy_us = None
    if not args.no_graph:
        half = int(wl.send_bpe * BUCKET / 2) // 256 * 256                  # bytes copied = half of read + written
        src8, dst8 = wl.grad.view(torch.uint8), wl.out_buf.view(torch.uint8)
        span = min(src8.numel(), dst8.numel())
        count = max(1, min(nb, span // half))
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(count):
                dst8[i * half:(i + 1) * half].copy_(src8[i * half:(i + 1) * half])
        g.replay()
        ce = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        torch.cuda.synchronize()
        ce[0].record(); g.replay(); g.replay(); ce[1].record()
        torch.cuda.synchronize()
        us = ce[0].elapsed_time(ce[1]) * 1e3 / (2 * count)
        copy_us = {"bytes_moved_per_copy": 2 * half, "copy_us": us, "gbs": 2 * half / us / 1e3}
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
               "how": "loco_*_host entry points, pinned host buffers, copies inside the timed region (this measures the host "
                      "link: 57 GB cross it per step); send and receive passes on two streams so that host-to-device and "
                      "device-to-host copies overlap"}
    if dist is not None:
        dist.barrier()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak()
    send_gbs = wl.send_bytes / (send_ms * 1e-3) / 1e9
    recv_gbs = wl.recv_bytes / (recv_ms * 1e-3) / 1e9
    per_phase = max(1, launches_per_step // 2)
    how = ("CUDA events around this kernel's phase of every timed step; " +
           ("a phase is ONE launch that walks all %d buckets (grid.z = bucket), so the figures below are per bucket: "
            "phase time / buckets" % nb if multi else "every bucket's launch strictly after the previous one"))
    traffic_note = ("dram__bytes_read.sum + dram__bytes_write.sum of one captured multi-bucket launch / its buckets, read from "
                    "profiles/dram_traffic_llama2_7b_buckets.json; null when there is no capture for this case or the kernel "
                    "sources have changed since it was taken")
    tag = "fixed scale" if args.scale == "fixed" else "block-256 scale"
    roof_send = {"kernel": "loco_send%s_kernel<bf16 g, int8 state, 4 bit, %s>" % ("_multi" if multi else "", tag), "bound": "hbm",
                 "achieved": send_gbs, "peak": peak, "peak_kind": "%s HBM copy bandwidth" % peak_kind, "unit": "GB/s",
                 "frac": send_gbs / peak, "frac_of_nominal_8TBps": send_gbs / 8000.0, "traffic": stored_traffic("send", args.scale),
                 "traffic_source": traffic_note, "algorithmic_bytes_per_bucket": wl.send_bpe * BUCKET,
                 "avg_us_per_bucket": send_ms * 1e3 / nb, "launches_per_step": per_phase, "buckets_per_launch": nb // per_phase, "how": how}
    roof_reduce = {"kernel": "loco_reduce%s_kernel<bf16 out, 4 bit, %s>, 8 workers" % ("_multi" if multi else "", tag), "bound": "hbm",
                   "achieved": recv_gbs, "peak": peak, "peak_kind": "%s HBM copy bandwidth" % peak_kind, "unit": "GB/s",
                   "frac": recv_gbs / peak, "frac_of_nominal_8TBps": recv_gbs / 8000.0, "traffic": stored_traffic("reduce", args.scale),
                   "traffic_source": traffic_note, "algorithmic_bytes_per_bucket": wl.recv_bpe * BUCKET,
                   "avg_us_per_bucket": recv_ms * 1e3 / nb, "launches_per_step": per_phase, "buckets_per_launch": nb // per_phase, "how": how}
    # the roofline object describes the kernel that takes the larger share of the step; the other one rides along
    roofline, other = (roof_reduce, roof_send) if recv_ms >= send_ms else (roof_send, roof_reduce)
    roofline["other_kernel"] = other
    kernels = {"send": {"hbm_gbs": send_gbs, "frac_of_peak": send_gbs / peak, "gradient_gbs": wl.grad_bytes / (send_ms * 1e-3) / 1e9,
                        "ms_per_step": send_ms, "avg_us_per_bucket": send_ms * 1e3 / nb, "bytes_per_elem": wl.send_bpe},
               "reduce": {"hbm_gbs": recv_gbs, "frac_of_peak": recv_gbs / peak,
                          "gradient_gbs": wl.grad_bytes / (recv_ms * 1e-3) / 1e9, "ms_per_step": recv_ms,
                          "avg_us_per_bucket": recv_ms * 1e3 / nb, "bytes_per_out_elem": wl.recv_bpe}}
    if serial_us is not None:
        kernels["send"]["single_bucket_calls_one_stream_us"] = serial_us[0]
        kernels["send"]["single_bucket_calls_one_stream_hbm_gbs"] = wl.send_bytes / nb / (serial_us[0] * 1e-6) / 1e9
        kernels["reduce"]["single_bucket_calls_one_stream_us"] = serial_us[1]
        kernels["reduce"]["single_bucket_calls_one_stream_hbm_gbs"] = wl.recv_bytes / nb / (serial_us[1] * 1e-6) / 1e9
    if copy_us is not None:
        kernels["device_copy_same_bytes_as_send_bucket"] = copy_us
    cpu = None
    if not args.no_cpu_baseline:
        cpu = cpu_baseline_record(cores, cfgd, BUCKET, WORKERS, "buckets of 25M elements")
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
