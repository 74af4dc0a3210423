"""Two CPU ranks (gloo) walk the multi-worker path of Sec. 3.3: every rank compresses its own gradient into the
partitioned communication buffer, the parts are exchanged with one all-to-all (rank r keeps part r of every
worker), and every rank averages the parts it received.  The buffers are produced and reduced by the oracle; the
sizes, strides and part boundaries come from the CUDA library's host-side layout functions, which need no GPU.
The gathered result must equal the one-process reduction over both workers' whole buffers."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import loco_oracle as orc
from paper_2407_04480_b200 import build as loco_build
from paper_2407_04480_b200 import inputs, loco

WORLD = 2
N_ELEMS = 100_003
KW = dict(bits=4, s=2.0 ** 12, s_e=2.0 ** 14, beta=0.5, reset_period=0, state_fmt=0, grad_dtype=1, out_dtype=0,
          num_partitions=WORLD)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker_buffers(rank, steps=2):
    ocfg = orc.OracleConfig(**KW)
    state, comm = orc.new_state(ocfg, N_ELEMS), orc.new_comm(ocfg, N_ELEMS)
    for k in range(steps):
        g = inputs.gaussian(N_ELEMS, 1e-3, seed=77, worker=rank, step=k, dtype=torch.bfloat16)
        orc.send_step(ocfg, inputs.as_numpy_bits(g), state, comm, k + 1)
    return ocfg, comm


def _rank_main(rank, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=WORLD)
    try:
        gcfg = loco.Config(**KW)
        ocfg, comm = _worker_buffers(rank)
        stride = loco.loco_partition_bytes(gcfg, N_ELEMS)
        assert comm.size == loco.loco_packed_bytes(gcfg, N_ELEMS) == WORLD * stride
        # all-to-all: part j of this worker goes to rank j; part `rank` of every worker arrives here
        send = torch.from_numpy(comm.copy())
        recv = torch.empty_like(send)
        dist.all_to_all_single(recv, send, [stride] * WORLD, [stride] * WORLD)
        received = recv.numpy()
        # what arrived from worker w is its part `rank`; rebuild, per worker, a buffer that holds that part in place
        per_worker = []
        for w in range(WORLD):
            buf = np.zeros(WORLD * stride, dtype=np.uint8)
            buf[rank * stride:(rank + 1) * stride] = received[w * stride:(w + 1) * stride]
            per_worker.append(buf)
        mine = orc.reduce(ocfg, N_ELEMS, per_worker, first=rank, count=1)
        assert mine.size == loco.loco_partition_elems(gcfg, N_ELEMS, rank)
        np.save(os.path.join(out_dir, "part%d.npy" % rank), mine)
        # the timing rule of the benchmark: the job's step time is the slowest rank's
        t = torch.tensor([float(rank + 1)], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert float(t.item()) == float(WORLD)
    finally:
        dist.destroy_process_group()


def test_two_ranks_all_to_all_then_reduce(tmp_path):
    loco_build.build()
    orc.lib()
    mp.spawn(_rank_main, args=(_free_port(), str(tmp_path)), nprocs=WORLD, join=True)
    parts = [np.load(os.path.join(str(tmp_path), "part%d.npy" % r)) for r in range(WORLD)]
    ocfg = orc.OracleConfig(**KW)
    whole = orc.reduce(ocfg, N_ELEMS, [_worker_buffers(r)[1] for r in range(WORLD)])
    got = np.concatenate(parts)
    assert got.size == N_ELEMS
    assert np.array_equal(got.view(np.uint32), whole.view(np.uint32))
    assert np.abs(whole).max() > 0


def test_rank_parts_tile_the_bucket():
    """Part boundaries are the same on every rank and cover the bucket exactly once, for even and ragged sizes."""
    loco_build.build()
    for n in (1, 255, 256, 1000, 100_003, 25_000_000):
        for P in (2, 4, 8):
            cfg = loco.Config(**{**KW, "num_partitions": P})
            lp = loco.loco_partition_capacity(cfg, n)
            elems = [loco.loco_partition_elems(cfg, n, j) for j in range(P)]
            assert sum(elems) == n and all(0 <= e <= lp for e in elems)
            # parts are filled in order: once one is short, the rest are empty
            short = [j for j in range(P) if elems[j] < lp]
            assert all(elems[j] == 0 for j in short[1:])
            assert loco.loco_partition_bytes(cfg, n) % 128 == 0
