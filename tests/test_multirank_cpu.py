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


# ---- the peer-store transport's host logic: slots, destination tables, the two alternating areas ----------------

STEPS = 4


def _peer_store_rank(rank, port, out_dir, arena):
    """arena: one shared host tensor standing in for the ranks' symmetric memory; the 'address' of rank j's area a
    is its offset in the arena.  The oracle produces and reduces the buffers; a byte copy stands in for the send
    kernel's stores; the group's barrier stands in for the ordering collective.  There is deliberately no second
    barrier per step: the alternation of the two areas has to make that safe."""
    from paper_2407_04480_b200 import exchange
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=WORLD)
    try:
        gcfg = loco.Config(**KW)
        ocfg = orc.OracleConfig(**KW)
        stride = loco.loco_partition_bytes(gcfg, N_ELEMS)
        abytes = exchange.area_bytes(gcfg, N_ELEMS)
        assert abytes == WORLD * stride
        area_addr = [[(a * WORLD + j) * abytes for j in range(WORLD)] for a in range(2)]     # [area][rank]
        tables = [exchange.scatter_table(area_addr[a], gcfg, N_ELEMS, rank) for a in range(2)]
        mem = arena.numpy()
        state, comm = orc.new_state(ocfg, N_ELEMS), orc.new_comm(ocfg, N_ELEMS)
        for k in range(STEPS):
            g = inputs.gaussian(N_ELEMS, 1e-3, seed=77, worker=rank, step=k, dtype=torch.bfloat16)
            orc.send_step(ocfg, inputs.as_numpy_bits(g), state, comm, k)
            a = exchange.area_index(k)
            for j in range(WORLD):                                   # the scattering stores
                mem[tables[a][j]:tables[a][j] + stride] = comm[j * stride:(j + 1) * stride]
            dist.barrier()                                           # everybody has stored
            if rank == 1 and k % 2 == 0:
                import time
                time.sleep(0.3)                                      # a slow reader: the other rank runs ahead
            mine = area_addr[a][rank]
            slots = []
            for w in range(WORLD):
                buf = np.zeros(WORLD * stride, dtype=np.uint8)
                off = mine + exchange.slot_offset(gcfg, N_ELEMS, w)
                buf[rank * stride:(rank + 1) * stride] = mem[off:off + stride]
                slots.append(buf)
            out = orc.reduce(ocfg, N_ELEMS, slots, first=rank, count=1)
            assert out.size == exchange.shard_elems(gcfg, N_ELEMS, rank)
            np.save(os.path.join(out_dir, "ps_step%d_part%d.npy" % (k, rank)), out)
    finally:
        dist.destroy_process_group()


def test_two_ranks_peer_store_slots_and_alternating_areas(tmp_path):
    from paper_2407_04480_b200 import exchange
    loco_build.build()
    orc.lib()
    gcfg = loco.Config(**KW)
    arena = torch.zeros(2 * WORLD * exchange.area_bytes(gcfg, N_ELEMS), dtype=torch.uint8).share_memory_()
    mp.spawn(_peer_store_rank, args=(_free_port(), str(tmp_path), arena), nprocs=WORLD, join=True)
    # one process, both workers, whole buffers
    ocfg = orc.OracleConfig(**KW)
    states = [orc.new_state(ocfg, N_ELEMS) for _ in range(WORLD)]
    comms = [orc.new_comm(ocfg, N_ELEMS) for _ in range(WORLD)]
    for k in range(STEPS):
        for r in range(WORLD):
            g = inputs.gaussian(N_ELEMS, 1e-3, seed=77, worker=r, step=k, dtype=torch.bfloat16)
            orc.send_step(ocfg, inputs.as_numpy_bits(g), states[r], comms[r], k)
        whole = orc.reduce(ocfg, N_ELEMS, comms)
        got = np.concatenate([np.load(os.path.join(str(tmp_path), "ps_step%d_part%d.npy" % (k, r))) for r in range(WORLD)])
        assert np.array_equal(got.view(np.uint32), whole.view(np.uint32)), "step %d" % k


def test_exchange_host_helpers():
    from paper_2407_04480_b200 import exchange
    loco_build.build()
    cfg = loco.Config(**{**KW, "num_partitions": 8})
    n = 25_000_000
    part = loco.loco_partition_bytes(cfg, n)
    assert exchange.area_bytes(cfg, n) == 8 * part
    assert [exchange.slot_offset(cfg, n, r) for r in range(8)] == [r * part for r in range(8)]
    with pytest.raises(ValueError):
        exchange.slot_offset(cfg, n, 8)
    bases = [1 << 40, 2 << 40, 3 << 40, 4 << 40, 5 << 40, 6 << 40, 7 << 40, 8 << 40]
    assert exchange.scatter_table(bases, cfg, n, 3) == [b + 3 * part for b in bases]
    with pytest.raises(ValueError):
        exchange.scatter_table(bases[:7], cfg, n, 0)
    assert [exchange.area_index(k) for k in range(5)] == [0, 1, 0, 1, 0]
    assert sum(exchange.shard_elems(cfg, n, r) for r in range(8)) == n
    with pytest.raises(RuntimeError):
        exchange.BucketExchange(cfg, n)          # no process group: refuses, does not fall back to anything
