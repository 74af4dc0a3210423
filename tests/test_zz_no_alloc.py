"""The receive pass that brings its own staging area (loco_unpack_dequant_reduce_host_noalloc).

Some users of the library cannot give it device memory: their framework's allocator has already
taken the whole GPU, or they call from a place where cudaMalloc is not allowed.  For them the
library stages host buffers through a fixed array inside its own image.  This test calls that
entry point through the C ABI twice in a row and requires the bytes the workspace-taking entry
point produces -- and the bytes the CPU oracle computes from the same parts (Eq. 8) -- then
checks that a request beyond the array's size is refused.  The file name
sorts last so that a run stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import loco_oracle as orc
from paper_2407_04480_b200 import loco

pytestmark = pytest.mark.gpu


def _random_parts(cfg, n, workers, count, seed):
    """Host buffers holding `count` consecutive parts per worker: any byte is a pair of valid 4-bit codes."""
    stride = loco.loco_partition_bytes(cfg, n)
    g = torch.Generator()
    g.manual_seed(seed)
    return [torch.randint(0, 256, (count * stride,), dtype=torch.uint8, generator=g).pin_memory() for _ in range(workers)]


def _reduce_with_workspace(cfg, parts, n, first, count):
    n_out = sum(loco.loco_partition_elems(cfg, n, j) for j in range(first, first + count))
    out = torch.zeros(n_out, dtype=torch.bfloat16).pin_memory()
    work = torch.empty(loco.loco_reduce_host_workspace_bytes(cfg, n, len(parts), count), dtype=torch.uint8, device="cuda")
    loco.loco_unpack_dequant_reduce_host(cfg, parts, n, out, work, first_partition=first, partition_count=count)
    torch.cuda.synchronize()
    return out


def _reduce_without_allocation(cfg, parts, n, first, count):
    n_out = sum(loco.loco_partition_elems(cfg, n, j) for j in range(first, first + count))
    out = torch.zeros(n_out, dtype=torch.bfloat16).pin_memory()
    loco.loco_unpack_dequant_reduce_host_noalloc(cfg, parts, n, out, first_partition=first, partition_count=count)
    torch.cuda.synchronize()
    return out


def test_noalloc_reduce_matches_the_workspace_variant_twice():
    cfg = loco.Config(bits=4, s=2.0 ** 12, s_e=2.0 ** 14, beta=0.5, reset_period=0, state_fmt=loco.STATE_NONE,
                      grad_dtype=loco.BF16, out_dtype=loco.BF16, num_partitions=4)
    # first call: a large request (close to the array's size); second call: a smaller, different one,
    # so that bytes left behind by the first call would show up if they were read
    for n, workers, first, count, seed in ((1_200_003, 8, 1, 2, 41), (70_001, 3, 0, 4, 42)):
        assert loco.loco_reduce_host_workspace_bytes(cfg, n, workers, count) <= loco.NOALLOC_SCRATCH_BYTES
        parts = _random_parts(cfg, n, workers, count, seed)
        want = _reduce_with_workspace(cfg, parts, n, first, count)
        got = _reduce_without_allocation(cfg, parts, n, first, count)
        assert want.abs().max() > 0
        # same kernel on the same bytes: the outputs are identical, which is inside every tolerance in use
        assert np.array_equal(got.view(torch.int16).numpy(), want.view(torch.int16).numpy())
        # and they are what the oracle averages from these parts: each worker's host buffer holds parts first..first+count-1,
        # which the oracle addresses inside a whole communication buffer
        ocfg = orc.OracleConfig(bits=4, s=2.0 ** 12, s_e=2.0 ** 14, beta=0.5, reset_period=0, state_fmt=orc.STATE_NONE,
                                grad_dtype=orc.BF16, out_dtype=orc.BF16, num_partitions=4)
        stride = orc.partition_bytes(ocfg, n)
        comms = []
        for p in parts:
            whole = np.zeros(orc.packed_bytes(ocfg, n), dtype=np.uint8)
            whole[first * stride:(first + count) * stride] = p.numpy()
            comms.append(whole)
        oracle = orc.reduce(ocfg, n, comms, first=first, count=count)
        assert np.array_equal(got.view(torch.int16).numpy().view(np.uint16), oracle)


def test_noalloc_reduce_refuses_requests_beyond_its_array():
    cfg = loco.Config(bits=4, s=2.0 ** 12, s_e=2.0 ** 14, state_fmt=loco.STATE_NONE, grad_dtype=loco.BF16,
                      out_dtype=loco.BF16, num_partitions=1)
    n, workers = 2_000_000, 8
    assert loco.loco_reduce_host_workspace_bytes(cfg, n, workers, 1) > loco.NOALLOC_SCRATCH_BYTES
    parts = _random_parts(cfg, n, workers, 1, 43)
    out = torch.full((n,), 7.0, dtype=torch.bfloat16).pin_memory()
    with pytest.raises(loco.LocoError) as ei:
        loco.loco_unpack_dequant_reduce_host_noalloc(cfg, parts, n, out)
    assert ei.value.code == loco.ERR_SIZE
    torch.cuda.synchronize()
    assert bool((out == 7.0).all()), "a refused call must not touch the output"
