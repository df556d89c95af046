"""Two-rank CPU (gloo) check of the multi-GPU scheme: shard the chunks, accumulate locally, all-reduce the
accumulator once, add the same counter-based noise on every rank.  The arithmetic here is the oracle's (no GPU in
this test); what is under test is the sharding / all-reduce / identical-noise logic the benchmark uses for N > 1."""
import os
import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2109_12191_b200 import synth
from paper_2109_12191_b200.sharding import shard_range, allreduce_accumulator, global_batch

SIZES, BN, CHUNKS, C, SIGMA = [300, 17], 4, 5, 0.3, 1.2


def _chunk(c):
    return [synth.normal_f32((BN, p), 950, c, l, scale=0.05) for l, p in enumerate(SIZES)]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lo, hi = shard_range(CHUNKS, rank, world)
    acc = None
    for c in range(lo, hi):
        acc, _, _ = oracle.clipped_sum(_chunk(c), C, "global", acc)
    if acc is None:
        acc = [np.zeros(p) for p in SIZES]
    flat = torch.from_numpy(np.concatenate(acc))
    allreduce_accumulator(flat, dist)
    total = global_batch(BN * (hi - lo), dist)            # 5 chunks on 2 ranks: the shares are 3 and 2 chunks
    res = oracle.noise_average(flat.numpy(), 0, SIGMA, C, total, 7, 3)
    out[rank] = res
    out[f"total{rank}"] = total
    dist.barrier()
    dist.destroy_process_group()


def test_shard_range_covers_everything_once():
    for n in (0, 1, 5, 16, 17):
        for world in (1, 2, 3, 8):
            spans = [shard_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            assert max(h - l for l, h in spans) - min(h - l for l, h in spans) <= 1
    with pytest.raises(ValueError):
        shard_range(4, 2, 2)


@pytest.mark.timeout(120)
def test_two_ranks_reproduce_the_single_process_step():
    world = 2
    port = 29500 + os.getpid() % 2000
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    ref, _, _ = oracle.privatise([_chunk(c) for c in range(CHUNKS)], C, SIGMA, "global", 7, 3)
    ref = np.concatenate(ref)
    for r in range(world):
        assert out[f"total{r}"] == BN * CHUNKS             # uneven shares still add up to the step's batch
        np.testing.assert_allclose(out[r], ref, rtol=1e-12, atol=1e-15)
    np.testing.assert_array_equal(out[0], out[1])          # every rank holds the same noised average
