"""Multi-process path on CPU (gloo, world_size 2): requests are independent, so ranks shard the
batch with no data-path collective; the only exchange is the max-over-ranks of the elapsed time.
Each rank runs the oracle on its shard; together they must reproduce the single-process result."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_20734_b200 import sharding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from tests.helpers import make_problem, oracle_attention

    seq = [40, 7, 130, 65, 18]
    prob = make_problem(5, 2, len(seq), 4, 2, 16, seq)
    lo, hi = sharding.request_shard(len(seq), rank, world)
    mask = np.zeros(len(seq), np.uint8)
    mask[lo:hi] = 1
    out, _ = oracle_attention(prob, "local", [16, 16], [2, 2], request_mask=mask)
    # whole-job rate = all ranks' tokens over the slowest rank's time
    elapsed = sharding.max_over_ranks(0.5 + rank)
    total = sharding.sum_over_ranks(hi - lo)
    ret[rank] = (lo, hi, out[:, lo:hi].copy(), elapsed, total)
    dist.barrier()
    dist.destroy_process_group()


def test_request_sharding_two_ranks_gloo():
    world = 2
    with mp.Manager() as m:
        ret = m.dict()
        mp.spawn(_worker, args=(world, 29611, ret), nprocs=world, join=True)
        res = dict(ret)
    from tests.helpers import make_problem, oracle_attention

    seq = [40, 7, 130, 65, 18]
    prob = make_problem(5, 2, len(seq), 4, 2, 16, seq)
    whole, _ = oracle_attention(prob, "local", [16, 16], [2, 2])
    covered = []
    for r in range(world):
        lo, hi, part, elapsed, total = res[r]
        covered += list(range(lo, hi))
        np.testing.assert_array_equal(part, whole[:, lo:hi])
        assert elapsed == 1.5 and total == len(seq)
    assert covered == list(range(len(seq)))


def test_request_shard_covers_everything_once():
    for n in (0, 1, 5, 16, 17):
        for world in (1, 2, 3, 8):
            spans = [sharding.request_shard(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
