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


def _free_port():
    import socket

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


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
        mp.spawn(_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
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


def _tp_problem():
    from tests.helpers import make_problem
    from paper_2609_20734_b200 import synth

    L, B, Hq, Hkv, D, d_ext, d_h = 2, 3, 8, 4, 16, 5, 12
    prob = make_problem(8, L, B, Hq, Hkv, D, [40, 7, 130])
    head = dict(W1=synth.gauss_f32_tensor(3, synth.STREAM_W1, (d_h, d_ext + Hq * D), std=0.1),
                b1=synth.gauss_f32_tensor(3, synth.STREAM_B1, (d_h,), std=0.1),
                w2=synth.gauss_f32_tensor(3, synth.STREAM_W2, (d_h,), std=0.1),
                b2=synth.gauss_f32_tensor(3, synth.STREAM_B2, (1,), std=0.1))
    fe = synth.gauss_f32_tensor(3, synth.STREAM_FEAT, (B, d_ext))
    return prob, head, fe, d_ext, d_h


def _tp_worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import oda_oracle as orc
    from paper_2609_20734_b200 import tensor_parallel as tp

    prob, head, fe, d_ext, d_h = _tp_problem()
    L, B, Hq, Hkv, D, lay = prob["L"], prob["B"], prob["Hq"], prob["Hkv"], prob["D"], prob["layout"]
    sh = tp.head_shard(rank, world, Hq, Hkv, D, d_ext, True)
    # the rank's heads: a slice of q, and the caches entered at its first KV head
    q = np.ascontiguousarray(prob["q"][:, :, sh.q_head_begin:sh.q_head_begin + sh.q_heads])
    off = sh.kv_head_begin * lay.head_stride
    out, _ = orc.attention("local", q, prob["k"][off:], prob["v"][off:], prob["table"], prob["seq_lens"],
                           num_kv_heads=sh.kv_heads, block_size=16, layout=lay, layer_window=[16, 16],
                           layer_sinks=[2, 2])
    x = out[L - 1].reshape(B, -1)
    if sh.d_ext:
        x = np.concatenate([fe.astype(np.float64), x], axis=1)
    assert x.shape[1] == sh.col_count
    W = head["W1"][:, sh.col_begin:sh.col_begin + sh.col_count].astype(np.float64)
    pre = torch.from_numpy(x @ W.T)
    tp.sum_over_ranks(pre)                           # the step's one collective
    a = pre.numpy() + head["b1"].astype(np.float64)
    z = (a / (1.0 + np.exp(-a))) @ head["w2"].astype(np.float64) + float(head["b2"][0])
    ret[rank] = (sh, out, z)
    dist.barrier()
    dist.destroy_process_group()


def test_kv_head_tensor_parallel_two_ranks_gloo():
    """Ranks own disjoint KV heads and W1 columns; after one all-reduce of the first-layer
    products every rank holds the logits of the unsharded head, and the heads' outputs tile
    the unsharded attention output."""
    world = 2
    with mp.Manager() as m:
        ret = m.dict()
        mp.spawn(_tp_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
        res = dict(ret)
    from oracle import oda_oracle as orc
    from tests.helpers import oracle_attention

    prob, head, fe, d_ext, d_h = _tp_problem()
    whole, _ = oracle_attention(prob, "local", [16, 16], [2, 2])
    z, _ = orc.recall_head(fe, whole[prob["L"] - 1], head["W1"], head["b1"], head["w2"], head["b2"])
    cols = []
    for r in range(world):
        sh, out, zr = res[r]
        np.testing.assert_array_equal(out, whole[:, :, sh.q_head_begin:sh.q_head_begin + sh.q_heads])
        np.testing.assert_allclose(zr, z, rtol=0, atol=1e-12)
        np.testing.assert_array_equal(zr, res[0][2])     # identical on every rank
        cols += list(range(sh.col_begin, sh.col_begin + sh.col_count))
    assert cols == list(range(d_ext + prob["Hq"] * prob["D"]))


def test_head_shard_arithmetic():
    from paper_2609_20734_b200 import tensor_parallel as tp
    import pytest

    for world in (1, 2, 4, 8):
        shards = [tp.head_shard(r, world, 32, 8, 128, 24, True) for r in range(world)]
        assert sum(s.kv_heads for s in shards) == 8 and sum(s.q_heads for s in shards) == 32
        assert sum(s.col_count for s in shards) == shards[0].d_in == 24 + 32 * 128
        assert all(a.col_begin + a.col_count == b.col_begin for a, b in zip(shards, shards[1:]))
        assert all(s.q_head_begin == s.kv_head_begin * 4 for s in shards)
        assert [s.d_ext for s in shards] == [24] + [0] * (world - 1)
    with pytest.raises(ValueError):
        tp.head_shard(0, 3, 32, 8, 128)
    with pytest.raises(ValueError):
        tp.head_shard(2, 2, 32, 8, 128)


_SP_SEQ = [40, 7, 130, 65, 18]


def _sp_worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import oda_oracle as orc
    from paper_2609_20734_b200 import tensor_parallel as tp
    from tests.helpers import make_problem

    prob = make_problem(6, 2, len(_SP_SEQ), 4, 2, 16, _SP_SEQ)
    B, width = len(_SP_SEQ), prob["table"].shape[1]
    table = np.zeros((B, width), np.int32)
    held = np.zeros(B, np.int32)
    for b, t in enumerate(_SP_SEQ):
        lo, hi, held[b] = tp.sequence_shard(rank, world, t)
        table[b, :hi - lo] = prob["table"][b, lo:hi]
    out, lse = orc.attention("full", prob["q"], prob["k"], prob["v"], table, np.maximum(held, 1),
                             num_kv_heads=2, block_size=16, layout=prob["layout"], layer_window=[16, 16],
                             layer_sinks=[2, 2], request_mask=(held > 0).astype(np.uint8))
    out = torch.from_numpy(np.nan_to_num(out))
    lse = torch.from_numpy(np.where(np.isnan(lse), -np.inf, lse))
    outs = torch.empty((world,) + tuple(out.shape), dtype=out.dtype)
    lses = torch.empty((world,) + tuple(lse.shape), dtype=lse.dtype)
    tp.gather_over_ranks(outs, out)
    tp.gather_over_ranks(lses, lse)
    m = lses.max(0).values
    wgt = torch.exp(lses - m)
    merged = (wgt[..., None] * outs).sum(0) / wgt.sum(0)[..., None]
    ret[rank] = (held.copy(), merged.numpy(), (m + torch.log(wgt.sum(0))).numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_sequence_sharded_full_two_ranks_gloo():
    """Ranks hold page ranges of every request; their (out, lse) pairs, gathered and combined by
    log-sum-exp, are Full attention over the whole history on every rank."""
    world = 2
    with mp.Manager() as m:
        ret = m.dict()
        mp.spawn(_sp_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
        res = dict(ret)
    from tests.helpers import make_problem, oracle_attention

    prob = make_problem(6, 2, len(_SP_SEQ), 4, 2, 16, _SP_SEQ)
    whole, whole_lse = oracle_attention(prob, "full", [16, 16], [2, 2])
    assert (sum(res[r][0] for r in range(world)) == np.array(_SP_SEQ)).all()
    assert (res[1][0] == 0).any()                    # the 7-token request fits one rank
    for r in range(world):
        np.testing.assert_allclose(res[r][1], whole, rtol=0, atol=1e-12)
        np.testing.assert_allclose(res[r][2], whole_lse, rtol=0, atol=1e-12)


def test_sequence_shard_covers_every_position_once():
    from paper_2609_20734_b200 import tensor_parallel as tp

    for t in (1, 15, 16, 17, 100, 2500):
        for world in (1, 2, 3, 8):
            parts = [tp.sequence_shard(r, world, t) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == (t + 15) // 16
            assert all(a[1] == b[0] for a, b in zip(parts, parts[1:]))
            assert sum(p[2] for p in parts) == t


def _bench_mode_worker(rank, world, port, ret):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2609_20734_b200 import sharded_bench, sharding, workloads

    res = {}
    for shard, name in (("heads", "llama8b"), ("sequence", "batched")):
        # the same argument path as `bench.py --gpus 2 --shard ...`
        args = bench.parse(["--gpus", str(world), "--shard", shard, "--config", name, "--steps", "4", "--warmup", "3"])
        wl = workloads.make(args.config)
        mine, info = sharded_bench.plan(wl, shard, rank, world)
        infos = [None] * world
        dist.all_gather_object(infos, info)
        total_ms = sharding.max_over_ranks(10.0 * (rank + 1))       # the slowest rank's time counts
        line = sharded_bench.line(bench, args, wl, shard, world, total_ms, 1e9, 3, {}) if rank == 0 else None
        res[shard] = (mine, infos, line)
    ret[rank] = res
    dist.barrier()
    dist.destroy_process_group()


def test_bench_shard_modes_two_ranks_gloo():
    """`bench.py --shard heads|sequence`: what each rank holds tiles the workload exactly once, and rank 0's
    line has the contract's keys with the slowest rank's time (the timed half needs one GPU per rank)."""
    world = 2
    with mp.Manager() as m:
        ret = m.dict()
        mp.spawn(_bench_mode_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
        res = dict(ret)
    from paper_2609_20734_b200 import workloads

    wl = workloads.make("llama8b")
    mine0, infos, line = res[0]["heads"]
    assert [i["kv_heads"] for i in infos] == [[0, 4], [4, 8]]
    assert [i["w1_columns"] for i in infos] == [[0, 2048], [2048, 4096]] and infos[0]["d_in"] == 4096
    assert infos[0]["exchange_bytes_per_step"] == wl.B * 256 * 4
    assert sum(res[r]["heads"][0].kv_token_bytes for r in range(world)) == wl.kv_token_bytes
    assert (mine0.Hq, mine0.Hkv) == (16, 4) and res[1]["heads"][0].seed != mine0.seed
    assert line["scaling"] == "strong" and line["n_gpus"] == 2 and line["ms_per_step"] == 20.0 / 4
    assert line["value"] == wl.B * 4 / 20e-3 and line["config"]["parallelism"].startswith("tp2")
    assert line["config"]["global_batch"] == wl.B and "llama8b" in line["config"]["workload"]
    wl = workloads.make("batched")
    _, infos, line = res[0]["sequence"]
    lens = np.asarray(wl.seq_lens0)
    assert (np.asarray(infos[0]["tokens_held"]) + np.asarray(infos[1]["tokens_held"]) == lens).all()
    for b in range(wl.B):
        (a0, a1), (b0, b1) = infos[0]["pages"][b], infos[1]["pages"][b]
        assert a0 == 0 and a1 == b0 and b1 == (int(lens[b]) + 15) // 16
    assert line["config"]["parallelism"].startswith("sp2") and line["shard"] == "sequence"
    for key in ("metric", "value", "unit", "steps", "warmup", "higher_is_better", "vs_baseline", "dtype", "data", "gpu_launches"):
        assert key in line
