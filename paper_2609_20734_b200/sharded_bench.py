"""Benchmark modes in which the ranks of `bench.py --gpus N` share ONE batch of requests instead of
serving a batch each (strong scaling):

  --shard heads     KV-head tensor parallelism: rank r holds KV heads [r*Hkv/N, (r+1)*Hkv/N) of every
                    layer and request.  A step is tensor_parallel.tp_step: Local pass over the rank's
                    heads, the rank's share of the recall head's first layer, ONE all-reduce of
                    batch x d_hidden floats (NCCL), the decision, the gated Full pass.
  --shard sequence  rank r holds pages [ceil(r*n/N), ceil((r+1)*n/N)) of every request's history.  A
                    step is tensor_parallel.sp_full_step: the gated Full pass over the rank's pages, an
                    all-gather of the partial rows and their log-sum-exps (NCCL), the merge.  The Local
                    pass and the decision are not part of this mode (the window lives on the last rank).

Both use the library's kernels between plain NCCL collectives: no peer-memory kernels, no multicast.
The planning half (what each rank holds, the line's format) is plain Python and is what the CPU tests
drive with gloo ranks; the timing half needs one GPU per rank.
"""
from __future__ import annotations

import json
import os
from dataclasses import replace

import numpy as np

from . import tensor_parallel as tp
from . import workloads

P = 16


def plan(wl, shard: str, rank: int, world: int):
    """What rank `rank` of `world` holds and reads.  Returns (rank's workload, info dict)."""
    if shard == "heads":
        if wl.Hkv % world:
            raise ValueError(f"{wl.Hkv} KV heads do not divide over {world} ranks")
        head = wl.head if wl.head else (0, 1, 256)     # the decision needs a head for there to be an exchange
        hs = tp.head_shard(rank, world, wl.Hq, wl.Hkv, wl.D, d_ext=head[0], use_attn_out=bool(head[1]))
        # the rank's stack: its own heads; its recall head multiplies its own columns of W1
        mine = replace(wl, Hq=hs.q_heads, Hkv=hs.kv_heads, head=(hs.d_ext, head[1], head[2]), seed=wl.seed + 1000 * rank)
        info = {"kv_heads": [hs.kv_head_begin, hs.kv_head_begin + hs.kv_heads], "w1_columns": [hs.col_begin, hs.col_begin + hs.col_count],
                "exchange_bytes_per_step": wl.B * head[2] * 4, "d_hidden": head[2], "d_in": hs.d_in,
                "kv_bytes_per_token": mine.kv_token_bytes}
        return mine, info
    if shard == "sequence":
        lens = np.asarray(wl.seq_lens0, dtype=np.int64)
        lo, hi, held = zip(*[tp.sequence_shard(rank, world, int(t), P) for t in lens])
        mine = replace(wl, seq_lens0=np.maximum(np.asarray(held, np.int32), 0), seed=wl.seed + 1000 * rank)
        info = {"pages": [[int(a), int(b)] for a, b in zip(lo, hi)], "tokens_held": [int(h) for h in held],
                "exchange_bytes_per_step": wl.L * wl.B * wl.Hq * (wl.D + 1) * 4 * (world - 1)}
        return mine, info
    raise ValueError(shard)


def line(bench, args, wl, shard, world, total_ms, step_bytes, launches_per_step, extra):
    """Rank 0's JSON line (same keys as the default mode's)."""
    realised = 1.0 if shard == "sequence" else wl.recall_rate
    if shard == "heads" and not wl.head:
        wl = replace(wl, head=(0, 1, 256))    # the head this mode adds so that the decision has an exchange
    d = {"metric": bench.METRIC, "value": wl.B * args.steps / (total_ms * 1e-3), "unit": bench.UNIT, "n_gpus": world,
         "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
         "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
         "config": bench.config_dict(wl, args, realised, shard), "launch": "eager launches between NCCL collectives",
         "arithmetic": bench.ARITHMETIC_TEXT, "gpu_launches": launches_per_step * args.steps,
         "step_gbs": step_bytes / (total_ms / args.steps * 1e-3) / 1e9, "shard": shard}
    d.update(extra)
    return d


def _max_over_ranks(x, dist, device):
    import torch

    t = torch.tensor([x], dtype=torch.float64, device=device)
    if dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run(args, wl, bench):
    import torch
    import torch.distributed as dist

    from . import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if "MASTER_ADDR" not in os.environ:   # a plain one-process run still goes through the collective calls
        os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT="29532")
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", local_rank))
    args.warmup = max(args.warmup, 3)
    nsteps = args.warmup + args.steps
    wl.steps = nsteps + 1
    mine, info = plan(wl, args.shard, rank, world)
    mine.steps = wl.steps
    flush = bench.L2Flush(torch)
    B, L = wl.B, wl.L

    def barrier():
        dist.barrier()
        torch.cuda.synchronize()

    if args.shard == "heads":
        st = workloads.materialize(mine)
        ctx = binding.OdaContext(workloads.oda_config(mine, st.num_blocks, variant=args.variant))
        hs = tp.head_shard(rank, world, wl.Hq, wl.Hkv, wl.D, d_ext=info["d_in"] - wl.Hq * wl.D, use_attn_out=True)
        # every rank generates the same full first-layer matrix and reads only its columns
        full = replace(wl, head=(info["d_in"] - wl.Hq * wl.D, 1, info["d_hidden"]))
        hh = full.head_host()
        head = {k: torch.from_numpy(np.ascontiguousarray(v)).cuda() for k, v in hh.items() if k != "use_attn_out"}
        qs = [workloads.q_device(mine, s) for s in range(nsteps)]
        flags_h = bench.schedule_flags(wl, args.warmup, args.steps)
        ovs = [torch.from_numpy(f).cuda() for f in flags_h]
        out = torch.zeros((L, B, mine.Hq, wl.D), device="cuda")
        pre = torch.zeros((B, info["d_hidden"]), device="cuda")
        scores = torch.zeros(B, device="cuda")
        flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
        seq0 = st.seq_lens.clone()

        def step(s):
            tp.tp_step(ctx, hs, B, qs[s], st.k_cache, st.v_cache, st.block_table, st.seq_lens, out,
                       W1=head["W1"], b1=head["b1"], w2=head["w2"], b2=head["b2"], threshold=wl.threshold,
                       pre=pre, scores=scores, flags=flags, override_flags=ovs[s])
            ctx.advance_seq_lens(B, st.seq_lens)

        seq_steps = [np.asarray(wl.seq_lens0) + s for s in range(args.warmup, nsteps)]
        step_bytes = float(np.mean([sum(wl.algorithmic_bytes(sl, f)) for sl, f in zip(seq_steps, flags_h[args.warmup:])]))
    else:
        # this rank's slice of every request: its own pool of pages, a local table and local lengths
        st = workloads.materialize(mine)
        ctx = binding.OdaContext(workloads.oda_config(mine, st.num_blocks, variant=args.variant, allow_empty=1))
        qs = [workloads.q_device(wl, s) for s in range(nsteps)]       # same queries on every rank
        ones = torch.ones(B, dtype=torch.uint8, device="cuda")
        part_out = torch.zeros((L, B, wl.Hq, wl.D), device="cuda")
        part_lse = torch.zeros((L, B, wl.Hq), device="cuda")
        parts_out = torch.zeros((world,) + tuple(part_out.shape), device="cuda")
        parts_lse = torch.zeros((world,) + tuple(part_lse.shape), device="cuda")
        out = torch.zeros_like(part_out)
        held = torch.tensor(info["tokens_held"], dtype=torch.int32, device="cuda")
        tokens = torch.zeros((world, B), dtype=torch.int32, device="cuda")
        dist.all_gather(list(tokens.unbind(0)), held)
        seq0 = st.seq_lens.clone()

        def step(s):
            tp.sp_full_step(ctx, world, B, qs[s], st.k_cache, st.v_cache, st.block_table, st.seq_lens, tokens, ones,
                            part_out, part_lse, parts_out, parts_lse, out)

        step_bytes = float(sum(int(t) for t in wl.seq_lens0) * sum(wl.gated) * wl.kv_token_bytes)

    before = ctx.launch_count
    step(0)
    launches_per_step = ctx.launch_count - before
    torch.cuda.synchronize()

    def one_pass():
        st.seq_lens.copy_(seq0)
        for s in range(args.warmup):
            flush.fill_(s)
            step(s)
        barrier()
        evs = []
        for s in range(args.warmup, nsteps):
            flush.fill_(s)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            step(s)
            e1.record()
            evs.append((e0, e1))
        barrier()
        return float(sum(a.elapsed_time(b) for a, b in evs))

    one_pass()
    sampler = bench.ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    totals = sorted(_max_over_ranks(one_pass(), dist, "cuda") for _ in range(max(1, args.passes)))
    total_ms = totals[len(totals) // 2]
    assert ctx.read_device_status() == 0, "device status word set during the timed region"
    if rank == 0:
        extra = {"passes": {"measured": len(totals), "statistic": "median", "ms_per_step": [t / args.steps for t in totals]},
                 "rank0_holds": info, "clocks": sampler.stop(),
                 "note": "steps are launched eagerly (a collective sits between the library's kernels), so the host's "
                         "launch path is inside the events"}
        print(json.dumps(line(bench, args, wl, args.shard, world, total_ms, step_bytes, launches_per_step, extra)))
    dist.barrier()
    dist.destroy_process_group()
