#!/usr/bin/env python
"""Benchmark of the ODA decode-attention step (one JSON line on stdout).

A step is one pass of the whole hot path -- Local attention on every layer, recall score,
device-side flags, gated Full attention, seq_lens advance -- for one batch of synthetic
requests of the Llama-3-8B-shaped configuration (32 layers, 32q/8kv heads, D=128, batch 1,
context 32768, window 1024 + 4 sinks, block size 16, bf16 KV ~ N(0,1), flags forced by a
seeded Bernoulli draw).  The step is replayed from one CUDA graph; its time is taken with
CUDA events around each replay, with an untimed L2 flush between steps.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attention_tokens_per_s"
UNIT = "tokens/s"
SWEEP_RATES = [0.0, 0.1, 0.25, 0.5, 1.0]
FLUSH_BYTES = 256 << 20


class L2Flush:
    """Untimed L2 flush between timed launches: a 256 MiB write (twice the 126 MB L2), then a 256 MiB
    read of a second buffer.  The write evicts the previous iteration's data; the read pushes the
    write's own dirty lines out, so that the cache the timed launch starts with is cold AND clean.
    After the write alone the timed launch pays, inside its own events, for writing back up to
    126 MB of this buffer's dirty lines (measured: 18 us of a 646 us pass, 4 us of a 41 us one)."""

    def __init__(self, torch):
        self.torch = torch
        self.w = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
        self.r = torch.zeros(FLUSH_BYTES // 4, dtype=torch.int32, device="cuda")

    def fill_(self, tag):
        self.w.fill_(int(tag) & 0xFF)
        self.r.max()   # result unused: the point is the read traffic


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="llama8b")
    ap.add_argument("--recall-rate", type=float, default=0.25)
    ap.add_argument("--variant", type=int, default=0, help="0 auto, 1 SIMT, 2 TMA+MMA")
    ap.add_argument("--sinks", type=int, default=None)
    ap.add_argument("--phys-layers", type=int, default=0,
                    help="alias the layers onto this many physical cache slices (bounds memory for the large "
                         "configs); -1 = one slice per layer")
    ap.add_argument("--context", type=int, default=0, help="override every request's context length")
    ap.add_argument("--reuse-local", action="store_true",
                    help="variant: the gated pass reads only the positions Local did not and merges with the "
                         "Local result (exact here because the synthetic stack uses the same queries for both)")
    ap.add_argument("--shuffled", type=int, default=-1,
                    help="1: physical blocks in a seeded random order, 0: in logical order (default: the config's own)")
    ap.add_argument("--l2-resident-mib", type=int, default=64,
                    help="budget of the back-to-back context run that keeps leading layers' Local windows in L2")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--kernel-reps", type=int, default=10)
    ap.add_argument("--no-calibrate", action="store_true", help="keep the equal split of work across CTAs")
    ap.add_argument("--paper-sweep", action="store_true",
                    help="attention-only decode at the paper's seven prompt lengths (batch 1, w=2048+4 sinks, "
                         "first-k-of-16 schedules); prints one JSON table and exits")
    ap.add_argument("--kernels-only", action="store_true",
                    help="time only the Local and the all-flagged Full attention launches (for ncu captures)")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy bandwidth)"
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                 "--format=csv,noheader,nounits", "-lms", "25"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        deadline = time.time() + 2.0      # a very short run can end before nvidia-smi has printed its first row
        while not self.rows and time.time() < deadline and self.proc.poll() is None:
            time.sleep(0.02)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def schedule_flags(wl, warmup, steps):
    """Forced flags of a run, one uint8 array [B] per step (None if the head decides).  For the seeded
    Bernoulli schedule the draw is conditioned on its sum: every request recalls on exactly
    round(rate * steps) of the timed steps, at positions chosen by a seeded shuffle, so that the
    realised rate equals the target whatever the number of timed steps is (an unconditioned draw over
    a handful of steps can land anywhere: 0.8 instead of 0.25 over 5 steps).  Warm-up steps keep the
    plain hashed draw."""
    if wl.schedule != "bernoulli":
        return [wl.override_flags(s) for s in range(warmup + steps)]
    flags = [wl.override_flags(s) for s in range(warmup)]
    timed = np.zeros((steps, wl.B), np.uint8)
    k = int(round(wl.recall_rate * steps))
    for b in range(wl.B):
        order = np.random.default_rng([wl.seed, b, steps]).permutation(steps)
        timed[order[:k], b] = 1
    return flags + [timed[s] for s in range(steps)]


def reference_arm(args, wl, realised_rate=None):
    """The oracle, as it stands, timed on the host cores.  A step is a bounded sample of the
    workload: Local on `nl` layers and Full on `nf` layers of the stack, extrapolated to all
    layers and combined at the realised recall rate of the same forced-flag schedule."""
    from oracle import oda_oracle as orc
    from paper_2609_20734_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = orc.host_threads()
    nl = nf = min(8, wl.L)      # sampled layers; they read one generated cache slice (each with its own queries)
    table, nb = wl.tables()
    lay = orc.hnd_layout(nb, wl.Hkv, 16, wl.D)
    kk, vk = synth.stream_key(wl.seed, synth.STREAM_K), synth.stream_key(wl.seed, synth.STREAM_V)
    idx = np.arange(0, lay.layer_stride, dtype=np.uint64)
    k, v = synth.gauss_bf16(kk, idx), synth.gauss_bf16(vk, idx)
    flags = schedule_flags(wl, args.warmup, args.steps)
    realised = float(np.mean([f.mean() for f in flags[args.warmup:]])) if realised_rate is None else realised_rate

    def one(step, mode, n, threads=None):
        q = wl.q_host(step)[:n]
        t0 = time.perf_counter()
        orc.attention(mode, q, k, v, table, np.asarray(wl.seq_lens0) + step, num_kv_heads=wl.Hkv,
                      block_size=16, layout=lay, layer_window=wl.windows[:n], layer_sinks=wl.sinks[:n],
                      layer_kv_index=[0] * n, nthreads=cores if threads is None else threads)
        return time.perf_counter() - t0

    for s in range(args.warmup):
        one(s, "local", nl)
    tl, tf = [], []
    for s in range(args.steps):
        tl.append(one(args.warmup + s, "local", nl) * wl.L / nl)
        if s < max(1, min(args.steps, 3)):
            tf.append(one(args.warmup + s, "full", nf) * sum(wl.gated) / nf)
    step_s = float(np.mean(tl) + realised * np.mean(tf))
    val = wl.B / step_s
    # the same sample on one thread (one Local and one Full call)
    step_1 = one(args.warmup, "local", nl, 1) * wl.L / nl + realised * one(args.warmup, "full", nf, 1) * sum(wl.gated) / nf
    sample = (f"per step: Local on {nl} of {wl.L} layers (every step) and Full on {nf} of {wl.L} layers "
              f"({len(tf)} steps), scaled to all layers and combined at the realised recall rate {realised:.3f}")
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_s * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": dict(config_dict(wl, args, realised), arithmetic="f64 (the oracle)",
                                                launch="host threads over (layer, request, head) units"),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "value_1_thread": wl.B / step_1},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def config_dict(wl, args, realised):
    return {"workload": f"{wl.name}: L={wl.L} B={wl.B} Hq={wl.Hq} Hkv={wl.Hkv} D={wl.D} "
                        f"context={int(np.max(wl.seq_lens0))} window={wl.windows[0]} sinks={wl.sinks[0]} block=16 "
                        f"bf16 KV ~N(0,1), "
                        f"{'seeded Bernoulli flags conditioned on their count' if wl.schedule == 'bernoulli' else wl.schedule + ' flags'}, "
                        f"{'shuffled' if wl.shuffled else 'in-order'} block tables",
            "recall_rate_target": wl.recall_rate, "recall_rate_realised": realised,
            "global_batch": wl.B * args.gpus, "parallelism": f"dp{args.gpus} (requests sharded, no collective)",
            "l2": "flushed between timed steps (256 MiB write, then 256 MiB read so that no dirty lines are left; untimed)",
            "launch": "one CUDA graph replay per step",
            "arithmetic": "bf16 K/V/q, bf16 tensor-core products with f32 accumulation, f32 softmax and outputs",
            "gated_pass": "remainder S^F minus S^L merged with Local" if getattr(wl, "reuse_local", False) else "recomputes all of S^F"}


PAPER_LENGTHS = [4139, 15918, 31400, 63852, 128852, 261696, 516788]


def paper_sweep(args):
    """Tokens/s of the attention path at the paper's prompt lengths: native Full alone, Local
    alone, and ODA steps with Full on the first 2 / 4 / 8 of every 16 steps (12.5 / 25 / 50 %)."""
    import torch

    from paper_2609_20734_b200 import binding, workloads

    torch.cuda.set_device(0)
    flush = L2Flush(torch)
    rows = []
    for n in PAPER_LENGTHS:
        wl = workloads.make("paper", seq_lens0=np.array([n], np.int32), steps=40)
        st = workloads.materialize(wl)
        ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks, variant=args.variant))
        B, L = wl.B, wl.L
        shape = (L, B, wl.Hq, wl.D)
        q = workloads.q_device(wl, 0)
        out = torch.zeros(shape, device="cuda")
        scores = torch.zeros(B, device="cuda")
        flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
        ov = torch.zeros(B, dtype=torch.uint8, device="cuda")
        ones = torch.ones(B, dtype=torch.uint8, device="cuda")
        seq0 = st.seq_lens.clone()
        if not args.no_calibrate:
            ctx.calibration_begin()
            ctx.full_decode_gated(0, L, B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens, ones, out, None)
            ctx.calibration_end()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())

        def capture(fn):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    fn(side.cuda_stream)
            return g

        g_step = capture(lambda s_: ctx.step(ctx.step_args(B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens,
                                                             out, scores, flags, override_flags=ov,
                                                             advance_seq_lens=True), stream=s_))
        g_full = capture(lambda s_: ctx.full_decode_gated(0, L, B, q, st.k_cache, st.v_cache, st.block_table,
                                                            st.seq_lens, ones, out, None, stream=s_))
        g_local = capture(lambda s_: ctx.local_decode(0, L, B, q, st.k_cache, st.v_cache, st.block_table,
                                                        st.seq_lens, out, None, stream=s_))
        torch.cuda.synchronize()

        def timed(graph, steps, first_k=None):
            st.seq_lens.copy_(seq0)
            tot = 0.0
            for s_ in range(steps + 2):
                if first_k is not None:
                    ov.fill_(1 if (s_ % 16) < first_k else 0)
                flush.fill_(s_ & 0xFF)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                graph.replay()
                e1.record()
                torch.cuda.synchronize()
                if s_ >= 2:
                    tot += e0.elapsed_time(e1)
            return B * steps / (tot * 1e-3)

        row = {"input_tokens": n, "full_only_tok_s": timed(g_full, 8), "local_only_tok_s": timed(g_local, 8)}
        for k, name in ((2, "oda_12.5"), (4, "oda_25"), (8, "oda_50")):
            # 32 timed steps after 2 warm-ups: two whole 16-step periods, phase shifted by 2
            row[name + "_tok_s"] = timed(g_step, 32, first_k=k)
        for name in ("local_only", "oda_12.5", "oda_25", "oda_50"):
            row[name + "_speedup_vs_full"] = row[name + "_tok_s"] / row["full_only_tok_s"]
        rows.append(row)
        del st, ctx, g_step, g_full, g_local
        torch.cuda.empty_cache()
    print(json.dumps({"paper_sweep": rows, "shape": "28 layers, 16q/8kv heads, head_dim 128, batch 1, window 2048 + 4 sinks",
                      "note": "attention path only; the paper's table times the whole model in vLLM on A100s"}))


def main():
    args = parse()
    from paper_2609_20734_b200 import workloads

    if args.impl == "ours" and not args.kernels_only:
        args.warmup = max(args.warmup, 3)   # the timing rules want at least three untimed steps; reported as run
    if args.paper_sweep:
        paper_sweep(args)
        return

    ov = {"recall_rate": args.recall_rate}
    if args.shuffled >= 0:
        ov["shuffled"] = bool(args.shuffled)
    wl = workloads.make(args.config, **ov)
    if args.sinks is not None:
        wl.sinks = [args.sinks if g else s for g, s in zip(wl.gated, wl.sinks)]
    wl.steps = args.steps + args.warmup + 1
    if args.phys_layers > 0:
        wl.kv_index = [l % args.phys_layers for l in range(wl.L)]
    elif args.phys_layers < 0:
        wl.kv_index = None
    if args.context > 0:
        wl.seq_lens0 = np.full(wl.B, args.context, np.int32)
    wl.reuse_local = bool(args.reuse_local)
    if args.impl == "reference":
        reference_arm(args, wl)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus > 1 and world == 1:
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", "29531", os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))

    import torch
    import torch.distributed as dist

    from paper_2609_20734_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    # requests are independent: every rank serves its own batch of the same shape (weak scaling)
    wl.seed = wl.seed + rank

    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks, variant=args.variant))
    B, L = wl.B, wl.L
    shape = (L, B, wl.Hq, wl.D)
    nsteps = args.warmup + args.steps
    qs = [workloads.q_device(wl, s) for s in range(nsteps)]
    flags_h = schedule_flags(wl, args.warmup, args.steps)
    head_decides = flags_h[0] is None        # flags come from the recall head (no forced schedule)
    ovs = None if head_decides else [torch.from_numpy(f).cuda() for f in flags_h]
    flags_log = torch.zeros((nsteps, B), dtype=torch.uint8, device="cuda")
    feats = [None if wl.feat_host(s) is None else torch.from_numpy(wl.feat_host(s)).cuda() for s in range(nsteps)]
    q_s = torch.empty_like(qs[0])
    ov_s = torch.zeros(B, dtype=torch.uint8, device="cuda")
    fe_s = None if feats[0] is None else torch.empty_like(feats[0])
    out = torch.zeros(shape, device="cuda")
    lse = torch.zeros(shape[:3], device="cuda")
    scores = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    counters = torch.zeros((B, 2), dtype=torch.int32, device="cuda")
    flush = L2Flush(torch)
    seq0 = torch.from_numpy(np.asarray(wl.seq_lens0, dtype=np.int32)).cuda()

    step_args = ctx.step_args(B, q_s, st.k_cache, st.v_cache, st.block_table, st.seq_lens, out, scores,
                              flags, feat_ext=fe_s, head=st.head, threshold=wl.threshold,
                              override_flags=None if head_decides else ov_s, lse=lse, counters=counters,
                              advance_seq_lens=True)
    calib = 0.0
    if not args.no_calibrate:  # set-up, once: per-SM streaming rates measured on two all-flagged Full passes
        ctx.calibration_begin()
        for _ in range(2):
            ctx.full_decode_gated(0, L, B, qs[0], st.k_cache, st.v_cache, st.block_table, st.seq_lens,
                                  torch.ones(B, dtype=torch.uint8, device="cuda"), out, lse)
        calib = ctx.calibration_end()

    # capture one step; every replay reads lengths and flags on the device
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    before = ctx.launch_count
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            ctx.step(step_args, stream=side.cuda_stream)
    launches_per_step = ctx.launch_count - before
    torch.cuda.synchronize()

    def set_inputs(s):
        q_s.copy_(qs[s])
        if ovs is not None:
            ov_s.copy_(ovs[s])
        if fe_s is not None:
            fe_s.copy_(feats[s])

    def run_steps(first, count, timed):
        evs = []
        for s in range(first, first + count):
            set_inputs(s)
            flush.fill_(s & 0xFF)  # evict the previous step's KV from L2 (untimed)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            flags_log[s].copy_(flags)     # the step's decisions, for the byte count (after the timed region)
            evs.append((e0, e1))
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs] if timed else None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.kernels_only:
        args.steps, args.warmup, args.no_sweep, args.no_e2e, args.no_cpu_baseline = 1, 1, True, True, True
    st.seq_lens.copy_(seq0)
    run_steps(0, args.warmup, False)
    sampler = ClockSampler(local_rank)
    barrier()
    if rank == 0:
        sampler.start()
    t_wall = time.perf_counter()
    ms = run_steps(args.warmup, args.steps, True)
    barrier()
    t_wall = time.perf_counter() - t_wall
    total_ms = float(np.sum(ms))
    if world > 1:
        t = torch.tensor([total_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    if head_decides:
        flags_h = list(flags_log.cpu().numpy())
        args.no_sweep = True                  # the sweep forces rates; this configuration decides by itself
    realised = float(np.mean([f.mean() for f in flags_h[args.warmup:]]))
    assert ctx.read_device_status() == 0, "device status word set during the timed region"
    assert int(counters[0, 0].item()) == args.warmup + args.steps, "the recall kernel did not run once per step"
    value = world * B * args.steps / (total_ms * 1e-3)

    # per-step algorithmic bytes (exact tokens of Eq. 1, not rounded to pages)
    seq_steps = [np.asarray(wl.seq_lens0) + s for s in range(args.warmup, nsteps)]
    ab = [wl.algorithmic_bytes(sl, f) for sl, f in zip(seq_steps, flags_h[args.warmup:])]
    step_bytes = float(np.mean([a + b for a, b in ab]))

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "config": config_dict(wl, args, realised),
            "gpu_launches": launches_per_step * args.steps,
            "step_gbs": step_bytes / (total_ms / args.steps * 1e-3) / 1e9,
            "variant": {1: "simt", 2: "tma_mma"}.get(ctx.variant, str(ctx.variant)),
            "attention_grid": ctx.attention_grid,
            "sm_bandwidth_calibration": {"applied": calib > 0, "slowest_over_fastest_sm": calib},
            "wall_s_timed_region_incl_flush": t_wall}

    # ---- end to end: host buffers through oda_step_host, copies inside the timed region; every rank
    #      runs it at the same time, the slowest rank's time counts ----
    e2e = None
    if not args.no_e2e and not args.kernels_only:
        q_hs = [q.cpu().pin_memory() for q in qs]
        ov_hs = [None if head_decides else torch.from_numpy(f).pin_memory() for f in flags_h]
        fe_hs = [None if f is None else f.cpu().pin_memory() for f in feats]
        out_h = torch.zeros(shape).pin_memory()
        sc_h = torch.zeros(B).pin_memory()
        fl_h = torch.zeros(B, dtype=torch.uint8).pin_memory()
        st.seq_lens.copy_(seq0)
        barrier()
        tot, up, down = 0.0, 0, 0
        for s in range(nsteps):
            a = ctx.step_args(B, q_hs[s], st.k_cache, st.v_cache, st.block_table, st.seq_lens, out_h,
                              sc_h, fl_h, feat_ext=fe_hs[s], head=st.head, threshold=wl.threshold,
                              override_flags=ov_hs[s], counters=counters, advance_seq_lens=True)
            flush.fill_(s & 0xFF)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            up, down = ctx.step_host(a)
            dt = time.perf_counter() - t0
            if s >= args.warmup:
                tot += dt
        if world > 1:
            t = torch.tensor([tot], device="cuda", dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            tot = float(t.item())
        e2e = {"value": world * B * args.steps / tot, "unit": UNIT, "h2d_bytes_per_step": up,
               "d2h_bytes_per_step": down, "ms_per_step": tot / args.steps * 1e3,
               "note": "oda_step_host: pinned host q/flags pulled in by one kernel, out/scores/flags back in pinned host memory "
                       "(written in place over the bus by the kernels when the stack has no recall head, copied "
                       "otherwise), stream sync inside; KV cache, block table and head weights are device-resident state"}

    if rank == 0:
        peak, peak_src = peaks()
        # ---- the two attention kernels alone, events around each launch, L2 flushed ----
        reps = args.kernel_reps
        ones = torch.ones(B, dtype=torch.uint8, device="cuda")
        st.seq_lens.copy_(seq0)
        kt = {"local": [], "full": []}
        # each launch is captured in a graph of its own, so that the events time the kernel and
        # not the host's launch path
        kgraphs = {}
        for name in ("local", "full"):
            gk = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(gk, stream=side):
                    if name == "local":
                        ctx.local_decode(0, L, B, qs[0], st.k_cache, st.v_cache, st.block_table, st.seq_lens,
                                         out, lse, stream=side.cuda_stream)
                    else:
                        ctx.full_decode_gated(0, L, B, qs[0], st.k_cache, st.v_cache, st.block_table,
                                              st.seq_lens, ones, out, lse, stream=side.cuda_stream)
            kgraphs[name] = gk
        torch.cuda.synchronize()
        for r in range(reps + 2):
            for name in ("local", "full"):
                flush.fill_(r)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                kgraphs[name].replay()
                e1.record()
                torch.cuda.synchronize()
                if r >= 2:
                    kt[name].append(e0.elapsed_time(e1))
        # the same two launches back to back without the flush: what the 126 MB L2 keeps of the
        # previous pass (nothing of a 4 GB Full pass, most of a 137 MB Local pass)
        kt_warm = {"local": [], "full": []}
        for name in ("local", "full"):
            for r in range(reps + 2):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                kgraphs[name].replay()
                e1.record()
                torch.cuda.synchronize()
                if r >= 2:
                    kt_warm[name].append(e0.elapsed_time(e1))
        # what a backbone with other work between its layers sees: the Local pass as one launch per
        # layer (chained by programmatic dependent launch inside one graph)
        g_layers = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g_layers, stream=side):
                for l in range(L):
                    ctx.local_decode(l, l + 1, B, qs[0], st.k_cache, st.v_cache, st.block_table, st.seq_lens,
                                     out, lse, stream=side.cuda_stream)
        torch.cuda.synchronize()
        t_layers = []
        for r in range(reps + 2):
            flush.fill_(r)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g_layers.replay()
            e1.record()
            torch.cuda.synchronize()
            if r >= 2:
                t_layers.append(e0.elapsed_time(e1))
        lb, fb = wl.algorithmic_bytes(np.asarray(wl.seq_lens0), np.ones(B))
        kernels = {}
        for name, nbytes in (("local", lb), ("full", fb)):
            t = float(np.mean(kt[name])) * 1e-3
            kernels[name] = {"bound": "hbm", "achieved": nbytes / t / 1e9, "peak": peak, "unit": "GB/s",
                             "frac": nbytes / t / 1e9 / peak, "traffic": None,
                             "algorithmic_bytes": nbytes, "us": t * 1e6, "frac_of_8000_nominal": nbytes / t / 8e12,
                             "us_l2_warm": float(np.mean(kt_warm[name])) * 1e3}
        dominant = "full" if realised * kernels["full"]["us"] > kernels["local"]["us"] else "local"
        line["roofline"] = dict(kernels[dominant], kernel=f"splitkv ({dominant} pass)", peak_source=peak_src)
        line["roofline_other"] = dict(kernels["local" if dominant == "full" else "full"],
                                      kernel=f"splitkv ({'local' if dominant == 'full' else 'full'} pass)")
        line["local_pass_one_launch_per_layer"] = {
            "us": float(np.mean(t_layers)) * 1e3, "launches": L,
            "gbs": lb / (float(np.mean(t_layers)) * 1e-3) / 1e9,
            "note": "context: the same Local work as one launch per layer in one graph, L2 flushed before the graph"}
        traffic_path = os.path.join(ROOT, "profiles", "traffic.json")
        if os.path.exists(traffic_path):  # DRAM bytes per launch from the committed ncu summary
            tr = json.load(open(traffic_path))
            line["roofline"]["traffic"] = tr.get(dominant)
            line["roofline_other"]["traffic"] = tr.get("local" if dominant == "full" else "full")

        # ---- recall-rate sweep: step time must be affine in the realised rate ----
        if not args.no_sweep:
            sweep = []
            n_sw = min(args.steps, 32)
            for rate in SWEEP_RATES:
                wl_r = workloads.make(args.config, recall_rate=rate)
                fl = schedule_flags(wl_r, 0, n_sw)
                st.seq_lens.copy_(seq0)
                tms = []
                for s in range(n_sw):
                    q_s.copy_(qs[s % nsteps])
                    ov_s.copy_(torch.from_numpy(fl[s]).cuda())
                    flush.fill_(s & 0xFF)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    graph.replay()
                    e1.record()
                    torch.cuda.synchronize()
                    tms.append(e0.elapsed_time(e1))
                rr = float(np.mean([f.mean() for f in fl]))
                bts = np.mean([sum(wl.algorithmic_bytes(np.asarray(wl.seq_lens0) + s, fl[s])) for s in range(n_sw)])
                sweep.append({"rate": rate, "realised": rr, "ms_per_step": float(np.mean(tms)),
                              "tokens_per_s": B / (float(np.mean(tms)) * 1e-3),
                              "gbs": float(bts) / (float(np.mean(tms)) * 1e-3) / 1e9})
            x = np.array([s["realised"] for s in sweep])
            y = np.array([s["ms_per_step"] for s in sweep])
            A = np.vstack([x, np.ones_like(x)]).T
            coef, res, *_ = np.linalg.lstsq(A, y, rcond=None)
            ss_tot = float(((y - y.mean()) ** 2).sum())
            r2 = 1.0 - float(((A @ coef - y) ** 2).sum()) / ss_tot if ss_tot > 0 else 1.0
            line["sweep"] = sweep
            line["affine_fit"] = {"slope_ms": float(coef[0]), "intercept_ms": float(coef[1]), "r2": r2}

        # ---- context: the same steps replayed back to back, no flush, one pair of events around all of
        #      them (what a decode loop sees: launches overlap the previous step; the 137 MB Local
        #      working set partly stays in L2, the 4.3 GB Full pass does not) ----
        if not args.kernels_only and ovs is not None:
            st.seq_lens.copy_(seq0)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for s in range(args.warmup, nsteps):
                set_inputs(s)
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            line["back_to_back"] = {"tokens_per_s": B * args.steps / (e0.elapsed_time(e1) * 1e-3),
                                    "ms_per_step": e0.elapsed_time(e1) / args.steps,
                                    "note": "not the headline: no L2 flush between steps, input copies inside the timed region"}
            # the same loop with half of L2 given to the Local windows of the leading layers
            # (oda_set_cache_resident_bytes; a new capture, since a graph keeps the hints it was captured with)
            ctx.set_cache_resident_bytes(args.l2_resident_mib << 20)
            graph2 = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph2, stream=side):
                    ctx.step(step_args, stream=side.cuda_stream)
            ctx.set_cache_resident_bytes(0)
            st.seq_lens.copy_(seq0)
            torch.cuda.synchronize()
            for s in range(args.warmup):
                set_inputs(s)
                graph2.replay()
            e0.record()
            for s in range(args.warmup, nsteps):
                set_inputs(s)
                graph2.replay()
            e1.record()
            torch.cuda.synchronize()
            line["back_to_back"]["ms_per_step_l2_resident"] = e0.elapsed_time(e1) / args.steps
            line["back_to_back"]["l2_resident_mib"] = args.l2_resident_mib

        if e2e is not None:
            line["e2e"] = e2e
        line["clocks"] = sampler.stop()

        # ---- the oracle on the host cores, bounded sample ----
        if not args.no_cpu_baseline and world == 1:
            import contextlib
            import io

            buf = io.StringIO()
            ref_args = argparse.Namespace(**vars(args))
            ref_args.steps, ref_args.warmup = 3, 1
            with contextlib.redirect_stdout(buf):
                reference_arm(ref_args, workloads.make(args.config, recall_rate=args.recall_rate), realised)
            line["cpu_baseline"] = json.loads(buf.getvalue())["cpu_baseline"]
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
