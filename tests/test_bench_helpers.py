"""Host-side pieces of bench.py that need no GPU: the forced-flag schedule, the line's bookkeeping and
what both arms must fill identically."""
import argparse

import numpy as np

import bench
from paper_2609_20734_b200 import workloads


def test_conditioned_bernoulli_schedule_hits_the_rate_exactly():
    for name, steps in (("llama8b", 20), ("batched", 16), ("70b", 20), ("hybrid", 20)):
        wl = workloads.make(name)
        fl = bench.schedule_flags(wl, 3, steps)
        assert len(fl) == 3 + steps and all(f.shape == (wl.B,) and f.dtype == np.uint8 for f in fl)
        timed = np.stack(fl[3:])
        assert (timed.sum(0) == round(wl.recall_rate * steps)).all()          # every request, exactly
        assert abs(timed.mean() - wl.recall_rate) < 1e-12
        again = bench.schedule_flags(workloads.make(name), 3, steps)
        assert all((a == b).all() for a, b in zip(fl, again))                 # seeded
    wl = workloads.make("llama8b", recall_rate=0.0)
    assert not np.stack(bench.schedule_flags(wl, 0, 8)).any()
    wl = workloads.make("llama8b", recall_rate=1.0)
    assert np.stack(bench.schedule_flags(wl, 0, 8)).all()


def test_both_arms_describe_the_same_config():
    args = bench.parse(["--steps", "20", "--warmup", "5"])
    wl = workloads.make(args.config)
    ours = bench.config_dict(wl, args, 0.25)
    ref = bench.config_dict(workloads.make(args.config), bench.parse(["--impl", "reference", "--steps", "20", "--warmup", "5"]), 0.25)
    assert ours == ref
    assert "launch" not in ours and "arithmetic" not in ours and ours["parallelism"].startswith("dp1")
    assert "llama8b" in ours["workload"] and "context=32768" in ours["workload"] and "window=1024 sinks=4" in ours["workload"]
    hyb = bench.workload_text(workloads.make("hybrid"))
    assert "12 gated layers window=1024 sinks=4" in hyb and "36 fixed-window layers window=512 sinks=0" in hyb
    assert "recall head 4096->256->1" in hyb
    bat = bench.workload_text(workloads.make("batched"))
    assert "shuffled block tables" in bat and "context=" in bat and ".." in bat


def test_roofline_entry_arithmetic_and_flag_above_one():
    e = bench.roofline_entry(134742016, 34.8, 6460.2)
    assert abs(e["achieved"] - 134742016 / 34.8e-6 / 1e9) < 1e-9 and abs(e["frac"] - e["achieved"] / 6460.2) < 1e-12
    assert abs(e["frac_of_8000_nominal"] - e["achieved"] / 8000.0) < 1e-12 and "frac_note" not in e
    e = bench.roofline_entry(4294967296, 604.0, 6460.2)
    assert e["frac"] > 1.0 and "copy" in e["frac_note"]


def test_algorithmic_bytes_of_the_configs():
    wl = workloads.make("llama8b")
    lb, fb = wl.algorithmic_bytes(np.asarray(wl.seq_lens0), np.ones(1))
    assert (lb, fb) == (32 * 1028 * 4096, 32 * 32768 * 4096)
    lb0, fb0 = wl.algorithmic_bytes(np.asarray(wl.seq_lens0), np.zeros(1))
    assert (lb0, fb0) == (lb, 0)
    hyb = workloads.make("hybrid")
    lb, fb = hyb.algorithmic_bytes(np.asarray(hyb.seq_lens0), np.ones(4))
    assert lb == 4 * (36 * 512 + 12 * 1028) * 4096 and fb == 4 * 12 * 262144 * 4096


def test_clock_sampler_without_a_gpu_reports_instead_of_failing():
    s = bench.ClockSampler(0)
    s.start()
    out = s.stop()
    assert set(out) >= {"sm_mhz", "sm_max_mhz", "reasons", "samples"}
    assert out["samples"] >= 0 and isinstance(out["reasons"], list)


def test_argument_defaults_finish_in_minutes():
    a = bench.parse([])
    assert (a.gpus, a.steps, a.warmup, a.passes, a.impl, a.shard) == (1, 64, 3, 3, "ours", "requests")
    assert set(a.configs.split(",")) == {"tiny", "batched", "70b", "hybrid"}
    assert isinstance(a, argparse.Namespace)
