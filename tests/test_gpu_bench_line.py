"""The benchmark's own arm on a GPU: one JSON line with every key of the contract, internally
consistent (a short run of the real configuration; the numbers themselves are not judged here)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_prints_one_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "8", "--warmup", "3", "--no-sweep",
                        "--kernel-reps", "2", "--configs", "tiny", "--no-paper-head"], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["metric"] == "decode_attention_tokens_per_s" and d["unit"] == "tokens/s" and "impl" not in d
    assert d["n_gpus"] == 1 and d["steps"] == 8 and d["warmup"] == 3 and d["higher_is_better"] is True
    assert d["scaling"] == "weak" and d["vs_baseline"] is None and d["data"] == "synthetic" and d["dtype"] == "bf16"
    assert abs(d["value"] - 1e3 / d["ms_per_step"]) < 1e-6 * d["value"]          # batch 1: tokens/s = 1 / step time
    assert "llama8b" in d["config"]["workload"] and "flushed" in d["config"]["l2"]
    assert d["config"]["recall_rate_realised"] == 0.25
    assert d["gpu_launches"] == 2 * d["steps"]
    roof = d["roofline"]
    assert roof["bound"] == "hbm" and roof["unit"] == "GB/s" and roof["peak"] > 0 and roof["traffic"] > 0
    assert abs(roof["frac"] - roof["achieved"] / roof["peak"]) < 1e-9
    assert abs(roof["achieved"] - roof["algorithmic_bytes"] / (roof["us"] * 1e-6) / 1e9) < 1e-6 * roof["achieved"]
    assert 0.98 < roof["traffic"] / roof["algorithmic_bytes"] < 1.1
    e2e = d["e2e"]
    assert e2e["unit"] == "tokens/s" and 0 < e2e["value"] < d["value"]
    assert e2e["h2d_bytes_per_step"] == 32 * 32 * 128 * 2 + 1                       # q (bf16) and one forced flag
    assert e2e["d2h_bytes_per_step"] == 32 * 32 * 128 * 4 + 4 + 1                   # rows (f32), score, flag
    cpu = d["cpu_baseline"]
    assert cpu["kind"] == "oracle" and cpu["cores"] >= 1 and cpu["value"] > 0 and cpu["sample"]
    clk = d["clocks"]
    assert clk["sm_max_mhz"] >= clk["sm_mhz"] > 0 and isinstance(clk["reasons"], list) and clk["samples"] >= 10
    # three measured passes, the median one is the headline
    ps = d["passes"]
    assert ps["measured"] == 3 and sorted(ps["ms_per_step"])[1] == d["ms_per_step"]
    assert d["roofline_other"]["floor_us"] > 0 and d["roofline_other"]["frac_above_floor"] > d["roofline_other"]["frac"]
    # the Local launch once more with its code warm and its data cold: context beside the flushed figure
    cw = d["roofline_other"]["code_warm"]
    assert 0 < cw["us"] < 2 * d["roofline_other"]["us"] and cw["frac"] > 0
    # the arm-specific descriptions sit beside `config`, which both arms fill identically
    assert "launch" in d and "arithmetic" in d and "launch" not in d["config"]
    (tiny,) = d["configs"]
    assert tiny["name"] == "tiny" and tiny["recall_rate_realised"] == 0.25 and tiny["tokens_per_s"] > 0
    assert tiny["head"]["us"] > 0 and tiny["local"]["us"] > 0 and tiny["full"]["us"] > 0


@pytest.mark.parametrize("shard", ["heads", "sequence"])
def test_bench_shard_modes_run_at_world_size_one(shard):
    """The GPU half of `bench.py --shard ...` with one rank: the library's kernels on either side of an
    NCCL collective (which a one-rank group performs on itself), one contract line."""
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "1", "--shard", shard, "--steps", "4",
                        "--warmup", "3"], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["shard"] == shard and d["scaling"] == "strong" and d["n_gpus"] == 1 and d["steps"] == 4
    assert d["value"] > 0 and abs(d["value"] - 1e3 / d["ms_per_step"]) < 1e-6 * d["value"]
    assert d["passes"]["measured"] == 3 and d["gpu_launches"] == (5 if shard == "heads" else 2) * 4
    assert d["config"]["parallelism"].startswith("tp1" if shard == "heads" else "sp1")
