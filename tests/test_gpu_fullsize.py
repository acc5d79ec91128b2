"""Parity at the benchmark's full size and launch configuration (one CUDA-graph replay of
oda_step), plus the other configurations' shapes at reduced layer counts: the oracle recomputes
sampled (layer, request, kv head) units one by one from regenerated host slices of the cache."""
import numpy as np
import pytest
import torch

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import binding, workloads
from tests import gpu_helpers as gh

pytestmark = pytest.mark.gpu


def oracle_unit(wl, st, step, seq_lens, layer, b, g, mode):
    """Oracle output [G, D] and lse [G] of one unit, from host-regenerated K/V pages."""
    t = int(seq_lens[b])
    k, v, table = wl.host_unit(st.table_host, st.num_blocks, layer, b, g, t)
    G = wl.G
    q = wl.q_host(step)[layer:layer + 1, b:b + 1, g * G:(g + 1) * G]
    lay = orc.hnd_layout(table.shape[1], 1, 16, wl.D)
    out, lse = orc.attention(mode, np.ascontiguousarray(q), k, v, table, np.array([t], np.int32),
                             num_kv_heads=1, block_size=16, layout=lay,
                             layer_window=[wl.windows[layer]], layer_sinks=[wl.sinks[layer]], nthreads=8)
    return out[0, 0], lse[0, 0]


def run_graph_step(wl, st, ctx, step, override, advance=False):
    B = wl.B
    shape = (wl.L, B, wl.Hq, wl.D)
    q = workloads.q_device(wl, step)
    out = torch.zeros(shape, device="cuda")
    lse = torch.zeros(shape[:3], device="cuda")
    scores = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    ov = None if override is None else torch.from_numpy(np.asarray(override, np.uint8)).cuda()
    args = ctx.step_args(B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens, out, scores, flags,
                         head=st.head, threshold=wl.threshold, override_flags=ov, lse=lse,
                         advance_seq_lens=advance)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            ctx.step(args, stream=s.cuda_stream)
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    return out.cpu().numpy(), lse.cpu().numpy(), scores.cpu().numpy(), flags.cpu().numpy(), q


def check_units(wl, st, step, seq_lens, out, lse, flags, units):
    G = wl.G
    worst = 0.0
    for (l, b, g) in units:
        mode = "full" if (wl.gated[l] and flags[b]) else "local"
        ref, rlse = oracle_unit(wl, st, step, seq_lens, l, b, g, mode)
        worst = max(worst, gh.assert_close(out[l, b, g * G:(g + 1) * G], ref, gh.ATOL_OUT, f"unit {(l, b, g)} {mode}"))
        gh.assert_close(lse[l, b, g * G:(g + 1) * G], rlse, gh.ATOL_LSE, f"unit {(l, b, g)} lse")
    return worst


def test_llama8b_full_size_graph_step():
    """Configuration 2 exactly as bench.py runs it: 32 layers, 32q/8kv, D=128, context 32768,
    window 1024 + 4 sinks, 4.3 GB of KV; flags forced to 1, then to 0."""
    wl = workloads.make("llama8b", steps=4)
    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    assert ctx.variant == binding.VARIANT_TMA_MMA
    seq = np.asarray(wl.seq_lens0)
    rng = np.random.RandomState(1)
    units = [(int(rng.randint(wl.L)), 0, int(rng.randint(wl.Hkv))) for _ in range(5)] + [(0, 0, 0), (31, 0, 7)]
    out1, lse1, _, fl1, q = run_graph_step(wl, st, ctx, 0, [1])
    assert fl1[0] == 1
    check_units(wl, st, 0, seq, out1, lse1, fl1, units)
    out0, lse0, _, fl0, _ = run_graph_step(wl, st, ctx, 0, [0])
    check_units(wl, st, 0, seq, out0, lse0, fl0, units[:4])
    # all flags 0 => exactly the Local pass; Full really differs from Local at this length
    loc = torch.zeros_like(torch.from_numpy(out0)).cuda()
    ctx.local_decode(0, wl.L, 1, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens, loc, None)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(loc.cpu().numpy(), out0)
    assert np.abs(out1 - out0).max() > 1e-2
    # properties that hold at any size: every output row is finite and inside the value range
    assert np.isfinite(out1).all() and np.abs(out1).max() < 5.0
    assert (lse1 >= lse0 - 1e-4).all()          # Full's set contains Local's
    assert ctx.read_device_status() == 0


def test_batched_mixed_lengths_shape_with_learned_flags():
    """Configuration 3's shape (batch 16, lengths uniform in [8192, 65536], shuffled block
    tables, head 4096->256->1 deciding the flags) on 2 layers."""
    wl = workloads.make("batched", L=2, windows=[1024] * 2, sinks=[4] * 2, gated=[1, 1], steps=2)
    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    seq = np.asarray(wl.seq_lens0)
    # threshold = median of the scores of an all-Local pass, so about half the requests recall
    _, _, sc, _, _ = run_graph_step(wl, st, ctx, 0, np.zeros(wl.B, np.uint8))
    wl.threshold = float(np.median(sc))
    out, lse, scores, flags, _ = run_graph_step(wl, st, ctx, 0, None)
    np.testing.assert_allclose(scores, sc, rtol=0, atol=0)      # same Local pass, same head
    decided = np.abs(sc - wl.threshold) >= gh.FLAG_BAND
    np.testing.assert_array_equal(flags[decided], (sc > wl.threshold).astype(np.uint8)[decided])
    assert 4 <= flags.sum() <= 12
    shortest, longest = int(np.argmin(seq)), int(np.argmax(seq))
    flagged = [int(b) for b in np.nonzero(flags)[0]][:2]
    unflagged = [int(b) for b in np.nonzero(flags == 0)[0]][:1]
    units = [(1, shortest, 3), (0, longest, 5)] + [(1, b, 0) for b in flagged] + [(0, b, 7) for b in unflagged]
    check_units(wl, st, 0, seq, out, lse, flags, units)
    # the head saw the oracle-grade Local output: teacher-forced score check on the GPU's features
    hh = wl.head_host()
    loc = torch.zeros((wl.L, wl.B, wl.Hq, wl.D), device="cuda")
    ctx.local_decode(0, wl.L, wl.B, workloads.q_device(wl, 0), st.k_cache, st.v_cache, st.block_table,
                     st.seq_lens, loc, None)
    torch.cuda.synchronize()
    z, s = orc.recall_head(None, loc[1].cpu().numpy().astype(np.float64).reshape(wl.B, -1), hh["W1"],
                           hh["b1"], hh["w2"], hh["b2"])
    np.testing.assert_allclose(scores, s, rtol=0, atol=gh.ATOL_SCORE)
    assert ctx.read_device_status() == 0


def test_70b_shape_group_of_eight():
    """Configuration 4's shape (64q/8kv: G = 8, batch 4, context 131072, window 2048) on 2 layers
    that share one physical cache slice; per-request flags."""
    wl = workloads.make("70b", L=2, windows=[2048] * 2, sinks=[4] * 2, gated=[1, 1], kv_index=[0, 0], steps=2)
    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    seq = np.asarray(wl.seq_lens0)
    ov = np.array([0, 1, 0, 0], np.uint8)
    out, lse, _, flags, _ = run_graph_step(wl, st, ctx, 0, ov)
    check_units(wl, st, 0, seq, out, lse, flags, [(0, 1, 2), (1, 0, 7), (1, 3, 0)])
    assert ctx.read_device_status() == 0


def test_hybrid_shape_fixed_and_gated_layers():
    """Configuration 5's shape: of every 4 layers 3 are fixed-window (512, no sinks) and 1 is
    ODA-gated (1024 + 4 sinks); batch 4; here 8 layers and context 65536 with aliased slices."""
    L = 8
    gated = [1 if l % 4 == 3 else 0 for l in range(L)]
    wl = workloads.make("hybrid", L=L, gated=gated, windows=[1024 if g else 512 for g in gated],
                        sinks=[4 if g else 0 for g in gated], kv_index=[0, 1, 2, 3, 0, 1, 2, 4],
                        seq_lens0=np.array([65536, 40000, 65521, 9000], np.int32), steps=2)
    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    seq = np.asarray(wl.seq_lens0)
    ov = np.array([1, 0, 1, 0], np.uint8)
    out, lse, scores, flags, _ = run_graph_step(wl, st, ctx, 0, ov)
    units = [(3, 0, 1), (7, 2, 6), (7, 1, 0), (2, 0, 3), (4, 2, 5), (6, 3, 2)]
    check_units(wl, st, 0, seq, out, lse, flags, units)
    assert np.isfinite(scores).all()
    assert ctx.read_device_status() == 0


def test_longest_paper_context_one_layer():
    """The paper's longest prompt (516,788 tokens, s=4, w=2048, 16q/8kv heads, D=128) on one layer:
    32,300 pages per unit, every span a partial of some unit; Full and Local units sampled."""
    wl = workloads.make("paper", L=1, windows=[2048], sinks=[4], gated=[1],
                        seq_lens0=np.array([516788], np.int32), steps=2)
    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    seq = np.asarray(wl.seq_lens0)
    out1, lse1, _, fl1, _ = run_graph_step(wl, st, ctx, 0, [1])
    check_units(wl, st, 0, seq, out1, lse1, fl1, [(0, 0, 5)])
    out0, lse0, _, fl0, _ = run_graph_step(wl, st, ctx, 0, [0])
    check_units(wl, st, 0, seq, out0, lse0, fl0, [(0, 0, 0), (0, 0, 7)])
    assert (lse1 >= lse0 - 1e-4).all()
    assert ctx.read_device_status() == 0


def test_batched_full_size_offsets_beyond_32_bits():
    """Configuration 3 at its full size: 32 layers, batch 16, lengths uniform in [8192, 65536],
    shuffled block tables, 38 G bf16 elements per cache tensor (77 GB in all), so page addresses
    need 64-bit arithmetic everywhere.  One graph-replayed step with a mixed gate pattern; sampled
    units across the whole address range against the oracle."""
    free, _ = torch.cuda.mem_get_info()
    wl = workloads.make("batched", steps=2)
    need = 2 * wl.phys_layers * int(wl.blocks_needed.sum()) * wl.Hkv * 16 * wl.D * 2
    if free < need + (6 << 30):
        pytest.skip(f"needs {need / 2**30:.0f} GiB of device memory")
    st = workloads.materialize(wl)
    assert st.k_cache.numel() > 2**32
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    seq = np.asarray(wl.seq_lens0)
    ov = (np.arange(wl.B) % 3 == 0).astype(np.uint8)
    out, lse, scores, flags, _ = run_graph_step(wl, st, ctx, 0, ov)
    np.testing.assert_array_equal(flags, ov)
    longest, shortest = int(np.argmax(seq)), int(np.argmin(seq))
    # units whose pages lie in the first, a middle and the last layer slice; flagged and not
    units = [(0, 0, 0), (31, 15, 7), (31, longest, 3), (16, shortest, 5), (30, 3, 1), (17, 4, 6), (31, 1, 0)]
    check_units(wl, st, 0, seq, out, lse, flags, units)
    assert np.isfinite(out).all()
    assert ctx.read_device_status() == 0
    del st, ctx
    torch.cuda.empty_cache()


def _fits(wl, slack=6 << 30):
    free, _ = torch.cuda.mem_get_info()
    need = 2 * wl.phys_layers * int(wl.blocks_needed.sum()) * wl.Hkv * 16 * wl.D * 2
    return free >= need + slack, need


def test_70b_full_size_eighty_layers():
    """Configuration 4 at its full shape: 80 layers, 64q/8kv (G = 8), batch 4, context 131072,
    window 2048 + 4 sinks; the 80 layers read 16 physical cache slices (the whole cache would be
    160 GiB).  One request recalls: only its pages may be read by the gated pass."""
    wl = workloads.make("70b", steps=2)
    ok, need = _fits(wl)
    if not ok:
        pytest.skip(f"needs {need / 2**30:.0f} GiB of device memory")
    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    seq = np.asarray(wl.seq_lens0)
    ov = np.array([0, 0, 1, 0], np.uint8)
    out, lse, _, flags, _ = run_graph_step(wl, st, ctx, 0, ov)
    np.testing.assert_array_equal(flags, ov)
    check_units(wl, st, 0, seq, out, lse, flags, [(79, 2, 7), (0, 2, 0), (40, 0, 3), (79, 3, 1), (17, 1, 5)])
    assert np.isfinite(out).all()
    assert ctx.read_device_status() == 0
    del st, ctx
    torch.cuda.empty_cache()


def test_hybrid_full_size_forty_eight_layers():
    """Configuration 5 at its full shape: 48 layers (36 fixed-window 512 without sinks on 3 shared
    slices, 12 gated 1024 + 4 sinks with a slice each), batch 4, context 262144."""
    wl = workloads.make("hybrid", steps=2)
    ok, need = _fits(wl)
    if not ok:
        pytest.skip(f"needs {need / 2**30:.0f} GiB of device memory")
    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    seq = np.asarray(wl.seq_lens0)
    # the flags come from this configuration's head; the threshold is set between its scores
    _, _, sc, _, _ = run_graph_step(wl, st, ctx, 0, np.zeros(wl.B, np.uint8))
    srt = np.sort(sc)
    wl.threshold = float(0.5 * (srt[2] + srt[3]))          # one of the four requests recalls
    assert srt[3] - wl.threshold > 2 * gh.FLAG_BAND and wl.threshold - srt[2] > 2 * gh.FLAG_BAND
    out, lse, scores, flags, _ = run_graph_step(wl, st, ctx, 0, None)
    assert flags.sum() == 1
    b1 = int(np.argmax(flags))
    b0 = (b1 + 1) % wl.B
    check_units(wl, st, 0, seq, out, lse, flags, [(47, b1, 7), (3, b1, 0), (47, b0, 2), (46, b1, 4), (0, b0, 6)])
    assert np.isfinite(out).all()
    assert ctx.read_device_status() == 0
    del st, ctx
    torch.cuda.empty_cache()
