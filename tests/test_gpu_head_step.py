"""GPU parity of the recall head, the decision rule, the whole step (eager, host-buffer and
CUDA-graph forms) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import binding, synth, workloads
from tests import gpu_helpers as gh
from tests.helpers import make_problem

pytestmark = pytest.mark.gpu


def _head(seed, d_in, d_h, std=0.02):
    return dict(W1=synth.gauss_f32_tensor(seed, synth.STREAM_W1, (d_h, d_in), std=std),
                b1=synth.gauss_f32_tensor(seed, synth.STREAM_B1, (d_h,), std=std),
                w2=synth.gauss_f32_tensor(seed, synth.STREAM_W2, (d_h,), std=std),
                b2=synth.gauss_f32_tensor(seed, synth.STREAM_B2, (1,), std=std), use_attn_out=1)


@pytest.mark.parametrize("B,d_ext,Hq,D,d_h", [(1, 256, 4, 64, 64), (16, 0, 32, 128, 256), (5, 7, 2, 64, 3)])
def test_recall_score_parity(B, d_ext, Hq, D, d_h):
    prob = make_problem(1, 1, B, Hq, Hq, D, [20] * B)
    ctx = gh.make_ctx(prob, [8], [0], [1], head=(d_ext, 1, d_h))
    head = _head(5, d_ext + Hq * D, d_h, std=0.05)
    hd = gh.head_to_device(head)
    fe = synth.gauss_f32_tensor(5, synth.STREAM_FEAT, (B, d_ext)) if d_ext else None
    attn = synth.gauss_f32_tensor(6, synth.STREAM_FEAT, (B, Hq, D))
    z, s = orc.recall_head(fe, attn.astype(np.float64), head["W1"], head["b1"], head["w2"], head["b2"])
    tau = float(np.median(s)) if B > 1 else 0.5
    scores = torch.zeros(B, device="cuda")
    logits = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    counters = torch.zeros((B, 2), dtype=torch.int32, device="cuda")
    fe_d = None if fe is None else torch.from_numpy(fe).cuda()
    attn_d = torch.from_numpy(attn).cuda()
    for _ in range(2):
        ctx.recall_score(B, fe_d, attn_d, hd["W1"], hd["b1"], hd["w2"], hd["b2"], tau, None, scores,
                         logits, flags, counters)
    torch.cuda.synchronize()
    np.testing.assert_allclose(scores.cpu().numpy(), s, rtol=0, atol=gh.ATOL_SCORE)
    np.testing.assert_allclose(logits.cpu().numpy(), z, rtol=0, atol=5e-5)
    want = orc.flags(z, s, tau)
    decided = np.abs(s - tau) >= gh.FLAG_BAND
    np.testing.assert_array_equal(flags.cpu().numpy()[decided], want[decided])
    c = counters.cpu().numpy()
    assert (c[:, 0] == 2).all() and (c[:, 1] == 2 * flags.cpu().numpy()).all()
    # override: the head still runs, the flags are the forced ones
    ov = (np.arange(B) % 2).astype(np.uint8)
    ctx.recall_score(B, fe_d, attn_d, hd["W1"], hd["b1"], hd["w2"], hd["b2"], tau,
                     torch.from_numpy(ov).cuda(), scores, None, flags, None)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(flags.cpu().numpy(), ov)
    np.testing.assert_allclose(scores.cpu().numpy(), s, rtol=0, atol=gh.ATOL_SCORE)


def test_decision_rule_edges_on_device():
    """Strict '>' at equality, and every nonfinite logit (NaN, +inf, -inf) selects Full."""
    B, D = 4, 64
    prob = make_problem(2, 1, B, 1, 1, D, [20] * B)
    ctx = gh.make_ctx(prob, [8], [0], [1], head=(0, 1, 1))
    W1 = torch.zeros((1, D), device="cuda")
    W1[0, 0] = 1.0
    attn = torch.zeros((B, 1, D), device="cuda")
    # hidden pre-activation a = x0; z = w2*SiLU(a) + b2 with w2 = 1
    attn[:, 0, 0] = torch.tensor([0.0, float("nan"), float("inf"), 1.0])
    scores = torch.zeros(B, device="cuda")
    logits = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    one, zero = torch.ones(1, device="cuda"), torch.zeros(1, device="cuda")
    ctx.recall_score(B, None, attn, W1, zero, one, zero, 0.5, None, scores, logits, flags, None)
    torch.cuda.synchronize()
    # z = [0, nan, inf, SiLU(1)]: score 0.5 is not > 0.5; nan and inf are nonfinite
    np.testing.assert_array_equal(flags.cpu().numpy(), [0, 1, 1, 1])
    ctx.recall_score(B, None, attn, W1, zero, -one, zero, 0.5, None, scores, logits, flags, None)
    torch.cuda.synchronize()
    # w2 = -1: z = [0 (or -0), nan, -inf, -SiLU(1)]: -inf is nonfinite too
    np.testing.assert_array_equal(flags.cpu().numpy(), [0, 1, 1, 0])
    assert scores[0].item() == 0.5


def _oracle_step(wl, table, nb, seq_lens, step, head, tau, override):
    lay = (orc.hnd_layout if wl.layout == "hnd" else orc.nhd_layout)(nb, wl.Hkv, 16, wl.D)
    n = wl.phys_layers * lay.layer_stride
    k = synth.gauss_bf16_tensor(wl.seed, synth.STREAM_K, (n,))
    v = synth.gauss_bf16_tensor(wl.seed, synth.STREAM_V, (n,))
    return orc.step(wl.q_host(step), None, k, v, table, seq_lens, num_kv_heads=wl.Hkv, block_size=16,
                    layout=lay, layer_window=wl.windows, layer_sinks=wl.sinks, layer_gated=wl.gated,
                    layer_kv_index=wl.kv_index, head=head, feat_ext=wl.feat_host(step), tau=tau,
                    override_flags=override, nthreads=8)


def test_tiny_config_eight_steps_with_learned_flags():
    """Configuration 1: 8 decode steps, flags from the head, threshold between the 2nd and 3rd
    largest oracle scores so that 2 of 8 steps recall."""
    wl = workloads.make("tiny")
    st = workloads.materialize(wl)
    head = wl.head_host()
    seq0 = np.asarray(wl.seq_lens0)
    pre = [_oracle_step(wl, st.table_host, st.num_blocks, seq0 + k, k, head, 0.5, None) for k in range(wl.steps)]
    sc = np.sort(np.array([r.score[0] for r in pre]))[::-1]
    tau = 0.5 * (sc[1] + sc[2])
    assert sc[1] - tau > 2e-4 and tau - sc[2] > 2e-4
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    out = torch.zeros((wl.L, wl.B, wl.Hq, wl.D), device="cuda")
    lse = torch.zeros((wl.L, wl.B, wl.Hq), device="cuda")
    scores = torch.zeros(wl.B, device="cuda")
    flags = torch.zeros(wl.B, dtype=torch.uint8, device="cuda")
    counters = torch.zeros((wl.B, 2), dtype=torch.int32, device="cuda")
    recalls = 0
    for k in range(wl.steps):
        ref = _oracle_step(wl, st.table_host, st.num_blocks, seq0 + k, k, head, tau, None)
        q = workloads.q_device(wl, k)
        fe = torch.from_numpy(wl.feat_host(k)).cuda()
        args = ctx.step_args(wl.B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens, out, scores,
                             flags, feat_ext=fe, head=st.head, threshold=tau, lse=lse,
                             counters=counters, advance_seq_lens=True)
        ctx.step(args)
        torch.cuda.synchronize()
        assert st.seq_lens.item() == seq0[0] + k + 1          # advanced on the device
        np.testing.assert_allclose(scores.cpu().numpy(), ref.score, rtol=0, atol=gh.ATOL_SCORE)
        np.testing.assert_array_equal(flags.cpu().numpy(), ref.flags)
        gh.assert_close(out.cpu().numpy(), ref.out, gh.ATOL_OUT, f"step {k} out")
        gh.assert_close(lse.cpu().numpy(), ref.lse, gh.ATOL_LSE, f"step {k} lse")
        recalls += int(ref.flags[0])
    assert recalls == 2
    c = counters.cpu().numpy()
    assert c[0, 0] == wl.steps and c[0, 1] == 2
    assert ctx.read_device_status() == 0
    assert ctx.launch_count == wl.steps * 3   # Local, head, gated Full (which also advances seq_lens)


def _small_batched():
    L = 4
    return workloads.make("batched", L=L, B=5, windows=[64, 32, 64, 32], sinks=[4, 0, 4, 0],
                          gated=[1, 0, 1, 0], seq_lens0=np.array([100, 900, 33, 2500, 64], np.int32),
                          steps=4, head=(0, 1, 16))


def test_step_forms_agree_eager_host_graph():
    """Mixed-length batch, hybrid stack, shuffled tables: oda_step eager vs the oracle; the
    host-buffer entry point and a CUDA-graph replay give the same bits as eager."""
    wl = _small_batched()
    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    head = wl.head_host()
    B = wl.B
    shape = (wl.L, B, wl.Hq, wl.D)
    seq0 = np.asarray(wl.seq_lens0)
    ov_h = np.array([1, 0, 1, 1, 0], np.uint8)
    ov = torch.from_numpy(ov_h).cuda()
    q = workloads.q_device(wl, 0)

    def run_eager():
        out = torch.zeros(shape, device="cuda")
        lse = torch.zeros(shape[:3], device="cuda")
        scores = torch.zeros(B, device="cuda")
        flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
        args = ctx.step_args(B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens, out, scores, flags,
                             head=st.head, threshold=0.5, override_flags=ov, lse=lse)
        ctx.step(args)
        torch.cuda.synchronize()
        return out, lse, scores, flags

    out, lse, scores, flags = run_eager()
    ref = _oracle_step(wl, st.table_host, st.num_blocks, seq0, 0, head, 0.5, ov_h)
    gh.assert_close(out.cpu().numpy(), ref.out, gh.ATOL_OUT, "step out")
    gh.assert_close(lse.cpu().numpy(), ref.lse, gh.ATOL_LSE, "step lse")
    np.testing.assert_allclose(scores.cpu().numpy(), ref.score, rtol=0, atol=gh.ATOL_SCORE)
    np.testing.assert_array_equal(flags.cpu().numpy(), ov_h)

    # host-buffer form
    q_h = q.cpu().pin_memory()
    ov_p = torch.from_numpy(ov_h).pin_memory()
    out_h = torch.zeros(shape).pin_memory()
    lse_h = torch.zeros(shape[:3]).pin_memory()
    sc_h = torch.zeros(B).pin_memory()
    fl_h = torch.zeros(B, dtype=torch.uint8).pin_memory()
    args = ctx.step_args(B, q_h, st.k_cache, st.v_cache, st.block_table, st.seq_lens, out_h, sc_h, fl_h,
                         head=st.head, threshold=0.5, override_flags=ov_p, lse=lse_h)
    up, down = ctx.step_host(args)
    assert up == q_h.numel() * 2 + B and down == out_h.numel() * 4 + lse_h.numel() * 4 + B * 4 + B
    assert torch.equal(out_h, out.cpu()) and torch.equal(lse_h, lse.cpu()) and torch.equal(fl_h, flags.cpu())

    # graph replay vs eager: same bits, and the device-side advance makes replays walk the sequence
    g_out = torch.zeros(shape, device="cuda")
    g_scores = torch.zeros(B, device="cuda")
    g_flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    args = ctx.step_args(B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens, g_out, g_scores,
                         g_flags, head=st.head, threshold=0.5, override_flags=ov, advance_seq_lens=True)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(graph, stream=s):
            ctx.step(args, stream=s.cuda_stream)
    torch.cuda.synchronize()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(g_out, out)
    np.testing.assert_array_equal(st.seq_lens.cpu().numpy(), seq0 + 1)
    graph.replay()
    torch.cuda.synchronize()
    ref2 = _oracle_step(wl, st.table_host, st.num_blocks, seq0 + 1, 0, head, 0.5, ov_h)
    gh.assert_close(g_out.cpu().numpy(), ref2.out, gh.ATOL_OUT, "graph replay 2")
    assert ctx.read_device_status() == 0


@pytest.mark.parametrize("pinned", [True, False])
def test_host_step_without_a_head(pinned):
    """Head-less stack, forced flags.  With pinned buffers the kernels write every output in place
    over the bus, with pageable ones everything goes through staging copies: either way the
    host-buffer entry point gives the bits of the device-pointer one (which is checked against the
    oracle), twice in a row, scores and flags included."""
    from tests.helpers import make_problem
    L, Hq, Hkv, D = 3, 8, 2, 128
    seq = [700, 33, 1, 2100, 257]
    B = len(seq)
    windows, sinks, gated = [64, 32, 64], [4, 0, 4], [1, 0, 1]
    prob = make_problem(77, L, B, Hq, Hkv, D, seq)
    ctx = gh.make_ctx(prob, windows, sinks, gated)
    dev = gh.upload(prob)
    ov_h = np.array([1, 0, 1, 1, 0], np.uint8)
    out, lse = gh.new_out(prob)
    scores = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    ctx.step(ctx.step_args(B, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out, scores, flags,
                           override_flags=torch.from_numpy(ov_h).cuda(), lse=lse))
    torch.cuda.synchronize()
    ref = orc.step(prob["q"], None, prob["k"], prob["v"], prob["table"], prob["seq_lens"], num_kv_heads=Hkv,
                   block_size=16, layout=prob["layout"], layer_window=windows, layer_sinks=sinks, layer_gated=gated,
                   override_flags=ov_h, nthreads=4)
    gh.assert_close(out.cpu().numpy(), ref.out, gh.ATOL_OUT, "eager out")

    place = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    q_h = place(dev["q"].cpu())
    out_h = place(torch.full((L, B, Hq, D), 9.0))
    lse_h = place(torch.full((L, B, Hq), 9.0))
    sc_h, fl_h = place(torch.zeros(B)), place(torch.zeros(B, dtype=torch.uint8))
    lg_h = place(torch.full((B,), 9.0))
    ov_p = place(torch.from_numpy(ov_h.copy()))     # the argument block holds addresses, not references
    args = ctx.step_args(B, q_h, dev["k"], dev["v"], dev["table"], dev["seq_lens"], out_h, sc_h, fl_h,
                         override_flags=ov_p, lse=lse_h, logits=lg_h)
    for _ in range(2):
        up, down = ctx.step_host(args)
        assert up == q_h.numel() * 2 + B and down == out_h.numel() * 4 + lse_h.numel() * 4 + B * 4 + B * 4 + B
        assert torch.equal(out_h, out.cpu()) and torch.equal(lse_h, lse.cpu())
        np.testing.assert_array_equal(fl_h.numpy(), ov_h)
        assert torch.equal(sc_h, scores.cpu()) and (lg_h == 0).all()    # no head: score 0.5, logit 0
        out_h.fill_(9.0), lse_h.fill_(9.0), sc_h.fill_(9.0), fl_h.fill_(9), lg_h.fill_(9.0)
    assert ctx.read_device_status() == 0


def test_step_flag_invariants_on_device():
    wl = _small_batched()
    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    B, shape = wl.B, (wl.L, wl.B, wl.Hq, wl.D)
    q = workloads.q_device(wl, 1)
    loc = torch.zeros(shape, device="cuda")
    ctx.local_decode(0, wl.L, B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens, loc, None)
    res = {}
    for name, ov_h in (("zeros", np.zeros(B, np.uint8)), ("ones", np.ones(B, np.uint8))):
        out = torch.zeros(shape, device="cuda")
        scores = torch.zeros(B, device="cuda")
        flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
        ctx.step(ctx.step_args(B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens, out, scores,
                               flags, head=st.head, override_flags=torch.from_numpy(ov_h).cuda()))
        torch.cuda.synchronize()
        res[name] = out
    assert torch.equal(res["zeros"], loc)                           # all flags 0 => Local
    full = torch.zeros(shape, device="cuda")
    ctx.full_decode_gated(0, wl.L, B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens,
                          torch.ones(B, dtype=torch.uint8, device="cuda"), full, None)
    torch.cuda.synchronize()
    for l in range(wl.L):
        assert torch.equal(res["ones"][l], full[l] if wl.gated[l] else loc[l])  # all flags 1 => Full on gated layers


def test_remainder_only_gated_pass_equals_full():
    """Option 'reuse_local': the gated pass reads only S^F \\ S^L and merges with the Local result.
    With q_full == q_local that is Full attention: same oracle bar, and within rounding of the
    recompute-from-scratch path; requests whose window already covers everything are left alone."""
    L = 4
    wl = workloads.make("batched", L=L, B=6, windows=[64, 32, 64, 32], sinks=[4, 0, 4, 0], gated=[1, 0, 1, 0],
                        seq_lens0=np.array([100, 900, 33, 2500, 68, 69], np.int32), steps=2, head=(0, 1, 16))
    st = workloads.materialize(wl)
    head = wl.head_host()
    B, shape = wl.B, (wl.L, wl.B, wl.Hq, wl.D)
    ov_h = np.array([1, 1, 1, 0, 1, 1], np.uint8)
    ov = torch.from_numpy(ov_h).cuda()
    q = workloads.q_device(wl, 0)
    outs = {}
    for reuse in (0, 1):
        cfg = workloads.oda_config(wl, st.num_blocks, reuse_local=reuse)
        ctx = binding.OdaContext(cfg)
        out = torch.zeros(shape, device="cuda")
        lse = torch.zeros(shape[:3], device="cuda")
        scores = torch.zeros(B, device="cuda")
        flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
        for keep_lse in (True, False):   # the step keeps its own lse when the caller passes none
            ctx.step(ctx.step_args(B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens, out, scores, flags,
                                   head=st.head, override_flags=ov, lse=lse if keep_lse else None))
            torch.cuda.synchronize()
            outs[(reuse, keep_lse)] = (out.cpu().numpy().copy(), lse.cpu().numpy().copy())
        assert ctx.read_device_status() == 0
    ref = _oracle_step(wl, st.table_host, st.num_blocks, np.asarray(wl.seq_lens0), 0, head, 0.5, ov_h)
    for key, (o, l) in outs.items():
        gh.assert_close(o, ref.out, gh.ATOL_OUT, f"reuse={key}")
    gh.assert_close(outs[(1, True)][1], ref.lse, gh.ATOL_LSE, "merged lse")
    np.testing.assert_allclose(outs[(1, True)][0], outs[(0, True)][0], rtol=0, atol=1e-5)
    np.testing.assert_array_equal(outs[(1, False)][0], outs[(1, True)][0])


@pytest.mark.parametrize("first_k,expect", [(2, 126), (4, 252), (8, 504)])
def test_prescribed_schedule_counts_over_1008_routed_steps(first_k, expect):
    """The paper's timing protocol: Full on the first k of every 16 routed steps, 1,008 steps.  The
    device counters of one graph-replayed step (head still running, lengths advancing on the device)
    must read exactly 1,008 steps and 126 / 252 / 504 Full calls."""
    steps = 1008
    wl = workloads.make("tiny", seq_lens0=np.array([100], np.int32), steps=steps + 2, schedule="periodic")
    st = workloads.materialize(wl)
    ctx = binding.OdaContext(workloads.oda_config(wl, st.num_blocks))
    out = torch.zeros((wl.L, wl.B, wl.Hq, wl.D), device="cuda")
    scores = torch.zeros(wl.B, device="cuda")
    flags = torch.zeros(wl.B, dtype=torch.uint8, device="cuda")
    counters = torch.zeros((wl.B, 2), dtype=torch.int32, device="cuda")
    ov = torch.zeros(wl.B, dtype=torch.uint8, device="cuda")
    fe = torch.from_numpy(wl.feat_host(0)).cuda()
    q = workloads.q_device(wl, 0)
    args = ctx.step_args(wl.B, q, st.k_cache, st.v_cache, st.block_table, st.seq_lens, out, scores, flags,
                         feat_ext=fe, head=st.head, threshold=0.5, override_flags=ov, counters=counters,
                         advance_seq_lens=True)
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            ctx.step(args, stream=s.cuda_stream)
    sched = torch.from_numpy(np.stack([synth.periodic_flags(t, wl.B, first_k) for t in range(steps)])).cuda()
    for t in range(steps):
        ov.copy_(sched[t])
        g.replay()
    torch.cuda.synchronize()
    c = counters.cpu().numpy()
    assert c[0, 0] == steps and c[0, 1] == expect
    assert st.seq_lens.item() == 100 + steps
    assert ctx.read_device_status() == 0
