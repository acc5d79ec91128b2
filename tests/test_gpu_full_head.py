"""GPU parity of the paper's full recall head (three towers, interaction vector, fusion, SwiGLU
blocks) against the fp64 oracle, at toy sizes and at the paper's 28,325,889-parameter size."""
import numpy as np
import pytest
import torch

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import binding, synth
from tests import gpu_helpers as gh
from tests.helpers import make_problem
from tests.test_oracle_full_head import _layout, _pack

pytestmark = pytest.mark.gpu


def _params(seed, dm, T, F, nb):
    parts = {}
    for i, (n, shp) in enumerate(_layout(dm, T, F, nb)):
        fan_in = shp[-1] if len(shp) == 2 else 1
        std = 1.0 / np.sqrt(fan_in) if len(shp) == 2 else 0.1
        parts[n] = synth.gauss_f32_tensor(seed, 200 + i, shp, std=std)
        if n.startswith("g") or n.startswith("bg"):
            parts[n] = (1.0 + parts[n]).astype(np.float32)
    return _pack(parts, dm, T, F, nb)


def _ctx():
    prob = make_problem(1, 1, 1, 1, 1, 64, [20])
    return gh.make_ctx(prob, [8], [0], [1])


def _fused_available(ctx):
    """The persistent variant needs a cooperative launch of one CTA per SM with 225 KB of shared memory."""
    dm, T, F, nb, B = 64, 32, 40, 1, 1
    p = torch.from_numpy(_params(1, dm, T, F, nb)).cuda()
    x = [torch.zeros((B, dm), device="cuda") for _ in range(3)]
    try:
        ctx.recall_score_full(B, p, T, F, nb, x[0], x[1], x[2], 0.5, None, torch.zeros(B, device="cuda"), None,
                              torch.zeros(B, dtype=torch.uint8, device="cuda"), variant=2)
        torch.cuda.synchronize()
        return True
    except binding.OdaError as e:
        if e.status == 2:
            return False
        raise


@pytest.mark.parametrize("dm,T,F,nb,B,variant", [
    (64, 32, 40, 2, 5, 0), (128, 64, 96, 1, 20, 0), (2048, 1024, 2048, 2, 4, 1),   # one launch per stage
    (2048, 1024, 2048, 2, 4, 2), (2048, 1024, 2048, 2, 1, 2),                      # persistent kernel, paper size
    (64, 32, 40, 2, 3, 2), (128, 64, 96, 0, 1, 2),                                 # fewer rows than CTAs, no blocks
    (4104, 24, 2052, 1, 2, 2)])                                                    # k longer than a ring slot, ragged
def test_full_head_parity(dm, T, F, nb, B, variant):
    ctx = _ctx()
    if variant == 2 and not _fused_available(ctx):
        pytest.skip("no cooperative launch of one CTA per SM on this device")
    params = _params(3, dm, T, F, nb)
    assert params.size == binding.load_library().oda_full_head_param_count(dm, T, F, nb)
    if (dm, T, F, nb) == (2048, 1024, 2048, 2):
        assert params.size == 28325889
    x = [synth.gauss_f32_tensor(4, i, (B, dm)) for i in range(3)]
    q, s = orc.full_head(params, *x, d_tower=T, d_ff=F, n_blocks=nb)
    srt = np.sort(s)
    tau = float(0.5 * (srt[B // 2 - 1] + srt[B // 2])) if B > 1 else 0.5
    scores = torch.zeros(B, device="cuda")
    logits = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    counters = torch.zeros((B, 2), dtype=torch.int32, device="cuda")
    pd = torch.from_numpy(params).cuda()
    xd = [torch.from_numpy(v).cuda() for v in x]
    scratch = None
    for _ in range(2):   # twice: tickets and scratch must be reusable
        scratch = ctx.recall_score_full(B, pd, T, F, nb, xd[0], xd[1], xd[2], tau, None, scores, logits, flags,
                                        counters, scratch=scratch, variant=variant)
    torch.cuda.synchronize()
    np.testing.assert_allclose(logits.cpu().numpy(), q, rtol=0, atol=1e-4)
    np.testing.assert_allclose(scores.cpu().numpy(), s, rtol=0, atol=2e-5)
    decided = np.abs(s - tau) >= gh.FLAG_BAND
    np.testing.assert_array_equal(flags.cpu().numpy()[decided], orc.flags(q, s, tau)[decided])
    c = counters.cpu().numpy()
    assert (c[:, 0] == 2).all() and (c[:, 1] == 2 * flags.cpu().numpy()).all()
    # forced flags: the head still runs
    ov = (np.arange(B) % 2).astype(np.uint8)
    ctx.recall_score_full(B, pd, T, F, nb, xd[0], xd[1], xd[2], tau, torch.from_numpy(ov).cuda(), scores, None,
                          flags, None, scratch=scratch, variant=variant)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(flags.cpu().numpy(), ov)
    np.testing.assert_allclose(scores.cpu().numpy(), s, rtol=0, atol=2e-5)


@pytest.mark.parametrize("dm,T,F,nb,B", [(64, 32, 40, 2, 5), (128, 64, 96, 1, 20), (2048, 1024, 2048, 2, 1),
                                          (2048, 1024, 2048, 2, 4), (4104, 24, 2052, 1, 2)])
def test_full_head_in_two_parts(dm, T, F, nb, B):
    """The part that needs only h_prev and emb first (its own call), then the rest on the same scratch:
    same scores as the oracle, flags exact outside the band, and the same bits on a second round."""
    ctx = _ctx()
    params = _params(3, dm, T, F, nb)
    x = [synth.gauss_f32_tensor(4, i, (B, dm)) for i in range(3)]
    q, s = orc.full_head(params, *x, d_tower=T, d_ff=F, n_blocks=nb)
    srt = np.sort(s)
    tau = float(0.5 * (srt[B // 2 - 1] + srt[B // 2])) if B > 1 else 0.5
    scores = torch.zeros(B, device="cuda")
    logits = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    pd = torch.from_numpy(params).cuda()
    xd = [torch.from_numpy(v).cuda() for v in x]
    scratch = ctx.full_head_scratch(B, dm, T, F, nb)
    scratch.fill_(0xFF)     # NaN patterns: nothing may be read before it is written
    # the Local hidden state does not exist yet when the first part runs: hand the second part a buffer
    # that is only filled in between
    h_local = torch.full_like(xd[2], float("nan"))
    rounds = []
    for _ in range(2):
        h_local.fill_(float("nan"))
        ctx.recall_score_full_pre(B, pd, T, F, nb, xd[0], xd[1], scratch)
        h_local.copy_(xd[2])
        ctx.recall_score_full(B, pd, T, F, nb, xd[0], xd[1], h_local, tau, None, scores, logits, flags,
                              scratch=scratch, variant=3)
        torch.cuda.synchronize()
        rounds.append(logits.clone())
    assert torch.equal(rounds[0], rounds[1])
    np.testing.assert_allclose(logits.cpu().numpy(), q, rtol=0, atol=1e-4)
    np.testing.assert_allclose(scores.cpu().numpy(), s, rtol=0, atol=2e-5)
    decided = np.abs(s - tau) >= gh.FLAG_BAND
    np.testing.assert_array_equal(flags.cpu().numpy()[decided], orc.flags(q, s, tau)[decided])
    assert ctx.read_device_status() == 0


def test_full_head_nonfinite_input_selects_full_and_bad_dims_are_refused():
    ctx = _ctx()
    dm, T, F, nb, B = 64, 32, 40, 1, 3
    params = torch.from_numpy(_params(5, dm, T, F, nb)).cuda()
    x = [torch.from_numpy(synth.gauss_f32_tensor(6, i, (B, dm))).cuda() for i in range(3)]
    x[2][1, 7] = float("nan")
    scores = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    ctx.recall_score_full(B, params, T, F, nb, x[0], x[1], x[2], 2.0, None, scores, None, flags)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(flags.cpu().numpy(), [0, 1, 0])   # threshold 2 is never exceeded; NaN forces Full
    with pytest.raises(binding.OdaError) as e:
        ctx.recall_score_full(B, params, 36, F, nb, x[0], x[1], x[2], 0.5, None, scores, None, flags)
    assert e.value.status == 2


def test_fused_head_graph_replay_is_bitwise_stable_and_forced_variant_limits():
    """The persistent kernel is captured in a CUDA graph (cooperative launch node) and replayed: the
    same bits every time, equal to the eager call.  Batch > 4 with the fused variant forced is refused."""
    ctx = _ctx()
    if not _fused_available(ctx):
        pytest.skip("no cooperative launch of one CTA per SM on this device")
    dm, T, F, nb, B = 2048, 1024, 2048, 2, 2
    pd = torch.from_numpy(_params(3, dm, T, F, nb)).cuda()
    xd = [torch.from_numpy(synth.gauss_f32_tensor(4, i, (B, dm))).cuda() for i in range(3)]
    scores = torch.zeros(B, device="cuda")
    logits = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    scratch = ctx.recall_score_full(B, pd, T, F, nb, xd[0], xd[1], xd[2], 0.5, None, scores, logits, flags, variant=2)
    torch.cuda.synchronize()
    eager = logits.clone()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            ctx.recall_score_full(B, pd, T, F, nb, xd[0], xd[1], xd[2], 0.5, None, scores, logits, flags,
                                  scratch=scratch, variant=2)
    for _ in range(3):
        logits.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(logits, eager)
    assert ctx.read_device_status() == 0
    x5 = [torch.zeros((5, dm), device="cuda") for _ in range(3)]
    with pytest.raises(binding.OdaError) as e:
        ctx.recall_score_full(5, pd, T, F, nb, x5[0], x5[1], x5[2], 0.5, None, torch.zeros(5, device="cuda"), None,
                              torch.zeros(5, dtype=torch.uint8, device="cuda"), variant=2)
    assert e.value.status == 2


def test_step_decides_with_the_papers_head():
    """oda_step with the paper's head in place of the two-layer one: Local pass, the head on the
    caller's hidden states, gated Full pass for the requests it flags -- against the oracle's head
    feeding the oracle's step, eager and as one CUDA graph."""
    L, B, Hq, Hkv, D = 3, 4, 8, 2, 128
    windows, sinks, gated = [64, 32, 64], [4, 0, 4], [1, 0, 1]
    prob = make_problem(77, L, B, Hq, Hkv, D, [100, 900, 33, 2500])
    dm, T, F, nb = 128, 64, 96, 2
    params = _params(8, dm, T, F, nb)
    x = [synth.gauss_f32_tensor(9, i, (B, dm)) for i in range(3)]
    q_ref, s_ref = orc.full_head(params, *x, d_tower=T, d_ff=F, n_blocks=nb)
    srt = np.sort(s_ref)
    tau = float(0.5 * (srt[1] + srt[2]))
    assert srt[2] - tau > 2 * gh.FLAG_BAND and tau - srt[1] > 2 * gh.FLAG_BAND
    want_flags = orc.flags(q_ref, s_ref, tau)
    assert want_flags.sum() == 2
    ref = orc.step(prob["q"], None, prob["k"], prob["v"], prob["table"], prob["seq_lens"], num_kv_heads=Hkv,
                   block_size=16, layout=prob["layout"], layer_window=windows, layer_sinks=sinks,
                   layer_gated=gated, override_flags=want_flags, nthreads=4)
    ctx = gh.make_ctx(prob, windows, sinks, gated)          # no two-layer head configured
    dev = gh.upload(prob)
    out, lse = gh.new_out(prob)
    scores = torch.zeros(B, device="cuda")
    logits = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    fh = dict(params=torch.from_numpy(params).cuda(), d_tower=T, d_ff=F, n_blocks=nb,
              h_prev=torch.from_numpy(x[0]).cuda(), emb=torch.from_numpy(x[1]).cuda(),
              h_local=torch.from_numpy(x[2]).cuda(), scratch=ctx.full_head_scratch(B, dm, T, F, nb))
    args = ctx.step_args(B, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out, scores, flags,
                         threshold=tau, lse=lse, logits=logits, full_head=fh)
    ctx.step(args)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(flags.cpu().numpy(), want_flags)
    np.testing.assert_allclose(scores.cpu().numpy(), s_ref, rtol=0, atol=2e-5)
    np.testing.assert_allclose(logits.cpu().numpy(), q_ref, rtol=0, atol=1e-4)
    gh.assert_close(out.cpu().numpy(), ref.out, gh.ATOL_OUT, "out")
    gh.assert_close(lse.cpu().numpy(), ref.lse, gh.ATOL_LSE, "lse")
    eager = out.clone()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            ctx.step(args, stream=s.cuda_stream)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager)
    assert ctx.read_device_status() == 0
    # the host-buffer form has no place for the head's device inputs
    with pytest.raises(binding.OdaError):
        ctx.step_host(args)
