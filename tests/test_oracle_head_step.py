"""Pins for the oracle's recall head, decision rule, and whole-step gating.  CPU only."""
import math

import numpy as np

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import synth
from tests.helpers import make_problem, oracle_attention
from tests.test_oracle_attention import golden


def test_head_hand_example():
    """x = [ln3, ln3], W1 = diag(1,-1): hidden = [ln3, -ln3]; SiLU(a) = a*sigmoid(a) gives
    [ln3*3/4, -ln3*1/4]; w2 = [2,2], b2 = 0 -> z = ln3, sigmoid(z) = 3/4."""
    x = np.array([[math.log(3.0), math.log(3.0)]], dtype=np.float64)
    W1 = np.array([[1, 0], [0, -1]], dtype=np.float32)
    z, s = orc.recall_head(None, x, W1, np.zeros(2, np.float32), np.array([2, 2], np.float32), 0.0)
    assert abs(z[0] - math.log(3.0)) < 1e-15 and abs(s[0] - 0.75) < 1e-15
    # the same numbers with the input split between the external and the attention part
    z2, s2 = orc.recall_head(x[:, :1].astype(np.float32), x[:, 1:], W1, np.zeros(2, np.float32),
                             np.array([2, 2], np.float32), 0.0)
    assert abs(z2[0] - z[0]) < 1e-7 and abs(s2[0] - 0.75) < 1e-7  # fp32 rounding of ln3 only
    # bias paths: b1 shifts the hidden pre-activation, b2 the logit
    z3, _ = orc.recall_head(None, np.zeros((1, 2)), W1, np.array([math.log(3.0), 0], np.float32),
                            np.array([4, 0], np.float32), 1.0)
    assert abs(z3[0] - (4 * np.float64(np.float32(math.log(3.0))) * 0.75 + 1.0)) < 1e-6


def test_head_zero_weights_and_monotone_in_b2():
    B, d = 3, 10
    x = synth.gauss_f32_tensor(1, synth.STREAM_FEAT, (B, d))
    W1 = np.zeros((4, d), np.float32)
    for b2 in (-2.0, 0.0, 0.7):
        z, s = orc.recall_head(x, None, W1, np.zeros(4, np.float32), np.ones(4, np.float32), b2)
        np.testing.assert_allclose(z, np.float32(b2), atol=0)
        np.testing.assert_allclose(s, 1 / (1 + math.exp(-float(np.float32(b2)))), atol=1e-15)
    W1 = synth.gauss_f32_tensor(2, synth.STREAM_W1, (4, d), std=0.5)
    prev = None
    for b2 in np.linspace(-3, 3, 7):
        _, s = orc.recall_head(x, None, W1, np.zeros(4, np.float32), np.ones(4, np.float32), b2)
        if prev is not None:
            assert (s > prev).all()
        prev = s


def test_head_matches_numpy_formula():
    B, de, da, dh = 4, 6, 10, 7
    fe = synth.gauss_f32_tensor(3, synth.STREAM_FEAT, (B, de))
    af = synth.gauss_f32_tensor(4, synth.STREAM_FEAT, (B, da)).astype(np.float64) * 1.3
    W1 = synth.gauss_f32_tensor(3, synth.STREAM_W1, (dh, de + da), std=0.3)
    b1 = synth.gauss_f32_tensor(3, synth.STREAM_B1, (dh,), std=0.3)
    w2 = synth.gauss_f32_tensor(3, synth.STREAM_W2, (dh,), std=0.3)
    b2 = np.float32(0.1)
    z, s = orc.recall_head(fe, af, W1, b1, w2, b2)
    x = np.concatenate([fe.astype(np.float64), af], axis=1)
    a = x @ W1.astype(np.float64).T + b1.astype(np.float64)
    zr = (a / (1 + np.exp(-a))) @ w2.astype(np.float64) + np.float64(b2)
    np.testing.assert_allclose(z, zr, rtol=0, atol=1e-13)
    np.testing.assert_allclose(s, 1 / (1 + np.exp(-zr)), rtol=0, atol=1e-14)
    # the order of the two input parts matters: swapping them changes the result
    z_sw, _ = orc.recall_head(fe, af, np.roll(W1, de, axis=1), b1, w2, b2)
    assert np.abs(z_sw - z).max() > 1e-6


def test_decision_rule():
    z = np.array([0.0, 1e-9, -1e-9, np.nan, np.inf, -np.inf, 5.0])
    score = 1 / (1 + np.exp(-z))
    f = orc.flags(z, score, 0.5)
    # strict '>': score == tau stays Local; every nonfinite logit (also -inf) goes to Full
    np.testing.assert_array_equal(f, [0, 1, 0, 1, 1, 1, 1])
    np.testing.assert_array_equal(orc.flags(z, score, 1.0), [0, 0, 0, 1, 1, 1, 0])
    ov = np.array([1, 0, 1, 0, 0, 0, 0], dtype=np.uint8)
    np.testing.assert_array_equal(orc.flags(z, score, 0.5, ov), ov)
    np.testing.assert_array_equal(orc.flags(None, None, 0.5, ov), ov)


def test_nan_feature_forces_full():
    x = np.array([[0.3, np.nan], [0.3, 0.1]], dtype=np.float32)
    W1 = np.ones((2, 2), np.float32)
    z, s = orc.recall_head(x, None, W1, np.zeros(2, np.float32), np.ones(2, np.float32), -50.0)
    np.testing.assert_array_equal(orc.flags(z, s, 0.5), [1, 0])


def _head(seed, d_in, d_h, std=0.02):
    return dict(W1=synth.gauss_f32_tensor(seed, synth.STREAM_W1, (d_h, d_in), std=std),
                b1=synth.gauss_f32_tensor(seed, synth.STREAM_B1, (d_h,), std=std),
                w2=synth.gauss_f32_tensor(seed, synth.STREAM_W2, (d_h,), std=std),
                b2=synth.gauss_f32_tensor(seed, synth.STREAM_B2, (1,), std=std)[0], use_attn_out=1)


def _step(prob, windows, sinks, gated, **kw):
    return orc.step(prob["q"], kw.pop("q_full", None), prob["k"], prob["v"], prob["table"],
                    prob["seq_lens"], num_kv_heads=prob["Hkv"], block_size=prob["P"],
                    layout=prob["layout"], layer_window=windows, layer_sinks=sinks,
                    layer_gated=gated, **kw)


def test_step_gating_invariants():
    L, B, Hq, Hkv, D = 4, 3, 4, 2, 16
    seq = [100, 31, 64]
    windows, sinks, gated = [16, 8, 16, 8], [4, 0, 4, 0], [1, 0, 1, 0]
    prob = make_problem(7, L, B, Hq, Hkv, D, seq)
    loc, _ = oracle_attention(prob, "local", windows, sinks)
    ful, _ = oracle_attention(prob, "full", windows, sinks)
    head = _head(7, 5 + Hq * D, 8)
    fe = synth.gauss_f32_tensor(7, synth.STREAM_FEAT, (B, 5))
    # all flags 0 => output == Local everywhere
    r0 = _step(prob, windows, sinks, gated, head=head, feat_ext=fe, override_flags=np.zeros(B, np.uint8))
    np.testing.assert_array_equal(r0.out, loc)
    np.testing.assert_array_equal(r0.out_local, loc)
    # all flags 1 => gated layers == Full, fixed-window layers == Local
    r1 = _step(prob, windows, sinks, gated, head=head, feat_ext=fe, override_flags=np.ones(B, np.uint8))
    for l in range(L):
        np.testing.assert_array_equal(r1.out[l], ful[l] if gated[l] else loc[l])
    # mixed flags select per request
    ov = np.array([1, 0, 1], np.uint8)
    rm = _step(prob, windows, sinks, gated, head=head, feat_ext=fe, override_flags=ov)
    for l in range(L):
        for b in range(B):
            np.testing.assert_array_equal(rm.out[l, b], ful[l, b] if (gated[l] and ov[b]) else loc[l, b])
    np.testing.assert_array_equal(rm.flags, ov)
    # the head sees [feat_ext ; Local output of the LAST gated layer (2)], also under an override
    z, s = orc.recall_head(fe, loc[2].reshape(B, -1), head["W1"], head["b1"], head["w2"], head["b2"])
    np.testing.assert_array_equal(rm.z, z)
    np.testing.assert_array_equal(rm.score, s)
    # without an override the flags come from the rule; a threshold between sorted scores splits them
    srt = np.sort(s)
    tau = 0.5 * (srt[0] + srt[1])
    rt = _step(prob, windows, sinks, gated, head=head, feat_ext=fe, tau=tau)
    np.testing.assert_array_equal(rt.flags, (s > tau).astype(np.uint8))
    assert rt.flags.sum() == B - 1
    for l in range(L):
        for b in range(B):
            np.testing.assert_array_equal(rt.out[l, b], ful[l, b] if (gated[l] and rt.flags[b]) else loc[l, b])


def test_step_full_uses_q_full_and_window_covering_everything():
    L, B, Hq, Hkv, D = 2, 2, 2, 1, 8
    prob = make_problem(9, L, B, Hq, Hkv, D, [20, 33])
    qf = synth.gauss_bf16_tensor(9, synth.STREAM_QFULL, (L, B, Hq, D))
    ones = np.ones(B, np.uint8)
    r = _step(prob, [4, 4], [1, 1], [1, 1], override_flags=ones, q_full=qf)
    alt = dict(prob, q=qf)
    ful, _ = oracle_attention(alt, "full", [4, 4], [1, 1])
    np.testing.assert_array_equal(r.out, ful)
    # window >= seq_len: flags do not matter
    ra = _step(prob, [64, 64], [0, 0], [1, 1], override_flags=ones)
    rb = _step(prob, [64, 64], [0, 0], [1, 1], override_flags=np.zeros(B, np.uint8))
    np.testing.assert_array_equal(ra.out, rb.out)


def test_prescribed_schedule_counts_match_paper():
    g = golden()
    for k, name in [(2, "full_calls_first2"), (4, "full_calls_first4"), (8, "full_calls_first8")]:
        calls = sum(int(synth.periodic_flags(t, 1, k, g["period"])[0]) for t in range(g["routed_steps"]))
        assert calls == g[name]
        assert calls / g["routed_steps"] == k / g["period"]


def test_bernoulli_flags_rates():
    for rate in (0.0, 0.1, 0.25, 0.5, 1.0):
        f = np.concatenate([synth.bernoulli_flags(20734, t, 16, rate) for t in range(512)])
        if rate in (0.0, 1.0):
            assert f.mean() == rate
        else:
            assert abs(f.mean() - rate) < 0.02
