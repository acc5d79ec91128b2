"""Pins for the oracle's selected-state commit (Algorithm 1, line 8): the candidate K/V of the
current token lands at position seq_len-1 of the right requests and nowhere else; the selected
branch supplies output, hidden row and cache contents.  CPU only."""
import numpy as np

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import synth
from tests.helpers import dense_kv, make_problem, oracle_attention


def _cands(seed, L, B, Hkv, D):
    return (synth.gauss_bf16_tensor(seed, 40, (L, B, Hkv, D)), synth.gauss_bf16_tensor(seed, 41, (L, B, Hkv, D)))


def test_write_current_kv_touches_only_position_t_minus_1():
    seq = [17, 48, 5]
    for layout in ("hnd", "nhd"):
        prob = make_problem(3, 2, 3, 4, 2, 16, seq, layout=layout)
        k0, v0 = prob["k"].copy(), prob["v"].copy()
        kc, vc = _cands(3, 2, 3, 2, 16)
        mask = np.array([1, 0, 1], np.uint8)
        orc.write_current_kv(kc, vc, prob["k"], prob["v"], prob["table"], prob["seq_lens"], block_size=16,
                             layout=prob["layout"], mask=mask)
        changed_k = np.nonzero(prob["k"] != k0)[0]
        assert len(changed_k) <= 2 * 2 * 2 * 16           # layers x masked requests x heads x D
        for l in range(2):
            for b, t in enumerate(seq):
                for g in range(2):
                    rows_k = dense_kv(prob, prob["k"], l, b, g)
                    rows_v = dense_kv(prob, prob["v"], l, b, g)
                    old = dict(prob, k=k0, v=v0)
                    ok, ov = dense_kv(old, k0, l, b, g), dense_kv(old, v0, l, b, g)
                    np.testing.assert_array_equal(rows_k[:t - 1], ok[:t - 1])    # history untouched
                    np.testing.assert_array_equal(rows_v[:t - 1], ov[:t - 1])
                    if mask[b]:
                        np.testing.assert_array_equal(rows_k[t - 1], synth.bf16_bits_to_f32(kc[l, b, g]))
                        np.testing.assert_array_equal(rows_v[t - 1], synth.bf16_bits_to_f32(vc[l, b, g]))
                    else:
                        np.testing.assert_array_equal(rows_k[t - 1], ok[t - 1])
        # mask None writes every request
        orc.write_current_kv(kc, vc, prob["k"], prob["v"], prob["table"], prob["seq_lens"], block_size=16,
                             layout=prob["layout"])
        np.testing.assert_array_equal(dense_kv(prob, prob["k"], 1, 1, 0)[47], synth.bf16_bits_to_f32(kc[1, 1, 0]))


def test_select_rows():
    lo = np.arange(12, dtype=np.float32).reshape(3, 4)
    fu = -lo
    out = orc.select_rows(lo, fu, np.array([0, 1, 0], np.uint8))
    np.testing.assert_array_equal(out, np.stack([lo[0], fu[1], lo[2]]))


def test_step_with_commit_selected_branch_everywhere():
    L, B, Hq, Hkv, D = 2, 3, 4, 2, 16
    seq = [40, 70, 23]
    prob = make_problem(9, L, B, Hq, Hkv, D, seq)
    kl, vl = _cands(1, L, B, Hkv, D)
    kf, vf = _cands(2, L, B, Hkv, D)
    qf = synth.gauss_bf16_tensor(9, synth.STREAM_QFULL, (L, B, Hq, D))
    ov = np.array([1, 0, 1], np.uint8)
    hl = synth.gauss_f32_tensor(5, 1, (B, 6))
    hf = synth.gauss_f32_tensor(5, 2, (B, 6))
    windows, sinks, gated = [16, 16], [2, 2], [1, 1]
    r = orc.step_with_commit(prob["q"], qf, prob["k"], prob["v"], prob["table"], prob["seq_lens"],
                             k_cur_local=kl, v_cur_local=vl, k_cur_full=kf, v_cur_full=vf, num_kv_heads=Hkv,
                             block_size=16, layout=prob["layout"], layer_window=windows, layer_sinks=sinks,
                             layer_gated=gated, override_flags=ov, hidden_local=hl, hidden_full=hf)
    # independent check: build the two caches by hand and attend
    for b, t in enumerate(seq):
        for l in range(L):
            for g in range(Hkv):
                want_k = kf if ov[b] else kl
                np.testing.assert_array_equal(dense_kv(prob, prob["k"], l, b, g)[t - 1],
                                              synth.bf16_bits_to_f32(want_k[l, b, g]))
    np.testing.assert_array_equal(r.hidden, np.stack([hf[0], hl[1], hf[2]]))
    # the cache now holds the selected candidates: Full on it with q_full reproduces the flagged rows,
    alt = dict(prob, q=qf)
    full, _ = oracle_attention(alt, "full", windows, sinks)
    for b in range(B):
        if ov[b]:
            np.testing.assert_array_equal(r.out[:, b], full[:, b])
    # and the unflagged rows equal Local on the same cache (their candidate is the Local one)
    loc, _ = oracle_attention(prob, "local", windows, sinks)
    np.testing.assert_array_equal(r.out[:, 1], loc[:, 1])
    # the Local pass of a flagged request saw the LOCAL candidate, not the Full one
    assert np.abs(r.out_local[:, 0] - loc[:, 0]).max() > 1e-6
