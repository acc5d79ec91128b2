"""Pins for the oracle's attention: brute force, an independent library routine,
closed forms, the paper's set identities and invariants.  CPU only."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import synth
from tests.helpers import (brute_attention, dense_kv, full_set_1based, local_set_1based,
                           make_problem, oracle_attention)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = int(v)
    return out


@pytest.mark.parametrize("layout", ["hnd", "nhd"])
def test_brute_force_grid(layout):
    """Literal 1-based sets of Eq. 1, extended precision, no max subtraction."""
    seq = [1, 37, 80]
    prob = make_problem(11, L=2, B=3, Hq=4, Hkv=2, D=16, seq_lens=seq, layout=layout)
    for s, w in itertools.product([0, 1, 4, 17], [1, 5, 16, 33, 100]):
        out_l, lse_l = oracle_attention(prob, "local", [w, w], [s, s])
        out_f, lse_f = oracle_attention(prob, "full", [w, w], [s, s])
        for l, b, h in itertools.product(range(2), range(3), range(4)):
            t = seq[b]
            ref, rl = brute_attention(prob, l, b, h, local_set_1based(t, s, w))
            np.testing.assert_allclose(out_l[l, b, h], ref, rtol=0, atol=1e-12)
            assert abs(lse_l[l, b, h] - rl) < 1e-12
            ref, rl = brute_attention(prob, l, b, h, full_set_1based(t))
            np.testing.assert_allclose(out_f[l, b, h], ref, rtol=0, atol=1e-12)
            assert abs(lse_f[l, b, h] - rl) < 1e-12


def test_cardinality_of_local_set():
    for t, s, w in itertools.product(range(1, 40), [0, 1, 4, 9], [1, 3, 8, 50]):
        assert len(local_set_1based(t, s, w)) == min(t, s + w)


def test_against_masked_sdpa():
    """The 'independent materialized-window attention calculation' of the paper's own
    numerical checks: a library attention routine with a boolean mask, fp64."""
    seq = [70, 129]
    prob = make_problem(5, L=1, B=2, Hq=8, Hkv=2, D=32, seq_lens=seq, layout="nhd")
    s, w = 4, 24
    out_l, _ = oracle_attention(prob, "local", [w], [s])
    out_f, _ = oracle_attention(prob, "full", [w], [s])
    for b, t in enumerate(seq):
        for h in range(8):
            K = torch.from_numpy(dense_kv(prob, prob["k"], 0, b, h // 4))
            V = torch.from_numpy(dense_kv(prob, prob["v"], 0, b, h // 4))
            q = torch.from_numpy(synth.bf16_bits_to_f32(prob["q"][0, b, h]).astype(np.float64))
            mask = torch.zeros(1, t, dtype=torch.bool)
            for i in local_set_1based(t, s, w):
                mask[0, i - 1] = True
            o = torch.nn.functional.scaled_dot_product_attention(q[None, None], K[None], V[None], attn_mask=mask)
            np.testing.assert_allclose(out_l[0, b, h], o[0, 0].numpy(), rtol=0, atol=1e-10)
            o = torch.nn.functional.scaled_dot_product_attention(q[None, None], K[None], V[None])
            np.testing.assert_allclose(out_f[0, b, h], o[0, 0].numpy(), rtol=0, atol=1e-10)


def _set_row(prob, cache, kv_layer, b, j, g, values_f32):
    lay, P, D = prob["layout"], prob["P"], prob["D"]
    blk = int(prob["table"][b, j // P])
    off = kv_layer * lay.layer_stride + blk * lay.block_stride + (j % P) * lay.token_stride + g * lay.head_stride
    cache[off:off + D] = synth.f32_to_bf16_bits(np.asarray(values_f32, dtype=np.float32))


def test_closed_forms():
    D = 16
    # t = 1: the output is v_0 whatever q, s, w are
    prob = make_problem(3, L=1, B=1, Hq=2, Hkv=1, D=D, seq_lens=[1])
    out, lse = oracle_attention(prob, "local", [7], [2])
    v0 = dense_kv(prob, prob["v"], 0, 0, 0)[0]
    np.testing.assert_array_equal(out[0, 0, 0], v0)
    np.testing.assert_array_equal(out[0, 0, 1], v0)
    # q = 0: uniform weights -> the mean of V over the set, lse = ln |set|
    prob = make_problem(4, L=1, B=1, Hq=2, Hkv=1, D=D, seq_lens=[50])
    prob["q"][:] = 0
    s, w = 3, 10
    out, lse = oracle_attention(prob, "local", [w], [s])
    V = dense_kv(prob, prob["v"], 0, 0, 0)
    members = sorted(i - 1 for i in local_set_1based(50, s, w))
    np.testing.assert_allclose(out[0, 0, 0], V[members].mean(axis=0), rtol=0, atol=1e-14)
    assert abs(lse[0, 0, 0] - np.log(len(members))) < 1e-14
    out, lse = oracle_attention(prob, "full", [w], [s])
    np.testing.assert_allclose(out[0, 0, 0], V.mean(axis=0), rtol=0, atol=1e-14)
    # all keys equal: again the mean
    prob = make_problem(6, L=1, B=1, Hq=1, Hkv=1, D=D, seq_lens=[33])
    for j in range(33):
        _set_row(prob, prob["k"], 0, 0, j, 0, np.linspace(-1, 1, D))
    out, _ = oracle_attention(prob, "full", [8], [0])
    np.testing.assert_allclose(out[0, 0, 0], dense_kv(prob, prob["v"], 0, 0, 0).mean(axis=0), atol=1e-13, rtol=0)
    # V constant: the output is that constant
    for j in range(33):
        _set_row(prob, prob["v"], 0, 0, j, 0, np.full(D, 1.5))
    prob["k"] = synth.gauss_bf16_tensor(99, synth.STREAM_K, prob["k"].shape)
    out, _ = oracle_attention(prob, "local", [8], [2])
    np.testing.assert_allclose(out[0, 0, 0], np.full(D, 1.5), atol=1e-14, rtol=0)


def test_key_shift_invariance():
    """Adding one vector c to every key adds the constant q.c to every logit: the softmax
    weights, hence the output, do not change; lse moves by scale * q.c.  Small-integer
    keys keep k + c exact in bf16."""
    D, t = 8, 21
    prob = make_problem(8, L=1, B=1, Hq=1, Hkv=1, D=D, seq_lens=[t])
    rng = np.random.RandomState(0)
    keys = rng.randint(-2, 3, size=(t, D)).astype(np.float32)
    c = rng.randint(-3, 4, size=D).astype(np.float32)
    qv = rng.randint(-2, 3, size=D).astype(np.float32)
    prob["q"][0, 0, 0] = synth.f32_to_bf16_bits(qv)
    for j in range(t):
        _set_row(prob, prob["k"], 0, 0, j, 0, keys[j])
    o1, l1 = oracle_attention(prob, "local", [9], [2])
    for j in range(t):
        _set_row(prob, prob["k"], 0, 0, j, 0, keys[j] + c)
    o2, l2 = oracle_attention(prob, "local", [9], [2])
    np.testing.assert_allclose(o1, o2, rtol=0, atol=1e-13)
    assert abs((l2 - l1)[0, 0, 0] - float(qv @ c) / np.sqrt(D)) < 1e-12


def test_needle_inside_and_outside_the_local_set():
    """A key with a dominant logit at position s (1-based: the last sink) is seen by Local;
    one position later it is outside Local once t > s + w, and only Full sees it."""
    D, t, s, w = 16, 64, 4, 16
    for needle_pos_1based, local_sees in [(s, True), (s + 1, False)]:
        prob = make_problem(21, L=1, B=1, Hq=1, Hkv=1, D=D, seq_lens=[t])
        prob["q"][0, 0, 0] = synth.f32_to_bf16_bits(np.full(D, 4.0, dtype=np.float32))
        for j in range(t):
            _set_row(prob, prob["k"], 0, 0, j, 0, np.zeros(D))
        _set_row(prob, prob["k"], 0, 0, needle_pos_1based - 1, 0, np.full(D, 4.0))  # logit 64
        V = dense_kv(prob, prob["v"], 0, 0, 0)
        o_l, _ = oracle_attention(prob, "local", [w], [s])
        o_f, _ = oracle_attention(prob, "full", [w], [s])
        needle_v = V[needle_pos_1based - 1]
        np.testing.assert_allclose(o_f[0, 0, 0], needle_v, atol=1e-20 + 1e-12)
        if local_sees:
            np.testing.assert_allclose(o_l[0, 0, 0], needle_v, atol=1e-12)
        else:
            members = sorted(i - 1 for i in local_set_1based(t, s, w))
            np.testing.assert_allclose(o_l[0, 0, 0], V[members].mean(axis=0), atol=1e-13)


def test_paper_set_identity_2052_2053():
    """Paper: with s=4, w=2048 Local and Full coincide through position 2,052 and first
    differ at 2,053."""
    g = golden()
    s, w = g["sinks"], g["window"]
    assert s + w == g["last_coinciding_position"]
    for t in (g["last_coinciding_position"], g["first_differing_position"]):
        assert (local_set_1based(t, s, w) == full_set_1based(t)) == (t <= g["last_coinciding_position"])
        prob = make_problem(31, L=1, B=1, Hq=2, Hkv=1, D=8, seq_lens=[t])
        o_l, l_l = oracle_attention(prob, "local", [w], [s])
        o_f, l_f = oracle_attention(prob, "full", [w], [s])
        if t <= g["last_coinciding_position"]:
            np.testing.assert_array_equal(o_l, o_f)
            np.testing.assert_array_equal(l_l, l_f)
        else:
            assert np.abs(o_l - o_f).max() > 1e-9
            assert len(full_set_1based(t) - local_set_1based(t, s, w)) == 1
    # at most 2,051 committed positions + the current one are visible to Local
    assert max(len(local_set_1based(t, s, w)) for t in (2052, 2053, 5000, 100000)) - 1 == g["max_committed_local_positions"]
    assert g["ring_recent_positions"] == w - 1
    assert g["local_max_blocks"] * g["local_block_positions"] >= s + w


def test_window_covering_sequence_gives_full():
    seq = [5, 40, 64]
    prob = make_problem(41, L=1, B=3, Hq=4, Hkv=4, D=16, seq_lens=seq)
    for w in (64, 65, 1000):
        o_l, l_l = oracle_attention(prob, "local", [w], [0])
        o_f, l_f = oracle_attention(prob, "full", [w], [0])
        np.testing.assert_array_equal(o_l, o_f)
        np.testing.assert_array_equal(l_l, l_f)


def test_invariants_superset_range_permutation_merge():
    seq = [90, 47]
    s, w = 4, 20
    prob = make_problem(51, L=2, B=2, Hq=4, Hkv=2, D=16, seq_lens=seq, shuffled=False)
    o_l, l_l = oracle_attention(prob, "local", [w, w], [s, s])
    o_f, l_f = oracle_attention(prob, "full", [w, w], [s, s])
    assert (l_f >= l_l).all()  # Full's set contains Local's
    for l, b, h in itertools.product(range(2), range(2), range(4)):
        V = dense_kv(prob, prob["v"], l, b, h // 2)
        mem = sorted(i - 1 for i in local_set_1based(seq[b], s, w))
        assert (o_l[l, b, h] <= V[mem].max(axis=0) + 1e-15).all()
        assert (o_l[l, b, h] >= V[mem].min(axis=0) - 1e-15).all()
        # merging Local's partial with the partial over Full \ Local reproduces Full
        rest = full_set_1based(seq[b]) - local_set_1based(seq[b], s, w)
        o_r, l_r = brute_attention(prob, l, b, h, rest)
        m = max(l_l[l, b, h], l_r)
        wl, wr = np.exp(l_l[l, b, h] - m), np.exp(l_r - m)
        merged = (wl * o_l[l, b, h] + wr * o_r) / (wl + wr)
        np.testing.assert_allclose(merged, o_f[l, b, h], rtol=0, atol=1e-12)
        assert abs(m + np.log(wl + wr) - l_f[l, b, h]) < 1e-12
    # the same logical content under a permuted physical placement gives the same bits
    perm = make_problem(51, L=2, B=2, Hq=4, Hkv=2, D=16, seq_lens=seq, shuffled=True)
    lay, P, D = prob["layout"], 16, 16
    for l in range(2):
        for b in range(2):
            for pg in range((seq[b] + P - 1) // P):
                src, dst = int(prob["table"][b, pg]), int(perm["table"][b, pg])
                so = l * lay.layer_stride + src * lay.block_stride
                do = l * lay.layer_stride + dst * lay.block_stride
                perm["k"][do:do + lay.block_stride] = prob["k"][so:so + lay.block_stride]
                perm["v"][do:do + lay.block_stride] = prob["v"][so:so + lay.block_stride]
    perm["q"] = prob["q"]
    o_p, l_p = oracle_attention(perm, "local", [w, w], [s, s])
    np.testing.assert_array_equal(o_p, o_l)
    np.testing.assert_array_equal(l_p, l_l)


def test_gqa_mapping_and_layer_kv_index():
    """Query head h reads KV head h // G; layer_kv_index redirects a layer's cache slice."""
    prob = make_problem(61, L=3, B=1, Hq=6, Hkv=3, D=8, seq_lens=[30], kv_layers=2)
    kvmap = [1, 0, 1]
    out, lse = oracle_attention(prob, "local", [12] * 3, [1] * 3, layer_kv_index=kvmap)
    for l in range(3):
        for h in range(6):
            ref, rl = brute_attention(prob, l, 0, h, local_set_1based(30, 1, 12), kv_layer=kvmap[l])
            np.testing.assert_allclose(out[l, 0, h], ref, atol=1e-12, rtol=0)


def test_layer_range_mask_and_threads():
    prob = make_problem(71, L=3, B=3, Hq=2, Hkv=1, D=8, seq_lens=[9, 33, 17])
    full, _ = oracle_attention(prob, "local", [5, 6, 7], [1, 0, 2])
    part, _ = oracle_attention(prob, "local", [5, 6, 7], [1, 0, 2], layer_begin=1, layer_end=2,
                               request_mask=np.array([1, 0, 1], dtype=np.uint8), nthreads=4)
    assert np.isnan(part[0]).all() and np.isnan(part[2]).all() and np.isnan(part[1, 1]).all()
    np.testing.assert_array_equal(part[1, 0], full[1, 0])
    np.testing.assert_array_equal(part[1, 2], full[1, 2])
    par, _ = oracle_attention(prob, "local", [5, 6, 7], [1, 0, 2], nthreads=4)
    np.testing.assert_array_equal(par, full)


def test_custom_scale():
    prob = make_problem(81, L=1, B=1, Hq=1, Hkv=1, D=8, seq_lens=[12])
    out, lse = oracle_attention(prob, "full", [4], [0], sm_scale=0.37)
    ref, rl = brute_attention(prob, 0, 0, 0, full_set_1based(12), sm_scale=0.37)
    np.testing.assert_allclose(out[0, 0, 0], ref, atol=1e-13, rtol=0)
    assert abs(lse[0, 0, 0] - rl) < 1e-13
