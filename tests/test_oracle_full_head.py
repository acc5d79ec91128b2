"""Pins for the oracle's version of the paper's recall head: the printed parameter count, closed
forms, and an independent small-dimension computation written out term by term.  CPU only."""
import math

import numpy as np

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import synth
from tests.test_oracle_attention import golden


def test_parameter_count_is_the_papers():
    g = golden()
    n = orc.full_head_param_count(g["head_d_model"], g["head_d_tower"], g["head_d_ff"], g["head_blocks"])
    assert n == g["head_parameters"]
    assert 9 * g["head_d_tower"] == g["head_interaction_dim"]
    # the pieces: a biased down projection or biased gate/up would not give the printed number
    tower = 2048 + 2048 * 1024 + 1024
    assert n == 3 * tower + (1024 * 9216 + 1024) + 2 * (1024 + 3 * 2048 * 1024) + (1024 + 1024 + 1)


def _layout(dm, T, F, nb):
    """(name, shape) in storage order."""
    out = []
    for i in range(3):
        out += [(f"g{i}", (dm,)), (f"W{i}", (T, dm)), (f"b{i}", (T,))]
    out += [("Wf", (T, 9 * T)), ("bf", (T,))]
    for k in range(nb):
        out += [(f"bg{k}", (T,)), (f"Wg{k}", (F, T)), (f"Wu{k}", (F, T)), (f"Wd{k}", (T, F))]
    out += [("go", (T,)), ("w", (T,)), ("bias", (1,))]
    return out


def _pack(parts, dm, T, F, nb):
    return np.concatenate([np.asarray(parts[n], np.float32).reshape(-1) for n, _ in _layout(dm, T, F, nb)])


def _random_parts(seed, dm, T, F, nb, std=0.3):
    parts = {}
    for i, (n, shp) in enumerate(_layout(dm, T, F, nb)):
        parts[n] = synth.gauss_f32_tensor(seed, 100 + i, shp, std=std)
        if n.startswith("g") or n.startswith("bg"):
            parts[n] = (1.0 + parts[n]).astype(np.float32)
    return parts


def test_zero_weights_closed_forms():
    dm, T, F, nb, B = 6, 4, 5, 2, 3
    parts = {n: np.zeros(s, np.float32) for n, s in _layout(dm, T, F, nb)}
    for n in parts:
        if n.startswith("g") or n.startswith("bg"):
            parts[n][:] = 1.0
    parts["bias"][0] = 0.37
    x = [synth.gauss_f32_tensor(1, i, (B, dm)) for i in range(3)]
    q, s = orc.full_head(_pack(parts, dm, T, F, nb), *x, d_tower=T, d_ff=F, n_blocks=nb)
    # a = b = c = SiLU(0) = 0 -> u = 0 -> z0 = SiLU(0)/2 = 0 -> blocks add 0 -> q = bias
    np.testing.assert_allclose(q, np.float32(0.37), atol=1e-15)
    np.testing.assert_allclose(s, 1 / (1 + math.exp(-float(np.float32(0.37)))), atol=1e-15)
    # tower biases only: a = b = c = SiLU(b_i); with W_f = 0: z0 = (a+b+c)/2; w picks one coordinate
    parts["b0"][:] = 1.0
    parts["b1"][:] = 2.0
    parts["b2"][:] = -1.0
    parts["w"][2] = 1.0
    silu = lambda t: t / (1 + math.exp(-t))
    z0 = 0.5 * (silu(1.0) + silu(2.0) + silu(-1.0))
    q, _ = orc.full_head(_pack(parts, dm, T, F, nb), *x, d_tower=T, d_ff=F, n_blocks=nb, eps=0.0)
    # z is the constant vector z0: RMSNorm of a constant vector is sign(z0) in every coordinate
    np.testing.assert_allclose(q, np.float32(0.37) + math.copysign(1.0, z0), atol=1e-12)


def test_small_head_term_by_term():
    dm, T, F, nb, B = 5, 3, 4, 2, 2
    parts = _random_parts(7, dm, T, F, nb)
    x = [synth.gauss_f32_tensor(2, i, (B, dm)) for i in range(3)]
    eps = 1e-6
    q, s = orc.full_head(_pack(parts, dm, T, F, nb), *x, d_tower=T, d_ff=F, n_blocks=nb, eps=eps)
    P = {k: v.astype(np.float64) for k, v in parts.items()}
    silu = lambda t: t / (1.0 + np.exp(-t))
    rms = lambda v, g: v / np.sqrt(np.mean(v * v) + eps) * g
    for b in range(B):
        abc = [silu(P[f"W{i}"] @ rms(x[i][b].astype(np.float64), P[f"g{i}"]) + P[f"b{i}"]) for i in range(3)]
        a, bb, c = abc
        u = np.concatenate([a, bb, c, a * bb, np.abs(a - bb), a * c, np.abs(a - c), bb * c, np.abs(bb - c)])
        z = 0.5 * (a + bb + c + silu(P["Wf"] @ u + P["bf"]))
        for k in range(nb):
            n = rms(z, P[f"bg{k}"])
            z = z + P[f"Wd{k}"] @ (silu(P[f"Wg{k}"] @ n) * (P[f"Wu{k}"] @ n))
        want = float(P["w"] @ rms(z, P["go"]) + P["bias"][0])
        assert abs(q[b] - want) < 1e-12
        assert abs(s[b] - 1 / (1 + math.exp(-want))) < 1e-14
    # the three inputs are not interchangeable, nor are gate and up
    q_sw, _ = orc.full_head(_pack(parts, dm, T, F, nb), x[1], x[0], x[2], d_tower=T, d_ff=F, n_blocks=nb, eps=eps)
    assert np.abs(q_sw - q).max() > 1e-6
    swapped = dict(parts, Wg0=parts["Wu0"], Wu0=parts["Wg0"])
    q_gu, _ = orc.full_head(_pack(swapped, dm, T, F, nb), *x, d_tower=T, d_ff=F, n_blocks=nb, eps=eps)
    assert np.abs(q_gu - q).max() > 1e-6


# ---------------------------------------------------------------------------------------------
# Hand pins.  Every expected number below was worked out on paper from the definitions in the
# paper's appendix "Recall-head architecture" and typed in as a decimal; nothing here evaluates
# the head's formula a second time.  Two identities keep the arithmetic hand-sized:
#   sigmoid(ln k) = k / (k + 1),  so  SiLU(ln 3) = 3/4 ln 3,  SiLU(-ln 3) = -1/4 ln 3,
#   SiLU(ln 2) = 2/3 ln 2,  SiLU(ln 4) = 4/5 ln 4,  SiLU(-ln 4) = -1/5 ln 4,  SiLU(ln 5) = 5/6 ln 5;
#   SiLU(x) - SiLU(-x) = x  exactly (x sigmoid(x) + x sigmoid(-x) = x).
# The scalar output is q = w . RMSNorm(z) + bias, so with bias 0, unit output gain and w = e_j the
# two calls j = 0, 1 return z_0 / r and z_1 / r with the same r: their ratio is z_0 / z_1.
LN2, LN3, LN5 = math.log(2.0), math.log(3.0), math.log(5.0)


def _hand_towers():
    """Towers (d_model 4 -> d_tower 2) whose outputs are closed forms.  eps = 0 throughout.
    tower 0: x = (2,-2,2,-2): rms 2 -> (1,-1,1,-1); gain (ln3, ln2, 2ln2, 7) -> n = (ln3,-ln2,2ln2,-7);
             W = [[1,0,0,0],[0,1,1,0]], bias 0 -> pre = (ln3, -ln2 + 2ln2 = ln2) -> a = (3/4 ln3, 2/3 ln2)
    tower 1: x = (3,3,-3,3): rms 3 -> (1,1,-1,1); gain (ln4,1,1,1) -> n = (ln4,1,-1,1);
             W = [[-1,0,0,0],[0,0,0,0]], bias (0,-ln3) -> pre = (-ln4, -ln3) -> b = (-1/5 ln4, -1/4 ln3)
    tower 2: x = (0,0,0,5): mean square 25/4, rms 5/2 -> (0,0,0,2); gain (1,1,1,1/2) -> n = (0,0,0,1);
             W = [[0,0,0,ln5],[0,0,0,ln4]], bias 0 -> pre = (ln5, ln4) -> c = (5/6 ln5, 4/5 ln4)"""
    parts = {
        "g0": [LN3, LN2, 2 * LN2, 7.0], "W0": [[1, 0, 0, 0], [0, 1, 1, 0]], "b0": [0, 0],
        "g1": [2 * LN2, 1, 1, 1], "W1": [[-1, 0, 0, 0], [0, 0, 0, 0]], "b1": [0, -LN3],
        "g2": [1, 1, 1, 0.5], "W2": [[0, 0, 0, LN5], [0, 0, 0, 2 * LN2]], "b2": [0, 0],
    }
    x = [np.array([[2, -2, 2, -2]], np.float32), np.array([[3, 3, -3, 3]], np.float32),
         np.array([[0, 0, 0, 5]], np.float32)]
    return parts, x


# a = ( 0.8239592165010823,  0.4620981203732969)
# b = (-0.2772588722239781, -0.2746530721670274)
# c = ( 1.3411982603617503,  1.1090354888959125)
# The interaction vector in the paper's order [a; b; c; a.b; |a-b|; a.c; |a-c|; b.c; |b-c|],
# two coordinates per segment, multiplied / subtracted by hand from the six numbers above:
U_HAND = [
    0.8239592165010823, 0.4620981203732969,      # a
    -0.2772588722239781, -0.2746530721670274,    # b
    1.3411982603617503, 1.1090354888959125,      # c
    -0.2284500031256427, -0.1269166684031348,    # a . b
    1.1012180887250604, 0.7367511925403243,      # |a - b|
    1.1050926677802820, 0.5124832148460815,      # a . c
    0.5172390438606680, 0.6469373685226156,      # |a - c|
    -0.3718591170966603, -0.3046000041675236,    # b . c
    1.6184571325857284, 1.3836885610629399,      # |b - c|
]
S0_HAND = 1.8878986046388545   # a_0 + b_0 + c_0
S1_HAND = 1.2964805371021819   # a_1 + b_1 + c_1


def _ratio(parts, x, dm, T, F, nb, eps):
    """z_0 / z_1 of the state that enters the final RMSNorm (unit gain, bias 0, w = e_0 then e_1)."""
    qs = []
    for j in range(2):
        p = dict(parts, go=[1.0] * T, w=[1.0 if k == j else 0.0 for k in range(T)], bias=[0.0])
        q, _ = orc.full_head(_pack(p, dm, T, F, nb), *x, d_tower=T, d_ff=F, n_blocks=nb, eps=eps)
        qs.append(float(q[0]))
    return qs[0] / qs[1]


def test_hand_towers_feed_the_sum():
    # W_f = 0, b_f = 0: z0 = (a + b + c + SiLU(0)) / 2 = (S0, S1) / 2, so z0_0 / z0_1 = S0 / S1
    parts, x = _hand_towers()
    parts.update(Wf=np.zeros((2, 18)), bf=[0, 0])
    assert abs(_ratio(parts, x, 4, 2, 3, 0, 0.0) - 1.4561719598649555) < 2e-6   # S0 / S1 by hand
    # the three inputs are tied to their towers: exchanging h_prev and the embedding changes a and b
    assert abs(_ratio(parts, [x[1], x[0], x[2]], 4, 2, 3, 0, 0.0) - 1.4561719598649555) > 1e-2


def test_hand_interaction_vector_order_by_one_hot_rows():
    # One row of W_f is +e_k or -e_k, the other row and b_f are zero.  With the probe in row 0:
    #   z0_0 = (S0 + SiLU(+-u_k)) / 2,  z0_1 = S1 / 2   ->   R(+) - R(-) = u_k / S1
    # and with the probe in row 1 the same holds for 1/R with S0.  This reads u_k itself out of the
    # oracle, coordinate by coordinate, and compares it with the hand table: any reordering of the
    # nine segments, a transposed W_f or a product taken for a difference fails it.
    parts, x = _hand_towers()
    got = []
    for k in range(18):
        row = k % 2   # also alternate the row, so that the row index of W_f is pinned
        r = {}
        for sign in (+1.0, -1.0):
            Wf = np.zeros((2, 18))
            Wf[row, k] = sign
            p = dict(parts, Wf=Wf, bf=[0, 0])
            r[sign] = _ratio(p, x, 4, 2, 3, 0, 0.0)
        got.append((r[1.0] - r[-1.0]) * S1_HAND if row == 0 else (1 / r[1.0] - 1 / r[-1.0]) * S0_HAND)
    np.testing.assert_allclose(got, U_HAND, atol=2e-6, rtol=0)   # fp32 storage of ln 2, ln 3, ln 5
    # all 18 hand values are distinct, so no two positions can be exchanged unnoticed
    assert len({round(v, 6) for v in U_HAND}) == 18


def test_hand_fusion_bias_and_half():
    # towers silent (zero weights and biases: a = b = c = 0, u = 0): z0 = SiLU(b_f) / 2.
    parts = {n: np.zeros(s, np.float32) for n, s in _layout(4, 2, 3, 0)}
    for n in ("g0", "g1", "g2"):
        parts[n][:] = 1.0
    x = [np.ones((1, 4), np.float32)] * 3
    # b_f = (ln 3, ln 2): z0 = (3/8 ln 3, 1/3 ln 2); ratio 9 ln 3 / (8 ln 2) = 1.7830828133113007
    parts["bf"][:] = [LN3, LN2]
    assert abs(_ratio(parts, x, 4, 2, 3, 0, 0.0) - 1.7830828133113007) < 2e-6
    # b_f = (60, 80): SiLU(x) = x (1 - 1/(1 + e^x)) is x to 1e-24 here, so z0 = (30, 40); with
    # eps = 350 the final norm divides by sqrt((900 + 1600)/2 + 350) = 40: n = (3/4, 1).
    parts["bf"][:] = [60.0, 80.0]
    parts.update(go=[3.0, -2.0], w=[1.0, 1.0], bias=[0.25])
    q, s = orc.full_head(_pack(parts, 4, 2, 3, 0), *x, d_tower=2, d_ff=3, n_blocks=0, eps=350.0)
    assert abs(q[0] - (3.0 * 0.75 - 2.0 * 1.0 + 0.25)) < 1e-12          # = 0.5
    # eps is added to the mean square, not to the sum and not outside the root: eps = 0 gives
    # n = (30, 40) / sqrt(1250) = (3 sqrt2 / 5, 4 sqrt2 / 5) and q = sqrt2 (9/5 - 8/5) + 1/4
    q, _ = orc.full_head(_pack(parts, 4, 2, 3, 0), *x, d_tower=2, d_ff=3, n_blocks=0, eps=0.0)
    assert abs(q[0] - (0.2 * math.sqrt(2.0) + 0.25)) < 1e-12
    # score = sigmoid(q): w = 0, bias = ln 3 -> 3/4
    parts.update(w=[0.0, 0.0], bias=[LN3])
    _, s = orc.full_head(_pack(parts, 4, 2, 3, 0), *x, d_tower=2, d_ff=3, n_blocks=0, eps=0.0)
    assert abs(s[0] - 0.75) < 1e-7


def _hand_block():
    """One SwiGLU block (d_tower 2, d_ff 3) entered with z = (30, 40) and eps = 350:
      RMSNorm: (30, 40) / 40 = (3/4, 1), gain (2, 1/2)              -> n    = (3/2, 1/2)
      W_gate = [[2/3 ln3, 0], [0, -2 ln3], [2/3 ln2, 0]]            -> gate = (ln3, -ln3, ln2)
      SiLU(gate)                                                    =  (3/4 ln3, -1/4 ln3, 2/3 ln2)
      W_up   = [[2, 4], [1, -1], [0, 6]]                            -> up   = (5, 1, 3)
      SiLU(gate) . up                                               =  (15/4 ln3, -1/4 ln3, 2 ln2)
      W_down = [[1, 2, -1], [-1, 3, 1/2]]   -> (15/4 - 1/2) ln3 - 2 ln2,  (-15/4 - 3/4) ln3 + ln2
      z'     = (30 + 13/4 ln3 - 2 ln2,  40 - 9/2 ln3 + ln2) = (32.18419557705147, 35.74939188155345)
    SiLU on `up` instead of `gate` would give SiLU(5) ln3 ... instead; a unit block gain n = (3/4, 1)."""
    return {"bg": [2.0, 0.5], "Wg": [[2 * LN3 / 3, 0], [0, -2 * LN3], [2 * LN2 / 3, 0]],
            "Wu": [[2, 4], [1, -1], [0, 6]], "Wd": [[1, 2, -1], [-1, 3, 0.5]]}


def _silent_towers_z0_30_40(nb):
    parts = {n: np.zeros(s, np.float32) for n, s in _layout(4, 2, 3, nb)}
    for n in ("g0", "g1", "g2"):
        parts[n][:] = 1.0
    parts["bf"][:] = [60.0, 80.0]
    return parts, [np.ones((1, 4), np.float32)] * 3


def test_hand_swiglu_block():
    blk = _hand_block()
    parts, x = _silent_towers_z0_30_40(1)
    parts.update(bg0=blk["bg"], Wg0=blk["Wg"], Wu0=blk["Wu"], Wd0=blk["Wd"])
    # z'_0 / z'_1 = 32.18419557705147 / 35.74939188155345
    assert abs(_ratio(parts, x, 4, 2, 3, 1, 350.0) - 0.9002725328499472) < 1e-7
    # and the value itself through the final norm (eps = 350 again):
    #   r = sqrt((32.184...^2 + 35.749...^2)/2 + 350) = 38.81907691356647;  z'_0 / r = 0.8290819394987661
    p = dict(parts, go=[1.0, 1.0], w=[1.0, 0.0], bias=[0.0])
    q, _ = orc.full_head(_pack(p, 4, 2, 3, 1), *x, d_tower=2, d_ff=3, n_blocks=1, eps=350.0)
    assert abs(q[0] - 0.8290819394987661) < 1e-7
    # no block: the residual stream is untouched, ratio 30 / 40
    parts0, _ = _silent_towers_z0_30_40(0)
    assert abs(_ratio(parts0, x, 4, 2, 3, 0, 350.0) - 0.75) < 1e-12


def test_hand_two_blocks_each_read_their_own_parameters():
    # A block whose down projection is zero leaves z alone whatever its gate / up weights are.
    # Put the hand block first and such a block second, then the other way round: both must give
    # the one-block result, which fails if a block reads the other block's parameters.
    blk = _hand_block()
    junk = {"bg": [1.5, -0.7], "Wg": [[0.3, -1.1], [0.9, 0.2], [-0.4, 0.8]],
            "Wu": [[1.2, 0.1], [-0.6, 0.5], [0.7, -0.9]], "Wd": np.zeros((2, 3))}
    for first, second in ((blk, junk), (junk, blk)):
        parts, x = _silent_towers_z0_30_40(2)
        for k, b in enumerate((first, second)):
            parts.update({f"bg{k}": b["bg"], f"Wg{k}": b["Wg"], f"Wu{k}": b["Wu"], f"Wd{k}": b["Wd"]})
        assert abs(_ratio(parts, x, 4, 2, 3, 2, 350.0) - 0.9002725328499472) < 1e-7
