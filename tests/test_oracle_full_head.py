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
