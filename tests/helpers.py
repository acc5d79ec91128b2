"""Shared test scaffolding: small paged-KV problems built from the seeded generator,
and an independent brute-force attention used to pin the oracle."""
from __future__ import annotations

import numpy as np

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import synth


def make_problem(seed, L, B, Hq, Hkv, D, seq_lens, P=16, layout="hnd", shuffled=True,
                 spare_blocks=3, kv_layers=None):
    """Host-side problem: q [L,B,Hq,D], caches (flat uint16 bf16 bits), block table."""
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    assert len(seq_lens) == B
    need = (np.maximum(seq_lens, 1) + P - 1) // P
    max_blocks = int(need.max()) + 1 if B else 1
    table, pool = synth.block_tables(seed, need, max_blocks, shuffled,
                                     num_blocks=int(need.sum()) + spare_blocks)
    Lkv = L if kv_layers is None else kv_layers
    lay = (orc.hnd_layout if layout == "hnd" else orc.nhd_layout)(pool, Hkv, P, D)
    n = Lkv * lay.layer_stride
    k = synth.gauss_bf16_tensor(seed, synth.STREAM_K, (n,))
    v = synth.gauss_bf16_tensor(seed, synth.STREAM_V, (n,))
    q = synth.gauss_bf16_tensor(seed, synth.STREAM_Q, (L, B, Hq, D))
    return dict(L=L, B=B, Hq=Hq, Hkv=Hkv, D=D, P=P, q=q, k=k, v=v, table=table,
                seq_lens=seq_lens, layout=lay, pool=pool, kv_layers=Lkv)


def dense_kv(prob, cache, kv_layer, b, kv_head):
    """De-page one (layer, request, kv head) into a dense [t, D] float array (exact)."""
    lay, P, D = prob["layout"], prob["P"], prob["D"]
    t = int(prob["seq_lens"][b])
    rows = np.empty((t, D), dtype=np.float64)
    for j in range(t):
        blk = int(prob["table"][b, j // P])
        off = (kv_layer * lay.layer_stride + blk * lay.block_stride + (j % P) * lay.token_stride
               + kv_head * lay.head_stride)
        rows[j] = synth.bf16_bits_to_f32(cache[off:off + D]).astype(np.float64)
    return rows


def local_set_1based(t, s, w):
    """Eq. 1, literally, with 1-based positions."""
    return set(range(1, min(s, t) + 1)) | set(range(max(1, t - w + 1), t + 1))


def full_set_1based(t):
    return set(range(1, t + 1))


def brute_attention(prob, l, b, h, members_1based, sm_scale=None, kv_layer=None):
    """Softmax attention over an explicit 1-based index set, in extended precision and
    without max subtraction: out = sum e^{z_i} v_i / sum e^{z_i}, lse = ln sum e^{z_i}."""
    D = prob["D"]
    G = prob["Hq"] // prob["Hkv"]
    g = h // G
    kvl = l if kv_layer is None else kv_layer
    K = dense_kv(prob, prob["k"], kvl, b, g).astype(np.longdouble)
    V = dense_kv(prob, prob["v"], kvl, b, g).astype(np.longdouble)
    q = synth.bf16_bits_to_f32(prob["q"][l, b, h]).astype(np.longdouble)
    scale = np.longdouble(1.0) / np.sqrt(np.longdouble(D)) if sm_scale is None else np.longdouble(sm_scale)
    num = np.zeros(D, dtype=np.longdouble)
    den = np.longdouble(0.0)
    for i in sorted(members_1based):
        e = np.exp(scale * np.dot(q, K[i - 1]))
        num += e * V[i - 1]
        den += e
    return (num / den).astype(np.float64), float(np.log(den))


def oracle_attention(prob, mode, windows, sinks, **kw):
    return orc.attention(mode, prob["q"], prob["k"], prob["v"], prob["table"], prob["seq_lens"],
                         num_kv_heads=prob["Hkv"], block_size=prob["P"], layout=prob["layout"],
                         layer_window=windows, layer_sinks=sinks, **kw)
