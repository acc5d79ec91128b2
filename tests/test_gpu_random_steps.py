"""Seeded random sweep of whole ODA steps against the oracle: layer counts, group sizes, head
dims, layouts, per-layer windows / sinks / gating, cache-layer aliasing, ragged lengths around the
page and window edges, distinct Full-branch queries, learned or forced flags, both kernels."""
import numpy as np
import pytest
import torch

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import binding, synth
from tests import gpu_helpers as gh
from tests.helpers import make_problem

pytestmark = pytest.mark.gpu


def _draw(case):
    rng = np.random.default_rng(9000 + case)
    D = int(rng.choice([64, 128]))
    G = int(rng.choice([1, 2, 4, 8]))
    Hkv = int(rng.choice([1, 2, 3]))
    L = int(rng.integers(1, 6))
    B = int(rng.integers(1, 8))
    layout = str(rng.choice(["hnd", "nhd"]))
    # at most four distinct (window, sinks, gated) layer classes per context (the library's limit)
    palette = [(int(rng.choice([1, 7, 16, 33, 64, 200])), int(rng.choice([0, 1, 4, 17])), int(rng.random() < 0.6))
               for _ in range(3)]
    palette.append((int(rng.choice([16, 64])), 4, 1))          # always one gated class
    picks = [palette[int(rng.integers(0, 4))] for _ in range(L - 1)] + [palette[3]]
    windows, sinks, gated = [list(v) for v in zip(*picks)]
    kv_layers = int(rng.integers(1, L + 1))
    kv_index = [int(rng.integers(0, kv_layers)) for _ in range(L)]
    # lengths: 1, page edges, window edges, a few hundred
    pool = [1, 2, 15, 16, 17, 31, 32, 33, 63, 64, 65, 100, 255, 256, 257, 400, 700]
    seq = [int(rng.choice(pool)) for _ in range(B)]
    forced = bool(rng.random() < 0.5)
    distinct_qf = bool(rng.random() < 0.5)
    variant = int(rng.choice([binding.VARIANT_SIMT, binding.VARIANT_TMA_MMA]))
    return dict(D=D, Hq=G * Hkv, Hkv=Hkv, L=L, B=B, layout=layout, windows=windows, sinks=sinks, gated=gated,
                kv_layers=kv_layers, kv_index=kv_index, seq=seq, forced=forced, distinct_qf=distinct_qf,
                variant=variant, seed=int(rng.integers(1, 10**6)))


@pytest.mark.parametrize("case", range(24))
def test_random_step_matches_oracle(case):
    c = _draw(case)
    L, B, Hq, Hkv, D = c["L"], c["B"], c["Hq"], c["Hkv"], c["D"]
    prob = make_problem(c["seed"], L, B, Hq, Hkv, D, c["seq"], layout=c["layout"], kv_layers=c["kv_layers"])
    qf = synth.gauss_bf16_tensor(c["seed"], synth.STREAM_QFULL, (L, B, Hq, D)) if c["distinct_qf"] else None
    d_ext, d_h = 12, 9
    head = dict(W1=synth.gauss_f32_tensor(c["seed"], synth.STREAM_W1, (d_h, d_ext + Hq * D), std=0.05),
                b1=synth.gauss_f32_tensor(c["seed"], synth.STREAM_B1, (d_h,), std=0.05),
                w2=synth.gauss_f32_tensor(c["seed"], synth.STREAM_W2, (d_h,), std=0.3),
                b2=synth.gauss_f32_tensor(c["seed"], synth.STREAM_B2, (1,), std=0.05), use_attn_out=1)
    fe = synth.gauss_f32_tensor(c["seed"], synth.STREAM_FEAT, (B, d_ext))
    ov = (np.random.default_rng(c["seed"]).random(B) < 0.5).astype(np.uint8) if c["forced"] else None
    kw = dict(num_kv_heads=Hkv, block_size=16, layout=prob["layout"], layer_window=c["windows"],
              layer_sinks=c["sinks"], layer_gated=c["gated"], layer_kv_index=c["kv_index"], head=head,
              feat_ext=fe, override_flags=ov, nthreads=4)
    first = orc.step(prob["q"], qf, prob["k"], prob["v"], prob["table"], prob["seq_lens"], tau=0.5, **kw)
    # a threshold no score is close to, so that the learned flags are decided
    edges = np.concatenate([[first.score.min() - 0.02], np.sort(first.score), [first.score.max() + 0.02]])
    j = int(np.argmax(np.diff(edges)))
    tau = float(0.5 * (edges[j] + edges[j + 1]))     # the middle of the widest gap between scores
    ref = orc.step(prob["q"], qf, prob["k"], prob["v"], prob["table"], prob["seq_lens"], tau=tau, **kw)
    assert np.abs(ref.score - tau).min() > 2 * gh.FLAG_BAND

    ctx = gh.make_ctx(prob, c["windows"], c["sinks"], c["gated"], head=(d_ext, 1, d_h), kv_index=c["kv_index"],
                      variant=c["variant"])
    dev = gh.upload(prob)
    out, lse = gh.new_out(prob)
    scores = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    args = ctx.step_args(B, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out, scores, flags,
                         q_full=None if qf is None else synth.bf16_bits_to_torch(qf, "cuda"),
                         feat_ext=torch.from_numpy(fe).cuda(), head=gh.head_to_device(head), threshold=tau,
                         override_flags=None if ov is None else torch.from_numpy(ov).cuda(), lse=lse)
    ctx.step(args)
    torch.cuda.synchronize()
    assert ctx.read_device_status() == 0
    np.testing.assert_array_equal(flags.cpu().numpy(), ref.flags, err_msg=str(c))
    np.testing.assert_allclose(scores.cpu().numpy(), ref.score, rtol=0, atol=gh.ATOL_SCORE, err_msg=str(c))
    gh.assert_close(out.cpu().numpy(), ref.out, gh.ATOL_OUT, f"out {c}")
    gh.assert_close(lse.cpu().numpy(), ref.lse, gh.ATOL_LSE, f"lse {c}")
