"""GPU parity of the selected-state commit (Algorithm 1, line 8): byte-exact cache contents and
hidden rows, attention outputs within the usual bar, against the oracle's step_with_commit."""
import numpy as np
import pytest
import torch

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import binding, synth
from tests import gpu_helpers as gh
from tests.helpers import make_problem

pytestmark = pytest.mark.gpu


def _cands(seed, L, B, Hkv, D):
    return (synth.gauss_bf16_tensor(seed, 40, (L, B, Hkv, D)), synth.gauss_bf16_tensor(seed, 41, (L, B, Hkv, D)))


@pytest.mark.parametrize("layout", ["hnd", "nhd"])
def test_write_current_kv_is_byte_exact(layout):
    seq = [17, 48, 5, 2053]
    L, B, Hq, Hkv, D = 3, 4, 8, 2, 128
    prob = make_problem(3, L, B, Hq, Hkv, D, seq, layout=layout)
    ctx = gh.make_ctx(prob, [16] * L, [0] * L, [1] * L)
    dev = gh.upload(prob)
    kc, vc = _cands(3, L, B, Hkv, D)
    mask = np.array([1, 0, 1, 1], np.uint8)
    ctx.write_current_kv(B, synth.bf16_bits_to_torch(kc, "cuda"), synth.bf16_bits_to_torch(vc, "cuda"),
                         torch.from_numpy(mask).cuda(), dev["k"], dev["v"], dev["table"], dev["seq_lens"])
    torch.cuda.synchronize()
    orc.write_current_kv(kc, vc, prob["k"], prob["v"], prob["table"], prob["seq_lens"], block_size=16,
                         layout=prob["layout"], mask=mask)
    np.testing.assert_array_equal(synth.torch_to_bf16_bits(dev["k"]), prob["k"])
    np.testing.assert_array_equal(synth.torch_to_bf16_bits(dev["v"]), prob["v"])
    assert ctx.read_device_status() == 0


def test_step_with_commit_matches_oracle():
    L, B, Hq, Hkv, D = 4, 5, 8, 2, 128
    seq = [400, 70, 2053, 16, 1000]
    windows, sinks, gated = [64, 32, 64, 32], [4, 0, 4, 0], [1, 0, 1, 0]
    prob = make_problem(9, L, B, Hq, Hkv, D, seq)
    head_shape = (0, 1, 16)
    ctx = gh.make_ctx(prob, windows, sinks, gated, head=head_shape)
    dev = gh.upload(prob)
    kl, vl = _cands(1, L, B, Hkv, D)
    kf, vf = _cands(2, L, B, Hkv, D)
    qf = synth.gauss_bf16_tensor(9, synth.STREAM_QFULL, (L, B, Hq, D))
    hl = synth.gauss_f32_tensor(5, 1, (B, 64))
    hf = synth.gauss_f32_tensor(5, 2, (B, 64))
    head = dict(W1=synth.gauss_f32_tensor(7, synth.STREAM_W1, (16, Hq * D), std=0.05),
                b1=synth.gauss_f32_tensor(7, synth.STREAM_B1, (16,), std=0.05),
                w2=synth.gauss_f32_tensor(7, synth.STREAM_W2, (16,), std=0.05),
                b2=synth.gauss_f32_tensor(7, synth.STREAM_B2, (1,), std=0.05), use_attn_out=1)
    # threshold between the sorted oracle scores of a dry run, so that the head itself splits the batch
    dry = dict(prob, k=prob["k"].copy(), v=prob["v"].copy())
    r0 = orc.step_with_commit(prob["q"], qf, dry["k"], dry["v"], prob["table"], prob["seq_lens"],
                              k_cur_local=kl, v_cur_local=vl, k_cur_full=kf, v_cur_full=vf, num_kv_heads=Hkv,
                              block_size=16, layout=prob["layout"], layer_window=windows, layer_sinks=sinks,
                              layer_gated=gated, head=head, tau=2.0, nthreads=8)
    srt = np.sort(r0.score)
    tau = float(0.5 * (srt[2] + srt[3]))       # two of the five requests recall
    assert np.abs(r0.score - tau).min() > gh.FLAG_BAND
    ref = orc.step_with_commit(prob["q"], qf, prob["k"], prob["v"], prob["table"], prob["seq_lens"],
                               k_cur_local=kl, v_cur_local=vl, k_cur_full=kf, v_cur_full=vf, num_kv_heads=Hkv,
                               block_size=16, layout=prob["layout"], layer_window=windows, layer_sinks=sinks,
                               layer_gated=gated, head=head, tau=tau, hidden_local=hl, hidden_full=hf, nthreads=8)
    assert 0 < ref.flags.sum() < B
    out = torch.zeros((L, B, Hq, D), device="cuda")
    scores = torch.zeros(B, device="cuda")
    flags = torch.zeros(B, dtype=torch.uint8, device="cuda")
    hidden = torch.zeros((B, 64), device="cuda")
    seq_dev = dev["seq_lens"].clone()
    args = ctx.step_args(B, dev["q"], dev["k"], dev["v"], dev["table"], seq_dev, out, scores, flags,
                         q_full=synth.bf16_bits_to_torch(qf, "cuda"), head=gh.head_to_device(head), threshold=tau,
                         k_cur_local=synth.bf16_bits_to_torch(kl, "cuda"), v_cur_local=synth.bf16_bits_to_torch(vl, "cuda"),
                         k_cur_full=synth.bf16_bits_to_torch(kf, "cuda"), v_cur_full=synth.bf16_bits_to_torch(vf, "cuda"),
                         hidden_local=torch.from_numpy(hl).cuda(), hidden_full=torch.from_numpy(hf).cuda(),
                         hidden_out=hidden, advance_seq_lens=True)
    ctx.step(args)
    torch.cuda.synchronize()
    np.testing.assert_allclose(scores.cpu().numpy(), ref.score, rtol=0, atol=gh.ATOL_SCORE)
    decided = np.abs(ref.score - tau) >= gh.FLAG_BAND
    np.testing.assert_array_equal(flags.cpu().numpy()[decided], ref.flags[decided])
    assert decided.all()
    gh.assert_close(out.cpu().numpy(), ref.out, gh.ATOL_OUT, "step-with-commit out")
    np.testing.assert_array_equal(hidden.cpu().numpy(), ref.hidden)
    np.testing.assert_array_equal(synth.torch_to_bf16_bits(dev["k"]), prob["k"])   # the selected candidates, byte for byte
    np.testing.assert_array_equal(synth.torch_to_bf16_bits(dev["v"]), prob["v"])
    np.testing.assert_array_equal(seq_dev.cpu().numpy(), np.asarray(seq) + 1)
    assert ctx.read_device_status() == 0


def test_advance_seq_lens_moves_only_the_requests_of_the_call():
    prob = make_problem(4, 1, 5, 4, 2, 64, [3, 40, 7, 16, 2053])
    ctx = gh.make_ctx(prob, [16], [0], [1])
    seq = torch.from_numpy(prob["seq_lens"]).cuda()
    ctx.advance_seq_lens(3, seq)
    ctx.advance_seq_lens(5, seq)
    ctx.advance_seq_lens(0, seq)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(seq.cpu().numpy(), np.array([5, 42, 9, 17, 2054], np.int32))
    with pytest.raises(binding.OdaError):
        ctx.advance_seq_lens(6, seq)
