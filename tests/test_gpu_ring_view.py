"""The Local workspace variant (sink slots + a ring of recent positions beside the paged history, the
commit writing both views): the Local pass over the ring view must give the bits of the Local pass
over the paged history at every step, across page boundaries and ring wrap-arounds, and match the
oracle; positions outside the live window are poisoned so that a stale or early read shows."""
import numpy as np
import pytest
import torch

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import binding, ring_view, synth
from tests import gpu_helpers as gh
from tests.helpers import make_problem, oracle_attention

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("w,s", [(32, 4), (256, 0), (48, 20)])
def test_local_over_ring_view_equals_local_over_paged_history(w, s):
    L, Hq, Hkv, D, steps = 2, 8, 2, 128, 70
    seq0 = np.array([5, 40, 700], np.int32)
    B = len(seq0)
    prob = make_problem(21, L, B, Hq, Hkv, D, seq0 + steps, shuffled=True)
    prob["seq_lens"] = seq0.copy()
    dev = gh.upload(prob)
    ctx = gh.make_ctx(prob, [w] * L, [s] * L, [1] * L)
    geo = ring_view.geometry(B, [w] * L, [s] * L)
    lay = prob["layout"]
    n_ring = L * geo.num_blocks * Hkv * 16 * D
    poison = torch.full((n_ring,), float("nan"), dtype=torch.bfloat16, device="cuda")
    ring_k, ring_v = poison.clone(), poison.clone()
    ring_tab_h = ring_view.table(geo, B, prob["table"].shape[1])
    ring_tab = torch.from_numpy(ring_tab_h).cuda()
    ring_view.fill_from_paged(geo, ring_k, ring_v, dev["k"], dev["v"], prob["table"], seq0, [w] * L, [s] * L,
                              phys_layers=L, paged_blocks=prob["pool"], kv_heads=Hkv, head_dim=D)
    rcfg = binding.OdaConfig(
        num_layers=L, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=B,
        max_blocks_per_seq=prob["table"].shape[1], layer_window=[w] * L, layer_sinks=[s] * L, layer_gated=[1] * L,
        kv_layer_stride=geo.num_blocks * Hkv * 16 * D, kv_block_stride=lay.block_stride,
        kv_token_stride=lay.token_stride, kv_head_stride=lay.head_stride)
    rctx = binding.OdaContext(rcfg)
    seq = dev["seq_lens"]
    for step in range(steps):
        if step:   # the step's commit: the new position's K/V goes into both views
            kc = synth.gauss_bf16_tensor(50 + step, 40, (L, B, Hkv, D))
            vc = synth.gauss_bf16_tensor(50 + step, 41, (L, B, Hkv, D))
            seq.add_(1)
            prob["seq_lens"] = prob["seq_lens"] + 1
            kd, vd = synth.bf16_bits_to_torch(kc, "cuda"), synth.bf16_bits_to_torch(vc, "cuda")
            ctx.write_current_kv(B, kd, vd, None, dev["k"], dev["v"], dev["table"], seq)
            rctx.write_current_kv(B, kd, vd, None, ring_k, ring_v, ring_tab, seq)
            orc.write_current_kv(kc, vc, prob["k"], prob["v"], prob["table"], prob["seq_lens"], block_size=16,
                                 layout=lay)
        out_p, lse_p = gh.new_out(prob)
        out_r, lse_r = gh.new_out(prob)
        ctx.local_decode(0, L, B, dev["q"], dev["k"], dev["v"], dev["table"], seq, out_p, lse_p)
        rctx.local_decode(0, L, B, dev["q"], ring_k, ring_v, ring_tab, seq, out_r, lse_r)
        torch.cuda.synchronize()
        assert torch.equal(out_r, out_p) and torch.equal(lse_r, lse_p), f"step {step}"
        if step % 23 == 0 or step == steps - 1:
            want, want_lse = oracle_attention(prob, "local", [w] * L, [s] * L)
            gh.assert_close(out_r.cpu().numpy(), want, gh.ATOL_OUT, f"ring view, step {step}")
            gh.assert_close(lse_r.cpu().numpy(), want_lse, gh.ATOL_LSE, f"ring view lse, step {step}")
    assert ctx.read_device_status() == 0 and rctx.read_device_status() == 0
