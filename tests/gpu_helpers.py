"""Upload host problems (tests.helpers.make_problem) and run them through the C-ABI binding."""
from __future__ import annotations

import numpy as np
import torch

from paper_2609_20734_b200 import binding, synth

ATOL_OUT = 2e-3   # max-abs bar on attention outputs (bf16 in, fp32 accumulate, fp32 out)
ATOL_LSE = 1e-3
FLAG_BAND = 1e-4  # flags must match unless |score - threshold| < band
ATOL_SCORE = 1e-5


def make_ctx(prob, windows, sinks, gated, *, head=None, kv_index=None, variant=binding.VARIANT_AUTO,
             out_dtype=0, sm_scale=0.0, max_batch=None):
    lay = prob["layout"]
    d_ext, use_attn, d_h = head if head else (0, 0, 0)
    cfg = binding.OdaConfig(
        num_layers=prob["L"], num_q_heads=prob["Hq"], num_kv_heads=prob["Hkv"], head_dim=prob["D"],
        max_batch=max_batch or max(prob["B"], 1), max_blocks_per_seq=prob["table"].shape[1],
        layer_window=windows, layer_sinks=sinks, layer_gated=gated, layer_kv_index=kv_index,
        kv_layer_stride=lay.layer_stride, kv_block_stride=lay.block_stride,
        kv_token_stride=lay.token_stride, kv_head_stride=lay.head_stride, out_dtype=out_dtype,
        sm_scale=sm_scale, variant=variant, head_d_ext=d_ext, head_use_attn_out=use_attn,
        head_d_hidden=d_h)
    return binding.OdaContext(cfg)


def upload(prob):
    dev = {}
    dev["q"] = synth.bf16_bits_to_torch(prob["q"], "cuda")
    dev["k"] = synth.bf16_bits_to_torch(prob["k"], "cuda")
    dev["v"] = synth.bf16_bits_to_torch(prob["v"], "cuda")
    dev["table"] = torch.from_numpy(prob["table"]).cuda()
    dev["seq_lens"] = torch.from_numpy(prob["seq_lens"]).cuda()
    return dev


def new_out(prob, fill=float("nan"), dtype=torch.float32):
    L, B, Hq, D = prob["L"], prob["B"], prob["Hq"], prob["D"]
    out = torch.full((L, B, Hq, D), fill, dtype=dtype, device="cuda")
    lse = torch.full((L, B, Hq), fill, dtype=torch.float32, device="cuda")
    return out, lse


def gpu_local(ctx, prob, dev, lb=0, le=None, batch=None):
    out, lse = new_out(prob)
    ctx.local_decode(lb, prob["L"] if le is None else le, prob["B"] if batch is None else batch,
                     dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out, lse)
    torch.cuda.synchronize()
    return out.cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)


def head_to_device(head):
    return {k: torch.from_numpy(np.ascontiguousarray(np.asarray(v, dtype=np.float32).reshape(-1) if k == "b2" else v)).cuda()
            for k, v in head.items() if k != "use_attn_out"}


def assert_close(got, want, atol, what=""):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    mask = ~np.isnan(want)
    assert np.isfinite(got[mask]).all(), f"{what}: non-finite values in the GPU result"
    err = np.abs(got[mask] - want[mask]).max() if mask.any() else 0.0
    assert err <= atol, f"{what}: max abs error {err:.3e} > {atol:.1e}"
    return err
