"""oda_local_decode_static: the Local pass for callers that cannot allocate device memory (its
scratch is a fixed array inside the library).  Checked against the regular entry point, which
uses a caller-provided workspace, on two calls in a row -- the second call finds the array as
the first one left it.  Collected last so that a run stopping at the first failure has already
run every other test."""
import numpy as np
import pytest
import torch

from paper_2609_20734_b200 import binding
from tests import gpu_helpers as gh
from tests.helpers import make_problem

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_workspace_entry_point_twice():
    seq = [1, 17, 300, 2053, 64, 999]
    D, Hq, Hkv, w, s = 128, 8, 2, 256, 4
    prob = make_problem(77, 1, len(seq), Hq, Hkv, D, seq, layout="hnd")
    dev = gh.upload(prob)
    lay = prob["layout"]
    ctx = gh.make_ctx(prob, [w], [s], [1])
    ref, ref_lse = gh.gpu_local(ctx, prob, dev)
    B = len(seq)
    for call in range(2):
        # different queries on the second call: stale partials or tickets would show
        if call == 1:
            dev["q"] = torch.flip(dev["q"], dims=[2]).contiguous()
            ref, ref_lse = gh.gpu_local(ctx, prob, dev)
        out = torch.full((B, Hq, D), float("nan"), device="cuda")
        lse = torch.full((B, Hq), float("nan"), device="cuda")
        binding.local_decode_static(B, Hq, Hkv, D, w, s, 0.0, lay.block_stride, lay.token_stride,
                                    lay.head_stride, prob["table"].shape[1], dev["q"], dev["k"],
                                    dev["v"], dev["table"], dev["seq_lens"], out, lse)
        torch.cuda.synchronize()
        gh.assert_close(out.cpu().numpy(), ref[0], gh.ATOL_OUT, f"static call {call} out")
        gh.assert_close(lse.cpu().numpy(), ref_lse[0], gh.ATOL_LSE, f"static call {call} lse")


def test_static_scratch_entry_point_rejects_sizes_beyond_its_array():
    z = torch.zeros(16, device="cuda")
    for batch, hq, hkv in ((17, 8, 2), (16, 64, 32)):
        with pytest.raises(binding.OdaError) as e:
            binding.local_decode_static(batch, hq, hkv, 128, 16, 0, 0.0, 4096, 128, 2048, 4, z, z, z, z, z, z)
        assert e.value.status == 2
