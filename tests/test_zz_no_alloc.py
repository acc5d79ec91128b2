"""oda_local_decode_static: the Local pass for callers that cannot allocate device memory (its
scratch is a fixed array inside the library).  Checked against the oracle and against the regular
entry point, which uses a caller-provided workspace, on two calls in a row -- the second call
finds the array as the first one left it.  Collected last so that a run stopping at the first
failure has already run every other test."""
import numpy as np
import pytest
import torch

from paper_2609_20734_b200 import binding
from tests import gpu_helpers as gh
from tests.helpers import make_problem, oracle_attention

pytestmark = pytest.mark.gpu


def _call_static(prob, dev, w, s):
    B, Hq, Hkv, D, lay = prob["B"], prob["Hq"], prob["Hkv"], prob["D"], prob["layout"]
    out = torch.full((B, Hq, D), float("nan"), device="cuda")
    lse = torch.full((B, Hq), float("nan"), device="cuda")
    binding.local_decode_static(B, Hq, Hkv, D, w, s, 0.0, lay.block_stride, lay.token_stride,
                                lay.head_stride, prob["table"].shape[1], dev["q"], dev["k"],
                                dev["v"], dev["table"], dev["seq_lens"], out, lse)
    torch.cuda.synchronize()
    return out, lse


def _check_two_calls(prob, w, s, what):
    dev = gh.upload(prob)
    ctx = gh.make_ctx(prob, [w], [s], [1])
    binding.local_decode_static_status()   # start from a clean status word whatever ran before
    for call in range(2):
        # different queries on the second call: stale partials or tickets would show
        if call == 1:
            prob = dict(prob, q=np.ascontiguousarray(prob["q"][:, :, ::-1, :]))
            dev["q"] = torch.flip(dev["q"], dims=[2]).contiguous()
        want_out, want_lse = oracle_attention(prob, "local", [w], [s], nthreads=8)
        ws_out, ws_lse = gh.gpu_local(ctx, prob, dev)
        out, lse = _call_static(prob, dev, w, s)
        gh.assert_close(out.cpu().numpy(), want_out[0], gh.ATOL_OUT, f"{what}, static call {call}: out vs oracle")
        gh.assert_close(lse.cpu().numpy(), want_lse[0], gh.ATOL_LSE, f"{what}, static call {call}: lse vs oracle")
        gh.assert_close(out.cpu().numpy(), ws_out[0], gh.ATOL_OUT, f"{what}, static call {call}: out vs workspace path")
        gh.assert_close(lse.cpu().numpy(), ws_lse[0], gh.ATOL_LSE, f"{what}, static call {call}: lse vs workspace path")
    assert binding.local_decode_static_status() == 0


def test_static_scratch_entry_point_matches_oracle_and_workspace_entry_point_twice():
    seq = [1, 17, 300, 2053, 64, 999]
    prob = make_problem(77, 1, len(seq), 8, 2, 128, seq, layout="hnd")
    _check_two_calls(prob, 256, 4, "D128 G4")


def test_static_scratch_entry_point_at_its_size_limits():
    # batch 16 x 16 kv heads = the 256-unit limit, windows long enough that every span has work:
    # partial slots up to (spans + units) are in use
    rng = np.random.default_rng(5)
    seq = [int(x) for x in rng.integers(700, 1400, 16)]
    prob = make_problem(78, 1, 16, 16, 16, 128, seq, layout="hnd")
    _check_two_calls(prob, 640, 4, "D128 G1 at 256 units")
    # the widest partial rows per unit: group 8, and head_dim 64
    seq = [int(x) for x in rng.integers(100, 900, 16)]
    prob = make_problem(79, 1, 16, 128, 16, 64, seq, layout="hnd")
    _check_two_calls(prob, 512, 4, "D64 G8 at 256 units")


def test_static_scratch_entry_point_allocates_nothing():
    seq = [40, 900, 333]
    prob = make_problem(80, 1, len(seq), 8, 2, 128, seq, layout="hnd")
    dev = gh.upload(prob)
    _call_static(prob, dev, 256, 4)           # first call on the device: set-up
    out = torch.empty((3, 8, 128), device="cuda")
    lse = torch.empty((3, 8), device="cuda")
    lay = prob["layout"]
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(2):
        binding.local_decode_static(3, 8, 2, 128, 256, 4, 0.0, lay.block_stride, lay.token_stride,
                                    lay.head_stride, prob["table"].shape[1], dev["q"], dev["k"],
                                    dev["v"], dev["table"], dev["seq_lens"], out, lse)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
    assert free1 == free0, "device memory in use changed across calls that must not allocate"


def test_static_scratch_entry_point_reports_a_skipped_request():
    # one request of length 0: its rows stay untouched, the others are right, and the status word
    # says so until it is read (it is not reset by the next call)
    seq = [50, 0, 700]
    prob = make_problem(81, 1, len(seq), 8, 2, 128, seq, layout="hnd")
    dev = gh.upload(prob)
    binding.local_decode_static_status()
    out, lse = _call_static(prob, dev, 256, 4)
    good = dict(prob, seq_lens=np.array([50, 1, 700], np.int32))   # the oracle refuses length 0: row 1 is not compared
    want_out, _ = oracle_attention(good, "local", [256], [4])
    o = out.cpu().numpy()
    for b in (0, 2):
        gh.assert_close(o[b], want_out[0, b], gh.ATOL_OUT, f"request {b} beside a skipped one")
    assert np.isnan(o[1]).all() and torch.isnan(lse[1]).all()
    ok = dict(prob, seq_lens=np.array([50, 3, 700], np.int32))
    dev_ok = dict(dev, seq_lens=torch.from_numpy(ok["seq_lens"]).cuda())
    _call_static(ok, dev_ok, 256, 4)          # a clean call in between does not clear the word
    assert binding.local_decode_static_status() == 1
    assert binding.local_decode_static_status() == 0


def test_static_scratch_entry_point_rejects_sizes_beyond_its_array():
    z = torch.zeros(16, device="cuda")
    for batch, hq, hkv in ((17, 8, 2), (16, 64, 32)):
        with pytest.raises(binding.OdaError) as e:
            binding.local_decode_static(batch, hq, hkv, 128, 16, 0, 0.0, 4096, 128, 2048, 4, z, z, z, z, z, z)
        assert e.value.status == 2
    # arguments the workspace path refuses at creation are refused here too
    for scale, block_stride in ((float("inf"), 4096), (0.0, 1024)):
        with pytest.raises(binding.OdaError) as e:
            binding.local_decode_static(1, 8, 2, 128, 16, 0, scale, block_stride, 128, 2048, 4, z, z, z, z, z, z)
        assert e.value.status == 1
