"""KV-head tensor-parallel step: the ranks of a 2- and 4-way split run one after another on one
GPU (their kernels never wait on each other; the exchange between the two phases is a plain sum
here), and the assembled result is compared with the unsharded oracle step."""
import numpy as np
import pytest
import torch

from oracle import oda_oracle as orc
from paper_2609_20734_b200 import synth
from paper_2609_20734_b200 import tensor_parallel as tp
from tests import gpu_helpers as gh
from tests.helpers import make_problem

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world,layout,d_ext", [(2, "hnd", 32), (4, "nhd", 0), (1, "hnd", 6)])
def test_tensor_parallel_step_matches_unsharded_oracle(world, layout, d_ext):
    L, B, Hq, Hkv, D, d_h = 3, 5, 8, 4, 128, 40
    windows, sinks, gated = [64, 32, 64], [4, 0, 4], [1, 1, 0]
    prob = make_problem(31, L, B, Hq, Hkv, D, [100, 900, 33, 2500, 64], layout=layout)
    lay = prob["layout"]
    d_in = d_ext + Hq * D
    head = dict(W1=synth.gauss_f32_tensor(9, synth.STREAM_W1, (d_h, d_in), std=0.05),
                b1=synth.gauss_f32_tensor(9, synth.STREAM_B1, (d_h,), std=0.05),
                w2=synth.gauss_f32_tensor(9, synth.STREAM_W2, (d_h,), std=0.05),
                b2=synth.gauss_f32_tensor(9, synth.STREAM_B2, (1,), std=0.05), use_attn_out=1)
    fe = synth.gauss_f32_tensor(9, synth.STREAM_FEAT, (B, d_ext)) if d_ext else None
    kw = dict(num_kv_heads=Hkv, block_size=16, layout=lay, layer_window=windows, layer_sinks=sinks,
              layer_gated=gated, head=head, feat_ext=fe, nthreads=4)
    sc = np.sort(orc.step(prob["q"], None, prob["k"], prob["v"], prob["table"], prob["seq_lens"], tau=0.5, **kw).score)
    tau = float(0.5 * (sc[2] + sc[3]))              # two of the five requests recall
    assert sc[3] - tau > 2 * gh.FLAG_BAND and tau - sc[2] > 2 * gh.FLAG_BAND
    ref = orc.step(prob["q"], None, prob["k"], prob["v"], prob["table"], prob["seq_lens"], tau=tau, **kw)
    assert ref.flags.sum() == 2

    dev = gh.upload(prob)
    hd = gh.head_to_device(head)
    fe_d = None if fe is None else torch.from_numpy(fe).cuda()
    q_all = dev["q"].view(L, B, Hq, D)
    ranks = []
    for r in range(world):
        sh = tp.head_shard(r, world, Hq, Hkv, D, d_ext, True)
        rp = dict(prob, Hq=sh.q_heads, Hkv=sh.kv_heads)
        ctx = gh.make_ctx(rp, windows, sinks, gated, head=(sh.d_ext, 1, d_h))
        off = sh.kv_head_begin * lay.head_stride      # the rank's heads inside the shared test cache
        st = dict(sh=sh, ctx=ctx, k=dev["k"][off:], v=dev["v"][off:],
                  q=q_all[:, :, sh.q_head_begin:sh.q_head_begin + sh.q_heads].contiguous(),
                  out=torch.full((L, B, sh.q_heads, D), float("nan"), device="cuda"),
                  lse=torch.full((L, B, sh.q_heads), float("nan"), device="cuda"),
                  pre=torch.full((B, d_h), float("nan"), device="cuda"),
                  scores=torch.zeros(B, device="cuda"), logits=torch.zeros(B, device="cuda"),
                  flags=torch.zeros(B, dtype=torch.uint8, device="cuda"))
        ranks.append(st)
    for st in ranks:
        tp.tp_local_and_preact(st["ctx"], st["sh"], B, st["q"], st["k"], st["v"], dev["table"], dev["seq_lens"],
                               st["out"], W1=hd["W1"], pre=st["pre"], feat_ext=fe_d, lse=st["lse"])
    pre_sum = torch.stack([st["pre"] for st in ranks]).sum(0)     # stands in for the all-reduce
    for st in ranks:
        tp.tp_decide_and_recompute(st["ctx"], B, st["q"], st["k"], st["v"], dev["table"], dev["seq_lens"],
                                   st["out"], pre_sum=pre_sum.clone(), b1=hd["b1"], w2=hd["w2"], b2=hd["b2"],
                                   threshold=tau, scores=st["scores"], flags=st["flags"], logits=st["logits"],
                                   lse=st["lse"])
    torch.cuda.synchronize()
    for st in ranks:
        assert st["ctx"].read_device_status() == 0
        np.testing.assert_array_equal(st["flags"].cpu().numpy(), ref.flags)
        np.testing.assert_allclose(st["scores"].cpu().numpy(), ref.score, rtol=0, atol=gh.ATOL_SCORE)
        # every rank holds the same sums, so the decisions are bitwise the same
        assert torch.equal(st["scores"], ranks[0]["scores"]) and torch.equal(st["logits"], ranks[0]["logits"])
    out = torch.cat([st["out"] for st in ranks], dim=2).cpu().numpy()
    lse = torch.cat([st["lse"] for st in ranks], dim=2).cpu().numpy()
    gh.assert_close(out, ref.out, gh.ATOL_OUT, "assembled out")
    gh.assert_close(lse, ref.lse, gh.ATOL_LSE, "assembled lse")


def test_preact_plus_finalize_equals_fused_head():
    """world = 1: the two-call head agrees with the fused one to fp32 rounding, odd widths included."""
    B, d_ext, Hq, D, d_h = 7, 7, 2, 64, 19
    prob = make_problem(1, 1, B, Hq, Hq, D, [20] * B)
    ctx = gh.make_ctx(prob, [8], [0], [1], head=(d_ext, 1, d_h))
    d_in = d_ext + Hq * D
    hd = {k: torch.from_numpy(v).cuda() for k, v in dict(
        W1=synth.gauss_f32_tensor(5, synth.STREAM_W1, (d_h, d_in), std=0.05),
        b1=synth.gauss_f32_tensor(5, synth.STREAM_B1, (d_h,), std=0.05),
        w2=synth.gauss_f32_tensor(5, synth.STREAM_W2, (d_h,), std=0.05),
        b2=synth.gauss_f32_tensor(5, synth.STREAM_B2, (1,), std=0.05)).items()}
    fe = torch.from_numpy(synth.gauss_f32_tensor(5, synth.STREAM_FEAT, (B, d_ext))).cuda()
    attn = torch.from_numpy(synth.gauss_f32_tensor(6, synth.STREAM_FEAT, (B, Hq, D))).cuda()
    s1, z1, s2, z2 = (torch.zeros(B, device="cuda") for _ in range(4))
    f1, f2 = (torch.zeros(B, dtype=torch.uint8, device="cuda") for _ in range(2))
    pre = torch.zeros((B, d_h), device="cuda")
    ctx.recall_score(B, fe, attn, hd["W1"], hd["b1"], hd["w2"], hd["b2"], 0.5, None, s1, z1, f1)
    ctx.recall_preact(B, fe, attn, hd["W1"], d_in, pre)
    ctx.recall_finalize(B, pre, hd["b1"], hd["w2"], hd["b2"], 0.5, None, s2, z2, f2)
    torch.cuda.synchronize()
    np.testing.assert_allclose(s2.cpu().numpy(), s1.cpu().numpy(), rtol=0, atol=1e-6)
    np.testing.assert_allclose(z2.cpu().numpy(), z1.cpu().numpy(), rtol=0, atol=1e-5)
    x = torch.cat([fe, attn.reshape(B, -1)], dim=1).double()
    np.testing.assert_allclose(pre.cpu().numpy(), (x @ hd["W1"].double().T).cpu().numpy(), rtol=0, atol=1e-5)


@pytest.mark.parametrize("world", [1, 2, 4])
def test_sequence_sharded_full_pass_matches_oracle(world):
    """Each 'rank' runs the gated Full pass over its page range of every request (ranks run one
    after another on this GPU); the merged rows equal the oracle's Full attention over the whole
    history, short requests that leave ranks empty included."""
    L, B, Hq, Hkv, D = 3, 6, 8, 2, 128
    windows, sinks, gated = [64, 32, 64], [4, 0, 4], [1, 0, 1]
    seq = [100, 900, 5, 2500, 64, 17]
    prob = make_problem(41, L, B, Hq, Hkv, D, seq)
    flags_h = np.array([1, 1, 1, 1, 0, 1], np.uint8)
    want, want_lse = orc.attention("full", prob["q"], prob["k"], prob["v"], prob["table"], prob["seq_lens"],
                                   num_kv_heads=Hkv, block_size=16, layout=prob["layout"], layer_window=windows,
                                   layer_sinks=sinks, request_mask=flags_h, nthreads=4)
    dev = gh.upload(prob)
    flags = torch.from_numpy(flags_h).cuda()
    lay = prob["layout"]
    cfg = dict(num_layers=L, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=B,
               max_blocks_per_seq=prob["table"].shape[1], layer_window=windows, layer_sinks=sinks,
               layer_gated=gated, kv_layer_stride=lay.layer_stride, kv_block_stride=lay.block_stride,
               kv_token_stride=lay.token_stride, kv_head_stride=lay.head_stride, allow_empty=1)
    from paper_2609_20734_b200 import binding
    ctx = binding.OdaContext(binding.OdaConfig(**cfg))
    width = prob["table"].shape[1]
    parts_out = torch.full((world, L, B, Hq, D), float("nan"), device="cuda")
    parts_lse = torch.full((world, L, B, Hq), float("nan"), device="cuda")
    tokens = np.zeros((world, B), np.int32)
    for r in range(world):
        table_r = np.zeros((B, width), np.int32)
        for b, t in enumerate(seq):
            lo, hi, held = tp.sequence_shard(r, world, t)
            table_r[b, :hi - lo] = prob["table"][b, lo:hi]
            tokens[r, b] = held
        ctx.full_decode_gated(0, L, B, dev["q"], dev["k"], dev["v"], torch.from_numpy(table_r).cuda(),
                              torch.from_numpy(tokens[r]).cuda(), flags, parts_out[r], parts_lse[r])
    assert (tokens.sum(0) == np.array(seq)).all() and (world == 1 or (tokens == 0).any())
    out = torch.full((L, B, Hq, D), 7.0, device="cuda")
    lse = torch.full((L, B, Hq), 7.0, device="cuda")
    ctx.merge_partials(world, 0, L, B, parts_out, parts_lse, flags, out, lse, part_tokens=torch.from_numpy(tokens).cuda())
    torch.cuda.synchronize()
    assert ctx.read_device_status() == 0
    o, ls = out.cpu().numpy(), lse.cpu().numpy()
    for l in range(L):
        for b in range(B):
            if gated[l] and flags_h[b]:
                gh.assert_close(o[l, b], want[l, b], gh.ATOL_OUT, f"layer {l} request {b} out")
                gh.assert_close(ls[l, b], want_lse[l, b], gh.ATOL_LSE, f"layer {l} request {b} lse")
            else:
                assert (o[l, b] == 7.0).all() and (ls[l, b] == 7.0).all()   # untouched


def test_sharded_steps_through_nccl_on_one_rank():
    """The two sharded compositions with their collectives issued through torch.distributed's NCCL
    backend (a one-rank group: the library calls and the collectives share the current stream the
    way they do on several GPUs).  Results equal the unsharded library calls bitwise."""
    import os
    import socket

    import torch.distributed as dist

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    try:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
        probe = torch.ones(1, device="cuda")
        dist.all_reduce(probe)
        torch.cuda.synchronize()
    except Exception as e:  # no usable NCCL in this environment: the composition is covered by the tests above
        if dist.is_initialized():
            dist.destroy_process_group()
        pytest.skip(f"NCCL one-rank group unavailable: {e}")
    try:
        L, B, Hq, Hkv, D, d_ext, d_h = 2, 3, 8, 2, 128, 8, 24
        windows, sinks, gated = [64, 32], [4, 0], [1, 1]
        prob = make_problem(91, L, B, Hq, Hkv, D, [300, 40, 1000])
        head = dict(W1=synth.gauss_f32_tensor(9, synth.STREAM_W1, (d_h, d_ext + Hq * D), std=0.05),
                    b1=synth.gauss_f32_tensor(9, synth.STREAM_B1, (d_h,), std=0.05),
                    w2=synth.gauss_f32_tensor(9, synth.STREAM_W2, (d_h,), std=0.3),
                    b2=synth.gauss_f32_tensor(9, synth.STREAM_B2, (1,), std=0.05), use_attn_out=1)
        hd = gh.head_to_device(head)
        fe = torch.from_numpy(synth.gauss_f32_tensor(9, synth.STREAM_FEAT, (B, d_ext))).cuda()
        ctx = gh.make_ctx(prob, windows, sinks, gated, head=(d_ext, 1, d_h))
        dev = gh.upload(prob)
        # reference: the fused single-GPU step
        out0, lse0 = gh.new_out(prob)
        sc0 = torch.zeros(B, device="cuda")
        fl0 = torch.zeros(B, dtype=torch.uint8, device="cuda")
        ctx.step(ctx.step_args(B, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out0, sc0, fl0,
                               feat_ext=fe, head=hd, threshold=0.5, lse=lse0))
        # tensor-parallel composition on the one rank
        sh = tp.head_shard(0, 1, Hq, Hkv, D, d_ext, True)
        out1, lse1 = gh.new_out(prob)
        sc1 = torch.zeros(B, device="cuda")
        fl1 = torch.zeros(B, dtype=torch.uint8, device="cuda")
        pre = torch.zeros((B, d_h), device="cuda")
        tp.tp_step(ctx, sh, B, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out1, W1=hd["W1"],
                   b1=hd["b1"], w2=hd["w2"], b2=hd["b2"], threshold=0.5, pre=pre, scores=sc1, flags=fl1,
                   feat_ext=fe, lse=lse1)
        torch.cuda.synchronize()
        assert torch.equal(fl1, fl0)
        np.testing.assert_allclose(sc1.cpu().numpy(), sc0.cpu().numpy(), rtol=0, atol=1e-6)
        assert torch.equal(out1, out0) and torch.equal(lse1, lse0)
        # sequence-sharded composition on the one rank: gather + merge of a single part is the identity
        ones = torch.ones(B, dtype=torch.uint8, device="cuda")
        part_out, part_lse = gh.new_out(prob)
        parts_out = torch.zeros((1,) + tuple(part_out.shape), device="cuda")
        parts_lse = torch.zeros((1,) + tuple(part_lse.shape), device="cuda")
        out2 = torch.zeros_like(part_out)
        lse2 = torch.zeros_like(part_lse)
        tokens = dev["seq_lens"].reshape(1, B).contiguous()
        tp.sp_full_step(ctx, 1, B, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], tokens, ones,
                        part_out, part_lse, parts_out, parts_lse, out2, lse2)
        torch.cuda.synchronize()
        full, flse = gh.new_out(prob)
        ctx.full_decode_gated(0, L, B, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], ones, full, flse)
        torch.cuda.synchronize()
        np.testing.assert_allclose(out2.cpu().numpy(), full.cpu().numpy(), rtol=0, atol=1e-6)
        np.testing.assert_allclose(lse2.cpu().numpy(), flse.cpu().numpy(), rtol=0, atol=1e-6)
        assert ctx.read_device_status() == 0
    finally:
        dist.destroy_process_group()


def _exchange_setup(world, B, d_h, seed=3):
    recv = [torch.full((2, world, B, d_h), float("nan"), device="cuda") for _ in range(world)]
    arrived = [torch.zeros(world, dtype=torch.int32, device="cuda") for _ in range(world)]
    return recv, arrived


@pytest.mark.parametrize("world", [1, 2, 4, 8])
def test_fused_exchange_decision_matches_oracle_and_agrees_across_ranks(world):
    """The tensor-parallel decision with its exchange inside the kernel (peer stores + arrival
    flags instead of a collective call).  The ranks are the CTAs of one cooperative launch with
    separate buffers; three consecutive steps exercise the epoch flags and the alternating buffers."""
    B, d_in, d_h = 5, 8 * 64, 40
    ctx = gh.make_ctx(make_problem(1, 1, B, 8, 8, 64, [20] * B), [8], [0], [1], head=(0, 1, d_h))
    head = dict(W1=synth.gauss_f32_tensor(9, synth.STREAM_W1, (d_h, d_in), std=0.05),
                b1=synth.gauss_f32_tensor(9, synth.STREAM_B1, (d_h,), std=0.05),
                w2=synth.gauss_f32_tensor(9, synth.STREAM_W2, (d_h,), std=0.3),
                b2=synth.gauss_f32_tensor(9, synth.STREAM_B2, (1,), std=0.05), use_attn_out=1)
    hd = gh.head_to_device(head)
    recv, arrived = _exchange_setup(world, B, d_h)
    cols = d_in // world
    for step in range(3):
        x = synth.gauss_f32_tensor(20 + step, synth.STREAM_FEAT, (B, d_in))
        z, s = orc.recall_head(None, x.astype(np.float64), head["W1"], head["b1"], head["w2"], head["b2"])
        srt = np.sort(s)
        tau = float(0.5 * (srt[B // 2 - 1] + srt[B // 2]))
        xd = torch.from_numpy(x).cuda()
        ranks = []
        for r in range(world):   # each rank's share of W1 x: its columns only (fp64 product rounded to fp32)
            share = (xd[:, r * cols:(r + 1) * cols].double() @ hd["W1"][:, r * cols:(r + 1) * cols].double().T).float()
            ranks.append(dict(pre_local=share.contiguous(), scores=torch.zeros(B, device="cuda"),
                              logits=torch.zeros(B, device="cuda"),
                              flags=torch.full((B,), 7, dtype=torch.uint8, device="cuda"),
                              counters=torch.zeros((B, 2), dtype=torch.int32, device="cuda")))
        ctx.recall_finalize_exchange(B, world, 0, ranks, recv, arrived, step + 1, hd["b1"], hd["w2"], hd["b2"], tau)
        torch.cuda.synchronize()
        want = orc.flags(z, s, tau)
        decided = np.abs(s - tau) >= gh.FLAG_BAND
        for r in range(world):
            np.testing.assert_allclose(ranks[r]["scores"].cpu().numpy(), s, rtol=0, atol=gh.ATOL_SCORE)
            np.testing.assert_array_equal(ranks[r]["flags"].cpu().numpy()[decided], want[decided])
            assert torch.equal(ranks[r]["logits"], ranks[0]["logits"])       # bit for bit on every rank
            assert torch.equal(ranks[r]["flags"], ranks[0]["flags"])
            assert (ranks[r]["counters"][:, 0] == 1).all()
            assert (arrived[r] == step + 1).all()
    assert ctx.read_device_status() == 0


def test_fused_exchange_wait_runs_out_when_a_rank_never_arrives():
    """Three of four ranks make the call; the fourth never does.  Their waits end after the given
    limit, the status word says so, and the outputs are left alone (no trap, no hang)."""
    world, B, d_h = 4, 3, 16
    ctx = gh.make_ctx(make_problem(1, 1, B, 2, 2, 64, [20] * B), [8], [0], [1], head=(0, 1, d_h))
    recv, arrived = _exchange_setup(world, B, d_h)
    w = torch.zeros(d_h, device="cuda")
    one = torch.zeros(1, device="cuda")
    ranks = [dict(pre_local=torch.zeros((B, d_h), device="cuda"), scores=torch.full((B,), -1.0, device="cuda"),
                  flags=torch.full((B,), 9, dtype=torch.uint8, device="cuda")) for _ in range(3)]
    ctx.recall_finalize_exchange(B, world, 0, ranks, recv, arrived, 1, w, w, one, 0.5, timeout_ns=2_000_000)
    torch.cuda.synchronize()
    assert ctx.read_device_status() & 4
    for r in ranks:
        assert (r["scores"] == -1.0).all() and (r["flags"] == 9).all()
    assert ctx.read_device_status() == 0          # reading the word clears it


def test_tp_step_fused_on_one_rank_equals_the_fused_single_gpu_step():
    """world = 1: the step with the exchange kernel (a rank that only exchanges with itself) against
    the library's own single-GPU step, bit for bit on the attention outputs."""
    L, B, Hq, Hkv, D, d_ext, d_h = 2, 3, 8, 2, 128, 8, 24
    windows, sinks, gated = [64, 32], [4, 0], [1, 1]
    prob = make_problem(93, L, B, Hq, Hkv, D, [300, 40, 1000])
    head = dict(W1=synth.gauss_f32_tensor(9, synth.STREAM_W1, (d_h, d_ext + Hq * D), std=0.05),
                b1=synth.gauss_f32_tensor(9, synth.STREAM_B1, (d_h,), std=0.05),
                w2=synth.gauss_f32_tensor(9, synth.STREAM_W2, (d_h,), std=0.3),
                b2=synth.gauss_f32_tensor(9, synth.STREAM_B2, (1,), std=0.05), use_attn_out=1)
    hd = gh.head_to_device(head)
    fe = torch.from_numpy(synth.gauss_f32_tensor(9, synth.STREAM_FEAT, (B, d_ext))).cuda()
    ctx = gh.make_ctx(prob, windows, sinks, gated, head=(d_ext, 1, d_h))
    dev = gh.upload(prob)
    out0, lse0 = gh.new_out(prob)
    sc0 = torch.zeros(B, device="cuda")
    fl0 = torch.zeros(B, dtype=torch.uint8, device="cuda")
    ctx.step(ctx.step_args(B, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out0, sc0, fl0,
                           feat_ext=fe, head=hd, threshold=0.5, lse=lse0))
    sh = tp.head_shard(0, 1, Hq, Hkv, D, d_ext, True)
    bufs = tp.ExchangeBuffers.local(1, B, d_h)
    out1, lse1 = gh.new_out(prob)
    sc1 = torch.zeros(B, device="cuda")
    fl1 = torch.zeros(B, dtype=torch.uint8, device="cuda")
    pre = torch.zeros((B, d_h), device="cuda")
    for _ in range(2):   # two steps: epochs 1 and 2
        tp.tp_step_fused(ctx, sh, B, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out1, W1=hd["W1"],
                         b1=hd["b1"], w2=hd["w2"], b2=hd["b2"], threshold=0.5, pre=pre, scores=sc1, flags=fl1,
                         buffers=bufs, feat_ext=fe, lse=lse1)
    torch.cuda.synchronize()
    assert bufs.epoch == 2
    assert torch.equal(fl1, fl0) and torch.equal(out1, out0) and torch.equal(lse1, lse0)
    np.testing.assert_allclose(sc1.cpu().numpy(), sc0.cpu().numpy(), rtol=0, atol=1e-6)
    assert ctx.read_device_status() == 0


def _sp_problem(world, seed=41):
    L, B, Hq, Hkv, D = 3, 6, 8, 2, 128
    windows, sinks, gated = [64, 32, 64], [4, 0, 4], [1, 0, 1]
    seq = [100, 900, 5, 2500, 64, 17]
    prob = make_problem(seed, L, B, Hq, Hkv, D, seq)
    lay = prob["layout"]
    cfg = dict(num_layers=L, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, max_batch=B,
               max_blocks_per_seq=prob["table"].shape[1], layer_window=windows, layer_sinks=sinks,
               layer_gated=gated, kv_layer_stride=lay.layer_stride, kv_block_stride=lay.block_stride,
               kv_token_stride=lay.token_stride, kv_head_stride=lay.head_stride, allow_empty=1)
    from paper_2609_20734_b200 import binding
    ctx = binding.OdaContext(binding.OdaConfig(**cfg))
    width = prob["table"].shape[1]
    tables, tokens = [], np.zeros((world, B), np.int32)
    for r in range(world):
        table_r = np.zeros((B, width), np.int32)
        for b, t in enumerate(seq):
            lo, hi, held = tp.sequence_shard(r, world, t)
            table_r[b, :hi - lo] = prob["table"][b, lo:hi]
            tokens[r, b] = held
        tables.append(torch.from_numpy(table_r).cuda())
    return ctx, prob, (windows, sinks, gated), tables, tokens


@pytest.mark.parametrize("world", [1, 2, 4, 8])
def test_fused_merge_exchange_matches_oracle_on_every_rank(world):
    """Sequence-sharded Full pass whose exchange runs inside the merge kernel.  The ranks are the
    CTA columns of one cooperative launch (kernels that wait on one another never run as separate
    launches on one GPU).  Three exchanges in a row with different flags: every rank ends with the
    oracle's whole-history rows, bit-identical across ranks; unflagged rows stay untouched."""
    ctx, prob, (windows, sinks, gated), tables, tokens = _sp_problem(world)
    L, B, Hq, D = prob["q"].shape
    dev = gh.upload(prob)
    bufs = tp.MergeExchangeBuffers.local(world, L, B, Hq, D)
    for step, flags_h in enumerate([np.array([1, 1, 1, 1, 0, 1], np.uint8), np.array([0, 1, 0, 0, 1, 0], np.uint8),
                                    np.ones(6, np.uint8)]):
        want, want_lse = orc.attention("full", prob["q"], prob["k"], prob["v"], prob["table"], prob["seq_lens"],
                                       num_kv_heads=2, block_size=16,
                                       layout=prob["layout"], layer_window=windows, layer_sinks=sinks,
                                       request_mask=flags_h, nthreads=4)
        flags = torch.from_numpy(flags_h).cuda()
        ranks = []
        for r in range(world):
            po = torch.full((L, B, Hq, D), float("nan"), device="cuda")
            pl = torch.full((L, B, Hq), float("nan"), device="cuda")
            tok = torch.from_numpy(tokens[r]).cuda()
            ctx.full_decode_gated(0, L, B, dev["q"], dev["k"], dev["v"], tables[r], tok, flags, po, pl)
            ranks.append(dict(part_out=po, part_lse=pl, tokens_local=tok, flags=flags,
                              out=torch.full((L, B, Hq, D), 7.0, device="cuda"),
                              lse=torch.full((L, B, Hq), 7.0, device="cuda")))
        ctx.merge_partials_exchange(world, 0, ranks, bufs.recv_out, bufs.recv_lse, bufs.arrived, bufs.next_epoch(),
                                    0, L, B, timeout_ns=2_000_000_000)
        torch.cuda.synchronize()
        assert ctx.read_device_status() == 0
        o0, l0 = ranks[0]["out"].cpu().numpy(), ranks[0]["lse"].cpu().numpy()
        for r in range(1, world):
            np.testing.assert_array_equal(ranks[r]["out"].cpu().numpy(), o0)
            np.testing.assert_array_equal(ranks[r]["lse"].cpu().numpy(), l0)
        for l in range(L):
            for b in range(B):
                if gated[l] and flags_h[b]:
                    gh.assert_close(o0[l, b], want[l, b], gh.ATOL_OUT, f"step {step} layer {l} request {b} out")
                    gh.assert_close(l0[l, b], want_lse[l, b], gh.ATOL_LSE, f"step {step} layer {l} request {b} lse")
                else:
                    assert (o0[l, b] == 7.0).all() and (l0[l, b] == 7.0).all()
        for r in range(world):
            assert (bufs.arrived[r] == step + 1).all()


def test_fused_merge_exchange_equals_the_gathered_merge():
    """Same partial rows through the gathered merge and through the exchange kernel: same bits
    (both combine the parts in rank order with the same arithmetic)."""
    world = 4
    ctx, prob, _, tables, tokens = _sp_problem(world, seed=43)
    L, B, Hq, D = prob["q"].shape
    dev = gh.upload(prob)
    flags = torch.ones(B, dtype=torch.uint8, device="cuda")
    parts_out = torch.zeros((world, L, B, Hq, D), device="cuda")
    parts_lse = torch.zeros((world, L, B, Hq), device="cuda")
    toks = [torch.from_numpy(tokens[r]).cuda() for r in range(world)]
    for r in range(world):
        ctx.full_decode_gated(0, L, B, dev["q"], dev["k"], dev["v"], tables[r], toks[r], flags, parts_out[r], parts_lse[r])
    out_a = torch.zeros((L, B, Hq, D), device="cuda")
    lse_a = torch.zeros((L, B, Hq), device="cuda")
    ctx.merge_partials(world, 0, L, B, parts_out, parts_lse, flags, out_a, lse_a, part_tokens=torch.from_numpy(tokens).cuda())
    bufs = tp.MergeExchangeBuffers.local(world, L, B, Hq, D)
    ranks = [dict(part_out=parts_out[r], part_lse=parts_lse[r], tokens_local=toks[r], flags=flags,
                  out=torch.zeros((L, B, Hq, D), device="cuda"), lse=torch.zeros((L, B, Hq), device="cuda"))
             for r in range(world)]
    ctx.merge_partials_exchange(world, 0, ranks, bufs.recv_out, bufs.recv_lse, bufs.arrived, bufs.next_epoch(), 0, L, B)
    torch.cuda.synchronize()
    assert ctx.read_device_status() == 0
    np.testing.assert_array_equal(ranks[2]["out"].cpu().numpy(), out_a.cpu().numpy())
    np.testing.assert_array_equal(ranks[2]["lse"].cpu().numpy(), lse_a.cpu().numpy())


def test_fused_merge_exchange_wait_runs_out_when_a_rank_never_arrives():
    """One of two ranks makes the call.  Its wait ends at the limit, the status word says so, the
    output stays as it was."""
    world = 2
    ctx, prob, _, tables, tokens = _sp_problem(world)
    L, B, Hq, D = prob["q"].shape
    bufs = tp.MergeExchangeBuffers.local(world, L, B, Hq, D)
    rank0 = dict(part_out=torch.zeros((L, B, Hq, D), device="cuda"), part_lse=torch.zeros((L, B, Hq), device="cuda"),
                 out=torch.full((L, B, Hq, D), 7.0, device="cuda"), lse=torch.full((L, B, Hq), 7.0, device="cuda"))
    ctx.merge_partials_exchange(world, 0, [rank0], bufs.recv_out, bufs.recv_lse, bufs.arrived, 1, 0, L, B,
                                timeout_ns=2_000_000)
    torch.cuda.synchronize()
    assert ctx.read_device_status() & 4
    assert (rank0["out"] == 7.0).all() and (rank0["lse"] == 7.0).all()


def test_sp_full_step_fused_on_one_rank_equals_the_plain_full_pass():
    ctx, prob, (windows, sinks, gated), tables, tokens = _sp_problem(1)
    L, B, Hq, D = prob["q"].shape
    dev = gh.upload(prob)
    flags = torch.from_numpy(np.array([1, 0, 1, 1, 0, 1], np.uint8)).cuda()
    tok = torch.from_numpy(tokens[0]).cuda()
    ref_out = torch.full((L, B, Hq, D), 7.0, device="cuda")
    ref_lse = torch.full((L, B, Hq), 7.0, device="cuda")
    ctx.full_decode_gated(0, L, B, dev["q"], dev["k"], dev["v"], tables[0], tok, flags, ref_out, ref_lse)
    out = torch.full((L, B, Hq, D), 7.0, device="cuda")
    lse = torch.full((L, B, Hq), 7.0, device="cuda")
    bufs = tp.MergeExchangeBuffers.local(1, L, B, Hq, D)
    for _ in range(2):
        tp.sp_full_step_fused(ctx, 1, 0, B, dev["q"], dev["k"], dev["v"], tables[0], tok, flags,
                              torch.zeros((L, B, Hq, D), device="cuda"), torch.zeros((L, B, Hq), device="cuda"),
                              out, lse, buffers=bufs)
    torch.cuda.synchronize()
    assert ctx.read_device_status() == 0
    np.testing.assert_array_equal(out.cpu().numpy(), ref_out.cpu().numpy())
    np.testing.assert_array_equal(lse.cpu().numpy(), ref_lse.cpu().numpy())

