"""GPU parity: the CUDA attention kernels, called through the C-ABI, against the fp64 oracle on
the same seeded inputs, element by element."""
import numpy as np
import pytest
import torch

from paper_2609_20734_b200 import binding, synth
from tests import gpu_helpers as gh
from tests.helpers import make_problem, oracle_attention

pytestmark = pytest.mark.gpu

VARIANTS = [binding.VARIANT_SIMT, binding.VARIANT_TMA_MMA]
RAGGED = [1, 15, 16, 17, 300, 1000, 2053]


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("D,Hq,Hkv", [(128, 8, 2), (128, 8, 1), (64, 4, 1), (64, 4, 4), (128, 4, 2)])
@pytest.mark.parametrize("layout", ["hnd", "nhd"])
def test_local_parity_ragged(variant, D, Hq, Hkv, layout):
    L = 3
    prob = make_problem(100 + D + Hq, L, len(RAGGED), Hq, Hkv, D, RAGGED, layout=layout)
    windows, sinks, gated = [256, 64, 1024], [4, 0, 17], [1, 0, 1]
    ctx = gh.make_ctx(prob, windows, sinks, gated, variant=variant)
    dev = gh.upload(prob)
    out, lse = gh.gpu_local(ctx, prob, dev)
    ref, rlse = oracle_attention(prob, "local", windows, sinks, nthreads=8)
    gh.assert_close(out, ref, gh.ATOL_OUT, "local out")
    gh.assert_close(lse, rlse, gh.ATOL_LSE, "local lse")
    assert ctx.read_device_status() == 0


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("D,Hq,Hkv", [(128, 8, 2), (64, 8, 1)])
def test_full_gated_parity_and_untouched_rows(variant, D, Hq, Hkv):
    L = 4
    seq = [700, 33, 1, 4100, 257]
    prob = make_problem(7 + D, L, len(seq), Hq, Hkv, D, seq, layout="hnd")
    windows, sinks, gated = [64, 32, 64, 32], [4, 0, 4, 0], [1, 0, 1, 0]
    ctx = gh.make_ctx(prob, windows, sinks, gated, variant=variant)
    dev = gh.upload(prob)
    flags_h = np.array([1, 0, 1, 1, 0], dtype=np.uint8)
    flags = torch.from_numpy(flags_h).cuda()
    out, lse = gh.new_out(prob, fill=-77.0)
    ctx.full_decode_gated(0, L, len(seq), dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"],
                          flags, out, lse)
    torch.cuda.synchronize()
    out, lse = out.cpu().numpy(), lse.cpu().numpy()
    ref, rlse = oracle_attention(prob, "full", windows, sinks, nthreads=8)
    for l in range(L):
        for b in range(len(seq)):
            if gated[l] and flags_h[b]:
                gh.assert_close(out[l, b], ref[l, b], gh.ATOL_OUT, f"full out l{l} b{b}")
                gh.assert_close(lse[l, b], rlse[l, b], gh.ATOL_LSE, f"full lse l{l} b{b}")
            else:
                assert (out[l, b] == -77.0).all() and (lse[l, b] == -77.0).all()
    # all flags 0: nothing is written at all
    out2, lse2 = gh.new_out(prob, fill=-5.0)
    ctx.full_decode_gated(0, L, len(seq), dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"],
                          torch.zeros(len(seq), dtype=torch.uint8, device="cuda"), out2, lse2)
    torch.cuda.synchronize()
    assert (out2 == -5.0).all().item()
    assert ctx.read_device_status() == 0


@pytest.mark.parametrize("variant", VARIANTS)
def test_window_covering_sequence_equals_full(variant):
    seq = [5, 640, 1023]
    prob = make_problem(3, 2, 3, 8, 2, 128, seq)
    ctx = gh.make_ctx(prob, [1024, 2048], [0, 4], [1, 1], variant=variant)
    dev = gh.upload(prob)
    loc, llse = gh.gpu_local(ctx, prob, dev)
    out, lse = gh.new_out(prob)
    ctx.full_decode_gated(0, 2, 3, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"],
                          torch.ones(3, dtype=torch.uint8, device="cuda"), out, lse)
    torch.cuda.synchronize()
    np.testing.assert_allclose(out.cpu().numpy(), loc, rtol=0, atol=1e-6)
    np.testing.assert_allclose(lse.cpu().numpy(), llse, rtol=0, atol=1e-6)


@pytest.mark.parametrize("variant", VARIANTS)
def test_slots_past_the_sequence_and_unused_table_entries_are_never_used(variant):
    """Slots after position t-1 of the last page hold NaN bit patterns and table entries past
    ceil(t/16) are -1: the result must not change."""
    seq = [37, 130]
    prob = make_problem(9, 1, 2, 4, 1, 128, seq, shuffled=True)
    ref, _ = oracle_attention(prob, "local", [48], [4])
    lay = prob["layout"]
    for b, t in enumerate(seq):
        blk = int(prob["table"][b, (t - 1) // 16])
        for slot in range(t % 16, 16) if t % 16 else []:
            off = blk * lay.block_stride + slot * lay.token_stride
            prob["k"][off:off + 128] = 0x7FC0
            prob["v"][off:off + 128] = 0x7FC0
    assert (prob["table"][0, 3:] == -1).all()
    ctx = gh.make_ctx(prob, [48], [4], [1], variant=variant)
    out, _ = gh.gpu_local(ctx, prob, gh.upload(prob))
    gh.assert_close(out, ref, gh.ATOL_OUT, "poisoned tail")


@pytest.mark.parametrize("variant", VARIANTS)
def test_layer_ranges_kv_index_batch_prefix_and_determinism(variant):
    seq = [90, 500, 31]
    prob = make_problem(13, 4, 3, 8, 2, 128, seq, kv_layers=2)
    kvmap = [1, 0, 1, 0]
    windows, sinks, gated = [64] * 4, [4] * 4, [1] * 4
    ctx = gh.make_ctx(prob, windows, sinks, gated, kv_index=kvmap, variant=variant)
    dev = gh.upload(prob)
    ref, _ = oracle_attention(prob, "local", windows, sinks, layer_kv_index=kvmap, nthreads=8)
    whole, _ = gh.gpu_local(ctx, prob, dev)
    gh.assert_close(whole, ref, gh.ATOL_OUT, "kv_index")
    part, _ = gh.gpu_local(ctx, prob, dev, lb=1, le=3)
    assert np.isnan(part[0]).all() and np.isnan(part[3]).all()
    np.testing.assert_allclose(part[1:3], whole[1:3], rtol=0, atol=1e-5)   # another split of the same sums
    again, _ = gh.gpu_local(ctx, prob, dev)
    np.testing.assert_array_equal(again, whole)                # same call, same bits: determinism
    # batch = 0 and an empty layer range are no-ops
    out, lse = gh.new_out(prob, fill=3.0)
    ctx.local_decode(0, 4, 0, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out, lse)
    ctx.local_decode(2, 2, 3, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out, lse)
    torch.cuda.synchronize()
    assert (out == 3.0).all().item()


@pytest.mark.parametrize("variant", VARIANTS)
def test_custom_scale_and_bf16_output(variant):
    seq = [200, 77]
    prob = make_problem(17, 1, 2, 4, 2, 64, seq)
    ctx = gh.make_ctx(prob, [96], [2], [1], variant=variant, sm_scale=0.2, out_dtype=1)
    dev = gh.upload(prob)
    out = torch.zeros((1, 2, 4, 64), dtype=torch.bfloat16, device="cuda")
    ctx.local_decode(0, 1, 2, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out, None)
    torch.cuda.synchronize()
    ref, _ = oracle_attention(prob, "local", [96], [2], sm_scale=0.2)
    got = out.float().cpu().numpy().astype(np.float64)
    # bf16 output: within half a bf16 ulp of a value that meets the fp32 bar
    assert (np.abs(got - ref) <= gh.ATOL_OUT + np.abs(ref) * 2.0 ** -8).all()


@pytest.mark.parametrize("variant", VARIANTS)
def test_bad_seq_len_sets_status_without_trapping(variant):
    prob = make_problem(19, 1, 2, 4, 1, 64, [40, 40])
    ctx = gh.make_ctx(prob, [16], [0], [1], variant=variant)
    dev = gh.upload(prob)
    dev["seq_lens"] = torch.tensor([0, 40], dtype=torch.int32, device="cuda")
    out, lse = gh.new_out(prob, fill=9.0)
    ctx.local_decode(0, 1, 2, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], out, lse)
    torch.cuda.synchronize()
    assert ctx.read_device_status() & 1
    assert ctx.read_device_status() == 0           # reading clears it
    assert (out[0, 0] == 9.0).all().item()         # the bad row is left alone
    ref, _ = oracle_attention(prob, "local", [16], [0])
    gh.assert_close(out[0, 1].cpu().numpy(), ref[0, 1], gh.ATOL_OUT, "good row")


@pytest.mark.parametrize("variant", VARIANTS)
def test_peaked_softmax_short_sequences(variant):
    """Few tokens and large logits: the regime where rounding of the softmax weights would show."""
    seq = [2, 3, 5, 9]
    prob = make_problem(23, 1, 4, 8, 1, 128, seq)
    q = synth.bf16_bits_to_f32(prob["q"]) * 3.0
    prob["q"] = synth.f32_to_bf16_bits(q).reshape(prob["q"].shape)
    ctx = gh.make_ctx(prob, [4], [1], [1], variant=variant)
    dev = gh.upload(prob)
    out, lse = gh.gpu_local(ctx, prob, dev)
    ref, rlse = oracle_attention(prob, "local", [4], [1])
    gh.assert_close(out, ref, gh.ATOL_OUT, "peaked local")
    out2, _ = gh.new_out(prob)
    ctx.full_decode_gated(0, 1, 4, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"],
                          torch.ones(4, dtype=torch.uint8, device="cuda"), out2, None)
    torch.cuda.synchronize()
    reff, _ = oracle_attention(prob, "full", [4], [1])
    gh.assert_close(out2.cpu().numpy(), reff, gh.ATOL_OUT, "peaked full")


def test_calibrated_split_gives_the_same_result():
    """After a calibration run the spans follow the measured per-SM streaming rates: same oracle
    bar, same bits on a second run, and agreement with the equal split up to summation order."""
    seq = [40000, 700, 33, 20530, 1]
    prob = make_problem(29, 3, len(seq), 8, 2, 128, seq)
    windows, sinks, gated = [512, 64, 512], [4, 0, 4], [1, 0, 1]
    ctx = gh.make_ctx(prob, windows, sinks, gated, variant=binding.VARIANT_TMA_MMA)
    dev = gh.upload(prob)
    ones = torch.ones(len(seq), dtype=torch.uint8, device="cuda")
    before, _ = gh.new_out(prob)
    ctx.calibration_begin()
    ctx.full_decode_gated(0, 3, len(seq), dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], ones, before, None)
    spread = ctx.calibration_end()
    assert 0.3 < spread <= 1.0
    out, lse = gh.gpu_local(ctx, prob, dev)
    ref, rlse = oracle_attention(prob, "local", windows, sinks, nthreads=8)
    gh.assert_close(out, ref, gh.ATOL_OUT, "calibrated local")
    again, _ = gh.gpu_local(ctx, prob, dev)
    np.testing.assert_array_equal(again, out)
    full, flse = gh.new_out(prob)
    for _ in range(2):   # twice: the per-SM claim table must be re-armed between launches
        ctx.full_decode_gated(0, 3, len(seq), dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"], ones, full, flse)
    torch.cuda.synchronize()
    reff, _ = oracle_attention(prob, "full", windows, sinks, nthreads=8)
    for l in (0, 2):
        gh.assert_close(full[l].cpu().numpy(), reff[l], gh.ATOL_OUT, f"calibrated full layer {l}")
        np.testing.assert_allclose(full[l].cpu().numpy(), before[l].cpu().numpy(), rtol=0, atol=1e-5)
    assert ctx.read_device_status() == 0


@pytest.mark.parametrize("variant", VARIANTS)
def test_maximum_batch_many_layers_tiny_sequences(variant):
    """128 requests (the batch limit) of 1..200 tokens on 40 layers with three layer classes:
    many tiny units per span, most spans crossing many unit boundaries."""
    B, L = 128, 40
    rng = np.random.RandomState(5)
    seq = rng.randint(1, 201, size=B).tolist()
    seq[0], seq[1], seq[2] = 1, 16, 17
    prob = make_problem(31, L, B, 4, 2, 64, seq, layout="nhd")
    windows = [32 if l % 3 == 0 else (48 if l % 3 == 1 else 300) for l in range(L)]
    sinks = [4 if l % 3 == 0 else (0 if l % 3 == 1 else 2) for l in range(L)]
    gated = [1 if l % 3 != 1 else 0 for l in range(L)]
    ctx = gh.make_ctx(prob, windows, sinks, gated, variant=variant)
    dev = gh.upload(prob)
    out, lse = gh.gpu_local(ctx, prob, dev)
    ref, rlse = oracle_attention(prob, "local", windows, sinks, nthreads=8)
    gh.assert_close(out, ref, gh.ATOL_OUT, "max-batch local")
    gh.assert_close(lse, rlse, gh.ATOL_LSE, "max-batch lse")
    flags_h = (rng.rand(B) < 0.3).astype(np.uint8)
    full, _ = gh.new_out(prob, fill=-3.0)
    ctx.full_decode_gated(0, L, B, dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"],
                          torch.from_numpy(flags_h).cuda(), full, None)
    torch.cuda.synchronize()
    reff, _ = oracle_attention(prob, "full", windows, sinks, nthreads=8)
    full = full.cpu().numpy()
    for l in range(L):
        for b in range(B):
            if gated[l] and flags_h[b]:
                gh.assert_close(full[l, b], reff[l, b], gh.ATOL_OUT, f"max-batch full l{l} b{b}")
            else:
                assert (full[l, b] == -3.0).all()
    assert ctx.read_device_status() == 0


@pytest.mark.parametrize("variant", VARIANTS)
def test_layer_and_batch_limits_together(variant):
    """256 layers x 128 requests (both limits of a context) with four layer classes and group
    size 1: 32,768 units of 1..7 pages on one launch; one step beyond either limit is refused."""
    B, L = 128, 256
    rng = np.random.RandomState(11)
    seq = rng.randint(1, 100, size=B).tolist()
    prob = make_problem(57, L, B, 1, 1, 64, seq, kv_layers=2)
    classes = [(16, 0, 1), (40, 4, 1), (7, 1, 0), (64, 2, 1)]
    windows, sinks, gated = (list(v) for v in zip(*[classes[(l * 7) % 4] for l in range(L)]))
    kv_index = [l % 2 for l in range(L)]
    ctx = gh.make_ctx(prob, windows, sinks, gated, kv_index=kv_index, variant=variant)
    dev = gh.upload(prob)
    out, lse = gh.gpu_local(ctx, prob, dev)
    ref, rlse = oracle_attention(prob, "local", windows, sinks, layer_kv_index=kv_index, nthreads=8)
    gh.assert_close(out, ref, gh.ATOL_OUT, "limits local")
    gh.assert_close(lse, rlse, gh.ATOL_LSE, "limits lse")
    assert ctx.read_device_status() == 0
    with pytest.raises(binding.OdaError):
        gh.make_ctx(dict(prob, L=257), windows + [16], sinks + [0], gated + [1], kv_index=kv_index + [0], variant=variant)
    with pytest.raises(binding.OdaError):
        gh.make_ctx(prob, windows, sinks, gated, kv_index=kv_index, variant=variant, max_batch=129)


@pytest.mark.parametrize("layout", ["hnd", "nhd"])
def test_unit_aligned_split_parity(layout):
    """A short launch whose (layer, request, kv head) units are about one CTA's share each is cut at
    unit boundaries: every unit is streamed whole by one CTA and written without partials.  The
    shape below falls under that rule on a 148-SM part (checked; skipped elsewhere), with units of 32 and 33
    pages, a sink page each, and more CTAs than units; so does the Full pass over the same requests
    (units of 94 and 95 pages)."""
    L, Hq, Hkv, D = 10, 16, 8, 128
    seq = [1500, 1504, 1519]        # windows of 33, 32 and 33 pages
    windows, sinks, gated = [512] * L, [4] * L, [1] * L
    prob = make_problem(321, L, len(seq), Hq, Hkv, D, seq, layout=layout)
    ctx = gh.make_ctx(prob, windows, sinks, gated, variant=binding.VARIANT_TMA_MMA)
    units, pages = L * len(seq) * Hkv, L * Hkv * (33 + 32 + 33)
    span = pages / ctx.attention_grid
    if not (pages >= 16 * ctx.attention_grid and span <= 128 and span <= 32 and 33 <= 1.5 * span):
        pytest.skip(f"{units} units of 32-33 pages on {ctx.attention_grid} CTAs: outside the unit-aligned rule")
    dev = gh.upload(prob)
    out, lse = gh.gpu_local(ctx, prob, dev)
    ref, rlse = oracle_attention(prob, "local", windows, sinks, nthreads=8)
    gh.assert_close(out, ref, gh.ATOL_OUT, "local out")
    gh.assert_close(lse, rlse, gh.ATOL_LSE, "local lse")
    again, _ = gh.gpu_local(ctx, prob, dev)
    np.testing.assert_array_equal(again, out)
    fo, fl = gh.new_out(prob)
    ctx.full_decode_gated(0, L, len(seq), dev["q"], dev["k"], dev["v"], dev["table"], dev["seq_lens"],
                          torch.ones(len(seq), dtype=torch.uint8, device="cuda"), fo, fl)
    torch.cuda.synchronize()
    ref, rlse = oracle_attention(prob, "full", windows, sinks, nthreads=8)
    gh.assert_close(fo.cpu().numpy(), ref, gh.ATOL_OUT, "full out")
    gh.assert_close(fl.cpu().numpy(), rlse, gh.ATOL_LSE, "full lse")
    assert ctx.read_device_status() == 0


def _unit_aligned_case(case, grid):
    """Draws shapes until one falls under the unit-aligned rule of the plan (average span of at most
    128 pages, at least 16; every unit between 1 and 3/2 of it) on a launch of `grid` CTAs."""
    rng = np.random.default_rng(4400 + case)
    for _ in range(10000):
        L, B, Hkv = int(rng.integers(2, 13)), int(rng.integers(1, 5)), int(rng.choice([1, 2, 4, 8]))
        w, s = int(rng.choice([128, 200, 256, 384, 512, 777])), int(rng.choice([0, 4, 17]))
        seq = [int(rng.integers(max(2, w // 2), 3 * w)) for _ in range(B)]
        pages = []
        for t in seq:   # pages of the window segment (Eq. 1); a separate sink page is not part of the unit's length
            lo = 0 if t - w <= s else t - w
            pages.append((t + 15) // 16 - lo // 16)
        total, span = L * Hkv * sum(pages), L * Hkv * sum(pages) / grid
        if total >= 16 * grid and span <= 128 and span <= min(pages) and max(pages) <= 1.5 * span:
            return dict(L=L, B=B, Hkv=Hkv, w=w, s=s, seq=seq, G=int(rng.choice([1, 2, 4, 8])),
                        layout=str(rng.choice(["hnd", "nhd"])), seed=int(rng.integers(1, 10**6)))
    raise AssertionError("no eligible shape drawn")


@pytest.mark.parametrize("case", range(6))
def test_unit_aligned_split_random_shapes(case):
    probe = gh.make_ctx(make_problem(1, 1, 1, 8, 8, 128, [40]), [16], [0], [1], variant=binding.VARIANT_TMA_MMA)
    c = _unit_aligned_case(case, probe.attention_grid)
    L, B, Hkv = c["L"], c["B"], c["Hkv"]
    windows, sinks, gated = [c["w"]] * L, [c["s"]] * L, [1] * L
    prob = make_problem(c["seed"], L, B, c["G"] * Hkv, Hkv, 128, c["seq"], layout=c["layout"])
    ctx = gh.make_ctx(prob, windows, sinks, gated, variant=binding.VARIANT_TMA_MMA)
    assert ctx.attention_grid == probe.attention_grid
    dev = gh.upload(prob)
    out, lse = gh.gpu_local(ctx, prob, dev)
    ref, rlse = oracle_attention(prob, "local", windows, sinks, nthreads=8)
    gh.assert_close(out, ref, gh.ATOL_OUT, f"local out {c}")
    gh.assert_close(lse, rlse, gh.ATOL_LSE, f"local lse {c}")
    assert ctx.read_device_status() == 0


def test_cache_resident_hint_changes_no_bits():
    """The L2 evict-last hint on the leading layers' windows is a hint: same bits with any budget."""
    L, Hq, Hkv, D = 6, 8, 2, 128
    seq = [900, 70, 2053]
    windows, sinks, gated = [256] * L, [4] * L, [1] * L
    prob = make_problem(55, L, len(seq), Hq, Hkv, D, seq)
    ctx = gh.make_ctx(prob, windows, sinks, gated, variant=binding.VARIANT_TMA_MMA)
    dev = gh.upload(prob)
    base, base_lse = gh.gpu_local(ctx, prob, dev)
    per_layer = len(seq) * Hkv * (256 + 4) * D * 4
    for budget in (per_layer - 1, 3 * per_layer, 1 << 40):   # no layer, three layers, all of them
        ctx.set_cache_resident_bytes(budget)
        out, lse = gh.gpu_local(ctx, prob, dev)
        np.testing.assert_array_equal(out, base)
        np.testing.assert_array_equal(lse, base_lse)
    ctx.set_cache_resident_bytes(0)
    ref, _ = oracle_attention(prob, "local", windows, sinks, nthreads=8)
    gh.assert_close(base, ref, gh.ATOL_OUT, "local out")
    assert ctx.read_device_status() == 0


@pytest.mark.parametrize("layout,t", [("hnd", 700), ("nhd", 1024), ("hnd", 519), ("hnd", 400)])
def test_batch_one_unit_per_cta_parity(layout, t):
    """Batch 1 with about as many (layer, kv head) units as CTAs: the plan gives CTA u unit u without
    any scan.  Lengths: window and sinks apart (unaligned and page-aligned), window just past the
    sinks, and shorter than the window (one range); layers alias three cache slices."""
    L, Hq, Hkv, D = 30, 16, 8, 128
    windows, sinks, gated = [512] * L, [4] * L, [1] * L
    kv_index = [l % 3 for l in range(L)]
    prob = make_problem(808 + t, L, 1, Hq, Hkv, D, [t], layout=layout, kv_layers=3)
    ctx = gh.make_ctx(prob, windows, sinks, gated, kv_index=kv_index, variant=binding.VARIANT_TMA_MMA)
    grid, units = ctx.attention_grid, L * Hkv
    if not (units <= grid <= 1.5 * units):
        pytest.skip(f"{units} units on {grid} CTAs: outside the one-unit-per-CTA rule")
    dev = gh.upload(prob)
    out, lse = gh.gpu_local(ctx, prob, dev)
    ref, rlse = oracle_attention(prob, "local", windows, sinks, nthreads=8, layer_kv_index=kv_index)
    gh.assert_close(out, ref, gh.ATOL_OUT, "local out")
    gh.assert_close(lse, rlse, gh.ATOL_LSE, "local lse")
    again, _ = gh.gpu_local(ctx, prob, dev)
    np.testing.assert_array_equal(again, out)
    assert ctx.read_device_status() == 0



@pytest.mark.parametrize("layout,Hq,Hkv,D,w,s", [("hnd", 32, 8, 128, 1024, 4), ("nhd", 8, 2, 128, 256, 0),
                                                 ("hnd", 8, 1, 64, 100, 17), ("hnd", 16, 2, 128, 2048, 4)])
def test_batch_one_identical_units_plan_in_registers(layout, Hq, Hkv, D, w, s):
    """Batch 1 over layers of one class: every unit has the same length and the equal split is taken in
    closed form from the one length (no shared plan).  Whole stacks and layer ranges (one launch per
    layer is what a backbone issues), lengths around the page, sink and window edges; the layers alias
    cache slices so that the per-item layer lookup is exercised; same bits on a second run, and the
    same bits as the same request inside a batch of two (which takes the general plan)."""
    L = 5
    kv_index = [l % 2 for l in range(L)]
    for t in (1, 16, 17, w + s - 1, w + s, w + s + 1, 3 * w + 9):
        prob = make_problem(4000 + t, L, 1, Hq, Hkv, D, [t], layout=layout, kv_layers=2)
        ctx = gh.make_ctx(prob, [w] * L, [s] * L, [1] * L, kv_index=kv_index, variant=binding.VARIANT_TMA_MMA)
        dev = gh.upload(prob)
        ref, rlse = oracle_attention(prob, "local", [w] * L, [s] * L, nthreads=8, layer_kv_index=kv_index)
        whole, whole_lse = gh.gpu_local(ctx, prob, dev)
        gh.assert_close(whole, ref, gh.ATOL_OUT, f"t={t} whole stack")
        gh.assert_close(whole_lse, rlse, gh.ATOL_LSE, f"t={t} whole stack lse")
        for lb, le in ((0, 1), (2, 3), (1, 4), (4, 5)):
            out, lse = gh.gpu_local(ctx, prob, dev, lb, le)
            gh.assert_close(out[lb:le], ref[lb:le], gh.ATOL_OUT, f"t={t} layers [{lb},{le})")
            gh.assert_close(lse[lb:le], rlse[lb:le], gh.ATOL_LSE, f"t={t} layers [{lb},{le}) lse")
            assert np.isnan(out[:lb]).all() and np.isnan(out[le:]).all()      # other layers untouched
        again, _ = gh.gpu_local(ctx, prob, dev)
        np.testing.assert_array_equal(again, whole)
        # the same request as request 0 of a batch of two: the general plan cuts the same spans
        prob2 = dict(prob, B=2, q=np.ascontiguousarray(np.repeat(prob["q"], 2, axis=1)),
                     table=np.ascontiguousarray(np.repeat(prob["table"], 2, axis=0)),
                     seq_lens=np.array([t, t], np.int32))
        ctx2 = gh.make_ctx(prob2, [w] * L, [s] * L, [1] * L, kv_index=kv_index, variant=binding.VARIANT_TMA_MMA)
        dev2 = gh.upload(prob2)
        both, _ = gh.gpu_local(ctx2, prob2, dev2)
        gh.assert_close(both[:, 0], ref[:, 0], gh.ATOL_OUT, f"t={t} as request 0 of two")
        gh.assert_close(both[:, 1], ref[:, 0], gh.ATOL_OUT, f"t={t} as request 1 of two")
        assert ctx.read_device_status() == 0 and ctx2.read_device_status() == 0
