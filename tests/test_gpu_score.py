"""pvf_score against the fp64 oracle, element by element, through the C interface."""
import numpy as np
import pytest
import torch

from oracle import score as oscore
from paper_2601_12247_b200 import binding, synth
from gpu_util import check_score, check_score_properties, dev, make_ctx, to_np, upload_bits

pytestmark = pytest.mark.gpu


def run_and_compare(w_bits, h_bits, plan_ids, max_rows=None, rows=None):
    ctx = make_ctx(w_bits, plan_ids, max_rows or max(1, h_bits.shape[0]))
    h = upload_bits(h_bits)
    got = to_np(ctx.score(h))
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    again = to_np(ctx.score(h))
    torch.cuda.synchronize()
    for k in got:
        assert np.array_equal(got[k], again[k]), "run-to-run difference in " + k
    sub = h_bits if rows is None else h_bits[rows]
    want = oscore.score(w_bits, sub, plan_ids)
    near = check_score(got, want, w_bits.shape[0], plan_ids, rows)
    check_score_properties(got, w_bits.shape[0], plan_ids)
    ctx.close()
    return got, want, near


@pytest.mark.parametrize("stress", [False, True])
def test_config0_tiny(stress):
    st = synth.config0(stress=stress)
    got, want, near = run_and_compare(st.w_bits, st.h_bits, st.plan_ids)
    assert near <= 2


@pytest.mark.parametrize("V,D,M", [(4096, 256, 1), (4096, 256, 7), (4096, 256, 128), (4096, 256, 129),
                                   (5000, 200, 150), (1000, 64, 33), (16, 8, 3), (70000, 512, 300),
                                   (4096, 256, 16), (4096, 256, 17), (4096, 256, 31), (4096, 256, 32),
                                   (5000, 200, 20), (70000, 512, 30), (100, 64, 5), (300, 72, 9), (40000, 136, 32),
                                   (4096, 256, 40), (5000, 200, 64), (300, 72, 50), (70000, 512, 160), (40000, 136, 191),
                                   (5000, 200, 192), (100, 64, 130), (4100, 256, 65), (4100, 256, 193),
                                   (4096, 256, 257), (5000, 200, 290), (70000, 512, 448), (300, 72, 449), (40000, 136, 400)])
def test_ragged_shapes(V, D, M):
    # several row tiles, vocabulary not a multiple of 16 or 32, hidden size not a multiple of 64; up to 32 rows take
    # the swapped-operand streaming kernel, 33 .. 64, 129 .. 192 and 257 .. 448 rows the swapped paired kernel (rows
    # padded to a multiple of 32; above 256 in two column groups; vocabularies of fewer granules than pairs of
    # SMs), other counts the 128-row GEMM kernel or the paired kernel
    pos = np.arange(M)
    st = synth.build_step("ragged", 4242, V, D, min(64, V), [(pos, np.ones(M, np.uint8))], M, M,
                          dict(tau_high=0.9, budget=4), amp_max=40.0 * (256.0 / D) ** 0.5)
    run_and_compare(st.w_bits, st.h_bits, st.plan_ids)


def test_uniform_and_peaked_closed_forms():
    # all-zero hidden state -> p = 1/V, H = ln V, token 0;  W = c*I -> one logit a*c, the rest 0
    V = 256
    w = synth.f32_to_bf16_bits(0.5 * np.eye(V, dtype=np.float32))
    h = np.zeros((3, V), np.float32); h[1, 17] = 8.0; h[2, 255] = 30.0
    ctx = make_ctx(w, [17], 8)
    got = to_np(ctx.score(upload_bits(synth.f32_to_bf16_bits(h))))
    assert got["tok"].tolist() == [0, 17, 255] and got["in_plan"].tolist() == [0, 1, 0]
    Z = np.exp(4.0) + V - 1
    assert abs(got["conf"][0] - 1.0 / V) < 1e-6 and abs(got["ent"][0] - np.log(V)) < 1e-4
    assert abs(got["conf"][1] - np.exp(4.0) / Z) < 1e-5 and abs(got["ent"][1] - (np.log(Z) - 4.0 * np.exp(4.0) / Z)) < 1e-4
    Z2 = np.exp(15.0) + V - 1
    assert abs(got["conf"][2] - np.exp(15.0) / Z2) < 1e-5
    assert abs(got["ent"][2] - (np.log(Z2) - 15.0 * np.exp(15.0) / Z2)) < 1e-4
    ctx.close()


def test_exact_tie_goes_to_lowest_id_across_ranges():
    # identical weight rows far apart in the vocabulary: equal logits in different blocks' ranges
    V, D = 4096, 64
    w = synth.make_w(9, V, D)
    w[3000] = w[10]; w[4095] = w[10]
    h = (synth.bf16_bits_to_f32(w[10]).astype(np.float32) * 400.0)[None, :]
    ctx = make_ctx(w, [10], 8)
    got = to_np(ctx.score(upload_bits(synth.f32_to_bf16_bits(h))))
    assert got["tok"][0] == 10 and got["in_plan"][0] == 1
    ctx.close()


@pytest.mark.parametrize("M", [1, 20, 40, 100, 150, 300])
def test_exact_ties_inside_one_range(M):
    # equal logits at ids that one block sees on the same accumulator lane (10 and 138), in its other
    # 128-entry slice (138), in a later tile (300) and in another block's range (60000)
    V, D = 70000, 64
    w = synth.make_w(11, V, D)
    for v in (138, 300, 60000):
        w[v] = w[10]
    w[20000] = w[19999]
    h = np.zeros((M, D), np.float32)
    h[:] = synth.bf16_bits_to_f32(w[10]).astype(np.float32) * 400.0
    h[M - 1] = synth.bf16_bits_to_f32(w[19999]).astype(np.float32) * 400.0
    ctx = make_ctx(w, [10], 512)
    got = to_np(ctx.score(upload_bits(synth.f32_to_bf16_bits(h))))
    assert (got["tok"][:M - 1] == 10).all() and got["tok"][M - 1] == 19999
    ctx.close()


@pytest.mark.parametrize("max_rows", [33, 64, 100, 129, 192, 200, 300, 448, 460, 600])
def test_workspace_covers_every_row_count_up_to_max_rows(max_rows):
    # the kernels leave a different number of partial states per row (148 in the swapped paired kernel's windows,
    # 74 just above them): a context sized for max_rows must serve every smaller call
    V, D = 4800, 64
    w = synth.make_w(5, V, D)
    ctx = make_ctx(w, [1], max_rows)
    h = upload_bits(synth.make_w(6, max_rows, D))
    for M in sorted({1, 32, 33, 64, 65, 128, 129, 192, 193, 256, 257, 448, 449, 512, max_rows}):
        if M <= max_rows:
            out = ctx.score(h[:M])
            assert out["tok"].shape[0] == M
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    ctx.close()


def test_argument_errors_launch_nothing():
    st = synth.config0()
    ctx = make_ctx(st.w_bits, st.plan_ids, 64)
    h = upload_bits(st.h_bits)
    out = ctx.score(h[:0])                                        # M = 0 is a no-op
    assert out["tok"].numel() == 0
    big = upload_bits(np.concatenate([st.h_bits, st.h_bits]))
    with pytest.raises(binding.PvfError) as e:
        ctx.score(big)                                            # above max_rows
    assert e.value.code == binding.PVF_ERR_INVALID
    flat = torch.empty(64 * 256 + 8, dtype=torch.bfloat16, device=dev())
    mis = flat[1:1 + 64 * 256].view(64, 256)                      # 2-byte offset: not 16-byte aligned
    with pytest.raises(binding.PvfError) as e:
        ctx.score(mis)
    assert e.value.code == binding.PVF_ERR_ALIGN
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    ctx.close()


@pytest.mark.parametrize("M", [8, 48, 100, 160, 300])
def test_non_finite_hidden_rows_stay_in_bounds_and_do_not_disturb_other_rows(M):
    # rows holding NaN or Inf have unspecified outputs, but the call terminates, reports no error, returns valid
    # token ids, and every other row is scored as if they were not there (all four kernels)
    V, D = 5000, 200
    pos = np.arange(M)
    st = synth.build_step("nonfinite", 99, V, D, 64, [(pos, np.ones(M, np.uint8))], M, M,
                          dict(tau_high=0.9, budget=4), amp_max=40.0 * (256.0 / D) ** 0.5)
    h = st.h_bits.copy()
    nan, inf, ninf = 0x7FC0, 0x7F80, 0xFF80                       # bf16 bit patterns
    bad = [1, M // 2, M - 1]
    h[bad[0], 3] = nan
    h[bad[1], :] = inf
    h[bad[2], 0] = ninf
    ctx = make_ctx(st.w_bits, st.plan_ids, M)
    got = to_np(ctx.score(upload_bits(h)))
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    assert np.all((got["tok"] >= 0) & (got["tok"] < V)) and np.all(got["in_plan"] <= 1)
    good = np.setdiff1d(np.arange(M), bad)
    want = oscore.score(st.w_bits, st.h_bits[good], st.plan_ids)
    check_score(got, want, V, st.plan_ids, rows=good)
    ctx.close()


@pytest.mark.parametrize("copies", [1, 2, 5, 32, 256])
def test_small_tail_terms_are_not_lost_beside_a_dominant_logit(copies):
    # One logit 11 .. 20 above a narrow bulk (hidden size 1024: the other logits spread by 0.5 only): every other
    # term e^{x - max} is near or below the fp32 rounding unit of 1.0, yet there are 70000 of them and together
    # they hold up to a per cent of the probability mass.  A running sum that contains the dominant term's 1.0
    # rounds them away -- the more, the longer the vocabulary range one block sweeps, i.e. the more rows the call
    # has: 64 distinct rows are scored once (swapped paired kernel, 74 ranges), twice over (128 rows: 128-row
    # kernel, 148 ranges), 5 times over (320 rows: swapped paired kernel in two column groups), 32 times over (2048
    # rows, paired kernel) and 256 times over (16384 rows, few ranges per row tile).
    V, D, M = 70000, 1024, 64
    w = synth.make_w(21, V, D)
    targets = (np.arange(M) * 331 + 7) % V
    amps = np.linspace(18.0, 32.0, M)
    keys = np.stack([np.zeros(M, np.int64), np.arange(M), np.zeros(M, np.int64)], axis=1)
    h = synth.make_hidden_rows(w, targets, amps, 21, synth.TAG_NOISE, keys)
    plan = synth.make_plan_ids(21, V, 64)
    want = oscore.score(w, h, plan)
    assert ((1.0 - want["conf"]) > 1e-3).sum() >= M // 4 and want["gap"].min() > 8.0     # the case under test is present
    ctx = make_ctx(w, plan, M * copies)
    got = to_np(ctx.score(upload_bits(np.tile(h, (copies, 1)))))
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    for c in sorted({0, copies // 2, copies - 1}):
        rows = np.arange(c * M, (c + 1) * M)
        check_score(got, want, V, plan, rows=rows)
        # far inside the tolerance: a lost tail shows as an error of a fifth to a half of 1 - conf (up to 1e-3 here)
        assert np.max(np.abs(got["conf"][rows] - want["conf"])) <= 1e-4
        assert np.max(np.abs(got["ent"][rows] - want["ent"])) <= 3e-4
    ctx.close()


@pytest.mark.parametrize("M", [24, 48, 200, 300])
def test_hidden_states_written_just_before_the_call_are_the_ones_scored(M):
    """Stream order: the scoring kernels fetch weights ahead of the work queued before them, never hidden states.
    One buffer is overwritten on the stream right before every call, alternating between two sets of rows, with no
    synchronisation in between; every call must see the rows written last (each kernel kind: streaming, swapped
    paired, paired, swapped paired with two column groups)."""
    V, D = 4096, 256
    pos = np.arange(M)
    st = synth.build_step("order", 4300, V, D, 64, [(pos, np.ones(M, np.uint8))], M, M, dict(tau_high=0.9, budget=4),
                          amp_max=40.0)
    w_bits, plan_ids = st.w_bits, st.plan_ids
    sets = [st.h_bits, np.ascontiguousarray(st.h_bits[::-1])]          # the same rows in reverse order
    want = [oscore.score(w_bits, s, plan_ids) for s in sets]
    assert not np.array_equal(want[0]["tok"], want[1]["tok"])
    ctx = make_ctx(w_bits, plan_ids, M)
    src = [upload_bits(s) for s in sets]
    h = torch.zeros_like(src[0])
    outs = []
    for i in range(12):
        h.copy_(src[i % 2])                       # a kernel on the same stream, queued right before the call
        outs.append(ctx.score(h))
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    for i, out in enumerate(outs):
        check_score(to_np(out), want[i % 2], V, plan_ids)
    ctx.close()
