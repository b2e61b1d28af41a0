"""The whole step (score -> commit -> select -> verification-pass score -> verify) on the synthetic
configurations, GPU against oracle.  LLaDA-shaped cases score every row on the GPU in the launch
geometry the benchmark times and check a sample of rows against the oracle one by one."""
import numpy as np
import pytest
import torch

from oracle import score as oscore
from oracle import step as ostep
from paper_2601_12247_b200 import binding, synth
from gpu_util import (FRAGILE, NEAR_TIE, check_score, check_score_properties, dev, make_ctx, params_of, t_i32, t_u8,
                      to_np, upload_bits)

pytestmark = pytest.mark.gpu


def fragile_rows(conf, thresholds):
    bad = np.zeros(len(conf), bool)
    for t in thresholds:
        bad |= np.abs(conf - float(np.float32(t))) < FRAGILE
    return bad


def full_step(ctx, st, flags=0):
    """GPU step and oracle step, each on its own scores; decisions must agree on every sequence
    that holds no near-tie or threshold-fragile row."""
    p = st.params
    prm = params_of(st, flags)
    seg, pos, act = t_i32(st.seg_off), t_i32(st.row_pos), t_u8(st.active)
    sc = ctx.score(upload_bits(st.h_bits))
    cm = ctx.commit(prm, seg, pos, act, sc["tok"], sc["conf"])
    sel = ctx.select_drafts(prm, seg, pos, act, sc["tok"], sc["conf"], sc["in_plan"], cm["commit"])
    torch.cuda.synchronize()

    osc = oscore.score(st.w_bits, st.h_bits, st.plan_ids)
    check_score(to_np(sc), osc, st.vocab, st.plan_ids)
    force = bool(flags & binding.PVF_FORCE_PROGRESS)
    ocm = ostep.commit(osc["conf"], osc["tok"], st.seg_off, st.row_pos, st.active, p["tau_high"], force)
    osel = ostep.select_drafts(osc["conf"], osc["tok"], osc["in_plan"], ocm["commit"], st.seg_off, st.row_pos,
                               st.active, p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"], p["budget"])
    bad_row = (osc["gap"] < NEAR_TIE) | fragile_rows(osc["conf"], [p["tau_high"], p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"]])
    seq_ok = np.array([not bad_row[st.seg_off[b]:st.seg_off[b + 1]].any() for b in range(st.n_seq)])
    # top-k fragility: K-th and (K+1)-th candidate closer than FRAGILE
    for b in range(st.n_seq):
        rows = np.arange(st.seg_off[b], st.seg_off[b + 1])
        cand = [m for m in rows if st.active[m] and not ocm["commit"][m] and osc["in_plan"][m]
                and np.float32(p["tau_plan_lo"]) <= osc["conf"][m] < np.float32(p["tau_plan_hi"])]
        cs = sorted((osc["conf"][m] for m in cand), reverse=True)
        K = p["budget"]
        if len(cs) > K and cs[K - 1] - cs[K] < FRAGILE:
            seq_ok[b] = False
    g_cm, g_sel = to_np(cm), to_np(sel)
    row_ok = np.repeat(seq_ok, np.diff(st.seg_off))
    assert np.array_equal(g_cm["commit"][row_ok], ocm["commit"][row_ok])
    for b in np.nonzero(seq_ok)[0]:
        assert np.array_equal(g_sel["draft_rows"][b], osel["draft_rows"][b])
        assert g_sel["route"][b] == osel["route"][b] and g_sel["n_drafts"][b] == osel["n_drafts"][b]
    return sc, cm, sel, osc, ocm, osel, seq_ok


def verify_pass(ctx, st, sc, cm, sel, osc, ocm, osel, seq_ok, flags=0):
    """Verification pass laid out from the ORACLE's draft decisions (so that it lines up even when a
    fragile sequence made the GPU draft differently): the GPU scores it and verifies it with the
    oracle's selection uploaded; everything is compared sequence by sequence."""
    p = st.params
    prm = params_of(st, flags)
    v = synth.make_verify_pass(st, osel["rem_rows"], osel["rem_off"], osel["n_drafts"])
    assert np.array_equal(v.v_off, osel["v_off"])
    scv = ctx.score(upload_bits(v.hv_bits))
    seg, pos = t_i32(st.seg_off), t_i32(st.row_pos)
    sel_up = dict(rem_rows=t_i32(osel["rem_rows"]), rem_off=t_i32(osel["rem_off"]), v_off=t_i32(osel["v_off"]),
                  draft_rows=t_i32(osel["draft_rows"]), n_drafts=t_i32(osel["n_drafts"]), route=t_u8(osel["route"]))
    ver = ctx.verify(prm, seg, pos, sel_up, t_i32(osc["tok"]), scv["tok"], scv["conf"], t_u8(ocm["commit"]))
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    oscv = oscore.score(st.w_bits, v.hv_bits, st.plan_ids)
    if v.hv_bits.shape[0]:
        check_score(to_np(scv), oscv, st.vocab, st.plan_ids)
    over = ostep.verify(osc["tok"], ocm["commit"], st.seg_off, st.row_pos, osel["rem_rows"], osel["rem_off"],
                        osel["v_off"], osel["draft_rows"], osel["n_drafts"], osel["route"], oscv["tok"], oscv["conf"],
                        p["tau_high"], p["budget"])
    gv = to_np(ver)
    bad_v = (oscv["gap"] < NEAR_TIE) | fragile_rows(oscv["conf"], [p["tau_high"]])
    margins = ostep.c_total_margins(osel["rem_rows"], osel["rem_off"], osel["v_off"], osel["draft_rows"],
                                    osel["n_drafts"], osel["route"], oscv["conf"], over["accept"])
    n_checked = 0
    for b in range(st.n_seq):
        if bad_v[osel["v_off"][b]:osel["v_off"][b + 1]].any() or margins[b] < 1e-3:
            continue
        n_checked += 1
        assert np.array_equal(gv["accept"][b], over["accept"][b]) and gv["choice"][b] == over["choice"][b]
        rows = slice(st.seg_off[b], st.seg_off[b + 1])
        assert np.array_equal(gv["final_commit"][rows], over["final_commit"][rows])
    assert n_checked >= (st.n_seq + 1) // 2 or st.n_seq == 1
    return over, n_checked


@pytest.mark.parametrize("stress", [False, True])
def test_config0_full_step(stress):
    st = synth.config0(stress=stress)
    ctx = make_ctx(st.w_bits, st.plan_ids, 4096)
    parts = full_step(ctx, st)
    verify_pass(ctx, st, *parts)
    ctx.close()


@pytest.mark.parametrize("stress", [False, True])
def test_config2_and_3_at_small_vocab(stress):
    # the batched and large-batch row layouts at a vocabulary the oracle scores in seconds
    w = synth.make_w(2002, 8192, 256)
    ctx = make_ctx(w, synth.make_plan_ids(1002, 8192, 2048), 8192, 64, 16)
    st2 = synth.config2(stress=stress, w_bits=w, vocab=8192, hidden=256)
    over = verify_pass(ctx, st2, *full_step(ctx, st2))
    ctx.close()
    st3 = synth.config3(stress=stress, w_bits=w, vocab=8192, hidden=256, n_seq=8, gen_len=128)
    ctx = make_ctx(w, st3.plan_ids, 65536, 64, 16)
    verify_pass(ctx, st3, *full_step(ctx, st3))
    ctx.close()


@pytest.mark.parametrize("force", [0, binding.PVF_FORCE_PROGRESS])
def test_step_calls_equal_the_four_calls(force):
    # pvf_draft_step / pvf_verify_step (two launches each) against pvf_score, pvf_commit, pvf_select_drafts, pvf_verify
    # called one by one: the same kernels on the same inputs, so every output is bit-identical, canvas included
    w = synth.make_w(2002, 8192, 256)
    st = synth.config2(stress=True, w_bits=w, vocab=8192, hidden=256)
    ctx = make_ctx(w, st.plan_ids, 8192, 64, 16)
    prm = params_of(st, force, tau_high=0.97 if force else st.params["tau_high"])
    seg, pos, act = t_i32(st.seg_off), t_i32(st.row_pos), t_u8(st.active)
    h = upload_bits(st.h_bits)
    y_a = torch.full((st.n_seq, st.gen_len), -1, dtype=torch.int32, device=dev())
    y_b = y_a.clone()
    sc = ctx.score(h)
    cm = ctx.commit(prm, seg, pos, act, sc["tok"], sc["conf"], y=y_a)
    sel = ctx.select_drafts(prm, seg, pos, act, sc["tok"], sc["conf"], sc["in_plan"], cm["commit"])
    d = ctx.draft_step(prm, h, seg, pos, act, y=y_b)
    torch.cuda.synchronize()
    one, two = dict(to_np(sc), **to_np(cm), **to_np(sel)), to_np(d)
    n_rem = int(one["rem_off"][-1])
    for k in one:
        a, b = (one[k][:n_rem], two[k][:n_rem]) if k == "rem_rows" else (one[k], two[k])
        assert np.array_equal(a.view(np.uint8), b.view(np.uint8)), k
    assert torch.equal(y_a, y_b)
    v = synth.make_verify_pass(st, one["rem_rows"][:n_rem], one["rem_off"], one["n_drafts"])
    assert v.hv_bits.shape[0] > 0
    hv = upload_bits(v.hv_bits)
    scv = ctx.score(hv)
    ver = ctx.verify(prm, seg, pos, sel, sc["tok"], scv["tok"], scv["conf"], cm["commit"], y=y_a)
    vs = ctx.verify_step(prm, hv, seg, pos, d, y=y_b)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    assert torch.equal(scv["tok"], vs["tok_v"]) and torch.equal(scv["conf"].view(torch.int32), vs["conf_v"].view(torch.int32))
    for k in ("accept", "choice", "final_commit"):
        assert torch.equal(ver[k], vs[k]), k
    assert torch.equal(y_a, y_b) and (to_np(ver)["choice"] > 0).any()
    ctx.close()


def test_scores_are_identical_from_run_to_run():
    # the tail's merge is done by whichever block finishes last, in an order fixed by the data layout alone: repeated
    # calls give the same bits, for every kernel (row counts of the streaming, swapped, 128-row and paired kernels)
    w = synth.make_w(2003, 20000, 512)
    pos = np.arange(600)
    st = synth.build_step("repeat", 2003, 20000, 512, 256, [(pos, np.ones(600, np.uint8))], 600, 600,
                          dict(tau_high=0.9, budget=4), stress=True, w_bits=w)
    ctx = make_ctx(w, st.plan_ids, 1024)
    kernels = set()
    for rows in (24, 60, 100, 170, 256, 300, 600):
        h = upload_bits(st.h_bits[:rows])
        kernels.add(ctx.score_kernel_name(rows))
        first = to_np(ctx.score(h))
        for _ in range(5):
            again = to_np(ctx.score(h))
            for k in first:
                assert np.array_equal(first[k].view(np.uint8), again[k].view(np.uint8)), (rows, k)
    assert len(kernels) == 4 and ctx.last_status() == 0
    ctx.close()


# ------------------------------------------------------------------------------ LLaDA shape
@pytest.fixture(scope="module")
def llada():
    w_bits = synth.make_w(1001, synth.LLADA_VOCAB, synth.LLADA_HIDDEN)
    plan = synth.make_plan_ids(1001, synth.LLADA_VOCAB, 2048)
    ctx = make_ctx(w_bits, plan, 32768, 64, 16)
    yield w_bits, plan, ctx
    ctx.close()


def sampled_parity(ctx, st, w_bits, plan, sample):
    h = upload_bits(st.h_bits)
    got = to_np(ctx.score(h))
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    check_score_properties(got, st.vocab, plan)
    want = oscore.score(w_bits, st.h_bits[sample], plan)
    check_score(got, want, st.vocab, plan, rows=sample)
    return got


def test_config1a_every_row(llada):
    w_bits, plan, ctx = llada
    st = synth.config1("a", w_bits=w_bits)
    assert ctx.score_plan(32)["ctas"] == torch.cuda.get_device_properties(0).multi_processor_count
    parts = full_step(ctx, st)
    assert parts[-1].all()


def test_config1a_stress_every_row(llada):
    w_bits, plan, ctx = llada
    st = synth.config1("a", stress=True, w_bits=w_bits)
    full_step(ctx, st)


def test_config1b_sampled(llada):
    w_bits, plan, ctx = llada
    st = synth.config1("b", w_bits=w_bits)
    sampled_parity(ctx, st, w_bits, plan, np.array([0, 31, 32, 127, 128, 129, 200, 255]))


def test_config2_full_step_on_the_oracles_own_scores(llada):
    # every draft and verification row of config 2 scored by the oracle itself: decisions compared end to end
    w_bits, _, _ = llada
    st = synth.config2(w_bits=w_bits)
    ctx = make_ctx(w_bits, st.plan_ids, 8192, 64, 16)          # config 2 has a planning vocabulary of its own
    over, n_checked = verify_pass(ctx, st, *full_step(ctx, st))
    assert n_checked >= st.n_seq // 2
    ctx.close()


def test_config2_at_batch_24_sampled(llada):
    # config 2's recipe with 24 sequences: 354 rows, which the swapped paired kernel takes in two column groups
    # (rows 0..255 and 256..383 of one accumulator); sampled on both sides of the group boundary, at the edges of
    # the 32-row chunks the epilogue warps alternate on, and on the last real row
    w_bits, plan, ctx = llada
    st = synth.config2(w_bits=w_bits, n_seq=24)
    assert 256 < st.n_rows <= 448 and ctx.score_kernel_name(st.n_rows) == "pvf_score_swap_pair_kernel"
    M = st.n_rows
    sampled_parity(ctx, st, w_bits, plan, np.array([0, 31, 32, 127, 128, 255, 256, 257, 287, 288, 319, 320, M - 1]))


def test_config2_sampled_rows_and_decisions_on_gpu_scores(llada):
    w_bits, plan, ctx = llada
    st = synth.config2(w_bits=w_bits)
    M = st.n_rows
    got = sampled_parity(ctx, st, w_bits, plan, np.unique(np.linspace(0, M - 1, 12).astype(int)))
    # consistency of the decision kernels with the scoring kernel's outputs: fed the same fp32 numbers, the
    # oracle's decision rules must give the same sets (the scores themselves are checked on sampled rows above
    # and on every row in test_config2_full_step_on_the_oracles_own_scores)
    p = st.params
    prm = params_of(st)
    seg, pos, act = t_i32(st.seg_off), t_i32(st.row_pos), t_u8(st.active)
    sc = ctx.score(upload_bits(st.h_bits))
    cm = ctx.commit(prm, seg, pos, act, sc["tok"], sc["conf"])
    sel = ctx.select_drafts(prm, seg, pos, act, sc["tok"], sc["conf"], sc["in_plan"], cm["commit"])
    ocm = ostep.commit(got["conf"], got["tok"], st.seg_off, st.row_pos, st.active, p["tau_high"])
    osel = ostep.select_drafts(got["conf"], got["tok"], got["in_plan"], ocm["commit"], st.seg_off, st.row_pos,
                               st.active, p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"], p["budget"])
    assert np.array_equal(to_np(cm)["commit"], ocm["commit"])
    gs = to_np(sel)
    for k in ("draft_rows", "n_drafts", "route", "rem_off", "v_off"):
        assert np.array_equal(gs[k], osel[k]), k
    v = synth.make_verify_pass(st, osel["rem_rows"], osel["rem_off"], osel["n_drafts"])
    scv = ctx.score(upload_bits(v.hv_bits))
    ver = ctx.verify(prm, seg, pos, sel, sc["tok"], scv["tok"], scv["conf"], cm["commit"])
    gscv = to_np(scv)
    over = ostep.verify(got["tok"], ocm["commit"], st.seg_off, st.row_pos, osel["rem_rows"], osel["rem_off"],
                        osel["v_off"], osel["draft_rows"], osel["n_drafts"], osel["route"], gscv["tok"], gscv["conf"],
                        p["tau_high"], p["budget"])
    gv = to_np(ver)
    for k in ("accept", "choice", "final_commit"):
        assert np.array_equal(gv[k], over[k]), k
    Mv = v.hv_bits.shape[0]
    if Mv:
        rows = np.unique(np.linspace(0, Mv - 1, 6).astype(int))
        check_score(gscv, oscore.score(w_bits, v.hv_bits[rows], plan), st.vocab, plan, rows=rows)


def test_paired_kernel_two_waves_sampled(llada):
    # 4096 rows: 16 tiles of 256 rows, 8 in flight, 9 vocabulary ranges, 2 waves of the paired kernel
    w_bits, plan, ctx = llada
    st = synth.config3(w_bits=w_bits, n_seq=8)
    assert st.n_rows == 4096 and ctx.score_kernel_name(4096) == "pvf_score_gemm_pair_kernel"
    assert ctx.score_plan(4096)["waves"] == 2
    sampled_parity(ctx, st, w_bits, plan, np.array([0, 127, 128, 255, 256, 2047, 2048, 2303, 2304, 4095]))


def test_second_model_shape_sampled():
    # Dream-7B-like LM head: 56 k-panels, 9504 vocabulary granules (64.2 per block): all four kernels
    V, D = synth.DREAM_VOCAB, synth.DREAM_HIDDEN
    w_bits = synth.make_w(1005, V, D)
    plan = synth.make_plan_ids(1005, V, 2048)
    ctx = make_ctx(w_bits, plan, 512, 8, 8)
    st = synth.config1("b", stress=True, w_bits=w_bits, vocab=V, hidden=D)
    h_bits = np.concatenate([st.h_bits, st.h_bits[:64][::-1]])            # 320 rows: the last 64 repeat earlier ones
    for rows, kernel, sample in ((32, "pvf_score_stream_kernel", np.array([0, 1, 15, 16, 30, 31])),
                                 (48, "pvf_score_swap_pair_kernel", np.array([0, 23, 24, 32, 47])),
                                 (100, "pvf_score_gemm_kernel", np.array([0, 31, 32, 64, 99])),
                                 (170, "pvf_score_swap_pair_kernel", np.array([0, 95, 96, 128, 169])),
                                 (256, "pvf_score_gemm_pair_kernel", np.array([0, 127, 128, 129, 255])),
                                 (300, "pvf_score_swap_pair_kernel", np.array([0, 127, 128, 255, 256, 277, 278, 299]))):
        assert ctx.score_kernel_name(rows) == kernel
        got = to_np(ctx.score(upload_bits(h_bits[:rows])))
        torch.cuda.synchronize()
        assert ctx.last_status() == 0
        check_score_properties(got, V, plan)
        check_score(got, oscore.score(w_bits, h_bits[sample], plan), V, plan, rows=sample)
    ctx.close()


def test_config3_large_batch_sampled(llada):
    w_bits, plan, ctx = llada
    st = synth.config3(w_bits=w_bits)
    assert st.n_rows == 32768
    geo = ctx.score_plan(st.n_rows)
    assert geo["waves"] >= 2 and geo["ctas"] <= torch.cuda.get_device_properties(0).multi_processor_count
    sample = np.array([0, 127, 128, 4735, 4736, 16383, 20000, 32767])
    got = sampled_parity(ctx, st, w_bits, plan, sample)
    p = st.params
    prm = params_of(st)
    seg, pos, act = t_i32(st.seg_off), t_i32(st.row_pos), t_u8(st.active)
    sc = dict(tok=t_i32(got["tok"]), conf=torch.from_numpy(got["conf"]).to(dev()), in_plan=t_u8(got["in_plan"]))
    cm = ctx.commit(prm, seg, pos, act, sc["tok"], sc["conf"])
    sel = ctx.select_drafts(prm, seg, pos, act, sc["tok"], sc["conf"], sc["in_plan"], cm["commit"])
    ocm = ostep.commit(got["conf"], got["tok"], st.seg_off, st.row_pos, st.active, p["tau_high"])
    osel = ostep.select_drafts(got["conf"], got["tok"], got["in_plan"], ocm["commit"], st.seg_off, st.row_pos,
                               st.active, p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"], p["budget"])
    assert np.array_equal(to_np(cm)["commit"], ocm["commit"])
    gs = to_np(sel)
    for k in ("draft_rows", "n_drafts", "route", "rem_off", "v_off"):
        assert np.array_equal(gs[k], osel[k]), k
    # every one of the 32768 rows against a second reference: torch's fp64 matmul and log-softmax on the GPU (not
    # the oracle -- the oracle checks 8 + 512 rows of this launch above and below, and pins this reference on the
    # sampled rows); it is what catches an error that only a few rows in ten thousand show
    wd = ctx.w_head.double()
    hd = upload_bits(st.h_bits)
    ref_conf = np.empty(st.n_rows); ref_ent = np.empty(st.n_rows); ref_tok = np.empty(st.n_rows, np.int64); ref_gap = np.empty(st.n_rows)
    for r0 in range(0, st.n_rows, 1024):
        lp = torch.log_softmax(hd[r0:r0 + 1024].double() @ wd.t(), dim=1)
        top2 = lp.topk(2, dim=1)
        ref_conf[r0:r0 + 1024] = top2.values[:, 0].exp().cpu().numpy()
        ref_tok[r0:r0 + 1024] = top2.indices[:, 0].cpu().numpy()
        ref_gap[r0:r0 + 1024] = (top2.values[:, 0] - top2.values[:, 1]).cpu().numpy()
        ref_ent[r0:r0 + 1024] = (-(lp.exp() * lp).sum(dim=1)).cpu().numpy()
        del lp
    want_s = oscore.score(w_bits, st.h_bits[sample], plan)
    assert np.max(np.abs(ref_conf[sample] - want_s["conf"])) < 1e-9 and np.max(np.abs(ref_ent[sample] - want_s["ent"])) < 1e-9
    assert np.array_equal(ref_tok[sample], want_s["tok"])
    assert np.max(np.abs(got["conf"] - ref_conf)) <= 1e-3 and np.max(np.abs(got["ent"] - ref_ent)) <= 1e-3
    clear = ref_gap >= NEAR_TIE
    assert np.array_equal(got["tok"][clear], ref_tok[clear]) and (~clear).sum() < 100
    del wd
    # one whole sequence end to end on the oracle's own scores (512 rows is what the oracle scores in seconds)
    b = 41
    r0, r1 = int(st.seg_off[b]), int(st.seg_off[b + 1])
    osc = oscore.score(w_bits, st.h_bits[r0:r1], plan)
    check_score(got, osc, st.vocab, plan, rows=np.arange(r0, r1))
    one = np.array([0, r1 - r0], np.int32)
    ocm1 = ostep.commit(osc["conf"], osc["tok"], one, st.row_pos[r0:r1], st.active[r0:r1], p["tau_high"])
    osel1 = ostep.select_drafts(osc["conf"], osc["tok"], osc["in_plan"], ocm1["commit"], one, st.row_pos[r0:r1],
                                st.active[r0:r1], p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"], p["budget"])
    taus = [p["tau_high"], p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"]]
    if not ((osc["gap"] < NEAR_TIE) | fragile_rows(osc["conf"], taus)).any():
        assert np.array_equal(to_np(cm)["commit"][r0:r1], ocm1["commit"])
        want_rows = np.where(osel1["draft_rows"][0] >= 0, osel1["draft_rows"][0] + r0, -1)
        assert np.array_equal(gs["draft_rows"][b], want_rows)
        assert gs["route"][b] == osel1["route"][0] and gs["n_drafts"][b] == osel1["n_drafts"][0]
        assert gs["rem_off"][b + 1] - gs["rem_off"][b] == osel1["rem_off"][1]


def torch_fp64_reference(w_head, h_dev, chunk=1024):
    """Every row of a launch against a second reference (torch's fp64 matmul and log-softmax on the GPU): conf, ent,
    tok and the top-2 gap.  Not the oracle: the caller pins it to the oracle on sampled rows."""
    n = h_dev.shape[0]
    wd = w_head.double()
    conf = np.empty(n); ent = np.empty(n); tok = np.empty(n, np.int64); gap = np.empty(n)
    for r0 in range(0, n, chunk):
        lp = torch.log_softmax(h_dev[r0:r0 + chunk].double() @ wd.t(), dim=1)
        top2 = lp.topk(2, dim=1)
        conf[r0:r0 + chunk] = top2.values[:, 0].exp().cpu().numpy()
        tok[r0:r0 + chunk] = top2.indices[:, 0].cpu().numpy()
        gap[r0:r0 + chunk] = (top2.values[:, 0] - top2.values[:, 1]).cpu().numpy()
        ent[r0:r0 + chunk] = (-(lp.exp() * lp).sum(dim=1)).cpu().numpy()
        del lp
    del wd
    return conf, ent, tok, gap


def test_config3_verification_pass_sampled():
    # Config 3's verification pass at its stated size: the 64 sequences' (1 + K_t) * |R_b| rows (about 10^5, eleven
    # passes over W of the paired kernel, the last one a partial wave) scored in the geometry the benchmark times.  Sampled rows against the
    # oracle one by one, every row against the torch fp64 reference that is pinned to the oracle on that sample, and
    # pvf_verify on the GPU's own fp32 numbers against the oracle's rule fed the same numbers.
    w_bits = synth.make_w(1001, synth.LLADA_VOCAB, synth.LLADA_HIDDEN)
    st = synth.config3(w_bits=w_bits)
    plan = st.plan_ids
    p = st.params
    K = int(p["budget"])
    ctx = make_ctx(w_bits, plan, 131072, 64, 16)
    prm = params_of(st)
    seg, pos, act = t_i32(st.seg_off), t_i32(st.row_pos), t_u8(st.active)
    sc = ctx.score(upload_bits(st.h_bits))
    cm = ctx.commit(prm, seg, pos, act, sc["tok"], sc["conf"])
    sel = ctx.select_drafts(prm, seg, pos, act, sc["tok"], sc["conf"], sc["in_plan"], cm["commit"])
    torch.cuda.synchronize()
    g_sc, g_cm, gs = to_np(sc), to_np(cm), to_np(sel)
    # the draft-pass decisions follow the oracle's rules on the GPU's own numbers (the scores themselves are checked
    # in test_config3_large_batch_sampled)
    ocm = ostep.commit(g_sc["conf"], g_sc["tok"], st.seg_off, st.row_pos, st.active, p["tau_high"])
    osel = ostep.select_drafts(g_sc["conf"], g_sc["tok"], g_sc["in_plan"], ocm["commit"], st.seg_off, st.row_pos,
                               st.active, p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"], K)
    assert np.array_equal(g_cm["commit"], ocm["commit"])
    for k in ("draft_rows", "n_drafts", "route", "rem_off", "v_off"):
        assert np.array_equal(gs[k], osel[k]), k
    n_rem = int(osel["rem_off"][-1])
    assert np.array_equal(gs["rem_rows"][:n_rem], osel["rem_rows"][:n_rem])
    v = synth.make_verify_pass(st, osel["rem_rows"], osel["rem_off"], osel["n_drafts"])
    Mv = int(v.hv_bits.shape[0])
    assert np.array_equal(v.v_off, osel["v_off"]) and Mv > 65536
    geo = ctx.score_plan(Mv)
    assert geo["waves"] >= 8 and ctx.score_kernel_name(Mv) == "pvf_score_gemm_pair_kernel"
    full = binding.score_plan_for_shape(st.vocab, st.hidden, torch.cuda.get_device_properties(0).multi_processor_count, Mv)
    hv = upload_bits(v.hv_bits)
    scv = ctx.score(hv)
    ver = ctx.verify(prm, seg, pos, sel, sc["tok"], scv["tok"], scv["conf"], cm["commit"])
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
    g_scv, gv = to_np(scv), to_np(ver)
    check_score_properties(g_scv, st.vocab, plan)
    # sampled rows: first and last row, both sides of a 128-row tile edge, of a wave edge (rows per pass over W) and
    # of sequence boundaries of the [b][c][r] layout
    rows_per_wave = min(256 * full["tiles_per_wave"], Mv - 1)
    last_wave = rows_per_wave * (full["waves"] - 1)                   # first row of the last wave (split over more pairs)
    sample = np.unique(np.clip(np.array([0, 127, 128, 255, 256, rows_per_wave - 1, rows_per_wave, int(v.v_off[1]) - 1,
                                         int(v.v_off[1]), int(v.v_off[32]), Mv // 2, last_wave - 1, last_wave, Mv - 129,
                                         Mv - 128, Mv - 1]), 0, Mv - 1))
    want = oscore.score(w_bits, v.hv_bits[sample], plan)
    check_score(g_scv, want, st.vocab, plan, rows=sample)
    ref_conf, ref_ent, ref_tok, ref_gap = torch_fp64_reference(ctx.w_head, hv)
    assert np.max(np.abs(ref_conf[sample] - want["conf"])) < 1e-9 and np.max(np.abs(ref_ent[sample] - want["ent"])) < 1e-9
    assert np.array_equal(ref_tok[sample], want["tok"])
    assert np.max(np.abs(g_scv["conf"] - ref_conf)) <= 1e-3 and np.max(np.abs(g_scv["ent"] - ref_ent)) <= 1e-3
    clear = ref_gap >= NEAR_TIE
    assert np.array_equal(g_scv["tok"][clear], ref_tok[clear]) and (~clear).sum() < 300
    # acceptance, branch choice and final commit: the oracle's rule on the GPU's own verification-pass numbers
    over = ostep.verify(g_sc["tok"], ocm["commit"], st.seg_off, st.row_pos, osel["rem_rows"], osel["rem_off"], osel["v_off"],
                        osel["draft_rows"], osel["n_drafts"], osel["route"], g_scv["tok"], g_scv["conf"].astype(np.float64),
                        p["tau_high"], K)
    for k in ("accept", "choice", "final_commit"):
        assert np.array_equal(gv[k], over[k]), k
    assert (osel["route"] > 0).sum() >= st.n_seq // 2                  # the pass is not an empty formality
    ctx.close()
