"""Planning-vocabulary calibration on the GPU (verified information gain, token statistics, filtering rule)
against the oracle, through the C interface."""
import numpy as np
import pytest
import torch

from oracle import calib as ocal
from oracle import score as oscore
from oracle import step as ostep
from paper_2601_12247_b200 import binding, synth
from gpu_util import dev, make_ctx, params_of, t_f32, t_i32, t_u8, to_np, upload_bits

pytestmark = pytest.mark.gpu

Q32 = 2.0 ** 32


def random_step(rng, n_seq, max_rows, K, vocab, tau_high):
    """Random draft-pass decisions (via the oracle's selection in calibration mode) and a random
    verification pass over them, all as arrays."""
    sizes = rng.integers(0, max_rows + 1, n_seq)
    seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    M = int(seg[-1])
    pos = np.concatenate([np.arange(s) for s in sizes]).astype(np.int32) if M else np.zeros(0, np.int32)
    conf = rng.random(M).astype(np.float32)
    tok = rng.integers(0, vocab, M).astype(np.int32)
    act = (rng.random(M) < 0.9).astype(np.uint8)
    cm = ostep.commit(conf, tok, seg, pos, act, tau_high)
    sel = ostep.select_drafts(conf, tok, np.zeros(M, np.uint8), cm["commit"], seg, pos, act, 0.15, 0.6, 0.1, K,
                              any_token=True, ar_fallback=False)
    Mv = int(sel["v_off"][-1])
    tok_v = np.zeros(Mv, np.int32)
    for b in range(n_seq):                                          # branches mostly agree with the base branch
        nR = int(sel["rem_off"][b + 1] - sel["rem_off"][b])
        if sel["n_drafts"][b] == 0:
            continue
        base = rng.integers(0, 4, nR)
        for c in range(1 + int(sel["n_drafts"][b])):
            o = int(sel["v_off"][b]) + c * nR
            tok_v[o:o + nR] = base if c == 0 else np.where(rng.random(nR) < 0.9, base, 9)
    conf_v = rng.random(Mv).astype(np.float32)
    ent_v = (rng.random(Mv) * 8).astype(np.float32)
    return dict(seg=seg, pos=pos, tok=tok, commit=cm["commit"], sel=sel, tok_v=tok_v, conf_v=conf_v, ent_v=ent_v)


def upload_sel(sel):
    return dict(rem_rows=t_i32(sel["rem_rows"]) if len(sel["rem_rows"]) else torch.zeros(1, dtype=torch.int32, device=dev()),
                rem_off=t_i32(sel["rem_off"]), v_off=t_i32(sel["v_off"]), draft_rows=t_i32(sel["draft_rows"]),
                n_drafts=t_i32(sel["n_drafts"]), route=t_u8(sel["route"]))


@pytest.mark.parametrize("n_seq,max_rows,K,exclude_self", [(1, 8, 4, False), (16, 32, 8, False), (64, 64, 16, True),
                                                           (40, 512, 64, False)])
def test_accumulate_and_filter_on_arrays(n_seq, max_rows, K, exclude_self):
    V, tau_high = 300, 0.7
    ctx = binding.Context(upload_bits(synth.make_w(3, V, 64)), [1], n_seq * max_rows + 1, max(n_seq, 1), K)
    flags = binding.PVF_EXCLUDE_SELF_FROM_IMPACT if exclude_self else 0
    prm = binding.make_params(tau_high, 0.15, 0.6, 0.1, K, flags)
    rng = np.random.default_rng(n_seq * 7 + K)
    stats = ctx.new_calib_stats()
    want = ocal.new_stats(V)
    n_events = 0
    for step in range(3):                                            # statistics accumulate across steps
        s = random_step(rng, n_seq, max_rows, K, V, tau_high)
        sel = s["sel"]
        over = ostep.verify(s["tok"], s["commit"], s["seg"], s["pos"], sel["rem_rows"], sel["rem_off"], sel["v_off"],
                            sel["draft_rows"], sel["n_drafts"], sel["route"], s["tok_v"], s["conf_v"], tau_high, K,
                            exclude_self)
        evs = ocal.events(s["tok"], sel["rem_rows"], sel["rem_off"], sel["v_off"], sel["draft_rows"], sel["n_drafts"],
                          sel["route"], s["tok_v"], s["conf_v"], s["ent_v"], tau_high, exclude_self)
        ocal.accumulate(want, evs)
        n_events += len(evs)
        # the GPU's own acceptance flags feed the accumulation, as in the real pipeline
        sel_d = upload_sel(sel)
        seg_d, pos_d = t_i32(s["seg"]), t_i32(s["pos"]) if len(s["pos"]) else torch.zeros(1, dtype=torch.int32, device=dev())
        one = lambda a, f: f(a) if len(a) else f(np.zeros(1, a.dtype))
        tok_d, tokv_d = one(s["tok"], t_i32), one(s["tok_v"], t_i32)
        confv_d, entv_d = one(s["conf_v"], t_f32), one(s["ent_v"], t_f32)
        ver = ctx.verify(prm, seg_d, pos_d, sel_d, tok_d, tokv_d, confv_d, one(s["commit"], t_u8))
        assert np.array_equal(to_np(ver)["accept"], over["accept"])
        vig_out = torch.full((n_seq, K), 7.0, dtype=torch.float64, device=dev())
        ctx.calib_accumulate(prm, sel_d, tok_d, confv_d, entv_d, ver["accept"], stats, vig_out)
        torch.cuda.synchronize()
        vig = vig_out.cpu().numpy()
        expect = np.zeros((n_seq, K))
        for e in evs:
            expect[e["seq"], e["j"] - 1] = e["VIG"]
        assert np.max(np.abs(vig - expect), initial=0.0) <= 1e-12
    got = to_np(stats)
    assert n_events > 0
    assert np.array_equal(got["n_v"], want["n"]) and np.array_equal(got["m_v"], want["m"])
    assert np.array_equal(got["sum_a"], want["sum_a"])
    assert np.max(np.abs(got["sum_vig_q32"] / Q32 - want["sum_vig"])) <= 1e-9 * max(1, n_events)
    assert ctx.last_status() == 0

    for n_min, m_min, rho, gam in [(1, 0, 0.0, -100.0), (2, 1, 0.5, 0.0), (3, 2, 0.9, 0.03), (1, 1, 1.0, 0.5)]:
        cal = binding.pvf_calib_params(0.15, 0.25, n_min, m_min, rho, gam)
        bitmap, n_plan = ctx.calib_filter(cal, stats)
        torch.cuda.synchronize()
        bits = np.unpackbits(bitmap.cpu().numpy().view(np.uint8), bitorder="little")[:V]
        keep = ocal.filter_tokens(want, n_min, m_min, rho, gam)
        want_bits = np.zeros(V, np.uint8); want_bits[keep] = 1
        vig_hat = np.divide(want["sum_vig"], np.maximum(want["n"], 1))
        dist = np.abs(vig_hat - float(np.float32(gam)))
        fragile = (want["n"] > 0) & (dist > 0) & (dist < 1e-7)       # a hair off the gamma threshold: may flip
        assert np.array_equal(bits[~fragile], want_bits[~fragile]) and fragile.sum() <= 2
        assert abs(int(n_plan.item()) - len(keep)) <= int(fragile.sum())
    ctx.close()


def test_calibration_pipeline_builds_a_planning_vocabulary():
    """score -> commit -> select (calibration candidates) -> score of the verification pass (with entropies)
    -> verify -> accumulate -> filter -> install the vocabulary, on synthetic hidden states."""
    V, D, n_seq, L = 4096, 256, 8, 32
    seed = 4321
    seg_rows = [(np.arange(L), np.ones(L, np.uint8)) for _ in range(n_seq)]
    st = synth.build_step("calib", seed, V, D, 256, seg_rows, L, L, dict(tau_high=0.9, budget=8), stress=True)
    p = dict(st.params, tau_plan_lo=0.15, tau_plan_hi=0.6)
    K = 8
    ctx = make_ctx(st.w_bits, st.plan_ids, n_seq * L * (2 + K), n_seq, K)
    prm = binding.make_params(p["tau_high"], p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"], K,
                              binding.PVF_SELECT_ANY_TOKEN | binding.PVF_NO_AR_FALLBACK)
    seg, pos = t_i32(st.seg_off), t_i32(st.row_pos)
    sc = ctx.score(upload_bits(st.h_bits))
    cm = ctx.commit(prm, seg, pos, None, sc["tok"], sc["conf"])
    sel = ctx.select_drafts(prm, seg, pos, None, sc["tok"], sc["conf"], None, cm["commit"])
    torch.cuda.synchronize()
    g_sc, g_cm, g_sel = to_np(sc), to_np(cm), to_np(sel)
    # the oracle on the GPU's own fp32 scores: decisions must agree exactly
    ocm = ostep.commit(g_sc["conf"], g_sc["tok"], st.seg_off, st.row_pos, None, p["tau_high"])
    osel = ostep.select_drafts(g_sc["conf"], g_sc["tok"], g_sc["in_plan"], ocm["commit"], st.seg_off, st.row_pos, None,
                               p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"], K, any_token=True, ar_fallback=False)
    assert np.array_equal(g_cm["commit"], ocm["commit"])
    for k in ("draft_rows", "n_drafts", "route", "rem_off", "v_off"):
        assert np.array_equal(g_sel[k], osel[k]), k
    assert (osel["route"] != 2).all() and osel["n_drafts"].sum() >= 8      # candidates exist, never the AR route
    vp = synth.make_verify_pass(st, osel["rem_rows"], osel["rem_off"], osel["n_drafts"])
    scv = ctx.score(upload_bits(vp.hv_bits))
    ver = ctx.verify(prm, seg, pos, sel, sc["tok"], scv["tok"], scv["conf"], cm["commit"])
    stats = ctx.new_calib_stats()
    ctx.calib_accumulate(prm, sel, sc["tok"], scv["conf"], scv["ent"], ver["accept"], stats)
    torch.cuda.synchronize()
    g_scv, g_ver = to_np(scv), to_np(ver)
    # entropies of the verification pass against the fp64 oracle
    oscv = oscore.score(st.w_bits, vp.hv_bits, st.plan_ids)
    assert np.max(np.abs(g_scv["ent"].astype(np.float64) - oscv["ent"])) <= 1e-3
    # statistics against the oracle fed with the GPU's fp32 verification-pass outputs
    evs = ocal.events(g_sc["tok"], osel["rem_rows"], osel["rem_off"], osel["v_off"], osel["draft_rows"], osel["n_drafts"],
                      osel["route"], g_scv["tok"], g_scv["conf"], g_scv["ent"], p["tau_high"])
    assert [e["A"] for e in evs] == [int(g_ver["accept"][e["seq"], e["j"] - 1]) for e in evs]
    want = ocal.accumulate(ocal.new_stats(V), evs)
    got = to_np(stats)
    assert np.array_equal(got["n_v"], want["n"]) and np.array_equal(got["m_v"], want["m"])
    assert np.array_equal(got["sum_a"], want["sum_a"])
    assert np.max(np.abs(got["sum_vig_q32"] / Q32 - want["sum_vig"])) <= 1e-8
    # filter with thresholds this small sample can meet, install the result and see pvf_score use it
    cal = binding.pvf_calib_params(0.15, 0.6, 1, 1, 0.5, -100.0)
    bitmap, n_plan = ctx.calib_filter(cal, stats)
    keep = ocal.filter_tokens(want, 1, 1, 0.5, -100.0)
    assert int(n_plan.item()) == len(keep) and len(keep) > 0
    ctx.set_plan_bitmap(bitmap)
    sc2 = to_np(ctx.score(upload_bits(st.h_bits)))
    assert np.array_equal(sc2["in_plan"], np.isin(sc2["tok"], keep).astype(np.uint8))
    assert ctx.last_status() == 0
    ctx.close()
