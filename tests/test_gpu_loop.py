"""Config 4: the synthetic decode loop on the GPU against the oracle's loop, state by state."""
import numpy as np
import pytest
import torch

from oracle import loop as oloop
from oracle import score as oscore
from paper_2601_12247_b200 import binding, decode_loop, synth
from gpu_util import FRAGILE, NEAR_TIE, check_score, dev, make_ctx, to_np


def fragile_step(h, p):
    """True if the oracle's step holds a row whose decision could legitimately flip on the GPU."""
    def bad(sc, taus):
        f = sc["gap"] < NEAR_TIE
        for t in taus:
            f |= np.abs(sc["conf"] - float(np.float32(t))) < FRAGILE
        return bool(f.any())
    return bad(h["score"], [p["tau_high"], p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"]])


@pytest.mark.gpu
@pytest.mark.parametrize("budget,q_plan,n_sparse", [(4, 0.5, 0), (0, 0.0, 0), (3, 0.0, 0), (4, 0.5, 5), (0, 0.0, 8)])
def test_loop_tiny_shape_state_by_state(budget, q_plan, n_sparse):
    V, D, B, L, S, seed = 4096, 256, 4, 64, 32, 1004
    w = synth.make_w(seed, V, D)
    plan = synth.make_plan_ids(seed, V, 256)
    tg = synth.loop_targets(seed, V, B, L, plan, q_plan, avoid=V - 1)
    p = dict(tau_high=0.9, budget=budget, **synth.DEFAULT_BAND)
    mask = V - 1
    want = oloop.decode(synth, w, plan, tg, seed, L, S, p, mask, trace=True, n_sparse=n_sparse)
    ctx = make_ctx(w, plan, B * 2 * S * (2 + budget), B, max(budget, 1))
    trace = []
    got = decode_loop.decode(ctx, w, tg, seed, L, S, p, mask, on_step=lambda s, d: trace.append(d), n_sparse=n_sparse)
    assert got["status"] == 0
    n_same = 0
    for s, (g, o) in enumerate(zip(trace, want["history"])):
        if fragile_step(o, p):
            break
        assert np.array_equal(g["positions"], o["positions"]) and np.array_equal(g["seq_ids"], o["seq_ids"])
        check_score(to_np(g["score"]), o["score"], V, plan)
        assert np.array_equal(to_np(g["commit"])["commit"], o["commit"]["commit"])
        if budget > 0:
            gs, os_ = to_np(g["select"]), o["select"]
            for k in ("draft_rows", "n_drafts", "route", "rem_off", "v_off"):
                assert np.array_equal(gs[k], os_[k]), (s, k)
            if os_["v_off"][-1] > 0:
                osv = oscore.score(w, g["hv_bits"], plan)
                if (osv["gap"] < NEAR_TIE).any() or (np.abs(osv["conf"] - float(np.float32(0.9))) < FRAGILE).any():
                    break
                gv = to_np(g["verify"])
                for k in ("accept", "choice", "final_commit"):
                    assert np.array_equal(gv[k], o["verify"][k]), (s, k)
        assert np.array_equal(g["y"], o["y"]), s
        n_same += 1
    assert n_same >= min(5, want["steps"])
    if n_same == want["steps"]:
        assert got["steps"] == want["steps"] and np.array_equal(got["y"], want["y"])
        assert np.array_equal(got["steps_per_seq"], want["steps_per_seq"])
    # invariants that hold whatever happened
    assert not (got["y"] == mask).any()
    prev = np.full((B, L), mask, np.int32)
    for g in trace:
        keep = prev != mask
        assert np.array_equal(g["y"][keep], prev[keep])
        prev = g["y"]
    ctx.close()


@pytest.mark.gpu
def test_loop_llada_shape_two_sequences_sampled_rows():
    # full vocabulary and hidden size, short canvas: every step's scores are checked on sampled rows
    V, D, B, L, S, seed = synth.LLADA_VOCAB, synth.LLADA_HIDDEN, 2, 32, 16, 1004
    w = synth.make_w(seed, V, D)
    plan = synth.make_plan_ids(seed, V, 2048)
    tg = synth.loop_targets(seed, V, B, L, plan, 0.5, avoid=V - 128)
    p = dict(tau_high=0.9, budget=4, **synth.DEFAULT_BAND)
    ctx = make_ctx(w, plan, 4096, B, 4)
    checked = []

    def on_step(s, d):
        if s < 3 and len(d["positions"]):
            rows = np.unique(np.linspace(0, len(d["positions"]) - 1, 3).astype(int))
            check_score(to_np(d["score"]), oscore.score(w, d["h_bits"][rows], plan), V, plan, rows=rows)
            checked.append(s)

    got = decode_loop.decode(ctx, w, tg, seed, L, S, p, V - 128, on_step=on_step)
    assert got["status"] == 0 and not (got["y"] == V - 128).any() and len(checked) >= 2
    base = decode_loop.decode(ctx, w, tg, seed, L, S, dict(p, budget=0), V - 128)
    assert got["steps_per_seq"].sum() <= base["steps_per_seq"].sum() + 2
    ctx.close()


@pytest.mark.gpu
@pytest.mark.parametrize("mode", ["random", "planning"])
def test_exploration_loop_state_by_state(mode):
    V, D, B, L, S, seed = 4096, 256, 4, 64, 32, 1004
    w = synth.make_w(seed, V, D)
    plan = synth.make_plan_ids(seed, V, 256)
    tg = synth.loop_targets(seed, V, B, L, plan, 0.5, avoid=V - 1)
    p = dict(tau_high=0.9, budget=0, **synth.DEFAULT_BAND)
    mask = V - 1
    want = oloop.decode(synth, w, plan, tg, seed, L, S, p, mask, trace=True, explore=mode)
    ctx = make_ctx(w, plan, B * S * 2, B, 1)
    trace = []
    got = decode_loop.decode(ctx, w, tg, seed, L, S, p, mask, on_step=lambda s, d: trace.append(
        dict(d, commit_np=d["commit"]["commit"].cpu().numpy(), explore_np=d["explore_row"].cpu().numpy())), explore=mode)
    assert got["status"] == 0 and not (got["y"] == mask).any()
    n_same = 0
    for g, o in zip(trace, want["history"]):
        if fragile_step(o, p):
            break
        assert np.array_equal(g["positions"], o["positions"])
        check_score(to_np(g["score"]), o["score"], V, plan)
        assert np.array_equal(g["explore_np"], o["explore"]["explore_row"])
        assert np.array_equal(g["commit_np"], o["explore"]["commit"])          # base commit plus the explored row
        assert np.array_equal(g["y"], o["y"])
        n_same += 1
    assert n_same >= min(4, want["steps"])
    if n_same == want["steps"]:
        assert got["steps"] == want["steps"] and np.array_equal(got["y"], want["y"])
    ctx.close()


@pytest.mark.gpu
@pytest.mark.parametrize("K,band,min_widest", [(8, (None, 0.6), 1), (32, (0.02, 0.9), 9)])
def test_calibration_trajectory_matches_oracle(K, band, min_widest):
    # K = 8 with a band a little wider than the paper's; and K = 32 = the block size with a band so wide that more
    # than 8 rows of a sequence fall into it at once: with the budget at least the block size every candidate of
    # C_t^cal is measured, which is the paper's rule (Appendix, "Calibration trajectory") -- the oracle runs with the
    # same budget, which then never binds.
    from oracle import calib as ocal
    from paper_2601_12247_b200 import calibrate
    V, D, B, L, S, seed = 4096, 256, 4, 64, 32, 1006
    w = synth.make_w(seed, V, D)
    pool = synth.make_plan_ids(seed, V, 24)
    tg = synth.loop_targets(seed, V, B, L, pool, 1.0, avoid=V - 1)
    mask = V - 1
    cal = binding.default_calib_params()
    if band[0] is not None:
        cal.tau_cal_lo = band[0]
    cal.tau_cal_hi = band[1]                                 # a wider band than the paper's: more events in a tiny run
    want = ocal.calibrate(synth, w, tg, seed, L, S, 0.9, cal.tau_cal_lo, cal.tau_cal_hi, K, mask, trace=True)
    ctx = make_ctx(w, [], B * S * (2 + K), B, K)
    trace = []
    got = calibrate.calibrate(ctx, w, tg, seed, L, S, 0.9, cal, K, mask, on_step=lambda s, d: trace.append(d))
    assert got["status"] == 0
    taus = [0.9, cal.tau_cal_lo, cal.tau_cal_hi]
    clean = True
    for g, o in zip(trace, want["history"]):
        bad = (o["score"]["gap"] < NEAR_TIE).any() or any((np.abs(o["score"]["conf"] - float(np.float32(t))) < FRAGILE).any() for t in taus)
        if o["score_v"] is not None:
            bad = bad or (o["score_v"]["gap"] < NEAR_TIE).any() or (np.abs(o["score_v"]["conf"] - float(np.float32(0.9))) < FRAGILE).any()
        if bad:
            clean = False
            break
        gs = to_np(g["select"])
        for k in ("draft_rows", "n_drafts", "route", "rem_off", "v_off"):
            assert np.array_equal(gs[k], o["select"][k]), k
        if o["events"]:
            vig = g["vig"].cpu().numpy()
            for e in o["events"]:
                assert abs(vig[e["seq"], e["j"] - 1] - e["VIG"]) <= 2e-3       # entropies within 1e-3 on both branches
        assert np.array_equal(g["y"], o["y"])
    assert want["n_events"] > 0
    widest = max(int(o["select"]["n_drafts"].max()) for o in want["history"])
    assert min_widest <= widest <= K and (K < S or widest < K)              # K = S: the budget never binds
    if clean:
        st = to_np(got["stats"])
        assert got["steps"] == want["steps"] and got["n_events"] == want["n_events"]
        assert np.array_equal(st["n_v"], want["stats"]["n"]) and np.array_equal(st["m_v"], want["stats"]["m"])
        assert np.array_equal(st["sum_a"], want["stats"]["sum_a"])
        assert np.max(np.abs(st["sum_vig_q32"] / 2.0 ** 32 - want["stats"]["sum_vig"])) <= 2e-3 * max(1, want["n_events"])
    ctx.close()


@pytest.mark.gpu
@pytest.mark.parametrize("q_plan", [0.0, 0.5])
def test_loop_config4_full_size(q_plan):
    # Config 4 at its stated size (Algorithm 1): LLaDA-shaped head, 32 sequences, 256 tokens, blocks of 32, budget 4,
    # forced progress.  Per step: sampled draft and verification rows against the oracle one by one, and every
    # decision of the step against the oracle's rules fed the GPU's own fp32 outputs.  At the end: no mask left,
    # committed tokens never changed, and PVF needs no more forwards than threshold-only decoding (K = 0).
    V, D, B, L, S, K, seed = synth.LLADA_VOCAB, synth.LLADA_HIDDEN, 32, 256, 32, 4, 1004
    mask = V - 128
    w = synth.make_w(seed, V, D)
    plan = synth.make_plan_ids(seed, V, 2048)
    tg = synth.loop_targets(seed, V, B, L, plan, q_plan, avoid=mask)
    p = dict(tau_high=0.9, budget=K, **synth.DEFAULT_BAND)
    ctx = make_ctx(w, plan, B * S * (2 + K), B, K)
    state = dict(prev=np.full((B, L), mask, np.int32), rows=0, rows_v=0, routes=np.zeros(3, np.int64), checked=0, checked_v=0)

    def on_step(s, d):
        from oracle import step as ostep
        pos, seg = d["positions"], d["seg_off"]
        n = len(pos)
        act = np.ones(n, np.uint8)
        g_sc = to_np(d["score"])
        assert n <= B * S and np.all(np.diff(seg) <= S)
        if n and (s < 4 or s % 4 == 0):                                    # sampled rows against the oracle
            rows = np.unique(np.array([0, n // 2, n - 1]))
            check_score(g_sc, oscore.score(w, d["h_bits"][rows], plan), V, plan, rows=rows)
            state["checked"] += len(rows)
        conf64 = g_sc["conf"].astype(np.float64)
        ocm = ostep.commit(conf64, g_sc["tok"], seg, pos, act, p["tau_high"], force_progress=True)
        assert np.array_equal(to_np(d["commit"])["commit"], ocm["commit"])
        osel = ostep.select_drafts(conf64, g_sc["tok"], g_sc["in_plan"], ocm["commit"], seg, pos, act,
                                   p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"], K)
        gs = to_np(d["select"])
        for k in ("draft_rows", "n_drafts", "route", "rem_off", "v_off"):
            assert np.array_equal(gs[k], osel[k]), (s, k)
        state["routes"] += np.bincount(osel["route"], minlength=3)
        Mv = int(osel["v_off"][-1])
        g_scv = to_np(d["score_v"])
        if Mv and (s < 4 or s % 4 == 0):
            rows = np.unique(np.array([0, Mv // 2, Mv - 1]))
            check_score(g_scv, oscore.score(w, d["hv_bits"][rows], plan), V, None, rows=rows)    # (no in_plan for this pass)
            state["checked_v"] += len(rows)
        over = ostep.verify(g_sc["tok"], ocm["commit"], seg, pos, osel["rem_rows"], osel["rem_off"], osel["v_off"],
                            osel["draft_rows"], osel["n_drafts"], osel["route"], g_scv["tok"][:max(Mv, 0)],
                            g_scv["conf"][:max(Mv, 0)].astype(np.float64), p["tau_high"], K)
        gv = to_np(d["verify"])
        for k in ("accept", "choice", "final_commit"):
            assert np.array_equal(gv[k], over[k]), (s, k)
        # the canvas: exactly the final commits are written, with the draft pass's tokens; nothing else changes
        want_y = state["prev"].copy()
        fin = over["final_commit"].astype(bool)
        want_y[d["seq_ids"][fin], pos[fin]] = g_sc["tok"][fin]
        assert np.array_equal(d["y"], want_y)
        assert fin.sum() >= (np.diff(seg) > 0).sum()                       # forced progress: every live sequence moves
        state["prev"] = d["y"]
        state["rows"] += n
        state["rows_v"] += Mv

    got = decode_loop.decode(ctx, w, tg, seed, L, S, p, mask, on_step=on_step)
    assert got["status"] == 0 and not (got["y"] == mask).any()
    assert state["checked"] >= 9 and got["scored_rows"] == state["rows"] + state["rows_v"]
    assert state["routes"][1] + state["routes"][2] > 0 and state["rows_v"] > 0
    if q_plan > 0:
        assert state["routes"][1] > 0 and state["checked_v"] > 0         # the planning route was taken
    base = decode_loop.decode(ctx, w, tg, seed, L, S, dict(p, budget=0), mask)
    assert base["status"] == 0 and not (base["y"] == mask).any()
    assert got["steps"] <= base["steps"] and got["tokens_per_forward"] >= base["tokens_per_forward"] - 1e-9
    assert 1.0 <= base["tokens_per_forward"] <= S and got["steps_per_seq"].min() >= L // S
    ctx.close()
