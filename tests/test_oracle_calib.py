"""Pins of the calibration oracle (verified information gain, token statistics, filtering rule).  CPU only."""
import math
import os

import numpy as np

from oracle import calib as ocal
from oracle import step as ostep

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def golden():
    g = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "paper_hyperparameters.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            g[k] = float(v)
    return g


def one_sequence(n_rem, drafts, tok_v, conf_v, ent_v, tok=None):
    """A single sequence whose remaining rows are 0..n_rem-1 and whose candidates are `drafts`."""
    K = max(len(drafts), 1)
    dr = np.full((1, K), -1, np.int32)
    dr[0, :len(drafts)] = drafts
    tok = np.arange(100, 100 + n_rem, dtype=np.int32) if tok is None else np.asarray(tok, np.int32)
    return dict(tok=tok, rem_rows=np.arange(n_rem, dtype=np.int32), rem_off=np.array([0, n_rem], np.int32),
                v_off=np.array([0, (1 + len(drafts)) * n_rem], np.int32), draft_rows=dr,
                n_drafts=np.array([len(drafts)], np.int32), route=np.array([1], np.uint8),
                tok_v=np.asarray(tok_v, np.int32), conf_v=np.asarray(conf_v, np.float64),
                ent_v=np.asarray(ent_v, np.float64))


def test_hand_computed_event():
    # 3 remaining rows, candidate = row 1.  Base branch: rows 0 and 2 confident (impact set {0, 2}).
    # Branch 1 keeps both tokens -> A = 1.  Entropies base (1.0, 9.9, 3.0), branch (0.5, 9.9, 2.0):
    # R = {0, 2}, dH = ((1.0 - 0.5) + (3.0 - 2.0)) / 2 = 0.75, VIG = 0.75.
    s = one_sequence(3, [1], tok_v=[7, 8, 9, 7, 5, 9], conf_v=[0.95, 0.3, 0.92, 0.9, 0.9, 0.9],
                     ent_v=[1.0, 9.9, 3.0, 0.5, 9.9, 2.0])
    (e,) = ocal.events(tau_high=0.9, **s)
    assert (e["token"], e["impact"], e["A"]) == (101, 1, 1)
    assert math.isclose(e["dH"], 0.75) and math.isclose(e["VIG"], 0.75)
    # flip one impact token in the branch: A = 0, the gain is still measured but VIG is 0
    s["tok_v"][5] = 4
    (e,) = ocal.events(tau_high=0.9, **s)
    assert e["A"] == 0 and math.isclose(e["dH"], 0.75) and e["VIG"] == 0.0 and e["impact"] == 1
    # no confident base row: vacuous -> A = 0 and the event does not count towards m_v
    s["conf_v"][:3] = [0.5, 0.3, 0.6]
    (e,) = ocal.events(tau_high=0.9, **s)
    assert e["impact"] == 0 and e["A"] == 0 and e["VIG"] == 0.0
    # entropy can also go up: negative gain
    s = one_sequence(2, [0], tok_v=[1, 2, 1, 2], conf_v=[0.1, 0.99, 0.5, 0.99], ent_v=[2.0, 1.0, 2.0, 1.5])
    (e,) = ocal.events(tau_high=0.9, **s)
    assert e["A"] == 1 and math.isclose(e["VIG"], -0.5)


def test_candidate_position_is_left_out_and_empty_region_gives_zero():
    # the candidate's own entropy change (here huge) must not enter dH
    s = one_sequence(2, [0], tok_v=[1, 2, 1, 2], conf_v=[0.95, 0.95, 0.9, 0.9], ent_v=[8.0, 1.0, 0.0, 0.25])
    (e,) = ocal.events(tau_high=0.9, **s)
    assert math.isclose(e["dH"], 0.75)
    # a single remaining row that is itself the candidate: R empty -> dH = 0 by definition
    s = one_sequence(1, [0], tok_v=[1, 1], conf_v=[0.95, 0.95], ent_v=[3.0, 0.1])
    (e,) = ocal.events(tau_high=0.9, **s)
    assert e["dH"] == 0.0 and e["VIG"] == 0.0 and e["A"] == 1
    (e,) = ocal.events(tau_high=0.9, exclude_self=True, **s)
    assert e["A"] == 0 and e["impact"] == 0                   # the only impact row was the candidate itself


def test_acceptance_agrees_with_the_decode_steps_verify():
    rng = np.random.default_rng(5)
    for _ in range(50):
        n_rem, K = int(rng.integers(1, 9)), int(rng.integers(1, 5))
        kt = min(K, n_rem)
        drafts = rng.permutation(n_rem)[:kt].astype(np.int32)
        n_v = (1 + kt) * n_rem
        base_tok = rng.integers(0, 3, n_rem)
        tok_v = np.concatenate([base_tok] + [np.where(rng.random(n_rem) < 0.8, base_tok, 5) for _ in range(kt)])
        conf_v = rng.random(n_v)
        s = one_sequence(n_rem, drafts, tok_v, conf_v, rng.random(n_v) * 5)
        evs = ocal.events(tau_high=0.7, **s)
        ver = ostep.verify(s["tok"], np.zeros(n_rem, np.uint8), np.array([0, n_rem], np.int32), np.arange(n_rem),
                           s["rem_rows"], s["rem_off"], s["v_off"], s["draft_rows"], s["n_drafts"], s["route"],
                           s["tok_v"], s["conf_v"], 0.7, s["draft_rows"].shape[1])
        assert [e["A"] for e in evs] == ver["accept"][0, :kt].tolist()
        for e in evs:
            assert abs(e["dH"]) <= 5.0 and e["VIG"] == e["A"] * e["dH"]


def test_aggregation_against_a_dictionary_restatement():
    rng = np.random.default_rng(11)
    V = 50
    evs = [dict(token=int(rng.integers(0, V)), impact=int(rng.random() < 0.7), A=0, dH=float(rng.normal()), VIG=0.0)
           for _ in range(2000)]
    for e in evs:
        e["A"] = int(e["impact"] and rng.random() < 0.8)
        e["VIG"] = e["A"] * e["dH"]
    st = ocal.accumulate(ocal.new_stats(V), evs)
    by_tok = {}
    for e in evs:
        by_tok.setdefault(e["token"], []).append(e)
    for v in range(V):
        ev = by_tok.get(v, [])
        assert st["n"][v] == len(ev) and st["m"][v] == sum(e["impact"] for e in ev)
        assert st["sum_a"][v] == sum(e["A"] for e in ev)
        assert math.isclose(st["sum_vig"][v], math.fsum(e["VIG"] for e in ev), abs_tol=1e-12)
    assert st["n"].sum() == len(evs) and np.all(st["sum_a"] <= st["m"]) and np.all(st["m"] <= st["n"])
    # accumulating in two halves gives the same statistics
    st2 = ocal.accumulate(ocal.accumulate(ocal.new_stats(V), evs[:700]), evs[700:])
    assert np.array_equal(st2["n"], st["n"]) and np.allclose(st2["sum_vig"], st["sum_vig"], atol=1e-12)


def test_filter_rule_boundaries_with_the_papers_thresholds():
    g = golden()
    n_min, m_min, rho, gam = int(g["n_min"]), int(g["m_min"]), g["rho_ver"], g["gamma_vig"]
    assert (n_min, m_min, rho, gam) == (50, 20, 0.9, 0.03) and (g["tau_cal_lo"], g["tau_cal_hi"]) == (0.15, 0.25)
    st = ocal.new_stats(8)

    def put(v, n, m, a, vig_mean):
        st["n"][v], st["m"][v], st["sum_a"][v], st["sum_vig"][v] = n, m, a, vig_mean * n

    put(0, 50, 20, 18, 0.05)          # exactly at n_min, m_min and r = 0.9: kept
    put(1, 49, 20, 20, 0.05)          # support too small
    put(2, 80, 19, 19, 0.05)          # too few non-vacuous verifications
    put(3, 80, 40, 35, 0.05)          # r = 0.875 < 0.9
    put(4, 80, 40, 40, 0.0299)        # average gain below gamma
    put(5, 80, 40, 40, 0.031)         # kept
    put(6, 60, 0, 0, 0.5)             # m = 0 -> r = 0
    put(7, 0, 0, 0, 0.0)              # never seen
    assert ocal.filter_tokens(st, n_min, m_min, rho, gam).tolist() == [0, 5]
    # with every threshold at its minimum, every token that was seen at least once is kept
    assert ocal.filter_tokens(st, 1, 0, 0.0, -1e9).tolist() == [0, 1, 2, 3, 4, 5, 6]


def test_calibration_candidates_are_the_band_without_vocabulary_filter():
    # thresholds cross the interface as fp32: rows 4 and 5 sit exactly on the fp32 band edges
    conf = np.array([0.95, 0.2, 0.16, 0.24, float(np.float32(0.25)), float(np.float32(0.15)), 0.1, 0.22], np.float64)
    M = len(conf)
    seg, pos, act = np.array([0, M], np.int32), np.arange(M), np.ones(M, np.uint8)
    tok, in_plan = np.arange(M), np.zeros(M, np.uint8)
    cm = ostep.commit(conf, tok, seg, pos, act, 0.9)
    sel = ostep.select_drafts(conf, tok, in_plan, cm["commit"], seg, pos, act, 0.15, 0.25, 0.1, 8,
                              any_token=True, ar_fallback=False)
    # rows in [0.15, 0.25): 1, 2, 3, 5, 7 -- by confidence: 3 (0.24), 7 (0.22), 1 (0.2), 2 (0.16), 5 (0.15)
    assert sel["route"][0] == 1 and sel["draft_rows"][0, :5].tolist() == [3, 7, 1, 2, 5] and sel["n_drafts"][0] == 5
    # the same call without the switches finds no planning candidate and falls back to AR
    sel2 = ostep.select_drafts(conf, tok, in_plan, cm["commit"], seg, pos, act, 0.15, 0.25, 0.1, 8)
    assert sel2["route"][0] == 2
    # an empty band proposes nothing and does not fall back
    sel3 = ostep.select_drafts(conf, tok, in_plan, cm["commit"], seg, pos, act, 0.5, 0.6, 0.1, 8,
                               any_token=True, ar_fallback=False)
    assert sel3["route"][0] == 0 and sel3["n_drafts"][0] == 0 and sel3["v_off"][-1] == 0


def test_calibration_trajectory_is_threshold_decoding_plus_measurement():
    from oracle import loop as oloop
    from paper_2601_12247_b200 import synth
    V, D, B, L, S, seed, mask = 1024, 64, 3, 64, 32, 1004, 1023
    w = synth.make_w(seed, V, D)
    plan = synth.make_plan_ids(seed, V, 128)
    tg = synth.loop_targets(seed, V, B, L, plan, 0.5, avoid=mask)
    r = ocal.calibrate(synth, w, tg, seed, L, S, 0.9, 0.15, 0.6, 8, mask, trace=True)
    # the trajectory itself is confidence-threshold decoding: measuring commits nothing
    base = oloop.decode(synth, w, plan, tg, seed, L, S, dict(tau_high=0.9, tau_plan_lo=0.2, tau_plan_hi=0.65,
                                                             tau_ar_lo=0.1, budget=0), mask)
    assert np.array_equal(r["y"], base["y"]) and r["steps"] == base["steps"]
    st = r["stats"]
    assert r["n_events"] > 0 and st["n"].sum() == r["n_events"]
    assert np.all(st["sum_a"] <= st["m"]) and np.all(st["m"] <= st["n"])
    seen = set()
    for h in r["history"]:
        assert (h["select"]["route"] != 2).all()
        for e in h["events"]:
            assert abs(e["dH"]) <= np.log(V) + 1e-9
            seen.add(e["token"])
    assert set(np.nonzero(st["n"])[0].tolist()) == seen
    keep = ocal.filter_tokens(st, 1, 1, 0.5, -100.0)
    assert set(keep.tolist()) <= seen
