"""Pins of the step oracle (commit / draft proposal / verification): hand-built cases, brute
force on small candidate sets, library cross-checks and the step's invariants (CPU only)."""
import itertools

import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import step as ostep

F = lambda x: float(np.float32(x))


def one_seq(n):
    return np.array([0, n], np.int32), np.arange(n, dtype=np.int32), np.ones(n, np.uint8)


# ----------------------------------------------------------------------------- commit
def test_commit_threshold_is_inclusive_and_gated_by_active():
    seg, pos, act = one_seq(5)
    act[4] = 0
    conf = np.array([F(0.9), np.nextafter(np.float32(0.9), np.float32(0)), 0.95, 0.1, 0.99])
    r = ostep.commit(conf, np.arange(5) + 100, seg, pos, act, 0.9)
    assert r["commit"].tolist() == [1, 0, 1, 0, 0]          # p >= tau commits; inactive never
    assert r["n_commit"].tolist() == [2]


def test_commit_writes_only_committed_positions():
    seg = np.array([0, 3, 5], np.int32)
    pos = np.array([2, 5, 7, 0, 1], np.int32)
    conf = np.array([0.95, 0.2, 0.91, 0.3, 0.99])
    tok = np.array([11, 12, 13, 14, 15], np.int32)
    y = np.full((2, 8), -7, np.int32)
    y[0, 0] = 42                                              # an already committed token
    r = ostep.commit(conf, tok, seg, pos, None, 0.9, y=y)
    want = y.copy(); want[0, 2] = 11; want[0, 7] = 13; want[1, 1] = 15
    assert np.array_equal(r["y"], want)
    assert r["n_commit"].tolist() == [2, 1]


def test_commit_force_progress():
    seg = np.array([0, 4, 6, 6], np.int32)
    pos = np.array([0, 1, 2, 3, 0, 1], np.int32)
    act = np.array([1, 1, 1, 0, 1, 1], np.uint8)
    conf = np.array([0.3, 0.5, 0.5, 0.8, 0.95, 0.1])
    r0 = ostep.commit(conf, np.zeros(6, np.int32), seg, pos, act, 0.9)
    assert r0["commit"].tolist() == [0, 0, 0, 0, 1, 0]
    r1 = ostep.commit(conf, np.zeros(6, np.int32), seg, pos, act, 0.9, force_progress=True)
    # sequence 0: best ACTIVE row, lowest position on the 0.5 tie; sequence 1 already progresses;
    # sequence 2 has no rows
    assert r1["commit"].tolist() == [0, 1, 0, 0, 1, 0]
    assert r1["n_commit"].tolist() == [1, 1, 0]
    # tau_high above 1: empty base set, or exactly one row per sequence with forced progress
    assert ostep.commit(conf, np.zeros(6, np.int32), seg, pos, act, 1.5)["commit"].sum() == 0
    assert ostep.commit(conf, np.zeros(6, np.int32), seg, pos, act, 1.5, True)["n_commit"].tolist() == [1, 1, 0]


# ----------------------------------------------------------------------------- select
def brute_force_topk(cands, conf, pos, K):
    """Enumerate every subset of size min(K, n): the chosen one has the lexicographically largest
    sorted key list (confidence descending, then position ascending)."""
    k = min(K, len(cands))
    key = lambda m: (-conf[m], pos[m])
    best = None
    for sub in itertools.combinations(cands, k):
        ks = sorted(key(m) for m in sub)
        if best is None or ks < best[0]:
            best = (ks, sorted(sub, key=key))
    return best[1] if best else []


def test_select_bruteforce_small_candidate_sets():
    rng = np.random.default_rng(5)
    for trial in range(60):
        n = int(rng.integers(1, 9))
        seg, pos, act = one_seq(n)
        conf = rng.choice([0.1, 0.25, 0.3, 0.3, 0.5, 0.64, 0.65, 0.7, 0.95], size=n).astype(np.float32).astype(np.float64)
        in_plan = rng.integers(0, 2, n).astype(np.uint8)
        act = rng.integers(0, 4, n).astype(bool).astype(np.uint8)
        K = int(rng.integers(0, 5))
        cm = ostep.commit(conf, np.zeros(n, np.int32), seg, pos, act, 0.9)["commit"]
        r = ostep.select_drafts(conf, np.zeros(n, np.int32), in_plan, cm, seg, pos, act, 0.2, 0.65, 0.1, K)
        rem = [m for m in range(n) if act[m] and not cm[m]]
        cands = [m for m in rem if in_plan[m] and F(0.2) <= conf[m] < F(0.65)]
        if K == 0:
            assert r["n_drafts"][0] == 0 and r["route"][0] == 0
        elif cands:
            assert r["route"][0] == 1
            assert r["draft_rows"][0, :r["n_drafts"][0]].tolist() == brute_force_topk(cands, conf, pos, K)
        else:
            ar = [m for m in rem if conf[m] >= F(0.1)][:K]
            assert r["draft_rows"][0, :r["n_drafts"][0]].tolist() == ar
            assert r["route"][0] == (2 if ar else 0)
        assert r["rem_rows"].tolist() == rem
        assert np.all(r["draft_rows"][0, r["n_drafts"][0]:] == -1)


def test_select_whole_vocab_plan_and_wide_band_is_plain_topk():
    rng = np.random.default_rng(11)
    n, K = 40, 6
    seg, pos, act = one_seq(n)
    conf = rng.random(n).astype(np.float32).astype(np.float64) * 0.89
    r = ostep.select_drafts(conf, np.zeros(n, np.int32), np.ones(n, np.uint8), np.zeros(n, np.uint8),
                            seg, pos, act, 0.0, 0.9, 0.1, K)
    assert r["draft_rows"][0].tolist() == np.argsort(-conf, kind="stable")[:K].tolist()
    assert r["route"][0] == 1 and r["n_drafts"][0] == K


def test_select_band_is_half_open_and_ties_go_left():
    seg, pos, act = one_seq(6)
    conf = np.array([F(0.65), F(0.2), 0.4, 0.4, np.nextafter(np.float32(0.2), np.float32(0)), 0.5])
    r = ostep.select_drafts(conf, np.zeros(6, np.int32), np.ones(6, np.uint8), np.zeros(6, np.uint8),
                            seg, pos, act, 0.2, 0.65, 0.1, 8)
    # 0.65 is outside [0.2, 0.65), 0.2 inside, just-below-0.2 outside; equal 0.4s in position order
    assert r["draft_rows"][0, :4].tolist() == [5, 2, 3, 1] and r["n_drafts"][0] == 4


def test_select_ar_route_when_no_planning_candidate():
    seg, pos, act = one_seq(7)
    conf = np.array([0.05, 0.3, 0.95, 0.12, 0.09, 0.7, 0.4])
    cm = np.array([0, 0, 1, 0, 0, 0, 0], np.uint8)
    r = ostep.select_drafts(conf, np.zeros(7, np.int32), np.zeros(7, np.uint8), cm, seg, pos, act,
                            0.2, 0.65, 0.1, 3)
    assert r["route"][0] == 2
    assert r["draft_rows"][0].tolist() == [1, 3, 5]        # leftmost qualifying, gaps allowed, base skipped
    assert r["rem_rows"].tolist() == [0, 1, 3, 4, 5, 6]
    assert r["v_off"].tolist() == [0, 4 * 6]


def test_select_offsets_over_several_sequences():
    seg = np.array([0, 3, 3, 7], np.int32)
    pos = np.array([4, 5, 6, 0, 1, 2, 3], np.int32)
    conf = np.array([0.95, 0.3, 0.01, 0.5, 0.92, 0.02, 0.03])
    in_plan = np.array([0, 1, 0, 0, 0, 0, 0], np.uint8)
    cm = ostep.commit(conf, np.zeros(7, np.int32), seg, pos, None, 0.9)["commit"]
    r = ostep.select_drafts(conf, np.zeros(7, np.int32), in_plan, cm, seg, pos, None, 0.2, 0.65, 0.1, 2)
    assert r["rem_off"].tolist() == [0, 2, 2, 5] and r["rem_rows"].tolist() == [1, 2, 3, 5, 6]
    assert r["route"].tolist() == [1, 0, 2] and r["n_drafts"].tolist() == [1, 0, 1]
    assert r["draft_rows"].tolist() == [[1, -1], [-1, -1], [3, -1]]
    assert r["v_off"].tolist() == [0, 4, 4, 10]


@settings(max_examples=150, deadline=None)
@given(st.data())
def test_select_invariants(data):
    n_seq = data.draw(st.integers(1, 4))
    lens = [data.draw(st.integers(0, 12)) for _ in range(n_seq)]
    seg = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    M = int(seg[-1])
    pos = np.concatenate([np.sort(np.random.default_rng(i).permutation(40)[:l]) for i, l in enumerate(lens)] + [np.zeros(0, int)]).astype(np.int32)
    conf = np.array([data.draw(st.sampled_from([0.0, 0.1, 0.15, 0.2, 0.33, 0.5, 0.5, 0.649, 0.65, 0.8, 0.9, 0.97]))
                     for _ in range(M)], dtype=np.float32).astype(np.float64)
    in_plan = np.array([data.draw(st.integers(0, 1)) for _ in range(M)], np.uint8)
    act = np.array([data.draw(st.integers(0, 3)) > 0 for _ in range(M)], np.uint8)
    K = data.draw(st.integers(0, 5))
    cm = ostep.commit(conf, np.zeros(M, np.int32), seg, pos, act, 0.9)["commit"]
    r = ostep.select_drafts(conf, np.zeros(M, np.int32), in_plan, cm, seg, pos, act, 0.2, 0.65, 0.1, K)
    lo, hi, ar = F(0.2), F(0.65), F(0.1)
    for b in range(n_seq):
        rows = list(range(seg[b], seg[b + 1]))
        nd = int(r["n_drafts"][b])
        d = r["draft_rows"][b, :nd].tolist()
        assert nd <= K and len(set(d)) == nd
        elig = [m for m in rows if act[m] and not cm[m] and in_plan[m] and lo <= conf[m] < hi]
        for m in d:
            assert m in rows and act[m] and not cm[m]                       # drafts never touch the base set
        if r["route"][b] == 1:
            assert nd == min(K, len(elig)) and set(d) <= set(elig)
            assert all(conf[d[i]] >= conf[d[i + 1]] for i in range(nd - 1))
            worst = (-conf[d[-1]], pos[d[-1]])
            assert all((-conf[m], pos[m]) >= worst for m in elig if m not in d)
        else:
            assert not elig or K == 0                                       # planning has priority
            if r["route"][b] == 2:
                assert all(conf[m] >= ar for m in d)
                assert all(pos[d[i]] < pos[d[i + 1]] for i in range(nd - 1))
            else:
                assert nd == 0


# ----------------------------------------------------------------------------- verify
def planning_case(conf_base, tok_base, branch_tok, branch_conf, draft_r, tau=0.9, exclude_self=False):
    """One sequence, nR remaining rows (= all rows), drafts given as indices into them."""
    nR = len(conf_base)
    K = len(draft_r)
    seg, pos, act = one_seq(nR)
    rem = np.arange(nR, dtype=np.int32)
    rem_off = np.array([0, nR], np.int32)
    v_off = np.array([0, (1 + K) * nR], np.int32)
    tok_v = np.concatenate([tok_base] + list(branch_tok)).astype(np.int32)
    conf_v = np.concatenate([conf_base] + list(branch_conf)).astype(np.float64)
    return ostep.verify(np.arange(nR, dtype=np.int32) + 1000, np.zeros(nR, np.uint8), seg, pos, rem, rem_off,
                        v_off, np.array([draft_r], np.int32), np.array([K], np.int32), np.array([1], np.uint8),
                        tok_v, conf_v, tau, K, exclude_self=exclude_self)


def test_verify_all_branches_agree_choose_largest_c_total():
    conf_base = np.array([0.95, 0.3, 0.2, 0.92])
    tok_base = np.array([5, 6, 7, 8])
    bt = [tok_base.copy(), tok_base.copy()]
    bc = [np.array([0.9, 0.99, 0.1, 0.9]), np.array([0.9, 0.5, 0.99, 0.9])]
    # draft 1 sits at r=1, draft 2 at r=2; C_1 = 0.9+0.1+0.9 = 1.9, C_2 = 0.9+0.5+0.9 = 2.3
    r = planning_case(conf_base, tok_base, bt, bc, [1, 2])
    assert r["accept"].tolist() == [[1, 1]] and r["choice"].tolist() == [2]
    assert r["final_commit"].tolist() == [0, 0, 1, 0]


def test_verify_one_flipped_impact_token_rejects_that_branch_only():
    conf_base = np.array([0.95, 0.3, 0.2, 0.92])
    tok_base = np.array([5, 6, 7, 8])
    b1 = tok_base.copy(); b1[3] = 99            # row 3 is in the impact set
    b2 = tok_base.copy(); b2[1] = 99            # row 1 is not (0.3 < tau): harmless
    conf = [np.full(4, 0.5), np.full(4, 0.4)]
    r = planning_case(conf_base, tok_base, [b1, b2], conf, [1, 2])
    assert r["accept"].tolist() == [[0, 1]] and r["choice"].tolist() == [2]


def test_verify_empty_impact_set_rejects_everything():
    conf_base = np.array([0.5, 0.3, 0.2, 0.89])
    tok_base = np.array([5, 6, 7, 8])
    r = planning_case(conf_base, tok_base, [tok_base, tok_base], [np.ones(4), np.ones(4)], [0, 1])
    assert r["accept"].tolist() == [[0, 0]] and r["choice"].tolist() == [0]
    assert r["final_commit"].sum() == 0


def test_verify_impact_threshold_inclusive_and_self_position_counts():
    conf_base = np.array([F(0.9), 0.3, 0.2])
    tok_base = np.array([5, 6, 7])
    b1 = tok_base.copy(); b1[0] = 77            # the draft sits on the only impact row and changes it
    r = planning_case(conf_base, tok_base, [b1], [np.full(3, 0.5)], [0])
    assert r["accept"].tolist() == [[0]]
    r = planning_case(conf_base, tok_base, [b1], [np.full(3, 0.5)], [0], exclude_self=True)
    assert r["accept"].tolist() == [[0]]        # impact set without the draft's own row is empty
    conf_base2 = np.array([F(0.9), 0.95, 0.2])
    r = planning_case(conf_base2, tok_base, [b1], [np.full(3, 0.5)], [0], exclude_self=True)
    assert r["accept"].tolist() == [[1]] and r["choice"].tolist() == [1]


def test_verify_c_total_excludes_the_draft_row_and_ties_take_lowest_j():
    conf_base = np.array([0.95, 0.3, 0.2])
    tok_base = np.array([5, 6, 7])
    bc = [np.array([0.25, 1.0, 0.5]), np.array([0.5, 0.25, 0.123])]   # C_1 = 0.75 (row 1 left out), C_2 = 0.75
    r = planning_case(conf_base, tok_base, [tok_base, tok_base], bc, [1, 2])
    assert r["choice"].tolist() == [1]


def ar_case(flip):
    """AR route, 5 remaining rows, drafts at rows 1, 2, 4; `flip` lists (branch k, fill r) pairs whose
    verification token differs from the drafted token."""
    nR, K = 5, 3
    seg, pos, act = one_seq(nR)
    tok = np.array([10, 11, 12, 13, 14], np.int32)
    drafts = [1, 2, 4]
    tok_v = np.tile(tok, 1 + K).astype(np.int32)
    for k, r in flip:
        tok_v[k * nR + drafts[r - 1]] = 999
    conf_v = np.full((1 + K) * nR, 0.5)
    return ostep.verify(tok, np.zeros(nR, np.uint8), seg, pos, np.arange(nR, dtype=np.int32),
                        np.array([0, nR], np.int32), np.array([0, (1 + K) * nR], np.int32),
                        np.array([drafts], np.int32), np.array([K], np.int32), np.array([2], np.uint8),
                        tok_v, conf_v, 0.9, K)


def test_verify_ar_longest_verified_extension():
    r = ar_case([])
    assert r["accept"].tolist() == [[1, 1, 1]] and r["choice"].tolist() == [3]
    assert r["final_commit"].tolist() == [0, 1, 1, 0, 1]
    r = ar_case([(3, 2)])                       # fill 2 changes under branch 3 only
    assert r["accept"].tolist() == [[1, 1, 0]] and r["choice"].tolist() == [2]
    assert r["final_commit"].tolist() == [0, 1, 1, 0, 0]
    r = ar_case([(1, 1), (2, 1), (3, 1)])       # fill 1 unstable everywhere
    assert r["accept"].tolist() == [[0, 0, 0]] and r["choice"].tolist() == [0]
    r = ar_case([(1, 1)])                       # K^AR need not be prefix-closed: k*=max
    assert r["accept"].tolist() == [[0, 1, 1]] and r["choice"].tolist() == [3]


@settings(max_examples=120, deadline=None)
@given(st.data())
def test_verify_invariants(data):
    nR = data.draw(st.integers(1, 7))
    K = data.draw(st.integers(1, 4))
    Kt = data.draw(st.integers(1, min(K, nR)))
    route = data.draw(st.sampled_from([1, 2]))
    seg, pos, act = one_seq(nR + 1)
    cm = np.zeros(nR + 1, np.uint8); cm[0] = 1              # row 0 is base-committed
    rem = np.arange(1, nR + 1, dtype=np.int32)
    drafts = sorted(data.draw(st.permutations(list(range(1, nR + 1))))[:Kt])
    dr = np.full((1, K), -1, np.int32); dr[0, :Kt] = drafts
    tok = np.arange(nR + 1, dtype=np.int32) + 50
    tok_v = np.array([data.draw(st.sampled_from([0, 1])) * 7 + tok[rem[i % nR]] for i in range((1 + Kt) * nR)], np.int32)
    conf_v = np.array([data.draw(st.sampled_from([0.1, 0.5, 0.9, 0.95])) for _ in range((1 + Kt) * nR)], np.float32).astype(np.float64)
    r = ostep.verify(tok, cm, seg, pos, rem, np.array([0, nR], np.int32), np.array([0, (1 + Kt) * nR], np.int32),
                     dr, np.array([Kt], np.int32), np.array([route], np.uint8), tok_v, conf_v, 0.9, K)
    acc, ch, fin = r["accept"][0], int(r["choice"][0]), r["final_commit"]
    assert np.all(fin >= cm)                                 # committed positions are never re-masked
    assert acc[Kt:].sum() == 0
    extra = [m for m in range(nR + 1) if fin[m] and not cm[m]]
    if ch > 0:
        assert acc[ch - 1] == 1                              # the chosen branch passed verification
    else:
        assert extra == []
    if route == 1:
        assert extra == ([drafts[ch - 1]] if ch else [])
        impact = [i for i in range(nR) if conf_v[i] >= F(0.9)]
        for j in range(1, Kt + 1):
            if acc[j - 1]:                                   # acceptance implies agreement with the backbone
                assert impact and all(tok_v[j * nR + i] == tok_v[i] for i in impact)
    else:
        assert extra == drafts[:ch] and len(extra) <= K
        if ch:
            assert all(tok_v[ch * nR + (drafts[q] - 1)] == tok[drafts[q]] for q in range(ch))


# ----------------------------------------------------------------------------- C_total margins (Section 4.2, Filter 2)
def margins_case(branch_conf, draft_r, accept, route=1):
    """One sequence with nR remaining rows; returns c_total_margins for hand-written branch confidences."""
    nR = len(branch_conf[0])
    K = len(draft_r)
    conf_v = np.concatenate([np.full(nR, 0.95)] + [np.asarray(c, dtype=np.float64) for c in branch_conf])
    return ostep.c_total_margins(np.arange(nR, dtype=np.int32), np.array([0, nR], np.int32),
                                 np.array([0, (1 + K) * nR], np.int32), np.array([draft_r], np.int32),
                                 np.array([K], np.int32), np.array([route], np.uint8), conf_v,
                                 np.array([accept], np.uint8))


def test_c_total_margins_hand_built_three_branches():
    # drafts at rows 1, 2, 3 of five; each branch's own draft row carries a large value that must be left out:
    #   C_1 = 0.5 + 0.6 + 0.4 + 0.4    = 1.9       (row 1 = 9.0 left out)
    #   C_2 = 0.5 + 0.6 + 0.6 + 0.6    = 2.3       (row 2 = 7.0 left out)
    #   C_3 = 0.5 + 0.6 + 0.6 + 0.6005 = 2.3005    (row 3 = 5.0 left out)
    bc = [[0.5, 9.0, 0.6, 0.4, 0.4], [0.5, 0.6, 7.0, 0.6, 0.6], [0.5, 0.6, 0.6, 5.0, 0.6005]]
    m = margins_case(bc, [1, 2, 3], [1, 1, 1])
    assert m.shape == (1,) and abs(m[0] - 0.0005) < 1e-12
    # only accepted branches count: without branch 3 the closest pair is C_2 - C_1 = 0.4
    assert abs(margins_case(bc, [1, 2, 3], [1, 1, 0])[0] - 0.4) < 1e-12
    assert abs(margins_case(bc, [1, 2, 3], [1, 0, 1])[0] - 0.4005) < 1e-12
    # the result does not depend on the order the branches come in
    assert abs(margins_case([bc[2], bc[0], bc[1]], [3, 1, 2], [1, 1, 1])[0] - 0.0005) < 1e-12


def test_c_total_margins_is_inf_without_two_accepted_planning_branches():
    bc = [[0.5, 9.0, 0.6], [0.5, 0.6, 7.0]]
    assert np.isinf(margins_case(bc, [1, 2], [1, 0])[0])
    assert np.isinf(margins_case(bc, [1, 2], [0, 0])[0])
    assert np.isinf(margins_case(bc, [1, 2], [1, 1], route=2)[0])        # AR route: Filter 2 does not apply
    assert np.isinf(margins_case(bc, [1, 2], [1, 1], route=0)[0])
    assert abs(margins_case(bc, [1, 2], [1, 1])[0] - 0.0) < 1e-12        # C_1 = C_2 = 1.1: an exact tie


def test_c_total_margins_agree_with_verifys_choice():
    # verify picks the accepted branch with the largest C_total; margins computed independently must rank the
    # same branch on top whenever the margin is clear, on random cases of several sequences
    rng = np.random.default_rng(5)
    for _ in range(40):
        n_seq, K = 3, 3
        nRs = rng.integers(3, 7, n_seq)
        seg = np.concatenate([[0], np.cumsum(nRs)]).astype(np.int32)
        M = int(seg[-1])
        pos = np.concatenate([np.arange(n) for n in nRs]).astype(np.int32)
        rem, rem_off = np.arange(M, dtype=np.int32), seg.copy()
        dr = np.stack([seg[b] + np.sort(rng.permutation(nRs[b])[:K]) for b in range(n_seq)]).astype(np.int32)
        nd = np.full(n_seq, K, np.int32)
        v_off = np.concatenate([[0], np.cumsum((1 + K) * nRs)]).astype(np.int32)
        tok = np.arange(M, dtype=np.int32)
        tok_v = np.concatenate([np.tile(tok[seg[b]:seg[b + 1]], 1 + K) for b in range(n_seq)]).astype(np.int32)
        conf_v = rng.uniform(0.0, 1.0, int(v_off[-1]))
        for b in range(n_seq):
            conf_v[v_off[b]] = 0.99                                       # a non-empty impact set everywhere
        route = np.ones(n_seq, np.uint8)
        r = ostep.verify(tok, np.zeros(M, np.uint8), seg, pos, rem, rem_off, v_off, dr, nd, route, tok_v, conf_v, 0.9, K)
        assert r["accept"].all()
        m = ostep.c_total_margins(rem, rem_off, v_off, dr, nd, route, conf_v, r["accept"])
        for b in range(n_seq):
            nR = int(nRs[b])
            cs = []
            for j in range(1, K + 1):
                blk = conf_v[v_off[b] + j * nR: v_off[b] + (j + 1) * nR].copy()
                blk[dr[b, j - 1] - seg[b]] = 0.0
                cs.append(blk.sum())
            srt = np.sort(cs)
            assert abs(m[b] - np.min(np.diff(srt))) < 1e-12
            assert int(r["choice"][b]) == int(np.argmax(cs)) + 1
