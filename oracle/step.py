"""CPU oracle for the decisions of one PVF step -- TEST INFRASTRUCTURE, not part of the product.

Plain Python loops over rows, written from the paper's set definitions.  Notation follows the
paper: M_t masked positions of the working block B_t, p the top-1 confidence, y^ the top-1
token, S_base, P_t^plan, S_impact, A_t^j, C_total, K^AR.

Row bookkeeping (an input convention, not the paper's): the scored rows of sequence b are
seg_off[b] .. seg_off[b+1]-1, sorted by ascending canvas position row_pos[m]; active[m] says
whether the position belongs to B_t.

Readings where the paper is silent:
  * top-k ties: higher confidence first, then the lower position;
  * branch-choice ties in C_total: the lower draft index;
  * the draft's own position is NOT removed from the impact set unless exclude_self is set;
  * a step whose planning drafts all fail commits the base branch only (no AR attempt);
  * with force_progress, a sequence whose base set is empty commits its single most confident
    active row (the lowest position on ties), so that a decode loop always terminates.

All comparisons are done in fp64 on the numbers handed in; thresholds are handed in as the
fp32 numbers the C interface carries.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np

ROUTE_NONE, ROUTE_PLAN, ROUTE_AR = 0, 1, 2


def f32(x: float) -> float:
    """The double that equals the fp32 rounding of x (thresholds cross the C interface as float)."""
    return float(np.float32(x))


def commit(conf, tok, seg_off, row_pos, active, tau_high: float, force_progress: bool = False,
           y: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Base set S_base = {i in M_t : p_i >= tau_high} and base branch z_base (Section 3).

    Returns commit[M] (uint8), n_commit[n_seq] and, when a canvas y[n_seq][L] is given, a copy
    with y^ written at the committed positions (every other entry untouched).
    """
    conf = np.asarray(conf, dtype=np.float64)
    M = len(conf)
    n_seq = len(seg_off) - 1
    act = np.ones(M, np.uint8) if active is None else np.asarray(active)
    out = np.zeros(M, dtype=np.uint8)
    n_commit = np.zeros(n_seq, dtype=np.int32)
    tau = f32(tau_high)
    for b in range(n_seq):
        rows = range(int(seg_off[b]), int(seg_off[b + 1]))
        for m in rows:
            if act[m] and conf[m] >= tau:
                out[m] = 1
        if force_progress and not any(out[m] for m in rows):
            best = -1
            for m in rows:                                   # ascending position
                if act[m] and (best < 0 or conf[m] > conf[best]):
                    best = m
            if best >= 0:
                out[best] = 1
        n_commit[b] = sum(int(out[m]) for m in rows)
    res = dict(commit=out, n_commit=n_commit)
    if y is not None:
        y2 = np.array(y, copy=True)
        for b in range(n_seq):
            for m in range(int(seg_off[b]), int(seg_off[b + 1])):
                if out[m]:
                    y2[b, int(row_pos[m])] = int(tok[m])
        res["y"] = y2
    return res


def select_drafts(conf, tok, in_plan, commit_mask, seg_off, row_pos, active, tau_plan_lo: float,
                  tau_plan_hi: float, tau_ar_lo: float, budget: int, any_token: bool = False,
                  ar_fallback: bool = True) -> Dict[str, np.ndarray]:
    """Draft proposal of one step (Sections 4.1 and 4.3).

    Planning candidates  P_t^plan = {i in M_t \\ S_base : y^_i in P^plan, tau_l <= p_i < tau_u};
    the K_t = min(K, |P_t^plan|) most confident are the drafts, in rank order (route 1).
    If P_t^plan is empty the AR fallback proposes the leftmost <= K positions of M_t \\ S_base
    with p_i >= tau_AR^l, in position order (route 2).  Route 0: nothing to propose.

    ``any_token`` drops the planning-vocabulary condition and ``ar_fallback=False`` the second route:
    together they give the candidate set of the offline calibration, C_t^cal = {i in M_t \\ S_base :
    tau_cal^l <= p_i < tau_cal^u} (Appendix, planning-token set construction), capped at the K most
    confident.

    Also returns the remaining rows R_b = active, not base-committed rows of each sequence
    (rem_rows / rem_off) and the row offsets v_off of the verification pass, whose rows are laid
    out [b][c][r] with 1 + K_t branches per sequence that has drafts and none otherwise.
    """
    conf = np.asarray(conf, dtype=np.float64)
    M = len(conf)
    n_seq = len(seg_off) - 1
    K = int(budget)
    act = np.ones(M, np.uint8) if active is None else np.asarray(active)
    lo, hi, ar = f32(tau_plan_lo), f32(tau_plan_hi), f32(tau_ar_lo)
    draft_rows = np.full((n_seq, max(K, 1)), -1, dtype=np.int32)[:, :K]
    n_drafts = np.zeros(n_seq, dtype=np.int32)
    route = np.zeros(n_seq, dtype=np.uint8)
    rem_rows = []
    rem_off = np.zeros(n_seq + 1, dtype=np.int32)
    v_off = np.zeros(n_seq + 1, dtype=np.int32)
    for b in range(n_seq):
        rem = [m for m in range(int(seg_off[b]), int(seg_off[b + 1])) if act[m] and not commit_mask[m]]
        rem_rows.extend(rem)
        rem_off[b + 1] = rem_off[b] + len(rem)
        plan = [m for m in rem if (any_token or in_plan[m]) and lo <= conf[m] < hi]
        chosen = []
        if K > 0 and plan:
            order = sorted(plan, key=lambda m: (-conf[m], int(row_pos[m])))
            chosen = order[:K]
            route[b] = ROUTE_PLAN
        elif K > 0 and ar_fallback:
            chosen = [m for m in rem if conf[m] >= ar][:K]
            route[b] = ROUTE_AR if chosen else ROUTE_NONE
        n_drafts[b] = len(chosen)
        for j, m in enumerate(chosen):
            draft_rows[b, j] = m
        v_off[b + 1] = v_off[b] + ((1 + len(chosen)) * len(rem) if chosen else 0)
    return dict(draft_rows=draft_rows, n_drafts=n_drafts, route=route,
                rem_rows=np.asarray(rem_rows, dtype=np.int32), rem_off=rem_off, v_off=v_off)


def verify(tok, commit_mask, seg_off, row_pos, rem_rows, rem_off, v_off, draft_rows, n_drafts, route,
           tok_v, conf_v, tau_high: float, budget: int, exclude_self: bool = False,
           y: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Acceptance check and final commit of one step (Sections 3, 4.2, 4.3).

    tok_v / conf_v are the top-1 tokens and confidences of the verification pass, rows
    [b][c][r]: index v_off[b] + c * nR_b + r, c = 0 the base branch z_base, c = j the branch
    that adds draft j (planning) or the first j fills (AR), r over the remaining rows R_b.

    Planning route: impact set S_impact = {r in R_b : conf_v[base][r] >= tau_high} (Eq. 1);
      A_j = 1 iff S_impact is non-empty and branch j keeps the base branch's top-1 token on all
      of it (Eq. 3);  C_j = sum of conf_v[j][r] over the rows still masked in branch j, i.e.
      R_b without draft j;  j* = argmax of C_j over accepted branches; none accepted -> base only.
    AR route: k is verified iff for every r <= k the top-1 token of branch k at fill position
      i_r equals the drafted token y^_{i_r};  k* = the largest verified k (0 if none).
    """
    n_seq = len(seg_off) - 1
    K = int(budget)
    M = len(commit_mask)
    tau = f32(tau_high)
    conf_v = np.asarray(conf_v, dtype=np.float64)
    accept = np.zeros((n_seq, max(K, 1)), dtype=np.uint8)[:, :K]
    choice = np.zeros(n_seq, dtype=np.int32)
    final = np.array(commit_mask, dtype=np.uint8, copy=True)
    for b in range(n_seq):
        rem = [int(m) for m in rem_rows[int(rem_off[b]):int(rem_off[b + 1])]]
        nR = len(rem)
        Kt = int(n_drafts[b])
        if Kt == 0 or route[b] == ROUTE_NONE:
            continue
        base = int(v_off[b])
        idx = lambda c, r: base + c * nR + r
        r_of = {m: r for r, m in enumerate(rem)}
        drafts = [int(draft_rows[b, j]) for j in range(Kt)]
        if route[b] == ROUTE_PLAN:
            best_j, best_c = 0, None
            for j in range(1, Kt + 1):
                rj = r_of[drafts[j - 1]]
                impact = [r for r in range(nR)
                          if conf_v[idx(0, r)] >= tau and not (exclude_self and r == rj)]
                ok = len(impact) > 0 and all(tok_v[idx(j, r)] == tok_v[idx(0, r)] for r in impact)
                accept[b, j - 1] = 1 if ok else 0
                if ok:
                    c_total = 0.0
                    for r in range(nR):
                        if r != rj:
                            c_total += conf_v[idx(j, r)]
                    if best_c is None or c_total > best_c:
                        best_j, best_c = j, c_total
            choice[b] = best_j
            if best_j > 0:
                final[drafts[best_j - 1]] = 1
        else:                                                # AR fallback
            k_star = 0
            for k in range(1, Kt + 1):
                ok = all(tok_v[idx(k, r_of[drafts[r - 1]])] == tok[drafts[r - 1]] for r in range(1, k + 1))
                accept[b, k - 1] = 1 if ok else 0
                if ok:
                    k_star = k
            choice[b] = k_star
            for r in range(k_star):
                final[drafts[r]] = 1
    res = dict(accept=accept, choice=choice, final_commit=final)
    if y is not None:
        y2 = np.array(y, copy=True)
        for b in range(n_seq):
            for m in range(int(seg_off[b]), int(seg_off[b + 1])):
                if final[m]:
                    y2[b, int(row_pos[m])] = int(tok[m])
        res["y"] = y2
    return res


def c_total_margins(rem_rows, rem_off, v_off, draft_rows, n_drafts, route, conf_v, accept):
    """Smallest |C_a - C_b| between two accepted planning branches, per sequence (inf if < 2)."""
    n_seq = len(rem_off) - 1
    out = np.full(n_seq, np.inf)
    for b in range(n_seq):
        if route[b] != ROUTE_PLAN:
            continue
        rem = [int(m) for m in rem_rows[int(rem_off[b]):int(rem_off[b + 1])]]
        nR = len(rem)
        cs = []
        for j in range(1, int(n_drafts[b]) + 1):
            if accept[b, j - 1]:
                rj = rem.index(int(draft_rows[b, j - 1]))
                cs.append(sum(float(conf_v[int(v_off[b]) + j * nR + r]) for r in range(nR) if r != rj))
        cs.sort()
        for a, c in zip(cs, cs[1:]):
            out[b] = min(out[b], c - a)
    return out


def explore_commit(conf, tok, in_plan, commit_mask, seg_off, row_pos, active, tau_lo: float, tau_hi: float,
                   u, planning: bool, y: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Exploration variants of the appendix ("Planning tokens beyond high-confidence decoding"): after the
    high-confidence commits, commit exactly one more token per sequence from the closed confidence bin
    [tau_lo, tau_hi].

    Eligible rows: active, not base-committed, tau_lo <= p <= tau_hi.  "Random" draws one of them
    uniformly; "Planning" draws uniformly from the eligible rows whose top-1 token is in P^plan and falls
    back to the Random rule when there is none.  The uniform draw is an input: u[b] in [0, 1) selects the
    floor(u * n)-th of the n rows of the chosen set in position order (product taken in fp32, the precision
    of the interface).  Returns the updated commit mask and explore_row[n_seq] (-1: bin empty).
    """
    conf = np.asarray(conf, dtype=np.float64)
    M = len(conf)
    n_seq = len(seg_off) - 1
    act = np.ones(M, np.uint8) if active is None else np.asarray(active)
    lo, hi = f32(tau_lo), f32(tau_hi)
    out = np.array(commit_mask, dtype=np.uint8, copy=True)
    explore_row = np.full(n_seq, -1, dtype=np.int32)
    for b in range(n_seq):
        rows = range(int(seg_off[b]), int(seg_off[b + 1]))
        eligible = [m for m in rows if act[m] and not commit_mask[m] and lo <= conf[m] <= hi]
        pool = eligible
        if planning:
            plan = [m for m in eligible if in_plan[m]]
            if plan:
                pool = plan
        if pool:
            n = len(pool)
            idx = min(int(np.float32(u[b]) * np.float32(n)), n - 1)
            explore_row[b] = pool[idx]
            out[pool[idx]] = 1
    res = dict(commit=out, explore_row=explore_row)
    if y is not None:
        y2 = np.array(y, copy=True)
        for b in range(n_seq):
            if explore_row[b] >= 0:
                y2[b, int(row_pos[explore_row[b]])] = int(tok[explore_row[b]])
        res["y"] = y2
    return res
