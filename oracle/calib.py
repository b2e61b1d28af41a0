"""CPU oracle for the planning-token calibration statistics -- TEST INFRASTRUCTURE, not part of the product.

Written from the paper's definitions: verified information gain (Section 3, "Verified information
gain") and the token-level aggregation and filtering rule of the planning-token set construction
(Appendix, "Planning Token Set Construction").  Plain Python loops, fp64.

A calibration step looks at the candidate positions C_t^cal = {i in M_t \\ S_base : tau_cal^l <= p_i <
tau_cal^u} (any top-1 token, no planning-vocabulary filter), builds one planning branch per candidate and
measures, per candidate j with token v = y^_{i_(j)}:

    A_j      verified compatibility (Eq. 3), as in the decode step
    R_j      the positions of B_t still masked in the base branch, without i_(j)
    dH_j     mean over R_j of  H_i(z_base) - H_i(z_plan,j)      (0 when R_j is empty)
    VIG_j    A_j * dH_j

and adds to the token's statistics  n_v += 1,  m_v += [S_impact non-empty],  sum_A_v += A_j,
sum_VIG_v += VIG_j.  The vocabulary keeps a token iff
    n_v >= n_min,  m_v >= m_min,  sum_A_v / m_v >= rho_ver (0 when m_v = 0),  sum_VIG_v / n_v >= gamma_vig.

Rows of the verification pass are laid out as in oracle/step.py: index v_off[b] + c * nR_b + r, c = 0 the
base branch, c = j the branch of candidate j, r over the remaining rows R_b.

Readings where the paper is silent: entropies in nats; at most `budget` candidates per sequence and step
are measured (the most confident first, as in the decode step's TopK); "S_impact non-empty" refers to the
same set whose non-emptiness A_j requires (so it follows the exclude_self switch).
"""
from __future__ import annotations

from typing import Dict

import numpy as np

from .step import ROUTE_PLAN, f32


def events(tok, rem_rows, rem_off, v_off, draft_rows, n_drafts, route, tok_v, conf_v, ent_v,
           tau_high: float, exclude_self: bool = False):
    """One record per measured candidate: (sequence, j, token, impact_nonempty, A_j, dH_j, VIG_j)."""
    tau = f32(tau_high)
    conf_v = np.asarray(conf_v, dtype=np.float64)
    ent_v = np.asarray(ent_v, dtype=np.float64)
    out = []
    n_seq = len(rem_off) - 1
    for b in range(n_seq):
        if route[b] != ROUTE_PLAN:
            continue
        rem = [int(m) for m in rem_rows[int(rem_off[b]):int(rem_off[b + 1])]]
        nR = len(rem)
        base = int(v_off[b])
        for j in range(1, int(n_drafts[b]) + 1):
            row = int(draft_rows[b, j - 1])
            rj = rem.index(row)
            impact = [r for r in range(nR) if conf_v[base + r] >= tau and not (exclude_self and r == rj)]
            a_j = 1 if (impact and all(tok_v[base + j * nR + r] == tok_v[base + r] for r in impact)) else 0
            region = [r for r in range(nR) if r != rj]                        # R_t^j
            if region:
                d_h = sum(ent_v[base + r] - ent_v[base + j * nR + r] for r in region) / len(region)
            else:
                d_h = 0.0
            out.append(dict(seq=b, j=j, token=int(tok[row]), impact=1 if impact else 0, A=a_j, dH=d_h,
                            VIG=a_j * d_h))
    return out


def new_stats(vocab: int) -> Dict[str, np.ndarray]:
    return dict(n=np.zeros(vocab, np.int64), m=np.zeros(vocab, np.int64), sum_a=np.zeros(vocab, np.int64),
                sum_vig=np.zeros(vocab, np.float64))


def accumulate(stats: Dict[str, np.ndarray], evs) -> Dict[str, np.ndarray]:
    """Token-level aggregation over the event set E_v."""
    for e in evs:
        v = e["token"]
        stats["n"][v] += 1
        stats["m"][v] += e["impact"]
        stats["sum_a"][v] += e["A"]
        stats["sum_vig"][v] += e["VIG"]
    return stats


def filter_tokens(stats: Dict[str, np.ndarray], n_min: int, m_min: int, rho_ver: float, gamma_vig: float) -> np.ndarray:
    """The planning-token vocabulary: sorted ids of the tokens that pass all four thresholds."""
    rho, gam = f32(rho_ver), f32(gamma_vig)
    keep = []
    for v in range(len(stats["n"])):
        n, m = int(stats["n"][v]), int(stats["m"][v])
        if n < n_min or m < m_min or n == 0:
            continue
        r_ver = stats["sum_a"][v] / m if m > 0 else 0.0
        vig_hat = stats["sum_vig"][v] / n
        if r_ver >= rho and vig_hat >= gam:
            keep.append(v)
    return np.asarray(keep, dtype=np.int32)


def calibrate(synth, w_bits, targets, seed: int, gen_len: int, block: int, tau_high: float, tau_cal_lo: float,
              tau_cal_hi: float, budget: int, mask_id: int, max_steps: int = 100000, trace: bool = False) -> Dict:
    """Calibration trajectory on synthetic hidden states (Appendix, "Calibration trajectory").

    The canvas is decoded with the confidence-threshold base rule alone (forced progress as in the decode
    loop).  At every step the candidates C_t^cal are measured -- one planning branch each, scored by the
    generator's verification-pass hidden states -- and their events are added to the token statistics; the
    branches are never committed.  Returns the statistics, the number of events and steps."""
    from . import loop as oloop
    from . import score as oscore
    from . import step as ostep
    n_seq = targets.shape[0]
    vocab = w_bits.shape[0]
    y = np.full((n_seq, gen_len), mask_id, dtype=np.int32)
    stats = new_stats(vocab)
    n_events = n_steps = 0
    history = []
    while (y == mask_id).any():
        if n_steps >= max_steps:
            raise RuntimeError("calibration loop did not terminate")
        seq_ids, positions, seg_off = oloop.working_rows(y, mask_id, block)
        frac = (y != mask_id).sum(axis=1) / float(gen_len)
        h = synth.loop_hidden(w_bits, targets, seed, n_steps, 0, seq_ids, positions, frac)
        sc = oscore.score(w_bits, h, None)
        active = np.ones(len(positions), np.uint8)
        cm = ostep.commit(sc["conf"], sc["tok"], seg_off, positions, active, tau_high, force_progress=True)
        sel = ostep.select_drafts(sc["conf"], sc["tok"], sc["in_plan"], cm["commit"], seg_off, positions, active,
                                  tau_cal_lo, tau_cal_hi, 0.0, budget, any_token=True, ar_fallback=False)
        vb, vi, vc = [], [], []
        for b in range(n_seq):
            rem = sel["rem_rows"][sel["rem_off"][b]:sel["rem_off"][b + 1]]
            if sel["n_drafts"][b] > 0:
                for c in range(1 + int(sel["n_drafts"][b])):
                    for m in rem:
                        vb.append(b); vi.append(int(positions[m])); vc.append(c)
        evs = []
        scv = None
        if vb:
            hv = synth.loop_verify_hidden(w_bits, targets, seed, n_steps, np.asarray(vb, np.int32),
                                          np.asarray(vi, np.int32), np.asarray(vc, np.int32), frac)
            scv = oscore.score(w_bits, hv, None)
            evs = events(sc["tok"], sel["rem_rows"], sel["rem_off"], sel["v_off"], sel["draft_rows"], sel["n_drafts"],
                         sel["route"], scv["tok"], scv["conf"], scv["ent"], tau_high)
            accumulate(stats, evs)
            n_events += len(evs)
        for m in range(len(positions)):                      # only the base set is committed
            if cm["commit"][m]:
                y[seq_ids[m], positions[m]] = sc["tok"][m]
        if trace:
            history.append(dict(positions=positions.copy(), seq_ids=seq_ids.copy(), score=sc, commit=cm, select=sel,
                                score_v=scv, events=evs, y=y.copy()))
        n_steps += 1
    out = dict(stats=stats, n_events=n_events, steps=n_steps, y=y)
    if trace:
        out["history"] = history
    return out
