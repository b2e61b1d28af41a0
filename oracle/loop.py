"""CPU oracle for the decode loop (Algorithm 1) on synthetic hidden states -- TEST INFRASTRUCTURE.

The transformer is replaced by the seeded generator: at every step the hidden states of the
scored rows are re-drawn from (seed, step, sequence, position) with an amplitude that grows with
the sequence's committed fraction.  Decoding is semi-autoregressive (Appendix A.1): the working
block of a sequence is its first block that still holds a mask, and the scored rows are that
block's masked positions.  One loop step = one batched forward (draft pass and verification
branches counted together).

`decode(..., budget=0)` is confidence-threshold decoding (Section 2): nothing is drafted, every
step commits the base set only.  `n_sparse` is the early cross-block threshold N_s (Appendix,
"Planning-Guided Early Cross-Block Revelation", Eq. 4; 0 = strict block order).
"""
from __future__ import annotations

from typing import Dict

import numpy as np

from . import score as oscore
from . import step as ostep


def working_set(y: np.ndarray, mask_id: int, block: int, n_sparse: int = 0):
    """Rows of the current step with early cross-block revelation (Appendix, Eq. 4).

    For each sequence: k_t is the first block that holds a mask and M_active its masked
    positions.  The working index set B_t is M_active, widened by the whole index range of
    block k_t + 1 when |M_active| <= N_s (``n_sparse``) and that block exists.  The scored rows
    are the masked positions of B_t, ascending.  N_s = 0 never widens (|M_active| >= 1).
    Returns seq_ids, positions, seg_off and the per-sequence flag ``expanded``."""
    n_seq, L = y.shape
    seq_ids, positions = [], []
    seg_off = np.zeros(n_seq + 1, dtype=np.int32)
    expanded = np.zeros(n_seq, dtype=np.uint8)
    for b in range(n_seq):
        masked = [int(i) for i in range(L) if y[b, i] == mask_id]
        if masked:
            k = masked[0] // block                               # k_t (0-based)
            m_active = [i for i in masked if k * block <= i < (k + 1) * block]
            b_t = set(m_active)
            if len(m_active) <= n_sparse and (k + 1) * block < L:
                b_t |= set(range((k + 1) * block, min((k + 2) * block, L)))   # I_{k_t+1}
                expanded[b] = 1
            pos = [i for i in masked if i in b_t]
            seq_ids.extend([b] * len(pos))
            positions.extend(pos)
        seg_off[b + 1] = len(positions)
    return np.asarray(seq_ids, np.int32), np.asarray(positions, np.int32), seg_off, expanded


def working_rows(y: np.ndarray, mask_id: int, block: int, n_sparse: int = 0):
    """seq_ids, positions (ascending per sequence), seg_off of the current step's rows."""
    seq_ids, positions, seg_off, _ = working_set(y, mask_id, block, n_sparse)
    return seq_ids, positions, seg_off


def decode(synth, w_bits, plan_ids, targets, seed: int, gen_len: int, block: int, params: Dict,
           mask_id: int, max_steps: int = 100000, trace: bool = False, n_sparse: int = 0,
           explore: str = "") -> Dict:
    """Run Algorithm 1 until no masks remain.  ``synth`` is the input-generator module.

    ``explore`` = "random" or "planning" runs the appendix's exploration loop instead ("Planning tokens
    beyond high-confidence decoding"): every step commits the base set and then exactly one more token
    from the closed confidence bin [tau_plan_lo, tau_plan_hi]; nothing is drafted or verified (the budget
    is ignored).  The uniform draws come from the input generator."""
    n_seq = targets.shape[0]
    K = 0 if explore else int(params["budget"])
    y = np.full((n_seq, gen_len), mask_id, dtype=np.int32)
    steps_per_seq = np.zeros(n_seq, dtype=np.int32)
    scored_rows = 0
    n_steps = 0
    history = []
    while (y == mask_id).any():
        if n_steps >= max_steps:
            raise RuntimeError("decode loop did not terminate")
        seq_ids, positions, seg_off = working_rows(y, mask_id, block, n_sparse)
        frac = (y != mask_id).sum(axis=1) / float(gen_len)
        h = synth.loop_hidden(w_bits, targets, seed, n_steps, 0, seq_ids, positions, frac)
        sc = oscore.score(w_bits, h, plan_ids)
        active = np.ones(len(positions), np.uint8)
        cm = ostep.commit(sc["conf"], sc["tok"], seg_off, positions, active, params["tau_high"],
                          force_progress=True)
        scored_rows += len(positions)
        final = cm["commit"]
        sel = ver = exp = None
        if explore:
            exp = ostep.explore_commit(sc["conf"], sc["tok"], sc["in_plan"], cm["commit"], seg_off, positions, active,
                                       params["tau_plan_lo"], params["tau_plan_hi"],
                                       synth.loop_uniforms(seed, n_steps, n_seq), explore == "planning")
            final = exp["commit"]
        if K > 0:
            sel = ostep.select_drafts(sc["conf"], sc["tok"], sc["in_plan"], cm["commit"], seg_off,
                                      positions, active, params["tau_plan_lo"], params["tau_plan_hi"],
                                      params["tau_ar_lo"], K)
            vb, vi, vc = [], [], []
            for b in range(n_seq):
                rem = sel["rem_rows"][sel["rem_off"][b]:sel["rem_off"][b + 1]]
                if sel["n_drafts"][b] > 0:
                    for c in range(1 + int(sel["n_drafts"][b])):
                        for m in rem:
                            vb.append(b); vi.append(int(positions[m])); vc.append(c)
            hv = synth.loop_verify_hidden(w_bits, targets, seed, n_steps, np.asarray(vb, np.int32),
                                          np.asarray(vi, np.int32), np.asarray(vc, np.int32), frac)
            scv = oscore.score(w_bits, hv, plan_ids)
            scored_rows += len(vb)
            ver = ostep.verify(sc["tok"], cm["commit"], seg_off, positions, sel["rem_rows"],
                               sel["rem_off"], sel["v_off"], sel["draft_rows"], sel["n_drafts"],
                               sel["route"], scv["tok"], scv["conf"], params["tau_high"], K)
            final = ver["final_commit"]
        for m in range(len(positions)):
            if final[m]:
                y[seq_ids[m], positions[m]] = sc["tok"][m]
        for b in range(n_seq):
            if seg_off[b + 1] > seg_off[b]:
                steps_per_seq[b] += 1
        if trace:
            history.append(dict(positions=positions.copy(), seq_ids=seq_ids.copy(), score=sc,
                                commit=cm, select=sel, verify=ver, explore=exp, y=y.copy()))
        n_steps += 1
    out = dict(y=y, steps=n_steps, steps_per_seq=steps_per_seq, scored_rows=scored_rows,
               tokens_per_forward=float(np.mean(gen_len / np.maximum(steps_per_seq, 1))))
    if trace:
        out["history"] = history
    return out
