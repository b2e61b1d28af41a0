"""Pins of the decode-loop oracle (Algorithm 1 on synthetic hidden states), CPU only."""
import numpy as np

from oracle import loop as oloop
from oracle import score as oscore
from paper_2601_12247_b200 import synth

V, D, B, L, S = 1024, 64, 3, 64, 32
SEED = 1004
P = dict(tau_high=0.9, tau_plan_lo=0.2, tau_plan_hi=0.65, tau_ar_lo=0.1, budget=4)
MASK = V - 1


def setup():
    w = synth.make_w(SEED, V, D)
    plan = synth.make_plan_ids(SEED, V, 128)
    tg = synth.loop_targets(SEED, V, B, L, plan, 0.5, avoid=MASK)
    return w, plan, tg


def threshold_only(w, plan, tg):
    """Independent restatement of confidence-threshold decoding (Section 2) with the same
    forced-progress rule: per step commit every masked position of the working block whose
    confidence reaches tau_high, else the single most confident one."""
    y = np.full((B, L), MASK, np.int32)
    steps = np.zeros(B, np.int32)
    s = 0
    while (y == MASK).any():
        frac = (y != MASK).sum(axis=1) / float(L)
        for b in range(B):
            masked = np.nonzero(y[b] == MASK)[0]
            if not len(masked):
                continue
            k = masked[0] // S
            pos = masked[(masked >= k * S) & (masked < (k + 1) * S)].astype(np.int32)
            h = synth.loop_hidden(w, tg, SEED, s, 0, np.full(len(pos), b, np.int32), pos, frac)
            sc = oscore.score(w, h)
            take = sc["conf"] >= float(np.float32(P["tau_high"]))
            if not take.any():
                take[int(np.argmax(sc["conf"]))] = True
            y[b, pos[take]] = sc["tok"][take]
            steps[b] += 1
        s += 1
    return y, steps


def test_loop_terminates_monotone_and_counts_commits():
    w, plan, tg = setup()
    r = oloop.decode(synth, w, plan, tg, SEED, L, S, P, MASK, trace=True)
    assert not (r["y"] == MASK).any()
    prev = np.full((B, L), MASK, np.int32)
    for h in r["history"]:
        y = h["y"]
        keep = prev != MASK
        assert np.array_equal(y[keep], prev[keep])           # committed tokens never change or re-mask
        new = int(((y != MASK) & ~keep).sum())
        ver, cm, sel = h["verify"], h["commit"], h["select"]
        extra = 0
        for b in range(B):
            if sel["route"][b] == 1:
                extra += 1 if ver["choice"][b] > 0 else 0
            elif sel["route"][b] == 2:
                extra += int(ver["choice"][b])
            assert sel["n_drafts"][b] <= P["budget"]
        assert new == int(cm["commit"].sum()) + extra
        prev = y
    assert r["steps"] == len(r["history"]) and r["steps_per_seq"].max() == r["steps"]


def test_budget_zero_is_threshold_decoding():
    w, plan, tg = setup()
    r0 = oloop.decode(synth, w, plan, tg, SEED, L, S, dict(P, budget=0), MASK)
    y, steps = threshold_only(w, plan, tg)
    assert np.array_equal(r0["y"], y)
    assert np.array_equal(r0["steps_per_seq"], steps)


def test_pvf_needs_no_more_forwards_than_threshold_decoding_here():
    w, plan, tg = setup()
    r = oloop.decode(synth, w, plan, tg, SEED, L, S, P, MASK)
    r0 = oloop.decode(synth, w, plan, tg, SEED, L, S, dict(P, budget=0), MASK)
    assert r["steps_per_seq"].sum() <= r0["steps_per_seq"].sum()
    assert r["tokens_per_forward"] >= 1.0


def test_early_cross_block_revelation_loop_terminates_and_never_skips_ahead():
    # Eq. 4: with N_s > 0 the loop may fill positions of block k+1 while block k still holds masks,
    # but never anything beyond block k+1; it still terminates and never changes a committed token.
    w, plan, tg = setup()
    r = oloop.decode(synth, w, plan, tg, SEED, L, S, P, MASK, trace=True, n_sparse=6)
    assert not (r["y"] == MASK).any()
    prev = np.full((B, L), MASK, np.int32)
    for h in r["history"]:
        keep = prev != MASK
        assert np.array_equal(h["y"][keep], prev[keep])
        for b in range(B):
            masked = np.nonzero(prev[b] == MASK)[0]
            if len(masked):
                k = masked[0] // S
                new = np.nonzero((h["y"][b] != MASK) & (prev[b] == MASK))[0]
                assert np.all(new < (k + 2) * S)
        prev = h["y"]


def test_exploration_loops_commit_one_extra_token_per_step():
    w, plan, tg = setup()
    base = oloop.decode(synth, w, plan, tg, SEED, L, S, dict(P, budget=0), MASK)
    for mode in ("random", "planning"):
        r = oloop.decode(synth, w, plan, tg, SEED, L, S, P, MASK, trace=True, explore=mode)
        assert not (r["y"] == MASK).any()
        assert r["steps_per_seq"].sum() <= base["steps_per_seq"].sum()      # never slower than threshold decoding
        extra_total = 0
        for h in r["history"]:
            ex = h["explore"]
            extra = (ex["commit"].astype(int) - h["commit"]["commit"].astype(int))
            assert extra.min() >= 0 and h["select"] is None and h["verify"] is None
            for b in range(B):
                rows = np.nonzero(h["seq_ids"] == b)[0]
                assert extra[rows].sum() == (1 if ex["explore_row"][b] >= 0 else 0)
                if ex["explore_row"][b] >= 0:
                    p = h["score"]["conf"][ex["explore_row"][b]]
                    assert float(np.float32(P["tau_plan_lo"])) <= p <= float(np.float32(P["tau_plan_hi"]))
            extra_total += int(extra.sum())
        assert extra_total > 0
