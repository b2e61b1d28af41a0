"""Pins of the exploration-variant oracle (appendix: one extra in-bin commit, Random or Planning).  CPU only."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import step as ostep


def setup(conf, in_plan=None, commit=None, active=None):
    M = len(conf)
    seg = np.array([0, M], np.int32)
    return dict(conf=np.asarray(conf, np.float64), tok=np.arange(100, 100 + M), in_plan=np.zeros(M, np.uint8) if in_plan is None else np.asarray(in_plan, np.uint8),
                commit_mask=np.zeros(M, np.uint8) if commit is None else np.asarray(commit, np.uint8), seg_off=seg,
                row_pos=np.arange(M), active=active)


def test_closed_bin_and_position_order():
    lo, hi = float(np.float32(0.2)), float(np.float32(0.6))
    s = setup([0.95, lo, 0.4, hi, 0.61, 0.19, 0.5], commit=[1, 0, 0, 0, 0, 0, 0])
    # eligible in position order: rows 1 (on the lower edge), 2, 3 (on the upper edge), 6
    picks = [int(ostep.explore_commit(tau_lo=0.2, tau_hi=0.6, u=[u], planning=False, **s)["explore_row"][0])
             for u in (0.0, 0.24, 0.25, 0.49, 0.5, 0.74, 0.75, 0.999)]
    assert picks == [1, 1, 2, 2, 3, 3, 6, 6]
    r = ostep.explore_commit(tau_lo=0.2, tau_hi=0.6, u=[0.5], planning=False, **s)
    assert r["commit"].tolist() == [1, 0, 0, 1, 0, 0, 0]       # exactly one extra commit, the base commit kept


def test_planning_prefers_the_planning_subset_and_falls_back():
    s = setup([0.3, 0.4, 0.5, 0.55], in_plan=[0, 1, 0, 1])
    picks = [int(ostep.explore_commit(tau_lo=0.2, tau_hi=0.6, u=[u], planning=True, **s)["explore_row"][0])
             for u in (0.0, 0.49, 0.5, 0.99)]
    assert picks == [1, 1, 3, 3]                                # only rows whose token is in P^plan
    s = setup([0.3, 0.4, 0.5, 0.55])                            # no planning token in the bin: Random rule
    picks = [int(ostep.explore_commit(tau_lo=0.2, tau_hi=0.6, u=[u], planning=True, **s)["explore_row"][0])
             for u in (0.0, 0.3, 0.6, 0.9)]
    assert picks == [0, 1, 2, 3]
    s = setup([0.7, 0.1])                                       # empty bin: nothing happens
    r = ostep.explore_commit(tau_lo=0.2, tau_hi=0.6, u=[0.3], planning=True, **s)
    assert r["explore_row"][0] == -1 and r["commit"].sum() == 0


def test_uniform_over_the_eligible_rows():
    rng = np.random.default_rng(1)
    conf = rng.random(40)
    s = setup(conf, active=(rng.random(40) < 0.8).astype(np.uint8))
    elig = [m for m in range(40) if s["active"][m] and 0.2 <= conf[m] <= 0.6]
    counts = {m: 0 for m in elig}
    N = 1200 * len(elig)
    for k in range(N):                                          # an even grid of draws hits every row equally often
        m = int(ostep.explore_commit(tau_lo=0.2, tau_hi=0.6, u=[(k + 0.5) / N], planning=False, **s)["explore_row"][0])
        counts[m] += 1
    assert set(counts.values()) == {1200}


@settings(max_examples=150, deadline=None)
@given(st.integers(0, 2 ** 31 - 1), st.booleans())
def test_invariants(seed, planning):
    rng = np.random.default_rng(seed)
    sizes = rng.integers(0, 12, 4)
    seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    M = int(seg[-1])
    conf = rng.random(M)
    tok = rng.integers(0, 9, M)
    inp = (rng.random(M) < 0.3).astype(np.uint8)
    act = (rng.random(M) < 0.8).astype(np.uint8)
    pos = np.concatenate([np.arange(s) for s in sizes]) if M else np.zeros(0, int)
    base = ostep.commit(conf, tok, seg, pos, act, 0.9)["commit"]
    y = np.full((4, 12), -1, np.int64)
    r = ostep.explore_commit(conf, tok, inp, base, seg, pos, act, 0.2, 0.6, rng.random(4), planning, y=y)
    lo, hi = float(np.float32(0.2)), float(np.float32(0.6))
    for b in range(4):
        rows = np.arange(seg[b], seg[b + 1])
        elig = [m for m in rows if act[m] and not base[m] and lo <= conf[m] <= hi]
        extra = [m for m in rows if r["commit"][m] and not base[m]]
        assert len(extra) == (1 if elig else 0)
        if elig:
            m = extra[0]
            assert m == r["explore_row"][b] and m in elig and r["y"][b, pos[m]] == tok[m]
            if planning and any(inp[e] for e in elig):
                assert inp[m]
        else:
            assert r["explore_row"][b] == -1
    assert np.all(r["commit"] >= base) and (r["y"] != -1).sum() == (r["explore_row"] >= 0).sum()
