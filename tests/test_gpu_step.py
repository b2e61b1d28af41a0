"""pvf_commit / pvf_select_drafts / pvf_verify against the oracle on hand-made and random arrays
(bit-exact: both sides decide on the same fp32 numbers)."""
import numpy as np
import pytest
import torch

from oracle import step as ostep
from paper_2601_12247_b200 import binding, synth
from gpu_util import dev, make_ctx, t_f32, t_i32, t_u8, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    w = synth.make_w(1, 256, 64)
    c = make_ctx(w, [1, 2, 3], max_rows=40000, max_seqs=4096, max_budget=32)
    yield c
    c.close()


def random_case(rng, n_seq, max_len, K, grid=True, inactive=True):
    lens = rng.integers(0, max_len + 1, n_seq)
    seg = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    M = int(seg[-1])
    L = max_len + 8
    pos = np.concatenate([np.sort(rng.permutation(L)[:l]) for l in lens] + [np.zeros(0, np.int64)]).astype(np.int32)
    if grid:      # many exact ties and values exactly on the thresholds
        conf = rng.choice(np.array([0.0, 0.05, 0.1, 0.15, 0.2, 0.3, 0.3, 0.5, 0.64, 0.65, 0.8, 0.9, 0.95, 1.0], np.float32), M)
    else:
        conf = rng.random(M).astype(np.float32)
    tok = rng.integers(0, 1000, M).astype(np.int32)
    in_plan = (rng.random(M) < 0.4).astype(np.uint8)
    active = (rng.random(M) < 0.85).astype(np.uint8) if inactive else np.ones(M, np.uint8)
    return dict(seg=seg, pos=pos, conf=conf, tok=tok, in_plan=in_plan, active=active, M=M, L=L, n_seq=n_seq, K=K)


def run_step(ctx, c, tau_high=0.9, flags=0, rng=None, agree=0.7):
    """Runs commit -> select -> verify on the GPU and in the oracle; compares everything."""
    prm = binding.make_params(tau_high, 0.2, 0.65, 0.1, c["K"], flags)
    seg, pos, act = t_i32(c["seg"]), t_i32(c["pos"]), t_u8(c["active"])
    tok, conf, inp = t_i32(c["tok"]), t_f32(c["conf"]), t_u8(c["in_plan"])
    y0 = np.full((c["n_seq"], c["L"]), -1, np.int32)
    y = t_i32(y0)
    cm = ctx.commit(prm, seg, pos, act, tok, conf, y=y)
    force = bool(flags & binding.PVF_FORCE_PROGRESS)
    ocm = ostep.commit(c["conf"], c["tok"], c["seg"], c["pos"], c["active"], tau_high, force, y=y0)
    g = to_np(cm)
    assert np.array_equal(g["commit"], ocm["commit"]) and np.array_equal(g["n_commit"], ocm["n_commit"])
    assert np.array_equal(y.cpu().numpy(), ocm["y"])

    sel = ctx.select_drafts(prm, seg, pos, act, tok, conf, inp, cm["commit"])
    osel = ostep.select_drafts(c["conf"], c["tok"], c["in_plan"], ocm["commit"], c["seg"], c["pos"], c["active"],
                               0.2, 0.65, 0.1, c["K"])
    gs = to_np(sel)
    n_rem = int(osel["rem_off"][-1])
    for k in ("draft_rows", "n_drafts", "route", "rem_off", "v_off"):
        assert np.array_equal(gs[k], osel[k]), k
    assert np.array_equal(gs["rem_rows"][:n_rem], osel["rem_rows"])
    # the fused call (one launch) gives what the two calls gave, bit for bit, canvas included
    y2 = t_i32(y0)
    both = to_np(ctx.commit_select(prm, seg, pos, act, tok, conf, inp, y=y2))
    assert np.array_equal(both["commit"], g["commit"]) and np.array_equal(both["n_commit"], g["n_commit"])
    assert np.array_equal(y2.cpu().numpy(), ocm["y"])
    for k in ("draft_rows", "n_drafts", "route", "rem_off", "v_off"):
        assert np.array_equal(both[k], gs[k]), k
    assert np.array_equal(both["rem_rows"][:n_rem], osel["rem_rows"])

    # verification-pass outputs: start from "every branch repeats the draft-pass token", then flip some
    rng = rng or np.random.default_rng(0)
    Mv = int(osel["v_off"][-1])
    tok_v = np.zeros(Mv, np.int32)
    conf_v = rng.choice(np.array([0.1, 0.5, 0.89, 0.9, 0.95, 0.99], np.float32), Mv) if Mv else np.zeros(0, np.float32)
    for b in range(c["n_seq"]):
        rem = osel["rem_rows"][osel["rem_off"][b]:osel["rem_off"][b + 1]]
        if osel["n_drafts"][b] > 0:
            for cc in range(1 + osel["n_drafts"][b]):
                o = osel["v_off"][b] + cc * len(rem)
                tok_v[o:o + len(rem)] = c["tok"][rem]
    flip = rng.random(Mv) > agree
    tok_v[flip] += 1
    ver = ctx.verify(prm, seg, pos, sel, tok, t_i32(tok_v), t_f32(conf_v), cm["commit"], y=y)
    over = ostep.verify(c["tok"], ocm["commit"], c["seg"], c["pos"], osel["rem_rows"], osel["rem_off"], osel["v_off"],
                        osel["draft_rows"], osel["n_drafts"], osel["route"], tok_v, conf_v, tau_high, c["K"],
                        exclude_self=bool(flags & binding.PVF_EXCLUDE_SELF_FROM_IMPACT), y=ocm["y"])
    gv = to_np(ver)
    for k in ("accept", "choice", "final_commit"):
        assert np.array_equal(gv[k], over[k]), k
    assert np.array_equal(y.cpu().numpy(), over["y"])
    torch.cuda.synchronize()
    return osel, over


@pytest.mark.parametrize("seed", range(6))
def test_random_steps_with_ties_and_threshold_values(ctx, seed):
    rng = np.random.default_rng(seed)
    c = random_case(rng, n_seq=int(rng.integers(1, 40)), max_len=int(rng.integers(1, 70)), K=int(rng.integers(0, 9)))
    run_step(ctx, c, rng=rng, flags=[0, 1, 2, 3][seed % 4])


def test_long_sequences_budget_16(ctx):
    rng = np.random.default_rng(77)
    c = random_case(rng, n_seq=64, max_len=512, K=16, grid=False)
    osel, over = run_step(ctx, c, tau_high=0.95, rng=rng, agree=0.97)
    assert (osel["route"] == 1).any() and (over["choice"] > 0).any()


def test_ar_route_and_forced_progress(ctx):
    rng = np.random.default_rng(5)
    c = random_case(rng, n_seq=30, max_len=40, K=4)
    c["in_plan"][:] = 0                                   # no planning candidate anywhere -> AR route
    osel, over = run_step(ctx, c, rng=rng, flags=binding.PVF_FORCE_PROGRESS, agree=0.9)
    assert set(np.unique(osel["route"]).tolist()) <= {0, 2} and (osel["route"] == 2).any()
    assert (over["choice"] > 1).any()


def test_many_short_sequences_and_empty_ones(ctx):
    rng = np.random.default_rng(9)
    c = random_case(rng, n_seq=1500, max_len=6, K=3)
    run_step(ctx, c, rng=rng)


def test_single_row_and_budget_zero(ctx):
    rng = np.random.default_rng(3)
    c = random_case(rng, n_seq=1, max_len=1, K=0)
    run_step(ctx, c, rng=rng)
    c = random_case(rng, n_seq=5, max_len=20, K=0)
    osel, over = run_step(ctx, c, rng=rng)
    assert osel["n_drafts"].sum() == 0 and over["choice"].sum() == 0       # K = 0: threshold decoding only


@pytest.mark.parametrize("seed", range(8))
def test_single_sequence_writes_its_offsets_directly(ctx, seed):
    """One sequence takes a path of its own in draft selection (no ticket, no packing): every budget, both routes,
    lengths around a block of 256 threads, rows with and without the active flag."""
    rng = np.random.default_rng(100 + seed)
    max_len = [1, 7, 32, 64, 255, 256, 257, 600][seed]
    c = random_case(rng, n_seq=1, max_len=max_len, K=[0, 1, 3, 4, 8, 16, 2, 5][seed], inactive=bool(seed % 2))
    while c["M"] == 0:                                    # a sequence without rows says nothing here
        c = random_case(rng, n_seq=1, max_len=max_len, K=c["K"], inactive=bool(seed % 2))
    if seed % 3 == 0:
        c["in_plan"][:] = 0                               # AR route (or none)
    osel, over = run_step(ctx, c, rng=rng, flags=[0, 1, 2, 3][seed % 4])
    assert osel["rem_off"][0] == 0 and osel["v_off"][0] == 0


def test_argument_errors(ctx):
    prm = binding.make_params(0.9, 0.2, 0.65, 0.1, 64)      # budget above the context's limit
    seg = t_i32([0, 1])
    z = t_i32([0]); f = t_f32([0.5]); u = t_u8([1])
    with pytest.raises(binding.PvfError) as e:
        ctx.commit(prm, seg, z, u, z, f)
    assert e.value.code == binding.PVF_ERR_INVALID
    prm = binding.make_params(0.9, 0.2, 0.65, 0.1, 2)
    rc = ctx.lib.pvf_commit(ctx.handle, prm, 1, 1, None, None, None, None, None, None, None, None, 0, None)
    assert rc == binding.PVF_ERR_INVALID
    # zero sequences is a no-op
    rc = ctx.lib.pvf_commit(ctx.handle, prm, 0, 0, None, None, None, None, None, None, None, None, 0, None)
    assert rc == binding.PVF_OK
