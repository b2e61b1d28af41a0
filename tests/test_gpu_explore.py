"""pvf_explore_commit (appendix exploration variants) against the oracle, bit for bit, and the Static
baseline (one most confident token per step) through pvf_commit."""
import numpy as np
import pytest
import torch

from oracle import step as ostep
from paper_2601_12247_b200 import binding, synth
from gpu_util import dev, make_ctx, t_f32, t_i32, t_u8, to_np

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    st = synth.config0()
    c = make_ctx(st.w_bits, st.plan_ids, 40000, max_seqs=128)
    yield c
    c.close()


@pytest.mark.parametrize("n_seq,max_rows", [(1, 40), (16, 32), (64, 512), (128, 3), (5, 700)])
@pytest.mark.parametrize("mode", [binding.PVF_EXPLORE_RANDOM, binding.PVF_EXPLORE_PLANNING])
def test_random_arrays(ctx, n_seq, max_rows, mode):
    rng = np.random.default_rng(n_seq * 31 + max_rows + mode)
    for trial in range(4):
        sizes = rng.integers(0, max_rows + 1, n_seq)
        seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
        M = int(seg[-1])
        if M == 0:
            continue
        pos = np.concatenate([np.arange(s) for s in sizes]).astype(np.int32)
        conf = rng.random(M).astype(np.float32)
        conf[rng.random(M) < 0.05] = np.float32(0.2)               # rows exactly on the closed bin's edges
        conf[rng.random(M) < 0.05] = np.float32(0.6)
        tok = rng.integers(0, 4096, M).astype(np.int32)
        inp = (rng.random(M) < (0.0 if trial == 3 else 0.3)).astype(np.uint8)   # last trial: always the fallback
        act = (rng.random(M) < 0.8).astype(np.uint8)
        u = rng.random(n_seq).astype(np.float32)
        base = ostep.commit(conf, tok, seg, pos, act, 0.9)["commit"]
        L = int(max(sizes.max(), 1))
        y0 = np.full((n_seq, L), -1, np.int32)
        want = ostep.explore_commit(conf, tok, inp, base, seg, pos, act, 0.2, 0.6, u, mode == binding.PVF_EXPLORE_PLANNING, y=y0)
        prm = binding.make_params(0.9, 0.2, 0.6, 0.1, 4)
        commit_d, y_d = t_u8(base), t_i32(y0)
        row = ctx.explore_commit(prm, mode, t_i32(seg), t_i32(pos), t_u8(act), t_i32(tok), t_f32(conf), t_u8(inp), t_f32(u),
                                 commit_d, y=y_d)
        torch.cuda.synchronize()
        assert np.array_equal(row.cpu().numpy(), want["explore_row"])
        assert np.array_equal(commit_d.cpu().numpy(), want["commit"])
        assert np.array_equal(y_d.cpu().numpy(), want["y"])
    assert ctx.last_status() == 0


def test_static_baseline_is_commit_with_forced_progress(ctx):
    # tau_high above 1 commits nothing by threshold; forced progress then commits the single most confident
    # active row of every sequence (the lowest position on ties): one token per step, as the Static baseline
    rng = np.random.default_rng(3)
    sizes = rng.integers(1, 60, 32)
    seg = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    M = int(seg[-1])
    pos = np.concatenate([np.arange(s) for s in sizes]).astype(np.int32)
    conf = rng.random(M).astype(np.float32)
    conf[seg[3]:seg[4]] = np.float32(0.5)                          # a sequence of exact ties
    tok = rng.integers(0, 4096, M).astype(np.int32)
    prm = binding.make_params(1.5, 0.2, 0.6, 0.1, 0, binding.PVF_FORCE_PROGRESS)
    cm = to_np(ctx.commit(prm, t_i32(seg), t_i32(pos), None, t_i32(tok), t_f32(conf)))
    for b in range(32):
        rows = np.arange(seg[b], seg[b + 1])
        assert cm["commit"][rows].sum() == 1 and cm["commit"][rows[np.argmax(conf[rows])]] == 1
    assert (cm["n_commit"] == 1).all()
