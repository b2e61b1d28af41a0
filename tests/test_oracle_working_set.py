"""Pins of the working-set oracle: semi-autoregressive block order (Appendix A.1) with early
cross-block revelation (Appendix, Eq. 4).  CPU only."""
import os

import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import loop as oloop

MASK = -7
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def canvas(rows):
    """'M' = mask, anything else = a committed token."""
    return np.array([[MASK if c == "M" else 11 for c in r.replace(" ", "")] for r in rows], np.int32)


def test_hand_built_cases():
    # block size 4; blocks are separated by spaces
    y = canvas(["ttMM MMMM MMMM",      # 2 masks left in block 0
                "tttt tMtM MMMM",      # block 0 done, 2 masks left in block 1
                "tttt tttt MMtM",      # last block: nothing to reveal
                "tttt tttt tttt",      # finished
                "MttM MtMM MMMM"])     # next block already partly committed by an earlier revelation
    # N_s = 1: no sequence has <= 1 masks in its active block -> plain block order
    seq, pos, seg, exp = oloop.working_set(y, MASK, 4, 1)
    assert exp.tolist() == [0, 0, 0, 0, 0]
    assert seg.tolist() == [0, 2, 4, 7, 7, 9]
    assert pos.tolist() == [2, 3, 5, 7, 8, 9, 11, 0, 3]
    assert seq.tolist() == [0, 0, 1, 1, 2, 2, 2, 4, 4]
    # N_s = 2: sequences 0, 1 and 4 reveal their next block; sequence 2 has 3 masks and no next block
    seq, pos, seg, exp = oloop.working_set(y, MASK, 4, 2)
    assert exp.tolist() == [1, 1, 0, 0, 1]
    assert pos[seg[0]:seg[1]].tolist() == [2, 3, 4, 5, 6, 7]
    assert pos[seg[1]:seg[2]].tolist() == [5, 7, 8, 9, 10, 11]
    assert pos[seg[2]:seg[3]].tolist() == [8, 9, 11]
    assert seg[3] == seg[4]
    assert pos[seg[4]:seg[5]].tolist() == [0, 3, 4, 6, 7]      # only the masked positions of block 1
    # N_s = 3 additionally meets the last block's 3 masks, which still has nothing to reveal
    _, pos3, seg3, exp3 = oloop.working_set(y, MASK, 4, 3)
    assert exp3.tolist() == [1, 1, 0, 0, 1] and pos3[seg3[2]:seg3[3]].tolist() == [8, 9, 11]


def plain_block_rule(y, block):
    """Independent vectorised restatement of strict block order: the masked positions of the first
    block that holds a mask."""
    masked = y == MASK
    out = []
    for b in range(y.shape[0]):
        per_block = masked[b].reshape(-1, block).sum(axis=1)
        nz = np.nonzero(per_block)[0]
        if len(nz) == 0:
            out.append(np.zeros(0, np.int64))
        else:
            k = nz[0]
            out.append(k * block + np.nonzero(masked[b, k * block:(k + 1) * block])[0])
    return out


@settings(max_examples=200, deadline=None)
@given(st.integers(1, 4), st.integers(1, 5), st.sampled_from([2, 4, 8]), st.integers(0, 9), st.integers(0, 2 ** 31 - 1))
def test_invariants(n_seq, n_blocks, block, n_sparse, seed):
    rng = np.random.default_rng(seed)
    L = n_blocks * block
    y = np.where(rng.random((n_seq, L)) < rng.random(), MASK, 5).astype(np.int32)
    seq, pos, seg, exp = oloop.working_set(y, MASK, block, n_sparse)
    plain = plain_block_rule(y, block)
    _, pos0, seg0, exp0 = oloop.working_set(y, MASK, block, 0)
    assert not exp0.any()
    _, pos_more, seg_more, _ = oloop.working_set(y, MASK, block, n_sparse + 1)
    for b in range(n_seq):
        rows = pos[seg[b]:seg[b + 1]]
        assert np.array_equal(pos0[seg0[b]:seg0[b + 1]], plain[b])            # N_s = 0 is strict block order
        assert (seq[seg[b]:seg[b + 1]] == b).all()
        assert np.all(np.diff(rows) > 0) and np.all(y[b, rows] == MASK)
        if len(plain[b]) == 0:
            assert len(rows) == 0 and not exp[b]
            continue
        k = plain[b][0] // block
        assert rows[0] == plain[b][0]                                          # first masked position of the canvas
        should = len(plain[b]) <= n_sparse and k + 1 < n_blocks
        assert bool(exp[b]) == should
        if should:
            nxt = (k + 1) * block + np.nonzero(y[b, (k + 1) * block:(k + 2) * block] == MASK)[0]
            assert np.array_equal(rows, np.concatenate([plain[b], nxt]))
        else:
            assert np.array_equal(rows, plain[b])
        assert set(rows.tolist()) <= set(pos_more[seg_more[b]:seg_more[b + 1]].tolist())   # monotone in N_s


def test_papers_printed_thresholds():
    golden = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "paper_hyperparameters.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            golden[k] = float(v)
    # Table 5: N_s = 5 with block 64 (GSM8K, MMLU-Pro), N_s = 0 (HumanEval, MATH)
    S = int(golden["block_size"])
    y = np.full((1, 3 * S), MASK, np.int32)
    y[0, :S - 5] = 1                                        # 5 masks left in block 0
    _, pos, _, exp = oloop.working_set(y, MASK, S, int(golden["early_reveal_Ns"]))
    assert exp[0] == 1 and len(pos) == 5 + S
    y[0, S - 6] = MASK                                      # 6 masks left: above the threshold
    _, pos, _, exp = oloop.working_set(y, MASK, S, int(golden["early_reveal_Ns"]))
    assert exp[0] == 0 and len(pos) == 6
    _, pos, _, exp = oloop.working_set(y[:, :], MASK, S, int(golden["alt_early_reveal_Ns"]))
    assert exp[0] == 0
