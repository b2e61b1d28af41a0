"""pvf_working_set (block order and early cross-block revelation, Eq. 4) against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import loop as oloop
from paper_2601_12247_b200 import binding, synth
from gpu_util import dev, make_ctx, to_np

pytestmark = pytest.mark.gpu

MASK = 4095


@pytest.fixture(scope="module")
def ctx():
    st = synth.config0()
    c = make_ctx(st.w_bits, st.plan_ids, 64, max_seqs=300)
    yield c
    c.close()


def compare(ctx, y, block, n_sparse):
    out = to_np(ctx.working_set(torch.from_numpy(y).to(dev()), block, n_sparse, MASK))
    torch.cuda.synchronize()
    seq, pos, seg, exp = oloop.working_set(y, MASK, block, n_sparse)
    assert np.array_equal(out["seg_off"], seg)
    n = int(seg[-1])
    assert np.array_equal(out["row_pos"][:n], pos) and np.array_equal(out["row_seq"][:n], seq)
    assert (out["active"][:n] == 1).all() and np.array_equal(out["expanded"][:y.shape[0]], exp)


@pytest.mark.parametrize("n_seq,L,block", [(1, 32, 32), (5, 64, 16), (64, 512, 64), (33, 256, 32), (3, 1000, 300),
                                           (7, 50, 16), (300, 96, 32)])
def test_random_canvases(ctx, n_seq, L, block):
    rng = np.random.default_rng(n_seq * 1000 + L)
    for trial in range(6):
        y = rng.integers(0, 50, (n_seq, L)).astype(np.int32)
        frac = rng.random((n_seq, 1)) ** 2                         # from nearly finished to fully masked
        y[rng.random((n_seq, L)) < frac] = MASK
        if n_seq > 1:
            y[0] = 3                                               # a finished sequence
        first_block_done = rng.random(n_seq) < 0.5                 # block order: earlier blocks resolved
        y[first_block_done, :block] = 7
        for n_sparse in (0, 1, 5, block, 10 * block):
            compare(ctx, y, block, n_sparse)


def test_all_masked_all_done_and_single_mask(ctx):
    y = np.full((4, 128), MASK, np.int32)
    compare(ctx, y, 32, 0)
    compare(ctx, y, 32, 32)                                        # |M_active| = 32 <= 32: two blocks
    y[:] = 1
    compare(ctx, y, 32, 5)                                         # nothing left: M = 0
    y[2, 127] = MASK                                               # one mask in the last block
    compare(ctx, y, 32, 5)
    y[1, 31] = MASK                                                # one mask at the end of block 0: reveals block 1, all committed
    compare(ctx, y, 32, 5)


def test_argument_errors(ctx):
    y = torch.full((2, 64), MASK, dtype=torch.int32, device=dev())
    out = ctx.working_set(y, 16, 0, MASK)
    small = dict(out, row_pos=out["row_pos"][:10])
    with pytest.raises(binding.PvfError) as e:
        ctx.working_set(y, 16, 0, MASK, out=small)                 # capacity below n_seq * 2 * block
    assert e.value.code == binding.PVF_ERR_INVALID
    with pytest.raises(binding.PvfError):
        ctx.working_set(y, 0, 0, MASK)
    torch.cuda.synchronize()
    assert ctx.last_status() == 0
