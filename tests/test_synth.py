"""The input generator: determinism, order independence, shapes and value ranges (CPU only)."""
import numpy as np

from paper_2601_12247_b200 import synth


def test_bf16_round_trip_and_rounding():
    x = np.array([0.0, 1.0, -2.5, 0.02, 1.00390625, 1.01171875, 3.0e38], np.float32)
    b = synth.f32_to_bf16_bits(x)
    back = synth.bf16_bits_to_f32(b)
    assert back[0] == 0.0 and back[1] == 1.0 and back[2] == -2.5
    assert back[4] == 1.0                       # tie (1 + 2^-8) rounds to even
    assert back[5] == np.float32(1.015625)      # 1 + 3*2^-8 is a tie too: rounds up to the even 1 + 2^-6
    assert np.all(np.abs(back[:6] - x[:6]) <= np.abs(x[:6]) * 2.0 ** -8)
    assert np.array_equal(synth.f32_to_bf16_bits(back), b)


def test_values_depend_only_on_seed_tag_indices():
    a = synth.make_w(5, 3000, 32, workers=1)
    b = synth.make_w(5, 3000, 32, workers=4)
    assert np.array_equal(a, b)
    assert np.array_equal(synth.make_w(5, 1024, 32), a[:1024])
    assert not np.array_equal(synth.make_w(6, 1024, 32), a[:1024])
    s1, s2 = synth.config0(), synth.config0()
    assert np.array_equal(s1.h_bits, s2.h_bits) and np.array_equal(s1.plan_ids, s2.plan_ids)


def test_config_shapes():
    s = synth.config0()
    assert (s.vocab, s.hidden, s.n_rows, s.n_seq) == (4096, 256, 64, 1)
    assert s.active.sum() == 32 and len(s.plan_ids) == 256 and len(set(s.plan_ids.tolist())) == 256
    assert s.params["budget"] == 4 and s.params["tau_high"] == 0.9
    w = synth.make_w(1, 512, 64)
    s2 = synth.config2(w_bits=w, vocab=512, hidden=64)
    assert s2.n_seq == 16 and s2.seg_off[-1] == s2.n_rows
    for b in range(16):
        pos = s2.row_pos[s2.seg_off[b]:s2.seg_off[b + 1]]
        assert 1 <= len(pos) <= 32 and np.all(np.diff(pos) > 0)
        assert pos.min() // 32 == pos.max() // 32           # one active block per sequence
    s3 = synth.config3(w_bits=w, vocab=512, hidden=64, n_seq=2, gen_len=16)
    assert s3.n_rows == 32 and s3.params["budget"] == 16 and s3.params["tau_high"] == 0.95
    std = synth.bf16_bits_to_f32(w).std()
    assert abs(std - 0.02) < 0.001


def test_verify_pass_layout():
    w = synth.make_w(1, 512, 64)
    s = synth.config2(w_bits=w, vocab=512, hidden=64, n_seq=3)
    rem_rows = np.arange(s.n_rows, dtype=np.int32)
    rem_off = s.seg_off.copy()
    n_drafts = np.array([2, 0, 1], np.int32)
    v = synth.make_verify_pass(s, rem_rows, rem_off, n_drafts)
    n = np.diff(s.seg_off)
    assert v.v_off.tolist() == [0, 3 * n[0], 3 * n[0], 3 * n[0] + 2 * n[2]]
    assert v.hv_bits.shape == (v.v_off[-1], 64)
    assert np.array_equal(v.target_v[:n[0]], s.target[:n[0]])          # base branch aims at the row's target
    assert np.all((v.agree_rate >= 0.3) & (v.agree_rate <= 0.9))
