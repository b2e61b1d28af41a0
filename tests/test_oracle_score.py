"""Pins of the fp64 scoring oracle against what the mathematics fixes (CPU only)."""
import math

import numpy as np
import pytest
from scipy.special import log_softmax

from oracle import score as oscore
from paper_2601_12247_b200 import synth


def bits(x):
    return synth.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def as_f64(b):
    return synth.bf16_bits_to_f32(b).astype(np.float64)


def test_uniform_row_closed_form():
    # h = 0  =>  every logit is 0  =>  p = 1/V, H = ln V, argmax = lowest id
    V, D = 300, 24
    w = synth.make_w(7, V, D)
    o = oscore.score(w, bits(np.zeros((2, D))))
    assert o["tok"].tolist() == [0, 0]
    assert np.allclose(o["conf"], 1.0 / V, rtol=0, atol=1e-15)
    assert np.allclose(o["ent"], math.log(V), rtol=0, atol=1e-12)
    assert np.all(o["gap"] == 0.0)


@pytest.mark.parametrize("t", [0, 5, 63])
def test_identity_weights_closed_form(t):
    # W = c I (V = D), h = a e_t  =>  logits a c at t and 0 elsewhere
    V = 64
    c, a = 0.5, 4.0                      # exactly representable in bf16
    w = bits(c * np.eye(V))
    h = np.zeros((1, V)); h[0, t] = a
    o = oscore.score(w, bits(h))
    Z = math.exp(a * c) + V - 1
    p = math.exp(a * c) / Z
    H = math.log(Z) - p * a * c
    assert o["tok"][0] == t
    assert abs(o["conf"][0] - p) < 1e-14
    assert abs(o["ent"][0] - H) < 1e-12
    assert abs(o["gap"][0] - a * c) < 1e-14


def test_tie_goes_to_lowest_id():
    V, D = 16, 4
    w = np.zeros((V, D)); w[3, 0] = 1.0; w[9, 0] = 1.0; w[12, 0] = 0.5
    h = np.zeros((1, D)); h[0, 0] = 2.0
    o = oscore.score(bits(w), bits(h))
    assert o["tok"][0] == 3 and o["gap"][0] == 0.0
    # two equal maxima e^2, one e^1 and 13 zeros
    Z = 2 * math.exp(2) + math.exp(1) + 13
    assert abs(o["conf"][0] - math.exp(2) / Z) < 1e-14


def test_logits_are_h_dot_w_rows_not_transposed():
    # V != D, hand-computed entries: x[m][v] = sum_k H[m][k] W[v][k]
    V, D, M = 7, 3, 2
    w = np.arange(V * D, dtype=np.float64).reshape(V, D) - 4.0      # small integers: exact in bf16
    h = np.array([[1.0, -2.0, 0.5], [0.0, 3.0, -1.0]])
    o = oscore.score(bits(w), bits(h), want_logits=True)
    for m in range(M):
        for v in range(V):
            want = sum(h[m][k] * w[v][k] for k in range(D))
            assert o["logits"][m, v] == want
    assert o["tok"].tolist() == [int(np.argmax(h[m] @ w.T)) for m in range(M)]


def test_matches_scipy_log_softmax_on_small_shapes():
    for seed, (V, D, M) in enumerate([(50, 8, 5), (257, 33, 4), (1000, 64, 3)]):
        st = synth.build_step("t", 50 + seed, V, D, 8, [(np.arange(M), np.ones(M, np.uint8))], M, M,
                              dict(tau_high=0.9, budget=2), amp_max=25.0)
        o = oscore.score(st.w_bits, st.h_bits, st.plan_ids, want_logits=True)
        x = as_f64(st.h_bits) @ as_f64(st.w_bits).T
        assert np.allclose(o["logits"], x, rtol=0, atol=1e-12)
        ls = log_softmax(x, axis=1)
        assert np.array_equal(o["tok"], np.argmax(x, axis=1))
        assert np.allclose(o["conf"], np.exp(ls.max(axis=1)), rtol=1e-12, atol=0)
        assert np.allclose(o["ent"], -(np.exp(ls) * ls).sum(axis=1), rtol=0, atol=1e-11)
        srt = np.sort(x, axis=1)
        assert np.allclose(o["gap"], srt[:, -1] - srt[:, -2], rtol=0, atol=1e-12)
        member = np.isin(o["tok"], st.plan_ids).astype(np.uint8)
        assert np.array_equal(o["in_plan"], member)


def test_brute_force_argmax_and_probabilities_tiny_vocab():
    V, D, M = 37, 5, 6
    st = synth.build_step("t", 91, V, D, 4, [(np.arange(M), np.ones(M, np.uint8))], M, M,
                          dict(tau_high=0.9, budget=2), amp_max=60.0)
    o = oscore.score(st.w_bits, st.h_bits, st.plan_ids)
    W, H = as_f64(st.w_bits), as_f64(st.h_bits)
    for m in range(M):
        x = [sum(H[m][k] * W[v][k] for k in range(D)) for v in range(V)]
        best = 0
        for v in range(V):
            if x[v] > x[best]:
                best = v
        Z = sum(math.exp(xv - x[best]) for xv in x)
        q = [math.exp(xv - x[best]) / Z for xv in x]
        assert o["tok"][m] == best
        assert abs(o["conf"][m] - max(q)) < 1e-14
        assert abs(o["ent"][m] + sum(qv * math.log(qv) for qv in q if qv > 0)) < 1e-12


def test_shift_invariance_constant_column():
    # a column of ones in W makes h[0] a common shift of all logits: p, H, y^ must not move
    V, D = 200, 16
    w = as_f64(synth.make_w(3, V, D)); w[:, 0] = 1.0
    g = np.random.default_rng(3)
    h = g.standard_normal((1, D)) * 4.0
    outs = []
    for shift in (0.0, 8.0, -32.0):
        h2 = h.copy(); h2[0, 0] = shift
        outs.append(oscore.score(bits(w), bits(h2)))
    for o in outs[1:]:
        assert o["tok"][0] == outs[0]["tok"][0]
        assert abs(o["conf"][0] - outs[0]["conf"][0]) < 1e-12
        assert abs(o["ent"][0] - outs[0]["ent"][0]) < 1e-11


def test_row_permutation_of_w_permutes_tokens_only():
    V, D, M = 128, 12, 8
    st = synth.build_step("t", 17, V, D, 8, [(np.arange(M), np.ones(M, np.uint8))], M, M,
                          dict(tau_high=0.9, budget=2), amp_max=30.0)
    perm = np.random.default_rng(1).permutation(V)          # new row r holds old row perm[r]
    o1 = oscore.score(st.w_bits, st.h_bits)
    o2 = oscore.score(st.w_bits[perm], st.h_bits)
    assert np.array_equal(perm[o2["tok"]], o1["tok"])
    assert np.allclose(o1["conf"], o2["conf"], rtol=1e-13, atol=0)
    assert np.allclose(o1["ent"], o2["ent"], rtol=0, atol=1e-11)


def test_bounds_hold_on_every_row():
    st = synth.config0()
    o = oscore.score(st.w_bits, st.h_bits, st.plan_ids)
    V = st.vocab
    p, H = o["conf"], o["ent"]
    assert np.all(p >= 1.0 / V - 1e-15) and np.all(p <= 1.0)
    assert np.all(H >= -1e-12) and np.all(H <= math.log(V) + 1e-12)
    assert np.all(-np.log(p) <= H + 1e-12)                  # min-entropy <= Shannon entropy
    hb = -(p * np.log(p) + np.where(p < 1, (1 - p) * np.log1p(-np.minimum(p, 1 - 1e-300)), 0.0))
    assert np.all(H >= hb - 1e-10)                          # grouping: H >= h_b(p)
    assert np.all(H <= hb + (1 - p) * math.log(V - 1) + 1e-10)


def test_streaming_recurrence_equals_two_pass_definition():
    # The online form (running max m, s = sum e^{x-m}, t = sum (x-m) e^{x-m}; on a new max m'
    # s <- s e^{m-m'}, t <- (t + (m-m') s) e^{m-m'};  p = 1/s,  H = ln s - t/s) must reproduce the
    # oracle's two-pass numbers, in any chunking and when partial states are merged.
    st = synth.config0()
    o = oscore.score(st.w_bits, st.h_bits[:6], want_logits=True)

    def stream(x):
        m, s, t, arg = -math.inf, 0.0, 0.0, -1
        for v, xv in enumerate(x):
            if xv > m:
                if s > 0.0:
                    c = math.exp(m - xv)
                    t = (t + (m - xv) * s) * c
                    s = s * c
                m, arg = xv, v
            e = math.exp(xv - m)
            s += e
            t += (xv - m) * e
        return m, arg, s, t

    def merge(a, b):                                         # a covers the lower ids
        (ma, ia, sa, ta), (mb, ib, sb, tb) = a, b
        m = max(ma, mb)
        arg = ia if ma >= mb else ib
        ca, cb = math.exp(ma - m), math.exp(mb - m)
        return m, arg, sa * ca + sb * cb, (ta + (ma - m) * sa) * ca + (tb + (mb - m) * sb) * cb

    for r in range(6):
        x = o["logits"][r]
        for parts in (1, 3, 148):
            edges = np.linspace(0, len(x), parts + 1).astype(int)
            acc = None
            for lo, hi in zip(edges[:-1], edges[1:]):
                if hi == lo:
                    continue
                m, arg, s, t = stream(x[lo:hi])
                piece = (m, arg + lo, s, t)
                acc = piece if acc is None else merge(acc, piece)
            m, arg, s, t = acc
            assert arg == o["tok"][r]
            assert abs(1.0 / s - o["conf"][r]) < 1e-12
            assert abs(math.log(s) - t / s - o["ent"][r]) < 1e-11


def test_row_stats_entry_point_matches_score():
    st = synth.config0()
    o = oscore.score(st.w_bits, st.h_bits[:3], want_logits=True)
    for r in range(3):
        tok, conf, ent, gap = oscore.row_stats(o["logits"][r])
        assert (tok, conf, ent, gap) == (o["tok"][r], o["conf"][r], o["ent"][r], o["gap"][r])
