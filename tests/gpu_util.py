"""Shared helpers of the GPU parity tests: contexts, uploads and the comparison rules."""
import math

import numpy as np
import torch

from paper_2601_12247_b200 import binding, synth

TOL = 1e-3          # absolute tolerance on confidence and entropy
NEAR_TIE = 1e-3     # rows whose oracle top-2 logit gap is below this are exempt from token equality
FRAGILE = 1e-4      # distance of an oracle confidence to a threshold below which a decision may flip


def dev():
    return torch.device("cuda:0")


def upload_bits(bits):
    return binding.bf16_from_bits(bits, dev())


def t_i32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev())


def t_u8(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint8)).to(dev())


def t_f32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dev())


def to_np(d):
    return {k: v.detach().cpu().numpy() for k, v in d.items()}


def make_ctx(w_bits, plan_ids, max_rows, max_seqs=64, max_budget=16):
    w = upload_bits(w_bits)
    return binding.Context(w, plan_ids, max_rows, max_seqs, max_budget)


def params_of(step, flags=0, **over):
    p = dict(step.params)
    p.update(over)
    return binding.make_params(p["tau_high"], p["tau_plan_lo"], p["tau_plan_hi"], p["tau_ar_lo"], p["budget"], flags)


def check_score(got, want, vocab, plan_ids=None, rows=None):
    """got: numpy dict of GPU outputs; want: oracle dict on the same rows (or on `rows` of them).
    Returns the number of near-tie rows that were exempt from token equality."""
    g = {k: (v if rows is None else v[rows]) for k, v in got.items()}
    assert np.all(np.isfinite(g["conf"])) and np.all(np.isfinite(g["ent"]))
    assert np.max(np.abs(g["conf"].astype(np.float64) - want["conf"])) <= TOL
    assert np.max(np.abs(g["ent"].astype(np.float64) - want["ent"])) <= TOL
    near = want["gap"] < NEAR_TIE
    assert np.array_equal(g["tok"][~near], want["tok"][~near])
    if plan_ids is not None:
        assert np.array_equal(g["in_plan"][~near], want["in_plan"][~near])
        assert np.array_equal(g["in_plan"], np.isin(g["tok"], plan_ids).astype(np.uint8))
    return int(near.sum())


def check_score_properties(got, vocab, plan_ids):
    c, e = got["conf"].astype(np.float64), got["ent"].astype(np.float64)
    assert np.all((got["tok"] >= 0) & (got["tok"] < vocab))
    assert np.all(c >= 1.0 / vocab - 1e-6) and np.all(c <= 1.0 + 1e-6)
    assert np.all(e >= -TOL) and np.all(e <= math.log(vocab) + TOL)
    assert np.all(-np.log(np.minimum(c, 1.0)) <= e + TOL)
    assert np.array_equal(got["in_plan"], np.isin(got["tok"], plan_ids).astype(np.uint8))
