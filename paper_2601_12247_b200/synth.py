"""Seeded synthetic inputs for one PVF decode step.

This module only *draws inputs*: LM-head weights, hidden states, the planning
vocabulary, the row -> (sequence, position) bookkeeping and the hidden states
of a verification pass.  It holds none of the method's arithmetic (no softmax,
no thresholds, no selection) and is the only code shared by the CPU oracle's
tests and the CUDA path's tests and benchmark.

Every value depends only on ``(seed, tag, indices)``: each draw builds its own
Philox generator whose key is ``(seed, tag)`` and whose 256-bit counter has the
indices in its three high words, so the order in which things are drawn never
matters.

The inputs stand in for LLaDA-8B-Instruct hidden states on the paper's
benchmarks (Section 5.1): they take only the shapes (vocabulary, hidden size,
generation length, block size, small verification width).  No dataset item,
prompt or model weight is used.

bf16 tensors are carried as ``numpy.uint16`` bit patterns.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Dict, Optional

import numpy as np

TAG_W = 1
TAG_PLAN = 2
TAG_TARGET = 3
TAG_AMP = 4
TAG_NOISE = 5
TAG_MASK = 6
TAG_VERIFY_AMP = 7
TAG_VERIFY_AGREE = 8
TAG_VERIFY_TOKEN = 9
TAG_VERIFY_NOISE = 10
TAG_SEQ = 11
TAG_LOOP_AMP = 12
TAG_LOOP_NOISE = 13
TAG_PLAN_PICK = 14
TAG_EXPLORE = 15

LLADA_VOCAB = 126464
LLADA_HIDDEN = 4096
# Second backbone of the paper's experiments (Dream-7B-Instruct).  The paper states neither number; these
# are the vocabulary and hidden size of the public Qwen2.5-7B family that model is built on, taken as a
# second LM-head shape (hidden size not a multiple of 256, vocabulary not a multiple of the 148 blocks).
DREAM_VOCAB = 152064
DREAM_HIDDEN = 3584


def _rng(seed: int, tag: int, i0: int = 0, i1: int = 0, i2: int = 0) -> np.random.Generator:
    """Generator for the stream named by (seed, tag, i0, i1, i2)."""
    bitgen = np.random.Philox(key=[np.uint64(seed), np.uint64(tag)],
                              counter=[0, np.uint64(i2), np.uint64(i1), np.uint64(i0)])
    return np.random.Generator(bitgen)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def make_w(seed: int, vocab: int, hidden: int, std: float = 0.02, chunk: int = 1024,
           workers: Optional[int] = None) -> np.ndarray:
    """LM-head weight W[V][D] ~ bf16(std * N(0,1)), as uint16 bit patterns.

    Row chunk c is drawn from its own stream (seed, TAG_W, c), so the result does not depend
    on the number of worker threads."""
    w = np.empty((vocab, hidden), dtype=np.uint16)

    def fill(c: int) -> None:
        r0 = c * chunk
        r1 = min(vocab, r0 + chunk)
        g = _rng(seed, TAG_W, c)
        x = g.standard_normal((r1 - r0, hidden), dtype=np.float32) * np.float32(std)
        w[r0:r1] = f32_to_bf16_bits(x)

    n_chunks = (vocab + chunk - 1) // chunk
    if workers is None:
        workers = min(16, os.cpu_count() or 1)
    if workers <= 1 or n_chunks == 1:
        for c in range(n_chunks):
            fill(c)
    else:
        with ThreadPoolExecutor(max_workers=workers) as ex:
            list(ex.map(fill, range(n_chunks)))
    return w


def make_plan_ids(seed: int, vocab: int, n_plan: int) -> np.ndarray:
    """Planning-token vocabulary: n_plan distinct ids, sorted ascending (int32)."""
    perm = _rng(seed, TAG_PLAN).permutation(vocab)
    return np.sort(perm[:n_plan]).astype(np.int32)


def make_hidden_rows(w_bits: np.ndarray, targets: np.ndarray, amps: np.ndarray,
                     seed: int, tag: int, keys: np.ndarray, noise_std: float = 0.05) -> np.ndarray:
    """h = bf16( a * W[t] / ||W[t]||_2 + noise_std * N(0, I_D) ), one row per (target, amp, key).

    ``keys`` is an int array [n, 3]: the three counter indices of each row's noise stream.
    """
    n = len(targets)
    hidden = w_bits.shape[1]
    out = np.empty((n, hidden), dtype=np.uint16)
    for r in range(n):
        wt = bf16_bits_to_f32(w_bits[int(targets[r])]).astype(np.float64)
        nrm = np.sqrt(np.sum(wt * wt))
        g = _rng(seed, tag, int(keys[r, 0]), int(keys[r, 1]), int(keys[r, 2]))
        noise = g.standard_normal(hidden, dtype=np.float32).astype(np.float64) * noise_std
        out[r] = f32_to_bf16_bits((float(amps[r]) * wt / nrm + noise).astype(np.float32))
    return out


@dataclass
class StepInputs:
    """Inputs of one decode step (draft pass)."""
    name: str
    seed: int
    vocab: int
    hidden: int
    n_seq: int
    gen_len: int            # L
    block: int              # S, block size in tokens
    w_bits: np.ndarray      # [V][D] uint16
    h_bits: np.ndarray      # [M][D] uint16
    plan_ids: np.ndarray    # sorted int32
    seg_off: np.ndarray     # [n_seq+1] int32, rows of sequence b are seg_off[b]..seg_off[b+1]-1
    row_pos: np.ndarray     # [M] int32 canvas position of each row (ascending inside a sequence)
    active: np.ndarray      # [M] uint8, position belongs to the working block B_t
    target: np.ndarray      # [M] int32 generator's target token per row
    amp: np.ndarray         # [M] float64 generator's amplitude per row
    params: Dict[str, float] = field(default_factory=dict)

    @property
    def n_rows(self) -> int:
        return int(self.h_bits.shape[0])


# Default thresholds where the configs are silent: planning band and AR bound of the
# paper's Table 5 (GSM8K / MMLU-Pro rows).
DEFAULT_BAND = dict(tau_plan_lo=0.2, tau_plan_hi=0.65, tau_ar_lo=0.1)


def _targets_and_amps(seed: int, vocab: int, plan_ids: np.ndarray, seq_of_row: np.ndarray,
                      row_pos: np.ndarray, amp_max: float, q_plan: float):
    """Per (sequence, position): target token uniform on the vocabulary (with probability
    q_plan drawn from the planning ids instead) and amplitude ~ U(0, amp_max)."""
    n = len(row_pos)
    target = np.empty(n, dtype=np.int32)
    amp = np.empty(n, dtype=np.float64)
    for r in range(n):
        b, i = int(seq_of_row[r]), int(row_pos[r])
        g = _rng(seed, TAG_TARGET, b, i)
        t = int(g.integers(0, vocab))
        if q_plan > 0.0:
            gp = _rng(seed, TAG_PLAN_PICK, b, i)
            if gp.random() < q_plan:
                t = int(plan_ids[int(gp.integers(0, len(plan_ids)))])
        target[r] = t
        amp[r] = _rng(seed, TAG_AMP, b, i).random() * amp_max
    return target, amp


def _stress_amp_max(vocab: int, hidden: int) -> float:
    # puts confidence 0.5 mid-range: the target logit a*||W[t]|| (||W[t]|| ~ 0.02 sqrt(D))
    # reaches ln(V) at half of this amplitude
    return 2.0 * np.log(vocab) / (0.02 * np.sqrt(hidden))


def build_step(name: str, seed: int, vocab: int, hidden: int, n_plan: int, seg_rows,
               gen_len: int, block: int, params: Dict[str, float], stress: bool = False,
               w_bits: Optional[np.ndarray] = None, amp_max: float = 40.0) -> StepInputs:
    """Assemble a step from per-sequence row lists.

    ``seg_rows`` is a list (one entry per sequence) of (positions, active_flags) arrays,
    positions ascending.
    """
    if w_bits is None:
        w_bits = make_w(seed, vocab, hidden)
    plan_ids = make_plan_ids(seed, vocab, n_plan)
    seg_off = np.zeros(len(seg_rows) + 1, dtype=np.int32)
    pos_l, act_l, seq_l = [], [], []
    for b, (pos, act) in enumerate(seg_rows):
        seg_off[b + 1] = seg_off[b] + len(pos)
        pos_l.append(np.asarray(pos, dtype=np.int32))
        act_l.append(np.asarray(act, dtype=np.uint8))
        seq_l.append(np.full(len(pos), b, dtype=np.int32))
    row_pos = np.concatenate(pos_l) if pos_l else np.zeros(0, np.int32)
    active = np.concatenate(act_l) if act_l else np.zeros(0, np.uint8)
    seq_of_row = np.concatenate(seq_l) if seq_l else np.zeros(0, np.int32)
    if stress:
        amp_max = _stress_amp_max(vocab, hidden)
    target, amp = _targets_and_amps(seed, vocab, plan_ids, seq_of_row, row_pos, amp_max,
                                    0.5 if stress else 0.0)
    keys = np.stack([seq_of_row, row_pos, np.zeros_like(row_pos)], axis=1) if len(row_pos) else np.zeros((0, 3), np.int64)
    h_bits = make_hidden_rows(w_bits, target, amp, seed, TAG_NOISE, keys)
    p = dict(DEFAULT_BAND)
    p.update(params)
    return StepInputs(name=name + ("-stress" if stress else ""), seed=seed, vocab=vocab, hidden=hidden,
                      n_seq=len(seg_rows), gen_len=gen_len, block=block, w_bits=w_bits, h_bits=h_bits,
                      plan_ids=plan_ids, seg_off=seg_off, row_pos=row_pos, active=active,
                      target=target, amp=amp, params=p)


def config0(stress: bool = False, vocab: int = 4096, hidden: int = 256) -> StepInputs:
    """Tiny step: one sequence, 64 masked positions, the first 32-position block active."""
    pos = np.arange(64)
    act = (pos < 32).astype(np.uint8)
    return build_step("cfg0-tiny", 1000, vocab, hidden, 256, [(pos, act)], 64, 32,
                      dict(tau_high=0.9, budget=4), stress)


def config1(variant: str = "a", stress: bool = False, w_bits: Optional[np.ndarray] = None,
            vocab: int = LLADA_VOCAB, hidden: int = LLADA_HIDDEN) -> StepInputs:
    """LLaDA-8B-shaped single step, one sequence of L=256, block 0 (32 positions) fully masked
    and active.  Variant "a" scores the 32 active rows, "b" all 256 masked rows."""
    n = 32 if variant == "a" else 256
    pos = np.arange(n)
    act = (pos < 32).astype(np.uint8)
    return build_step("cfg1" + variant, 1001, vocab, hidden, 2048, [(pos, act)], 256, 32,
                      dict(tau_high=0.9, budget=4), stress, w_bits)


def config2(stress: bool = False, w_bits: Optional[np.ndarray] = None,
            vocab: int = LLADA_VOCAB, hidden: int = LLADA_HIDDEN, n_seq: int = 16) -> StepInputs:
    """Batched decode step: per sequence a uniformly drawn active block whose masked
    fraction is U(0.1, 1); rows are the masked positions of the active block."""
    seed, gen_len, block = 1002, 256, 32
    seg = []
    for b in range(n_seq):
        g = _rng(seed, TAG_MASK, b)
        blk = int(g.integers(0, gen_len // block))
        phi = 0.1 + 0.9 * g.random()
        n = max(1, int(round(block * phi)))
        pos = np.sort(g.permutation(block)[:n]) + blk * block
        seg.append((pos, np.ones(n, np.uint8)))
    return build_step("cfg2-batched", seed, vocab, hidden, 2048, seg, gen_len, block,
                      dict(tau_high=0.9, budget=8), stress, w_bits)


def config3(stress: bool = False, w_bits: Optional[np.ndarray] = None,
            vocab: int = LLADA_VOCAB, hidden: int = LLADA_HIDDEN, n_seq: int = 64,
            gen_len: int = 512) -> StepInputs:
    """Large-batch step: every position of every sequence masked, one block of gen_len."""
    pos = np.arange(gen_len)
    seg = [(pos, np.ones(gen_len, np.uint8)) for _ in range(n_seq)]
    return build_step("cfg3-large", 1003, vocab, hidden, 4096, seg, gen_len, gen_len,
                      dict(tau_high=0.95, budget=16), stress, w_bits)


@dataclass
class VerifyInputs:
    """Hidden states of the verification pass, rows laid out [b][c][r]:
    row index = v_off[b] + c * nR_b + r, c = 0 the base branch, c = j draft j,
    r indexing the sequence's remaining (active, not base-committed) rows."""
    hv_bits: np.ndarray     # [Mv][D] uint16
    v_off: np.ndarray       # [n_seq+1] int32
    target_v: np.ndarray    # [Mv] int32
    agree_rate: np.ndarray  # [n_seq] float64


def make_verify_pass(step: StepInputs, rem_rows: np.ndarray, rem_off: np.ndarray,
                     n_drafts: np.ndarray, amp_boost: float = 15.0) -> VerifyInputs:
    """Draw the verification pass for the given remaining rows and per-sequence draft counts.

    Base branch rows aim at the row's own target with amplitude a + U(0, amp_boost).  Rows of
    branch c >= 1 aim at the same target with probability r_b (per sequence, U(0.3, 0.9)) and
    at another uniformly drawn token otherwise.  Agreement is thus defined on the targets.
    """
    n_seq = step.n_seq
    seed = step.seed
    v_off = np.zeros(n_seq + 1, dtype=np.int32)
    tg, am, keys = [], [], []
    agree = np.zeros(n_seq, dtype=np.float64)
    for b in range(n_seq):
        rows = rem_rows[rem_off[b]:rem_off[b + 1]]
        n_r = len(rows)
        k_t = int(n_drafts[b])
        n_br = (1 + k_t) if k_t > 0 else 0
        v_off[b + 1] = v_off[b] + n_br * n_r
        agree[b] = 0.3 + 0.6 * _rng(seed, TAG_SEQ, b).random()
        for c in range(n_br):
            for m in rows:
                i = int(step.row_pos[m])
                a = step.amp[m] + amp_boost * _rng(seed, TAG_VERIFY_AMP, b, i).random()
                t = int(step.target[m])
                if c >= 1:
                    g = _rng(seed, TAG_VERIFY_AGREE, b, i, c)
                    if g.random() >= agree[b]:
                        t2 = int(_rng(seed, TAG_VERIFY_TOKEN, b, i, c).integers(0, step.vocab - 1))
                        t = t2 if t2 < t else t2 + 1      # uniformly among the other tokens
                tg.append(t)
                am.append(a)
                keys.append((b, i, c))
    tg = np.asarray(tg, dtype=np.int32)
    am = np.asarray(am, dtype=np.float64)
    keys = np.asarray(keys, dtype=np.int64).reshape(-1, 3)
    hv = make_hidden_rows(step.w_bits, tg, am, seed, TAG_VERIFY_NOISE, keys)
    return VerifyInputs(hv_bits=hv, v_off=v_off, target_v=tg, agree_rate=agree)


def loop_targets(seed: int, vocab: int, n_seq: int, gen_len: int, plan_ids: Optional[np.ndarray] = None,
                 q_plan: float = 0.0, avoid: Optional[int] = None) -> np.ndarray:
    """Target token of every (sequence, position) of the decode loop; fixed across steps.  A target
    equal to ``avoid`` (the mask id: committing it would leave the position masked for ever) is moved
    to the next id."""
    t = np.empty((n_seq, gen_len), dtype=np.int32)
    for b in range(n_seq):
        for i in range(gen_len):
            v = int(_rng(seed, TAG_TARGET, b, i).integers(0, vocab))
            if q_plan > 0.0 and plan_ids is not None:
                gp = _rng(seed, TAG_PLAN_PICK, b, i)
                if gp.random() < q_plan:
                    v = int(plan_ids[int(gp.integers(0, len(plan_ids)))])
            if avoid is not None and v == avoid:
                v = (v + 1) % vocab
            t[b, i] = v
    return t


def loop_hidden(w_bits: np.ndarray, targets: np.ndarray, seed: int, step_no: int, branch: int,
                seq_ids: np.ndarray, positions: np.ndarray, committed_frac: np.ndarray,
                amp_max: float = 40.0, row_targets: Optional[np.ndarray] = None) -> np.ndarray:
    """Hidden states re-drawn at a loop step: a = amp_max * (f_b + (1 - f_b) * u) with
    u ~ U(0,1) from (seed, step, b, i) and f_b the committed fraction of sequence b at the
    start of the step.  ``branch`` separates the noise of the verification branches."""
    n = len(positions)
    tg = np.empty(n, dtype=np.int32)
    am = np.empty(n, dtype=np.float64)
    keys = np.empty((n, 3), dtype=np.int64)
    for r in range(n):
        b, i = int(seq_ids[r]), int(positions[r])
        u = _rng(seed, TAG_LOOP_AMP, step_no, b, i).random()
        f = float(committed_frac[b])
        am[r] = amp_max * (f + (1.0 - f) * u)
        tg[r] = targets[b, i] if row_targets is None else row_targets[r]
        keys[r] = (step_no * 64 + branch, b, i)
    return make_hidden_rows(w_bits, tg, am, seed, TAG_LOOP_NOISE, keys)


def loop_verify_hidden(w_bits: np.ndarray, targets: np.ndarray, seed: int, step_no: int,
                       seq_ids: np.ndarray, positions: np.ndarray, branches: np.ndarray,
                       committed_frac: np.ndarray, amp_max: float = 40.0,
                       amp_boost: float = 15.0) -> np.ndarray:
    """Hidden states of a loop step's verification pass, one row per (sequence, position, branch).

    Amplitude: the draft pass's a (same (seed, step, b, i) stream) plus U(0, amp_boost).  Branch 0
    aims at the position's target; branch c >= 1 keeps it with the sequence's agreement rate
    r_b ~ U(0.3, 0.9) and otherwise aims at another uniformly drawn token."""
    n = len(positions)
    vocab = w_bits.shape[0]
    tg = np.empty(n, dtype=np.int32)
    am = np.empty(n, dtype=np.float64)
    keys = np.empty((n, 3), dtype=np.int64)
    for r in range(n):
        b, i, c = int(seq_ids[r]), int(positions[r]), int(branches[r])
        u = _rng(seed, TAG_LOOP_AMP, step_no, b, i).random()
        f = float(committed_frac[b])
        am[r] = amp_max * (f + (1.0 - f) * u) + amp_boost * _rng(seed, TAG_VERIFY_AMP, step_no, b, i).random()
        t = int(targets[b, i])
        if c >= 1:
            r_b = 0.3 + 0.6 * _rng(seed, TAG_SEQ, b).random()
            if _rng(seed, TAG_VERIFY_AGREE, step_no * 64 + c, b, i).random() >= r_b:
                t2 = int(_rng(seed, TAG_VERIFY_TOKEN, step_no * 64 + c, b, i).integers(0, vocab - 1))
                t = t2 if t2 < t else t2 + 1
        tg[r] = t
        keys[r] = (step_no * 64 + 1 + c, b, i)
    return make_hidden_rows(w_bits, tg, am, seed, TAG_LOOP_NOISE, keys)


def loop_uniforms(seed: int, step_no: int, n_seq: int) -> np.ndarray:
    """One uniform number in [0, 1) per sequence for a loop step (float32): the random draws that the
    exploration variants take as an input."""
    return np.array([_rng(seed, TAG_EXPLORE, step_no, b).random() for b in range(n_seq)], dtype=np.float32)
