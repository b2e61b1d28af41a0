"""Synthetic PVF decode loop on the GPU (Algorithm 1), driving the C interface step by step.

The transformer is replaced by the seeded generator of ``synth``: at every step the hidden states of
the scored rows are re-drawn on the host from (seed, step, sequence, position), with an amplitude that
grows with the sequence's committed fraction, and uploaded.  Decoding is semi-autoregressive: the
working block of a sequence is its first block that still holds a mask; the scored rows are that block's
masked positions, widened by the next block under early cross-block revelation (``n_sparse``); the rows
come from pvf_working_set on the device.  One step = pvf_draft_step (draft-pass score, base commit and draft selection) and
pvf_verify_step (verification-pass score, verify); it counts as one batched forward.  ``budget = 0`` gives confidence-threshold decoding.

This is a harness around the library (the hot path is the library's kernels); it reports steps,
tokens per forward, scored rows and the kernel time per step measured with CUDA events.

    python -m paper_2601_12247_b200.decode_loop [--n-seq 32] [--gen-len 256] [--block 32] [--budget 4]
"""
from __future__ import annotations

import argparse
import json
from typing import Callable, Dict, Optional

import numpy as np
import torch

from . import binding, synth


def decode(ctx: binding.Context, w_bits: np.ndarray, targets: np.ndarray, seed: int, gen_len: int, block: int,
           params: Dict, mask_id: int, max_steps: int = 100000,
           on_step: Optional[Callable[[int, Dict], None]] = None, n_sparse: int = 0, explore: str = "") -> Dict:
    """Run the loop until no masks remain.  ``params`` holds tau_high, tau_plan_lo, tau_plan_hi, tau_ar_lo
    and budget; ``n_sparse`` is the early cross-block threshold N_s (Eq. 4; 0 = strict block order).
    ``explore`` = "random" / "planning" runs the appendix's exploration loop instead (base commit plus one
    token from the closed bin [tau_plan_lo, tau_plan_hi] per step, no drafts, no verification).
    Returns y, step counts, scored rows and kernel times."""
    dev = ctx.device
    n_seq = targets.shape[0]
    K = 0 if explore else int(params["budget"])
    prm = binding.make_params(params["tau_high"], params["tau_plan_lo"], params["tau_plan_hi"], params["tau_ar_lo"],
                              K, binding.PVF_FORCE_PROGRESS)
    y_dev = torch.full((n_seq, gen_len), mask_id, dtype=torch.int32, device=dev)
    y = np.full((n_seq, gen_len), mask_id, dtype=np.int32)
    steps_per_seq = np.zeros(n_seq, dtype=np.int32)
    scored_rows, n_steps, kernel_ms = 0, 0, 0.0
    while (y == mask_id).any():
        if n_steps >= max_steps:
            raise RuntimeError("decode loop did not terminate")
        ws = ctx.working_set(y_dev, block, n_sparse, mask_id)          # rows of this step, built on the device
        seg_off = ws["seg_off"].cpu().numpy()
        n_rows = int(seg_off[-1])
        positions = ws["row_pos"][:n_rows].cpu().numpy()
        seq_ids = ws["row_seq"][:n_rows].cpu().numpy()
        frac = (y != mask_id).sum(axis=1) / float(gen_len)
        h_bits = synth.loop_hidden(w_bits, targets, seed, n_steps, 0, seq_ids, positions, frac)
        h = binding.bf16_from_bits(h_bits, dev)
        seg, pos = ws["seg_off"], ws["row_pos"][:n_rows]
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        e[0].record()
        sel = ver = scv = exp_row = None
        hv_bits = None
        if K > 0 and not explore:
            # score, then base commit and draft proposal in one launch
            d = ctx.draft_step(prm, h, seg, pos, None, y=y_dev)
            sc = {k: d[k] for k in ("tok", "conf", "ent", "in_plan")}
            cm = {k: d[k] for k in ("commit", "n_commit")}
            sel = {k: d[k] for k in ("draft_rows", "n_drafts", "route", "rem_rows", "rem_off", "v_off")}
        else:
            sc = ctx.score(h)
            cm = ctx.commit(prm, seg, pos, None, sc["tok"], sc["conf"], y=y_dev)
        if explore:
            u = torch.from_numpy(synth.loop_uniforms(seed, n_steps, n_seq)).to(dev)
            mode = binding.PVF_EXPLORE_PLANNING if explore == "planning" else binding.PVF_EXPLORE_RANDOM
            exp_row = ctx.explore_commit(prm, mode, seg, pos, None, sc["tok"], sc["conf"], sc["in_plan"], u, cm["commit"], y=y_dev)
        e[1].record()
        scored_rows += len(positions)
        if K > 0:
            # the "model forward" of the verification branches: host-side generator
            s = {k: v.cpu().numpy() for k, v in sel.items()}
            vb, vi, vc = [], [], []
            for b in range(n_seq):
                if s["n_drafts"][b] > 0:
                    rem = s["rem_rows"][s["rem_off"][b]:s["rem_off"][b + 1]]
                    for c in range(1 + int(s["n_drafts"][b])):
                        vb.append(np.full(len(rem), b, np.int32)); vi.append(positions[rem]); vc.append(np.full(len(rem), c, np.int32))
            cat = lambda l: np.concatenate(l) if l else np.zeros(0, np.int32)
            vb, vi, vc = cat(vb), cat(vi), cat(vc)
            hv_bits = synth.loop_verify_hidden(w_bits, targets, seed, n_steps, vb, vi, vc, frac)
            hv = binding.bf16_from_bits(hv_bits, dev)
            e[2].record()
            vs = ctx.verify_step(prm, hv, seg, pos, d, y=y_dev)
            scv = dict(tok=vs["tok_v"], conf=vs["conf_v"], ent=vs["ent_v"])
            ver = {k: vs[k] for k in ("accept", "choice", "final_commit")}
            e[3].record()
            scored_rows += len(vb)
        torch.cuda.synchronize()
        kernel_ms += e[0].elapsed_time(e[1]) + (e[2].elapsed_time(e[3]) if K > 0 else 0.0)
        y = y_dev.cpu().numpy()
        steps_per_seq += (np.diff(seg_off) > 0).astype(np.int32)
        if on_step is not None:
            on_step(n_steps, dict(seq_ids=seq_ids, positions=positions, seg_off=seg_off, h_bits=h_bits, hv_bits=hv_bits,
                                  score=sc, commit=cm, select=sel, score_v=scv, verify=ver, explore_row=exp_row, y=y.copy()))
        n_steps += 1
    status = ctx.last_status()
    return dict(y=y, steps=n_steps, steps_per_seq=steps_per_seq, scored_rows=scored_rows, status=status,
                tokens_per_forward=float(np.mean(gen_len / np.maximum(steps_per_seq, 1))),
                kernel_ms_per_step=kernel_ms / max(n_steps, 1), kernel_ms_total=kernel_ms)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--vocab", type=int, default=synth.LLADA_VOCAB)
    ap.add_argument("--hidden", type=int, default=synth.LLADA_HIDDEN)
    ap.add_argument("--n-seq", type=int, default=32)
    ap.add_argument("--gen-len", type=int, default=256)
    ap.add_argument("--block", type=int, default=32)
    ap.add_argument("--budget", type=int, default=4)
    ap.add_argument("--n-plan", type=int, default=2048)
    ap.add_argument("--q-plan", type=float, default=0.0, help="fraction of targets drawn from the planning ids")
    ap.add_argument("--n-sparse", type=int, default=0, help="early cross-block threshold N_s (Eq. 4)")
    ap.add_argument("--explore", action="store_true", help="also run the Random / Planning exploration loops")
    ap.add_argument("--seed", type=int, default=1004)
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    w_bits = synth.make_w(args.seed, args.vocab, args.hidden)
    plan = synth.make_plan_ids(args.seed, args.vocab, args.n_plan)
    targets = synth.loop_targets(args.seed, args.vocab, args.n_seq, args.gen_len, plan, args.q_plan, avoid=args.vocab - 128)
    ctx = binding.Context(binding.bf16_from_bits(w_bits, dev), plan, args.n_seq * args.block * (2 + args.budget),
                          args.n_seq, max(args.budget, 1))
    p = dict(tau_high=0.9, budget=args.budget, **synth.DEFAULT_BAND)
    out = {}
    for name, budget in (("pvf", args.budget), ("threshold_only", 0)):
        r = decode(ctx, w_bits, targets, args.seed, args.gen_len, args.block, dict(p, budget=budget), args.vocab - 128,
                   n_sparse=args.n_sparse)
        out[name] = dict(steps=r["steps"], mean_steps_per_sequence=float(r["steps_per_seq"].mean()),
                         tokens_per_forward=r["tokens_per_forward"], scored_rows=r["scored_rows"],
                         kernel_ms_per_step=r["kernel_ms_per_step"], status=r["status"])
    if args.explore:
        for mode in ("random", "planning"):
            r = decode(ctx, w_bits, targets, args.seed, args.gen_len, args.block, p, args.vocab - 128,
                       n_sparse=args.n_sparse, explore=mode)
            out["explore_" + mode] = dict(steps=r["steps"], mean_steps_per_sequence=float(r["steps_per_seq"].mean()),
                                          tokens_per_forward=r["tokens_per_forward"], scored_rows=r["scored_rows"],
                                          kernel_ms_per_step=r["kernel_ms_per_step"], status=r["status"])
    out["config"] = dict(vocab=args.vocab, hidden=args.hidden, n_seq=args.n_seq, gen_len=args.gen_len, block=args.block,
                         budget=args.budget, q_plan=args.q_plan, n_sparse=args.n_sparse, data="synthetic")
    print(json.dumps(out))


if __name__ == "__main__":
    main()
