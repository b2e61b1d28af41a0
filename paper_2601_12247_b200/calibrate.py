"""Offline construction of the planning-token vocabulary on synthetic trajectories, driving the C interface
(Appendix, "Planning Token Set Construction").

The canvas is decoded with the confidence-threshold base rule alone.  At every step the calibration candidates
(non-base masked positions of the working block whose confidence lies in the calibration band, any top-1 token)
are measured -- all of them, as in the paper, when ``budget`` is at least the block size (the default; the library
takes budgets up to 64); a smaller budget keeps the most confident ones only, which is a caller's choice that departs
from the paper: one planning branch each, scored with
entropies, checked with pvf_verify, and their events added to the per-token statistics with
pvf_calib_accumulate.  The branches are never committed.  pvf_calib_filter turns the statistics into the
vocabulary.  The transformer is replaced by the seeded generator of ``synth`` (the paper's calibration corpora
are not available here): this is a harness around the library that shows the whole path and reports its
kernel time.

    python -m paper_2601_12247_b200.calibrate [--n-seq 32] [--gen-len 256] [--block 32] [--budget min(64, block)]
"""
from __future__ import annotations

import argparse
import json
from typing import Callable, Dict, Optional

import numpy as np
import torch

from . import binding, synth


def calibrate(ctx: binding.Context, w_bits: np.ndarray, targets: np.ndarray, seed: int, gen_len: int, block: int,
              tau_high: float, cal: binding.pvf_calib_params, budget: int, mask_id: int, max_steps: int = 100000,
              on_step: Optional[Callable[[int, Dict], None]] = None) -> Dict:
    """Run the calibration trajectory until no masks remain; returns the device statistics, event and step
    counts and the kernel time.  ``cal`` supplies the calibration band."""
    dev = ctx.device
    n_seq = targets.shape[0]
    K = int(budget)
    prm = binding.make_params(tau_high, cal.tau_cal_lo, cal.tau_cal_hi, 0.0, K,
                              binding.PVF_FORCE_PROGRESS | binding.PVF_SELECT_ANY_TOKEN | binding.PVF_NO_AR_FALLBACK)
    y_dev = torch.full((n_seq, gen_len), mask_id, dtype=torch.int32, device=dev)
    y = np.full((n_seq, gen_len), mask_id, dtype=np.int32)
    stats = ctx.new_calib_stats()
    n_events, n_steps, kernel_ms = 0, 0, 0.0
    while (y == mask_id).any():
        if n_steps >= max_steps:
            raise RuntimeError("calibration loop did not terminate")
        ws = ctx.working_set(y_dev, block, 0, mask_id)
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
        sc = ctx.score(h)
        cm = ctx.commit(prm, seg, pos, None, sc["tok"], sc["conf"], y=y_dev)          # only the base set is committed
        sel = ctx.select_drafts(prm, seg, pos, None, sc["tok"], sc["conf"], None, cm["commit"])
        e[1].record()
        s = {k: v.cpu().numpy() for k, v in sel.items()}
        vb, vi, vc = [], [], []
        for b in range(n_seq):
            if s["n_drafts"][b] > 0:
                rem = s["rem_rows"][s["rem_off"][b]:s["rem_off"][b + 1]]
                for c in range(1 + int(s["n_drafts"][b])):
                    vb.append(np.full(len(rem), b, np.int32)); vi.append(positions[rem]); vc.append(np.full(len(rem), c, np.int32))
        scv = ver = vig = hv_bits = None
        if vb:
            vb, vi, vc = np.concatenate(vb), np.concatenate(vi), np.concatenate(vc)
            hv_bits = synth.loop_verify_hidden(w_bits, targets, seed, n_steps, vb, vi, vc, frac)
            hv = binding.bf16_from_bits(hv_bits, dev)
            vig = torch.zeros((n_seq, K), dtype=torch.float64, device=dev)
            e[2].record()
            scv = ctx.score(hv)
            ver = ctx.verify(prm, seg, pos, sel, sc["tok"], scv["tok"], scv["conf"], cm["commit"])   # acceptance only
            ctx.calib_accumulate(prm, sel, sc["tok"], scv["conf"], scv["ent"], ver["accept"], stats, vig)
            e[3].record()
            n_events += int(s["n_drafts"][s["route"] == 1].sum())
        torch.cuda.synchronize()
        kernel_ms += e[0].elapsed_time(e[1]) + (e[2].elapsed_time(e[3]) if scv is not None else 0.0)
        y = y_dev.cpu().numpy()
        if on_step is not None:
            on_step(n_steps, dict(seq_ids=seq_ids, positions=positions, seg_off=seg_off, h_bits=h_bits, hv_bits=hv_bits,
                                  score=sc, commit=cm, select=sel, score_v=scv, verify=ver, vig=vig, y=y.copy()))
        n_steps += 1
    return dict(stats=stats, n_events=n_events, steps=n_steps, y=y, status=ctx.last_status(),
                kernel_ms_per_step=kernel_ms / max(n_steps, 1))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--vocab", type=int, default=synth.LLADA_VOCAB)
    ap.add_argument("--hidden", type=int, default=synth.LLADA_HIDDEN)
    ap.add_argument("--n-seq", type=int, default=32)
    ap.add_argument("--gen-len", type=int, default=256)
    ap.add_argument("--block", type=int, default=32)
    ap.add_argument("--budget", type=int, default=None,
                    help="candidates measured per sequence and step; default min(64, block): every candidate of the band")
    ap.add_argument("--n-tokens", type=int, default=64, help="targets are drawn from this many token ids, so that tokens repeat")
    ap.add_argument("--n-min", type=int, default=5)
    ap.add_argument("--m-min", type=int, default=2)
    ap.add_argument("--seed", type=int, default=1006)
    args = ap.parse_args()
    if args.budget is None:
        args.budget = min(64, args.block)
    dev = torch.device("cuda:0")
    w_bits = synth.make_w(args.seed, args.vocab, args.hidden)
    pool = synth.make_plan_ids(args.seed, args.vocab, args.n_tokens)
    targets = synth.loop_targets(args.seed, args.vocab, args.n_seq, args.gen_len, pool, 1.0, avoid=args.vocab - 128)
    ctx = binding.Context(binding.bf16_from_bits(w_bits, dev), [], args.n_seq * args.block * (2 + args.budget),
                          args.n_seq, args.budget)
    cal = binding.default_calib_params()
    r = calibrate(ctx, w_bits, targets, args.seed, args.gen_len, args.block, 0.9, cal, args.budget, args.vocab - 128)
    cal.n_min, cal.m_min = args.n_min, args.m_min          # a 32-sequence sample cannot meet the paper's 50 / 20
    bitmap, n_plan = ctx.calib_filter(cal, r["stats"])
    ctx.set_plan_bitmap(bitmap)
    torch.cuda.synchronize()
    st = {k: v.cpu().numpy() for k, v in r["stats"].items()}
    print(json.dumps(dict(steps=r["steps"], events=r["n_events"], tokens_seen=int((st["n_v"] > 0).sum()),
                          accepted=int(st["sum_a"].sum()), non_vacuous=int(st["m_v"].sum()),
                          mean_vig=float(st["sum_vig_q32"].sum() / 2.0 ** 32 / max(1, st["n_v"].sum())),
                          n_plan=int(n_plan.item()), kernel_ms_per_step=r["kernel_ms_per_step"], status=r["status"],
                          config=dict(vocab=args.vocab, hidden=args.hidden, n_seq=args.n_seq, gen_len=args.gen_len,
                                      block=args.block, budget=args.budget, band=[cal.tau_cal_lo, cal.tau_cal_hi],
                                      n_min=cal.n_min, m_min=cal.m_min, rho_ver=cal.rho_ver, gamma_vig=cal.gamma_vig,
                                      data="synthetic"))))
    ctx.close()


if __name__ == "__main__":
    main()
