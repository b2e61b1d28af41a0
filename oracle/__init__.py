"""CPU oracle for the PVF decode step -- TEST INFRASTRUCTURE, not part of the product.

A plain, slow, fp64 restatement of what the paper's step computes, written from the paper's
definitions (Sections 2-4, Algorithm 1).  Only ``tests/``, ``__graft_entry__.smoke()`` and the
``cpu_baseline`` / ``--impl reference`` legs of ``bench.py`` may import it.  It shares no code
with the CUDA library and never imports it.

  score.py   logits -> (top-1 token, confidence, entropy, top-2 gap, planning eligibility);
             thin ctypes wrapper around pvf_oracle_score.c
  step.py    base commit, planning / AR draft proposal, impact-set verification, branch choice
  loop.py    Algorithm 1 on synthetic hidden states, the threshold-only loop, and the working
             set with early cross-block revelation (Eq. 4)
  calib.py   verified information gain, per-token calibration statistics and the filtering
             rule that builds the planning-token vocabulary

Pins (tests/test_oracle_*.py): closed forms (uniform row, identity weights), invariances,
scipy's fp64 log_softmax on tiny shapes, brute-force argmax / top-k, a streaming recurrence
versus the two-pass definition, hand-built verification cases and the step's invariants;
hand-built canvases and an independent block rule for the working set; hand-computed
information-gain events, a dictionary restatement of the token statistics and the filter's
boundaries at the paper's printed thresholds; closed-bin edges and even-grid uniformity of
the exploration variants.
The paper prints no worked numeric example of a step, so parity with printed values is
unpinned; its printed hyper-parameters (Table 5, Section 5.1) are pinned as defaults.
"""
