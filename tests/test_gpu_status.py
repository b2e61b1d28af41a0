"""The device status word: what a kernel leaves there when one of its bounded waits runs out, and how
pvf_last_status reads it.  The expiry is exercised in its harmless form only: a self-test kernel of the library
waits, with the projection kernels' own bounded wait and a limit of a millisecond, on a barrier that nothing
arrives on -- no copy, no tensor-core work and no tensor memory is in flight, the kernel returns by itself."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import score as oscore
from paper_2601_12247_b200 import binding, synth
from gpu_util import check_score, dev, make_ctx, to_np, upload_bits

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_sets_the_status_word_and_the_context_stays_usable():
    st = synth.config0(stress=True)
    ctx = make_ctx(st.w_bits, st.plan_ids, 256)
    lib = binding.load()
    lib.pvf_selftest_wait_expiry.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_void_p]
    lib.pvf_selftest_wait_expiry.restype = ctypes.c_int
    h = upload_bits(st.h_bits)
    want = oscore.score(st.w_bits, st.h_bits, st.plan_ids)
    check_score(to_np(ctx.score(h)), want, st.vocab, st.plan_ids)
    assert ctx.last_status() == 0
    gave_up = torch.zeros(1, dtype=torch.int32, device=dev())
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert lib.pvf_selftest_wait_expiry(ctx.handle, 1_000_000, ctypes.c_void_p(gave_up.data_ptr()), stream) == binding.PVF_OK
    torch.cuda.synchronize()                                   # the kernel ended by itself
    assert int(gave_up.item()) == 2                            # the wait that ran out, and the one that saw the abort flag
    assert ctx.last_status() == binding.PVF_ERR_TIMEOUT
    assert "wait" in binding.strerror(binding.PVF_ERR_TIMEOUT)
    assert ctx.last_status() == 0                              # reading it cleared it
    for rows in (64, 20, 40):                                  # and the context scores correctly afterwards
        got = to_np(ctx.score(upload_bits(st.h_bits[:rows])))
        check_score(got, {k: v[:rows] for k, v in want.items()}, st.vocab, st.plan_ids)
    assert ctx.last_status() == 0
    # limits outside (0, 0.1 s] are refused on the host, nothing is launched
    assert lib.pvf_selftest_wait_expiry(ctx.handle, 0, ctypes.c_void_p(gave_up.data_ptr()), stream) == binding.PVF_ERR_INVALID
    assert lib.pvf_selftest_wait_expiry(ctx.handle, 10**9, ctypes.c_void_p(gave_up.data_ptr()), stream) == binding.PVF_ERR_INVALID
    ctx.close()


def test_last_status_waits_for_non_blocking_streams():
    # pvf_last_status synchronises the whole device: a score call on a non-blocking side stream (which the legacy
    # default stream does not wait for) has finished, and its status is the one read, without any other synchronisation
    V, D = 70000, 1024
    w_bits = synth.make_w(9, V, D)
    pos = np.arange(512)
    st = synth.build_step("status", 9, V, D, 64, [(pos, np.ones(512, np.uint8))], 512, 512, dict(tau_high=0.9, budget=4),
                          w_bits=w_bits)
    ctx = make_ctx(w_bits, st.plan_ids, 512)
    h = upload_bits(st.h_bits)
    out = dict(tok=torch.full((512,), -7, dtype=torch.int32, device=dev()), conf=torch.zeros(512, device=dev()),
               ent=torch.zeros(512, device=dev()), in_plan=torch.zeros(512, dtype=torch.uint8, device=dev()))
    torch.cuda.synchronize()
    side = torch.cuda.Stream(device=dev())                     # torch's side streams are non-blocking
    with torch.cuda.stream(side):
        for _ in range(20):
            ctx.score(h, out)
        assert ctx.last_status() == 0                          # returns only after the 20 launches have run
        assert side.query()                                    # nothing left in flight on the side stream
    got = to_np(out)
    sample = np.array([0, 255, 511])
    check_score(got, oscore.score(w_bits, st.h_bits[sample], st.plan_ids), V, st.plan_ids, rows=sample)
    ctx.close()
