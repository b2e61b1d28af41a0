"""pvf_score_static -- the scoring entry point for callers that cannot allocate device memory (its
scratch is a fixed array inside the library) -- must give what pvf_score gives.

Collected last on purpose (file name): a run that stops at the first failure has then already run every
other test.  Each case makes two calls in a row with different row counts, because all calls share the
one built-in array and it keeps the previous call's contents.  Passes alone in a fresh process and after
the other tests."""
import numpy as np
import pytest
import torch

from oracle import score as oscore
from paper_2601_12247_b200 import binding, synth
from gpu_util import TOL, check_score, dev, make_ctx, to_np, upload_bits

pytestmark = pytest.mark.gpu


def outputs(M):
    return dict(tok=torch.full((M,), -1, dtype=torch.int32, device=dev()),
                conf=torch.full((M,), -1.0, dtype=torch.float32, device=dev()),
                ent=torch.full((M,), -1.0, dtype=torch.float32, device=dev()),
                in_plan=torch.full((M,), 9, dtype=torch.uint8, device=dev()))


def bitmap_of(plan_ids, vocab):
    words = np.zeros((vocab + 31) // 32, dtype=np.uint32)
    for v in plan_ids:
        words[v >> 5] |= np.uint32(1) << np.uint32(v & 31)
    return torch.from_numpy(words.view(np.int32)).to(dev())


def compare(static_out, ctx_out):
    s, c = to_np(static_out), to_np(ctx_out)
    assert np.array_equal(s["tok"], c["tok"]) and np.array_equal(s["in_plan"], c["in_plan"])
    assert np.max(np.abs(s["conf"].astype(np.float64) - c["conf"])) <= TOL
    assert np.max(np.abs(s["ent"].astype(np.float64) - c["ent"])) <= TOL


@pytest.mark.parametrize("V,D,rows", [(4096, 256, (150, 64)), (5000, 200, (33, 300)), (70000, 512, (1024, 1))])
def test_two_calls_in_a_row_match_pvf_score(V, D, rows):
    M_max = max(rows)
    pos = np.arange(M_max)
    st = synth.build_step("static", 777, V, D, 64, [(pos, np.ones(M_max, np.uint8))], M_max, M_max,
                          dict(tau_high=0.9, budget=4), amp_max=40.0 * (256.0 / D) ** 0.5)
    ctx = make_ctx(st.w_bits, st.plan_ids, M_max)
    w = ctx.w_head
    bitmap = bitmap_of(st.plan_ids, V)
    for M in rows:                                    # second call reuses the array the first one filled
        h = upload_bits(st.h_bits[:M])
        out = outputs(M)
        rc = binding.score_static(w, h, out, bitmap)
        assert rc == binding.PVF_OK, binding.strerror(rc)
        torch.cuda.synchronize()
        assert binding.score_static_status() == 0
        compare(out, ctx.score(h))
    ctx.close()


def test_rejects_more_rows_than_the_array_holds_and_bad_arguments():
    V, D = 4096, 256
    w = upload_bits(synth.make_w(3, V, D))
    M = binding.PVF_STATIC_MAX_ROWS + 1
    h = torch.zeros((M, D), dtype=torch.bfloat16, device=dev())
    out = outputs(M)
    assert binding.score_static(w, h[:8], outputs(8), None) == binding.PVF_ERR_INVALID   # in_plan without a bitmap
    out.pop("in_plan")
    assert binding.score_static(w, h, out, None) == binding.PVF_ERR_TOO_LARGE
    assert "scratch" in binding.strerror(binding.PVF_ERR_TOO_LARGE)
    torch.cuda.synchronize()
    assert float(out["conf"].max()) == -1.0                                         # nothing was launched
    ok = outputs(8); ok.pop("in_plan")
    assert binding.score_static(w, h[:8], ok, None) == binding.PVF_OK              # zero rows -> uniform
    torch.cuda.synchronize()
    assert np.allclose(ok["conf"].cpu().numpy(), 1.0 / V, atol=1e-7) and ok["tok"].cpu().numpy().tolist() == [0] * 8


def test_llada_shape_two_calls():
    V, D = synth.LLADA_VOCAB, synth.LLADA_HIDDEN
    w_bits = synth.make_w(1001, V, D)
    st = synth.config1("a", w_bits=w_bits)
    ctx = make_ctx(w_bits, st.plan_ids, 256)
    bitmap = bitmap_of(st.plan_ids, V)
    for M in (32, 17):
        h = upload_bits(st.h_bits[:M])
        out = outputs(M)
        assert binding.score_static(ctx.w_head, h, out, bitmap) == binding.PVF_OK
        torch.cuda.synchronize()
        assert binding.score_static_status() == 0
        compare(out, ctx.score(h))
    ctx.close()


def test_matches_the_oracle_directly_and_allocates_no_device_memory():
    # The property the entry point exists for: once a device has made its first call, further calls leave the
    # amount of free device memory exactly as it was (cudaMemGetInfo through torch), whatever the row count and
    # the kernel that serves it.  And its outputs are checked against the fp64 oracle itself, not only against
    # pvf_score.
    V, D, M_max = 4096, 256, 300
    pos = np.arange(M_max)
    st = synth.build_step("static-oracle", 778, V, D, 64, [(pos, np.ones(M_max, np.uint8))], M_max, M_max,
                          dict(tau_high=0.9, budget=4))
    w = upload_bits(st.w_bits)
    bitmap = bitmap_of(st.plan_ids, V)
    cases = [(M, upload_bits(st.h_bits[:M]), outputs(M)) for M in (150, 20, 300, 64)]   # every tensor exists beforehand
    assert binding.score_static(w, cases[0][1], cases[0][2], bitmap) == binding.PVF_OK  # the device's set-up call
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for M, h, out in cases:
        assert binding.score_static(w, h, out, bitmap) == binding.PVF_OK
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert binding.score_static_status() == 0
    for M, h, out in cases:
        check_score(to_np(out), oscore.score(st.w_bits, st.h_bits[:M], st.plan_ids), V, st.plan_ids)
