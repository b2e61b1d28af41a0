"""The host-buffer entry points give exactly what the device entry points give."""
import numpy as np
import pytest
import torch

from paper_2601_12247_b200 import binding, synth
from gpu_util import make_ctx, params_of, t_i32, t_u8, to_np, upload_bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("stress,pinned,bounce", [(False, True, True), (True, False, True), (True, True, False)])
def test_host_step_equals_device_step(stress, pinned, bounce):
    w = synth.make_w(2002, 8192, 256)
    st = synth.config2(stress=stress, w_bits=w, vocab=8192, hidden=256)
    ctx = make_ctx(w, st.plan_ids, 16384, 64, 16)
    prm = params_of(st)
    K = int(st.params["budget"])
    seg, pos, act = t_i32(st.seg_off), t_i32(st.row_pos), t_u8(st.active)
    sc = ctx.score(upload_bits(st.h_bits))
    cm = ctx.commit(prm, seg, pos, act, sc["tok"], sc["conf"])
    sel = ctx.select_drafts(prm, seg, pos, act, sc["tok"], sc["conf"], sc["in_plan"], cm["commit"])
    s = to_np(sel)
    n_rem = int(s["rem_off"][-1])
    vp = synth.make_verify_pass(st, s["rem_rows"][:n_rem], s["rem_off"], s["n_drafts"])
    Mv = vp.hv_bits.shape[0]
    scv = ctx.score(upload_bits(vp.hv_bits))
    ver = ctx.verify(prm, seg, pos, sel, sc["tok"], scv["tok"], scv["conf"], cm["commit"])
    torch.cuda.synchronize()

    with pytest.raises(binding.PvfError) as e:                                   # no staging attached yet
        ctx.draft_step_host(prm, binding.bf16_from_bits(st.h_bits, "cpu"), torch.from_numpy(st.seg_off),
                            torch.from_numpy(st.row_pos), None, {})
    assert e.value.code == binding.PVF_ERR_WORKSPACE
    ctx.attach_host_staging(bounce=bounce)
    hb = binding.host_buffers(st.n_rows, st.n_seq, K, Mv, pinned=pinned)
    mk = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    ctx.draft_step_host(prm, mk(binding.bf16_from_bits(st.h_bits, "cpu")), mk(torch.from_numpy(st.seg_off)),
                        mk(torch.from_numpy(st.row_pos)), mk(torch.from_numpy(st.active)), hb)
    g = {k: v.numpy() for k, v in hb.items()}
    d = dict(to_np(sc), **to_np(cm), **s)
    for k in ("tok", "conf", "ent", "in_plan", "commit", "draft_rows", "n_drafts", "route", "rem_off", "v_off"):
        assert np.array_equal(g[k], d[k]), k
    assert np.array_equal(g["rem_rows"][:n_rem], s["rem_rows"][:n_rem])
    ctx.verify_step_host(prm, mk(binding.bf16_from_bits(vp.hv_bits, "cpu")) if Mv else None, hb)
    dv = dict(tok_v=scv["tok"].cpu().numpy(), conf_v=scv["conf"].cpu().numpy(), **to_np(ver))
    assert np.array_equal(g["tok_v"][:Mv], dv["tok_v"]) and np.array_equal(g["conf_v"][:Mv], dv["conf_v"])
    for k in ("accept", "choice", "final_commit"):
        assert np.array_equal(g[k], dv[k]), k
    # again and again on the same context: the results of every call are the call's own (nothing left over from
    # the one before is taken for them)
    for _ in range(4):
        for v in hb.values():
            v.zero_()
        ctx.draft_step_host(prm, mk(binding.bf16_from_bits(st.h_bits, "cpu")), mk(torch.from_numpy(st.seg_off)),
                            mk(torch.from_numpy(st.row_pos)), mk(torch.from_numpy(st.active)), hb)
        for k in ("tok", "conf", "ent", "in_plan", "commit", "draft_rows", "n_drafts", "route", "rem_off", "v_off"):
            assert np.array_equal(hb[k].numpy(), d[k]), k
        ctx.verify_step_host(prm, mk(binding.bf16_from_bits(vp.hv_bits, "cpu")) if Mv else None, hb)
        assert np.array_equal(hb["tok_v"].numpy()[:Mv], dv["tok_v"])
        for k in ("accept", "choice", "final_commit"):
            assert np.array_equal(hb[k].numpy(), dv[k]), k
    assert ctx.last_status() == 0
    ctx.close()
