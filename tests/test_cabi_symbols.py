"""The C-ABI library builds for sm_100a, loads without a GPU and exports everything pvf.h declares."""
import ctypes
import os
import re

from paper_2601_12247_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "pvf.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pvf_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(build.build())
    names = declared_functions()
    assert {"pvf_score", "pvf_commit", "pvf_select_drafts", "pvf_verify", "pvf_create", "pvf_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_defaults_are_the_papers_printed_values():
    golden = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "paper_hyperparameters.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            golden[k] = float(v)
    p = binding.default_params()
    f32 = lambda x: ctypes.c_float(x).value
    assert p.tau_high == f32(golden["tau_high"]) and p.budget == int(golden["budget_K"])
    assert p.tau_plan_lo == f32(golden["tau_plan_lo"]) and p.tau_plan_hi == f32(golden["tau_plan_hi"])
    assert p.tau_ar_lo == f32(golden["tau_ar_lo"]) and p.flags == 0
    c = binding.default_calib_params()
    assert c.tau_cal_lo == f32(golden["tau_cal_lo"]) and c.tau_cal_hi == f32(golden["tau_cal_hi"])
    assert c.n_min == int(golden["n_min"]) and c.m_min == int(golden["m_min"])
    assert c.rho_ver == f32(golden["rho_ver"]) and c.gamma_vig == f32(golden["gamma_vig"])
    from paper_2601_12247_b200 import synth
    assert synth.DEFAULT_BAND == dict(tau_plan_lo=golden["tau_plan_lo"], tau_plan_hi=golden["tau_plan_hi"],
                                      tau_ar_lo=golden["tau_ar_lo"])


def test_error_strings_and_host_side_argument_checks():
    assert binding.strerror(0) == "ok"
    for code in range(-6, 0):
        assert binding.strerror(code) not in ("ok", "unknown error")
    lib = binding.load()
    # NULL context / shape are rejected on the host, before any CUDA call
    assert lib.pvf_score(None, None, 4, None, None, None, None, None) == binding.PVF_ERR_INVALID
    assert lib.pvf_workspace_bytes(None) == 0
    assert lib.pvf_create(None, None, None, None, 0, None, 0) == binding.PVF_ERR_INVALID


def test_host_only_entry_points_work_without_a_gpu():
    lib = binding.load()
    # every error code has a message of its own
    codes = [0, -1, -2, -3, -4, -5, -6, -7]
    msgs = [binding.strerror(c) for c in codes]
    assert len(set(msgs)) == len(codes) and binding.strerror(-99) == "unknown error"
    # staging and bounce sizes are pure arithmetic on the shape
    small = binding.pvf_shape(4096, 256, 64, 4, 4)
    big = binding.pvf_shape(4096, 256, 128, 4, 4)
    s_small = lib.pvf_host_staging_bytes(ctypes.byref(small))
    s_big = lib.pvf_host_staging_bytes(ctypes.byref(big))
    assert s_small >= 64 * 256 * 2 and s_big - s_small >= 64 * 256 * 2
    b_small = lib.pvf_host_bounce_bytes(ctypes.byref(small))
    assert 0 < b_small < s_small and s_small - b_small >= 64 * 256 * 2          # the bounce buffer holds no hidden states
    bad = binding.pvf_shape(0, 256, 64, 4, 4)
    assert lib.pvf_host_staging_bytes(ctypes.byref(bad)) == 0 and lib.pvf_host_bounce_bytes(ctypes.byref(bad)) == 0
    # calls that need a context refuse a missing one instead of touching the device
    assert lib.pvf_score(None, None, 4, None, None, None, None, None) == binding.PVF_ERR_INVALID
    assert lib.pvf_attach_host_staging(None, None, 0) == binding.PVF_ERR_INVALID
    assert lib.pvf_working_set(None, None, 1, 8, 4, 0, 0, None, None, None, None, None, 8, None) == binding.PVF_ERR_INVALID
    assert lib.pvf_score_kernel_name(None, 4) is None
    st = ctypes.c_int32(7)
    assert lib.pvf_last_status(None, ctypes.byref(st)) == binding.PVF_ERR_INVALID
