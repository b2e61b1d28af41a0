"""Thin ctypes binding of libpvf.so: argument marshalling only.

Every function here has the name and meaning of the C entry point it calls (see include/pvf.h);
torch is used for device memory and for the current stream, nothing else.  There is no fallback:
if the library has not been built, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpvf.so")

PVF_OK = 0
PVF_ERR_INVALID, PVF_ERR_ALIGN, PVF_ERR_UNSUPPORTED, PVF_ERR_CUDA, PVF_ERR_TIMEOUT, PVF_ERR_WORKSPACE = -1, -2, -3, -4, -5, -6
PVF_ERR_TOO_LARGE = -7
PVF_STATIC_MAX_ROWS = 1024
PVF_FORCE_PROGRESS = 1
PVF_EXCLUDE_SELF_FROM_IMPACT = 2
PVF_EXPLORE_RANDOM, PVF_EXPLORE_PLANNING = 0, 1
PVF_SELECT_ANY_TOKEN = 4
PVF_NO_AR_FALLBACK = 8


class pvf_shape(ctypes.Structure):
    _fields_ = [("vocab", ctypes.c_int32), ("hidden", ctypes.c_int32), ("max_rows", ctypes.c_int32),
                ("max_seqs", ctypes.c_int32), ("max_budget", ctypes.c_int32)]


class pvf_params(ctypes.Structure):
    _fields_ = [("tau_high", ctypes.c_float), ("tau_plan_lo", ctypes.c_float), ("tau_plan_hi", ctypes.c_float),
                ("tau_ar_lo", ctypes.c_float), ("budget", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class pvf_calib_params(ctypes.Structure):
    _fields_ = [("tau_cal_lo", ctypes.c_float), ("tau_cal_hi", ctypes.c_float), ("n_min", ctypes.c_int32),
                ("m_min", ctypes.c_int32), ("rho_ver", ctypes.c_float), ("gamma_vig", ctypes.c_float)]


class PvfError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s failed: %d (%s)" % (what, code, strerror(code)))
        self.code = code


_lib = None


def load() -> ctypes.CDLL:
    """Load libpvf.so; raises if it is missing (build it with paper_2601_12247_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            # not built yet: build it now if this machine has nvcc; there is no CPU or PyTorch fallback
            try:
                from . import build as _build
                if os.path.abspath(LIB_PATH) == os.path.abspath(_build.LIB):
                    _build.build()
            except Exception as exc:
                raise RuntimeError("libpvf.so is not built and could not be built here (%s): run "
                                   "`python -m paper_2601_12247_b200.build` (there is no CPU or PyTorch fallback)" % exc)
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libpvf.so is not built: run `python -m paper_2601_12247_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        pp = ctypes.POINTER(pvf_params)
        ps = ctypes.POINTER(pvf_shape)
        lib.pvf_default_params.argtypes = [pp]; lib.pvf_default_params.restype = None
        lib.pvf_strerror.argtypes = [ctypes.c_int]; lib.pvf_strerror.restype = ctypes.c_char_p
        lib.pvf_workspace_bytes.argtypes = [ps]; lib.pvf_workspace_bytes.restype = sz
        lib.pvf_create.argtypes = [ctypes.POINTER(vp), ps, vp, vp, i32, vp, sz]; lib.pvf_create.restype = ctypes.c_int
        lib.pvf_destroy.argtypes = [vp]; lib.pvf_destroy.restype = ctypes.c_int
        lib.pvf_last_status.argtypes = [vp, ctypes.POINTER(i32)]; lib.pvf_last_status.restype = ctypes.c_int
        lib.pvf_set_score_events.argtypes = [vp, vp, vp]; lib.pvf_set_score_events.restype = ctypes.c_int
        lib.pvf_score_plan.argtypes = [vp, i32] + [ctypes.POINTER(i32)] * 4; lib.pvf_score_plan.restype = ctypes.c_int
        lib.pvf_score_plan_for_shape.argtypes = [i32] * 4 + [ctypes.POINTER(i32)] * 8
        lib.pvf_score_plan_for_shape.restype = ctypes.c_int
        lib.pvf_score_kernel_name.argtypes = [vp, i32]; lib.pvf_score_kernel_name.restype = ctypes.c_char_p
        lib.pvf_score_clock.argtypes = [vp, i32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)]
        lib.pvf_score_clock.restype = ctypes.c_int
        lib.pvf_score.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp]; lib.pvf_score.restype = ctypes.c_int
        lib.pvf_commit.argtypes = [vp, pp, i32, i32] + [vp] * 8 + [i32, vp]; lib.pvf_commit.restype = ctypes.c_int
        lib.pvf_select_drafts.argtypes = [vp, pp, i32, i32] + [vp] * 13 + [vp]; lib.pvf_select_drafts.restype = ctypes.c_int
        lib.pvf_verify.argtypes = [vp, pp, i32, i32] + [vp] * 16 + [i32, vp]; lib.pvf_verify.restype = ctypes.c_int
        lib.pvf_commit_select.argtypes = [vp, pp, i32, i32] + [vp] * 9 + [i32] + [vp] * 6 + [vp]
        lib.pvf_commit_select.restype = ctypes.c_int
        lib.pvf_draft_step.argtypes = [vp, pp, vp, i32, i32] + [vp] * 10 + [i32] + [vp] * 6 + [vp]
        lib.pvf_draft_step.restype = ctypes.c_int
        lib.pvf_verify_step.argtypes = [vp, pp, vp, i32, i32, i32] + [vp] * 17 + [i32, vp]
        lib.pvf_verify_step.restype = ctypes.c_int
        lib.pvf_explore_commit.argtypes = [vp, pp, i32, i32, i32] + [vp] * 10 + [i32, vp]
        lib.pvf_explore_commit.restype = ctypes.c_int
        pc = ctypes.POINTER(pvf_calib_params)
        lib.pvf_default_calib_params.argtypes = [pc]; lib.pvf_default_calib_params.restype = None
        lib.pvf_calib_accumulate.argtypes = [vp, pp, i32] + [vp] * 15 + [vp]; lib.pvf_calib_accumulate.restype = ctypes.c_int
        lib.pvf_calib_filter.argtypes = [vp, pc] + [vp] * 6 + [vp]; lib.pvf_calib_filter.restype = ctypes.c_int
        lib.pvf_set_plan_bitmap.argtypes = [vp, vp, vp]; lib.pvf_set_plan_bitmap.restype = ctypes.c_int
        lib.pvf_working_set.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32, vp]
        lib.pvf_working_set.restype = ctypes.c_int
        lib.pvf_host_staging_bytes.argtypes = [ps]; lib.pvf_host_staging_bytes.restype = sz
        lib.pvf_attach_host_staging.argtypes = [vp, vp, sz]; lib.pvf_attach_host_staging.restype = ctypes.c_int
        lib.pvf_host_bounce_bytes.argtypes = [ps]; lib.pvf_host_bounce_bytes.restype = sz
        lib.pvf_attach_host_bounce.argtypes = [vp, vp, sz]; lib.pvf_attach_host_bounce.restype = ctypes.c_int
        lib.pvf_draft_step_host.argtypes = [vp, pp, vp, i32, i32] + [vp] * 14 + [vp]; lib.pvf_draft_step_host.restype = ctypes.c_int
        lib.pvf_verify_step_host.argtypes = [vp, pp, vp, i32] + [vp] * 5 + [vp]; lib.pvf_verify_step_host.restype = ctypes.c_int
        lib.pvf_score_static.argtypes = [vp, i32, i32, vp, i32, vp, vp, vp, vp, vp, vp]; lib.pvf_score_static.restype = ctypes.c_int
        lib.pvf_score_static_status.argtypes = [ctypes.POINTER(i32)]; lib.pvf_score_static_status.restype = ctypes.c_int
        _lib = lib
    return _lib


def strerror(code: int) -> str:
    return load().pvf_strerror(int(code)).decode()


def default_params() -> pvf_params:
    p = pvf_params()
    load().pvf_default_params(ctypes.byref(p))
    return p


def score_plan_for_shape(vocab: int, hidden: int, n_sm: int, M: int) -> Dict[str, int]:
    """pvf_score_plan_for_shape: the work split pvf_score would use, computed on the host (no GPU needed)."""
    v = [ctypes.c_int32() for _ in range(8)]
    _check(load().pvf_score_plan_for_shape(int(vocab), int(hidden), int(n_sm), int(M), *[ctypes.byref(x) for x in v]),
           "pvf_score_plan_for_shape")
    return dict(zip(("ctas", "splits", "waves", "kernel", "row_tiles", "tiles_per_wave", "last_wave_tiles", "last_wave_splits"),
                    (x.value for x in v)))


def default_calib_params() -> pvf_calib_params:
    c = pvf_calib_params()
    load().pvf_default_calib_params(ctypes.byref(c))
    return c


def make_params(tau_high: float, tau_plan_lo: float, tau_plan_hi: float, tau_ar_lo: float, budget: int,
                flags: int = 0) -> pvf_params:
    return pvf_params(tau_high, tau_plan_lo, tau_plan_hi, tau_ar_lo, int(budget), int(flags))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc: int, what: str):
    if rc != PVF_OK:
        raise PvfError(rc, what)


class Context:
    """Owns a pvf_ctx, its workspace and a reference to the LM-head weight."""

    def __init__(self, w_head: torch.Tensor, plan_ids, max_rows: int, max_seqs: int, max_budget: int):
        lib = load()
        assert w_head.is_cuda and w_head.dtype == torch.bfloat16 and w_head.is_contiguous() and w_head.dim() == 2
        self.lib = lib
        self.w_head = w_head
        self.device = w_head.device
        self.shape = pvf_shape(w_head.shape[0], w_head.shape[1], int(max_rows), int(max_seqs), int(max_budget))
        with torch.cuda.device(self.device):
            nbytes = lib.pvf_workspace_bytes(ctypes.byref(self.shape))
            if nbytes == 0:
                raise PvfError(PVF_ERR_INVALID, "pvf_workspace_bytes")
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            off = (-self.workspace.data_ptr()) % 256
            ids = np.ascontiguousarray(np.asarray(plan_ids, dtype=np.int32))
            self.handle = ctypes.c_void_p()
            rc = lib.pvf_create(ctypes.byref(self.handle), ctypes.byref(self.shape), _ptr(w_head),
                                ids.ctypes.data_as(ctypes.c_void_p), len(ids),
                                ctypes.c_void_p(self.workspace.data_ptr() + off), nbytes)
        _check(rc, "pvf_create")

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle.value:
            self.lib.pvf_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def last_status(self) -> int:
        st = ctypes.c_int32()
        _check(self.lib.pvf_last_status(self.handle, ctypes.byref(st)), "pvf_last_status")
        return int(st.value)

    def set_score_events(self, start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]):
        """Timing hook: events recorded around the GEMM kernel of every following score call."""
        for ev in (start, stop):
            if ev is not None and not ev.cuda_event:
                ev.record()                      # torch creates the CUDA event lazily, on first record
        a = None if start is None else ctypes.c_void_p(start.cuda_event)
        b = None if stop is None else ctypes.c_void_p(stop.cuda_event)
        _check(self.lib.pvf_set_score_events(self.handle, a, b), "pvf_set_score_events")

    def score_plan(self, M: int) -> Dict[str, int]:
        v = [ctypes.c_int32() for _ in range(4)]
        _check(self.lib.pvf_score_plan(self.handle, int(M), *[ctypes.byref(x) for x in v]), "pvf_score_plan")
        return dict(ctas=v[0].value, splits=v[1].value, waves=v[2].value, launches=v[3].value)

    def score_clock(self, which: int) -> Dict[str, float]:
        """pvf_score_clock: mean run time, SM clock and count of the projection launches since the last call
        (which = 0: pvf_score / draft pass, 1: verification pass); synchronises the device and clears the sums."""
        ms, mhz, n = ctypes.c_double(), ctypes.c_double(), ctypes.c_int64()
        _check(self.lib.pvf_score_clock(self.handle, int(which), ctypes.byref(ms), ctypes.byref(mhz), ctypes.byref(n)), "pvf_score_clock")
        return dict(ms=ms.value, sm_mhz=mhz.value, launches=int(n.value), sm_cycles=ms.value * mhz.value * 1e3)

    def score_kernel_name(self, M: int) -> str:
        name = self.lib.pvf_score_kernel_name(self.handle, int(M))
        if name is None:
            raise PvfError(PVF_ERR_INVALID, "pvf_score_kernel_name")
        return name.decode()

    # ------------------------------------------------------------------ host-buffer variants
    def attach_host_staging(self, bounce: bool = True):
        """Allocate the device staging buffer of the host-buffer calls (and, with ``bounce``, the pinned host
        bounce buffer that packs their copies) and hand them to the context."""
        nbytes = self.lib.pvf_host_staging_bytes(ctypes.byref(self.shape))
        self.staging = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.staging.data_ptr()) % 256
        _check(self.lib.pvf_attach_host_staging(self.handle, ctypes.c_void_p(self.staging.data_ptr() + off), nbytes),
               "pvf_attach_host_staging")
        if bounce:
            hbytes = self.lib.pvf_host_bounce_bytes(ctypes.byref(self.shape))
            self.bounce = torch.empty(hbytes, dtype=torch.uint8).pin_memory()
            _check(self.lib.pvf_attach_host_bounce(self.handle, ctypes.c_void_p(self.bounce.data_ptr()), hbytes),
                   "pvf_attach_host_bounce")
        else:
            _check(self.lib.pvf_attach_host_bounce(self.handle, None, 0), "pvf_attach_host_bounce")

    def draft_step_host(self, params: pvf_params, hidden_host: torch.Tensor, seg_off: torch.Tensor, row_pos: torch.Tensor,
                        active: Optional[torch.Tensor], out: Dict[str, torch.Tensor]):
        """pvf_draft_step_host: all tensors are CPU tensors; returns after the results are in ``out``."""
        hp = lambda k: _ptr(out.get(k))
        rc = self.lib.pvf_draft_step_host(self.handle, ctypes.byref(params), _ptr(hidden_host), hidden_host.shape[0],
                                          seg_off.shape[0] - 1, _ptr(seg_off), _ptr(row_pos), _ptr(active),
                                          hp("tok"), hp("conf"), hp("ent"), hp("in_plan"), hp("commit"), hp("draft_rows"),
                                          hp("n_drafts"), hp("route"), hp("rem_rows"), hp("rem_off"), hp("v_off"), _stream())
        _check(rc, "pvf_draft_step_host")
        return out

    def verify_step_host(self, params: pvf_params, hidden_v_host: Optional[torch.Tensor], out: Dict[str, torch.Tensor]):
        """pvf_verify_step_host: continues the last draft_step_host of this context."""
        Mv = 0 if hidden_v_host is None else hidden_v_host.shape[0]
        hp = lambda k: _ptr(out.get(k))
        rc = self.lib.pvf_verify_step_host(self.handle, ctypes.byref(params), _ptr(hidden_v_host), Mv,
                                           hp("tok_v"), hp("conf_v"), hp("accept"), hp("choice"), hp("final_commit"), _stream())
        _check(rc, "pvf_verify_step_host")
        return out

    def explore_commit(self, params: pvf_params, mode: int, seg_off, row_pos, active, tok, conf, in_plan, u, commit, y=None):
        """pvf_explore_commit: updates ``commit`` in place; returns explore_row [n_seq]."""
        M, n_seq = conf.shape[0], seg_off.shape[0] - 1
        explore_row = torch.empty(max(n_seq, 1), dtype=torch.int32, device=self.device)
        L = 0 if y is None else y.shape[1]
        rc = self.lib.pvf_explore_commit(self.handle, ctypes.byref(params), int(mode), M, n_seq, _ptr(seg_off), _ptr(row_pos),
                                         _ptr(active), _ptr(tok), _ptr(conf), _ptr(in_plan), _ptr(u), _ptr(commit),
                                         _ptr(explore_row), _ptr(y), L, _stream())
        _check(rc, "pvf_explore_commit")
        return explore_row[:n_seq]

    # ------------------------------------------------------------------ planning-vocabulary calibration
    def new_calib_stats(self) -> Dict[str, torch.Tensor]:
        """Zeroed per-token statistics (n_v, m_v, sum_a int32; sum_vig_q32 int64) on the context's device."""
        V = self.shape.vocab
        z = lambda dt: torch.zeros(V, dtype=dt, device=self.device)
        return dict(n_v=z(torch.int32), m_v=z(torch.int32), sum_a=z(torch.int32), sum_vig_q32=z(torch.int64))

    def calib_accumulate(self, params: pvf_params, sel: Dict[str, torch.Tensor], tok, conf_v, ent_v, accept,
                         stats: Dict[str, torch.Tensor], vig_out: Optional[torch.Tensor] = None):
        n_seq = sel["n_drafts"].shape[0]
        rc = self.lib.pvf_calib_accumulate(self.handle, ctypes.byref(params), n_seq, _ptr(sel["rem_rows"]),
                                           _ptr(sel["rem_off"]), _ptr(sel["v_off"]), _ptr(sel["draft_rows"]),
                                           _ptr(sel["n_drafts"]), _ptr(sel["route"]), _ptr(tok), _ptr(conf_v), _ptr(ent_v),
                                           _ptr(accept), _ptr(stats["n_v"]), _ptr(stats["m_v"]), _ptr(stats["sum_a"]),
                                           _ptr(stats["sum_vig_q32"]), _ptr(vig_out), _stream())
        _check(rc, "pvf_calib_accumulate")

    def calib_filter(self, cal: pvf_calib_params, stats: Dict[str, torch.Tensor]):
        """Returns (bitmap int32 tensor of ceil(V/32) words, n_plan int32 tensor of one element)."""
        words = (self.shape.vocab + 31) // 32
        bitmap = torch.empty(words, dtype=torch.int32, device=self.device)
        n_plan = torch.empty(1, dtype=torch.int32, device=self.device)
        rc = self.lib.pvf_calib_filter(self.handle, ctypes.byref(cal), _ptr(stats["n_v"]), _ptr(stats["m_v"]),
                                       _ptr(stats["sum_a"]), _ptr(stats["sum_vig_q32"]), _ptr(bitmap), _ptr(n_plan), _stream())
        _check(rc, "pvf_calib_filter")
        return bitmap, n_plan

    def set_plan_bitmap(self, bitmap: torch.Tensor):
        _check(self.lib.pvf_set_plan_bitmap(self.handle, _ptr(bitmap), _stream()), "pvf_set_plan_bitmap")

    def working_set(self, y: torch.Tensor, block: int, n_sparse: int, mask_id: int, out=None):
        """pvf_working_set: rows of the next step from the canvas y [n_seq][L] (int32, on the device)."""
        assert y.is_cuda and y.dtype == torch.int32 and y.is_contiguous() and y.dim() == 2
        n_seq, L = y.shape
        cap = n_seq * min(2 * int(block), L)
        if out is None:
            dev = self.device
            out = dict(seg_off=torch.empty(n_seq + 1, dtype=torch.int32, device=dev),
                       row_pos=torch.empty(max(cap, 1), dtype=torch.int32, device=dev),
                       row_seq=torch.empty(max(cap, 1), dtype=torch.int32, device=dev),
                       active=torch.empty(max(cap, 1), dtype=torch.uint8, device=dev),
                       expanded=torch.empty(max(n_seq, 1), dtype=torch.uint8, device=dev))
        rc = self.lib.pvf_working_set(self.handle, _ptr(y), n_seq, L, int(block), int(n_sparse), int(mask_id),
                                      _ptr(out["seg_off"]), _ptr(out["row_pos"]), _ptr(out.get("row_seq")),
                                      _ptr(out.get("active")), _ptr(out.get("expanded")), out["row_pos"].shape[0], _stream())
        _check(rc, "pvf_working_set")
        return out

    # ------------------------------------------------------------------ the four calls
    def score(self, hidden: torch.Tensor, out: Optional[Dict[str, torch.Tensor]] = None) -> Dict[str, torch.Tensor]:
        assert hidden.is_cuda and hidden.dtype == torch.bfloat16 and hidden.is_contiguous()
        M = hidden.shape[0]
        if out is None:
            out = dict(tok=torch.empty(M, dtype=torch.int32, device=self.device),
                       conf=torch.empty(M, dtype=torch.float32, device=self.device),
                       ent=torch.empty(M, dtype=torch.float32, device=self.device),
                       in_plan=torch.empty(M, dtype=torch.uint8, device=self.device))
        rc = self.lib.pvf_score(self.handle, _ptr(hidden), M, _ptr(out["tok"]), _ptr(out["conf"]),
                                _ptr(out.get("ent")), _ptr(out.get("in_plan")), _stream())
        _check(rc, "pvf_score")
        return out

    def commit(self, params: pvf_params, seg_off, row_pos, active, tok, conf, y=None, out=None):
        M, n_seq = conf.shape[0], seg_off.shape[0] - 1
        if out is None:
            out = dict(commit=torch.empty(M, dtype=torch.uint8, device=self.device),
                       n_commit=torch.empty(n_seq, dtype=torch.int32, device=self.device))
        L = 0 if y is None else y.shape[1]
        rc = self.lib.pvf_commit(self.handle, ctypes.byref(params), M, n_seq, _ptr(seg_off), _ptr(row_pos),
                                 _ptr(active), _ptr(tok), _ptr(conf), _ptr(out["commit"]), _ptr(out["n_commit"]),
                                 _ptr(y), L, _stream())
        _check(rc, "pvf_commit")
        return out

    def select_drafts(self, params: pvf_params, seg_off, row_pos, active, tok, conf, in_plan, commit, out=None):
        M, n_seq, K = conf.shape[0], seg_off.shape[0] - 1, int(params.budget)
        if out is None:
            dev = self.device
            out = dict(draft_rows=torch.empty((n_seq, K), dtype=torch.int32, device=dev),
                       n_drafts=torch.empty(n_seq, dtype=torch.int32, device=dev),
                       route=torch.empty(n_seq, dtype=torch.uint8, device=dev),
                       rem_rows=torch.empty(max(M, 1), dtype=torch.int32, device=dev),
                       rem_off=torch.empty(n_seq + 1, dtype=torch.int32, device=dev),
                       v_off=torch.empty(n_seq + 1, dtype=torch.int32, device=dev))
        rc = self.lib.pvf_select_drafts(self.handle, ctypes.byref(params), M, n_seq, _ptr(seg_off), _ptr(row_pos),
                                        _ptr(active), _ptr(tok), _ptr(conf), _ptr(in_plan), _ptr(commit),
                                        _ptr(out["draft_rows"]), _ptr(out["n_drafts"]), _ptr(out["route"]),
                                        _ptr(out["rem_rows"]), _ptr(out["rem_off"]), _ptr(out["v_off"]), _stream())
        _check(rc, "pvf_select_drafts")
        return out

    def _step_outputs(self, M: int, n_seq: int, K: int) -> Dict[str, torch.Tensor]:
        dev = self.device
        return dict(commit=torch.empty(M, dtype=torch.uint8, device=dev),
                    n_commit=torch.empty(n_seq, dtype=torch.int32, device=dev),
                    draft_rows=torch.empty((n_seq, K), dtype=torch.int32, device=dev),
                    n_drafts=torch.empty(n_seq, dtype=torch.int32, device=dev),
                    route=torch.empty(n_seq, dtype=torch.uint8, device=dev),
                    rem_rows=torch.empty(max(M, 1), dtype=torch.int32, device=dev),
                    rem_off=torch.empty(n_seq + 1, dtype=torch.int32, device=dev),
                    v_off=torch.empty(n_seq + 1, dtype=torch.int32, device=dev))

    def commit_select(self, params: pvf_params, seg_off, row_pos, active, tok, conf, in_plan, y=None, out=None):
        """pvf_commit_select: pvf_commit + pvf_select_drafts in one launch; ``out`` holds both calls' outputs."""
        M, n_seq, K = conf.shape[0], seg_off.shape[0] - 1, int(params.budget)
        if out is None:
            out = self._step_outputs(M, n_seq, K)
        L = 0 if y is None else y.shape[1]
        rc = self.lib.pvf_commit_select(self.handle, ctypes.byref(params), M, n_seq, _ptr(seg_off), _ptr(row_pos),
                                        _ptr(active), _ptr(tok), _ptr(conf), _ptr(in_plan), _ptr(out["commit"]),
                                        _ptr(out.get("n_commit")), _ptr(y), L, _ptr(out["draft_rows"]), _ptr(out["n_drafts"]),
                                        _ptr(out["route"]), _ptr(out["rem_rows"]), _ptr(out["rem_off"]), _ptr(out["v_off"]),
                                        _stream())
        _check(rc, "pvf_commit_select")
        return out

    def draft_step(self, params: pvf_params, hidden, seg_off, row_pos, active, y=None, out=None):
        """pvf_draft_step: pvf_score + pvf_commit_select (two launches).  ``out`` holds tok, conf, ent, in_plan and the
        outputs of commit_select."""
        M, n_seq, K = hidden.shape[0], seg_off.shape[0] - 1, int(params.budget)
        if out is None:
            out = self._step_outputs(M, n_seq, K)
            out.update(tok=torch.empty(M, dtype=torch.int32, device=self.device),
                       conf=torch.empty(M, dtype=torch.float32, device=self.device),
                       ent=torch.empty(M, dtype=torch.float32, device=self.device),
                       in_plan=torch.empty(M, dtype=torch.uint8, device=self.device))
        L = 0 if y is None else y.shape[1]
        rc = self.lib.pvf_draft_step(self.handle, ctypes.byref(params), _ptr(hidden), M, n_seq, _ptr(seg_off), _ptr(row_pos),
                                     _ptr(active), _ptr(out["tok"]), _ptr(out["conf"]), _ptr(out.get("ent")), _ptr(out["in_plan"]),
                                     _ptr(out["commit"]), _ptr(out.get("n_commit")), _ptr(y), L, _ptr(out["draft_rows"]),
                                     _ptr(out["n_drafts"]), _ptr(out["route"]), _ptr(out["rem_rows"]), _ptr(out["rem_off"]),
                                     _ptr(out["v_off"]), _stream())
        _check(rc, "pvf_draft_step")
        return out

    def verify_step(self, params: pvf_params, hidden_v, seg_off, row_pos, draft: Dict[str, torch.Tensor], y=None, out=None):
        """pvf_verify_step: pvf_score on the verification pass + pvf_verify (two launches).  ``draft`` is the
        output of draft_step (or of score + commit_select); ``out`` holds tok_v, conf_v, accept, choice, final_commit."""
        Mv = 0 if hidden_v is None else hidden_v.shape[0]
        M, n_seq, K = draft["commit"].shape[0], seg_off.shape[0] - 1, int(params.budget)
        if out is None:
            dev = self.device
            out = dict(tok_v=torch.empty(max(Mv, 1), dtype=torch.int32, device=dev),
                       conf_v=torch.empty(max(Mv, 1), dtype=torch.float32, device=dev),
                       ent_v=torch.empty(max(Mv, 1), dtype=torch.float32, device=dev),
                       accept=torch.empty((n_seq, K), dtype=torch.uint8, device=dev),
                       choice=torch.empty(n_seq, dtype=torch.int32, device=dev),
                       final_commit=torch.empty(M, dtype=torch.uint8, device=dev))
        L = 0 if y is None else y.shape[1]
        rc = self.lib.pvf_verify_step(self.handle, ctypes.byref(params), _ptr(hidden_v), Mv, M, n_seq, _ptr(seg_off),
                                      _ptr(row_pos), _ptr(draft["rem_rows"]), _ptr(draft["rem_off"]), _ptr(draft["v_off"]),
                                      _ptr(draft["draft_rows"]), _ptr(draft["n_drafts"]), _ptr(draft["route"]),
                                      _ptr(draft["tok"]), _ptr(draft["commit"]), _ptr(out["tok_v"]), _ptr(out["conf_v"]),
                                      _ptr(out.get("ent_v")), _ptr(out["accept"]), _ptr(out["choice"]), _ptr(out["final_commit"]),
                                      _ptr(y), L, _stream())
        _check(rc, "pvf_verify_step")
        return out

    def verify(self, params: pvf_params, seg_off, row_pos, sel: Dict[str, torch.Tensor], tok, tok_v, conf_v,
               commit, y=None, out=None):
        M, n_seq, K = commit.shape[0], seg_off.shape[0] - 1, int(params.budget)
        if out is None:
            dev = self.device
            out = dict(accept=torch.empty((n_seq, K), dtype=torch.uint8, device=dev),
                       choice=torch.empty(n_seq, dtype=torch.int32, device=dev),
                       final_commit=torch.empty(M, dtype=torch.uint8, device=dev))
        L = 0 if y is None else y.shape[1]
        rc = self.lib.pvf_verify(self.handle, ctypes.byref(params), M, n_seq, _ptr(seg_off), _ptr(row_pos),
                                 _ptr(sel["rem_rows"]), _ptr(sel["rem_off"]), _ptr(sel["v_off"]),
                                 _ptr(sel["draft_rows"]), _ptr(sel["n_drafts"]), _ptr(sel["route"]),
                                 _ptr(tok), _ptr(tok_v), _ptr(conf_v), _ptr(commit),
                                 _ptr(out["accept"]), _ptr(out["choice"]), _ptr(out["final_commit"]),
                                 _ptr(y), L, _stream())
        _check(rc, "pvf_verify")
        return out


def host_buffers(M: int, n_seq: int, budget: int, Mv: int = 0, pinned: bool = True) -> Dict[str, torch.Tensor]:
    """Host tensors (pinned by default) for every output of the host-buffer step calls."""
    mk = lambda shape, dt: (torch.empty(shape, dtype=dt).pin_memory() if pinned else torch.empty(shape, dtype=dt))
    return dict(tok=mk(M, torch.int32), conf=mk(M, torch.float32), ent=mk(M, torch.float32), in_plan=mk(M, torch.uint8),
                commit=mk(M, torch.uint8), draft_rows=mk((n_seq, budget), torch.int32), n_drafts=mk(n_seq, torch.int32),
                route=mk(n_seq, torch.uint8), rem_rows=mk(max(M, 1), torch.int32), rem_off=mk(n_seq + 1, torch.int32),
                v_off=mk(n_seq + 1, torch.int32), tok_v=mk(max(Mv, 1), torch.int32), conf_v=mk(max(Mv, 1), torch.float32),
                accept=mk((n_seq, budget), torch.uint8), choice=mk(n_seq, torch.int32), final_commit=mk(M, torch.uint8))


def bf16_from_bits(bits: np.ndarray, device) -> torch.Tensor:
    """uint16 bf16 bit patterns (numpy) -> torch.bfloat16 tensor on `device`."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def score_static(w_head: torch.Tensor, hidden: torch.Tensor, out: Dict[str, torch.Tensor],
                 plan_bitmap: Optional[torch.Tensor] = None) -> int:
    """pvf_score_static: scoring without a context or workspace, for callers that cannot allocate.

    Everything is passed in: ``out`` holds the preallocated tok / conf (and optionally ent, in_plan)
    tensors, ``plan_bitmap`` an optional int32 device tensor of ceil(V/32) words.  Returns the C return
    code (PVF_OK, or e.g. PVF_ERR_TOO_LARGE above PVF_STATIC_MAX_ROWS rows) instead of raising, and
    allocates nothing itself.  Calls that overlap on the GPU race on the library's built-in scratch
    array; make the first call on a device before any stream capture."""
    lib = load()
    V, D = w_head.shape
    return int(lib.pvf_score_static(_ptr(w_head), V, D, _ptr(hidden), hidden.shape[0], _ptr(plan_bitmap),
                                    _ptr(out["tok"]), _ptr(out["conf"]), _ptr(out.get("ent")), _ptr(out.get("in_plan")),
                                    _stream()))


def score_static_status() -> int:
    """Status word of the most recent pvf_score_static call on the current device (synchronises)."""
    st = ctypes.c_int32()
    _check(load().pvf_score_static_status(ctypes.byref(st)), "pvf_score_static_status")
    return int(st.value)
