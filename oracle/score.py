"""ctypes wrapper around the fp64 scoring oracle (pvf_oracle_score.c).  Test infrastructure only."""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pvf_oracle_score.c")
_LIB = os.path.join(_HERE, "libpvf_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle (gcc, OpenMP).  Rebuilds when the source is newer than the library."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u16p = ctypes.POINTER(ctypes.c_uint16)
        lib.pvf_oracle_score.restype = ctypes.c_int
        lib.pvf_oracle_score.argtypes = [u16p, u16p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                         ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                         ctypes.c_void_p]
        lib.pvf_oracle_row_stats.restype = None
        lib.pvf_oracle_row_stats.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p,
                                             ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.pvf_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().pvf_oracle_threads())


def plan_membership(plan_ids: np.ndarray, vocab: int) -> np.ndarray:
    member = np.zeros(vocab, dtype=np.uint8)
    member[np.asarray(plan_ids, dtype=np.int64)] = 1
    return member


def score(w_bits: np.ndarray, h_bits: np.ndarray, plan_ids: Optional[np.ndarray] = None,
          want_logits: bool = False) -> Dict[str, np.ndarray]:
    """Score every row of ``h_bits`` ([M][D] bf16 bit patterns) against ``w_bits`` ([V][D]).

    Returns tok (int32), conf, ent, gap (float64), in_plan (uint8) and optionally logits [M][V].
    """
    lib = _load()
    w = np.ascontiguousarray(w_bits, dtype=np.uint16)
    h = np.ascontiguousarray(h_bits, dtype=np.uint16)
    V, D = w.shape
    M = h.shape[0]
    assert h.ndim == 2 and (M == 0 or h.shape[1] == D)
    tok = np.zeros(M, dtype=np.int32)
    conf = np.zeros(M, dtype=np.float64)
    ent = np.zeros(M, dtype=np.float64)
    gap = np.zeros(M, dtype=np.float64)
    in_plan = np.zeros(M, dtype=np.uint8)
    member = plan_membership(plan_ids, V) if plan_ids is not None else None
    logits = np.zeros((M, V), dtype=np.float64) if want_logits else None
    u16p = ctypes.POINTER(ctypes.c_uint16)
    rc = lib.pvf_oracle_score(w.ctypes.data_as(u16p), h.ctypes.data_as(u16p), M, V, D,
                              member.ctypes.data if member is not None else None,
                              tok.ctypes.data, conf.ctypes.data, ent.ctypes.data, gap.ctypes.data,
                              in_plan.ctypes.data, logits.ctypes.data if logits is not None else None)
    if rc != 0:
        raise RuntimeError("pvf_oracle_score failed: %d" % rc)
    out = dict(tok=tok, conf=conf, ent=ent, gap=gap, in_plan=in_plan)
    if logits is not None:
        out["logits"] = logits
    return out


def row_stats(x: np.ndarray):
    """Softmax statistics of one fp64 logit row: (tok, conf, ent, gap)."""
    lib = _load()
    x = np.ascontiguousarray(x, dtype=np.float64)
    tok = ctypes.c_int32()
    conf, ent, gap = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
    lib.pvf_oracle_row_stats(x.ctypes.data, x.shape[0], ctypes.byref(tok), ctypes.byref(conf),
                             ctypes.byref(ent), ctypes.byref(gap))
    return int(tok.value), float(conf.value), float(ent.value), float(gap.value)
