"""The paper's CPU method (Algorithm 2, Section V-A) in plain C, with its plain front end.

Test and measurement infrastructure, not product code: a second, independent CPU implementation that
follows the method's own steps (pack, one multiplication per block, add the carried product, split),
checked against the plain definition in ``tests/`` and timed beside it by ``bench.py``'s CPU leg, which
restates the paper's CPU experiment (Section VI-A) on this host.  Layouts come from ``oracle.plan``
(Eq. 6-8 with the 1-D guard-bit rule), narrowed by an exact range check of the packed operands
where Eq. 7 holds with equality for signed values.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Optional

import numpy as np

from . import plan

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hikonv_alg2.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "libalg2.so")
_lock = threading.Lock()
_lib = None
_I64P = ctypes.POINTER(ctypes.c_int64)


def build(force: bool = False) -> str:
    os.makedirs(_OUT_DIR, exist_ok=True)
    stale = (not os.path.exists(_LIB_PATH)) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.alg2_conv1d.argtypes = [_I64P, ctypes.c_int64, _I64P, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_int, _I64P]
            lib.alg2_conv1d.restype = ctypes.c_int
            _lib = lib
    return _lib


def layout(p: int, q: int, K: int, signed: bool) -> Optional[dict]:
    """(N, S) for a 32x32 multiplier and a K-tap kernel held in one word, or None when none fits."""
    best = plan.search(p, q, 32, 32, plan.MODE_1D, K_fixed=K)
    N, S = best["N"], best["S"]
    if N < 1:
        return None
    if signed:
        # exact operand range: the all-minimum block must not leave int32
        while N >= 1 and sum((1 << (p - 1)) << (S * n) for n in range(N)) > (1 << 31):
            N -= 1
        if sum((1 << (q - 1)) << (S * k) for k in range(K)) > (1 << 31) or N < 1:
            return None
    if S * (N + K - 1) > 64:
        return None
    return {"N": N, "S": S, "Gb": best["Gb"]}


def conv1d_full(f, g, p: int, q: int, signed: bool, threads: int = 0) -> np.ndarray:
    f = np.ascontiguousarray(f, dtype=np.int64)
    g = np.ascontiguousarray(g, dtype=np.int64)
    lay = layout(p, q, int(g.size), signed)
    if lay is None:
        raise ValueError("no packed layout fits a 32x32 multiplier for p=%d q=%d K=%d" % (p, q, g.size))
    y = np.empty(f.size + g.size - 1, dtype=np.int64)
    rc = _load().alg2_conv1d(f.ctypes.data_as(_I64P), f.size, g.ctypes.data_as(_I64P), int(g.size), lay["S"], lay["N"],
                             int(bool(signed)), int(threads), y.ctypes.data_as(_I64P))
    if rc != 0:
        raise ValueError("layout rejected by the C routine")
    return y
