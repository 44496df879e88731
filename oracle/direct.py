"""Plain-definition oracle: ctypes front end of ``hikonv_oracle.c`` (int64, CPU).

Test infrastructure, not product code.  Every function takes integer *values*
(not storage bytes) as numpy arrays, converts them to int64 and evaluates the
textbook definition:

* ``conv1d_full``  - Eq. 2-4, full linear convolution, ``len + K - 1`` outputs.
* ``conv2d_nchw``  - Eq. 16 (cross-correlation, stride 1) on a zero-padded input.
* ``requant``      - ``clamp(floor(acc / 2**shift), lo, hi)``.
* ``maxpool2x2``   - 2x2 window, stride 2.
* ``cnn_forward``  - a chain of the above (conv, requantize, optional pool) plus
                     a final convolution with int64 output.
* ``pack_words``   - Eq. 5, ``A = sum_n f[n] * 2**(S*n)`` reduced modulo the word size.
* ``count_out_of_range`` - how many values lie outside the p-bit code range the paper assumes
                     (``[0, 2**p - 1]`` or ``[-2**(p-1), 2**(p-1) - 1]``, the ranges behind Eq. 6-8).

The C file is compiled on first use with ``gcc -O2 -fopenmp`` into
``oracle/_build/`` (never committed).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hikonv_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "liboracle.so")
_lock = threading.Lock()
_lib = None

_I64P = ctypes.POINTER(ctypes.c_int64)


def build(force: bool = False) -> str:
    """Compile the C oracle if the shared object is missing or older than its source."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    stale = (not os.path.exists(_LIB_PATH)) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC],
            check=True,
        )
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.oracle_num_threads.restype = ctypes.c_int
            lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
            lib.oracle_conv1d_full.argtypes = [_I64P, ctypes.c_int64, _I64P, ctypes.c_int64, _I64P]
            lib.oracle_conv2d_nchw.argtypes = [_I64P] + [ctypes.c_int64] * 4 + [_I64P] + [ctypes.c_int64] * 3 + [_I64P]
            lib.oracle_requant.argtypes = [_I64P] + [ctypes.c_int64] * 4 + [_I64P]
            lib.oracle_maxpool2x2.argtypes = [_I64P] + [ctypes.c_int64] * 3 + [_I64P]
            _lib = lib
    return _lib


def _i64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.int64)


def _p(a: np.ndarray):
    return a.ctypes.data_as(_I64P)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def conv1d_full(f, g) -> np.ndarray:
    """Eq. 2-4: y[m] = sum_k h[m-k] g[k] for m = 0 .. len+K-2 (h = f zero-extended)."""
    f = _i64(f).ravel()
    g = _i64(g).ravel()
    if g.size == 0:
        raise ValueError("kernel must have at least one tap")
    y = np.zeros(max(f.size + g.size - 1, 0), dtype=np.int64)
    if f.size:
        _load().oracle_conv1d_full(_p(f), f.size, _p(g), g.size, _p(y))
    return y


def conv2d_nchw(x, w, pad: int) -> np.ndarray:
    """Eq. 16 on the zero-padded input: stride 1, no kernel flip.  x [B,Ci,H,W], w [Co,Ci,K,K]."""
    x = _i64(x)
    w = _i64(w)
    B, Ci, H, W = x.shape
    Co, Ci2, K, K2 = w.shape
    if Ci != Ci2 or K != K2:
        raise ValueError("shape mismatch")
    Ho, Wo = H + 2 * pad - K + 1, W + 2 * pad - K + 1
    out = np.zeros((B, Co, max(Ho, 0), max(Wo, 0)), dtype=np.int64)
    if out.size:
        _load().oracle_conv2d_nchw(_p(x), B, Ci, H, W, _p(w), Co, K, pad, _p(out))
    return out


def requant(acc, shift: int, lo: int, hi: int) -> np.ndarray:
    """clamp(floor(acc / 2**shift), lo, hi)."""
    acc = _i64(acc)
    out = np.empty_like(acc)
    if acc.size:
        _load().oracle_requant(_p(acc), acc.size, shift, lo, hi, _p(out))
    return out


def maxpool2x2(x) -> np.ndarray:
    """2x2 max-pool with stride 2 over the last two axes of [B,C,H,W]."""
    x = _i64(x)
    B, C, H, W = x.shape
    out = np.empty((B, C, H // 2, W // 2), dtype=np.int64)
    if out.size:
        _load().oracle_maxpool2x2(_p(x), B * C, H, W, _p(out))
    return out


def cnn_forward(x, layers, head_w):
    """Integer CNN: for each layer conv3x3(pad 1) -> requantize -> optional 2x2 pool; then a head conv.

    ``layers`` is a list of dicts ``{"w": [Co,Ci,K,K], "pad": int, "shift": int, "lo": int,
    "hi": int, "pool": bool}``; ``head_w`` is ``[Co,Ci,K,K]`` (pad 0).  Returns the int64 head
    output and the list of per-layer activations (after requantize/pool) for inspection.
    """
    acts = []
    a = _i64(x)
    for L in layers:
        a = conv2d_nchw(a, L["w"], L["pad"])
        a = requant(a, L["shift"], L["lo"], L["hi"])
        if L["pool"]:
            a = maxpool2x2(a)
        acts.append(a)
    return conv2d_nchw(a, head_w, 0), acts


def pack_words(values, S: int, N: int, word_bits: int) -> np.ndarray:
    """Eq. 5: word[x] = sum_{n<N} values[x*N+n] * 2**(S*n), taken modulo 2**word_bits.

    The input is zero-extended to a multiple of N.  Negative values enter as
    themselves, so the word is the two's-complement image of the integer sum.
    Returned as uint64.
    """
    if word_bits not in (32, 64):
        raise ValueError("word_bits must be 32 or 64")
    v = _i64(values).ravel()
    n_words = (v.size + N - 1) // N
    padded = np.zeros(n_words * N, dtype=np.int64)
    padded[: v.size] = v
    padded = padded.reshape(n_words, N)
    words = np.zeros(n_words, dtype=np.uint64)
    with np.errstate(over="ignore"):
        for n in range(N):
            sh = S * n
            if sh >= 64:
                continue  # 2**sh vanishes modulo 2**64
            words += padded[:, n].astype(np.uint64) << np.uint64(sh)
    if word_bits == 32:
        words &= np.uint64(0xFFFFFFFF)
    return words


def count_out_of_range(values, bits: int, signed: bool) -> int:
    """Number of values outside the p-bit code range (Section IV-A: p-bit unsigned or two's-complement inputs)."""
    v = _i64(values).ravel()
    lo, hi = (-(1 << (bits - 1)), (1 << (bits - 1)) - 1) if signed else (0, (1 << bits) - 1)
    return int(np.count_nonzero((v < lo) | (v > hi)))
