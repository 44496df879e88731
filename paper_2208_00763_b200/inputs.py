"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no convolution, packing or planning arithmetic: it only draws
integer codes with ``numpy.random.default_rng(seed)`` and converts between code
values and their int8 storage.  Both the CPU oracle (through the tests) and the
CUDA path are fed from here, so the two sides see the same buffers.

The paper evaluates on randomly generated feature and kernel vectors (1-D sweep
over bitwidths 1-8, a 4-bit layer, a full 4-bit CNN on camera frames); its
vector lengths, trained weights and images are not available, so uniform codes
of the stated bitwidth stand in for them.
"""
from __future__ import annotations

from typing import Dict, List, Tuple

import numpy as np


def code_range(bits: int, signed: bool) -> Tuple[int, int]:
    """Inclusive range of a ``bits``-wide code: [0, 2^b - 1] or [-2^(b-1), 2^(b-1) - 1]."""
    if signed:
        return -(1 << (bits - 1)), (1 << (bits - 1)) - 1
    return 0, (1 << bits) - 1


def uniform_codes(rng: np.random.Generator, shape, bits: int, signed: bool) -> np.ndarray:
    lo, hi = code_range(bits, signed)
    return rng.integers(lo, hi + 1, size=shape, dtype=np.int64)


def to_storage(values: np.ndarray) -> np.ndarray:
    """Code values -> the int8 bytes the library reads (unsigned 8-bit codes wrap into int8)."""
    v = np.asarray(values)
    if v.min(initial=0) < -128 or v.max(initial=0) > 255:
        raise ValueError("code does not fit one byte")
    return np.ascontiguousarray(v.astype(np.int64) & 0xFF).astype(np.uint8).view(np.int8)


def to_dense(values: np.ndarray, bits: int) -> np.ndarray:
    """Code values -> dense storage: 8 / bits codes per byte, code e at bit (e * bits) % 8 of byte
    (e * bits) // 8, two's complement for negative codes.  bits must divide 8."""
    if bits not in (1, 2, 4, 8):
        raise ValueError("bits must divide 8")
    v = np.asarray(values).astype(np.int64).ravel() & ((1 << bits) - 1)
    per = 8 // bits
    pad = (-v.size) % per
    v = np.concatenate([v, np.zeros(pad, dtype=np.int64)]).reshape(-1, per)
    shifts = (np.arange(per) * bits).astype(np.int64)
    return np.ascontiguousarray((v << shifts).sum(axis=1).astype(np.uint8))


def from_dense(dense: np.ndarray, count: int, bits: int, signed: bool) -> np.ndarray:
    """Dense storage -> the first ``count`` code values (the inverse of ``to_dense``)."""
    if bits not in (1, 2, 4, 8):
        raise ValueError("bits must divide 8")
    per = 8 // bits
    b = np.asarray(dense, dtype=np.uint8).astype(np.int64)
    shifts = (np.arange(per) * bits).astype(np.int64)
    v = ((b[:, None] >> shifts) & ((1 << bits) - 1)).reshape(-1)[:count]
    if signed:
        v = np.where(v >= (1 << (bits - 1)), v - (1 << bits), v)
    return v


def from_storage(stored: np.ndarray, signed: bool) -> np.ndarray:
    """int8 storage bytes -> code values as int64."""
    s = np.asarray(stored)
    if signed:
        return s.view(np.int8).astype(np.int64)
    return s.view(np.uint8).astype(np.int64)


# ----------------------------------------------------------------------------
# 1-D workloads
# ----------------------------------------------------------------------------

def conv1d_case(length: int, K: int, p: int, q: int, f_signed: bool, g_signed: bool, seed: int):
    rng = np.random.default_rng(seed)
    f = uniform_codes(rng, (length,), p, f_signed)
    g = uniform_codes(rng, (K,), q, g_signed)
    return f, g


def c1():
    """Single channel, unsigned 4-bit, length 4096, K = 3, seed 0."""
    return conv1d_case(4096, 3, 4, 4, False, False, 0)


def c2_cases(length: int = 1 << 24) -> List[Dict]:
    """The bitwidth sweep: p = q in 1..8, K in {3,5,7}, unsigned and signed: 48 cases."""
    cases = []
    for bits in range(1, 9):
        for K in (3, 5, 7):
            for signed in (False, True):
                cases.append({
                    "length": length, "K": K, "p": bits, "q": bits,
                    "f_signed": signed, "g_signed": signed,
                    "seed": 1000 + 100 * bits + 10 * K + int(signed),
                })
    return cases


def extreme_1d(length: int, K: int, p: int, q: int, f_signed: bool, g_signed: bool):
    """Inputs that stress the guard bits: every combination of all-min / all-max codes, and an
    alternating min/max pattern."""
    flo, fhi = code_range(p, f_signed)
    glo, ghi = code_range(q, g_signed)
    out = []
    for fv in (flo, fhi):
        for gv in (glo, ghi):
            out.append((np.full(length, fv, dtype=np.int64), np.full(K, gv, dtype=np.int64)))
    alt_f = np.where(np.arange(length) % 2 == 0, flo, fhi).astype(np.int64)
    alt_g = np.where(np.arange(K) % 2 == 0, ghi, glo).astype(np.int64)
    out.append((alt_f, alt_g))
    return out


# ----------------------------------------------------------------------------
# 2-D workloads
# ----------------------------------------------------------------------------

def conv2d_case(B, Ci, H, W, Co, K, p, q, x_signed, w_signed, seed, zero_frac: float = 0.0):
    rng = np.random.default_rng(seed)
    x = uniform_codes(rng, (B, Ci, H, W), p, x_signed)
    if zero_frac > 0.0:
        x = np.where(rng.random(x.shape) < zero_frac, 0, x)
    w = uniform_codes(rng, (Co, Ci, K, K), q, w_signed)
    return x, w


C3_SHAPE = dict(B=32, Ci=64, H=56, W=56, Co=64, K=3, pad=1, p=4, q=4, x_signed=True, w_signed=True,
                requant=True, shift=6, lo=-8, hi=7, seed=3, zero_frac=0.0)
C4_SHAPE = dict(B=64, Ci=256, H=14, W=14, Co=256, K=3, pad=1, p=4, q=4, x_signed=False, w_signed=True,
                requant=False, shift=0, lo=0, hi=0, seed=4, zero_frac=0.3)


def layer_case(shape: Dict, batch: int | None = None):
    """Inputs for a 2-D layer description such as ``C3_SHAPE``; ``batch`` overrides B."""
    B = shape["B"] if batch is None else batch
    return conv2d_case(B, shape["Ci"], shape["H"], shape["W"], shape["Co"], shape["K"], shape["p"],
                       shape["q"], shape["x_signed"], shape["w_signed"], shape["seed"],
                       shape.get("zero_frac", 0.0))


def extreme_2d(B, Ci, H, W, Co, K, p, q, x_signed, w_signed):
    xlo, xhi = code_range(p, x_signed)
    wlo, whi = code_range(q, w_signed)
    out = []
    for xv in (xlo, xhi):
        for wv in (wlo, whi):
            out.append((np.full((B, Ci, H, W), xv, dtype=np.int64),
                        np.full((Co, Ci, K, K), wv, dtype=np.int64)))
    idx = np.indices((B, Ci, H, W)).sum(axis=0)
    widx = np.indices((Co, Ci, K, K)).sum(axis=0)
    out.append((np.where(idx % 2 == 0, xlo, xhi).astype(np.int64),
                np.where(widx % 2 == 0, whi, wlo).astype(np.int64)))
    return out


# ----------------------------------------------------------------------------
# Compact 4-bit CNN (8 conv3x3 layers, pools after the first four, 1x1 head)
# ----------------------------------------------------------------------------

C5_CHANNELS = [3, 16, 32, 64, 64, 64, 64, 64, 64]
C5_POOL = [True, True, True, True, False, False, False, False]
# Per-layer right shifts.  The paper gives none (it has no requantisation); these keep the
# 4-bit codes of uniform random data spread over [0, 15] instead of saturating.
C5_SHIFTS = [8, 5, 6, 6, 6, 6, 6, 6]
C5_HEAD_CHANNELS = 36


def c5_network(seed: int = 5, batch: int = 64, H: int = 160, W: int = 320):
    """Input image batch (8-bit unsigned) and 4-bit signed weights for the compact CNN."""
    rng = np.random.default_rng(seed)
    x = uniform_codes(rng, (batch, C5_CHANNELS[0], H, W), 8, False)
    layers = []
    for i in range(8):
        w = uniform_codes(rng, (C5_CHANNELS[i + 1], C5_CHANNELS[i], 3, 3), 4, True)
        layers.append({"w": w, "pad": 1, "shift": C5_SHIFTS[i], "lo": 0, "hi": 15,
                       "pool": C5_POOL[i], "p": 8 if i == 0 else 4, "q": 4,
                       "x_signed": False, "w_signed": True})
    head_w = uniform_codes(rng, (C5_HEAD_CHANNELS, C5_CHANNELS[-1], 1, 1), 4, True)
    return x, layers, head_w
