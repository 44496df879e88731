"""Slot-width rule, operand-fit constraints, guard bits and the throughput search
(Eq. 6-8, Eq. 11, the 1-D and DNN guard-bit rules, Eq. 24-26, Algorithm 1), by
brute force in Python.  Test infrastructure only.

Readings taken where the printed text is loose:

* Algorithm 1 prints strict "<" loop bounds derived from (L - p)/(p + q) + 1 and
  writes "p + q + G_b" inside the two conditions.  Taken literally it cannot
  return the operation counts the paper itself prints (13 at 4 bits on a
  32x32 multiplier, 60 at 1 bit on a 27x18 multiplier).  Here the search runs
  over every n in 1..L_A and k in 1..L_B and the conditions use the slot width
  S of Eq. 6, which reproduces the printed counts.
* G_b depends on min(K, N), which depends on S, which depends on G_b: it is
  evaluated per candidate pair (n, k), as the algorithm's loop body does.
"""
from __future__ import annotations

from typing import Dict, Optional

MODE_SINGLE = 0   # Eq. 11:  ceil(log2 min(K, N))
MODE_1D = 1       # 1-D extension:  ceil(log2 K)
MODE_DNN = 2      # DNN extension:  ceil(log2(M * min(K, N)))


def ceil_log2(v: int) -> int:
    if v < 1:
        raise ValueError("log2 of a non-positive number")
    return (v - 1).bit_length()


def guard_bits(mode: int, N: int, K: int, M: int = 1) -> int:
    if mode == MODE_SINGLE:
        return ceil_log2(min(K, N))
    if mode == MODE_1D:
        return ceil_log2(K)
    if mode == MODE_DNN:
        return ceil_log2(M * min(K, N))
    raise ValueError("unknown guard-bit mode")


def slice_bits(p: int, q: int, Gb: int) -> int:
    """Eq. 6."""
    if p == 1:
        return q + Gb
    if q == 1:
        return p + Gb
    return p + q + Gb


def fits(p: int, q: int, N: int, K: int, S: int, LA: int, LB: int) -> bool:
    """Eq. 7 and Eq. 8."""
    return p + (N - 1) * S <= LA and q + (K - 1) * S <= LB


def ops(N: int, K: int) -> int:
    """Eq. 24: N K multiplications plus (N-1)(K-1) additions."""
    return N * K + (N - 1) * (K - 1)


def search(p: int, q: int, LA: int, LB: int, mode: int = MODE_SINGLE, M: int = 1,
           K_fixed: Optional[int] = None) -> Dict[str, int]:
    """Algorithm 1: the (N, K) pair with the most operations per multiplication.

    With ``K_fixed`` the kernel length is given (the 1-D / DNN use) and only N is searched.
    Ties keep the first pair found with k ascending, n ascending.
    """
    best = {"N": 0, "K": 0, "S": 0, "Gb": 0, "ops": 0}
    ks = range(1, LB + 1) if K_fixed is None else [K_fixed]
    for k in ks:
        for n in range(1, LA + 1):
            Gb = guard_bits(mode, n, k, M)
            S = slice_bits(p, q, Gb)
            if not fits(p, q, n, k, S, LA, LB):
                continue
            cur = ops(n, k)
            if cur > best["ops"]:
                best = {"N": n, "K": k, "S": S, "Gb": Gb, "ops": cur}
    return best
