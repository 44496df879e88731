"""The packed-multiply method in Python big integers (test infrastructure only).

This follows the paper's steps in the paper's order and notation, for small
inputs, so that the identities the GPU path relies on can be checked against
the plain definitions in ``oracle.direct`` and against the printed example:

* Eq. 5     pack:   A = sum_n f[n] 2^(S n),  B = sum_k g[k] 2^(S k)
* Eq. 9-10  one multiply:  Prod = A * B = sum_m y[m] 2^(S m),  m = 0 .. N+K-2
* Eq. 28    signed slot contents:  slot_n = f[n] - A[S n - 1]
* Eq. 29    signed split:  y[m] = Prod[S(m+1)-1 : S m] + Prod[S m - 1]
* Theorem 2 overlap-add of blocks:  y[n] = sum_x y_x[n - x N]
* Theorem 3 a conv layer as row-wise 1-D convolutions with the reversed kernel
            row, read at index w + K - 1, products of all (ci, kh) summed
            before the split (the DNN guard-bit rule).

Python integers are unbounded, so "the multiplier" here is exact; the operand
widths are checked separately by ``oracle.plan``.
"""
from __future__ import annotations

from typing import List, Sequence


def pack(vals: Sequence[int], S: int) -> int:
    """Eq. 5 as an exact integer (negative when the top element is negative)."""
    return sum(int(v) << (S * n) for n, v in enumerate(vals))


def to_word(a: int, bits: int) -> int:
    """Two's-complement image of ``a`` in a ``bits``-wide register."""
    return a & ((1 << bits) - 1)


def from_word(u: int, bits: int) -> int:
    """Signed value of a ``bits``-wide register image."""
    u &= (1 << bits) - 1
    return u - (1 << bits) if u >> (bits - 1) else u


def pack_signed_fields(vals: Sequence[int], S: int, bits: int) -> int:
    """Eq. 28: build the word slot by slot, slot n = f[n] - (bit S n - 1 of what is below)."""
    word = 0
    for n, v in enumerate(vals):
        borrow = (word >> (S * n - 1)) & 1 if n > 0 else 0
        field = (int(v) - borrow) & ((1 << S) - 1)
        word |= field << (S * n)
    # the slots above the last element hold the sign extension of the last slot
    top = S * len(vals)
    if top < bits and len(vals) > 0 and (word >> (top - 1)) & 1:
        word |= ((1 << bits) - 1) ^ ((1 << top) - 1)
    return word & ((1 << bits) - 1)


def split_unsigned(prod: int, S: int, count: int) -> List[int]:
    """Algorithm 2's unsigned split: shift and mask."""
    mask = (1 << S) - 1
    return [(prod >> (S * m)) & mask for m in range(count)]


def split_signed(prod: int, S: int, count: int) -> List[int]:
    """Eq. 29: S-bit field plus the bit just below it, read as an S-bit signed number."""
    mask = (1 << S) - 1
    out = []
    for m in range(count):
        field = (prod >> (S * m)) & mask
        below = (prod >> (S * m - 1)) & 1 if m > 0 else 0
        v = (field + below) & mask
        out.append(v - (1 << S) if v >> (S - 1) else v)
    return out


def f_nk(f: Sequence[int], g: Sequence[int], S: int, signed: bool) -> List[int]:
    """Theorem 1: the N+K-1 outputs of F_{N,K}(f, g) from one multiplication."""
    prod = pack(f, S) * pack(g, S)
    count = len(f) + len(g) - 1
    return split_signed(prod, S, count) if signed else split_unsigned(prod, S, count)


def conv1d_blocks(f: Sequence[int], g: Sequence[int], N: int, S: int, signed: bool) -> List[int]:
    """Theorem 2: cut f into N-element blocks, run F_{N,K} on each, add the index-shifted outputs."""
    f = list(f)
    K = len(g)
    X = (len(f) + N - 1) // N
    f = f + [0] * (X * N - len(f))
    y = [0] * (X * N + K - 1)
    for x in range(X):
        yx = f_nk(f[x * N:(x + 1) * N], g, S, signed)
        for i, v in enumerate(yx):
            y[x * N + i] += v
    return y


def conv1d_carry(f: Sequence[int], g: Sequence[int], N: int, S: int, signed: bool) -> List[int]:
    """Theorem 2 with the overlap-add done on the products, before the split.

    Block x's product P_x is added to what block x-1 left above its N low
    segments (the "previous product shifted right, current one aligned" step of
    Section V-A), then the N low segments are split off.  Segment m of the sum
    then holds a complete output with K terms, which is why the 1-D guard-bit
    rule is ceil(log2 K).
    """
    f = list(f)
    K = len(g)
    X = (len(f) + N - 1) // N
    f = f + [0] * (X * N - len(f))
    B = pack(g, S)
    y: List[int] = []
    carry = 0
    for x in range(X):
        C = pack(f[x * N:(x + 1) * N], S) * B + carry
        seg = split_signed(C, S, N) if signed else split_unsigned(C, S, N)
        y.extend(seg)
        low = sum(v << (S * m) for m, v in enumerate(seg))
        carry = (C - low) >> (S * N)      # exact: C - low is a multiple of 2^(S N)
    tail = split_signed(carry, S, K - 1) if signed else split_unsigned(carry, S, K - 1)
    return y + tail


def conv2d_rows(x, w, pad: int, N: int, S: int, signed: bool):
    """Theorem 3: O[co][h][w] = sum_{ci,kh} y_{ci,co,h,kh}[w + K - 1].

    ``x`` is [Ci][H][W] (one image), ``w`` is [Co][Ci][K][K], both nested lists of
    ints.  Each padded input row is cut into N-element blocks; for every block the
    products with the reversed kernel rows of all (ci, kh) are summed first
    (Eq. 23's accumulation before the split), then overlap-added and split.
    Returns [Co][Ho][Wo].
    """
    Ci, H, W = len(x), len(x[0]), len(x[0][0])
    Co, K = len(w), len(w[0][0])
    Hp, Wp = H + 2 * pad, W + 2 * pad
    Ho, Wo = Hp - K + 1, Wp - K + 1

    def prow(ci, r):  # zero-padded row r of channel ci (Eq. 19)
        rr = r - pad
        if rr < 0 or rr >= H:
            return [0] * Wp
        return [0] * pad + list(x[ci][rr]) + [0] * pad

    X = (Wp + N - 1) // N
    out = [[[0] * Wo for _ in range(Ho)] for _ in range(Co)]
    for co in range(Co):
        for h in range(Ho):
            # accumulate the per-block products over ci and kh
            acc = [0] * X
            for ci in range(Ci):
                for kh in range(K):
                    row = prow(ci, h + kh)
                    row = row + [0] * (X * N - Wp)
                    B = pack(list(reversed(w[co][ci][kh])), S)      # g = W[co][ci][kh][K-1:0]
                    for xb in range(X):
                        acc[xb] += pack(row[xb * N:(xb + 1) * N], S) * B
            # overlap-add across blocks on the accumulated products, then split
            y: List[int] = []
            carry = 0
            for xb in range(X):
                C = acc[xb] + carry
                seg = split_signed(C, S, N) if signed else split_unsigned(C, S, N)
                y.extend(seg)
                low = sum(v << (S * m) for m, v in enumerate(seg))
                carry = (C - low) >> (S * N)
            y += split_signed(carry, S, K - 1) if signed else split_unsigned(carry, S, K - 1)
            for ww in range(Wo):
                out[co][h][ww] = y[ww + K - 1]                       # Eq. 17
    return out
