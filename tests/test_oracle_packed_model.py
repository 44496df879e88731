"""Pins for the big-integer model of the packed method (CPU only).

The model restates Eq. 5, Theorem 1-3, Eq. 28 and Eq. 29.  It is checked against the
paper's printed numbers and against the plain-definition oracle, which is pinned on
its own in ``test_oracle_direct.py``.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import direct, packed_model as pm, plan

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#") or "=" not in line:
                continue
            k, v = line.split("=", 1)
            vals[k.strip()] = v.strip()
    return vals


def test_printed_example_words_and_product():
    g = _golden("worked_example_f32.txt")
    f = [int(t) for t in g["f"].split()]
    k = [int(t) for t in g["g"].split()]
    y = [int(t) for t in g["y"].split()]
    S = int(g["S"])
    # the figure stores the first element in the top slot: mirror the sequences, then Eq. 5
    A = pm.pack(f[::-1], S)
    B = pm.pack(k[::-1], S)
    assert A == int(g["multiplicand_f"])
    assert B == int(g["multiplicand_g"])
    assert A * B == int(g["product"])
    assert bin(A * B)[2:] == g["product_binary"]
    # mirrored packing mirrors the segments: the outputs come out high slot first
    assert pm.split_unsigned(A * B, S, 4) == y[::-1]
    # Eq. 5 order (first element in the lowest slot) gives them low slot first
    assert pm.f_nk(f, k, S, signed=False) == y


def test_multichannel_int4_identity():
    # Eq. 1: (V2 2^11 + V1)(W2 2^22 + W1) = V2W2 2^33 + V1W2 2^22 + V2W1 2^11 + V1W1
    rng = np.random.default_rng(1)
    for _ in range(200):
        v1, v2 = (int(t) for t in rng.integers(0, 16, 2))       # unsigned 4-bit
        w1, w2 = (int(t) for t in rng.integers(-8, 8, 2))       # signed 4-bit
        prod = (v2 * 2 ** 11 + v1) * (w2 * 2 ** 22 + w1)
        assert prod == v2 * w2 * 2 ** 33 + v1 * w2 * 2 ** 22 + v2 * w1 * 2 ** 11 + v1 * w1
        assert pm.split_signed(prod, 11, 4) == [v1 * w1, v2 * w1, v1 * w2, v2 * w2]


def _codes(rng, n, bits, signed):
    lo, hi = (-(1 << (bits - 1)), 1 << (bits - 1)) if signed else (0, 1 << bits)
    return [int(t) for t in rng.integers(lo, hi, n)]


def _slot(p, q, signed_f, signed_g, terms):
    """Smallest slot that holds `terms` products exactly, with the symmetric signed range Eq. 29 needs."""
    flo, fhi = (-(1 << (p - 1)), (1 << (p - 1)) - 1) if signed_f else (0, (1 << p) - 1)
    glo, ghi = (-(1 << (q - 1)), (1 << (q - 1)) - 1) if signed_g else (0, (1 << q) - 1)
    prods = [a * b for a in (flo, fhi) for b in (glo, ghi)]
    lo, hi = terms * min(prods), terms * max(prods)
    S = 1
    if signed_f or signed_g:
        while not (-(1 << (S - 1)) + 1 <= lo and hi <= (1 << (S - 1)) - 1):
            S += 1
    else:
        while hi > (1 << S) - 1:
            S += 1
    return S


@pytest.mark.parametrize("signed", [False, True])
def test_theorem1_single_multiplication(signed):
    rng = np.random.default_rng(2 + signed)
    for _ in range(300):
        p, q = int(rng.integers(1, 9)), int(rng.integers(1, 9))
        N, K = int(rng.integers(1, 7)), int(rng.integers(1, 7))
        S = _slot(p, q, signed, signed, min(N, K))
        f, g = _codes(rng, N, p, signed), _codes(rng, K, q, signed)
        assert pm.f_nk(f, g, S, signed) == direct.conv1d_full(f, g).tolist()


def test_paper_slot_width_is_enough_unsigned():
    # Eq. 6 with Eq. 11 guard bits holds the extreme unsigned products for every p, q, N, K that fit 32x32
    for p in range(1, 9):
        for q in range(1, 9):
            for N in range(1, 9):
                for K in range(1, 9):
                    S = plan.slice_bits(p, q, plan.guard_bits(plan.MODE_SINGLE, N, K))
                    if not plan.fits(p, q, N, K, S, 32, 32):
                        continue
                    f, g = [(1 << p) - 1] * N, [(1 << q) - 1] * K
                    assert pm.f_nk(f, g, S, False) == direct.conv1d_full(f, g).tolist()


@pytest.mark.parametrize("signed", [False, True])
def test_theorem2_overlap_add(signed):
    rng = np.random.default_rng(4 + signed)
    for _ in range(200):
        p, q = int(rng.integers(1, 9)), int(rng.integers(1, 9))
        N, K = int(rng.integers(1, 6)), int(rng.integers(1, 6))
        n = int(rng.integers(1, 40))
        f, g = _codes(rng, n, p, signed), _codes(rng, K, q, signed)
        ref = direct.conv1d_full(f, g).tolist()
        # split-then-add needs min(N, K) terms per slot, add-then-split needs K terms
        y1 = pm.conv1d_blocks(f, g, N, _slot(p, q, signed, signed, min(N, K)), signed)
        y2 = pm.conv1d_carry(f, g, N, _slot(p, q, signed, signed, K), signed)
        assert y1[:len(ref)] == ref and not any(y1[len(ref):])
        assert y2[:len(ref)] == ref and not any(y2[len(ref):])


def test_theorem2_extreme_codes():
    for p in range(1, 9):
        for signed in (False, True):
            lo, hi = (-(1 << (p - 1)), (1 << (p - 1)) - 1) if signed else (0, (1 << p) - 1)
            for K in (3, 5, 7):
                N = 3
                S = _slot(p, p, signed, signed, K)
                for fv, gv in itertools.product((lo, hi), repeat=2):
                    f, g = [fv] * 11, [gv] * K
                    ref = direct.conv1d_full(f, g).tolist()
                    assert pm.conv1d_carry(f, g, N, S, signed)[:len(ref)] == ref


def test_exhaustive_tiny_signed_split():
    # every signed 2-bit F_{2,2}: Eq. 29 recovers every output
    S = _slot(2, 2, True, True, 2)
    for f in itertools.product(range(-2, 2), repeat=2):
        for g in itertools.product(range(-2, 2), repeat=2):
            assert pm.f_nk(f, g, S, True) == direct.conv1d_full(f, g).tolist()


def test_signed_pack_decrementer_form():
    # Eq. 28 builds the same register image as the two's-complement sum of Eq. 5
    rng = np.random.default_rng(8)
    for _ in range(300):
        p = int(rng.integers(1, 9))
        S = p + int(rng.integers(1, 10))        # a slot is always wider than the code (S >= p + q)
        N = max(1, min(int(rng.integers(1, 6)), (32 - p) // S + 1))
        f = _codes(rng, N, p, True)
        assert pm.pack_signed_fields(f, S, 32) == pm.to_word(pm.pack(f, S), 32)
        if -(1 << 31) <= pm.pack(f, S) < (1 << 31):
            assert pm.from_word(pm.to_word(pm.pack(f, S), 32), 32) == pm.pack(f, S)


def test_eq7_boundary_case_for_signed_operands():
    # Eq. 7 admits p + (N-1) S = L_A exactly.  For signed codes the top slot then has to hold
    # f[N-1] minus the borrow of the slots below it, one value more than p bits can take:
    # the all-minimum operand no longer fits the register, so a planner has to test the exact
    # operand range instead of Eq. 7 alone.
    p, S, N, L = 2, 10, 4, 32
    assert p + (N - 1) * S == L
    worst = pm.pack([-1, -1, -1, -2], S)
    assert worst < -(1 << (L - 1))
    assert pm.from_word(pm.to_word(worst, L), L) != worst
    # one bit of slack is enough
    assert -(1 << (L - 1)) <= pm.pack([-2, -2, -2], S) and pm.pack([1, 1, 1], S) < (1 << (L - 1))


@pytest.mark.parametrize("signed_x,signed_w", [(False, False), (True, True), (False, True)])
def test_theorem3_layer(signed_x, signed_w):
    rng = np.random.default_rng(20 + 2 * signed_x + signed_w)
    for (Ci, H, W, Co, K, pad, N) in ((3, 5, 7, 2, 3, 1, 3), (2, 4, 6, 3, 3, 0, 2), (4, 3, 5, 2, 1, 0, 4),
                                      (2, 6, 6, 2, 5, 2, 3)):
        p, q = 4, 4
        x = np.array(_codes(rng, Ci * H * W, p, signed_x)).reshape(Ci, H, W)
        w = np.array(_codes(rng, Co * Ci * K * K, q, signed_w)).reshape(Co, Ci, K, K)
        S = _slot(p, q, signed_x, signed_w, Ci * K * K)          # M = Ci*K products per slot, K terms each
        got = pm.conv2d_rows(x.tolist(), w.tolist(), pad, N, S, signed_x or signed_w)
        ref = direct.conv2d_nchw(x[None], w, pad)[0]
        assert np.array_equal(np.array(got), ref)
