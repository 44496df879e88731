"""Pins for the brute-force planner oracle: the operation counts and the 4-bit configuration
the paper prints."""
import os

import pytest

from oracle import plan

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows():
    rows = []
    with open(os.path.join(GOLDEN, "ops_per_multiply.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            rows.append(tuple(int(t) for t in line.split()))
    return rows


@pytest.mark.parametrize("LA,LB,p,q,printed", _rows())
def test_printed_ops_per_multiply(LA, LB, p, q, printed):
    best = plan.search(p, q, LA, LB, plan.MODE_SINGLE)
    if (LA, LB, p) == (32, 32, 1):
        # The printed 128 cannot be reached under Eq. 6-8 with Eq. 11: the maximum is 113 at
        # N = K = 8, S = 4.  128 is N = 9, K = 8, S = 4, whose packed A needs 1 + 8*4 = 33 bits.
        assert best["ops"] == 113 and (best["N"], best["K"], best["S"]) == (8, 8, 4)
        relaxed = plan.search(p, q, 33, 32, plan.MODE_SINGLE)
        assert relaxed["ops"] == printed and (relaxed["N"], relaxed["K"], relaxed["S"]) == (9, 8, 4)
        assert not plan.fits(1, 1, 9, 8, 4, 32, 32)
    else:
        assert best["ops"] == printed


def test_printed_splits_of_the_counts():
    # 27x18, 1-bit: N = 9, K = 4 -> 36 multiplications and 24 additions
    best = plan.search(1, 1, 27, 18, plan.MODE_SINGLE)
    assert (best["N"], best["K"]) == (9, 4)
    assert best["N"] * best["K"] == 36 and (best["N"] - 1) * (best["K"] - 1) == 24
    # the text prints S = 4 for this case, but Eq. 6 with Gb = ceil(log2 4) = 2 gives S = 3,
    # and S = 4 would need 1 + 8*4 = 33 > 27 bits
    assert best["S"] == 3 and not plan.fits(1, 1, 9, 4, 4, 27, 18)
    # 27x18, 4-bit: 6 multiplications + 2 additions
    best = plan.search(4, 4, 27, 18, plan.MODE_SINGLE)
    assert best["N"] * best["K"] == 6 and (best["N"] - 1) * (best["K"] - 1) == 2


def test_printed_4bit_1d_configuration():
    vals = {}
    with open(os.path.join(GOLDEN, "config_4bit_1d.txt")) as fh:
        for line in fh:
            if "=" in line and not line.startswith("#"):
                k, v = line.split("=")
                vals[k.strip()] = int(v)
    best = plan.search(vals["p"], vals["q"], vals["LA"], vals["LB"], plan.MODE_1D, K_fixed=vals["K"])
    assert (best["N"], best["K"], best["Gb"], best["S"]) == (vals["N"], vals["K"], vals["Gb"], vals["S"])


def test_guard_bit_rules_and_ops_formula():
    assert plan.guard_bits(plan.MODE_SINGLE, 3, 3) == 2
    assert plan.guard_bits(plan.MODE_SINGLE, 9, 4) == 2
    assert plan.guard_bits(plan.MODE_1D, 100, 5) == 3
    assert plan.guard_bits(plan.MODE_DNN, 3, 3, M=7) == 5          # ceil(log2 21)
    assert plan.slice_bits(1, 4, 2) == 6 and plan.slice_bits(4, 1, 2) == 6 and plan.slice_bits(4, 4, 2) == 10
    # Eq. 24 counts every product and every addition of the full N+K-1 outputs
    for N in range(1, 8):
        for K in range(1, 8):
            mults = N * K
            adds = sum(max(min(m + 1, N, K, N + K - 1 - m) - 1, 0) for m in range(N + K - 1))
            assert plan.ops(N, K) == mults + adds


def test_literal_algorithm1_bounds_do_not_reproduce_the_counts():
    # Algorithm 1 as printed: Max_N = (LA-p)/(p+q)+1, loops with strict "<".  At 1 bit on 27x18 it
    # stops at n < 14, k < 9 with slot p+q+Gb = 4, and finds fewer operations than the printed 60.
    def literal(p, q, LA, LB):
        max_n, max_k = (LA - p) // (p + q) + 1, (LB - q) // (p + q) + 1
        best = 0
        for k in range(1, max_k):
            for n in range(1, max_n):
                S = p + q + plan.guard_bits(plan.MODE_SINGLE, n, k)
                if p + (n - 1) * S <= LA and q + (k - 1) * S <= LB:
                    best = max(best, plan.ops(n, k))
        return best
    assert literal(1, 1, 27, 18) < 60
    assert literal(5, 5, 32, 32) < plan.search(5, 5, 32, 32)["ops"]
