"""The C restatement of the paper's CPU loop (Algorithm 2) against the plain definition (CPU only)."""
import numpy as np
import pytest

from oracle import algorithm2, direct, packed_model as pm


def _codes(rng, n, bits, signed):
    lo, hi = (-(1 << (bits - 1)), 1 << (bits - 1)) if signed else (0, 1 << bits)
    return rng.integers(lo, hi, n)


def test_printed_configuration():
    # the 4-bit configuration of the CPU evaluation: N = 3, K = 3, Gb = 2, S = 10
    lay = algorithm2.layout(4, 4, 3, False)
    assert (lay["N"], lay["S"], lay["Gb"]) == (3, 10, 2)


@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("bits", range(1, 9))
@pytest.mark.parametrize("K", [2, 3, 5, 7])
def test_matches_plain_definition(bits, K, signed):
    if algorithm2.layout(bits, bits, K, signed) is None:
        pytest.skip("kernel does not fit one 32-bit word at this width")
    rng = np.random.default_rng(100 * bits + 10 * K + signed)
    for n in (1, 2, 7, 64, 1001, 40000):
        f, g = _codes(rng, n, bits, signed), _codes(rng, K, bits, signed)
        for threads in (1, 5):
            assert np.array_equal(algorithm2.conv1d_full(f, g, bits, bits, signed, threads), direct.conv1d_full(f, g))


@pytest.mark.parametrize("signed", [False, True])
def test_extreme_codes(signed):
    for bits in range(1, 9):
        for K in (3, 5):
            if algorithm2.layout(bits, bits, K, signed) is None:
                continue
            lo, hi = (-(1 << (bits - 1)), (1 << (bits - 1)) - 1) if signed else (0, (1 << bits) - 1)
            for fv in (lo, hi):
                for gv in (lo, hi):
                    f, g = np.full(500, fv), np.full(K, gv)
                    assert np.array_equal(algorithm2.conv1d_full(f, g, bits, bits, signed, 3), direct.conv1d_full(f, g))


def test_agrees_with_big_integer_model():
    # same steps in Python big integers (no 64-bit wrap anywhere): block products, carry, Eq. 29 split
    rng = np.random.default_rng(3)
    for signed in (False, True):
        lay = algorithm2.layout(4, 4, 3, signed)
        f, g = _codes(rng, 50, 4, signed), _codes(rng, 3, 4, signed)
        ref = pm.conv1d_carry(list(map(int, f)), list(map(int, g)), lay["N"], lay["S"], signed)
        got = algorithm2.conv1d_full(f, g, 4, 4, signed, 1)
        assert got.tolist() == ref[:got.size]


def test_unfit_layout_is_refused():
    assert algorithm2.layout(8, 8, 7, False) is None
    with pytest.raises(ValueError):
        algorithm2.conv1d_full(np.zeros(10), np.zeros(7), 8, 8, False)
