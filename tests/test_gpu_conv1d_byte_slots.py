"""GPU parity of the 1-D kernels with register-aligned slots (S = 8, 16 and 17..21) against the int64 oracle, bit for bit.

``hikonv_conv1d`` takes these kernels by itself whenever the sums of K products fit such a slot and K <= 8;
``hikonv_conv1d_layout`` reports the layout that runs.  Every bitwidth, kernel length 1..8, sign combination,
both per-lane run lengths, extreme codes, ragged and unaligned buffers.
"""
import numpy as np
import pytest
import torch

from oracle import direct
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs
from gpu_util import assert_exact, dev

pytestmark = pytest.mark.gpu

SIGNS = [(False, False), (True, True), (False, True), (True, False)]


def _run(f, g, p, q, fs, gs, tune=None):
    return hk.conv1d(dev(f), dev(g), p, q, fs, gs, algo=hk.ALGO_PACKED32, tune=tune)


def test_layout_that_runs_is_reported():
    # the sweep's cases: one-byte slots at 1-3 bits, two-byte slots at 4-7 bits, 17 to 19 bits at 8 bits
    for bits in range(1, 9):
        for K in (3, 5, 7):
            for signed in (False, True):
                L = hk.conv1d_layout(bits, bits, signed, signed, K)
                assert (L["N"], L["S"]) in ((4, 8), (2, 16), (2, 17), (2, 18), (2, 19)), (bits, K, signed, L)
                plan = hk.layout(bits, bits, signed, signed, K, 1)
                forced = hk.conv1d_layout(bits, bits, signed, signed, K, tune={"tile": -1})
                assert forced["S"] == plan["S"]
    L1 = hk.conv1d_layout(1, 1, False, False, 3)
    assert (L1["N"], L1["S"], L1["Kc"], L1["J"]) == (4, 8, 3, 1)
    assert hk.conv1d_layout(3, 3, False, False, 7)["S"] == 16          # 7 * 49 = 343 needs nine bits
    assert hk.conv1d_layout(3, 3, True, True, 7)["S"] == 8             # [-84, 112] fits a signed byte
    assert hk.conv1d_layout(7, 7, False, False, 5)["S"] == 17          # 5 * 127^2 = 80645 needs 17 bits
    assert hk.conv1d_layout(7, 7, True, True, 7)["S"] == 16
    L8 = hk.conv1d_layout(8, 8, True, True, 7)
    assert (L8["N"], L8["S"], L8["Kc"], L8["J"]) == (2, 18, 2, 4)
    L8u = hk.conv1d_layout(8, 8, False, False, 7)
    assert (L8u["N"], L8u["S"], L8u["Kc"], L8u["J"]) == (2, 19, 2, 4)      # 7 * 255^2 = 455175 < 2^19


@pytest.mark.parametrize("signs", SIGNS)
@pytest.mark.parametrize("bits", range(1, 9))
def test_every_width_kernel_length_and_sign(bits, signs):
    fs, gs = signs
    for K in range(1, 9):
        for n in (1, 3, 767, 768, 769, 50021):
            f, g = inputs.conv1d_case(n, K, bits, bits, fs, gs, seed=7000 + 100 * bits + 10 * K + n % 7)
            assert_exact(_run(f, g, bits, bits, fs, gs), direct.conv1d_full(f, g),
                         "p=%d K=%d n=%d signs=%s" % (bits, K, n, signs))


@pytest.mark.parametrize("signs", SIGNS)
def test_extreme_codes(signs):
    fs, gs = signs
    for bits in range(1, 9):
        for K in (1, 2, 3, 4, 5, 7, 8):
            for f, g in inputs.extreme_1d(3001, K, bits, bits, fs, gs):
                assert_exact(_run(f, g, bits, bits, fs, gs), direct.conv1d_full(f, g),
                             "extreme p=%d K=%d signs=%s" % (bits, K, signs))


def test_unequal_widths():
    rng = np.random.default_rng(77)
    for (p, q, fs, gs) in ((1, 8, False, True), (8, 1, True, True), (2, 6, True, False), (7, 3, False, False), (4, 8, True, False),
                           (8, 4, False, True), (8, 2, False, False), (3, 5, True, True), (6, 2, False, True)):
        for K in (1, 2, 3, 4, 6, 8):
            f = inputs.uniform_codes(rng, (20011,), p, fs)
            g = inputs.uniform_codes(rng, (K,), q, gs)
            assert_exact(_run(f, g, p, q, fs, gs), direct.conv1d_full(f, g), "p=%d q=%d K=%d" % (p, q, K))
            for fx, gx in inputs.extreme_1d(1500, K, p, q, fs, gs):
                assert_exact(_run(fx, gx, p, q, fs, gs), direct.conv1d_full(fx, gx), "extreme p=%d q=%d K=%d" % (p, q, K))


@pytest.mark.parametrize("budget", [-24, -25])
@pytest.mark.parametrize("signed", [False, True])
def test_both_register_budgets(signed, budget):
    # every kernel is built for four and for five resident CTAs per SM; the default takes one of them per kernel
    for bits in range(1, 9):
        for K in (3, 5, 7):
            for n in (100003, 1025):
                f, g = inputs.conv1d_case(n, K, bits, bits, signed, signed, seed=900 + bits * 10 + K)
                assert_exact(_run(f, g, bits, bits, signed, signed, {"tile": budget}), direct.conv1d_full(f, g),
                             "budget %d: p=%d K=%d n=%d signed=%d" % (budget, bits, K, n, signed))


def test_full_size_cases_of_the_widest_slots():
    # the 8-bit and unsigned 7-bit cases of the sweep at 2^24 codes with the other register budget than the
    # default one (tests/test_gpu_conv1d.py runs all 48 cases in the default configuration)
    for case in inputs.c2_cases():
        if case["p"] < 7:
            continue
        f, g = inputs.conv1d_case(case["length"], case["K"], case["p"], case["q"], case["f_signed"], case["g_signed"], case["seed"])
        J = hk.conv1d_layout(case["p"], case["q"], case["f_signed"], case["g_signed"], case["K"])["J"]
        y = _run(f, g, case["p"], case["q"], case["f_signed"], case["g_signed"], {"tile": -24 if J <= 2 else -25})
        assert_exact(y, direct.conv1d_full(f, g), str(case))


@pytest.mark.parametrize("bits", [2, 5, 8])
def test_unaligned_pointers(bits):
    rng = np.random.default_rng(78)
    for signed in (False, True):
        f = inputs.uniform_codes(rng, (20000,), bits, signed)
        g = inputs.uniform_codes(rng, (5,), bits, signed)
        ref = direct.conv1d_full(f, g)
        for shift in (1, 2, 3):
            big_f = torch.zeros(20016, dtype=torch.int8, device="cuda")
            big_y = torch.full((20032,), -7, dtype=torch.int32, device="cuda")
            big_f[shift:shift + 20000] = dev(f)
            y = big_y[shift:shift + 20004]
            hk.conv1d(big_f[shift:shift + 20000], dev(g), bits, bits, signed, signed, out=y)
            assert_exact(y, ref, "offset %d" % shift)
            torch.cuda.synchronize()
            assert int(big_y[shift - 1]) == -7 and int(big_y[shift + 20004]) == -7     # nothing written outside
