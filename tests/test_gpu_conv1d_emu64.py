"""GPU parity of HIKONV_ALGO_PACKED64EMU (64-bit packed words, 64x64 -> 128 product built from 32-bit
multiplies; the wider multiplier of Section V-A) against the int64 oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import direct
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs
from gpu_util import assert_exact, dev

pytestmark = pytest.mark.gpu

EMU = hk.ALGO_PACKED64EMU


def _run(f, g, p, q, fs, gs, tune=None):
    return hk.conv1d(dev(f), dev(g), p, q, fs, gs, algo=EMU, tune=tune)


def test_c1():
    f, g = inputs.c1()
    assert_exact(_run(f, g, 4, 4, False, False), direct.conv1d_full(f, g), "C1")


@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("bits", range(1, 9))
def test_bitwidth_sweep_small(bits, signed):
    # several steps of 32 blocks per warp, several warps, a ragged tail
    for K in (3, 5, 7):
        for n in (100003, 4097):
            f, g = inputs.conv1d_case(n, K, bits, bits, signed, signed, seed=bits * 100 + K)
            assert_exact(_run(f, g, bits, bits, signed, signed), direct.conv1d_full(f, g),
                         "p=%d K=%d n=%d signed=%d" % (bits, K, n, signed))


@pytest.mark.parametrize("signed", [False, True])
def test_extreme_codes(signed):
    # all-min, all-max and alternating codes fill every slot of the 128-bit product to its bound
    for bits in range(1, 9):
        for K in (3, 5, 7):
            for f, g in inputs.extreme_1d(2051, K, bits, bits, signed, signed):
                assert_exact(_run(f, g, bits, bits, signed, signed), direct.conv1d_full(f, g),
                             "extreme p=%d K=%d signed=%d" % (bits, K, signed))


def test_mixed_signedness_and_widths():
    rng = np.random.default_rng(15)
    for (p, q, fs, gs) in ((4, 4, False, True), (8, 4, False, True), (4, 8, True, False), (1, 8, False, True),
                           (8, 1, True, True), (2, 6, True, False), (7, 3, False, False)):
        for K in (1, 2, 3, 4, 9, 16):
            f = inputs.uniform_codes(rng, (5000,), p, fs)
            g = inputs.uniform_codes(rng, (K,), q, gs)
            assert_exact(_run(f, g, p, q, fs, gs), direct.conv1d_full(f, g), "p=%d q=%d K=%d" % (p, q, K))


def test_tiny_and_degenerate_lengths():
    rng = np.random.default_rng(16)
    for n in (1, 2, 3, 5, 31, 32, 33, 95, 96, 97, 191, 193):
        for K in (1, 3, 7):
            f = inputs.uniform_codes(rng, (n,), 4, True)
            g = inputs.uniform_codes(rng, (K,), 4, True)
            assert_exact(_run(f, g, 4, 4, True, True), direct.conv1d_full(f, g), "n=%d K=%d" % (n, K))


def test_forced_layouts_cover_every_block_size():
    # every N from 1 to 16 (each its own kernel instance), the kernel in one word and in chunks
    rng = np.random.default_rng(17)
    f1 = inputs.uniform_codes(rng, (30011,), 1, False)
    f4 = inputs.uniform_codes(rng, (30011,), 4, True)
    for K in (3, 7):
        g1 = inputs.uniform_codes(rng, (K,), 1, False)
        g4 = inputs.uniform_codes(rng, (K,), 4, True)
        ref1, ref4 = direct.conv1d_full(f1, g1), direct.conv1d_full(f4, g4)
        for N in range(1, 17):
            assert_exact(_run(f1, g1, 1, 1, False, False, {"N": N}), ref1, "1-bit N=%d K=%d" % (N, K))
            if N <= hk.layout_emu64(4, 4, True, True, K)["N"]:
                assert_exact(_run(f4, g4, 4, 4, True, True, {"N": N}), ref4, "4-bit N=%d K=%d" % (N, K))
    # the paper's printed slot width for 4 bits, and a wider one; short and long runs per warp
    f = inputs.uniform_codes(rng, (30011,), 4, False)
    g = inputs.uniform_codes(rng, (3,), 4, False)
    ref = direct.conv1d_full(f, g)
    for tune in ({"N": 7, "S": 10}, {"N": 3, "S": 10}, {"N": 4, "S": 14}, {"N": 7, "S": 10, "tile": 1}, {"tile": 3}):
        assert_exact(_run(f, g, 4, 4, False, False, tune), ref, str(tune))
    with pytest.raises(hk.HikonvError):
        _run(f, g, 4, 4, False, False, {"N": 8, "S": 10})


def test_unaligned_pointers():
    rng = np.random.default_rng(18)
    f = inputs.uniform_codes(rng, (20000,), 4, True)
    g = inputs.uniform_codes(rng, (3,), 4, True)
    ref = direct.conv1d_full(f, g)
    for shift in (1, 3):
        big_f = torch.zeros(20016, dtype=torch.int8, device="cuda")
        big_y = torch.full((20016,), -7, dtype=torch.int32, device="cuda")
        big_f[shift:shift + 20000] = dev(f)
        y = big_y[shift:shift + 20002]
        hk.conv1d(big_f[shift:shift + 20000], dev(g), 4, 4, True, True, algo=EMU, out=y)
        assert_exact(y, ref, "offset %d" % shift)
        torch.cuda.synchronize()
        assert int(big_y[shift - 1]) == -7 and int(big_y[shift + 20002]) == -7     # nothing written outside


def test_full_size_cases():
    # benchmark length 2^24, in the launch configuration the benchmark table times: the narrowest, the
    # printed 4-bit and the widest codes
    for case in inputs.c2_cases():
        if (case["p"], case["K"]) not in ((1, 7), (4, 3), (8, 7)):
            continue
        f, g = inputs.conv1d_case(case["length"], case["K"], case["p"], case["q"], case["f_signed"], case["g_signed"], case["seed"])
        y = _run(f, g, case["p"], case["q"], case["f_signed"], case["g_signed"])
        assert_exact(y, direct.conv1d_full(f, g), str(case))
