"""GPU parity, 1-D: the CUDA path through the C interface against the int64 oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import direct
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs
from gpu_util import assert_exact, dev

pytestmark = pytest.mark.gpu

# "planner": the packed kernels on the planner's layout (most outputs per multiply); without it the packed call
# takes byte-aligned slots wherever the sums fit them (tests/test_gpu_conv1d_byte_slots.py covers those further)
PLANNER = "planner-layout"
ALGOS = [hk.ALGO_PACKED32, PLANNER, hk.ALGO_UNPACKED_IMAD]


def _run(f, g, p, q, fs, gs, algo, tune=None):
    if algo == PLANNER:
        algo = hk.ALGO_PACKED32
        if not tune:
            tune = {"tile": -1}
    return hk.conv1d(dev(f), dev(g), p, q, fs, gs, algo=algo, tune=tune)


@pytest.mark.parametrize("algo", ALGOS)
def test_c1(algo):
    f, g = inputs.c1()
    y = _run(f, g, 4, 4, False, False, algo)
    assert y.numel() == 4098
    assert_exact(y, direct.conv1d_full(f, g), "C1")


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("bits", range(1, 9))
def test_bitwidth_sweep_small(bits, signed, algo):
    # several chunks of 32 blocks per warp, several warps, and a ragged tail
    for K in (3, 5, 7):
        for n in (100003, 4097):
            f, g = inputs.conv1d_case(n, K, bits, bits, signed, signed, seed=bits * 100 + K)
            assert_exact(_run(f, g, bits, bits, signed, signed, algo), direct.conv1d_full(f, g),
                         "p=%d K=%d n=%d signed=%d" % (bits, K, n, signed))


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("signed", [False, True])
def test_bitwidth_sweep_shuffle_kernels(signed, algo):
    # tile > 0 selects the general kernels (any N, J, K), which the automatic choice only uses for
    # layouts the register-resident kernels are not instantiated for
    for bits in range(1, 9):
        for K in (3, 5, 7):
            f, g = inputs.conv1d_case(40009, K, bits, bits, signed, signed, seed=bits * 10 + K)
            assert_exact(_run(f, g, bits, bits, signed, signed, algo, tune={"tile": 4}), direct.conv1d_full(f, g),
                         "general kernel p=%d K=%d signed=%d" % (bits, K, signed))


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("signed", [False, True])
def test_extreme_codes(signed, algo):
    for bits in range(1, 9):
        for K in (3, 5, 7):
            for f, g in inputs.extreme_1d(2051, K, bits, bits, signed, signed):
                assert_exact(_run(f, g, bits, bits, signed, signed, algo), direct.conv1d_full(f, g),
                             "extreme p=%d K=%d signed=%d" % (bits, K, signed))


@pytest.mark.parametrize("algo", ALGOS)
def test_mixed_signedness_and_widths(algo):
    rng = np.random.default_rng(5)
    for (p, q, fs, gs) in ((4, 4, False, True), (8, 4, False, True), (4, 8, True, False), (1, 8, False, True),
                           (8, 1, True, True), (2, 6, True, False), (7, 3, False, False)):
        for K in (1, 2, 3, 4, 9, 16):
            f = inputs.uniform_codes(rng, (5000,), p, fs)
            g = inputs.uniform_codes(rng, (K,), q, gs)
            assert_exact(_run(f, g, p, q, fs, gs, algo), direct.conv1d_full(f, g), "p=%d q=%d K=%d" % (p, q, K))


@pytest.mark.parametrize("algo", ALGOS)
def test_tiny_and_degenerate_lengths(algo):
    rng = np.random.default_rng(6)
    for n in (1, 2, 3, 5, 31, 32, 33, 95, 96, 97):
        for K in (1, 3, 7):
            f = inputs.uniform_codes(rng, (n,), 4, True)
            g = inputs.uniform_codes(rng, (K,), 4, True)
            assert_exact(_run(f, g, 4, 4, True, True, algo), direct.conv1d_full(f, g), "n=%d K=%d" % (n, K))


def test_forced_layouts():
    # other (N, S) than the automatic choice, including the paper's N = 3, S = 10 at 4 bits
    rng = np.random.default_rng(7)
    f = inputs.uniform_codes(rng, (30011,), 4, False)
    g = inputs.uniform_codes(rng, (3,), 4, False)
    ref = direct.conv1d_full(f, g)
    for tune in ({"N": 3, "S": 10}, {"N": 2, "S": 10}, {"N": 1, "S": 12}, {"N": 2, "S": 14}, {"N": 3, "S": 10, "tile": 1},
                 {"N": 3, "S": 10, "tile": 3}):
        assert_exact(_run(f, g, 4, 4, False, False, hk.ALGO_PACKED32, tune), ref, str(tune))
    fs = inputs.uniform_codes(rng, (30011,), 3, True)
    gs = inputs.uniform_codes(rng, (5,), 3, True)
    for tune in ({"N": 4}, {"N": 3}, {"N": 2, "S": 12}):
        assert_exact(_run(fs, gs, 3, 3, True, True, hk.ALGO_PACKED32, tune), direct.conv1d_full(fs, gs), str(tune))


@pytest.mark.parametrize("signed", [False, True])
def test_planner_block_sizes_that_the_automatic_choice_replaces(signed):
    # without a forced layout the call runs N = 8 / N = 4 where the planner says 11 / 5; the planner's own
    # layouts stay reachable by forcing N, and both must give the oracle's result
    for bits, K in ((1, 3), (2, 3), (2, 5), (2, 7)):
        f, g = inputs.conv1d_case(60013, K, bits, bits, signed, signed, seed=300 + 10 * bits + K)
        ref = direct.conv1d_full(f, g)
        n_plan = hk.layout(bits, bits, signed, signed, K, 1)["N"]
        assert_exact(_run(f, g, bits, bits, signed, signed, hk.ALGO_PACKED32), ref, "automatic p=%d K=%d" % (bits, K))
        assert_exact(_run(f, g, bits, bits, signed, signed, hk.ALGO_PACKED32, {"N": n_plan}), ref,
                     "planner N=%d p=%d K=%d" % (n_plan, bits, K))
    # a layout whose smaller block would need one more kernel chunk keeps the planner's block size
    rng = np.random.default_rng(31)
    f = inputs.uniform_codes(rng, (60013,), 1, False)
    g = inputs.uniform_codes(rng, (9,), 2, True)
    assert_exact(_run(f, g, 1, 2, False, True, hk.ALGO_PACKED32), direct.conv1d_full(f, g), "1-bit x s2, K=9")


@pytest.mark.parametrize("shape", [-32, -24, -25])
@pytest.mark.parametrize("algo", [hk.ALGO_UNPACKED_IMAD, hk.ALGO_DP4A])
def test_comparators_in_every_launch_shape(algo, shape):
    # tile = -32: runs of 32 outputs per lane; -24 / -25: runs of 24 with the register budget of four / five
    # resident CTAs per SM (the default picks between the last two by kernel length)
    for signed in (False, True):
        for bits in (1, 4, 8):
            for K in (3, 5, 7):
                for n in (100003, 1023):
                    f, g = inputs.conv1d_case(n, K, bits, bits, signed, signed, seed=500 + bits * 10 + K)
                    assert_exact(_run(f, g, bits, bits, signed, signed, algo, {"tile": shape}), direct.conv1d_full(f, g),
                                 "shape %d: p=%d K=%d n=%d signed=%d" % (shape, bits, K, n, signed))


@pytest.mark.parametrize("algo", ALGOS)
def test_unaligned_pointers(algo):
    rng = np.random.default_rng(8)
    f = inputs.uniform_codes(rng, (20000,), 4, True)
    g = inputs.uniform_codes(rng, (3,), 4, True)
    ref = direct.conv1d_full(f, g)
    for shift in (1, 3):
        big_f = torch.zeros(20016, dtype=torch.int8, device="cuda")
        big_y = torch.full((20016,), -7, dtype=torch.int32, device="cuda")
        big_f[shift:shift + 20000] = dev(f)
        y = big_y[shift:shift + 20002]
        hk.conv1d(big_f[shift:shift + 20000], dev(g), 4, 4, True, True, algo=hk.ALGO_PACKED32 if algo == PLANNER else algo,
                  tune={"tile": -1} if algo == PLANNER else None, out=y)
        assert_exact(y, ref, "offset %d" % shift)
        torch.cuda.synchronize()
        assert int(big_y[shift - 1]) == -7 and int(big_y[shift + 20002]) == -7     # nothing written outside


def test_host_buffer_entry_point():
    f, g = inputs.conv1d_case(50000, 5, 4, 4, True, True, seed=9)
    h_f = torch.from_numpy(inputs.to_storage(f)).pin_memory()
    h_g = torch.from_numpy(inputs.to_storage(g)).pin_memory()
    h_y = torch.empty(50004, dtype=torch.int32).pin_memory()
    ws = torch.empty(hk.conv1d_host_workspace_bytes(50000, 5), dtype=torch.uint8, device="cuda")
    hk.conv1d_host(h_f, h_g, 4, 4, True, True, h_y, ws)
    torch.cuda.synchronize()
    assert np.array_equal(h_y.numpy().astype(np.int64), direct.conv1d_full(f, g))
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(hk.HikonvError):
        hk.conv1d_host(h_f, h_g, 4, 4, True, True, h_y, small)


@pytest.mark.parametrize("algo", ALGOS)
def test_full_size_sweep(algo):
    # the 48 benchmark cases at 2^24, in the launch configuration the benchmark times
    for case in inputs.c2_cases():
        f, g = inputs.conv1d_case(case["length"], case["K"], case["p"], case["q"], case["f_signed"], case["g_signed"], case["seed"])
        y = _run(f, g, case["p"], case["q"], case["f_signed"], case["g_signed"], algo)
        assert_exact(y, direct.conv1d_full(f, g), str(case))


# ---- the byte dot-product comparator (dp4a), kernels of up to eight taps

@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("bits", range(1, 9))
def test_dp4a_bitwidth_sweep_and_extremes(bits, signed):
    for K in (3, 5, 7):
        for n in (100003, 4097):
            f, g = inputs.conv1d_case(n, K, bits, bits, signed, signed, seed=bits * 100 + K + 1)
            assert_exact(_run(f, g, bits, bits, signed, signed, hk.ALGO_DP4A), direct.conv1d_full(f, g),
                         "dp4a p=%d K=%d n=%d signed=%d" % (bits, K, n, signed))
        for f, g in inputs.extreme_1d(2051, K, bits, bits, signed, signed):
            assert_exact(_run(f, g, bits, bits, signed, signed, hk.ALGO_DP4A), direct.conv1d_full(f, g),
                         "dp4a extreme p=%d K=%d signed=%d" % (bits, K, signed))


def test_dp4a_mixed_signs_every_kernel_length_and_tiny_signals():
    rng = np.random.default_rng(41)
    for (p, q, fs, gs) in ((4, 4, False, True), (8, 4, False, True), (4, 8, True, False), (8, 8, True, True), (8, 8, False, False)):
        for K in range(1, 9):
            for n in (1, 2, 5, 33, 1023, 1024, 1025, 5000):
                f = inputs.uniform_codes(rng, (n,), p, fs)
                g = inputs.uniform_codes(rng, (K,), q, gs)
                assert_exact(_run(f, g, p, q, fs, gs, hk.ALGO_DP4A), direct.conv1d_full(f, g), "dp4a p=%d q=%d K=%d n=%d" % (p, q, K, n))
    f = inputs.uniform_codes(rng, (100,), 4, False)
    with pytest.raises(hk.HikonvError):
        _run(f, inputs.uniform_codes(rng, (9,), 4, False), 4, 4, False, False, hk.ALGO_DP4A)


def test_dp4a_unaligned_pointers_and_full_size():
    rng = np.random.default_rng(42)
    f = inputs.uniform_codes(rng, (20000,), 8, False)
    g = inputs.uniform_codes(rng, (7,), 4, True)
    ref = direct.conv1d_full(f, g)
    for shift in (1, 3):
        big_f = torch.zeros(20016, dtype=torch.int8, device="cuda")
        big_y = torch.full((20032,), -7, dtype=torch.int32, device="cuda")
        big_f[shift:shift + 20000] = dev(f)
        y = big_y[shift:shift + 20006]
        hk.conv1d(big_f[shift:shift + 20000], dev(g), 8, 4, False, True, algo=hk.ALGO_DP4A, out=y)
        assert_exact(y, ref, "dp4a offset %d" % shift)
        torch.cuda.synchronize()
        assert int(big_y[shift - 1]) == -7 and int(big_y[shift + 20006]) == -7
    for case in inputs.c2_cases():
        if (case["p"], case["K"]) in ((1, 3), (4, 5), (8, 7)):
            f, g = inputs.conv1d_case(case["length"], case["K"], case["p"], case["q"], case["f_signed"], case["g_signed"], case["seed"])
            y = _run(f, g, case["p"], case["q"], case["f_signed"], case["g_signed"], hk.ALGO_DP4A)
            assert_exact(y, direct.conv1d_full(f, g), "dp4a " + str(case))
