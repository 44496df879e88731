"""GPU parity of the dense-input 1-D convolution against the int64 oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import direct
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs
from gpu_util import assert_exact, dev

pytestmark = pytest.mark.gpu


def _run(f, g, bits, signed, offset=0):
    dense = inputs.to_dense(f, bits)
    buf = torch.zeros(dense.size + 8, dtype=torch.uint8, device="cuda")
    buf[offset:offset + dense.size] = torch.from_numpy(dense).cuda()
    view = buf[offset:offset + dense.size]
    return hk.conv1d_dense(view, f.size, dev(g), bits, bits, signed, signed)


@pytest.mark.parametrize("signed", [False, True])
@pytest.mark.parametrize("K", [3, 5, 7])
@pytest.mark.parametrize("bits", [1, 2, 4])
def test_matches_oracle(bits, K, signed):
    # lengths below one tile, ragged tails, several tiles per warp
    for n in (1, 2, 9, 777, 4096, 100003, (1 << 20) + 5):
        f, g = inputs.conv1d_case(n, K, bits, bits, signed, signed, seed=bits * 100 + K * 10 + signed + n)
        assert_exact(_run(f, g, bits, signed), direct.conv1d_full(f, g), "bits=%d K=%d signed=%d n=%d" % (bits, K, signed, n))


@pytest.mark.parametrize("bits", [1, 2, 4])
def test_extreme_codes_and_unaligned_buffers(bits):
    for signed in (False, True):
        for f, g in inputs.extreme_1d(50000, 5, bits, bits, signed, signed):
            assert_exact(_run(f, g, bits, signed), direct.conv1d_full(f, g), "extreme bits=%d signed=%d" % (bits, signed))
        f, g = inputs.conv1d_case(70001, 3, bits, bits, signed, signed, seed=5 + bits)
        ref = direct.conv1d_full(f, g)
        for offset in (1, 2, 3):
            assert_exact(_run(f, g, bits, signed, offset), ref, "offset %d" % offset)


@pytest.mark.parametrize("bits", [1, 2, 4])
def test_full_size_sweep_cases(bits):
    # the 18 dense cases the benchmark times (1, 2 and 4 bits; K = 3, 5, 7; both signs) at 2^24 codes against the
    # oracle: at this length every warp of the persistent grid walks several tiles
    for case in inputs.c2_cases():
        if case["p"] != bits:
            continue
        f, g = inputs.conv1d_case(case["length"], case["K"], case["p"], case["q"], case["f_signed"], case["g_signed"], case["seed"])
        assert_exact(_run(f, g, bits, case["f_signed"]), direct.conv1d_full(f, g), "dense " + str(case))


def test_same_results_as_byte_storage_at_full_size():
    # the benchmark length, one case: dense and one-code-per-byte inputs give identical outputs
    f, g = inputs.conv1d_case(1 << 24, 3, 4, 4, True, True, seed=1431)
    a = _run(f, g, 4, True)
    b = hk.conv1d(dev(f), dev(g), 4, 4, True, True)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    idx = np.random.default_rng(0).integers(0, f.size, 2000)
    fz = np.concatenate([np.zeros(2, dtype=np.int64), f])
    want = np.array([int(fz[i + 2] * g[0] + fz[i + 1] * g[1] + fz[i] * g[2]) for i in idx])   # y[m] = sum_k f[m-k] g[k]
    assert np.array_equal(a.cpu().numpy()[idx], want)


@pytest.mark.parametrize("bits", [1, 2, 4])
def test_mixed_signedness(bits):
    # unsigned codes against signed taps and the reverse, random and extreme, several tiles and a ragged tail
    for fs, gs in ((False, True), (True, False)):
        for K in (3, 5, 7):
            for n in (5, 4099, 200003):
                f, g = inputs.conv1d_case(n, K, bits, bits, fs, gs, seed=40 + bits * 10 + K)
                y = hk.conv1d_dense(torch.from_numpy(inputs.to_dense(f, bits)).cuda(), f.size, dev(g), bits, bits, fs, gs)
                assert_exact(y, direct.conv1d_full(f, g), "mixed bits=%d K=%d fs=%d n=%d" % (bits, K, fs, n))
            for f, g in inputs.extreme_1d(30001, K, bits, bits, fs, gs):
                y = hk.conv1d_dense(torch.from_numpy(inputs.to_dense(f, bits)).cuda(), f.size, dev(g), bits, bits, fs, gs)
                assert_exact(y, direct.conv1d_full(f, g), "mixed extreme bits=%d K=%d fs=%d" % (bits, K, fs))


def test_unsupported_combinations_are_refused():
    f, g = inputs.conv1d_case(1000, 3, 4, 2, False, True, seed=1)
    with pytest.raises(hk.HikonvError):
        hk.conv1d_dense(torch.from_numpy(inputs.to_dense(f, 4)).cuda(), f.size, dev(g), 4, 2, False, True)   # unequal widths: another layout
    f, g = inputs.conv1d_case(1000, 3, 3, 3, False, False, seed=2)
    with pytest.raises(hk.HikonvError):
        hk.conv1d_dense(torch.zeros(1000, dtype=torch.uint8, device="cuda"), f.size, dev(g), 3, 3, False, False)   # 3 bits straddle bytes
