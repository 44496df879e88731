"""Seeded random configurations of both convolutions against the int64 oracle, bit for bit: unequal
bitwidths, mixed signedness, odd shapes, forced layouts."""
import numpy as np
import pytest
import torch

from oracle import direct
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs
from gpu_util import assert_exact, dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", range(40))
def test_conv1d_random_configuration(seed):
    rng = np.random.default_rng(9000 + seed)
    p, q = int(rng.integers(1, 9)), int(rng.integers(1, 9))
    fs, gs = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
    K = int(rng.choice([1, 2, 3, 4, 5, 7, 9, 16, 33]))
    n = int(rng.choice([1, 5, 63, 1000, 4097, 33333, 262144 + 17]))
    f, g = inputs.conv1d_case(n, K, p, q, fs, gs, seed=seed)
    ref = direct.conv1d_full(f, g)
    for algo in (hk.ALGO_PACKED32, hk.ALGO_UNPACKED_IMAD):
        assert_exact(hk.conv1d(dev(f), dev(g), p, q, fs, gs, algo=algo), ref,
                     "p=%d q=%d fs=%d gs=%d K=%d n=%d algo=%d" % (p, q, fs, gs, K, n, algo))
    # the general (shuffle) kernel on the same case
    assert_exact(hk.conv1d(dev(f), dev(g), p, q, fs, gs, tune={"tile": 3}), ref, "general kernel, seed %d" % seed)


@pytest.mark.parametrize("seed", range(40))
def test_conv2d_random_configuration(seed):
    rng = np.random.default_rng(7000 + seed)
    p, q = int(rng.integers(1, 9)), int(rng.integers(1, 9))
    xs, ws = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
    K = int(rng.choice([1, 2, 3, 3, 3, 5]))
    pad = int(rng.integers(0, K))
    B, Ci, Co = int(rng.integers(1, 4)), int(rng.integers(1, 40)), int(rng.integers(1, 45))
    H, W = int(rng.integers(K, 20)), int(rng.integers(K, 90))
    x, w = inputs.conv2d_case(B, Ci, H, W, Co, K, p, q, xs, ws, seed=seed)
    ref = direct.conv2d_nchw(x, w, pad)
    what = "B=%d Ci=%d H=%d W=%d Co=%d K=%d pad=%d p=%d q=%d xs=%d ws=%d" % (B, Ci, H, W, Co, K, pad, p, q, xs, ws)
    for algo in (hk.ALGO_PACKED32, hk.ALGO_UNPACKED_IMAD):
        try:
            got = hk.conv2d(dev(x), dev(w), pad, p, q, xs, ws, algo=algo)
        except hk.HikonvError as e:
            # wide codes with long kernel rows may have no packed layout; that has to be said, not mis-computed
            assert algo == hk.ALGO_PACKED32 and e.status in (hk.ERR_NO_FIT, hk.ERR_UNSUPPORTED), what
            continue
        assert_exact(got, ref, what + " algo=%d" % algo)
    shift = int(rng.integers(0, 8))
    lo, hi = (-(1 << (p - 1)), (1 << (p - 1)) - 1) if xs else (0, (1 << p) - 1)
    try:
        got = hk.conv2d(dev(x), dev(w), pad, p, q, xs, ws, requant=(shift, lo, hi))
    except hk.HikonvError:
        return
    torch.cuda.synchronize()
    g = got.cpu().numpy()
    g = g.astype(np.int64) if lo < 0 else g.view(np.uint8).astype(np.int64)
    assert np.array_equal(g, direct.requant(ref, shift, lo, hi)), what + " requant"


@pytest.mark.parametrize("seed", range(24))
def test_conv2d_deep_and_wide_layers(seed):
    # many input channels (several carry-save moves, every schedule) and rows wider than one tile segment
    rng = np.random.default_rng(5000 + seed)
    p, q = int(rng.choice([1, 2, 3, 4, 4, 4, 5, 8])), int(rng.choice([1, 2, 4, 4, 4, 6, 8]))
    xs, ws = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
    K = int(rng.choice([1, 3, 3, 3, 5]))
    pad = K // 2
    Ci, Co = int(rng.integers(40, 300)), int(rng.integers(1, 140))
    if seed % 2:
        B, H, W = 1, int(rng.integers(1, 5)), int(rng.integers(150, 400))
    else:
        B, H, W = int(rng.integers(1, 5)), int(rng.integers(1, 9)), int(rng.integers(1, 30))
    x, w = inputs.conv2d_case(B, Ci, H, W, Co, K, p, q, xs, ws, seed=seed)
    ref = direct.conv2d_nchw(x, w, pad)
    what = "B=%d Ci=%d H=%d W=%d Co=%d K=%d p=%d q=%d xs=%d ws=%d" % (B, Ci, H, W, Co, K, p, q, xs, ws)
    for algo in (hk.ALGO_PACKED32, hk.ALGO_UNPACKED_IMAD):
        try:
            got = hk.conv2d(dev(x), dev(w), pad, p, q, xs, ws, algo=algo)
        except hk.HikonvError as e:
            assert algo == hk.ALGO_PACKED32 and e.status in (hk.ERR_NO_FIT, hk.ERR_UNSUPPORTED), what
            continue
        assert_exact(got, ref, what + " algo=%d" % algo)
