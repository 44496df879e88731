"""GPU parity of the 2-D layer on seeded random shapes, bit widths, signs, kernel sizes and paddings against the int64
oracle, bit for bit: exact sums and requantised codes, random and extreme codes."""
import numpy as np
import pytest
import torch

from oracle import direct
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [101, 102, 103])
def test_random_layers(seed):
    rng = np.random.default_rng(seed)
    ran = 0
    for _ in range(120):
        K = int(rng.choice([1, 2, 3, 3, 3, 5]))
        pad = int(rng.integers(0, K))
        B = int(rng.integers(1, 4))
        Ci = int(rng.choice([1, 2, 3, 5, 8, 16, 31, 32, 40, 64, 100, 128, 131, 200]))
        H = int(rng.integers(max(1, K - 2 * pad), 24))
        W = int(rng.integers(max(1, K - 2 * pad), 70))
        if rng.random() < 0.15:                                   # wide rows: several row segments
            W, H = int(rng.integers(100, 400)), int(rng.integers(max(1, K - 2 * pad), 6))
        Co = int(rng.choice([1, 3, 4, 7, 16, 17, 40, 64, 70]))
        p, q = int(rng.integers(1, 9)), int(rng.integers(1, 9))
        xs, ws = bool(rng.integers(0, 2)), bool(rng.integers(0, 2))
        if Ci * K * K * (1 << p) * (1 << q) >= (1 << 30):         # sums beyond int32 are refused by the library
            continue
        x, w = inputs.conv2d_case(B, Ci, H, W, Co, K, p, q, xs, ws, seed=int(rng.integers(1 << 30)))
        if rng.random() < 0.2:                                    # every code at an end of its range
            (lo_x, hi_x), (lo_w, hi_w) = inputs.code_range(p, xs), inputs.code_range(q, ws)
            x[...] = hi_x if rng.random() < 0.5 else lo_x
            w[...] = lo_w if rng.random() < 0.5 else hi_w
        case = (B, Ci, H, W, Co, K, pad, p, q, xs, ws)
        ref = direct.conv2d_nchw(x, w, pad)
        d_x, d_w = torch.from_numpy(inputs.to_storage(x)).cuda(), torch.from_numpy(inputs.to_storage(w)).cuda()
        got = hk.conv2d(d_x, d_w, pad, p, q, xs, ws)
        torch.cuda.synchronize()
        assert np.array_equal(got.cpu().numpy().astype(np.int64), ref), case
        if rng.random() < 0.5:
            signed_out = bool(rng.integers(0, 2))
            rq = (int(rng.integers(0, 12)), -8, 7) if signed_out else (int(rng.integers(0, 12)), 0, 15)
            got8 = hk.conv2d(d_x, d_w, pad, p, q, xs, ws, requant=rq)
            torch.cuda.synchronize()
            assert np.array_equal(inputs.from_storage(got8.cpu().numpy(), signed_out), direct.requant(ref, *rq)), (case, rq)
        ran += 1
    assert ran > 80
