"""GPU parity for the standalone packing kernel and the 2x2 max-pool."""
import os

import numpy as np
import pytest
import torch

from oracle import direct
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs
from gpu_util import dev

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_pack_matches_eq5():
    rng = np.random.default_rng(1)
    for signed in (False, True):
        for (bits, S, N, wb) in ((4, 10, 3, 32), (4, 13, 3, 32), (1, 3, 11, 32), (8, 18, 2, 32), (4, 10, 7, 64), (8, 21, 3, 64),
                                 (2, 6, 5, 32), (4, 4, 8, 32)):
            for n in (1, N, 1000, 100003):
                v = inputs.uniform_codes(rng, (n,), bits, signed)
                words = hk.pack(dev(v), bits, signed, S, N, wb)
                torch.cuda.synchronize()
                got = words.cpu().numpy()
                got = got.view(np.uint32).astype(np.uint64) if wb == 32 else got.view(np.uint64)
                assert np.array_equal(got, direct.pack_words(v, S, N, wb)), (bits, S, N, wb, n, signed)


def test_pack_reproduces_the_printed_multiplicands():
    vals = {}
    with open(os.path.join(GOLDEN, "worked_example_f32.txt")) as fh:
        for line in fh:
            if "=" in line and not line.startswith("#"):
                k, v = line.split("=", 1)
                vals[k.strip()] = v.strip()
    f = np.array([int(t) for t in vals["f"].split()])
    g = np.array([int(t) for t in vals["g"].split()])
    # the figure stores the first element in the top slot: feed the mirrored sequences
    A = hk.pack(dev(f[::-1].copy()), 4, False, 10, 3, 32)
    B = hk.pack(dev(g[::-1].copy()), 4, False, 10, 2, 32)
    torch.cuda.synchronize()
    assert int(A[0]) == int(vals["multiplicand_f"]) and int(B[0]) == int(vals["multiplicand_g"])
    assert int(A[0]) * int(B[0]) == int(vals["product"])


def test_maxpool():
    rng = np.random.default_rng(2)
    for signed in (False, True):
        # widths that take the scalar kernel, the 8-byte kernel (W % 8 == 0) and the 16-byte kernel (W % 16 == 0)
        for shape in ((1, 1, 2, 2), (2, 3, 6, 10), (3, 5, 7, 9), (2, 3, 9, 24), (2, 4, 6, 40), (4, 16, 40, 80), (3, 7, 5, 48)):
            v = inputs.uniform_codes(rng, shape, 8, signed)
            out = hk.maxpool2x2_i8(dev(v), signed)
            torch.cuda.synchronize()
            got = inputs.from_storage(out.cpu().numpy(), signed)
            assert np.array_equal(got, direct.maxpool2x2(v)), (shape, signed)
        # a view that starts 8 bytes into an allocation: the 16-byte kernel must not be chosen for it
        v = inputs.uniform_codes(rng, (2, 3, 4, 32), 8, signed)
        buf = torch.zeros(v.size + 16, dtype=torch.int8, device="cuda")
        buf[8:8 + v.size] = dev(v).reshape(-1)
        out = hk.maxpool2x2_i8(buf[8:8 + v.size].view(2, 3, 4, 32), signed)
        torch.cuda.synchronize()
        assert np.array_equal(inputs.from_storage(out.cpu().numpy(), signed), direct.maxpool2x2(v))


def test_check_range_counts_codes_outside_their_range():
    # 8-bit values checked against every narrower range: sizes around the 16-byte pieces, unaligned starts
    rng = np.random.default_rng(21)
    for signed in (False, True):
        for n in (1, 15, 16, 17, 47, 1000, 1000003):
            v = inputs.uniform_codes(rng, (n + 3,), 8, signed)
            d = dev(v)
            for off in (0, 1, 3):
                for bits in range(1, 9):
                    want = direct.count_out_of_range(v[off:off + n], bits, signed)
                    assert hk.check_range(d[off:off + n], bits, signed) == want, (signed, n, off, bits)
    # in-range data of every width, the extremes included, passes; one bad code is found wherever it sits
    for signed in (False, True):
        for bits in range(1, 8):
            lo, hi = inputs.code_range(bits, signed)
            v = inputs.uniform_codes(rng, (5000,), bits, signed)
            v[:2] = (lo, hi)
            assert hk.check_range(dev(v), bits, signed) == 0
            for pos in (0, 7, 16, 4999):
                w = v.copy()
                w[pos] = hi + 1
                assert hk.check_range(dev(w), bits, signed) == 1
                w[pos] = lo - 1
                assert hk.check_range(dev(w), bits, signed) == 1
    # the status code of the C interface
    bad = dev(np.array([0, 1, 16, 3]))
    count = torch.zeros(1, dtype=torch.int64, device="cuda")
    assert hk.lib().hikonv_check_range(bad.data_ptr(), 4, 4, 0, count.data_ptr(), None, None) == hk.ERR_RANGE
    assert int(count.item()) == 1
    assert hk.lib().hikonv_check_range(bad.data_ptr(), 4, 5, 0, count.data_ptr(), None, None) == hk.OK
    assert hk.status_string(hk.ERR_RANGE)
