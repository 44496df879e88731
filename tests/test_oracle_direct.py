"""Pins for the plain-definition oracle (CPU only).

Each check compares ``oracle.direct`` with something that is not itself: the
paper's printed example, a library routine, an algebraic identity, a closed
form, or an exhaustive enumeration through a different formulation
(polynomial multiplication by Kronecker substitution).
"""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import direct

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


# ---------------------------------------------------------------- 1-D

def test_conv1d_paper_example():
    g = _golden("worked_example_f32.txt")
    f = [int(t) for t in g["f"].split()]
    k = [int(t) for t in g["g"].split()]
    y = [int(t) for t in g["y"].split()]
    assert direct.conv1d_full(f, k).tolist() == y


def _kronecker_conv(f, g):
    """Coefficients of (sum f x^n)(sum g x^k) for non-negative f, g, read off one big product."""
    base_bits = 40
    F = sum(int(v) << (base_bits * i) for i, v in enumerate(f))
    G = sum(int(v) << (base_bits * i) for i, v in enumerate(g))
    P = F * G
    mask = (1 << base_bits) - 1
    return [(P >> (base_bits * m)) & mask for m in range(len(f) + len(g) - 1)]


def test_conv1d_exhaustive_tiny_unsigned():
    # every 2-bit input of length 3 against every 2-bit kernel of length 2
    for f in itertools.product(range(4), repeat=3):
        for g in itertools.product(range(4), repeat=2):
            assert direct.conv1d_full(f, g).tolist() == _kronecker_conv(f, g)


def test_conv1d_exhaustive_tiny_signed():
    # signed 2-bit codes: shift both operands to non-negative, expand the product by hand
    #   (f+2)*(g+2) = f*g + 2*(1*g) + 2*(f*1) + 4*(1*1)   (all '*' are convolutions)
    for f in itertools.product(range(-2, 2), repeat=3):
        for g in itertools.product(range(-2, 2), repeat=2):
            fs = [v + 2 for v in f]
            gs = [v + 2 for v in g]
            ones_f, ones_g = [1] * 3, [1] * 2
            lhs = _kronecker_conv(fs, gs)
            a = _kronecker_conv(fs, ones_g)     # (f+2) * 1
            b = _kronecker_conv(ones_f, gs)     # 1 * (g+2)
            c = _kronecker_conv(ones_f, ones_g)
            # f*g = (f+2)*(g+2) - 2*((f+2)*1) - 2*(1*(g+2)) + 4*(1*1)
            expect = [lhs[m] - 2 * a[m] - 2 * b[m] + 4 * c[m] for m in range(4)]
            assert direct.conv1d_full(f, g).tolist() == expect


@pytest.mark.parametrize("n,k,signed", [(1, 1, False), (1, 5, True), (7, 1, True), (64, 3, False),
                                        (1000, 7, True), (4097, 5, True), (33, 40, True)])
def test_conv1d_vs_numpy_convolve(n, k, signed):
    rng = np.random.default_rng(n * 100 + k)
    lo, hi = (-128, 128) if signed else (0, 256)
    f = rng.integers(lo, hi, n)
    g = rng.integers(lo, hi, k)
    assert np.array_equal(direct.conv1d_full(f, g), np.convolve(f, g, mode="full"))


def test_conv1d_invariants():
    rng = np.random.default_rng(7)
    f = rng.integers(-8, 8, 50)
    f2 = rng.integers(-8, 8, 50)
    g = rng.integers(-8, 8, 5)
    y = direct.conv1d_full(f, g)
    assert y.size == 54
    assert int(y.sum()) == int(f.sum()) * int(g.sum())                    # sum rule
    assert np.array_equal(y, direct.conv1d_full(g, f))                     # commutative
    assert np.array_equal(direct.conv1d_full(f + 3 * f2, g), y + 3 * direct.conv1d_full(f2, g))  # linear
    delta = np.zeros(5, dtype=np.int64)
    delta[2] = 1
    shifted = direct.conv1d_full(f, delta)                                  # delta kernel = shift
    assert np.array_equal(shifted[2:52], f) and not shifted[:2].any() and not shifted[52:].any()
    ramp = direct.conv1d_full(np.ones(10, dtype=np.int64), np.ones(3, dtype=np.int64))
    assert ramp.tolist() == [1, 2, 3, 3, 3, 3, 3, 3, 3, 3, 2, 1]           # edge term counts


def test_conv1d_empty_input():
    assert direct.conv1d_full([], [1, 2, 3]).tolist() == [0, 0]


# ---------------------------------------------------------------- 2-D

@pytest.mark.parametrize("B,Ci,H,W,Co,K,pad", [(2, 3, 7, 9, 4, 3, 1), (1, 5, 6, 4, 2, 3, 0), (2, 2, 5, 8, 3, 5, 2),
                                               (1, 4, 3, 3, 5, 1, 0), (1, 1, 4, 6, 1, 2, 1)])
def test_conv2d_vs_torch(B, Ci, H, W, Co, K, pad):
    rng = np.random.default_rng(B * 1000 + Ci * 100 + H * 10 + K)
    x = rng.integers(-8, 16, (B, Ci, H, W))
    w = rng.integers(-8, 8, (Co, Ci, K, K))
    ref = torch.nn.functional.conv2d(torch.tensor(x, dtype=torch.float64),
                                     torch.tensor(w, dtype=torch.float64), padding=pad)
    got = direct.conv2d_nchw(x, w, pad)
    assert got.shape == tuple(ref.shape)
    assert np.array_equal(got, ref.numpy().astype(np.int64))


def test_conv2d_constant_closed_form():
    # constant input a, constant weight w, 3x3, pad 1: interior Ci*9*a*w, edges 6/9, corners 4/9
    Ci, a, wv = 5, 7, -3
    x = np.full((1, Ci, 6, 8), a)
    w = np.full((2, Ci, 3, 3), wv)
    out = direct.conv2d_nchw(x, w, 1)
    full = Ci * 9 * a * wv
    assert out.shape == (1, 2, 6, 8)
    assert (out[0, :, 1:-1, 1:-1] == full).all()
    assert (out[0, :, 0, 1:-1] == full * 6 // 9).all() and (out[0, :, 1:-1, 0] == full * 6 // 9).all()
    assert (out[0, :, -1, 1:-1] == full * 6 // 9).all() and (out[0, :, 1:-1, -1] == full * 6 // 9).all()
    for r, c in ((0, 0), (0, -1), (-1, 0), (-1, -1)):
        assert (out[0, :, r, c] == full * 4 // 9).all()


def test_conv2d_1x1_is_matrix_product():
    rng = np.random.default_rng(11)
    x = rng.integers(0, 16, (3, 6, 4, 5))
    w = rng.integers(-8, 8, (7, 6, 1, 1))
    out = direct.conv2d_nchw(x, w, 0)
    ref = np.einsum("oc,bchw->bohw", w[:, :, 0, 0], x)
    assert np.array_equal(out, ref)


def test_conv2d_single_row_is_1d_correlation():
    rng = np.random.default_rng(12)
    row = rng.integers(-8, 8, 20)
    k = rng.integers(-8, 8, 3)
    x = row.reshape(1, 1, 1, 20)
    w = np.zeros((1, 1, 3, 3), dtype=np.int64)
    w[0, 0, 1, :] = k                       # only the middle kernel row is non-zero
    out = direct.conv2d_nchw(x, w, 1)[0, 0, 0]
    assert np.array_equal(out, np.correlate(np.pad(row, 1), k, mode="valid"))
    # the same through the 1-D oracle: correlation = convolution with the reversed kernel, read at K-1
    y = direct.conv1d_full(np.pad(row, 1), k[::-1])
    assert np.array_equal(out, y[2:2 + 20])


def test_conv2d_distinguishes_axes():
    # a kernel with a single 1 at (kh, kw) = (0, 2) picks I[h-1][w+1]: catches flips and transposes
    x = np.arange(2 * 3 * 4 * 5).reshape(2, 3, 4, 5)
    w = np.zeros((3, 3, 3, 3), dtype=np.int64)
    for c in range(3):
        w[c, c, 0, 2] = 1
    out = direct.conv2d_nchw(x, w, 1)
    expect = np.zeros_like(x)
    expect[:, :, 1:, :-1] = x[:, :, :-1, 1:]
    assert np.array_equal(out, expect)


# ---------------------------------------------------------------- requantize / pool / pack

def test_requant_exhaustive():
    acc = np.arange(-600, 600)
    for shift in (0, 1, 3, 6):
        for lo, hi in ((-8, 7), (0, 15)):
            got = direct.requant(acc, shift, lo, hi)
            expect = [min(max(int(a) // (1 << shift), lo), hi) for a in acc]   # Python // floors
            assert got.tolist() == expect


def test_maxpool_vs_numpy():
    rng = np.random.default_rng(5)
    x = rng.integers(-20, 20, (2, 3, 6, 10))
    ref = x.reshape(2, 3, 3, 2, 5, 2).max(axis=(3, 5))
    assert np.array_equal(direct.maxpool2x2(x), ref)
    odd = rng.integers(-20, 20, (1, 1, 5, 7))
    assert direct.maxpool2x2(odd).shape == (1, 1, 2, 3)
    assert np.array_equal(direct.maxpool2x2(odd), odd[:, :, :4, :6].reshape(1, 1, 2, 2, 3, 2).max(axis=(3, 5)))


def test_relu_requant_pool_commute():
    # clamp, floor-shift and max are all non-decreasing, so pooling before or after gives the same codes
    rng = np.random.default_rng(6)
    acc = rng.integers(-5000, 5000, (1, 2, 8, 8))
    a = direct.maxpool2x2(direct.requant(acc, 5, 0, 15))
    b = direct.requant(direct.maxpool2x2(acc), 5, 0, 15)
    assert np.array_equal(a, b)


def test_pack_words_against_python_ints():
    rng = np.random.default_rng(9)
    for signed in (False, True):
        for (S, N, bits) in ((10, 3, 32), (13, 3, 32), (16, 2, 32), (3, 11, 32), (10, 6, 64), (21, 3, 64)):
            lo, hi = (-8, 8) if signed else (0, 16)
            v = rng.integers(lo, hi, 50)
            words = direct.pack_words(v, S, N, bits)
            padded = list(v) + [0] * (-len(v) % N)
            for x, wv in enumerate(words):
                exact = sum(int(padded[x * N + n]) << (S * n) for n in range(N))
                assert int(wv) == exact % (1 << bits)


def test_count_out_of_range_against_enumeration():
    # every int8 value against every width, by the definition of a p-bit code: representable values are
    # exactly those that survive a round trip through p bits
    vals = np.arange(-128, 256)
    for bits in range(1, 9):
        for signed in (False, True):
            def representable(v):
                u = v & ((1 << bits) - 1)
                back = u - (1 << bits) if signed and (u >> (bits - 1)) else u
                return back == v
            want = sum(0 if representable(int(v)) else 1 for v in vals)
            assert direct.count_out_of_range(vals, bits, signed) == want
    assert direct.count_out_of_range([0, 15, 16, -1], 4, False) == 2
    assert direct.count_out_of_range([-8, 7, 8, -9], 4, True) == 2


def test_pack_words_printed_multiplicands():
    # Section V-A-2's worked example: f = (11, 9, 7) and g = (3, 2) with S = 10 are printed packed as 11543559
    # and 3074, element 0 in the TOP slot; Eq. 5 puts element 0 in the lowest slot, so the mirrored sequences
    # must reproduce the printed words, and the product of the two words must be the printed one
    g = _golden("worked_example_f32.txt")
    f = [int(t) for t in g["f"].split()]
    k = [int(t) for t in g["g"].split()]
    S = int(g["S"])
    wf = direct.pack_words(f[::-1], S, len(f), 32)
    wg = direct.pack_words(k[::-1], S, len(k), 32)
    assert wf.tolist() == [int(g["multiplicand_f"])] and wg.tolist() == [int(g["multiplicand_g"])]
    assert int(wf[0]) * int(wg[0]) == int(g["product"])
    # a second block and a ragged tail: (11, 9, 7, 5) in blocks of three -> the printed word and 5 alone
    assert direct.pack_words([7, 9, 11, 5], S, 3, 64).tolist() == [int(g["multiplicand_f"]), 5]
    # signed codes: Eq. 28's slot-by-slot form, written out by hand for (-1, 2) at S = 4: slot 0 holds 15,
    # slot 1 holds 2 - 1 (the borrow of the negative slot below): 0x1F
    assert direct.pack_words([-1, 2], 4, 2, 32).tolist() == [0x1F]
    # (-1, -1): slot 0 holds 15, slot 1 holds -1 - 1 = 14 (mod 16), the sign fills the rest of the register
    assert direct.pack_words([-1, -1], 4, 2, 32).tolist() == [0xFFFFFFEF]


def _torch_network(x, layers, head_w):
    """The same chain through library routines: float64 conv2d (exact below 2^53), floor division by 2^shift,
    clamp, max_pool2d."""
    a = torch.tensor(np.asarray(x), dtype=torch.float64)
    acts = []
    for L in layers:
        a = torch.nn.functional.conv2d(a, torch.tensor(np.asarray(L["w"]), dtype=torch.float64), padding=L["pad"])
        a = torch.clamp(torch.floor(a / float(1 << L["shift"])), L["lo"], L["hi"])
        if L["pool"]:
            a = torch.nn.functional.max_pool2d(a, 2, 2)
        acts.append(a.numpy().astype(np.int64))
    head = torch.nn.functional.conv2d(a, torch.tensor(np.asarray(head_w), dtype=torch.float64))
    return head.numpy().astype(np.int64), acts


def test_cnn_forward_vs_library_chain():
    # a pooled layer, an unpooled one, a signed clamp range and the pad-0 1x1 head; odd sizes so that the pool
    # drops a row and a column
    rng = np.random.default_rng(77)
    x = rng.integers(0, 256, (2, 3, 11, 14))
    layers = [
        {"w": rng.integers(-8, 8, (5, 3, 3, 3)), "pad": 1, "shift": 7, "lo": 0, "hi": 15, "pool": True},
        {"w": rng.integers(-8, 8, (6, 5, 3, 3)), "pad": 1, "shift": 3, "lo": 0, "hi": 15, "pool": False},
        {"w": rng.integers(-8, 8, (4, 6, 3, 3)), "pad": 0, "shift": 4, "lo": -8, "hi": 7, "pool": True},
    ]
    head_w = rng.integers(-8, 8, (7, 4, 1, 1))
    head, acts = direct.cnn_forward(x, layers, head_w)
    ref_head, ref_acts = _torch_network(x, layers, head_w)
    assert [a.shape for a in acts] == [(2, 5, 5, 7), (2, 6, 5, 7), (2, 4, 1, 2)]
    for a, r in zip(acts, ref_acts):
        assert np.array_equal(a, r)
    assert head.shape == (2, 7, 1, 2) and np.array_equal(head, ref_head)
    # the activations are not degenerate: the clamps bite on both sides somewhere and the values spread
    assert acts[0].min() == 0 and acts[0].max() == 15 and len(np.unique(acts[1])) > 4


def test_cnn_forward_one_pixel_network_by_hand():
    # 1x1 input, one channel, 1x1 kernels: layer 1: 200 * 3 = 600 >> 4 = 37 -> clamp [0, 15] = 15;
    # layer 2: 15 * (-2) = -30 >> 2 = floor(-7.5) = -8 -> clamp [-8, 7] = -8; head: -8 * 5 = -40
    layers = [{"w": [[[[3]]]], "pad": 0, "shift": 4, "lo": 0, "hi": 15, "pool": False},
              {"w": [[[[-2]]]], "pad": 0, "shift": 2, "lo": -8, "hi": 7, "pool": False}]
    head, acts = direct.cnn_forward([[[[200]]]], layers, [[[[5]]]])
    assert [int(a.ravel()[0]) for a in acts] == [15, -8] and int(head.ravel()[0]) == -40
