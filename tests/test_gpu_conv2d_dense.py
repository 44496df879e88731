"""GPU parity of ``hikonv_conv2d_dense`` (densely stored activations, weights and requantised outputs, optional fused
2x2 max-pool) against the int64 oracle on code values, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import direct
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs
from gpu_util import assert_exact

pytestmark = pytest.mark.gpu

ALGOS = [hk.ALGO_PACKED32, hk.ALGO_UNPACKED_IMAD]


def _store(values, bits, store_bits):
    """Device tensor of the codes: one per byte (store_bits == 8) or dense."""
    if store_bits == 8:
        return torch.from_numpy(inputs.to_storage(values).reshape(-1)).cuda()
    assert store_bits == bits
    return torch.from_numpy(inputs.to_dense(values, bits)).cuda()


def _reference(x, w, pad, requant, pool):
    acc = direct.conv2d_nchw(x, w, pad)
    if not requant:
        return acc
    out = direct.requant(acc, *requant)
    return direct.maxpool2x2(out) if pool else out


def _run(x, w, pad, p, q, xs, ws, x_store, w_store, requant, out_store, pool, algo, tune=None):
    got = hk.conv2d_dense(_store(x, p, x_store), x.shape, x_store, _store(w, q, w_store), w.shape, w_store, pad, p, q, xs, ws,
                          requant=requant, out_store_bits=out_store, pool=pool, algo=algo, tune=tune)
    torch.cuda.synchronize()
    ref = _reference(x, w, pad, requant, pool)
    if not requant:
        return got.cpu().numpy().astype(np.int64), ref
    if out_store == 8:
        return inputs.from_storage(got.cpu().numpy(), requant[1] < 0), ref
    return inputs.from_dense(got.cpu().numpy(), ref.size, out_store, requant[1] < 0).reshape(ref.shape), ref


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("bits", [1, 2, 4])
def test_dense_inputs_and_weights(bits, algo):
    # every storage combination of activations and weights, both signs, exact int32 sums
    for xs, ws in ((False, False), (True, True), (False, True), (True, False)):
        for (B, Ci, H, W, Co, K, pad) in ((2, 5, 9, 11, 7, 3, 1), (1, 16, 12, 20, 24, 3, 1), (3, 3, 7, 13, 4, 5, 2), (2, 8, 6, 6, 8, 1, 0)):
            x, w = inputs.conv2d_case(B, Ci, H, W, Co, K, bits, bits, xs, ws, seed=bits * 100 + Ci + K)
            for x_store, w_store in ((bits, bits), (bits, 8), (8, bits)):
                got, ref = _run(x, w, pad, bits, bits, xs, ws, x_store, w_store, None, 32, False, algo)
                assert np.array_equal(got, ref), (bits, xs, ws, (B, Ci, H, W, Co, K, pad), x_store, w_store)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("pool", [False, True])
def test_dense_requantised_output(pool, algo):
    # 4-bit network layers: dense in, dense out (signed and unsigned clamp ranges), with and without the fused pool;
    # widths whose rows fill whole bytes, several row segments (W = 160) and ragged channel counts
    rng = np.random.default_rng(17)
    for (B, Ci, H, W, Co) in ((2, 16, 12, 20, 24), (1, 6, 10, 240, 5), (3, 32, 8, 40, 36), (2, 4, 16, 8, 3)):
        for xs, (shift, lo, hi) in ((True, (5, -8, 7)), (False, (6, 0, 15)), (False, (4, 0, 3)), (True, (7, -1, 0))):
            x, w = inputs.conv2d_case(B, Ci, H, W, Co, 3, 4, 4, xs, True, seed=int(rng.integers(1 << 30)))
            out_bits = 4 if hi > 3 or lo < -2 else (2 if hi > 1 or lo < -1 else 1)
            for out_store in (out_bits, 8):
                Wq = W // 2 if pool else W
                if (Wq * out_store) % 8 != 0:        # rows that do not fill whole bytes are refused, nothing is launched
                    with pytest.raises(hk.HikonvError) as err:
                        _run(x, w, 1, 4, 4, xs, True, 4, 4, (shift, lo, hi), out_store, pool, algo)
                    assert err.value.status == hk.ERR_UNSUPPORTED
                    continue
                got, ref = _run(x, w, 1, 4, 4, xs, True, 4, 4, (shift, lo, hi), out_store, pool, algo)
                assert np.array_equal(got, ref), ((B, Ci, H, W, Co), xs, (shift, lo, hi), out_store, pool)


def test_first_layer_bytes_in_dense_out_pooled():
    # 8-bit unsigned image (one code per byte) x dense 4-bit weights -> pooled dense 4-bit codes, as in the compact CNN
    x, w = inputs.conv2d_case(2, 3, 32, 64, 16, 3, 8, 4, False, True, seed=5)
    got, ref = _run(x, w, 1, 8, 4, False, True, 8, 4, (8, 0, 15), 4, True, hk.ALGO_PACKED32)
    assert np.array_equal(got, ref)


def test_deep_layer_dense_in_and_out_on_shifted_codes():
    # 128 and more input channels, unsigned dense activations against signed dense weights: the layer runs on codes
    # shifted by 2^(p-1); dense, pooled and plain outputs
    for (B, Ci, H, W, Co, bits) in ((2, 128, 8, 16, 12, 4), (1, 200, 6, 32, 5, 2), (2, 136, 4, 8, 9, 1)):
        x, w = inputs.conv2d_case(B, Ci, H, W, Co, 3, bits, 4 if bits == 4 else bits, False, True, seed=900 + Ci)
        q = 4 if bits == 4 else bits
        got, ref = _run(x, w, 1, bits, q, False, True, bits, q, None, 32, False, hk.ALGO_PACKED32)
        assert np.array_equal(got, ref), (B, Ci, H, W, Co, bits)
        for pool in (False, True):
            for out_store in (4, 8):
                got, ref = _run(x, w, 1, bits, q, False, True, bits, q, (bits + q - 1, 0, 15), out_store, pool, hk.ALGO_PACKED32)
                assert np.array_equal(got, ref), (B, Ci, H, W, Co, bits, pool, out_store)


def test_extreme_codes_dense():
    for xs, ws in ((True, True), (False, True)):
        for x, w in inputs.extreme_2d(2, 20, 8, 16, 9, 3, 4, 4, xs, ws):
            got, ref = _run(x, w, 1, 4, 4, xs, ws, 4, 4, (4, -8, 7) if xs else (4, 0, 15), 4, True, hk.ALGO_PACKED32)
            assert np.array_equal(got, ref)
            got, ref = _run(x, w, 1, 4, 4, xs, ws, 4, 4, None, 32, False, hk.ALGO_PACKED32)
            assert np.array_equal(got, ref)


def test_c3_layer_dense_every_image():
    # the 4-bit benchmark layer with all three tensors dense, all 32 images
    s = inputs.C3_SHAPE
    x, w = inputs.layer_case(s)
    got, ref = _run(x, w, s["pad"], 4, 4, True, True, 4, 4, (s["shift"], s["lo"], s["hi"]), 4, False, hk.ALGO_PACKED32)
    assert np.array_equal(got, ref)
    got, ref = _run(x, w, s["pad"], 4, 4, True, True, 4, 4, (s["shift"], s["lo"], s["hi"]), 4, True, hk.ALGO_PACKED32)
    assert np.array_equal(got, ref)


def test_refusals():
    x, w = inputs.conv2d_case(1, 4, 6, 7, 4, 3, 4, 4, False, True, seed=1)
    d_x, d_w = _store(x, 4, 4), _store(w, 4, 4)
    with pytest.raises(hk.HikonvError):      # rows of 7 four-bit codes do not fill whole bytes
        hk.conv2d_dense(d_x, x.shape, 4, d_w, w.shape, 4, 1, 4, 4, False, True, requant=(4, 0, 15), out_store_bits=4)
    with pytest.raises(hk.HikonvError):      # odd output size with the fused pool
        hk.conv2d_dense(d_x, x.shape, 4, d_w, w.shape, 4, 1, 4, 4, False, True, requant=(4, 0, 15), out_store_bits=8, pool=True)
    with pytest.raises(hk.HikonvError):      # clamp range wider than the stored width
        hk.conv2d_dense(d_x, x.shape, 4, d_w, w.shape, 4, 1, 4, 4, False, True, requant=(4, 0, 15), out_store_bits=2)
    x3, w3 = inputs.conv2d_case(1, 4, 6, 8, 4, 3, 3, 3, False, False, seed=2)
    with pytest.raises(hk.HikonvError):      # 3-bit codes straddle bytes: no dense format
        hk.conv2d_dense(_store(x3, 3, 8), x3.shape, 3, _store(w3, 3, 8), w3.shape, 8, 1, 3, 3, False, False)
