"""GPU parity, 2-D layers and the compact CNN, against the int64 oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import direct
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs
from paper_2208_00763_b200 import network
from gpu_util import assert_exact, dev

pytestmark = pytest.mark.gpu

ALGOS = [hk.ALGO_PACKED32, hk.ALGO_UNPACKED_IMAD]


def _layer(x, w, pad, p, q, xs, ws, algo, requant=None, tune=None):
    return hk.conv2d(dev(x), dev(w), pad, p, q, xs, ws, requant=requant, algo=algo, tune=tune)


SHAPES = [
    # B, Ci, H, W, Co, K, pad
    (1, 1, 1, 1, 1, 1, 0),
    (1, 3, 5, 7, 2, 3, 1),
    (2, 5, 9, 11, 7, 3, 1),
    (3, 16, 14, 14, 40, 3, 1),      # several images per tile
    (2, 8, 6, 70, 20, 3, 1),        # wide rows: row segments
    (1, 4, 20, 300, 16, 3, 1),
    (2, 6, 8, 9, 5, 3, 0),          # valid convolution
    (1, 7, 10, 12, 9, 5, 2),        # 5x5: the kernel row is cut into chunks
    (2, 3, 9, 10, 4, 7, 3),
    (2, 12, 5, 6, 36, 1, 0),        # 1x1
    (1, 2, 4, 5, 3, 2, 1),          # even kernel
    (5, 9, 3, 4, 70, 3, 1),         # more than 64 output channels, tiny images
]


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("shape", SHAPES)
def test_layer_shapes(shape, algo):
    B, Ci, H, W, Co, K, pad = shape
    for (p, q, xs, ws) in ((4, 4, True, True), (4, 4, False, True), (8, 4, False, True), (2, 2, False, False)):
        x, w = inputs.conv2d_case(B, Ci, H, W, Co, K, p, q, xs, ws, seed=sum(shape) + p)
        ref = direct.conv2d_nchw(x, w, pad)
        assert_exact(_layer(x, w, pad, p, q, xs, ws, algo), ref, "%s p=%d q=%d" % (shape, p, q))


@pytest.mark.parametrize("bits", range(1, 9))
def test_every_bitwidth(bits):
    # 3x3 and pointwise layers; shallow (no carry-save moves) and deep enough to need them
    for signed in (False, True):
        for (Ci, K, pad) in ((10, 3, 1), (10, 1, 0), (150, 3, 1), (150, 1, 0)):
            x, w = inputs.conv2d_case(2, Ci, 7, 13, 12, K, bits, bits, signed, signed, seed=bits + Ci + K)
            ref = direct.conv2d_nchw(x, w, pad)
            for algo in ALGOS:
                assert_exact(_layer(x, w, pad, bits, bits, signed, signed, algo), ref,
                             "bits=%d signed=%d Ci=%d K=%d algo=%d" % (bits, signed, Ci, K, algo))


@pytest.mark.parametrize("n", [1, 2, 3, 4])
def test_forced_words_per_block(n):
    # four 4-bit codes per word leave no room to accumulate even one channel, so N = 4 runs on narrower codes
    for bits in ((4,) if n < 4 else (2, 3)):
        x, w = inputs.conv2d_case(2, 40, 9, 17, 24, 3, bits, bits, True, True, seed=40 + n)
        ref = direct.conv2d_nchw(x, w, 1)
        run = lambda tune: _layer(x, w, 1, bits, bits, True, True, hk.ALGO_PACKED32, tune=tune)
        assert_exact(run({"N": n}), ref, "N=%d" % n)
        # the shortest split period the kernel accepts (one channel's three kernel rows): a split after every channel
        assert_exact(run({"N": n, "M": 3}), ref, "N=%d M=3" % n)
        assert_exact(run({"N": n, "tile": 1}), ref, "N=%d one row per tile" % n)
        with pytest.raises(hk.HikonvError):
            run({"N": n, "M": 1})
    if n == 4:
        x, w = inputs.conv2d_case(1, 4, 5, 9, 4, 3, 4, 4, True, True, seed=1)
        with pytest.raises(hk.HikonvError):
            _layer(x, w, 1, 4, 4, True, True, hk.ALGO_PACKED32, tune={"N": 4})


@pytest.mark.parametrize("ci", [4, 7, 20, 64, 130, 256])
def test_carry_save_schedules(ci):
    # 3x3 layers at N = 3, S = 13 move slot bits to the second accumulator at stage ends (s4 x s4, and any layer
    # with tile < 0) or at fixed places inside groups of 3 or 4 channels (u4 x s4, by depth); channel counts that
    # are not multiples of the group leave zero-weight channels in the last group
    for (xs, ws) in ((True, True), (False, True)):
        x, w = inputs.conv2d_case(2, ci, 6, 17, 12, 3, 4, 4, xs, ws, seed=300 + ci)
        ref = direct.conv2d_nchw(x, w, 1)
        for tune in (None, {"tile": -1}):
            assert_exact(_layer(x, w, 1, 4, 4, xs, ws, hk.ALGO_PACKED32, tune=tune), ref, "ci=%d xs=%d tune=%s" % (ci, xs, tune))
    for x, w in inputs.extreme_2d(1, ci, 5, 9, 8, 3, 4, 4, False, True):
        for tune in (None, {"tile": -1}):
            assert_exact(_layer(x, w, 1, 4, 4, False, True, hk.ALGO_PACKED32, tune=tune), direct.conv2d_nchw(x, w, 1), "extreme ci=%d" % ci)


@pytest.mark.parametrize("p", [1, 2, 3, 4, 5, 6, 8])
def test_deep_unsigned_layers_on_shifted_codes(p):
    # unsigned activations x signed weights with 128 or more input channels may be packed as x - 2^(p-1) (the padding
    # included) and get 2^(p-1) * (the channel's weight sum) back in the epilogue: image borders, valid convolution,
    # several kernel sizes, channel counts that are not multiples of four, requantised output, extreme codes
    for (K, pad, q, Co) in ((3, 1, 4, 7), (3, 0, 2, 4), (1, 0, 4, 18), (5, 2, 2, 5), (3, 2, 3, 6)):
        x, w = inputs.conv2d_case(2, 131, 6, 11, Co, K, p, q, False, True, seed=7000 + 10 * p + K + pad)
        ref = direct.conv2d_nchw(x, w, pad)
        assert_exact(_layer(x, w, pad, p, q, False, True, hk.ALGO_PACKED32), ref, "p=%d q=%d K=%d pad=%d" % (p, q, K, pad))
        rq = (p + q - 2, 0, 15)
        assert_exact(_layer(x, w, pad, p, q, False, True, hk.ALGO_PACKED32, requant=rq), direct.requant(ref, *rq),
                     "requant p=%d q=%d K=%d pad=%d" % (p, q, K, pad))
    for x, w in inputs.extreme_2d(1, 160, 5, 9, 6, 3, p, 4, False, True):
        assert_exact(_layer(x, w, 1, p, 4, False, True, hk.ALGO_PACKED32), direct.conv2d_nchw(x, w, 1), "extreme p=%d" % p)


@pytest.mark.parametrize("algo", ALGOS)
def test_extreme_codes(algo):
    for (p, q, xs, ws) in ((4, 4, True, True), (4, 4, False, True), (8, 4, False, True), (8, 8, True, True), (1, 1, True, True)):
        for x, w in inputs.extreme_2d(2, 70, 6, 10, 8, 3, p, q, xs, ws):
            assert_exact(_layer(x, w, 1, p, q, xs, ws, algo), direct.conv2d_nchw(x, w, 1), "extreme p=%d q=%d" % (p, q))


@pytest.mark.parametrize("algo", ALGOS)
def test_unaligned_input_pointer(algo):
    # an input that does not start on a 4-byte boundary takes the byte-wise row fetch
    x, w = inputs.conv2d_case(2, 9, 7, 13, 8, 3, 4, 4, True, True, seed=91)
    ref = direct.conv2d_nchw(x, w, 1)
    flat = torch.zeros(x.size + 8, dtype=torch.int8, device="cuda")
    for shift in (1, 2, 3):
        flat[shift:shift + x.size] = dev(x).reshape(-1)
        view = flat[shift:shift + x.size].view(2, 9, 7, 13)
        assert view.data_ptr() % 4 == shift
        assert_exact(hk.conv2d(view, dev(w), 1, 4, 4, True, True, algo=algo), ref, "offset %d" % shift)


@pytest.mark.parametrize("algo", ALGOS)
def test_requantize(algo):
    x, w = inputs.conv2d_case(2, 32, 10, 12, 16, 3, 4, 4, True, True, seed=77)
    acc = direct.conv2d_nchw(x, w, 1)
    for (shift, lo, hi) in ((6, -8, 7), (0, -128, 127), (5, 0, 15), (3, 0, 255)):
        got = _layer(x, w, 1, 4, 4, True, True, algo, requant=(shift, lo, hi))
        torch.cuda.synchronize()
        g = got.cpu().numpy()
        g = g.astype(np.int64) if lo < 0 else g.view(np.uint8).astype(np.int64)
        assert np.array_equal(g, direct.requant(acc, shift, lo, hi)), (shift, lo, hi)


@pytest.mark.parametrize("algo", ALGOS)
def test_c3_layer_every_image(algo):
    # full-size launch (batch 32); the oracle checks all 32 images of it, codes and (packed algorithm) exact sums
    s = inputs.C3_SHAPE
    x, w = inputs.layer_case(s)
    acc = direct.conv2d_nchw(x, w, s["pad"])
    got = _layer(x, w, s["pad"], s["p"], s["q"], s["x_signed"], s["w_signed"], algo, requant=(s["shift"], s["lo"], s["hi"]))
    assert_exact(got, direct.requant(acc, s["shift"], s["lo"], s["hi"]), "C3 codes")
    if algo == hk.ALGO_PACKED32:
        assert_exact(_layer(x, w, s["pad"], s["p"], s["q"], s["x_signed"], s["w_signed"], algo), acc, "C3 sums")


@pytest.mark.parametrize("algo", ALGOS)
def test_c4_layer_every_image(algo):
    # full-size launch (batch 64), all 64 images against the oracle
    s = inputs.C4_SHAPE
    x, w = inputs.layer_case(s)
    assert abs(float((x == 0).mean()) - (0.3 + 0.7 / 16)) < 0.01
    got = _layer(x, w, s["pad"], s["p"], s["q"], s["x_signed"], s["w_signed"], algo)
    assert_exact(got, direct.conv2d_nchw(x, w, s["pad"]), "C4 sums")


def test_host_buffer_entry_point():
    x, w = inputs.conv2d_case(2, 8, 9, 10, 12, 3, 4, 4, False, True, seed=5)
    h_x = torch.from_numpy(inputs.to_storage(x)).pin_memory()
    h_w = torch.from_numpy(inputs.to_storage(w)).pin_memory()
    h_o = torch.empty((2, 12, 9, 10), dtype=torch.int32).pin_memory()
    ws = torch.empty(hk.conv2d_host_workspace_bytes(2, 8, 9, 10, 12, 3, 1, False), dtype=torch.uint8, device="cuda")
    hk.conv2d_host(h_x, h_w, 1, 4, 4, False, True, h_o, ws)
    torch.cuda.synchronize()
    assert np.array_equal(h_o.numpy().astype(np.int64), direct.conv2d_nchw(x, w, 1))


@pytest.mark.parametrize("algo", ALGOS)
def test_compact_cnn_small_batch(algo):
    x, layers, head_w = inputs.c5_network(batch=2, H=32, W=64)
    ref_head, ref_acts = direct.cnn_forward(x, layers, head_w)
    net = network.CompactCnn(layers, head_w, device="cuda")
    head, acts = net.forward(dev(x), algo=algo, keep_activations=True)
    for i, (a, r) in enumerate(zip(acts, ref_acts)):
        assert_exact(a, r, "layer %d" % (i + 1))
    assert_exact(head, ref_head, "head")


@pytest.mark.parametrize("fused_pool", [True, False])
def test_compact_cnn_with_pools_fused_into_the_layers_or_launched_apart(fused_pool):
    x, layers, head_w = inputs.c5_network(batch=3, H=32, W=64)
    ref_head, ref_acts = direct.cnn_forward(x, layers, head_w)
    net = network.CompactCnn(layers, head_w, device="cuda")
    head, acts = net.forward(dev(x), keep_activations=True, fused_pool=fused_pool)
    for i, (a, r) in enumerate(zip(acts, ref_acts)):
        assert_exact(a, r, "layer %d" % (i + 1))
    assert_exact(head, ref_head, "head")


def test_compact_cnn_full_size_every_image():
    # the benchmark configuration (batch 64, 3x160x320): head output and every layer's activations of all 64
    # images against the oracle (the oracle runs the batch in four parts to bound its int64 buffers)
    # ... once with the library's own tiles, once with the tiles the network's tuning pass picks on the device
    x, layers, head_w = inputs.c5_network()
    net = network.CompactCnn(layers, head_w, device="cuda")
    d_x = dev(x)
    results = [net.forward(d_x, keep_activations=True)]
    kept = net.tune_tiles(d_x)
    assert len(kept) == len(layers) and all(t is None or t["tile"] > 0 for t in kept)
    results.append(net.forward(d_x, keep_activations=True))
    torch.cuda.synchronize()
    got = [(head.cpu().numpy().astype(np.int64), [a.cpu().numpy() for a in acts]) for head, acts in results]
    assert got[0][0].shape == (64, 36, 10, 20)
    for b0 in range(0, 64, 16):
        ref_head, ref_acts = direct.cnn_forward(x[b0:b0 + 16], layers, head_w)
        for which, (g, g_acts) in enumerate(got):
            assert np.array_equal(g[b0:b0 + 16], ref_head), "head, images %d..%d, pass %d" % (b0, b0 + 15, which)
            for i, (a, r) in enumerate(zip(g_acts, ref_acts)):
                assert np.array_equal(a[b0:b0 + 16].astype(np.int64), r), "layer %d, images %d..%d, pass %d" % (i + 1, b0, b0 + 15, which)


@pytest.mark.parametrize("co", [8, 12, 16, 24, 40, 72])
def test_first_layer_kernel_with_eight_or_four_channels_per_thread(co):
    # 8-bit activations, few input channels: the kernel without second accumulators holds eight output channels per
    # thread when the channel count is a multiple of eight, four otherwise; ragged rows, several row segments, several
    # images per tile, exact sums and requantised codes
    for (B, Ci, H, W) in ((2, 3, 9, 21, ), (1, 1, 5, 300), (5, 2, 3, 7), (1, 3, 33, 64)):
        L = hk.conv2d_layout(B, Ci, H, W, co, 3, 1, 8, 4, False, True)
        assert (L["N"], L["J"]) == (2, 2) and L["M"] >= Ci * 3 and L["S"] == (17 if Ci > 1 else 16)    # one channel: the general kernel
        x, w = inputs.conv2d_case(B, Ci, H, W, co, 3, 8, 4, False, True, seed=4000 + co + W)
        ref = direct.conv2d_nchw(x, w, 1)
        assert_exact(_layer(x, w, 1, 8, 4, False, True, hk.ALGO_PACKED32), ref, "co=%d %s" % (co, (B, Ci, H, W)))
        assert_exact(_layer(x, w, 1, 8, 4, False, True, hk.ALGO_PACKED32, requant=(8, 0, 15)), direct.requant(ref, 8, 0, 15),
                     "requant co=%d %s" % (co, (B, Ci, H, W)))
    for x, w in inputs.extreme_2d(2, 3, 6, 10, co, 3, 8, 4, False, True):
        assert_exact(_layer(x, w, 1, 8, 4, False, True, hk.ALGO_PACKED32), direct.conv2d_nchw(x, w, 1), "extreme co=%d" % co)


def test_tuner_times_tiles_and_returns_one_that_gives_the_same_result():
    for (B, Ci, H, W, Co, p, xs, pool) in ((4, 16, 12, 20, 24, 4, True, False), (8, 64, 10, 20, 64, 4, False, True), (2, 3, 16, 40, 16, 8, False, False)):
        x, w = inputs.conv2d_case(B, Ci, H, W, Co, 3, p, 4, xs, True, seed=77 + Ci)
        rq = (6, -8, 7) if xs else (6, 0, 15)
        want = direct.requant(direct.conv2d_nchw(x, w, 1), *rq)
        if pool:
            want = direct.maxpool2x2(want)
        d_x, d_w = dev(x), dev(w)
        found = hk.conv2d_tune(d_x.reshape(-1), x.shape, 8, d_w.reshape(-1), w.shape, 8, 1, p, 4, xs, True, requant=rq, pool=pool, repeats=2)
        assert found["us"] > 0 and found["default_us"] > 0 and found["us"] <= found["default_us"]
        assert found["tune"] is None or (found["tune"]["tile"] > 0 and found["us"] <= 0.97 * found["default_us"])
        assert_exact(found["out"], want, "output left by the tuner")
        again = hk.conv2d_dense(d_x.reshape(-1), x.shape, 8, d_w.reshape(-1), w.shape, 8, 1, p, 4, xs, True, requant=rq, pool=pool,
                                tune=found["tune"])
        assert_exact(again, want, "layer with the tuned tile %s" % (found["tune"],))
    # argument errors come back as they would from the layer call
    with pytest.raises(hk.HikonvError) as err:
        hk.conv2d_tune(d_x.reshape(-1), x.shape, 8, d_w.reshape(-1), w.shape, 8, 5, p, 4, xs, True, requant=rq)      # pad >= K
    assert err.value.status == hk.ERR_UNSUPPORTED


def test_layer_chain_captured_in_a_cuda_graph():
    # a layer, a requantised layer and a pool captured once and replayed: the kernels are launched with
    # programmatic dependencies, which a captured graph has to preserve
    x, w = inputs.conv2d_case(2, 16, 12, 20, 24, 3, 4, 4, True, True, seed=3)
    d_x, d_w = dev(x), dev(w)
    ws = torch.empty(hk.conv2d_workspace_bytes(2, 16, 12, 20, 24, 3, 1), dtype=torch.uint8, device="cuda")
    out = torch.empty((2, 24, 12, 20), dtype=torch.int32, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        hk.conv2d(d_x, d_w, 1, 4, 4, True, True, workspace=ws, out=out)          # first call outside the capture
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        hk.conv2d(d_x, d_w, 1, 4, 4, True, True, workspace=ws, out=out)
        o8 = hk.conv2d(d_x, d_w, 1, 4, 4, True, True, requant=(6, -8, 7), workspace=ws)
        pooled = hk.maxpool2x2_i8(o8, True)
    out.zero_()
    graph.replay()
    graph.replay()
    ref = direct.conv2d_nchw(x, w, 1)
    assert_exact(out, ref, "captured layer")
    assert_exact(pooled, direct.maxpool2x2(direct.requant(ref, 6, -8, 7)), "captured requantised layer and pool")
