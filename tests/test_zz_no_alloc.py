"""GPU check of the allocation-free layer entry point.

``hikonv_conv2d_static_scratch`` serves callers that cannot hand the library any device scratch
(they own only the input and output tensors, or may not allocate once their service has started).
It must give exactly what ``hikonv_conv2d`` gives with a caller-provided workspace (and what the
oracle gives), on consecutive calls that reuse the built-in buffer with different contents, without
taking any device memory, up to the very capacity of that buffer, and it must refuse layers whose
packed rows do not fit it.  This file sorts last on purpose, so a run that stops at the
first failure has already exercised every other test.
"""
import numpy as np
import pytest
import torch

from oracle import direct
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs

pytestmark = pytest.mark.gpu


def _case(B, Ci, H, W, Co, K, p, q, xs, ws, seed, with_values=False):
    x, w = inputs.conv2d_case(B, Ci, H, W, Co, K, p, q, xs, ws, seed)
    d = (torch.from_numpy(inputs.to_storage(x)).cuda(), torch.from_numpy(inputs.to_storage(w)).cuda())
    return d + (x, w) if with_values else d


def test_static_scratch_matches_workspace_path_on_consecutive_calls():
    # two different layers back to back: the second call finds the first call's words in the buffer
    calls = [
        dict(shape=(2, 24, 10, 14, 20, 3), p=4, q=4, xs=True, ws=True, pad=1, requant=None, algo=hk.ALGO_PACKED32),
        dict(shape=(3, 7, 9, 11, 33, 5), p=4, q=4, xs=False, ws=True, pad=2, requant=(4, 0, 15), algo=hk.ALGO_PACKED32),
        dict(shape=(1, 12, 8, 8, 16, 3), p=8, q=4, xs=False, ws=True, pad=1, requant=None, algo=hk.ALGO_UNPACKED_IMAD),
    ]
    for rep in range(2):
        for i, c in enumerate(calls):
            B, Ci, H, W, Co, K = c["shape"]
            d_x, d_w, x, w = _case(B, Ci, H, W, Co, K, c["p"], c["q"], c["xs"], c["ws"], seed=100 + 10 * rep + i, with_values=True)
            ref = hk.conv2d(d_x, d_w, c["pad"], c["p"], c["q"], c["xs"], c["ws"], requant=c["requant"], algo=c["algo"])
            out = torch.empty_like(ref)
            hk.conv2d_static_scratch(d_x, d_w, c["pad"], c["p"], c["q"], c["xs"], c["ws"], out, requant=c["requant"],
                                     algo=c["algo"])
            torch.cuda.synchronize()
            assert torch.equal(out, ref), "call %d of round %d differs from the workspace path" % (i, rep)
            want = direct.conv2d_nchw(x, w, c["pad"])
            if c["requant"]:
                want = direct.requant(want, *c["requant"])
            assert np.array_equal(out.cpu().numpy().astype(np.int64), want), "call %d of round %d differs from the oracle" % (i, rep)


def test_static_scratch_takes_no_device_memory():
    # after a first call (which looks up the buffer's address), a call with a preallocated output must leave both
    # the driver's free-memory figure and torch's allocator untouched
    d_x, d_w = _case(2, 16, 12, 20, 24, 3, 4, 4, True, True, seed=7)
    out = torch.empty((2, 24, 12, 20), dtype=torch.int32, device="cuda")
    hk.conv2d_static_scratch(d_x, d_w, 1, 4, 4, True, True, out)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    torch_before = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
    for _ in range(3):
        hk.conv2d_static_scratch(d_x, d_w, 1, 4, 4, True, True, out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == torch_before


def test_static_scratch_at_its_capacity():
    # the largest batch of this layer whose packed rows still fit the built-in buffer, and the next one
    Ci, H, W, Co, K, pad = 16, 24, 24, 16, 3, 1
    B = 1
    while hk.conv2d_workspace_bytes(B + 1, Ci, H, W, Co, K, pad) <= hk.STATIC_SCRATCH_BYTES:
        B += 1
    assert hk.conv2d_workspace_bytes(B, Ci, H, W, Co, K, pad) > 0.9 * hk.STATIC_SCRATCH_BYTES, "layer does not come near the limit"
    d_x, d_w, x, w = _case(B + 1, Ci, H, W, Co, K, 4, 4, False, True, seed=9, with_values=True)
    out = torch.empty((B, Co, H, W), dtype=torch.int32, device="cuda")
    hk.conv2d_static_scratch(d_x[:B], d_w, pad, 4, 4, False, True, out)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().astype(np.int64), direct.conv2d_nchw(x[:B], w, pad))
    over = torch.empty((B + 1, Co, H, W), dtype=torch.int32, device="cuda")
    with pytest.raises(hk.HikonvError) as err:
        hk.conv2d_static_scratch(d_x, d_w, pad, 4, 4, False, True, over)
    assert err.value.status == hk.ERR_TOO_LARGE


def test_static_scratch_checks_its_output_tensor():
    # the caller computes the output shape here, so a wrong one must be refused before any kernel sees its address
    d_x, d_w = _case(1, 4, 6, 6, 4, 3, 4, 4, True, True, seed=3)
    for bad in (torch.empty((1, 4, 6, 5), dtype=torch.int32, device="cuda"),
                torch.empty((1, 4, 6, 6), dtype=torch.int8, device="cuda"),
                torch.empty((1, 4, 6, 12), dtype=torch.int32, device="cuda")[..., ::2],
                torch.empty((1, 4, 6, 6), dtype=torch.int32)):
        with pytest.raises(ValueError):
            hk.conv2d_static_scratch(d_x, d_w, 1, 4, 4, True, True, bad)


def test_static_scratch_rejects_layers_beyond_its_capacity():
    # 512 x 512 x 3 x 3 needs 512*3*3*512*4 bytes = 9.4 MB of packed kernel rows alone: more than the built-in 4 MiB
    assert hk.conv2d_workspace_bytes(1, 512, 4, 4, 512, 3, 1) > hk.STATIC_SCRATCH_BYTES
    d_x = torch.zeros((1, 512, 4, 4), dtype=torch.int8, device="cuda")
    d_w = torch.zeros((512, 512, 3, 3), dtype=torch.int8, device="cuda")
    out = torch.empty((1, 512, 4, 4), dtype=torch.int32, device="cuda")
    with pytest.raises(hk.HikonvError) as err:
        hk.conv2d_static_scratch(d_x, d_w, 1, 4, 4, True, True, out)
    assert err.value.status == hk.ERR_TOO_LARGE
    assert "static buffer" in hk.status_string(hk.ERR_TOO_LARGE)
