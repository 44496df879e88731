"""GPU check of the allocation-free layer entry point.

``hikonv_conv2d_static_scratch`` serves callers that cannot hand the library any device scratch
(they own only the input and output tensors, or may not allocate once their service has started).
It must give exactly what ``hikonv_conv2d`` gives with a caller-provided workspace, on consecutive
calls that reuse the built-in buffer with different contents, and it must refuse layers whose
packed rows do not fit that buffer.  This file sorts last on purpose, so a run that stops at the
first failure has already exercised every other test.
"""
import numpy as np
import pytest
import torch

from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import inputs

pytestmark = pytest.mark.gpu


def _case(B, Ci, H, W, Co, K, p, q, xs, ws, seed):
    x, w = inputs.conv2d_case(B, Ci, H, W, Co, K, p, q, xs, ws, seed)
    return (torch.from_numpy(inputs.to_storage(x)).cuda(), torch.from_numpy(inputs.to_storage(w)).cuda())


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
            d_x, d_w = _case(B, Ci, H, W, Co, K, c["p"], c["q"], c["xs"], c["ws"], seed=100 + 10 * rep + i)
            ref = hk.conv2d(d_x, d_w, c["pad"], c["p"], c["q"], c["xs"], c["ws"], requant=c["requant"], algo=c["algo"])
            out = torch.empty_like(ref)
            hk.conv2d_static_scratch(d_x, d_w, c["pad"], c["p"], c["q"], c["xs"], c["ws"], out, requant=c["requant"],
                                     algo=c["algo"])
            torch.cuda.synchronize()
            assert torch.equal(out, ref), "call %d of round %d differs from the workspace path" % (i, rep)


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
