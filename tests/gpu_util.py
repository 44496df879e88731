"""Helpers shared by the GPU parity tests: move code arrays to the device, compare bit-exactly."""
import numpy as np
import torch

from paper_2208_00763_b200 import inputs


def dev(values):
    return torch.from_numpy(inputs.to_storage(values)).cuda()


def host_i64(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().astype(np.int64)


def assert_exact(got: torch.Tensor, ref: np.ndarray, what: str = ""):
    torch.cuda.synchronize()
    g = host_i64(got)
    assert g.shape == ref.shape, "%s: shape %s vs %s" % (what, g.shape, ref.shape)
    if not np.array_equal(g, ref):
        bad = np.argwhere(g != ref)
        first = tuple(bad[0])
        raise AssertionError("%s: %d of %d values differ, first at %s: got %d, expected %d"
                             % (what, len(bad), ref.size, first, g[first], ref[first]))
