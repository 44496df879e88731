"""The integer-pipe microbenchmark behind the "alu" rooflines: every kind runs and lands in the range the hardware
allows (at most 32 lanes per clock and SM for the 32x32->64 multiply-add, 64 for 32-bit integer instructions)."""
import pytest
import torch

from paper_2208_00763_b200 import binding as hk

pytestmark = pytest.mark.gpu


def test_every_kind_gives_a_plausible_rate():
    rates = {kind: hk.pipe_rate(kind, iters=512) for kind in hk.PIPE_KINDS}
    for kind, r in rates.items():
        assert r["ops_per_second"] > 0 and r["lanes_per_clock_per_sm"] > 0, kind
    for kind in ("mad_wide_u32", "mad_wide_s32"):
        assert 16.0 < rates[kind]["lanes_per_clock_per_sm"] <= 33.0, (kind, rates[kind])
    for kind in ("mad_lo_s32", "logic", "shift", "prmt"):
        assert 32.0 < rates[kind]["lanes_per_clock_per_sm"] <= 66.0, (kind, rates[kind])
    # logic instructions between the multiply-adds do not come for free, and cannot cost more than their own issue slots
    mixed, pure = rates["mad_wide_with_logic"]["lanes_per_clock_per_sm"], rates["mad_wide_u32"]["lanes_per_clock_per_sm"]
    assert 0.6 * pure < mixed <= 1.02 * pure, (mixed, pure)


def test_bad_arguments_are_refused():
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    for kind, iters in ((-1, 16), (len(hk.PIPE_KINDS), 16), (0, 0), (0, (1 << 20) + 1)):
        ops = hk.ctypes.c_double(0.0)
        rc = hk.lib().hikonv_pipe_rate(kind, iters, word.data_ptr(), hk.ctypes.byref(ops), None, None)
        assert rc == hk.ERR_INVALID_ARG, (kind, iters, rc)
