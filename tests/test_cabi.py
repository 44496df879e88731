"""CPU checks of the C interface: the library builds, loads and exports every declared entry
point; the host-only planning calls agree with the brute-force oracle and with the paper's
printed numbers; argument validation returns status codes without touching a GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import direct, packed_model as pm, plan as oplan
from paper_2208_00763_b200 import binding as hk
from paper_2208_00763_b200 import build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    lib_build.build()
    return hk.lib()


def _declared_names():
    text = open(os.path.join(ROOT, "include", "hikonv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hikonv_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared_names()
    assert "hikonv_pack" in names and "hikonv_conv1d" in names and "hikonv_conv2d" in names
    raw = ctypes.CDLL(hk.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), "library does not export %s" % n
    assert sorted(hk.exported_names()) == names


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(hk, "_lib", None)
    monkeypatch.setattr(hk, "LIB_PATH", os.path.join(ROOT, "does_not_exist.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        hk.lib()


@pytest.mark.parametrize("mode", [hk.GB_SINGLE, hk.GB_1D, hk.GB_DNN])
def test_plan_matches_bruteforce_oracle(mode):
    for LA, LB in ((32, 32), (27, 18)):
        for p in range(1, 9):
            for q in range(1, 9):
                for M in ((1,) if mode != hk.GB_DNN else (1, 4, 21)):
                    got = hk.plan(p, q, LA, LB, mode, M)
                    assert got == oplan.search(p, q, LA, LB, mode, M)
                    for K in (1, 3, 5):
                        ref = oplan.search(p, q, LA, LB, mode, M, K_fixed=K)
                        if ref["ops"] == 0:
                            with pytest.raises(hk.HikonvError):
                                hk.plan(p, q, LA, LB, mode, M, K)
                        else:
                            assert hk.plan(p, q, LA, LB, mode, M, K) == ref


def test_plan_printed_counts():
    assert hk.plan(4, 4)["ops"] == 13 and hk.plan(8, 8)["ops"] == 5
    assert hk.plan(1, 1, 27, 18)["ops"] == 60 and hk.plan(4, 4, 27, 18)["ops"] == 8 and hk.plan(8, 8, 27, 18)["ops"] == 2
    assert hk.plan(1, 1)["ops"] == 113 and hk.plan(1, 1, 33, 32)["ops"] == 128
    four = hk.plan(4, 4, 32, 32, hk.GB_1D, 1, 3)
    assert (four["N"], four["K"], four["Gb"], four["S"]) == (3, 3, 2, 10)


def test_plan_rejects_bad_arguments():
    out = hk.PlanT()
    lib = hk.lib()
    assert lib.hikonv_plan(0, 4, 32, 32, 0, 1, 0, ctypes.byref(out)) == hk.ERR_INVALID_ARG
    assert lib.hikonv_plan(4, 4, 32, 32, 7, 1, 0, ctypes.byref(out)) == hk.ERR_INVALID_ARG
    assert lib.hikonv_plan(4, 4, 32, 32, 0, 1, 0, None) == hk.ERR_INVALID_ARG
    assert lib.hikonv_plan(8, 8, 4, 4, 0, 1, 0, ctypes.byref(out)) == hk.ERR_NO_FIT
    assert hk.status_string(hk.ERR_NO_FIT) and hk.status_string(99) == "unknown status"


def _extreme_vectors(p, q, fs, gs, n, K):
    flo, fhi = (-(1 << (p - 1)), (1 << (p - 1)) - 1) if fs else (0, (1 << p) - 1)
    glo, ghi = (-(1 << (q - 1)), (1 << (q - 1)) - 1) if gs else (0, (1 << q) - 1)
    out = []
    for fv in (flo, fhi):
        for gv in (glo, ghi):
            out.append(([fv] * n, [gv] * K))
    out.append(([flo if i % 2 else fhi for i in range(n)], [ghi if i % 2 else glo for i in range(K)]))
    return out


def _model_conv1d(f, g, L, bias_per_slot, word_bits=32):
    """The kernel's arithmetic in big integers: chunked kernel, carries added before the split,
    slots lifted by a bias instead of Eq. 29's borrow increment; operands of `word_bits`, product of twice as many."""
    N, S, Kc, J = L["N"], L["S"], L["Kc"], L["J"]
    n_out = len(f) + len(g) - 1
    nb = (n_out + N - 1) // N
    fpad = list(f) + [0] * ((nb + 1) * N)
    A = [pm.pack(fpad[x * N:(x + 1) * N], S) for x in range(nb)]
    Bw = [pm.pack(g[j * Kc:(j + 1) * Kc], S) for j in range(J)]
    lim = 1 << (word_bits - 1)
    for a in A:
        assert (-lim <= a < lim) if L["signed_prod"] else (0 <= a < 2 * lim)
    for b in Bw:
        assert (-lim <= b < lim) if L["signed_prod"] else (0 <= b < 2 * lim)
    bias = sum(b << (S * m) for m, b in enumerate(bias_per_slot))
    y, prev_hi = [], bias >> (S * N)
    for x in range(nb):
        Q = bias + sum(A[x - j] * Bw[j] for j in range(J) if x - j >= 0)
        assert 0 <= Q < (1 << (2 * word_bits))
        D = Q + prev_hi
        for m in range(N):
            carry_bias = bias_per_slot[m] + (bias_per_slot[m + N] if m + N < len(bias_per_slot) else 0)
            y.append(((D >> (S * m)) & ((1 << S) - 1)) - carry_bias)
        prev_hi = Q >> (S * N)
    return y[:n_out]


@pytest.mark.parametrize("signed", [False, True])
def test_layout_1d_is_exact_on_extreme_codes(signed):
    # every (p, K) of the bitwidth sweep: the layout the kernels use reproduces the plain
    # convolution on the inputs that stress the slots hardest
    for p in range(1, 9):
        for K in (1, 2, 3, 5, 7, 9):
            L = hk.layout(p, p, signed, signed, K, 1)
            assert L["J"] == -(-K // L["Kc"]) and L["segments"] == L["N"] + L["Kc"] - 1
            assert L["S"] >= L["S_paper"] and L["S"] * (L["segments"] - 1) < 64
            lo_f = -(1 << (p - 1)) if signed else 0
            hi_f = (1 << (p - 1)) - 1 if signed else (1 << p) - 1
            pmin = min(a * b for a in (lo_f, hi_f) for b in (lo_f, hi_f))
            T = [0] * L["segments"]
            for j in range(L["J"]):
                kc = min(L["Kc"], K - j * L["Kc"])
                for n in range(L["N"]):
                    for k in range(kc):
                        T[n + k] += 1
            bias = [-t * pmin for t in T]
            for f, g in _extreme_vectors(p, p, signed, signed, 3 * L["N"] + 2, K):
                assert _model_conv1d(f, g, L, bias) == direct.conv1d_full(f, g).tolist()


@pytest.mark.parametrize("signed", [False, True])
def test_layout_emu64_is_exact_on_extreme_codes(signed):
    # the 64x64 -> 128 variant: same check with 64-bit operands and a 128-bit product, and a wider
    # multiplier never yields fewer outputs per multiply than the 32-bit one
    for p in range(1, 9):
        for K in (1, 2, 3, 5, 7, 9):
            L = hk.layout_emu64(p, p, signed, signed, K)
            L32 = hk.layout(p, p, signed, signed, K, 1)
            assert L["J"] == -(-K // L["Kc"]) and L["segments"] == L["N"] + L["Kc"] - 1
            assert L["S"] >= L["S_paper"] and L["S"] * (L["segments"] - 1) < 128 and 1 <= L["N"] <= 16
            assert L["N"] / L["J"] >= min(L32["N"], 16) / L32["J"]
            lo_f = -(1 << (p - 1)) if signed else 0
            hi_f = (1 << (p - 1)) - 1 if signed else (1 << p) - 1
            pmin = min(a * b for a in (lo_f, hi_f) for b in (lo_f, hi_f))
            T = [0] * L["segments"]
            for j in range(L["J"]):
                kc = min(L["Kc"], K - j * L["Kc"])
                for n in range(L["N"]):
                    for k in range(kc):
                        T[n + k] += 1
            bias = [-t * pmin for t in T]
            for f, g in _extreme_vectors(p, p, signed, signed, 3 * L["N"] + 2, K):
                assert _model_conv1d(f, g, L, bias, word_bits=64) == direct.conv1d_full(f, g).tolist()
    # the printed 4-bit slot width (S = 10 at K = 3) holds six codes in 64 bits... and seven: 4 + 6 * 10 = 64
    assert hk.layout_emu64(4, 4, False, False, 3, {"S": 10})["N"] == 7
    with pytest.raises(hk.HikonvError):
        hk.layout_emu64(4, 4, False, False, 3, {"S": 10, "N": 8})       # 4 + 7 * 10 = 74 bits


def test_layout_2d_known_cases():
    c3 = hk.layout(4, 4, True, True, 3, 2, 64 * 3)
    assert c3["J"] == 1 and c3["Kc"] == 3 and c3["M"] >= 1 and c3["S"] * (c3["segments"] - 1) < 64
    forced = hk.layout(4, 4, True, True, 3, 2, 64 * 3, {"N": 2})
    assert forced["N"] == 2
    with pytest.raises(hk.HikonvError):
        hk.layout(8, 8, True, True, 3, 2, 64 * 3, {"N": 4})     # four 8-bit codes never fit 32 bits with products
    with pytest.raises(hk.HikonvError):
        hk.layout(4, 4, True, True, 3, 2, 64 * 3, {"N": 3, "S": 13, "M": 1000})


def test_device_entry_points_validate_before_touching_cuda():
    lib = hk.lib()
    assert lib.hikonv_conv1d(None, 10, None, 3, 4, 4, 0, 0, None, 0, None, None) == hk.ERR_INVALID_ARG
    assert lib.hikonv_conv1d(8, 10, 8, 3, 9, 4, 0, 0, 8, 0, None, None) == hk.ERR_INVALID_ARG
    assert lib.hikonv_conv1d(8, 10, 8, 3, 4, 4, 0, 0, 8, 9, None, None) == hk.ERR_INVALID_ARG     # no such algorithm
    assert lib.hikonv_conv1d(8, 10, 8, 9, 4, 4, 0, 0, 8, hk.ALGO_DP4A, None, None) == hk.ERR_UNSUPPORTED   # dp4a comparator: K <= 8
    assert lib.hikonv_conv1d(8, 10, 8, 3, 4, 4, 0, 0, 9, 1, None, None) == hk.ERR_INVALID_ARG     # misaligned output
    assert lib.hikonv_conv1d(8, 10, 8, 0, 4, 4, 0, 0, 8, 0, None, None) == hk.ERR_INVALID_ARG
    # dense input: null pointers, widths that straddle bytes, layouts that are not instantiated
    assert lib.hikonv_conv1d_dense(None, 10, 8, 3, 4, 4, 0, 0, 8, None, None) == hk.ERR_INVALID_ARG
    assert lib.hikonv_conv1d_dense(8, 10, 8, 3, 3, 3, 0, 0, 8, None, None) == hk.ERR_UNSUPPORTED
    assert lib.hikonv_conv1d_dense(8, 10, 8, 3, 4, 2, 0, 1, 8, None, None) == hk.ERR_UNSUPPORTED     # unequal widths: a layout that is not built
    # the dense 2-D entry point: storage widths that match no code width, outputs that need requantisation
    assert lib.hikonv_conv2d_dense(8, 3, 1, 1, 4, 4, 8, 8, 1, 3, 1, 1, 4, 4, 0, 0, 8, 32, 0, 0, 0, 0, 0, 256, 1 << 20, 0, None, None) == hk.ERR_UNSUPPORTED
    assert lib.hikonv_conv2d_dense(8, 4, 1, 1, 4, 4, 8, 8, 1, 3, 1, 1, 4, 4, 0, 0, 8, 4, 0, 0, 0, 0, 0, 256, 1 << 20, 0, None, None) == hk.ERR_INVALID_ARG
    assert lib.hikonv_conv2d_dense(8, 4, 1, 1, 4, 4, 8, 8, 1, 3, 1, 1, 4, 4, 0, 0, 8, 32, 0, 0, 0, 0, 1, 256, 1 << 20, 0, None, None) == hk.ERR_INVALID_ARG   # pool without requant
    assert lib.hikonv_conv1d_dense(8, 10, 8, 9, 4, 4, 0, 0, 8, None, None) == hk.ERR_UNSUPPORTED     # K = 9
    assert lib.hikonv_pack(None, 10, 4, 0, 10, 3, 32, None, None) == hk.ERR_INVALID_ARG
    assert lib.hikonv_check_range(None, 10, 4, 0, 8, None, None) == hk.ERR_INVALID_ARG
    assert lib.hikonv_check_range(8, 10, 9, 0, 8, None, None) == hk.ERR_INVALID_ARG
    assert lib.hikonv_check_range(8, 10, 4, 0, 12, None, None) == hk.ERR_INVALID_ARG     # count word not 8-byte aligned
    assert lib.hikonv_pack(8, 10, 4, 0, 10, 4, 32, 8, None) == hk.ERR_NO_FIT
    assert lib.hikonv_conv2d(8, 1, 1, 4, 4, 8, 1, 3, 2, 1, 4, 4, 0, 0, 8, 0, 0, 0, 0, 256, 1 << 20, 0, None, None) == hk.ERR_UNSUPPORTED
    assert lib.hikonv_conv2d(8, 1, 1, 4, 4, 8, 1, 3, 1, 1, 4, 4, 0, 0, 8, 0, 0, 0, 0, None, 0, 0, None, None) == hk.ERR_WORKSPACE
    assert lib.hikonv_conv2d(8, 1, 1, 4, 4, 8, 1, 3, 1, 1, 4, 4, 0, 0, 8, 1, 40, 0, 15, 256, 1 << 20, 0, None, None) == hk.ERR_INVALID_ARG
    assert lib.hikonv_maxpool2x2_i8(None, 1, 1, 4, 4, 0, None, None) == hk.ERR_INVALID_ARG
    # room for the packed kernel rows and for one packed word per input pixel in the comparator's layout
    assert hk.conv2d_workspace_bytes(2, 64, 8, 8, 64, 3, 1) >= 64 * 3 * 3 * 64 * 4 + 64 * 2 * 10 * 11 * 4
    assert hk.conv2d_workspace_bytes(2, 64, 8, 8, 64, 3, 4) > 0 and hk.conv2d_workspace_bytes(2, 64, 2, 2, 64, 7, 0) == 0
    assert hk.conv1d_host_workspace_bytes(1000, 3) >= 1000 + 3 + 4 * 1002


def test_multiply_counts():
    # packed 4-bit K = 3 on the planner's layout: one multiply per block of N = 3 outputs; comparator: K per output
    n = 3000
    planner = {"tile": -1}
    assert hk.conv1d_multiplies(n, 3, 4, 4, False, False, hk.ALGO_PACKED32, planner) == -(-(n + 2) // 3)
    assert hk.conv1d_multiplies(n, 3, 4, 4, False, False, hk.ALGO_UNPACKED_IMAD) == (n + 2) * 3
    assert hk.conv1d_multiplies(n, 7, 4, 4, False, False, hk.ALGO_DP4A) == (n + 6) * 2
    assert hk.conv1d_multiplies(n, 3, 4, 4, False, False, hk.ALGO_PACKED64EMU) == -(-(n + 2) // hk.layout_emu64(4, 4, False, False, 3)["N"])
    # byte input without a forced layout: byte-aligned slots (the HBM-bound call takes the fewest instructions per
    # output, not the most outputs per multiply): 16-bit slots, N = 2, the three taps in two kernel words at
    # 4 bits; 8-bit slots, N = 4 at 1 and 2 bits; 18-bit slots, N = 2, two taps per kernel word for signed 8-bit codes
    assert hk.conv1d_multiplies(n, 3, 4, 4, False, False, hk.ALGO_PACKED32) == 2 * -(-(n + 2) // 2)
    assert hk.conv1d_multiplies(n, 3, 1, 1, False, False, hk.ALGO_PACKED32) == -(-(n + 2) // 4)
    assert hk.conv1d_multiplies(n, 5, 2, 2, False, False, hk.ALGO_PACKED32) == 2 * -(-(n + 4) // 4)
    assert hk.conv1d_multiplies(n, 7, 8, 8, True, True, hk.ALGO_PACKED32) == 4 * -(-(n + 6) // 2)
    L8 = hk.conv1d_layout(8, 8, True, True, 7)
    assert (L8["N"], L8["S"], L8["Kc"], L8["J"]) == (2, 18, 2, 4)
    assert hk.conv1d_layout(4, 4, False, False, 3) == dict(hk.conv1d_layout(4, 4, False, False, 3), N=2, S=16, Kc=2, J=2)
    # with tile = -1 the planner's layout runs, in blocks of 8 where the planner says 11 (1-bit, K = 3) and of 4
    # where it says 5 (2-bit, K = 5), unless N is forced; hikonv_layout keeps the planner's answer
    assert hk.layout(1, 1, False, False, 3, 1)["N"] == 11 and hk.layout(2, 2, False, False, 5, 1)["N"] == 5
    assert hk.conv1d_multiplies(n, 3, 1, 1, False, False, hk.ALGO_PACKED32, planner) == -(-(n + 2) // 8)
    assert hk.conv1d_multiplies(n, 5, 2, 2, False, False, hk.ALGO_PACKED32, planner) == -(-(n + 4) // 4)
    assert hk.conv1d_layout(1, 1, False, False, 3, planner)["N"] == 8
    assert hk.conv1d_multiplies(n, 3, 1, 1, False, False, hk.ALGO_PACKED32, {"N": 11}) == -(-(n + 2) // 11)
    # a smaller block that would need more kernel chunks is not taken: 1-bit codes x signed 2-bit taps, K = 9
    # fit two chunks of N = 5 taps but would need three of N = 4
    L9 = hk.layout(1, 2, False, True, 9, 1)
    assert (L9["N"], L9["J"]) == (5, 2)
    assert hk.conv1d_multiplies(n, 9, 1, 2, False, True, hk.ALGO_PACKED32) == 2 * -(-(n + 8) // 5)
    packed = hk.conv2d_multiplies(2, 8, 10, 12, 16, 3, 1, 4, 4, True, True, hk.ALGO_PACKED32)
    unpacked = hk.conv2d_multiplies(2, 8, 10, 12, 16, 3, 1, 4, 4, True, True, hk.ALGO_UNPACKED_IMAD)
    macs = 2 * 16 * 10 * 12 * 8 * 9
    assert 0 < packed < macs / 2 and unpacked >= macs


class _FakeDeviceTensor:
    """Stands in for a CUDA tensor where there is no GPU: only what the binding's checks look at."""

    def __init__(self, numel, dtype, device="cuda:0", contiguous=True, is_cuda=True):
        self._numel, self.dtype, self.device, self._contiguous, self.is_cuda = numel, dtype, device, contiguous, is_cuda

    def numel(self):
        return self._numel

    def is_contiguous(self):
        return self._contiguous

    def data_ptr(self):
        return 0x1000


def test_output_tensors_are_validated_before_any_launch():
    # the kernels see only an address: a short, mistyped, strided or misplaced `out` must be refused on the host
    import torch
    like = _FakeDeviceTensor(10, torch.int8)
    good = _FakeDeviceTensor(12, torch.int32)
    assert hk._dev_out(good, "out", 12, (torch.int32,), like) == 0x1000
    for bad in (_FakeDeviceTensor(11, torch.int32),                         # too short
                _FakeDeviceTensor(12, torch.int8),                          # bytes where int32 is written
                _FakeDeviceTensor(12, torch.int32, contiguous=False),       # strided view
                _FakeDeviceTensor(12, torch.int32, device="cuda:1"),        # another GPU
                _FakeDeviceTensor(12, torch.int32, is_cuda=False),          # host memory
                torch.empty(12, dtype=torch.int32)):                        # a real CPU tensor
        with pytest.raises(ValueError):
            hk._dev_out(bad, "out", 12, (torch.int32,), like)
    # through a public wrapper: a CPU tensor as `out` never reaches the library
    f = torch.zeros(8, dtype=torch.int8)
    with pytest.raises(ValueError):
        hk.conv1d(f, f[:3], 4, 4, False, False, out=torch.empty(10, dtype=torch.int32))


def test_register_aligned_layout_conditions():
    # hikonv_conv1d_layout takes slots of 8, 16 or 17..21 bits exactly when, recomputed here from the code ranges:
    # the (lifted) packed codes fit the multiplier's register, the kernel word fits it, the slots fit 64 bits and
    # K products fit the slot
    for p in range(1, 9):
        for q in range(1, 9):
            for fs in (False, True):
                for gs in (False, True):
                    flo, fhi = (-(1 << (p - 1)), (1 << (p - 1)) - 1) if fs else (0, (1 << p) - 1)
                    glo, ghi = (-(1 << (q - 1)), (1 << (q - 1)) - 1) if gs else (0, (1 << q) - 1)
                    prods = [a * b for a in (flo, fhi) for b in (glo, ghi)]
                    signed_mul = fs or gs
                    reg_hi = (1 << 31) - 1 if signed_mul else (1 << 32) - 1
                    for K in range(1, 10):
                        want = None
                        for S in (8, 16, 17, 18, 19, 20, 21):
                            N = 4 if S == 8 else 2
                            Kc = min(K, N)
                            # signed codes enter lifted: by 2^(p-1) with one-byte slots, by 128 otherwise
                            top = (1 << p) - 1 if (S == 8 or not fs) else 255
                            a_ok = sum(top << (S * n) for n in range(N)) <= reg_hi
                            b_lo = sum(glo << (S * k) for k in range(Kc))
                            b_hi = sum(ghi << (S * k) for k in range(Kc))
                            b_ok = b_hi <= reg_hi and (b_lo >= -(1 << 31) if signed_mul else b_lo >= 0)
                            lo, hi = K * min(prods), K * max(prods)
                            y_ok = (-(1 << (S - 1)) <= lo and hi <= (1 << (S - 1)) - 1) if signed_mul else hi <= (1 << S) - 1
                            if K <= 8 and a_ok and b_ok and y_ok and S * (N + Kc - 1) <= 63:
                                want = (N, S, Kc, -(-K // Kc))
                                break
                        L = hk.conv1d_layout(p, q, fs, gs, K)
                        got = (L["N"], L["S"], L["Kc"], L["J"])
                        if want is not None:
                            assert got == want, (p, q, fs, gs, K, got, want)
                        else:
                            plan = hk.conv1d_layout(p, q, fs, gs, K, {"tile": -1})
                            assert got == (plan["N"], plan["S"], plan["Kc"], plan["J"]), (p, q, fs, gs, K)


def test_conv2d_layout_reports_the_shifted_activation_codes():
    # deep layers with unsigned activations and signed weights run on codes x - 2^(p-1): the signed layout's larger M,
    # at least half again the unsigned one's; shallower layers, signed activations and unsigned weights keep their own
    deep = hk.conv2d_layout(64, 256, 14, 14, 256, 3, 1, 4, 4, False, True)
    own = hk.layout(4, 4, False, True, 3, 2, 256 * 3)
    signed = hk.layout(4, 4, True, True, 3, 2, 256 * 3)
    assert deep["x_shift"] == 8
    assert (deep["N"], deep["S"], deep["M"]) == (signed["N"], signed["S"], signed["M"])
    assert 2 * deep["M"] >= 3 * own["M"] and deep["N"] >= own["N"]
    assert hk.conv2d_layout(64, 64, 20, 40, 64, 3, 1, 4, 4, False, True)["x_shift"] == 0          # fewer than 128 channels, small layer
    assert hk.conv2d_layout(64, 32, 40, 80, 64, 3, 1, 4, 4, False, True)["x_shift"] == 8          # 32 channels on a large layer
    assert hk.conv2d_layout(64, 16, 80, 160, 32, 3, 1, 4, 4, False, True)["x_shift"] == 0         # fewer than 32 channels
    assert hk.conv2d_layout(32, 256, 14, 14, 64, 3, 1, 4, 4, True, True)["x_shift"] == 0          # signed already
    assert hk.conv2d_layout(32, 256, 14, 14, 64, 3, 1, 4, 4, False, False)["x_shift"] == 0        # products never negative
    for p in (1, 2, 3, 5, 8):
        L = hk.conv2d_layout(2, 200, 9, 11, 8, 3, 1, p, 4, False, True)
        assert L["x_shift"] in (0, 1 << (p - 1))
    # the multiply count follows the layout that runs
    L = hk.conv2d_layout(2, 130, 6, 17, 12, 3, 1, 4, 4, False, True)
    muls = hk.conv2d_multiplies(2, 130, 6, 17, 12, 3, 1, 4, 4, False, True, hk.ALGO_PACKED32)
    assert muls > 0 and muls % (130 * 3 * L["J"] * 12) == 0
    with pytest.raises(hk.HikonvError):
        hk.conv2d_layout(1, 4, 60000, 8, 4, 3, 1, 4, 4, True, True)                                # rows beyond the index arithmetic


def test_tuner_refuses_bad_arguments_before_touching_the_device():
    tile = ctypes.c_int(-1)
    args = [None, 8, 1, 1, 4, 4, None, 8, 1, 3, 1, 1, 4, 4, 1, 1, None, 8, 1, 6, -8, 7, 0, None, 0, hk.ALGO_PACKED32]
    assert hk.lib().hikonv_conv2d_tune(*args, 3, None, None, None, None) == hk.ERR_INVALID_ARG          # nowhere to put the tile
    assert hk.lib().hikonv_conv2d_tune(*args, 0, ctypes.byref(tile), None, None, None) == hk.ERR_INVALID_ARG
    assert hk.lib().hikonv_conv2d_tune(*args, 101, ctypes.byref(tile), None, None, None) == hk.ERR_INVALID_ARG
    assert tile.value == -1
