"""ctypes binding of ``libhikonv.so``: same names as the C interface, argument marshalling only.

PyTorch is used for device memory and streams; every arithmetic step runs in the CUDA
library.  Loading fails loudly when the library has not been built: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhikonv.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NO_FIT, ERR_WORKSPACE, ERR_CUDA, ERR_TOO_LARGE, ERR_RANGE = range(8)
STATIC_SCRATCH_BYTES = 4 << 20
ALGO_PACKED32, ALGO_PACKED64EMU, ALGO_UNPACKED_IMAD, ALGO_DP4A = 0, 1, 2, 3
GB_SINGLE, GB_1D, GB_DNN = 0, 1, 2
PIPE_KINDS = {"mad_wide_u32": 0, "mad_wide_s32": 1, "mad_lo_s32": 2, "logic": 3, "shift": 4, "prmt": 5,
              "mad_wide_with_logic": 6}


class HikonvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %s (status %d)" % (where, status_string(status), status))


class PlanT(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("N", "K", "S", "Gb", "ops")]


class LayoutT(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("N", "S", "Kc", "J", "segments", "top_bits", "M", "signed_prod", "S_paper", "carry_bits")]


class TuningT(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("N", "S", "M", "tile")]


_lib = None

_vp, _sz, _i, _d = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int, ctypes.c_double

_SIGNATURES = {
    "hikonv_plan": (_i, [_i] * 7 + [ctypes.POINTER(PlanT)]),
    "hikonv_layout": (_i, [_i] * 7 + [ctypes.POINTER(TuningT), ctypes.POINTER(LayoutT)]),
    "hikonv_layout_emu64": (_i, [_i] * 5 + [ctypes.POINTER(TuningT), ctypes.POINTER(LayoutT)]),
    "hikonv_pack": (_i, [_vp, _sz, _i, _i, _i, _i, _i, _vp, _vp]),
    "hikonv_check_range": (_i, [_vp, _sz, _i, _i, _vp, ctypes.POINTER(ctypes.c_ulonglong), _vp]),
    "hikonv_conv1d": (_i, [_vp, _sz, _vp, _i, _i, _i, _i, _i, _vp, _i, ctypes.POINTER(TuningT), _vp]),
    "hikonv_conv1d_layout": (_i, [_i] * 5 + [ctypes.POINTER(TuningT), ctypes.POINTER(LayoutT)]),
    "hikonv_conv1d_dense": (_i, [_vp, _sz, _vp, _i, _i, _i, _i, _i, _vp, ctypes.POINTER(TuningT), _vp]),
    "hikonv_conv1d_host_workspace_bytes": (_sz, [_sz, _i]),
    "hikonv_conv1d_host": (_i, [_vp, _sz, _vp, _i, _i, _i, _i, _i, _vp, _vp, _sz, _i, ctypes.POINTER(TuningT), _vp]),
    "hikonv_conv2d": (_i, [_vp, _i, _i, _i, _i, _vp, _i, _i, _i, _i, _i, _i, _i, _i, _vp, _i, _i, _i, _i, _vp, _sz, _i,
                           ctypes.POINTER(TuningT), _vp]),
    "hikonv_conv2d_dense": (_i, [_vp, _i, _i, _i, _i, _i, _vp, _i, _i, _i, _i, _i, _i, _i, _i, _i, _vp, _i, _i, _i, _i, _i, _i, _vp, _sz,
                                 _i, ctypes.POINTER(TuningT), _vp]),
    "hikonv_conv2d_tune": (_i, [_vp, _i, _i, _i, _i, _i, _vp, _i, _i, _i, _i, _i, _i, _i, _i, _i, _vp, _i, _i, _i, _i, _i, _i, _vp, _sz,
                                _i, _i, ctypes.POINTER(_i), ctypes.POINTER(_d), ctypes.POINTER(_d), _vp]),
    "hikonv_conv2d_workspace_bytes": (_sz, [_i] * 7),
    "hikonv_conv2d_static_scratch": (_i, [_vp, _i, _i, _i, _i, _vp, _i, _i, _i, _i, _i, _i, _i, _i, _vp, _i, _i, _i, _i, _i,
                                          ctypes.POINTER(TuningT), _vp]),
    "hikonv_conv2d_host_workspace_bytes": (_sz, [_i] * 8),
    "hikonv_conv2d_host": (_i, [_vp, _i, _i, _i, _i, _vp, _i, _i, _i, _i, _i, _i, _i, _i, _vp, _i, _i, _i, _i, _vp, _sz,
                                _i, ctypes.POINTER(TuningT), _vp]),
    "hikonv_maxpool2x2_i8": (_i, [_vp, _i, _i, _i, _i, _i, _vp, _vp]),
    "hikonv_conv1d_multiplies": (_d, [_sz, _i, _i, _i, _i, _i, _i, ctypes.POINTER(TuningT)]),
    "hikonv_conv2d_multiplies": (_d, [_i] * 12 + [ctypes.POINTER(TuningT)]),
    "hikonv_conv2d_layout": (_i, [_i] * 11 + [ctypes.POINTER(TuningT), ctypes.POINTER(LayoutT), ctypes.POINTER(_i)]),
    "hikonv_pipe_rate": (_i, [_i, _i, _vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), _vp]),
    "hikonv_status_string": (ctypes.c_char_p, [_i]),
}


def exported_names():
    return sorted(_SIGNATURES)


def lib():
    """The loaded CUDA library.  Raises if it has not been built (no CPU fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "CUDA library %s is missing: run `python -m paper_2208_00763_b200.build` "
                "(or __graft_entry__.build()) first; there is no CPU fallback" % LIB_PATH)
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def status_string(status: int) -> str:
    return lib().hikonv_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise HikonvError(status, where)


def _tune(tune: Optional[dict]):
    if not tune:
        return None
    t = TuningT(int(tune.get("N", 0)), int(tune.get("S", 0)), int(tune.get("M", 0)), int(tune.get("tile", 0)))
    return ctypes.byref(t)


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev_i8(t: torch.Tensor, name: str) -> int:
    if not t.is_cuda or t.dtype not in (torch.int8, torch.uint8) or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA int8/uint8 tensor" % name)
    return t.data_ptr()


def _dev_out(t: torch.Tensor, name: str, numel: int, dtypes, like: torch.Tensor) -> int:
    """Checks a caller-supplied output tensor before its address goes to a kernel: the library writes `numel`
    elements of one of `dtypes` there and cannot see the tensor's size, type, layout or device."""
    if not getattr(t, "is_cuda", False):
        raise ValueError("%s must be a CUDA tensor" % name)
    if t.device != like.device:
        raise ValueError("%s is on %s, the inputs are on %s" % (name, t.device, like.device))
    if t.dtype not in dtypes:
        raise ValueError("%s must have dtype %s, not %s" % (name, " or ".join(str(d) for d in dtypes), t.dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    if t.numel() != numel:
        raise ValueError("%s holds %d elements, the call writes %d" % (name, t.numel(), numel))
    return t.data_ptr()


_CODE_DTYPES = (torch.int8, torch.uint8)


# ------------------------------------------------------------------ host-only planning

def plan(p, q, LA=32, LB=32, mode=GB_SINGLE, M=1, K_fixed=0) -> dict:
    out = PlanT()
    _check(lib().hikonv_plan(p, q, LA, LB, mode, M, K_fixed, ctypes.byref(out)), "hikonv_plan")
    return {n: getattr(out, n) for n, _ in PlanT._fields_}


def layout(p, q, f_signed, g_signed, K, dims, total_terms=0, tune=None) -> dict:
    out = LayoutT()
    _check(lib().hikonv_layout(p, q, int(f_signed), int(g_signed), K, dims, total_terms, _tune(tune), ctypes.byref(out)),
           "hikonv_layout")
    return {n: getattr(out, n) for n, _ in LayoutT._fields_}


def layout_emu64(p, q, f_signed, g_signed, K, tune=None) -> dict:
    out = LayoutT()
    _check(lib().hikonv_layout_emu64(p, q, int(f_signed), int(g_signed), K, _tune(tune), ctypes.byref(out)),
           "hikonv_layout_emu64")
    return {n: getattr(out, n) for n, _ in LayoutT._fields_}


def conv1d_layout(p, q, f_signed, g_signed, K, tune=None) -> dict:
    """The layout ``conv1d`` (packed algorithm, one code per byte) runs with."""
    out = LayoutT()
    _check(lib().hikonv_conv1d_layout(p, q, int(f_signed), int(g_signed), K, _tune(tune), ctypes.byref(out)),
           "hikonv_conv1d_layout")
    return {n: getattr(out, n) for n, _ in LayoutT._fields_}


def conv2d_layout(B, Ci, H, W, Co, K, pad, p, q, x_signed, w_signed, tune=None) -> dict:
    """The layout ``conv2d`` (packed algorithm) runs this layer with, plus ``x_shift``: 0, or 2^(p-1) when the layer
    runs its unsigned activations as signed codes shifted by that much."""
    out, shift = LayoutT(), ctypes.c_int(0)
    _check(lib().hikonv_conv2d_layout(B, Ci, H, W, Co, K, pad, p, q, int(x_signed), int(w_signed), _tune(tune), ctypes.byref(out),
                                      ctypes.byref(shift)), "hikonv_conv2d_layout")
    d = {n: getattr(out, n) for n, _ in LayoutT._fields_}
    d["x_shift"] = shift.value
    return d


# ------------------------------------------------------------------ device entry points

def pack(d_in: torch.Tensor, bits: int, is_signed: bool, S: int, N: int, word_bits: int = 32, stream=None) -> torch.Tensor:
    n = d_in.numel()
    n_words = (n + N - 1) // N
    out = torch.empty(n_words, dtype=torch.int32 if word_bits == 32 else torch.int64, device=d_in.device)
    _check(lib().hikonv_pack(_dev_i8(d_in, "d_in"), n, bits, int(is_signed), S, N, word_bits, out.data_ptr(), _stream(stream)),
           "hikonv_pack")
    return out


def check_range(d_in: torch.Tensor, bits: int, is_signed: bool, stream=None) -> int:
    """Number of stored codes outside their range (0 = all valid).  Synchronises the stream."""
    d_count = torch.empty(1, dtype=torch.int64, device=d_in.device)
    found = ctypes.c_ulonglong(0)
    rc = lib().hikonv_check_range(_dev_i8(d_in, "d_in"), d_in.numel(), bits, int(is_signed), d_count.data_ptr(),
                                  ctypes.byref(found), _stream(stream))
    if rc not in (OK, ERR_RANGE):
        _check(rc, "hikonv_check_range")
    assert (rc == ERR_RANGE) == (found.value > 0)
    return int(found.value)


def conv1d(d_f: torch.Tensor, d_g: torch.Tensor, p: int, q: int, f_signed: bool, g_signed: bool,
           algo: int = ALGO_PACKED32, tune=None, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    n, K = d_f.numel(), d_g.numel()
    if out is None:
        out = torch.empty(n + K - 1, dtype=torch.int32, device=d_f.device)
    _check(lib().hikonv_conv1d(_dev_i8(d_f, "d_f"), n, _dev_i8(d_g, "d_g"), K, p, q, int(f_signed), int(g_signed),
                               _dev_out(out, "out", n + K - 1, (torch.int32,), d_f), algo, _tune(tune), _stream(stream)),
           "hikonv_conv1d")
    return out


def conv1d_dense(d_f_dense: torch.Tensor, n: int, d_g: torch.Tensor, p: int, q: int, f_signed: bool, g_signed: bool,
                 tune=None, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """`d_f_dense`: uint8 tensor holding `n` codes of p bits, 8 / p per byte."""
    K = d_g.numel()
    if d_f_dense.dtype != torch.uint8 or not d_f_dense.is_cuda or not d_f_dense.is_contiguous():
        raise ValueError("d_f_dense must be a contiguous CUDA uint8 tensor")
    if d_f_dense.numel() * 8 < n * p:
        raise ValueError("d_f_dense holds fewer than n codes")
    if out is None:
        out = torch.empty(n + K - 1, dtype=torch.int32, device=d_f_dense.device)
    _check(lib().hikonv_conv1d_dense(d_f_dense.data_ptr(), n, _dev_i8(d_g, "d_g"), K, p, q, int(f_signed), int(g_signed),
                                     _dev_out(out, "out", n + K - 1, (torch.int32,), d_f_dense), _tune(tune), _stream(stream)),
           "hikonv_conv1d_dense")
    return out


def conv1d_host_workspace_bytes(n: int, K: int) -> int:
    return int(lib().hikonv_conv1d_host_workspace_bytes(n, K))


def conv1d_host(h_f: torch.Tensor, h_g: torch.Tensor, p, q, f_signed, g_signed, h_y: torch.Tensor,
                d_workspace: torch.Tensor, algo: int = ALGO_PACKED32, tune=None, stream=None) -> None:
    """Host buffers in, host buffer out (pinned tensors make the copies asynchronous)."""
    n, K = h_f.numel(), h_g.numel()
    _check(lib().hikonv_conv1d_host(h_f.data_ptr(), n, h_g.data_ptr(), K, p, q, int(f_signed), int(g_signed),
                                    h_y.data_ptr(), d_workspace.data_ptr(), d_workspace.numel() * d_workspace.element_size(),
                                    algo, _tune(tune), _stream(stream)), "hikonv_conv1d_host")


def conv2d_workspace_bytes(B: int, Ci: int, H: int, W: int, Co: int, K: int, pad: int) -> int:
    return int(lib().hikonv_conv2d_workspace_bytes(B, Ci, H, W, Co, K, pad))


def conv2d(d_x: torch.Tensor, d_w: torch.Tensor, pad: int, p: int, q: int, x_signed: bool, w_signed: bool,
           requant: Optional[tuple] = None, algo: int = ALGO_PACKED32, tune=None, workspace: Optional[torch.Tensor] = None,
           out: Optional[torch.Tensor] = None, stride: int = 1, stream=None) -> torch.Tensor:
    """requant = (shift, lo, hi) selects int8 output, None the exact int32 sums."""
    B, Ci, H, W = d_x.shape
    Co, Ci2, K, K2 = d_w.shape
    if Ci != Ci2 or K != K2:
        raise ValueError("weight shape does not match the input")
    Ho, Wo = H + 2 * pad - K + 1, W + 2 * pad - K + 1
    if workspace is None:
        workspace = torch.empty(conv2d_workspace_bytes(B, Ci, H, W, Co, K, pad), dtype=torch.uint8, device=d_x.device)
    if out is None:
        out = torch.empty((B, Co, max(Ho, 0), max(Wo, 0)), dtype=torch.int8 if requant else torch.int32, device=d_x.device)
    shift, lo, hi = requant if requant else (0, 0, 0)
    out_ptr = _dev_out(out, "out", B * Co * max(Ho, 0) * max(Wo, 0), _CODE_DTYPES if requant else (torch.int32,), d_x)
    if not workspace.is_cuda or workspace.device != d_x.device or not workspace.is_contiguous():
        raise ValueError("workspace must be a contiguous CUDA tensor on the inputs' device")
    _check(lib().hikonv_conv2d(_dev_i8(d_x, "d_x"), B, Ci, H, W, _dev_i8(d_w, "d_w"), Co, K, stride, pad, p, q,
                               int(x_signed), int(w_signed), out_ptr, 1 if requant else 0, shift, lo, hi,
                               workspace.data_ptr(), workspace.numel() * workspace.element_size(), algo, _tune(tune),
                               _stream(stream)), "hikonv_conv2d")
    return out


def conv2d_tune(d_x: torch.Tensor, x_shape, x_store_bits: int, d_w: torch.Tensor, w_shape, w_store_bits: int, pad: int, p: int,
                q: int, x_signed: bool, w_signed: bool, requant: Optional[tuple] = None, out_store_bits: int = 8,
                pool: bool = False, algo: int = ALGO_PACKED32, workspace: Optional[torch.Tensor] = None,
                out: Optional[torch.Tensor] = None, stride: int = 1, stream=None, repeats: int = 3) -> dict:
    """Times the tile shapes of this layer on the device (``hikonv_conv2d_tune``; arguments as for ``conv2d_dense``).
    Returns ``{"tune": {"tile": t} or None, "us": best, "default_us": the automatic choice's, "out": the layer's output}``;
    pass ``tune`` to later calls on this shape.  Synchronises."""
    return conv2d_dense(d_x, x_shape, x_store_bits, d_w, w_shape, w_store_bits, pad, p, q, x_signed, w_signed, requant, out_store_bits,
                        pool, algo, None, workspace, out, stride, stream, _tuner_repeats=int(repeats))


def conv2d_dense(d_x: torch.Tensor, x_shape, x_store_bits: int, d_w: torch.Tensor, w_shape, w_store_bits: int, pad: int, p: int,
                 q: int, x_signed: bool, w_signed: bool, requant: Optional[tuple] = None, out_store_bits: int = 8,
                 pool: bool = False, algo: int = ALGO_PACKED32, tune=None, workspace: Optional[torch.Tensor] = None,
                 out: Optional[torch.Tensor] = None, stride: int = 1, stream=None, _tuner_repeats: Optional[int] = None):
    """``conv2d`` on densely stored tensors.  ``d_x`` / ``d_w`` are flat uint8 (dense) or int8 (one code per byte)
    tensors holding the codes of ``x_shape`` = (B, Ci, H, W) / ``w_shape`` = (Co, Ci, K, K).  Returns int32
    [B, Co, Ho, Wo] without ``requant``; with it a flat uint8 tensor of the (optionally pooled) output codes,
    ``out_store_bits`` per code (8: shaped [B, Co, Ho', Wo'] int8)."""
    B, Ci, H, W = x_shape
    Co, Ci2, K, K2 = w_shape
    if Ci != Ci2 or K != K2:
        raise ValueError("weight shape does not match the input")
    for t, n, bits, name in ((d_x, B * Ci * H * W, x_store_bits, "d_x"), (d_w, Co * Ci * K * K, w_store_bits, "d_w")):
        if not t.is_cuda or not t.is_contiguous() or t.dtype not in _CODE_DTYPES or t.numel() * 8 < n * bits:
            raise ValueError("%s must be a contiguous CUDA byte tensor holding all codes" % name)
    Ho, Wo = H + 2 * pad - K + 1, W + 2 * pad - K + 1
    Hq, Wq = (Ho // 2, Wo // 2) if pool else (Ho, Wo)
    count = B * Co * max(Hq, 0) * max(Wq, 0)
    if workspace is None:
        workspace = torch.empty(conv2d_workspace_bytes(B, Ci, H, W, Co, K, pad), dtype=torch.uint8, device=d_x.device)
    if not requant:
        if out is None:
            out = torch.empty((B, Co, max(Ho, 0), max(Wo, 0)), dtype=torch.int32, device=d_x.device)
        out_ptr, store = _dev_out(out, "out", B * Co * max(Ho, 0) * max(Wo, 0), (torch.int32,), d_x), 32
    else:
        nbytes = (count * out_store_bits + 7) // 8
        if out is None:
            out = (torch.empty((B, Co, Hq, Wq), dtype=torch.int8, device=d_x.device) if out_store_bits == 8
                   else torch.empty(nbytes, dtype=torch.uint8, device=d_x.device))
        out_ptr, store = _dev_out(out, "out", nbytes, _CODE_DTYPES, d_x), out_store_bits
    shift, lo, hi = requant if requant else (0, 0, 0)
    if _tuner_repeats is not None:
        tile, us, default_us = ctypes.c_int(0), ctypes.c_double(0.0), ctypes.c_double(0.0)
        with torch.cuda.device(d_x.device):
            _check(lib().hikonv_conv2d_tune(d_x.data_ptr(), x_store_bits, B, Ci, H, W, d_w.data_ptr(), w_store_bits, Co, K, stride, pad,
                                            p, q, int(x_signed), int(w_signed), out_ptr, store, 1 if requant else 0, shift, lo, hi,
                                            1 if pool else 0, workspace.data_ptr(), workspace.numel() * workspace.element_size(),
                                            algo, _tuner_repeats, ctypes.byref(tile), ctypes.byref(us), ctypes.byref(default_us),
                                            _stream(stream)), "hikonv_conv2d_tune")
        return {"tune": {"tile": tile.value} if tile.value else None, "us": us.value, "default_us": default_us.value, "out": out}
    _check(lib().hikonv_conv2d_dense(d_x.data_ptr(), x_store_bits, B, Ci, H, W, d_w.data_ptr(), w_store_bits, Co, K, stride, pad, p, q,
                                     int(x_signed), int(w_signed), out_ptr, store, 1 if requant else 0, shift, lo, hi,
                                     1 if pool else 0, workspace.data_ptr(), workspace.numel() * workspace.element_size(), algo,
                                     _tune(tune), _stream(stream)), "hikonv_conv2d_dense")
    return out


def conv2d_static_scratch(d_x: torch.Tensor, d_w: torch.Tensor, pad: int, p: int, q: int, x_signed: bool, w_signed: bool,
                          out: torch.Tensor, requant: Optional[tuple] = None, algo: int = ALGO_PACKED32, tune=None,
                          stride: int = 1, stream=None) -> torch.Tensor:
    """``conv2d`` without a workspace: the packed kernel and activation rows go to the library's built-in device buffer.

    For callers that may not allocate device memory when the layer runs (they own only the input and
    output tensors, or allocation is forbidden after start-up).  ``out`` must be preallocated by the
    caller.  Layers whose packed rows exceed ``STATIC_SCRATCH_BYTES`` raise ``ERR_TOO_LARGE``; calls
    that may overlap on the GPU must be ordered by the caller, since they share the buffer.
    """
    B, Ci, H, W = d_x.shape
    Co, Ci2, K, K2 = d_w.shape
    if Ci != Ci2 or K != K2:
        raise ValueError("weight shape does not match the input")
    shift, lo, hi = requant if requant else (0, 0, 0)
    Ho, Wo = H + 2 * pad - K + 1, W + 2 * pad - K + 1
    out_ptr = _dev_out(out, "out", B * Co * max(Ho, 0) * max(Wo, 0), _CODE_DTYPES if requant else (torch.int32,), d_x)
    if d_w.device != d_x.device:
        raise ValueError("d_w is on %s, d_x on %s" % (d_w.device, d_x.device))
    with torch.cuda.device(d_x.device):      # the built-in buffer that is used is the current device's
        _check(lib().hikonv_conv2d_static_scratch(_dev_i8(d_x, "d_x"), B, Ci, H, W, _dev_i8(d_w, "d_w"), Co, K, stride, pad, p, q,
                                                  int(x_signed), int(w_signed), out_ptr, 1 if requant else 0, shift, lo, hi,
                                                  algo, _tune(tune), _stream(stream)), "hikonv_conv2d_static_scratch")
    return out


def conv2d_host_workspace_bytes(B, Ci, H, W, Co, K, pad, requant) -> int:
    return int(lib().hikonv_conv2d_host_workspace_bytes(B, Ci, H, W, Co, K, pad, 1 if requant else 0))


def conv2d_host(h_x: torch.Tensor, h_w: torch.Tensor, pad, p, q, x_signed, w_signed, h_out: torch.Tensor,
                d_workspace: torch.Tensor, requant: Optional[tuple] = None, algo: int = ALGO_PACKED32, tune=None,
                stride: int = 1, stream=None) -> None:
    B, Ci, H, W = h_x.shape
    Co, _, K, _ = h_w.shape
    shift, lo, hi = requant if requant else (0, 0, 0)
    _check(lib().hikonv_conv2d_host(h_x.data_ptr(), B, Ci, H, W, h_w.data_ptr(), Co, K, stride, pad, p, q, int(x_signed),
                                    int(w_signed), h_out.data_ptr(), 1 if requant else 0, shift, lo, hi,
                                    d_workspace.data_ptr(), d_workspace.numel() * d_workspace.element_size(), algo,
                                    _tune(tune), _stream(stream)), "hikonv_conv2d_host")


def maxpool2x2_i8(d_in: torch.Tensor, is_signed: bool, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    B, C, H, W = d_in.shape
    if out is None:
        out = torch.empty((B, C, H // 2, W // 2), dtype=d_in.dtype, device=d_in.device)
    _check(lib().hikonv_maxpool2x2_i8(_dev_i8(d_in, "d_in"), B, C, H, W, int(is_signed),
                                      _dev_out(out, "out", B * C * (H // 2) * (W // 2), _CODE_DTYPES, d_in), _stream(stream)),
           "hikonv_maxpool2x2_i8")
    return out


def conv1d_multiplies(n, K, p, q, f_signed, g_signed, algo=ALGO_PACKED32, tune=None) -> float:
    return float(lib().hikonv_conv1d_multiplies(n, K, p, q, int(f_signed), int(g_signed), algo, _tune(tune)))


def conv2d_multiplies(B, Ci, H, W, Co, K, pad, p, q, x_signed, w_signed, algo=ALGO_PACKED32, tune=None) -> float:
    return float(lib().hikonv_conv2d_multiplies(B, Ci, H, W, Co, K, pad, p, q, int(x_signed), int(w_signed), algo, _tune(tune)))


def pipe_rate(kind: str, iters: int = 2048, device=None, stream=None) -> dict:
    """Measured rate of one integer instruction (see ``PIPE_KINDS``): operations per second (instructions x 32
    lanes) and lanes per clock per SM at the device's maximum SM clock.  Synchronises."""
    word = torch.zeros(1, dtype=torch.int32, device=device or "cuda")
    ops, lanes = ctypes.c_double(0.0), ctypes.c_double(0.0)
    with torch.cuda.device(word.device):
        _check(lib().hikonv_pipe_rate(PIPE_KINDS[kind], int(iters), word.data_ptr(), ctypes.byref(ops), ctypes.byref(lanes),
                                      _stream(stream)), "hikonv_pipe_rate")
    return {"ops_per_second": ops.value, "lanes_per_clock_per_sm": lanes.value}
