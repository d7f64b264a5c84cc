"""Thin ctypes binding over ``libeden.so`` (declared in ``include/eden.h``).

Argument marshalling only: every step of EDEN's sender and receiver runs in the CUDA
kernels of the library.  PyTorch supplies device memory and the stream.  Importing this
module fails loudly if the library has not been built (``python -m
paper_2108_08842_b200.build``); there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libeden.so")

if not os.path.exists(_LIB_PATH):
    raise ImportError(
        "libeden.so is missing: build it with `python -m paper_2108_08842_b200.build` "
        "(needs nvcc); this package has no CPU fallback")

_lib = ctypes.CDLL(_LIB_PATH)

_u32, _u64, _f64, _vp, _int = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_double, ctypes.c_void_p, ctypes.c_int


class ClientStat(ctypes.Structure):
    _fields_ = [("norm2", _f64), ("dot", _f64), ("received", _f64), ("flags", _u32), ("reserved", _u32)]


def _sig(name, restype, argtypes):
    fn = getattr(_lib, name)
    fn.restype = restype
    fn.argtypes = argtypes
    return fn


_sig("eden_kept_count", _u64, [_u64, _f64])
_sig("eden_rot_dim", _u64, [_u64, _f64])
_sig("eden_code_width", _u32, [_f64])
_sig("eden_code_bytes", _u64, [_u64, _f64])
_sig("eden_num_packets", _u64, [_u64, _f64])
_sig("eden_recv_mask_words", _u64, [_u64, _f64])
_sig("eden_workspace_bytes", _u64, [_u64, _u32])
_sig("eden_host_workspace_bytes", _u64, [_u64, _u32])
_sig("eden_table", _int, [_u32, _vp, _vp])
_sig("eden_pass_plan", _int, [_u64, _f64, _vp, _u32, ctypes.POINTER(_u32)])
_sig("eden_create", _int, [ctypes.POINTER(_vp), _int, _vp, _vp, _u64])
_sig("eden_destroy", _int, [_vp])
_sig("eden_encode", _int, [_vp, _vp, _u64, _u64, _u32, _vp, _vp, _vp, _vp])
_sig("eden_decode_accumulate", _int, [_vp, _vp, _vp, _vp, _vp, _vp, _u64, _u32, _vp, _vp])
_sig("eden_mean", _int, [_vp, _vp, _vp, _vp, _vp, _vp, _u64, _u32, _vp])
_sig("eden_sparsification_mask", _int, [_vp, _u64, _u64, _f64, _vp])
_sig("eden_encode_host", _int, [_vp, _vp, _u64, _u64, _u32, _vp, _vp, _vp, _vp])
_sig("eden_mean_host", _int, [_vp, _vp, _vp, _vp, _vp, _vp, _u64, _u32, _vp])
_sig("eden_status", _int, [_vp, ctypes.POINTER(_u32)])
_sig("eden_client_stats", _int, [_vp, _u32, _vp])
_sig("eden_launch_count", _u64, [_vp])
_sig("eden_sparsification_mask_noalloc", _int, [_int, _vp, _u64, _u64, _f64, _vp])
_sig("eden_strerror", ctypes.c_char_p, [_int])
_sig("eden_mean_partial", _int, [_vp, _vp, _vp, _vp, _vp, _vp, _u64, _u32, _u64, _vp])
_sig("eden_uniform_entropy", _f64, [_f64])
_sig("eden_uniform_delta", _f64, [_f64])
_sig("eden_uniform_values", _int, [_f64, _vp])
_sig("eden_uniform_index_bytes", _u64, [_u64])
_sig("eden_encode_uniform", _int, [_vp, _vp, _u64, _u64, _u32, _vp, _vp, _vp, _vp])
_sig("eden_decode_accumulate_uniform", _int, [_vp, _vp, _vp, _vp, _vp, _vp, _u64, _u32, _vp, _vp])
_sig("eden_mean_uniform", _int, [_vp, _vp, _vp, _vp, _vp, _vp, _u64, _u32, _vp])
_sig("eden_index_histogram", _int, [_vp, _vp, _u64, _u32, _vp])
_sig("eden_profile_enable", _int, [_vp, _int])
_sig("eden_force_generic_kernels", _int, [_vp, _int])
_sig("eden_set_option", _int, [_vp, _int, _int])
_sig("eden_self_check", _int, [])
_sig("eden_mask_threshold_band", _int, [_u64, _u64, _int, _vp, _vp])
_sig("eden_after_kept_count", _u64, [_u64, _f64])
_sig("eden_after_code_bytes", _u64, [_u64, _f64])
_sig("eden_after_workspace_bytes", _u64, [_u64, _u32])
_sig("eden_encode_sparsify_after", _int, [_vp, _vp, _u64, _u64, _u32, _vp, _vp, _vp, _vp])
_sig("eden_mean_sparsify_after", _int, [_vp, _vp, _vp, _vp, _vp, _u64, _u32, _vp])
_sig("eden_decode_accumulate_sparsify_after", _int, [_vp, _vp, _vp, _vp, _vp, _u64, _u32, _vp, _vp])
_sig("eden_profile_collect", _int, [_vp, ctypes.POINTER(_u32)])
_sig("eden_profile_get", _int, [_vp, _u32, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(_u64),
                                ctypes.POINTER(_f64), ctypes.POINTER(_f64)])

STATUS_ZERO_VECTOR, STATUS_NONFINITE, STATUS_NO_DATA, STATUS_TIMEOUT, STATUS_SCRATCH = 1, 2, 4, 8, 16
OPT_PLAN_VARIANT, OPT_ROW_STAGING, OPT_SEL_ROUNDS, OPT_SLAB_MIB, OPT_SLAB_STREAMS, OPT_SLAB_SIDES, OPT_SEL_BAND, OPT_SEL_AHEAD = 1, 2, 3, 4, 5, 6, 7, 8
PACKET_COORDS = 1024
UNIFORM_MAX_INDEX = 127
UNIFORM_MIN_DELTA = 0.0625


class EdenError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__("eden: %s (%d)" % (_lib.eden_strerror(code).decode(), code))


def _check(rc: int):
    if rc != 0:
        raise EdenError(rc)


# ---------------------------------------------------------------------------- size rules
def kept_count(d: int, bits: float) -> int:
    return int(_lib.eden_kept_count(d, bits))


def rot_dim(d: int, bits: float) -> int:
    return int(_lib.eden_rot_dim(d, bits))


def code_width(bits: float) -> int:
    return int(_lib.eden_code_width(bits))


def code_bytes(d: int, bits: float) -> int:
    return int(_lib.eden_code_bytes(d, bits))


def num_packets(d: int, bits: float) -> int:
    return int(_lib.eden_num_packets(d, bits))


def recv_mask_words(d: int, bits: float) -> int:
    return int(_lib.eden_recv_mask_words(d, bits))


def workspace_bytes(d_max: int, n_batch: int) -> int:
    return int(_lib.eden_workspace_bytes(d_max, n_batch))


def mask_threshold_band(d: int, k: int, tenths: int = 40):
    """eden_mask_threshold_band: (lo, hi) of the band of keys predicted to hold the mask's threshold."""
    lo, hi = ctypes.c_uint32(), ctypes.c_uint32()
    _check(_lib.eden_mask_threshold_band(d, k, tenths, ctypes.byref(lo), ctypes.byref(hi)))
    return int(lo.value), int(hi.value)


def after_kept_count(d: int, bits: float) -> int:
    return int(_lib.eden_after_kept_count(d, bits))


def after_code_bytes(d: int, bits: float) -> int:
    return int(_lib.eden_after_code_bytes(d, bits))


def after_workspace_bytes(d: int, n: int) -> int:
    return int(_lib.eden_after_workspace_bytes(d, n))


def host_workspace_bytes(d: int, n: int) -> int:
    return int(_lib.eden_host_workspace_bytes(d, n))


def pass_plan(d: int, bits: float):
    """Index bits transformed by each sweep over HBM for one client (sender order)."""
    buf = (_u32 * 8)()
    n = _u32(0)
    _check(_lib.eden_pass_plan(d, bits, buf, 8, ctypes.byref(n)))
    return list(buf[: n.value])


def table(W: int):
    """(values float32[2^W], boundaries float32[2^W - 1]) the kernels quantise with."""
    c = np.zeros(1 << W, dtype=np.float32)
    b = np.zeros(max((1 << W) - 1, 1), dtype=np.float32)
    _check(_lib.eden_table(W, c.ctypes.data, b.ctypes.data))
    return c, b[: (1 << W) - 1]


def uniform_entropy(delta: float) -> float:
    return float(_lib.eden_uniform_entropy(float(delta)))


def uniform_delta(bits: float) -> float:
    """Delta_b of Section 4.3 (0.0 if outside the supported widths)."""
    return float(_lib.eden_uniform_delta(float(bits)))


def uniform_values(delta: float) -> np.ndarray:
    """float32[128]: the value of each magnitude index, as the kernels use it."""
    v = np.zeros(128, dtype=np.float32)
    _check(_lib.eden_uniform_values(float(delta), v.ctypes.data))
    return v


def uniform_index_bytes(d: int) -> int:
    return int(_lib.eden_uniform_index_bytes(d))


def _f64s(v) -> np.ndarray:
    return np.ascontiguousarray(v, dtype=np.float64)


def _u64s(v) -> np.ndarray:
    return np.ascontiguousarray(v, dtype=np.uint64)


def _ptr_table(tensors: Sequence[Optional[torch.Tensor]]):
    arr = (ctypes.c_void_p * len(tensors))()
    for i, t in enumerate(tensors):
        arr[i] = None if t is None else t.data_ptr()
    return arr


class Context:
    """One device, one stream, one caller-owned workspace (a torch uint8 tensor)."""

    def __init__(self, device: int = 0, workspace_bytes_: Optional[int] = None,
                 d_max: int = 1 << 20, n_batch: int = 1, stream: Optional[torch.cuda.Stream] = None,
                 host_staging: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("eden: no CUDA device; this library has no CPU path")
        self.device = device
        if workspace_bytes_ is None:
            workspace_bytes_ = (host_workspace_bytes if host_staging else workspace_bytes)(d_max, n_batch)
        with torch.cuda.device(device):
            self.stream = stream if stream is not None else torch.cuda.current_stream()
            self.workspace = torch.empty(int(workspace_bytes_) + 256, dtype=torch.uint8, device="cuda:%d" % device)
        base = self.workspace.data_ptr()
        aligned = (base + 255) // 256 * 256
        self._h = _vp()
        self.workspace_bytes = int(workspace_bytes_)
        _check(_lib.eden_create(ctypes.byref(self._h), device, self.stream.cuda_stream,
                                aligned, self.workspace_bytes))

    def close(self):
        if self._h:
            _lib.eden_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ sender
    def alloc_codes(self, d: int, bits) -> List[torch.Tensor]:
        return [torch.empty(code_bytes(d, float(b)), dtype=torch.uint8, device="cuda:%d" % self.device)
                for b in bits]

    def encode(self, x: torch.Tensor, bits, seeds, codes: Optional[List[torch.Tensor]] = None,
               scales: Optional[torch.Tensor] = None):
        """eden_encode: x is a CUDA fp32 [n, d] tensor (row stride >= d).  Returns (codes, scales)."""
        assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1
        n, d = x.shape
        bits, seeds = _f64s(bits), _u64s(seeds)
        assert len(bits) == n and len(seeds) == n
        if codes is None:
            codes = self.alloc_codes(d, bits)
        if scales is None:
            scales = torch.empty(n, dtype=torch.float32, device=x.device)
        tab = _ptr_table(codes)
        _check(_lib.eden_encode(self._h, x.data_ptr(), x.stride(0), d, n, bits.ctypes.data,
                                seeds.ctypes.data, tab, scales.data_ptr()))
        return codes, scales

    def encode_uniform(self, x: torch.Tensor, delta, seeds, index: Optional[List[torch.Tensor]] = None,
                       scales: Optional[torch.Tensor] = None):
        """eden_encode_uniform: one int8 index per rotated coordinate.  Returns (index, scales)."""
        assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1
        n, d = x.shape
        delta, seeds = _f64s(delta), _u64s(seeds)
        assert len(delta) == n and len(seeds) == n
        if index is None:
            index = [torch.empty(uniform_index_bytes(d), dtype=torch.int8, device=x.device) for _ in range(n)]
        if scales is None:
            scales = torch.empty(n, dtype=torch.float32, device=x.device)
        _check(_lib.eden_encode_uniform(self._h, x.data_ptr(), x.stride(0), d, n, delta.ctypes.data,
                                        seeds.ctypes.data, _ptr_table(index), scales.data_ptr()))
        return index, scales

    def mean_uniform(self, index, scales, delta, seeds, d: int, recv_masks=None,
                     out: Optional[torch.Tensor] = None):
        if out is None:
            out = torch.empty(d, dtype=torch.float32, device=scales.device)
        return self._decode(_lib.eden_mean_uniform, index, scales, delta, seeds, recv_masks, d, out)

    def decode_accumulate_uniform(self, index, scales, delta, seeds, d: int, acc: torch.Tensor, recv_masks=None):
        used = _u32(0)
        self._decode(_lib.eden_decode_accumulate_uniform, index, scales, delta, seeds, recv_masks, d, acc,
                     extra=(ctypes.byref(used),))
        return int(used.value)

    def index_histogram(self, index, d: int, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """eden_index_histogram: int32 [n, 256], column v + 128 counts index v."""
        n = len(index)
        if out is None:
            out = torch.empty((n, 256), dtype=torch.int32, device=index[0].device)
        _check(_lib.eden_index_histogram(self._h, _ptr_table(index), d, n, out.data_ptr()))
        return out

    # ------------------------------------------------------------------ receiver
    def _decode(self, fn, codes, scales, bits, seeds, recv_masks, d, out, extra=()):
        n = len(codes)
        bits, seeds = _f64s(bits), _u64s(seeds)
        assert len(bits) == n and len(seeds) == n and scales.is_cuda and scales.dtype == torch.float32
        tab = _ptr_table(codes)
        mtab = None if recv_masks is None else _ptr_table(recv_masks)
        _check(fn(self._h, tab, scales.data_ptr(), bits.ctypes.data, seeds.ctypes.data, mtab,
                  d, n, out.data_ptr(), *extra))
        return out

    def mean(self, codes, scales, bits, seeds, d: int, recv_masks=None, out: Optional[torch.Tensor] = None):
        """eden_mean: (1/n) sum_c x_hat_c as a CUDA fp32 [d] tensor."""
        if out is None:
            out = torch.empty(d, dtype=torch.float32, device=scales.device)
        return self._decode(_lib.eden_mean, codes, scales, bits, seeds, recv_masks, d, out)

    def mean_partial(self, codes, scales, bits, seeds, d: int, n_total: int, recv_masks=None,
                     out: Optional[torch.Tensor] = None):
        """eden_mean_partial: (1/n_total) * sum over the given clients; the partial vectors of
        all GPUs add up to the mean over all n_total senders."""
        if out is None:
            out = torch.empty(d, dtype=torch.float32, device=scales.device)
        n = len(codes)
        bits, seeds = _f64s(bits), _u64s(seeds)
        assert len(bits) == n and len(seeds) == n
        tab = _ptr_table(codes)
        mtab = None if recv_masks is None else _ptr_table(recv_masks)
        _check(_lib.eden_mean_partial(self._h, tab, scales.data_ptr(), bits.ctypes.data, seeds.ctypes.data, mtab,
                                      d, n, int(n_total), out.data_ptr()))
        return out

    def decode_accumulate(self, codes, scales, bits, seeds, d: int, acc: torch.Tensor, recv_masks=None,
                          used_so_far: int = 0):
        """eden_decode_accumulate: acc += sum_c x_hat_c; returns used_so_far + the clients counted."""
        used = _u32(used_so_far)
        self._decode(_lib.eden_decode_accumulate, codes, scales, bits, seeds, recv_masks, d, acc,
                     extra=(ctypes.byref(used),))
        return int(used.value)

    # ------------------------------------------------------------------ sparsification after the rotation
    def encode_sparsify_after(self, x: torch.Tensor, bits, seeds, codes: Optional[List[torch.Tensor]] = None,
                              scales: Optional[torch.Tensor] = None):
        """eden_encode_sparsify_after: b < 1 with the mask over the rotated coordinates."""
        assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1
        n, d = x.shape
        bits, seeds = _f64s(bits), _u64s(seeds)
        if codes is None:
            codes = [torch.empty(after_code_bytes(d, float(b)), dtype=torch.uint8, device=x.device) for b in bits]
        if scales is None:
            scales = torch.empty(n, dtype=torch.float32, device=x.device)
        _check(_lib.eden_encode_sparsify_after(self._h, x.data_ptr(), x.stride(0), d, n, bits.ctypes.data,
                                               seeds.ctypes.data, _ptr_table(codes), scales.data_ptr()))
        return codes, scales

    def mean_sparsify_after(self, codes, scales, bits, seeds, d: int, out: Optional[torch.Tensor] = None):
        n = len(codes)
        bits, seeds = _f64s(bits), _u64s(seeds)
        if out is None:
            out = torch.empty(d, dtype=torch.float32, device=scales.device)
        _check(_lib.eden_mean_sparsify_after(self._h, _ptr_table(codes), scales.data_ptr(), bits.ctypes.data,
                                             seeds.ctypes.data, d, n, out.data_ptr()))
        return out

    def decode_accumulate_sparsify_after(self, codes, scales, bits, seeds, d: int, acc: torch.Tensor,
                                         used_so_far: int = 0):
        n = len(codes)
        bits, seeds = _f64s(bits), _u64s(seeds)
        used = _u32(used_so_far)
        _check(_lib.eden_decode_accumulate_sparsify_after(self._h, _ptr_table(codes), scales.data_ptr(),
                                                          bits.ctypes.data, seeds.ctypes.data, d, n,
                                                          acc.data_ptr(), ctypes.byref(used)))
        return int(used.value)

    def sparsification_mask(self, seed: int, d: int, bits: float) -> torch.Tensor:
        """Bitmap (int32 words, bit i of word i/32) of the coordinates kept for b < 1."""
        out = torch.zeros((d + 31) // 32, dtype=torch.int32, device="cuda:%d" % self.device)
        _check(_lib.eden_sparsification_mask(self._h, int(seed), d, float(bits), out.data_ptr()))
        return out

    # ------------------------------------------------------------------ host-buffer variants
    def encode_host(self, x: np.ndarray, bits, seeds, codes: List[np.ndarray], scales: np.ndarray):
        """eden_encode_host: numpy/pinned host buffers in, host buffers out (synchronous)."""
        n, d = x.shape
        bits, seeds = _f64s(bits), _u64s(seeds)
        tab = (ctypes.c_void_p * n)(*[c.ctypes.data for c in codes])
        _check(_lib.eden_encode_host(self._h, x.ctypes.data, x.strides[0] // 4, d, n, bits.ctypes.data,
                                     seeds.ctypes.data, tab, scales.ctypes.data))

    def mean_host(self, codes: List[np.ndarray], scales: np.ndarray, bits, seeds, d: int,
                  recv_masks: Optional[List[Optional[np.ndarray]]], out: np.ndarray):
        n = len(codes)
        bits, seeds = _f64s(bits), _u64s(seeds)
        tab = (ctypes.c_void_p * n)(*[c.ctypes.data for c in codes])
        mtab = None
        if recv_masks is not None:
            mtab = (ctypes.c_void_p * n)(*[None if m is None else m.ctypes.data for m in recv_masks])
        _check(_lib.eden_mean_host(self._h, tab, scales.ctypes.data, bits.ctypes.data, seeds.ctypes.data,
                                   mtab, d, n, out.ctypes.data))

    # ------------------------------------------------------------------ status
    def status(self) -> int:
        w = _u32(0)
        _check(_lib.eden_status(self._h, ctypes.byref(w)))
        return int(w.value)

    def client_stats(self, n: int):
        arr = (ClientStat * n)()
        _check(_lib.eden_client_stats(self._h, n, arr))
        return [dict(norm2=a.norm2, dot=a.dot, received=a.received, flags=a.flags) for a in arr]

    def force_generic_kernels(self, on: bool):
        _check(_lib.eden_force_generic_kernels(self._h, 1 if on else 0))

    def set_option(self, option: int, value: int):
        """eden_set_option: one of the OPT_* switches of this module."""
        _check(_lib.eden_set_option(self._h, int(option), int(value)))

    def profile(self, on: bool):
        _check(_lib.eden_profile_enable(self._h, 1 if on else 0))

    def profile_collect(self):
        """Per-kernel totals since profile(True): name -> dict(launches, ms, bytes)."""
        n = _u32(0)
        _check(_lib.eden_profile_collect(self._h, ctypes.byref(n)))
        out = {}
        for i in range(n.value):
            name, launches, ms, nbytes = ctypes.c_char_p(), _u64(0), _f64(0), _f64(0)
            _check(_lib.eden_profile_get(self._h, i, ctypes.byref(name), ctypes.byref(launches),
                                         ctypes.byref(ms), ctypes.byref(nbytes)))
            out[name.value.decode()] = dict(launches=int(launches.value), ms=float(ms.value),
                                            bytes=float(nbytes.value))
        return out

    @property
    def launch_count(self) -> int:
        return int(_lib.eden_launch_count(self._h))


NOALLOC_MAX_DIM = 1 << 24


def sparsification_mask_noalloc(seed: int, d: int, bits: float, out: torch.Tensor,
                                device: int = 0, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """eden_sparsification_mask_noalloc: the b < 1 mask bitmap for callers that cannot
    allocate device memory (no context, no workspace; scratch is a fixed array inside the
    library).  `out` is a caller-owned CUDA int32 tensor of ceil(d/32) words.  Calls that
    overlap on the GPU share that scratch and race; keep them on one stream."""
    assert out.is_cuda and out.dtype == torch.int32 and out.numel() >= (d + 31) // 32
    s = stream if stream is not None else torch.cuda.current_stream(device)
    _check(_lib.eden_sparsification_mask_noalloc(device, s.cuda_stream, int(seed), int(d), float(bits),
                                                 out.data_ptr()))
    return out


# module-level calls with the names of the C entry points ---------------------------------
def eden_encode(ctx: Context, x, bits, seeds, codes=None, scales=None):
    return ctx.encode(x, bits, seeds, codes, scales)


def eden_mean(ctx: Context, codes, scales, bits, seeds, d, recv_masks=None, out=None):
    return ctx.mean(codes, scales, bits, seeds, d, recv_masks, out)


def eden_decode_accumulate(ctx: Context, codes, scales, bits, seeds, d, acc, recv_masks=None):
    return ctx.decode_accumulate(codes, scales, bits, seeds, d, acc, recv_masks)


def eden_encode_uniform(ctx: Context, x, delta, seeds, index=None, scales=None):
    return ctx.encode_uniform(x, delta, seeds, index, scales)


def eden_mean_uniform(ctx: Context, index, scales, delta, seeds, d, recv_masks=None, out=None):
    return ctx.mean_uniform(index, scales, delta, seeds, d, recv_masks, out)


def eden_decode_accumulate_uniform(ctx: Context, index, scales, delta, seeds, d, acc, recv_masks=None):
    return ctx.decode_accumulate_uniform(index, scales, delta, seeds, d, acc, recv_masks)


def eden_index_histogram(ctx: Context, index, d, out=None):
    return ctx.index_histogram(index, d, out)


def eden_mean_partial(ctx: Context, codes, scales, bits, seeds, d, n_total, recv_masks=None, out=None):
    return ctx.mean_partial(codes, scales, bits, seeds, d, n_total, recv_masks, out)
