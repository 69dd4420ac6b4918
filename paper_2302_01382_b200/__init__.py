"""Thin Python binding of the qcfg C-ABI library (include/qcfg.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch is used for device memory and streams.  The shared library is loaded on first
use; if it is missing and cannot be built the call fails loudly -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

from .build import LIB, build_library

OK = 0
PER_TENSOR, PER_ROW = 0, 1
ACT_NONE, ACT_RELU, ACT_GELU_TANH = 0, 1, 2
SEARCH_BISECTION, SEARCH_GREEDY = 0, 1
STATUS_NAMES = {0: "OK", 1: "EINVAL", 2: "EBITS", 3: "ESHAPE", 4: "EALIGN", 5: "ENOMEM", 6: "ENONFINITE", 7: "EARCH",
                8: "ECUDA", 9: "ETIMEOUT", 11: "ESTATE"}
EINVAL, EBITS, ESHAPE, EALIGN, ENOMEM, ENONFINITE, EARCH, ECUDA, ETIMEOUT = range(1, 10)
ESTATE = 11

EXPORTS = ["qcfg_create", "qcfg_destroy", "qcfg_sync_status", "qcfg_selftest_wait_timeout", "qcfg_last_error", "qcfg_launch_count",
           "qcfg_set_fusion", "qcfg_set_pair_tiles", "qcfg_set_grouping", "qcfg_set_prefix_reuse", "qcfg_set_implicit_conv", "qcfg_set_gemm_chains", "qcfg_profile_enable", "qcfg_profile_read", "qcfg_calibrate", "qcfg_scales_from_absmax", "qcfg_quantize",
           "qcfg_quant_error_sweep", "qcfg_quant_error_sweep_static", "qcfg_gemm_i8", "qcfg_gemm_i8_requant", "qcfg_gemm_bf16", "qcfg_model_create",
           "qcfg_model_destroy", "qcfg_calibrate_model", "qcfg_model_act_absmax",
           "qcfg_model_weight_absmax", "qcfg_eval_config", "qcfg_latency_table", "qcfg_config_cost", "qcfg_noise_sensitivity", "qcfg_search", "qcfg_adjust_scales", "qcfg_scale_gradients", "qcfg_model_scales",
           "qcfg_model_reset_scales", "qcfg_debug_dump"]


class QcfgError(RuntimeError):
    def __init__(self, status: int, msg: str = ""):
        name = STATUS_NAMES.get(status, str(status))
        super().__init__(f"QCFG_{name}: {msg}")
        self.status = status


class LayerStruct(C.Structure):
    _fields_ = [("w_dev", C.c_void_p), ("n_out", C.c_int64), ("k_in", C.c_int64), ("src", C.c_int32),
                ("src_col0", C.c_int32), ("act", C.c_int32), ("kh", C.c_int32), ("kw", C.c_int32),
                ("stride", C.c_int32), ("pad", C.c_int32), ("in_h", C.c_int32), ("in_w", C.c_int32),
                ("in_c", C.c_int32), ("pool_before", C.c_int32), ("src_h", C.c_int32), ("src_w", C.c_int32),
                ("residual_from", C.c_int32)]


_lib = None


def load_library() -> C.CDLL:
    """Loads libqcfg.so (building it with nvcc first if it is absent)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB):
        build_library()
    lib = C.CDLL(LIB)
    vp, i64, i32, ci, f32 = C.c_void_p, C.c_int64, C.c_int32, C.c_int, C.c_float
    sig = {
        "qcfg_create": [C.POINTER(vp), ci],
        "qcfg_destroy": [vp],
        "qcfg_sync_status": [vp, vp],
        "qcfg_selftest_wait_timeout": [vp, C.c_uint64, vp],
        "qcfg_set_fusion": [vp, ci],
        "qcfg_set_pair_tiles": [vp, ci],
        "qcfg_set_grouping": [vp, ci],
        "qcfg_set_prefix_reuse": [vp, ci],
        "qcfg_set_implicit_conv": [vp, ci],
        "qcfg_set_gemm_chains": [vp, ci],
        "qcfg_profile_enable": [vp, ci],
        "qcfg_profile_read": [vp, ci, C.POINTER(C.c_double), C.POINTER(i64), C.POINTER(C.c_double), ci],
        "qcfg_calibrate": [vp, vp, i64, i64, i64, ci, vp, vp],
        "qcfg_scales_from_absmax": [vp, vp, i64, ci, vp, vp, vp],
        "qcfg_quantize": [vp, vp, i64, i64, i64, vp, ci, ci, vp, i64, vp],
        "qcfg_quant_error_sweep": [vp, C.POINTER(vp), C.POINTER(i64), C.POINTER(i64), i32, ci, ci, ci, vp, vp, vp],
        "qcfg_quant_error_sweep_static": [vp, C.POINTER(vp), C.POINTER(i64), C.POINTER(i64), i32, ci, ci, ci, vp, vp, vp],
        "qcfg_gemm_i8": [vp, vp, i64, vp, i64, i64, i64, i64, f32, vp, ci, vp, vp, vp],
        "qcfg_gemm_i8_requant": [vp, vp, i64, vp, i64, i64, i64, i64, f32, vp, ci, f32, ci, vp, i64, vp],
        "qcfg_gemm_bf16": [vp, vp, i64, vp, i64, i64, i64, i64, ci, vp, vp],
        "qcfg_model_create": [vp, C.POINTER(LayerStruct), i32, C.POINTER(vp)],
        "qcfg_model_destroy": [vp],
        "qcfg_calibrate_model": [vp, vp, vp, i64, vp],
        "qcfg_model_act_absmax": [vp, C.POINTER(f32)],
        "qcfg_model_weight_absmax": [vp, i32, C.POINTER(f32)],
        "qcfg_eval_config": [vp, vp, C.POINTER(C.c_uint8), vp, i64, C.POINTER(vp), vp],
        "qcfg_debug_dump": [vp, vp, i32, vp, vp, vp, vp],
        "qcfg_search": [vp, vp, ci, C.POINTER(i32), C.POINTER(C.c_uint8), i32, C.c_double, vp, i64, C.POINTER(C.c_uint8),
                        C.POINTER(C.c_uint8), C.POINTER(C.c_double), i32, C.POINTER(i32), vp],
        "qcfg_noise_sensitivity": [vp, vp, vp, i64, C.POINTER(C.c_void_p), C.c_float, C.POINTER(C.c_double), vp],
        "qcfg_adjust_scales": [vp, vp, C.POINTER(C.c_uint8), vp, i64, i32, C.c_double, C.POINTER(C.c_double), vp],
        "qcfg_scale_gradients": [vp, vp, C.POINTER(C.c_uint8), vp, i64, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                 C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_double), vp],
        "qcfg_model_scales": [vp, i32, ci, C.POINTER(f32), C.POINTER(f32), C.POINTER(f32), C.POINTER(f32)],
        "qcfg_model_reset_scales": [vp],
        "qcfg_latency_table": [vp, vp, vp, i64, C.POINTER(C.c_uint8), i32, i32, C.POINTER(C.c_float), vp],
        "qcfg_config_cost": [vp, C.POINTER(C.c_uint8), C.POINTER(C.c_uint8), i32, C.POINTER(C.c_float), C.POINTER(C.c_double),
                             C.POINTER(C.c_double)],
    }
    for name, args in sig.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = ci
    lib.qcfg_last_error.argtypes = [vp]
    lib.qcfg_last_error.restype = C.c_char_p
    lib.qcfg_launch_count.argtypes = [vp]
    lib.qcfg_launch_count.restype = i64
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


class Context:
    """Owns one qcfg_ctx.  Methods carry the C entry points' names without the prefix."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        h = C.c_void_p()
        rc = self.lib.qcfg_create(C.byref(h), device)
        if rc != OK:
            raise QcfgError(rc, "qcfg_create failed (an sm_100 CUDA device is required)")
        self.h = h
        self.device = device

    def close(self):
        if getattr(self, "h", None):
            self.lib.qcfg_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != OK:
            raise QcfgError(rc, self.last_error())

    def last_error(self) -> str:
        return self.lib.qcfg_last_error(self.h).decode()

    def launch_count(self) -> int:
        return int(self.lib.qcfg_launch_count(self.h))

    def sync_status(self, stream=None) -> int:
        return int(self.lib.qcfg_sync_status(self.h, _stream(stream)))

    def selftest_wait_timeout(self, limit_ns: int, stream=None):
        self._check(self.lib.qcfg_selftest_wait_timeout(self.h, int(limit_ns), _stream(stream)))

    def check_sync(self, stream=None):
        self._check(self.sync_status(stream))

    def set_fusion(self, enabled: bool):
        self._check(self.lib.qcfg_set_fusion(self.h, int(enabled)))

    def set_grouping(self, enabled: bool):
        self._check(self.lib.qcfg_set_grouping(self.h, int(enabled)))

    def set_prefix_reuse(self, enabled: bool):
        self._check(self.lib.qcfg_set_prefix_reuse(self.h, int(enabled)))

    def set_implicit_conv(self, enabled: bool):
        self._check(self.lib.qcfg_set_implicit_conv(self.h, int(enabled)))

    def set_gemm_chains(self, enabled: bool):
        self._check(self.lib.qcfg_set_gemm_chains(self.h, int(enabled)))

    def set_pair_tiles(self, enabled: bool):
        self._check(self.lib.qcfg_set_pair_tiles(self.h, int(enabled)))

    def profile_enable(self, mode):
        """0 off, 1 CUDA events around every launch, 2 in-kernel time stamps of the GEMM launches."""
        self._check(self.lib.qcfg_profile_enable(self.h, int(mode)))

    def profile_read(self, kernel_class: int, reset: bool = True):
        ms, n, ops = C.c_double(), C.c_int64(), C.c_double()
        self._check(self.lib.qcfg_profile_read(self.h, kernel_class, C.byref(ms), C.byref(n), C.byref(ops), int(reset)))
        return ms.value, n.value, ops.value

    # ---- tensor-level steps
    def calibrate(self, x: torch.Tensor, granularity: int, out: Optional[torch.Tensor] = None, stream=None):
        rows, cols = x.shape
        if out is None:
            out = torch.empty(1 if granularity == PER_TENSOR else rows, dtype=torch.float32, device=x.device)
        self._check(self.lib.qcfg_calibrate(self.h, _ptr(x), rows, cols, x.stride(0), granularity, _ptr(out), _stream(stream)))
        return out

    def scales_from_absmax(self, absmax: torch.Tensor, bits: int, stream=None):
        scale = torch.empty_like(absmax)
        inv = torch.empty_like(absmax)
        self._check(self.lib.qcfg_scales_from_absmax(self.h, _ptr(absmax), absmax.numel(), bits, _ptr(scale), _ptr(inv), _stream(stream)))
        return scale, inv

    def quantize(self, x: torch.Tensor, inv_scale: Optional[torch.Tensor], granularity: int, bits: int,
                 ldq: Optional[int] = None, stream=None) -> torch.Tensor:
        rows, cols = x.shape
        if ldq is None:
            ldq = (cols + 15) // 16 * 16
        q = torch.empty((rows, ldq), dtype=torch.bfloat16 if bits == 16 else torch.int8, device=x.device)
        self._check(self.lib.qcfg_quantize(self.h, _ptr(x), rows, cols, x.stride(0), _ptr(inv_scale), granularity, bits,
                                           _ptr(q), ldq, _stream(stream)))
        return q

    def quant_error_sweep(self, tensors: Sequence[torch.Tensor], granularity: int = PER_ROW, b_lo: int = 2, b_hi: int = 8,
                          sse: Optional[torch.Tensor] = None, absmax: Optional[torch.Tensor] = None, stream=None):
        n = len(tensors)
        nb = b_hi - b_lo + 1
        dev = tensors[0].device if n else torch.device("cuda", self.device)
        if sse is None:
            sse = torch.empty((n, nb), dtype=torch.float64, device=dev)
        if absmax is None:
            absmax = torch.empty(n, dtype=torch.float32, device=dev)
        ptrs = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in tensors])
        rows = (C.c_int64 * max(n, 1))(*[t.shape[0] for t in tensors])
        cols = (C.c_int64 * max(n, 1))(*[t.shape[1] for t in tensors])
        self._check(self.lib.qcfg_quant_error_sweep(self.h, ptrs, rows, cols, n, granularity, b_lo, b_hi, _ptr(sse),
                                                    _ptr(absmax), _stream(stream)))
        return sse, absmax

    def quant_error_sweep_static(self, tensors: Sequence[torch.Tensor], granularity: int = PER_ROW, b_lo: int = 2,
                                 b_hi: int = 8, sse: Optional[torch.Tensor] = None, absmax: Optional[torch.Tensor] = None,
                                 shapes: Optional[Sequence] = None, stream=None):
        """The sweep through the entry point that allocates no device memory (fixed scratch array
        inside the library, shared by all calls: do not overlap two of them on the GPU).  Pass
        `sse` and `absmax` to keep the binding from allocating either.  `shapes` overrides the
        (rows, cols) taken from the tensors."""
        n = len(tensors)
        nb = b_hi - b_lo + 1
        dev = tensors[0].device if n else torch.device("cuda", self.device)
        if sse is None:
            sse = torch.empty((n, nb), dtype=torch.float64, device=dev)
        if absmax is None:
            absmax = torch.empty(n, dtype=torch.float32, device=dev)
        shp = shapes if shapes is not None else [tuple(t.shape) for t in tensors]
        ptrs = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in tensors])
        rows = (C.c_int64 * max(n, 1))(*[s[0] for s in shp])
        cols = (C.c_int64 * max(n, 1))(*[s[1] for s in shp])
        self._check(self.lib.qcfg_quant_error_sweep_static(self.h, ptrs, rows, cols, n, granularity, b_lo, b_hi,
                                                           _ptr(sse), _ptr(absmax), _stream(stream)))
        return sse, absmax

    def gemm_i8(self, qx: torch.Tensor, qw: torch.Tensor, k: int, scale_x: float, scale_w: Optional[torch.Tensor],
                act: int = ACT_NONE, want_y: bool = True, want_acc: bool = False, stream=None):
        m, n = qx.shape[0], qw.shape[0]
        y = torch.empty((m, n), dtype=torch.float32, device=qx.device) if want_y else None
        acc = torch.empty((m, n), dtype=torch.int32, device=qx.device) if want_acc else None
        self._check(self.lib.qcfg_gemm_i8(self.h, _ptr(qx), qx.stride(0), _ptr(qw), qw.stride(0), m, n, k, scale_x,
                                          _ptr(scale_w), act, _ptr(y), _ptr(acc), _stream(stream)))
        return y, acc

    def gemm_i8_requant(self, qx: torch.Tensor, qw: torch.Tensor, k: int, scale_x: float, scale_w: torch.Tensor, act: int,
                        next_inv_scale: float, next_bits: int, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        m, n = qx.shape[0], qw.shape[0]
        if out is None:
            out = torch.zeros((m, (n + 15) // 16 * 16), dtype=torch.bfloat16 if next_bits == 16 else torch.int8, device=qx.device)
        self._check(self.lib.qcfg_gemm_i8_requant(self.h, _ptr(qx), qx.stride(0), _ptr(qw), qw.stride(0), m, n, k, scale_x,
                                                  _ptr(scale_w), act, next_inv_scale, next_bits, _ptr(out), out.stride(0),
                                                  _stream(stream)))
        return out

    def gemm_bf16(self, x: torch.Tensor, w: torch.Tensor, k: int, act: int = ACT_NONE, stream=None) -> torch.Tensor:
        m, n = x.shape[0], w.shape[0]
        y = torch.empty((m, n), dtype=torch.float32, device=x.device)
        self._check(self.lib.qcfg_gemm_bf16(self.h, _ptr(x), x.stride(0), _ptr(w), w.stride(0), m, n, k, act, _ptr(y), _stream(stream)))
        return y


class Model:
    """Owns one qcfg_model built from a list of layer descriptions and device weights."""

    def __init__(self, ctx: Context, layers, weights: Sequence[torch.Tensor]):
        self.ctx = ctx
        self.layers = list(layers)
        self.weights = list(weights)          # keeps the borrowed device memory alive
        arr = (LayerStruct * len(self.layers))()
        for i, (l, w) in enumerate(zip(self.layers, self.weights)):
            assert w.dtype == torch.float32 and w.is_contiguous() and tuple(w.shape) == (l.n_out, l.k_in)
            arr[i] = LayerStruct(w.data_ptr(), l.n_out, l.k_in, l.src, l.src_col0, l.act, l.kh, l.kw, l.stride, l.pad,
                                 l.in_h, l.in_w, l.in_c, l.pool_before, l.src_h, l.src_w, l.residual_from)
        h = C.c_void_p()
        ctx._check(ctx.lib.qcfg_model_create(ctx.h, arr, len(self.layers), C.byref(h)))
        self.h = h

    def close(self):
        if getattr(self, "h", None) and self.ctx.h:
            self.ctx.lib.qcfg_model_destroy(self.h)
        self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def calibrate_model(self, x: torch.Tensor, m: int, stream=None):
        self.ctx._check(self.ctx.lib.qcfg_calibrate_model(self.ctx.h, self.h, _ptr(x), m, _stream(stream)))

    def act_absmax(self) -> List[float]:
        out = (C.c_float * len(self.layers))()
        self.ctx._check(self.ctx.lib.qcfg_model_act_absmax(self.h, out))
        return list(out)

    def weight_absmax(self, layer: int):
        out = (C.c_float * self.layers[layer].n_out)()
        self.ctx._check(self.ctx.lib.qcfg_model_weight_absmax(self.h, layer, out))
        return list(out)

    def eval_config(self, bits, x: torch.Tensor, m: int, y: Optional[Sequence[Optional[torch.Tensor]]] = None, stream=None):
        n = len(self.layers)
        b = (C.c_uint8 * n)(*[int(v) for v in bits])
        yp = None
        if y is not None:
            yp = (C.c_void_p * n)(*[None if t is None else t.data_ptr() for t in y])
        self.ctx._check(self.ctx.lib.qcfg_eval_config(self.ctx.h, self.h, b, _ptr(x), m, yp, _stream(stream)))

    def search(self, algorithm: int, order, bs, target: float, x: torch.Tensor, m: int, capacity: int = 4096, stream=None):
        """Algorithm 1 (algorithm=0, bisection) or 2 (1, greedy).  Returns (bits, visited configurations, fidelities)."""
        n = len(self.layers)
        order_a = (C.c_int32 * n)(*[int(v) for v in order])
        bs_a = (C.c_uint8 * len(bs))(*[int(v) for v in bs])
        bits = (C.c_uint8 * n)()
        visited = (C.c_uint8 * (capacity * n))()
        acc = (C.c_double * capacity)()
        n_evals = C.c_int32()
        self.ctx._check(self.ctx.lib.qcfg_search(self.ctx.h, self.h, algorithm, order_a, bs_a, len(bs), float(target), _ptr(x), m,
                                                 bits, visited, acc, capacity, C.byref(n_evals), _stream(stream)))
        k = min(n_evals.value, capacity)
        vis = [list(visited[i * n:(i + 1) * n]) for i in range(k)]
        return list(bits), vis, list(acc[:k]), n_evals.value

    def noise_sensitivity(self, x: torch.Tensor, m: int, noises, lam: float, stream=None):
        """E_N per layer (Eqs. 3-5); noises[l] is a standard-normal tensor shaped like layer l's weight, or None."""
        n = len(self.layers)
        ptrs = (C.c_void_p * n)(*[None if t is None else t.data_ptr() for t in noises])
        out = (C.c_double * n)()
        self.ctx._check(self.ctx.lib.qcfg_noise_sensitivity(self.ctx.h, self.h, _ptr(x), m, ptrs, float(lam), out, _stream(stream)))
        return list(out)

    def adjust_scales(self, bits, x: torch.Tensor, m: int, steps: int, lr: float = 1e-5, stream=None):
        """Section 3.1's adjustment step: `steps` gradient steps on the scales.  Returns the losses (steps + 1)."""
        n = len(self.layers)
        b = (C.c_uint8 * n)(*[int(v) for v in bits])
        losses = (C.c_double * (steps + 1))()
        self.ctx._check(self.ctx.lib.qcfg_adjust_scales(self.ctx.h, self.h, b, _ptr(x), m, steps, float(lr), losses, _stream(stream)))
        return list(losses)

    def scale_gradients(self, bits, x: torch.Tensor, m: int, stream=None):
        """(loss, d_scale_x, d_inv_scale_x, d_scale_w, d_inv_scale_w); the last two are lists of per-channel lists."""
        n = len(self.layers)
        b = (C.c_uint8 * n)(*[int(v) for v in bits])
        dsx, dix, loss = (C.c_double * n)(), (C.c_double * n)(), C.c_double()
        bufs_s = [(C.c_double * l.n_out)() for l in self.layers]
        bufs_i = [(C.c_double * l.n_out)() for l in self.layers]
        ps = (C.c_void_p * n)(*[C.addressof(a) for a in bufs_s])
        pi = (C.c_void_p * n)(*[C.addressof(a) for a in bufs_i])
        self.ctx._check(self.ctx.lib.qcfg_scale_gradients(self.ctx.h, self.h, b, _ptr(x), m, dsx, dix, ps, pi, C.byref(loss), _stream(stream)))
        return loss.value, list(dsx), list(dix), [list(a) for a in bufs_s], [list(a) for a in bufs_i]

    def scales(self, layer: int, bits: int):
        """(scale_x, inv_scale_x, scale_w[n_out], inv_scale_w[n_out]) in use for `layer` at `bits`."""
        n_out = self.layers[layer].n_out
        sx, ix = C.c_float(), C.c_float()
        sw, iw = (C.c_float * n_out)(), (C.c_float * n_out)()
        self.ctx._check(self.ctx.lib.qcfg_model_scales(self.h, layer, bits, C.byref(sx), C.byref(ix), sw, iw))
        return sx.value, ix.value, list(sw), list(iw)

    def reset_scales(self):
        self.ctx._check(self.ctx.lib.qcfg_model_reset_scales(self.h))

    def latency_table(self, x: torch.Tensor, m: int, bs, reps: int = 5, stream=None):
        """Mean milliseconds of every layer at every width of bs: list of n_layers rows of len(bs) floats."""
        n = len(self.layers)
        bs_a = (C.c_uint8 * len(bs))(*[int(v) for v in bs])
        out = (C.c_float * (n * len(bs)))()
        self.ctx._check(self.ctx.lib.qcfg_latency_table(self.ctx.h, self.h, _ptr(x), m, bs_a, len(bs), reps, out, _stream(stream)))
        return [list(out[l * len(bs):(l + 1) * len(bs)]) for l in range(n)]

    def config_cost(self, bits, bs=None, table=None):
        """(latency in ms or None, size in bytes) of a configuration; latency needs bs and the table."""
        n = len(self.layers)
        b = (C.c_uint8 * n)(*[int(v) for v in bits])
        size = C.c_double()
        if table is None:
            self.ctx._check(self.ctx.lib.qcfg_config_cost(self.h, b, None, 0, None, None, C.byref(size)))
            return None, size.value
        bs_a = (C.c_uint8 * len(bs))(*[int(v) for v in bs])
        flat = (C.c_float * (n * len(bs)))(*[float(v) for row in table for v in row])
        lat = C.c_double()
        self.ctx._check(self.ctx.lib.qcfg_config_cost(self.h, b, bs_a, len(bs), flat, C.byref(lat), C.byref(size)))
        return lat.value, size.value

    def debug_dump(self, layer: int, qx: Optional[torch.Tensor], qw: Optional[torch.Tensor], acc: Optional[torch.Tensor], stream=None):
        self.ctx._check(self.ctx.lib.qcfg_debug_dump(self.ctx.h, self.h, layer, _ptr(qx), _ptr(qw), _ptr(acc), _stream(stream)))
