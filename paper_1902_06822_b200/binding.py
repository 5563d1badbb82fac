"""Thin ctypes binding of the C interface in include/omse.h.

Argument marshalling only: every step of the method runs in the CUDA kernels of libomse.so.
PyTorch supplies device memory and the stream; tensors are passed as raw device pointers.
The library must be present (build it with paper_1902_06822_b200.build.build()); there is no
fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

OK, EINVAL, ECUDA, ENOMEM, ELIMIT = 0, -1, -2, -3, -4
DEV_NONFINITE, DEV_DEGENERATE = 1, 2
MAX_CANDIDATES, MAX_KERNEL_LEN, MAX_KERNEL_LEN_MULTISWEEP, MAX_TENSORS = 4096, 28672, 25600, 4
STATIC_MAX_CANDIDATES = 2048

EXPORTS = [
    "omse_create", "omse_destroy", "omse_set_stream", "omse_workspace_bytes", "omse_quantize_weights",
    "omse_quantize_weights_batched", "omse_dual_quantize", "omse_select_key_layers", "omse_compression_ratio",
    "omse_alg1_quantize", "omse_read_evaluations", "omse_quantize_weights_offset", "omse_activation_scale_offset",
    "omse_activation_scale", "omse_residual_quantize", "omse_pack_int4", "omse_last_device_status",
    "omse_status_string", "omse_activation_scale_static", "omse_alg1_quantize_converge",
    "omse_quantize_weights_solver", "omse_quantize_weights_affine", "omse_quantize_key_layers",
    "omse_measure_fp32_peak", "omse_read_launches",
]
SOLVER_GRID, SOLVER_UNIFORM, SOLVER_ALTERNATING, SOLVER_GOLDEN = 0, 1, 2, 3
MAX_OFFSETS = 64


class OmseGrid(C.Structure):
    _fields_ = [("n_cand", C.c_int32), ("hi_frac", C.c_float), ("refine_iters", C.c_int32)]


class OmseWeightTensor(C.Structure):
    _fields_ = [("d_w", C.c_void_p), ("n_kernels", C.c_int64), ("kernel_len", C.c_int64), ("d_alpha", C.c_void_p),
                ("d_sse", C.c_void_p), ("d_best_idx", C.c_void_p), ("d_codes", C.c_void_p), ("d_packed", C.c_void_p)]


class OmseDualGrid(C.Structure):
    _fields_ = [("n_cand1", C.c_int32), ("n_cand2", C.c_int32), ("hi_frac1", C.c_float), ("hi_frac2", C.c_float)]


class OmseLayerError(C.Structure):
    _fields_ = [("d_sse", C.c_void_p), ("n_kernels", C.c_int64), ("kernel_len", C.c_int64)]


class OmseOffsetGrid(C.Structure):
    _fields_ = [("n_delta", C.c_int32), ("off_frac", C.c_float)]


class OmseKeyLayer(C.Structure):
    _fields_ = [("first", OmseWeightTensor), ("d_alpha2", C.c_void_p), ("d_sse2", C.c_void_p),
                ("d_codes2", C.c_void_p), ("d_packed2", C.c_void_p)]


class OmseError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: {status_string(code)} ({code})")
        self.code = code


_lib = None


def load_library() -> C.CDLL:
    """dlopen libomse.so and declare the prototypes; raises if the library has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_build.LIB_PATH):
        raise FileNotFoundError(f"{_build.LIB_PATH} is missing: run paper_1902_06822_b200.build.build() first")
    lib = C.CDLL(_build.LIB_PATH)
    vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int
    lib.omse_create.argtypes = [C.POINTER(vp), i32, vp]
    lib.omse_destroy.argtypes = [vp]
    lib.omse_set_stream.argtypes = [vp, vp]
    lib.omse_workspace_bytes.argtypes = [i64, i64, C.c_int32, C.c_int32]
    lib.omse_workspace_bytes.restype = C.c_size_t
    lib.omse_quantize_weights.argtypes = [vp, vp, i64, i64, i32, i32, C.POINTER(OmseGrid), vp, vp, vp, vp, vp]
    lib.omse_quantize_weights_batched.argtypes = [vp, C.POINTER(OmseWeightTensor), i32, i32, i32, C.POINTER(OmseGrid)]
    lib.omse_activation_scale.argtypes = [vp, vp, i64, i32, i32, C.POINTER(OmseGrid), vp, vp, vp, vp]
    lib.omse_residual_quantize.argtypes = [vp, vp, i64, i64, C.POINTER(C.c_int), i32, C.POINTER(OmseGrid), i32, i32,
                                           vp, vp, vp, vp]
    lib.omse_pack_int4.argtypes = [vp, vp, i64, i32, vp]
    lib.omse_quantize_weights_offset.argtypes = [vp, vp, i64, i64, i32, C.POINTER(OmseGrid), vp, vp, vp, vp, vp, vp]
    lib.omse_activation_scale_offset.argtypes = [vp, vp, i64, i32, C.POINTER(OmseGrid), vp, vp, vp, vp, vp]
    lib.omse_alg1_quantize.argtypes = [vp, vp, i64, i64, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(OmseGrid),
                                       i32, i32, vp, vp, vp, vp, vp]
    lib.omse_alg1_quantize_converge.argtypes = [vp, vp, i64, i64, C.POINTER(C.c_int), C.POINTER(C.c_int),
                                                C.POINTER(OmseGrid), i32, i32, C.c_float, vp, vp, vp, vp, vp, vp]
    lib.omse_quantize_weights_solver.argtypes = [vp, vp, i64, i64, i32, i32, i32, i32, C.POINTER(OmseGrid), vp, vp, vp,
                                                 vp, vp]
    lib.omse_quantize_weights_affine.argtypes = [vp, vp, i64, i64, i32, C.POINTER(OmseGrid), C.POINTER(OmseOffsetGrid),
                                                 vp, vp, vp, vp, vp, vp]
    lib.omse_quantize_key_layers.argtypes = [vp, C.POINTER(OmseKeyLayer), i32, i32, i32, C.POINTER(OmseGrid), C.c_float,
                                             vp, vp, vp]
    lib.omse_select_key_layers.argtypes = [vp, C.POINTER(OmseLayerError), i32, C.c_float, vp, vp]
    lib.omse_compression_ratio.argtypes = [C.POINTER(i64), C.POINTER(i64), C.POINTER(i32), C.POINTER(i32), i32]
    lib.omse_compression_ratio.restype = C.c_double
    lib.omse_dual_quantize.argtypes = [vp, vp, i64, i64, i32, i32, i32, C.POINTER(OmseDualGrid), vp, vp, vp, vp, vp]
    lib.omse_activation_scale_static.argtypes = [i32, vp, vp, i64, i32, i32, C.POINTER(OmseGrid), vp, vp, vp, vp, vp]
    lib.omse_last_device_status.argtypes = [vp, C.POINTER(C.c_uint32)]
    lib.omse_read_evaluations.argtypes = [vp, C.POINTER(C.c_uint64)]
    lib.omse_measure_fp32_peak.argtypes = [vp, i32, C.POINTER(C.c_double)]
    lib.omse_read_launches.argtypes = [vp, C.POINTER(C.c_uint64)]
    lib.omse_status_string.argtypes = [i32]
    lib.omse_status_string.restype = C.c_char_p
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().omse_status_string(code).decode()


def _ptr(t: torch.Tensor | None, dtype: torch.dtype | None = None):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def omse_activation_scale_static(x, n, bits, is_signed, n_cand, hi_frac, refine_iters, alpha, sse, best_idx=None,
                                 sse_curve=None, status=None, stream=None):
    """Per-tensor scale search that allocates nothing and needs no Context.

    For callers that must not allocate device memory (they cannot build a Context either, since that
    allocates the workspace): the scratch is a fixed array inside the library.  Runs on x's device and
    on `stream` (default: torch's current stream).  At most STATIC_MAX_CANDIDATES candidates; calls that
    may overlap on the GPU must not be issued, they share the scratch.  status: optional uint32-sized
    CUDA tensor (dtype int32) receiving this call's device status bits.
    """
    dev = x.device if n > 0 else alpha.device
    st = stream if stream is not None else torch.cuda.current_stream(dev)
    g = OmseGrid(n_cand, hi_frac, refine_iters)
    rc = load_library().omse_activation_scale_static(
        dev.index or 0, C.c_void_p(st.cuda_stream), _ptr(x, torch.float32), n, bits, int(is_signed), C.byref(g),
        _ptr(alpha, torch.float32), _ptr(sse, torch.float32), _ptr(best_idx, torch.int32),
        _ptr(sse_curve, torch.float64), _ptr(status, torch.int32))
    if rc != OK:
        raise OmseError(rc, "omse_activation_scale_static")


def omse_compression_ratio(n_kernels, kernel_len, bits, n_tensors) -> float:
    """Section 3.5 compression ratio of a set of layers (host arithmetic)."""
    n = len(n_kernels)
    return float(load_library().omse_compression_ratio((C.c_int64 * n)(*n_kernels), (C.c_int64 * n)(*kernel_len),
                                                       (C.c_int * n)(*bits), (C.c_int * n)(*n_tensors), n))


class Context:
    """An omse_ctx bound to a device and to the torch stream that is current at construction."""

    def __init__(self, device: int | torch.device = 0, stream: torch.cuda.Stream | None = None):
        lib = load_library()
        dev = torch.device(device) if not isinstance(device, int) else torch.device("cuda", device)
        self.device = dev
        self._stream = stream if stream is not None else torch.cuda.current_stream(dev)
        h = C.c_void_p()
        rc = lib.omse_create(C.byref(h), dev.index or 0, C.c_void_p(self._stream.cuda_stream))
        if rc != OK:
            raise OmseError(rc, "omse_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            load_library().omse_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_stream(self, stream: torch.cuda.Stream):
        self._stream = stream
        rc = load_library().omse_set_stream(self._h, C.c_void_p(stream.cuda_stream))
        if rc != OK:
            raise OmseError(rc, "omse_set_stream")

    @staticmethod
    def workspace_bytes(n_kernels: int = 1, kernel_len: int = 1, n_cand: int = 1, n_tensors: int = 1) -> int:
        return int(load_library().omse_workspace_bytes(n_kernels, kernel_len, n_cand, n_tensors))

    # -- the four calls of the library --------------------------------------------------------
    def omse_quantize_weights(self, w, n_kernels, kernel_len, bits, is_signed, n_cand, hi_frac, refine_iters,
                              alpha, sse, best_idx=None, codes=None, packed=None):
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        rc = load_library().omse_quantize_weights(
            self._h, _ptr(w, torch.float32), n_kernels, kernel_len, bits, int(is_signed), C.byref(g),
            _ptr(alpha, torch.float32), _ptr(sse, torch.float32), _ptr(best_idx, torch.int32),
            _ptr(codes, torch.int8), _ptr(packed, torch.uint8))
        if rc != OK:
            raise OmseError(rc, "omse_quantize_weights")

    def omse_quantize_weights_batched(self, tensors, bits, is_signed, n_cand, hi_frac, refine_iters):
        """tensors: sequence of dicts with keys w, n_kernels, kernel_len, alpha, sse and optionally
        best_idx, codes, packed (CUDA tensors), one per weight tensor; all quantized in one launch."""
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        arr = (OmseWeightTensor * len(tensors))()
        for d, t in zip(arr, tensors):
            d.d_w = _ptr(t["w"], torch.float32)
            d.n_kernels, d.kernel_len = t["n_kernels"], t["kernel_len"]
            d.d_alpha = _ptr(t["alpha"], torch.float32)
            d.d_sse = _ptr(t["sse"], torch.float32)
            d.d_best_idx = _ptr(t.get("best_idx"), torch.int32)
            d.d_codes = _ptr(t.get("codes"), torch.int8)
            d.d_packed = _ptr(t.get("packed"), torch.uint8)
        rc = load_library().omse_quantize_weights_batched(self._h, arr, len(tensors), bits, int(is_signed), C.byref(g))
        if rc != OK:
            raise OmseError(rc, "omse_quantize_weights_batched")

    def omse_activation_scale(self, x, n, bits, is_signed, n_cand, hi_frac, refine_iters, alpha, sse,
                              best_idx=None, sse_curve=None):
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        rc = load_library().omse_activation_scale(
            self._h, _ptr(x, torch.float32), n, bits, int(is_signed), C.byref(g), _ptr(alpha, torch.float32),
            _ptr(sse, torch.float32), _ptr(best_idx, torch.int32), _ptr(sse_curve, torch.float64))
        if rc != OK:
            raise OmseError(rc, "omse_activation_scale")

    def omse_residual_quantize(self, t, n_kernels, kernel_len, bits, is_signed, n_cand, hi_frac, refine_iters,
                               n_sweeps, alpha, sse, codes=None, packed=None):
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        b = (C.c_int * len(bits))(*bits)
        rc = load_library().omse_residual_quantize(
            self._h, _ptr(t, torch.float32), n_kernels, kernel_len, b, int(is_signed), C.byref(g), len(bits),
            n_sweeps, _ptr(alpha, torch.float32), _ptr(sse, torch.float32), _ptr(codes, torch.int8),
            _ptr(packed, torch.uint8))
        if rc != OK:
            raise OmseError(rc, "omse_residual_quantize")

    def omse_dual_quantize(self, t, n_kernels, kernel_len, bits1, bits2, is_signed, n_cand1, n_cand2, hi_frac1,
                           hi_frac2, alpha, sse, best_idx=None, codes=None, packed=None):
        g = OmseDualGrid(n_cand1, n_cand2, hi_frac1, hi_frac2)
        rc = load_library().omse_dual_quantize(
            self._h, _ptr(t, torch.float32), n_kernels, kernel_len, bits1, bits2, int(is_signed), C.byref(g),
            _ptr(alpha, torch.float32), _ptr(sse, torch.float32), _ptr(best_idx, torch.int32),
            _ptr(codes, torch.int8), _ptr(packed, torch.uint8))
        if rc != OK:
            raise OmseError(rc, "omse_dual_quantize")

    def omse_select_key_layers(self, layers, tau, mse, is_key=None):
        """layers: sequence of (sse tensor, n_kernels, kernel_len); mse: float64 [n]; is_key: int32 [n]."""
        arr = (OmseLayerError * len(layers))()
        for d, (sse, s, k) in zip(arr, layers):
            d.d_sse, d.n_kernels, d.kernel_len = _ptr(sse, torch.float32), s, k
        rc = load_library().omse_select_key_layers(self._h, arr, len(layers), tau, _ptr(mse, torch.float64),
                                                   _ptr(is_key, torch.int32))
        if rc != OK:
            raise OmseError(rc, "omse_select_key_layers")

    def omse_alg1_quantize(self, t, n_kernels, kernel_len, bits, is_signed, n_cand, hi_frac, refine_iters, n_sweeps,
                           alpha, sse, sse_history=None, codes=None, packed=None):
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        b = (C.c_int * len(bits))(*bits)
        f = (C.c_int * len(bits))(*[int(x) for x in is_signed])
        rc = load_library().omse_alg1_quantize(
            self._h, _ptr(t, torch.float32), n_kernels, kernel_len, b, f, C.byref(g), len(bits), n_sweeps,
            _ptr(alpha, torch.float32), _ptr(sse, torch.float32), _ptr(sse_history, torch.float32),
            _ptr(codes, torch.int8), _ptr(packed, torch.uint8))
        if rc != OK:
            raise OmseError(rc, "omse_alg1_quantize")

    def omse_alg1_quantize_converge(self, t, n_kernels, kernel_len, bits, is_signed, n_cand, hi_frac, refine_iters,
                                    max_sweeps, eps, alpha, sse, sse_history=None, sweeps_done=None, codes=None,
                                    packed=None):
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        b = (C.c_int * len(bits))(*bits)
        f = (C.c_int * len(bits))(*[int(x) for x in is_signed])
        rc = load_library().omse_alg1_quantize_converge(
            self._h, _ptr(t, torch.float32), n_kernels, kernel_len, b, f, C.byref(g), len(bits), max_sweeps, eps,
            _ptr(alpha, torch.float32), _ptr(sse, torch.float32), _ptr(sse_history, torch.float32),
            _ptr(sweeps_done, torch.int32), _ptr(codes, torch.int8), _ptr(packed, torch.uint8))
        if rc != OK:
            raise OmseError(rc, "omse_alg1_quantize_converge")

    def omse_quantize_weights_solver(self, w, n_kernels, kernel_len, bits, is_signed, solver, n_iter, n_cand, hi_frac,
                                     refine_iters, alpha, sse, best_idx=None, codes=None, packed=None):
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        rc = load_library().omse_quantize_weights_solver(
            self._h, _ptr(w, torch.float32), n_kernels, kernel_len, bits, int(is_signed), solver, n_iter, C.byref(g),
            _ptr(alpha, torch.float32), _ptr(sse, torch.float32), _ptr(best_idx, torch.int32),
            _ptr(codes, torch.int8), _ptr(packed, torch.uint8))
        if rc != OK:
            raise OmseError(rc, "omse_quantize_weights_solver")

    def omse_quantize_weights_affine(self, w, n_kernels, kernel_len, bits, n_cand, hi_frac, refine_iters, n_delta,
                                     off_frac, alpha, delta, sse, best_idx=None, codes=None, packed=None):
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        o = OmseOffsetGrid(n_delta, off_frac)
        rc = load_library().omse_quantize_weights_affine(
            self._h, _ptr(w, torch.float32), n_kernels, kernel_len, bits, C.byref(g), C.byref(o),
            _ptr(alpha, torch.float32), _ptr(delta, torch.float32), _ptr(sse, torch.float32),
            _ptr(best_idx, torch.int32), _ptr(codes, torch.int8), _ptr(packed, torch.uint8))
        if rc != OK:
            raise OmseError(rc, "omse_quantize_weights_affine")

    def omse_quantize_key_layers(self, layers, bits, is_signed, n_cand, hi_frac, refine_iters, tau, mse, is_key,
                                 cr=None):
        """layers: sequence of dicts with the keys of omse_quantize_weights_batched plus alpha2, sse2 and
        optionally codes2, packed2 (second tensor, written for key layers only)."""
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        arr = (OmseKeyLayer * len(layers))()
        for d, t in zip(arr, layers):
            d.first.d_w = _ptr(t["w"], torch.float32)
            d.first.n_kernels, d.first.kernel_len = t["n_kernels"], t["kernel_len"]
            d.first.d_alpha = _ptr(t["alpha"], torch.float32)
            d.first.d_sse = _ptr(t["sse"], torch.float32)
            d.first.d_best_idx = _ptr(t.get("best_idx"), torch.int32)
            d.first.d_codes = _ptr(t.get("codes"), torch.int8)
            d.first.d_packed = _ptr(t.get("packed"), torch.uint8)
            d.d_alpha2 = _ptr(t["alpha2"], torch.float32)
            d.d_sse2 = _ptr(t["sse2"], torch.float32)
            d.d_codes2 = _ptr(t.get("codes2"), torch.int8)
            d.d_packed2 = _ptr(t.get("packed2"), torch.uint8)
        rc = load_library().omse_quantize_key_layers(
            self._h, arr, len(layers), bits, int(is_signed), C.byref(g), tau, _ptr(mse, torch.float64),
            _ptr(is_key, torch.int32), _ptr(cr, torch.float64))
        if rc != OK:
            raise OmseError(rc, "omse_quantize_key_layers")

    def omse_quantize_weights_offset(self, w, n_kernels, kernel_len, bits, n_cand, hi_frac, refine_iters, alpha, delta,
                                     sse, best_idx=None, codes=None, packed=None):
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        rc = load_library().omse_quantize_weights_offset(
            self._h, _ptr(w, torch.float32), n_kernels, kernel_len, bits, C.byref(g), _ptr(alpha, torch.float32),
            _ptr(delta, torch.float32), _ptr(sse, torch.float32), _ptr(best_idx, torch.int32),
            _ptr(codes, torch.int8), _ptr(packed, torch.uint8))
        if rc != OK:
            raise OmseError(rc, "omse_quantize_weights_offset")

    def omse_activation_scale_offset(self, x, n, bits, n_cand, hi_frac, refine_iters, alpha, delta, sse,
                                     best_idx=None, sse_curve=None):
        g = OmseGrid(n_cand, hi_frac, refine_iters)
        rc = load_library().omse_activation_scale_offset(
            self._h, _ptr(x, torch.float32), n, bits, C.byref(g), _ptr(alpha, torch.float32),
            _ptr(delta, torch.float32), _ptr(sse, torch.float32), _ptr(best_idx, torch.int32),
            _ptr(sse_curve, torch.float64))
        if rc != OK:
            raise OmseError(rc, "omse_activation_scale_offset")

    def omse_pack_int4(self, codes, n, is_signed, packed):
        rc = load_library().omse_pack_int4(self._h, _ptr(codes, torch.int8), n, int(is_signed), _ptr(packed, torch.uint8))
        if rc != OK:
            raise OmseError(rc, "omse_pack_int4")

    def omse_read_evaluations(self) -> int:
        out = C.c_uint64(0)
        rc = load_library().omse_read_evaluations(self._h, C.byref(out))
        if rc != OK:
            raise OmseError(rc, "omse_read_evaluations")
        return out.value

    def omse_read_launches(self) -> int:
        """Kernels launched by this context's calls since the last read."""
        out = C.c_uint64(0)
        rc = load_library().omse_read_launches(self._h, C.byref(out))
        if rc != OK:
            raise OmseError(rc, "omse_read_launches")
        return out.value

    def omse_measure_fp32_peak(self, target_ms: int = 200) -> float:
        """Measured FP32 lane operations per second of the FMA pipe (packed fma loop on every SM)."""
        out = C.c_double(0.0)
        rc = load_library().omse_measure_fp32_peak(self._h, target_ms, C.byref(out))
        if rc != OK:
            raise OmseError(rc, "omse_measure_fp32_peak")
        return out.value

    def omse_last_device_status(self) -> int:
        out = C.c_uint32(0)
        rc = load_library().omse_last_device_status(self._h, C.byref(out))
        if rc != OK:
            raise OmseError(rc, "omse_last_device_status")
        return out.value
