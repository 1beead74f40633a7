"""Thin ctypes binding of libstwq.so: argument marshalling only.

Every method of `Context` has the name and argument order of the C entry point it calls
(see include/stwq.h). Tensors are torch CUDA tensors used purely as device memory; the
stream is torch's current stream unless one is given. All arithmetic runs in the library's
kernels.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libstwq.so")

ACT_NONE, ACT_GELU_ERF, ACT_GELU_TANH = 0, 1, 2
OUT_F32, OUT_BF16, OUT_INT32 = 0, 1, 2
OPT_GEMM_PATH, OPT_WAIT_LIMIT_MS = 1, 2
OPT_TILE_N, OPT_VARIANT, OPT_KSPLIT = 100, 101, 102
STATIC_MAX_CODES = 4 * 1024 * 1024

_SYMBOLS = ["stwq_create", "stwq_destroy", "stwq_reserve", "stwq_calibrate", "gps_fold", "stwq_quantize",
            "qlinear", "qlinear_q", "stwq_device_status", "stwq_set_option", "stwq_launch_count",
            "stwq_strerror", "stwq_last_cuda_error", "qlinear_static", "dtwq_quantize", "qlinear_dtwq", "qlinear_chain", "qlinear_chain_q", "stwq_quantize_bf16", "stwq_calibrate_asym", "gps_fold_asym",
            "stwq_quantize_asym", "qlinear_asym", "gps_scales", "qlinear_bf16"]

_lib = None


class StwqError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        super().__init__(f"{where}: status {code} ({detail})")


def library_path() -> str:
    return _LIB_PATH


def exported_symbols():
    """Names the header declares; each must resolve in the shared library."""
    return list(_SYMBOLS)


def load_library():
    """dlopen libstwq.so and declare the prototypes. Raises if the library is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise FileNotFoundError(
            f"{_LIB_PATH} not found: build it with `python -m paper_2601_21238_b200.build` "
            "(there is no CPU fallback)")
    L = C.CDLL(_LIB_PATH)
    vp, i32, i64, u32 = C.c_void_p, C.c_int, C.c_int64, C.c_uint32
    L.stwq_create.argtypes = [C.POINTER(vp), i32]
    L.stwq_destroy.argtypes = [vp]
    L.stwq_destroy.restype = None
    L.stwq_reserve.argtypes = [vp, i64, i32, i32]
    L.stwq_calibrate.argtypes = [vp, vp, vp, i64, i32, i32, vp, i32, u32, vp, vp]
    L.gps_fold.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp, vp]
    L.gps_scales.argtypes = [vp, vp, i64, i32, vp, i32, i32, u32, i32, vp, vp, vp]
    L.stwq_quantize.argtypes = [vp, vp, vp, i64, i32, vp, vp, i32, i32, vp, vp]
    L.qlinear.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, vp, i32, vp, vp, i32, i32, i32, vp, vp]
    L.qlinear_bf16.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, vp, i32, vp, vp, i32, i32, i32, vp, vp]
    L.qlinear_q.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, vp, i32, vp, i32, i32, vp, vp]
    L.qlinear_static.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, i32, vp, vp, i32, i32, i32, vp, vp]
    L.stwq_calibrate_asym.argtypes = [vp, vp, vp, i64, i32, i32, vp, i32, u32, vp, vp, vp]
    L.gps_fold_asym.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp, vp, vp, vp]
    L.stwq_quantize_asym.argtypes = [vp, vp, vp, i64, i32, vp, vp, vp, i32, i32, vp, vp, vp]
    L.qlinear_asym.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, vp, vp, vp, vp, i32, vp, vp, i32, i32, i32, vp, vp]
    L.stwq_quantize_bf16.argtypes = [vp, vp, vp, i64, i32, vp, vp, i32, i32, vp, vp]
    L.qlinear_chain.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, vp, i32, vp, vp, i32, i32, vp, vp, i32, vp, vp]
    L.qlinear_chain_q.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, vp, i32, vp, i32, vp, vp, i32, vp, vp]
    L.dtwq_quantize.argtypes = [vp, vp, i64, i32, vp, i32, vp, vp, vp]
    L.qlinear_dtwq.argtypes = [vp, vp, i64, i32, i32, vp, vp, vp, vp, i32, i32, i32, vp, vp]
    L.stwq_device_status.argtypes = [vp, vp]
    L.stwq_set_option.argtypes = [vp, i32, i32]
    L.stwq_launch_count.argtypes = [vp]
    L.stwq_launch_count.restype = i64
    L.stwq_strerror.argtypes = [i32]
    L.stwq_strerror.restype = C.c_char_p
    L.stwq_last_cuda_error.argtypes = [vp]
    for name in _SYMBOLS:
        getattr(L, name)          # raises AttributeError if a declared symbol is not exported
    _lib = L
    return L


def _p(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def qlinear_static(X, pos_ids, Wq, s_w, s_tok, s_ch, bias, bits, act, out_dtype, Y, stream=None):
    """The context-free, allocation-free entry point: same arguments as Context.qlinear, runs on
    the tensors' device (made current for the call), scratch limited to STATIC_MAX_CODES codes."""
    import torch
    L = load_library()
    M, K = X.shape
    N = Wq.shape[0]
    with torch.cuda.device(X.device):
        if stream is None:
            stream = torch.cuda.current_stream(X.device)
        rc = L.qlinear_static(_p(X), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok), s_tok.numel(),
                              _p(s_ch), _p(bias), bits, act, out_dtype, _p(Y), C.c_void_p(stream.cuda_stream))
    if rc != 0:
        raise StwqError(rc, "qlinear_static", L.stwq_strerror(rc).decode())


class Context:
    """Owns one stwq_ctx on one CUDA device."""

    def __init__(self, device: int = 0):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2601_21238_b200 needs a CUDA device (sm_100); there is no CPU path")
        self._torch = torch
        self._L = load_library()
        self.device = device
        h = C.c_void_p()
        self._check(self._L.stwq_create(C.byref(h), device), "stwq_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            self._L.stwq_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, where: str):
        if rc != 0:
            raise StwqError(rc, where, self._L.stwq_strerror(rc).decode())

    def _stream(self, stream):
        if stream is None:
            stream = self._torch.cuda.current_stream(self.device)
        return C.c_void_p(stream.cuda_stream)

    # ---- one method per C entry point, same name, same argument order -------------------
    def stwq_reserve(self, M, K, P):
        self._check(self._L.stwq_reserve(self._h, M, K, P), "stwq_reserve")

    def stwq_set_option(self, option, value):
        self._check(self._L.stwq_set_option(self._h, option, value), "stwq_set_option")

    def stwq_calibrate(self, Xcal, pos_ids, P, s_ch, bits, pct_ppm, s_tok, stream=None):
        rows, K = Xcal.shape
        self._check(self._L.stwq_calibrate(self._h, _p(Xcal), _p(pos_ids), rows, K, P, _p(s_ch), bits,
                                           pct_ppm, _p(s_tok), self._stream(stream)), "stwq_calibrate")

    def gps_scales(self, Xcal, W, bits, pct_ppm, variant, s_ch, k_star=None, stream=None):
        rows, K = Xcal.shape
        N = W.shape[0]
        self._check(self._L.gps_scales(self._h, _p(Xcal), rows, K, _p(W), N, bits, pct_ppm, variant, _p(s_ch),
                                       _p(k_star), self._stream(stream)), "gps_scales")

    def gps_fold(self, W, s_ch, bits, Wq, s_w, stream=None):
        N, K = W.shape
        self._check(self._L.gps_fold(self._h, _p(W), N, K, _p(s_ch), bits, _p(Wq), _p(s_w),
                                     self._stream(stream)), "gps_fold")

    def stwq_quantize(self, X, pos_ids, s_ch, s_tok, bits, Xq, stream=None):
        M, K = X.shape
        self._check(self._L.stwq_quantize(self._h, _p(X), _p(pos_ids), M, K, _p(s_ch), _p(s_tok),
                                          s_tok.numel(), bits, _p(Xq), self._stream(stream)),
                    "stwq_quantize")

    def stwq_quantize_bf16(self, X, pos_ids, s_ch, s_tok, bits, Xq, stream=None):
        M, K = X.shape
        self._check(self._L.stwq_quantize_bf16(self._h, _p(X), _p(pos_ids), M, K, _p(s_ch), _p(s_tok),
                                               s_tok.numel(), bits, _p(Xq), self._stream(stream)),
                    "stwq_quantize_bf16")

    def qlinear(self, X, pos_ids, Wq, s_w, s_tok, s_ch, bias, bits, act, out_dtype, Y, stream=None):
        M, K = X.shape
        N = Wq.shape[0]
        self._check(self._L.qlinear(self._h, _p(X), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok),
                                    s_tok.numel(), _p(s_ch), _p(bias), bits, act, out_dtype, _p(Y),
                                    self._stream(stream)), "qlinear")

    def qlinear_bf16(self, X, pos_ids, Wq, s_w, s_tok, s_ch, bias, bits, act, out_dtype, Y, stream=None):
        M, K = X.shape
        N = Wq.shape[0]
        self._check(self._L.qlinear_bf16(self._h, _p(X), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok),
                                    s_tok.numel(), _p(s_ch), _p(bias), bits, act, out_dtype, _p(Y),
                                    self._stream(stream)), "qlinear_bf16")

    def qlinear_q(self, Xq, pos_ids, Wq, s_w, s_tok, bias, act, out_dtype, Y, stream=None):
        M, K = Xq.shape
        N = Wq.shape[0]
        P = s_tok.numel() if s_tok is not None else 1
        self._check(self._L.qlinear_q(self._h, _p(Xq), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok),
                                      P, _p(bias), act, out_dtype, _p(Y), self._stream(stream)),
                    "qlinear_q")

    def qlinear_chain(self, X, pos_ids, Wq, s_w, s_tok, s_ch, bias, bits, act, s_ch_next, s_tok_next, bits_next,
                      Xq_next, stream=None):
        M, K = X.shape
        N = Wq.shape[0]
        self._check(self._L.qlinear_chain(self._h, _p(X), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok),
                                          s_tok.numel(), _p(s_ch), _p(bias), bits, act, _p(s_ch_next),
                                          _p(s_tok_next), bits_next, _p(Xq_next), self._stream(stream)),
                    "qlinear_chain")

    def qlinear_chain_q(self, Xq, pos_ids, Wq, s_w, s_tok, bias, act, s_ch_next, s_tok_next, bits_next, Xq_next,
                        stream=None):
        M, K = Xq.shape
        N = Wq.shape[0]
        self._check(self._L.qlinear_chain_q(self._h, _p(Xq), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok),
                                            s_tok.numel(), _p(bias), act, _p(s_ch_next), _p(s_tok_next),
                                            bits_next, _p(Xq_next), self._stream(stream)), "qlinear_chain_q")

    def stwq_calibrate_asym(self, Xcal, pos_ids, P, s_ch, bits, pct_ppm, s_tok, z_tok, stream=None):
        rows, K = Xcal.shape
        self._check(self._L.stwq_calibrate_asym(self._h, _p(Xcal), _p(pos_ids), rows, K, P, _p(s_ch), bits, pct_ppm,
                                                _p(s_tok), _p(z_tok), self._stream(stream)), "stwq_calibrate_asym")

    def gps_fold_asym(self, W, s_ch, bits, Wq, s_w, z_w, colsum, stream=None):
        N, K = W.shape
        self._check(self._L.gps_fold_asym(self._h, _p(W), N, K, _p(s_ch), bits, _p(Wq), _p(s_w), _p(z_w), _p(colsum),
                                          self._stream(stream)), "gps_fold_asym")

    def stwq_quantize_asym(self, X, pos_ids, s_ch, s_tok, z_tok, bits, Xq, rowcorr, stream=None):
        M, K = X.shape
        self._check(self._L.stwq_quantize_asym(self._h, _p(X), _p(pos_ids), M, K, _p(s_ch), _p(s_tok), _p(z_tok),
                                               s_tok.numel(), bits, _p(Xq), _p(rowcorr), self._stream(stream)),
                    "stwq_quantize_asym")

    def qlinear_asym(self, X, pos_ids, Wq, s_w, z_w, colsum, s_tok, z_tok, s_ch, bias, bits, act, out_dtype, Y,
                     stream=None):
        M, K = X.shape
        N = Wq.shape[0]
        self._check(self._L.qlinear_asym(self._h, _p(X), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(z_w), _p(colsum),
                                         _p(s_tok), _p(z_tok), s_tok.numel(), _p(s_ch), _p(bias), bits, act, out_dtype,
                                         _p(Y), self._stream(stream)), "qlinear_asym")

    def dtwq_quantize(self, X, s_ch, bits, Xq, s_row, stream=None):
        M, K = X.shape
        self._check(self._L.dtwq_quantize(self._h, _p(X), M, K, _p(s_ch), bits, _p(Xq), _p(s_row),
                                          self._stream(stream)), "dtwq_quantize")

    def qlinear_dtwq(self, X, Wq, s_w, s_ch, bias, bits, act, out_dtype, Y, stream=None):
        M, K = X.shape
        N = Wq.shape[0]
        self._check(self._L.qlinear_dtwq(self._h, _p(X), M, K, N, _p(Wq), _p(s_w), _p(s_ch), _p(bias), bits, act,
                                         out_dtype, _p(Y), self._stream(stream)), "qlinear_dtwq")

    def stwq_device_status(self, stream=None) -> int:
        return int(self._L.stwq_device_status(self._h, self._stream(stream)))

    def check_device_status(self, stream=None):
        self._check(self.stwq_device_status(stream), "device status")

    def stwq_launch_count(self) -> int:
        return int(self._L.stwq_launch_count(self._h))

    # ---- raw access for tests that pass hand-made pointers / sizes ----------------------
    @property
    def handle(self):
        return self._h

    @property
    def lib(self):
        return self._L
