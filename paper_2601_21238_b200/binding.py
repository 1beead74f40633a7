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

ACT_NONE, ACT_GELU_ERF, ACT_GELU_TANH, ACT_GELU_FAST = 0, 1, 2, 3
OUT_F32, OUT_BF16, OUT_INT32 = 0, 1, 2
OPT_GEMM_PATH, OPT_WAIT_LIMIT_MS = 1, 2
OPT_TILE_N, OPT_VARIANT, OPT_KSPLIT = 100, 101, 102
STATIC_MAX_CODES = 4 * 1024 * 1024

_SYMBOLS = ["stwq_create", "stwq_destroy", "stwq_reserve", "stwq_calibrate", "gps_fold", "stwq_quantize",
            "qlinear", "qlinear_q", "stwq_device_status", "stwq_set_option", "stwq_launch_count",
            "stwq_strerror", "stwq_last_cuda_error", "qlinear_static", "dtwq_quantize", "qlinear_dtwq", "qlinear_chain", "qlinear_chain_q", "stwq_quantize_bf16", "stwq_calibrate_asym", "gps_fold_asym",
            "stwq_quantize_asym", "qlinear_asym", "gps_scales", "qlinear_bf16", "stwq_reserve_layer",
            "stwq_workspace_generation", "stwq_selftest_wait_expiry", "stwq_probe_int8_peak", "gps_fold_packed4", "stwq_unpack4",
            "qlinear_w4", "kv_append", "qattention", "stwq_reserve_attention", "qattn_softmax_quantize", "qattn_pv",
            "dgc_select"]

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
    L.stwq_reserve_layer.argtypes = [vp, i64, i32, i32, i32]
    L.stwq_workspace_generation.argtypes = [vp]
    L.stwq_workspace_generation.restype = C.c_uint64
    L.stwq_selftest_wait_expiry.argtypes = [vp, vp, vp]
    L.stwq_probe_int8_peak.argtypes = [vp, i32, i32, C.POINTER(i64), vp]
    L.stwq_calibrate.argtypes = [vp, vp, vp, i64, i32, i32, vp, i32, u32, vp, vp]
    L.gps_fold.argtypes = [vp, vp, i32, i32, vp, i32, vp, vp, vp]
    L.gps_fold_packed4.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    L.stwq_unpack4.argtypes = [vp, vp, i32, i32, vp, vp]
    L.qlinear_w4.argtypes = [vp, vp, vp, i64, i32, i32, vp, vp, vp, i32, vp, vp, i32, i32, i32, vp, vp]
    L.kv_append.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, i32, i32, vp, vp, vp]
    L.qattention.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, vp, vp, i32, i32, i32, i32, vp, vp]
    L.stwq_reserve_attention.argtypes = [vp, i32, i32, i32, i32]
    L.qattn_softmax_quantize.argtypes = [vp, vp, i64, i32, i32, i32, i32, i32, vp, vp]
    L.qattn_pv.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, i32, vp, vp]
    L.dgc_select.argtypes = [vp, vp, i32, i32, u32, C.c_double, vp, vp, vp]
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


ERR_NULL, ERR_DIM, ERR_ALIGN, ERR_BITS, ERR_CUDA = -1, -2, -3, -4, -6
_F32, _BF16, _I8, _I32, _U8 = "torch.float32", "torch.bfloat16", "torch.int8", "torch.int32", "torch.uint8"
_OUT_DTYPES = {OUT_F32: _F32, OUT_BF16: _BF16, OUT_INT32: _I32}


def check_args(where, device, *specs):
    """Host-side check of the tensors handed to one C call, before any pointer is taken: every
    tensor must be a dense (contiguous) CUDA tensor on `device` with the element type and the exact
    shape the call's sizes imply. A spec is (name, tensor, dtype string, shape tuple, optional).
    The C library sees only raw addresses and sizes; a transposed view, a wrong dtype or a short
    vector would make a kernel read or write out of bounds. Raises StwqError; computes nothing."""
    for name, t, dtype, shape, optional in specs:
        if t is None:
            if optional:
                continue
            raise StwqError(ERR_NULL, where, f"{name} is None")
        if not getattr(t, "is_cuda", False):
            raise StwqError(ERR_CUDA, where, f"{name} is not a CUDA tensor")
        idx = t.device.index
        if device is not None and idx is not None and idx != device:
            raise StwqError(ERR_CUDA, where, f"{name} lives on cuda:{idx}, the call runs on cuda:{device}")
        if str(t.dtype) != dtype:
            raise StwqError(ERR_BITS, where, f"{name} has dtype {t.dtype}, expected {dtype}")
        if tuple(t.shape) != tuple(shape):
            raise StwqError(ERR_DIM, where, f"{name} has shape {tuple(t.shape)}, expected {tuple(shape)}")
        if not t.is_contiguous():
            raise StwqError(ERR_ALIGN, where, f"{name} is not contiguous (row-major dense storage is required)")


def _mk(X, what="X"):
    if X is None or len(X.shape) != 2:
        raise StwqError(ERR_DIM, what, "a 2-D tensor is required")
    return int(X.shape[0]), int(X.shape[1])


def _out_dtype(where, out_dtype):
    if out_dtype not in _OUT_DTYPES:
        raise StwqError(ERR_BITS, where, f"out_dtype {out_dtype} is not OUT_F32 / OUT_BF16 / OUT_INT32")
    return _OUT_DTYPES[out_dtype]


def _layer_specs(where, X, x_dtype, pos_ids, Wq, s_w, s_tok, s_ch, bias, out_dtype, Y, need_scales=True):
    """The tensors of a qlinear-shaped call: X [M,K], pos_ids [M], Wq [N,K], s_w [N], s_tok [P],
    s_ch [K] or None, bias [N] or None, Y [M,N] of the type out_dtype names."""
    M, K = _mk(X)
    N, _ = _mk(Wq, "Wq")
    P = int(s_tok.numel()) if s_tok is not None else 1
    ydt = _out_dtype(where, out_dtype)
    return M, K, N, P, [("X", X, x_dtype, (M, K), False), ("pos_ids", pos_ids, _I32, (M,), not need_scales),
                        ("Wq", Wq, _I8, (N, K), False), ("s_w", s_w, _F32, (N,), not need_scales),
                        ("s_tok", s_tok, _F32, (P,), not need_scales), ("s_ch", s_ch, _F32, (K,), True),
                        ("bias", bias, _F32, (N,), True), ("Y", Y, ydt, (M, N), False)]


def qlinear_static(X, pos_ids, Wq, s_w, s_tok, s_ch, bias, bits, act, out_dtype, Y, stream=None):
    """The context-free, allocation-free entry point: same arguments as Context.qlinear, runs on
    the tensors' device (made current for the call), scratch limited to STATIC_MAX_CODES codes."""
    import torch
    L = load_library()
    M, K, N, P, specs = _layer_specs("qlinear_static", X, _F32, pos_ids, Wq, s_w, s_tok, s_ch, bias, out_dtype, Y)
    check_args("qlinear_static", X.device.index if getattr(X, "is_cuda", False) else None, *specs)
    with torch.cuda.device(X.device):
        if stream is None:
            stream = torch.cuda.current_stream(X.device)
        rc = L.qlinear_static(_p(X), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok), P,
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

    def _args(self, where, *specs):
        check_args(where, self.device, *specs)

    # ---- one method per C entry point, same name, same argument order -------------------
    def stwq_reserve(self, M, K, P):
        self._check(self._L.stwq_reserve(self._h, M, K, P), "stwq_reserve")

    def stwq_reserve_layer(self, M, K, N, P):
        self._check(self._L.stwq_reserve_layer(self._h, M, K, N, P), "stwq_reserve_layer")

    def stwq_workspace_generation(self) -> int:
        return int(self._L.stwq_workspace_generation(self._h))

    def stwq_set_option(self, option, value):
        self._check(self._L.stwq_set_option(self._h, option, value), "stwq_set_option")

    def stwq_calibrate(self, Xcal, pos_ids, P, s_ch, bits, pct_ppm, s_tok, stream=None):
        rows, K = _mk(Xcal, "Xcal")
        self._args("stwq_calibrate", ("Xcal", Xcal, _F32, (rows, K), False), ("pos_ids", pos_ids, _I32, (rows,), False),
                   ("s_ch", s_ch, _F32, (K,), True), ("s_tok", s_tok, _F32, (P,), False))
        self._check(self._L.stwq_calibrate(self._h, _p(Xcal), _p(pos_ids), rows, K, P, _p(s_ch), bits,
                                           pct_ppm, _p(s_tok), self._stream(stream)), "stwq_calibrate")

    def gps_scales(self, Xcal, W, bits, pct_ppm, variant, s_ch, k_star=None, stream=None):
        rows, K = _mk(Xcal, "Xcal")
        N, _ = _mk(W, "W")
        self._args("gps_scales", ("Xcal", Xcal, _F32, (rows, K), False), ("W", W, _F32, (N, K), False),
                   ("s_ch", s_ch, _F32, (K,), False), ("k_star", k_star, _I32, (1,), True))
        self._check(self._L.gps_scales(self._h, _p(Xcal), rows, K, _p(W), N, bits, pct_ppm, variant, _p(s_ch),
                                       _p(k_star), self._stream(stream)), "gps_scales")

    def gps_fold(self, W, s_ch, bits, Wq, s_w, stream=None):
        N, K = _mk(W, "W")
        self._args("gps_fold", ("W", W, _F32, (N, K), False), ("s_ch", s_ch, _F32, (K,), True),
                   ("Wq", Wq, _I8, (N, K), False), ("s_w", s_w, _F32, (N,), False))
        self._check(self._L.gps_fold(self._h, _p(W), N, K, _p(s_ch), bits, _p(Wq), _p(s_w),
                                     self._stream(stream)), "gps_fold")

    def dgc_select(self, F, keep_ppm, ridge, rho, selected=None, stream=None):
        n, D = _mk(F, "F")
        k = min(n, max(1, (keep_ppm * n + 999999) // 1000000))
        self._args("dgc_select", ("F", F, _F32, (n, D), False), ("rho", rho, "torch.float64", (n,), False),
                   ("selected", selected, _I32, (k,), True))
        self._check(self._L.dgc_select(self._h, _p(F), n, D, keep_ppm, float(ridge), _p(rho), _p(selected),
                                       self._stream(stream)), "dgc_select")

    def gps_fold_packed4(self, W, s_ch, Wp, s_w, stream=None):
        N, K = _mk(W, "W")
        self._args("gps_fold_packed4", ("W", W, _F32, (N, K), False), ("s_ch", s_ch, _F32, (K,), True),
                   ("Wp", Wp, _U8, (N, K // 2), False), ("s_w", s_w, _F32, (N,), False))
        self._check(self._L.gps_fold_packed4(self._h, _p(W), N, K, _p(s_ch), _p(Wp), _p(s_w), self._stream(stream)),
                    "gps_fold_packed4")

    def stwq_unpack4(self, Wp, Wq, stream=None):
        N, K = _mk(Wq, "Wq")
        self._args("stwq_unpack4", ("Wp", Wp, _U8, (N, K // 2), False), ("Wq", Wq, _I8, (N, K), False))
        self._check(self._L.stwq_unpack4(self._h, _p(Wp), N, K, _p(Wq), self._stream(stream)), "stwq_unpack4")

    def qlinear_w4(self, X, pos_ids, Wp, s_w, s_tok, s_ch, bias, bits, act, out_dtype, Y, stream=None):
        M, K = _mk(X)
        N, _ = _mk(Wp, "Wp")
        P = int(s_tok.numel()) if s_tok is not None else 1
        self._args("qlinear_w4", ("X", X, _F32, (M, K), False), ("pos_ids", pos_ids, _I32, (M,), False),
                   ("Wp", Wp, _U8, (N, K // 2), False), ("s_w", s_w, _F32, (N,), False), ("s_tok", s_tok, _F32, (P,), False),
                   ("s_ch", s_ch, _F32, (K,), True), ("bias", bias, _F32, (N,), True),
                   ("Y", Y, _out_dtype("qlinear_w4", out_dtype), (M, N), False))
        self._check(self._L.qlinear_w4(self._h, _p(X), _p(pos_ids), M, K, N, _p(Wp), _p(s_w), _p(s_tok), P, _p(s_ch),
                                       _p(bias), bits, act, out_dtype, _p(Y), self._stream(stream)), "qlinear_w4")

    def kv_append(self, Knew, Vnew, pos0, s_k, s_v, bits, Kc, Vt, stream=None):
        G, t_new, d = (int(v) for v in Knew.shape)
        Tmax = int(Kc.shape[1])
        P = int(s_k.numel())
        self._args("kv_append", ("Knew", Knew, _F32, (G, t_new, d), False), ("Vnew", Vnew, _F32, (G, t_new, d), False),
                   ("s_k", s_k, _F32, (P,), False), ("s_v", s_v, _F32, (d,), False), ("Kc", Kc, _I8, (G, Tmax, d), False),
                   ("Vt", Vt, _I8, (G, d, Tmax), False))
        self._check(self._L.kv_append(self._h, _p(Knew), _p(Vnew), G, t_new, d, pos0, Tmax, _p(s_k), _p(s_v), P, bits,
                                      _p(Kc), _p(Vt), self._stream(stream)), "kv_append")

    def qattention(self, Q, pos_q, Tk, Kc, Vt, s_q, s_kcol, s_v, bits, causal, out_dtype, O, stream=None):
        G, Tq, d = (int(v) for v in Q.shape)
        Tmax = int(Kc.shape[1])
        P = int(s_q.numel())
        self._args("qattention", ("Q", Q, _F32, (G, Tq, d), False), ("pos_q", pos_q, _I32, (Tq,), False),
                   ("Kc", Kc, _I8, (G, Tmax, d), False), ("Vt", Vt, _I8, (G, d, Tmax), False), ("s_q", s_q, _F32, (P,), False),
                   ("s_kcol", s_kcol, _F32, (Tk,), False), ("s_v", s_v, _F32, (d,), False),
                   ("O", O, _out_dtype("qattention", out_dtype), (G, Tq, d), False))
        self._check(self._L.qattention(self._h, _p(Q), _p(pos_q), G, Tq, Tk, d, Tmax, _p(Kc), _p(Vt), _p(s_q), _p(s_kcol),
                                       _p(s_v), P, bits, int(bool(causal)), out_dtype, _p(O), self._stream(stream)),
                    "qattention")

    def stwq_reserve_attention(self, G, Tq, Tk, d):
        self._check(self._L.stwq_reserve_attention(self._h, G, Tq, Tk, d), "stwq_reserve_attention")

    def qattn_softmax_quantize(self, S, Tq, Tk, causal, bits, Pq, stream=None):
        rows, ld = _mk(S, "S")
        self._args("qattn_softmax_quantize", ("S", S, _F32, (rows, ld), False), ("Pq", Pq, _U8, (rows, ld), False))
        self._check(self._L.qattn_softmax_quantize(self._h, _p(S), rows, Tq, Tk, ld, int(bool(causal)), bits, _p(Pq),
                                                   self._stream(stream)), "qattn_softmax_quantize")

    def qattn_pv(self, Pq, Vt, s_v, delta_p, out_dtype, O, stream=None):
        G, Tq, Tk_pad = (int(v) for v in Pq.shape)
        d, Tmax = int(Vt.shape[1]), int(Vt.shape[2])
        self._args("qattn_pv", ("Pq", Pq, _U8, (G, Tq, Tk_pad), False), ("Vt", Vt, _I8, (G, d, Tmax), False),
                   ("s_v", s_v, _F32, (d,), out_dtype == OUT_INT32), ("delta_p", delta_p, _F32, (1,), out_dtype == OUT_INT32),
                   ("O", O, _out_dtype("qattn_pv", out_dtype), (G, Tq, d), False))
        self._check(self._L.qattn_pv(self._h, _p(Pq), G, Tq, Tk_pad, d, Tmax, _p(Vt), _p(s_v), _p(delta_p), out_dtype,
                                     _p(O), self._stream(stream)), "qattn_pv")

    def _quantize_specs(self, X, x_dtype, pos_ids, s_ch, s_tok, Xq):
        M, K = _mk(X)
        P = int(s_tok.numel()) if s_tok is not None else 1
        return M, K, P, [("X", X, x_dtype, (M, K), False), ("pos_ids", pos_ids, _I32, (M,), False),
                         ("s_ch", s_ch, _F32, (K,), True), ("s_tok", s_tok, _F32, (P,), False),
                         ("Xq", Xq, _I8, (M, K), False)]

    def stwq_quantize(self, X, pos_ids, s_ch, s_tok, bits, Xq, stream=None):
        M, K, P, specs = self._quantize_specs(X, _F32, pos_ids, s_ch, s_tok, Xq)
        self._args("stwq_quantize", *specs)
        self._check(self._L.stwq_quantize(self._h, _p(X), _p(pos_ids), M, K, _p(s_ch), _p(s_tok),
                                          P, bits, _p(Xq), self._stream(stream)), "stwq_quantize")

    def stwq_quantize_bf16(self, X, pos_ids, s_ch, s_tok, bits, Xq, stream=None):
        M, K, P, specs = self._quantize_specs(X, _BF16, pos_ids, s_ch, s_tok, Xq)
        self._args("stwq_quantize_bf16", *specs)
        self._check(self._L.stwq_quantize_bf16(self._h, _p(X), _p(pos_ids), M, K, _p(s_ch), _p(s_tok),
                                               P, bits, _p(Xq), self._stream(stream)), "stwq_quantize_bf16")

    def qlinear(self, X, pos_ids, Wq, s_w, s_tok, s_ch, bias, bits, act, out_dtype, Y, stream=None):
        M, K, N, P, specs = _layer_specs("qlinear", X, _F32, pos_ids, Wq, s_w, s_tok, s_ch, bias, out_dtype, Y)
        self._args("qlinear", *specs)
        self._check(self._L.qlinear(self._h, _p(X), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok),
                                    P, _p(s_ch), _p(bias), bits, act, out_dtype, _p(Y),
                                    self._stream(stream)), "qlinear")

    def qlinear_bf16(self, X, pos_ids, Wq, s_w, s_tok, s_ch, bias, bits, act, out_dtype, Y, stream=None):
        M, K, N, P, specs = _layer_specs("qlinear_bf16", X, _BF16, pos_ids, Wq, s_w, s_tok, s_ch, bias, out_dtype, Y)
        self._args("qlinear_bf16", *specs)
        self._check(self._L.qlinear_bf16(self._h, _p(X), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok),
                                         P, _p(s_ch), _p(bias), bits, act, out_dtype, _p(Y),
                                         self._stream(stream)), "qlinear_bf16")

    def qlinear_q(self, Xq, pos_ids, Wq, s_w, s_tok, bias, act, out_dtype, Y, stream=None):
        # raw accumulators (OUT_INT32) need no scales or positions
        M, K, N, P, specs = _layer_specs("qlinear_q", Xq, _I8, pos_ids, Wq, s_w, s_tok, None, bias, out_dtype, Y,
                                         need_scales=out_dtype != OUT_INT32)
        self._args("qlinear_q", *specs)
        self._check(self._L.qlinear_q(self._h, _p(Xq), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok),
                                      P, _p(bias), act, out_dtype, _p(Y), self._stream(stream)),
                    "qlinear_q")

    def _chain_specs(self, where, X, x_dtype, pos_ids, Wq, s_w, s_tok, s_ch, bias, s_ch_next, s_tok_next, Xq_next):
        M, K = _mk(X)
        N, _ = _mk(Wq, "Wq")
        P = int(s_tok.numel()) if s_tok is not None else 1
        return M, K, N, P, [("X", X, x_dtype, (M, K), False), ("pos_ids", pos_ids, _I32, (M,), False),
                            ("Wq", Wq, _I8, (N, K), False), ("s_w", s_w, _F32, (N,), False),
                            ("s_tok", s_tok, _F32, (P,), False), ("s_ch", s_ch, _F32, (K,), True),
                            ("bias", bias, _F32, (N,), True), ("s_ch_next", s_ch_next, _F32, (N,), True),
                            ("s_tok_next", s_tok_next, _F32, (P,), False), ("Xq_next", Xq_next, _I8, (M, N), False)]

    def qlinear_chain(self, X, pos_ids, Wq, s_w, s_tok, s_ch, bias, bits, act, s_ch_next, s_tok_next, bits_next,
                      Xq_next, stream=None):
        M, K, N, P, specs = self._chain_specs("qlinear_chain", X, _F32, pos_ids, Wq, s_w, s_tok, s_ch, bias, s_ch_next,
                                              s_tok_next, Xq_next)
        self._args("qlinear_chain", *specs)
        self._check(self._L.qlinear_chain(self._h, _p(X), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok),
                                          P, _p(s_ch), _p(bias), bits, act, _p(s_ch_next),
                                          _p(s_tok_next), bits_next, _p(Xq_next), self._stream(stream)),
                    "qlinear_chain")

    def qlinear_chain_q(self, Xq, pos_ids, Wq, s_w, s_tok, bias, act, s_ch_next, s_tok_next, bits_next, Xq_next,
                        stream=None):
        M, K, N, P, specs = self._chain_specs("qlinear_chain_q", Xq, _I8, pos_ids, Wq, s_w, s_tok, None, bias,
                                              s_ch_next, s_tok_next, Xq_next)
        self._args("qlinear_chain_q", *specs)
        self._check(self._L.qlinear_chain_q(self._h, _p(Xq), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(s_tok),
                                            P, _p(bias), act, _p(s_ch_next), _p(s_tok_next),
                                            bits_next, _p(Xq_next), self._stream(stream)), "qlinear_chain_q")

    def stwq_calibrate_asym(self, Xcal, pos_ids, P, s_ch, bits, pct_ppm, s_tok, z_tok, stream=None):
        rows, K = _mk(Xcal, "Xcal")
        self._args("stwq_calibrate_asym", ("Xcal", Xcal, _F32, (rows, K), False),
                   ("pos_ids", pos_ids, _I32, (rows,), False), ("s_ch", s_ch, _F32, (K,), True),
                   ("s_tok", s_tok, _F32, (P,), False), ("z_tok", z_tok, _I32, (P,), False))
        self._check(self._L.stwq_calibrate_asym(self._h, _p(Xcal), _p(pos_ids), rows, K, P, _p(s_ch), bits, pct_ppm,
                                                _p(s_tok), _p(z_tok), self._stream(stream)), "stwq_calibrate_asym")

    def gps_fold_asym(self, W, s_ch, bits, Wq, s_w, z_w, colsum, stream=None):
        N, K = _mk(W, "W")
        self._args("gps_fold_asym", ("W", W, _F32, (N, K), False), ("s_ch", s_ch, _F32, (K,), True),
                   ("Wq", Wq, _I8, (N, K), False), ("s_w", s_w, _F32, (N,), False), ("z_w", z_w, _I32, (N,), False),
                   ("colsum", colsum, _I32, (N,), False))
        self._check(self._L.gps_fold_asym(self._h, _p(W), N, K, _p(s_ch), bits, _p(Wq), _p(s_w), _p(z_w), _p(colsum),
                                          self._stream(stream)), "gps_fold_asym")

    def stwq_quantize_asym(self, X, pos_ids, s_ch, s_tok, z_tok, bits, Xq, rowcorr, stream=None):
        M, K, P, specs = self._quantize_specs(X, _F32, pos_ids, s_ch, s_tok, Xq)
        self._args("stwq_quantize_asym", *specs, ("z_tok", z_tok, _I32, (P,), False),
                   ("rowcorr", rowcorr, _I32, (M,), False))
        self._check(self._L.stwq_quantize_asym(self._h, _p(X), _p(pos_ids), M, K, _p(s_ch), _p(s_tok), _p(z_tok),
                                               P, bits, _p(Xq), _p(rowcorr), self._stream(stream)),
                    "stwq_quantize_asym")

    def qlinear_asym(self, X, pos_ids, Wq, s_w, z_w, colsum, s_tok, z_tok, s_ch, bias, bits, act, out_dtype, Y,
                     stream=None):
        M, K, N, P, specs = _layer_specs("qlinear_asym", X, _F32, pos_ids, Wq, s_w, s_tok, s_ch, bias, out_dtype, Y)
        self._args("qlinear_asym", *specs, ("z_w", z_w, _I32, (N,), False), ("colsum", colsum, _I32, (N,), False),
                   ("z_tok", z_tok, _I32, (P,), False))
        self._check(self._L.qlinear_asym(self._h, _p(X), _p(pos_ids), M, K, N, _p(Wq), _p(s_w), _p(z_w), _p(colsum),
                                         _p(s_tok), _p(z_tok), P, _p(s_ch), _p(bias), bits, act, out_dtype,
                                         _p(Y), self._stream(stream)), "qlinear_asym")

    def dtwq_quantize(self, X, s_ch, bits, Xq, s_row, stream=None):
        M, K = _mk(X)
        self._args("dtwq_quantize", ("X", X, _F32, (M, K), False), ("s_ch", s_ch, _F32, (K,), True),
                   ("Xq", Xq, _I8, (M, K), False), ("s_row", s_row, _F32, (M,), False))
        self._check(self._L.dtwq_quantize(self._h, _p(X), M, K, _p(s_ch), bits, _p(Xq), _p(s_row),
                                          self._stream(stream)), "dtwq_quantize")

    def qlinear_dtwq(self, X, Wq, s_w, s_ch, bias, bits, act, out_dtype, Y, stream=None):
        M, K = _mk(X)
        N, _ = _mk(Wq, "Wq")
        self._args("qlinear_dtwq", ("X", X, _F32, (M, K), False), ("Wq", Wq, _I8, (N, K), False),
                   ("s_w", s_w, _F32, (N,), False), ("s_ch", s_ch, _F32, (K,), True), ("bias", bias, _F32, (N,), True),
                   ("Y", Y, _out_dtype("qlinear_dtwq", out_dtype), (M, N), False))
        self._check(self._L.qlinear_dtwq(self._h, _p(X), M, K, N, _p(Wq), _p(s_w), _p(s_ch), _p(bias), bits, act,
                                         out_dtype, _p(Y), self._stream(stream)), "qlinear_dtwq")

    def stwq_device_status(self, stream=None) -> int:
        return int(self._L.stwq_device_status(self._h, self._stream(stream)))

    def check_device_status(self, stream=None):
        self._check(self.stwq_device_status(stream), "device status")

    def stwq_selftest_wait_expiry(self, waited_ns=None, stream=None):
        self._args("stwq_selftest_wait_expiry", ("waited_ns", waited_ns, "torch.int64", (1,), True))
        self._check(self._L.stwq_selftest_wait_expiry(self._h, _p(waited_ns), self._stream(stream)),
                    "stwq_selftest_wait_expiry")

    def stwq_probe_int8_peak(self, kblocks, cta_pairs=0, stream=None) -> int:
        """Launch the peak probe; returns the int8 operations the launch performs."""
        ops = C.c_int64(0)
        self._check(self._L.stwq_probe_int8_peak(self._h, kblocks, cta_pairs, C.byref(ops), self._stream(stream)),
                    "stwq_probe_int8_peak")
        return int(ops.value)

    def stwq_launch_count(self) -> int:
        return int(self._L.stwq_launch_count(self._h))

    # ---- raw access for tests that pass hand-made pointers / sizes ----------------------
    @property
    def handle(self):
        return self._h

    @property
    def lib(self):
        return self._L
