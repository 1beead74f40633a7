"""CPU oracle for the STWQ quantized linear layer: ctypes front end to stwq_oracle.c.

TEST INFRASTRUCTURE ONLY. Nothing on the product path imports this package; the
GPU library never calls it and it never imports the GPU library. It is loaded by
the tests, by the smoke check and by the benchmark's CPU-baseline leg.

All arithmetic lives in stwq_oracle.c (one plain C function per step of the
method, each citing the passage of the paper it follows). This module only
compiles that file with gcc and marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "stwq_oracle.c")
_LIB = os.path.join(_HERE, "libstwq_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with strict IEEE semantics (no contraction, no fast-math)."""
    if force or (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-D_GNU_SOURCE", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a, ct):
    return None if a is None else a.ctypes.data_as(C.POINTER(ct))


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            fp, ip, bp, dp = (C.POINTER(C.c_float), C.POINTER(C.c_int32), C.POINTER(C.c_int8),
                              C.POINTER(C.c_double))
            L.orc_num_threads.restype = C.c_int
            L.orc_delta.restype = C.c_float
            L.orc_delta.argtypes = [C.c_float, C.c_int]
            L.orc_eq1_quantize.argtypes = [fp, C.c_int64, C.c_float, C.c_float, C.c_int, ip, fp, ip]
            L.orc_eq1_dequantize.argtypes = [ip, C.c_int64, C.c_float, C.c_int32, fp]
            L.orc_quantize_div.argtypes = [fp, C.c_int64, C.c_float, C.c_int, bp]
            L.orc_gps_fold.argtypes = [fp, C.c_int, C.c_int, fp, C.c_int, bp, fp]
            L.orc_stwq_calibrate.restype = C.c_int
            L.orc_stwq_calibrate.argtypes = [fp, ip, C.c_int64, C.c_int, C.c_int, fp, C.c_int,
                                             C.c_uint32, fp]
            for f in (L.orc_quantize, L.orc_quantize_exact_div):
                f.restype = C.c_int
                f.argtypes = [fp, ip, C.c_int64, C.c_int, fp, fp, C.c_int, C.c_int, bp]
            L.orc_asym_params.argtypes = [C.c_float, C.c_float, C.c_int, fp, ip]
            L.orc_gps_fold_asym.argtypes = [fp, C.c_int, C.c_int, fp, C.c_int, bp, fp, ip, ip]
            L.orc_stwq_calibrate_asym.restype = C.c_int
            L.orc_stwq_calibrate_asym.argtypes = [fp, ip, C.c_int64, C.c_int, C.c_int, fp, C.c_int, C.c_uint32, fp, ip]
            L.orc_quantize_asym.restype = C.c_int
            L.orc_quantize_asym.argtypes = [fp, ip, C.c_int64, C.c_int, fp, fp, ip, C.c_int, C.c_int, bp, ip]
            L.orc_epilogue_asym.restype = C.c_int
            L.orc_epilogue_asym.argtypes = [ip, ip, C.c_int64, C.c_int, fp, ip, C.c_int, fp, ip, ip, ip, fp, C.c_int,
                                            dp, dp, ip]
            L.orc_dtwq_quantize.argtypes = [fp, C.c_int64, C.c_int, fp, C.c_int, bp, fp]
            L.orc_igemm.argtypes = [bp, bp, C.c_int64, C.c_int, C.c_int, ip]
            L.orc_epilogue.restype = C.c_int
            L.orc_epilogue.argtypes = [ip, ip, C.c_int64, C.c_int, fp, C.c_int, fp, fp, C.c_int, dp, dp]
            L.orc_chain_codes.restype = C.c_int
            L.orc_chain_codes.argtypes = [ip, ip, C.c_int64, C.c_int, fp, C.c_int, fp, fp, C.c_int, fp, fp, C.c_int,
                                          bp, fp, fp]
            L.orc_qlinear.restype = C.c_int
            L.orc_qlinear.argtypes = [fp, ip, C.c_int64, C.c_int, C.c_int, bp, fp, fp, C.c_int, fp, fp,
                                      C.c_int, C.c_int, dp, bp, ip, dp]
            L.orc_gps.argtypes = [fp, C.c_int64, C.c_int, fp, C.c_int, C.c_int, C.c_uint32, C.c_int,
                                  fp, ip]
            L.orc_pack4.restype = C.c_int
            L.orc_pack4.argtypes = [bp, C.c_int64, C.POINTER(C.c_uint8)]
            L.orc_unpack4.argtypes = [C.POINTER(C.c_uint8), C.c_int64, bp]
            L.orc_softmax_quantize.argtypes = [fp, C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_uint8), dp]
            L.orc_igemm_u8s8.argtypes = [C.POINTER(C.c_uint8), bp, C.c_int, C.c_int, C.c_int, ip]
            L.orc_dgc_select.restype = C.c_int
            L.orc_dgc_select.argtypes = [fp, C.c_int, C.c_int, C.c_uint32, C.c_double, dp, ip]
            L.orc_gps_gain.restype = C.c_double
            L.orc_gps_gain.argtypes = [C.c_double] * 4
            _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def delta(a: float, bits: int) -> float:
    """Scale of the symmetric b-bit quantizer with range [-a, a] (Eq. 1)."""
    return float(lib().orc_delta(np.float32(a), bits))


def eq1_quantize(x, x_down, x_up, bits):
    """Eq. 1 as printed: unsigned codes, scale and zero point."""
    x = _f32(x).ravel()
    code = np.empty(x.size, np.int32)
    d = C.c_float()
    z = C.c_int32()
    lib().orc_eq1_quantize(_ptr(x, C.c_float), x.size, np.float32(x_down), np.float32(x_up), bits,
                           _ptr(code, C.c_int32), C.byref(d), C.byref(z))
    return code, float(d.value), int(z.value)


def eq1_dequantize(code, delta_, z):
    code = np.ascontiguousarray(code, np.int32).ravel()
    out = np.empty(code.size, np.float32)
    lib().orc_eq1_dequantize(_ptr(code, C.c_int32), code.size, np.float32(delta_), int(z),
                             _ptr(out, C.c_float))
    return out


def quantize_div(x, delta_, bits):
    """Signed codes clamp(round(x / delta)) of the symmetric quantizer."""
    x = _f32(x)
    q = np.empty(x.shape, np.int8)
    lib().orc_quantize_div(_ptr(x, C.c_float), x.size, np.float32(delta_), bits, _ptr(q, C.c_int8))
    return q


def gps_fold(W, s_ch, bits):
    """Eq. 2 weight side + per-output-channel quantization. Returns (Wq int8 [N,K], s_w [N])."""
    W = _f32(W)
    s_ch = _f32(s_ch)
    N, K = W.shape
    Wq = np.empty((N, K), np.int8)
    s_w = np.empty(N, np.float32)
    lib().orc_gps_fold(_ptr(W, C.c_float), N, K, _ptr(s_ch, C.c_float), bits, _ptr(Wq, C.c_int8),
                       _ptr(s_w, C.c_float))
    return Wq, s_w


def stwq_calibrate(X, pos_ids, P, s_ch, bits, pct_ppm):
    """Section 4.2: per-position static scales by nearest-rank percentile. Returns s_tok [P]."""
    X = _f32(X)
    pos_ids = np.ascontiguousarray(pos_ids, np.int32)
    s_ch = _f32(s_ch)
    rows, K = X.shape
    s_tok = np.empty(P, np.float32)
    st = lib().orc_stwq_calibrate(_ptr(X, C.c_float), _ptr(pos_ids, C.c_int32), rows, K, P,
                                  _ptr(s_ch, C.c_float), bits, int(pct_ppm), _ptr(s_tok, C.c_float))
    if st == -1:
        raise ValueError("pos_ids outside [0, P)")
    if st == -2:
        raise ValueError("non-finite calibration value")
    return s_tok


def quantize(X, pos_ids, s_ch, s_tok, bits, exact_div=False):
    """Activation quantization with static per-position scales. Returns Xq int8 [M,K]."""
    X = _f32(X)
    pos_ids = np.ascontiguousarray(pos_ids, np.int32)
    s_ch = _f32(s_ch)
    s_tok = _f32(s_tok)
    M, K = X.shape
    Xq = np.empty((M, K), np.int8)
    f = lib().orc_quantize_exact_div if exact_div else lib().orc_quantize
    st = f(_ptr(X, C.c_float), _ptr(pos_ids, C.c_int32), M, K, _ptr(s_ch, C.c_float),
           _ptr(s_tok, C.c_float), s_tok.size, bits, _ptr(Xq, C.c_int8))
    if st != 0:
        raise ValueError("pos_ids outside [0, P)")
    return Xq


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def asym_params(x_down, x_up, bits):
    """Eq. 1 parameters for the range [x_down, x_up] widened to contain 0: (delta, signed zero point)."""
    d = C.c_float()
    z = C.c_int32()
    lib().orc_asym_params(np.float32(x_down), np.float32(x_up), bits, C.byref(d), C.byref(z))
    return float(d.value), int(z.value)


def gps_fold_asym(W, s_ch, bits):
    """Asymmetric per-output-channel weights. Returns (Wq int8, s_w, z_w int32, colsum int32)."""
    W, s_ch = _f32(W), _f32(s_ch)
    N, K = W.shape
    Wq = np.empty((N, K), np.int8)
    s_w = np.empty(N, np.float32)
    z_w = np.empty(N, np.int32)
    cs = np.empty(N, np.int32)
    lib().orc_gps_fold_asym(_ptr(W, C.c_float), N, K, _ptr(s_ch, C.c_float), bits, _ptr(Wq, C.c_int8),
                            _ptr(s_w, C.c_float), _ptr(z_w, C.c_int32), _ptr(cs, C.c_int32))
    return Wq, s_w, z_w, cs


def stwq_calibrate_asym(X, pos_ids, P, s_ch, bits, pct_ppm):
    """Asymmetric per-position calibration. Returns (s_tok [P], z_tok int32 [P])."""
    X, pos_ids, s_ch = _f32(X), _i32(pos_ids), _f32(s_ch)
    rows, K = X.shape
    s_tok = np.empty(P, np.float32)
    z_tok = np.empty(P, np.int32)
    st = lib().orc_stwq_calibrate_asym(_ptr(X, C.c_float), _ptr(pos_ids, C.c_int32), rows, K, P,
                                       _ptr(s_ch, C.c_float), bits, int(pct_ppm), _ptr(s_tok, C.c_float),
                                       _ptr(z_tok, C.c_int32))
    if st == -1:
        raise ValueError("pos_ids outside [0, P)")
    if st == -2:
        raise ValueError("non-finite calibration value")
    return s_tok, z_tok


def quantize_asym(X, pos_ids, s_ch, s_tok, z_tok, bits):
    """Asymmetric static activation quantization. Returns (Xq int8 [M,K], rowcorr int32 [M])."""
    X, pos_ids, s_ch, s_tok, z_tok = _f32(X), _i32(pos_ids), _f32(s_ch), _f32(s_tok), _i32(z_tok)
    M, K = X.shape
    Xq = np.empty((M, K), np.int8)
    rc = np.empty(M, np.int32)
    st = lib().orc_quantize_asym(_ptr(X, C.c_float), _ptr(pos_ids, C.c_int32), M, K, _ptr(s_ch, C.c_float),
                                 _ptr(s_tok, C.c_float), _ptr(z_tok, C.c_int32), s_tok.size, bits,
                                 _ptr(Xq, C.c_int8), _ptr(rc, C.c_int32))
    if st != 0:
        raise ValueError("pos_ids outside [0, P)")
    return Xq, rc


def epilogue_asym(acc, pos_ids, s_tok, z_tok, s_w, z_w, colsum, rowcorr, bias, act):
    """Zero-point correction, dequantize, bias, activation. Returns dict(Y, mag, acc_corr)."""
    acc, pos_ids = _i32(acc), _i32(pos_ids)
    M, N = acc.shape
    s_tok, s_w, bias = _f32(s_tok), _f32(s_w), _f32(bias)
    z_tok, z_w, colsum, rowcorr = _i32(z_tok), _i32(z_w), _i32(colsum), _i32(rowcorr)
    Y = np.empty((M, N), np.float64)
    mag = np.empty((M, N), np.float64)
    ac = np.empty((M, N), np.int32)
    st = lib().orc_epilogue_asym(_ptr(acc, C.c_int32), _ptr(pos_ids, C.c_int32), M, N, _ptr(s_tok, C.c_float),
                                 _ptr(z_tok, C.c_int32), s_tok.size, _ptr(s_w, C.c_float), _ptr(z_w, C.c_int32),
                                 _ptr(colsum, C.c_int32), _ptr(rowcorr, C.c_int32), _ptr(bias, C.c_float), act,
                                 _ptr(Y, C.c_double), _ptr(mag, C.c_double), _ptr(ac, C.c_int32))
    if st != 0:
        raise ValueError("pos_ids outside [0, P)")
    return {"Y": Y, "mag": mag, "acc": ac}


def qlinear_asym(X, pos_ids, Wq, s_w, z_w, colsum, s_tok, z_tok, s_ch, bias, bits, act=0):
    """The whole asymmetric quantized linear. Returns dict(Y, mag, acc (corrected), Xq, rowcorr)."""
    Xq, rowcorr = quantize_asym(X, pos_ids, s_ch, s_tok, z_tok, bits)
    raw = igemm(Xq, Wq)
    out = epilogue_asym(raw, pos_ids, s_tok, z_tok, s_w, z_w, colsum, rowcorr, bias, act)
    out.update(Xq=Xq, rowcorr=rowcorr, raw=raw)
    return out


def dtwq_quantize(X, s_ch, bits):
    """Dynamic token-wise quantization (per-row min-max at run time). Returns (Xq int8 [M,K], s_row [M])."""
    X = _f32(X)
    s_ch = _f32(s_ch)
    M, K = X.shape
    Xq = np.empty((M, K), np.int8)
    s_row = np.empty(M, np.float32)
    lib().orc_dtwq_quantize(_ptr(X, C.c_float), M, K, _ptr(s_ch, C.c_float), bits, _ptr(Xq, C.c_int8),
                            _ptr(s_row, C.c_float))
    return Xq, s_row


def igemm(Xq, Wq):
    """acc[m,n] = sum_k Xq[m,k] * Wq[n,k] in int32."""
    Xq = np.ascontiguousarray(Xq, np.int8)
    Wq = np.ascontiguousarray(Wq, np.int8)
    M, K = Xq.shape
    N, K2 = Wq.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    lib().orc_igemm(_ptr(Xq, C.c_int8), _ptr(Wq, C.c_int8), M, N, K, _ptr(acc, C.c_int32))
    return acc


def epilogue(acc, pos_ids, s_tok, s_w, bias, act):
    """Dequantize + bias + activation in double. Returns (Y, mag)."""
    acc = np.ascontiguousarray(acc, np.int32)
    pos_ids = np.ascontiguousarray(pos_ids, np.int32)
    s_tok, s_w, bias = _f32(s_tok), _f32(s_w), _f32(bias)
    M, N = acc.shape
    Y = np.empty((M, N), np.float64)
    mag = np.empty((M, N), np.float64)
    st = lib().orc_epilogue(_ptr(acc, C.c_int32), _ptr(pos_ids, C.c_int32), M, N, _ptr(s_tok, C.c_float),
                            s_tok.size, _ptr(s_w, C.c_float), _ptr(bias, C.c_float), act,
                            _ptr(Y, C.c_double), _ptr(mag, C.c_double))
    if st != 0:
        raise ValueError("pos_ids outside [0, P)")
    return Y, mag


def chain_codes(acc, pos_ids, s_tok, s_w, bias, act, s_ch_next, s_tok_next, bits_next):
    """Dequantize + bias + activation in fp32, then the next layer's static quantizer.
    Returns dict(codes int8 [M,N], u float32 (value before rounding), zmag float32)."""
    acc = np.ascontiguousarray(acc, np.int32)
    pos_ids = np.ascontiguousarray(pos_ids, np.int32)
    s_tok, s_w, bias = _f32(s_tok), _f32(s_w), _f32(bias)
    s_ch_next, s_tok_next = _f32(s_ch_next), _f32(s_tok_next)
    M, N = acc.shape
    codes = np.empty((M, N), np.int8)
    u = np.empty((M, N), np.float32)
    zmag = np.empty((M, N), np.float32)
    st = lib().orc_chain_codes(_ptr(acc, C.c_int32), _ptr(pos_ids, C.c_int32), M, N, _ptr(s_tok, C.c_float),
                               s_tok.size, _ptr(s_w, C.c_float), _ptr(bias, C.c_float), act,
                               _ptr(s_ch_next, C.c_float), _ptr(s_tok_next, C.c_float), bits_next,
                               _ptr(codes, C.c_int8), _ptr(u, C.c_float), _ptr(zmag, C.c_float))
    if st != 0:
        raise ValueError("pos_ids outside [0, P)")
    return {"codes": codes, "u": u, "zmag": zmag}


def qlinear(X, pos_ids, Wq, s_w, s_tok, s_ch, bias, bits, act=0):
    """The whole quantized linear. Returns dict(Y float64, Xq int8, acc int32, mag float64, act)."""
    X = _f32(X)
    pos_ids = np.ascontiguousarray(pos_ids, np.int32)
    Wq = np.ascontiguousarray(Wq, np.int8)
    s_w, s_tok, s_ch, bias = _f32(s_w), _f32(s_tok), _f32(s_ch), _f32(bias)
    M, K = X.shape
    N = Wq.shape[0]
    assert Wq.shape[1] == K
    Y = np.empty((M, N), np.float64)
    mag = np.empty((M, N), np.float64)
    Xq = np.empty((M, K), np.int8)
    acc = np.empty((M, N), np.int32)
    st = lib().orc_qlinear(_ptr(X, C.c_float), _ptr(pos_ids, C.c_int32), M, K, N, _ptr(Wq, C.c_int8),
                           _ptr(s_w, C.c_float), _ptr(s_tok, C.c_float), s_tok.size,
                           _ptr(s_ch, C.c_float), _ptr(bias, C.c_float), bits, act,
                           _ptr(Y, C.c_double), _ptr(Xq, C.c_int8), _ptr(acc, C.c_int32),
                           _ptr(mag, C.c_double))
    if st != 0:
        raise ValueError("pos_ids outside [0, P)")
    return {"Y": Y, "Xq": Xq, "acc": acc, "mag": mag, "act": act}


def gps(X, W, bits, pct_ppm=999900, variant=0):
    """Algorithm 1. X [T,K] calibration rows, W [N,K]. Returns (s [K] float32, k_star)."""
    X = _f32(X)
    W = _f32(W)
    T, K = X.shape
    N = W.shape[0]
    assert W.shape[1] == K
    s = np.empty(K, np.float32)
    ks = C.c_int32()
    lib().orc_gps(_ptr(X, C.c_float), T, K, _ptr(W, C.c_float), N, bits, int(pct_ppm), variant,
                  _ptr(s, C.c_float), C.byref(ks))
    return s, int(ks.value)


def gps_gain(A, B, s_k, s_i):
    """Scaling gain of Eq. 13 / Eq. 15 given A = sum W^2 dX^2 and B = sum dW^2 X^2."""
    return float(lib().orc_gps_gain(A, B, s_k, s_i))


def pack4(codes):
    """Signed 4-bit codes [..., K] (K even, values in [-8, 7]) -> bytes [..., K/2], low nibble = even channel."""
    codes = np.ascontiguousarray(codes, np.int8)
    assert codes.shape[-1] % 2 == 0
    out = np.empty(codes.shape[:-1] + (codes.shape[-1] // 2,), np.uint8)
    if lib().orc_pack4(_ptr(codes, C.c_int8), out.size, _ptr(out, C.c_uint8)) != 0:
        raise ValueError("a code lies outside [-8, 7]")
    return out


def unpack4(packed):
    """Bytes [..., K/2] -> signed 4-bit codes [..., K] as int8."""
    packed = np.ascontiguousarray(packed, np.uint8)
    out = np.empty(packed.shape[:-1] + (packed.shape[-1] * 2,), np.int8)
    lib().orc_unpack4(_ptr(packed, C.c_uint8), packed.size, _ptr(out, C.c_int8))
    return out


def softmax_quantize(S, causal, bits):
    """Row softmax of S [Tq, Tk] (fp32) then the probability quantizer (unsigned codes, delta = 1/(2^b - 1)).
    Returns (codes uint8 [Tq, Tk], u float64: the value before rounding)."""
    S = _f32(S)
    Tq, Tk = S.shape
    codes = np.empty((Tq, Tk), np.uint8)
    u = np.empty((Tq, Tk), np.float64)
    lib().orc_softmax_quantize(_ptr(S, C.c_float), Tq, Tk, int(bool(causal)), bits, _ptr(codes, C.c_uint8),
                               _ptr(u, C.c_double))
    return codes, u


def igemm_u8s8(P, Vq):
    """acc[i,c] = sum_j P[i,j] Vq[j,c]: unsigned probability codes [Tq, Tk] times signed value codes [Tk, C]."""
    P = np.ascontiguousarray(P, np.uint8)
    Vq = np.ascontiguousarray(Vq, np.int8)
    Tq, Tk = P.shape
    assert Vq.shape[0] == Tk
    acc = np.empty((Tq, Vq.shape[1]), np.int32)
    lib().orc_igemm_u8s8(_ptr(P, C.c_uint8), _ptr(Vq, C.c_int8), Tq, Tk, Vq.shape[1], _ptr(acc, C.c_int32))
    return acc


def qattention(Q, K, V, pos_q, pos_k, s_q, s_k, s_v, softmax_scale, bits, causal):
    """One head of quantized attention, composed of the steps above (queries / keys with per-position
    scales, values per channel, unsigned probability codes). Q [Tq,d], K, V [Tk,d]. Returns a dict with
    every intermediate: Qq, Kq, Vq, acc_qk, S (fp32), Pq, u, acc_pv, O (float64), mag."""
    ones = np.ones(1, np.float32)
    Qq = quantize(Q, pos_q, None, s_q, bits)
    Kq = quantize(K, pos_k, None, s_k, bits)
    Vq = quantize(V, np.zeros(V.shape[0], np.int32), s_v, ones, bits)
    acc_qk = igemm(Qq, Kq)
    s_kcol = (_f32(s_k)[np.asarray(pos_k)] * np.float32(softmax_scale)).astype(np.float32)
    S, _ = epilogue(acc_qk, pos_q, s_q, s_kcol, None, 0)
    S32 = S.astype(np.float32)
    Pq, u = softmax_quantize(S32, causal, bits)
    acc_pv = igemm_u8s8(Pq, Vq)
    delta_p = np.array([np.float32(1.0) / np.float32((1 << bits) - 1)], np.float32)
    O, mag = epilogue(acc_pv, np.zeros(Q.shape[0], np.int32), delta_p, s_v, None, 0)
    return {"Qq": Qq, "Kq": Kq, "Vq": Vq, "acc_qk": acc_qk, "s_kcol": s_kcol, "S": S32, "Pq": Pq, "u": u,
            "acc_pv": acc_pv, "delta_p": delta_p, "O": O, "mag": mag, "act": 0}


def dgc_select(F, keep_ppm=500000, ridge=0.0):
    """Mahalanobis distance of every sample (rows of F [n, D]) to the set, and the indices of the kept
    fraction, largest distance first. Returns (rho float64 [n], selected int32 [k])."""
    F = _f32(F)
    n, D = F.shape
    k = min(n, max(1, (keep_ppm * n + 999999) // 1000000))
    rho = np.empty(n, np.float64)
    sel = np.empty(k, np.int32)
    if lib().orc_dgc_select(_ptr(F, C.c_float), n, D, keep_ppm, float(ridge), _ptr(rho, C.c_double), _ptr(sel, C.c_int32)) != 0:
        raise ValueError("covariance not positive definite (use a ridge)")
    return rho, sel
