"""Test helper: the offline parameters of a workload layer, computed by the CPU oracle."""
from __future__ import annotations

import numpy as np

import oracle
import workloads as wl

PCT = 999900   # 99.99 % percentile calibration


def prepare(layer: wl.Layer, samples: int = 32, gps_n: int = 256):
    """Calibration set -> GPS scales (Algorithm 1) -> per-position scales -> folded int8 weights."""
    Xc, pc = wl.calibration(layer, samples)
    W = wl.weights(layer)
    s_ch = oracle.gps(wl.gps_rows(Xc, gps_n), W, layer.bits, PCT)[0] if layer.use_gps else None
    s_tok = oracle.stwq_calibrate(Xc, pc, layer.P, s_ch, layer.bits, PCT)
    Wq, s_w = oracle.gps_fold(W, s_ch, layer.bits)
    return dict(Xc=Xc, pc=pc, W=W, bias=wl.bias(layer), s_ch=s_ch, s_tok=s_tok, Wq=Wq, s_w=s_w)


def sample_rows(M: int, n: int = 768, tile: int = 128) -> np.ndarray:
    """Rows for a sampled comparison: the first and last tile in full, and one row of every tile."""
    rows = set(range(min(tile, M))) | set(range(max(0, M - tile), M))
    rows |= {min(M - 1, t * tile + (37 * t) % tile) for t in range((M + tile - 1) // tile)}
    extra = np.linspace(0, M - 1, max(0, n - len(rows))).astype(np.int64).tolist() if n > len(rows) else []
    return np.array(sorted(rows | set(extra)), dtype=np.int64)


def assert_close(Y, ref, rtol, what=""):
    """Element-by-element bound on |y - y_ref|, with mag = |acc * s_tok * s_w| + |bias|:

    * no activation (ref["act"] == 0): rtol * |y_ref| + 4 * 2^-24 * mag. The first term is the
      relative error the target names; the second is the fp32 rounding of the terms y is built from
      (int -> float of the accumulator, the scale product, the fused multiply-add), which is all that
      is left of y where the bias cancels the product and a pure relative error has no meaning.
    * with GELU (or when the reference does not say): rtol * (|y_ref| + mag). The bound is absolute in
      |z| on purpose: in GELU's negative tail y = z Phi(z) is many orders below |z|, and the kernel's
      Phi carries an absolute error (1.5e-7 for the erf form), so the error is a fraction of |z|, not
      of |y|."""
    Y = np.asarray(Y, np.float64)
    if ref.get("act", None) == 0:
        tol = rtol * np.abs(ref["Y"]) + 4.0 * 2.0 ** -24 * ref["mag"]
    else:
        tol = rtol * (np.abs(ref["Y"]) + ref["mag"])
    err = np.abs(Y - ref["Y"])
    bad = err > tol
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} outside rtol={rtol}; worst ratio "
                           f"{(err / np.maximum(tol, 1e-300)).max():.3g}")
