"""GPU-vs-oracle parity through the C ABI. Integer results (codes, scales chosen by an order
statistic, int32 accumulators) must be bit-exact; floating-point outputs within
|y - y_ref| <= rtol * (|y_ref| + |acc*s_tok*s_w| + |bias|), rtol = 1e-5 (fp32) / 1e-2 (bf16).
"""
import numpy as np
import pytest

import oracle
import workloads as wl
from layer_setup import PCT, assert_close, prepare, sample_rows

pytestmark = pytest.mark.gpu

RTOL = {"fp32": 1e-5, "bf16": 1e-2}


@pytest.fixture(scope="module")
def gpu():
    import torch

    import paper_2601_21238_b200 as pk
    from paper_2601_21238_b200 import binding as B
    from paper_2601_21238_b200 import build as pkbuild
    pkbuild.build()
    ctx = pk.Context(0)
    dev = torch.device("cuda:0")

    class G:
        pass
    g = G()
    g.torch, g.ctx, g.dev, g.B = torch, ctx, dev, B
    g.T = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    yield g
    ctx.close()


rng = np.random.default_rng(7)


def _out_tensor(g, M, N, out):
    dt = {"fp32": g.torch.float32, "bf16": g.torch.bfloat16, "int32": g.torch.int32}[out]
    return g.torch.full((M, N), -3, dtype=dt, device=g.dev)


def _out_code(g, out):
    return {"fp32": g.B.OUT_F32, "bf16": g.B.OUT_BF16, "int32": g.B.OUT_INT32}[out]


# ----------------------------------------------------------------------------- quantize
@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("shape", [(1, 16, 1), (7, 48, 3), (300, 1040, 11), (64, 1920, 64), (513, 512, 680),
                                   (40, 5120, 5), (1000, 16, 2), (512, 16, 4), (96, 48, 7), (4099, 256, 680)])
def test_quantize_codes_bit_exact(gpu, bits, shape):
    M, K, P = shape
    X = (rng.standard_normal((M, K)) * 3).astype(np.float32)
    pos = rng.integers(0, P, M).astype(np.int32)            # shuffled positions
    s_ch = rng.uniform(0.5, 2, K).astype(np.float32)
    s_tok = rng.uniform(0.01, 0.1, P).astype(np.float32)
    X.flat[:4] = [np.nan, np.inf, -np.inf, 1e30]            # NaN -> 0, Inf and huge saturate
    if M > 2:
        X[1] = 0.0                                          # all-zero row
        X[2] = 1e4                                          # saturating row
    for sc in (s_ch, None):
        ref = oracle.quantize(X, pos, sc, s_tok, bits)
        for variant in (7, 8):              # the register-streaming kernel, the TMA-ring kernel
            Xq = gpu.torch.full((M, K), 99, dtype=gpu.torch.int8, device=gpu.dev)
            gpu.ctx.stwq_set_option(gpu.B.OPT_VARIANT, variant)
            try:
                gpu.ctx.stwq_quantize(gpu.T(X), gpu.T(pos), gpu.T(sc), gpu.T(s_tok), bits, Xq)
                assert gpu.ctx.stwq_device_status() == 0
            finally:
                gpu.ctx.stwq_set_option(gpu.B.OPT_VARIANT, 0)
            np.testing.assert_array_equal(Xq.cpu().numpy(), ref)


def test_quantize_reports_bad_position_and_zeroes_the_row(gpu):
    M, K, P = 20, 64, 4
    X = rng.standard_normal((M, K)).astype(np.float32)
    pos = rng.integers(0, P, M).astype(np.int32)
    pos[5], pos[11] = P, -1
    s_tok = rng.uniform(0.01, 0.1, P).astype(np.float32)
    for variant in (7, 8):
        Xq = gpu.torch.full((M, K), 99, dtype=gpu.torch.int8, device=gpu.dev)
        gpu.ctx.stwq_set_option(gpu.B.OPT_VARIANT, variant)
        try:
            gpu.ctx.stwq_quantize(gpu.T(X), gpu.T(pos), None, gpu.T(s_tok), 8, Xq)
        finally:
            gpu.ctx.stwq_set_option(gpu.B.OPT_VARIANT, 0)
        assert gpu.ctx.stwq_device_status() == -8               # STWQ_ERR_POS_RANGE
        assert gpu.ctx.stwq_device_status() == 0                # reading clears it
        got = Xq.cpu().numpy()
        assert not got[5].any() and not got[11].any()
        good = np.ones(M, bool)
        good[[5, 11]] = False
        np.testing.assert_array_equal(got[good], oracle.quantize(X[good], pos[good], None, s_tok, 8))


def test_host_argument_validation(gpu):
    L, h = gpu.ctx.lib, gpu.ctx.handle
    X = gpu.torch.zeros((4, 32), device=gpu.dev)
    pos = gpu.torch.zeros(4, dtype=gpu.torch.int32, device=gpu.dev)
    s_tok = gpu.torch.ones(1, device=gpu.dev)
    Xq = gpu.torch.zeros((4, 32), dtype=gpu.torch.int8, device=gpu.dev)
    p = lambda t: t.data_ptr()
    assert L.stwq_quantize(h, p(X), p(pos), 4, 32, None, p(s_tok), 1, 7, p(Xq), None) == -4    # bits
    assert L.stwq_quantize(h, p(X), p(pos), 4, 24, None, p(s_tok), 1, 8, p(Xq), None) == -3    # K % 16
    assert L.stwq_quantize(h, p(X) + 4, p(pos), 4, 16, None, p(s_tok), 1, 8, p(Xq), None) == -3
    assert L.stwq_quantize(h, p(X), p(pos), 0, 32, None, p(s_tok), 1, 8, p(Xq), None) == -2    # M
    assert L.stwq_quantize(h, None, p(pos), 4, 32, None, p(s_tok), 1, 8, p(Xq), None) == -1
    assert L.stwq_calibrate(h, p(X), p(pos), 4, 32, 1, None, 8, 0, p(s_tok), None) == -4       # pct
    assert L.stwq_set_option(h, 99, 0) == -2
    # the later entry points: 4-bit codes are for weights only; GPS takes variant 0 or 1
    W = gpu.torch.zeros((8, 32), device=gpu.dev)
    Wq = gpu.torch.zeros((8, 32), dtype=gpu.torch.int8, device=gpu.dev)
    s_w = gpu.torch.zeros(8, device=gpu.dev)
    s_ch = gpu.torch.zeros(32, device=gpu.dev)
    assert L.gps_fold(h, p(W), 8, 32, None, 4, p(Wq), p(s_w), None) == 0
    assert L.gps_fold(h, p(W), 8, 32, None, 5, p(Wq), p(s_w), None) == -4
    assert L.stwq_quantize(h, p(X), p(pos), 4, 32, None, p(s_tok), 1, 4, p(Xq), None) == -4
    assert L.gps_scales(h, p(X), 4, 32, p(W), 8, 8, 999900, 2, p(s_ch), None, None) == -4     # variant
    assert L.gps_scales(h, p(X), 4, 32, p(W), 8, 8, 0, 0, p(s_ch), None, None) == -4          # pct
    assert L.gps_scales(h, p(X), 4, 32, p(W), 0, 8, 999900, 0, p(s_ch), None, None) == -2     # N
    assert L.gps_scales(h, p(X), 4, 32, None, 8, 8, 999900, 0, p(s_ch), None, None) == -1
    Xb = gpu.torch.zeros((4, 32), dtype=gpu.torch.bfloat16, device=gpu.dev)
    Y = gpu.torch.zeros((4, 8), device=gpu.dev)
    assert L.qlinear_bf16(h, p(Xb), p(pos), 4, 24, 8, p(Wq), p(s_w), p(s_tok), 1, None, None, 8, 0, 0, p(Y), None) == -3
    assert L.qlinear_bf16(h, p(Xb), p(pos), 4, 32, 8, p(Wq), p(s_w), p(s_tok), 1, None, None, 8, 4, 0, p(Y), None) == -4
    gpu.torch.cuda.synchronize()
    assert gpu.ctx.stwq_device_status() == 0


# ----------------------------------------------------------------------------- gps_fold
@pytest.mark.parametrize("bits", [8, 6, 4])
@pytest.mark.parametrize("shape", [(1, 16), (70, 208), (256, 1024), (33, 7680)])
def test_gps_fold_bit_exact(gpu, bits, shape):
    N, K = shape
    W = (0.02 * rng.standard_normal((N, K))).astype(np.float32)
    W[N // 2] = 0.0                                         # dead output channel -> s_w = 1
    s_ch = rng.uniform(0.3, 4, K).astype(np.float32)
    for sc in (s_ch, None):
        Wq_r, sw_r = oracle.gps_fold(W, sc, bits)
        Wq = gpu.torch.full((N, K), 99, dtype=gpu.torch.int8, device=gpu.dev)
        sw = gpu.torch.zeros(N, device=gpu.dev)
        gpu.ctx.gps_fold(gpu.T(W), gpu.T(sc), bits, Wq, sw)
        np.testing.assert_array_equal(sw.cpu().numpy(), sw_r)
        np.testing.assert_array_equal(Wq.cpu().numpy(), Wq_r)


# ----------------------------------------------------------------------------- gps_scales
@pytest.mark.parametrize("variant", [0, 1])
@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("shape", [(1, 16, 1), (37, 48, 5), (300, 1040, 70), (256, 1024, 3072), (4100, 520, 33)])
def test_gps_scales_match_the_oracle(gpu, shape, bits, variant):
    """Algorithm 1 on the GPU against the oracle: k* and the clamp decisions are exact; the scales
    agree to fp32 rounding (both sides sum in fp64, in different orders: relative difference of the
    sums below 1e-12, so the fp32 results differ by at most one unit in the last place)."""
    T, K, N = shape
    X = rng.standard_normal((T, K)).astype(np.float32) * rng.uniform(0.2, 3.0, K).astype(np.float32)
    X[:, K // 3] *= 25.0                                    # an outlier channel: the one with the widest range
    W = (0.02 * rng.standard_normal((N, K))).astype(np.float32)
    if K > 4:
        W[:, 1] = 0.0                                       # dead input channel: denominator 0 -> s = 1
        X[:, 2] = 0.0                                       # silent channel: numerator 0 -> s = 1
    s_ref, k_ref = oracle.gps(X, W, bits, PCT, variant)
    s = gpu.torch.zeros(K, device=gpu.dev)
    kstar = gpu.torch.full((1,), -1, dtype=gpu.torch.int32, device=gpu.dev)
    for _ in range(2):
        gpu.ctx.gps_scales(gpu.T(X), gpu.T(W), bits, PCT, variant, s, kstar)
        assert gpu.ctx.stwq_device_status() == 0
        assert int(kstar.item()) == int(k_ref)
        got = s.cpu().numpy()
        np.testing.assert_allclose(got, s_ref, rtol=2.5e-7, atol=0)
        if K > 4 and T > 1:
            assert got[1] == 1.0 and got[2] == 1.0
    first = s.clone()
    gpu.ctx.gps_scales(gpu.T(X), gpu.T(W), bits, PCT, variant, s, None)
    assert gpu.torch.equal(first, s)                        # fixed summation order: repeatable bit for bit


# ----------------------------------------------------------------------------- stwq_calibrate
@pytest.mark.parametrize("pct", [1000000, PCT, 990000, 500000, 1])
def test_calibrate_bit_exact(gpu, pct):
    S, P, K = 6, 9, 112
    pos = np.tile(np.arange(P, dtype=np.int32), S)
    X = (rng.standard_normal((S * P, K)) * (1 + pos[:, None])).astype(np.float32)
    X[3] = 0.0
    perm = rng.permutation(S * P)                           # row order must not matter
    X, pos = X[perm], pos[perm]
    s_ch = rng.uniform(0.5, 2, K).astype(np.float32)
    for bits in (8, 6):
        for sc in (s_ch, None):
            ref = oracle.stwq_calibrate(X, pos, P + 2, sc, bits, pct)   # two positions never seen
            out = gpu.torch.zeros(P + 2, device=gpu.dev)
            gpu.ctx.stwq_calibrate(gpu.T(X), gpu.T(pos), P + 2, gpu.T(sc), bits, pct, out)
            assert gpu.ctx.stwq_device_status() == 0
            np.testing.assert_array_equal(out.cpu().numpy(), ref)


def test_calibrate_config1_full_size(gpu):
    L = wl.config_layers(1)[0]
    par = prepare(L)
    out = gpu.torch.zeros(L.P, device=gpu.dev)
    gpu.ctx.stwq_calibrate(gpu.T(par["Xc"]), gpu.T(par["pc"]), L.P, gpu.T(par["s_ch"]), 8, PCT, out)
    assert gpu.ctx.stwq_device_status() == 0
    np.testing.assert_array_equal(out.cpu().numpy(), par["s_tok"])
    # 16 calibration rows of one sink-like position scaled up: only that position's scale moves
    Xs = par["Xc"].copy()
    Xs[par["pc"] == 0] *= 64
    out2 = gpu.torch.zeros(L.P, device=gpu.dev)
    gpu.ctx.stwq_calibrate(gpu.T(Xs), gpu.T(par["pc"]), L.P, gpu.T(par["s_ch"]), 8, PCT, out2)
    o2 = out2.cpu().numpy()
    np.testing.assert_array_equal(o2[1:], par["s_tok"][1:])
    assert o2[0] == par["s_tok"][0] * 64


def test_calibrate_flags_nonfinite_and_bad_positions(gpu):
    X = rng.standard_normal((12, 32)).astype(np.float32)
    pos = (np.arange(12) % 3).astype(np.int32)
    out = gpu.torch.zeros(3, device=gpu.dev)
    Xb = X.copy()
    Xb[4, 4] = np.inf
    gpu.ctx.stwq_calibrate(gpu.T(Xb), gpu.T(pos), 3, None, 8, PCT, out)
    assert gpu.ctx.stwq_device_status() == -9
    pb = pos.copy()
    pb[0] = 3
    gpu.ctx.stwq_calibrate(gpu.T(X), gpu.T(pb), 3, None, 8, PCT, out)
    assert gpu.ctx.stwq_device_status() == -8


# ----------------------------------------------------------------------------- GEMM accumulators
GEMM_SHAPES = [(1, 16, 16), (128, 256, 128), (128, 128, 2048), (129, 257, 16), (300, 520, 144), (77, 8, 48),
               (256, 512, 384), (640, 1000, 1008), (1000, 136, 8192), (257, 3072, 1024), (2000, 1920, 1920),
               # more tiles than CTA pairs with a last tile column half inside the matrix; one tile
               # more than there are pairs
               (2816, 1920, 256), (600, 640, 128), (19000, 256, 144)]


@pytest.mark.parametrize("path", [1, 3, 0])      # CTA-pair GEMM, single-CTA GEMM, automatic choice
@pytest.mark.parametrize("shape", GEMM_SHAPES)
def test_int32_accumulators_bit_exact(gpu, shape, path):
    M, N, K = shape
    Xq = rng.integers(-128, 128, (M, K)).astype(np.int8)
    Wq = rng.integers(-128, 128, (N, K)).astype(np.int8)
    Xq[0], Wq[0] = -128, -128                              # extreme accumulator K * 2^14
    ref = oracle.igemm(Xq, Wq)
    Y = _out_tensor(gpu, M, N, "int32")
    gpu.ctx.stwq_set_option(gpu.B.OPT_GEMM_PATH, path)
    try:
        gpu.ctx.qlinear_q(gpu.T(Xq), None, gpu.T(Wq), None, None, None, 0, gpu.B.OUT_INT32, Y)
        assert gpu.ctx.stwq_device_status() == 0
    finally:
        gpu.ctx.stwq_set_option(gpu.B.OPT_GEMM_PATH, 0)
    np.testing.assert_array_equal(Y.cpu().numpy(), ref)


def test_repeat_runs_are_bitwise_identical(gpu):
    M, N, K = 900, 1024, 2048
    Xq = gpu.T(rng.integers(-128, 128, (M, K)).astype(np.int8))
    Wq = gpu.T(rng.integers(-128, 128, (N, K)).astype(np.int8))
    a, b = _out_tensor(gpu, M, N, "int32"), _out_tensor(gpu, M, N, "int32")
    gpu.ctx.qlinear_q(Xq, None, Wq, None, None, None, 0, gpu.B.OUT_INT32, a)
    gpu.ctx.qlinear_q(Xq, None, Wq, None, None, None, 0, gpu.B.OUT_INT32, b)
    assert gpu.torch.equal(a, b)


# ----------------------------------------------------------------------------- whole qlinear
def _run_qlinear(gpu, L, par, X, pos, out, act=None, path=0):
    M = X.shape[0]
    Y = _out_tensor(gpu, M, L.N, out)
    gpu.ctx.stwq_set_option(gpu.B.OPT_GEMM_PATH, path)
    try:
        gpu.ctx.qlinear(gpu.T(X) if isinstance(X, np.ndarray) else X, gpu.T(pos) if isinstance(pos, np.ndarray) else pos,
                        gpu.T(par["Wq"]), gpu.T(par["s_w"]), gpu.T(par["s_tok"]), gpu.T(par["s_ch"]),
                        gpu.T(par["bias"]), L.bits, L.act if act is None else act, _out_code(gpu, out), Y)
        assert gpu.ctx.stwq_device_status() == 0
    finally:
        gpu.ctx.stwq_set_option(gpu.B.OPT_GEMM_PATH, 0)
    return Y.float().cpu().numpy() if out != "int32" else Y.cpu().numpy()


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("act", [0, 1, 2])
@pytest.mark.parametrize("out", ["fp32", "bf16"])
def test_qlinear_small_ragged(gpu, bits, act, out):
    """Several tiles with ragged M, N and K tails; every activation and output type."""
    L = wl.scaled(wl.config_layers(1)[0], K=400, N=328, P=37, batch=9, bits=bits, act=act)
    par = prepare(L, samples=8, gps_n=64)
    X, pos = wl.activations(L), wl.positions(L)
    ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], bits, act)
    acc = _run_qlinear(gpu, L, par, X, pos, "int32")
    np.testing.assert_array_equal(acc, ref["acc"])
    assert_close(_run_qlinear(gpu, L, par, X, pos, out), ref, RTOL[out], f"b{bits} act{act} {out}")
    assert_close(_run_qlinear(gpu, L, par, X, pos, out, path=3), ref, RTOL[out], "single-CTA kernel")
    # without bias and without channel scale
    par2 = dict(par, bias=None)
    ref2 = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], None, bits, act)
    assert_close(_run_qlinear(gpu, L, par2, X, pos, out), ref2, RTOL[out], "no bias")


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_match_the_oracle(gpu, seed):
    """Seeded random problem sizes (ragged in every dimension, N a multiple of 4 or of 16, with and
    without channel scale and bias) through every GEMM route: exact accumulators, outputs in tolerance."""
    r = np.random.default_rng(seed)
    for _ in range(10):
        M = int(r.choice([1, 7, 128, 129, 255, 257, 300, 511, int(r.integers(1, 700))]))
        N = int(4 * r.integers(1, 150)) if r.random() < 0.6 else int(16 * r.integers(1, 40))
        K = int(16 * r.integers(1, 64))
        P = int(r.integers(1, 20))
        act = int(r.integers(0, 3))
        path = int(r.choice([0, 0, 1, 3]))
        X = (r.standard_normal((M, K)) * 2).astype(np.float32)
        Wq = r.integers(-128, 128, (N, K)).astype(np.int8)
        pos = r.integers(0, P, M).astype(np.int32)
        s_w = r.uniform(1e-4, 1e-3, N).astype(np.float32)
        s_tok = r.uniform(0.01, 0.06, P).astype(np.float32)
        s_ch = r.uniform(0.5, 1.5, K).astype(np.float32) if r.random() < 0.5 else None
        bias = (0.5 * r.standard_normal(N)).astype(np.float32) if r.random() < 0.7 else None
        ref = oracle.qlinear(X, pos, Wq, s_w, s_tok, s_ch, bias, 8, act)
        what = f"seed {seed} M={M} N={N} K={K} act={act} path={path}"
        gpu.ctx.stwq_set_option(gpu.B.OPT_GEMM_PATH, path)
        try:
            for out in ("int32", "fp32", "bf16"):
                Y = _out_tensor(gpu, M, N, out)
                gpu.ctx.qlinear(gpu.T(X), gpu.T(pos), gpu.T(Wq), gpu.T(s_w), gpu.T(s_tok), gpu.T(s_ch), gpu.T(bias), 8,
                                0 if out == "int32" else act, _out_code(gpu, out), Y)
                assert gpu.ctx.stwq_device_status() == 0, what
                if out == "int32":
                    np.testing.assert_array_equal(Y.cpu().numpy(), ref["acc"], err_msg=what)
                else:
                    assert_close(Y.float().cpu().numpy(), ref, RTOL[out], what + " " + out)
        finally:
            gpu.ctx.stwq_set_option(gpu.B.OPT_GEMM_PATH, 0)


@pytest.mark.parametrize("act", [0, 1])
def test_qlinear_w4a8(gpu, act):
    """4-bit weights with 8-bit activations (Table 11's W4A8): the weight codes come from gps_fold
    with bits = 4 on the GPU, everything else is the 8-bit path."""
    L = wl.scaled(wl.config_layers(1)[0], K=528, N=584, P=37, batch=9, bits=8, act=act)
    par = prepare(L, samples=8, gps_n=64)
    Wq4_ref, sw4_ref = oracle.gps_fold(par["W"], par["s_ch"], 4)
    assert Wq4_ref.min() >= -8 and Wq4_ref.max() <= 7
    Wq4 = gpu.torch.empty((L.N, L.K), dtype=gpu.torch.int8, device=gpu.dev)
    sw4 = gpu.torch.empty(L.N, device=gpu.dev)
    gpu.ctx.gps_fold(gpu.T(par["W"]), gpu.T(par["s_ch"]), 4, Wq4, sw4)
    np.testing.assert_array_equal(Wq4.cpu().numpy(), Wq4_ref)
    np.testing.assert_array_equal(sw4.cpu().numpy(), sw4_ref)
    X, pos = wl.activations(L), wl.positions(L)
    ref = oracle.qlinear(X, pos, Wq4_ref, sw4_ref, par["s_tok"], par["s_ch"], par["bias"], 8, act)
    par4 = dict(par, Wq=Wq4_ref, s_w=sw4_ref)
    np.testing.assert_array_equal(_run_qlinear(gpu, L, par4, X, pos, "int32"), ref["acc"])
    for out in ("fp32", "bf16"):
        assert_close(_run_qlinear(gpu, L, par4, X, pos, out), ref, RTOL[out], f"W4A8 act{act} {out}")


@pytest.mark.parametrize("M", [37, 256, 700])
@pytest.mark.parametrize("act", [0, 1])
def test_packed_int4_weights(gpu, M, act):
    """W4A8 with the weights stored two codes per byte (Table 11's setting): the packed bytes and the
    scales equal the oracle's 4-bit fold packed by the oracle; unpacking on the GPU returns the
    codes; qlinear_w4 gives the accumulators and outputs of qlinear on the unpacked codes, on the
    few-row route (M <= 256) and on the tiled one."""
    torch = gpu.torch
    L = wl.scaled(wl.config_layers(1)[0], K=544, N=584, P=37, batch=19, bits=8, act=act)
    par = prepare(L, samples=8, gps_n=64)
    Wq4, sw4 = oracle.gps_fold(par["W"], par["s_ch"], 4)
    Wp_ref = oracle.pack4(Wq4)
    Wp = torch.full((L.N, L.K // 2), 0x5A, dtype=torch.uint8, device=gpu.dev)
    sw = torch.zeros(L.N, device=gpu.dev)
    gpu.ctx.gps_fold_packed4(gpu.T(par["W"]), gpu.T(par["s_ch"]), Wp, sw)
    np.testing.assert_array_equal(Wp.cpu().numpy(), Wp_ref)
    np.testing.assert_array_equal(sw.cpu().numpy(), sw4)
    back = torch.full((L.N, L.K), 99, dtype=torch.int8, device=gpu.dev)
    gpu.ctx.stwq_unpack4(Wp, back)
    np.testing.assert_array_equal(back.cpu().numpy(), Wq4)
    X, pos = wl.activations(L)[:M], wl.positions(L)[:M]
    ref = oracle.qlinear(X, pos, oracle.unpack4(Wp_ref), sw4, par["s_tok"], par["s_ch"], par["bias"], 8, act)
    d = {k: gpu.T(par[k]) for k in ("s_tok", "s_ch", "bias")}
    for out in ("int32", "fp32", "bf16"):
        Y = _out_tensor(gpu, M, L.N, out)
        gpu.ctx.qlinear_w4(gpu.T(X), gpu.T(pos), Wp, sw, d["s_tok"], d["s_ch"], d["bias"], 8, 0 if out == "int32" else act,
                           _out_code(gpu, out), Y)
        assert gpu.ctx.stwq_device_status() == 0
        if out == "int32":
            np.testing.assert_array_equal(Y.cpu().numpy(), ref["acc"])
        else:
            assert_close(Y.float().cpu().numpy(), ref, RTOL[out], f"qlinear_w4 M={M} {out}")


@pytest.mark.parametrize("out", ["fp32", "bf16"])
def test_config1_full(gpu, out):
    """Config 1: one W8A8 linear over the 680-token VAR pyramid, K = N = 1024, every element."""
    L = wl.config_layers(1)[0]
    par = prepare(L)
    X, pos = wl.activations(L), wl.positions(L)
    ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, 0)
    # the offline calls reproduce the oracle's parameters bit for bit
    Wq = gpu.torch.zeros((L.N, L.K), dtype=gpu.torch.int8, device=gpu.dev)
    sw = gpu.torch.zeros(L.N, device=gpu.dev)
    gpu.ctx.gps_fold(gpu.T(par["W"]), gpu.T(par["s_ch"]), 8, Wq, sw)
    np.testing.assert_array_equal(Wq.cpu().numpy(), par["Wq"])
    np.testing.assert_array_equal(sw.cpu().numpy(), par["s_w"])
    Xq = gpu.torch.zeros((L.M, L.K), dtype=gpu.torch.int8, device=gpu.dev)
    gpu.ctx.stwq_quantize(gpu.T(X), gpu.T(pos), gpu.T(par["s_ch"]), gpu.T(par["s_tok"]), 8, Xq)
    np.testing.assert_array_equal(Xq.cpu().numpy(), ref["Xq"])
    np.testing.assert_array_equal(_run_qlinear(gpu, L, par, X, pos, "int32"), ref["acc"])
    assert_close(_run_qlinear(gpu, L, par, X, pos, out), ref, RTOL[out], "config 1")


@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_config2_full(gpu, idx):
    """Config 2 (VAR-d16 block, batch 16 x 680 tokens): every element of every layer, in the
    launch configuration the benchmark times (bf16 output, fused GELU on fc1)."""
    L = wl.config_layers(2)[idx]
    par = prepare(L, samples=8)
    X, pos = wl.activations(L), wl.positions(L)
    ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, L.act)
    np.testing.assert_array_equal(_run_qlinear(gpu, L, par, X, pos, "int32"), ref["acc"])
    assert_close(_run_qlinear(gpu, L, par, X, pos, "bf16"), ref, RTOL["bf16"], L.name)
    assert_close(_run_qlinear(gpu, L, par, X, pos, "fp32"), ref, RTOL["fp32"], L.name)


def _sampled_full_size(gpu, L, samples=4):
    """Full-size layer drawn on the device; the oracle recomputes a sample of rows (all columns)."""
    par = prepare(L, samples=samples, gps_n=96)
    Xd, posd = wl.activations_device(L, gpu.dev)
    rows = sample_rows(L.M)
    rt = gpu.torch.from_numpy(rows).to(gpu.dev)
    Xs, ps = Xd[rt].cpu().numpy(), posd[rt].cpu().numpy()
    ref = oracle.qlinear(Xs, ps, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], L.bits, L.act)
    for out in ("int32", "bf16"):
        M = L.M
        Y = _out_tensor(gpu, M, L.N, out)
        gpu.ctx.qlinear(Xd, posd, gpu.T(par["Wq"]), gpu.T(par["s_w"]), gpu.T(par["s_tok"]), gpu.T(par["s_ch"]),
                        gpu.T(par["bias"]), L.bits, L.act, _out_code(gpu, out), Y)
        assert gpu.ctx.stwq_device_status() == 0
        got = Y[rt]
        if out == "int32":
            np.testing.assert_array_equal(got.cpu().numpy(), ref["acc"])
        else:
            assert_close(got.float().cpu().numpy(), ref, RTOL["bf16"], f"cfg{L.config} {L.name} b{L.bits}")
        del Y


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("idx", [0, 1, 2, 3])
def test_config3_sampled(gpu, idx, bits):
    """Config 3 (VAR-d30 block, batch 32 x 680, hidden 1920), W8A8 and W6A6, full size on the GPU."""
    _sampled_full_size(gpu, wl.config_layers(3, bits=bits)[idx])


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("idx", [0, 1])
def test_config5_sampled(gpu, idx, bits):
    """Config 5 (MAR-Huge prefill, M = 65536, hidden 1280), W6A6 and W8A8, full size on the GPU."""
    _sampled_full_size(gpu, wl.config_layers(5, bits=bits)[idx])


@pytest.mark.parametrize("path", [0, 1])
@pytest.mark.parametrize("idx", [0, 1])
def test_config4_decode_full(gpu, idx, path):
    """Config 4 (raster-order decode step): 256 rows that share one token position."""
    L = wl.config_layers(4)[idx]
    par = prepare(L, samples=4, gps_n=64)
    for step in (0, 1):
        X, pos = wl.activations(L, step), wl.positions(L, step)
        assert len(set(pos.tolist())) == 1
        ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, 0)
        np.testing.assert_array_equal(_run_qlinear(gpu, L, par, X, pos, "int32", path=path), ref["acc"])
        assert_close(_run_qlinear(gpu, L, par, X, pos, "bf16", path=path), ref, RTOL["bf16"], L.name)
        assert_close(_run_qlinear(gpu, L, par, X, pos, "fp32", path=path), ref, RTOL["fp32"], L.name)


def test_decode_rows_with_mixed_positions_and_few_rows(gpu):
    """The few-row path makes no assumption that positions are shared; also M = 1 and M = 37."""
    L = wl.scaled(wl.config_layers(4)[0], K=512, N=1024, P=16)
    par = prepare(L, samples=4, gps_n=64)
    for M in (1, 37, 256):
        X = wl.activations(L)[:M]
        pos = rng.integers(0, L.P, M).astype(np.int32)
        ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, 1)
        for path in (0, 2):
            np.testing.assert_array_equal(_run_qlinear(gpu, L, par, X, pos, "int32", act=1, path=path), ref["acc"])
            assert_close(_run_qlinear(gpu, L, par, X, pos, "fp32", act=1, path=path), ref, RTOL["fp32"], "decode")


@pytest.mark.parametrize("ksplit", [0, 2, 5])
@pytest.mark.parametrize("shape", [(256, 2048, 256), (200, 1536, 136), (37, 4096, 128), (1, 512, 1024)])
def test_decode_split_k_is_exact_and_repeatable(gpu, shape, ksplit):
    """The few-row path with K split over several CTA pairs: int32 partial sums through scratch
    memory, added up by whichever warp arrives last. Exact, and the counters return to zero, so a
    second call gives the same bits."""
    M, K, N = shape
    L = wl.scaled(wl.config_layers(4)[0], K=K, N=N, P=16)
    par = prepare(L, samples=4, gps_n=64)
    X = wl.activations(wl.scaled(L, batch=256))[:M]
    pos = rng.integers(0, L.P, M).astype(np.int32)
    ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, 2)
    gpu.ctx.stwq_set_option(gpu.B.OPT_KSPLIT, ksplit)
    try:
        for _ in range(2):
            np.testing.assert_array_equal(_run_qlinear(gpu, L, par, X, pos, "int32", act=2, path=2), ref["acc"])
            assert_close(_run_qlinear(gpu, L, par, X, pos, "fp32", act=2, path=2), ref, RTOL["fp32"], "decode fp32")
            assert_close(_run_qlinear(gpu, L, par, X, pos, "bf16", act=2, path=2), ref, RTOL["bf16"], "decode bf16")
    finally:
        gpu.ctx.stwq_set_option(gpu.B.OPT_KSPLIT, 0)


@pytest.mark.parametrize("ksplit", [-1, 0, 3, 7])
@pytest.mark.parametrize("shape", [(600, 520, 2064), (257, 1024, 1024), (1300, 264, 4096)])
def test_tiled_gemm_split_tail_is_exact_and_repeatable(gpu, shape, ksplit):
    """The tiled GEMM cuts the tiles of a partly filled last wave along K (here: every tile, the
    problems being smaller than one wave) and adds the int32 partial sums through scratch memory.
    -1 switches the split off, 0 lets the library choose, 3 and 7 force the number of K ranges."""
    M, N, K = shape
    Xq = rng.integers(-128, 128, (M, K)).astype(np.int8)
    Wq = rng.integers(-128, 128, (N, K)).astype(np.int8)
    pos = rng.integers(0, 5, M).astype(np.int32)
    s_tok = rng.uniform(0.01, 0.1, 5).astype(np.float32)
    s_w = rng.uniform(1e-4, 1e-3, N).astype(np.float32)
    bias = (0.5 * rng.standard_normal(N)).astype(np.float32)
    acc = oracle.igemm(Xq, Wq)
    Yref, mag = oracle.epilogue(acc, pos, s_tok, s_w, bias, 1)
    ref = {"Y": Yref, "mag": mag}
    d = [gpu.T(a) for a in (Xq, pos, Wq, s_w, s_tok, bias)]
    gpu.ctx.stwq_set_option(gpu.B.OPT_GEMM_PATH, 1)
    gpu.ctx.stwq_set_option(gpu.B.OPT_KSPLIT, ksplit)
    try:
        for _ in range(2):
            Yi = _out_tensor(gpu, M, N, "int32")
            gpu.ctx.qlinear_q(d[0], None, d[2], None, None, None, 0, gpu.B.OUT_INT32, Yi)
            np.testing.assert_array_equal(Yi.cpu().numpy(), acc)
            for out in ("bf16", "fp32"):
                Y = _out_tensor(gpu, M, N, out)
                gpu.ctx.qlinear_q(d[0], d[1], d[2], d[3], d[4], d[5], 1, _out_code(gpu, out), Y)
                assert gpu.ctx.stwq_device_status() == 0
                assert_close(Y.float().cpu().numpy(), ref, RTOL[out], f"split tail {out}")
    finally:
        gpu.ctx.stwq_set_option(gpu.B.OPT_KSPLIT, 0)
        gpu.ctx.stwq_set_option(gpu.B.OPT_GEMM_PATH, 0)


@pytest.mark.parametrize("cfg,idx", [(2, 2), (2, 3), (4, 0), (4, 1)])
def test_graph_replay_matches_the_oracle(gpu, cfg, idx):
    """The benchmark replays qlinear from a CUDA graph (with the two kernels of a call chained by
    programmatic dependent launch). The replayed call must give what the direct call gives."""
    torch = gpu.torch
    L = wl.config_layers(cfg)[idx]
    par = prepare(L, samples=4, gps_n=64)
    X, pos = wl.activations(L), wl.positions(L)
    ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], L.bits, L.act)
    d = {k: gpu.T(par[k]) for k in ("Wq", "s_w", "s_tok", "s_ch", "bias")}
    Xd, pd = gpu.T(X), gpu.T(pos)
    Y = _out_tensor(gpu, L.M, L.N, "bf16")
    Yi = _out_tensor(gpu, L.M, L.N, "int32")

    def calls():
        gpu.ctx.qlinear(Xd, pd, d["Wq"], d["s_w"], d["s_tok"], d["s_ch"], d["bias"], L.bits, L.act, gpu.B.OUT_BF16, Y)
        gpu.ctx.qlinear(Xd, pd, d["Wq"], d["s_w"], d["s_tok"], d["s_ch"], d["bias"], L.bits, L.act, gpu.B.OUT_INT32, Yi)
    calls()                                     # workspace is allocated outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            calls()
        Y.fill_(-3)
        Yi.fill_(-3)
        g.replay()
        g.replay()
    torch.cuda.synchronize()
    assert gpu.ctx.stwq_device_status() == 0
    np.testing.assert_array_equal(Yi.cpu().numpy(), ref["acc"])
    assert_close(Y.float().cpu().numpy(), ref, RTOL["bf16"], f"graph replay cfg{cfg} {L.name}")


@pytest.mark.parametrize("option,value", [("TILE_N", 128), ("TILE_N", 256), ("VARIANT", 1), ("VARIANT", 2), ("VARIANT", 5)])
def test_forced_kernel_variants_match_the_oracle(gpu, option, value):
    """Every variant the options name computes the same layer: tile width 128 / 256 of the
    CTA-pair GEMM, staged TMA stores / stores from registers, ordinary instead of programmatic
    dependent launches. Exact accumulators, outputs in tolerance, on a ragged multi-tile shape."""
    opt = {"TILE_N": gpu.B.OPT_TILE_N, "VARIANT": gpu.B.OPT_VARIANT}[option]
    L = wl.scaled(wl.config_layers(1)[0], K=656, N=1032, P=37, batch=21, bits=8, act=1)
    par = prepare(L, samples=4, gps_n=64)
    X, pos = wl.activations(L), wl.positions(L)
    ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, 1)
    ref0 = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, 0)
    gpu.ctx.stwq_set_option(opt, value)
    try:
        np.testing.assert_array_equal(_run_qlinear(gpu, L, par, X, pos, "int32", path=1), ref["acc"])
        for out in ("fp32", "bf16"):
            assert_close(_run_qlinear(gpu, L, par, X, pos, out, path=1), ref, RTOL[out], f"{option}={value} {out}")
            assert_close(_run_qlinear(gpu, L, par, X, pos, out, act=0, path=1), ref0, RTOL[out], f"{option}={value} {out}")
    finally:
        gpu.ctx.stwq_set_option(opt, 0)


def test_options_reject_values_they_do_not_name(gpu):
    L, h = gpu.ctx.lib, gpu.ctx.handle
    for opt, bad in ((gpu.B.OPT_TILE_N, 64), (gpu.B.OPT_TILE_N, 192), (gpu.B.OPT_VARIANT, 3), (gpu.B.OPT_VARIANT, 10),
                     (gpu.B.OPT_KSPLIT, -2), (gpu.B.OPT_KSPLIT, 65), (gpu.B.OPT_GEMM_PATH, 4),
                     (gpu.B.OPT_WAIT_LIMIT_MS, 0)):
        assert L.stwq_set_option(h, opt, bad) == -2
    for opt in (gpu.B.OPT_TILE_N, gpu.B.OPT_VARIANT, gpu.B.OPT_KSPLIT, gpu.B.OPT_GEMM_PATH):
        assert L.stwq_set_option(h, opt, 0) == 0


def test_peak_probe_and_reserve_layer(gpu):
    """The int8 peak probe launches, reports the operations it performs and leaves no error behind;
    stwq_reserve_layer makes a later call allocation-free (the workspace generation stays put)."""
    torch = gpu.torch
    ops = gpu.ctx.stwq_probe_int8_peak(64, 3)
    assert ops == 3 * 64 * 4 * 2 * 256 * 256 * 32
    ops_all = gpu.ctx.stwq_probe_int8_peak(16)
    assert ops_all % (16 * 4 * 2 * 256 * 256 * 32) == 0 and ops_all > 0
    assert gpu.ctx.stwq_device_status() == 0
    gpu.ctx.stwq_reserve_layer(200, 4096, 1024, 8)
    gen = gpu.ctx.stwq_workspace_generation()
    L = wl.scaled(wl.config_layers(4)[1], K=4096, N=1024, P=8)
    par = prepare(L, samples=2, gps_n=32)
    X = wl.activations(wl.scaled(L, batch=256))[:200]
    pos = rng.integers(0, L.P, 200).astype(np.int32)
    ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, 0)
    np.testing.assert_array_equal(_run_qlinear(gpu, L, par, X, pos, "int32", act=0), ref["acc"])     # splits K: uses the scratch
    assert gpu.ctx.stwq_workspace_generation() == gen


# ----------------------------------------------------------------------------- failure handling
def test_bounded_wait_expires_and_the_context_stays_usable(gpu):
    """The wait every GEMM kernel uses gives up after the limit, the kernel reports the timeout and
    returns; the status is read once and clears; the next call computes correctly. The wait that
    runs out belongs to a one-CTA self-test kernel (a barrier nothing arrives at), never to a
    kernel that moves data."""
    torch = gpu.torch
    waited = torch.zeros(1, dtype=torch.int64, device=gpu.dev)
    gpu.ctx.stwq_set_option(gpu.B.OPT_WAIT_LIMIT_MS, 2)
    try:
        gpu.ctx.stwq_selftest_wait_expiry(waited)
        assert gpu.ctx.stwq_device_status() == -7             # STWQ_ERR_DEVICE_TIMEOUT
        assert gpu.ctx.stwq_device_status() == 0              # reading clears it
        ns = int(waited.item())
        assert 2_000_000 <= ns < 200_000_000, ns               # it waited for the limit, not forever
    finally:
        gpu.ctx.stwq_set_option(gpu.B.OPT_WAIT_LIMIT_MS, 2000)
    M, N, K = 300, 520, 144
    Xq = rng.integers(-128, 128, (M, K)).astype(np.int8)
    Wq = rng.integers(-128, 128, (N, K)).astype(np.int8)
    Y = _out_tensor(gpu, M, N, "int32")
    gpu.ctx.qlinear_q(gpu.T(Xq), None, gpu.T(Wq), None, None, None, 0, gpu.B.OUT_INT32, Y)
    assert gpu.ctx.stwq_device_status() == 0
    np.testing.assert_array_equal(Y.cpu().numpy(), oracle.igemm(Xq, Wq))


def test_workspace_growth_is_refused_during_capture(gpu):
    """A call that would have to allocate workspace while its stream is being captured returns
    STWQ_ERR_CAPTURE and enqueues nothing; after stwq_reserve_layer the same capture succeeds, and
    the workspace generation tells a holder of older graphs that buffers moved."""
    torch = gpu.torch
    import paper_2601_21238_b200 as pk
    ctx = pk.Context(0)
    try:
        M, K, N, P = 384, 256, 512, 8
        X = torch.randn(M, K, device=gpu.dev)
        pos = torch.zeros(M, dtype=torch.int32, device=gpu.dev)
        Wq = torch.randint(-128, 128, (N, K), dtype=torch.int8, device=gpu.dev)
        s_w = torch.full((N,), 1e-3, device=gpu.dev)
        s_tok = torch.full((P,), 0.05, device=gpu.dev)
        Y = torch.zeros((M, N), device=gpu.dev)
        call = lambda: ctx.qlinear(X, pos, Wq, s_w, s_tok, None, None, 8, 0, gpu.B.OUT_F32, Y)
        gen0 = ctx.stwq_workspace_generation()
        side = torch.cuda.Stream()
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                with pytest.raises(pk.StwqError) as ei:
                    call()                                   # fresh context: no workspace yet
            assert ei.value.code == -11                       # STWQ_ERR_CAPTURE
        torch.cuda.synchronize()
        assert ctx.stwq_workspace_generation() == gen0        # nothing was allocated
        ctx.stwq_reserve_layer(M, K, N, P)
        gen1 = ctx.stwq_workspace_generation()
        assert gen1 > gen0
        with torch.cuda.stream(side):
            g2 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g2, stream=side):
                call()
            g2.replay()
        torch.cuda.synchronize()
        assert ctx.stwq_device_status() == 0
        assert ctx.stwq_workspace_generation() == gen1        # the capture and the replay allocated nothing
        want = torch.zeros((M, N), device=gpu.dev)
        ctx.qlinear(X, pos, Wq, s_w, s_tok, None, None, 8, 0, gpu.B.OUT_F32, want)
        torch.cuda.synchronize()
        assert torch.equal(Y, want)
        # a larger problem moves the buffer: the generation changes, which is the cue to re-capture
        X2 = torch.randn(4 * M, K, device=gpu.dev)
        pos2 = torch.zeros(4 * M, dtype=torch.int32, device=gpu.dev)
        Y2 = torch.zeros((4 * M, N), device=gpu.dev)
        ctx.qlinear(X2, pos2, Wq, s_w, s_tok, None, None, 8, 0, gpu.B.OUT_F32, Y2)
        torch.cuda.synchronize()
        assert ctx.stwq_workspace_generation() > gen1
    finally:
        ctx.close()


# ----------------------------------------------------------------------------- dynamic token-wise baseline
@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("shape", [(1, 16), (37, 1040), (300, 2048), (64, 5120), (9, 8192)])
def test_dtwq_codes_and_scales_bit_exact(gpu, bits, shape):
    M, K = shape
    X = (rng.standard_normal((M, K)) * rng.uniform(0.1, 30, (M, 1))).astype(np.float32)
    X.flat[:2] = [np.nan, 1e30]
    if M > 2:
        X[1] = 0.0
    s_ch = rng.uniform(0.5, 2, K).astype(np.float32)
    for sc in (s_ch, None):
        ref_q, ref_s = oracle.dtwq_quantize(X, sc, bits)
        Xq = gpu.torch.full((M, K), 99, dtype=gpu.torch.int8, device=gpu.dev)
        sr = gpu.torch.zeros(M, device=gpu.dev)
        gpu.ctx.dtwq_quantize(gpu.T(X), gpu.T(sc), bits, Xq, sr)
        np.testing.assert_array_equal(sr.cpu().numpy(), ref_s)
        np.testing.assert_array_equal(Xq.cpu().numpy(), ref_q)


@pytest.mark.parametrize("M", [200, 1500])
def test_qlinear_dtwq_matches_the_oracle(gpu, M):
    """qlinear with run-time per-row scales: codes from the dynamic quantizer, dequantizer fed
    with the row's own scale. M = 200 takes the few-row kernel, M = 1500 the tiled GEMM."""
    L = wl.scaled(wl.config_layers(2)[2], batch=3, K=1024, N=768)
    par = prepare(L, samples=4, gps_n=64)
    X = wl.activations(L)[:M]
    Xq, s_row = oracle.dtwq_quantize(X, par["s_ch"], 8)
    acc = oracle.igemm(Xq, par["Wq"])
    ids = np.arange(M, dtype=np.int32)
    Yref, mag = oracle.epilogue(acc, ids, s_row, par["s_w"], par["bias"], 1)
    ref = {"Y": Yref, "mag": mag}
    d = {k: gpu.T(par[k]) for k in ("Wq", "s_w", "s_ch", "bias")}
    Yi = _out_tensor(gpu, M, L.N, "int32")
    gpu.ctx.qlinear_dtwq(gpu.T(X), d["Wq"], d["s_w"], d["s_ch"], d["bias"], 8, 1, gpu.B.OUT_INT32, Yi)
    np.testing.assert_array_equal(Yi.cpu().numpy(), acc)
    for out in ("fp32", "bf16"):
        Y = _out_tensor(gpu, M, L.N, out)
        gpu.ctx.qlinear_dtwq(gpu.T(X), d["Wq"], d["s_w"], d["s_ch"], d["bias"], 8, 1, _out_code(gpu, out), Y)
        assert gpu.ctx.stwq_device_status() == 0
        assert_close(Y.float().cpu().numpy(), ref, RTOL[out], f"qlinear_dtwq {out}")


# ----------------------------------------------------------------------------- chained layers
@pytest.mark.parametrize("act", [0, 1, 2, 3])
@pytest.mark.parametrize("bits_next", [8, 6])
@pytest.mark.parametrize("shape", [(333, 400, 336), (1500, 1024, 1024), (77, 48, 32), (700, 272, 1040)])
def test_chained_output_codes(gpu, shape, bits_next, act):
    """qlinear_chain: the epilogue applies the next layer's static quantizer. Without activation
    the codes are bit-exact. With GELU (erf or tanh form) the activation is evaluated to fp32
    accuracy, and a code may differ from the oracle's (which rounds the exact activation to fp32)
    only where the oracle's pre-round value sits within fp32 noise of a rounding tie. The short
    GELU (act 3, asked for by name) moves y by up to 6e-4 |z| and is held to that."""
    M0, K, N = shape
    ref_act = 2 if act == 3 else act                      # the short form approximates the tanh form
    L = wl.scaled(wl.config_layers(2)[2], batch=3, P=680, K=K, N=N, act=ref_act)
    par = prepare(L, samples=4, gps_n=64)
    X, pos = wl.activations(L)[:M0], wl.positions(L)[:M0]
    first = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, ref_act)
    s_chn = rng.uniform(0.5, 2, N).astype(np.float32)
    # next-layer scales sized so that the codes use the range: y / (s_ch s_tok) of order 30
    typical = np.maximum(np.abs(first["Y"]).mean(axis=1), 1e-3)
    s_tokn = np.zeros(L.P, np.float32)
    for p_ in range(L.P):
        sel = pos == p_
        s_tokn[p_] = np.float32(typical[sel].mean() / 20) if sel.any() else np.float32(1)
    ref = oracle.chain_codes(first["acc"], pos, par["s_tok"], par["s_w"], par["bias"], ref_act, s_chn, s_tokn, bits_next)
    d = {k: gpu.T(par[k]) for k in ("Wq", "s_w", "s_tok", "s_ch", "bias")}
    out = gpu.torch.full((M0, N), 99, dtype=gpu.torch.int8, device=gpu.dev)
    gpu.ctx.qlinear_chain(gpu.T(X), gpu.T(pos), d["Wq"], d["s_w"], d["s_tok"], d["s_ch"], d["bias"], 8, act,
                          gpu.T(s_chn), gpu.T(s_tokn), bits_next, out)
    assert gpu.ctx.stwq_device_status() == 0
    got = out.cpu().numpy().astype(np.int32)
    want = ref["codes"].astype(np.int32)
    if act == 0:
        np.testing.assert_array_equal(got, want)
    else:
        diff = got != want
        assert np.abs(got - want).max() <= 1
        u = ref["u"].astype(np.float64)
        if act == 3:
            slack = 1e-3 * ref["zmag"].astype(np.float64) + 1e-3
            limit = 0.05
        else:
            # fp32 noise on u, plus the activation's own error carried to u: at most 3e-7 |z| on y
            # (the erf form's fitted polynomial 4e-8, its fp32 evaluation 5e-8, the hardware exp2
            # 2^-22 of Phi <= 1/2; the tanh form's exp2 / reciprocal are closer)
            slack = 8e-6 * np.maximum(1.0, np.abs(u)) + 1e-6 + 3e-7 * ref["zmag"].astype(np.float64)
            limit = 2e-3
        assert (np.abs(u - np.floor(u) - 0.5)[diff] <= slack[diff]).all()
        assert diff.mean() < limit
        print(f"chained codes act={act} bits_next={bits_next} {shape}: {diff.sum()} of {diff.size} differ by one")
    assert np.abs(got).max() > 2 ** (bits_next - 1) // 2       # the range is really used
    # the same from codes already held
    out2 = gpu.torch.full((M0, N), 99, dtype=gpu.torch.int8, device=gpu.dev)
    gpu.ctx.qlinear_chain_q(gpu.T(first["Xq"]), gpu.T(pos), d["Wq"], d["s_w"], d["s_tok"], d["bias"], act,
                            gpu.T(s_chn), gpu.T(s_tokn), bits_next, out2)
    assert gpu.torch.equal(out, out2)


@pytest.mark.parametrize("out", ["fp32", "bf16"])
@pytest.mark.parametrize("shape", [(333, 400, 328), (200, 2048, 512)])
def test_short_gelu_is_the_tanh_form_within_its_stated_error(gpu, shape, out):
    """STWQ_ACT_GELU_FAST: within 6e-4 |z| (+ output rounding) of the tanh form, on the tiled and
    the few-row route; inside the bf16 tolerance of either GELU form."""
    M, K, N = shape
    L = wl.scaled(wl.config_layers(1)[0], K=K, N=N, P=37, batch=1, bits=8, act=2)
    par = prepare(L, samples=4, gps_n=64)
    X = (rng.standard_normal((M, K)) * 2).astype(np.float32)
    pos = rng.integers(0, L.P, M).astype(np.int32)
    ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, 2)
    ref_erf = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, 1)
    Y = _run_qlinear(gpu, L, par, X, pos, out, act=gpu.B.ACT_GELU_FAST)
    zmag = ref["mag"]
    rounding = 2.0 ** -8 if out == "bf16" else 2.0 ** -22
    assert (np.abs(Y - ref["Y"]) <= 6e-4 * zmag + rounding * np.abs(ref["Y"]) + 1e-30).all()
    if out == "bf16":
        assert_close(Y, ref, RTOL["bf16"], "short GELU against the tanh form")
        assert_close(Y, ref_erf, RTOL["bf16"], "short GELU against the erf form")


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("shape", [(1, 16, 1), (7, 48, 3), (300, 1040, 11), (513, 512, 680), (40, 5120, 5)])
def test_quantize_bf16_input_bit_exact(gpu, bits, shape):
    """bf16 activations: the codes are those of the quantizer on the same values widened to fp32."""
    M, K, P = shape
    Xb = gpu.torch.from_numpy((rng.standard_normal((M, K)) * 3).astype(np.float32)).to(gpu.dev).to(gpu.torch.bfloat16)
    Xb.view(-1)[:3] = gpu.torch.tensor([float("nan"), float("inf"), 1e30], dtype=gpu.torch.bfloat16)
    X = Xb.float().cpu().numpy()
    pos = rng.integers(0, P, M).astype(np.int32)
    s_ch = rng.uniform(0.5, 2, K).astype(np.float32)
    s_tok = rng.uniform(0.01, 0.1, P).astype(np.float32)
    for sc in (s_ch, None):
        ref = oracle.quantize(X, pos, sc, s_tok, bits)
        Xq = gpu.torch.full((M, K), 99, dtype=gpu.torch.int8, device=gpu.dev)
        gpu.ctx.stwq_quantize_bf16(Xb, gpu.T(pos), gpu.T(sc), gpu.T(s_tok), bits, Xq)
        assert gpu.ctx.stwq_device_status() == 0
        np.testing.assert_array_equal(Xq.cpu().numpy(), ref)


@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("shape", [(333, 400, 328), (1500, 1024, 1024), (200, 2048, 512)])
def test_qlinear_bf16_matches_the_oracle(gpu, shape, act):
    """The whole layer on bf16 activations equals the oracle's layer on the widened values: exact
    accumulators, outputs within the usual tolerance (the last shape takes the few-row kernel)."""
    torch = gpu.torch
    M, K, N = shape
    L = wl.scaled(wl.config_layers(1)[0], K=K, N=N, P=37, batch=1, bits=8, act=act)
    par = prepare(L, samples=4, gps_n=64)
    Xb = torch.from_numpy((rng.standard_normal((M, K)) * 2).astype(np.float32)).to(gpu.dev).to(torch.bfloat16)
    X = Xb.float().cpu().numpy()
    pos = rng.integers(0, L.P, M).astype(np.int32)
    ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], 8, act)
    d = {k: gpu.T(par[k]) for k in ("Wq", "s_w", "s_tok", "s_ch", "bias")}
    for out in ("int32", "fp32", "bf16"):
        Y = _out_tensor(gpu, M, N, out)
        gpu.ctx.qlinear_bf16(Xb, gpu.T(pos), d["Wq"], d["s_w"], d["s_tok"], d["s_ch"], d["bias"], 8,
                             0 if out == "int32" else act, _out_code(gpu, out), Y)
        assert gpu.ctx.stwq_device_status() == 0
        if out == "int32":
            np.testing.assert_array_equal(Y.cpu().numpy(), ref["acc"])
        else:
            assert_close(Y.float().cpu().numpy(), ref, RTOL[out], f"qlinear_bf16 {out}")


# ----------------------------------------------------------------------------- asymmetric quantizer (Eq. 1 as printed)
@pytest.mark.parametrize("bits", [8, 6])
def test_asym_offline_calls_bit_exact(gpu, bits):
    torch = gpu.torch
    N, K = 70, 208
    W = (0.02 * rng.standard_normal((N, K)) + 0.01 * rng.standard_normal((N, 1))).astype(np.float32)
    W[5] = np.abs(W[5]) + 0.01
    W[6] = 0.0
    s_ch = rng.uniform(0.3, 4, K).astype(np.float32)
    for sc in (s_ch, None):
        ref = oracle.gps_fold_asym(W, sc, bits)
        Wq = torch.full((N, K), 99, dtype=torch.int8, device=gpu.dev)
        sw = torch.zeros(N, device=gpu.dev)
        zw = torch.zeros(N, dtype=torch.int32, device=gpu.dev)
        cs = torch.zeros(N, dtype=torch.int32, device=gpu.dev)
        gpu.ctx.gps_fold_asym(gpu.T(W), gpu.T(sc), bits, Wq, sw, zw, cs)
        for got, want in zip((Wq, sw, zw, cs), ref):
            np.testing.assert_array_equal(got.cpu().numpy(), want)
    S, P = 6, 9
    pos = np.tile(np.arange(P, dtype=np.int32), S)
    X = (rng.standard_normal((S * P, K)) * (1 + pos[:, None]) + 0.3 * pos[:, None]).astype(np.float32)
    X[pos == 2] = np.abs(X[pos == 2])
    perm = rng.permutation(S * P)
    X, pos = X[perm], pos[perm]
    for pct in (1000000, 990000, 500000):
        for sc in (s_ch, None):
            rs, rz = oracle.stwq_calibrate_asym(X, pos, P + 2, sc, bits, pct)
            st = torch.zeros(P + 2, device=gpu.dev)
            zt = torch.zeros(P + 2, dtype=torch.int32, device=gpu.dev)
            gpu.ctx.stwq_calibrate_asym(gpu.T(X), gpu.T(pos), P + 2, gpu.T(sc), bits, pct, st, zt)
            assert gpu.ctx.stwq_device_status() == 0
            np.testing.assert_array_equal(st.cpu().numpy(), rs)
            np.testing.assert_array_equal(zt.cpu().numpy(), rz)


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("act", [0, 1])
@pytest.mark.parametrize("shape", [(333, 400, 328), (1500, 1024, 768), (77, 48, 24), (700, 272, 1048)])
def test_qlinear_asym_matches_the_oracle(gpu, shape, act, bits):
    """Asymmetric codes and row corrections bit-exact; the corrected int32 accumulators (which equal
    sum_k (cs - zx)(ws - zw)) bit-exact; outputs within the usual tolerance."""
    torch = gpu.torch
    M, K, N = shape
    L = wl.scaled(wl.config_layers(2)[2], batch=3, P=680, K=K, N=N, act=act, bits=bits)
    W, b = wl.weights(L) + np.float32(0.004), wl.bias(L)
    X = (wl.activations(L)[:M] + np.float32(0.8)).astype(np.float32)           # off-centre on purpose
    pos = wl.positions(L)[:M]
    s_ch = rng.uniform(0.5, 2, K).astype(np.float32)
    s_tok, z_tok = oracle.stwq_calibrate_asym(X, pos, L.P, s_ch, bits, 999000)
    Wq, s_w, z_w, cs = oracle.gps_fold_asym(W, s_ch, bits)
    ref = oracle.qlinear_asym(X, pos, Wq, s_w, z_w, cs, s_tok, z_tok, s_ch, b, bits, act)
    Xq = torch.full((M, K), 99, dtype=torch.int8, device=gpu.dev)
    rc = torch.full((M,), 7, dtype=torch.int32, device=gpu.dev)
    gpu.ctx.stwq_quantize_asym(gpu.T(X), gpu.T(pos), gpu.T(s_ch), gpu.T(s_tok), gpu.T(z_tok), bits, Xq, rc)
    np.testing.assert_array_equal(Xq.cpu().numpy(), ref["Xq"])
    np.testing.assert_array_equal(rc.cpu().numpy(), ref["rowcorr"])
    args = [gpu.T(a) for a in (X, pos, Wq, s_w, z_w, cs, s_tok, z_tok, s_ch, b)]
    Yi = _out_tensor(gpu, M, N, "int32")
    gpu.ctx.qlinear_asym(*args, bits, act, gpu.B.OUT_INT32, Yi)
    np.testing.assert_array_equal(Yi.cpu().numpy(), ref["acc"])
    for out in ("fp32", "bf16"):
        Y = _out_tensor(gpu, M, N, out)
        gpu.ctx.qlinear_asym(*args, bits, act, _out_code(gpu, out), Y)
        assert gpu.ctx.stwq_device_status() == 0
        assert_close(Y.float().cpu().numpy(), ref, RTOL[out], f"qlinear_asym {out}")
