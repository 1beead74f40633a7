"""Quantized attention matmuls and the quantized KV cache on the GPU against the CPU oracle: cache
codes, integer accumulators and probability codes of every stage, then the composite call; and the
calibration-set selection by Mahalanobis distance (Section 4.3).
Integer results bit-exact; the probability codes (an integer decided by a floating-point softmax)
may differ by one where the oracle's value before rounding lies within fp32 noise of a tie."""
import numpy as np
import pytest

import oracle
from layer_setup import assert_close

pytestmark = pytest.mark.gpu

rng = np.random.default_rng(31)


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


def _head_data(G, T, d, P):
    """Seeded heads with per-position magnitude and a few outlier channels, and static scales sized
    like a calibration would (ranges near the data's abs-max per position / per channel)."""
    sig = rng.uniform(0.5, 3.0, (1, T, 1)).astype(np.float32)
    Q = (rng.standard_normal((G, T, d)).astype(np.float32) * sig)
    K = (rng.standard_normal((G, T, d)).astype(np.float32) * sig)
    V = rng.standard_normal((G, T, d)).astype(np.float32)
    V[:, :, :2] *= 6.0
    s_q = np.ones(P, np.float32)
    s_k = np.ones(P, np.float32)
    s_q[:T] = (np.abs(Q).max(axis=(0, 2)) * 2 / 255 * 0.9).astype(np.float32)      # a little saturation
    s_k[:T] = (np.abs(K).max(axis=(0, 2)) * 2 / 255).astype(np.float32)
    s_v = (np.abs(V).max(axis=(0, 1)) * 2 / 255).astype(np.float32)
    return Q, K, V, s_q, s_k, s_v


@pytest.mark.parametrize("bits", [8, 6])
def test_kv_append_writes_the_oracles_codes_into_both_cache_layouts(gpu, bits):
    torch = gpu.torch
    G, T, d, P, Tmax = 3, 21, 48, 24, 32
    _, K, V, _, s_k, s_v = _head_data(G, T, d, P)
    Kc = torch.full((G, Tmax, d), 77, dtype=torch.int8, device=gpu.dev)
    Vt = torch.full((G, d, Tmax), 77, dtype=torch.int8, device=gpu.dev)
    # prefill of 16 positions, then five single-position steps
    gpu.ctx.kv_append(gpu.T(K[:, :16]), gpu.T(V[:, :16]), 0, gpu.T(s_k), gpu.T(s_v), bits, Kc, Vt)
    for t in range(16, T):
        gpu.ctx.kv_append(gpu.T(K[:, t:t + 1]), gpu.T(V[:, t:t + 1]), t, gpu.T(s_k), gpu.T(s_v), bits, Kc, Vt)
    assert gpu.ctx.stwq_device_status() == 0
    pos = np.arange(T, dtype=np.int32)
    for g in range(G):
        want_k = oracle.quantize(K[g], pos, None, s_k, bits)
        want_v = oracle.quantize(V[g], np.zeros(T, np.int32), s_v, np.ones(1, np.float32), bits)
        np.testing.assert_array_equal(Kc[g, :T].cpu().numpy(), want_k)
        np.testing.assert_array_equal(Vt[g, :, :T].cpu().numpy(), want_v.T)
    assert (Kc[:, T:].cpu().numpy() == 77).all() and (Vt[:, :, T:].cpu().numpy() == 77).all()   # untouched slots
    # a position beyond the cache or the scale table is refused on the host
    with pytest.raises(Exception):
        gpu.ctx.kv_append(gpu.T(K[:, :4]), gpu.T(V[:, :4]), Tmax - 2, gpu.T(s_k), gpu.T(s_v), bits, Kc, Vt)


@pytest.mark.parametrize("case", [(2, 70, 64, 3, 96), (1, 33, 16, 31, 64), (5, 256, 128, 0, 256)])
def test_kv_append_blocks_of_positions_at_an_odd_offset(gpu, case):
    """Several 32-position tiles with a ragged last one, starting at a cache column that is not a
    multiple of 4: the transposed value cache is written in runs along the positions."""
    torch = gpu.torch
    G, t_new, d, pos0, Tmax = case
    P = Tmax
    _, K, V, _, _, s_v = _head_data(G, t_new, d, P)
    s_k = rng.uniform(0.01, 0.05, P).astype(np.float32)
    Kc = torch.full((G, Tmax, d), -5, dtype=torch.int8, device=gpu.dev)
    Vt = torch.full((G, d, Tmax), -5, dtype=torch.int8, device=gpu.dev)
    gpu.ctx.kv_append(gpu.T(K), gpu.T(V), pos0, gpu.T(s_k), gpu.T(s_v), 8, Kc, Vt)
    assert gpu.ctx.stwq_device_status() == 0
    pos = np.arange(pos0, pos0 + t_new, dtype=np.int32)
    kc, vt = Kc.cpu().numpy(), Vt.cpu().numpy()
    for g in range(G):
        np.testing.assert_array_equal(kc[g, pos0:pos0 + t_new], oracle.quantize(K[g], pos, None, s_k, 8))
        want_v = oracle.quantize(V[g], np.zeros(t_new, np.int32), s_v, np.ones(1, np.float32), 8)
        np.testing.assert_array_equal(vt[g, :, pos0:pos0 + t_new], want_v.T)
    assert (kc[:, :pos0] == -5).all() and (kc[:, pos0 + t_new:] == -5).all()
    assert (vt[:, :, :pos0] == -5).all() and (vt[:, :, pos0 + t_new:] == -5).all()


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("shape", [(5, 37, 37, True), (3, 1, 50, False), (2, 300, 300, True), (4, 20, 129, True)])
def test_softmax_quantizer_codes(gpu, shape, bits):
    torch = gpu.torch
    G, Tq, Tk, causal = shape
    ld = (Tk + 15) // 16 * 16
    S = (rng.standard_normal((G * Tq, ld)) * 4).astype(np.float32)
    Pq = torch.full((G * Tq, ld), 9, dtype=torch.uint8, device=gpu.dev)
    gpu.ctx.qattn_softmax_quantize(gpu.T(S), Tq, Tk, causal, bits, Pq)
    got = Pq.cpu().numpy().astype(np.int32)
    assert (got[:, Tk:] == 0).all()                       # padding columns
    flips = 0
    for g in range(G):
        want, u = oracle.softmax_quantize(S[g * Tq:(g + 1) * Tq, :Tk], causal, bits)
        diff = got[g * Tq:(g + 1) * Tq, :Tk] != want
        assert np.abs(got[g * Tq:(g + 1) * Tq, :Tk] - want.astype(np.int32)).max() <= 1
        # fp32 softmax: relative error of a probability below 2e-6 (exp2 of a rounded argument, a sum of Tk terms)
        assert (np.abs(u - np.floor(u) - 0.5)[diff] <= 2e-6 * np.maximum(1.0, u[diff]) * 8).all()
        flips += int(diff.sum())
    assert flips <= 1e-3 * got.size + 2


@pytest.mark.parametrize("shape", [(3, 37, 48, 64, 64), (2, 300, 304, 128, 320), (5, 1, 80, 64, 96), (1, 680, 688, 64, 688)])
def test_probability_value_matmul_is_exact(gpu, shape):
    """Unsigned probability codes times the transposed value cache: int32 accumulators bit-exact
    (a code above 127 must be read as unsigned), outputs within tolerance."""
    torch = gpu.torch
    G, Tq, Tk_pad, d, Tmax = shape
    Pc = rng.integers(0, 256, (G, Tq, Tk_pad)).astype(np.uint8)
    Vq = rng.integers(-128, 128, (G, Tmax, d)).astype(np.int8)          # columns beyond Tk_pad are never read
    s_v = rng.uniform(1e-3, 1e-2, d).astype(np.float32)
    delta = np.array([1.0 / 255.0], np.float32)
    Vt = np.ascontiguousarray(Vq.transpose(0, 2, 1))
    acc = torch.full((G, Tq, d), -3, dtype=torch.int32, device=gpu.dev)
    gpu.ctx.qattn_pv(gpu.T(Pc), gpu.T(Vt), None, None, gpu.B.OUT_INT32, acc)
    assert gpu.ctx.stwq_device_status() == 0
    for out, dt, rtol in (("fp32", torch.float32, 1e-5), ("bf16", torch.bfloat16, 1e-2)):
        O = torch.full((G, Tq, d), -3, dtype=dt, device=gpu.dev)
        gpu.ctx.qattn_pv(gpu.T(Pc), gpu.T(Vt), gpu.T(s_v), gpu.T(delta), gpu.B.OUT_F32 if out == "fp32" else gpu.B.OUT_BF16, O)
        for g in range(G):
            want = oracle.igemm_u8s8(Pc[g], Vq[g, :Tk_pad])
            np.testing.assert_array_equal(acc[g].cpu().numpy(), want)
            Y, mag = oracle.epilogue(want, np.zeros(Tq, np.int32), delta, s_v, None, 0)
            assert_close(O[g].float().cpu().numpy(), {"Y": Y, "mag": mag, "act": 0}, rtol, f"P V {out}")


@pytest.mark.parametrize("variant", [0, 9])
@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("shape", [(4, 37, 37, 64, True), (2, 1, 50, 64, False), (3, 129, 129, 128, True), (2, 40, 200, 48, True),
                                   (2, 680, 680, 64, True), (1, 300, 420, 128, False), (1, 200, 300, 256, True),
                                   (2, 130, 260, 16, True), (3, 1, 300, 64, False), (1, 256, 256, 144, True),
                                   (2, 3, 200, 48, True), (1, 4, 1000, 128, True), (2, 2, 90, 256, False), (1, 1, 2500, 64, False),
                                   (1, 5, 140, 64, True), (2, 8, 77, 64, True), (3, 2, 33, 32, True)])
def test_qattention_matches_the_oracle_stage_by_stage(gpu, shape, bits, variant):
    """The composite call against the oracle's head: the output differs from the oracle's only through
    probability codes that sit on a rounding tie (each such code moves O by delta_p |Vq| s_v), so O is
    compared with the usual tolerance plus that allowance for a handful of flips per row. Both forms of
    the call are held to it: the one-kernel head (several chunks of 128 keys, query tiles with a ragged
    last one, head dimensions below, at and above one 128-byte block; with at most four queries the
    decode-step kernel, up to eight queries, which reads the cache once per group of four queries) and the three separate stages."""
    torch = gpu.torch
    G, Tq, Tk, d, causal = shape
    gpu.ctx.stwq_set_option(gpu.B.OPT_VARIANT, variant)
    try:
        _check_qattention(gpu, shape, bits)
    finally:
        gpu.ctx.stwq_set_option(gpu.B.OPT_VARIANT, 0)


def _check_qattention(gpu, shape, bits):
    torch = gpu.torch
    G, Tq, Tk, d, causal = shape
    P, Tmax = Tk + 3, (Tk + 15) // 16 * 16 + 16
    Q, K, V, s_q, s_k, s_v = _head_data(G, Tk, d, P)
    Q = Q[:, Tk - Tq:]                                    # the queries are the last Tq positions
    pos_q = np.arange(Tk - Tq, Tk, dtype=np.int32)
    pos_k = np.arange(Tk, dtype=np.int32)
    scale = np.float32(1.0 / np.sqrt(d))
    s_kcol = (s_k[pos_k] * scale).astype(np.float32)
    Kc = torch.zeros((G, Tmax, d), dtype=torch.int8, device=gpu.dev)
    Vt = torch.full((G, d, Tmax), 55, dtype=torch.int8, device=gpu.dev)      # stale codes beyond Tk must not matter
    gpu.ctx.kv_append(gpu.T(K), gpu.T(V), 0, gpu.T(s_k), gpu.T(s_v), bits, Kc, Vt)
    levels = 2 ** bits - 1
    for out, dt, rtol in (("fp32", torch.float32, 1e-5), ("bf16", torch.bfloat16, 1e-2)):
        O = torch.full((G, Tq, d), -3, dtype=dt, device=gpu.dev)
        gpu.ctx.qattention(gpu.T(Q), gpu.T(pos_q), Tk, Kc, Vt, gpu.T(s_q), gpu.T(s_kcol), gpu.T(s_v), bits, causal,
                           gpu.B.OUT_F32 if out == "fp32" else gpu.B.OUT_BF16, O)
        assert gpu.ctx.stwq_device_status() == 0
        got = O.float().cpu().numpy().astype(np.float64)
        for g in range(G):
            r = oracle.qattention(Q[g], K[g], V[g], pos_q, pos_k, s_q, s_k, s_v, scale, bits, causal)
            np.testing.assert_array_equal(Kc[g, :Tk].cpu().numpy(), r["Kq"])
            flip = 4 * (1.0 / levels) * (2 ** (bits - 1)) * s_v[None, :].astype(np.float64)     # four flipped codes per row
            tol = rtol * (np.abs(r["O"]) + r["mag"]) + flip
            assert (np.abs(got[g] - r["O"]) <= tol).all(), f"{out} head {g}: worst {np.abs(got[g] - r['O']).max()}"
            # and it is a sensible attention: close to the float head computed from the same inputs
        assert np.isfinite(got).all()


@pytest.mark.parametrize("shape", [(3, 333, 333, 64, True), (2, 100, 700, 96, False)])
def test_one_kernel_head_agrees_with_the_separate_stages(gpu, shape):
    """Same codes except on rounding ties: the outputs of the two forms differ by at most a few
    flipped probability codes per row, and most rows agree to the last rounding of the dequantizer."""
    torch = gpu.torch
    G, Tq, Tk, d, causal = shape
    P, Tmax = Tk, (Tk + 15) // 16 * 16
    Q, K, V, s_q, s_k, s_v = _head_data(G, Tk, d, P)
    Q = Q[:, Tk - Tq:]
    pos_q = np.arange(Tk - Tq, Tk, dtype=np.int32)
    s_kcol = (s_k[:Tk] * np.float32(1.0 / np.sqrt(d))).astype(np.float32)
    Kc = torch.zeros((G, Tmax, d), dtype=torch.int8, device=gpu.dev)
    Vt = torch.zeros((G, d, Tmax), dtype=torch.int8, device=gpu.dev)
    gpu.ctx.kv_append(gpu.T(K), gpu.T(V), 0, gpu.T(s_k), gpu.T(s_v), 8, Kc, Vt)
    outs = []
    for variant in (0, 9):
        gpu.ctx.stwq_set_option(gpu.B.OPT_VARIANT, variant)
        try:
            O = torch.full((G, Tq, d), -3, dtype=torch.float32, device=gpu.dev)
            gpu.ctx.qattention(gpu.T(Q), gpu.T(pos_q), Tk, Kc, Vt, gpu.T(s_q), gpu.T(s_kcol), gpu.T(s_v), 8, causal,
                               gpu.B.OUT_F32, O)
            outs.append(O.cpu().numpy().astype(np.float64))
        finally:
            gpu.ctx.stwq_set_option(gpu.B.OPT_VARIANT, 0)
    assert gpu.ctx.stwq_device_status() == 0
    diff = np.abs(outs[0] - outs[1])
    flip = (1.0 / 255) * 128 * s_v[None, None, :].astype(np.float64)          # one code moved by one step
    assert (diff <= 4 * flip + 1e-6 * np.abs(outs[1])).all()
    rows_equal = (diff <= 1e-6 * np.abs(outs[1]) + 1e-12).all(axis=2).mean()
    assert rows_equal > 0.9, rows_equal


@pytest.mark.parametrize("variant", [0, 9])
def test_qattention_refuses_bad_arguments_and_reports_bad_positions(gpu, variant):
    """Host-side refusals (more queries than keys under a causal mask, a head dimension that is no
    multiple of 16, keys beyond the cache) leave no launch behind; a query position outside the scale
    table is reported through the device status word, and the context stays usable."""
    torch = gpu.torch
    G, T, d, P, Tmax = 2, 40, 64, 40, 48
    Q, K, V, s_q, s_k, s_v = _head_data(G, T, d, P)
    s_kcol = (s_k[:T] / 8).astype(np.float32)
    Kc = torch.zeros((G, Tmax, d), dtype=torch.int8, device=gpu.dev)
    Vt = torch.zeros((G, d, Tmax), dtype=torch.int8, device=gpu.dev)
    gpu.ctx.kv_append(gpu.T(K), gpu.T(V), 0, gpu.T(s_k), gpu.T(s_v), 8, Kc, Vt)
    O = torch.zeros((G, T, d), dtype=torch.float32, device=gpu.dev)
    pos = np.arange(T, dtype=np.int32)
    gpu.ctx.stwq_set_option(gpu.B.OPT_VARIANT, variant)
    try:
        args = lambda Tk, causal, pos_q=pos, Qx=Q, Ox=O: (gpu.T(Qx), gpu.T(pos_q), Tk, Kc, Vt, gpu.T(s_q), gpu.T(s_kcol[:Tk]),
                                                          gpu.T(s_v), 8, causal, gpu.B.OUT_F32, Ox)
        with pytest.raises(Exception):
            gpu.ctx.qattention(*args(T - 8, True))                              # causal with Tq > Tk
        with pytest.raises(Exception):
            gpu.ctx.qattention(*args(Tmax + 16, False))                         # more keys than the cache holds
        Kc24 = torch.zeros((G, Tmax, 24), dtype=torch.int8, device=gpu.dev)
        with pytest.raises(Exception):
            gpu.ctx.qattention(gpu.T(Q[:, :, :24]), gpu.T(pos), T, Kc24, torch.zeros((G, 24, Tmax), dtype=torch.int8, device=gpu.dev),
                               gpu.T(s_q), gpu.T(s_kcol), gpu.T(s_v[:24]), 8, True, gpu.B.OUT_F32,
                               torch.zeros((G, T, 24), dtype=torch.float32, device=gpu.dev))
        assert gpu.ctx.stwq_device_status() == 0
        bad = pos.copy()
        bad[7] = P + 5
        gpu.ctx.qattention(*args(T, True, bad))
        assert gpu.ctx.stwq_device_status() == -8                               # STWQ_ERR_POS_RANGE, cleared by the read
        gpu.ctx.qattention(*args(T, True))
        assert gpu.ctx.stwq_device_status() == 0
        r = oracle.qattention(Q[0], K[0], V[0], pos, pos, s_q, s_k, s_v, np.float32(1 / 8), 8, True)
        got = O[0].cpu().numpy().astype(np.float64)
        flip = 4 * (1.0 / 255) * 128 * s_v[None, :].astype(np.float64)
        assert (np.abs(got - r["O"]) <= 1e-5 * (np.abs(r["O"]) + r["mag"]) + flip).all()
    finally:
        gpu.ctx.stwq_set_option(gpu.B.OPT_VARIANT, 0)


# ----------------------------------------------------------------------------- distribution-guided calibration
@pytest.mark.parametrize("shape", [(128, 64, 0.0), (41, 5, 0.0), (300, 257, 0.0), (6, 12, 1e-6), (64, 1, 0.0), (20, 20, 1e-9)])
def test_dgc_select_matches_the_oracle(gpu, shape):
    """Eq. 17 on the GPU: distances agree with the oracle to fp64 rounding, the kept set and its order
    are the oracle's (the data hold no near-equal distances except the planted duplicates, whose order
    is fixed by index)."""
    torch = gpu.torch
    n, D, ridge = shape
    F = (rng.standard_normal((n, D)) @ rng.standard_normal((D, D)) + rng.standard_normal(D)).astype(np.float32)
    if n > 10:
        F[5] = F[3]                                        # duplicates: equal distances, index order
        F[7] += 4.0
    rho_ref, sel_ref = oracle.dgc_select(F, 500000, ridge)
    rho = torch.zeros(n, dtype=torch.float64, device=gpu.dev)
    sel = torch.full((len(sel_ref),), -1, dtype=torch.int32, device=gpu.dev)
    gpu.ctx.dgc_select(gpu.T(F), 500000, ridge, rho, sel)
    assert gpu.ctx.stwq_device_status() == 0
    np.testing.assert_allclose(rho.cpu().numpy(), rho_ref, rtol=1e-8, atol=1e-12)
    np.testing.assert_array_equal(sel.cpu().numpy(), sel_ref)
    # sum of squared distances = n D when nothing is added to the covariance (trace identity)
    if ridge == 0.0 and D < n:
        assert abs(float((rho ** 2).sum()) - n * D) < 1e-7 * n * D


def test_dgc_degenerate_sets(gpu):
    torch = gpu.torch
    rho = torch.full((5,), 3.0, dtype=torch.float64, device=gpu.dev)
    gpu.ctx.dgc_select(gpu.T(np.ones((5, 3), np.float32)), 500000, 1e-6, rho)      # no variance at all
    assert (rho.cpu().numpy() == 0).all()
    wide = rng.standard_normal((6, 12)).astype(np.float32)                          # singular, no ridge
    gpu.ctx.dgc_select(gpu.T(wide), 500000, 0.0, rho.new_zeros(6))
    assert gpu.ctx.stwq_device_status() == 0
