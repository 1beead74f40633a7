"""qlinear_static, the entry point for hosts that cannot allocate device memory (its scratch is
a fixed array inside the library image), must give what qlinear gives.

Collected last on purpose: a run that stops at the first failure has then already executed every
other test. The test does not depend on what ran before it: it works in a fresh process, where
its first call performs the one-time per-device set-up, and after the other GPU tests, where the
shared scratch array still holds whatever an earlier call left there.
"""
import numpy as np
import pytest

import oracle
import workloads as wl
from layer_setup import assert_close, prepare

pytestmark = pytest.mark.gpu


def test_qlinear_static_matches_qlinear_twice_in_a_row():
    import torch

    import paper_2601_21238_b200 as pk
    from paper_2601_21238_b200 import build as pkbuild
    pkbuild.build()
    dev = torch.device("cuda:0")
    T = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    ctx = pk.Context(0)
    try:
        # two different problems back to back, so the second call finds the first one's codes in
        # the shared scratch: ragged 333 x 400 -> 328 with GELU, then config 1 (680 x 1024 -> 1024)
        cases = [wl.scaled(wl.config_layers(1)[0], K=400, N=328, P=37, batch=9, bits=6, act=1),
                 wl.config_layers(1)[0]]
        for L in cases:
            par = prepare(L, samples=4, gps_n=64)
            X, pos = wl.activations(L), wl.positions(L)
            ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"],
                                 L.bits, L.act)
            d = {k: T(par[k]) for k in ("Wq", "s_w", "s_tok", "s_ch", "bias")}
            Xd, pd = T(X), T(pos)
            for out, dt, rtol in ((pk.OUT_INT32, torch.int32, None), (pk.OUT_F32, torch.float32, 1e-5),
                                  (pk.OUT_BF16, torch.bfloat16, 1e-2)):
                want = torch.full((L.M, L.N), -3, dtype=dt, device=dev)
                ctx.stwq_set_option(1, 1)            # the tiled GEMM, which is what qlinear_static runs
                ctx.qlinear(Xd, pd, d["Wq"], d["s_w"], d["s_tok"], d["s_ch"], d["bias"], L.bits, L.act, out, want)
                ctx.stwq_set_option(1, 0)
                assert ctx.stwq_device_status() == 0
                for _ in range(2):                   # two calls in a row
                    got = torch.full((L.M, L.N), -5, dtype=dt, device=dev)
                    pk.qlinear_static(Xd, pd, d["Wq"], d["s_w"], d["s_tok"], d["s_ch"], d["bias"], L.bits,
                                      L.act, out, got)
                    torch.cuda.synchronize()
                    if rtol is None:
                        assert torch.equal(got, want)
                        np.testing.assert_array_equal(got.cpu().numpy(), ref["acc"])
                    else:
                        # same kernels, same inputs: the two entry points agree to the last bit,
                        # and both sit inside the tolerance of the other parity tests
                        assert torch.equal(got, want)
                        assert_close(got.float().cpu().numpy(), ref, rtol, f"qlinear_static {L.name}")
        # a shape for which qlinear cuts its two tiles along K and exchanges partial sums through
        # scratch that its context allocates: qlinear_static must give the same bits without it,
        # and the device's free memory must not move across its calls (after one warm-up call,
        # which loads the kernel's code)
        L2 = wl.scaled(wl.config_layers(1)[0], K=4096, N=512, P=64, batch=4, bits=8, act=0)
        assert L2.M * L2.K <= pk.binding.STATIC_MAX_CODES
        par = prepare(L2, samples=2, gps_n=32)
        X, pos = wl.activations(L2), wl.positions(L2)
        ref = oracle.qlinear(X, pos, par["Wq"], par["s_w"], par["s_tok"], par["s_ch"], par["bias"], L2.bits, L2.act)
        d2 = {k: T(par[k]) for k in ("Wq", "s_w", "s_tok", "s_ch", "bias")}
        Xd, pd = T(X), T(pos)
        got = torch.full((L2.M, L2.N), -5, dtype=torch.int32, device=dev)
        args = (Xd, pd, d2["Wq"], d2["s_w"], d2["s_tok"], d2["s_ch"], d2["bias"], L2.bits, L2.act, pk.OUT_INT32, got)
        pk.qlinear_static(*args)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info(0)[0]
        for _ in range(3):
            pk.qlinear_static(*args)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info(0)[0] == free_before
        np.testing.assert_array_equal(got.cpu().numpy(), ref["acc"])
        # a problem larger than the fixed scratch is refused on the host, nothing is enqueued
        big_M = pk.binding.STATIC_MAX_CODES // 1024 + 1
        Xb = torch.zeros((big_M, 1024), device=dev)
        pb = torch.zeros(big_M, dtype=torch.int32, device=dev)
        Yb = torch.zeros((big_M, 1024), device=dev)
        L = cases[1]
        with pytest.raises(pk.StwqError) as ei:
            pk.qlinear_static(Xb, pb, d["Wq"], d["s_w"], d["s_tok"], None, None, 8, 0, pk.OUT_F32, Yb)
        assert ei.value.code == -2
    finally:
        ctx.close()
