"""The seeded input generators: counter based, reproducible, shaped like the five workloads."""
import numpy as np

import workloads as wl


def test_counter_based_slices_agree():
    a = wl.normals(7, wl.TAG_X, 0, 100000)
    b = wl.normals(7, wl.TAG_X, 54321, 1000)
    np.testing.assert_array_equal(a[54321:55321], b)
    assert abs(a.mean()) < 0.02 and abs(a.std() - 1) < 0.02
    assert not np.array_equal(a[:1000], wl.normals(8, wl.TAG_X, 0, 1000))
    assert not np.array_equal(a[:1000], wl.normals(7, wl.TAG_W, 0, 1000))


def test_config_shapes():
    M = {c: [(l.M, l.K, l.N) for l in wl.config_layers(c)] for c in range(1, 6)}
    assert M[1] == [(680, 1024, 1024)]
    assert M[2] == [(10880, 1024, 3072), (10880, 1024, 1024), (10880, 1024, 4096), (10880, 4096, 1024)]
    assert M[3] == [(21760, 1920, 5760), (21760, 1920, 1920), (21760, 1920, 7680), (21760, 7680, 1920)]
    assert M[4] == [(256, 2048, 8192), (256, 8192, 2048)]
    assert M[5] == [(65536, 1280, 5120), (65536, 5120, 1280)]


def test_activation_model():
    L = wl.scaled(wl.config_layers(1)[0], K=256, N=64)
    X, pos = wl.activations(L), wl.positions(L)
    assert X.shape == (680, 256) and X.dtype == np.float32 and pos.dtype == np.int32
    o = wl.outlier_factors(L)
    assert (o == 50).sum() == 3 and (o == 1).sum() == 253
    sig = wl.sigma_pos(L)
    assert sig.min() >= 0.5 and sig.max() <= 4.0
    # row slices reproduce the full tensor
    np.testing.assert_array_equal(wl.activations(L, rows=slice(100, 130)), X[100:130])
    # per-position profile is the same for calibration samples (position-invariant distribution)
    Xc, pc = wl.calibration(L, 8)
    ratio = np.abs(Xc[:, o == 1]).reshape(8, 680, -1).mean(axis=(0, 2)) / sig
    assert np.all(np.abs(ratio / np.sqrt(2 / np.pi) - 1) < 0.25)
    D = wl.config_layers(4)[0]
    assert len(set(wl.positions(D).tolist())) == 1 and wl.positions(D).size == 256
