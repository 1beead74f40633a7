"""Seeded synthetic inputs shaped like the linear layers of VAR / RAR / MAR decoders.

This module holds no arithmetic of the quantization method: it only produces
data (activations, weights, biases, position ids) that the tests and the
benchmark hand, unchanged, to both the CPU oracle and the GPU library.

Recipe. Activations follow the three properties the method relies on: a few
input channels carry outliers, the magnitude varies with the token position,
and that per-position profile is the same for every sample:

    X[m, k] = z * sigma_pos[pos[m]] * o[k],     z ~ N(0, 1)

where row m = sample * P + p sits at position p, sigma_pos is drawn once per
layer (uniform or log-normal), and o[k] is an outlier factor on a seeded subset
of channels and 1 elsewhere. Weights and biases are N(0, 0.02^2).

Host generator: counter based, so any element can be produced on its own:
u64 = splitmix64(seed * 2^44 + tag * 2^40 + index); two such words give two
24-bit uniforms, turned into a normal deviate by the Box-Muller transform in
double and rounded to fp32. For full-size layers the activations can instead be
drawn on the device with a seeded torch generator (the same statistical recipe;
rows the oracle needs are copied back).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

TAG_X, TAG_W, TAG_BIAS, TAG_SIGMA, TAG_OUTLIER, TAG_CALIB, TAG_POS = 1, 2, 3, 4, 5, 6, 7

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = x + np.uint64(0x9E3779B97F4A7C15)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def _key(seed: int, tag: int) -> np.uint64:
    return np.uint64(((seed & 0xFFFFF) << 44) | ((tag & 0xF) << 40))


def uniforms(seed: int, tag: int, start: int, count: int) -> np.ndarray:
    """count doubles in (0, 1), element i a function of (seed, tag, start + i) only."""
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        h = _splitmix64(_key(seed, tag) + idx)
    return ((h >> np.uint64(40)).astype(np.float64) + 0.5) / float(1 << 24)


def normals(seed: int, tag: int, start: int, count: int, chunk: int = 1 << 15) -> np.ndarray:
    """count N(0,1) deviates as fp32; element i depends on (seed, tag, start + i) only."""
    out = np.empty(count, np.float32)
    for c0 in range(0, count, chunk):
        n = min(chunk, count - c0)
        idx = np.arange(start + c0, start + c0 + n, dtype=np.uint64)
        with np.errstate(over="ignore"):
            h1 = _splitmix64(_key(seed, tag) + idx * np.uint64(2))
            h2 = _splitmix64(_key(seed, tag) + idx * np.uint64(2) + np.uint64(1))
        u1 = ((h1 >> np.uint64(40)).astype(np.float64) + 0.5) / float(1 << 24)
        u2 = ((h2 >> np.uint64(40)).astype(np.float64) + 0.5) / float(1 << 24)
        out[c0:c0 + n] = (np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)).astype(np.float32)
    return out


@dataclass(frozen=True)
class Layer:
    """One linear layer of a workload."""
    config: int            # 1..5, the workload family
    name: str
    batch: int             # samples per step
    P: int                 # token positions per sample
    K: int
    N: int
    bits: int = 8
    act: int = 0           # 0 none, 1 GELU (erf form), 2 GELU (tanh form)
    out_dtype: str = "bf16"
    sigma: tuple = ("uniform", 0.5, 4.0)   # or ("lognormal", 0.0, 1.0)
    outlier_frac: float = 0.01
    outlier_mult: float = 50.0
    use_gps: bool = True   # qkv / fc1 can absorb a per-channel scale; proj / fc2 run without
    decode: bool = False   # all rows of a step sit at one seeded position
    layer_index: int = 0

    @property
    def M(self) -> int:
        return self.batch if self.decode else self.batch * self.P

    @property
    def seed(self) -> int:
        return 1000 * self.config + self.layer_index

    @property
    def ops(self) -> float:
        return 2.0 * self.M * self.N * self.K


VAR_PYRAMID = (1, 4, 9, 16, 25, 36, 64, 100, 169, 256)   # 10 scales, 680 tokens
assert sum(VAR_PYRAMID) == 680


def config_layers(config: int, bits: int = 8, out_dtype: str | None = None):
    """The layers of workload family 1..5."""
    def mk(name, idx, batch, P, K, N, **kw):
        return Layer(config=config, name=name, batch=batch, P=P, K=K, N=N, bits=bits,
                     layer_index=idx, **kw)
    if config == 1:
        return [mk("single", 0, 1, 680, 1024, 1024, out_dtype=out_dtype or "fp32")]
    if config == 2:
        kw = dict(out_dtype=out_dtype or "bf16")
        return [mk("qkv", 0, 16, 680, 1024, 3072, **kw),
                mk("proj", 1, 16, 680, 1024, 1024, use_gps=False, **kw),
                mk("fc1", 2, 16, 680, 1024, 4096, act=1, **kw),
                mk("fc2", 3, 16, 680, 4096, 1024, use_gps=False, **kw)]
    if config == 3:
        kw = dict(out_dtype=out_dtype or "bf16", sigma=("lognormal", 0.0, 1.0),
                  outlier_frac=0.005, outlier_mult=100.0)
        return [mk("qkv", 0, 32, 680, 1920, 5760, **kw),
                mk("proj", 1, 32, 680, 1920, 1920, use_gps=False, **kw),
                mk("fc1", 2, 32, 680, 1920, 7680, **kw),
                mk("fc2", 3, 32, 680, 7680, 1920, use_gps=False, **kw)]
    if config == 4:
        kw = dict(out_dtype=out_dtype or "bf16", decode=True)
        return [mk("decodeA", 0, 256, 256, 2048, 8192, **kw),
                mk("decodeB", 1, 256, 256, 8192, 2048, use_gps=False, **kw)]
    if config == 5:
        kw = dict(out_dtype=out_dtype or "bf16", sigma=("uniform", 0.25, 8.0),
                  outlier_frac=0.02, outlier_mult=30.0)
        return [mk("fc1", 0, 256, 256, 1280, 5120, act=1, **kw),
                mk("fc2", 1, 256, 256, 5120, 1280, use_gps=False, **kw)]
    raise ValueError("config must be 1..5")


def scaled(layer: Layer, **kw) -> Layer:
    """A copy of a layer with some fields replaced (smaller batch, other bits, ...)."""
    d = {f: getattr(layer, f) for f in layer.__dataclass_fields__}
    d.update(kw)
    return Layer(**d)


# --------------------------------------------------------------------------- host data
def sigma_pos(layer: Layer) -> np.ndarray:
    u = uniforms(layer.seed, TAG_SIGMA, 0, layer.P)
    kind, a, b = layer.sigma
    if kind == "uniform":
        return (a + (b - a) * u).astype(np.float32)
    z = normals(layer.seed, TAG_SIGMA, 1 << 20, layer.P).astype(np.float64)
    return np.exp(a + b * z).astype(np.float32)


def outlier_factors(layer: Layer) -> np.ndarray:
    n_out = int(round(layer.outlier_frac * layer.K))
    o = np.ones(layer.K, np.float32)
    if n_out > 0:
        order = np.argsort(uniforms(layer.seed, TAG_OUTLIER, 0, layer.K), kind="stable")
        o[order[:n_out]] = layer.outlier_mult
    return o


def weights(layer: Layer) -> np.ndarray:
    return (0.02 * normals(layer.seed, TAG_W, 0, layer.N * layer.K)).reshape(layer.N, layer.K)


def bias(layer: Layer) -> np.ndarray:
    return 0.02 * normals(layer.seed, TAG_BIAS, 0, layer.N)


def decode_position(layer: Layer, step: int = 0) -> int:
    return int(uniforms(layer.seed, TAG_POS, step, 1)[0] * layer.P) % layer.P


def positions(layer: Layer, step: int = 0) -> np.ndarray:
    """pos_ids of one step: sample-major rows, or one shared position for decode."""
    if layer.decode:
        return np.full(layer.M, decode_position(layer, step), np.int32)
    return np.tile(np.arange(layer.P, dtype=np.int32), layer.batch)


def _rows(layer: Layer, tag: int, pos: np.ndarray, row0: int) -> np.ndarray:
    M = pos.size
    z = normals(layer.seed, tag, row0 * layer.K, M * layer.K).reshape(M, layer.K)
    return z * sigma_pos(layer)[pos][:, None] * outlier_factors(layer)[None, :]


def activations(layer: Layer, step: int = 0, rows: slice | None = None) -> np.ndarray:
    """X of one step on the host ([M, K] fp32), or a row slice of it."""
    pos = positions(layer, step)
    base = step * layer.M
    if rows is None:
        return _rows(layer, TAG_X, pos, base)
    r0 = rows.start or 0
    return _rows(layer, TAG_X, pos[rows], base + r0)


def calibration(layer: Layer, samples: int = 32):
    """Calibration set: `samples` full sequences. Returns (X [samples*P, K], pos_ids)."""
    pos = np.tile(np.arange(layer.P, dtype=np.int32), samples)
    return _rows(layer, TAG_CALIB, pos, 0), pos


def gps_rows(Xcal: np.ndarray, n: int = 256) -> np.ndarray:
    """An evenly strided subset of calibration rows for the GPS scale computation."""
    if Xcal.shape[0] <= n:
        return Xcal
    idx = np.linspace(0, Xcal.shape[0] - 1, n).astype(np.int64)
    return np.ascontiguousarray(Xcal[idx])


# --------------------------------------------------------------------------- device data
def activations_device(layer: Layer, device, step: int = 0):
    """X of one step drawn on the device (same recipe, torch's seeded generator).

    Returns (X [M,K] fp32 cuda tensor, pos_ids int32 cuda tensor). Used where the
    layer is too large to generate on the host in reasonable time; the rows the
    oracle needs are copied back from this tensor.
    """
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(layer.seed * 1000003 + step)
    pos = torch.from_numpy(positions(layer, step)).to(device)
    sig = torch.from_numpy(sigma_pos(layer)).to(device)
    o = torch.from_numpy(outlier_factors(layer)).to(device)
    X = torch.randn(layer.M, layer.K, device=device, dtype=torch.float32, generator=g)
    X.mul_(sig[pos.long()][:, None]).mul_(o[None, :])
    return X, pos
