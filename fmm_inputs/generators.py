"""Counter-based synthetic operand and gauge generators (no arithmetic of the method).

Recipe (stands in for the LLM linear-layer workloads the paper measures on; the models
and datasets themselves are not used):
  * every element is hash(seed, tensor id, flat index) -> uniform -> Box-Muller normal;
  * activations A: N(0,1) or Student-t(3), with a seeded choice of K-columns multiplied
    by a large factor ("outlier channels");
  * weights B: N(0, 0.02^2);
  * integer matrices: uniform integers in [-b, b] (exactness domain);
  * gauge matrices: N(0,1) entries, either rejected above a condition-number limit or
    re-conditioned to a log-uniform condition number through their SVD.
"""
from __future__ import annotations

import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on uint64 arrays (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        z = (z + _GOLD)
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def _key(seed: int, tid: int, stream: int) -> np.uint64:
    k = _mix(np.array([np.uint64(seed & 0xFFFFFFFFFFFFFFFF)], dtype=np.uint64))
    k = _mix(k ^ np.uint64(tid * 0x632BE59BD9B4E019 & 0xFFFFFFFFFFFFFFFF))
    k = _mix(k ^ np.uint64(stream * 0xD1342543DE82EF95 & 0xFFFFFFFFFFFFFFFF))
    return k[0]


def _bits(seed: int, tid: int, stream: int, start: int, count: int) -> np.ndarray:
    idx = np.arange(start, start + count, dtype=np.uint64)
    with np.errstate(over="ignore"):
        return _mix(idx * _GOLD ^ _key(seed, tid, stream))


def _uniform_flat(seed, tid, stream, start, count):
    """U[0,1) with 53 random bits."""
    return (_bits(seed, tid, stream, start, count) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


_CHUNK = 1 << 22


def _fill(shape, fn):
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float64)
    for s in range(0, n, _CHUNK):
        c = min(_CHUNK, n - s)
        out[s:s + c] = fn(s, c)
    return out.reshape(shape)


def uniform(seed: int, tid: int, shape, lo: float = 0.0, hi: float = 1.0, stream: int = 0) -> np.ndarray:
    return _fill(shape, lambda s, c: lo + (hi - lo) * _uniform_flat(seed, tid, stream, s, c))


def _normal_flat(seed, tid, stream, s, c):
    u1 = 1.0 - _uniform_flat(seed, tid, 2 * stream, s, c)       # (0,1]
    u2 = _uniform_flat(seed, tid, 2 * stream + 1, s, c)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def normal(seed: int, tid: int, shape, std: float = 1.0, stream: int = 0) -> np.ndarray:
    """N(0, std^2) by Box-Muller on two hashed uniforms per element."""
    return _fill(shape, lambda s, c: std * _normal_flat(seed, tid, stream, s, c))


def student_t3(seed: int, tid: int, shape) -> np.ndarray:
    """Student-t with 3 degrees of freedom: Z / sqrt((Z1^2+Z2^2+Z3^2)/3)."""
    def f(s, c):
        z = _normal_flat(seed, tid, 0, s, c)
        q = sum(_normal_flat(seed, tid, 1 + i, s, c) ** 2 for i in range(3))
        return z / np.sqrt(q / 3.0)
    return _fill(shape, f)


def outlier_columns(seed: int, tid: int, K: int, count: int) -> np.ndarray:
    """`count` distinct columns of K chosen by a seeded shuffle (smallest hashed keys)."""
    keys = _bits(seed, tid, 99, 0, K)
    return np.sort(np.argsort(keys, kind="stable")[:count])


def activations_outlier(seed: int, tid: int, M: int, K: int, dist: str = "normal",
                        frac: float = 0.005, factor: float = 100.0, at_least: int = 0) -> np.ndarray:
    """Activations with outlier channels: floor(frac*K) (at least `at_least`) K-columns,
    chosen by seed, multiplied by `factor`."""
    A = normal(seed, tid, (M, K)) if dist == "normal" else student_t3(seed, tid, (M, K))
    cnt = max(int(at_least), int(np.floor(frac * K)))
    if cnt > 0:
        cols = outlier_columns(seed, tid, K, cnt)
        A[:, cols] *= factor
    return A


def weights(seed: int, tid: int, K: int, N: int, std: float = 0.02) -> np.ndarray:
    """Weights N(0, std^2), returned as the K x N operand B."""
    return normal(seed, tid, (K, N), std=std)


def integer_matrix(seed: int, tid: int, shape, bound: int) -> np.ndarray:
    """Uniform integers in [-bound, bound] as float64."""
    u = uniform(seed, tid, shape)
    return np.floor(u * (2 * bound + 1)) - bound


def to_storage(x: np.ndarray, dtype: str):
    """Round an fp64 array to the storage dtype ('f32' | 'bf16').  Returns (torch CPU tensor of
    that dtype, fp64 numpy array holding exactly the stored values)."""
    import torch
    td = {"f32": torch.float32, "bf16": torch.bfloat16}[dtype]
    t = torch.from_numpy(np.ascontiguousarray(x)).to(td)
    return t, t.to(torch.float64).numpy()


def _gauss_matrix(seed: int, tid: int, d: int, attempt: int) -> np.ndarray:
    return normal(seed, tid, (d, d), stream=7 + attempt)


def gauge_cond_limited(seed: int, index: int, d: int, limit: float = 10.0) -> np.ndarray:
    """d x d matrix with N(0,1) entries, redrawn until its 2-norm condition number <= limit."""
    for attempt in range(10000):
        G = _gauss_matrix(seed, 1000 + index, d, attempt)
        if np.linalg.cond(G, 2) <= limit:
            return G
    raise RuntimeError("no well-conditioned draw")


def gauge_log_uniform_cond(seed: int, index: int, d: int, lo: float = 1.0, hi: float = 1e3) -> np.ndarray:
    """d x d matrix with the singular vectors of an N(0,1) draw and singular values spaced
    geometrically from kappa^(1/2) to kappa^(-1/2), kappa log-uniform in [lo, hi)."""
    G = _gauss_matrix(seed, 2000 + index, d, 0)
    X, _, Yt = np.linalg.svd(G)
    u = float(uniform(seed, 3000 + index, (1,))[0])
    kappa = lo * (hi / lo) ** u
    expo = np.linspace(0.5, -0.5, d)
    return X @ np.diag(kappa ** expo) @ Yt


# Shapes of the five benchmark configurations (scheme, storage/product/output dtypes, sizes).
WORKLOADS = {
    "c1": dict(scheme="strassen222", S="f32", Pd="bf16", O="f32", M=256, K=256, N=256, gauges=8),
    "c2": dict(scheme="strassen444", S="bf16", Pd="bf16", O="bf16", M=4096, K=4096, N=4096,
               outlier_frac=0.005, outlier_factor=100.0),
    "c3": dict(scheme="strassen222", S="bf16", Pd="bf16", O="bf16", M=2048, K=4096, N=4096,
               outlier_frac=0.005, outlier_factor=100.0, gauges=512),
    "c4": dict(scheme="strassen444", S="bf16", Pd="e4m3", O="bf16", T=2048,
               gemms=[(4096, 12288), (4096, 4096), (4096, 22016), (11008, 4096)],
               outlier_frac=0.001, outlier_factor=300.0, dist="t3"),
    "c5": dict(scheme="strassen444", S="bf16", Pd=("bf16", "e4m3"), O="bf16", T=8192,
               gemms=[(5120, 15360), (5120, 27648), (13824, 5120)],
               outlier_frac=0.001, outlier_factor=300.0, dist="t3", gauges=512, gauge_level="outer"),
}
