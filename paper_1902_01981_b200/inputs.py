"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU checker.

Only random draws and data movement live here -- none of the arithmetic of the
aggregation scheme.  Everything is generated on the host with NumPy's
`Generator(PCG64(seed))` and handed, as data, to whoever consumes it.

The value models follow the synthetic linear-regression recipe of the paper's
Section V (features and true model Gaussian, labels = features . model + Gaussian
noise); the aggregation-only workloads use Gaussian partition gradients, and the
integer mode uses uniform integers.
"""
from __future__ import annotations

import numpy as np


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def partition_gradients(P: int, d: int, seed: int, std: float = 1.0) -> np.ndarray:
    """One fp32 gradient vector per atomic data partition, N(0, std^2), shape [P, d]."""
    g = _rng(seed).standard_normal((P, d), dtype=np.float32)
    if std != 1.0:
        g *= np.float32(std)
    return g


def integer_gradients(P: int, d: int, seed: int, bound: int = 1 << 10) -> np.ndarray:
    """One int32 gradient vector per partition, uniform in [-bound, bound]."""
    return _rng(seed).integers(-bound, bound + 1, size=(P, d), dtype=np.int32)


def linreg_partitions(P: int, rows: int, d: int, seed: int, x_std: float = 1.0,
                      noise_std: float = 0.01):
    """P partitions of a linear-regression data set.

    Returns (X [P, rows, d] fp32 ~ N(0, x_std^2), y [P, rows] fp32, w_star [d] fp32)
    with y = X w_star + noise_std * N(0, 1), the products formed in fp64 and
    rounded once to fp32.
    """
    rng = _rng(seed)
    w_star = rng.standard_normal(d, dtype=np.float32)
    X = rng.standard_normal((P, rows, d), dtype=np.float32)
    if x_std != 1.0:
        X *= np.float32(x_std)
    noise = rng.standard_normal((P, rows), dtype=np.float32)
    y = np.empty((P, rows), dtype=np.float32)
    for p in range(P):
        y[p] = (X[p].astype(np.float64) @ w_star.astype(np.float64)
                + noise_std * noise[p].astype(np.float64)).astype(np.float32)
    return X, y, w_star


def logistic_partitions(P: int, rows: int, d: int, seed: int, x_std: float = 1.0):
    """P partitions of a two-class data set: X [P, rows, d] fp32 ~ N(0, x_std^2), labels y [P, rows]
    in {0, 1} drawn with probability 1 / (1 + exp(-x . w_star)), w_star [d] fp32 ~ N(0, I)."""
    rng = _rng(seed)
    w_star = rng.standard_normal(d, dtype=np.float32)
    X = rng.standard_normal((P, rows, d), dtype=np.float32)
    if x_std != 1.0:
        X *= np.float32(x_std)
    u = rng.random((P, rows))
    y = np.empty((P, rows), dtype=np.float32)
    for p in range(P):
        z = X[p].astype(np.float64) @ w_star.astype(np.float64)
        y[p] = (u[p] < 1.0 / (1.0 + np.exp(-z))).astype(np.float32)
    return X, y, w_star


def model_vector(d: int, seed: int) -> np.ndarray:
    """A start model w_0 ~ N(0, I), fp32."""
    return _rng(seed).standard_normal(d, dtype=np.float32)


def model_matrix(K: int, d: int, seed: int, spread: float = 0.1) -> np.ndarray:
    """K models around one start model, as a line search or an ensemble would hold them:
    W[k] = w_0 + spread * N(0, I), fp32, shape [K, d]."""
    rng = _rng(seed)
    w0 = rng.standard_normal(d, dtype=np.float32)
    return (w0[None, :] + np.float32(spread) * rng.standard_normal((K, d), dtype=np.float32)).astype(np.float32)


def tf32_representable(x: np.ndarray) -> np.ndarray:
    """Rounds fp32 values to the nearest value with a 10-bit mantissa (TF32), returned as fp32: the low
    13 mantissa bits are zero, so a tensor core reads these numbers without loss."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (bits + np.uint32(0x1000)) & np.uint32(0xFFFFE000)
    return rounded.view(np.float32)


def group_count(n: int, L: int) -> int:
    """Sibling groups of an (n, L) tree: one per parent, the master included."""
    return sum(n ** l for l in range(L))


def straggler_masks(n: int, L: int, s: int, batch: int, seed: int,
                    exactly_s: bool = False) -> np.ndarray:
    """Random straggler patterns, shape [batch, groups], dtype uint32.

    Bit j of masks[b, g] marks child j of sibling group g as a straggler.  Per
    group the number of stragglers is s (exactly_s) or uniform on {0..s}; the
    straggling children are a uniform subset of that size.
    """
    rng = _rng(seed)
    groups = group_count(n, L)
    masks = np.zeros((batch, groups), dtype=np.uint32)
    for b in range(batch):
        for g in range(groups):
            k = s if exactly_s else int(rng.integers(0, s + 1))
            chosen = rng.choice(n, size=k, replace=False) if k else []
            bits = 0
            for j in chosen:
                bits |= 1 << int(j)
            masks[b, g] = bits
    return masks


def shifted_exponential_times(count: int, load_points: float, a: float, mu: float, seed: int, trials: int = 1):
    """Computation times T with P[T <= t] = 1 - exp(-(mu / d_i)(t - a d_i)), t >= a d_i, for d_i =
    load_points data points per worker; shape [trials, count], float64."""
    return a * load_points + _rng(seed).exponential(load_points / mu, size=(trials, count))


def replicate_into_slots(G_parts: np.ndarray, slot_partition: np.ndarray) -> np.ndarray:
    """Copy partition gradients into per-node slots: out[v, j] = G_parts[slot_partition[v, j]].

    Every node that holds a partition computes the same gradient for it, so the
    slot buffer of an aggregation-only workload is this gather (pure data
    movement; `slot_partition` comes from whoever planned the allocation).
    """
    return G_parts[np.asarray(slot_partition, dtype=np.int64)]


# Benchmark workloads.  Tree shape, partition count, gradient length and value model of each; no
# arithmetic of the scheme.  `code` names the encoding-matrix family ("printed_3_1": the matrices the
# paper prints for n=3, s=1; "cyclic": random cyclic-support code; "repetition": 0/1 fractional
# repetition).  `P` of cfg3 is 48, the nearest count above the nominal 40 that the (4,2,1) tree can
# split into whole chunks.
CONFIGS = {
    "cfg1": dict(n=3, L=1, s=1, P=6, d=256, rows=64, code="printed_3_1", kind="linreg", x_std=1.0,
                 noise_std=0.01, iters=10, lr=5e-4, seed=0),
    "cfg2": dict(n=4, L=2, s=1, P=24, d=1 << 20, code="cyclic", kind="aggregate", std=1.0, iters=100,
                 batch=1, exactly_s=False, seed=0, mask_seed=1),
    "cfg3": dict(n=4, L=2, s=1, P=48, d=4096, rows=2048, code="cyclic", kind="linreg", x_std=1.0 / 64.0,
                 noise_std=0.01, iters=50, lr=0.1, seed=0, mask_seed=1),
    "cfg4": dict(n=5, L=2, s=2, P=40, d=1 << 24, code="cyclic", kind="aggregate", std=1e-3 ** 0.5, iters=20,
                 batch=1, exactly_s=True, seed=0, mask_seed=1),
    "cfg5": dict(n=3, L=4, s=1, P=195, d=1 << 22, code="printed_3_1", kind="aggregate", std=1.0, iters=5,
                 batch=64, exactly_s=False, seed=0, mask_seed=1, int_bound=1 << 10),
    # shaped like the paper's logistic-regression run: 6552 samples, p = 5001 (padded to 5004 so that rows
    # are 16-byte multiples), (12,2) tree with one straggler per group: 168 partitions of 39 samples
    "cfg_logit": dict(n=12, L=2, s=1, P=168, d=5004, rows=39, code="cyclic", kind="logistic", x_std=1.0 / 70.0,
                      iters=20, lr=0.5, seed=0, mask_seed=1),
    # the trees of the paper's clusters at a large gradient: (12,2) = 156 workers (stated for CR) and
    # (4,3) = 84 workers (the only regular tree with 84 nodes), one straggler per sibling group
    "cfg_tree12": dict(n=12, L=2, s=1, P=168, d=1 << 22, code="cyclic", kind="aggregate", std=1.0, iters=20,
                       batch=1, exactly_s=True, seed=0, mask_seed=1),
    "cfg_tree43": dict(n=4, L=3, s=1, P=112, d=1 << 22, code="cyclic", kind="aggregate", std=1.0, iters=20,
                       batch=1, exactly_s=True, seed=0, mask_seed=1),
    # shaped like the paper's CNN run: p ~ 1.2e5 parameters, (12,2) tree, 5 of 12 children straggling in
    # every group; (s+1) | n, so the 0/1 fractional repetition code exists (m = 36 slots per node)
    "cfg_cnn": dict(n=12, L=2, s=5, P=216, d=120000, code="repetition", kind="aggregate", std=1.0, iters=20,
                    batch=1, exactly_s=True, seed=0, mask_seed=1, int_bound=1 << 10),
    "cfg_rep": dict(n=4, L=2, s=1, P=24, d=1 << 20, code="repetition", kind="aggregate", std=1.0, iters=20,
                    batch=1, exactly_s=False, seed=0, mask_seed=1, int_bound=1 << 10),
}
