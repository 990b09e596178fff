"""Seeded synthetic inputs and shape tables for the synchronisation round.

This module serves the tests, the smoke check and the benchmark on both the
CPU-oracle side and the CUDA side.  It holds no arithmetic of the method: only
random draws, tensor shapes and the integer rule that turns a ratio into k.

The data stand in for the paper's workloads (ResNet-50 on ImageNet, softmax
regression on MNIST): only their shapes and structure are reproduced.
"""
import numpy as np


def k_from_ratio(d: int, num: int, den: int) -> int:
    """k = max(1, floor(d * num / den)) in integer arithmetic."""
    return max(1, (int(d) * int(num)) // int(den))


def resnet50_tensor_sizes():
    """Element counts of the 161 trainable tensors of ResNet-50, in definition order:
    conv1, bn1 (weight, bias), then the 16 bottleneck blocks (conv/bn triples, the
    first block of each stage followed by its downsample conv + bn), then fc weight
    and bias."""
    sizes = [64 * 3 * 7 * 7, 64, 64]
    inplanes = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            out = planes * 4
            sizes += [inplanes * planes, planes, planes,
                      planes * planes * 9, planes, planes,
                      planes * out, out, out]
            if b == 0:
                sizes += [inplanes * out, out, out]
            inplanes = out
    sizes += [2048 * 1000, 1000]
    return sizes


def segments_from_sizes(sizes):
    off = np.zeros(len(sizes) + 1, dtype=np.int64)
    off[1:] = np.cumsum(np.asarray(sizes, dtype=np.int64))
    return off


def k_per_tensor_ratio(sizes, num=1, den=1000):
    """Per-tensor k_t = max(1, floor(d_t * num / den))."""
    return np.asarray([k_from_ratio(n, num, den) for n in sizes], dtype=np.int64)


def k_per_tensor_capped(sizes, cap=1000):
    """The paper's ResNet-50 rule k_t = min(d_t, cap)."""
    return np.asarray([min(int(n), cap) for n in sizes], dtype=np.int64)


def scaled_sizes(sizes, factor):
    """A smaller table with the same structure: every tensor shrunk by `factor`
    (at least 1 element), used where the CPU oracle has to finish in seconds."""
    return [max(1, int(n) // int(factor)) for n in sizes]


def _rng(seed, stream):
    """Counter-based generator keyed by (seed, stream)."""
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def gaussian_round(R, d, seed=0, x_std=1.0, drift_std=1e-2, mem_std=1e-3):
    """Single-round inputs: x ~ N(0, x_std), xw_r = x + N(0, drift_std),
    mem_r ~ N(0, mem_std); the second parameters are standard deviations."""
    g = _rng(seed, 1)
    x = g.standard_normal(d, dtype=np.float32) * np.float32(x_std)
    xw = x[None, :] + g.standard_normal((R, d), dtype=np.float32) * np.float32(drift_std)
    mem = g.standard_normal((R, d), dtype=np.float32) * np.float32(mem_std)
    return x, np.ascontiguousarray(xw, dtype=np.float32), mem


def tensor_scales(nseg, seed=0, lo=1e-5, hi=1e-2):
    """Per-tensor drift scale, log-uniform in [lo, hi]."""
    g = _rng(seed, 2)
    return np.exp(g.uniform(np.log(lo), np.log(hi), nseg)).astype(np.float32)


def model_init(d, seed=0, std=0.05):
    g = _rng(seed, 3)
    return g.standard_normal(d, dtype=np.float32) * np.float32(std)


def laplace_drift(R, offsets, scales, seed, rnd):
    """Drift of every worker for one round: Laplace(0, b_t) inside tensor t."""
    g = _rng(seed, 4 + int(rnd))
    d = int(offsets[-1])
    per_elem = np.repeat(scales.astype(np.float32), np.diff(offsets))
    out = g.laplace(0.0, 1.0, (R, d)).astype(np.float32)
    out *= per_elem[None, :]
    return out


def gaussian_drift(R, d, seed, rnd, std=1e-3, outlier_frac=0.0, outlier_gain=100.0):
    """N(0, std) drift; a fraction of entries is multiplied by outlier_gain."""
    g = _rng(seed, 4 + int(rnd))
    out = g.standard_normal((R, d), dtype=np.float32) * np.float32(std)
    if outlier_frac > 0.0:
        hit = g.random((R, d), dtype=np.float32) < np.float32(outlier_frac)
        out[hit] *= np.float32(outlier_gain)
    return out


def gaussian_mixture(n, features, classes, seed=0, sigma=1.0, center_std=1.0):
    """n samples from `classes` Gaussian components (one per class), labels = component."""
    g = _rng(seed, 5)
    centers = g.standard_normal((classes, features), dtype=np.float32) * np.float32(center_std)
    labels = g.integers(0, classes, n).astype(np.int64)
    data = centers[labels] + g.standard_normal((n, features), dtype=np.float32) * np.float32(sigma)
    return data.astype(np.float32), labels


def split_by_class(labels, R):
    """Non-iid split: worker r owns the samples of the classes c with c % R == r."""
    return [np.nonzero(labels % R == r)[0] for r in range(R)]


def async_schedule(R, T, H, seed=0):
    """Per-worker synchronisation indicator (T x R, uint8): after each of its
    synchronisations a worker draws its next interval uniformly from 1..H, so
    every gap is at most H; all workers synchronise at the last step."""
    g = _rng(seed, 6)
    sched = np.zeros((T, R), dtype=np.uint8)
    for r in range(R):
        t = -1
        while True:
            t += int(g.integers(1, H + 1))
            if t >= T - 1:
                break
            sched[t, r] = 1
    sched[T - 1, :] = 1
    return sched
