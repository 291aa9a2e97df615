"""Seeded synthetic gradients shaped like the paper's workloads.

This module only draws inputs (numpy, CPU, fixed seeds) and picks the base ``b`` that
meets a keep-ratio target; it holds none of the method's arithmetic and imports neither
the CUDA binding nor the oracle, so that both can be fed the very same bits.

The paper trains sparse linear models on URL / KDD10 / KDD12 / WebSpam and an MLP on
MNIST (Sec. 4.1); none of those datasets is used here.  The generators below stand in
for them: dense DNN-sized gradients with per-layer scales, and a clustered-sparse
gradient of a sparse linear model.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

TAU = 128          # Sec. 4.2: recommended threshold, one byte per kept value
FLAG_BITS = 2      # Sec. 4.2: recommended length-flag size
GROUP_LOG2 = 14


def _rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([int(seed), int(stream), 0x2112_04291]))


def _block_bounds(n: int, blocks: int, layout_seed: int) -> np.ndarray:
    """Contiguous 'layer' blocks with heavy-tailed sizes (the real tensor shapes of the
    named networks are not available; sizes are a seeded random partition)."""
    r = _rng(layout_seed, 1000)
    w = np.exp(r.uniform(0.0, 6.0, blocks))
    sizes = np.maximum(1, np.floor(w / w.sum() * (n - blocks)).astype(np.int64) + 1)
    sizes[-1] += n - int(sizes.sum())
    assert sizes.min() >= 1 and int(sizes.sum()) == n
    return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)


def normal(n: int, seed: int = 0, sigma: float = 1e-3) -> np.ndarray:
    """config 1: i.i.d. N(0, sigma^2)."""
    v = _rng(seed).standard_normal(n, dtype=np.float32)
    v *= np.float32(sigma)
    return v


def student_t_layers(n: int, seed: int = 0, blocks: int = 161, df: float = 3.0,
                     lo: float = 1e-4, hi: float = 1e-1, layout_seed: int = 0) -> np.ndarray:
    """config 2: heavy-tailed values, Student-t(df) times a per-layer scale drawn
    log-uniformly in [lo, hi].  The layer layout and scales depend on `layout_seed`
    only (all simulated workers share the model), the values on `seed`."""
    bounds = _block_bounds(n, blocks, layout_seed)
    scales = np.exp(_rng(layout_seed, 1001).uniform(math.log(lo), math.log(hi), blocks))
    r = _rng(seed)
    v = np.empty(n, np.float32)
    step = 1 << 22
    for s in range(0, n, step):
        e = min(n, s + step)
        v[s:e] = r.standard_t(df, e - s).astype(np.float32)
    for i in range(blocks):
        v[bounds[i]:bounds[i + 1]] *= np.float32(scales[i])
    return v


def clustered_sparse(n: int, seed: int = 0, density: float = 1e-3, mean_run: float = 32.0,
                     scale: float = 1e-2) -> np.ndarray:
    """config 3: gradient of a sparse linear model: about density*n nonzeros placed in runs
    of Poisson(mean_run) consecutive indices at uniform starts (overlapping runs merge),
    values Laplace(0, scale), everything else exactly 0."""
    r = _rng(seed)
    v = np.zeros(n, np.float32)
    target = int(round(density * n))
    clusters = max(1, int(round(target / mean_run)))
    starts = r.integers(0, n, clusters)
    lens = r.poisson(mean_run, clusters)
    for s, ln in zip(starts.tolist(), lens.tolist()):
        e = min(n, s + ln)
        if e > s:
            v[s:e] = r.laplace(0.0, scale, e - s).astype(np.float32)
    return v


def normal_layers(n: int, seed: int = 0, blocks: int = 400, lo: float = 1e-5, hi: float = 1e-2,
                  layout_seed: int = 0) -> np.ndarray:
    """config 4: N(0, sigma_l^2) per layer block, sigma_l log-uniform in [lo, hi]."""
    bounds = _block_bounds(n, blocks, layout_seed)
    sig = np.exp(_rng(layout_seed, 1002).uniform(math.log(lo), math.log(hi), blocks))
    v = _rng(seed).standard_normal(n, dtype=np.float32)
    for i in range(blocks):
        v[bounds[i]:bounds[i + 1]] *= np.float32(sig[i])
    return v


def normal_outliers(n: int, seed: int = 0, sigma: float = 1e-3, frac: float = 0.01,
                    factor: float = 100.0) -> np.ndarray:
    """config 5: N(0, sigma^2) with a random `frac` of the entries multiplied by `factor`."""
    r = _rng(seed)
    v = r.standard_normal(n, dtype=np.float32)
    v *= np.float32(sigma)
    k = int(round(frac * n))
    if k:
        idx = r.integers(0, n, k)
        v[idx] *= np.float32(factor)
    return v


def base_for_keep(v: np.ndarray, keep: int, tau: int = TAU) -> float:
    """Harness-only choice of the base: the paper fixes b and tau and lets the kept count
    follow; the benchmark configs fix the kept count instead.  Since an entry survives iff
    |v| >= sum / b^tau, b = (sum / q)^(1/tau) with q the keep-th largest magnitude keeps
    about `keep` entries.  (A plain numpy sum is good enough to aim; the method's own sum
    is computed by the encoder.)"""
    a = np.abs(v)
    keep = int(max(1, min(keep, a.size)))
    q = float(np.partition(a, a.size - keep)[a.size - keep])
    s = float(a.sum(dtype=np.float64))
    if not (q > 0.0) or not (s > q):
        return 1.1
    b = (s / q) ** (1.0 / tau)
    return float(max(b, 1.0 + 1e-9))


def bases_for_keeps(v: np.ndarray, keeps, tau: int = TAU) -> list:
    """base_for_keep for several kept counts at once (one selection pass over |v|); the same values."""
    a = np.abs(v)
    ks = [int(max(1, min(int(k), a.size))) for k in keeps]
    a.partition(sorted(set(a.size - k for k in ks)))
    s = float(np.abs(v).sum(dtype=np.float64))
    out = []
    for k in ks:
        q = float(a[a.size - k])
        if not (q > 0.0) or not (s > q):
            out.append(1.1)
        else:
            out.append(float(max((s / q) ** (1.0 / tau), 1.0 + 1e-9)))
    return out


def _draw_workers(fn, n: int, seeds, threads: int) -> list:
    """One gradient per seed; with threads > 1 the workers are drawn side by side (numpy's generators
    release the interpreter lock), which changes nothing in the values."""
    if threads <= 1 or len(seeds) <= 1:
        return [fn(n, s) for s in seeds]
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=min(threads, len(seeds))) as ex:
        return list(ex.map(lambda s: fn(n, s), seeds))


@dataclass
class Workload:
    name: str
    n: int
    workers: int
    keep_fraction: float          # of n
    grads: list                   # one float32 array per worker
    base: float                   # one b per job (chosen on worker 0)
    tau: int = TAU
    flag_bits: int = FLAG_BITS
    group_log2: int = GROUP_LOG2


def make(name: str, n: int | None = None, workers: int | None = None, keep: float | None = None,
         seed: int = 0, threads: int = 1) -> Workload:
    """The five benchmark configurations (optionally at a reduced n for tests)."""
    if name == "c1":
        n = n or 1_048_576; workers = workers or 1; keep = keep if keep is not None else 0.01
        fn = normal
    elif name == "c2":
        n = n or 25_557_032; workers = workers or 4; keep = keep if keep is not None else 0.005
        fn = student_t_layers
    elif name == "c3":
        n = n or 50_000_000; workers = workers or 1
        fn = clustered_sparse
    elif name == "c4":
        n = n or 335_141_888; workers = workers or 8; keep = keep if keep is not None else 0.001
        fn = normal_layers
    elif name == "c5":
        n = n or (1 << 20); workers = workers or 1; keep = keep if keep is not None else 0.01
        fn = normal_outliers
    else:
        raise ValueError(name)
    grads = _draw_workers(fn, n, [seed + w for w in range(workers)], threads)
    if name == "c3":
        nnz = int(np.count_nonzero(grads[0]))
        kcount = (keep if keep is not None else 0.8) * nnz      # keep is a fraction of the nonzeros here
        keep = kcount / n
    else:
        kcount = keep * n
    b = base_for_keep(grads[0], int(round(kcount)))
    return Workload(name, n, workers, float(keep), grads, b)


def with_keeps(wl: Workload, keeps) -> list:
    """The same gradients at several keep ratios (fractions of n): one Workload per ratio, sharing the arrays."""
    bases = bases_for_keeps(wl.grads[0], [int(round(k * wl.n)) for k in keeps])
    return [Workload(wl.name, wl.n, wl.workers, float(k), wl.grads, b, wl.tau, wl.flag_bits, wl.group_log2)
            for k, b in zip(keeps, bases)]
