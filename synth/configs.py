"""Seeded synthetic workloads shaped like the paper's (flat fp32 gradients of tens
of workers, replication about 2-5). Used by both the oracle-side tests and the
CUDA-side tests / benchmark. This module holds NO arithmetic of the method:
no code construction, no bit allocation, no quantiser. Quantities the method
derives (code weights, allocated bits) are obtained by the caller.

The five workloads stand in for the paper's COCO / MobileNetV3 / ResNet-50 /
GPT-2-scale experiments (Sec. VI): only their shapes are taken.
"""
from dataclasses import dataclass, field

import numpy as np


@dataclass
class Workload:
    name: str
    n: int                 # workers
    k: int                 # partitions
    s: int                 # cyclic replication: worker i holds partitions i..i+s-1 (mod k)
    d: int                 # coordinates
    p: np.ndarray          # straggler probabilities, float64 [n]
    rounds: int
    seed: int
    value_model: str       # how the partial gradients are drawn
    bits: np.ndarray = None        # given bits, or None when they come from the allocator
    z_tot: int = 0                 # allocator budget when bits is None
    bits_range: tuple = (2, 8)
    realizations: int = 1          # straggler realisations decoded per encode
    extra: dict = field(default_factory=dict)


def _rng(seed, stream):
    return np.random.default_rng(np.random.SeedSequence([int(seed), int(stream)]))


def config1(seed=1):
    return Workload("cfg1", n=4, k=4, s=2, d=10_000, p=np.array([0.1, 0.2, 0.3, 0.4]),
                    rounds=100, seed=seed, value_model="normal",
                    bits=np.array([2, 3, 4, 8], np.uint8))


def config2(seed=2, d=1 << 20):
    r = _rng(seed, 0)
    return Workload("cfg2", n=16, k=16, s=3, d=d, p=r.uniform(0.05, 0.5, 16), rounds=1000,
                    seed=seed, value_model="partition_scale", z_tot=64, bits_range=(2, 8))


def config3(seed=3, d=25_557_032):
    p = np.repeat([0.02, 0.1, 0.3], [11, 11, 10]).astype(np.float64)
    return Workload("cfg3", n=32, k=32, s=4, d=d, p=p, rounds=200, seed=seed,
                    value_model="segments", z_tot=128, bits_range=(2, 8),
                    extra={"segments": 161})


def config4(seed=4, rows=1 << 20, features=4096):
    r = _rng(seed, 0)
    return Workload("cfg4", n=64, k=64, s=2, d=features, p=r.uniform(0.0, 0.4, 64), rounds=500,
                    seed=seed, value_model="least_squares",
                    bits=r.integers(2, 7, 64).astype(np.uint8),
                    extra={"rows": rows, "noise": 0.01})


def config5(seed=5, d=100_000_000):
    r = _rng(seed, 0)
    return Workload("cfg5", n=100, k=100, s=5, d=d, p=r.uniform(0.01, 0.6, 100), rounds=1,
                    seed=seed, value_model="student_t3",
                    bits=r.integers(1, 9, 100).astype(np.uint8), realizations=64)


def shifted_exponential_probs(n, seed=0, psi_range=(0.1, 2.0), tau_th=1.1):
    """Straggler probabilities of the paper's delay model (Sec. V-A / VI): worker i has rate
    psi_i ~ U(psi_range) and misses the deadline tau_th with p_i = exp(-psi_i (tau_th - 1))."""
    psi = _rng(seed, 21).uniform(psi_range[0], psi_range[1], n)
    return np.exp(-psi * (tau_th - 1.0))


def cyclic_support(wl):
    """Column lists of the cyclic assignment (sorted ascending)."""
    return [sorted(((i + t) % wl.k) for t in range(wl.s)) for i in range(wl.n)]


def straggler_masks(wl, rounds=None, realizations=None, stream=7):
    """uint8 [rounds, realizations, n]; 1 = the worker's message arrived.
    Independent Bernoulli(1 - p_i) draws (the paper's straggler model, Sec. II-A)."""
    rounds = wl.rounds if rounds is None else rounds
    realizations = wl.realizations if realizations is None else realizations
    r = _rng(wl.seed, stream)
    u = r.random((rounds, realizations, wl.n))
    return (u >= wl.p[None, None, :]).astype(np.uint8)


def segment_table(wl):
    """cfg3: 161 contiguous segments; lengths from seeded log-uniform weights
    normalised to d; per-segment std log-uniform in [1e-4, 1e-1]."""
    nseg = wl.extra["segments"]
    r = _rng(wl.seed, 11)
    wts = 10.0 ** r.uniform(0.0, 3.0, nseg)
    cuts = np.floor(np.cumsum(wts) / wts.sum() * wl.d).astype(np.int64)
    cuts[-1] = wl.d
    starts = np.concatenate([[0], cuts[:-1]])
    sigma = 10.0 ** r.uniform(-4.0, -1.0, nseg)
    return starts, cuts, sigma


def partition_scales(wl):
    """cfg2: per-partition scale log-uniform in [1e-3, 1]."""
    return 10.0 ** _rng(wl.seed, 12).uniform(-3.0, 0.0, wl.k)


def partials_numpy(wl, round_index=0, d=None):
    """k x d float32 partial gradients on the host (small workloads / slices)."""
    d = wl.d if d is None else d
    r = _rng(wl.seed, 1000 + round_index)
    if wl.value_model in ("normal", "least_squares"):
        # least_squares (cfg4): the partial gradients proper come from the harness's regression
        # problem on the device; host-side samples of that shape are standard normal
        return r.standard_normal((wl.k, d), dtype=np.float32)
    if wl.value_model == "partition_scale":
        g = r.standard_normal((wl.k, d), dtype=np.float32)
        return g * partition_scales(wl).astype(np.float32)[:, None]
    if wl.value_model == "segments":
        g = r.standard_normal((wl.k, d), dtype=np.float32)
        starts, ends, sigma = segment_table(wl)
        scale = np.empty(d, np.float32)
        for a, b, sg in zip(starts, ends, sigma):
            a2, b2 = min(a, d), min(b, d)
            scale[a2:b2] = sg
        return g * scale[None, :]
    if wl.value_model == "student_t3":
        z = r.standard_normal((wl.k, d), dtype=np.float32)
        chi = (r.standard_normal((3, wl.k, d), dtype=np.float32) ** 2).sum(axis=0)
        return (z / np.sqrt(chi / 3.0)).astype(np.float32)
    raise ValueError(wl.value_model)


def partials_torch(wl, device, round_index=0, d=None, ld=None, out=None):
    """k x d float32 partial gradients generated in place on a torch device
    (row by row, so the temporaries stay small). Returns a (k, ld) tensor whose
    first d columns are the data."""
    import torch
    d = wl.d if d is None else d
    ld = d if ld is None else ld
    gen = torch.Generator(device=device)
    gen.manual_seed(int(wl.seed) * 1_000_003 + 1000 + round_index)
    G = torch.empty((wl.k, ld), dtype=torch.float32, device=device) if out is None else out
    if ld > d:
        G[:, d:].zero_()
    if wl.value_model == "segments":
        starts, ends, sigma = segment_table(wl)
        scale = torch.empty(d, dtype=torch.float32, device=device)
        for a, b, sg in zip(starts, ends, sigma):
            scale[min(a, d):min(b, d)] = float(sg)
    elif wl.value_model == "partition_scale":
        ps = partition_scales(wl)
    for j in range(wl.k):
        row = G[j, :d]
        row.normal_(generator=gen)
        if wl.value_model == "normal":
            pass
        elif wl.value_model == "partition_scale":
            row.mul_(float(ps[j]))
        elif wl.value_model == "segments":
            row.mul_(scale)
        elif wl.value_model == "student_t3":
            chi = torch.zeros(d, dtype=torch.float32, device=device)
            tmp = torch.empty(d, dtype=torch.float32, device=device)
            for _ in range(3):
                tmp.normal_(generator=gen)
                chi.addcmul_(tmp, tmp)
            row.div_(torch.sqrt(chi / 3.0))
            del chi, tmp
        else:
            raise ValueError(wl.value_model)
    return G


def least_squares_problem(wl, device, rows=None, features=None):
    """cfg4: X ~ N(0,1) [rows, features], w* ~ N(0,1), y = X w* + noise*N(0,1).
    Partition j is the j-th block of rows/k consecutive rows."""
    import torch
    rows = wl.extra["rows"] if rows is None else rows
    features = wl.d if features is None else features
    gen = torch.Generator(device=device)
    gen.manual_seed(int(wl.seed) * 1_000_003 + 77)
    X = torch.empty((rows, features), dtype=torch.float32, device=device)
    X.normal_(generator=gen)
    w_star = torch.empty(features, dtype=torch.float32, device=device).normal_(generator=gen)
    noise = torch.empty(rows, dtype=torch.float32, device=device).normal_(generator=gen)
    y = X @ w_star + wl.extra["noise"] * noise
    return X, y, w_star
