"""Seeded synthetic inputs for the batched SPDY dynamic program.

This module only *makes inputs*: timing tables ``times[L][K]`` (int32 buckets), error tables
``errors[N][L][K]`` (fp32) and a budget ``B``.  It contains none of the solver's arithmetic and
is the one module that both the CPU oracle's tests and the CUDA path's tests/bench may share.

The shapes stand in for the paper's workloads (Section 4, "Setup"): the sparsity grid is the
paper's ``{0} ∪ {1 - 0.6·δ^i}`` with ``δ = ((1 - s_max)/0.6)^(1/(K-2))`` (K = 42, s_max = 0.99
there), time is discretised into ``B`` buckets (Section 3.2; B = 10^4 in the paper) and the layer
lists are those of ResNet-50 / BERT-base / BERT-large.  The paper's measured timing tables are
not available, so per-layer dense times are taken proportional to the layers' multiply-accumulate
counts and the sparse speed-up curve is the fixed stand-in ``1 - 0.85·s``.

All floating-point work is float64 with one cast at the end, so the arrays are reproducible
across machines with the same NumPy.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterator

import numpy as np

__all__ = [
    "Workload",
    "sparsity_levels",
    "resnet50_macs",
    "bert_macs",
    "make_times",
    "make_errors",
    "make_workload",
    "paper_shaped_errors",
    "tiny_random_instance",
    "sensitivity_samples",
    "mutation_draws",
    "synthetic_calibration_loss",
    "float_times",
    "CONFIG_NAMES",
]


@dataclass
class Workload:
    """One problem batch: everything the solver takes as input, plus a label."""

    name: str
    times: np.ndarray  # [L][K] int32
    errors: np.ndarray  # [N][L][K] float32
    B: int

    @property
    def N(self) -> int:
        return int(self.errors.shape[0])

    @property
    def L(self) -> int:
        return int(self.times.shape[0])

    @property
    def K(self) -> int:
        return int(self.times.shape[1])

    @property
    def nominal_cells(self) -> int:
        """N·L·K·B, the unit the throughput metric is quoted in."""
        return self.N * self.L * self.K * self.B


def sparsity_levels(K: int, s_max: float) -> np.ndarray:
    """Dense (0) followed by K-1 levels spaced geometrically in the remaining weights.

    Generalises the grid of Section 4 "Setup": s_0 = 0, s_{i+1} = 1 - 0.6·δ^i for i = 0..K-2 with
    δ = ((1 - s_max)/0.6)^(1/(K-2)), so that the last level equals ``s_max``.
    """
    if K < 3:
        raise ValueError("need K >= 3 for the geometric grid")
    delta = ((1.0 - s_max) / 0.6) ** (1.0 / (K - 2))
    s = np.empty(K, dtype=np.float64)
    s[0] = 0.0
    s[1:] = 1.0 - 0.6 * delta ** np.arange(K - 1, dtype=np.float64)
    return s


def resnet50_macs() -> np.ndarray:
    """Multiply-accumulates of the 53 convolutions of ResNet-50 at 224x224 (batch cancels)."""
    macs = [7 * 7 * 3 * 64 * 112 * 112]  # stem, stride 2
    in_ch, hw = 64, 56
    for stage, (width, blocks) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        out_ch = width * 4
        for b in range(blocks):
            stride = 2 if (b == 0 and stage > 0) else 1
            hw_out = hw // stride
            macs.append(in_ch * width * hw * hw)  # 1x1 reduce (stride sits on the 3x3)
            macs.append(3 * 3 * width * width * hw_out * hw_out)  # 3x3
            macs.append(width * out_ch * hw_out * hw_out)  # 1x1 expand
            if b == 0:
                macs.append(in_ch * out_ch * hw_out * hw_out)  # 1x1 projection shortcut
            in_ch, hw = out_ch, hw_out
    out = np.asarray(macs, dtype=np.float64)
    assert out.shape[0] == 53
    return out


def bert_macs(blocks: int, hidden: int, ffn: int) -> np.ndarray:
    """Weight-matrix sizes of the encoder's linear layers (tokens x batch scales all equally)."""
    one = [hidden * hidden] * 4 + [hidden * ffn, ffn * hidden]
    return np.asarray(one * blocks, dtype=np.float64)


def _round_half_away(x: np.ndarray) -> np.ndarray:
    return np.sign(x) * np.floor(np.abs(x) + 0.5)


def make_times(T_layer: np.ndarray, s: np.ndarray) -> np.ndarray:
    """times[l][k] = round(T_l · (1 - 0.85·s_k)), at least one bucket each."""
    t = _round_half_away(T_layer[:, None] * (1.0 - 0.85 * s[None, :]))
    t = t.astype(np.int32)
    if t.min() < 1:
        raise ValueError("a layer rounds to a zero-bucket time; use a finer budget")
    return t


def _g(s: np.ndarray) -> np.ndarray:
    return s * s / (1.0 - 0.9 * s)


def make_errors(c: np.ndarray, s: np.ndarray) -> np.ndarray:
    """errors[n][l][k] = fp32(c[n][l] · s_k² / (1 - 0.9·s_k)); the dense choice costs exactly +0."""
    e = (c[:, :, None] * _g(s)[None, None, :]).astype(np.float32)
    e[:, :, 0] = np.float32(0.0)
    return e


def _candidate_sensitivities(cfg: int, L: int, N: int, start: int = 0) -> np.ndarray:
    """c[n][l] = b_l · LogNormal(0, 0.5); one stream per config, so a smaller N is a prefix."""
    base = np.random.default_rng(2000 + cfg).lognormal(0.0, 1.0, size=L)
    rng = np.random.default_rng(3000 + cfg)
    out = np.empty((N, L), dtype=np.float64)
    # Draw row blocks in order so that the stream position depends only on the row index.
    pos, block = 0, 4096
    while pos < start + N:
        n = min(block, start + N - pos)
        z = rng.lognormal(0.0, 0.5, size=(n, L))
        lo, hi = max(pos, start), pos + n
        if hi > lo:
            out[lo - start : hi - start] = z[lo - pos : hi - pos]
        pos += n
    return out * base[None, :]


CONFIG_NAMES = {
    0: "tiny-L8-K4",
    1: "resnet50-L53-K42",
    2: "bert-base-L72-K42",
    3: "bert-large-L144-K64",
    4: "bert-base-sweep",
}


def make_workload(cfg: int, N: int | None = None, B: int | None = None, seed_shift: int = 0,
                  start: int = 0) -> Workload:
    """Build config ``cfg`` (0..4).  ``N``/``B`` override the config's defaults (config 4 sweeps
    them over config 2's shapes); ``seed_shift`` gives independent replicas (e.g. one per rank);
    ``start`` skips that many candidates of the stream (shards of one big batch)."""
    if cfg == 0:
        seed = seed_shift
        L, K = 8, 4
        s = np.array([0.0, 0.5, 0.75, 0.9])
        T = np.random.default_rng(1000 + seed).uniform(8.0, 40.0, size=L)
        Bv = int(min(256, _round_half_away(np.asarray(0.6 * T.sum())))) if B is None else int(B)
        times = make_times(T, s)
        n = 1 if N is None else int(N)
        c = np.random.default_rng(3000 + seed).lognormal(0.0, 1.0, size=(n, L))
        return Workload(f"{CONFIG_NAMES[0]}-seed{seed}", times, make_errors(c, s), Bv)

    if cfg == 1:
        L, K, s_max, n_def, B_def, speedup = 53, 42, 0.99, 1024, 10000, 2.5
        macs = resnet50_macs()
        u = np.random.default_rng(1000 + cfg + seed_shift).uniform(-1.0, 1.0, size=L)
        rel = macs * (1.0 + 0.2 * u)
    elif cfg in (2, 4):
        L, K, s_max, n_def, B_def, speedup = 72, 42, 0.99, 4096, 10000, 3.0
        rel = bert_macs(12, 768, 3072)
    elif cfg == 3:
        L, K, s_max, n_def, B_def, speedup = 144, 64, 0.995, 1024, 65536, 4.0
        rel = bert_macs(24, 1024, 4096)
    else:
        raise ValueError(f"unknown config {cfg}")

    Bv = B_def if B is None else int(B)
    n = n_def if N is None else int(N)
    s = sparsity_levels(K, s_max)
    T = rel / rel.sum() * (speedup * Bv)  # dense total = speedup · budget
    times = make_times(T, s)
    gen_cfg = 2 if cfg == 4 else cfg
    c = _candidate_sensitivities(gen_cfg + 10 * seed_shift, L, n, start=start)
    name = f"{CONFIG_NAMES[cfg]}-N{n}-B{Bv}"
    return Workload(name, times, make_errors(c, s), Bv)


def paper_shaped_errors(L: int, K: int, N: int, seed: int, mutate: bool = True) -> np.ndarray:
    """Error tables as the search itself would submit them (Eq. 4 and Algorithm 4).

    ``errors[n][l][k] = c[n][l]·(k/(K-1))²`` with sensitivities uniform in [0,1]^L; with
    ``mutate`` every candidate after the first is a copy of candidate 0 with at most
    ceil(0.1·L) entries resampled.
    """
    rng = np.random.default_rng(seed)
    if mutate:
        c = np.repeat(rng.uniform(0.0, 1.0, size=(1, L)), N, axis=0)
        dmax = int(np.ceil(0.1 * L))
        for n in range(1, N):
            d = int(rng.integers(1, dmax + 1))
            idx = rng.choice(L, size=d, replace=False)
            c[n, idx] = rng.uniform(0.0, 1.0, size=d)
    else:
        c = rng.uniform(0.0, 1.0, size=(N, L))
    q = (np.arange(K, dtype=np.float64) / (K - 1)) ** 2
    return (c[:, :, None] * q[None, None, :]).astype(np.float32)


def tiny_random_instance(seed: int, max_L: int = 6, max_K: int = 5, max_B: int = 64,
                         exact: bool = False, N: int = 1) -> Workload:
    """Small adversarial instances: ties, zero times, times above the budget, +inf errors.

    With ``exact`` the errors are small multiples of 1/4, so every partial sum is exact in fp32
    and equal-cost optima really tie.
    """
    rng = np.random.default_rng(seed)
    L = int(rng.integers(1, max_L + 1))
    K = int(rng.integers(1, max_K + 1))
    Bv = int(rng.integers(0, max_B + 1))
    hi = max(1, (2 * Bv) // max(L, 1) + 2)
    times = rng.integers(0, hi + 1, size=(L, K)).astype(np.int32)
    if rng.random() < 0.3:  # a choice that can never fit
        times[rng.integers(L), rng.integers(K)] = Bv + 1 + int(rng.integers(0, 5))
    if exact:
        errors = (rng.integers(0, 5, size=(N, L, K)) / 4.0).astype(np.float32)
    else:
        errors = rng.lognormal(0.0, 1.0, size=(N, L, K)).astype(np.float32)
        if rng.random() < 0.3:
            errors[:, rng.integers(L), :] *= np.float32(-1.0)  # negative scores are legal
        if rng.random() < 0.3:  # +inf marks a forbidden choice (-inf and NaN are not valid inputs)
            errors[:, rng.integers(L), rng.integers(K)] = np.float32(np.inf)
    return Workload(f"tiny-random-{seed}", times, errors, Bv)


def iter_sweep_points() -> Iterator[tuple[int, int]]:
    """(N, B) points of the throughput sweep over the BERT-base shapes."""
    for n in (1, 16, 256, 4096, 65536):
        yield n, 10000
    for b in (1000, 100000):
        yield 4096, b


# ---------------------------------------------------------------------------------------------
# Inputs of the coefficient search (Section 3.3 / Algorithm 4).  The random numbers the search
# draws are made here, so that every implementation is fed the same ones; none of the search's
# own steps live in this module.
# ---------------------------------------------------------------------------------------------

def sensitivity_samples(seed: int, L: int, count: int) -> np.ndarray:
    """``count`` coefficient vectors uniform in [0, 1]^L (fp32): the samples of Algorithm 4's first loop."""
    return np.random.default_rng([seed, 1]).uniform(0.0, 1.0, size=(count, L)).astype(np.float32)


def mutation_draws(seed: int, L: int):
    """``draws(d, j)`` -> (indices [d] without repetition, values [d] uniform in [0, 1], fp32): what
    trial j of neighbourhood size d of Algorithm 4 resamples.  Every (d, j) has its own
    counter-seeded generator, so the result does not depend on the order of the calls."""

    def draws(d: int, j: int):
        rng = np.random.default_rng([seed, 2, int(d), int(j)])
        idx = rng.choice(L, size=int(d), replace=False).astype(np.int64)
        val = rng.uniform(0.0, 1.0, size=int(d)).astype(np.float32)
        return idx, val

    return draws


def synthetic_calibration_loss(seed: int, L: int, K: int, s_max: float = 0.99):
    """Stand-in for the calibration loss of a stitched model (Section 3.4 needs the paper's models and
    data, which are not available): a fixed, deterministic function of the profile that is not
    additive over layers - per-layer convex penalties plus a coupling of neighbouring layers.
    An infeasible profile (bytes 0xFF) scores +inf.  Returns ``loss(profile) -> float``."""
    rng = np.random.default_rng([seed, 3])
    w = rng.lognormal(0.0, 1.0, size=L)
    s = sparsity_levels(K, s_max) if K >= 3 else np.linspace(0.0, s_max, K)
    g = s * s / (1.0 - 0.9 * s)
    couple = 0.25 * np.sqrt(w[:-1] * w[1:]) if L > 1 else np.zeros(0)

    def loss(profile) -> float:
        p = np.asarray(profile).astype(np.int64)
        if (p >= K).any():
            return float("inf")
        val = float(np.dot(w, g[p]))
        if L > 1:
            val += float(np.dot(couple, s[p[:-1]] * s[p[1:]]))
        return val

    return loss


def float_times(cfg: int, seed_shift: int = 0):
    """Real-valued layer timings (seconds, fp64) [L][K] of a named config before discretisation,
    with the dense total; inputs of the discretisation helpers."""
    wl = make_workload(cfg, N=1, seed_shift=seed_shift)
    rng = np.random.default_rng([4000 + cfg, seed_shift])
    scale = 1e-4 * (1.0 + rng.uniform())  # seconds per bucket, arbitrary
    t = wl.times.astype(np.float64) * scale * (1.0 + 1e-3 * rng.uniform(-1.0, 1.0, size=wl.times.shape))
    return t, float(t[:, 0].sum())
