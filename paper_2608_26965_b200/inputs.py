"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws numbers: it holds none of the method's arithmetic, so
both the CPU oracle's tests and the CUDA path's tests may use it.  All
randomness comes from the counter-based Philox generator keyed by
(seed of the workload, head index), so any subset of heads can be produced
without generating the others.

The five workloads stand in for the paper's evaluation inputs (TabPFN-3 on
tabular sets of 93k-634k rows, Wan 2.1 video latents with 40 heads of
dimension 128, DINOv2 token counts up to 143k; Section 4), whose activations
need model weights and datasets that are not available offline.

Arrays are float32 numpy arrays whose values are already representable in the
workload's storage type (bf16 workloads are rounded to bf16, nearest-even).
"""
from __future__ import annotations

import concurrent.futures
import math
import os
from dataclasses import dataclass, replace
from typing import Optional, Sequence, Tuple

import numpy as np

SEED_BASE = 26082696500


@dataclass(frozen=True)
class Workload:
    name: str
    config_id: int
    heads: int
    head_dim: int
    dtype: str                 # "fp32" | "bf16"
    n_q: int
    n_k: int
    cluster: int               # c (queries and keys use the same size here)
    keep: int                  # kept key clusters per query cluster
    compensate: bool
    kind: str                  # "mixture_iso" | "mixture_aniso" | "video"
    components: int = 0
    grid: Optional[Tuple[int, int, int]] = None

    @property
    def n_qc(self) -> int:
        return -(-self.n_q // self.cluster)

    @property
    def n_kc(self) -> int:
        return -(-self.n_k // self.cluster)

    def scaled(self, **kw) -> "Workload":
        """A reduced copy (fewer heads / rows) for tests; same generator."""
        return replace(self, **kw)


def keep_from_fraction(n_kc: int, fraction: float) -> int:
    return max(1, math.ceil(fraction * n_kc))


WORKLOADS = {
    "tiny": Workload("tiny", 1, 2, 64, "fp32", 1024, 1024, 64, 4, True, "mixture_iso", 8),
    "tabular": Workload("tabular", 2, 8, 64, "bf16", 16384, 131072, 128, 128, True,
                        "mixture_aniso", 32),
    "video480": Workload("video480", 3, 40, 128, "bf16", 32760, 32760, 128, 32, True, "video",
                         grid=(21, 30, 52)),
    "video720": Workload("video720", 4, 40, 128, "bf16", 75600, 75600, 128, 74, True, "video",
                         grid=(21, 45, 80)),
    "sweep": Workload("sweep", 5, 16, 128, "bf16", 131072, 131072, 128, 128, True,
                      "mixture_iso", 64),
}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even), kept as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    rounded = (u + (((u >> 16) & 1) + np.uint32(0x7FFF))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def _rng(w: Workload, head: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[SEED_BASE + w.config_id, head * 16 + stream]))


def _unit_rows(rng, n, d):
    g = rng.standard_normal((n, d))
    return g / np.linalg.norm(g, axis=1, keepdims=True)


def _mixture_iso(w: Workload, head: int):
    rng = _rng(w, head)
    d = w.head_dim
    means = 3.0 * _unit_rows(rng, w.components, d)
    out = []
    for n in (w.n_q, w.n_k):
        comp = rng.integers(0, w.components, size=n)
        out.append((means[comp] + rng.standard_normal((n, d))).astype(np.float32))
    V = rng.standard_normal((w.n_k, d)).astype(np.float32)
    return out[0], out[1], V


def _mixture_aniso(w: Workload, head: int):
    rng = _rng(w, head)
    d = w.head_dim
    means = 3.0 * _unit_rows(rng, w.components, d)
    bases, scales = [], []
    for _ in range(w.components):
        U, _ = np.linalg.qr(rng.standard_normal((d, d)))
        kappa = rng.uniform(1.0, 100.0)
        lam = kappa ** (-np.arange(d) / (d - 1))
        lam = lam / lam.mean()
        bases.append(U)
        scales.append(np.sqrt(lam))
    out = []
    for n in (w.n_q, w.n_k):
        comp = rng.integers(0, w.components, size=n)
        z = rng.standard_normal((n, d))
        x = np.empty((n, d), np.float32)
        for j in range(w.components):
            sel = np.nonzero(comp == j)[0]
            if len(sel):
                x[sel] = (means[j] + (z[sel] * scales[j]) @ bases[j].T).astype(np.float32)
        out.append(x)
    V = rng.standard_normal((w.n_k, d)).astype(np.float32)
    return out[0], out[1], V


def _video(w: Workload, head: int):
    assert w.n_q == w.n_k
    rng = _rng(w, head)
    d = w.head_dim
    T, Hh, Ww = w.grid
    n_full = T * Hh * Ww
    n = w.n_q
    t, y, x = np.meshgrid(np.arange(T) / T, np.arange(Hh) / Hh, np.arange(Ww) / Ww, indexing="ij")
    p = np.stack([t.ravel(), y.ravel(), x.ravel()], axis=1).astype(np.float32)[:n]
    n_waves = 8
    F = np.zeros((n, d), np.float32)
    for _ in range(n_waves):
        omega = rng.integers(0, 4, size=(d, 3))
        zero = np.nonzero((omega == 0).all(axis=1))[0]
        omega[zero, rng.integers(0, 3, size=len(zero))] = 1   # exclude the zero frequency
        a = (rng.standard_normal(d) / math.sqrt(n_waves)).astype(np.float32)
        phi = rng.uniform(0.0, 2.0 * math.pi, size=d).astype(np.float32)
        phase = (2.0 * math.pi) * (p @ omega.T.astype(np.float32)) + phi
        F += a * np.cos(phase, dtype=np.float32)
    sigma = 0.3
    Q = F + sigma * rng.standard_normal((n, d), dtype=np.float32)
    K = F + sigma * rng.standard_normal((n, d), dtype=np.float32)
    V = rng.standard_normal((n, d), dtype=np.float32)
    order = rng.permutation(n)
    assert n <= n_full
    return Q[order], K[order], V[order]


_KINDS = {"mixture_iso": _mixture_iso, "mixture_aniso": _mixture_aniso, "video": _video}


def generate_head(w: Workload, head: int):
    """(Q [n_q,d], K [n_k,d], V [n_k,d]) float32 for one head, storage-rounded."""
    Q, K, V = _KINDS[w.kind](w, head)
    if w.dtype == "bf16":
        Q, K, V = round_to_bf16(Q), round_to_bf16(K), round_to_bf16(V)
    return Q, K, V


def generate(w: Workload, heads: Optional[Sequence[int]] = None):
    """Stacked [H', n, d] float32 arrays for the listed heads (default: all).  Heads are drawn
    from their own generator streams, so they are produced side by side on the host's cores; the
    values do not depend on how many threads run."""
    heads = list(range(w.heads)) if heads is None else list(heads)
    d = w.head_dim
    out = (np.empty((len(heads), w.n_q, d), np.float32), np.empty((len(heads), w.n_k, d), np.float32),
           np.empty((len(heads), w.n_k, d), np.float32))

    def one(slot):
        for dst, src in zip(out, generate_head(w, heads[slot])):
            dst[slot] = src

    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:
        cores = os.cpu_count() or 1
    workers = max(1, min(len(heads), cores))
    if workers == 1:
        one(0)
    else:
        with concurrent.futures.ThreadPoolExecutor(max_workers=workers) as pool:
            list(pool.map(one, range(len(heads))))
    return out
