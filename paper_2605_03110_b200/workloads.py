"""Seeded synthetic activation workloads for representative-token selection.

This module only *draws inputs*: prototype-clustered activation matrices X^(l)
(T x d per sequence, one per layer) whose shapes follow the GPT-2 / GPT-J /
OPT-6.7B settings of the paper's Section 6.1.  It contains none of the
selection arithmetic (no norms, no Gram, no threshold), so both the CUDA path
and the CPU checker can be fed from it without sharing any of the method.

Recipe (all counts are exact floors, all draws come from counter-based Philox
streams keyed by (seed, config, sequence, layer)):

  layer 0   P prototype rows p_j ~ N(0, I_d).  floor(u*T) positions, chosen by a
            random permutation, hold unique rows ~ N(0, I_d); every other token
            is p_{j(t)} + sigma*N(0, I_d) with j(t) uniform.  With plant=True
            one token of each prototype is planted first, so that every
            prototype is present.
  layer l+1 X <- X + delta*N(0, I);  then floor(rho*T) random positions are
            replaced by p_{j'} + sigma*N(0, I) with a fresh uniform j';  then
            floor(phi*T) random positions are replaced by fresh N(0, I_d) rows.

The fp32 master copy is carried across layers; bf16 configurations hand out
round-to-nearest-even bf16 copies of every layer (as uint16 bit patterns).
Token labels (prototype id, or a unique negative id) are tracked per layer so
tests can predict the selection from labels alone.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Iterator, List, Optional, Tuple

import numpy as np

__all__ = [
    "WorkloadConfig", "CONFIGS", "sweep_config", "SWEEP_T", "SWEEP_Q",
    "LayerBatch", "generate_layers", "f32_to_bf16_bits", "bf16_bits_to_f32",
    "bf16_bits_to_f64", "as_f64",
]


@dataclass(frozen=True)
class WorkloadConfig:
    cfg_id: int          # 1..5, names the BASELINE configuration
    name: str
    dtype: str           # "f32" or "bf16" (storage type handed to the selection)
    B: int               # independent sequences
    T: int               # tokens per sequence
    d: int               # hidden width
    L: int               # layers
    P: int               # prototypes per sequence
    sigma: float         # within-cluster noise
    u: float             # fraction of unique tokens at layer 0
    delta: float         # per-layer additive drift
    rho: float           # per-layer fraction re-assigned to a random prototype
    phi: float           # per-layer fraction replaced by fresh unique rows
    tau: float = 0.3
    plant: bool = False  # plant one token of every prototype (sweep)

    @property
    def es(self) -> int:
        return 4 if self.dtype == "f32" else 2


CONFIGS = {
    1: WorkloadConfig(1, "gpt2-small-shaped", "f32", 1, 512, 768, 12, 96, 0.05, 0.10, 0.02, 0.0, 0.0),
    2: WorkloadConfig(2, "batched-mid-length", "bf16", 8, 2048, 768, 12, 128, 0.05, 0.05, 0.02, 0.01, 0.0),
    3: WorkloadConfig(3, "gptj-shaped", "bf16", 1, 2048, 4096, 28, 410, 0.05, 0.02, 0.02, 0.02, 0.0),
    4: WorkloadConfig(4, "opt6.7b-shaped-long", "bf16", 1, 8192, 4096, 32, 410, 0.05, 0.0, 0.03, 0.03, 0.005),
}

SWEEP_T = (512, 1024, 2048, 4096, 8192, 16384)
SWEEP_Q = (0.01, 0.05, 0.2, 0.5)


def sweep_config(T: int, q: float) -> WorkloadConfig:
    """One point of the crossover sweep: d=4096, bf16, one layer transition."""
    P = max(1, int(round(q * T)))
    return WorkloadConfig(5, f"sweep-T{T}-q{q:g}", "bf16", 1, T, 4096, 2, P,
                          0.05, 0.0, 0.02, 0.0, 0.0, plant=True)


def scaled(cfg: WorkloadConfig, **kw) -> WorkloadConfig:
    """A smaller / altered copy of a configuration (same recipe, other sizes)."""
    return replace(cfg, **kw)


# ----------------------------------------------------------------------------
# bf16 storage helpers (bit manipulation only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    return bf16_bits_to_f32(bits).astype(np.float64)


def as_f64(x: np.ndarray) -> np.ndarray:
    """Exact float64 view of a stored layer (uint16 = bf16 bits, else fp32)."""
    if x.dtype == np.uint16:
        return bf16_bits_to_f64(x)
    return x.astype(np.float64)


# ----------------------------------------------------------------------------
# generator
# ----------------------------------------------------------------------------
@dataclass
class LayerBatch:
    layer: int
    X: np.ndarray        # (B, T, d) float32, or uint16 bf16 bit patterns
    labels: np.ndarray   # (B, T) int64: prototype id >= 0, unique tokens < 0


def _rng(seed: int, cfg_id: int, seq: int, layer: int, purpose: int) -> np.random.Generator:
    key1 = (cfg_id << 48) | (seq << 32) | (layer << 8) | purpose
    return np.random.Generator(np.random.Philox(key=[int(seed), int(key1)]))


class _Sequence:
    """fp32 master state of one sequence."""

    def __init__(self, cfg: WorkloadConfig, seed: int, seq: int):
        self.cfg, self.seed, self.seq = cfg, seed, seq
        T, d, P = cfg.T, cfg.d, cfg.P
        g = _rng(seed, cfg.cfg_id, seq, 0, 0)
        self.protos = g.standard_normal((P, d), dtype=np.float32)
        perm = g.permutation(T)
        n_u = int(np.floor(cfg.u * T))
        labels = np.empty(T, dtype=np.int64)
        uniq_pos = perm[:n_u]
        rest = perm[n_u:]
        assign = g.integers(0, P, size=rest.size)
        if cfg.plant:
            n_pl = min(P, rest.size)
            assign[:n_pl] = np.arange(n_pl)
        labels[rest] = assign
        self._next_unique = 1
        labels[uniq_pos] = -np.arange(self._next_unique, self._next_unique + n_u)
        self._next_unique += n_u
        X = g.standard_normal((T, d), dtype=np.float32)          # noise / unique rows
        X[rest] *= np.float32(cfg.sigma)
        X[rest] += self.protos[assign]
        self.X, self.labels = X, labels

    def advance(self, layer: int) -> None:
        cfg = self.cfg
        T, d, P = cfg.T, cfg.d, cfg.P
        g = _rng(self.seed, cfg.cfg_id, self.seq, layer, 1)
        noise = g.standard_normal((T, d), dtype=np.float32)
        noise *= np.float32(cfg.delta)
        self.X += noise
        del noise
        n_re = int(np.floor(cfg.rho * T))
        if n_re:
            pos = g.permutation(T)[:n_re]
            j = g.integers(0, P, size=n_re)
            rows = g.standard_normal((n_re, d), dtype=np.float32)
            rows *= np.float32(cfg.sigma)
            rows += self.protos[j]
            self.X[pos] = rows
            self.labels[pos] = j
        n_fr = int(np.floor(cfg.phi * T))
        if n_fr:
            pos = g.permutation(T)[:n_fr]
            self.X[pos] = g.standard_normal((n_fr, d), dtype=np.float32)
            self.labels[pos] = -np.arange(self._next_unique, self._next_unique + n_fr)
            self._next_unique += n_fr


def generate_layers(cfg: WorkloadConfig, seed: int = 0,
                    n_layers: Optional[int] = None) -> Iterator[LayerBatch]:
    """Yield X^(0), X^(1), ... for all B sequences of a configuration."""
    L = cfg.L if n_layers is None else n_layers
    seqs = [_Sequence(cfg, seed, b) for b in range(cfg.B)]
    for layer in range(L):
        if layer > 0:
            for s in seqs:
                s.advance(layer)
        if cfg.dtype == "bf16":
            X = np.stack([f32_to_bf16_bits(s.X) for s in seqs])
        else:
            X = np.stack([s.X.copy() for s in seqs])
        labels = np.stack([s.labels.copy() for s in seqs])
        yield LayerBatch(layer, X, labels)


def generate_all(cfg: WorkloadConfig, seed: int = 0,
                 n_layers: Optional[int] = None) -> Tuple[List[np.ndarray], List[np.ndarray]]:
    Xs, labs = [], []
    for lb in generate_layers(cfg, seed, n_layers):
        Xs.append(lb.X)
        labs.append(lb.labels)
    return Xs, labs
