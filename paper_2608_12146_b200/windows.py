"""Seeded synthetic optimizer-step windows (inputs only; none of the method's arithmetic).

A *window* is what the planner receives from routing replay: one sequence length per
sample and, for every sample and MoE layer, how many of its top-k assignments went to
each logical expert (the paper's routing-replay input, Section 2.1).  Real replay
traces are not available, so each named workload below draws lengths and routing
counts from the distribution family its description asks for.  Routing counts are a
multinomial of ``k * t_i`` assignments over a per-layer expert popularity vector, so
the conservation law ``sum_e a[i,l,e] == k * t_i`` holds by construction.

Both the CPU oracle's tests and the CUDA path's tests/benchmark take their inputs from
here.  Nothing in this module places experts, packs rows, scores or anneals.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Tuple

import numpy as np


@dataclass(frozen=True)
class WindowSpec:
    """Shape and search budget of one named workload."""

    name: str
    n_samples: int          # N
    n_layers: int           # L   (MoE layers only)
    n_experts: int          # E   (logical experts per layer)
    top_k: int              # k
    token_cap: int          # C   (microbatch token capacity)
    dp_width: int           # D   (controller DP slots; EDP shards = DP slots by default)
    ep_width: int           # P   (modelled physical EP ranks)
    pop_size: int           # P_pop
    sweeps: int             # proposal steps per chain over the whole schedule
    data_seed: int
    n_levels: int = 20      # temperature levels; steps per level = sweeps / n_levels
    t0: float = 1e-3        # first temperature (relative-energy units)
    t_last: float = 1e-6    # last temperature
    p_reloc: float = 0.25   # relocation probability rho
    p_guide: float = 0.8    # guided-proposal probability
    alpha: Tuple[float, ...] = (1.0, 1.0)   # per attention stage: token-linear coefficient
    beta: Tuple[float, ...] = (0.0, 1.0)    # per attention stage: token-pair coefficient
    anneal_seed: int = 0

    @property
    def steps_per_level(self) -> int:
        return max(1, self.sweeps // self.n_levels)

    @property
    def t_ratio(self) -> float:
        if self.n_levels <= 1:
            return 1.0
        return float((self.t_last / self.t0) ** (1.0 / (self.n_levels - 1)))


SPECS: Dict[str, WindowSpec] = {
    "tiny": WindowSpec("tiny", 64, 4, 16, 2, 4096, 2, 4, 8, 200, data_seed=0),
    "medium": WindowSpec("medium", 512, 16, 64, 4, 32768, 8, 8, 256, 2000, data_seed=1),
    "large": WindowSpec("large", 2048, 24, 128, 8, 65536, 16, 16, 1024, 5000, data_seed=2),
    "wide": WindowSpec("wide", 4096, 48, 256, 8, 131072, 32, 32, 4096, 5000, data_seed=3),
    "heavy": WindowSpec("heavy", 8192, 32, 128, 8, 131072, 16, 32, 8192, 20000, data_seed=4),
}
ORDER = ("tiny", "medium", "large", "wide", "heavy")


@dataclass
class Window:
    spec: WindowSpec
    lengths: np.ndarray            # int32 [N]
    demand: np.ndarray             # int32 [N][L][E], expert index fastest
    popularity: np.ndarray = field(repr=False, default=None)  # float64 [L][E], for inspection only


def _lengths(spec: WindowSpec, rng: np.random.Generator) -> np.ndarray:
    n = spec.n_samples
    if spec.name == "tiny":
        t = np.clip(rng.lognormal(7.0, 1.0, n), 16, 4096)
    elif spec.name == "medium":
        t = np.clip(rng.lognormal(8.0, 1.2, n), 64, 16384)
    elif spec.name == "large":
        short = np.clip(rng.lognormal(7.0, 0.8, n), 16, spec.token_cap)
        long_ = rng.integers(8192, 32768, n, endpoint=True).astype(np.float64)
        t = np.where(rng.random(n) < 0.7, short, long_)
    elif spec.name == "wide":
        t = np.clip(rng.lognormal(8.5, 1.3, n), 128, 32768)
    elif spec.name == "heavy":
        t = np.clip(256.0 * (1.0 + rng.pareto(1.5, n)), 256, 65536)
    else:  # custom specs: medium-like mix scaled to the cap
        t = np.clip(rng.lognormal(np.log(spec.token_cap / 12.0), 1.0, n), 8, spec.token_cap // 2)
    return np.minimum(np.floor(t), spec.token_cap).astype(np.int32)


def _popularity(spec: WindowSpec, rng: np.random.Generator) -> np.ndarray:
    L, E = spec.n_layers, spec.n_experts
    tiny = 1e-30
    if spec.name == "medium":
        p = np.empty((L, E))
        p[0] = rng.dirichlet(np.full(E, 0.2))
        for l in range(1, L):  # 5% multiplicative per-layer drift
            v = np.maximum(p[l - 1], tiny) * np.exp(0.05 * rng.standard_normal(E))
            p[l] = v / v.sum()
    elif spec.name == "large":
        p = rng.dirichlet(np.full(E, 0.1), size=L)
        for l in range(L):  # 4 hot experts per layer get 3x mass
            hot = rng.choice(E, size=4, replace=False)
            p[l, hot] = np.maximum(p[l, hot], tiny) * 3.0
            p[l] /= p[l].sum()
    elif spec.name == "wide":
        p = rng.dirichlet(np.full(E, 0.15), size=L)
    elif spec.name == "heavy":
        p = np.empty((L, E))
        logit = np.log(np.maximum(rng.dirichlet(np.full(E, 0.05)), tiny))
        for l in range(L):  # random walk on the logits, layer by layer
            if l:
                logit = logit + 0.5 * rng.standard_normal(E)
            v = np.exp(logit - logit.max())
            p[l] = v / v.sum()
    else:  # tiny and custom
        p = rng.dirichlet(np.full(E, 0.3), size=L)
    p = np.maximum(p, 0.0)
    return p / p.sum(axis=1, keepdims=True)


def make_window(spec: WindowSpec | str, **overrides) -> Window:
    """Draw the window for ``spec`` (a name from SPECS or a WindowSpec).

    ``overrides`` replace fields of the spec (for example ``pop_size=64``) without
    changing the drawn data unless they change a data-shaping field.
    """
    if isinstance(spec, str):
        spec = SPECS[spec]
    if overrides:
        spec = replace(spec, **overrides)
    rng = np.random.default_rng(spec.data_seed)
    lengths = _lengths(spec, rng)
    pop = _popularity(spec, rng)
    n_tok = (spec.top_k * lengths.astype(np.int64))[:, None]
    if spec.name in SPECS:
        # numpy broadcasts n [N,1] against pvals [L,E] -> counts [N,L,E]
        demand = rng.multinomial(n_tok, pop).astype(np.int32)
    else:
        # custom specs: every sample follows one of four "topics", each a sharpened and
        # rotated copy of the layer popularity, so samples differ in which ranks they load
        topic = rng.integers(0, 4, spec.n_samples)
        tp = np.stack([np.roll(pop, 3 * k + 1, axis=1) ** (1.0 + 0.5 * k) for k in range(4)])
        tp /= tp.sum(axis=2, keepdims=True)
        demand = rng.multinomial(n_tok, tp[topic]).astype(np.int32)   # pvals [N,L,E]
    return Window(spec=spec, lengths=lengths, demand=np.ascontiguousarray(demand), popularity=pop)


def custom_spec(name: str, n_samples: int, n_layers: int, n_experts: int, top_k: int,
                token_cap: int, dp_width: int, ep_width: int, pop_size: int, sweeps: int,
                data_seed: int = 1234, **kw) -> WindowSpec:
    """A spec outside the five named workloads (edge-case and ragged-shape tests)."""
    return WindowSpec(name, n_samples, n_layers, n_experts, top_k, token_cap, dp_width,
                      ep_width, pop_size, sweeps, data_seed=data_seed, **kw)
