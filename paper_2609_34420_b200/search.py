"""Parallelism-strategy search of the paper's Alg. 1 ("Automatic Optimal Strategy Search") as a small host
utility: given W devices, L Transformer layers, a per-device memory limit and K micro-batches, enumerate the
factorisations W = P_pp * P_cp * P_dp and, for each (P_pp, P_cp), find by dynamic programming the contiguous
layer partition into P_pp pipeline stages that minimises the slowest stage,

    dp[i][k] = min over j < k of max(dp[i-1][j], T_comp(stage i, layers j+1..k, P_cp)),

skipping every stage whose predicted memory exceeds the limit; the winner is the configuration with the smallest
step latency  T = (K + P_pp - 1) * t_cycle + T_stall + t_allreduce  (Sec. "Cost Model Construction").

The cost terms are callables, so that they can be fed with kernel times measured through this library (for
example the per-layer forward + backward attention time of one context-parallel shard from `bench.py --mode
ring`) or with the paper's fitted model, for which `PiecewiseCost` restates the formulas with the constants left
to the caller (the paper does not print its fitted values).  Nothing here touches a GPU.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Callable, List, Optional, Sequence, Tuple

# (stage index, number of stages, layers in the stage, P_cp) -> cost
StageCost = Callable[[int, int, int, int], float]


@dataclass
class Strategy:
    p_pp: int
    p_cp: int
    p_dp: int
    partition: List[int]           # layers per pipeline stage, in stage order
    bottleneck: float              # slowest stage's full-batch compute time
    step_latency: float


def factorisations(w: int) -> List[Tuple[int, int, int]]:
    """All (P_pp, P_cp, P_dp) with P_pp * P_cp * P_dp == w."""
    out = []
    for pp in range(1, w + 1):
        if w % pp:
            continue
        for cp in range(1, w // pp + 1):
            if (w // pp) % cp == 0:
                out.append((pp, cp, w // pp // cp))
    return out


def best_partition(n_layers: int, p_pp: int, p_cp: int, time_cost: StageCost, mem_cost: StageCost,
                   mem_limit: float) -> Optional[Tuple[float, List[int]]]:
    """Min-max contiguous partition of `n_layers` layers into `p_pp` non-empty stages under the memory limit.
    Returns (bottleneck time, layers per stage) or None when no partition fits."""
    if p_pp > n_layers:
        return None
    inf = math.inf
    dp = [[inf] * (n_layers + 1) for _ in range(p_pp + 1)]
    cut = [[-1] * (n_layers + 1) for _ in range(p_pp + 1)]
    dp[0][0] = 0.0
    for i in range(1, p_pp + 1):
        for k in range(i, n_layers - (p_pp - i) + 1):           # later stages still need a layer each
            for j in range(i - 1, k):
                if dp[i - 1][j] == inf:
                    continue
                layers = k - j
                if mem_cost(i - 1, p_pp, layers, p_cp) > mem_limit:
                    continue
                t = max(dp[i - 1][j], time_cost(i - 1, p_pp, layers, p_cp))
                if t < dp[i][k]:
                    dp[i][k], cut[i][k] = t, j
    if dp[p_pp][n_layers] == inf:
        return None
    parts, k = [], n_layers
    for i in range(p_pp, 0, -1):                                # walk the recorded cuts back
        j = cut[i][k]
        parts.append(k - j)
        k = j
    return dp[p_pp][n_layers], parts[::-1]


def search_strategy(n_devices: int, n_layers: int, mem_limit: float, n_micro: int, time_cost: StageCost, mem_cost: StageCost,
                    step_latency: Callable[[float, int, int, int, int], float]) -> Optional[Strategy]:
    """Alg. 1.  `step_latency(bottleneck, P_pp, P_cp, P_dp, K)` turns the slowest stage's compute time into the
    latency of a training step.  Returns the best strategy, or None if nothing fits the memory limit."""
    best: Optional[Strategy] = None
    for pp, cp, dp_ in factorisations(n_devices):
        found = best_partition(n_layers, pp, cp, time_cost, mem_cost, mem_limit)
        if found is None:
            continue
        t_step = step_latency(found[0], pp, cp, dp_, n_micro)
        if best is None or t_step < best.step_latency:
            best = Strategy(pp, cp, dp_, found[1], found[0], t_step)
    return best


@dataclass
class PiecewiseCost:
    """The paper's cost formulas with caller-supplied constants (Sec. "Cost Model Construction").

    Time of a stage with l layers:  l * (t_fwd + t_bwd) * (gamma if l > l_break else 1) + t_emb [first stage]
    + t_proj [last stage], where t_fwd(P_cp), t_bwd(P_cp) are per-layer times of one context-parallel shard.
    Memory of a stage:  c_fp * l * (4 d^2 + 2 d d_ff) + extra weights [first / last stage]
    + l * b * S * (c_mlp d + c_attn h N) + b * S * (c_bias l N + c_feat d_in [first stage]) + m_fixed,
    with N = N' + N_s and S = N' / P_cp + N_s rows per rank."""
    t_fwd: Callable[[int], float]
    t_bwd: Callable[[int], float]
    t_emb: float = 0.0
    t_proj: float = 0.0
    l_break: float = math.inf
    gamma: float = 1.0
    t_p2p: Callable[[float], float] = lambda size: 0.0
    t_allreduce: Callable[[int], float] = lambda p_dp: 0.0
    t_stall: float = 0.0
    # memory
    batch: int = 1
    n_regular: int = 0
    n_super: int = 0
    d: int = 0
    d_ff: int = 0
    d_in: int = 0
    d_out: int = 0
    heads: int = 0
    c_fp: float = 0.0
    c_mlp: float = 0.0
    c_attn: float = 0.0
    c_bias: float = 0.0
    c_feat: float = 0.0
    m_fixed: float = 0.0

    def rows_per_rank(self, p_cp: int) -> float:
        return self.n_regular / p_cp + self.n_super

    def time_cost(self, stage: int, n_stages: int, layers: int, p_cp: int) -> float:
        t = layers * (self.t_fwd(p_cp) + self.t_bwd(p_cp)) * (self.gamma if layers > self.l_break else 1.0)
        return t + (self.t_emb if stage == 0 else 0.0) + (self.t_proj if stage == n_stages - 1 else 0.0)

    def mem_cost(self, stage: int, n_stages: int, layers: int, p_cp: int) -> float:
        n, s = self.n_regular + self.n_super, self.rows_per_rank(p_cp)
        weight = self.c_fp * layers * (4 * self.d ** 2 + 2 * self.d * self.d_ff)
        weight += self.c_fp * self.d_in * self.d if stage == 0 else 0.0
        weight += self.c_fp * self.d * self.d_out if stage == n_stages - 1 else 0.0
        act = layers * self.batch * s * (self.c_mlp * self.d + self.c_attn * self.heads * n)
        feat = self.batch * s * (self.c_bias * layers * n + (self.c_feat * self.d_in if stage == 0 else 0.0))
        return weight + act + feat + self.m_fixed

    def step_latency(self, bottleneck: float, p_pp: int, p_cp: int, p_dp: int, n_micro: int) -> float:
        s_act = (self.batch / n_micro) * self.rows_per_rank(p_cp) * self.d
        t_cycle = bottleneck / n_micro + self.t_p2p(s_act)
        return (n_micro + p_pp - 1) * t_cycle + self.t_stall + self.t_allreduce(p_dp)
