"""Alg. 1 (strategy search): the dynamic programme against brute force over every layer partition, the memory
pruning, and the paper's qualitative example (a heavier first stage gets fewer layers)."""
import itertools
import math

import pytest

from paper_2609_34420_b200 import search


def compositions(n, parts):
    for cuts in itertools.combinations(range(1, n), parts - 1):
        edges = (0,) + cuts + (n,)
        yield [edges[i + 1] - edges[i] for i in range(parts)]


def brute_force(n_devices, n_layers, mem_limit, k, time_cost, mem_cost, step_latency):
    best = None
    for pp, cp, dp in search.factorisations(n_devices):
        if pp > n_layers:
            continue
        for parts in compositions(n_layers, pp):
            if any(mem_cost(i, pp, l, cp) > mem_limit for i, l in enumerate(parts)):
                continue
            bott = max(time_cost(i, pp, l, cp) for i, l in enumerate(parts))
            t = step_latency(bott, pp, cp, dp, k)
            if best is None or t < best[0] - 1e-12:
                best = (t, pp, cp, dp, parts, bott)
    return best


def test_factorisations_cover_every_triple():
    f = search.factorisations(12)
    assert all(a * b * c == 12 for a, b, c in f) and len(f) == len(set(f)) == 18


@pytest.mark.parametrize("w,layers,limit", [(4, 9, 1e9), (8, 10, 1e9), (6, 7, 40.0), (4, 12, 25.0), (2, 5, 5.0)])
def test_search_equals_brute_force(w, layers, limit):
    # irregular but deterministic costs: per-layer time shrinks with P_cp, a superlinear term, stage extras
    def time_cost(i, n, l, cp):
        return l * (3.0 / cp + 0.4) + 0.05 * l * l + (1.7 if i == 0 else 0.0) + (0.6 if i == n - 1 else 0.0)

    def mem_cost(i, n, l, cp):
        return l * (6.0 / cp + 1.0) + (4.0 if i == 0 else 0.0)

    def step_latency(b, pp, cp, dp, k):
        return (k + pp - 1) * (b / k + 0.02 * cp) + 0.3 * math.log2(dp + 1)

    got = search.search_strategy(w, layers, limit, 4, time_cost, mem_cost, step_latency)
    ref = brute_force(w, layers, limit, 4, time_cost, mem_cost, step_latency)
    if ref is None:
        assert got is None
        return
    assert got is not None
    assert got.step_latency == pytest.approx(ref[0], rel=1e-12)
    assert got.bottleneck == pytest.approx(max(time_cost(i, got.p_pp, l, got.p_cp) for i, l in enumerate(got.partition)))
    assert sum(got.partition) == layers and len(got.partition) == got.p_pp and min(got.partition) >= 1
    assert got.p_pp * got.p_cp * got.p_dp == w
    assert all(mem_cost(i, got.p_pp, l, got.p_cp) <= limit for i, l in enumerate(got.partition))


def test_nothing_fits():
    assert search.search_strategy(2, 4, 0.5, 2, lambda *a: 1.0, lambda *a: 1.0, lambda b, *a: b) is None


def test_heavier_first_stage_gets_fewer_layers():
    """Four pipeline stages, 24 layers, an embedding stage that costs as much as four layers: the balanced
    partition is the paper's [3, 7, 7, 7] (Sec. "Heterogeneous pipeline parallelism"), not [6, 6, 6, 6]."""
    cost = search.PiecewiseCost(t_fwd=lambda cp: 1.0, t_bwd=lambda cp: 2.0, t_emb=12.0)
    found = search.best_partition(24, 4, 1, cost.time_cost, lambda *a: 0.0, 1.0)
    assert found is not None and found[1] == [3, 7, 7, 7] and found[0] == pytest.approx(21.0)


def test_piecewise_cost_formulas():
    c = search.PiecewiseCost(t_fwd=lambda cp: 4.0 / cp, t_bwd=lambda cp: 8.0 / cp, t_emb=1.0, t_proj=2.0, l_break=8, gamma=1.5,
                             t_p2p=lambda s: 1e-3 * s, t_allreduce=lambda dp: 0.0 if dp == 1 else 5.0, t_stall=3.0,
                             batch=4, n_regular=1000, n_super=24, d=64, d_ff=128, d_in=100, d_out=10, heads=8,
                             c_fp=16.0, c_mlp=2.0, c_attn=3.0, c_bias=1.0, c_feat=4.0, m_fixed=7.0)
    assert c.time_cost(0, 2, 8, 2) == pytest.approx(8 * 6.0 + 1.0)                  # at the break: no penalty
    assert c.time_cost(1, 2, 9, 2) == pytest.approx(9 * 6.0 * 1.5 + 2.0)            # beyond it: gamma
    s = 1000 / 2 + 24
    mem = 16.0 * 3 * (4 * 64 ** 2 + 2 * 64 * 128) + 16.0 * 100 * 64 + 3 * 4 * s * (2.0 * 64 + 3.0 * 8 * 1024) \
        + 4 * s * (1.0 * 3 * 1024 + 4.0 * 100) + 7.0
    assert c.mem_cost(0, 2, 3, 2) == pytest.approx(mem)
    t_cycle = 30.0 / 4 + 1e-3 * (4 / 4) * s * 64
    assert c.step_latency(30.0, 2, 2, 1, 4) == pytest.approx((4 + 2 - 1) * t_cycle + 3.0)
