"""Seeded synthetic inputs: graphs (CSR) and attention tensors.

This module holds input generation only: no distance computation, no attention
arithmetic.  Both the CUDA path's tests/benchmarks and the CPU oracle's tests draw
their inputs from here so that both sides see bit-identical data.

Graph recipes stand in for the sampled sub-graph batches of the paper's datasets
(Products, Reddit, Citeseer, ...), which are public benchmarks that cannot be
fetched in an offline build.  Every generator emits a symmetric, de-duplicated,
self-loop-free CSR with sorted rows (int32 ``row_ptr[n+1]``, int32 ``col_idx[nnz]``).

bf16 tensors are carried on the host as uint16 bit patterns (numpy has no bf16);
``bf16_bits_to_f64`` widens them exactly.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

CSR = Tuple[np.ndarray, np.ndarray]


# ----------------------------------------------------------------------------
# bf16 <-> float helpers (bit manipulation only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the uint16 patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rnd = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rnd) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


# ----------------------------------------------------------------------------
# CSR assembly
# ----------------------------------------------------------------------------
def csr_from_edges(n: int, src: np.ndarray, dst: np.ndarray, symmetric: bool = True) -> CSR:
    """Build a sorted, de-duplicated, self-loop-free CSR from an edge list."""
    src = np.asarray(src, dtype=np.int64)
    dst = np.asarray(dst, dtype=np.int64)
    if symmetric:
        src, dst = np.concatenate([src, dst]), np.concatenate([dst, src])
    keep = src != dst
    src, dst = src[keep], dst[keep]
    key = np.unique(src * n + dst)
    src, dst = key // n, key % n
    row_ptr = np.zeros(n + 1, dtype=np.int64)
    np.add.at(row_ptr, src + 1, 1)
    row_ptr = np.cumsum(row_ptr)
    return row_ptr.astype(np.int32), dst.astype(np.int32)


def csr_permute(csr: CSR, perm: np.ndarray) -> CSR:
    """Relabel nodes: new node i is old node perm[i].  Directed edges are kept as-is."""
    row_ptr, col_idx = csr
    n = len(row_ptr) - 1
    inv = np.empty(n, dtype=np.int64)
    inv[perm] = np.arange(n)
    deg = np.diff(row_ptr)
    src_old = np.repeat(np.arange(n), deg)
    return csr_from_edges(n, inv[src_old], inv[col_idx.astype(np.int64)], symmetric=False)


def csr_stats(csr: CSR) -> dict:
    row_ptr, col_idx = csr
    deg = np.diff(row_ptr)
    return {"n": int(len(row_ptr) - 1), "nnz": int(len(col_idx)), "deg_min": int(deg.min(initial=0)),
            "deg_mean": float(deg.mean()) if len(deg) else 0.0, "deg_max": int(deg.max(initial=0))}


# ----------------------------------------------------------------------------
# Graph generators
# ----------------------------------------------------------------------------
def erdos_renyi(n: int, p: float, seed: int) -> CSR:
    """G(n, p): every unordered pair is an edge independently with probability p."""
    rng = np.random.Generator(np.random.PCG64(seed))
    iu, ju = np.triu_indices(n, k=1)
    keep = rng.random(iu.shape[0]) < p
    return csr_from_edges(n, iu[keep], ju[keep])


def barabasi_albert(n: int, m: int, seed: int) -> CSR:
    """Preferential attachment: each new node links to m distinct earlier nodes drawn
    proportionally to degree (sampling from the list of all edge endpoints so far)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    endpoints = np.empty(2 * m * n, dtype=np.int64)
    n_end = 0
    src: List[int] = []
    dst: List[int] = []
    targets = list(range(m))                      # node m connects to the m seed nodes
    for v in range(m, n):
        for t in targets:
            src.append(v)
            dst.append(t)
            endpoints[n_end] = v
            endpoints[n_end + 1] = t
            n_end += 2
        chosen: set = set()
        while len(chosen) < m:
            draw = endpoints[rng.integers(0, n_end, size=m - len(chosen))]
            chosen.update(int(x) for x in draw)
        targets = sorted(chosen)
    return csr_from_edges(n, np.array(src), np.array(dst))


def chung_lu_power_law(n: int, avg_degree: float, gamma: float, seed: int) -> CSR:
    """Power-law expected-degree graph: weights w_i ~ (i + i0)^(-1/(gamma-1)), capped at
    sqrt(sum w); n*avg_degree/2 endpoint pairs are drawn proportionally to w, then loops and
    duplicates are dropped and the edge set is symmetrised."""
    rng = np.random.Generator(np.random.PCG64(seed))
    i0 = 10.0
    w = (np.arange(n, dtype=np.float64) + i0) ** (-1.0 / (gamma - 1.0))
    w *= (avg_degree * n) / w.sum()
    w = np.minimum(w, np.sqrt(w.sum()))
    p = w / w.sum()
    n_pairs = int(round(n * avg_degree / 2.0))
    cdf = np.cumsum(p)
    cdf[-1] = 1.0
    a = np.searchsorted(cdf, rng.random(n_pairs), side="right")
    b = np.searchsorted(cdf, rng.random(n_pairs), side="right")
    return csr_from_edges(n, a, b)


def random_geometric(n: int, avg_degree: float, seed: int) -> CSR:
    """n points uniform in the unit square; an edge joins two points closer than
    r = sqrt(avg_degree / (pi n))."""
    from scipy.spatial import cKDTree

    rng = np.random.Generator(np.random.PCG64(seed))
    pts = rng.random((n, 2))
    r = float(np.sqrt(avg_degree / (np.pi * n)))
    pairs = cKDTree(pts).query_pairs(r, output_type="ndarray")
    if pairs.size == 0:
        return csr_from_edges(n, np.zeros(0, np.int64), np.zeros(0, np.int64))
    return csr_from_edges(n, pairs[:, 0], pairs[:, 1])


def random_directed(n: int, avg_out_degree: float, seed: int) -> CSR:
    """Directed G(n,p) (used by tests: the library must be right for asymmetric input)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    mask = rng.random((n, n)) < (avg_out_degree / max(n - 1, 1))
    np.fill_diagonal(mask, False)
    s, d = np.nonzero(mask)
    return csr_from_edges(n, s, d, symmetric=False)


# ----------------------------------------------------------------------------
# Batches and SPD layout
# ----------------------------------------------------------------------------
def round_up(x: int, m: int) -> int:
    return (x + m - 1) // m * m


@dataclass
class GraphBatch:
    """A packed batch of G graphs.  ``row_ptr``/``col_idx`` form ONE block-diagonal CSR over
    the T = sum n_g packed nodes (column ids are packed ids)."""
    row_ptr: np.ndarray            # int32 [T+1]
    col_idx: np.ndarray            # int32 [nnz]
    cu_seqlens: np.ndarray         # int32 [G+1]
    spd_offsets: np.ndarray        # int64 [G+1] byte offset of each graph's SPD block
    spd_ld: np.ndarray             # int64 [G]   row pitch of each block (round_up(n_g,16))

    @property
    def n_graphs(self) -> int:
        return len(self.cu_seqlens) - 1

    @property
    def n_total(self) -> int:
        return int(self.cu_seqlens[-1])

    @property
    def max_seqlen(self) -> int:
        return int(np.diff(self.cu_seqlens).max())

    @property
    def spd_bytes(self) -> int:
        return int(self.spd_offsets[-1])

    @property
    def sum_n2(self) -> int:
        d = np.diff(self.cu_seqlens).astype(np.int64)
        return int((d * d).sum())

    def graph_csr(self, g: int) -> CSR:
        """Local CSR (ids 0..n_g-1) of graph g."""
        a, b = int(self.cu_seqlens[g]), int(self.cu_seqlens[g + 1])
        lo, hi = int(self.row_ptr[a]), int(self.row_ptr[b])
        return ((self.row_ptr[a:b + 1] - lo).astype(np.int32), (self.col_idx[lo:hi] - a).astype(np.int32))


def pack_graphs(graphs: List[CSR]) -> GraphBatch:
    sizes = np.array([len(rp) - 1 for rp, _ in graphs], dtype=np.int64)
    cu = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    rps, cis = [np.zeros(1, np.int64)], []
    nnz = 0
    for g, (rp, ci) in enumerate(graphs):
        rps.append(rp[1:].astype(np.int64) + nnz)
        cis.append(ci.astype(np.int64) + int(cu[g]))
        nnz += len(ci)
    ld = np.array([round_up(int(s), 16) for s in sizes], dtype=np.int64)
    off = np.concatenate([[0], np.cumsum(sizes * ld)]).astype(np.int64)
    col = np.concatenate(cis).astype(np.int32) if cis else np.zeros(0, np.int32)
    return GraphBatch(np.concatenate(rps).astype(np.int32), col, cu, off, ld)


# ----------------------------------------------------------------------------
# Attention tensors
# ----------------------------------------------------------------------------
@dataclass
class AttnTensors:
    q: np.ndarray       # uint16 bf16 bits [T,H,d]
    k: np.ndarray
    v: np.ndarray
    dout: np.ndarray
    bias: np.ndarray    # float32 [H, max_dist+2]


def make_attn_tensors(n_total: int, n_heads: int, head_dim: int, max_dist: int, seed: int,
                      qkv_std: float = 1.0, bias_std: float = 0.5) -> AttnTensors:
    """Q,K,V ~ N(0, qkv_std^2), dO ~ N(0,1) (fp32 draws rounded to bf16 RNE);
    bias table ~ N(0, bias_std^2) fp32 (0.5 is read as the standard deviation)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    shp = (n_total, n_heads, head_dim)

    def draw(std):
        return f32_to_bf16_bits((rng.standard_normal(shp, dtype=np.float32) * np.float32(std)))

    q, k, v = draw(qkv_std), draw(qkv_std), draw(qkv_std)
    dout = draw(1.0)
    bias = (rng.standard_normal((n_heads, max_dist + 2)) * bias_std).astype(np.float32)
    return AttnTensors(q, k, v, dout, bias)


# ----------------------------------------------------------------------------
# The five named workloads
# ----------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    batch: GraphBatch
    n_heads: int
    head_dim: int
    max_dist: int
    qkv_std: float = 1.0
    seed: int = 0
    n_kv_chunks: int = 1
    note: str = ""
    _tensors: Optional[AttnTensors] = field(default=None, repr=False)

    @property
    def n_buckets(self) -> int:
        return self.max_dist + 2

    def tensors(self) -> AttnTensors:
        if self._tensors is None:
            self._tensors = make_attn_tensors(self.batch.n_total, self.n_heads, self.head_dim,
                                              self.max_dist, self.seed + 1, self.qkv_std)
        return self._tensors

    def attn_flops(self) -> Tuple[float, float]:
        """(forward, backward) FLOPs: 4 and 10 times H*d*sum n_g^2 (2 and 5 GEMMs)."""
        base = float(self.n_heads) * self.head_dim * self.batch.sum_n2
        return 4.0 * base, 10.0 * base


WORKLOAD_NAMES = ("tiny_er256", "ba4096", "powerlaw16k", "powerlaw64k", "varlen_rgg64")


def make_workload(name: str, seed: int = 0) -> Workload:
    if name == "tiny_er256":
        g = erdos_renyi(256, 8.0 / 255.0, seed)
        return Workload(name, pack_graphs([g]), 4, 32, 8, seed=seed, note="Erdos-Renyi n=256 avg deg 8")
    if name == "tiny_er256_sparse":   # populates the clip and unreachable buckets
        g = erdos_renyi(256, 2.0 / 255.0, seed)
        return Workload(name, pack_graphs([g]), 4, 32, 8, seed=seed, note="Erdos-Renyi n=256 avg deg 2")
    if name == "ba4096":
        g = barabasi_albert(4096, 5, seed)
        return Workload(name, pack_graphs([g]), 8, 64, 16, seed=seed, note="Barabasi-Albert n=4096 m=5")
    if name == "powerlaw16k":
        g = chung_lu_power_law(16384, 14.0, 2.1, seed)
        return Workload(name, pack_graphs([g]), 8, 64, 20, qkv_std=1.0 / 8.0, seed=seed,
                        note="Chung-Lu power law gamma=2.1 n=16384 avg deg 14; Q,K,V ~ N(0,1)/sqrt(d)")
    if name == "powerlaw64k":
        g = chung_lu_power_law(65536, 12.0, 2.1, seed)
        return Workload(name, pack_graphs([g]), 8, 64, 24, seed=seed, n_kv_chunks=8,
                        note="Chung-Lu power law gamma=2.1 n=65536 avg deg 12")
    if name == "varlen_rgg64":
        rng = np.random.Generator(np.random.PCG64(seed))
        sizes = rng.integers(512, 2049, size=64)
        graphs = [random_geometric(int(s), 6.0, seed * 1000 + 17 + i) for i, s in enumerate(sizes)]
        return Workload(name, pack_graphs(graphs), 16, 64, 12, seed=seed,
                        note="64 random geometric graphs n_g~U[512,2048] avg deg 6, packed")
    raise ValueError(f"unknown workload {name!r}")


def small_workload(n_list: List[int], n_heads: int, head_dim: int, max_dist: int, seed: int,
                   avg_degree: float = 3.0, directed: bool = False, qkv_std: float = 1.0) -> Workload:
    """Small random graphs of arbitrary sizes for tail/edge-case parity tests."""
    graphs = []
    for i, n in enumerate(n_list):
        if directed:
            graphs.append(random_directed(n, avg_degree, seed * 7919 + i))
        else:
            graphs.append(erdos_renyi(n, min(1.0, avg_degree / max(n - 1, 1)), seed * 7919 + i))
    return Workload(f"small{n_list}", pack_graphs(graphs), n_heads, head_dim, max_dist,
                    qkv_std=qkv_std, seed=seed)
