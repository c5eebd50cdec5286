"""Pins for the SPD oracle (CPU only): brute force, closed forms, invariants, scipy."""
import numpy as np
import pytest

from oracle import spd as ospd
from paper_2609_34420_b200 import workloads as wl


def edges_csr(n, edges, symmetric=True):
    e = np.array(edges, dtype=np.int64).reshape(-1, 2)
    return wl.csr_from_edges(n, e[:, 0], e[:, 1], symmetric=symmetric)


def floyd_warshall_spd(csr, max_dist):
    """Independent brute force: all-pairs hop distances by Floyd-Warshall, then clip/map."""
    rp, ci = csr
    n = len(rp) - 1
    INF = 10 ** 9
    dist = np.full((n, n), INF, dtype=np.int64)
    for u in range(n):
        for e in range(rp[u], rp[u + 1]):
            dist[u, ci[e]] = 1
    np.fill_diagonal(dist, 0)
    for m in range(n):
        dist = np.minimum(dist, dist[:, m:m + 1] + dist[m:m + 1, :])
    return np.where(dist >= INF, max_dist + 1, np.minimum(dist, max_dist)).astype(np.uint8)


def reachability_by_matrix_power(csr):
    rp, ci = csr
    n = len(rp) - 1
    a = np.eye(n, dtype=bool)
    for u in range(n):
        a[u, ci[rp[u]:rp[u + 1]]] = True
    for _ in range(int(np.ceil(np.log2(max(n, 2)))) + 1):
        a = (a.astype(np.int64) @ a.astype(np.int64)) > 0
    return a


@pytest.mark.parametrize("n,deg,directed,seed", [(1, 0, False, 0), (2, 1, False, 1), (17, 2.0, False, 2),
                                                 (40, 1.2, False, 3), (64, 3.0, False, 4),
                                                 (33, 1.5, True, 5), (64, 2.0, True, 6), (50, 0.7, True, 7)])
@pytest.mark.parametrize("max_dist", [1, 3, 20])
def test_against_floyd_warshall(n, deg, directed, seed, max_dist):
    csr = wl.random_directed(n, deg, seed) if directed else wl.erdos_renyi(n, min(1.0, deg / max(n - 1, 1)), seed)
    got = ospd.spd_matrix(*csr, max_dist)[:, :n]
    np.testing.assert_array_equal(got, floyd_warshall_spd(csr, max_dist))
    reach = reachability_by_matrix_power(csr)
    np.testing.assert_array_equal(got <= max_dist, reach)


def test_path_graph_and_clipping():
    n = 37
    csr = edges_csr(n, [(i, i + 1) for i in range(n - 1)])
    i, j = np.indices((n, n))
    for D in (3, 10, 60):
        np.testing.assert_array_equal(ospd.spd_matrix(*csr, D)[:, :n], np.minimum(np.abs(i - j), D))


def test_cycle_graph():
    n = 30
    csr = edges_csr(n, [(i, (i + 1) % n) for i in range(n)])
    i, j = np.indices((n, n))
    d = np.abs(i - j)
    np.testing.assert_array_equal(ospd.spd_matrix(*csr, 20)[:, :n], np.minimum(d, n - d))


def test_directed_cycle_is_asymmetric():
    n = 9
    csr = edges_csr(n, [(i, (i + 1) % n) for i in range(n)], symmetric=False)
    i, j = np.indices((n, n))
    np.testing.assert_array_equal(ospd.spd_matrix(*csr, 20)[:, :n], (j - i) % n)


def test_complete_and_star():
    n = 12
    comp = edges_csr(n, [(i, j) for i in range(n) for j in range(i + 1, n)])
    np.testing.assert_array_equal(ospd.spd_matrix(*comp, 5)[:, :n], 1 - np.eye(n, dtype=np.int64))
    star = edges_csr(n, [(0, j) for j in range(1, n)])
    exp = np.full((n, n), 2)
    exp[0, :] = 1
    exp[:, 0] = 1
    np.fill_diagonal(exp, 0)
    np.testing.assert_array_equal(ospd.spd_matrix(*star, 5)[:, :n], exp)


def test_grid_is_manhattan():
    a, b = 5, 7
    idx = lambda x, y: x * b + y
    edges = [(idx(x, y), idx(x + 1, y)) for x in range(a - 1) for y in range(b)]
    edges += [(idx(x, y), idx(x, y + 1)) for x in range(a) for y in range(b - 1)]
    csr = edges_csr(a * b, edges)
    xs, ys = np.divmod(np.arange(a * b), b)
    exp = np.abs(xs[:, None] - xs[None, :]) + np.abs(ys[:, None] - ys[None, :])
    np.testing.assert_array_equal(ospd.spd_matrix(*csr, 30)[:, :a * b], exp)
    np.testing.assert_array_equal(ospd.spd_matrix(*csr, 4)[:, :a * b], np.minimum(exp, 4))


def test_hypercube_is_popcount():
    k = 5
    n = 1 << k
    csr = edges_csr(n, [(i, i ^ (1 << b)) for i in range(n) for b in range(k)])
    i, j = np.indices((n, n))
    pc = np.vectorize(lambda x: bin(x).count("1"))(i ^ j)
    np.testing.assert_array_equal(ospd.spd_matrix(*csr, 8)[:, :n], pc)


def test_empty_graph_and_disjoint_union():
    n = 10
    empty = (np.zeros(n + 1, np.int32), np.zeros(0, np.int32))
    exp = np.full((n, n), 7)
    np.fill_diagonal(exp, 0)
    np.testing.assert_array_equal(ospd.spd_matrix(*empty, 6)[:, :n], exp)
    # two triangles
    csr = edges_csr(6, [(0, 1), (1, 2), (0, 2), (3, 4), (4, 5), (3, 5)])
    got = ospd.spd_matrix(*csr, 4)[:, :6]
    assert (got[:3, 3:] == 5).all() and (got[3:, :3] == 5).all()
    assert (got[:3, :3] == 1 - np.eye(3, dtype=int)).all()


def test_self_loops_and_duplicates_are_ignored():
    rp = np.array([0, 3, 5, 6], np.int32)
    ci = np.array([0, 1, 1, 0, 2, 1], np.int32)     # 0:{0,1,1} 1:{0,2} 2:{1}
    np.testing.assert_array_equal(ospd.spd_matrix(rp, ci, 5)[:, :3], [[0, 1, 2], [1, 0, 1], [2, 1, 0]])


def test_padding_and_ld():
    csr = wl.erdos_renyi(21, 0.2, 0)
    m = ospd.spd_matrix(*csr, 5)
    assert m.shape == (21, 32) and (m[:, 21:] == 255).all()


@pytest.mark.parametrize("seed", [0, 1])
def test_invariants(seed):
    n, D = 300, 6
    csr = wl.erdos_renyi(n, 2.5 / n, seed)
    rp, ci = csr
    s = ospd.spd_matrix(*csr, D)[:, :n].astype(np.int64)
    assert (np.diag(s) == 0).all()
    adj = np.zeros((n, n), bool)
    adj[np.repeat(np.arange(n), np.diff(rp)), ci] = True
    off = ~np.eye(n, dtype=bool)
    np.testing.assert_array_equal((s == 1) & off, adj & off)
    np.testing.assert_array_equal(s, s.T)                      # symmetric CSR => symmetric SPD
    assert (s == D).any() and (s == D + 1).any()               # clip and unreachable both present
    # triangle inequality below the clip (unreachable treated as infinity)
    big = np.where(s > D, 10 ** 6, s)
    for j in range(0, n, 37):
        via = big[:, j:j + 1] + big[j:j + 1, :]
        ok = (np.minimum(via, D) >= np.minimum(big, D)) | (via >= 10 ** 6)
        assert ok.all()


def test_relabelling_equivariance():
    n, D = 120, 9
    csr = wl.random_directed(n, 1.8, 11)
    perm = np.random.default_rng(5).permutation(n)
    s = ospd.spd_matrix(*csr, D)[:, :n]
    s2 = ospd.spd_matrix(*wl.csr_permute(csr, perm), D)[:, :n]
    np.testing.assert_array_equal(s2, s[np.ix_(perm, perm)])


@pytest.mark.parametrize("name", ["tiny_er256", "tiny_er256_sparse", "ba4096"])
def test_against_scipy(name):
    import scipy.sparse as sp
    from scipy.sparse.csgraph import shortest_path

    w = wl.make_workload(name)
    rp, ci = w.batch.graph_csr(0)
    n = len(rp) - 1
    a = sp.csr_matrix((np.ones(len(ci)), ci, rp), shape=(n, n))
    d = shortest_path(a, method="D", unweighted=True, directed=True)
    exp = np.where(np.isinf(d), w.max_dist + 1, np.minimum(d, w.max_dist)).astype(np.uint8)
    np.testing.assert_array_equal(ospd.spd_matrix(rp, ci, w.max_dist)[:, :n], exp)


def test_packed_batch_layout():
    w = wl.small_workload([5, 33, 16, 1], 2, 32, 4, seed=3)
    b = w.batch
    flat = ospd.spd_packed(b.row_ptr, b.col_idx, b.cu_seqlens, w.max_dist)
    assert flat.size == b.spd_bytes
    for g in range(b.n_graphs):
        n_g = int(b.cu_seqlens[g + 1] - b.cu_seqlens[g])
        ld = int(b.spd_ld[g])
        blk = flat[int(b.spd_offsets[g]):int(b.spd_offsets[g]) + n_g * ld].reshape(n_g, ld)
        np.testing.assert_array_equal(blk[:, :n_g], floyd_warshall_spd(b.graph_csr(g), w.max_dist))


def test_source_subset_equals_full_rows():
    csr = wl.random_directed(90, 1.6, 2)
    full = ospd.spd_matrix(*csr, 7)
    rows = np.array([5, 0, 89, 33, 33])
    np.testing.assert_array_equal(ospd.spd_rows(*csr, 7, rows), full[rows])
