"""gt_spd_build vs the BFS oracle: bit-exact, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import spd as ospd
from paper_2609_34420_b200 import workloads as wl

from gpu_util import gpu_spd

pytestmark = pytest.mark.gpu


def check(w: wl.Workload):
    b = w.batch
    got = gpu_spd(w).cpu().numpy()
    exp = ospd.spd_packed(b.row_ptr, b.col_idx, b.cu_seqlens, w.max_dist)
    assert got.shape == exp.shape
    np.testing.assert_array_equal(got, exp)          # padding bytes included (255 on both sides)
    return got


def closed_form_workload(n, edges, D, symmetric=True):
    e = np.array(edges, dtype=np.int64).reshape(-1, 2)
    csr = wl.csr_from_edges(n, e[:, 0], e[:, 1], symmetric=symmetric)
    return wl.Workload("closed", wl.pack_graphs([csr]), 1, 32, D)


@pytest.mark.parametrize("n", [1, 2, 17, 31, 32, 33, 127, 128, 129, 255, 300, 1000])
@pytest.mark.parametrize("D", [1, 5, 254])
def test_small_sizes_and_tails(n, D):
    check(wl.small_workload([n], 1, 32, D, seed=n + D, avg_degree=2.2))


@pytest.mark.parametrize("directed", [False, True])
def test_varlen_batch_with_empty_and_tiny_graphs(directed):
    check(wl.small_workload([5, 33, 1, 64, 200, 16, 2, 97], 1, 32, 6, seed=4, avg_degree=1.7, directed=directed))


def test_path_graph_runs_to_exhaustion_and_clips():
    n = 700
    w = closed_form_workload(n, [(i, i + 1) for i in range(n - 1)], D=9)
    got = check(w).reshape(n, -1)[:, :n]
    i, j = np.indices((n, n))
    np.testing.assert_array_equal(got, np.minimum(np.abs(i - j), 9))


def test_directed_cycle():
    n = 100
    w = closed_form_workload(n, [(i, (i + 1) % n) for i in range(n)], D=120, symmetric=False)
    got = check(w).reshape(n, -1)[:, :n]
    i, j = np.indices((n, n))
    np.testing.assert_array_equal(got, (j - i) % n)


def _csr(n, src, dst):
    """CSR exactly as given (no symmetrisation, duplicates and self loops kept)."""
    src, dst = np.asarray(src, np.int64), np.asarray(dst, np.int64)
    order = np.lexsort((dst, src))
    rp = np.zeros(n + 1, np.int32)
    np.add.at(rp, src + 1, 1)
    return np.cumsum(rp).astype(np.int32), dst[order].astype(np.int32)


def _both_ways(edges):
    e = np.array(edges, np.int64).reshape(-1, 2)
    return np.concatenate([e[:, 0], e[:, 1]]), np.concatenate([e[:, 1], e[:, 0]])


def test_undirected_graphs_deeper_than_max_dist_stop_at_the_clip_level():
    """Beyond level max_dist an undirected graph only needs "same component or not".  One packed batch with: three
    paths of different lengths in one graph (far pairs, unreachable pairs), a grid, the same paths with duplicate
    edges and self loops, a directed chain (no reverse edges: the full search), the paths with ONE reverse edge
    missing (must not be taken for undirected: nodes behind the one-way edge reach forward only), and a deep
    graph with a hub of 80 leaves (beyond the degree up to which the reverse edges are checked)."""
    D = 6
    paths = [(i, i + 1) for i in range(0, 149)] + [(i, i + 1) for i in range(150, 199)] + [(i, i + 1) for i in range(200, 229)]
    g_paths = _csr(230, *_both_ways(paths))
    side = 23
    grid = [(r * side + c, r * side + c + 1) for r in range(side) for c in range(side - 1)] + \
           [(r * side + c, (r + 1) * side + c) for r in range(side - 1) for c in range(side)]
    g_grid = _csr(side * side, *_both_ways(grid))
    s, d = _both_ways(paths + paths[:40])
    g_dups = _csr(230, np.concatenate([s, np.arange(0, 230, 7)]), np.concatenate([d, np.arange(0, 230, 7)]))
    g_chain = _csr(120, np.arange(119), np.arange(1, 120))
    s, d = _both_ways(paths)
    keep = ~((s == 60) & (d == 59))
    g_oneway = _csr(230, s[keep], d[keep])
    hub = [(i, i + 1) for i in range(0, 99)] + [(50, 100 + j) for j in range(80)]
    g_hub = _csr(180, *_both_ways(hub))
    w = wl.Workload("deep", wl.pack_graphs([g_paths, g_grid, g_dups, g_chain, g_oneway, g_hub]), 1, 32, D)
    got = check(w)
    b = w.batch
    first = got[: b.spd_offsets[1]].reshape(230, -1)[:, :230]
    i, j = np.indices((230, 230))
    block = lambda x: np.where(x < 150, 0, np.where(x < 200, 1, 2))
    np.testing.assert_array_equal(first, np.where(block(i) == block(j), np.minimum(np.abs(i - j), D), D + 1))
    a = b.spd_offsets[4]
    oneway = got[a: a + 230 * 240].reshape(230, 240)[:, :230]
    assert oneway[70, 10] == D + 1 and oneway[10, 70] == D and oneway[61, 60] == 1 and oneway[60, 59] == D + 1


@pytest.mark.parametrize("n,D", [(3000, 3), (5000, 12), (12000, 6)])
def test_deep_undirected_single_graph(n, D):
    """Random geometric graph near its connectivity threshold: many levels, several components.  (At 12 000 nodes the
    graph's CSR no longer fits beside the labels in the component pre-pass's shared memory and is read in place.)"""
    w = wl.Workload("rgg", wl.pack_graphs([wl.random_geometric(n, 5.0, 11)]), 1, 32, D)
    check(w)


def test_star_hub_uses_warp_expansion():
    n = 600                                     # hub degree 599 > the per-lane expansion limit
    w = closed_form_workload(n, [(0, j) for j in range(1, n)], D=4)
    check(w)


def test_empty_graph():
    w = wl.Workload("empty", wl.pack_graphs([(np.zeros(41, np.int32), np.zeros(0, np.int32))]), 1, 32, 3)
    got = check(w).reshape(40, -1)[:, :40]
    exp = np.full((40, 40), 4)
    np.fill_diagonal(exp, 0)
    np.testing.assert_array_equal(got, exp)


@pytest.mark.parametrize("name", ["tiny_er256", "tiny_er256_sparse", "ba4096", "powerlaw16k", "varlen_rgg64"])
def test_named_workloads(name):
    check(wl.make_workload(name))


def test_single_graph_beyond_the_shared_memory_state_matches_and_is_deterministic():
    """A single graph of 14 500 nodes or more takes the bit-matrix build."""
    w = wl.Workload("pl20k", wl.pack_graphs([wl.chung_lu_power_law(20000, 8.0, 2.1, 3)]), 1, 32, 10)
    a = check(w)
    b = gpu_spd(w).cpu().numpy()
    np.testing.assert_array_equal(a, b)


@pytest.mark.parametrize("n", [14499, 14500, 16001])
def test_single_graphs_around_the_switch_to_the_bit_matrix_build(n):
    """14 499 nodes: multi-source BFS with the state in shared memory; 14 500 and 16 001: bit-matrix build with a
    ragged second column block.  Directed, so that the matrix is asymmetric."""
    rng = np.random.Generator(np.random.PCG64(n))
    m = 4 * n
    csr = wl.csr_from_edges(n, rng.integers(0, n - 50, m), rng.integers(0, n - 20, m), symmetric=False)
    check(wl.Workload("switch", wl.pack_graphs([csr]), 1, 32, 7))


def test_packed_batch_with_a_graph_beyond_the_shared_memory_state():
    """A packed batch that contains a graph above the shared-memory limit runs the multi-source BFS with its
    frontier / next / visited words in the workspace (atomics and plain loads on the same L2-resident words).
    Directed, with a hub of several thousand out-edges, vertices without out-edges and isolated vertices;
    two tiny graphs ride along.  Bit-exact against the oracle, twice."""
    n = 18000
    rng = np.random.Generator(np.random.PCG64(77))
    m = 2 * n
    src = np.concatenate([rng.integers(0, n - 300, m), np.full(4000, 11)])
    dst = np.concatenate([rng.integers(0, n - 150, m), rng.choice(n - 150, 4000, replace=False)])
    big = wl.csr_from_edges(n, src, dst, symmetric=False)
    mid = wl.random_directed(300, 2.0, 5)
    tiny = wl.random_directed(5, 1.5, 6)
    w = wl.Workload("packed_big", wl.pack_graphs([big, mid, tiny]), 1, 32, 9)
    from gpu_util import device_batch
    from paper_2609_34420_b200 import binding as gt
    assert gt.gt_spd_build_workspace(device_batch(w.batch), int(w.batch.col_idx.size), 9) > 12 * n    # per-CTA state slices
    a = check(w)
    b = gpu_spd(w).cpu().numpy()
    np.testing.assert_array_equal(a, b)


def test_packed_batch_with_a_deep_undirected_graph_beyond_the_shared_memory_state():
    """The same kernel variant (state in the workspace) where the search stops at level max_dist: a random geometric
    graph of 18 000 nodes (dozens of levels deep, several components) next to a small directed graph."""
    big = wl.random_geometric(18000, 5.5, 21)
    small = wl.random_directed(200, 2.0, 3)
    check(wl.Workload("packed_deep", wl.pack_graphs([big, small]), 1, 32, 7))


def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    """Device-timeout path end to end: the test hook makes the grid barrier of the next bit-matrix build wait
    for a thread block that does not exist; the bounded wait gives up, every thread block returns (the kernel
    has no asynchronous copies in flight), gt_check reports GT_ERR_DEVICE_TIMEOUT and clears the status word,
    and the same workspace then serves a normal, bit-exact build."""
    from gpu_util import device_batch, device_csr
    from paper_2609_34420_b200 import binding as gt
    w = wl.Workload("pl18k", wl.pack_graphs([wl.chung_lu_power_law(18000, 6.0, 2.1, 9)]), 1, 32, 8)
    bt = device_batch(w.batch)
    rp, ci = device_csr(w.batch)
    out = torch.empty(w.batch.spd_bytes, dtype=torch.uint8, device="cuda")
    ws = gt._workspace(gt.gt_spd_build_workspace(bt, int(ci.numel()), w.max_dist), "cuda")
    gt.gt_test_hook_barrier_overcount(1)
    gt.gt_spd_build(rp, ci, bt, w.max_dist, out, ws)
    with pytest.raises(gt.GtError) as e:
        gt.gt_check(ws)
    assert e.value.status == 5                      # GT_ERR_DEVICE_TIMEOUT
    gt.gt_check(ws)                                 # cleared by the report
    gt.gt_spd_build(rp, ci, bt, w.max_dist, out, ws)
    gt.gt_check(ws)
    exp = ospd.spd_packed(w.batch.row_ptr, w.batch.col_idx, w.batch.cu_seqlens, w.max_dist)
    np.testing.assert_array_equal(out.cpu().numpy(), exp)


def test_spd_validate_counts_entries_that_name_no_bucket():
    from gpu_util import device_batch
    from paper_2609_34420_b200 import binding as gt
    w = wl.small_workload([5, 33, 1, 64, 200, 16, 2, 97], 1, 32, 6, seed=4, avg_degree=1.7)
    b = w.batch
    bt = device_batch(b)
    spd = ospd.spd_packed(b.row_ptr, b.col_idx, b.cu_seqlens, w.max_dist).copy()
    good = torch.from_numpy(spd).cuda()
    ws = gt.gt_spd_validate(good, bt, w.max_dist)
    gt.gt_check(ws)                                 # padding bytes (255) are outside the valid region
    assert gt.gt_spd_validate_count(ws) == 0
    # plant invalid bytes inside valid regions: first and last valid byte of a row, a one-node graph, a tail word
    planted = 0
    for g, (i, j) in ((4, (0, 0)), (4, (199, 199)), (2, (0, 0)), (7, (96, 93)), (1, (32, 32)), (4, (17, 130))):
        n_g = int(b.cu_seqlens[g + 1] - b.cu_seqlens[g])
        ld = (n_g + 15) // 16 * 16
        spd[int(b.spd_offsets[g]) + i * ld + j] = w.max_dist + 2 + planted      # >= n_buckets
        planted += 1
    bad = torch.from_numpy(spd).cuda()
    ws = gt.gt_spd_validate(bad, bt, w.max_dist)
    with pytest.raises(gt.GtError) as e:
        gt.gt_check(ws)
    assert e.value.status == 7                      # GT_ERR_BAD_SPD
    assert gt.gt_spd_validate_count(ws) == planted


def test_spd_validate_on_a_single_graph_built_on_the_gpu():
    from gpu_util import device_batch
    from paper_2609_34420_b200 import binding as gt
    w = wl.make_workload("ba4096")
    bt = device_batch(w.batch)
    spd = gpu_spd(w)
    ws = gt.gt_spd_validate(spd, bt, w.max_dist)
    gt.gt_check(ws)
    assert gt.gt_spd_validate_count(ws) == 0
    ws = gt.gt_spd_validate(spd, bt, 3)             # declared with fewer buckets than the matrix holds: distances 4, 5 count
    with pytest.raises(gt.GtError) as e:
        gt.gt_check(ws)
    assert e.value.status == 7
    host = spd.cpu().numpy().reshape(4096, -1)[:, :4096]
    assert gt.gt_spd_validate_count(ws) == int((host >= 5).sum())


def test_a_workspace_whose_header_was_not_zeroed_is_reported_not_trusted():
    """The first 256 bytes of a workspace must be zero when it is first handed over; a dirty header shows up as
    an error from gt_check (which clears it), never as a silently accepted status."""
    from gpu_util import device_batch, device_csr
    from paper_2609_34420_b200 import binding as gt
    w = wl.small_workload([40], 1, 32, 5, seed=0)
    bt = device_batch(w.batch)
    rp, ci = device_csr(w.batch)
    out = torch.zeros(w.batch.spd_bytes, dtype=torch.uint8, device="cuda")
    ws = torch.full((max(gt.gt_spd_build_workspace(bt, int(ci.numel()), 5), 256),), 0xFF, dtype=torch.uint8, device="cuda")
    with pytest.raises(gt.GtError):
        gt.gt_check(ws)
    gt.gt_check(ws)                                 # the report cleared the status word
    ws[:256].zero_()
    gt.gt_spd_build(rp, ci, bt, 5, out, ws)
    gt.gt_check(ws)
    np.testing.assert_array_equal(out.cpu().numpy(), ospd.spd_packed(w.batch.row_ptr, w.batch.col_idx, w.batch.cu_seqlens, 5))


def test_invalid_arguments_are_rejected_without_launch():
    from paper_2609_34420_b200 import binding as gt
    w = wl.small_workload([40], 1, 32, 5, seed=0)
    from gpu_util import device_batch, device_csr
    bt = device_batch(w.batch)
    rp, ci = device_csr(w.batch)
    out = torch.zeros(w.batch.spd_bytes, dtype=torch.uint8, device="cuda")
    with pytest.raises(gt.GtError) as e:
        gt.gt_spd_build(rp, ci, bt, 0, out)
    assert e.value.status == 1
    with pytest.raises(gt.GtError) as e:
        gt.gt_spd_build(rp, ci, bt, 5, out, workspace=torch.zeros(256, dtype=torch.uint8, device="cuda")[:64])
    assert e.value.status == 3
