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


def test_large_state_in_global_memory_matches_and_is_deterministic():
    """n above the shared-memory state limit exercises the workspace-resident state."""
    w = wl.Workload("pl20k", wl.pack_graphs([wl.chung_lu_power_law(20000, 8.0, 2.1, 3)]), 1, 32, 10)
    a = check(w)
    b = gpu_spd(w).cpu().numpy()
    np.testing.assert_array_equal(a, b)


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
