"""gt_spd_build_static: the SPD build for callers that are not allowed to allocate device memory
(its scratch is an array built into the library).  Collected last on purpose.

The result must be bit-identical to gt_spd_build's on the same inputs and to the BFS oracle's, also on
the second of two calls in a row (the built-in array still holds the first call's leftovers then)."""
import numpy as np
import pytest
import torch

from oracle import spd as ospd
from paper_2609_34420_b200 import binding as gt
from paper_2609_34420_b200 import workloads as wl

from gpu_util import device_batch, device_csr

pytestmark = pytest.mark.gpu


def reference_build(w, bt, rp, ci):
    out = torch.full((w.batch.spd_bytes,), 0xEE, dtype=torch.uint8, device="cuda")
    gt.gt_check(gt.gt_spd_build(rp, ci, bt, w.max_dist, out))
    return out


@pytest.mark.parametrize("make", [lambda: wl.small_workload([5, 130, 1, 256, 300, 64, 2, 97], 1, 32, 6, seed=4, avg_degree=1.7,
                                                            directed=True),
                                  lambda: wl.make_workload("ba4096")])
def test_static_scratch_build_matches_workspace_build_twice_in_a_row(make):
    w = make()
    bt = device_batch(w.batch)
    rp, ci = device_csr(w.batch)
    assert gt.gt_spd_build_workspace(bt, int(ci.numel()), w.max_dist) <= gt.gt_spd_build_static_limit()
    ref = reference_build(w, bt, rp, ci)
    exp = ospd.spd_packed(w.batch.row_ptr, w.batch.col_idx, w.batch.cu_seqlens, w.max_dist)
    for _ in range(2):
        out = torch.full_like(ref, 0x55)
        gt.gt_spd_build_static(rp, ci, bt, w.max_dist, out)
        torch.cuda.synchronize()
        assert torch.equal(out, ref)
        assert np.array_equal(out.cpu().numpy(), exp)


def test_batches_beyond_the_built_in_array_are_refused():
    w = wl.Workload("pl20k", wl.pack_graphs([wl.chung_lu_power_law(20000, 8.0, 2.1, 3)]), 1, 32, 10)
    bt = device_batch(w.batch)
    rp, ci = device_csr(w.batch)
    assert gt.gt_spd_build_workspace(bt, int(ci.numel()), w.max_dist) > gt.gt_spd_build_static_limit()
    out = torch.zeros(w.batch.spd_bytes, dtype=torch.uint8, device="cuda")
    with pytest.raises(gt.GtError) as e:
        gt.gt_spd_build_static(rp, ci, bt, w.max_dist, out)
    assert e.value.status == 3          # GT_ERR_WORKSPACE: nothing was launched
    torch.cuda.synchronize()
    assert int(out.max()) == 0
