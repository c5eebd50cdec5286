"""Degenerate inputs and argument errors through the C ABI: batches that contain empty graphs, a
single-node batch, misaligned pointers, unsupported shapes.  Results against the oracle, errors by code."""
import numpy as np
import pytest
import torch

from oracle import attention as oattn
from oracle import spd as ospd
from paper_2609_34420_b200 import binding as gt
from paper_2609_34420_b200 import workloads as wl

from gpu_util import DeviceCase, gpu_spd, rel_l2, to_f64

pytestmark = pytest.mark.gpu


def test_packed_batch_with_empty_graphs_at_the_start_middle_and_end():
    graphs = [wl.erdos_renyi(n, 0.05, 3 + i) if n else (np.zeros(1, np.int32), np.zeros(0, np.int32))
              for i, n in enumerate([0, 70, 0, 0, 130, 1, 0])]
    w = wl.Workload("with_empty", wl.pack_graphs(graphs), 2, 64, 5, seed=3)
    bt = w.batch
    assert list(np.diff(bt.cu_seqlens)) == [0, 70, 0, 0, 130, 1, 0]
    got = gpu_spd(w).cpu().numpy()
    np.testing.assert_array_equal(got, ospd.spd_packed(bt.row_ptr, bt.col_idx, bt.cu_seqlens, w.max_dist))
    case = DeviceCase(w)
    out, lse = case.forward()
    dq, dk, dv, db = case.backward(out, lse)
    q, k, v, do, b = case.host_f64()
    ro, rl = oattn.forward_batch(q, k, v, case.spd_host, bt.spd_offsets, bt.cu_seqlens, b)
    ref = oattn.backward_batch(q, k, v, do, case.spd_host, bt.spd_offsets, bt.cu_seqlens, b)
    assert np.abs(to_f64(out) - ro).max() <= 1e-2 and np.abs(to_f64(lse) - rl).max() <= 1e-3
    for name, got_, want in zip(("dq", "dk", "dv", "dbias"), (dq, dk, dv, db), ref):
        assert rel_l2(to_f64(got_), want) <= 2e-2, name


def test_single_node_graph_attends_to_itself():
    w = wl.small_workload([1], 2, 32, 3, seed=1)
    case = DeviceCase(w)
    out, lse = case.forward()
    assert torch.equal(out, case.v)                         # softmax over one key: the output is its value row
    np.testing.assert_allclose(to_f64(lse)[:, 0],
                               (to_f64(case.q)[0] * to_f64(case.k)[0]).sum(-1) / np.sqrt(32.0) + to_f64(case.bias)[:, 0], atol=1e-3)
    dq, dk, dv, db = case.backward(out, lse)
    assert (to_f64(dq) == 0).all() and (to_f64(dk) == 0).all() and (to_f64(db) == 0).all()      # dS = P (dP - Delta) = 0
    assert torch.equal(dv, case.dout)


def _fwd_status(case, **over):
    a = dict(q=case.q, k=case.k, v=case.v, spd=case.spd, bias=case.bias, batch=case.batch, max_dist=case.w.max_dist,
             out=torch.empty_like(case.q), lse=torch.empty(case.H, case.T, device="cuda"))
    a.update(over)
    try:
        gt.gt_biased_attn_fwd(a["q"], a["k"], a["v"], a["spd"], a["bias"], a["batch"], a["max_dist"], a["out"], a["lse"])
    except gt.GtError as e:
        return e.status
    return 0


def test_argument_errors_are_codes_not_launches():
    case = DeviceCase(wl.small_workload([40], 2, 32, 5, seed=0))
    assert _fwd_status(case) == 0
    # a pointer that is not 16-byte aligned (TMA needs it): a view shifted by one bf16 element
    flat = torch.zeros(case.q.numel() + 8, dtype=torch.bfloat16, device="cuda")
    shifted = flat[1:1 + case.q.numel()].view_as(case.q)
    assert shifted.data_ptr() % 16 != 0
    assert _fwd_status(case, q=shifted) == 1                # GT_ERR_INVALID_ARG
    assert _fwd_status(case, max_dist=0) == 1 and _fwd_status(case, max_dist=255) == 1
    bad_batch = gt.Batch(n_total=40, n_graphs=2)            # two graphs without cu_seqlens / offsets
    assert _fwd_status(case, batch=bad_batch) == 1
    # head_dim outside {32, 64}
    x = torch.zeros(40, 2, 48, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(gt.GtError) as e:
        gt.gt_biased_attn_fwd(x, x, x, case.spd, case.bias, case.batch, 5, torch.empty_like(x), torch.empty(2, 40, device="cuda"))
    assert e.value.status == 2                              # GT_ERR_UNSUPPORTED
    # a workspace smaller than the query
    with pytest.raises(gt.GtError) as e:
        gt.gt_biased_attn_bwd(case.q, case.k, case.v, case.q, case.dout, torch.zeros(2, 40, device="cuda"), case.spd, case.bias,
                              case.batch, 5, *(torch.empty_like(case.q) for _ in range(3)), torch.empty_like(case.bias),
                              workspace=torch.zeros(512, dtype=torch.uint8, device="cuda"))
    assert e.value.status == 3                              # GT_ERR_WORKSPACE
    torch.cuda.synchronize()
