"""gt_feature_attn_fwd / gt_feature_attn_bwd (Eq. 1 with the four-feature bias) vs the fp64 oracle,
through the C ABI.  Same tolerances as the bucket form: output max-abs <= 1e-2 (or one bf16 ulp), LSE
max-abs <= 1e-3, dQ / dK / dV / dW relative-L2 <= 2e-2."""
import numpy as np
import pytest
import torch

from oracle import feature_attention as ofeat
from paper_2609_34420_b200 import binding as gt
from paper_2609_34420_b200 import workloads as wl

from gpu_util import bf16_tensor, rel_l2, to_f64

pytestmark = pytest.mark.gpu


def make_case(n, H, d, seed, weight_std=0.01, structured=False):
    rng = np.random.Generator(np.random.PCG64(seed))
    t = wl.make_attn_tensors(n, H, d, 4, seed)
    f = rng.integers(0, 256, size=(n, n, 4), dtype=np.uint8)
    if structured:                       # features with a large common part: three of them nearly constant
        f[:, :, 1:] = (200 + rng.integers(0, 4, size=(n, n, 3))).astype(np.uint8)
    w = (rng.standard_normal((H, 4)) * weight_std).astype(np.float32)
    return t, f, w


def run_case(n, H, d, seed, **kw):
    t, f, w = make_case(n, H, d, seed, **kw)
    dev = "cuda"
    q, k, v, do = (bf16_tensor(x, dev) for x in (t.q, t.k, t.v, t.dout))
    feat, wt = torch.from_numpy(f).to(dev), torch.from_numpy(w).to(dev)
    batch = gt.Batch(n)
    out = torch.full((n, H, d), float("nan"), dtype=torch.bfloat16, device=dev)
    lse = torch.full((H, n), float("nan"), device=dev)
    gt.gt_feature_attn_fwd(q, k, v, feat, wt, batch, out, lse)
    dq, dk, dv = (torch.full_like(q, float("nan")) for _ in range(3))
    dw = torch.full_like(wt, float("nan"))
    gt.gt_check(gt.gt_feature_attn_bwd(q, k, v, do, lse, feat, wt, batch, dq, dk, dv, dw))
    g = wl.bf16_bits_to_f64
    qf, kf, vf, dof, wf = g(t.q), g(t.k), g(t.v), g(t.dout), w.astype(np.float64)
    ro, rl = ofeat.forward_feature(qf, kf, vf, f, wf)
    rdq, rdk, rdv, rdw = ofeat.backward_feature(qf, kf, vf, dof, f, wf)
    o = to_f64(out)
    assert np.isfinite(o).all()
    assert (np.abs(o - ro) <= np.maximum(1e-2, np.abs(ro) * 2.0 ** -7)).all(), np.abs(o - ro).max()
    assert np.abs(to_f64(lse) - rl).max() <= 1e-3
    errs = {"dq": rel_l2(to_f64(dq), rdq), "dk": rel_l2(to_f64(dk), rdk), "dv": rel_l2(to_f64(dv), rdv), "dw": rel_l2(to_f64(dw), rdw)}
    per_head = max(rel_l2(to_f64(dw)[h], rdw[h]) for h in range(H))
    assert all(e <= 2e-2 for e in errs.values()) and per_head <= 2e-2, (errs, per_head)
    return errs


@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 130, 300])
@pytest.mark.parametrize("d", [32, 64])
def test_sizes_and_tails(n, d):
    run_case(n, 3, d, seed=n + d)


def test_larger_graph_with_peaked_softmax():
    run_case(1100, 4, 64, seed=7, weight_std=0.04)


def test_features_with_a_large_common_part():
    """Three of the four features are nearly the same for every pair: the weight gradient is then a small
    residue of large sums and only as good as the per-query term of the softmax gradient."""
    run_case(500, 2, 64, seed=8, structured=True)


def test_packed_batches_and_other_head_dims_are_refused():
    dev = "cuda"
    x = torch.zeros(64, 2, 16, dtype=torch.bfloat16, device=dev)
    feat = torch.zeros(64, 64, 4, dtype=torch.uint8, device=dev)
    wt = torch.zeros(2, 4, device=dev)
    lse = torch.zeros(2, 64, device=dev)
    with pytest.raises(gt.GtError) as e:
        gt.gt_feature_attn_fwd(x, x, x, feat, wt, gt.Batch(64), torch.empty_like(x), lse)
    assert e.value.status == 2
