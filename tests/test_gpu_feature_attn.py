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


# ------------------------------------------------------------------------------------------------------------------
# Categorical features through the code matrix and the tensor-core kernels of the bucket form
# ------------------------------------------------------------------------------------------------------------------
def categorical(n, n_vec, seed, common=False):
    rng = np.random.Generator(np.random.PCG64(seed))
    vec = rng.integers(0, 256, size=(n_vec, 4), dtype=np.uint8)
    if common:                               # a large common part: three features within 4 of 200
        vec[:, 1:] = (200 + rng.integers(0, 4, size=(n_vec, 3))).astype(np.uint8)
    p = rng.random(n_vec) ** 3               # a few vectors hold most pairs, as structural encodings do
    return vec[rng.choice(n_vec, size=(n, n), p=p / p.sum())]


def run_code_case(n, H, d, n_vec, seed, weight_std=0.01, common=False):
    t = wl.make_attn_tensors(n, H, d, 4, seed)
    f = categorical(n, n_vec, seed + 1, common)
    w = (np.random.Generator(np.random.PCG64(seed + 2)).standard_normal((H, 4)) * weight_std).astype(np.float32)
    dev = "cuda"
    q, k, v, do = (bf16_tensor(x, dev) for x in (t.q, t.k, t.v, t.dout))
    feat, wt = torch.from_numpy(f).to(dev), torch.from_numpy(w).to(dev)
    batch = gt.Batch(n)
    ld = (n + 15) // 16 * 16
    codes = torch.full((n * ld,), 77, dtype=torch.uint8, device=dev)
    vectors = torch.full((256,), -1, dtype=torch.int32, device=dev)
    ws = gt.gt_feature_encode(feat, batch, codes, vectors)
    gt.gt_check(ws)
    n_codes = gt.gt_feature_encode_count(ws)
    # the encoding itself: bit-exact against the oracle's numbering
    ref_code, ref_vec = ofeat.encode_features(f)
    assert n_codes == len(ref_vec)
    got = codes.cpu().numpy().reshape(n, ld)
    np.testing.assert_array_equal(got[:, :n], ref_code)
    assert (got[:, n:] == 255).all()
    vec_words = vectors.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(vec_words[:n_codes], ref_vec.astype(np.uint32) @ np.array([1, 256, 65536, 16777216], dtype=np.uint32))
    assert (vec_words[n_codes:] == 0).all()
    # attention through the bucket kernels (the route with the fp32 output: few codes hold nearly all pairs)
    width = max(n_codes, 3)
    table = torch.full((H, width), float("nan"), device=dev)
    gt.gt_feature_code_table(wt, vectors, table)
    out = torch.full((n, H, d), float("nan"), dtype=torch.bfloat16, device=dev)
    lse = torch.full((H, n), float("nan"), device=dev)
    out32 = torch.full((n, H, d), float("nan"), device=dev)
    gt.gt_check(gt.gt_biased_attn_fwd_ex(q, k, v, codes, table, batch, width - 2, out, lse, out32))
    dq, dk, dv = (torch.full_like(q, float("nan")) for _ in range(3))
    dtable = torch.full_like(table, float("nan"))
    gt.gt_check(gt.gt_biased_attn_bwd_ex(q, k, v, out, do, lse, codes, table, batch, width - 2, dq, dk, dv, dtable, out32))
    dw = torch.full_like(wt, float("nan"))
    gt.gt_feature_code_dweights(dtable, vectors, dw)
    g = wl.bf16_bits_to_f64
    qf, kf, vf, dof, wf = g(t.q), g(t.k), g(t.v), g(t.dout), w.astype(np.float64)
    ro, rl = ofeat.forward_feature(qf, kf, vf, f, wf)
    rdq, rdk, rdv, rdw = ofeat.backward_feature(qf, kf, vf, dof, f, wf)
    o = to_f64(out)
    assert (np.abs(o - ro) <= np.maximum(1e-2, np.abs(ro) * 2.0 ** -7)).all(), np.abs(o - ro).max()
    assert np.abs(to_f64(lse) - rl).max() <= 1e-3
    errs = {"dq": rel_l2(to_f64(dq), rdq), "dk": rel_l2(to_f64(dk), rdk), "dv": rel_l2(to_f64(dv), rdv), "dw": rel_l2(to_f64(dw), rdw)}
    per_head = max(rel_l2(to_f64(dw)[h], rdw[h]) for h in range(H))
    if n == 1:
        # One pair: P = 1 and dS = dP - Delta = 0 exactly, so dW = 0.  The kernel's dS is the fp32 rounding of that
        # difference (about 1e-5 of |Delta|), times features up to 255: there is no norm to be relative to.
        assert np.abs(rdw).max() <= 1e-9 and np.abs(to_f64(dw)).max() <= 255 * 2e-4 and errs["dv"] <= 2e-2
        return
    assert all(e <= 2e-2 for e in errs.values()) and per_head <= 2e-2, (errs, per_head)


@pytest.mark.parametrize("n,n_vec,d", [(1, 1, 32), (33, 2, 64), (300, 7, 64), (700, 30, 32), (1100, 256, 64)])
def test_categorical_features_through_the_code_matrix(n, n_vec, d):
    run_code_case(n, 3, d, n_vec, seed=n + n_vec)


def test_categorical_features_with_a_large_common_part():
    run_code_case(600, 2, 64, 12, seed=9, common=True, weight_std=0.02)


def test_more_than_256_distinct_vectors_are_reported_and_the_fallback_is_the_callers():
    n = 200
    rng = np.random.Generator(np.random.PCG64(1))
    f = rng.integers(0, 256, size=(n, n, 4), dtype=np.uint8)
    dev = "cuda"
    codes = torch.zeros(n * 208, dtype=torch.uint8, device=dev)
    vectors = torch.zeros(256, dtype=torch.int32, device=dev)
    ws = gt.gt_feature_encode(torch.from_numpy(f).to(dev), gt.Batch(n), codes, vectors)
    with pytest.raises(gt.GtError) as e:
        gt.gt_check(ws)
    assert e.value.status == 2
    assert gt.gt_feature_encode_count(ws) > 256
    gt.gt_check(ws)                                                  # the status was cleared by the first check
