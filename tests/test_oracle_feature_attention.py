"""Pins for the feature-bias oracle (CPU only): torch autograd through an einsum-built dense bias,
finite differences on the weights, reduction to the bucket form, a linear-dependence identity."""
import numpy as np
import pytest
import torch

from oracle import attention as oattn
from oracle import feature_attention as ofeat
from oracle import spd as ospd
from paper_2609_34420_b200 import workloads as wl


def make_case(n, H, d, C, seed, asym=True):
    rng = np.random.Generator(np.random.PCG64(seed))
    t = wl.make_attn_tensors(n, H, d, 4, seed)
    g = wl.bf16_bits_to_f64
    f = rng.integers(0, 256, size=(n, n, C), dtype=np.uint8)
    if not asym:
        f = np.maximum(f, f.transpose(1, 0, 2))
    w = rng.standard_normal((H, C)) * 0.01            # features go up to 255: keep the bias O(1)
    return g(t.q), g(t.k), g(t.v), g(t.dout), f, w


def torch_reference(q, k, v, dout, f, w):
    """Independent path: dense bias by einsum, SDPA with an additive mask, autograd in fp64."""
    tq, tk, tv = (torch.tensor(x.transpose(1, 0, 2)).requires_grad_(True) for x in (q, k, v))       # [H,n,d]
    tw = torch.tensor(w).requires_grad_(True)
    bias = torch.einsum("hc,ijc->hij", tw, torch.tensor(f.astype(np.float64)))
    o = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None], attn_mask=bias[None])[0]
    (o * torch.tensor(dout.transpose(1, 0, 2))).sum().backward()
    tr = lambda x: x.detach().numpy().transpose(1, 0, 2)
    s = tq.detach() @ tk.detach().transpose(1, 2) / np.sqrt(q.shape[2]) + bias.detach()
    return tr(o), torch.logsumexp(s, dim=-1).numpy(), tr(tq.grad), tr(tk.grad), tr(tv.grad), tw.grad.numpy()


@pytest.mark.parametrize("n,H,d,C", [(40, 2, 16, 4), (130, 3, 32, 4), (65, 2, 64, 2)])
def test_forward_backward_against_torch_autograd(n, H, d, C):
    q, k, v, do, f, w = make_case(n, H, d, C, seed=n)
    o, lse = ofeat.forward_feature(q, k, v, f, w)
    dq, dk, dv, dw = ofeat.backward_feature(q, k, v, do, f, w)
    ro, rl, rdq, rdk, rdv, rdw = torch_reference(q, k, v, do, f, w)
    for got, ref in ((o, ro), (lse, rl), (dq, rdq), (dk, rdk), (dv, rdv), (dw, rdw)):
        np.testing.assert_allclose(got, ref, rtol=1e-9, atol=1e-9)


def test_weight_gradient_by_central_finite_differences():
    q, k, v, do, f, w = make_case(12, 2, 4, 4, seed=3)
    _, _, _, dw = ofeat.backward_feature(q, k, v, do, f, w)
    loss = lambda ww: float((ofeat.forward_feature(q, k, v, f, ww)[0] * do).sum())
    eps = 1e-6
    for h in range(2):
        for c in range(4):
            wp, wm = w.copy(), w.copy()
            wp[h, c] += eps
            wm[h, c] -= eps
            fd = (loss(wp) - loss(wm)) / (2 * eps)
            assert abs(fd - dw[h, c]) <= 1e-6 * max(1.0, abs(dw[h, c])), (h, c, fd, dw[h, c])


def test_one_hot_features_reduce_to_the_bucket_form():
    """f = one-hot code of a distance matrix with four buckets (max_dist 2): W[h,c] is then the bucket
    table and dW the bucket-table gradient of the pinned bucket oracle."""
    n, H, d, D = 90, 3, 16, 2
    w_ = wl.small_workload([n], H, d, D, seed=5, avg_degree=1.2, directed=True)
    t = w_.tensors()
    g = wl.bf16_bits_to_f64
    q, k, v, do = g(t.q), g(t.k), g(t.v), g(t.dout)
    spd = ospd.spd_matrix(*w_.batch.graph_csr(0), D)[:, :n]
    assert set(np.unique(spd)) == {0, 1, 2, 3}
    f = np.zeros((n, n, 4), np.uint8)
    np.put_along_axis(f, spd[:, :, None].astype(np.int64), 1, axis=2)
    table = t.bias.astype(np.float64)                             # [H, 4]
    o, lse = ofeat.forward_feature(q, k, v, f, table)
    ro, rl = oattn.forward_single(q, k, v, spd, table)
    np.testing.assert_allclose(o, ro, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(lse, rl, rtol=1e-12, atol=1e-12)
    got = ofeat.backward_feature(q, k, v, do, f, table)
    ref = oattn.backward_single(q, k, v, do, spd, table)
    for a, b in zip(got, ref):
        np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-12)


def test_features_with_a_constant_linear_form_give_a_vanishing_directional_gradient():
    """If f[i,j,:] . u is the same for every pair, moving W along u shifts every score of a head by a
    constant, which the softmax ignores: the output is unchanged and dW . u = 0."""
    q, k, v, do, f, w = make_case(50, 2, 8, 4, seed=9)
    f = f.astype(np.int64)
    f[:, :, 0] = (f[:, :, 0] // 2) * 2                            # even, so that f0 / 2 is an integer
    f[:, :, 3] = 255 - f[:, :, 0] // 2                            # f0 / 2 + f3 = 255 for every pair
    f = f.astype(np.uint8)
    u = np.array([0.5, 0.0, 0.0, 1.0])
    assert np.all(f.astype(np.float64) @ u == 255.0)
    o1, l1 = ofeat.forward_feature(q, k, v, f, w)
    o2, l2 = ofeat.forward_feature(q, k, v, f, w + 0.003 * u)
    np.testing.assert_allclose(o1, o2, rtol=0, atol=1e-12)
    np.testing.assert_allclose(l2 - l1, 0.003 * 255.0, rtol=0, atol=1e-11)
    _, _, _, dw = ofeat.backward_feature(q, k, v, do, f, w)
    assert np.abs(dw @ u).max() <= 1e-9 * np.abs(dw).max()


def test_transposed_features_are_not_interchangeable():
    """The bias of the ordered pair (i -> j) is f[i,j]: swapping to f[j,i] must change the result
    (catches a transposed feature tile)."""
    q, k, v, do, f, w = make_case(30, 2, 8, 4, seed=11)
    o, _ = ofeat.forward_feature(q, k, v, f, w)
    ot, _ = ofeat.forward_feature(q, k, v, np.ascontiguousarray(f.transpose(1, 0, 2)), w)
    assert np.abs(o - ot).max() > 1e-3


def categorical_features(n, n_vec, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    vec = rng.integers(0, 256, size=(n_vec, 4), dtype=np.uint8)
    return vec[rng.integers(0, n_vec, size=(n, n))]


def test_codes_round_trip_and_are_numbered_by_ascending_word():
    f = categorical_features(37, 9, 3)
    code, vec = ofeat.encode_features(f)
    np.testing.assert_array_equal(vec[code], f)
    word = vec.astype(np.uint64) @ np.array([1, 256, 65536, 16777216], dtype=np.uint64)
    assert (np.diff(word.astype(np.int64)) > 0).all() and len(vec) <= 9
    # a hand-made case: three distinct vectors, the order decided by the LAST feature first
    g = np.zeros((2, 2, 4), np.uint8)
    g[0, 0] = (9, 0, 0, 0); g[0, 1] = (0, 0, 0, 1); g[1, 0] = (0, 1, 0, 0); g[1, 1] = (9, 0, 0, 0)
    code, vec = ofeat.encode_features(g)
    np.testing.assert_array_equal(code, [[0, 2], [1, 0]])
    np.testing.assert_array_equal(vec, [[9, 0, 0, 0], [0, 1, 0, 0], [0, 0, 0, 1]])


def test_the_code_form_is_the_feature_form_regrouped():
    """table[code] is the feature bias, and dW through the codes (the bucket oracle's scatter, then the contraction
    with the vectors) is backward_feature's dW."""
    from oracle import attention as oattn
    n, H, d = 41, 3, 8
    rng = np.random.Generator(np.random.PCG64(5))
    q, k, v, do = (rng.standard_normal((n, H, d)) for _ in range(4))
    w = rng.standard_normal((H, 4)) * 0.02
    f = categorical_features(n, 11, 8)
    code, vec = ofeat.encode_features(f)
    table = ofeat.code_table(w, vec)
    for h in range(H):
        np.testing.assert_allclose(table[h][code], ofeat.feature_bias(f, w[h]), rtol=0, atol=1e-12)
    o1, l1 = ofeat.forward_feature(q, k, v, f, w)
    o2, l2 = oattn.forward_single(q, k, v, code, table)
    np.testing.assert_allclose(o2, o1, atol=1e-12)
    np.testing.assert_allclose(l2, l1, atol=1e-12)
    dq1, dk1, dv1, dw1 = ofeat.backward_feature(q, k, v, do, f, w)
    dq2, dk2, dv2, dt = oattn.backward_single(q, k, v, do, code, table)
    np.testing.assert_allclose(dq2, dq1, atol=1e-11)
    np.testing.assert_allclose(ofeat.weights_gradient_from_table(dt, vec), dw1, atol=1e-9)
