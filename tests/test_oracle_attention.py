"""Pins for the attention oracle (CPU only): library cross-checks, closed forms, identities,
finite differences, equivariance, the hand-worked golden case."""
import os

import numpy as np
import pytest
import torch

from oracle import attention as oattn
from oracle import spd as ospd
from paper_2609_34420_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def make_case(n, H, d, D, seed, directed=False, deg=2.5, qkv_std=1.0):
    w = wl.small_workload([n], H, d, D, seed, avg_degree=deg, directed=directed, qkv_std=qkv_std)
    t = w.tensors()
    csr = w.batch.graph_csr(0)
    spd = ospd.spd_matrix(*csr, D)
    f = wl.bf16_bits_to_f64
    return f(t.q), f(t.k), f(t.v), f(t.dout), spd, t.bias.astype(np.float64)


def torch_reference(q, k, v, dout, spd, bias):
    """Independent path: torch SDPA in fp64 with the bias passed as a dense additive mask,
    gradients by autograd through the table gather."""
    n = q.shape[0]
    tq, tk, tv = (torch.tensor(x.transpose(1, 0, 2)).requires_grad_(True) for x in (q, k, v))  # [H,n,d]
    tb = torch.tensor(bias).requires_grad_(True)
    idx = torch.tensor(spd[:, :n].astype(np.int64))
    mask = tb[:, idx]                                                                       # [H,n,n]
    o = torch.nn.functional.scaled_dot_product_attention(tq[None], tk[None], tv[None], attn_mask=mask[None])[0]
    (o * torch.tensor(dout.transpose(1, 0, 2))).sum().backward()
    tr = lambda x: x.detach().numpy().transpose(1, 0, 2)
    s = tq.detach() @ tk.detach().transpose(1, 2) / np.sqrt(q.shape[2]) + mask.detach()
    return tr(o), torch.logsumexp(s, dim=-1).numpy(), tr(tq.grad), tr(tk.grad), tr(tv.grad), tb.grad.numpy()


@pytest.mark.parametrize("n,H,d,D,directed", [(50, 2, 32, 4, False), (200, 4, 64, 6, True), (129, 3, 16, 3, False)])
def test_forward_backward_against_torch_autograd(n, H, d, D, directed):
    q, k, v, do, spd, b = make_case(n, H, d, D, seed=n, directed=directed)
    o, lse = oattn.forward_single(q, k, v, spd, b)
    dq, dk, dv, db = oattn.backward_single(q, k, v, do, spd, b)
    ro, rl, rdq, rdk, rdv, rdb = torch_reference(q, k, v, do, spd, b)
    for got, ref in ((o, ro), (lse, rl), (dq, rdq), (dk, rdk), (dv, rdv), (db, rdb)):
        np.testing.assert_allclose(got, ref, rtol=1e-9, atol=1e-10)


def test_zero_bias_is_standard_attention():
    q, k, v, do, spd, b = make_case(150, 2, 32, 5, seed=1)
    b[:] = 0.0
    o, _ = oattn.forward_single(q, k, v, spd, b)
    tq, tk, tv = (torch.tensor(x.transpose(1, 0, 2))[None] for x in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0].numpy().transpose(1, 0, 2)
    np.testing.assert_allclose(o, ref, rtol=1e-10, atol=1e-12)


def test_golden_rational_softmax():
    vals = {}
    with open(os.path.join(GOLDEN, "eq1_rational_softmax.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, *nums = line.split()
            vals[key] = np.array([float(x) for x in nums])
    csr = wl.csr_from_edges(3, np.array([0, 1]), np.array([1, 2]))
    spd = ospd.spd_matrix(*csr, 2)
    np.testing.assert_array_equal(spd[:, :3], [[0, 1, 2], [1, 0, 1], [2, 1, 0]])
    bias = np.log(np.array([[1.0, 2.0, 3.0, 5.0]]))
    q = np.zeros((3, 1, 2))
    k = np.random.default_rng(0).standard_normal((3, 1, 2))        # irrelevant because Q = 0
    v = np.array([[6.0, 0.0], [0.0, 30.0], [30.0, 60.0]]).reshape(3, 1, 2)
    do = np.ones((3, 1, 2))
    o, lse = oattn.forward_single(q, k, v, spd, bias)
    np.testing.assert_allclose(o.reshape(-1), vals["O"], rtol=1e-13)
    np.testing.assert_allclose(lse.reshape(-1), vals["LSE"], rtol=1e-13)
    _, dk, _, db = oattn.backward_single(q, k, v, do, spd, bias)
    np.testing.assert_allclose(db.reshape(-1), vals["dB"], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dk, 0.0, atol=1e-14)                # dK = dS^T Q / sqrt(d) = 0


def test_closed_forms_q_zero_and_v_one():
    q, k, v, do, spd, b = make_case(90, 3, 32, 4, seed=7)
    n = q.shape[0]
    o, lse = oattn.forward_single(np.zeros_like(q), k, v, spd, b)
    for h in range(3):
        w = np.exp(b[h][spd[:, :n].astype(int)])
        np.testing.assert_allclose(o[:, h, :], (w @ v[:, h, :]) / w.sum(1, keepdims=True), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(lse[h], np.log(w.sum(1)), rtol=1e-12)
    o0, lse0 = oattn.forward_single(np.zeros_like(q), k, v, spd, np.zeros_like(b))
    np.testing.assert_allclose(o0, np.broadcast_to(v.mean(0), o0.shape), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse0, np.log(n), rtol=1e-13)
    o1, _ = oattn.forward_single(q, k, np.ones_like(v), spd, b)        # rows of P sum to one
    np.testing.assert_allclose(o1, 1.0, rtol=1e-13)


def test_shift_invariance_and_dominant_bucket():
    q, k, v, do, spd, b = make_case(64, 2, 32, 4, seed=9)
    o, lse = oattn.forward_single(q, k, v, spd, b)
    c = np.array([[1.7], [-0.3]])
    o2, lse2 = oattn.forward_single(q, k, v, spd, b + c)
    np.testing.assert_allclose(o2, o, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(lse2, lse + c, rtol=1e-12)
    b3 = b.copy()
    b3[:, 0] += 200.0                                                  # bucket 0 = the node itself
    o3, _ = oattn.forward_single(q, k, v, spd, b3)
    np.testing.assert_allclose(o3, v, rtol=1e-12, atol=1e-12)


def test_unreachable_pairs_still_attend():
    # two isolated nodes: each row has weights exp(B[0]) for itself and exp(B[D+1]) for the other
    spd = ospd.spd_matrix(np.zeros(3, np.int32), np.zeros(0, np.int32), 3)
    b = np.array([[0.0, 9.0, 9.0, 9.0, np.log(3.0)]])
    v = np.array([[1.0], [5.0]]).reshape(2, 1, 1)
    o, _ = oattn.forward_single(np.zeros((2, 1, 1)), np.zeros((2, 1, 1)), v, spd, b)
    np.testing.assert_allclose(o.reshape(-1), [(1 + 15) / 4, (5 + 3) / 4], rtol=1e-13)


def test_permutation_equivariance():
    n, H, d, D = 70, 2, 32, 5
    q, k, v, do, spd, b = make_case(n, H, d, D, seed=3, directed=True)
    perm = np.random.default_rng(1).permutation(n)
    sp = np.ascontiguousarray(spd[:, :n][np.ix_(perm, perm)])
    o, lse = oattn.forward_single(q, k, v, spd, b)
    dq, dk, dv, db = oattn.backward_single(q, k, v, do, spd, b)
    o2, lse2 = oattn.forward_single(q[perm], k[perm], v[perm], sp, b)
    dq2, dk2, dv2, db2 = oattn.backward_single(q[perm], k[perm], v[perm], do[perm], sp, b)
    np.testing.assert_allclose(o2, o[perm], rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(lse2, lse[:, perm], rtol=1e-12)
    np.testing.assert_allclose(dq2, dq[perm], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dk2, dk[perm], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dv2, dv[perm], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(db2, db, rtol=1e-9, atol=1e-10)


def test_finite_differences():
    n, H, d, D = 14, 2, 4, 3
    q, k, v, do, spd, b = make_case(n, H, d, D, seed=5)
    dq, dk, dv, db = oattn.backward_single(q, k, v, do, spd, b)

    def loss(q_, k_, v_, b_):
        return float((oattn.forward_single(q_, k_, v_, spd, b_)[0] * do).sum())

    eps = 1e-5
    rng = np.random.default_rng(0)
    for which, grad in (("q", dq), ("k", dk), ("v", dv), ("b", db)):
        base = {"q": q, "k": k, "v": v, "b": b}
        flat_idx = rng.choice(grad.size, size=min(grad.size, 25), replace=False)
        for fi in flat_idx:
            idx = np.unravel_index(fi, grad.shape)
            hi = {key: val.copy() for key, val in base.items()}
            lo = {key: val.copy() for key, val in base.items()}
            hi[which][idx] += eps
            lo[which][idx] -= eps
            fd = (loss(hi["q"], hi["k"], hi["v"], hi["b"]) - loss(lo["q"], lo["k"], lo["v"], lo["b"])) / (2 * eps)
            assert abs(fd - grad[idx]) <= 1e-6 * max(1.0, abs(grad[idx])), (which, idx, fd, grad[idx])


def test_backward_identities():
    q, k, v, do, spd, b = make_case(100, 3, 32, 4, seed=13)
    dq, dk, dv, db = oattn.backward_single(q, k, v, do, spd, b)
    # softmax is shift invariant => every row of dS sums to zero => sum_b dB[h,b] = 0
    assert np.abs(db.sum(axis=1)).max() <= 1e-10 * np.abs(db).max()
    # dO = 1  =>  dV[j] = column sums of P, and those sum to n over j
    _, _, dv1, _ = oattn.backward_single(q, k, v, np.ones_like(do), spd, b)
    np.testing.assert_allclose(dv1.sum(axis=0), 100.0, rtol=1e-12)
    # buckets that never occur get exactly zero
    n = 100
    present = np.bincount(spd[:, :n].reshape(-1), minlength=b.shape[1])[:b.shape[1]] > 0
    assert (db[:, ~present] == 0).all()


def test_row_subset_matches_full():
    q, k, v, do, spd, b = make_case(120, 2, 32, 4, seed=21)
    rows = np.array([3, 77, 5, 119])
    o, lse = oattn.forward_single(q, k, v, spd, b)
    o_r, lse_r = oattn.forward_single(q, k, v, spd, b, rows=rows)
    np.testing.assert_allclose(o_r, o[rows], rtol=1e-13)
    np.testing.assert_allclose(lse_r, lse[:, rows], rtol=1e-13)
    # dK/dV/dB over a row subset == full backward with dO zeroed outside the subset
    do_masked = np.zeros_like(do)
    do_masked[rows] = do[rows]
    full = oattn.backward_single(q, k, v, do_masked, spd, b)
    part = oattn.backward_single(q, k, v, do, spd, b, rows=rows)
    np.testing.assert_allclose(part[0], full[0][rows], rtol=1e-12, atol=1e-14)
    for a_, b_ in zip(part[1:], full[1:]):
        np.testing.assert_allclose(a_, b_, rtol=1e-12, atol=1e-14)


def test_chunk_lse_merges_to_full_and_uses_global_columns():
    n = 150
    q, k, v, do, spd, b = make_case(n, 2, 32, 6, seed=17, directed=True)     # asymmetric SPD
    assert (spd[:, :n] != spd[:, :n].T).any()
    _, lse = oattn.forward_single(q, k, v, spd, b)
    bounds = [(0, 64), (64, 128), (128, 150), (150, 150)]
    cl = oattn.chunk_lse(q, k, spd, b, bounds)
    assert np.isneginf(cl[3]).all()
    m = cl.max(axis=0)
    merged = m + np.log(np.exp(cl - m).sum(axis=0))
    np.testing.assert_allclose(merged, lse, rtol=1e-12)
    # brute force one chunk entry with the bias taken at the global column
    h, i = 1, 42
    s = (q[i, h] @ k[64:128, h].T) / np.sqrt(32.0) + b[h][spd[i, 64:128].astype(int)]
    np.testing.assert_allclose(cl[1, h, i], np.log(np.exp(s).sum()), rtol=1e-12)


def test_batch_equals_independent_graphs():
    w = wl.small_workload([40, 7, 65], 2, 32, 4, seed=2)
    t = w.tensors()
    f = wl.bf16_bits_to_f64
    q, k, v, do, b = f(t.q), f(t.k), f(t.v), f(t.dout), t.bias.astype(np.float64)
    bt = w.batch
    flat = ospd.spd_packed(bt.row_ptr, bt.col_idx, bt.cu_seqlens, w.max_dist)
    o, lse = oattn.forward_batch(q, k, v, flat, bt.spd_offsets, bt.cu_seqlens, b)
    dq, dk, dv, db = oattn.backward_batch(q, k, v, do, flat, bt.spd_offsets, bt.cu_seqlens, b)
    db_sum = np.zeros_like(db)
    for g in range(3):
        a, e = int(bt.cu_seqlens[g]), int(bt.cu_seqlens[g + 1])
        spd_g = ospd.spd_matrix(*bt.graph_csr(g), w.max_dist)
        ro, rl, rdq, rdk, rdv, rdb = torch_reference(q[a:e], k[a:e], v[a:e], do[a:e], spd_g, b)
        np.testing.assert_allclose(o[a:e], ro, rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(lse[:, a:e], rl, rtol=1e-10)
        np.testing.assert_allclose(dq[a:e], rdq, rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(dk[a:e], rdk, rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(dv[a:e], rdv, rtol=1e-9, atol=1e-11)
        db_sum += rdb
    np.testing.assert_allclose(db, db_sum, rtol=1e-9, atol=1e-11)


def test_bias_after_max_update_would_be_wrong():
    """The online-softmax rule of the context-parallel scheme: the bias slice must enter
    the score before the running max / sum are updated.  A blockwise merge that takes the
    statistics from the un-biased scores and adds the bias afterwards differs from the
    oracle whenever the bias spread is large; the per-chunk merge with bias folded in
    (checked above) does not."""
    n = 96
    q, k, v, do, spd, b = make_case(n, 1, 32, 4, seed=4)
    b = b * 20.0
    o, _ = oattn.forward_single(q, k, v, spd, b)
    s_nobias = (q[:, 0] @ k[:, 0].T) / np.sqrt(32.0)
    wrong_num, wrong_den = np.zeros((n, 32)), np.zeros((n, 1))
    for a in (0, 48):
        blk = s_nobias[:, a:a + 48]
        m = blk.max(1, keepdims=True)                      # statistics without the bias
        p = np.exp(blk - m)
        p = p / p.sum(1, keepdims=True) * np.exp(m)        # block-normalised, re-weighted by un-biased max
        p = p * np.exp(b[0][spd[:, a:a + 48].astype(int)])  # bias applied after normalisation
        wrong_num += p @ v[a:a + 48, 0]
        wrong_den += np.exp(blk).sum(1, keepdims=True)
    wrong = wrong_num / wrong_den
    assert np.abs(wrong - o[:, 0]).max() > 1e-2


def test_compact_spd_rows_match_full():
    q, k, v, do, spd, b = make_case(110, 2, 32, 4, seed=23, directed=True)
    rows = np.array([100, 3, 57])
    a = oattn.forward_single(q, k, v, spd, b, rows=rows)
    c = oattn.forward_single(q, k, v, np.ascontiguousarray(spd[rows]), b, rows=rows, compact_spd=True)
    np.testing.assert_array_equal(a[0], c[0])
    ga = oattn.backward_single(q, k, v, do, spd, b, rows=rows)
    gc = oattn.backward_single(q, k, v, do, np.ascontiguousarray(spd[rows]), b, rows=rows, compact_spd=True)
    for x, y in zip(ga, gc):
        np.testing.assert_array_equal(x, y)


def test_backward_chunked_sums_to_full_and_chunks_own_their_key_rows():
    n = 150
    q, k, v, do, spd, b = make_case(n, 2, 32, 6, seed=23, directed=True)
    out, lse = oattn.forward_single(q, k, v, spd, b)
    full = oattn.backward_single(q, k, v, do, spd, b)
    bounds = [(0, 64), (64, 128), (128, 150), (150, 150)]
    dq, dk, dv, db, db_c = oattn.backward_chunked(q, k, v, do, out, lse, spd, b, bounds)
    for got, ref in zip((dq, dk, dv, db), full):
        np.testing.assert_allclose(got, ref, rtol=1e-10, atol=1e-13)
    assert db_c.shape == (4, 2, b.shape[1]) and (db_c[3] == 0).all()
    # a chunk's bias gradient only sees its own key columns: brute force one bucket of one chunk
    h, c, (a_, b_) = 1, 1, bounds[1]
    s = (q[:, h] @ k[:, h].T) / np.sqrt(32.0) + b[h][spd[:, :n].astype(int)]
    p = np.exp(s - lse[h][:, None])
    ds = p * (do[:, h] @ v[:, h].T - (do[:, h] * out[:, h]).sum(1, keepdims=True))
    bucket = int(spd[3, 70])
    mask = spd[:, a_:b_] == bucket
    np.testing.assert_allclose(db_c[c, h, bucket], ds[:, a_:b_][mask].sum(), rtol=1e-10, atol=1e-13)
    # rows of dS sum to zero over ALL key columns, so the per-head total of dB vanishes only once every chunk is in
    np.testing.assert_allclose(db.sum(axis=1), 0.0, atol=1e-10)
    assert np.abs(db_c[:3].sum(axis=2)).min() > 1e-6


def test_ring_steps_with_two_part_key_slices_merge_to_the_full_forward():
    # 3 "ranks" of regular nodes plus a block of super nodes at the end of the index range; every step's key
    # block is a regular range plus (once only) the super-node range: two-part slicing of the bias columns
    n, n_super = 150, 22
    q, k, v, do, spd, b = make_case(n, 2, 32, 6, seed=31, directed=True)
    ro, rl = oattn.forward_single(q, k, v, spd, b)
    n_reg = n - n_super
    shards = [(0, 48), (48, 96), (96, n_reg)]
    rows = np.arange(16, 130)
    o = np.zeros((len(rows), 2, 32)); lse = np.full((2, len(rows)), -np.inf)
    for step, (a_, b_) in enumerate(shards):
        keys = np.concatenate([np.arange(a_, b_), np.arange(n_reg, n) if step == 1 else np.arange(0)])
        po, pl = oattn.attend_key_set(q, k, v, spd, b, rows, keys)
        o, lse = oattn.merge_state(o, lse, po, pl)
    np.testing.assert_allclose(o, ro[rows], rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(lse, rl[:, rows], rtol=1e-12)
    # a key subset's LSE by brute force, bias at the global column
    h, i = 1, 5
    keys = np.concatenate([np.arange(48, 96), np.arange(n_reg, n)])
    s = (q[rows[i], h] @ k[keys, h].T) / np.sqrt(32.0) + b[h][spd[rows[i], keys].astype(int)]
    _, pl = oattn.attend_key_set(q, k, v, spd, b, rows, keys)
    np.testing.assert_allclose(pl[h, i], np.log(np.exp(s).sum()), rtol=1e-12)
    # merging with an empty step changes nothing; merging into the empty state returns the step
    eo, el = oattn.attend_key_set(q, k, v, spd, b, rows, np.arange(0))
    o2, l2 = oattn.merge_state(o, lse, eo, el)
    np.testing.assert_array_equal(o2, o); np.testing.assert_array_equal(l2, lse)


def test_backward_blocks_over_a_partition_of_rows_and_keys_sum_to_the_full_backward():
    n = 150
    q, k, v, do, spd, b = make_case(n, 2, 32, 6, seed=41, directed=True)
    out, lse = oattn.forward_single(q, k, v, spd, b)
    full = oattn.backward_single(q, k, v, do, spd, b)
    row_parts = [np.arange(0, 48), np.arange(48, 128), np.arange(128, 150)]
    key_parts = [np.arange(0, 64), np.concatenate([np.arange(64, 100), np.arange(130, 150)]), np.arange(100, 130)]
    dq = np.zeros_like(q); dk = np.zeros_like(q); dv = np.zeros_like(q); db = np.zeros_like(b)
    for rows in row_parts:
        for keys in key_parts:
            pq, pk, pv, pb = oattn.backward_block(q, k, v, do, out, lse, spd, b, rows, keys)
            dq[rows] += pq; dk[keys] += pk; dv[keys] += pv; db += pb
    s = 1.0 / np.sqrt(32.0)
    for got, ref in zip((dq * s, dk * s, dv, db), full):
        np.testing.assert_allclose(got, ref, rtol=1e-10, atol=1e-13)
    # one block's dv by brute force
    rows, keys = row_parts[1], key_parts[1]
    _, _, pv, _ = oattn.backward_block(q, k, v, do, out, lse, spd, b, rows, keys)
    h, jj = 1, 40                                   # key 130 + (40 - 36)
    j = keys[jj]
    sc = (q[rows, h] @ k[j, h]) / np.sqrt(32.0) + b[h][spd[rows, j].astype(int)]
    np.testing.assert_allclose(pv[jj, h], (np.exp(sc - lse[h][rows])[:, None] * do[rows, h]).sum(0), rtol=1e-10, atol=1e-13)
