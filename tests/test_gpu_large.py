"""Parity at the full sizes the benchmark times (same entry points, same launch configuration).

At 16 384 nodes the fp64 oracle runs in full (every query row).  At 65 536 nodes it cannot
materialise 65536^2 scores per head in test time, so attention is checked with the row-slab protocol:
the oracle computes full rows for a subset R of query rows -- the first, a middle and the last
complete 256-row block of the launch (what one thread block of the forward owns) plus seeded random
rows -- giving forward O, LSE and dQ on R; the GPU backward is run with dO zeroed outside R, which
makes dK, dV and dBias depend on the rows of R only, so they are compared with the oracle's sums over R.
Gradients are compared over the whole tensor, per head and per block of 128 rows.
The SPD matrix is compared in full (bit-exact)."""
import numpy as np
import pytest
import torch

from oracle import attention as oattn
from oracle import spd as ospd
from paper_2609_34420_b200 import binding as gt
from paper_2609_34420_b200 import workloads as wl

from gpu_util import bf16_tensor, device_batch, device_csr, localized_rel_l2, rel_l2, to_f64

pytestmark = pytest.mark.gpu

O_MAX_ABS, LSE_MAX_ABS, GRAD_REL_L2, CHUNK_REL_L2 = 1e-2, 1e-3, 2e-2, 1e-3


def slab_rows(n: int, n_random: int) -> np.ndarray:
    """First, middle and last complete 256-row block plus `n_random` seeded rows elsewhere."""
    blocks = [0, (n // 512) * 256, (n // 256 - 1) * 256]
    fixed = np.unique(np.concatenate([np.arange(b, b + 256) for b in blocks]))
    rest = np.setdiff1d(np.arange(n), fixed)
    extra = np.random.default_rng(2024).choice(rest, size=n_random, replace=False)
    return np.sort(np.concatenate([fixed, extra]))


def run_large(name: str, n_slab: int, full_spd_oracle: bool):
    w = wl.make_workload(name)
    b, t = w.batch, w.tensors()
    n, H, d, D = b.n_total, w.n_heads, w.head_dim, w.max_dist
    dev = "cuda"
    bt = device_batch(b, dev)
    rp, ci = device_csr(b, dev)

    # ---- SPD: GPU build, bit-exact against the BFS oracle ----
    spd = torch.empty(b.spd_bytes, dtype=torch.uint8, device=dev)
    gt.gt_check(gt.gt_spd_build(rp, ci, bt, D, spd))
    rows = np.arange(n) if n_slab >= n else slab_rows(n, n_slab - 768)
    ld = int(b.spd_ld[0])
    if full_spd_oracle:
        ref = ospd.spd_matrix(b.row_ptr, b.col_idx, D)
        got = spd.cpu().numpy().reshape(n, ld)
        assert np.array_equal(got, ref)
        spd_rows = np.ascontiguousarray(ref[rows])
        del ref, got
    else:
        spd_rows = ospd.spd_rows(b.row_ptr, b.col_idx, D, rows)
        got_rows = spd.view(n, ld)[torch.from_numpy(rows).to(dev)].cpu().numpy()
        assert np.array_equal(got_rows, spd_rows)

    # ---- forward (unchunked and chunked) ----
    q, k, v, do = (bf16_tensor(x, dev) for x in (t.q, t.k, t.v, t.dout))
    bias = torch.tensor(t.bias, device=dev)
    out, out_c = torch.empty_like(q), torch.empty_like(q)
    lse, lse_c = torch.empty(H, n, device=dev), torch.empty(H, n, device=dev)
    gt.gt_check(gt.gt_biased_attn_fwd(q, k, v, spd, bias, bt, D, out, lse))
    gt.gt_check(gt.gt_biased_attn_fwd_chunked(q, k, v, spd, bias, bt, D, out_c, lse_c, max(w.n_kv_chunks, 2)))
    assert rel_l2(to_f64(out_c), to_f64(out)) <= CHUNK_REL_L2
    assert (lse_c - lse).abs().max().item() <= LSE_MAX_ABS

    f = wl.bf16_bits_to_f64
    qf, kf, vf, dof, bf = f(t.q), f(t.k), f(t.v), f(t.dout), t.bias.astype(np.float64)
    ro, rl = oattn.forward_single(qf, kf, vf, spd_rows, bf, rows=rows, compact_spd=True)
    rows_t = torch.from_numpy(rows).to(dev)
    assert np.abs(to_f64(out[rows_t]) - ro).max() <= O_MAX_ABS
    assert np.abs(to_f64(lse[:, rows_t]) - rl).max() <= LSE_MAX_ABS

    # ---- backward with dO restricted to the slab ----
    do_masked = torch.zeros_like(do)
    do_masked[rows_t] = do[rows_t]
    dq, dk, dv = (torch.empty_like(q) for _ in range(3))
    dbias = torch.empty_like(bias)
    gt.gt_check(gt.gt_biased_attn_bwd(q, k, v, out, do_masked, lse, spd, bias, bt, D, dq, dk, dv, dbias))
    rdq, rdk, rdv, rdb = oattn.backward_single(qf, kf, vf, dof, spd_rows, bf, rows=rows, compact_spd=True)
    errs = {"dq": rel_l2(to_f64(dq[rows_t]), rdq), "dk": rel_l2(to_f64(dk), rdk),
            "dv": rel_l2(to_f64(dv), rdv), "dbias": rel_l2(to_f64(dbias), rdb)}
    # the slab's rows in order: its three complete 256-row blocks are two 128-row blocks each
    for name_, got_, ref_ in (("dq", to_f64(dq[rows_t]), rdq), ("dk", to_f64(dk), rdk), ("dv", to_f64(dv), rdv)):
        loc = localized_rel_l2(got_, ref_)
        errs[name_ + "/head"], errs[name_ + "/block128"] = loc["head"], loc["block"]
    assert all(e <= GRAD_REL_L2 for e in errs.values()), errs
    mask = torch.ones(n, dtype=torch.bool, device=dev)
    mask[rows_t] = False
    if bool(mask.any()):
        assert (dq[mask].float().abs().max().item() == 0.0)

    # ---- chunked backward (same dO): equals the unchunked backward, chunk shares add up ----
    C = max(w.n_kv_chunks, 2)
    dq_c, dk_c, dv_c = (torch.empty_like(q) for _ in range(3))
    dbias_c = torch.empty_like(bias)
    db_chunks = torch.empty((C,) + tuple(bias.shape), device=dev)
    gt.gt_check(gt.gt_biased_attn_bwd_chunked(q, k, v, out, do_masked, lse, spd, bias, bt, D, C, dq_c, dk_c, dv_c, dbias_c, db_chunks))
    for got, ref_ in ((dq_c, dq), (dk_c, dk), (dv_c, dv), (dbias_c, dbias)):
        assert rel_l2(to_f64(got), to_f64(ref_)) <= CHUNK_REL_L2
    assert rel_l2(to_f64(db_chunks.sum(0)), to_f64(dbias_c)) <= 1e-5


def test_powerlaw16k_full_spd_and_full_oracle_attention():
    run_large("powerlaw16k", n_slab=16384, full_spd_oracle=True)


def test_powerlaw64k_full_spd_and_row_slab_attention():
    run_large("powerlaw64k", n_slab=2048, full_spd_oracle=True)


# ---- single graphs beyond the shared-memory BFS state: the bit-matrix build ----
def _spd_of(csr, max_dist):
    w = wl.Workload("big", wl.pack_graphs([csr]), 1, 32, max_dist)
    bt = device_batch(w.batch)
    rp, ci = device_csr(w.batch)
    spd = torch.empty(w.batch.spd_bytes, dtype=torch.uint8, device="cuda")
    gt.gt_spd_build(rp, ci, bt, max_dist, spd)
    torch.cuda.synchronize()
    n = w.batch.n_total
    return w, spd.cpu().numpy().reshape(n, -1)


def test_bit_matrix_build_directed_ragged_with_hub_and_isolated_vertices():
    n = 18001                                   # pitch 18016: padding columns; three column blocks, the last ragged
    rng = np.random.Generator(np.random.PCG64(5))
    m = 3 * n
    src = rng.integers(0, n - 200, size=m)      # the last 200 vertices have no out-edges
    dst = rng.integers(0, n - 100, size=m)      # the last 100 are isolated
    hub_dst = rng.choice(n - 100, size=3000, replace=False)      # a vertex split over many work items
    src = np.concatenate([src, np.full(3000, 7)])
    dst = np.concatenate([dst, hub_dst])
    csr = wl.csr_from_edges(n, src, dst, symmetric=False)
    w, got = _spd_of(csr, 7)
    exp = ospd.spd_matrix(w.batch.row_ptr, w.batch.col_idx, 7)
    assert got.shape == exp.shape
    np.testing.assert_array_equal(got, exp)


@pytest.mark.parametrize("base,one_longer", [(2, False), (2, True), (3, False), (6, True)])
def test_bit_matrix_build_depth_around_the_kept_levels(base, one_longer):
    """Chains of `base` vertices hanging off one centre (one of them a vertex longer if asked): the longest path
    has 2 * base (+ 1) hops.  The build keeps the frontiers of five levels for its output pass: 4 hops end before
    that, 5 exactly there (the pass runs while the last level still found pairs, the level after finds none),
    6 add one level and 13 add eight levels that blend into written rows.  Directed extras make the matrix
    asymmetric; a few vertices stay isolated."""
    n_chains = 17200 // base
    lengths = [base] * n_chains
    if one_longer:
        lengths[n_chains // 2] += 1
    firsts = 1 + np.concatenate([[0], np.cumsum(lengths)[:-1]])
    n = 1 + int(np.sum(lengths)) + 37           # 37 isolated vertices at the end
    src, dst = [], []
    for first, length in zip(firsts, lengths):
        src.append(0); dst.append(int(first))
        for t in range(length - 1):
            src.append(int(first) + t); dst.append(int(first) + t + 1)
    src, dst = np.array(src), np.array(dst)
    both_src, both_dst = np.concatenate([src, dst]), np.concatenate([dst, src])
    # one-way shortcuts from some chain ends to the first vertex of the next chain
    pick = np.arange(0, n_chains - 1, 97)
    ends = firsts[pick] + np.array(lengths)[pick] - 1
    both_src = np.concatenate([both_src, ends]); both_dst = np.concatenate([both_dst, firsts[pick + 1]])
    csr = wl.csr_from_edges(n, both_src, both_dst, symmetric=False)
    w, got = _spd_of(csr, 24)
    exp = ospd.spd_matrix(w.batch.row_ptr, w.batch.col_idx, 24)
    assert int(exp[exp <= 24].max()) == 2 * base + (1 if one_longer else 0)
    np.testing.assert_array_equal(got, exp)


def test_bit_matrix_build_ring_runs_thousands_of_levels_and_clips():
    n = 17500
    i = np.arange(n)
    csr = wl.csr_from_edges(n, i, (i + 1) % n, symmetric=True)
    w, got = _spd_of(csr, 50)
    rows = np.array([0, 1, 8191, 8192, 12345, n - 1])
    j = np.arange(n)
    for r in rows:
        ring = np.minimum((j - r) % n, (r - j) % n)
        np.testing.assert_array_equal(got[r, :n], np.minimum(ring, 50))
    assert (got[:, n:] == 255).all()
