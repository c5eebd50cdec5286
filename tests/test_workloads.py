"""Seeded generators: determinism, structure and the shapes the named workloads promise."""
import numpy as np
import pytest

from paper_2609_34420_b200 import workloads as wl


def check_csr(rp, ci, n):
    assert rp.dtype == np.int32 and ci.dtype == np.int32 and len(rp) == n + 1 and rp[0] == 0 and rp[-1] == len(ci)
    assert (np.diff(rp) >= 0).all()
    src = np.repeat(np.arange(n), np.diff(rp))
    assert (src != ci).all()                                   # no self loops
    key = src.astype(np.int64) * n + ci
    assert (np.diff(key) > 0).all()                            # sorted rows, no duplicates
    assert set(map(tuple, np.stack([ci, src], 1).tolist())) == set(map(tuple, np.stack([src, ci], 1).tolist()))


@pytest.mark.parametrize("name,n,H,d,D,deg", [("tiny_er256", 256, 4, 32, 8, 8.0), ("ba4096", 4096, 8, 64, 16, 10.0),
                                              ("powerlaw16k", 16384, 8, 64, 20, 14.0)])
def test_named_workloads(name, n, H, d, D, deg):
    w = wl.make_workload(name)
    assert (w.batch.n_total, w.n_heads, w.head_dim, w.max_dist) == (n, H, d, D)
    check_csr(w.batch.row_ptr, w.batch.col_idx, n)
    assert abs(wl.csr_stats((w.batch.row_ptr, w.batch.col_idx))["deg_mean"] - deg) < 0.1 * deg
    w2 = wl.make_workload(name)
    np.testing.assert_array_equal(w.batch.col_idx, w2.batch.col_idx)
    t, t2 = w.tensors(), w2.tensors()
    np.testing.assert_array_equal(t.q, t2.q)
    assert t.q.shape == (n, H, d) and t.q.dtype == np.uint16 and t.bias.shape == (H, D + 2)


def test_varlen_batch_layout():
    w = wl.make_workload("varlen_rgg64")
    b = w.batch
    sizes = np.diff(b.cu_seqlens)
    assert b.n_graphs == 64 and sizes.min() >= 512 and sizes.max() <= 2048
    assert (b.spd_ld == (sizes + 15) // 16 * 16).all() and (b.spd_offsets % 16 == 0).all()
    # block diagonal: every edge stays inside its graph
    src = np.repeat(np.arange(b.n_total), np.diff(b.row_ptr))
    g_of = np.searchsorted(b.cu_seqlens, np.arange(b.n_total), side="right") - 1
    assert (g_of[src] == g_of[b.col_idx]).all()
    rp, ci = b.graph_csr(5)
    check_csr(rp, ci, int(sizes[5]))


def test_bf16_round_trip_is_rne():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.1415927, 1e-30, 65504.0], np.float32)
    bits = wl.f32_to_bf16_bits(x)
    # 1.00390625 = 1 + 2^-8 is a tie between 1.0 and 1+2^-7 -> even (1.0); 1.01171875 = 1 + 3*2^-8 -> 1+2^-6
    assert wl.bf16_bits_to_f32(bits)[1] == 1.0 and wl.bf16_bits_to_f32(bits)[2] == 1.015625
    import torch
    ref = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, ref)
