"""Run the hot path a few times on one named workload and print CUDA-event timings.

    python -m paper_2609_34420_b200.profile_case WORKLOAD [REPS] [spd|fwd|bwd|chunked|all]
    python -m paper_2609_34420_b200.profile_case featN [REPS] [VECTORS]

WORKLOAD is one of the named workloads (tiny_er256, ba4096, powerlaw16k, powerlaw64k,
varlen_rgg64) or plN for a power-law graph of N nodes (H=8, d=64, max_dist=24).  A small,
self-contained timing command line for one entry point at a time.  featN times the feature-bias
variant on N nodes (H=8, d=64) with VECTORS distinct feature vectors (default 12): the fp32 path on
the CUDA cores, and the code matrix through the tensor-core kernels of the bucket form.
"""
from __future__ import annotations

import sys

import torch

from . import binding as gt
from . import workloads as wl


def timed_ms(fn, reps):
    fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def feature_timings(n: int, reps: int, n_vec: int, cuda_core_path: bool = True) -> dict:
    """CUDA-event timings (ms) of the feature-bias variant on n nodes, H=8, d=64, n_vec distinct feature vectors."""
    H, d = 8, 64
    dev = torch.device("cuda", torch.cuda.current_device())
    g = torch.Generator(device=dev).manual_seed(1)
    q, k, v, do = (torch.randn(n, H, d, device=dev, generator=g).bfloat16() for _ in range(4))
    wt = torch.randn(H, 4, device=dev, generator=g) * 0.01
    vec = torch.randint(0, 256, (n_vec, 4), device=dev, generator=g, dtype=torch.uint8)
    feat = vec[torch.randint(0, n_vec, (n, n), device=dev, generator=g)].contiguous()
    batch = gt.Batch(n)
    out, dq, dk, dv = (torch.empty_like(q) for _ in range(4))
    lse, dw = torch.empty(H, n, device=dev), torch.empty_like(wt)
    res = {"n": n, "n_heads": H, "head_dim": d, "fwd_flops": 4.0 * H * d * n * n, "bwd_flops": 10.0 * H * d * n * n}
    if cuda_core_path:
        res["fp32_fwd_ms"] = timed_ms(lambda: gt.gt_feature_attn_fwd(q, k, v, feat, wt, batch, out, lse), reps)
        ws_b = gt.gt_feature_attn_bwd(q, k, v, do, lse, feat, wt, batch, dq, dk, dv, dw)
        res["fp32_bwd_ms"] = timed_ms(lambda: gt.gt_feature_attn_bwd(q, k, v, do, lse, feat, wt, batch, dq, dk, dv, dw, ws_b), reps)
        gt.gt_check(ws_b)
    ld = (n + 15) // 16 * 16
    codes = torch.empty(n * ld, dtype=torch.uint8, device=dev)
    vectors = torch.empty(256, dtype=torch.int32, device=dev)
    ws_e = gt.gt_feature_encode(feat, batch, codes, vectors)
    gt.gt_check(ws_e)
    width = max(gt.gt_feature_encode_count(ws_e), 3)
    res["codes"] = width
    res["encode_ms"] = timed_ms(lambda: gt.gt_feature_encode(feat, batch, codes, vectors, ws_e), reps)
    table, dtable = torch.empty(H, width, device=dev), torch.empty(H, width, device=dev)
    out32 = torch.empty(n, H, d, device=dev)

    def fwd(ws=None):
        gt.gt_feature_code_table(wt, vectors, table)
        return gt.gt_biased_attn_fwd_ex(q, k, v, codes, table, batch, width - 2, out, lse, out32, ws)

    def bwd(ws=None):
        ws = gt.gt_biased_attn_bwd_ex(q, k, v, out, do, lse, codes, table, batch, width - 2, dq, dk, dv, dtable, out32, ws)
        gt.gt_feature_code_dweights(dtable, vectors, dw)
        return ws

    ws_f, ws_bb = fwd(), bwd()
    res["codes_fwd_ms"] = timed_ms(lambda: fwd(ws_f), reps)
    res["codes_bwd_ms"] = timed_ms(lambda: bwd(ws_bb), reps)
    gt.gt_check(ws_f)
    gt.gt_check(ws_bb)
    return res


def feature_case(n: int, reps: int, n_vec: int) -> int:
    r = feature_timings(n, reps, n_vec)
    tf = lambda flops, ms: flops / ms / 1e9
    print(f"feature fwd (CUDA cores) {r['fp32_fwd_ms']:.3f} ms  {tf(r['fwd_flops'], r['fp32_fwd_ms']):.1f} TFLOP/s")
    print(f"feature bwd (CUDA cores) {r['fp32_bwd_ms']:.3f} ms  {tf(r['bwd_flops'], r['fp32_bwd_ms']):.1f} TFLOP/s")
    print(f"feature encode {r['encode_ms']:.3f} ms  {n * n * 5 / r['encode_ms'] / 1e6:.1f} GB/s  ({r['codes']} codes)")
    print(f"feature fwd (codes, fp32 output too) {r['codes_fwd_ms']:.3f} ms  {tf(r['fwd_flops'], r['codes_fwd_ms']):.1f} TFLOP/s")
    print(f"feature bwd (codes) {r['codes_bwd_ms']:.3f} ms  {tf(r['bwd_flops'], r['codes_bwd_ms']):.1f} TFLOP/s")
    return 0


def main(argv) -> int:
    name = argv[1] if len(argv) > 1 else "powerlaw16k"
    reps = int(argv[2]) if len(argv) > 2 else 1
    if name.startswith("feat") and name[4:].isdigit():
        return feature_case(int(name[4:]), reps, int(argv[3]) if len(argv) > 3 else 12)
    what = argv[3] if len(argv) > 3 else "all"
    if name.startswith("pl") and name[2:].isdigit():
        w = wl.Workload(name, wl.pack_graphs([wl.chung_lu_power_law(int(name[2:]), 12.0, 2.1, 0)]), 8, 64, 24)
    else:
        w = wl.make_workload(name)
    b = w.batch
    T, H, d, D = b.n_total, w.n_heads, w.head_dim, w.max_dist
    dev = torch.device("cuda", 0)
    single = b.n_graphs == 1
    batch = gt.Batch(T, b.n_graphs, b.max_seqlen,
                     None if single else torch.from_numpy(b.cu_seqlens).to(dev),
                     None if single else torch.from_numpy(b.spd_offsets).to(dev))
    rp, ci = torch.from_numpy(b.row_ptr).to(dev), torch.from_numpy(b.col_idx).to(dev)
    g = torch.Generator(device=dev).manual_seed(1)
    q, k, v, do = (torch.randn(T, H, d, device=dev, generator=g).bfloat16() for _ in range(4))
    bias = torch.randn(H, D + 2, device=dev, generator=g) * 0.5
    spd = torch.empty(b.spd_bytes, dtype=torch.uint8, device=dev)
    out, dq, dk, dv, out_c = (torch.empty_like(q) for _ in range(5))
    lse, lse_c = torch.empty(H, T, device=dev), torch.empty(H, T, device=dev)
    dbias = torch.empty_like(bias)
    ws_spd = gt.gt_spd_build(rp, ci, batch, D, spd)
    ws_fwd = gt.gt_biased_attn_fwd(q, k, v, spd, bias, batch, D, out, lse)
    ws_bwd = gt.gt_biased_attn_bwd(q, k, v, out, do, lse, spd, bias, batch, D, dq, dk, dv, dbias)
    for ws in (ws_spd, ws_fwd, ws_bwd):
        gt.gt_check(ws)

    def timed(fn):
        return timed_ms(fn, reps)

    f_fwd, f_bwd = w.attn_flops()
    if what in ("all", "spd"):
        ms = timed(lambda: gt.gt_spd_build(rp, ci, batch, D, spd, ws_spd))
        print(f"spd_build {ms:.3f} ms  {b.spd_bytes / ms / 1e6:.1f} GB/s")
    if what in ("all", "fwd"):
        ms = timed(lambda: gt.gt_biased_attn_fwd(q, k, v, spd, bias, batch, D, out, lse, ws_fwd))
        print(f"fwd {ms:.3f} ms  {f_fwd / ms / 1e9:.1f} TFLOP/s")
    if what in ("all", "bwd"):
        ms = timed(lambda: gt.gt_biased_attn_bwd(q, k, v, out, do, lse, spd, bias, batch, D, dq, dk, dv, dbias, ws_bwd))
        print(f"bwd {ms:.3f} ms  {f_bwd / ms / 1e9:.1f} TFLOP/s")
    if what in ("all", "chunked") and single:
        ws_c = gt.gt_biased_attn_fwd_chunked(q, k, v, spd, bias, batch, D, out_c, lse_c, max(w.n_kv_chunks, 2))
        ms = timed(lambda: gt.gt_biased_attn_fwd_chunked(q, k, v, spd, bias, batch, D, out_c, lse_c,
                                                         max(w.n_kv_chunks, 2), None, ws_c))
        print(f"fwd_chunked {ms:.3f} ms  {f_fwd / ms / 1e9:.1f} TFLOP/s")
        gt.gt_check(ws_c)
    for ws in (ws_spd, ws_fwd, ws_bwd):
        gt.gt_check(ws)
    return 0


if __name__ == "__main__":
    sys.exit(main(sys.argv))
