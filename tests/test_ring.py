"""Ring schedule of graph-aware context parallelism on CPU ranks (gloo, world size 3): every rank
drives `ring.ring_forward` with a step function built from the oracle, and the gathered result
must equal the one-shot forward.  Checks which block is where at which step, the two-part key
slices (super nodes once), and the carried state — not the CUDA kernels."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


N, N_SUPER, H, D_HEAD, MAX_DIST = 150, 22, 2, 32, 6


def _case():
    from paper_2609_34420_b200 import workloads as wl
    w = wl.small_workload([N], H, D_HEAD, MAX_DIST, seed=5, avg_degree=2.0, directed=True)
    t = w.tensors()
    f = wl.bf16_bits_to_f64
    from oracle import spd as ospd
    spd = ospd.spd_matrix(w.batch.row_ptr, w.batch.col_idx, MAX_DIST)
    return f(t.q), f(t.k), f(t.v), spd, t.bias.astype(np.float64)


def _worker(rank, world, port, out_q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from oracle import attention as oattn
    from paper_2609_34420_b200 import ring
    dist.init_process_group("gloo", rank=rank, world_size=world)
    q, k, v, spd, bias = _case()
    layout = ring.RingLayout.even(N, N_SUPER, world)
    a, b = layout.shards[rank]
    share = max(e - s for s, e in layout.shards)
    sa, sb = layout.super_range

    def block(x):                                   # own regular rows (padded to the common length) + super nodes
        blk = np.zeros((share + N_SUPER,) + x.shape[1:])
        blk[: b - a] = x[a:b]
        blk[share:] = x[sa:sb]
        return torch.from_numpy(blk)

    o = np.zeros((N, H, D_HEAD)); lse = np.full((H, N), -np.inf)
    seen = []

    def step(q_range, kv_range, sup, k_blk, v_blk, owner):
        # rebuild the key rows of this step from the ARRIVED block only (what a rank really holds)
        ka, kb = kv_range
        kk, vv = np.zeros_like(k), np.zeros_like(v)
        kk[ka:kb] = k_blk.numpy()[: kb - ka]; vv[ka:kb] = v_blk.numpy()[: kb - ka]
        kk[sa:sb] = k_blk.numpy()[share:]; vv[sa:sb] = v_blk.numpy()[share:]
        keys = np.concatenate([np.arange(ka, kb), np.arange(*sup)])
        rows = np.arange(*q_range)
        po, pl = oattn.attend_key_set(q, kk, vv, spd, bias, rows, keys)
        o[rows], lse[:, rows] = oattn.merge_state(o[rows], lse[:, rows], po, pl)
        seen.append((q_range, owner))

    ring.ring_forward(layout, block(k), block(v), step)
    out_q.put((rank, o[a:b], lse[:, a:b], o[sa:sb], lse[:, sa:sb], seen))
    dist.barrier()
    dist.destroy_process_group()


def test_three_rank_ring_reproduces_the_forward():
    world = 3
    ctx = mp.get_context("spawn")
    out_q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out_q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((out_q.get(timeout=180) for _ in range(world)), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    from oracle import attention as oattn
    from paper_2609_34420_b200 import ring
    q, k, v, spd, bias = _case()
    ro, rl = oattn.forward_single(q, k, v, spd, bias)
    layout = ring.RingLayout.even(N, N_SUPER, world)
    sa, sb = layout.super_range
    for rank, o_sh, l_sh, o_sup, l_sup, seen in res:
        a, b = layout.shards[rank]
        np.testing.assert_allclose(o_sh, ro[a:b], rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(l_sh, rl[:, a:b], rtol=1e-12)
        np.testing.assert_allclose(o_sup, ro[sa:sb], rtol=1e-10, atol=1e-13)      # every rank's replica of the super rows
        np.testing.assert_allclose(l_sup, rl[:, sa:sb], rtol=1e-12)
        owners = [own for (qr, own) in seen if qr == layout.shards[rank]]
        assert owners == [(rank - s) % world for s in range(world)]               # blocks arrive round the ring


def _bwd_worker(rank, world, port, out_q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from oracle import attention as oattn
    from paper_2609_34420_b200 import ring, workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    q, k, v, spd, bias = _case()
    w = wl.small_workload([N], H, D_HEAD, MAX_DIST, seed=5, avg_degree=2.0, directed=True)
    do = wl.bf16_bits_to_f64(w.tensors().dout)
    out, lse = oattn.forward_single(q, k, v, spd, bias)
    layout = ring.RingLayout.even(N, N_SUPER, world)
    a, b = layout.shards[rank]
    share = max(e - s for s, e in layout.shards)
    sa, sb = layout.super_range

    def block(x):
        blk = np.zeros((share,) + x.shape[1:]); blk[: b - a] = x[a:b]
        return torch.from_numpy(blk)

    # accumulators this rank owns: dq of its rows (and its share for the super rows), super-key dk / dv, dbias
    dq = np.zeros_like(q); dk_sup = np.zeros((N_SUPER, H, D_HEAD)); dv_sup = np.zeros((N_SUPER, H, D_HEAD)); db = np.zeros_like(bias)

    def step(q_range, kv_range, sup, k_blk, v_blk, dk_blk, dv_blk, owner):
        ka, kb = kv_range
        kk, vv = np.zeros_like(k), np.zeros_like(v)
        kk[ka:kb] = k_blk.numpy()[: kb - ka]; vv[ka:kb] = v_blk.numpy()[: kb - ka]       # the arrived block ...
        kk[sa:sb] = k[sa:sb]; vv[sa:sb] = v[sa:sb]                                      # ... and the local super-node replica
        rows = np.arange(*q_range); keys = np.concatenate([np.arange(ka, kb), np.arange(*sup)])
        pq, pk, pv, pb = oattn.backward_block(q, kk, vv, do, out, lse, spd, bias, rows, keys)
        dq[rows] += pq
        dk_blk.numpy()[: kb - ka] += pk[: kb - ka]; dv_blk.numpy()[: kb - ka] += pv[: kb - ka]
        if sup[1] > sup[0]:
            dk_sup[:] += pk[kb - ka:]; dv_sup[:] += pv[kb - ka:]
        db[:] += pb

    dk_own, dv_own = ring.ring_backward(layout, block(k), block(v), step)
    red = [torch.from_numpy(x) for x in (dq[sa:sb].copy(), dk_sup, dv_sup, db)]
    for t in red:
        dist.all_reduce(t)
    out_q.put((rank, dq[a:b], dk_own.numpy()[: b - a], dv_own.numpy()[: b - a], [t.numpy() for t in red]))
    dist.barrier()
    dist.destroy_process_group()


def test_three_rank_backward_ring_reproduces_the_backward():
    world = 3
    ctx = mp.get_context("spawn")
    out_q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_bwd_worker, args=(r, world, port, out_q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((out_q.get(timeout=180) for _ in range(world)), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    from oracle import attention as oattn
    from paper_2609_34420_b200 import ring, workloads as wl
    q, k, v, spd, bias = _case()
    w = wl.small_workload([N], H, D_HEAD, MAX_DIST, seed=5, avg_degree=2.0, directed=True)
    do = wl.bf16_bits_to_f64(w.tensors().dout)
    rdq, rdk, rdv, rdb = oattn.backward_single(q, k, v, do, spd, bias)
    layout = ring.RingLayout.even(N, N_SUPER, world)
    sa, sb = layout.super_range
    s_ = 1.0 / np.sqrt(float(D_HEAD))
    for rank, dq_sh, dk_sh, dv_sh, (dq_sup, dk_sup, dv_sup, db) in res:
        a, b = layout.shards[rank]
        np.testing.assert_allclose(dq_sh * s_, rdq[a:b], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dk_sh * s_, rdk[a:b], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dv_sh, rdv[a:b], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dq_sup * s_, rdq[sa:sb], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dk_sup * s_, rdk[sa:sb], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dv_sup, rdv[sa:sb], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(db, rdb, rtol=1e-9, atol=1e-12)


def _cp_worker(rank, world, port, out_q):
    """Forward ring, then backward ring fed by the forward's carried state, then the all-reduce of the replicated
    pieces: `ring.context_parallel_pass` end to end with oracle-backed step functions."""
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import torch.distributed as dist
    from oracle import attention as oattn
    from paper_2609_34420_b200 import ring, workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    q, k, v, spd, bias = _case()
    w = wl.small_workload([N], H, D_HEAD, MAX_DIST, seed=5, avg_degree=2.0, directed=True)
    do = wl.bf16_bits_to_f64(w.tensors().dout)
    layout = ring.RingLayout.even(N, N_SUPER, world)
    a, b = layout.shards[rank]
    share = max(e - s for s, e in layout.shards)
    sa, sb = layout.super_range

    def block(x, with_super):
        blk = np.zeros((share + (N_SUPER if with_super else 0),) + x.shape[1:])
        blk[: b - a] = x[a:b]
        if with_super:
            blk[share:] = x[sa:sb]
        return torch.from_numpy(blk)

    o = np.zeros((N, H, D_HEAD)); lse = np.full((H, N), -np.inf)

    def fwd_step(q_range, kv_range, sup, k_blk, v_blk, owner):
        ka, kb = kv_range
        kk, vv = np.zeros_like(k), np.zeros_like(v)
        kk[ka:kb] = k_blk.numpy()[: kb - ka]; vv[ka:kb] = v_blk.numpy()[: kb - ka]
        kk[sa:sb] = k_blk.numpy()[share:]; vv[sa:sb] = v_blk.numpy()[share:]
        rows = np.arange(*q_range); keys = np.concatenate([np.arange(ka, kb), np.arange(*sup)])
        po, pl = oattn.attend_key_set(q, kk, vv, spd, bias, rows, keys)
        o[rows], lse[:, rows] = oattn.merge_state(o[rows], lse[:, rows], po, pl)

    dq = np.zeros_like(q); dk_sup = np.zeros((N_SUPER, H, D_HEAD)); dv_sup = np.zeros((N_SUPER, H, D_HEAD)); db = np.zeros_like(bias)

    def bwd_step(q_range, kv_range, sup, k_blk, v_blk, dk_blk, dv_blk, owner):
        ka, kb = kv_range
        kk, vv = np.zeros_like(k), np.zeros_like(v)
        kk[ka:kb] = k_blk.numpy()[: kb - ka]; vv[ka:kb] = v_blk.numpy()[: kb - ka]
        kk[sa:sb] = k[sa:sb]; vv[sa:sb] = v[sa:sb]
        rows = np.arange(*q_range); keys = np.concatenate([np.arange(ka, kb), np.arange(*sup)])
        # the forward state of THIS rank (its rows only are final): what the backward of a rank may use
        pq, pk, pv, pb = oattn.backward_block(q, kk, vv, do, o, lse, spd, bias, rows, keys)
        dq[rows] += pq
        dk_blk.numpy()[: kb - ka] += pk[: kb - ka]; dv_blk.numpy()[: kb - ka] += pv[: kb - ka]
        if sup[1] > sup[0]:
            dk_sup[:] += pk[kb - ka:]; dv_sup[:] += pv[kb - ka:]
        db[:] += pb

    red = [torch.from_numpy(x) for x in (dk_sup, dv_sup, db)]
    dq_sup = torch.zeros(N_SUPER, H, D_HEAD, dtype=torch.float64)
    done = []

    def between():
        done.append("forward state final")

    dk_own, dv_own = ring.context_parallel_pass(layout, (block(k, True), block(v, True)), fwd_step,
                                                (block(k, False), block(v, False)), bwd_step, replicated=red, between=between)
    dq_sup += torch.from_numpy(dq[sa:sb]); dist.all_reduce(dq_sup)
    out_q.put((rank, o[a:b], dq[a:b], dk_own.numpy()[: b - a], dv_own.numpy()[: b - a], dq_sup.numpy(), [t.numpy() for t in red], done))
    dist.barrier()
    dist.destroy_process_group()


def test_three_rank_forward_then_backward_pass_with_the_all_reduce_of_the_replicated_sums():
    world = 3
    ctx = mp.get_context("spawn")
    out_q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_cp_worker, args=(r, world, port, out_q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((out_q.get(timeout=180) for _ in range(world)), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    from oracle import attention as oattn
    from paper_2609_34420_b200 import ring, workloads as wl
    q, k, v, spd, bias = _case()
    w = wl.small_workload([N], H, D_HEAD, MAX_DIST, seed=5, avg_degree=2.0, directed=True)
    do = wl.bf16_bits_to_f64(w.tensors().dout)
    ro, _ = oattn.forward_single(q, k, v, spd, bias)
    rdq, rdk, rdv, rdb = oattn.backward_single(q, k, v, do, spd, bias)
    layout = ring.RingLayout.even(N, N_SUPER, world)
    sa, sb = layout.super_range
    s_ = 1.0 / np.sqrt(float(D_HEAD))
    for rank, o_sh, dq_sh, dk_sh, dv_sh, dq_sup, (dk_sup, dv_sup, db), done in res:
        a, b = layout.shards[rank]
        assert done == ["forward state final"]
        np.testing.assert_allclose(o_sh, ro[a:b], rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(dq_sh * s_, rdq[a:b], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dk_sh * s_, rdk[a:b], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dv_sh, rdv[a:b], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dq_sup * s_, rdq[sa:sb], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dk_sup * s_, rdk[sa:sb], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(dv_sup, rdv[sa:sb], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(db, rdb, rtol=1e-9, atol=1e-12)
