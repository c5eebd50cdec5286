"""Graph-aware context parallelism over `torch.distributed` (Sec. GA-CP): the ring that drives
`gt_biased_attn_fwd_step`.

Rank r owns the regular nodes of shard r (its query rows and its K/V block) and a replica of the
super nodes.  A forward pass is P steps: at step s the rank attends to the K/V block of rank
(r - s) mod P, which is in its receive buffer, while the block travels on to rank r + 1.  The bias
columns of a step are the block's GLOBAL node indices (two-part slice: the block's regular range,
plus the super-node range at step 0 only, so that the replicated super nodes are counted once).
The softmax state (o_acc, lse_acc) is carried from step to step by the step function.

Everything here is plumbing: which block is where, what to send, when to call the step.  The
arithmetic is the step function's — `device_step` wraps the C-ABI call; tests drive the same
schedule on CPU ranks (gloo) with a step function of their own.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist

Range = Tuple[int, int]


@dataclass
class RingLayout:
    """Global index ranges: shard r of the regular nodes is rows [shards[r]), the super nodes are
    rows [super_range) (replicated on every rank; may be empty)."""
    shards: List[Range]
    super_range: Range

    @staticmethod
    def even(n_total: int, n_super: int, world: int, align: int = 16) -> "RingLayout":
        """Regular nodes [0, n_total - n_super) in `world` contiguous shards whose starts are multiples
        of `align` (the step kernel fetches bias columns in aligned pieces); super nodes last."""
        n_reg = n_total - n_super
        share = ((n_reg + world - 1) // world + align - 1) // align * align
        return RingLayout([(min(r * share, n_reg), min((r + 1) * share, n_reg)) for r in range(world)],
                          (n_reg, n_total))


# step(q_range, kv_range, super_range_or_empty, k_block, v_block, block_owner) -> None
StepFn = Callable[[Range, Range, Range, torch.Tensor, torch.Tensor, int], None]


def ring_forward(layout: RingLayout, k_own: torch.Tensor, v_own: torch.Tensor, step: StepFn,
                 group: Optional[dist.ProcessGroup] = None, rank: Optional[int] = None,
                 world: Optional[int] = None) -> None:
    """One context-parallel forward on this rank.

    k_own, v_own: this rank's K/V block, rows = its regular shard followed by the super nodes
    ([shard_len + n_super, H, d]); all ranks' blocks have the same shape (pad the last shard).
    `step` is called once per ring step and once more for the super nodes' own query rows per step;
    it receives the block that is current at that step and must have consumed it when it returns
    (or have ordered its use before later writes to the buffer on the same stream)."""
    if world is None:
        world = dist.get_world_size(group) if dist.is_initialized() else 1
    if rank is None:
        rank = dist.get_rank(group) if dist.is_initialized() else 0
    assert len(layout.shards) == world
    cur_k, cur_v = k_own, v_own
    bufs = [(torch.empty_like(k_own), torch.empty_like(v_own)) for _ in range(2)] if world > 1 else []
    empty: Range = (0, 0)
    for s in range(world):
        owner = (rank - s) % world
        reqs = []
        if s + 1 < world:                       # pass the block on while it is being used
            nxt_k, nxt_v = bufs[s % 2]          # the current block sits in the own tensors or in bufs[(s - 1) % 2]
            dst, src = (rank + 1) % world, (rank - 1) % world
            reqs = dist.batch_isend_irecv([dist.P2POp(dist.isend, cur_k, dst, group), dist.P2POp(dist.isend, cur_v, dst, group),
                                           dist.P2POp(dist.irecv, nxt_k, src, group), dist.P2POp(dist.irecv, nxt_v, src, group)])
        sup = layout.super_range if s == 0 else empty
        step(layout.shards[rank], layout.shards[owner], sup, cur_k, cur_v, owner)         # the shard's rows
        if layout.super_range[1] > layout.super_range[0]:
            step(layout.super_range, layout.shards[owner], sup, cur_k, cur_v, owner)      # the super nodes' rows
        for r in reqs:
            r.wait()
        if s + 1 < world:
            cur_k, cur_v = bufs[s % 2]


def device_step(binding, q, k_full, v_full, spd, bias, batch, max_dist: int, layout: RingLayout,
                o_acc, lse_acc, out=None, workspace=None) -> StepFn:
    """Step function backed by `gt_biased_attn_fwd_step`.  The C ABI addresses keys by global row in
    full-size K/V tensors, so an arriving block is first copied to its rows of `k_full` / `v_full`
    (device-to-device, same stream); `q`, `spd` hold the rows this rank needs at their global
    positions."""
    n_super = layout.super_range[1] - layout.super_range[0]
    state = {"ws": workspace}

    def step(q_range: Range, kv_range: Range, sup: Range, k_blk, v_blk, owner: int) -> None:
        a, b = kv_range
        k_full[a:b].copy_(k_blk[: b - a], non_blocking=True)
        v_full[a:b].copy_(v_blk[: b - a], non_blocking=True)
        if sup[1] > sup[0]:
            k_full[sup[0]:sup[1]].copy_(k_blk[k_blk.shape[0] - n_super:], non_blocking=True)
            v_full[sup[0]:sup[1]].copy_(v_blk[v_blk.shape[0] - n_super:], non_blocking=True)
        state["ws"] = binding.gt_biased_attn_fwd_step(q, k_full, v_full, spd, bias, batch, max_dist, q_range, kv_range, sup,
                                                      o_acc, lse_acc, out, state["ws"])

    return step


# bwd_step(q_range, kv_range, super_range_or_empty, k_block, v_block, dk_block, dv_block, block_owner) -> None
BwdStepFn = Callable[[Range, Range, Range, torch.Tensor, torch.Tensor, torch.Tensor, torch.Tensor, int], None]


def ring_backward(layout: RingLayout, k_own: torch.Tensor, v_own: torch.Tensor, step: BwdStepFn,
                  group: Optional[dist.ProcessGroup] = None, rank: Optional[int] = None,
                  world: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """One context-parallel backward on this rank; returns (dk_own, dv_own), the unscaled sums of this rank's
    own regular key rows after they have been round the ring.

    k_own, v_own: the rank's REGULAR key/value rows only ([shard_len, H, d], same shape on all ranks; the
    super nodes' K/V are replicated and do not travel).  A block travels together with its dk / dv sums:
    at step s the rank holds the block of rank (r - s) mod P, adds what its queries contribute, and passes
    it on; after P hops the block is home again.  Pairs are visited exactly once:
      * the rank's regular queries see every regular block once, and the super-node keys at step 0;
      * the super-node QUERY rows are handled at a block's home rank (step 0) for its regular keys, and on
        rank 0 for the super-node keys.
    What is replicated ends up as per-rank partial sums — dq of the super rows, dk / dv of the super keys,
    dbias — and is summed by the caller (all-reduce) after this function: the step function owns those
    accumulators, this function only moves the blocks."""
    if world is None:
        world = dist.get_world_size(group) if dist.is_initialized() else 1
    if rank is None:
        rank = dist.get_rank(group) if dist.is_initialized() else 0
    assert len(layout.shards) == world
    # the sums travel in fp32 when K/V are 16-bit tensors (they are unscaled partial sums over many query rows)
    sum_dtype = torch.float32 if k_own.dtype in (torch.bfloat16, torch.float16) else k_own.dtype
    cur = [k_own, v_own, torch.zeros_like(k_own, dtype=sum_dtype), torch.zeros_like(v_own, dtype=sum_dtype)]
    bufs = [[torch.empty_like(cur[t]) for t in range(4)] for _ in range(2)] if world > 1 else []
    empty: Range = (0, 0)
    has_super = layout.super_range[1] > layout.super_range[0]
    for s in range(world):
        owner = (rank - s) % world
        step(layout.shards[rank], layout.shards[owner], layout.super_range if s == 0 else empty, *cur, owner)
        if has_super and s == 0:
            step(layout.super_range, layout.shards[owner], layout.super_range if rank == 0 else empty, *cur, owner)
        if world > 1:                           # the sums always move on (the last hop takes them home), K and V only while needed
            nxt = bufs[s % 2]
            dst, src = (rank + 1) % world, (rank - 1) % world
            which = range(4) if s + 1 < world else range(2, 4)
            ops = [dist.P2POp(dist.isend, cur[t], dst, group) for t in which] + [dist.P2POp(dist.irecv, nxt[t], src, group) for t in which]
            for r in dist.batch_isend_irecv(ops):
                r.wait()
            cur = [nxt[t] if t in which else cur[t] for t in range(4)]
    return cur[2], cur[3]


def device_bwd_step(binding, q, k_full, v_full, dout, bias, batch, max_dist: int, layout: RingLayout,
                    dq_acc, dk_acc, dv_acc, dbias_acc, context) -> BwdStepFn:
    """Backward step function backed by `gt_biased_attn_bwd_step` (counterpart of `device_step`).

    The C ABI addresses keys by global row: an arriving block's K/V rows are copied to their rows of the
    full-length `k_full` / `v_full`, and the sums that travel with the block (`dk_blk`, `dv_blk`, unscaled
    fp32) are copied to the same rows of the full-length accumulators `dk_acc` / `dv_acc` before the call and
    back into the travelling buffers after it, all on the current stream.  The super nodes' K/V are the
    rank's own replica (already in `k_full` / `v_full`); their dK/dV rows of the accumulators, the super
    rows of `dq_acc` and `dbias_acc` are this rank's partial sums, which the caller all-reduces at the end.
    `context` comes from `gt_biased_attn_bwd_step_prepare`."""

    def step(q_range: Range, kv_range: Range, sup: Range, k_blk, v_blk, dk_blk, dv_blk, owner: int) -> None:
        a, b = kv_range
        if b > a:
            k_full[a:b].copy_(k_blk[: b - a], non_blocking=True)
            v_full[a:b].copy_(v_blk[: b - a], non_blocking=True)
            dk_acc[a:b].copy_(dk_blk[: b - a], non_blocking=True)
            dv_acc[a:b].copy_(dv_blk[: b - a], non_blocking=True)
        binding.gt_biased_attn_bwd_step(q, k_full, v_full, dout, bias, batch, max_dist, q_range, kv_range, sup,
                                        dq_acc, dk_acc, dv_acc, dbias_acc, context)
        if b > a:
            dk_blk[: b - a].copy_(dk_acc[a:b], non_blocking=True)
            dv_blk[: b - a].copy_(dv_acc[a:b], non_blocking=True)

    return step


def context_parallel_pass(layout: RingLayout, fwd_blocks: Tuple[torch.Tensor, torch.Tensor], fwd_step: StepFn,
                          bwd_blocks: Tuple[torch.Tensor, torch.Tensor], bwd_step: BwdStepFn,
                          replicated: Sequence[torch.Tensor] = (), between: Optional[Callable[[], None]] = None,
                          group: Optional[dist.ProcessGroup] = None, rank: Optional[int] = None,
                          world: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """One forward + backward of graph-aware context parallelism on this rank: the forward ring (K/V blocks
    with the super nodes attached), `between()` (e.g. the backward's prepare call, once the forward state is
    final), the backward ring (regular K/V rows travelling with their dK/dV sums), then the all-reduce of
    what is replicated on every rank (`replicated`: the super rows of dq, the super keys' dk / dv, dbias --
    per-rank partial sums until here).  Returns the rank's own (dk, dv) sums as `ring_backward` does."""
    ring_forward(layout, fwd_blocks[0], fwd_blocks[1], fwd_step, group, rank, world)
    if between is not None:
        between()
    dk_own, dv_own = ring_backward(layout, bwd_blocks[0], bwd_blocks[1], bwd_step, group, rank, world)
    if dist.is_initialized() and (world is None or world > 1):
        for t in replicated:
            dist.all_reduce(t, group=group)
    return dk_own, dv_own
