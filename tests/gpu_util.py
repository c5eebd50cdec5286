"""Helpers for the GPU parity tests: move a seeded workload to the device, widen results."""
import numpy as np
import torch

from paper_2609_34420_b200 import binding as gt
from paper_2609_34420_b200 import workloads as wl


def device_batch(b: wl.GraphBatch, dev="cuda"):
    single = b.n_graphs == 1
    return gt.Batch(n_total=b.n_total, n_graphs=b.n_graphs, max_seqlen=b.max_seqlen,
                    cu_seqlens=None if single else torch.tensor(b.cu_seqlens, dtype=torch.int32, device=dev),
                    spd_offsets=None if single else torch.tensor(b.spd_offsets, dtype=torch.int64, device=dev))


def device_csr(b: wl.GraphBatch, dev="cuda"):
    rp = torch.tensor(b.row_ptr, dtype=torch.int32, device=dev)
    ci = torch.tensor(b.col_idx if b.col_idx.size else np.zeros(1, np.int32), dtype=torch.int32, device=dev)
    return rp, ci[:b.col_idx.size]


def bf16_tensor(bits: np.ndarray, dev="cuda") -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).to(dev).view(torch.bfloat16)


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def gpu_spd(w: wl.Workload, dev="cuda") -> torch.Tensor:
    """Run gt_spd_build on the workload's packed CSR; returns the flat uint8 device tensor."""
    bt = device_batch(w.batch, dev)
    rp, ci = device_csr(w.batch, dev)
    out = torch.full((w.batch.spd_bytes,), 0xEE, dtype=torch.uint8, device=dev)
    ws = gt.gt_spd_build(rp, ci, bt, w.max_dist, out)
    gt.gt_check(ws)
    return out


def rel_l2(x: np.ndarray, r: np.ndarray) -> float:
    den = float(np.linalg.norm(r.reshape(-1)))
    return float(np.linalg.norm((x - r).reshape(-1))) / (den if den > 0 else 1.0)


def localized_rel_l2(x: np.ndarray, r: np.ndarray, block: int = 128) -> dict:
    """Relative-L2 error of a [rows, H, d] gradient per head and per block of `block` consecutive rows
    (each over all heads), worst of each: an error confined to one head, one tile of rows or one row cannot
    hide in the norm of the whole tensor.  A block is measured against its own norm, but not below the
    average block norm (a block of nearly zero gradient has no meaningful relative error)."""
    n = x.shape[0]
    per_head = max(rel_l2(x[:, h], r[:, h]) for h in range(x.shape[1]))
    n_blocks = (n + block - 1) // block
    err = np.array([np.linalg.norm((x[b * block:(b + 1) * block] - r[b * block:(b + 1) * block]).reshape(-1)) for b in range(n_blocks)])
    ref = np.array([np.linalg.norm(r[b * block:(b + 1) * block].reshape(-1)) for b in range(n_blocks)])
    floor = float(np.sqrt((ref ** 2).mean()))
    den = np.maximum(ref, floor)
    return {"head": per_head, "block": float((err / np.where(den > 0, den, 1.0)).max())}


class DeviceCase:
    """A workload moved to the device, with the SPD either from the oracle (default, so that
    attention parity does not depend on the SPD kernel) or from gt_spd_build."""

    def __init__(self, w: wl.Workload, spd_from_gpu: bool = False, dev="cuda"):
        from oracle import spd as ospd
        self.w = w
        b = w.batch
        t = w.tensors()
        self.batch = device_batch(b, dev)
        self.spd_host = ospd.spd_packed(b.row_ptr, b.col_idx, b.cu_seqlens, w.max_dist)
        self.spd = gpu_spd(w, dev) if spd_from_gpu else torch.from_numpy(self.spd_host).to(dev)
        self.q, self.k, self.v, self.dout = (bf16_tensor(x, dev) for x in (t.q, t.k, t.v, t.dout))
        self.bias = torch.tensor(t.bias, device=dev)
        self.T, self.H, self.d = t.q.shape

    def host_f64(self):
        t = self.w.tensors()
        f = wl.bf16_bits_to_f64
        return f(t.q), f(t.k), f(t.v), f(t.dout), t.bias.astype(np.float64)

    def forward(self):
        out = torch.full((self.T, self.H, self.d), float("nan"), dtype=torch.bfloat16, device=self.q.device)
        lse = torch.full((self.H, self.T), float("nan"), dtype=torch.float32, device=self.q.device)
        ws = gt.gt_biased_attn_fwd(self.q, self.k, self.v, self.spd, self.bias, self.batch, self.w.max_dist, out, lse)
        gt.gt_check(ws)
        return out, lse

    def forward_ex(self):
        """Forward that also returns the fp32 output (before its rounding to bf16)."""
        out = torch.full((self.T, self.H, self.d), float("nan"), dtype=torch.bfloat16, device=self.q.device)
        out32 = torch.full((self.T, self.H, self.d), float("nan"), dtype=torch.float32, device=self.q.device)
        lse = torch.full((self.H, self.T), float("nan"), dtype=torch.float32, device=self.q.device)
        ws = gt.gt_biased_attn_fwd_ex(self.q, self.k, self.v, self.spd, self.bias, self.batch, self.w.max_dist, out, lse, out32)
        gt.gt_check(ws)
        return out, lse, out32

    def backward_ex(self, out, lse, out32):
        dq, dk, dv = (torch.full_like(self.q, float("nan")) for _ in range(3))
        dbias = torch.full_like(self.bias, float("nan"))
        ws = gt.gt_biased_attn_bwd_ex(self.q, self.k, self.v, out, self.dout, lse, self.spd, self.bias, self.batch,
                                      self.w.max_dist, dq, dk, dv, dbias, out32)
        gt.gt_check(ws)
        return dq, dk, dv, dbias

    def forward_chunked(self, n_chunks, want_chunk_lse=False):
        out = torch.full((self.T, self.H, self.d), float("nan"), dtype=torch.bfloat16, device=self.q.device)
        lse = torch.full((self.H, self.T), float("nan"), dtype=torch.float32, device=self.q.device)
        cl = torch.full((n_chunks, self.H, self.T), float("nan"), dtype=torch.float32,
                        device=self.q.device) if want_chunk_lse else None
        ws = gt.gt_biased_attn_fwd_chunked(self.q, self.k, self.v, self.spd, self.bias, self.batch, self.w.max_dist,
                                           out, lse, n_chunks, cl)
        gt.gt_check(ws)
        return out, lse, cl

    def backward_chunked(self, out, lse, n_chunks, want_chunk_dbias=False):
        dq, dk, dv = (torch.full_like(self.q, float("nan")) for _ in range(3))
        dbias = torch.full_like(self.bias, float("nan"))
        dbc = torch.full((n_chunks,) + tuple(self.bias.shape), float("nan"), dtype=torch.float32,
                         device=self.q.device) if want_chunk_dbias else None
        ws = gt.gt_biased_attn_bwd_chunked(self.q, self.k, self.v, out, self.dout, lse, self.spd, self.bias, self.batch,
                                           self.w.max_dist, n_chunks, dq, dk, dv, dbias, dbc)
        gt.gt_check(ws)
        return dq, dk, dv, dbias, dbc

    def backward(self, out, lse, dout=None):
        dout = self.dout if dout is None else dout
        dq, dk, dv = (torch.full_like(self.q, float("nan")) for _ in range(3))
        dbias = torch.full_like(self.bias, float("nan"))
        ws = gt.gt_biased_attn_bwd(self.q, self.k, self.v, out, dout, lse, self.spd, self.bias, self.batch,
                                   self.w.max_dist, dq, dk, dv, dbias)
        gt.gt_check(ws)
        return dq, dk, dv, dbias
