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
