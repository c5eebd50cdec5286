"""ctypes binding of libgtattn.so: same names as the C ABI, argument marshalling only.

Every function takes torch CUDA tensors (device memory owned by the caller), passes raw
pointers and sizes through the C ABI on torch's current stream and raises ``GtError`` on a
non-zero status.  There is no CPU fallback: if the CUDA library has not been built the
import of the library fails loudly on first use.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("GT_ATTN_LIB", os.path.join(_HERE, "libgtattn.so"))

GT_OK = 0
STATUS_NAMES = {0: "GT_OK", 1: "GT_ERR_INVALID_ARG", 2: "GT_ERR_UNSUPPORTED", 3: "GT_ERR_WORKSPACE",
                4: "GT_ERR_CUDA", 5: "GT_ERR_DEVICE_TIMEOUT", 6: "GT_ERR_NO_DEVICE", 7: "GT_ERR_BAD_SPD"}

EXPORTS = ("gt_status_string", "gt_check",
           "gt_spd_build_workspace", "gt_spd_build", "gt_spd_build_static_limit", "gt_spd_build_static",
           "gt_spd_validate_workspace", "gt_spd_validate", "gt_spd_validate_count", "gt_test_hook_barrier_overcount",
           "gt_biased_attn_fwd_workspace", "gt_biased_attn_fwd", "gt_biased_attn_fwd_ex",
           "gt_biased_attn_bwd_workspace", "gt_biased_attn_bwd", "gt_biased_attn_bwd_ex", "gt_profile_bwd_kernel_events",
           "gt_biased_attn_fwd_chunked_workspace", "gt_biased_attn_fwd_chunked",
           "gt_biased_attn_bwd_chunked_workspace", "gt_biased_attn_bwd_chunked",
           "gt_biased_attn_fwd_step_workspace", "gt_biased_attn_fwd_step",
           "gt_biased_attn_bwd_step_context_bytes", "gt_biased_attn_bwd_step_prepare", "gt_biased_attn_bwd_step_prepare_ex",
           "gt_biased_attn_bwd_step", "gt_biased_attn_bwd_step_finish",
           "gt_feature_attn_fwd", "gt_feature_attn_bwd_workspace", "gt_feature_attn_bwd",
           "gt_feature_encode_workspace", "gt_feature_encode", "gt_feature_encode_count",
           "gt_feature_code_table", "gt_feature_code_dweights")


class GtError(RuntimeError):
    def __init__(self, status: int, where: str):
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")
        self.status = status


class _GtBatch(ctypes.Structure):
    _fields_ = [("n_total", ctypes.c_int32), ("n_graphs", ctypes.c_int32),
                ("cu_seqlens", ctypes.c_void_p), ("max_seqlen", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load libgtattn.so (built in-tree by ``paper_2609_34420_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_34420_b200.build` "
                              "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
        bp = ctypes.POINTER(_GtBatch)
        L.gt_status_string.restype = ctypes.c_char_p
        L.gt_status_string.argtypes = [ctypes.c_int]
        L.gt_check.restype = ctypes.c_int
        L.gt_check.argtypes = [vp, vp]
        L.gt_spd_build_workspace.restype = sz
        L.gt_spd_build_workspace.argtypes = [bp, i64, i32]
        L.gt_spd_build.restype = ctypes.c_int
        L.gt_spd_build.argtypes = [vp, vp, i64, bp, i32, vp, vp, vp, sz, vp]
        L.gt_spd_build_static_limit.restype = sz
        L.gt_spd_build_static_limit.argtypes = []
        L.gt_spd_build_static.restype = ctypes.c_int
        L.gt_spd_build_static.argtypes = [vp, vp, i64, bp, i32, vp, vp, vp]
        L.gt_spd_validate_workspace.restype = sz
        L.gt_spd_validate_workspace.argtypes = []
        L.gt_spd_validate.restype = ctypes.c_int
        L.gt_spd_validate.argtypes = [vp, vp, bp, i32, vp, sz, vp]
        L.gt_spd_validate_count.restype = ctypes.c_int
        L.gt_spd_validate_count.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int64)]
        L.gt_test_hook_barrier_overcount.restype = None
        L.gt_test_hook_barrier_overcount.argtypes = [i32]
        L.gt_biased_attn_fwd_workspace.restype = sz
        L.gt_biased_attn_fwd_workspace.argtypes = [bp, i32, i32]
        L.gt_biased_attn_fwd.restype = ctypes.c_int
        L.gt_biased_attn_fwd.argtypes = [vp, vp, vp, vp, vp, vp, bp, i32, i32, i32, vp, vp, vp, sz, vp]
        L.gt_biased_attn_fwd_ex.restype = ctypes.c_int
        L.gt_biased_attn_fwd_ex.argtypes = [vp, vp, vp, vp, vp, vp, bp, i32, i32, i32, vp, vp, vp, vp, sz, vp]
        L.gt_biased_attn_bwd_workspace.restype = sz
        L.gt_biased_attn_bwd_workspace.argtypes = [bp, i32, i32, i32]
        L.gt_biased_attn_bwd.restype = ctypes.c_int
        L.gt_biased_attn_bwd.argtypes = [vp] * 9 + [bp, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.gt_biased_attn_bwd_ex.restype = ctypes.c_int
        L.gt_biased_attn_bwd_ex.argtypes = [vp] * 9 + [bp, i32, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.gt_profile_bwd_kernel_events.restype = None
        L.gt_profile_bwd_kernel_events.argtypes = [vp, vp, i32]
        L.gt_biased_attn_fwd_chunked_workspace.restype = sz
        L.gt_biased_attn_fwd_chunked_workspace.argtypes = [bp, i32, i32, i32]
        L.gt_biased_attn_fwd_chunked.restype = ctypes.c_int
        L.gt_biased_attn_fwd_chunked.argtypes = [vp, vp, vp, vp, vp, vp, bp, i32, i32, i32, vp, vp, i32, vp, vp, sz, vp]
        L.gt_biased_attn_fwd_step_workspace.restype = sz
        L.gt_biased_attn_fwd_step_workspace.argtypes = [bp, i32, i32]
        L.gt_biased_attn_fwd_step.restype = ctypes.c_int
        L.gt_biased_attn_fwd_step.argtypes = [vp] * 5 + [bp, i32, i32, i32] + [i32] * 6 + [vp, vp, vp, vp, sz, vp]
        L.gt_biased_attn_bwd_step_context_bytes.restype = sz
        L.gt_biased_attn_bwd_step_context_bytes.argtypes = [bp, i32, i32]
        L.gt_biased_attn_bwd_step_prepare.restype = ctypes.c_int
        L.gt_biased_attn_bwd_step_prepare.argtypes = [vp, vp, vp, vp, bp, i32, i32, i32, vp, sz, vp]
        L.gt_biased_attn_bwd_step_prepare_ex.restype = ctypes.c_int
        L.gt_biased_attn_bwd_step_prepare_ex.argtypes = [vp, vp, vp, vp, vp, bp, i32, i32, i32, vp, sz, vp]
        L.gt_biased_attn_bwd_step.restype = ctypes.c_int
        L.gt_biased_attn_bwd_step.argtypes = [vp] * 5 + [bp, i32, i32, i32] + [i32] * 6 + [vp, vp, vp, vp, vp, sz, vp]
        L.gt_biased_attn_bwd_step_finish.restype = ctypes.c_int
        L.gt_biased_attn_bwd_step_finish.argtypes = [vp, vp, vp, vp, bp, i32, i32, i32, vp, vp, vp, vp, vp]
        L.gt_biased_attn_bwd_chunked_workspace.restype = sz
        L.gt_biased_attn_bwd_chunked_workspace.argtypes = [bp, i32, i32, i32, i32]
        L.gt_biased_attn_bwd_chunked.restype = ctypes.c_int
        L.gt_biased_attn_bwd_chunked.argtypes = [vp] * 8 + [bp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.gt_feature_attn_fwd.restype = ctypes.c_int
        L.gt_feature_attn_fwd.argtypes = [vp] * 5 + [bp, i32, i32, vp, vp, vp]
        L.gt_feature_attn_bwd_workspace.restype = sz
        L.gt_feature_attn_bwd_workspace.argtypes = [bp, i32]
        L.gt_feature_attn_bwd.restype = ctypes.c_int
        L.gt_feature_attn_bwd.argtypes = [vp] * 7 + [bp, i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.gt_feature_encode_workspace.restype = sz
        L.gt_feature_encode_workspace.argtypes = []
        L.gt_feature_encode.restype = ctypes.c_int
        L.gt_feature_encode.argtypes = [vp, bp, vp, vp, vp, sz, vp]
        L.gt_feature_encode_count.restype = ctypes.c_int
        L.gt_feature_encode_count.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
        L.gt_feature_code_table.restype = ctypes.c_int
        L.gt_feature_code_table.argtypes = [vp, vp, i32, i32, vp, vp]
        L.gt_feature_code_dweights.restype = ctypes.c_int
        L.gt_feature_code_dweights.argtypes = [vp, vp, i32, i32, vp, vp]
        _lib = L
    return _lib


@dataclass
class Batch:
    """Packed batch: device ``cu_seqlens`` int32[G+1] and ``spd_offsets`` int64[G+1]
    (both None for a single graph)."""
    n_total: int
    n_graphs: int = 1
    max_seqlen: Optional[int] = None
    cu_seqlens: Optional[torch.Tensor] = None
    spd_offsets: Optional[torch.Tensor] = None

    def c_struct(self) -> _GtBatch:
        return _GtBatch(self.n_total, self.n_graphs, _ptr(self.cu_seqlens),
                        self.n_total if self.max_seqlen is None else self.max_seqlen)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _raise(status: int, where: str) -> None:
    if status != GT_OK:
        raise GtError(status, where)


def _workspace(nbytes: int, device) -> torch.Tensor:
    ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    ws[:256].zero_()
    return ws


def gt_check(workspace: torch.Tensor) -> None:
    """Synchronise the current stream and raise if a kernel recorded a device-side error."""
    _raise(lib().gt_check(_ptr(workspace), _stream()), "gt_check")


# ------------------------------------------------------------------------------------------
def gt_spd_build_workspace(batch: Batch, nnz: int, max_dist: int) -> int:
    b = batch.c_struct()
    return int(lib().gt_spd_build_workspace(ctypes.byref(b), int(nnz), int(max_dist)))


def gt_spd_build(row_ptr: torch.Tensor, col_idx: torch.Tensor, batch: Batch, max_dist: int,
                 spd_out: torch.Tensor, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Enqueue the SPD build; returns the workspace used (pass it to ``gt_check``)."""
    nnz = int(col_idx.numel())
    if workspace is None:
        workspace = _workspace(gt_spd_build_workspace(batch, nnz, max_dist), row_ptr.device)
    b = batch.c_struct()
    st = lib().gt_spd_build(_ptr(row_ptr), _ptr(col_idx) if nnz else None, nnz, ctypes.byref(b), int(max_dist),
                            _ptr(batch.spd_offsets), _ptr(spd_out), _ptr(workspace), workspace.numel(), _stream())
    _raise(st, "gt_spd_build")
    return workspace


def gt_spd_build_static_limit() -> int:
    return int(lib().gt_spd_build_static_limit())


def gt_spd_build_static(row_ptr: torch.Tensor, col_idx: torch.Tensor, batch: Batch, max_dist: int,
                        spd_out: torch.Tensor) -> None:
    """SPD build for callers that must not allocate: the scratch is a fixed array inside the
    library (one per device, shared by every call, so calls that overlap on the GPU race).
    Raises GtError(GT_ERR_WORKSPACE) when the batch needs more than gt_spd_build_static_limit()."""
    nnz = int(col_idx.numel())
    b = batch.c_struct()
    st = lib().gt_spd_build_static(_ptr(row_ptr), _ptr(col_idx) if nnz else None, nnz, ctypes.byref(b), int(max_dist),
                                   _ptr(batch.spd_offsets), _ptr(spd_out), _stream())
    _raise(st, "gt_spd_build_static")


def gt_biased_attn_fwd_workspace(batch: Batch, n_heads: int, head_dim: int) -> int:
    b = batch.c_struct()
    return int(lib().gt_biased_attn_fwd_workspace(ctypes.byref(b), n_heads, head_dim))


def gt_biased_attn_fwd(q, k, v, spd, bias, batch: Batch, max_dist: int, out, lse,
                       workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    _, H, d = q.shape
    if workspace is None:
        workspace = _workspace(gt_biased_attn_fwd_workspace(batch, H, d), q.device)
    b = batch.c_struct()
    st = lib().gt_biased_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(spd), _ptr(batch.spd_offsets), _ptr(bias),
                                  ctypes.byref(b), H, d, int(max_dist), _ptr(out), _ptr(lse),
                                  _ptr(workspace), workspace.numel(), _stream())
    _raise(st, "gt_biased_attn_fwd")
    return workspace


def gt_biased_attn_fwd_ex(q, k, v, spd, bias, batch: Batch, max_dist: int, out, lse, out_f32: Optional[torch.Tensor],
                          workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Forward that also writes the fp32 output (before its rounding to bf16) into ``out_f32``."""
    _, H, d = q.shape
    if workspace is None:
        workspace = _workspace(gt_biased_attn_fwd_workspace(batch, H, d), q.device)
    b = batch.c_struct()
    st = lib().gt_biased_attn_fwd_ex(_ptr(q), _ptr(k), _ptr(v), _ptr(spd), _ptr(batch.spd_offsets), _ptr(bias),
                                     ctypes.byref(b), H, d, int(max_dist), _ptr(out), _ptr(lse), _ptr(out_f32),
                                     _ptr(workspace), workspace.numel(), _stream())
    _raise(st, "gt_biased_attn_fwd_ex")
    return workspace


def gt_biased_attn_bwd_workspace(batch: Batch, n_heads: int, head_dim: int, max_dist: int) -> int:
    b = batch.c_struct()
    return int(lib().gt_biased_attn_bwd_workspace(ctypes.byref(b), n_heads, head_dim, max_dist))


def gt_biased_attn_bwd(q, k, v, out, dout, lse, spd, bias, batch: Batch, max_dist: int, dq, dk, dv, dbias,
                       workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    _, H, d = q.shape
    if workspace is None:
        workspace = _workspace(gt_biased_attn_bwd_workspace(batch, H, d, max_dist), q.device)
    b = batch.c_struct()
    st = lib().gt_biased_attn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(dout), _ptr(lse), _ptr(spd),
                                  _ptr(batch.spd_offsets), _ptr(bias), ctypes.byref(b), H, d, int(max_dist),
                                  _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dbias),
                                  _ptr(workspace), workspace.numel(), _stream())
    _raise(st, "gt_biased_attn_bwd")
    return workspace


def gt_biased_attn_bwd_ex(q, k, v, out, dout, lse, spd, bias, batch: Batch, max_dist: int, dq, dk, dv, dbias,
                          out_f32: Optional[torch.Tensor], workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Backward whose per-query term dout . out is formed from the fp32 forward output ``out_f32``."""
    _, H, d = q.shape
    if workspace is None:
        workspace = _workspace(gt_biased_attn_bwd_workspace(batch, H, d, max_dist), q.device)
    b = batch.c_struct()
    st = lib().gt_biased_attn_bwd_ex(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(dout), _ptr(lse), _ptr(spd),
                                     _ptr(batch.spd_offsets), _ptr(bias), ctypes.byref(b), H, d, int(max_dist),
                                     _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dbias), _ptr(out_f32),
                                     _ptr(workspace), workspace.numel(), _stream())
    _raise(st, "gt_biased_attn_bwd_ex")
    return workspace


def gt_spd_validate(spd, batch: Batch, max_dist: int, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Enqueue the check of an SPD matrix for entries that name no bucket; ``gt_check`` on the returned
    workspace raises GtError(GT_ERR_BAD_SPD) if there are any, ``gt_spd_validate_count`` gives their number."""
    if workspace is None:
        workspace = _workspace(int(lib().gt_spd_validate_workspace()), spd.device)
    b = batch.c_struct()
    st = lib().gt_spd_validate(_ptr(spd), _ptr(batch.spd_offsets), ctypes.byref(b), int(max_dist),
                               _ptr(workspace), workspace.numel(), _stream())
    _raise(st, "gt_spd_validate")
    return workspace


def gt_spd_validate_count(workspace: torch.Tensor) -> int:
    c = ctypes.c_int64(0)
    _raise(lib().gt_spd_validate_count(_ptr(workspace), _stream(), ctypes.byref(c)), "gt_spd_validate_count")
    return int(c.value)


def gt_test_hook_barrier_overcount(extra: int) -> None:
    """Test hook: the next bit-matrix SPD build waits for ``extra`` thread blocks that do not exist."""
    lib().gt_test_hook_barrier_overcount(int(extra))


def gt_biased_attn_fwd_chunked_workspace(batch: Batch, n_heads: int, head_dim: int, n_kv_chunks: int) -> int:
    b = batch.c_struct()
    return int(lib().gt_biased_attn_fwd_chunked_workspace(ctypes.byref(b), n_heads, head_dim, n_kv_chunks))


def gt_biased_attn_fwd_chunked(q, k, v, spd, bias, batch: Batch, max_dist: int, out, lse, n_kv_chunks: int,
                               lse_chunks: Optional[torch.Tensor] = None,
                               workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    _, H, d = q.shape
    if workspace is None:
        workspace = _workspace(gt_biased_attn_fwd_chunked_workspace(batch, H, d, n_kv_chunks), q.device)
    b = batch.c_struct()
    st = lib().gt_biased_attn_fwd_chunked(_ptr(q), _ptr(k), _ptr(v), _ptr(spd), _ptr(batch.spd_offsets), _ptr(bias),
                                          ctypes.byref(b), H, d, int(max_dist), _ptr(out), _ptr(lse),
                                          int(n_kv_chunks), _ptr(lse_chunks),
                                          _ptr(workspace), workspace.numel(), _stream())
    _raise(st, "gt_biased_attn_fwd_chunked")
    return workspace


def gt_biased_attn_bwd_chunked_workspace(batch: Batch, n_heads: int, head_dim: int, max_dist: int, n_kv_chunks: int) -> int:
    b = batch.c_struct()
    return int(lib().gt_biased_attn_bwd_chunked_workspace(ctypes.byref(b), n_heads, head_dim, max_dist, n_kv_chunks))


def gt_biased_attn_bwd_chunked(q, k, v, out, dout, lse, spd, bias, batch: Batch, max_dist: int, n_kv_chunks: int,
                               dq, dk, dv, dbias, dbias_chunks: Optional[torch.Tensor] = None,
                               workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    _, H, d = q.shape
    if workspace is None:
        workspace = _workspace(gt_biased_attn_bwd_chunked_workspace(batch, H, d, max_dist, n_kv_chunks), q.device)
    b = batch.c_struct()
    st = lib().gt_biased_attn_bwd_chunked(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(dout), _ptr(lse), _ptr(spd),
                                          _ptr(bias), ctypes.byref(b), H, d, int(max_dist), int(n_kv_chunks),
                                          _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dbias), _ptr(dbias_chunks),
                                          _ptr(workspace), workspace.numel(), _stream())
    _raise(st, "gt_biased_attn_bwd_chunked")
    return workspace


def gt_biased_attn_fwd_step_workspace(batch: Batch, n_heads: int, head_dim: int) -> int:
    b = batch.c_struct()
    return int(lib().gt_biased_attn_fwd_step_workspace(ctypes.byref(b), n_heads, head_dim))


def gt_biased_attn_fwd_step(q, k, v, spd, bias, batch: Batch, max_dist: int, q_range, kv_range0, kv_range1,
                            o_acc, lse_acc, out: Optional[torch.Tensor] = None,
                            workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    _, H, d = q.shape
    if workspace is None:
        workspace = _workspace(gt_biased_attn_fwd_step_workspace(batch, H, d), q.device)
    b = batch.c_struct()
    st = lib().gt_biased_attn_fwd_step(_ptr(q), _ptr(k), _ptr(v), _ptr(spd), _ptr(bias), ctypes.byref(b), H, d,
                                       int(max_dist), int(q_range[0]), int(q_range[1]),
                                       int(kv_range0[0]), int(kv_range0[1]), int(kv_range1[0]), int(kv_range1[1]),
                                       _ptr(o_acc), _ptr(lse_acc), _ptr(out),
                                       _ptr(workspace), workspace.numel(), _stream())
    _raise(st, "gt_biased_attn_fwd_step")
    return workspace


def gt_biased_attn_bwd_step_context_bytes(batch: Batch, n_heads: int, head_dim: int) -> int:
    b = batch.c_struct()
    return int(lib().gt_biased_attn_bwd_step_context_bytes(ctypes.byref(b), n_heads, head_dim))


def gt_biased_attn_bwd_step_prepare(out, dout, lse, spd, batch: Batch, max_dist: int,
                                    context: Optional[torch.Tensor] = None,
                                    out_f32: Optional[torch.Tensor] = None) -> torch.Tensor:
    """``out_f32`` (the fp32 o_acc of the forward steps) selects gt_biased_attn_bwd_step_prepare_ex."""
    _, H, d = dout.shape
    if context is None:
        context = _workspace(gt_biased_attn_bwd_step_context_bytes(batch, H, d), dout.device)
    b = batch.c_struct()
    if out_f32 is None:
        st = lib().gt_biased_attn_bwd_step_prepare(_ptr(out), _ptr(dout), _ptr(lse), _ptr(spd), ctypes.byref(b), H, d,
                                                   int(max_dist), _ptr(context), context.numel(), _stream())
    else:
        st = lib().gt_biased_attn_bwd_step_prepare_ex(_ptr(out), _ptr(out_f32), _ptr(dout), _ptr(lse), _ptr(spd),
                                                      ctypes.byref(b), H, d, int(max_dist),
                                                      _ptr(context), context.numel(), _stream())
    _raise(st, "gt_biased_attn_bwd_step_prepare")
    return context


def gt_biased_attn_bwd_step(q, k, v, dout, bias, batch: Batch, max_dist: int, q_range, kv_range0, kv_range1,
                            dq_acc, dk_acc, dv_acc, dbias_acc, context: torch.Tensor) -> None:
    _, H, d = q.shape
    b = batch.c_struct()
    st = lib().gt_biased_attn_bwd_step(_ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(bias), ctypes.byref(b), H, d, int(max_dist),
                                       int(q_range[0]), int(q_range[1]), int(kv_range0[0]), int(kv_range0[1]),
                                       int(kv_range1[0]), int(kv_range1[1]),
                                       _ptr(dq_acc), _ptr(dk_acc), _ptr(dv_acc), _ptr(dbias_acc),
                                       _ptr(context), context.numel(), _stream())
    _raise(st, "gt_biased_attn_bwd_step")


def gt_biased_attn_bwd_step_finish(dq_acc, dk_acc, dv_acc, dbias_acc, batch: Batch, max_dist: int, dq, dk, dv, dbias) -> None:
    _, H, d = dq_acc.shape
    b = batch.c_struct()
    st = lib().gt_biased_attn_bwd_step_finish(_ptr(dq_acc), _ptr(dk_acc), _ptr(dv_acc), _ptr(dbias_acc), ctypes.byref(b), H, d,
                                              int(max_dist), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dbias), _stream())
    _raise(st, "gt_biased_attn_bwd_step_finish")


def gt_feature_attn_fwd(q, k, v, features, weights, batch: Batch, out, lse) -> None:
    """Forward with the feature bias: features uint8 [N, N, 4], weights fp32 [H, 4]."""
    _, H, d = q.shape
    b = batch.c_struct()
    st = lib().gt_feature_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(features), _ptr(weights), ctypes.byref(b), H, d,
                                   _ptr(out), _ptr(lse), _stream())
    _raise(st, "gt_feature_attn_fwd")


def gt_feature_attn_bwd_workspace(batch: Batch, n_heads: int) -> int:
    b = batch.c_struct()
    return int(lib().gt_feature_attn_bwd_workspace(ctypes.byref(b), n_heads))


def gt_feature_attn_bwd(q, k, v, dout, lse, features, weights, batch: Batch, dq, dk, dv, dweights,
                        workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    _, H, d = q.shape
    if workspace is None:
        workspace = _workspace(gt_feature_attn_bwd_workspace(batch, H), q.device)
    b = batch.c_struct()
    st = lib().gt_feature_attn_bwd(_ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(lse), _ptr(features), _ptr(weights),
                                   ctypes.byref(b), H, d, _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dweights),
                                   _ptr(workspace), workspace.numel(), _stream())
    _raise(st, "gt_feature_attn_bwd")
    return workspace


_profile_keepalive = None


def gt_profile_bwd_kernel_events(before, after) -> None:
    """Have the next ``len(before)`` backward calls record the given torch CUDA events (created with
    ``enable_timing=True``) around their main kernel; pass empty lists to switch the hook off."""
    global _profile_keepalive
    n = len(before)
    if n == 0:
        lib().gt_profile_bwd_kernel_events(None, None, 0)
        _profile_keepalive = None
        return
    for e in list(before) + list(after):
        e.record()                                   # torch creates the CUDA event lazily, at its first record
    arr_t = ctypes.c_void_p * n
    a, b = arr_t(*[e.cuda_event for e in before]), arr_t(*[e.cuda_event for e in after])
    _profile_keepalive = (a, b, list(before), list(after))
    lib().gt_profile_bwd_kernel_events(a, b, n)


def gt_feature_encode(features, batch: Batch, codes, vectors, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Categorical features uint8 [N, N, 4] -> codes (uint8, N rows of pitch N rounded up to 16) and vectors (int32/uint32 [256])."""
    if workspace is None:
        workspace = _workspace(int(lib().gt_feature_encode_workspace()), features.device)
    b = batch.c_struct()
    st = lib().gt_feature_encode(_ptr(features), ctypes.byref(b), _ptr(codes), _ptr(vectors), _ptr(workspace),
                                 workspace.numel(), _stream())
    _raise(st, "gt_feature_encode")
    return workspace


def gt_feature_encode_count(workspace: torch.Tensor) -> int:
    """Synchronises; the number of distinct feature vectors the last gt_feature_encode on this workspace found."""
    c = ctypes.c_int32(0)
    _raise(lib().gt_feature_encode_count(_ptr(workspace), _stream(), ctypes.byref(c)), "gt_feature_encode_count")
    return int(c.value)


def gt_feature_code_table(weights, vectors, table) -> None:
    H, n_codes = table.shape
    _raise(lib().gt_feature_code_table(_ptr(weights), _ptr(vectors), H, n_codes, _ptr(table), _stream()), "gt_feature_code_table")


def gt_feature_code_dweights(dtable, vectors, dweights) -> None:
    H, n_codes = dtable.shape
    _raise(lib().gt_feature_code_dweights(_ptr(dtable), _ptr(vectors), H, n_codes, _ptr(dweights), _stream()),
           "gt_feature_code_dweights")
