"""CPU ORACLE -- TEST INFRASTRUCTURE ONLY (never imported by the product path).

Biased graph attention with a FEATURE bias instead of the distance-bucket table: the model the
paper trains has an "attention bias dimension of 4" (Sec. "Experiments", end-to-end setup), i.e.
every ordered node pair carries a small feature vector and each head weights it linearly.  The
paper gives the dimension only; the reading taken here (and stated in the design notes) is

    b_attn[h,i,j] = sum_c W[h,c] * f[i,j,c] ,   f uint8 [n, n, C] (C = 4),  W fp [H, C]

plugged into Eq. 1 unchanged:

    S[h,i,j] = (q[i,h,:] . k[j,h,:]) / sqrt(d) + b_attn[h,i,j],   P = softmax_j S,   O = P V,
    LSE[h,i] = log sum_j exp S[h,i,j].

Backward for L = sum(O * dO), by the chain rule (as for the bucket form), with the bias gradient now a
plain contraction instead of a scatter:

    dS[h,i,j] = P (dO_i . v_j - dO_i . O_i),    dW[h,c] = sum_{i,j} dS[h,i,j] * f[i,j,c].

fp64 numpy, full score rows, no key tiling; query rows are processed a block at a time only to bound
memory.  One graph per call (a packed batch is a loop over graphs with dW summed).

Pinned by tests against torch autograd in fp64 through an einsum-built dense bias, central finite
differences on W, the reduction to the bucket form when f is the one-hot code of a distance matrix, and
the identity sum_c dW[h,c] * u[c] = 0 when every pair's features satisfy f . u = const.

Categorical features (few distinct feature vectors, as structural encodings are): the feature form IS a bucket
form.  With the distinct 4-vectors numbered c = 0..n_codes-1,

    b_attn[h,i,j] = table[h, code[i,j]],  table[h,c] = sum_x W[h,x] * vec[c,x],   dW[h,x] = sum_c dTable[h,c] * vec[c,x]

exactly (same sums, regrouped).  encode_features / code_table / weights_gradient_from_table write that out; they
are pinned by the round trip vec[code] == f, by table[code] == feature_bias, and by dW through the codes equalling
backward_feature's dW.
"""
from __future__ import annotations

from typing import Tuple

import numpy as np

ROW_BLOCK = 1024


def feature_bias(f_rows: np.ndarray, w_h: np.ndarray) -> np.ndarray:
    """b[i,j] = sum_c w_h[c] * f_rows[i,j,c] for one head; f_rows uint8 [r,n,C], w_h [C]."""
    return f_rows.astype(np.float64) @ w_h


def forward_feature(q: np.ndarray, k: np.ndarray, v: np.ndarray, f: np.ndarray, w: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """q,k,v fp64 [n,H,d]; f uint8 [n,n,C]; w fp64 [H,C].  Returns O [n,H,d], LSE [H,n]."""
    n, H, d = q.shape
    out = np.zeros((n, H, d))
    lse = np.zeros((H, n))
    inv_sqrt_d = 1.0 / np.sqrt(float(d))
    for r0 in range(0, n, ROW_BLOCK):
        r1 = min(n, r0 + ROW_BLOCK)
        for h in range(H):
            s = (q[r0:r1, h, :] @ k[:, h, :].T) * inv_sqrt_d + feature_bias(f[r0:r1, :n], w[h])
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            l = e.sum(axis=1, keepdims=True)
            out[r0:r1, h, :] = (e / l) @ v[:, h, :]
            lse[h, r0:r1] = (m + np.log(l))[:, 0]
    return out, lse


def backward_feature(q: np.ndarray, k: np.ndarray, v: np.ndarray, dout: np.ndarray, f: np.ndarray, w: np.ndarray):
    """Returns dQ, dK, dV [n,H,d] and dW [H,C]."""
    n, H, d = q.shape
    C = w.shape[1]
    dq, dk, dv = np.zeros((n, H, d)), np.zeros((n, H, d)), np.zeros((n, H, d))
    dw = np.zeros((H, C))
    inv_sqrt_d = 1.0 / np.sqrt(float(d))
    for r0 in range(0, n, ROW_BLOCK):
        r1 = min(n, r0 + ROW_BLOCK)
        ff = f[r0:r1, :n].astype(np.float64)                       # [r,n,C]
        for h in range(H):
            s = (q[r0:r1, h, :] @ k[:, h, :].T) * inv_sqrt_d + ff @ w[h]
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            p = e / e.sum(axis=1, keepdims=True)
            do = dout[r0:r1, h, :]
            o = p @ v[:, h, :]
            delta = (do * o).sum(axis=1, keepdims=True)
            ds = p * (do @ v[:, h, :].T - delta)
            dv[:, h, :] += p.T @ do
            dq[r0:r1, h, :] = (ds @ k[:, h, :]) * inv_sqrt_d
            dk[:, h, :] += (ds.T @ q[r0:r1, h, :]) * inv_sqrt_d
            dw[h] += np.tensordot(ds, ff, axes=([0, 1], [0, 1]))
    return dq, dk, dv, dw


def encode_features(f: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """f uint8 [n,n,4] -> (code int64 [n,n], vec uint8 [n_codes,4]).  Codes number the distinct feature vectors in
    ascending order of the 32-bit word f0 + 256 f1 + 65536 f2 + 16777216 f3."""
    n = f.shape[0]
    assert f.shape == (n, n, 4) and f.dtype == np.uint8
    word = (f[..., 0].astype(np.uint32) | (f[..., 1].astype(np.uint32) << 8) |
            (f[..., 2].astype(np.uint32) << 16) | (f[..., 3].astype(np.uint32) << 24))
    distinct, inverse = np.unique(word.reshape(-1), return_inverse=True)
    vec = np.stack([(distinct >> (8 * x)) & 0xff for x in range(4)], axis=1).astype(np.uint8)
    return inverse.reshape(n, n).astype(np.int64), vec


def code_table(w: np.ndarray, vec: np.ndarray) -> np.ndarray:
    """table[h,c] = sum_x w[h,x] * vec[c,x]; w fp64 [H,4], vec uint8 [n_codes,4]."""
    return w @ vec.astype(np.float64).T


def weights_gradient_from_table(dtable: np.ndarray, vec: np.ndarray) -> np.ndarray:
    """dW[h,x] = sum_c dtable[h,c] * vec[c,x]."""
    return dtable @ vec.astype(np.float64)
