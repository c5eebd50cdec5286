"""CPU ORACLE -- TEST INFRASTRUCTURE ONLY (never imported by the product path).

Biased graph attention, forward and analytic backward, in fp64 numpy, written out from
the definition (the paper's Eq. 1 with the structural-encoding bias realised as a
per-head table indexed by the shortest-path-distance bucket):

    S[h,i,j]  = (q[i,h,:] . k[j,h,:]) / sqrt(d) + B[h, spd[i,j]]
    P[h,i,:]  = softmax_j S[h,i,:]                    O[i,h,:] = sum_j P[h,i,j] v[j,h,:]
    LSE[h,i]  = log sum_j exp S[h,i,j]

Every node attends to every node of its own graph (no mask; unreachable pairs use the
learnable bucket max_dist+1).  Each score row is materialised in full; there is no key
tiling and no online softmax.  The only concession to memory is that query rows are
processed a block at a time (rows are independent in the forward; in the backward the
per-key sums dK, dV, dB are accumulated over row blocks in fixed order).

Backward for the loss L = sum(O * dO), derived by the chain rule through softmax:

    Delta[i]  = sum_c dO[i,c] O[i,c]            dP[i,j] = sum_c dO[i,c] v[j,c]
    dS[i,j]   = P[i,j] (dP[i,j] - Delta[i])
    dV[j]     = sum_i P[i,j] dO[i]
    dQ[i]     = (1/sqrt d) sum_j dS[i,j] k[j]   dK[j] = (1/sqrt d) sum_i dS[i,j] q[i]
    dB[h,b]   = sum_{(i,j): spd[i,j]=b} dS[h,i,j]          (summed over all graphs)

The key-chunked result of the graph-aware context-parallel scheme (Eq. 2 plus the
bias-before-online-softmax rule) equals the unchunked one exactly, so the oracle for it is
the unchunked definition; ``chunk_lse`` gives the per-chunk log-sum-exp by its direct
definition so that the per-chunk statistic can be checked too.

Pinned by tests against torch's scaled_dot_product_attention (with and without a dense
additive mask) and torch autograd in fp64, central finite differences, closed forms
(Q=0, V=1, hand-worked rational softmax), shift invariance, permutation equivariance and
the identity sum_b dB[h,b] = 0.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np

ROW_BLOCK = 2048


def _scores(q_rows: np.ndarray, k: np.ndarray, spd_rows: np.ndarray, bias_h: np.ndarray) -> np.ndarray:
    """S[i,j] for the given query rows of one head of one graph; q_rows [r,d], k [n,d],
    spd_rows uint8 [r,n], bias_h [nb]."""
    d = q_rows.shape[1]
    return (q_rows @ k.T) / np.sqrt(float(d)) + bias_h[spd_rows.astype(np.int64)]


def _softmax_rows(s: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    return e / l, (m + np.log(l))[:, 0]


def forward_single(q: np.ndarray, k: np.ndarray, v: np.ndarray, spd: np.ndarray, bias: np.ndarray,
                   rows: Optional[np.ndarray] = None, compact_spd: bool = False) -> Tuple[np.ndarray, np.ndarray]:
    """One graph.  q,k,v fp64 [n,H,d]; spd uint8 [n, >=n]; bias fp64 [H,nb].
    Returns O fp64 [r,H,d] and LSE fp64 [H,r] for the selected query rows (default all).
    With compact_spd, spd holds only the selected rows: spd[i] is the SPD row of rows[i]."""
    n, H, d = q.shape
    rows = np.arange(n) if rows is None else np.asarray(rows)
    out = np.zeros((len(rows), H, d))
    lse = np.zeros((H, len(rows)))
    for r0 in range(0, len(rows), ROW_BLOCK):
        rr = rows[r0:r0 + ROW_BLOCK]
        spd_rows = spd[r0:r0 + len(rr), :n] if compact_spd else spd[rr, :n]
        for h in range(H):
            p, l = _softmax_rows(_scores(q[rr, h, :], k[:, h, :], spd_rows, bias[h]))
            out[r0:r0 + len(rr), h, :] = p @ v[:, h, :]
            lse[h, r0:r0 + len(rr)] = l
    return out, lse


def backward_single(q: np.ndarray, k: np.ndarray, v: np.ndarray, dout: np.ndarray, spd: np.ndarray,
                    bias: np.ndarray, rows: Optional[np.ndarray] = None, compact_spd: bool = False):
    """One graph.  dout fp64 [n,H,d] (only the selected rows are read).  Returns
    (dQ [r,H,d] for the selected rows, dK [n,H,d], dV [n,H,d], dB [H,nb]) where dK, dV, dB
    are the sums over the selected query rows only (all rows by default)."""
    n, H, d = q.shape
    nb = bias.shape[1]
    rows = np.arange(n) if rows is None else np.asarray(rows)
    dq = np.zeros((len(rows), H, d))
    dk = np.zeros((n, H, d))
    dv = np.zeros((n, H, d))
    db = np.zeros((H, nb))
    inv_sqrt_d = 1.0 / np.sqrt(float(d))
    for r0 in range(0, len(rows), ROW_BLOCK):
        rr = rows[r0:r0 + ROW_BLOCK]
        spd_rows = spd[r0:r0 + len(rr), :n] if compact_spd else spd[rr, :n]
        idx = spd_rows.astype(np.int64).reshape(-1)
        for h in range(H):
            p, _ = _softmax_rows(_scores(q[rr, h, :], k[:, h, :], spd_rows, bias[h]))
            o = p @ v[:, h, :]
            do = dout[rr, h, :]
            delta = (do * o).sum(axis=1, keepdims=True)
            dp = do @ v[:, h, :].T
            ds = p * (dp - delta)
            dv[:, h, :] += p.T @ do
            dq[r0:r0 + len(rr), h, :] = (ds @ k[:, h, :]) * inv_sqrt_d
            dk[:, h, :] += (ds.T @ q[rr, h, :]) * inv_sqrt_d
            db[h] += np.bincount(idx, weights=ds.reshape(-1), minlength=nb)[:nb]
    return dq, dk, dv, db


def chunk_lse(q: np.ndarray, k: np.ndarray, spd: np.ndarray, bias: np.ndarray,
              chunk_bounds: Sequence[Tuple[int, int]], rows: Optional[np.ndarray] = None) -> np.ndarray:
    """Per-chunk log-sum-exp, by definition: LSE_c[h,i] = log sum_{j in [a_c,b_c)} exp S[h,i,j],
    with the bias taken at the GLOBAL (i,j) position.  Empty chunks give -inf.
    Returns fp64 [C,H,r]."""
    n, H, d = q.shape
    rows = np.arange(n) if rows is None else np.asarray(rows)
    res = np.full((len(chunk_bounds), H, len(rows)), -np.inf)
    for r0 in range(0, len(rows), ROW_BLOCK):
        rr = rows[r0:r0 + ROW_BLOCK]
        spd_rows = spd[rr, :n]
        for h in range(H):
            s = _scores(q[rr, h, :], k[:, h, :], spd_rows, bias[h])
            for c, (a, b) in enumerate(chunk_bounds):
                if b > a:
                    sc = s[:, a:b]
                    m = sc.max(axis=1)
                    res[c, h, r0:r0 + len(rr)] = m + np.log(np.exp(sc - m[:, None]).sum(axis=1))
    return res


# ----------------------------------------------------------------------------------
# Packed batches: block-diagonal attention, one shared bias table, dB summed over graphs.
# ----------------------------------------------------------------------------------
def attend_key_set(q: np.ndarray, k: np.ndarray, v: np.ndarray, spd: np.ndarray, bias: np.ndarray,
                   rows: np.ndarray, keys: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Attention of the query rows `rows` over the key subset `keys` only (one graph), with the bias
    taken at the GLOBAL key indices (Eq. 2: Score_local = Q_i K_j^T + b_i[:, Indices(K_j)]).
    Returns the normalised output [r,H,d] and LSE [H,r] of that subset (LSE = -inf, output 0 if empty)."""
    rows, keys = np.asarray(rows), np.asarray(keys)
    n, H, d = q.shape
    o = np.zeros((len(rows), H, d))
    lse = np.full((H, len(rows)), -np.inf)
    if len(keys) == 0:
        return o, lse
    inv_sqrt_d = 1.0 / np.sqrt(float(d))
    b_idx = spd[np.ix_(rows, keys)].astype(np.int64)
    for h in range(H):
        s = (q[rows, h, :] @ k[keys, h, :].T) * inv_sqrt_d + bias[h][b_idx]
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        l = e.sum(axis=1, keepdims=True)
        o[:, h, :] = (e / l) @ v[keys, h, :]
        lse[h] = (m + np.log(l))[:, 0]
    return o, lse


def merge_state(o_acc: np.ndarray, lse_acc: np.ndarray, o_new: np.ndarray, lse_new: np.ndarray):
    """Online-softmax state carried between ring steps (Sec. GA-CP, item 3), in its normalised form:
    (running_max m, running_sum l, unnormalised accumulator A) is kept as lse = m + log l and o = A / l.
    Merging a step's result:  lse' = log(exp lse + exp lse_new),  o' = (exp(lse - lse') o + exp(lse_new - lse') o_new)."""
    m = np.maximum(lse_acc, lse_new)
    safe = np.where(np.isneginf(m), 0.0, m)
    wa, wb = np.exp(lse_acc - safe), np.exp(lse_new - safe)
    tot = wa + wb
    lse = np.where(tot > 0, safe + np.log(np.where(tot > 0, tot, 1.0)), -np.inf)
    fa = np.where(tot > 0, wa / np.where(tot > 0, tot, 1.0), 0.0)
    fb = np.where(tot > 0, wb / np.where(tot > 0, tot, 1.0), 0.0)
    o = fa.T[:, :, None] * o_acc + fb.T[:, :, None] * o_new
    return o, lse


def backward_chunked(q: np.ndarray, k: np.ndarray, v: np.ndarray, dout: np.ndarray, out: np.ndarray,
                     lse: np.ndarray, spd: np.ndarray, bias: np.ndarray, bounds: Sequence[Tuple[int, int]]):
    """Backward pass of Eq. 1 taken one key/value chunk at a time, the way a ring step of the
    paper's context parallelism sees it (Sec. GA-CP): the step holds the key rows [a, b) only, plus
    the forward results `out` [n,H,d] and `lse` [H,n] of the WHOLE row.  With
        P_ij = exp(S_ij - lse_i),  Delta_i = dout_i . out_i,  dS_ij = P_ij (dout_i . v_j - Delta_i)   for j in [a, b)
    a chunk yields dK, dV of its own rows completely, and its share of dQ and dB.  One graph.
    Returns dQ [n,H,d] (sum over chunks), dK, dV [n,H,d], dB [H,nb] (sum) and dB_c [C,H,nb]."""
    n, H, d = q.shape
    nb = bias.shape[1]
    inv_sqrt_d = 1.0 / np.sqrt(float(d))
    dq = np.zeros((n, H, d))
    dk = np.zeros((n, H, d))
    dv = np.zeros((n, H, d))
    db_c = np.zeros((len(bounds), H, nb))
    for c, (a, b) in enumerate(bounds):
        if b <= a:
            continue
        idx = spd[:n, a:b].astype(np.int64).reshape(-1)
        for h in range(H):
            s = (q[:, h, :] @ k[a:b, h, :].T) * inv_sqrt_d + bias[h][spd[:n, a:b]]
            p = np.exp(s - lse[h][:, None])
            do = dout[:, h, :]
            delta = (do * out[:, h, :]).sum(axis=1, keepdims=True)
            ds = p * (do @ v[a:b, h, :].T - delta)
            dv[a:b, h, :] = p.T @ do
            dk[a:b, h, :] = (ds.T @ q[:, h, :]) * inv_sqrt_d
            dq[:, h, :] += (ds @ k[a:b, h, :]) * inv_sqrt_d
            db_c[c, h] = np.bincount(idx, weights=ds.reshape(-1), minlength=nb)[:nb]
    return dq, dk, dv, db_c.sum(axis=0), db_c


def backward_block(q: np.ndarray, k: np.ndarray, v: np.ndarray, dout: np.ndarray, out: np.ndarray,
                   lse: np.ndarray, spd: np.ndarray, bias: np.ndarray, rows: np.ndarray, keys: np.ndarray):
    """What one rank adds at one ring step of the backward (Sec. GA-CP): the pairs (i, j) with i in `rows`
    (the rank's queries) and j in `keys` (the block it holds), given the forward results of the whole rows:
        P_ij = exp(S_ij - lse_i),  dS_ij = P_ij (dout_i . v_j - dout_i . out_i)
    Returns the UNSCALED sums  dq_part [r,H,d] = sum_j dS_ij k_j,  dk_part [m,H,d] = sum_i dS_ij q_i,
    dv_part [m,H,d] = sum_i P_ij dout_i  and db_part [H,nb]; dQ = dq / sqrt(d) and dK = dk / sqrt(d) once
    all blocks are in.  One graph."""
    rows, keys = np.asarray(rows), np.asarray(keys)
    n, H, d = q.shape
    nb = bias.shape[1]
    dq = np.zeros((len(rows), H, d)); dk = np.zeros((len(keys), H, d)); dv = np.zeros((len(keys), H, d))
    db = np.zeros((H, nb))
    if len(rows) == 0 or len(keys) == 0:
        return dq, dk, dv, db
    inv_sqrt_d = 1.0 / np.sqrt(float(d))
    idx = spd[np.ix_(rows, keys)].astype(np.int64)
    for h in range(H):
        s = (q[rows, h, :] @ k[keys, h, :].T) * inv_sqrt_d + bias[h][idx]
        p = np.exp(s - lse[h][rows][:, None])
        do = dout[rows, h, :]
        delta = (do * out[rows, h, :]).sum(axis=1, keepdims=True)
        ds = p * (do @ v[keys, h, :].T - delta)
        dq[:, h, :] = ds @ k[keys, h, :]
        dk[:, h, :] = ds.T @ q[rows, h, :]
        dv[:, h, :] = p.T @ do
        db[h] = np.bincount(idx.reshape(-1), weights=ds.reshape(-1), minlength=nb)[:nb]
    return dq, dk, dv, db


def _spd_block(spd_packed: np.ndarray, spd_offsets: np.ndarray, g: int, n_g: int) -> np.ndarray:
    ld = (n_g + 15) // 16 * 16
    a = int(spd_offsets[g])
    return spd_packed[a:a + n_g * ld].reshape(n_g, ld)


def forward_batch(q, k, v, spd_packed, spd_offsets, cu_seqlens, bias):
    """q,k,v fp64 [T,H,d] packed; returns O [T,H,d], LSE [H,T]."""
    T, H, d = q.shape
    out = np.zeros((T, H, d))
    lse = np.zeros((H, T))
    for g in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[g]), int(cu_seqlens[g + 1])
        if b == a:
            continue
        o_g, l_g = forward_single(q[a:b], k[a:b], v[a:b], _spd_block(spd_packed, spd_offsets, g, b - a), bias)
        out[a:b] = o_g
        lse[:, a:b] = l_g
    return out, lse


def backward_batch(q, k, v, dout, spd_packed, spd_offsets, cu_seqlens, bias):
    """Returns dQ, dK, dV [T,H,d] and dB [H,nb] (summed over the graphs of the batch)."""
    T, H, d = q.shape
    dq, dk, dv = np.zeros((T, H, d)), np.zeros((T, H, d)), np.zeros((T, H, d))
    db = np.zeros_like(bias, dtype=np.float64)
    for g in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[g]), int(cu_seqlens[g + 1])
        if b == a:
            continue
        r = backward_single(q[a:b], k[a:b], v[a:b], dout[a:b], _spd_block(spd_packed, spd_offsets, g, b - a), bias)
        dq[a:b], dk[a:b], dv[a:b] = r[0], r[1], r[2]
        db += r[3]
    return dq, dk, dv, db
