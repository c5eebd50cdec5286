"""CPU ORACLE -- TEST INFRASTRUCTURE ONLY (never imported by the product path).

Shortest-path-distance index matrix: thin ctypes wrapper over ``spd_bfs.c`` (textbook
queue BFS per source), plus the packed-batch layout helper.  The arithmetic lives in the
C file; this module only compiles it on demand with gcc and marshals numpy arrays.

Pinned by tests against Floyd-Warshall brute force, closed-form graphs (path, cycle,
star, grid, hypercube, complete, empty, disjoint union), structural invariants and
scipy's unweighted shortest_path.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spd_bfs.c")
_LIB = os.path.join(_HERE, "liboracle_spd.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile spd_bfs.c into liboracle_spd.so (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_spd_bfs.restype = ctypes.c_int
        lib.oracle_spd_bfs.argtypes = [ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                       ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p]
        lib.oracle_spd_bfs_sources.restype = ctypes.c_int
        lib.oracle_spd_bfs_sources.argtypes = [ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32,
                                               ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p]
        _lib = lib
    return _lib


def spd_matrix(row_ptr: np.ndarray, col_idx: np.ndarray, max_dist: int, ld: int | None = None) -> np.ndarray:
    """uint8 [n, ld] SPD index matrix of one graph (local node ids 0..n-1).

    spd[s][t] = min(hops(s->t), max_dist) if reachable else max_dist+1; padding = 255.
    """
    n = len(row_ptr) - 1
    if ld is None:
        ld = (n + 15) // 16 * 16
    rp = np.ascontiguousarray(row_ptr, dtype=np.int32)
    ci = np.ascontiguousarray(col_idx, dtype=np.int32)
    if ci.size == 0:
        ci = np.zeros(1, np.int32)
    out = np.empty((n, ld), dtype=np.uint8)
    rc = _load().oracle_spd_bfs(n, rp.ctypes.data, ci.ctypes.data, int(max_dist), int(ld), out.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"oracle_spd_bfs failed with code {rc}")
    return out


def spd_rows(row_ptr: np.ndarray, col_idx: np.ndarray, max_dist: int, sources: np.ndarray) -> np.ndarray:
    """uint8 [len(sources), ld]: the SPD rows of the listed sources only (BFS from each)."""
    n = len(row_ptr) - 1
    ld = (n + 15) // 16 * 16
    rp = np.ascontiguousarray(row_ptr, dtype=np.int32)
    ci = np.ascontiguousarray(col_idx, dtype=np.int32)
    if ci.size == 0:
        ci = np.zeros(1, np.int32)
    src = np.ascontiguousarray(sources, dtype=np.int32)
    out = np.empty((len(src), ld), dtype=np.uint8)
    rc = _load().oracle_spd_bfs_sources(n, rp.ctypes.data, ci.ctypes.data, int(max_dist), int(ld),
                                        len(src), src.ctypes.data, out.ctypes.data)
    if rc != 0:
        raise RuntimeError(f"oracle_spd_bfs_sources failed with code {rc}")
    return out


def spd_packed(row_ptr: np.ndarray, col_idx: np.ndarray, cu_seqlens: np.ndarray, max_dist: int) -> np.ndarray:
    """Packed SPD of a block-diagonal batch: graph g's n_g x ld_g block (ld_g = n_g rounded
    up to 16) starts at byte sum_{g'<g} n_g' * ld_g'.  Returns a flat uint8 array."""
    blocks = []
    for g in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[g]), int(cu_seqlens[g + 1])
        lo, hi = int(row_ptr[a]), int(row_ptr[b])
        rp = (np.asarray(row_ptr[a:b + 1], dtype=np.int64) - lo).astype(np.int32)
        ci = (np.asarray(col_idx[lo:hi], dtype=np.int64) - a).astype(np.int32)
        blocks.append(spd_matrix(rp, ci, max_dist).reshape(-1))
    return np.concatenate(blocks) if blocks else np.zeros(0, np.uint8)
