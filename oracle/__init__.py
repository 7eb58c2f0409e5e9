"""CPU oracle of the selection path (ctypes front end of ks_oracle.cpp).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import this package. It neither imports nor is imported by
the CUDA package; inputs come in as numpy arrays with the record layouts declared in
ks_oracle.cpp.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ks_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

ROW = 64
_lib = None


def build(force: bool = False) -> str:
    """Compile ks_oracle.cpp (g++, -O2, no FMA contraction, OpenMP over problems)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared",
               "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def _p(a, ctype=ctypes.c_void_p):
    return None if a is None else a.ctypes.data_as(ctype)


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(lib().orc_threads())


def set_threads(n: int) -> None:
    lib().orc_set_threads(ctypes.c_int(n))


def _check(arr, itemsize, name):
    if arr is None:
        return None
    a = np.ascontiguousarray(arr)
    if a.dtype.itemsize != itemsize:
        raise ValueError(f"{name}: itemsize {a.dtype.itemsize}, expected {itemsize}")
    return a


def _desc(desc):
    d = np.ascontiguousarray(desc)
    if d.nbytes != 80:
        raise ValueError("gpu descriptor must be 80 bytes")
    return d


def _pairs(P, C, seg_off):
    return int(seg_off[-1]) if seg_off is not None else P * C


def featurize(problems, candidates, desc, seg_off=None, seg_idx=None):
    p = _check(problems, 16, "problems")
    c = _check(candidates, 16, "candidates")
    so = None if seg_off is None else np.ascontiguousarray(seg_off, dtype=np.int64)
    si = None if seg_idx is None else np.ascontiguousarray(seg_idx, dtype=np.int32)
    out = np.empty((_pairs(len(p), len(c), so), ROW), dtype=np.float32)
    lib().orc_featurize(_p(p), ctypes.c_int(len(p)), _p(c), ctypes.c_int(len(c)), _p(so), _p(si),
                        _p(_desc(desc)), _p(out))
    return out


def score_gbdt(features, tree_offsets, nodes, base_score=0.0, want_leaf_idx=False):
    f = np.ascontiguousarray(features, dtype=np.float32).reshape(-1, ROW)
    off = np.ascontiguousarray(tree_offsets, dtype=np.int64)
    nd = _check(nodes, 12, "nodes")
    n_trees = len(off) - 1
    scores = np.empty(len(f), dtype=np.float32)
    leaf = np.empty((len(f), n_trees), dtype=np.uint16) if want_leaf_idx else None
    lib().orc_score_gbdt(_p(f), ctypes.c_int64(len(f)), ctypes.c_int(n_trees), _p(off), _p(nd),
                         ctypes.c_float(base_score), _p(scores), _p(leaf))
    return (scores, leaf) if want_leaf_idx else scores


def _mlp_args(mlp):
    widths = np.ascontiguousarray(mlp["widths"], dtype=np.int32)
    L = len(widths) - 1
    ws = [np.ascontiguousarray(w, dtype=np.uint16) for w in mlp["weights"]]
    bs = [np.ascontiguousarray(b, dtype=np.float32) for b in mlp["biases"]]
    mu = np.ascontiguousarray(mlp["mu"], dtype=np.float32)
    sigma = np.ascontiguousarray(mlp["sigma"], dtype=np.float32)
    wp = (ctypes.c_void_p * L)(*[w.ctypes.data for w in ws])
    bp = (ctypes.c_void_p * L)(*[b.ctypes.data for b in bs])
    keep = (widths, ws, bs, mu, sigma, wp, bp)
    return L, widths, wp, bp, mu, sigma, keep


def score_mlp(features, mlp):
    f = np.ascontiguousarray(features, dtype=np.float32).reshape(-1, ROW)
    L, widths, wp, bp, mu, sigma, _keep = _mlp_args(mlp)
    scores = np.empty(len(f), dtype=np.float32)
    lib().orc_score_mlp(_p(f), ctypes.c_int64(len(f)), ctypes.c_int(L), _p(widths), wp, bp, _p(mu),
                        _p(sigma), _p(scores))
    return scores


def topk(scores, P, k, rows_per_problem=0, seg_off=None, seg_idx=None):
    s = np.ascontiguousarray(scores, dtype=np.float32)
    so = None if seg_off is None else np.ascontiguousarray(seg_off, dtype=np.int64)
    si = None if seg_idx is None else np.ascontiguousarray(seg_idx, dtype=np.int32)
    idx = np.empty((P, k), dtype=np.int32)
    sc = np.empty((P, k), dtype=np.float32)
    lib().orc_topk(_p(s), ctypes.c_int(P), ctypes.c_int64(rows_per_problem), _p(so), _p(si),
                   ctypes.c_int(k), _p(idx), _p(sc))
    return idx, sc


def select(problems, candidates, desc, k, gbdt=None, mlp=None, seg_off=None, seg_idx=None,
           want_scores=False, static=False):
    """Featurize + score + full sort per problem. gbdt = (tree_offsets, nodes, base_score);
    static=True ranks by the static sampling score instead of a learned model."""
    if (gbdt is not None) + (mlp is not None) + bool(static) != 1:
        raise ValueError("pass exactly one of gbdt / mlp / static")
    p = _check(problems, 16, "problems")
    c = _check(candidates, 16, "candidates")
    so = None if seg_off is None else np.ascontiguousarray(seg_off, dtype=np.int64)
    si = None if seg_idx is None else np.ascontiguousarray(seg_idx, dtype=np.int32)
    P = len(p)
    idx = np.empty((P, k), dtype=np.int32)
    sc = np.empty((P, k), dtype=np.float32)
    allsc = np.empty(_pairs(P, len(c), so), dtype=np.float32) if want_scores else None
    if static:
        lib().orc_select(_p(p), ctypes.c_int(P), _p(c), ctypes.c_int(len(c)), _p(so), _p(si),
                         _p(_desc(desc)), ctypes.c_int(2), ctypes.c_int(0), None, None,
                         ctypes.c_float(0.0), ctypes.c_int(0), None, None, None, None, None,
                         ctypes.c_int(k), _p(idx), _p(sc), _p(allsc))
    elif gbdt is not None:
        off = np.ascontiguousarray(gbdt[0], dtype=np.int64)
        nd = _check(gbdt[1], 12, "nodes")
        base = float(gbdt[2]) if len(gbdt) > 2 else 0.0
        lib().orc_select(_p(p), ctypes.c_int(P), _p(c), ctypes.c_int(len(c)), _p(so), _p(si),
                         _p(_desc(desc)), ctypes.c_int(0), ctypes.c_int(len(off) - 1), _p(off),
                         _p(nd), ctypes.c_float(base), ctypes.c_int(0), None, None, None, None, None,
                         ctypes.c_int(k), _p(idx), _p(sc), _p(allsc))
    else:
        L, widths, wp, bp, mu, sigma, _keep = _mlp_args(mlp)
        lib().orc_select(_p(p), ctypes.c_int(P), _p(c), ctypes.c_int(len(c)), _p(so), _p(si),
                         _p(_desc(desc)), ctypes.c_int(1), ctypes.c_int(0), None, None,
                         ctypes.c_float(0.0), ctypes.c_int(L), _p(widths), wp, bp, _p(mu), _p(sigma),
                         ctypes.c_int(k), _p(idx), _p(sc), _p(allsc))
    return (idx, sc, allsc) if want_scores else (idx, sc)


CANDIDATE_BYTES = 16


def catalogue_size() -> int:
    lib().orc_catalogue_size.restype = ctypes.c_int64
    return int(lib().orc_catalogue_size())


def enumerate_candidates(first: int, count: int, dtype) -> np.ndarray:
    """Search-space records with ids first .. first+count-1 (dtype: a 16-byte record dtype)."""
    out = np.zeros(count, dtype=dtype)
    assert out.dtype.itemsize == CANDIDATE_BYTES
    lib().orc_enumerate(ctypes.c_int64(first), ctypes.c_int64(count), _p(out))
    return out


def valid_catalogue(problem, desc, flags: int, candidates=None, count=None, dtype=None):
    """Stable filter of `candidates` (None: the search space's first `count` ids) by the static
    validity rules. Returns (kept records, their positions int32)."""
    p = _check(problem, 16, "problem")
    c = None if candidates is None else _check(candidates, 16, "candidates")
    C = len(c) if c is not None else (catalogue_size() if count is None else int(count))
    dt = c.dtype if c is not None else dtype
    out_c = np.zeros(C, dtype=dt)
    out_i = np.empty(C, dtype=np.int32)
    f = lib().orc_valid_catalogue
    f.restype = ctypes.c_int64
    n = int(f(_p(p), _p(c), ctypes.c_int64(C), _p(_desc(desc)), ctypes.c_uint(flags), _p(out_c), _p(out_i)))
    return out_c[:n].copy(), out_i[:n].copy()
