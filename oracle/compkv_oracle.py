"""ctypes front end of the CPU oracle (compkv_oracle.c) -- TEST INFRASTRUCTURE, NOT A PRODUCT PATH.

Only tests, the smoke check and the bench's CPU-baseline leg may import this
module.  It never touches the CUDA library; it compiles the C file with gcc on
first use and marshals numpy arrays.  Every function works on one unit: one KV
head of one sequence with the G query heads sharing it (Sec. 3.1).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "compkv_oracle.c")
_LIB = os.path.join(_HERE, "libcompkv_oracle.so")
_lib = None

_F = ctypes.POINTER(ctypes.c_float)
_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, -O2, no fast-math); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.ckvo_group_of.restype = ctypes.c_int
        lib.ckvo_select.restype = ctypes.c_int
        lib.ckvo_kl.restype = ctypes.c_double
        for name in ("ckvo_dense", "ckvo_stats", "ckvo_scores", "ckvo_sparse", "ckvo_token_dists",
                     "ckvo_exact_blocks"):
            getattr(lib, name).restype = None
        _lib = lib
    return _lib


def _f(a):
    assert a.dtype == np.float32 and a.flags.c_contiguous
    return a.ctypes.data_as(_F)


def _d(a):
    assert a.dtype == np.float64 and a.flags.c_contiguous
    return a.ctypes.data_as(_D)


def _i(a):
    assert a.dtype == np.int32 and a.flags.c_contiguous
    return a.ctypes.data_as(_I)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


_ci, _cd = ctypes.c_int, ctypes.c_double


def default_scale(d: int) -> float:
    return 1.0 / float(np.sqrt(d))


def group_of(i: int, d: int, r: int, layout: int) -> int:
    return int(_load().ckvo_group_of(_ci(i), _ci(d), _ci(r), _ci(layout)))


def dense(q, K, V, scale: Optional[float] = None):
    """Dense attention of the unit's G heads: returns (out [G][d], lse [G])."""
    q, K, V = _f32(q), _f32(K), _f32(V)
    G, d = q.shape
    N = K.shape[0]
    out = np.zeros((G, d)); lse = np.zeros(G)
    _load().ckvo_dense(_f(q), _f(K), _f(V), _ci(N), _ci(G), _ci(d), _cd(scale or default_scale(d)), _d(out), _d(lse))
    return out, lse


@dataclass
class Stats:
    cnt: np.ndarray    # int32 [X]
    kmean: np.ndarray  # float64 [X][d]
    Dbar: np.ndarray   # float64 [X][r]
    vmean: np.ndarray  # float64 [X][d]
    bs: int
    r: int
    layout: int


def stats(K, V, bs: int, r: int = 4, layout: int = 1, first_block: int = 0, nblocks: Optional[int] = None) -> Stats:
    """Block summaries of a cache (Eq. 8 right half, Sec. 4.2)."""
    K, V = _f32(K), _f32(V)
    N, d = K.shape
    X = -(-N // bs)
    nb = X - first_block if nblocks is None else nblocks
    cnt = np.zeros(nb, np.int32); km = np.zeros((nb, d)); D = np.zeros((nb, r)); vm = np.zeros((nb, d))
    _load().ckvo_stats(_f(K), _f(V), _ci(N), _ci(d), _ci(bs), _ci(r), _ci(layout), _ci(first_block), _ci(nb),
                       _i(cnt), _d(km), _d(D), _d(vm))
    return Stats(cnt, km, D, vm, bs, r, layout)


def append(st: Stats, K, V) -> Stats:
    """Summaries after the cache grew to K/V: every completed block keeps its summary, the
    active (last) block -- and any block the new tokens opened -- is recomputed from its tokens
    (Sec. 4.2: summaries are updated as new K/V states enter the active block)."""
    K, V = _f32(K), _f32(V)
    N = K.shape[0]
    X_new = -(-N // st.bs)
    first = max(len(st.cnt) - 1, 0)
    tail = stats(K, V, st.bs, st.r, st.layout, first_block=first, nblocks=X_new - first)
    return Stats(np.concatenate([st.cnt[:first], tail.cnt]), np.concatenate([st.kmean[:first], tail.kmean]),
                 np.concatenate([st.Dbar[:first], tail.Dbar]), np.concatenate([st.vmean[:first], tail.vmean]),
                 st.bs, st.r, st.layout)


@dataclass
class Scores:
    zbar: np.ndarray    # [G][X]
    sigma2: np.ndarray  # [G][X]
    phat: np.ndarray    # [G][X]
    S: np.ndarray       # [X]


def scores(q, st: Stats, scale: Optional[float] = None, mass_order: int = 2, outer_var: int = 1) -> Scores:
    """Eq. 8 (left), Eq. 9, Eq. 10."""
    q = _f32(q)
    G, d = q.shape
    X = len(st.cnt)
    zb = np.zeros((G, X)); s2 = np.zeros((G, X)); ph = np.zeros((G, X)); S = np.zeros(X)
    _load().ckvo_scores(_f(q), _i(st.cnt), _d(st.kmean), _d(st.Dbar), _ci(X), _ci(G), _ci(d), _ci(st.r),
                        _ci(st.layout), _cd(scale or default_scale(d)), _ci(mass_order), _ci(outer_var),
                        _d(zb), _d(s2), _d(ph), _d(S))
    return Scores(zb, s2, ph, S)


def select(S, K: int, sink: int = 1, recent: int = 2) -> np.ndarray:
    """Eq. 11: ascending block ids; raises if the budget cannot hold the mandatory blocks."""
    S = np.ascontiguousarray(S, dtype=np.float64)
    X = len(S)
    ids = np.zeros(max(X, 1), np.int32)
    n = _load().ckvo_select(_d(S), _ci(X), _ci(K), _ci(sink), _ci(recent), _i(ids))
    if n < 0:
        raise ValueError("budget of %d blocks cannot hold the mandatory blocks" % K)
    return ids[:n].copy()


def sparse(q, K, V, st: Stats, ids: Sequence[int], scale: Optional[float] = None, drop: bool = False):
    """Eq. 12 (or its Drop variant): returns (out [G][d], lse [G])."""
    q, K, V = _f32(q), _f32(K), _f32(V)
    G, d = q.shape
    N = K.shape[0]
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    out = np.zeros((G, d)); lse = np.zeros(G)
    _load().ckvo_sparse(_f(q), _f(K), _f(V), _ci(N), _ci(G), _ci(d), _ci(st.bs), _i(st.cnt), _d(st.kmean),
                        _d(st.vmean), _i(ids), _ci(len(ids)), _cd(scale or default_scale(d)), _ci(int(drop)),
                        _d(out), _d(lse))
    return out, lse


def token_dists(qg, K, bs: int, ids: Sequence[int], scale: Optional[float] = None, drop: bool = False):
    """Token-level P, Phat(S) of one head and log D, log Dhat (Eq. 1, App. A.1)."""
    qg, K = _f32(qg), _f32(K)
    N, d = K.shape
    ids = np.ascontiguousarray(ids, dtype=np.int32)
    P = np.zeros(N); Ph = np.zeros(N); a = _cd(0.0); b = _cd(0.0)
    _load().ckvo_token_dists(_f(qg), _f(K), _ci(N), _ci(d), _ci(bs), _i(ids), _ci(len(ids)),
                             _cd(scale or default_scale(d)), _ci(int(drop)), _d(P), _d(Ph),
                             ctypes.byref(a), ctypes.byref(b))
    return P, Ph, a.value, b.value


def kl(A, B) -> float:
    A = np.ascontiguousarray(A, dtype=np.float64); B = np.ascontiguousarray(B, dtype=np.float64)
    return float(_load().ckvo_kl(_d(A), _d(B), _ci(len(A))))


@dataclass
class ExactBlocks:
    p: np.ndarray
    sigma2: np.ndarray
    rho: np.ndarray
    ratio: np.ndarray
    logZ: np.ndarray


def exact_blocks(qg, K, bs: int, scale: Optional[float] = None) -> ExactBlocks:
    """Eq. 3 and the exact compensation residual of App. B.1 for one head."""
    qg, K = _f32(qg), _f32(K)
    N, d = K.shape
    X = -(-N // bs)
    arrs = [np.zeros(X) for _ in range(5)]
    _load().ckvo_exact_blocks(_f(qg), _f(K), _ci(N), _ci(d), _ci(bs), _cd(scale or default_scale(d)),
                              *[_d(a) for a in arrs])
    return ExactBlocks(*arrs)


def decode_unit(q, K, V, st: Stats, budget_tokens: int, sink: int = 1, recent: int = 2,
                scale: Optional[float] = None):
    """One decode step of a unit: scores -> selection -> compensated attention.
    Returns (out [G][d], lse [G], ids, Scores)."""
    sc = scores(q, st, scale)
    ids = select(sc.S, budget_tokens // st.bs, sink, recent)
    out, lse = sparse(q, K, V, st, ids, scale)
    return out, lse, ids, sc
