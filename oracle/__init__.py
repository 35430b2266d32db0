"""CPU oracle of the CAOTE eviction step — TEST INFRASTRUCTURE, not part of the product.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
CUDA library never does, and this package never imports the CUDA library. The arithmetic of the
scoring step lives in ``caote_oracle.c`` (plain C, double precision); selection and compaction are
written here with numpy sorts and fancy indexing, straight from their definitions.

Pins (see the CPU tests): attention against torch's fp64 scaled-dot-product attention; scores against
leave-one-out recomputation (Theorem 3.2) and against the weight-renormalisation identity
(Theorem 3.1); closed forms for q = 0 and n = 2; invariances; the H2O mass theorem (Appendix D.1);
selection against a tuple sort; compaction against multiset preservation. The FastCAOTE and joint
multi-token helpers are pinned by their reductions to the single-token score and by brute force (the
greedy sequence by recomputing the output from scratch after every pick, by the joint score of the set it
chose and by exhaustive search over pairs); the post-eviction output against torch attention over the retained set and against the correction formula.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "caote_oracle.c")
_LIB = os.path.join(_HERE, "libcaote_oracle.so")

BASE_MODES = {"last_query": 0, "chunk_sum": 1, "accum": 2, "external": 3}
AGG_MODES = {"weights": 0, "sum_errors": 1}


class _Params(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32),
        ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("capacity", ctypes.c_int32),
        ("n_new", ctypes.c_int32),
        ("scale", ctypes.c_double),
        ("base_mode", ctypes.c_int32),
        ("agg_mode", ctypes.c_int32),
    ]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (``-O2 -fopenmp``) next to its source; returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        fp = ctypes.POINTER(ctypes.c_float)
        ip = ctypes.POINTER(ctypes.c_int32)
        lib.caote_oracle_score.restype = ctypes.c_int
        lib.caote_oracle_score.argtypes = [ctypes.POINTER(_Params), fp, fp, fp, ip, dp, dp, dp, dp, dp]
        lib.caote_oracle_fast_scores.restype = None
        lib.caote_oracle_fast_scores.argtypes = [dp, fp, ctypes.c_int, ctypes.c_int, dp]
        lib.caote_oracle_joint_score.restype = ctypes.c_double
        lib.caote_oracle_joint_score.argtypes = [dp, fp, ctypes.c_int, ctypes.c_int, ip, ctypes.c_int]
        lib.caote_oracle_greedy_evict.restype = ctypes.c_int
        lib.caote_oracle_greedy_evict.argtypes = [dp, fp, ip, ctypes.c_int, ctypes.c_int, ctypes.c_int, ip, dp, dp]
        _lib = lib
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _ptr(a: Optional[np.ndarray], ctype):
    if a is None:
        return ctypes.cast(None, ctypes.POINTER(ctype))
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def num_threads() -> int:
    """Threads the C oracle will use (OpenMP default: the cores this process may run on)."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


def score(q, K, V, lens, *, scale: float, n_new: int = 1, base_mode: str = "last_query",
          base: Optional[np.ndarray] = None, agg_mode: str = "weights"):
    """Scoring step for all units.

    q [B,Hq,m,d], K/V [B,Hkv,cap,d] (float32 arrays holding the exact input values), lens [B].
    ``base`` [B,Hkv,cap] float64 is required for "accum" (a fresh updated copy is returned) and
    "external". Returns a dict with o [B,Hq,m,d], scores [B,Hkv,cap] (NaN behind each length),
    w [B,Hkv,cap], X [B,Hkv,d], base (updated copy or None); all float64.
    """
    q, K, V = _f32(q), _f32(K), _f32(V)
    B, Hq, m, d = q.shape
    _, Hkv, cap, _ = K.shape
    assert m == n_new and K.shape == V.shape and K.shape[0] == B and K.shape[3] == d
    lens = np.ascontiguousarray(np.asarray(lens, dtype=np.int32))
    p = _Params(B, Hq, Hkv, d, cap, m, float(scale), BASE_MODES[base_mode], AGG_MODES[agg_mode])
    o = np.zeros((B, Hq, m, d), dtype=np.float64)
    scores = np.full((B, Hkv, cap), np.nan, dtype=np.float64)
    w = np.full((B, Hkv, cap), np.nan, dtype=np.float64)
    X = np.zeros((B, Hkv, d), dtype=np.float64)
    base_io = None
    if base is not None:
        base_io = np.ascontiguousarray(np.array(base, dtype=np.float64, copy=True))
    rc = _load().caote_oracle_score(
        ctypes.byref(p), _ptr(q, ctypes.c_float), _ptr(K, ctypes.c_float), _ptr(V, ctypes.c_float),
        _ptr(lens, ctypes.c_int32), _ptr(base_io, ctypes.c_double), _ptr(o, ctypes.c_double),
        _ptr(scores, ctypes.c_double), _ptr(w, ctypes.c_double), _ptr(X, ctypes.c_double))
    if rc != 0:
        raise ValueError("caote_oracle_score: bad argument")
    return {"o": o, "scores": scores, "w": w, "X": X, "base": base_io}


def fast_scores(w, V) -> np.ndarray:
    """FastCAOTE scores of one unit (Sec. 3.3): w [n] normalised weights, V [n,d]."""
    w = np.ascontiguousarray(np.asarray(w, dtype=np.float64))
    V = _f32(V)
    n, d = V.shape
    c = np.zeros(n, dtype=np.float64)
    _load().caote_oracle_fast_scores(_ptr(w, ctypes.c_double), _ptr(V, ctypes.c_float), n, d,
                                     _ptr(c, ctypes.c_double))
    return c


def joint_score(w, V, evicted) -> float:
    """Joint eviction error of a set of tokens of one unit (Appendix B)."""
    w = np.ascontiguousarray(np.asarray(w, dtype=np.float64))
    V = _f32(V)
    E = np.ascontiguousarray(np.asarray(evicted, dtype=np.int32))
    n, d = V.shape
    return float(_load().caote_oracle_joint_score(_ptr(w, ctypes.c_double), _ptr(V, ctypes.c_float),
                                                  n, d, _ptr(E, ctypes.c_int32), len(E)))


def greedy_evict(w, V, k: int, pos=None):
    """Greedy multi-token eviction of one unit (Appendix B chained): k times evict the token whose removal
    changes the current output least, renormalise the weights of the rest and update the output.

    w [n] normalised weights, V [n,d], pos [n] tie-break keys or None (slot index). Returns
    (order [k] slots in eviction order, step_score [k] each pick's score at its step,
    cum_err [k] distance between the original output and the output after each eviction).
    """
    w = np.ascontiguousarray(np.asarray(w, dtype=np.float64))
    V = _f32(V)
    n, d = V.shape
    order = np.zeros(k, dtype=np.int32)
    step = np.zeros(k, dtype=np.float64)
    cum = np.zeros(k, dtype=np.float64)
    pos_a = None if pos is None else np.ascontiguousarray(np.asarray(pos, dtype=np.int32))
    rc = _load().caote_oracle_greedy_evict(_ptr(w, ctypes.c_double), _ptr(V, ctypes.c_float),
                                           _ptr(pos_a, ctypes.c_int32), n, d, int(k),
                                           _ptr(order, ctypes.c_int32), _ptr(step, ctypes.c_double),
                                           _ptr(cum, ctypes.c_double))
    if rc != 0:
        raise ValueError("caote_oracle_greedy_evict: bad argument (need 0 <= k < n)")
    return order, step, cum


def post_evict_output(q, K, V, lens, evict, *, scale: float, n_new: int = 1) -> np.ndarray:
    """Attention output over the retained tokens (Sec. 2: the budgeted cache attends over what it kept).

    Written from the definition, row by row: query i of the block sees slots j <= n - m + i; the evicted
    slots ``evict[b][h]`` are taken out; softmax over what is left, in double. A row left with nothing to
    see gets zeros. q [B,Hq,m,d], K/V [B,Hkv,cap,d]; returns [B,Hq,m,d] float64.
    """
    q, K, V = _f32(q).astype(np.float64), _f32(K).astype(np.float64), _f32(V).astype(np.float64)
    B, Hq, m, d = q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    assert m == n_new
    out = np.zeros((B, Hq, m, d), dtype=np.float64)
    for b in range(B):
        n = int(lens[b])
        if n == 0:
            continue
        for h in range(Hkv):
            gone = np.zeros(n, dtype=bool)
            gone[np.asarray(evict[b][h], dtype=np.int64)] = True
            for g in range(G):
                for i in range(m):
                    keep = ~gone
                    keep[n - m + i + 1:] = False
                    if not keep.any():
                        continue
                    s = scale * (K[b, h, :n][keep] @ q[b, h * G + g, i])
                    w = np.exp(s - s.max())
                    out[b, h * G + g, i] = (w / w.sum()) @ V[b, h, :n][keep]
    return out


def select_evict(scores, lens, budget, pos=None) -> Tuple[list, np.ndarray]:
    """Tokens to evict (Sec. 2: the top-b tokens by score are retained).

    For sequence b, k = max(0, len[b] - budget[b]); every unit evicts its k smallest entries under
    the order (score, pos) ascending (tie-break towards the older token is this build's reading; the
    paper does not say). Returns (evict[b][h] = ascending array of slot indices, n_evict [B]).
    """
    scores = np.asarray(scores)
    B, Hkv, cap = scores.shape
    lens = np.asarray(lens, dtype=np.int64)
    budget = np.maximum(np.asarray(budget, dtype=np.int64), 1)
    n_evict = np.maximum(lens - budget, 0).astype(np.int32)
    out = []
    for b in range(B):
        row = []
        n, k = int(lens[b]), int(n_evict[b])
        for h in range(Hkv):
            c = scores[b, h, :n]
            key2 = np.arange(n) if pos is None else np.asarray(pos)[b, h, :n]
            order = np.lexsort((key2, c))  # primary key: score, secondary: pos
            row.append(np.sort(order[:k]).astype(np.int32))
        out.append(row)
    return out, n_evict


def compact(arrays, lens, evict):
    """Drop the evicted slots, keeping the survivors in their order (the STABLE layout).

    ``arrays``: list of arrays shaped [B,Hkv,cap,...]; returns (new arrays, new lens); slots behind
    the new length are zero-filled.
    """
    lens = np.asarray(lens, dtype=np.int64)
    outs = [np.zeros_like(a) for a in arrays]
    new_lens = lens.copy()
    B, Hkv = arrays[0].shape[:2]
    for b in range(B):
        n = int(lens[b])
        for h in range(Hkv):
            keep = np.setdiff1d(np.arange(n), evict[b][h])
            for a, o in zip(arrays, outs):
                o[b, h, : len(keep)] = a[b, h, keep]
        new_lens[b] = n - len(evict[b][0])
    return outs, new_lens.astype(np.int32)
