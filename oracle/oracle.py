"""numpy front end of the fp64 CPU oracle in calidrop_oracle.c.

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the bench's
CPU-baseline leg may use this module.  It shares nothing with the CUDA path; it only
marshals numpy arrays into the plain-C oracle (built with gcc on first use).

All tensors that the method treats as bf16 are passed as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "calidrop_oracle.c")
_LIB = os.path.join(_HERE, "libcalidrop_oracle.so")
_lib = None


def build_oracle(force: bool = False) -> str:
    """Compile calidrop_oracle.c with gcc (OpenMP, no fast-math) if it is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build_oracle())
        _lib.oracle_max_threads.restype = C.c_int
        _lib.oracle_compress.restype = C.c_int
        _lib.oracle_calibrate_given_indices.restype = C.c_int
    return _lib


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def default_scale(D: int) -> float:
    return 1.0 / math.sqrt(D)


def full_attention(q, K, V, scale=None):
    """Brute-force softmax attention: q [nq, D], K and V [n, D] (bf16 bits) -> out [nq, D], lse [nq]."""
    q, K, V = _u16(q), _u16(K), _u16(V)
    nq, D = q.shape
    n = K.shape[0]
    out = np.zeros((nq, D), dtype=np.float64)
    lse = np.zeros((nq,), dtype=np.float64)
    _load().oracle_full_attention(_p(q), _p(K), _p(V), C.c_int(nq), C.c_int64(n), C.c_int(D),
                                  C.c_double(scale or default_scale(D)), _p(out), _p(lse))
    return out, lse


def pool_votes(vote, pool):
    vote = np.ascontiguousarray(vote, dtype=np.float64)
    out = np.empty_like(vote)
    _load().oracle_pool(_p(vote), C.c_int64(vote.size), C.c_int(pool), _p(out))
    return out


def topk(score, k):
    score = np.ascontiguousarray(score, dtype=np.float64)
    out = np.empty((k,), dtype=np.int32)
    _load().oracle_topk(_p(score), C.c_int64(score.size), C.c_int64(k), _p(out))
    return out


def compress(Q_obs, K, V, *, window, pool, budget, n_cal=1, cap=None, scale=None, calib_size=None):
    """Oracle compress-and-calibrate.  Q_obs [B,Hq,W,D], K,V [B,Hkv,L,D] bf16 bits.
    calib_size: None = every evicted token is calibrated (Algorithm 1 as printed); m >= 0 = only the
    m evicted tokens of highest pooled vote (the "calibration size" of the paper's Section 4.4),
    whose ascending indices are returned as calib_idx [B,Hkv,min(m, number evicted)]."""
    Q_obs, K, V = _u16(Q_obs), _u16(K), _u16(V)
    B, Hq, W, D = Q_obs.shape
    _, Hkv, L, _ = K.shape
    assert W == window
    n_kept = min(budget, L)
    cap = cap or n_kept
    n_cand = max(L - W, 0)
    r = SimpleNamespace(
        kept_idx=np.zeros((B, Hkv, n_kept), dtype=np.int32),
        K_kept=np.zeros((B, Hkv, cap, D), dtype=np.uint16),
        V_kept=np.zeros((B, Hkv, cap, D), dtype=np.uint16),
        O_c=np.zeros((B, Hq, n_cal, D), dtype=np.float64),
        LSE_c=np.zeros((B, Hq, n_cal), dtype=np.float64),
        C_q=np.zeros((B, Hq, n_cal, D), dtype=np.uint16),
        vote=np.zeros((B, Hkv, n_cand), dtype=np.float64),
        pooled=np.zeros((B, Hkv, n_cand), dtype=np.float64),
        row_lse=np.zeros((B, Hq, W), dtype=np.float64),
        n_kept=n_kept, cap=cap, calib_idx=None,
    )
    m = -1
    if calib_size is not None and budget < L:
        m = min(int(calib_size), n_cand - (budget - W))
        r.calib_idx = np.zeros((B, Hkv, m), dtype=np.int32)
    rc = _load().oracle_compress(
        _p(Q_obs), _p(K), _p(V), C.c_int(B), C.c_int(Hq), C.c_int(Hkv), C.c_int64(L), C.c_int(D),
        C.c_int(W), C.c_int(pool), C.c_int64(budget), C.c_int(n_cal), C.c_int64(cap),
        C.c_double(scale or default_scale(D)),
        _p(r.kept_idx), _p(r.K_kept), _p(r.V_kept), _p(r.O_c), _p(r.LSE_c), _p(r.C_q),
        _p(r.vote), _p(r.pooled), _p(r.row_lse), C.c_int64(m), _p(r.calib_idx))
    if rc != 0:
        raise ValueError("oracle_compress: arguments outside the method's definition")
    return r


def calibrate_given_indices(Q_obs, K, V, kept_idx, *, n_cal=1, cap=None, scale=None):
    """Gather and calibrate for an externally supplied kept list kept_idx [B,Hkv,n_kept]."""
    Q_obs, K, V = _u16(Q_obs), _u16(K), _u16(V)
    kept_idx = np.ascontiguousarray(kept_idx, dtype=np.int32)
    B, Hq, W, D = Q_obs.shape
    _, Hkv, L, _ = K.shape
    n_kept = kept_idx.shape[-1]
    cap = cap or n_kept
    r = SimpleNamespace(
        kept_idx=kept_idx,
        K_kept=np.zeros((B, Hkv, cap, D), dtype=np.uint16),
        V_kept=np.zeros((B, Hkv, cap, D), dtype=np.uint16),
        O_c=np.zeros((B, Hq, n_cal, D), dtype=np.float64),
        LSE_c=np.zeros((B, Hq, n_cal), dtype=np.float64),
        C_q=np.zeros((B, Hq, n_cal, D), dtype=np.uint16),
        n_kept=n_kept, cap=cap,
    )
    rc = _load().oracle_calibrate_given_indices(
        _p(Q_obs), _p(K), _p(V), C.c_int(B), C.c_int(Hq), C.c_int(Hkv), C.c_int64(L), C.c_int(D),
        C.c_int(W), C.c_int(n_cal), C.c_int64(cap), C.c_double(scale or default_scale(D)),
        _p(kept_idx), C.c_int64(n_kept), _p(r.K_kept), _p(r.V_kept), _p(r.O_c), _p(r.LSE_c),
        _p(r.C_q))
    if rc != 0:
        raise ValueError("oracle_calibrate_given_indices: bad arguments")
    return r


def decode(q, k_new, v_new, K_kept, V_kept, kv_len, O_c, LSE_c, C_q, *,
           theta1=0.7, theta2=0.85, scale=None, force_c=None, force_apply=None):
    """One oracle decode step.  K_kept/V_kept [B,Hkv,cap,D] are updated in place."""
    q = _u16(q)
    B, Hq, D = q.shape
    assert K_kept.dtype == np.uint16 and K_kept.flags.c_contiguous
    assert V_kept.dtype == np.uint16 and V_kept.flags.c_contiguous
    _, Hkv, cap, _ = K_kept.shape
    O_c = np.ascontiguousarray(O_c, dtype=np.float64)
    LSE_c = np.ascontiguousarray(LSE_c, dtype=np.float64)
    C_q = _u16(C_q)
    n_cal = LSE_c.shape[-1]
    if k_new is not None:
        k_new, v_new = _u16(k_new), _u16(v_new)
        assert kv_len + 1 <= cap
    if force_c is not None:
        force_c = np.ascontiguousarray(force_c, dtype=np.int32)
    if force_apply is not None:
        force_apply = np.ascontiguousarray(force_apply, dtype=np.int32)
    r = SimpleNamespace(
        out=np.zeros((B, Hq, D), dtype=np.float64),
        lse=np.zeros((B, Hq), dtype=np.float64),
        lse_a=np.zeros((B, Hq), dtype=np.float64),
        rho=np.zeros((B, Hq, n_cal), dtype=np.float64),
        flags=np.zeros((B, Hq), dtype=np.uint8),
    )
    _load().oracle_decode(
        _p(q), _p(k_new), _p(v_new), _p(K_kept), _p(V_kept), C.c_int64(kv_len),
        _p(O_c), _p(LSE_c), _p(C_q), C.c_int(B), C.c_int(Hq), C.c_int(Hkv), C.c_int(D),
        C.c_int(n_cal), C.c_int64(cap), C.c_double(scale or default_scale(D)),
        C.c_double(theta1), C.c_double(theta2), _p(force_c), _p(force_apply),
        _p(r.out), _p(r.lse), _p(r.lse_a), _p(r.rho), _p(r.flags))
    return r


def streaming_indices(L, budget, n_sink):
    """StreamingLLM's rule (Section 4.1.3): the first n_sink prompt rows and the most recent ones, min(budget, L) in all."""
    n_kept = min(budget, L)
    n_sink = min(n_sink, n_kept)
    return np.concatenate([np.arange(n_sink), np.arange(L - (n_kept - n_sink), L)]).astype(np.int32)


def select_from_scores(scores, *, tail, budget, pool=1):
    """Kept list from per-row scores [L]: the last `tail` rows plus the budget - tail rows of [0, L - tail) with
    the largest (pooled) score, ties to the lower index; ascending.  With H2O's accumulated attention score and
    tail = budget / 2 this is H2O's rule (Section 4.1.3)."""
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    L = scores.shape[-1]
    assert 0 < tail < budget < L
    pooled = pool_votes(scores[:L - tail], pool)
    return np.concatenate([topk(pooled, budget - tail), np.arange(L - tail, L)]).astype(np.int32)


def accumulated_attention(Q_full, K, scale=None):
    """H2O's importance: for one kv head, the causal softmax attention of every prompt query of its query group
    (Q_full [G, L, D], K [L, D], bf16 bits), summed over the queries and the group: score[t] = sum_g sum_{i >= t} a[g,i,t]."""
    Q_full, K = _u16(Q_full), _u16(K)
    G, L, D = Q_full.shape
    scale = scale or default_scale(D)
    Kf = (K.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    score = np.zeros((L,), dtype=np.float64)
    for g in range(G):
        Qf = (Q_full[g].astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        for i in range(L):
            s = (Kf[:i + 1] @ Qf[i]) * scale
            e = np.exp(s - s.max())
            score[:i + 1] += e / e.sum()
    return score
