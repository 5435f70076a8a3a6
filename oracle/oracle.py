"""ctypes front end of the C oracle (test infrastructure only).

Arrays are numpy: fp32 tensors as float32, bf16 tensors as uint16 bit patterns
(the oracle widens them exactly). Index outputs are int32, weights float32.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "exfold_oracle.c")
_LIB = os.path.join(_HERE, "libexfold_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no contraction, no fast-math, OpenMP over tokens)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-fPIC",
                               "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _L():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dt(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    raise TypeError(f"oracle tensors are float32 or uint16 (bf16 bits), got {a.dtype}")


def _c(a, dtype=None) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if dtype is not None and a.dtype != dtype:
        a = a.astype(dtype)
    return a


def num_threads() -> int:
    return int(_L().orc_num_threads())


def gate(logits: np.ndarray, K: int):
    """Eq. 2. Returns (ids [T,K] int32, w [T,K] float32, w64 [T,K] float64)."""
    logits = _c(logits, np.float32)
    T, N = logits.shape
    ids = np.empty((T, K), np.int32)
    w = np.empty((T, K), np.float32)
    w64 = np.empty((T, K), np.float64)
    rc = _L().orc_gate(_p(logits), C.c_int64(T), N, K, _p(ids), _p(w), _p(w64))
    assert rc == 0, rc
    return ids, w, w64


def router_logits(x, wr):
    """Router scores r = W_r x that Eq. 2 ranks. Returns (float32 [T,N], float64 [T,N])."""
    x, wr = _c(x), _c(wr)
    assert x.dtype == wr.dtype
    T, d = x.shape
    N = wr.shape[0]
    assert wr.shape == (N, d)
    r32 = np.empty((T, N), np.float32)
    r64 = np.empty((T, N), np.float64)
    rc = _L().orc_router_logits(_p(x), _dt(x), C.c_int64(T), d, _p(wr), N, _p(r32), _p(r64))
    assert rc == 0, rc
    return r32, r64


def moe_apply(x, wg, wu, wd, ids, w, n_experts: int, n_shared: int = 0, tok_idx=None) -> np.ndarray:
    """y_i = sum_j w[i,j] E_{ids[i,j]}(x_i) (+ shared expert). Returns float32 [n_sel, d]."""
    x, wg, wu, wd = _c(x), _c(wg), _c(wu), _c(wd)
    ids = _c(ids, np.int32)
    w = _c(w, np.float32)
    T, d = x.shape
    I = wg.shape[1]
    Kr = ids.shape[1]
    assert wg.shape[0] == n_experts + n_shared and wd.shape == (wg.shape[0], d, I)
    if tok_idx is None:
        n_sel, ti = T, None
    else:
        ti = _c(tok_idx, np.int64)
        n_sel = ti.shape[0]
    y = np.empty((n_sel, d), np.float32)
    rc = _L().orc_moe_apply(_p(x), _dt(x), C.c_int64(n_sel), _p(ti), d, I, n_experts, n_shared,
                            _p(wg), _p(wu), _p(wd), Kr, _p(ids), _p(w), _p(y))
    assert rc == 0, rc
    return y


def expert_outputs(x, wg, wu, wd, ids) -> np.ndarray:
    """Unweighted outputs of every routed expert: float64 [m, K, d]."""
    x, wg, wu, wd = _c(x), _c(wg), _c(wu), _c(wd)
    ids = _c(ids, np.int32)
    m, d = x.shape
    I = wg.shape[1]
    K = ids.shape[1]
    out = np.empty((m, K, d), np.float64)
    rc = _L().orc_expert_outputs(_p(x), _dt(x), C.c_int64(m), d, I, _p(wg), _p(wu), _p(wd), K,
                                 _p(ids), _p(out))
    assert rc == 0, rc
    return out


def calibrate(x, logits, wg, wu, wd, n_experts: int, K: int, lam: float = 1e-3, clip_lo: float = -4.0,
              clip_hi: float = 4.0, eps: float = 1e-12, mode: int = 0):
    """Eq. 6-9. Returns dict(S, L, h, lnh, n_obs, stats=(A,B,C), unobserved)."""
    x, wg, wu, wd = _c(x), _c(wg), _c(wu), _c(wd)
    logits = _c(logits, np.float32)
    m, d = x.shape
    I = wg.shape[1]
    N = n_experts
    S = np.empty((N, N), np.float32)
    L = np.empty((N, N), np.float32)
    h = np.empty(N, np.float32)
    lnh = np.empty(N, np.float32)
    n_obs = np.empty((N, N), np.int32)
    stats = np.empty((3, N, N), np.float64)
    rc = _L().orc_calibrate(_p(x), _dt(x), C.c_int64(m), d, I, N, K, _p(wg), _p(wu), _p(wd),
                            _p(logits), C.c_double(lam), C.c_double(clip_lo), C.c_double(clip_hi),
                            C.c_double(eps), mode, _p(S), _p(L), _p(h), _p(lnh), _p(n_obs), _p(stats))
    assert rc >= 0, rc
    return dict(S=S, L=L, h=h, lnh=lnh, n_obs=n_obs, stats=stats, unobserved=rc)


def prefill_fold(logits, K: int, Kp: int, S, L, h, lnh):
    """Eq. 10, 12, 13. Returns dict(ids [T,K'], w [T,K'], omit_src, omit_tgt [T,K-K'], mismatch)."""
    logits = _c(logits, np.float32)
    S, L, h, lnh = _c(S, np.float32), _c(L, np.float32), _c(h, np.float32), _c(lnh, np.float32)
    T, N = logits.shape
    ids = np.empty((T, Kp), np.int32)
    w = np.empty((T, Kp), np.float32)
    osrc = np.empty((T, K - Kp), np.int32)
    otgt = np.empty((T, K - Kp), np.int32)
    mism = np.zeros(1, np.int64)
    rc = _L().orc_prefill_fold(_p(logits), C.c_int64(T), N, K, Kp, _p(S), _p(L), _p(h), _p(lnh),
                               _p(ids), _p(w), _p(osrc), _p(otgt), _p(mism))
    assert rc == 0, rc
    return dict(ids=ids, w=w, omit_src=osrc, omit_tgt=otgt, mismatch=int(mism[0]))


def prefill_eq4(x, logits, wg, wu, wd, n_experts, n_shared, K, Kp, S, L, lnh) -> np.ndarray:
    """Eq. 4 written out (every term evaluates its expert). float32 [T, d]."""
    x, wg, wu, wd = _c(x), _c(wg), _c(wu), _c(wd)
    logits = _c(logits, np.float32)
    S, L, lnh = _c(S, np.float32), _c(L, np.float32), _c(lnh, np.float32)
    T, d = x.shape
    I = wg.shape[1]
    y = np.empty((T, d), np.float32)
    rc = _L().orc_prefill_eq4(_p(x), _dt(x), C.c_int64(T), d, I, n_experts, n_shared, _p(wg), _p(wu),
                              _p(wd), _p(logits), K, Kp, _p(S), _p(L), _p(lnh), _p(y))
    assert rc == 0, rc
    return y


def decode_fold(logits, K: int, M: int, S, L, h):
    """Eq. 11, 12, 14. Returns dict(pool_ids [M] (-1 padded), pool_size, pool_mask, ids, w [B,K],
    target [N], scale [N], score [N] float64, min_gap)."""
    logits = _c(logits, np.float32)
    S, L, h = _c(S, np.float32), _c(L, np.float32), _c(h, np.float32)
    B, N = logits.shape
    pool_ids = np.empty(M, np.int32)
    pool_size = np.zeros(1, np.int32)
    pool_mask = np.zeros((N + 31) // 32, np.uint32)
    ids = np.empty((B, K), np.int32)
    w = np.empty((B, K), np.float32)
    target = np.empty(N, np.int32)
    scale = np.empty(N, np.float32)
    score = np.empty(N, np.float64)
    gap = np.zeros(1, np.float64)
    rc = _L().orc_decode_fold(_p(logits), C.c_int64(B), N, K, M, _p(S), _p(L), _p(h), _p(pool_ids),
                              _p(pool_size), _p(pool_mask), _p(ids), _p(w), _p(target), _p(scale),
                              _p(score), _p(gap))
    assert rc == 0, rc
    return dict(pool_ids=pool_ids, pool_size=int(pool_size[0]), pool_mask=pool_mask, ids=ids, w=w,
                target=target, scale=scale, score=score, min_gap=float(gap[0]))


def decode_eq4(x, logits, wg, wu, wd, n_experts, n_shared, K, pool, S, L) -> np.ndarray:
    """Eq. 4 written out for a given decode pool. float32 [B, d]."""
    x, wg, wu, wd = _c(x), _c(wg), _c(wu), _c(wd)
    logits = _c(logits, np.float32)
    S, L = _c(S, np.float32), _c(L, np.float32)
    pool = _c(pool, np.int32)
    B, d = x.shape
    I = wg.shape[1]
    y = np.empty((B, d), np.float32)
    rc = _L().orc_decode_eq4(_p(x), _dt(x), C.c_int64(B), d, I, n_experts, n_shared, _p(wg), _p(wu),
                             _p(wd), _p(logits), K, _p(pool), int(pool.shape[0]), _p(S), _p(L), _p(y))
    assert rc == 0, rc
    return y


def sort_routes(ids, n_groups: int):
    """Expert-sorted permutation. Returns (perm [R] int32, offsets [G+1] int32)."""
    flat = _c(ids, np.int32).reshape(-1)
    R = flat.shape[0]
    perm = np.empty(R, np.int32)
    offsets = np.empty(n_groups + 1, np.int32)
    rc = _L().orc_sort_routes(_p(flat), C.c_int64(R), n_groups, _p(perm), _p(offsets))
    assert rc == 0, rc
    return perm, offsets


def static_pool(M: int, S, L, h):
    """Static decode pool from the calibration norms. Returns dict(pool_ids [M], target [N], scale [N])."""
    S, L, h = _c(S, np.float32), _c(L, np.float32), _c(h, np.float32)
    N = h.shape[0]
    pool_ids = np.empty(M, np.int32)
    target = np.empty(N, np.int32)
    scale = np.empty(N, np.float32)
    rc = _L().orc_static_pool(N, M, _p(S), _p(L), _p(h), _p(pool_ids), _p(target), _p(scale))
    assert rc == 0, rc
    return dict(pool_ids=pool_ids, target=target, scale=scale)


def decode_static(logits, K: int, target, scale):
    """Per-route remap with precomputed target/scale tables. Returns dict(ids [B,K], w [B,K])."""
    logits = _c(logits, np.float32)
    target, scale = _c(target, np.int32), _c(scale, np.float32)
    B, N = logits.shape
    ids = np.empty((B, K), np.int32)
    w = np.empty((B, K), np.float32)
    rc = _L().orc_decode_static(_p(logits), C.c_int64(B), N, K, _p(target), _p(scale), _p(ids), _p(w))
    assert rc == 0, rc
    return dict(ids=ids, w=w)


def prefill_fold_safe(logits, K: int, Kp: int, S, L, lnh, loss_thr: float = float("inf"), rescale: bool = False,
                      confidence: bool = False):
    """Prefill folding with the loss-threshold / rescale / confidence-split safeguards.
    Returns dict(ids, w, omit_src, omit_tgt); omit_tgt is -1 for a dropped route."""
    logits = _c(logits, np.float32)
    S, L, lnh = _c(S, np.float32), _c(L, np.float32), _c(lnh, np.float32)
    T, N = logits.shape
    ids = np.empty((T, Kp), np.int32)
    w = np.empty((T, Kp), np.float32)
    osrc = np.empty((T, K - Kp), np.int32)
    otgt = np.empty((T, K - Kp), np.int32)
    rc = _L().orc_prefill_fold_safe(_p(logits), C.c_int64(T), N, K, Kp, _p(S), _p(L), _p(lnh), C.c_double(loss_thr),
                                    int(rescale), int(confidence), _p(ids), _p(w), _p(osrc), _p(otgt))
    assert rc == 0, rc
    return dict(ids=ids, w=w, omit_src=osrc, omit_tgt=otgt)
