"""FlowCache hot-path ORACLE (test infrastructure, not product code).

ctypes front end of ``libfc_oracle.so`` — the plain fp64 CPU statement of the
paper's definitions in ``fc_oracle.cpp``.  Only the tests, the smoke check and
the benchmark's CPU-baseline leg may import this package; the CUDA library
never does, and this package never imports the CUDA library.

Arrays are numpy; bf16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libfc_oracle.so")
_SRC = os.path.join(_HERE, "fc_oracle.cpp")

BF16, F32 = 0, 1
RED_AUTO, RED_PLAIN, RED_MEANKEY, RED_MAXSIM = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved)."""
    stale = (not os.path.exists(_SO)) or any(
        os.path.getmtime(os.path.join(_HERE, f)) > os.path.getmtime(_SO)
        for f in ("fc_oracle.cpp", "fc_oracle.h"))
    if force or stale:
        subprocess.check_call(
            ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread",
             "-o", _SO, _SRC])
    return _SO


class _AttnDesc(C.Structure):
    _fields_ = [("H_q", C.c_int32), ("H_kv", C.c_int32), ("d", C.c_int32),
                ("W", C.c_int32), ("q_hs", C.c_int64), ("q_rs", C.c_int64),
                ("k_hs", C.c_int64), ("k_rs", C.c_int64), ("v_hs", C.c_int64),
                ("v_rs", C.c_int64), ("scale", C.c_double)]


class _ScoreDesc(C.Structure):
    _fields_ = [("H_q", C.c_int32), ("H_kv", C.c_int32), ("d", C.c_int32),
                ("L_q", C.c_int32), ("L_k", C.c_int32), ("q_hs", C.c_int64),
                ("q_rs", C.c_int64), ("k_hs", C.c_int64), ("k_rs", C.c_int64),
                ("scale", C.c_double), ("lambda_", C.c_double),
                ("pool_k", C.c_int32), ("red_mode", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.fco_hardware_threads.restype = C.c_int
    return _lib


def hardware_threads() -> int:
    return int(lib().fco_hardware_threads())


def _ptr(a):
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.flags["C_CONTIGUOUS"], "need a C-contiguous numpy array"
    return a.ctypes.data_as(C.c_void_p)


def _dtype_of(a: np.ndarray) -> int:
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float32:
        return F32
    raise TypeError(f"oracle takes uint16 (bf16 bits) or float32, got {a.dtype}")


def _i32(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


def chunk_decide(cur, prev, chunk_elem_off, chunk_step, warmup_m, eps, acc,
                 force=None, n_threads=0):
    """Eqs. 5 and 8.  Returns dict(l1rel, recompute, acc, active_ids, n_active);
    ``acc`` is the accumulator AFTER the step (the input array is not modified)."""
    off = np.ascontiguousarray(np.asarray(chunk_elem_off, dtype=np.int64))
    n = len(off) - 1
    step = _i32(chunk_step)
    acc_out = np.array(acc, dtype=np.float32, copy=True)
    l1rel = np.zeros(n, np.float32)
    rec = np.zeros(n, np.uint8)
    ids = np.full(n, -1, np.int32)
    cnt = np.zeros(1, np.int32)
    frc = None if force is None else np.ascontiguousarray(np.asarray(force, dtype=np.uint8))
    rc = lib().fco_chunk_decide(_ptr(cur), _ptr(prev), _dtype_of(cur), _ptr(off), n,
                                _ptr(step), int(warmup_m), C.c_float(eps), _ptr(frc),
                                _ptr(acc_out), _ptr(l1rel), _ptr(rec), _ptr(ids),
                                _ptr(cnt), int(n_threads))
    if rc:
        raise ValueError(f"fco_chunk_decide -> {rc}")
    return dict(l1rel=l1rel, recompute=rec, acc=acc_out, active_ids=ids[:cnt[0]].copy(),
                n_active=int(cnt[0]))


def chunk_decide_uniform(cur, prev, chunk_elem_off, chunk_step, warmup_m, eps, acc,
                         force=None, n_threads=0):
    """The uniform policy of the caption of Fig. 3 (one shared decision; forced and warm-up chunks
    are computed anyway).  Same returns as chunk_decide."""
    off = np.ascontiguousarray(np.asarray(chunk_elem_off, dtype=np.int64))
    n = len(off) - 1
    step = _i32(chunk_step)
    acc_out = np.array(acc, dtype=np.float32, copy=True)
    l1rel = np.zeros(n, np.float32)
    rec = np.zeros(n, np.uint8)
    ids = np.full(n, -1, np.int32)
    cnt = np.zeros(1, np.int32)
    frc = None if force is None else np.ascontiguousarray(np.asarray(force, dtype=np.uint8))
    rc = lib().fco_chunk_decide_uniform(_ptr(cur), _ptr(prev), _dtype_of(cur), _ptr(off), n,
                                        _ptr(step), int(warmup_m), C.c_float(eps), _ptr(frc),
                                        _ptr(acc_out), _ptr(l1rel), _ptr(rec), _ptr(ids),
                                        _ptr(cnt), int(n_threads))
    if rc:
        raise ValueError(f"fco_chunk_decide_uniform -> {rc}")
    return dict(l1rel=l1rel, recompute=rec, acc=acc_out, active_ids=ids[:cnt[0]].copy(),
                n_active=int(cnt[0]))


def chunk_cache_apply(x_in, y, cache, chunk_elem_off, recompute, n_threads=0):
    """Activation-cache step (Sec. 3.2): computed chunks store y - x into the cache, skipped chunks
    get y = x + cache.  Returns new (y, cache) arrays; the inputs are not modified."""
    off = np.ascontiguousarray(np.asarray(chunk_elem_off, dtype=np.int64))
    n = len(off) - 1
    y_out = np.array(y, copy=True)
    c_out = np.array(cache, copy=True)
    rec = np.ascontiguousarray(np.asarray(recompute, dtype=np.uint8))
    assert x_in.dtype == y_out.dtype == c_out.dtype and len(rec) == n
    rc = lib().fco_chunk_cache_apply(_ptr(np.ascontiguousarray(x_in)), _ptr(y_out), _ptr(c_out),
                                     _dtype_of(y_out), _ptr(off), n, _ptr(rec), int(n_threads))
    if rc:
        raise ValueError(f"fco_chunk_cache_apply -> {rc}")
    return y_out, c_out


def chunk_attention(Q, K, V, q_chunk_row_off, kv_visible_len, seg_logical_off,
                    seg_phys_off, active_ids, *, H_kv=None, scale=0.0,
                    kv_token_index=None, sample_rows=None, O_init=None, n_threads=0):
    """Chunk-causal attention (Sec. 3.3).  Q [H_q, R, d]; K, V [H_kv, L_phys, d].
    Returns (O float64, lse float64): full [H_q, R, d] / [H_q, R] (starting from
    ``O_init`` or zeros; inactive rows untouched), or packed over ``sample_rows``."""
    H_q, R, d = Q.shape
    H_kv = H_kv or K.shape[0]
    W = len(q_chunk_row_off) - 1
    desc = _AttnDesc(H_q, H_kv, d, W, R * d, d, K.shape[1] * d, d, V.shape[1] * d, d, scale)
    qoff, vis = _i32(q_chunk_row_off), _i32(kv_visible_len)
    slo = None if seg_logical_off is None else _i32(seg_logical_off)
    spo = None if seg_phys_off is None else _i32(seg_phys_off)
    n_seg = 0 if spo is None else len(spo)
    act = _i32(active_ids)
    tok = None if kv_token_index is None else _i32(kv_token_index)
    tok_hs = 0 if tok is None else tok.shape[1]
    if sample_rows is None:
        O = np.zeros((H_q, R, d), np.float64) if O_init is None else np.array(O_init, np.float64, copy=True)
        lse = np.full((H_q, R), np.nan, np.float64)
        smp, n_smp = None, 0
    else:
        smp = _i32(sample_rows)
        n_smp = len(smp)
        O = np.zeros((H_q, n_smp, d), np.float64)
        lse = np.full((H_q, n_smp), np.nan, np.float64)
    rc = lib().fco_chunk_attention(C.byref(desc), _ptr(Q), _ptr(K), _ptr(V), _dtype_of(Q),
                                   _ptr(qoff), _ptr(vis), _ptr(slo), _ptr(spo), n_seg,
                                   _ptr(tok), C.c_int64(tok_hs), _ptr(act), len(act),
                                   _ptr(smp), n_smp, _ptr(O), C.c_int64(R * d), C.c_int64(d),
                                   _ptr(lse), int(n_threads))
    if rc:
        raise ValueError(f"fco_chunk_attention -> {rc}")
    return O, lse


def kv_score(Q_obs, K_cand, *, lambda_=0.07, pool_k=7, red_mode=RED_AUTO, scale=0.0,
             imp_accum=None, accum_phase=0, n_steps=1, n_threads=0):
    """Eqs. 9-12.  Q_obs [H_q, L_q, d], K_cand [H_kv, L_k, d].  Returns dict(imp,
    imp_pooled, red (float64), score (float32)); in phase 1 only imp_accum is updated."""
    H_q, L_q, d = Q_obs.shape
    H_kv, L_k, _ = K_cand.shape
    desc = _ScoreDesc(H_q, H_kv, d, L_q, L_k, L_q * d, d, L_k * d, d, scale, lambda_,
                      pool_k, red_mode)
    imp = np.zeros((H_kv, L_k), np.float64)
    pooled = np.zeros((H_kv, L_k), np.float64)
    red = np.zeros((H_kv, L_k), np.float64)
    score = np.zeros((H_kv, L_k), np.float32)
    if imp_accum is not None:
        assert imp_accum.dtype == np.float64 and imp_accum.shape == (H_kv, L_k)
    rc = lib().fco_kv_score(C.byref(desc), _ptr(Q_obs), _ptr(K_cand), _dtype_of(K_cand),
                            _ptr(imp_accum), int(accum_phase), int(n_steps), _ptr(imp),
                            _ptr(pooled), _ptr(red), _ptr(score), int(n_threads))
    if rc:
        raise ValueError(f"fco_kv_score -> {rc}")
    return dict(imp=imp, imp_pooled=pooled, red=red, score=score)


def key_similarity_columns(K_cand, cols, red_mode=RED_PLAIN, n_threads=0):
    """The softmax argument of Eq. 11 (column mean of the cosine matrix with zeroed diagonal; or, with
    RED_MAXSIM, the largest similarity to another token) for the columns ``cols`` only.  [H, len(cols)]."""
    H, L_k, d = K_cand.shape
    cols = _i32(cols)
    out = np.zeros((H, len(cols)), np.float64)
    rc = lib().fco_key_similarity_columns(_ptr(K_cand), _dtype_of(K_cand), H, L_k, d, C.c_int64(L_k * d),
                                          C.c_int64(d), _ptr(cols), len(cols), int(red_mode), _ptr(out),
                                          int(n_threads))
    if rc:
        raise ValueError(f"fco_key_similarity_columns -> {rc}")
    return out


def kv_select_compact(score, B, K_src=None, V_src=None, n_threads=0):
    """Top-B per head (score desc, index asc) and row retention.  score [H, L_k] f32;
    K_src, V_src [H, L_k, d] (any 2- or 4-byte dtype).  Returns dict(kept_idx
    [H, min(B, L_k)] ascending, n_kept, K_dst, V_dst)."""
    score = np.ascontiguousarray(score, dtype=np.float32)
    H, L_k = score.shape
    n_keep = min(B, L_k)
    kept = np.zeros((H, n_keep), np.int32)
    cnt = np.zeros(1, np.int32)
    K_dst = V_dst = None
    eb = d = 0
    if K_src is not None:
        d = K_src.shape[2]
        eb = K_src.dtype.itemsize
        K_dst = np.zeros((H, n_keep, d), K_src.dtype)
        V_dst = np.zeros((H, n_keep, d), V_src.dtype)
    rc = lib().fco_kv_select_compact(_ptr(score), H, L_k, int(B), _ptr(K_src), _ptr(V_src),
                                     _ptr(K_dst), _ptr(V_dst), eb, d, C.c_int64(L_k * d),
                                     C.c_int64(d), C.c_int64(n_keep * d), C.c_int64(d),
                                     _ptr(kept), _ptr(cnt), int(n_threads))
    if rc:
        raise ValueError(f"fco_kv_select_compact -> {rc}")
    return dict(kept_idx=kept, n_kept=int(cnt[0]), K_dst=K_dst, V_dst=V_dst)


def kv_select_units(score, B, unit=1, n_protect=0, n_threads=0):
    """Selection by units of ``unit`` consecutive tokens (unit score = mean of the tokens' scores) with the last
    ``n_protect`` tokens' units always kept.  Returns dict(kept_idx [H, min(B, L_k)] ascending, n_kept)."""
    score = np.ascontiguousarray(score, dtype=np.float32)
    H, L_k = score.shape
    n_keep = min(B, L_k)
    kept = np.zeros((H, n_keep), np.int32)
    cnt = np.zeros(1, np.int32)
    rc = lib().fco_kv_select_units(_ptr(score), H, L_k, int(B), int(unit), int(n_protect), _ptr(kept), _ptr(cnt),
                                   int(n_threads))
    if rc:
        raise ValueError(f"fco_kv_select_units -> {rc}")
    return dict(kept_idx=kept, n_kept=int(cnt[0]))

