"""ctypes binding of libfc.so: argument marshalling only (pointers, sizes, strides, the stream)."""
from __future__ import annotations

import ctypes as C
import os
import re

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
# FC_LIB=debug selects the bounds-checking build (libfc_debug.so, see build.py); anything else the normal library
_LIB_PATH = os.path.join(_PKG, "libfc_debug.so" if os.environ.get("FC_LIB") == "debug" else "libfc.so")
_HEADER = os.path.join(_ROOT, "include", "fc.h")

BF16, F32 = 0, 1
POLICY_CHUNKWISE, POLICY_UNIFORM = 0, 1
RED_MEANKEY, RED_TILED, RED_TILED_MAX = 0, 1, 2
STATUS_BITS = {"timeout": 1, "nan_score": 2, "bad_index": 4}


class FcError(RuntimeError):
    pass


class _AttnDesc(C.Structure):
    _fields_ = [("H_q", C.c_int32), ("H_kv", C.c_int32), ("d", C.c_int32), ("W", C.c_int32),
                ("q_hs", C.c_int64), ("q_rs", C.c_int64), ("k_hs", C.c_int64), ("k_rs", C.c_int64),
                ("v_hs", C.c_int64), ("v_rs", C.c_int64), ("o_hs", C.c_int64), ("o_rs", C.c_int64),
                ("kv_rows", C.c_int64), ("scale", C.c_float), ("impl", C.c_int32)]


class _ScoreDesc(C.Structure):
    _fields_ = [("H_q", C.c_int32), ("H_kv", C.c_int32), ("d", C.c_int32), ("L_q", C.c_int32),
                ("L_k", C.c_int32), ("q_hs", C.c_int64), ("q_rs", C.c_int64), ("k_hs", C.c_int64),
                ("k_rs", C.c_int64), ("scale", C.c_float), ("lambda_", C.c_float),
                ("pool_k", C.c_int32), ("impl", C.c_int32), ("red_mode", C.c_int32)]


class _SelectOpts(C.Structure):
    _fields_ = [("unit", C.c_int32), ("n_protect", C.c_int32)]


class _CompactStrides(C.Structure):
    _fields_ = [("src_hs", C.c_int64), ("src_rs", C.c_int64), ("dst_hs", C.c_int64), ("dst_rs", C.c_int64)]


_lib = None


def lib_path() -> str:
    return _LIB_PATH


def lib():
    """Load libfc.so.  There is no fallback: a missing library is an error."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise FcError(f"{_LIB_PATH} is missing: build it with `python -m paper_2602_10825_b200.build` "
                          "(or __graft_entry__.build()); this package has no CPU or PyTorch fallback")
        L = C.CDLL(_LIB_PATH)
        L.fc_status_string.restype = C.c_char_p
        L.fc_last_cuda_error.restype = C.c_char_p
        for name in ("fc_chunk_decide_static_max_bytes", "fc_chunk_decide_workspace_bytes", "fc_chunk_attention_workspace_bytes",
                     "fc_kv_score_workspace_bytes", "fc_kv_select_compact_workspace_bytes",
                     "fc_kv_select_compact_ex_workspace_bytes"):
            getattr(L, name).restype = C.c_size_t
        L.fc_chunk_decide_workspace_bytes.argtypes = [C.c_int64, C.c_int]
        _lib = L
    return _lib


def declared_symbols():
    """Names of the functions include/fc.h declares."""
    text = open(_HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fc_[a-z_0-9]+)\s*\(", text)))


def exported_symbols():
    """Subset of the declared names that libfc.so actually exports."""
    L = lib()
    return sorted(n for n in declared_symbols() if hasattr(L, n))


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise FcError(f"unsupported tensor dtype {t.dtype}")


def _dev(t, name, dtype=None):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda):
        raise FcError(f"{name} must be a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise FcError(f"{name} must have dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _hsr(t, name):
    """(head stride, row stride) in elements of a [heads, rows, d] tensor with contiguous d."""
    if t.dim() != 3 or t.stride(2) != 1:
        raise FcError(f"{name} must be [heads, rows, d] with a contiguous last dimension")
    return int(t.stride(0)), int(t.stride(1))


def _host_i32(x):
    a = np.ascontiguousarray(np.asarray(x, dtype=np.int32))
    return a, a.ctypes.data_as(C.c_void_p)


class Context:
    """A libfc context on one CUDA device (fc_create / fc_destroy)."""

    def __init__(self, device: int = 0):
        self._h = C.c_void_p()
        self._L = lib()
        self.device = int(device)
        rc = self._L.fc_create(C.byref(self._h), self.device)
        self._check(rc, "fc_create")
        self._ws = {}

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            self._L.fc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def sm_count(self) -> int:
        return int(self._L.fc_sm_count(self._h))

    def _check(self, rc, what):
        if rc != 0:
            msg = self._L.fc_status_string(rc).decode()
            if rc == -6:
                msg += ": " + self._L.fc_last_cuda_error().decode()
            raise FcError(f"{what} failed ({rc}): {msg}")

    def _stream(self):
        return C.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)

    def workspace(self, key, n_bytes):
        """A cached device scratch buffer (the binding's convenience; the C call never allocates)."""
        n_bytes = max(int(n_bytes), 256)
        buf = self._ws.get(key)
        if buf is None or buf.numel() < n_bytes:
            buf = torch.empty(n_bytes, dtype=torch.uint8, device=f"cuda:{self.device}")
            self._ws[key] = buf
        return buf

    # ------------------------------------------------------------------ fc_selftest_bounded_wait
    def selftest_bounded_wait(self, limit_ns, status, waited_ns=None):
        rc = self._L.fc_selftest_bounded_wait(self._h, self._stream(), C.c_uint64(int(limit_ns)),
                                              _dev(status, "status", torch.int32), _dev(waited_ns, "waited_ns", torch.int32))
        self._check(rc, "fc_selftest_bounded_wait")

    # ------------------------------------------------------------------ fc_chunk_decide
    def chunk_decide(self, cur, prev, chunk_elem_off, chunk_step, warmup_m, eps, acc, *, force=None,
                     policy=POLICY_CHUNKWISE, l1rel=None, recompute=None, active_ids=None, n_active=None, status=None, ws=None):
        off = np.ascontiguousarray(np.asarray(chunk_elem_off, dtype=np.int64))
        n = len(off) - 1
        dev = cur.device
        l1rel = torch.empty(n, dtype=torch.float32, device=dev) if l1rel is None else l1rel
        recompute = torch.empty(n, dtype=torch.uint8, device=dev) if recompute is None else recompute
        active_ids = torch.empty(n, dtype=torch.int32, device=dev) if active_ids is None else active_ids
        n_active = torch.empty(1, dtype=torch.int32, device=dev) if n_active is None else n_active
        need = self._L.fc_chunk_decide_workspace_bytes(C.c_int64(int(off[-1])), n)
        ws = self.workspace("decide", need) if ws is None else ws
        rc = self._L.fc_chunk_decide(
            self._h, self._stream(), _dev(cur, "cur"), _dev(prev, "prev"), _dt(cur),
            off.ctypes.data_as(C.c_void_p), n, _dev(chunk_step, "chunk_step", torch.int32), int(warmup_m),
            C.c_float(eps), _dev(force, "force", torch.uint8), int(policy), _dev(acc, "acc", torch.float32),
            _dev(l1rel, "l1rel", torch.float32), _dev(recompute, "recompute", torch.uint8),
            _dev(active_ids, "active_ids", torch.int32), _dev(n_active, "n_active", torch.int32),
            _dev(status, "status", torch.int32), _dev(ws, "ws"), C.c_size_t(ws.numel()))
        self._check(rc, "fc_chunk_decide")
        return dict(l1rel=l1rel, recompute=recompute, active_ids=active_ids, n_active=n_active, acc=acc)

    def chunk_decide_static(self, cur, prev, chunk_elem_off, chunk_step, warmup_m, eps, acc, *, l1rel, recompute,
                            active_ids, n_active, force=None, policy=POLICY_CHUNKWISE, status=None):
        """fc_chunk_decide_static: the decision without a workspace, for callers that cannot allocate device
        memory (the scratch is a fixed 1 MiB array inside the library).  Every output tensor is passed in, so
        this wrapper allocates nothing on the device either."""
        off = np.ascontiguousarray(np.asarray(chunk_elem_off, dtype=np.int64))
        n = len(off) - 1
        rc = self._L.fc_chunk_decide_static(
            self._h, self._stream(), _dev(cur, "cur"), _dev(prev, "prev"), _dt(cur),
            off.ctypes.data_as(C.c_void_p), n, _dev(chunk_step, "chunk_step", torch.int32), int(warmup_m),
            C.c_float(eps), _dev(force, "force", torch.uint8), int(policy), _dev(acc, "acc", torch.float32),
            _dev(l1rel, "l1rel", torch.float32), _dev(recompute, "recompute", torch.uint8),
            _dev(active_ids, "active_ids", torch.int32), _dev(n_active, "n_active", torch.int32),
            _dev(status, "status", torch.int32))
        self._check(rc, "fc_chunk_decide_static")
        return dict(l1rel=l1rel, recompute=recompute, active_ids=active_ids, n_active=n_active, acc=acc)

    # ------------------------------------------------------------------ fc_chunk_cache_apply
    def chunk_cache_apply(self, x_in, y_io, cache, chunk_elem_off, recompute, *, status=None):
        off = np.ascontiguousarray(np.asarray(chunk_elem_off, dtype=np.int64))
        if not (x_in.dtype == y_io.dtype == cache.dtype):
            raise FcError("x_in, y_io and cache must share one dtype")
        for name, t in (("x_in", x_in), ("y_io", y_io), ("cache", cache)):
            if not t.is_contiguous() or t.numel() < int(off[-1]):
                raise FcError(f"{name} must be contiguous and hold every chunk's elements")
        rc = self._L.fc_chunk_cache_apply(
            self._h, self._stream(), _dev(x_in, "x_in"), _dev(y_io, "y_io"), _dev(cache, "cache"), _dt(x_in),
            off.ctypes.data_as(C.c_void_p), len(off) - 1, _dev(recompute, "recompute", torch.uint8),
            _dev(status, "status", torch.int32))
        self._check(rc, "fc_chunk_cache_apply")
        return y_io, cache

    # ------------------------------------------------------------------ fc_chunk_attention
    def chunk_attention(self, Q, K, V, q_chunk_row_off, kv_visible_len, seg_logical_off, seg_phys_off,
                        active_ids, n_active, O, *, lse=None, kv_token_index=None, scale=0.0, impl=0,
                        status=None, ws=None):
        q_hs, q_rs = _hsr(Q, "Q")
        k_hs, k_rs = _hsr(K, "K")
        v_hs, v_rs = _hsr(V, "V")
        o_hs, o_rs = _hsr(O, "O")
        W = len(q_chunk_row_off) - 1
        desc = _AttnDesc(Q.shape[0], K.shape[0], Q.shape[2], W, q_hs, q_rs, k_hs, k_rs, v_hs, v_rs, o_hs, o_rs,
                         K.shape[1], scale, impl)
        qo, qo_p = _host_i32(q_chunk_row_off)
        vis, vis_p = _host_i32(kv_visible_len)
        if seg_phys_off is not None:
            sl, sl_p = _host_i32(seg_logical_off)
            sp, sp_p = _host_i32(seg_phys_off)
            n_seg = len(sp)
        else:
            sl_p = sp_p = None
            n_seg = 0
        tok_hs = 0
        if kv_token_index is not None:
            if kv_token_index.dim() != 2 or kv_token_index.stride(1) != 1:
                raise FcError("kv_token_index must be [H_kv, L_logical] with contiguous rows")
            tok_hs = int(kv_token_index.stride(0))
        lse_hs = 0 if lse is None else int(lse.stride(0))
        need = self._L.fc_chunk_attention_workspace_bytes(C.byref(desc))
        ws = self.workspace("attention", need) if ws is None else ws
        if O.dtype != Q.dtype or K.dtype != Q.dtype or V.dtype != Q.dtype:
            raise FcError("Q, K, V, O must share one dtype")
        rc = self._L.fc_chunk_attention(
            self._h, self._stream(), C.byref(desc), _dev(Q, "Q"), _dev(K, "K"), _dev(V, "V"), _dt(Q), qo_p,
            vis_p, sl_p, sp_p, n_seg, _dev(kv_token_index, "kv_token_index", torch.int32), C.c_int64(tok_hs),
            _dev(active_ids, "active_ids", torch.int32), _dev(n_active, "n_active", torch.int32), _dev(O, "O"),
            _dev(lse, "lse", torch.float32), C.c_int64(lse_hs), _dev(status, "status", torch.int32),
            _dev(ws, "ws"), C.c_size_t(ws.numel()))
        self._check(rc, "fc_chunk_attention")
        return O

    # ------------------------------------------------------------------ fc_kv_score
    def kv_score(self, Q_obs, K_cand, *, lambda_=0.07, pool_k=7, scale=0.0, imp_accum=None, accum_phase=0,
                 n_steps=1, imp=None, red=None, score=None, impl=0, red_mode=RED_MEANKEY, status=None, ws=None):
        q_hs, q_rs = _hsr(Q_obs, "Q_obs")
        k_hs, k_rs = _hsr(K_cand, "K_cand")
        H_kv, L_k, d = K_cand.shape
        desc = _ScoreDesc(Q_obs.shape[0], H_kv, d, Q_obs.shape[1], L_k, q_hs, q_rs, k_hs, k_rs, scale, lambda_,
                          pool_k, impl, red_mode)
        if score is None and accum_phase != 1:
            score = torch.empty((H_kv, L_k), dtype=torch.float32, device=K_cand.device)
        for name, t in (("imp", imp), ("red", red), ("score", score), ("imp_accum", imp_accum)):
            if t is not None and not (t.is_contiguous() and tuple(t.shape) == (H_kv, L_k)):
                raise FcError(f"{name} must be a contiguous [H_kv, L_k] tensor")
        need = self._L.fc_kv_score_workspace_bytes(C.byref(desc))
        ws = self.workspace("score", need) if ws is None else ws
        rc = self._L.fc_kv_score(
            self._h, self._stream(), C.byref(desc), _dev(Q_obs, "Q_obs"), _dev(K_cand, "K_cand"), _dt(K_cand),
            _dev(imp_accum, "imp_accum", torch.float32), int(accum_phase), int(n_steps),
            _dev(imp, "imp", torch.float32), _dev(red, "red", torch.float32), _dev(score, "score", torch.float32),
            _dev(status, "status", torch.int32), _dev(ws, "ws"), C.c_size_t(ws.numel()))
        self._check(rc, "fc_kv_score")
        return dict(imp=imp, red=red, score=score)

    # ------------------------------------------------------------------ fc_kv_select_compact
    def kv_select_compact(self, score, B, K_src=None, V_src=None, K_dst=None, V_dst=None, *, kept_idx=None,
                          n_kept=None, status=None, ws=None, unit=1, n_protect=0):
        """fc_kv_select_compact, or fc_kv_select_compact_ex when a selection unit or a protected tail is given."""
        H, L_k = score.shape
        if not score.is_contiguous():
            raise FcError("score must be contiguous [n_heads, L_k]")
        n_keep = min(int(B), L_k)
        dev = score.device
        kept_idx = torch.empty((H, n_keep), dtype=torch.int32, device=dev) if kept_idx is None else kept_idx
        n_kept = torch.empty(1, dtype=torch.int32, device=dev) if n_kept is None else n_kept
        strides, dtype, d = None, BF16, 0
        if K_src is not None:
            s_hs, s_rs = _hsr(K_src, "K_src")
            if _hsr(V_src, "V_src") != (s_hs, s_rs):
                raise FcError("K_src and V_src must share strides")
            if K_dst is None:
                K_dst = torch.empty((H, n_keep, K_src.shape[2]), dtype=K_src.dtype, device=dev)
                V_dst = torch.empty_like(K_dst)
            d_hs, d_rs = _hsr(K_dst, "K_dst")
            if _hsr(V_dst, "V_dst") != (d_hs, d_rs):
                raise FcError("K_dst and V_dst must share strides")
            strides = _CompactStrides(s_hs, s_rs, d_hs, d_rs)
            dtype, d = _dt(K_src), K_src.shape[2]
        if unit != 1 or n_protect != 0:
            need = self._L.fc_kv_select_compact_ex_workspace_bytes(H, L_k, int(unit))
            ws = self.workspace("select", need) if ws is None else ws
            opts = _SelectOpts(int(unit), int(n_protect))
            rc = self._L.fc_kv_select_compact_ex(
                self._h, self._stream(), _dev(score, "score", torch.float32), H, L_k, int(B), C.byref(opts),
                _dev(K_src, "K_src"), _dev(V_src, "V_src"), _dev(K_dst, "K_dst"), _dev(V_dst, "V_dst"), dtype, d,
                None if strides is None else C.byref(strides), _dev(kept_idx, "kept_idx", torch.int32),
                _dev(n_kept, "n_kept", torch.int32), _dev(status, "status", torch.int32), _dev(ws, "ws"),
                C.c_size_t(ws.numel()))
            self._check(rc, "fc_kv_select_compact_ex")
            return dict(kept_idx=kept_idx, n_kept=n_kept, K_dst=K_dst, V_dst=V_dst)
        need = self._L.fc_kv_select_compact_workspace_bytes(H, L_k)
        ws = self.workspace("select", need) if ws is None else ws
        rc = self._L.fc_kv_select_compact(
            self._h, self._stream(), _dev(score, "score", torch.float32), H, L_k, int(B), _dev(K_src, "K_src"),
            _dev(V_src, "V_src"), _dev(K_dst, "K_dst"), _dev(V_dst, "V_dst"), dtype, d,
            None if strides is None else C.byref(strides), _dev(kept_idx, "kept_idx", torch.int32),
            _dev(n_kept, "n_kept", torch.int32), _dev(status, "status", torch.int32), _dev(ws, "ws"),
            C.c_size_t(ws.numel()))
        self._check(rc, "fc_kv_select_compact")
        return dict(kept_idx=kept_idx, n_kept=n_kept, K_dst=K_dst, V_dst=V_dst)
