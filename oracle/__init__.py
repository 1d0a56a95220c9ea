"""ctypes front end of the CPU oracle (oracle/hawk_oracle.c).

Test infrastructure only: tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; the CUDA binding never does.  bf16 tensors are numpy uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "hawk_oracle.c"
_LIB = _HERE / "libhawk_oracle.so"
_lock = threading.Lock()
_lib = None

FLAG_BAD_DRAFT = 2
FLAG_NONFINITE = 4


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (-O2, OpenMP across independent units, no fp contraction)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            _lib = ctypes.CDLL(str(build()))
            _lib.hawk_oracle_residual.restype = ctypes.c_double
            _lib.hawk_oracle_cfg_accept.restype = ctypes.c_int
            _lib.hawk_oracle_target_probs.restype = ctypes.c_int
            _lib.hawk_oracle_target_probs_rows.restype = ctypes.c_int
            _lib.hawk_oracle_tree_accept.restype = ctypes.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _gomp():
    return ctypes.CDLL("libgomp.so.1")


def threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS or the host's cores, unless set_threads() changed it)."""
    _load()
    return int(_gomp().omp_get_max_threads())


def set_threads(n: int) -> None:
    """Number of threads for the OpenMP loops from now on (timing only: results do not depend on it, every
    parallel loop runs over independent units)."""
    _load()
    _gomp().omp_set_num_threads(int(n))


def verify_attn(q, k_cache, v_cache, prefix_len, sm_scale) -> np.ndarray:
    """q [S,K,H,D], caches [S,H_kv,L_cap,D] (uint16 bf16 bits), prefix_len [S] -> fp64 [S,K,H*D]."""
    q = _c(q, np.uint16); k_cache = _c(k_cache, np.uint16); v_cache = _c(v_cache, np.uint16)
    prefix_len = _c(prefix_len, np.int32)
    S, K, H, D = q.shape
    _, H_kv, L_cap, _ = k_cache.shape
    out = np.empty((S, K, H * D), dtype=np.float64)
    _load().hawk_oracle_verify_attn(_p(q), _p(k_cache), _p(v_cache), _p(prefix_len), _p(out),
                                    S, K, H, H_kv, D, L_cap, ctypes.c_double(float(sm_scale)))
    return out


def verify_attn_tree(q, k_cache, v_cache, prefix_len, anc_mask, sm_scale) -> np.ndarray:
    """q [S,N,H,D], caches [S,H_kv,L_cap,D] (uint16 bf16 bits), prefix_len [S], anc_mask uint64 [N] (N <= 64)
    -> fp64 [S,N,H*D]; node i sees the prefix and the block rows whose bit is set in anc_mask[i]."""
    q = _c(q, np.uint16); k_cache = _c(k_cache, np.uint16); v_cache = _c(v_cache, np.uint16)
    prefix_len = _c(prefix_len, np.int32); anc_mask = _c(anc_mask, np.uint64)
    S, N, H, D = q.shape
    _, H_kv, L_cap, _ = k_cache.shape
    assert anc_mask.shape == (N,) and N <= 64
    out = np.empty((S, N, H * D), dtype=np.float64)
    _load().hawk_oracle_verify_attn_tree(_p(q), _p(k_cache), _p(v_cache), _p(prefix_len), _p(anc_mask), _p(out),
                                         S, N, H, H_kv, D, L_cap, ctypes.c_double(float(sm_scale)))
    return out


def head_proj(x, w, v_begin=0, v_end=None, fill=np.nan) -> np.ndarray:
    """x [M,hidden], w [V,hidden] (uint16 bf16 bits) -> fp32 [M,V]; columns outside the range = fill."""
    x = _c(x, np.uint16); w = _c(w, np.uint16)
    M, hidden = x.shape
    V = w.shape[0]
    v_end = V if v_end is None else v_end
    logits = np.full((M, V), fill, dtype=np.float32)
    _load().hawk_oracle_head_proj(_p(x), _p(w), _p(logits), M, hidden, V, v_begin, v_end)
    return logits


def head_proj_cfg(x, w, cfg_scale, temperature, v_begin=0, v_end=None, fill=np.nan) -> np.ndarray:
    """x [2B,rows,hidden], w [V,hidden] (uint16 bf16 bits) -> guided logits fp32 [B,rows,V]."""
    x = _c(x, np.uint16); w = _c(w, np.uint16)
    S, rows, hidden = x.shape
    assert S % 2 == 0
    B, V = S // 2, w.shape[0]
    v_end = V if v_end is None else v_end
    guided = np.full((B, rows, V), fill, dtype=np.float32)
    _load().hawk_oracle_head_proj_cfg(_p(x), _p(w), _p(guided), B, rows, hidden, V, v_begin, v_end,
                                      ctypes.c_float(cfg_scale), ctypes.c_float(temperature))
    return guided


def target_probs(lc, lu, v_begin, v_end, cfg_scale, temperature, top_k):
    """One position: fp32 rows lc, lu [V] -> (p fp64 [V], flags)."""
    lc = _c(lc, np.float32); lu = _c(lu, np.float32)
    V = lc.shape[0]
    p = np.empty(V, dtype=np.float64)
    flags = _load().hawk_oracle_target_probs(_p(lc), _p(lu), V, v_begin, v_end,
                                             ctypes.c_float(cfg_scale), ctypes.c_float(temperature),
                                             int(top_k), _p(p))
    return p, flags


def target_probs_rows(logits, v_begin, v_end, cfg_scale, temperature, top_k):
    """logits fp32 [2B,rows,V] -> (p fp64 [B,rows,V], flags)."""
    logits = _c(logits, np.float32)
    S, rows, V = logits.shape
    B = S // 2
    p = np.empty((B, rows, V), dtype=np.float64)
    flags = _load().hawk_oracle_target_probs_rows(_p(logits), B, rows, V, v_begin, v_end,
                                                  ctypes.c_float(cfg_scale),
                                                  ctypes.c_float(temperature), int(top_k), _p(p))
    return p, flags


def residual(p, q, v_begin, v_end):
    """p fp64 [V], q fp32 [V] -> (r fp64 [V] un-normalised, total mass)."""
    p = _c(p, np.float64); q = _c(q, np.float32)
    V = p.shape[0]
    r = np.empty(V, dtype=np.float64)
    total = _load().hawk_oracle_residual(_p(p), _p(q), V, v_begin, v_end, _p(r))
    return r, total


def cfg_accept(logits, q_probs, draft, u_accept, u_resample, v_begin, v_end, cfg_scale,
               temperature, top_k, has_bonus_row=False, diagnostics=True) -> dict:
    """Chain verification; see hawk_oracle_cfg_accept in the C source for the contract."""
    logits = _c(logits, np.float32); q_probs = _c(q_probs, np.float32)
    draft = _c(draft, np.int32); u_accept = _c(u_accept, np.float32)
    u_resample = _c(u_resample, np.float32)
    B, K, V = q_probs.shape
    rows = K + (1 if has_bonus_row else 0)
    assert logits.shape == (2 * B, rows, V), (logits.shape, (2 * B, rows, V))
    assert draft.shape == (B, K) and u_accept.shape == (B, K) and u_resample.shape == (B, K + 1)
    accept_len = np.empty(B, dtype=np.int32)
    token = np.empty(B, dtype=np.int32)
    ratio = np.empty((B, K), dtype=np.float64) if diagnostics else None
    acc_margin = np.empty((B, K), dtype=np.float64) if diagnostics else None
    res_margin = np.empty(B, dtype=np.float64) if diagnostics else None
    flags = _load().hawk_oracle_cfg_accept(
        _p(logits), _p(q_probs), _p(draft), _p(u_accept), _p(u_resample), B, K, V, v_begin, v_end,
        ctypes.c_float(cfg_scale), ctypes.c_float(temperature), int(top_k), int(bool(has_bonus_row)),
        _p(accept_len), _p(token), _p(ratio), _p(acc_margin), _p(res_margin))
    return dict(accept_len=accept_len, token=token, ratio=ratio, accept_margin=acc_margin,
                resample_margin=res_margin, flags=flags)


def tree_accept(logits, q_probs, node_token, node_q, child_begin, u_accept, u_resample, v_begin, v_end,
                cfg_scale, temperature, top_k, max_depth=None, diagnostics=True) -> dict:
    """Verification of a candidate tree; see hawk_oracle_tree_accept in the C source for the contract."""
    logits = _c(logits, np.float32); q_probs = _c(q_probs, np.float32)
    node_token = _c(node_token, np.int32); node_q = _c(node_q, np.int32)
    child_begin = _c(child_begin, np.int32)
    u_accept = _c(u_accept, np.float32); u_resample = _c(u_resample, np.float32)
    B, NQ, V = q_probs.shape
    N = node_q.shape[0]
    assert logits.shape == (2 * B, N, V), (logits.shape, (2 * B, N, V))
    assert node_token.shape == (B, N) and child_begin.shape == (N + 1,)
    assert u_accept.shape == (B, N) and u_resample.shape == (B, N)
    max_depth = N if max_depth is None else max_depth
    accept_len = np.empty(B, dtype=np.int32)
    token = np.empty(B, dtype=np.int32)
    path = np.empty((B, max_depth), dtype=np.int32)
    acc_margin = np.empty((B, N), dtype=np.float64) if diagnostics else None
    res_margin = np.empty(B, dtype=np.float64) if diagnostics else None
    flags = _load().hawk_oracle_tree_accept(
        _p(logits), _p(q_probs), _p(node_token), _p(node_q), _p(child_begin), _p(u_accept), _p(u_resample),
        B, N, NQ, V, v_begin, v_end, ctypes.c_float(cfg_scale), ctypes.c_float(temperature), int(top_k),
        _p(accept_len), _p(token), _p(path), max_depth, _p(acc_margin), _p(res_margin))
    return dict(accept_len=accept_len, token=token, path=path, accept_margin=acc_margin,
                resample_margin=res_margin, flags=flags)
