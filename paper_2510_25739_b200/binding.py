"""Thin Python binding of the C-ABI library: argument marshalling only.

Every function takes torch CUDA tensors, checks dtype/contiguity/device, and passes raw pointers,
sizes and the current CUDA stream to the entry point of the same name in libhawk_verify.so.  No
step of the verify path is computed here, and there is no fallback: a missing library raises.
"""
from __future__ import annotations

import contextlib
import ctypes
from pathlib import Path
from typing import Optional

import torch

_PKG = Path(__file__).resolve().parent
_LIB_PATH = _PKG / "libhawk_verify.so"
_lib: Optional[ctypes.CDLL] = None

DEV_TIMEOUT, DEV_BAD_DRAFT, DEV_NONFINITE, DEV_BAD_PREFIX, DEV_BAD_TREE, DEV_BOUNDS = 1, 2, 4, 8, 16, 32

EXPORTS = (
    "hawk_status_string", "hawk_version",
    "hawk_verify_attn_workspace_bytes", "hawk_verify_attn",
    "hawk_head_proj",
    "hawk_cfg_accept_workspace_bytes", "hawk_cfg_accept",
    "hawk_verify_step_host",
    "hawk_cfg_accept_noalloc_max_rows", "hawk_cfg_accept_noalloc",
    "hawk_tree_accept_workspace_bytes", "hawk_tree_accept", "hawk_verify_attn_tree",
    "hawk_spec_cache_slots", "hawk_spec_cache_slot", "hawk_spec_cache_clear", "hawk_spec_cache_put",
    "hawk_pool_build", "hawk_pool_sample_workspace_bytes", "hawk_pool_sample",
    "hawk_head_proj_cfg", "hawk_cfg_accept_guided", "hawk_tree_accept_guided",
)


def _step_fields():
    vp, i32, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    ints = ("B", "K", "H", "H_kv", "D", "L_cap", "max_prefix_len", "V", "v_begin", "v_end", "top_k")
    floats = ("sm_scale", "cfg_scale", "temperature")
    ptrs = ("h_q", "h_x", "h_q_probs", "h_draft", "h_u_accept", "h_u_resample", "h_accept_len", "h_out_token",
            "d_k_cache", "d_v_cache", "d_prefix_len", "d_w",
            "d_q", "d_x", "d_q_probs", "d_draft", "d_u_accept", "d_u_resample",
            "d_attn_out", "d_logits", "d_accept_len", "d_out_token", "d_attn_workspace")
    return ([(n, i32) for n in ints] + [(n, f32) for n in floats] + [(n, vp) for n in ptrs]
            + [("attn_workspace_bytes", sz), ("d_accept_workspace", vp), ("accept_workspace_bytes", sz),
               ("d_status", vp)])


class StepHostArgs(ctypes.Structure):
    """Mirror of hawk_step_host_args (include/hawk.h)."""
    _fields_ = _step_fields()


class HawkError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: status {code} ({status_string(code)})")


def library_path() -> Path:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Loads libhawk_verify.so (built in-tree by paper_2510_25739_b200.build); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2510_25739_b200.build` "
            "(or __graft_entry__.build()); there is no fallback path")
    _lib = _open(_LIB_PATH)
    return _lib


@contextlib.contextmanager
def alternate_library(path):
    """Routes every call of this module to another build of the same library while the block runs (the tests of
    the kernels' give-up paths load a variant with short waits this way); the regular library is back afterwards."""
    global _lib
    if not Path(path).exists():
        raise RuntimeError(f"{path} is missing")
    saved = _lib
    _lib = _open(Path(path))
    try:
        yield _lib
    finally:
        _lib = saved


def _open(path: Path) -> ctypes.CDLL:
    """dlopens one build of the library and declares the argument types of its entry points."""
    lib = ctypes.CDLL(str(path))
    vp, i32, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.hawk_status_string.restype = ctypes.c_char_p
    lib.hawk_status_string.argtypes = [i32]
    lib.hawk_version.restype = i32
    lib.hawk_version.argtypes = []
    lib.hawk_verify_attn_workspace_bytes.restype = sz
    lib.hawk_verify_attn_workspace_bytes.argtypes = [i32] * 6
    lib.hawk_verify_attn.restype = i32
    lib.hawk_verify_attn.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, f32, vp, sz, vp, vp]
    lib.hawk_verify_attn_tree.restype = i32
    lib.hawk_verify_attn_tree.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, f32, vp, sz, vp, vp]
    lib.hawk_head_proj.restype = i32
    lib.hawk_head_proj.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp]
    lib.hawk_cfg_accept_workspace_bytes.restype = sz
    lib.hawk_cfg_accept_workspace_bytes.argtypes = [i32] * 3
    lib.hawk_cfg_accept.restype = i32
    lib.hawk_cfg_accept.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, f32, i32, i32,
                                    vp, vp, vp, vp, sz, vp, vp]
    lib.hawk_cfg_accept_noalloc_max_rows.restype = sz
    lib.hawk_cfg_accept_noalloc_max_rows.argtypes = []
    lib.hawk_cfg_accept_noalloc.restype = i32
    lib.hawk_cfg_accept_noalloc.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, f32, i32, i32,
                                            vp, vp, vp, vp]
    lib.hawk_tree_accept_workspace_bytes.restype = sz
    lib.hawk_tree_accept_workspace_bytes.argtypes = [i32, i32]
    lib.hawk_tree_accept.restype = i32
    lib.hawk_tree_accept.argtypes = [vp] * 7 + [i32] * 6 + [f32, f32, i32, i32] + [vp, vp, vp, vp, sz, vp, vp]
    lib.hawk_head_proj_cfg.restype = i32
    lib.hawk_head_proj_cfg.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, f32, f32, vp, vp]
    lib.hawk_cfg_accept_guided.restype = i32
    lib.hawk_cfg_accept_guided.argtypes = [vp] * 5 + [i32] * 7 + [vp, vp, vp, vp, sz, vp, vp]
    lib.hawk_tree_accept_guided.restype = i32
    lib.hawk_tree_accept_guided.argtypes = [vp] * 7 + [i32] * 8 + [vp, vp, vp, vp, sz, vp, vp]
    lib.hawk_spec_cache_slots.restype = i32
    lib.hawk_spec_cache_slots.argtypes = [i32, i32]
    lib.hawk_spec_cache_slot.restype = i32
    lib.hawk_spec_cache_slot.argtypes = [i32, i32, i32, i32]
    lib.hawk_spec_cache_clear.restype = i32
    lib.hawk_spec_cache_clear.argtypes = [vp, i32, i32, i32, vp]
    lib.hawk_spec_cache_put.restype = i32
    lib.hawk_spec_cache_put.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.hawk_pool_build.restype = i32
    lib.hawk_pool_build.argtypes = [vp] * 6 + [i32] * 5 + [vp]
    lib.hawk_pool_sample_workspace_bytes.restype = sz
    lib.hawk_pool_sample_workspace_bytes.argtypes = [i32, i32]
    lib.hawk_pool_sample.restype = i32
    lib.hawk_pool_sample.argtypes = [vp] * 4 + [i32] * 6 + [vp, sz, vp, vp]
    lib.hawk_verify_step_host.restype = i32
    lib.hawk_verify_step_host.argtypes = [ctypes.POINTER(StepHostArgs), vp]
    return lib


def status_string(code: int) -> str:
    return load_library().hawk_status_string(int(code)).decode()


def version() -> int:
    return load_library().hawk_version()


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _check(t: torch.Tensor, dtype, name: str, shape=None):
    if t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if not t.is_cuda:
        raise ValueError(f"{name}: must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name}: must be contiguous")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise ValueError(f"{name}: expected shape {tuple(shape)}, got {tuple(t.shape)}")


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def verify_attn_workspace_bytes(S: int, K: int, H: int, H_kv: int, D: int, max_prefix_len: int) -> int:
    return int(load_library().hawk_verify_attn_workspace_bytes(S, K, H, H_kv, D, max_prefix_len))


def verify_attn(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, prefix_len: torch.Tensor,
                max_prefix_len: int, sm_scale: float, out: Optional[torch.Tensor] = None,
                workspace: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                anc_mask: Optional[torch.Tensor] = None) -> torch.Tensor:
    """q [S,K,H,D], caches [S,H_kv,L_cap,D] (bf16), prefix_len [S] int32 -> out [S,K,H*D] bf16.
    With anc_mask (int64 tensor holding the uint64 masks, [K]) the K rows are tree nodes (hawk_verify_attn_tree)."""
    lib = load_library()
    S, K, H, D = q.shape
    _, H_kv, L_cap, _ = k_cache.shape
    _check(q, torch.bfloat16, "q")
    _check(k_cache, torch.bfloat16, "k_cache", (S, H_kv, L_cap, D))
    _check(v_cache, torch.bfloat16, "v_cache", (S, H_kv, L_cap, D))
    _check(prefix_len, torch.int32, "prefix_len", (S,))
    if out is None:
        out = torch.empty((S, K, H * D), dtype=torch.bfloat16, device=q.device)
    _check(out, torch.bfloat16, "out", (S, K, H * D))
    need = verify_attn_workspace_bytes(S, K, H, H_kv, D, max_prefix_len)
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    if anc_mask is not None:
        _check(anc_mask, torch.int64, "anc_mask", (K,))
        rc = lib.hawk_verify_attn_tree(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(prefix_len), _ptr(anc_mask),
                                       _ptr(out), S, K, H, H_kv, D, L_cap, int(max_prefix_len), float(sm_scale),
                                       _ptr(workspace), ws_bytes, _ptr(dev_status), _stream())
        if rc != 0:
            raise HawkError(rc, "hawk_verify_attn_tree")
        return out
    rc = lib.hawk_verify_attn(_ptr(q), _ptr(k_cache), _ptr(v_cache), _ptr(prefix_len), _ptr(out), S, K, H, H_kv, D,
                              L_cap, int(max_prefix_len), float(sm_scale), _ptr(workspace), ws_bytes,
                              _ptr(dev_status), _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_verify_attn")
    return out


def verify_attn_tree(q: torch.Tensor, k_cache: torch.Tensor, v_cache: torch.Tensor, prefix_len: torch.Tensor,
                     anc_mask: torch.Tensor, max_prefix_len: int, sm_scale: float, **kwargs) -> torch.Tensor:
    """hawk_verify_attn_tree: the N rows of q are tree nodes, anc_mask [N] their ancestor bit masks."""
    return verify_attn(q, k_cache, v_cache, prefix_len, max_prefix_len, sm_scale, anc_mask=anc_mask, **kwargs)


def head_proj(x: torch.Tensor, w: torch.Tensor, v_begin: int = 0, v_end: Optional[int] = None,
              logits: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """x [M,hidden], w [V,hidden] (bf16) -> logits [M,V] fp32 (only columns [v_begin,v_end) written)."""
    lib = load_library()
    M, hidden = x.shape
    V = w.shape[0]
    v_end = V if v_end is None else v_end
    _check(x, torch.bfloat16, "x")
    _check(w, torch.bfloat16, "w", (V, hidden))
    if logits is None:
        logits = torch.empty((M, V), dtype=torch.float32, device=x.device)
    _check(logits, torch.float32, "logits", (M, V))
    rc = lib.hawk_head_proj(_ptr(x), _ptr(w), _ptr(logits), M, hidden, V, int(v_begin), int(v_end),
                            _ptr(dev_status), _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_head_proj")
    return logits


def head_proj_cfg(x: torch.Tensor, w: torch.Tensor, cfg_scale: float, temperature: float, v_begin: int = 0,
                  v_end: Optional[int] = None, guided: Optional[torch.Tensor] = None,
                  dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """x [2B,rows,hidden], w [V,hidden] (bf16) -> guided logits [B,rows,V] fp32 (columns [v_begin,v_end) written)."""
    lib = load_library()
    S, rows, hidden = x.shape
    if S % 2:
        raise ValueError("x: the first dimension holds B conditional then B unconditional streams")
    B = S // 2
    V = w.shape[0]
    v_end = V if v_end is None else v_end
    _check(x, torch.bfloat16, "x")
    _check(w, torch.bfloat16, "w", (V, hidden))
    if guided is None:
        guided = torch.empty((B, rows, V), dtype=torch.float32, device=x.device)
    _check(guided, torch.float32, "guided", (B, rows, V))
    rc = lib.hawk_head_proj_cfg(_ptr(x), _ptr(w), _ptr(guided), B, rows, hidden, V, int(v_begin), int(v_end),
                                float(cfg_scale), float(temperature), _ptr(dev_status), _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_head_proj_cfg")
    return guided


def cfg_accept_guided(guided: torch.Tensor, q_probs: torch.Tensor, draft: torch.Tensor, u_accept: torch.Tensor,
                      u_resample: torch.Tensor, v_begin: int, v_end: int, top_k: int, has_bonus_row: bool = False,
                      accept_len: Optional[torch.Tensor] = None, out_token: Optional[torch.Tensor] = None,
                      p_debug: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                      dev_status: Optional[torch.Tensor] = None):
    """guided [B,K(+1),V] fp32 (from head_proj_cfg), otherwise as cfg_accept -> (accept_len, out_token)."""
    lib = load_library()
    B, K, V = q_probs.shape
    rows = K + (1 if has_bonus_row else 0)
    _check(guided, torch.float32, "guided", (B, rows, V))
    _check(q_probs, torch.float32, "q_probs")
    _check(draft, torch.int32, "draft", (B, K))
    _check(u_accept, torch.float32, "u_accept", (B, K))
    _check(u_resample, torch.float32, "u_resample", (B, K + 1))
    dev = guided.device
    if accept_len is None:
        accept_len = torch.empty(B, dtype=torch.int32, device=dev)
    if out_token is None:
        out_token = torch.empty(B, dtype=torch.int32, device=dev)
    _check(accept_len, torch.int32, "accept_len", (B,))
    _check(out_token, torch.int32, "out_token", (B,))
    if p_debug is not None:
        _check(p_debug, torch.float32, "p_debug", (B, rows, V))
    need = cfg_accept_workspace_bytes(B, K, V)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    ws_bytes = workspace.numel() * workspace.element_size()
    rc = lib.hawk_cfg_accept_guided(_ptr(guided), _ptr(q_probs), _ptr(draft), _ptr(u_accept), _ptr(u_resample), B, K, V,
                                    int(v_begin), int(v_end), int(top_k), int(bool(has_bonus_row)), _ptr(accept_len),
                                    _ptr(out_token), _ptr(p_debug), _ptr(workspace), ws_bytes, _ptr(dev_status),
                                    _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_cfg_accept_guided")
    return accept_len, out_token


def cfg_accept_workspace_bytes(B: int, K: int, V: int) -> int:
    return int(load_library().hawk_cfg_accept_workspace_bytes(B, K, V))


def cfg_accept(logits: torch.Tensor, q_probs: torch.Tensor, draft: torch.Tensor, u_accept: torch.Tensor,
               u_resample: torch.Tensor, v_begin: int, v_end: int, cfg_scale: float, temperature: float,
               top_k: int, has_bonus_row: bool = False, accept_len: Optional[torch.Tensor] = None,
               out_token: Optional[torch.Tensor] = None, p_debug: Optional[torch.Tensor] = None,
               workspace: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None):
    """logits [2B,K(+1),V] fp32, q_probs [B,K,V] fp32, draft [B,K] int32, uniforms -> (accept_len, out_token)."""
    lib = load_library()
    B, K, V = q_probs.shape
    rows = K + (1 if has_bonus_row else 0)
    _check(logits, torch.float32, "logits", (2 * B, rows, V))
    _check(q_probs, torch.float32, "q_probs")
    _check(draft, torch.int32, "draft", (B, K))
    _check(u_accept, torch.float32, "u_accept", (B, K))
    _check(u_resample, torch.float32, "u_resample", (B, K + 1))
    dev = logits.device
    if accept_len is None:
        accept_len = torch.empty(B, dtype=torch.int32, device=dev)
    if out_token is None:
        out_token = torch.empty(B, dtype=torch.int32, device=dev)
    _check(accept_len, torch.int32, "accept_len", (B,))
    _check(out_token, torch.int32, "out_token", (B,))
    if p_debug is not None:
        _check(p_debug, torch.float32, "p_debug", (B, rows, V))
    need = cfg_accept_workspace_bytes(B, K, V)
    if workspace is None:
        workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    ws_bytes = workspace.numel() * workspace.element_size()
    rc = lib.hawk_cfg_accept(_ptr(logits), _ptr(q_probs), _ptr(draft), _ptr(u_accept), _ptr(u_resample), B, K, V,
                             int(v_begin), int(v_end), float(cfg_scale), float(temperature), int(top_k),
                             int(bool(has_bonus_row)), _ptr(accept_len), _ptr(out_token), _ptr(p_debug),
                             _ptr(workspace), ws_bytes, _ptr(dev_status), _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_cfg_accept")
    return accept_len, out_token


def cfg_accept_noalloc_max_rows() -> int:
    return int(load_library().hawk_cfg_accept_noalloc_max_rows())


def cfg_accept_noalloc(logits: torch.Tensor, q_probs: torch.Tensor, draft: torch.Tensor, u_accept: torch.Tensor,
                       u_resample: torch.Tensor, v_begin: int, v_end: int, cfg_scale: float, temperature: float,
                       top_k: int, accept_len: torch.Tensor, out_token: torch.Tensor, has_bonus_row: bool = False,
                       dev_status: Optional[torch.Tensor] = None):
    """cfg_accept for callers that cannot lend a workspace: the verdict scratch is the library's built-in
    array.  Nothing is allocated here either, so both result tensors ([B] int32) must be passed in.
    Steps with B * (K + 1) above cfg_accept_noalloc_max_rows() are refused (HawkError, workspace)."""
    lib = load_library()
    B, K, V = q_probs.shape
    rows = K + (1 if has_bonus_row else 0)
    _check(logits, torch.float32, "logits", (2 * B, rows, V))
    _check(q_probs, torch.float32, "q_probs")
    _check(draft, torch.int32, "draft", (B, K))
    _check(u_accept, torch.float32, "u_accept", (B, K))
    _check(u_resample, torch.float32, "u_resample", (B, K + 1))
    _check(accept_len, torch.int32, "accept_len", (B,))
    _check(out_token, torch.int32, "out_token", (B,))
    rc = lib.hawk_cfg_accept_noalloc(_ptr(logits), _ptr(q_probs), _ptr(draft), _ptr(u_accept), _ptr(u_resample),
                                     B, K, V, int(v_begin), int(v_end), float(cfg_scale), float(temperature),
                                     int(top_k), int(bool(has_bonus_row)), _ptr(accept_len), _ptr(out_token),
                                     _ptr(dev_status), _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_cfg_accept_noalloc")
    return accept_len, out_token


def tree_accept(logits: torch.Tensor, q_probs: torch.Tensor, node_token: torch.Tensor, node_q: torch.Tensor,
                child_begin: torch.Tensor, u_accept: torch.Tensor, u_resample: torch.Tensor, v_begin: int,
                v_end: int, cfg_scale: float, temperature: float, top_k: int, max_depth: Optional[int] = None,
                dev_status: Optional[torch.Tensor] = None):
    """Candidate-tree verification: logits [2B,N,V], q_probs [B,NQ,V], node_token [B,N], node_q [N],
    child_begin [N+1], uniforms [B,N] -> (accept_len [B], out_token [B], path [B,max_depth])."""
    lib = load_library()
    B, NQ, V = q_probs.shape
    N = node_q.shape[0]
    max_depth = N if max_depth is None else int(max_depth)
    _check(logits, torch.float32, "logits", (2 * B, N, V))
    _check(q_probs, torch.float32, "q_probs")
    _check(node_token, torch.int32, "node_token", (B, N))
    _check(node_q, torch.int32, "node_q", (N,))
    _check(child_begin, torch.int32, "child_begin", (N + 1,))
    _check(u_accept, torch.float32, "u_accept", (B, N))
    _check(u_resample, torch.float32, "u_resample", (B, N))
    dev = logits.device
    accept_len = torch.empty(B, dtype=torch.int32, device=dev)
    out_token = torch.empty(B, dtype=torch.int32, device=dev)
    path = torch.empty((B, max_depth), dtype=torch.int32, device=dev)
    need = int(lib.hawk_tree_accept_workspace_bytes(B, N))
    workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    rc = lib.hawk_tree_accept(_ptr(logits), _ptr(q_probs), _ptr(node_token), _ptr(node_q), _ptr(child_begin),
                              _ptr(u_accept), _ptr(u_resample), B, N, NQ, V, int(v_begin), int(v_end),
                              float(cfg_scale), float(temperature), int(top_k), max_depth, _ptr(accept_len),
                              _ptr(out_token), _ptr(path), _ptr(workspace), workspace.numel(), _ptr(dev_status),
                              _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_tree_accept")
    return accept_len, out_token, path


def tree_accept_guided(guided: torch.Tensor, q_probs: torch.Tensor, node_token: torch.Tensor, node_q: torch.Tensor,
                       child_begin: torch.Tensor, u_accept: torch.Tensor, u_resample: torch.Tensor, v_begin: int,
                       v_end: int, top_k: int, max_depth: Optional[int] = None,
                       dev_status: Optional[torch.Tensor] = None):
    """guided [B,N,V] fp32 (from head_proj_cfg), otherwise as tree_accept -> (accept_len, out_token, path)."""
    lib = load_library()
    B, NQ, V = q_probs.shape
    N = node_q.shape[0]
    max_depth = N if max_depth is None else int(max_depth)
    _check(guided, torch.float32, "guided", (B, N, V))
    _check(q_probs, torch.float32, "q_probs")
    _check(node_token, torch.int32, "node_token", (B, N))
    _check(node_q, torch.int32, "node_q", (N,))
    _check(child_begin, torch.int32, "child_begin", (N + 1,))
    _check(u_accept, torch.float32, "u_accept", (B, N))
    _check(u_resample, torch.float32, "u_resample", (B, N))
    dev = guided.device
    accept_len = torch.empty(B, dtype=torch.int32, device=dev)
    out_token = torch.empty(B, dtype=torch.int32, device=dev)
    path = torch.empty((B, max_depth), dtype=torch.int32, device=dev)
    need = int(lib.hawk_tree_accept_workspace_bytes(B, N))
    workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    rc = lib.hawk_tree_accept_guided(_ptr(guided), _ptr(q_probs), _ptr(node_token), _ptr(node_q), _ptr(child_begin),
                                     _ptr(u_accept), _ptr(u_resample), B, N, NQ, V, int(v_begin), int(v_end),
                                     int(top_k), max_depth, _ptr(accept_len), _ptr(out_token), _ptr(path),
                                     _ptr(workspace), workspace.numel(), _ptr(dev_status), _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_tree_accept_guided")
    return accept_len, out_token, path


def spec_cache_slots(IW: int, VSD: int) -> int:
    """Rows of the speculation cache per sequence, IW * VSD * (VSD + 1) / 2."""
    return int(load_library().hawk_spec_cache_slots(int(IW), int(VSD)))


def spec_cache_slot(IW: int, VSD: int, position: int, depth: int) -> int:
    return int(load_library().hawk_spec_cache_slot(int(IW), int(VSD), int(position), int(depth)))


def spec_cache_new(B: int, IW: int, VSD: int, V: int, device="cuda"):
    """Allocates (cache_rows [B,slots,V] fp32, cache_tags [B,slots] int32) and marks every slot unwritten."""
    slots = spec_cache_slots(IW, VSD)
    rows = torch.empty((B, slots, V), dtype=torch.float32, device=device)
    tags = torch.empty((B, slots), dtype=torch.int32, device=device)
    spec_cache_clear(tags, IW, VSD)
    return rows, tags


def spec_cache_clear(cache_tags: torch.Tensor, IW: int, VSD: int) -> None:
    B = cache_tags.shape[0]
    _check(cache_tags, torch.int32, "cache_tags", (B, spec_cache_slots(IW, VSD)))
    rc = load_library().hawk_spec_cache_clear(_ptr(cache_tags), B, int(IW), int(VSD), _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_spec_cache_clear")


def spec_cache_put(q_vert: torch.Tensor, position: torch.Tensor, cache_rows: torch.Tensor,
                   cache_tags: torch.Tensor, IW: int) -> None:
    """Stores the vertical predictions q_vert [B,VSD,V] made at position [B] into the cache."""
    B, VSD, V = q_vert.shape
    slots = spec_cache_slots(IW, VSD)
    _check(q_vert, torch.float32, "q_vert")
    _check(position, torch.int32, "position", (B,))
    _check(cache_rows, torch.float32, "cache_rows", (B, slots, V))
    _check(cache_tags, torch.int32, "cache_tags", (B, slots))
    rc = load_library().hawk_spec_cache_put(_ptr(q_vert), _ptr(position), _ptr(cache_rows), _ptr(cache_tags), B,
                                            int(IW), VSD, V, _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_spec_cache_put")


def pool_build(q_horiz: torch.Tensor, cache_rows: torch.Tensor, cache_tags: torch.Tensor, position: torch.Tensor,
               IW: int, VSD: int, with_source: bool = True):
    """q_horiz [B,K,V] + cache -> (pool_q [B,K*(1+VSD),V], pool_source [B,K*(1+VSD)] or None)."""
    B, K, V = q_horiz.shape
    slots = spec_cache_slots(IW, VSD)
    _check(q_horiz, torch.float32, "q_horiz")
    _check(cache_rows, torch.float32, "cache_rows", (B, slots, V))
    _check(cache_tags, torch.int32, "cache_tags", (B, slots))
    _check(position, torch.int32, "position", (B,))
    NQ = K * (1 + VSD)
    pool_q = torch.empty((B, NQ, V), dtype=torch.float32, device=q_horiz.device)
    source = torch.empty((B, NQ), dtype=torch.int32, device=q_horiz.device) if with_source else None
    rc = load_library().hawk_pool_build(_ptr(q_horiz), _ptr(cache_rows), _ptr(cache_tags), _ptr(position),
                                        _ptr(pool_q), _ptr(source), B, K, int(IW), int(VSD), V, _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_pool_build")
    return pool_q, source


def pool_sample_workspace_bytes(B: int, NQ: int) -> int:
    return int(load_library().hawk_pool_sample_workspace_bytes(int(B), int(NQ)))


def pool_sample(pool_q: torch.Tensor, u: torch.Tensor, node_q: torch.Tensor, v_begin: int, v_end: int,
                dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """One draw per pool row, handed to the tree nodes: returns node_token [B,N] int32."""
    B, NQ, V = pool_q.shape
    N = node_q.shape[0]
    _check(pool_q, torch.float32, "pool_q")
    _check(u, torch.float32, "u", (B, NQ))
    _check(node_q, torch.int32, "node_q", (N,))
    node_token = torch.empty((B, N), dtype=torch.int32, device=pool_q.device)
    need = pool_sample_workspace_bytes(B, NQ)
    workspace = torch.empty(max(need, 16), dtype=torch.uint8, device=pool_q.device)
    rc = load_library().hawk_pool_sample(_ptr(pool_q), _ptr(u), _ptr(node_q), _ptr(node_token), B, NQ, N, V,
                                         int(v_begin), int(v_end), _ptr(workspace), workspace.numel(),
                                         _ptr(dev_status), _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_pool_sample")
    return node_token


def verify_step_host(args: StepHostArgs) -> None:
    """Queues one whole verify step (copies in, three kernels, copies out) on the current stream."""
    rc = load_library().hawk_verify_step_host(ctypes.byref(args), _stream())
    if rc != 0:
        raise HawkError(rc, "hawk_verify_step_host")
