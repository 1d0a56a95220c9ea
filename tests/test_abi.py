"""The C-ABI library loads, exports every function include/hawk.h declares, and its host-side
argument checks return the documented codes.  Nothing here launches a kernel: every call below is
rejected (or is a no-op) before the library touches a device."""
import ctypes
import re
from pathlib import Path

import pytest

from paper_2510_25739_b200 import binding, build

HEADER = Path(__file__).resolve().parent.parent / "include" / "hawk.h"
OK, E_NULL, E_SHAPE, E_ALIGN, E_UNSUP, E_WS, E_PARAM, E_CUDA = range(8)


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def _declared_functions():
    text = re.sub(r"/\*.*?\*/", "", HEADER.read_text(), flags=re.S)
    return sorted(set(re.findall(r"\b(hawk_[a-z_]+)\s*\(", text)))


def test_every_declared_function_is_exported(lib):
    names = _declared_functions()
    assert {"hawk_verify_attn", "hawk_head_proj", "hawk_cfg_accept"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in hawk.h but not exported"
    assert set(binding.EXPORTS) == set(names)


def test_version_and_status_strings(lib):
    assert lib.hawk_version() >= 100
    seen = {lib.hawk_status_string(c).decode() for c in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert lib.hawk_status_string(99).decode() == "unknown status"


def test_step_struct_matches_the_header():
    text = HEADER.read_text()
    body = text[text.index("typedef struct {"):text.index("} hawk_step_host_args;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    names = []
    for decl in body.split(";"):
        decl = decl.replace("typedef struct {", "").strip()
        if not decl:
            continue
        parts = re.sub(r"^(const\s+)?(void|float|int32_t|int|size_t)\b", "", decl).split(",")
        names += [p.replace("*", "").strip() for p in parts]
    assert names == [f[0] for f in binding.StepHostArgs._fields_]


def test_workspace_queries(lib):
    # invalid shapes report 0; a launch that cuts items needs two 16-row fp32 partial slots per share
    assert lib.hawk_verify_attn_workspace_bytes(0, 4, 16, 16, 64, 128) == 0
    assert lib.hawk_verify_attn_workspace_bytes(2, 4, 16, 16, 96, 128) == 0
    need = lib.hawk_verify_attn_workspace_bytes(64, 6, 24, 24, 64, 1144)   # 1536 items cut into equal shares
    assert need > 0 and need % (2 * 8 * 66 * 4) == 0          # K = 6 rows round up to 8 per item
    # 320 long items of 8 rows: the four warps of a block share an item and merge in shared memory
    assert lib.hawk_verify_attn_workspace_bytes(16, 5, 20, 20, 64, 1144) == 0
    # the same items with 24 tree rows each are cut into shares again
    assert lib.hawk_verify_attn_workspace_bytes(16, 22, 20, 20, 64, 1144) > 0
    # one tile per item and one share per tile: nothing is cut, no workspace
    assert lib.hawk_verify_attn_workspace_bytes(2, 1, 1, 1, 64, 0) == 0
    assert lib.hawk_cfg_accept_workspace_bytes(8, 5, 16384) >= 8 * 5 * 4
    assert lib.hawk_cfg_accept_workspace_bytes(0, 5, 16384) == 0


def test_attn_argument_checks(lib):
    p = ctypes.c_void_p(0x1000)          # never dereferenced: every call below fails a host check first
    odd = ctypes.c_void_p(0x1004)
    f = lib.hawk_verify_attn
    args = dict(S=2, K=4, H=16, H_kv=16, D=64, L_cap=132, mpl=128, scale=0.125)

    def call(q=p, k=p, v=p, pl=p, out=p, ws=None, wsb=0, **kw):
        a = {**args, **kw}
        return f(q, k, v, pl, out, a["S"], a["K"], a["H"], a["H_kv"], a["D"], a["L_cap"], a["mpl"], a["scale"],
                 ws, wsb, None, None)

    assert call(S=0) == OK
    assert call(S=-1) == E_SHAPE
    assert call(q=None) == E_NULL
    assert call(out=None) == E_NULL
    assert call(K=0) == E_UNSUP and call(K=65, L_cap=300) == E_UNSUP
    assert call(D=96) == E_UNSUP
    assert call(H=16, H_kv=3) == E_UNSUP
    assert call(mpl=129) == E_SHAPE                      # prefix + K exceeds the cache capacity
    assert call(scale=0.0) == E_PARAM and call(scale=float("nan")) == E_PARAM
    assert call(scale=float("inf")) == E_PARAM
    assert call(k=odd) == E_ALIGN
    assert call(S=2 ** 20, L_cap=2 ** 12, mpl=100) == E_UNSUP   # row index would overflow 31 bits


def test_head_argument_checks(lib):
    p, odd = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1008)
    f = lib.hawk_head_proj
    assert f(p, p, p, 0, 1024, 16384, 0, 16384, None, None) == OK
    assert f(p, p, p, 8, 1024, 16384, 5, 5, None, None) == OK       # empty range
    assert f(p, p, p, -1, 1024, 16384, 0, 16384, None, None) == E_SHAPE
    assert f(p, p, p, 8, 1024, 16384, 0, 16385, None, None) == E_SHAPE
    assert f(p, p, p, 8, 1024, 16384, 9, 8, None, None) == E_SHAPE
    assert f(None, p, p, 8, 1024, 16384, 0, 16384, None, None) == E_NULL
    assert f(p, p, p, 8, 1000, 16384, 0, 16384, None, None) == E_UNSUP   # hidden not a multiple of 64
    assert f(p, odd, p, 8, 1024, 16384, 0, 16384, None, None) == E_ALIGN


def test_accept_argument_checks(lib):
    p, odd = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1004)
    f = lib.hawk_cfg_accept

    def call(lg=p, q=p, d=p, ua=p, ur=p, B=2, K=4, V=1024, vb=0, ve=1024, s=3.0, T=1.0, k=100, al=p, tok=p,
             ws=p, wsb=1 << 20):
        return f(lg, q, d, ua, ur, B, K, V, vb, ve, s, T, k, 0, al, tok, None, ws, wsb, None, None)

    assert call(B=0) == OK
    assert call(B=-1) == E_SHAPE
    assert call(lg=None) == E_NULL and call(tok=None) == E_NULL
    assert call(vb=10, ve=10) == E_SHAPE and call(ve=2000) == E_SHAPE
    assert call(K=0) == E_UNSUP and call(K=17) == E_UNSUP
    assert call(V=40000, ve=40000) == E_UNSUP            # more valid ids than one block holds
    assert call(T=0.0) == E_PARAM and call(T=-1.0) == E_PARAM and call(T=float("nan")) == E_PARAM
    assert call(s=float("inf")) == E_PARAM
    assert call(q=odd) == E_ALIGN
    assert call(ws=None) == E_WS and call(wsb=4) == E_WS


def test_step_host_argument_checks(lib):
    assert lib.hawk_verify_step_host(None, None) == E_NULL
    a = binding.StepHostArgs()
    a.B = 0
    assert lib.hawk_verify_step_host(ctypes.byref(a), None) == OK
    a.B, a.K, a.H, a.D, a.V = 1, 4, 16, 64, 16384
    assert lib.hawk_verify_step_host(ctypes.byref(a), None) == E_NULL     # no buffers given


def test_step_host_checks_every_stage_before_it_queues_anything(lib):
    """The step call runs the argument checks of all three stages before its first copy: a bad argument of the
    LAST stage is reported although the first two stages' arguments are fine (the pointers are never touched:
    every call below is refused on the host)."""
    def good():
        a = binding.StepHostArgs()
        a.B, a.K, a.H, a.H_kv, a.D, a.L_cap, a.max_prefix_len = 2, 4, 16, 16, 64, 132, 128
        a.V, a.v_begin, a.v_end, a.top_k = 16384, 0, 16384, 1000
        a.sm_scale, a.cfg_scale, a.temperature = 0.125, 4.0, 1.0
        for name, _ in binding.StepHostArgs._fields_:
            if name.startswith(("h_", "d_")) and name != "d_status":
                setattr(a, name, 0x1000)
        a.attn_workspace_bytes, a.accept_workspace_bytes = 1 << 20, 1 << 20
        return a

    def call(**kw):
        a = good()
        for k, v in kw.items():
            setattr(a, k, v)
        return lib.hawk_verify_step_host(ctypes.byref(a), None)

    # accept stage (the last one)
    assert call(temperature=0.0) == E_PARAM
    assert call(cfg_scale=float("nan")) == E_PARAM
    assert call(K=17, L_cap=200) == E_UNSUP                       # attention takes 17 rows, accept does not
    assert call(accept_workspace_bytes=4) == E_WS
    assert call(d_accept_workspace=None) == E_WS
    assert call(d_q_probs=0x1004) == E_ALIGN
    assert call(v_begin=10, v_end=10) == E_SHAPE
    # head projection
    assert call(H=15) == E_UNSUP                                  # hidden 960 is a multiple of 64, 15 heads of 16 kv heads are not
    assert call(d_logits=0x1008) == E_ALIGN
    assert call(v_end=20000) == E_SHAPE
    # attention
    assert call(D=96) == E_UNSUP
    assert call(max_prefix_len=130) == E_SHAPE                    # 130 + 4 rows exceed the cache capacity
    assert call(sm_scale=0.0) == E_PARAM
    assert call(H_kv=-1) == E_SHAPE
    assert call(d_k_cache=0x1002) == E_ALIGN


def test_tree_accept_argument_checks(lib):
    p, odd = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1004)
    f = lib.hawk_tree_accept

    def call(lg=p, q=p, tok=p, nq=p, cb=p, ua=p, ur=p, B=2, N=7, NQ=4, V=1024, vb=0, ve=1024, s=3.0, T=1.0, k=100,
             depth=2, al=p, out=p, path=p, ws=p, wsb=1 << 20):
        return f(lg, q, tok, nq, cb, ua, ur, B, N, NQ, V, vb, ve, s, T, k, depth, al, out, path, ws, wsb, None, None)

    assert lib.hawk_tree_accept_workspace_bytes(4, 22) == (4 + 1) * 22 * 4   # verdicts and one parent per node
    assert lib.hawk_tree_accept_workspace_bytes(0, 22) == 0
    assert call(B=0) == OK
    assert call(B=-1) == E_SHAPE and call(depth=-1) == E_SHAPE
    assert call(cb=None) == E_NULL and call(out=None) == E_NULL
    assert call(N=0) == E_SHAPE and call(NQ=0) == E_SHAPE
    assert call(ve=2000) == E_SHAPE
    assert call(N=70000) == E_UNSUP
    assert call(V=40000, ve=40000) == E_UNSUP
    assert call(T=0.0) == E_PARAM
    assert call(lg=odd) == E_ALIGN
    assert call(ws=None) == E_WS and call(wsb=8) == E_WS


def test_attn_tree_argument_checks(lib):
    p = ctypes.c_void_p(0x1000)
    f = lib.hawk_verify_attn_tree
    assert f(p, p, p, p, None, p, 2, 7, 4, 4, 64, 100, 90, 0.125, None, 0, None, None) == E_NULL   # no mask
    assert f(p, p, p, p, p, p, 0, 7, 4, 4, 64, 100, 90, 0.125, None, 0, None, None) == OK
    assert f(p, p, p, p, p, p, 2, 65, 4, 4, 64, 200, 90, 0.125, None, 0, None, None) == E_UNSUP
    assert f(p, p, p, p, p, p, 2, 22, 4, 4, 64, 100, 90, 0.125, None, 0, None, None) == E_SHAPE    # 90 + 22 > 100


def test_guided_head_and_accept_argument_checks(lib):
    p, odd = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1008)
    f = lib.hawk_head_proj_cfg
    c = ctypes.c_float

    def head(x=p, w=p, out=p, B=2, rows=4, hidden=1024, V=16384, vb=0, ve=16384, s=3.0, T=1.0):
        return f(x, w, out, B, rows, hidden, V, vb, ve, c(s), c(T), None, None)

    assert head(B=0) == OK
    assert head(B=-1) == E_SHAPE and head(rows=-1) == E_SHAPE
    assert head(ve=16385) == E_SHAPE
    assert head(x=None) == E_NULL and head(out=None) == E_NULL
    assert head(hidden=1000) == E_UNSUP
    assert head(T=0.0) == E_PARAM and head(T=float("nan")) == E_PARAM and head(s=float("inf")) == E_PARAM
    assert head(w=odd) == E_ALIGN

    g = lib.hawk_cfg_accept_guided

    def acc(lg=p, q=p, d=p, ua=p, ur=p, B=2, K=4, V=1024, vb=0, ve=1024, k=100, al=p, tok=p, ws=p, wsb=1 << 20):
        return g(lg, q, d, ua, ur, B, K, V, vb, ve, k, 0, al, tok, None, ws, wsb, None, None)

    assert acc(B=0) == OK
    assert acc(B=-1) == E_SHAPE
    assert acc(lg=None) == E_NULL and acc(al=None) == E_NULL
    assert acc(vb=10, ve=10) == E_SHAPE
    assert acc(K=17) == E_UNSUP
    assert acc(q=odd) == E_ALIGN
    assert acc(ws=None) == E_WS

    t = lib.hawk_tree_accept_guided

    def tree(lg=p, q=p, tokn=p, nq=p, cb=p, ua=p, ur=p, B=2, N=7, NQ=4, V=1024, vb=0, ve=1024, k=100, md=3, al=p, tok=p,
             path=p, ws=p, wsb=1 << 20):
        return t(lg, q, tokn, nq, cb, ua, ur, B, N, NQ, V, vb, ve, k, md, al, tok, path, ws, wsb, None, None)

    assert tree(B=0) == OK
    assert tree(N=0) == E_SHAPE and tree(NQ=0) == E_SHAPE and tree(md=-1) == E_SHAPE
    assert tree(cb=None) == E_NULL
    assert tree(V=40000, ve=40000) == E_UNSUP
    assert tree(wsb=8) == E_WS


def test_cache_and_pool_argument_checks(lib):
    p, odd = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1004)
    assert lib.hawk_spec_cache_slots(32, 2) == 96 and lib.hawk_spec_cache_slots(48, 3) == 288
    assert lib.hawk_spec_cache_slots(0, 2) == 0 and lib.hawk_spec_cache_slots(32, 0) == 0
    # slots of one column and depth cycle with period `depth`; different depths never share a slot
    assert lib.hawk_spec_cache_slot(4, 2, 0, 1) == 0 and lib.hawk_spec_cache_slot(4, 2, 4, 1) == 0
    assert lib.hawk_spec_cache_slot(4, 2, 0, 2) == 1 and lib.hawk_spec_cache_slot(4, 2, 4, 2) == 2
    assert lib.hawk_spec_cache_slot(4, 2, 8, 2) == 1 and lib.hawk_spec_cache_slot(4, 2, 1, 1) == 3
    assert lib.hawk_spec_cache_slot(4, 2, -1, 1) == -1 and lib.hawk_spec_cache_slot(4, 2, 0, 3) == -1
    assert lib.hawk_spec_cache_clear(None, 2, 4, 2, None) == E_NULL
    assert lib.hawk_spec_cache_clear(p, 0, 4, 2, None) == OK
    assert lib.hawk_spec_cache_clear(p, 2, 0, 2, None) == E_SHAPE
    put = lib.hawk_spec_cache_put
    assert put(p, p, p, p, 0, 4, 2, 64, None) == OK
    assert put(None, p, p, p, 2, 4, 2, 64, None) == E_NULL
    assert put(p, p, p, p, 2, 4, 2, 0, None) == E_SHAPE
    assert put(p, p, p, p, 2, 4, 9, 64, None) == E_UNSUP
    build_ = lib.hawk_pool_build
    assert build_(p, p, p, p, p, None, 0, 3, 4, 2, 64, None) == OK
    assert build_(p, p, p, p, p, None, 2, 0, 4, 2, 64, None) == OK
    assert build_(p, p, p, p, None, None, 2, 3, 4, 2, 64, None) == E_NULL
    assert build_(p, p, p, p, p, None, 2, 3, 0, 2, 64, None) == E_SHAPE
    assert build_(p, p, p, p, p, None, 2, 3, 4, 9, 64, None) == E_UNSUP
    assert lib.hawk_pool_sample_workspace_bytes(2, 9) == 72 and lib.hawk_pool_sample_workspace_bytes(0, 9) == 0
    samp = lib.hawk_pool_sample

    def sample(pq=p, u=p, nq=p, out=p, B=2, NQ=9, N=22, V=1024, vb=0, ve=1024, ws=p, wsb=1 << 10):
        return samp(pq, u, nq, out, B, NQ, N, V, vb, ve, ws, wsb, None, None)

    assert sample(B=0) == OK
    assert sample(B=-1) == E_SHAPE and sample(NQ=0) == E_SHAPE and sample(vb=5, ve=5) == E_SHAPE
    assert sample(out=None) == E_NULL
    assert sample(V=40000, ve=40000) == E_UNSUP
    assert sample(pq=odd) == E_ALIGN
    assert sample(wsb=8) == E_WS
