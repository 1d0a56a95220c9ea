"""The kernels' give-up paths: a wait that runs out ends the kernel in an orderly way, reports
HAWK_DEV_TIMEOUT, and leaves the context usable.

Nothing here faults or hangs a GPU.  A second build of the library (paper_2510_25739_b200.build.build_stall_variant:
every wait limited to 2 ms, and ONE stage per launch armed for 16 bytes more than its copies deliver) makes exactly
one wait per launch run out; the kernel then takes the same exit a real stall would take: the waiting role raises
the block's abort flag, the other roles leave their loops, copies in flight are waited for (again bounded),
tensor memory is freed, and the block returns.  Each case then runs the regular library on the same stream and
inputs and checks the result against the oracle: the stalled launch left nothing behind.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_25739_b200 import binding, build
from paper_2510_25739_b200 import workloads as wl
from tests._util import bf16_to_torch, to_dev, torch_bf16_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def stall_lib():
    return build.build_stall_variant()


def _attn_case(cfg, seed, stall_lib):
    import paper_2510_25739_b200 as hawk
    a = wl.make_attn_inputs(cfg, seed)
    args = (bf16_to_torch(a["q"]), bf16_to_torch(a["k_cache"]), bf16_to_torch(a["v_cache"]), to_dev(a["prefix_len"]),
            cfg.L, float(a["sm_scale"]))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with binding.alternate_library(stall_lib):
        hawk.verify_attn(*args, dev_status=status)
        torch.cuda.synchronize()
    assert int(status.item()) & binding.DEV_TIMEOUT, "the stalled stage must be reported"
    # the context is intact: the regular library gives the oracle's result on the same inputs
    status.zero_()
    out = hawk.verify_attn(*args, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = oracle.verify_attn(a["q"], a["k_cache"], a["v_cache"], a["prefix_len"], a["sm_scale"])
    got = torch_bf16_to_f64(out)
    rms = np.sqrt((want ** 2).mean())
    assert (np.abs(got - want) <= 2e-2 * np.abs(want) + 1e-2 * rms).all()


@pytest.mark.parametrize("name,overrides", [
    ("equal shares and merge kernel", dict(B=8, K=6, H=24, H_kv=24, L=1144)),       # 384 items cut into shares
    ("item merged inside a block", dict(B=8, K=5, H=20, H_kv=20, L=1144)),           # 320 long items of 8 rows
    ("one warp per item", dict(B=4, K=5, H=8, H_kv=8, L=120)),                       # short prefix, nothing cut
])
def test_attention_wait_runs_out(name, overrides, stall_lib):
    _attn_case(wl.config(2, **overrides), 8100 + len(name), stall_lib)


def _head_case(M, hidden, V, seed, stall_lib, guided_pairs=0):
    import paper_2510_25739_b200 as hawk
    rng = np.random.default_rng(seed)
    x = wl.f32_to_bf16_bits(rng.standard_normal((M, hidden)).astype(np.float32))
    w = wl.f32_to_bf16_bits((rng.standard_normal((V, hidden)) * 0.02).astype(np.float32))
    xt, wt = bf16_to_torch(x), bf16_to_torch(w)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    logits = torch.zeros((M, V), dtype=torch.float32, device="cuda")
    with binding.alternate_library(stall_lib):
        hawk.head_proj(xt, wt, 0, V, logits=logits, dev_status=status)
        torch.cuda.synchronize()
    assert int(status.item()) & binding.DEV_TIMEOUT
    status.zero_()
    hawk.head_proj(xt, wt, 0, V, logits=logits, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = oracle.head_proj(x, w).astype(np.float64)
    got = logits.cpu().numpy().astype(np.float64)
    rms = np.sqrt((want ** 2).mean())
    assert (np.abs(got - want) <= 1e-5 * np.abs(want) + 1e-5 * rms).all()


@pytest.mark.parametrize("name,M,hidden,V", [
    ("one block per tile", 80, 512, 4096),
    ("tiles split along hidden", 48, 2048, 2048),
    ("pairs of blocks, 256-id tiles", 640, 256, 2048),
    ("pairs of blocks, one wide tile", 384, 256, 1024),
])
def test_head_wait_runs_out(name, M, hidden, V, stall_lib):
    _head_case(M, hidden, V, 8200 + M, stall_lib)


def test_guided_head_wait_runs_out(stall_lib):
    import paper_2510_25739_b200 as hawk
    B, K, hidden, V = 4, 5, 512, 2048
    rng = np.random.default_rng(8300)
    x = wl.f32_to_bf16_bits(rng.standard_normal((2 * B, K, hidden)).astype(np.float32))
    w = wl.f32_to_bf16_bits((rng.standard_normal((V, hidden)) * 0.02).astype(np.float32))
    xt, wt = bf16_to_torch(x), bf16_to_torch(w)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    with binding.alternate_library(stall_lib):
        hawk.head_proj_cfg(xt, wt, 3.0, 1.0, dev_status=status)
        torch.cuda.synchronize()
    assert int(status.item()) & binding.DEV_TIMEOUT
    status.zero_()
    got = hawk.head_proj_cfg(xt, wt, 3.0, 1.0, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = oracle.head_proj_cfg(x, w, 3.0, 1.0).astype(np.float64)
    g = got.cpu().numpy().astype(np.float64)
    rms = np.sqrt((want ** 2).mean())
    assert (np.abs(g - want) <= 1e-4 * np.abs(want) + 1e-4 * rms).all()   # guided = lu + 3 (lc - lu): errors of both logits, scaled
