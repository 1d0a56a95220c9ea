"""Host logic of the data-parallel path: two gloo ranks on CPU each verify their shard of the
sequences (with the oracle standing in for the device), gather, and must reproduce the unsharded result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2510_25739_b200 import sharding
from paper_2510_25739_b200 import workloads as wl


def test_sequence_ranges_cover_the_batch_once():
    for B in (0, 1, 2, 7, 8, 64, 65):
        for world in (1, 2, 3, 8):
            spans = [sharding.sequence_range(B, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.sequence_range(4, 2, 2)


def test_stream_rows_keep_both_streams_of_a_sequence_together():
    rows = sharding.stream_rows(8, 2, 5)
    assert rows.tolist() == [2, 3, 4, 10, 11, 12]


def _inputs(cfg, seed):
    a = wl.make_attn_inputs(cfg, seed, ragged=True)
    logits = wl.make_logits(cfg, seed)
    q = wl.random_probs(cfg, seed).astype(np.float32)
    u = wl.draw_uniforms(cfg, seed)
    return dict(q=a["q"], k_cache=a["k_cache"], v_cache=a["v_cache"], prefix_len=a["prefix_len"], logits=logits,
                q_probs=q, draft=wl.draw_drafts(q, seed), u_accept=u["u_accept"], u_resample=u["u_resample"],
                x=wl.make_head_inputs(cfg, seed)["x"], sm_scale=a["sm_scale"])


def _verify(cfg, d):
    attn = oracle.verify_attn(d["q"], d["k_cache"], d["v_cache"], d["prefix_len"], d["sm_scale"])
    r = oracle.cfg_accept(d["logits"], d["q_probs"], d["draft"], d["u_accept"], d["u_resample"], cfg.v_begin,
                          cfg.v_end, cfg.cfg_scale, cfg.temperature, cfg.top_k, diagnostics=False)
    return attn, r["accept_len"], r["token"]


def _worker(rank, world, port, B, ret):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = wl.config(1, B=B, K=3, H=2, H_kv=2, L=40, V=512, v_end=512, top_k=50)
        full = _inputs(cfg, 11)
        mine = sharding.shard_step_inputs(full, B, world, rank)
        b0, b1 = sharding.sequence_range(B, world, rank)
        assert mine["q"].shape[0] == 2 * (b1 - b0) and mine["x"].shape[0] == 2 * (b1 - b0) * cfg.K
        attn, alen, tok = _verify(cfg, mine)
        lens, toks = sharding.gather_results(torch.from_numpy(alen), torch.from_numpy(tok), B)
        want_attn, want_len, want_tok = _verify(cfg, full)
        ok = (lens.numpy() == want_len).all() and (toks.numpy() == want_tok).all()
        ok = ok and np.array_equal(attn, want_attn[sharding.stream_rows(B, b0, b1)])
        ret[rank] = bool(ok)
    finally:
        dist.destroy_process_group()


def test_two_ranks_reproduce_the_unsharded_step():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    oracle.build()
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        ret = m.dict()
        procs = [ctx.Process(target=_worker, args=(r, 2, port, 5, ret)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        assert dict(ret) == {0: True, 1: True}
