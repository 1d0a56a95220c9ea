#!/usr/bin/env python
"""Benchmark of the verify step (attention -> head projection -> CFG accept) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

One "step" is one pass of the whole verify path over one batch of synthetic inputs.  Without --config the
headline is workload 5 (acceptance stress: the largest of the five that fit one GPU) and the line also carries a
`per_config` table of all five workloads; --config C measures workload C alone.  Rank 0 prints ONE JSON line.

* value            verified draft positions per second, inputs resident in HBM, whole job (all ranks);
                   each step is a CUDA-graph replay of the three C-ABI calls.
* e2e              same metric through hawk_verify_step_host: pinned host buffers, host->device
                   copies of the step's inputs and device->host copy of the results inside the
                   timed region.
* roofline         the kernel with the largest share of the step, timed alone with CUDA events on the bench stream.
* per_config       for workloads 1..5: step time, positions/s, per-kernel mean / median / min microseconds and each
                   kernel's fraction of the roofline that bounds it (HBM for attention, accept and the head at few
                   token rows; tensor for the head at many).
* cpu_baseline     the CPU oracle timed on the host cores on a bounded sample (rank 0, N=1 only), all cores and once
                   single-threaded.
* --impl reference times that same oracle as the reference arm.

Inputs rotate over enough replicas that consecutive steps never find their data in L2.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from dataclasses import replace
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

from paper_2510_25739_b200 import workloads as wl  # noqa: E402

METRIC = "verified draft positions/sec per B200 (verify step)"
HEADLINE_CONFIG = 5            # the largest of the five workloads that fits one GPU
UNIT = "positions/s"
L2_BYTES = 126 * 1024 * 1024


NOMINAL_HBM_GBS = 7700.0       # HBM3e figure of the HGX B200 data sheet
NOMINAL_BF16_TFLOPS = 2250.0   # dense bf16
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one hawk_verify_attn call, attention kernel
# plus merge kernel, from the ncu captures summarised in profiles/ (not measured by this script); an entry is
# dropped when the attention kernels change and no new capture exists.
ATTN_TRAFFIC_BYTES = {2: 94_543_000 + 3_216_000,                 # attention kernel read + write (no merge kernel at this shape)
                      4: 317_123_000 + 3_759_000,               # the same at the 7B shape
                      5: 679_410_000 + 4_565_000 + 4_757_000}   # attention read + write, merge kernel read


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------------ bytes / flops
def attn_bytes(cfg) -> int:
    """Algorithmic HBM bytes of one attention launch: K and V rows every query can see, plus Q and O."""
    kv = cfg.S * cfg.H_kv * (cfg.L + cfg.K) * cfg.D * 2 * 2
    qo = 2 * cfg.S * cfg.K * cfg.H * cfg.D * 2
    return kv + qo


def head_bytes(cfg) -> int:
    return cfg.V_valid * cfg.hidden * 2 + cfg.M * cfg.hidden * 2 + cfg.M * cfg.V_valid * 4


def head_flops(cfg) -> int:
    return 2 * cfg.M * cfg.hidden * cfg.V_valid


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, uuid: str = "", period_s: float = 0.01):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = None
            if uuid:
                try:
                    self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
                except Exception:
                    self.h = None
            if self.h is None:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _once(self):
        nv = self.nv
        self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
        try:
            r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
        except Exception:
            r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
        names = {
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        for k, bit in names.items():
            if r & bit:
                self.reasons.add(k)

    def _run(self):
        while not self._stop.is_set():
            try:
                self._once()
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.nv is None:
            return
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self):
        if self._thread:
            self._stop.set()
            self._thread.join()
            self._thread = None
            self._stop.clear()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------ inputs
def synth_q(cfg, x, w, gen, torch):
    """Draft probabilities q = a*p + (1-a)*r for the bench (input synthesis with library ops only).

    p is the target distribution of the logits the head will produce for these x and w (matmul, top-k
    threshold and softmax by torch), r a random dense distribution over the valid ids.
    """
    lg = (x.float() @ w[cfg.v_begin:cfg.v_end].float().t()).view(cfg.S, cfg.K, cfg.V_valid)
    g = torch.addcmul(lg[cfg.B:], lg[:cfg.B] - lg[cfg.B:], torch.tensor(cfg.cfg_scale, device=x.device))
    g = g / cfg.temperature
    if 0 < cfg.top_k < cfg.V_valid:
        tau = torch.topk(g, cfg.top_k, dim=-1).values[..., -1:]
        g = torch.where(g >= tau, g, torch.full_like(g, float("-inf")))
    p = torch.softmax(g.double(), dim=-1)
    r = torch.softmax(torch.randn(p.shape, generator=gen, device=x.device, dtype=torch.float64), dim=-1)
    if cfg.q_recipe == "own":
        qv = r
    elif cfg.q_recipe == "mix_row_uniform":
        a = 0.3 + 0.65 * torch.rand((cfg.B, cfg.K, 1), generator=gen, device=x.device, dtype=torch.float64)
        qv = a * p + (1 - a) * r
    else:
        qv = cfg.q_alpha * p + (1 - cfg.q_alpha) * r
    q = torch.zeros((cfg.B, cfg.K, cfg.V), dtype=torch.float32, device=x.device)
    q[..., cfg.v_begin:cfg.v_end] = qv.float()
    draft = torch.multinomial(qv.view(-1, cfg.V_valid).float(), 1, generator=gen).view(cfg.B, cfg.K) + cfg.v_begin
    return q, draft.int()


class Replica:
    """Device-resident inputs, intermediates and outputs of one step."""

    def __init__(self, cfg, seed, torch, hawk):
        dev = torch.device("cuda")
        gen = torch.Generator(device=dev)
        gen.manual_seed(seed)
        S, K, H, Hkv, D, Lc = cfg.S, cfg.K, cfg.H, cfg.H_kv, cfg.D, cfg.L_cap
        bf = torch.bfloat16
        self.q = torch.randn((S, K, H, D), generator=gen, device=dev).to(bf)
        self.k_cache = torch.randn((S, Hkv, Lc, D), generator=gen, device=dev).to(bf)
        self.v_cache = torch.randn((S, Hkv, Lc, D), generator=gen, device=dev).to(bf)
        self.prefix_len = torch.full((S,), cfg.L, dtype=torch.int32, device=dev)
        self.x = torch.randn((cfg.M, cfg.hidden), generator=gen, device=dev).to(bf)
        self.w = (0.02 * torch.randn((cfg.V, cfg.hidden), generator=gen, device=dev)).to(bf)
        self.q_probs, self.draft = synth_q(cfg, self.x, self.w, gen, torch)
        self.u_accept = torch.rand((cfg.B, K), generator=gen, device=dev)
        self.u_resample = torch.rand((cfg.B, K + 1), generator=gen, device=dev)
        self.attn_out = torch.empty((S, K, H * D), dtype=bf, device=dev)
        self.logits = torch.zeros((cfg.M, cfg.V), dtype=torch.float32, device=dev)
        self.accept_len = torch.empty(cfg.B, dtype=torch.int32, device=dev)
        self.out_token = torch.empty(cfg.B, dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        ws = hawk.verify_attn_workspace_bytes(S, K, H, Hkv, D, cfg.L)
        self.attn_ws = torch.empty(max(ws, 16), dtype=torch.uint8, device=dev)
        self.attn_split = ws > 0
        self.acc_ws = torch.empty(max(hawk.cfg_accept_workspace_bytes(cfg.B, K, cfg.V), 16), dtype=torch.uint8,
                                  device=dev)
        self.sm_scale = 1.0 / float(np.sqrt(D))

    def bytes(self) -> int:
        ts = (self.q, self.k_cache, self.v_cache, self.x, self.w, self.q_probs, self.logits)
        return sum(t.numel() * t.element_size() for t in ts)


def run_attn(cfg, r, hawk):
    hawk.verify_attn(r.q, r.k_cache, r.v_cache, r.prefix_len, cfg.L, r.sm_scale, out=r.attn_out,
                     workspace=r.attn_ws, dev_status=r.status)


def run_head(cfg, r, hawk):
    hawk.head_proj(r.x, r.w, cfg.v_begin, cfg.v_end, logits=r.logits, dev_status=r.status)


def run_accept(cfg, r, hawk):
    hawk.cfg_accept(r.logits.view(cfg.S, cfg.K, cfg.V), r.q_probs, r.draft, r.u_accept, r.u_resample, cfg.v_begin,
                    cfg.v_end, cfg.cfg_scale, cfg.temperature, cfg.top_k, accept_len=r.accept_len,
                    out_token=r.out_token, workspace=r.acc_ws, dev_status=r.status)


def run_head_cfg(cfg, r, hawk):
    hawk.head_proj_cfg(r.x.view(cfg.S, cfg.K, cfg.hidden), r.w, cfg.cfg_scale, cfg.temperature, cfg.v_begin, cfg.v_end,
                       guided=r.guided, dev_status=r.status)


def run_accept_guided(cfg, r, hawk):
    hawk.cfg_accept_guided(r.guided, r.q_probs, r.draft, r.u_accept, r.u_resample, cfg.v_begin, cfg.v_end, cfg.top_k,
                           accept_len=r.accept_len2, out_token=r.out_token2, workspace=r.acc_ws, dev_status=r.status)


# ------------------------------------------------------------------------------------------ CPU oracle leg
def oracle_sample(cfg, seed, reps, threads=None):
    """Times the CPU oracle (as it stands) on `reps` full steps of `cfg`; returns (positions/s, seconds, threads)."""
    import oracle
    a = wl.make_attn_inputs(cfg, seed)
    h = wl.make_head_inputs(cfg, seed)
    q = wl.make_q(replace(cfg, q_recipe="own"), seed, None)   # timing only: any dense q will do
    drafts = wl.draw_drafts(q, seed)
    u = wl.draw_uniforms(cfg, seed)
    oracle.build()
    all_threads = oracle.threads()
    if threads is not None:
        oracle.set_threads(threads)
    try:
        t0 = time.perf_counter()
        for _ in range(reps):
            oracle.verify_attn(a["q"], a["k_cache"], a["v_cache"], a["prefix_len"], a["sm_scale"])
            lg = oracle.head_proj(h["x"], h["w"], cfg.v_begin, cfg.v_end, fill=0.0)
            oracle.cfg_accept(lg.reshape(cfg.S, cfg.K, cfg.V), q, drafts, u["u_accept"], u["u_resample"], cfg.v_begin,
                              cfg.v_end, cfg.cfg_scale, cfg.temperature, cfg.top_k, diagnostics=False)
        dt = time.perf_counter() - t0
        used = oracle.threads()
    finally:
        if threads is not None:
            oracle.set_threads(all_threads)
    return cfg.B * cfg.K * reps / dt, dt, used


def workload_name(cfg, cid):
    return (f"config {cid} ({cfg.name}): B={cfg.B} x2 CFG streams, K={cfg.K}, {cfg.H} heads x {cfg.D}, "
            f"hidden {cfg.hidden}, KV length {cfg.L}, vocab {cfg.V} ({cfg.V_valid} valid), "
            f"cfg {cfg.cfg_scale}, top-k {cfg.top_k}, T {cfg.temperature}")


def reference_arm(args, cfg, cid):
    """The CPU oracle as the reference arm: exactly --steps timed steps after --warmup untimed ones.  A step is the
    whole workload when that keeps the run within minutes, else the first sequences of it (a bounded sample)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    seed = wl.seed_for(cid)
    steps, warmup = max(args.steps, 1), max(args.warmup, 1)
    probe_B = min(cfg.B, 4)
    _, t_probe, cores = oracle_sample(replace(cfg, B=probe_B), seed, 1)    # also warms the build and the page cache
    _, t_probe, cores = oracle_sample(replace(cfg, B=probe_B), seed, 1)
    per_seq = t_probe / probe_B
    budget_s = 150.0
    B_step = int(max(1, min(cfg.B, budget_s / ((steps + warmup) * per_seq))))
    scfg = replace(cfg, B=B_step)
    oracle_sample(scfg, seed, warmup)
    v, total, cores = oracle_sample(scfg, seed, steps)
    sample = (f"{steps} full steps of the workload" if B_step == cfg.B else
              f"{steps} steps of the first {B_step} of {cfg.B} sequences of the workload (all {cfg.K} positions, both streams)")
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": 1e3 * total / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg, cid), "note": "CPU oracle; " + sample},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------ timing helpers
def time_graph(torch, stream, body, launches_per_replay, samples, warm=3, min_launches=32):
    """Captures `body()` into one CUDA graph; a sample is the graph replayed back to back until it covers at least
    `min_launches` launches (so that the event records between samples are amortised), bracketed by its own events
    on `stream`.  Returns the list of microseconds per launch, one entry per sample."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        body()
    for _ in range(warm):
        g.replay()
    stream.synchronize()
    m = max(1, -(-min_launches // launches_per_replay))
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(samples + 1)]
    evs[0].record(stream)
    for i in range(samples):
        for _ in range(m):
            g.replay()
        evs[i + 1].record(stream)
    stream.synchronize()
    return [evs[i].elapsed_time(evs[i + 1]) * 1e3 / (m * launches_per_replay) for i in range(samples)]


def stats(us_list):
    return {"us": statistics.mean(us_list), "us_median": statistics.median(us_list), "us_min": min(us_list),
            "samples": len(us_list)}


def accept_traffic_model(cfg, accept_len):
    """Bytes of the accept stage from the verdicts of one step (accept_len: int tensor [B] on the host).

    definition : both logit rows of every position, plus the q row of each sequence's first rejection (the rows
                 the stage's definition needs when every position is examined);
    chain      : only the positions a sequential chain would look at (up to and including the first rejection),
                 plus the same q rows — the least any schedule can read.
    """
    row = cfg.V_valid * 4
    rejecting = int((accept_len < cfg.K).sum())
    examined = int(np.minimum(accept_len + 1, cfg.K).sum())
    return {"definition": 2 * cfg.B * cfg.K * row + rejecting * row, "chain": 2 * examined * row + rejecting * row,
            "rejecting_sequences": rejecting, "positions_on_chain": examined}


# DRAM bytes of one hawk_cfg_accept call from the ncu captures summarised in profiles/ (rows kernel, read + write;
# at workload 5 the figure depends on how many rows see an earlier rejection in time: 33 to 38 MB in two launches)
ACCEPT_TRAFFIC_BYTES = {2: 6_066_000, 4: 1_877_000, 5: 35_968_000}


def launches_per_step(cfg, first, sms):
    """Kernels one verify step launches: attention (+ its merge kernel when items are cut), head, accept rows +
    per-sequence pass (+ a marking kernel from 1.5 waves of rows on)."""
    accept_marks = cfg.B * cfg.K > sms + sms // 2
    return (2 if first.attn_split else 1) + 1 + (3 if accept_marks else 2)


def run_config(cid, args, torch, hawk, binding, world, rank, local_rank, dist, headline):
    """Measures one workload: the step (CUDA-graph replay of the three calls over rotating replicas), each kernel
    alone, the two-call form, and — for the headline workload — the extras and the end-to-end call."""
    cfg = wl.config(cid)
    peaks = measured_peaks()
    W = max(args.warmup, 3)
    K_steps = max(args.steps, 1) if headline else max(20, min(args.steps, 300))
    sms = torch.cuda.get_device_properties(local_rank).multi_processor_count

    # ---- replicas: enough bytes that a step never finds its inputs in L2
    first = Replica(cfg, 1000 * cid + 17 * rank, torch, hawk)
    n_rep = max(2, -(-3 * L2_BYTES // first.bytes()))
    n_rep = min(n_rep, 64)
    reps = [first] + [Replica(cfg, 1000 * cid + 17 * rank + 101 * i, torch, hawk) for i in range(1, n_rep)]
    stream = torch.cuda.Stream()
    n_launch = launches_per_step(cfg, first, sms)

    graphs = []
    with torch.cuda.stream(stream):
        for r in reps:                       # warm the kernels (function attributes are set on first use)
            run_attn(cfg, r, hawk); run_head(cfg, r, hawk); run_accept(cfg, r, hawk)
        stream.synchronize()
        for r in reps:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                run_attn(cfg, r, hawk)
                run_head(cfg, r, hawk)
                run_accept(cfg, r, hawk)
            graphs.append(g)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(local_rank).uuid)
    except Exception:
        uuid = ""
    sampler = ClockSampler(local_rank, uuid) if headline else None
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        for i in range(W):
            graphs[i % n_rep].replay()
        barrier()
        if sampler:
            sampler.start()
        start.record(stream)
        for i in range(K_steps):
            graphs[i % n_rep].replay()
        stop.record(stream)
        barrier()
    elapsed_ms = start.elapsed_time(stop)
    if dist is not None:
        t = torch.tensor([elapsed_ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        elapsed_ms = float(t.item())
    ms_per_step = elapsed_ms / K_steps
    positions = cfg.B * cfg.K
    value = positions * world / (ms_per_step * 1e-3)
    status = int(sum(int(r.status.item()) for r in reps))

    # ---- each kernel alone: one CUDA graph holding the call for every replica (L2-cold), every replay timed with its
    # own events on the bench stream (issuing the launches of a call one by one from Python costs more host time
    # than the call takes on the device); the clock sampler keeps running so that these loops are covered too
    n_samples = max(5, min(30, K_steps // 4 + 1))
    kern, warm = {}, {}
    with torch.cuda.stream(stream):
        for name, fn in (("attn", run_attn), ("head", run_head), ("accept", run_accept)):
            kern[name] = stats(time_graph(torch, stream, lambda: [fn(cfg, r, hawk) for r in reps], n_rep, n_samples))
            # the same call with ONE replica repeated: inputs L2-warm where they fit (labelled as such)
            warm[name] = statistics.median(time_graph(torch, stream, lambda: [fn(cfg, first, hawk) for _ in range(4)],
                                                      4, 10))
        if cfg.V_valid < cfg.V:        # the head over ALL columns where only part of the vocabulary is valid
            full_logits = torch.zeros((cfg.M, cfg.V), dtype=torch.float32, device="cuda")
            kern["head_full_vocab"] = stats(time_graph(
                torch, stream, lambda: [hawk.head_proj(r.x, r.w, 0, cfg.V, logits=full_logits, dev_status=r.status)
                                        for r in reps], n_rep, 10))
            del full_logits
    if sampler:
        sampler.stop()

    # ---- the two-call form: guidance combined in the head's epilogue, accept reads one guided row per position
    for r in reps:
        r.guided = torch.zeros((cfg.B, cfg.K, cfg.V), dtype=torch.float32, device="cuda")
        r.accept_len2 = torch.empty_like(r.accept_len)
        r.out_token2 = torch.empty_like(r.out_token)
    with torch.cuda.stream(stream):
        for r in reps:
            run_head_cfg(cfg, r, hawk); run_accept_guided(cfg, r, hawk)
        stream.synchronize()
        for name, fn in (("head_cfg", run_head_cfg), ("accept_guided", run_accept_guided)):
            kern[name] = stats(time_graph(torch, stream, lambda: [fn(cfg, r, hawk) for r in reps], n_rep, n_samples))
        graphs2 = []
        for r in reps:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                run_attn(cfg, r, hawk)
                run_head_cfg(cfg, r, hawk)
                run_accept_guided(cfg, r, hawk)
            graphs2.append(g)
        for i in range(W):
            graphs2[i % n_rep].replay()
        stream.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        for i in range(K_steps):
            graphs2[i % n_rep].replay()
        a1.record(stream)
        stream.synchronize()
        us_step2 = a0.elapsed_time(a1) * 1e3 / K_steps
    same = all(bool(torch.equal(r.accept_len, r.accept_len2)) and bool(torch.equal(r.out_token, r.out_token2))
               for r in reps)

    # ---- bytes, flops, fractions
    hbm, tens = peaks["hbm_gbs"], peaks["bf16_tflops"]
    models = [accept_traffic_model(cfg, r.accept_len.cpu().numpy()) for r in reps]
    acc_def = sum(m["definition"] for m in models) / n_rep
    acc_chain = sum(m["chain"] for m in models) / n_rep
    mean_len = float(sum(float(r.accept_len.float().mean().item()) for r in reps) / n_rep)
    head_tensor_bound = head_flops(cfg) / (tens * 1e12) > head_bytes(cfg) / (hbm * 1e9)

    def hbm_leg(st, nbytes):
        return {**st, "bytes": nbytes, "GB/s": nbytes / st["us"] / 1e3, "frac_hbm": nbytes / st["us"] / 1e3 / hbm,
                "frac_hbm_best": nbytes / st["us_min"] / 1e3 / hbm,
                "frac_hbm_nominal": nbytes / st["us"] / 1e3 / NOMINAL_HBM_GBS}

    attn = {**hbm_leg(kern["attn"], attn_bytes(cfg)), "bound": "hbm", "frac": None,
            "us_one_replica_l2_warm": warm["attn"]}
    attn["frac"] = attn["frac_hbm"]
    head = {**hbm_leg(kern["head"], head_bytes(cfg)), "flops": head_flops(cfg),
            "TFLOP/s": head_flops(cfg) / kern["head"]["us"] / 1e6,
            "frac_tensor": head_flops(cfg) / kern["head"]["us"] / 1e6 / tens,
            "frac_tensor_sustained_peak": head_flops(cfg) / kern["head"]["us"] / 1e6 / peaks["bf16_tflops_sustained"],
            "frac_tensor_nominal": head_flops(cfg) / kern["head"]["us"] / 1e6 / NOMINAL_BF16_TFLOPS,
            "bound": "tensor" if head_tensor_bound else "hbm", "us_one_replica_l2_warm": warm["head"]}
    head["frac"] = head["frac_tensor"] if head_tensor_bound else head["frac_hbm"]
    accept = {**hbm_leg(kern["accept"], acc_def), "bound": "hbm", "us_one_replica_l2_warm": warm["accept"],
              "bytes_counted": "both logit rows of every position + the q row of each sequence's first rejection",
              "bytes_chain": acc_chain, "frac_hbm_chain_bytes": acc_chain / kern["accept"]["us"] / 1e3 / hbm,
              "bytes_chain_counted": "only positions up to and including each sequence's first rejection (the least "
                                     "any schedule reads); rows behind a rejection may or may not be read",
              "dram_bytes_ncu": ACCEPT_TRAFFIC_BYTES.get(cid),
              "dram_bytes_ncu_source": "profiles/ (not measured in this run)" if cid in ACCEPT_TRAFFIC_BYTES else None}
    accept["frac"] = accept["frac_hbm"]
    floor_us = (attn_bytes(cfg) / hbm + max(head_bytes(cfg) / hbm, head_flops(cfg) / tens / 1e3) + acc_def / hbm) / 1e3
    stage = {
        "attn": attn, "head": head, "accept": accept, "mean_accept_len": mean_len,
        "sequences_with_rejection": sum(m["rejecting_sequences"] for m in models) / n_rep,
        "positions_on_chain": sum(m["positions_on_chain"] for m in models) / n_rep,
        "step_floor_us": floor_us, "step_frac_of_floor": floor_us / (ms_per_step * 1e3),
        **({"head_full_vocab": {
            **kern["head_full_vocab"], "columns": cfg.V,
            "TFLOP/s": 2.0 * cfg.M * cfg.hidden * cfg.V / kern["head_full_vocab"]["us"] / 1e6,
            "frac_hbm": (cfg.V * cfg.hidden * 2 + cfg.M * cfg.hidden * 2 + cfg.M * cfg.V * 4)
                        / kern["head_full_vocab"]["us"] / 1e3 / hbm}} if "head_full_vocab" in kern else {}),
        "two_call_form": {
            "what": "hawk_head_proj_cfg + hawk_cfg_accept_guided: one guided logits row per position crosses HBM",
            "head_cfg": kern["head_cfg"], "accept_guided": kern["accept_guided"],
            "step_us": us_step2, "positions_per_s": positions * world / (us_step2 * 1e-6),
            "same_verdicts_as_three_calls": same},
    }
    seed = 1000 * cid + 17 * rank
    stage["tree_attn"] = bench_tree_attn(cfg, stream, torch, hawk, peaks, seed)
    stage["tree_accept"] = bench_tree(cfg, stream, torch, hawk, peaks, seed)
    if headline or cid == 2:
        stage["pool"] = bench_pool(cfg, stream, torch, hawk, peaks, seed)
    if cid == 2:   # the LlamaGen-XL-shaped workload sweeps the KV length over the image: 120 .. 1144
        stage["attn_kv_sweep"] = {str(L): bench_tree_attn(replace(cfg, L=L), stream, torch, hawk, peaks,
                                                          1000 * cid + L, branching=None)
                                  for L in wl.XL_PREFIX_SWEEP}
    e2e = None
    if headline and not args.no_e2e:
        e2e = bench_e2e(cfg, reps, stream, torch, hawk, binding, world, dist, min(K_steps, 500), W,
                        eager=args.e2e_eager)
    out = {"cid": cid, "cfg": cfg, "value": value, "ms_per_step": ms_per_step, "steps": K_steps, "warmup": W,
           "positions": positions, "n_rep": n_rep, "replica_bytes": first.bytes(), "launches_per_step": n_launch,
           "kernels": stage, "status": status, "e2e": e2e, "clocks": sampler.summary() if sampler else None}
    del graphs, graphs2, reps, first
    torch.cuda.empty_cache()
    return out


def compact(res):
    """One workload's entry of `per_config`: the step, the three kernels (mean / median / min microseconds) and each
    kernel's fraction of the roofline that bounds it."""
    k = res["kernels"]

    def leg(d, keys):
        return {key: d[key] for key in keys if key in d}

    kk = ("us", "us_median", "us_min", "bound", "frac", "frac_hbm", "frac_tensor", "bytes", "flops", "frac_hbm_chain_bytes")
    return {"workload": workload_name(res["cfg"], res["cid"]), "step_us": res["ms_per_step"] * 1e3, "steps": res["steps"],
            "positions_per_s": res["value"], "attn": leg(k["attn"], kk), "head": leg(k["head"], kk),
            "accept": leg(k["accept"], kk), "step_floor_us": k["step_floor_us"],
            "step_frac_of_floor": k["step_frac_of_floor"], "mean_accept_len": k["mean_accept_len"],
            "two_call_step_us": k["two_call_form"]["step_us"],
            "same_verdicts_as_three_calls": k["two_call_form"]["same_verdicts_as_three_calls"],
            "tree_attn": leg(k["tree_attn"], ("us", "frac_hbm")), "tree_accept": leg(k["tree_accept"], ("us", "frac_hbm")),
            "dev_status": res["status"]}


# ------------------------------------------------------------------------------------------ main arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=0,
                    help="workload id 1..5; default: headline on workload 5 (the largest) plus a per_config table of all five")
    ap.add_argument("--impl", default="hawk", choices=["hawk", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--e2e-eager", action="store_true", help="time the end-to-end call eagerly instead of as a graph")
    args = ap.parse_args()
    cid = args.config if args.config else HEADLINE_CONFIG
    cfg = wl.config(cid)
    if args.impl == "reference":
        reference_arm(args, cfg, cid)
        return

    import torch
    import paper_2510_25739_b200 as hawk
    from paper_2510_25739_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    hawk.load_library()

    res = run_config(cid, args, torch, hawk, binding, world, rank, local_rank, dist, headline=True)
    peaks = measured_peaks()
    k = res["kernels"]
    # the dominant kernel of the step: whichever of the three calls takes the largest share of it
    dom = max(("attn", "head", "accept"), key=lambda n: k[n]["us"])
    d = k[dom]
    if d["bound"] == "tensor":
        roofline = {"kernel": "hawk_head_proj", "bound": "tensor", "achieved": d["TFLOP/s"], "peak": peaks["bf16_tflops"],
                    "unit": "TFLOP/s", "frac": d["frac_tensor"], "algorithmic_flops": d["flops"], "traffic": None}
    else:
        name = {"attn": "hawk_verify_attn", "head": "hawk_head_proj", "accept": "hawk_cfg_accept"}[dom]
        traffic = ATTN_TRAFFIC_BYTES.get(cid) if dom == "attn" else None
        roofline = {"kernel": name, "bound": "hbm", "achieved": d["GB/s"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": d["frac_hbm"], "algorithmic_bytes": d["bytes"], "traffic": traffic,
                    "traffic_source": ("ncu capture summarised in profiles/ (dram read + write of one call; not "
                                       "measured in this run)") if traffic else None}
    roofline.update({"peak_source": f"of {peaks['source']}", "us_per_launch": d["us"], "us_per_launch_median": d["us_median"],
                     "us_per_launch_min": d["us_min"], "share_of_step": d["us"] / (res["ms_per_step"] * 1e3),
                     "timing": "CUDA graph of the call over the rotating replicas (L2-cold), every replay bracketed by "
                               "events on the bench stream"})

    per_config = None
    if world == 1 and not args.config and not args.no_per_config:
        per_config = {}
        for c in (1, 2, 3, 4, 5):
            per_config[str(c)] = compact(res if c == cid else
                                         run_config(c, args, torch, hawk, binding, world, rank, local_rank, dist, False))

    line = {
        "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": res["steps"],
        "warmup": res["warmup"], "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_name(cfg, cid), "positions_per_step_per_gpu": res["positions"],
                   "arithmetic": "bf16 operands (Q, K, V, X, W), fp32 accumulation, fp32 logits and accept stage",
                   "l2": f"inputs rotate over {res['n_rep']} replicas "
                         f"({res['n_rep'] * res['replica_bytes'] / 1e6:.0f} MB > 3x L2)",
                   "launch": "one CUDA graph replay per step (3 C-ABI calls captured)",
                   "parallelism": f"{world} independent replicas, sequences sharded, no collective"},
        "clocks": res["clocks"], "e2e": res["e2e"], "gpu_launches": res["launches_per_step"] * res["steps"],
        "roofline": roofline, "kernels": k, "dev_status": res["status"], "per_config": per_config,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        seed = wl.seed_for(cid)
        oracle_sample(replace(cfg, B=min(cfg.B, 2)), seed, 1)        # builds the oracle, warms the page cache
        _, t1, _ = oracle_sample(cfg, seed, 1)
        reps_cpu = max(1, min(2000, int(18.0 / max(t1, 1e-3))))      # 10 to 30 s of CPU work in all
        v, dt, cores = oracle_sample(cfg, seed, reps_cpu)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{reps_cpu} full steps of the workload ({dt:.1f} s)"}
        # once single-threaded, on a bounded sample: the first sequences of the workload (the oracle's cost is
        # linear in the number of sequences)
        B1 = max(1, min(cfg.B, int(cfg.B * 5.0 / max(t1 * cores, 1e-3))))
        v1, dt1, c1 = oracle_sample(replace(cfg, B=B1), seed, 1, threads=1)
        line["cpu_baseline"]["single_thread"] = {
            "value": v1, "unit": UNIT, "cores": c1,
            "sample": f"1 step of the first {B1} of {cfg.B} sequences of the workload ({dt1:.1f} s)"}
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def bench_tree(cfg, stream, torch, hawk, peaks, seed, branching=(3, 2, 2)):
    """Times hawk_tree_accept alone on random logits of the workload's vocabulary (replicas rotating)."""
    tree = wl.make_tree(branching)
    N, NQ, B = tree["N"], tree["NQ"], cfg.B
    dev = torch.device("cuda")
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed + 5)
    row_bytes = cfg.V_valid * 4
    n_rep = max(2, min(16, -(-3 * L2_BYTES // (2 * B * N * row_bytes))))
    std = 0.02 * float(np.sqrt(cfg.hidden))
    child_begin = torch.from_numpy(tree["child_begin"]).to(dev)
    node_q = torch.from_numpy(tree["node_q"]).to(dev)
    sets = []
    for _ in range(n_rep):
        logits = torch.full((2 * B, N, cfg.V), float("nan"), device=dev)
        logits[..., cfg.v_begin:cfg.v_end] = std * torch.randn((2 * B, N, cfg.V_valid), generator=gen, device=dev)
        g = torch.addcmul(logits[B:, 0, cfg.v_begin:cfg.v_end],
                          logits[:B, 0, cfg.v_begin:cfg.v_end] - logits[B:, 0, cfg.v_begin:cfg.v_end],
                          torch.tensor(cfg.cfg_scale, device=dev))
        p0 = torch.softmax(g.double(), dim=-1)[:, None, :]
        r = torch.softmax(torch.randn((B, NQ, cfg.V_valid), generator=gen, device=dev, dtype=torch.float64), dim=-1)
        qv = 0.7 * p0 + 0.3 * r
        q = torch.zeros((B, NQ, cfg.V), device=dev)
        q[..., cfg.v_begin:cfg.v_end] = qv.float()
        draw = torch.multinomial(qv.view(-1, cfg.V_valid).float(), 1, generator=gen).view(B, NQ) + cfg.v_begin
        tok = draw[:, node_q.long()].int().contiguous()
        ua = torch.rand((B, N), generator=gen, device=dev)
        ur = torch.rand((B, N), generator=gen, device=dev)
        sets.append((logits, q, tok, ua, ur))
    lens = []

    def run(t):
        a, _, _ = hawk.tree_accept(t[0], t[1], t[2], node_q, child_begin, t[3], t[4], cfg.v_begin, cfg.v_end,
                                   cfg.cfg_scale, cfg.temperature, cfg.top_k, max_depth=len(branching))
        return a

    with torch.cuda.stream(stream):
        for t in sets:
            lens.append(run(t))
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for t in sets:
                run(t)
        for _ in range(3):
            g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 20
        e0.record(stream)
        for _ in range(n):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (n * n_rep)
    nbytes = 2 * B * N * row_bytes
    return {"us": us, "tree": f"branching {branching}, {N} nodes, {NQ} draft rows per sequence", "rows": B * N,
            "logit_bytes": nbytes, "GB/s": nbytes / us / 1e3, "frac_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"],
            "mean_accept_len": float(torch.stack(lens).float().mean().item()),
            "timing": "graph of back-to-back calls, replicas rotating"}


def bench_pool(cfg, stream, torch, hawk, peaks, seed, IW=32, VSD=2, K=3, branching=(3, 2, 2)):
    """Times the drafting-side bookkeeping that feeds the tree verification: cache put, pool build, candidate draw
    (32 x 32 token image, two vertical depths, three horizontal offsets: the 9 draft rows of the (3, 2, 2) tree)."""
    tree = wl.make_tree(branching)
    B, N, NQ = cfg.B, tree["N"], K * (1 + VSD)
    assert tree["NQ"] == NQ
    dev = torch.device("cuda")
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed + 9)
    node_q = torch.from_numpy(tree["node_q"]).to(dev)
    row_bytes = cfg.V * 4
    n_rep = max(2, min(16, -(-3 * L2_BYTES // (2 * B * NQ * row_bytes))))

    def probs(rows):
        z = torch.zeros((B, rows, cfg.V), device=dev)
        z[..., cfg.v_begin:cfg.v_end] = torch.softmax(
            4.0 * torch.randn((B, rows, cfg.V_valid), generator=gen, device=dev), dim=-1)
        return z

    sets = [(probs(VSD), probs(K), torch.rand((B, NQ), generator=gen, device=dev)) for _ in range(n_rep)]
    rows, tags = hawk.spec_cache_new(B, IW, VSD, cfg.V)
    base = 2 * IW + 3
    with torch.cuda.stream(stream):
        for T in range(base + n_rep + 1):        # a step at every position so far: every lookup finds its row
            hawk.spec_cache_put(sets[T % n_rep][0], torch.full((B,), T, dtype=torch.int32, device=dev), rows, tags, IW)
        pos = [torch.full((B,), base + i, dtype=torch.int32, device=dev) for i in range(n_rep)]
        pools = [hawk.pool_build(sets[i][1], rows, tags, pos[i], IW, VSD)[0] for i in range(n_rep)]
        stream.synchronize()

        def timed(fn, n=50):
            """us per call: one CUDA graph holding the call for every replica, replayed n times."""
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for i in range(n_rep):
                    fn(i)
            for _ in range(3):
                g.replay()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(n):
                g.replay()
            e1.record(stream)
            stream.synchronize()
            return e0.elapsed_time(e1) * 1e3 / (n * n_rep)

        us_put = timed(lambda i: hawk.spec_cache_put(sets[i][0], pos[i], rows, tags, IW))
        us_build = timed(lambda i: hawk.pool_build(sets[i][1], rows, tags, pos[i], IW, VSD, with_source=False))
        us_sample = timed(lambda i: hawk.pool_sample(pools[i], sets[i][2], node_q, cfg.v_begin, cfg.v_end))
    b_put, b_build, b_sample = 2 * B * VSD * row_bytes, 2 * B * NQ * row_bytes, B * NQ * cfg.V_valid * 4
    leg = lambda us, nb: {"us": us, "bytes": nb, "GB/s": nb / us / 1e3, "frac_hbm": nb / us / 1e3 / peaks["hbm_gbs"]}
    return {"shape": f"IW {IW}, VSD {VSD}, K {K}: {NQ} pool rows and {N} tree nodes per sequence, "
                     f"cache {hawk.spec_cache_slots(IW, VSD)} rows per sequence",
            "cache_put": leg(us_put, b_put), "pool_build": leg(us_build, b_build),
            "pool_sample": leg(us_sample, b_sample),
            "timing": "each call alone in a CUDA graph over rotating replicas"}


def bench_tree_attn(cfg, stream, torch, hawk, peaks, seed, branching=(3, 2, 2)):
    """Times hawk_verify_attn_tree alone: the workload's KV shape with the 22 nodes of a (3, 2, 2) tree as queries."""
    if branching is None:      # the chain of K drafts (causal block) instead of a tree
        N, masks = cfg.K, None
    else:
        tree = wl.make_tree(branching)
        N = tree["N"]
        masks = torch.from_numpy(wl.tree_ancestor_masks(tree["child_begin"]).view(np.int64)).cuda()
    dev = torch.device("cuda")
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed + 9)
    S, H, Hkv, D, L = cfg.S, cfg.H, cfg.H_kv, cfg.D, cfg.L
    kv_bytes = 2 * S * Hkv * (L + N) * D * 2
    n_rep = max(2, min(8, -(-3 * L2_BYTES // kv_bytes)))
    bf = torch.bfloat16
    sets = []
    for _ in range(n_rep):
        q = torch.randn((S, N, H, D), generator=gen, device=dev).to(bf)
        kc = torch.randn((S, Hkv, L + N, D), generator=gen, device=dev).to(bf)
        vc = torch.randn((S, Hkv, L + N, D), generator=gen, device=dev).to(bf)
        sets.append((q, kc, vc, torch.empty((S, N, H * D), dtype=bf, device=dev)))
    pl = torch.full((S,), L, dtype=torch.int32, device=dev)
    ws = torch.empty(max(16, hawk.verify_attn_workspace_bytes(S, N, H, Hkv, D, L)), dtype=torch.uint8, device=dev)
    scale = 1.0 / float(np.sqrt(D))

    def run(t):
        hawk.verify_attn(t[0], t[1], t[2], pl, L, scale, out=t[3], workspace=ws, anc_mask=masks)

    with torch.cuda.stream(stream):
        for t in sets:
            run(t)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for t in sets:
                run(t)
        g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n = 30
        e0.record(stream)
        for _ in range(n):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (n * n_rep)
    nbytes = kv_bytes + 2 * S * N * H * D * 2
    return {"us": us, "queries": f"tree, branching {branching}, {N} nodes" if branching else f"chain of {N} drafts",
            "kv_length": L, "algorithmic_bytes": nbytes,
            "GB/s": nbytes / us / 1e3, "frac_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"],
            "timing": "graph of back-to-back calls, replicas rotating"}


def bench_e2e(cfg, reps, stream, torch, hawk, binding, world, dist, steps, warmup, eager=False):
    """Steps through hawk_verify_step_host with pinned host inputs; returns the e2e object."""
    import ctypes
    n_rep = len(reps)
    args_list, keep = [], []
    for r in reps:
        host = {k: getattr(r, k).cpu().pin_memory() for k in ("q", "x", "q_probs", "draft", "u_accept", "u_resample")}
        h_len = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
        h_tok = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
        a = binding.StepHostArgs()
        a.B, a.K, a.H, a.H_kv, a.D, a.L_cap = cfg.B, cfg.K, cfg.H, cfg.H_kv, cfg.D, cfg.L_cap
        a.max_prefix_len, a.V, a.v_begin, a.v_end, a.top_k = cfg.L, cfg.V, cfg.v_begin, cfg.v_end, cfg.top_k
        a.sm_scale, a.cfg_scale, a.temperature = r.sm_scale, cfg.cfg_scale, cfg.temperature
        a.h_q, a.h_x, a.h_q_probs = host["q"].data_ptr(), host["x"].data_ptr(), host["q_probs"].data_ptr()
        a.h_draft, a.h_u_accept, a.h_u_resample = (host["draft"].data_ptr(), host["u_accept"].data_ptr(),
                                                   host["u_resample"].data_ptr())
        a.h_accept_len, a.h_out_token = h_len.data_ptr(), h_tok.data_ptr()
        a.d_k_cache, a.d_v_cache, a.d_prefix_len, a.d_w = (r.k_cache.data_ptr(), r.v_cache.data_ptr(),
                                                           r.prefix_len.data_ptr(), r.w.data_ptr())
        a.d_q, a.d_x, a.d_q_probs, a.d_draft = r.q.data_ptr(), r.x.data_ptr(), r.q_probs.data_ptr(), r.draft.data_ptr()
        a.d_u_accept, a.d_u_resample = r.u_accept.data_ptr(), r.u_resample.data_ptr()
        a.d_attn_out, a.d_logits = r.attn_out.data_ptr(), r.logits.data_ptr()
        a.d_accept_len, a.d_out_token = r.accept_len.data_ptr(), r.out_token.data_ptr()
        a.d_attn_workspace, a.attn_workspace_bytes = r.attn_ws.data_ptr(), r.attn_ws.numel()
        a.d_accept_workspace, a.accept_workspace_bytes = r.acc_ws.data_ptr(), r.acc_ws.numel()
        a.d_status = r.status.data_ptr()
        args_list.append(a)
        keep.append((host, h_len, h_tok))
    h2d = sum(t.numel() * t.element_size() for t in keep[0][0].values())
    d2h = 2 * cfg.B * 4
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        for i in range(max(warmup, n_rep)):      # eager first: the library sets itself up outside any capture
            hawk.verify_step_host(args_list[i % n_rep])
        stream.synchronize()
        steps_fn, mode = None, "eager calls"
        if not eager:
            try:                                  # the same call captured once per replica, replayed per step
                graphs = []
                for a in args_list:
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        hawk.verify_step_host(a)
                    graphs.append(g)
                steps_fn, mode = (lambda i: graphs[i % n_rep].replay()), "one CUDA graph replay per step"
            except Exception as exc:              # capture refused: time the eager calls
                mode = f"eager calls (graph capture failed: {type(exc).__name__})"
        if steps_fn is None:
            steps_fn = lambda i: hawk.verify_step_host(args_list[i % n_rep])
        for i in range(warmup):
            steps_fn(i)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        start.record(stream)
        for i in range(steps):
            steps_fn(i)
        stop.record(stream)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
    ms = start.elapsed_time(stop)
    # the floor of such a step on this machine: the same host buffers copied to the same device buffers, nothing else
    with torch.cuda.stream(stream):
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_copy = max(5, min(steps, 50))
        pairs = [[(getattr(r, k), keep[j][0][k]) for k in ("q", "x", "q_probs", "draft", "u_accept", "u_resample")]
                 for j, r in enumerate(reps)]
        for dst, src in pairs[0]:
            dst.copy_(src, non_blocking=True)
        stream.synchronize()
        c0.record(stream)
        for it in range(n_copy):
            for dst, src in pairs[it % n_rep]:
                dst.copy_(src, non_blocking=True)
        c1.record(stream)
        stream.synchronize()
    copy_ms = c0.elapsed_time(c1) / n_copy
    if dist is not None:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return {"value": cfg.B * cfg.K * world / (ms / steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms / steps, "steps": steps,
            "h2d_GB/s": h2d / (ms / steps) / 1e6,
            "copy_floor_ms_per_step": copy_ms, "copy_floor_GB/s": h2d / copy_ms / 1e6,
            "step_over_copy_floor": (ms / steps) / copy_ms,
            "bound": "the host-to-device copy of the draft distributions (q_probs is most of the step's host bytes); "
                     "the kernels run under it on the caller's stream while it travels on the library's side stream",
            "api": "hawk_verify_step_host (pinned host inputs -> device, 3 kernels, results -> host)",
            "launch": mode}


if __name__ == "__main__":
    main()
