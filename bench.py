#!/usr/bin/env python
"""Benchmark of the KV swap + paged decode hot path on one B200 (or N independent replicas).

One "step" is one pass of the whole hot path over the Llama-3-8B-shaped workload (32 layers, 8 KV
heads, head_dim 128, bf16, block 16; 64 resident requests with 1k-4k contexts in fragmented block
tables; a seeded 16 of them are preempted):

  phase A  ps_swap_out of the 16 victims (gather kernels + device-to-host copies on the copy
           streams) while ps_step keeps decoding the 48 other requests, until every offload has
           been reaped and its blocks are back in the pool;
  phase B  ps_swap_in_begin of the 16, then ps_step with a per-step copy budget (layer-pipelined
           host-to-device copies + scatter kernels, attention of reloaded requests gated on the
           per-layer events) until all 64 decode again.

value = bytes moved over the host link (out + in) / time of the step, in GB/s.  The same run
reports each direction against the measured pinned-copy peak, the attention kernel against the HBM
roofline, the gather / scatter kernels against HBM, the budget sweep of the overlap workload
(decode batch 128, lognormal contexts, 8 reloading requests; hidden fraction of the reload), and the
CPU checker timed on the host cores.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-overlap]
  python bench.py --workload long_context | churn | decode_shapes   (other workloads, a line of their own)
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2512_12928_b200 import workloads as wl

METRIC = "swap-out/in GB/s vs host-link peak; decode+reload step us vs no-reload step"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1400.0


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return float(p["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def read_bf16_peak():
    """Dense bf16 TFLOP/s of a long-running GEMM: measured if the file is there, else the pool's earlier figure."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        if "bf16_tflops_sustained" in p:
            return float(p["bf16_tflops_sustained"]), "measured"
    return FALLBACK_BF16_TFLOPS, "fallback"


def kernel_code_sha256(path):
    """Hash of a CUDA source with comments and white space removed (a comment edit is not a kernel change)."""
    import hashlib
    import re
    text = open(path).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"//[^\n]*", "", text)
    text = re.sub(r"\s+", "", text)
    return hashlib.sha256(text.encode()).hexdigest()


def read_traffic_ratio():
    """DRAM bytes per algorithmic byte of the attention kernel from the committed ncu summary, or None when
    the kernel's code has changed since that capture (the counters then describe another kernel)."""
    import glob
    import re
    src = os.path.join(ROOT, "paper_2512_12928_b200", "csrc", "ps_attn_kernels.cu")
    try:
        sha = kernel_code_sha256(src)
    except OSError:
        return None
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "decode_attn_mma_*.md"))):
        text = open(path).read()
        m_sha = re.search(r"^kernel_code_sha256:\s*([0-9a-f]{64})", text, re.M)
        m_ratio = re.search(r"^dram_bytes_per_algorithmic_byte:\s*([0-9.]+)", text, re.M)
        if m_sha and m_ratio and m_sha.group(1) == sha:
            return float(m_ratio.group(1))
    return None


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.lines = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return

        def pump():
            for line in self.proc.stdout:
                self.lines.append(line.strip())
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# -------------------------------------------------------------------------------------------------
# CPU checker timing (the reference arm and the cpu_baseline leg; the only users of oracle/ here)
# -------------------------------------------------------------------------------------------------

def oracle_swap_pass(n_req: int = 4, ctx: int = 2048, seed: int = 0):
    """Builds a small Llama-8B-shaped checker instance; returns (callable doing one out+in pass, bytes per pass)."""
    from oracle import ps_oracle as po
    sh = wl.KVShape(32, 8, 32, 128, 16, n_req * (ctx // 16) + 64)
    rng = np.random.default_rng(seed)
    dims = (sh.num_layers, sh.num_gpu_blocks, sh.block_size, sh.num_kv_heads, sh.head_dim)
    K = wl.randn_bf16_bits(rng, dims)              # N(0,1) as bf16, like every other input
    V = wl.randn_bf16_bits(rng, dims)
    orc = po.PsOracle(sh.num_layers, sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size,
                      sh.num_gpu_blocks, rng.permutation(sh.num_gpu_blocks), K, V)
    grown = 0
    while grown < ctx:                     # interleaved growth: fragmented tables
        grown += sh.block_size
        for r in range(n_req):
            assert orc.kv_alloc(r, grown) == 0
    nbytes = 2 * n_req * sh.blocks_for(ctx) * sh.block_bytes

    def one_pass():
        for r in range(n_req):
            assert orc.swap_out(r) == 0
        orc.reap()
        for r in range(n_req):
            assert orc.swap_in_begin(r) == 0
        orc.step(-1)
    return one_pass, nbytes, orc, sh


def oracle_attention_step(step_layers: int, step_tokens: int, n_layers: int = 2, n_req: int = 8, ctx: int = 2048):
    """The checker's fp64 decode attention on n_layers x n_req requests of ctx tokens (8B KV shape, 32 query
    heads), and its linear extrapolation to a whole decode step of step_layers layers over step_tokens KV tokens
    (attention is linear in both).  NumPy's BLAS may use every host core the process is allowed."""
    from oracle import ps_oracle as po
    sh = wl.KVShape(n_layers, 8, 32, 128, 16, n_req * (ctx // 16) + 16)
    rng = np.random.default_rng(2)
    dims = (sh.num_layers, sh.num_gpu_blocks, sh.block_size, sh.num_kv_heads, sh.head_dim)
    orc = po.PsOracle(sh.num_layers, sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size, sh.num_gpu_blocks,
                      rng.permutation(sh.num_gpu_blocks), wl.randn_bf16_bits(rng, dims), wl.randn_bf16_bits(rng, dims))
    for r in range(n_req):
        assert orc.kv_alloc(r, ctx) == 0
    q = wl.randn_bf16_bits(rng, (n_layers, n_req, sh.num_q_heads, sh.head_dim))
    reqs = list(range(n_req))
    t0 = time.perf_counter()
    for l in range(n_layers):
        orc.decode_attn(l, q[l], reqs)
    sample_s = time.perf_counter() - t0
    scale = (step_layers / n_layers) * (step_tokens / (n_req * ctx))
    return {"attn_sample_s": sample_s,
            "attn_sample": f"fp64 decode attention, {n_layers} layers x {n_req} requests x {ctx} tokens x 32 query heads",
            "attn_step_s_extrapolated": sample_s * scale,
            "attn_step_extrapolation": f"sample x ({step_layers} / {n_layers} layers) x ({step_tokens} / {n_req * ctx} KV "
                                       f"tokens) = x {scale:.1f}: one decode step of the bench's 64 requests"}


def time_oracle(target_s: float = 10.0, step_layers: int = 32, step_tokens: int = 0):
    one_pass, nbytes, orc, sh = oracle_swap_pass()
    one_pass()                                   # touch the pages once
    t0 = time.perf_counter()
    n = 0
    while True:
        one_pass()
        n += 1
        if time.perf_counter() - t0 >= target_s:
            break
    dt = time.perf_counter() - t0
    del orc
    cores = len(os.sched_getaffinity(0))
    res = {
        "value": n * nbytes / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
        "sample": f"{n} passes of swap-out + reap + unbudgeted swap-in of 4 requests x 2048 tokens "
                  f"(8B KV shape, {nbytes / 2**30:.2f} GiB moved per pass) in {dt:.1f} s, single thread",
        "host_cores_available": cores, "attn_blas_threads_allowed": cores,
    }
    if step_tokens > 0:
        res.update(oracle_attention_step(step_layers, step_tokens))
    return res


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    one_pass, nbytes, _, _ = oracle_swap_pass()
    for _ in range(args.warmup):
        one_pass()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        one_pass()
    dt = time.perf_counter() - t0
    val = args.steps * nbytes / dt / 1e9
    sample = ("each step = swap-out + reap + unbudgeted swap-in of 4 requests x 2048 tokens of the 8B KV shape "
              f"({nbytes / 2**30:.2f} GiB moved), CPU checker, single thread")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "llama8b_swap (bounded sample)", "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# -------------------------------------------------------------------------------------------------
# GPU arm
# -------------------------------------------------------------------------------------------------

def fill_pools(torch, L, nb, S, Hkv, D, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    K = torch.empty((L, nb, S, Hkv, D), dtype=torch.bfloat16, device="cuda")
    V = torch.empty_like(K)
    for l in range(L):
        K[l].normal_(generator=g)
        V[l].normal_(generator=g)
    return K, V


def make_ctx(B, w, K, V, nb, *, max_batch, host_pool_bytes, flags=0, staging_bytes=0):
    sh = w.shape
    return B.KVSwap(num_layers=sh.num_layers, num_kv_heads=sh.num_kv_heads, num_q_heads=sh.num_q_heads,
                    head_dim=sh.head_dim, block_size=sh.block_size, num_gpu_blocks=nb,
                    max_blocks_per_req=max(sh.blocks_for(c) for c in w.ctx_lens) + 1, max_batch=max_batch,
                    host_pool_bytes=host_pool_bytes, staging_bytes=staging_bytes, initial_free_order=w.free_order,
                    k_pools=[K[l][:nb] for l in range(sh.num_layers)],
                    v_pools=[V[l][:nb] for l in range(sh.num_layers)], flags=flags)


def sub_batch(t, n):
    """A contiguous [L][n][Hq][D] view over the front of t's storage (values are irrelevant for timing)."""
    L, _, Hq, D = t.shape
    return t.flatten()[: L * n * Hq * D].view(L, n, Hq, D)


def swap_workload_step(torch, B, lib, w, q, out, q_res, out_res, budget, e2e_bufs=None):
    """One pass: phase A (offload under decode) and phase B (budgeted reload under decode).

    Returns a dict of times (ms, CUDA events on the compute stream) and counts."""
    stream = torch.cuda.current_stream()
    all_reqs = list(range(len(w.ctx_lens)))
    vict = set(w.victims)
    residents = [r for r in all_reqs if r not in vict]
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]

    def decode(reqs, qq, oo, bud):
        if e2e_bufs is not None:
            # end-to-end: queries and outputs live in pinned HOST memory; ps_step_host makes both copies
            qh, oh = e2e_bufs[qq.shape[1]]
            rc, mask, st = lib.step_host(qh, oh, reqs, bud)
        else:
            rc, mask, st = lib.step(qq, oo, reqs, bud)
        if rc != 0:
            raise RuntimeError(f"ps_step: {rc} {lib.last_error()}")
        stream.synchronize()                         # an engine reads the step's result before the next step
        return mask, st

    torch.cuda.synchronize()
    ev[0].record()
    for r in w.victims:
        rc = lib.swap_out(r)
        if rc != 0:
            raise RuntimeError(f"ps_swap_out: {rc} {lib.last_error()}")
    steps_a = 0
    while True:
        decode(residents, q_res, out_res, 0)
        steps_a += 1
        lib.poll()
        if lib.req_state(w.victims[-1]) == B.PS_REQ_HOST:      # offloads complete in issue order
            break
    ev[1].record()
    for r in w.victims:
        rc = lib.swap_in_begin(r)
        if rc != 0:
            raise RuntimeError(f"ps_swap_in_begin: {rc} {lib.last_error()}")
    steps_b = 0
    launches = 0
    while True:
        mask, st = decode(all_reqs, q, out, budget)
        steps_b += 1
        if all(mask):
            break
    if lib.sync() != 0:
        raise RuntimeError(f"ps_sync: {lib.last_error()}")
    ev[2].record()
    ev[2].synchronize()
    return {"out_ms": ev[0].elapsed_time(ev[1]), "in_ms": ev[1].elapsed_time(ev[2]),
            "steps_out": steps_a, "steps_in": steps_b}


def time_decode_steps(torch, lib, reqs, q, out, n):
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(n):
        rc, mask, st = lib.step(q, out, reqs, 0)
        assert rc == 0, lib.last_error()
        stream.synchronize()
    e1.record()
    e1.synchronize()
    return e0.elapsed_time(e1) / n


def kv_bytes_per_layer(sh, ctx_lens, reqs):
    """K and V bytes one layer of decode attention addresses for these requests (the algorithmic bytes)."""
    return sum(ctx_lens[r] for r in reqs) * 2 * sh.num_kv_heads * sh.head_dim * 2


def decode_roofline(torch, lib, sh, ctx_lens, reqs, q, out, steps=5):
    """Decode-only steps (nothing to reload): average duration of one attention launch, CUDA events around
    `steps` whole steps on the compute stream (no per-launch events), and the HBM rate that implies."""
    n0 = lib.launch_count()
    step_ms = time_decode_steps(torch, lib, reqs, q, out, steps)
    launches = (lib.launch_count() - n0) / steps
    alg = kv_bytes_per_layer(sh, ctx_lens, reqs)
    us = step_ms * 1e3 / sh.num_layers
    return {"us_per_layer": us, "launches_per_layer": launches / sh.num_layers, "algorithmic_bytes_per_launch": alg,
            "gbs": alg / us / 1e3, "step_us": step_ms * 1e3}


def single_launch_rate(torch, lib, sh, ctx_lens, reqs, q, out, rounds=3):
    """The same kernel through ps_decode_attn, one layer per call (what an engine that computes the next
    layer's queries from this layer's output can use): launches back to back, no overlap between layers."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for l in range(sh.num_layers):
        assert lib.decode_attn(l, q[l], out[l], reqs) == 0, lib.last_error()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(rounds):
        for l in range(sh.num_layers):
            assert lib.decode_attn(l, q[l], out[l], reqs) == 0, lib.last_error()
    e1.record(); e1.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (rounds * sh.num_layers)
    alg = kv_bytes_per_layer(sh, ctx_lens, reqs)
    return {"us_per_launch": us, "gbs": alg / us / 1e3}


def overlap_sweep(torch, B, K, V, peaks_hbm, w=None, label=None, pipelined_budgets=None, sync_budgets=None):
    """Overlap workload: decode batch 128 + 8 preempted requests reloading under 16/64/256 MiB budgets (or
    another workload with victims, e.g. the long-context one).

    Contexts carry no per-launch profiling events: under host-link load those events delay the compute
    stream's commands and would be charged to the reload."""
    w = w or wl.overlap()
    sh = w.shape
    nb = sh.num_gpu_blocks
    host_bytes = sum(sh.blocks_for(w.ctx_lens[r]) for r in w.victims) * sh.block_bytes + (64 << 20)
    res = {"workload": label or "overlap: decode batch 128, lognormal contexts (mean 2k, cap 8k), 8 preempted requests"}
    stream = torch.cuda.current_stream()
    if pipelined_budgets is None:
        pipelined_budgets = w.budgets + ["adaptive", -1]
    if sync_budgets is None:
        sync_budgets = [256 * wl.MiB, -1]
    for mode in ("pipelined", "sync_reload"):
        flags = B.PS_FLAG_SYNC_RELOAD if mode == "sync_reload" else 0
        if not (pipelined_budgets if mode == "pipelined" else sync_budgets):
            continue
        lib = make_ctx(B, w, K, V, nb, max_batch=len(w.ctx_lens), host_pool_bytes=host_bytes, flags=flags)
        for r, n in wl.build_order_round_robin(w):
            assert lib.kv_alloc(r, n) == 0, lib.last_error()
        all_reqs = list(range(len(w.ctx_lens)))
        batch = [r for r in all_reqs if r not in w.victims]
        g = torch.Generator(device="cuda")
        g.manual_seed(w.seed)
        q = torch.randn((sh.num_layers, len(all_reqs), sh.num_q_heads, sh.head_dim), generator=g, device="cuda",
                        dtype=torch.float32).to(torch.bfloat16)
        out = torch.zeros_like(q)
        reload_bytes = sum(sh.blocks_for(w.ctx_lens[r]) for r in w.victims) * sh.block_bytes
        # "adaptive": B_copy chosen every step by ps_copy_budget (Section 4.3) from the measured decode time per
        # token and the measured copy time per block (no latency budget: case 2 of the procedure)
        budgets = pipelined_budgets if mode == "pipelined" else sync_budgets
        model = None
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if mode == "pipelined":
            for _ in range(3):
                time_decode_steps(torch, lib, batch, sub_batch(q, len(batch)), sub_batch(out, len(batch)), 1)
            rf = decode_roofline(torch, lib, sh, w.ctx_lens, batch, sub_batch(q, len(batch)), sub_batch(out, len(batch)))
            res["attn_gbs"] = rf["gbs"]
            res["attn_frac_of_hbm"] = rf["gbs"] / peaks_hbm
            res["attn_us_per_layer"] = rf["us_per_layer"]
            link_gbs = B.ps_link_probe(256 << 20, 0, 5)
            model = {"a_d": rf["step_us"] / sum(w.ctx_lens[r] for r in batch), "b_d": 0.0, "t_c": 0.0,
                     "t_block": sh.block_bytes / (link_gbs * 1e3) * (1.0 + 1.0 / sh.num_layers), "t_budget": 1e12}
            # the largest budget whose transfer fits under a decode step: link rate x step time, less the
            # first layer chunk, which nothing can hide
            res["hideable_budget_mib"] = link_gbs * 1e3 * rf["step_us"] * (1.0 - 1.0 / sh.num_layers) / wl.MiB
            res["link_h2d_gbs_256mib_probe"] = link_gbs
            res["adaptive_model"] = dict(model, note="a_d: measured decode step us per KV token; t_block: block bytes / "
                                         "measured H2D rate, plus one layer chunk of pipeline fill")
        if mode == "pipelined":
            res.update(offload_rates(torch, B, lib, w, batch, sub_batch(q, len(batch)), sub_batch(out, len(batch)),
                                     reload_bytes))
        else:
            for r in w.victims:
                assert lib.swap_out(r) == 0, lib.last_error()
            assert lib.sync() == 0
        for budget in budgets:
            # (1) reload alone, no attention: the transfer time the decode steps have to hide
            for r in w.victims:
                assert lib.swap_in_begin(r) == 0
            torch.cuda.synchronize()
            e0.record()
            chosen = []

            def step_budget(reqs_now):
                if budget != "adaptive":
                    return budget
                rc, blocks, nbytes, case = lib.copy_budget(reqs_now, **model)
                assert rc == 0, lib.last_error()
                chosen.append(nbytes)
                return nbytes

            while any(lib.missing_blocks(r) for r in w.victims):
                rc, _, _ = lib.step(None, None, [], step_budget(all_reqs))
                assert rc == 0, lib.last_error()
                assert lib.sync() == 0
            e1.record(); e1.synchronize()
            alone_stepwise_ms = e0.elapsed_time(e1)
            chosen.clear()
            for r in w.victims:
                assert lib.swap_out(r) == 0
            assert lib.sync() == 0
            # (1b) the same steps issued back to back, one wait at the end: the transfer without a host round
            # trip per step (the denominator of the hidden fraction)
            for r in w.victims:
                assert lib.swap_in_begin(r) == 0
            torch.cuda.synchronize()
            e0.record()
            while any(lib.missing_blocks(r) for r in w.victims):
                rc, _, _ = lib.step(None, None, [], step_budget(all_reqs))
                assert rc == 0, lib.last_error()
            assert lib.sync() == 0
            e1.record(); e1.synchronize()
            alone_ms = e0.elapsed_time(e1)
            chosen.clear()
            for r in w.victims:
                assert lib.swap_out(r) == 0
            assert lib.sync() == 0
            # (2) the same reload under decode steps
            for _ in range(3):
                time_decode_steps(torch, lib, batch, sub_batch(q, len(batch)), sub_batch(out, len(batch)), 1)
            for r in w.victims:
                assert lib.swap_in_begin(r) == 0
            masks = []
            torch.cuda.synchronize()
            e0.record()
            while True:
                rc, mask, st = lib.step(q, out, all_reqs, step_budget(all_reqs))
                assert rc == 0, lib.last_error()
                stream.synchronize()
                masks.append(mask)
                if all(mask):
                    break
            e1.record(); e1.synchronize()
            with_ms = e0.elapsed_time(e1)
            assert lib.sync() == 0
            # (3) the same sequence of decode sets with nothing to reload
            sets = [[r for r, m in zip(all_reqs, mk) if m] for mk in masks]
            for _ in range(2):
                time_decode_steps(torch, lib, sets[0], sub_batch(q, len(sets[0])), sub_batch(out, len(sets[0])), 1)
            torch.cuda.synchronize()
            e0.record()
            for rs in sets:
                rc, _, _ = lib.step(sub_batch(q, len(rs)), sub_batch(out, len(rs)), rs, 0)
                assert rc == 0, lib.last_error()
                stream.synchronize()
            e1.record(); e1.synchronize()
            without_ms = e0.elapsed_time(e1)
            n_steps = len(masks)
            hidden = 1.0 - max(0.0, with_ms - without_ms) / alone_ms if alone_ms > 0 else None
            key = f"{mode}_" + ("adaptive" if budget == "adaptive" else "unlimited" if budget < 0
                                else str(budget // wl.MiB) + "MiB")
            res[key] = {"steps": n_steps, "step_us_with_reload": with_ms / n_steps * 1e3,
                        "step_us_no_reload": without_ms / n_steps * 1e3,
                        "reload_alone_ms": alone_ms, "reload_alone_gbs": reload_bytes / alone_ms / 1e6,
                        "reload_alone_stepwise_ms": alone_stepwise_ms,
                        "reload_alone_stepwise_gbs": reload_bytes / alone_stepwise_ms / 1e6,
                        "hidden_frac_vs_stepwise": (1.0 - max(0.0, with_ms - without_ms) / alone_stepwise_ms)
                        if alone_stepwise_ms > 0 else None,
                        "reload_under_decode_gbs": reload_bytes / with_ms / 1e6, "hidden_frac": hidden}
            if budget == "adaptive":
                res[key]["chosen_budget_mib_per_step"] = [round(c / wl.MiB, 1) for c in chosen]
            for r in w.victims:
                assert lib.swap_out(r) == 0
            assert lib.sync() == 0
        lib.destroy()
    if w.name == "overlap" and "pipelined_adaptive" in res:
        res["recompute_arm"] = recompute_arm(B, w, res)
    return res


def offload_rates(torch, B, lib, w, batch, q_b, out_b, nbytes):
    """Swap-out of the workload's victims, alone and then under running decode steps; leaves them on the host."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stream = torch.cuda.current_stream()
    torch.cuda.synchronize()
    e0.record()
    for r in w.victims:
        assert lib.swap_out(r) == 0, lib.last_error()
    assert lib.sync() == 0
    e1.record(); e1.synchronize()
    alone_ms = e0.elapsed_time(e1)
    for r in w.victims:
        assert lib.swap_in_begin(r) == 0, lib.last_error()
    rc, _, _ = lib.step(None, None, [], -1)
    assert rc == 0 and lib.sync() == 0, lib.last_error()
    torch.cuda.synchronize()
    e0.record()
    for r in w.victims:
        assert lib.swap_out(r) == 0, lib.last_error()
    steps = 0
    while True:
        rc, _, _ = lib.step(q_b, out_b, batch, 0)
        assert rc == 0, lib.last_error()
        stream.synchronize()
        steps += 1
        lib.poll()
        if lib.req_state(w.victims[-1]) == B.PS_REQ_HOST:      # offloads complete in issue order
            break
    e1.record(); e1.synchronize()
    under_ms = e0.elapsed_time(e1)
    assert lib.sync() == 0
    return {"offload_alone_gbs": nbytes / alone_ms / 1e6, "offload_under_decode_gbs": nbytes / under_ms / 1e6,
            "offload_bytes": nbytes, "decode_steps_during_offload": steps,
            "decode_step_us_during_offload": under_ms / steps * 1e3}


def recompute_arm(B, w, res):
    """The evaluation's "Recompute" ablation arm (blocks discarded at eviction, the context prefilled again on
    resume) against the measured reload, for the overlap workload's preempted requests.  The recompute side is
    NOT measured: it is ps_resume_cost with estimator coefficients set to a lower bound, the prefill's matrix
    and attention FLOPs at the dense bf16 rate of a long-running library GEMM on this GPU (a real prefill is
    slower).  hidden and ffn are the public dimensions of the 8B model family whose KV shape the workload has."""
    sh = w.shape
    hidden, ffn = 4096, 14336
    kv_dim = sh.num_kv_heads * sh.head_dim
    layer_params = hidden * (hidden + 2 * kv_dim) + hidden * hidden + 3 * hidden * ffn
    tflops, kind = read_bf16_peak()
    flop_per_us = tflops * 1e6
    pair_flops = 4 * sh.num_q_heads * sh.head_dim * sh.num_layers       # q.k and p.v, one (query, key) pair
    model = B.PsLatencyModel(a_p_us=0.5 * pair_flops / flop_per_us, b_p_us=pair_flops / flop_per_us,
                             c_p_us=2.0 * layer_params * sh.num_layers / flop_per_us, a_d_us=0.0, b_d_us=0.0,
                             t_c_us=0.0)
    t_block = res["adaptive_model"]["t_block"]
    reload_us = recompute_us = 0.0
    for r in w.victims:
        rc, a, b = B.ps_resume_cost(model, w.ctx_lens[r], 2048, sh.block_size, t_block)
        assert rc == 0
        reload_us += a
        recompute_us += b
    row = res["pipelined_adaptive"]
    exposed_ms = max(0.0, row["step_us_with_reload"] - row["step_us_no_reload"]) * row["steps"] / 1e3
    return {
        "tokens": sum(w.ctx_lens[r] for r in w.victims), "chunk_tokens": 2048,
        "recompute_lower_bound_ms": recompute_us / 1e3, "bf16_tflops": tflops, "bf16_peak_kind": kind,
        "coefficients_us": {"a_p": model.a_p_us, "b_p": model.b_p_us, "c_p": model.c_p_us},
        "reload_estimate_ms": reload_us / 1e3, "reload_alone_measured_ms": row["reload_alone_ms"],
        "reload_exposed_under_decode_measured_ms": exposed_ms,
        "note": "recompute side is a cost model at 100 % of the GEMM rate, not a measurement; the reload sides are "
                "the measured transfer alone and the measured step-time inflation under the adaptive budget",
    }


def proactive_offload_leg(torch, B, lib, w, n_off=16):
    """Time from eviction to reclaimable blocks, on demand and after proactive incremental offloading
    (Section 4.3: a copy for every n_off newly filled blocks, done in the background before eviction)."""
    sh = w.shape

    def evict_and_wait():
        t0 = time.perf_counter()
        for r in w.victims:
            assert lib.swap_out(r) == 0, lib.last_error()
        assert lib.sync() == 0, lib.last_error()
        return (time.perf_counter() - t0) * 1e3

    def reload_all():
        for r in w.victims:
            assert lib.swap_in_begin(r) == 0, lib.last_error()
        rc, _, _ = lib.step(None, None, [], -1)
        assert rc == 0 and lib.sync() == 0, lib.last_error()

    on_demand_ms = evict_and_wait()
    reload_all()
    copied = 0
    t0 = time.perf_counter()
    for r in w.victims:
        rc, n = lib.offload_progress(r, n_off)
        assert rc == 0, lib.last_error()
        copied += n
    assert lib.sync() == 0
    background_ms = (time.perf_counter() - t0) * 1e3
    tail_ms = evict_and_wait()
    reload_all()
    total = sum(sh.blocks_for(w.ctx_lens[r]) for r in w.victims)
    return {"n_off": n_off, "victim_blocks": total, "blocks_copied_ahead": copied,
            "evict_to_reclaim_ms_on_demand": on_demand_ms, "evict_to_reclaim_ms_after_proactive": tail_ms,
            "background_copy_ms": background_ms}


def kernel_rates(torch, B, lib, sh, nb, hbm_peak, iters=20):
    """The swap path's own kernels alone (no host link), in the launch shapes the path gives them: payload read
    once + written once per launch.  gather_image_kernel at the size of a staging slot (64 MiB over 8 layers
    of a request), scatter_image_kernel at the layer chunks ps_step issues for 16 / 64 / 256 MiB per step and
    for an unlimited budget.  Launches are enqueued back to back (the ids are uploaded once)."""
    import ctypes as C
    rng = np.random.default_rng(3)
    Bl = sh.layer_block_bytes
    cases = [("gather_slot_64mib", 0, 128, 8), ("scatter_slot_64mib", 1, 1024, 1),
             ("scatter_chunk_256mib_step", 1, 256 * wl.MiB // sh.block_bytes, 1),
             ("scatter_chunk_64mib_step", 1, 64 * wl.MiB // sh.block_bytes, 1),
             ("scatter_chunk_16mib_step", 1, 16 * wl.MiB // sh.block_bytes, 4)]
    res = {}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name, direction, n_blocks, n_layers in cases:          # scatters overwrite pool blocks: the caller runs this last
        ids = (C.c_int32 * n_blocks)(*[int(v) for v in rng.permutation(nb)[:n_blocks]])
        stage = torch.empty((n_layers, n_blocks, 2, sh.block_size, sh.num_kv_heads, sh.head_dim), dtype=torch.bfloat16,
                            device="cuda")
        payload = n_layers * n_blocks * Bl

        def launch(i):
            rc = lib.lib.ps_copy_blocks(lib.h, (i * n_layers) % (sh.num_layers - n_layers + 1), n_layers, ids, n_blocks,
                                        C.c_void_p(stage.data_ptr()), direction)
            assert rc == 0, lib.last_error()

        for i in range(3):
            launch(i)
        torch.cuda.synchronize()
        e0.record()
        for i in range(iters):
            launch(i)
        e1.record(); e1.synchronize()
        ms = e0.elapsed_time(e1) / iters
        res[name] = {"kernel": "gather_image_kernel" if direction == 0 else "scatter_image_kernel",
                     "blocks": n_blocks, "layers": n_layers, "payload_bytes_per_launch": payload,
                     "us_per_launch": ms * 1e3, "gbs_rw": 2 * payload / ms / 1e6,
                     "frac_of_hbm": 2 * payload / ms / 1e6 / hbm_peak}
        del stage
    res["launches_timed"] = iters
    return res


def long_context_leg(torch, B, hbm_peak, compact=False):
    """70B-shaped KV (80 layers, block 32): decode batch 64 x 4096 tokens, one 32k-token request (10 GiB) offloaded
    under decode and reloaded layer-pipelined across steps."""
    w = wl.long_context()
    sh = w.shape
    K, V = fill_pools(torch, sh.num_layers, sh.num_gpu_blocks, sh.block_size, sh.num_kv_heads, sh.head_dim, w.seed)
    torch.cuda.synchronize()
    res = overlap_sweep(torch, B, K, V, hbm_peak, w=w,
                        label="long_context: decode batch 64 x 4096 tokens, one 32768-token request of 10 GiB",
                        pipelined_budgets=[256 * wl.MiB, "adaptive"] if compact else [256 * wl.MiB, "adaptive", -1],
                        sync_budgets=[] if compact else [256 * wl.MiB])
    del K, V
    return res


def churn_leg(torch, B, hbm_peak, steps):
    """Qwen3-32B-shaped KV (64 layers), 256 live requests of 512-16k tokens on an oversubscribed instance: every
    step swaps out 2-16 low-priority residents and swaps in 2-16 host-resident requests (a seeded script clipped
    to capacity), unlimited copy budget, decode over whoever is resident.  Reports the sustained two-way rate
    over the host link and how much longer a step takes than decoding the same set with no swap."""
    w = wl.churn(steps=steps)
    sh = w.shape
    host_bytes = 12 * wl.GiB
    init, script = wl.churn_script(w, host_bytes)
    K, V = fill_pools(torch, sh.num_layers, sh.num_gpu_blocks, sh.block_size, sh.num_kv_heads, sh.head_dim, w.seed)
    torch.cuda.synchronize()
    nreq = len(w.ctx_lens)
    lib = make_ctx(B, w, K, V, sh.num_gpu_blocks, max_batch=nreq, host_pool_bytes=2 * host_bytes)
    for r in init["host"]:                           # host-resident requests pass through the device first
        assert lib.kv_alloc(r, w.ctx_lens[r]) == 0, lib.last_error()
        assert lib.swap_out(r) == 0, lib.last_error()
        assert lib.sync() == 0
    for r in init["resident"]:
        assert lib.kv_alloc(r, w.ctx_lens[r]) == 0, lib.last_error()
    known = sorted(init["host"] + init["resident"])
    g = torch.Generator(device="cuda")
    g.manual_seed(w.seed)
    q = torch.randn((sh.num_layers, nreq, sh.num_q_heads, sh.head_dim), generator=g, device="cuda",
                    dtype=torch.float32).to(torch.bfloat16)
    out = torch.zeros_like(q)
    duplex_gbs = B.ps_link_probe(256 << 20, 2, 5)
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    q_l, out_l = sub_batch(q, len(known)), sub_batch(out, len(known))
    for _ in range(3):
        rc, mask, _ = lib.step(q_l, out_l, known, 0)
        assert rc == 0, lib.last_error()
    torch.cuda.synchronize()
    bytes_out = bytes_in = n_out = n_in = decoded = 0
    step_ms = []
    bound_ms = 0.0                                   # per step the busier direction at half the two-way rate
    e0.record()
    for stp in script:
        assert lib.sync() == 0                       # the previous step's swaps have completed
        o0, i0 = bytes_out, bytes_in
        for r in stp["out"]:
            if lib.swap_out(r) == 0:
                bytes_out += sh.blocks_for(w.ctx_lens[r]) * sh.block_bytes
                n_out += 1
        for r in stp["inn"]:
            if lib.swap_in_begin(r) == 0:
                bytes_in += sh.blocks_for(w.ctx_lens[r]) * sh.block_bytes
                n_in += 1
        bound_ms += max(bytes_out - o0, bytes_in - i0) / (duplex_gbs / 2) / 1e6
        s0.record()
        rc, mask, st = lib.step(q_l, out_l, known, -1)
        assert rc == 0, lib.last_error()
        s1.record()
        stream.synchronize()
        step_ms.append(s0.elapsed_time(s1))
        decoded += sum(mask)
    assert lib.sync() == 0
    e1.record(); e1.synchronize()
    total_ms = e0.elapsed_time(e1)
    resident = [r for r in known if lib.block_table(r)[1] == B.PS_REQ_RESIDENT]
    q_r, out_r = sub_batch(q, len(resident)), sub_batch(out, len(resident))
    rf = decode_roofline(torch, lib, sh, w.ctx_lens, resident, q_r, out_r, steps=3)
    lib.destroy()
    del K, V
    return {
        "workload": f"churn: 64 layers, {nreq} live requests (512-16k tokens), {len(known)} of them holding KV, "
                    f"{steps} scripted steps, unlimited copy budget, device pool 96 GiB, host images 12 GiB planned",
        "steps": steps, "swap_outs": n_out, "swap_ins": n_in, "bytes_out": bytes_out, "bytes_in": bytes_in,
        "two_way_gbs": (bytes_out + bytes_in) / total_ms / 1e6, "link_two_way_peak_gbs": duplex_gbs,
        "frac_of_two_way_peak": (bytes_out + bytes_in) / total_ms / 1e6 / duplex_gbs,
        "schedule_bound_ms": bound_ms, "total_ms": total_ms, "frac_of_schedule_bound": bound_ms / total_ms,
        "schedule_bound": "the swaps of a step complete in that step, so a step cannot end before its busier "
                          "direction has crossed the link at half the measured two-way rate",
        "step_ms_mean_with_swaps": total_ms / steps, "compute_stream_step_ms_mean": float(np.mean(step_ms)),
        "decode_step_ms_no_swap": rf["step_us"] / 1e3, "requests_decoding_at_end": len(resident),
        "decoded_request_steps": decoded, "attn_gbs": rf["gbs"], "attn_frac_of_hbm": rf["gbs"] / hbm_peak,
    }


def churn_loop_leg(torch, B, hbm_peak, rounds):
    """The priority-churn workload driven by the paper's closed loop (engine_loop.SchedulerStub over the library):
    queue order -> eviction from the tail (asynchronous offloads) -> readmission from the head -> ps_copy_budget
    -> ps_step_ruled (budget consumed under the partial-copy rule) while the resident set decodes.  The latency
    model's coefficients are measured first (decode time per KV token, copy time per block), so the adaptive
    budget aims at what this GPU and this link can hide."""
    from paper_2512_12928_b200 import engine_loop as el
    w = wl.churn()
    sh = w.shape
    K, V = fill_pools(torch, sh.num_layers, sh.num_gpu_blocks, sh.block_size, sh.num_kv_heads, sh.head_dim, w.seed)
    torch.cuda.synchronize()
    params = el.config4_params()
    lib = B.KVSwap(num_layers=sh.num_layers, num_kv_heads=sh.num_kv_heads, num_q_heads=sh.num_q_heads,
                   head_dim=sh.head_dim, block_size=sh.block_size, num_gpu_blocks=sh.num_gpu_blocks,
                   max_blocks_per_req=1040, max_batch=params.max_batch, host_pool_bytes=30 * wl.GiB,
                   initial_free_order=w.free_order, k_pools=[K[l] for l in range(sh.num_layers)],
                   v_pools=[V[l] for l in range(sh.num_layers)])
    class TimedBackend(el.LibBackend):
        """Brackets every step with CUDA events on the compute stream: the step's device time, without the
        host time this Python stub spends between steps."""
        spans = []

        def step(self, *a):
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s0.record()
            res = super().step(*a)
            s1.record()
            self.spans.append((s0, s1))
            return res

    stub = el.SchedulerStub(TimedBackend(lib), w.ctx_lens, w.priority, sh.block_size, sh.block_bytes,
                            sh.num_gpu_blocks, params, seed=w.seed)
    placed = stub.fill()
    g = torch.Generator(device="cuda")
    g.manual_seed(w.seed)
    q = torch.randn((sh.num_layers, params.max_batch, sh.num_q_heads, sh.head_dim), generator=g, device="cuda",
                    dtype=torch.float32).to(torch.bfloat16)
    out = torch.zeros_like(q)
    # the latency model, measured: decode step = c0 + a_d * KV tokens (two batch sizes), t_block from the link
    tok = lambda rs: sum(stub.live[r].tokens for r in rs)
    half = placed[: len(placed) // 2]
    for rs in (placed, half):
        time_decode_steps(torch, lib, rs, sub_batch(q, len(rs)), sub_batch(out, len(rs)), 2)
    us_full = time_decode_steps(torch, lib, placed, sub_batch(q, len(placed)), sub_batch(out, len(placed)), 3) * 1e3
    us_half = time_decode_steps(torch, lib, half, sub_batch(q, len(half)), sub_batch(out, len(half)), 3) * 1e3
    tokens_full = tok(placed)
    a_d = (us_full - us_half) / (tok(placed) - tok(half))
    c0 = max(0.0, us_full - a_d * tok(placed))
    h2d_gbs = B.ps_link_probe(256 << 20, 0, 5)
    d2h_gbs = B.ps_link_probe(256 << 20, 1, 5)
    duplex_gbs = B.ps_link_probe(256 << 20, 2, 5)
    # offloads and reloads share the link in this loop: a block's copy time is taken at the rate one direction
    # gets while both run
    h2d_loaded = min(h2d_gbs, duplex_gbs / 2)
    params.a_d_us, params.b_d_us, params.t_c_us = a_d, 0.0, c0
    params.t_block_us = sh.block_bytes / (h2d_loaded * 1e3) * (1.0 + 1.0 / sh.num_layers)
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tot = dict(evicted=0, readmitted=0, admitted=0, finished=0, blocks_in=0, blocks_out=0, decoded=0, skipped=0,
               decode_tokens=0, reloads_completed=0)
    cases = {}
    no_swap_us = 0.0
    torch.cuda.synchronize()
    e0.record()
    for _ in range(rounds):
        rep = stub.round(q, out)
        stream.synchronize()                         # an engine reads the step's result before the next round
        tot["evicted"] += len(rep.evicted)
        tot["readmitted"] += len(rep.readmitted)
        tot["admitted"] += len(rep.admitted)
        tot["finished"] += len(rep.finished)
        tot["blocks_in"] += rep.stats["blocks_copied"]
        tot["blocks_out"] += sum(stub.blocks_for(stub.live[v].tokens) for v in rep.evicted if v in stub.live)
        tot["decoded"] += sum(rep.mask)
        tot["skipped"] += rep.skipped_by_rule
        tot["decode_tokens"] += rep.decode_tokens
        tot["reloads_completed"] += rep.stats["reloads_completed"]
        cases[rep.budget_case] = cases.get(rep.budget_case, 0) + 1
        no_swap_us += c0 + a_d * rep.decode_tokens
    e1.record(); e1.synchronize()
    loop_ms = e0.elapsed_time(e1)
    steps_ms = sum(a.elapsed_time(b) for a, b in TimedBackend.spans)
    assert lib.sync() == 0, lib.last_error()
    lib.destroy()
    del K, V, q, out
    bytes_in, bytes_out = tot["blocks_in"] * sh.block_bytes, tot["blocks_out"] * sh.block_bytes
    transfer_alone_ms = bytes_in / (h2d_gbs * 0.95) / 1e6           # a reload alone runs at about 0.95 of the probe
    hidden = 1.0 - max(0.0, steps_ms - no_swap_us / 1e3) / transfer_alone_ms if transfer_alone_ms > 0 else None
    return {
        "workload": f"churn, closed loop: 64 layers, 256 live requests (512-16k tokens, two classes), {len(placed)} "
                    f"resident at the start, {rounds} rounds of the scheduler stub (order, evict, readmit, adaptive "
                    "budget, partial-copy rule)",
        "rounds": rounds, **tot, "budget_cases": {str(k): v for k, v in sorted(cases.items())},
        "bytes_in": bytes_in, "bytes_out": bytes_out, "loop_ms": loop_ms, "round_ms_mean_wall": loop_ms / rounds,
        "step_ms_mean": steps_ms / rounds,
        "no_swap_step_ms_model": no_swap_us / 1e3 / rounds,
        "reload_gbs_sustained": bytes_in / loop_ms / 1e6, "offload_gbs_sustained": bytes_out / loop_ms / 1e6,
        "reload_frac_of_link": bytes_in / loop_ms / 1e6 / h2d_gbs, "offload_frac_of_link": bytes_out / loop_ms / 1e6 / d2h_gbs,
        "hidden_frac_estimate": hidden,
        "hidden_frac_how": "1 - (sum of the steps' device times - sum over rounds of the measured decode model c0 + a_d * KV tokens of the "
                           "round's batch) / (reloaded bytes at 0.95 of the probed H2D rate); offloads are "
                           "asynchronous and never on a step's critical path",
        "model": {"a_d_us_per_token": a_d, "c0_us": c0, "t_block_us": params.t_block_us, "h2d_gbs": h2d_gbs,
                  "d2h_gbs": d2h_gbs, "duplex_sum_gbs": duplex_gbs, "decode_us_full_set": us_full, "tokens_full_set": tokens_full},
    }


def decode_shapes_leg(torch, B, hbm_peak):
    """Decode attention alone for the KV shapes of the paper's model families under tensor parallelism: 8 / 4 / 2 / 1
    KV heads per GPU (8B-like 32 layers G = 4; Qwen2-7B-like 28 layers G = 7 and its 2- and 4-way shards).
    Batch 128, lognormal contexts (mean 2048, cap 8192); in-step rate (ps_step) and one launch per call."""
    rows = []
    nb = 24576
    for L, Hkv, Hq in [(32, 8, 32), (28, 4, 28), (28, 2, 14), (28, 1, 7)]:
        sh = wl.KVShape(L, Hkv, Hq, 128, 16, nb)
        rng = np.random.default_rng(wl.SEED_BASE + 9)
        ctx = wl.lognormal_ctx(rng, 128, 2048.0, 0.8, 8192)
        w = wl.Workload("decode_shapes", 9, sh, wl.SEED_BASE + 9, ctx, [], rng.permutation(nb).astype(np.int32),
                        decode_batch=128)
        K, V = fill_pools(torch, L, nb, sh.block_size, Hkv, sh.head_dim, w.seed)
        lib = make_ctx(B, w, K, V, nb, max_batch=128, host_pool_bytes=64 << 20)
        for r, n in wl.build_order_round_robin(w):
            assert lib.kv_alloc(r, n) == 0, lib.last_error()
        reqs = list(range(128))
        g = torch.Generator(device="cuda")
        g.manual_seed(w.seed)
        q = torch.randn((L, 128, Hq, sh.head_dim), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        out = torch.zeros_like(q)
        time_decode_steps(torch, lib, reqs, q, out, 3)
        rf = decode_roofline(torch, lib, sh, ctx, reqs, q, out, steps=5)
        sg = single_launch_rate(torch, lib, sh, ctx, reqs, q, out)
        rows.append({"layers": L, "kv_heads": Hkv, "q_heads": Hq, "bytes_per_launch": rf["algorithmic_bytes_per_launch"],
                     "in_step_gbs": rf["gbs"], "in_step_frac_of_hbm": rf["gbs"] / hbm_peak,
                     "in_step_us_per_launch": rf["us_per_layer"], "single_launch_gbs": sg["gbs"],
                     "single_launch_us": sg["us_per_launch"]})
        lib.destroy()
        del K, V, lib, q, out
        torch.cuda.empty_cache()
    return {"workload": "decode attention alone, batch 128, lognormal contexts, four KV shapes", "shapes": rows}


def run_extra(args):
    """The other workloads of the evaluation, one JSON line each (single GPU; not the headline line)."""
    import torch

    from paper_2512_12928_b200 import binding as B
    from paper_2512_12928_b200 import build as ps_build
    torch.cuda.set_device(0)
    ps_build.build()
    B.load()
    hbm_peak, peak_kind = read_peaks()
    sampler = ClockSampler(0)
    sampler.start()
    if args.workload == "long_context":
        detail = long_context_leg(torch, B, hbm_peak)
        value = detail["pipelined_adaptive"]["reload_under_decode_gbs"]
        metric = "reload GB/s under decode (adaptive copy budget); hidden fraction in detail"
    elif args.workload == "decode_shapes":
        detail = decode_shapes_leg(torch, B, hbm_peak)
        value = detail["shapes"][1]["in_step_gbs"]
        metric = "decode attention GB/s of KV read, 28 layers x 4 KV heads x 28 query heads (in ps_step)"
    else:
        detail = {"closed_loop": churn_loop_leg(torch, B, hbm_peak, args.churn_rounds)}
        torch.cuda.empty_cache()
        detail["scripted_unlimited_budget"] = churn_leg(torch, B, hbm_peak, args.churn_steps)
        value = detail["closed_loop"]["reload_gbs_sustained"] + detail["closed_loop"]["offload_gbs_sustained"]
        metric = "sustained swap-out + swap-in GB/s over the host link under decode, closed loop"
    clocks = sampler.stop()
    print(json.dumps({"metric": metric, "value": value, "unit": UNIT, "n_gpus": 1, "higher_is_better": True,
                      "dtype": "bf16", "data": "synthetic", "config": {"workload": args.workload},
                      "peak_kind": peak_kind, "clocks": clocks, "detail": detail}))


def run_gpu(args):
    import torch

    from paper_2512_12928_b200 import binding as B
    from paper_2512_12928_b200 import build as ps_build

    from paper_2512_12928_b200 import replicas

    rank, world, local_rank = replicas.env()
    torch.cuda.set_device(local_rank)
    if world > 1:
        replicas.bind_near_gpu(local_rank)           # pinned host pools from the memory nearest to this GPU's link
    group = replicas.Group("nccl", torch.device("cuda", local_rank))
    if rank == 0:
        ps_build.build()
    group.barrier()
    B.load()
    hbm_peak, peak_kind = read_peaks()

    # host link peaks (pinned cudaMemcpyAsync, 1 GiB, best of 10)
    link = {"h2d_gbs": B.ps_link_probe(1 << 30, 0, 10), "d2h_gbs": B.ps_link_probe(1 << 30, 1, 10),
            "duplex_sum_gbs": B.ps_link_probe(1 << 30, 2, 5)}

    w = wl.llama8b_swap()
    sh = w.shape
    w3 = wl.overlap()
    nb_alloc = max(sh.num_gpu_blocks, w3.shape.num_gpu_blocks) if not args.no_overlap else sh.num_gpu_blocks
    K, V = fill_pools(torch, sh.num_layers, nb_alloc, sh.block_size, sh.num_kv_heads, sh.head_dim,
                      replicas.replica_seed(w.seed, rank))
    torch.cuda.synchronize()

    victim_bytes = sum(sh.blocks_for(w.ctx_lens[r]) for r in w.victims) * sh.block_bytes
    nreq = len(w.ctx_lens)
    g = torch.Generator(device="cuda")
    g.manual_seed(w.seed)
    q = torch.randn((sh.num_layers, nreq, sh.num_q_heads, sh.head_dim), generator=g, device="cuda",
                    dtype=torch.float32).to(torch.bfloat16)
    out = torch.zeros_like(q)
    budget = args.budget_mib * wl.MiB if args.budget_mib >= 0 else -1
    n_res = nreq - len(w.victims)
    q_res = sub_batch(q, n_res).clone()
    out_res = torch.zeros_like(q_res)
    # end-to-end arm: queries and outputs in pinned host memory, one pair of buffers per batch size
    e2e_bufs = {nreq: (q.cpu().pin_memory(), torch.zeros_like(q, device="cpu").pin_memory()),
                n_res: (q_res.cpu().pin_memory(), torch.zeros_like(q_res, device="cpu").pin_memory())}

    def fresh_ctx(flags):
        lib = make_ctx(B, w, K, V, sh.num_gpu_blocks, max_batch=nreq, host_pool_bytes=victim_bytes + (256 << 20),
                       flags=flags, staging_bytes=args.staging_mib * wl.MiB)
        for r, n in wl.build_order_round_robin(w):
            assert lib.kv_alloc(r, n) == 0, lib.last_error()
        return lib

    # ---- the timed region: no per-launch events (they delay the compute stream under host-link load)
    lib = fresh_ctx(0)
    for _ in range(args.warmup):
        swap_workload_step(torch, B, lib, w, q, out, q_res, out_res, budget)
    launches0 = lib.launch_count()
    sampler = ClockSampler(local_rank)
    sampler.start()
    group.barrier()
    torch.cuda.synchronize()
    t_wall0 = time.perf_counter()
    recs = [swap_workload_step(torch, B, lib, w, q, out, q_res, out_res, budget) for _ in range(args.steps)]
    torch.cuda.synchronize()
    group.barrier()
    wall_ms = (time.perf_counter() - t_wall0) * 1e3
    launches = lib.launch_count() - launches0

    out_ms = sum(r["out_ms"] for r in recs)
    in_ms = sum(r["in_ms"] for r in recs)
    total_ms = out_ms + in_ms
    total_ms, out_ms, in_ms = group.max_over_ranks([total_ms, out_ms, in_ms])
    (moved,) = group.sum_over_ranks([2 * victim_bytes * args.steps])
    value = moved / total_ms / 1e6

    # ---- the dominant kernel, live, in the launch configuration of the step: decode-only steps of the
    # whole batch between two CUDA events on the compute stream (still inside the clock-sampled region)
    all_reqs = list(range(nreq))
    residents = [r for r in all_reqs if r not in set(w.victims)]
    time_decode_steps(torch, lib, all_reqs, q, out, 2)
    rf_all = decode_roofline(torch, lib, sh, w.ctx_lens, all_reqs, q, out, steps=5)
    time_decode_steps(torch, lib, residents, q_res, out_res, 2)
    rf_res = decode_roofline(torch, lib, sh, w.ctx_lens, residents, q_res, out_res, steps=5)
    # the same kernel over half a second of decode-only steps: the board reaches its power cap and the SM clock
    # settles lower than in the burst above
    rf_sust = decode_roofline(torch, lib, sh, w.ctx_lens, all_reqs, q, out, steps=150)
    rf_single = single_launch_rate(torch, lib, sh, w.ctx_lens, all_reqs, q, out)
    # the same with PS_FLAG_ATTN_PLAIN_LAUNCH: no set-up under the predecessor's tail (the default has it)
    elib = make_ctx(B, w, K, V, sh.num_gpu_blocks, max_batch=nreq, host_pool_bytes=64 << 20,
                    flags=B.PS_FLAG_ATTN_PLAIN_LAUNCH)
    for r, n in wl.build_order_round_robin(w):
        assert elib.kv_alloc(r, n) == 0, elib.last_error()
    rf_single_plain = single_launch_rate(torch, elib, sh, w.ctx_lens, all_reqs, q, out)
    elib.destroy()
    del elib
    clocks = sampler.stop()

    # ---- end-to-end arm: the same pass through ps_step_host (host buffers in, host buffers out)
    e2e_recs = [swap_workload_step(torch, B, lib, w, q, out, q_res, out_res, budget, e2e_bufs)
                for _ in range(max(1, min(args.steps, 2)))]
    e2e_ms = sum(r["out_ms"] + r["in_ms"] for r in e2e_recs)
    (e2e_ms,) = group.max_over_ranks([e2e_ms])
    row_bytes = sh.num_layers * sh.num_q_heads * sh.head_dim * 2
    io_bytes = sum(r["steps_out"] * n_res + r["steps_in"] * nreq for r in e2e_recs) * row_bytes / len(e2e_recs)
    e2e = {"value": 2 * victim_bytes * len(e2e_recs) * world / e2e_ms / 1e6, "unit": UNIT,
           "h2d_bytes_per_step": int(victim_bytes + io_bytes), "d2h_bytes_per_step": int(victim_bytes + io_bytes),
           "api": "ps_step_host: queries from and outputs to pinned host memory through the C ABI, every decode step",
           "decode_steps_per_pass": sum(r["steps_out"] + r["steps_in"] for r in e2e_recs) / len(e2e_recs),
           "decode_step_us_during_swap_out": sum(r["out_ms"] for r in e2e_recs) / sum(r["steps_out"] for r in e2e_recs) * 1e3,
           "note": "bytes per step = the swapped KV each way (host images live in pinned host memory by "
                   "definition) + the queries (up) / outputs (down) of every decode step: 48 rows while the "
                   "offload drains, 64 rows in the reload step"}

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "llama8b_swap", "layers": sh.num_layers, "kv_heads": sh.num_kv_heads,
                   "q_heads": sh.num_q_heads, "head_dim": sh.head_dim, "block_size": sh.block_size,
                   "gpu_blocks": sh.num_gpu_blocks, "resident_requests": nreq, "victims": len(w.victims),
                   "victim_bytes": victim_bytes, "copy_budget_mib_per_step": args.budget_mib,
                   "l2": "inputs larger than L2 (6 GiB swapped each way, ~0.6 GiB of KV read per attention launch)",
                   "parallelism": "independent replicas" if world > 1 else "single GPU"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "wall_ms": wall_ms,
    }
    flat = {}                                        # scalars that go into the roofline object (see below)
    if rank == 0:
        ratio = read_traffic_ratio()
        read_peak = B.ps_hbm_probe(4 << 30, 0, 5)
        copy_peak = B.ps_hbm_probe(2 << 30, 1, 5)
        result["roofline"] = {
            "kernel": "decode_attn_mma_kernel (paged GQA decode attention, split-KV combined in the kernel)",
            "bound": "hbm", "achieved": rf_all["gbs"], "peak": hbm_peak, "peak_kind": f"{peak_kind} copy bandwidth",
            "unit": "GB/s", "frac": rf_all["gbs"] / hbm_peak,
            "traffic": ratio * rf_all["algorithmic_bytes_per_launch"] if ratio else None,
            "algorithmic_bytes_per_launch": rf_all["algorithmic_bytes_per_launch"],
            "us_per_launch": rf_all["us_per_layer"], "launches_per_layer": rf_all["launches_per_layer"],
            "how": "CUDA events around 5 decode-only ps_step calls (32 launches each, 64 requests); launches of "
                   "consecutive layers overlap head to tail",
            "frac_of_nominal_8TBs": rf_all["gbs"] / 8000.0,
            # the kernel only reads: a read-only stream of this library's probe kernel, measured in this run,
            # is the like-for-like ceiling (the copy peak counts read + written bytes)
            "read_peak_gbs": read_peak, "frac_of_read_peak": rf_all["gbs"] / read_peak,
            "probe_copy_peak_gbs": copy_peak,
            "single_launch_gbs": rf_single["gbs"], "single_launch_us": rf_single["us_per_launch"],
            "single_launch_frac": rf_single["gbs"] / hbm_peak,
            "single_launch_frac_of_read_peak": rf_single["gbs"] / read_peak,
            "single_launch_plain_gbs": rf_single_plain["gbs"],
            "single_launch_plain_us": rf_single_plain["us_per_launch"],
            "single_launch_plain_frac": rf_single_plain["gbs"] / hbm_peak,
            "residents48_gbs": rf_res["gbs"], "residents48_us_per_launch": rf_res["us_per_layer"],
            "sustained_150_steps_gbs": rf_sust["gbs"], "sustained_150_steps_us_per_launch": rf_sust["us_per_layer"],
            "sustained_150_steps_frac": rf_sust["gbs"] / hbm_peak,
        }
        result["swap"] = {
            "swap_out_gbs": victim_bytes * args.steps / out_ms / 1e6, "swap_in_gbs": victim_bytes * args.steps / in_ms / 1e6,
            "out_ms_per_step": [round(r["out_ms"], 2) for r in recs], "in_ms_per_step": [round(r["in_ms"], 2) for r in recs],
            "swap_out_frac_of_link": victim_bytes * args.steps / out_ms / 1e6 / link["d2h_gbs"],
            "swap_in_frac_of_link": victim_bytes * args.steps / in_ms / 1e6 / link["h2d_gbs"],
            "decode_steps_during_out": recs[-1]["steps_out"], "decode_steps_during_in": recs[-1]["steps_in"],
            "decode_step_us_during_out": recs[-1]["out_ms"] / recs[-1]["steps_out"] * 1e3,
            "decode_step_us_no_swap": rf_res["step_us"],
            "link": link,
        }
        sw = result["swap"]
        flat.update({"swap_out_gbs": sw["swap_out_gbs"], "swap_in_gbs": sw["swap_in_gbs"],
                     "swap_out_frac_of_link": sw["swap_out_frac_of_link"],
                     "swap_in_frac_of_link": sw["swap_in_frac_of_link"], "link_h2d_gbs": link["h2d_gbs"],
                     "link_d2h_gbs": link["d2h_gbs"], "link_duplex_sum_gbs": link["duplex_sum_gbs"],
                     "decode_step_us_during_swap_out": sw["decode_step_us_during_out"],
                     "decode_step_us_no_swap_48req": sw["decode_step_us_no_swap"]})
        result["proactive_offload"] = proactive_offload_leg(torch, B, lib, w)
        # the swap path's own gather / scatter kernels alone (the scatters overwrite pool blocks: last use of lib)
        kr = kernel_rates(torch, B, lib, sh, sh.num_gpu_blocks, hbm_peak)
        result["gather_scatter_alone"] = kr
        for name, row in kr.items():
            if isinstance(row, dict):
                flat[name + "_gbs_rw"] = row["gbs_rw"]
                flat[name + "_frac_of_hbm"] = row["frac_of_hbm"]
                flat[name + "_us"] = row["us_per_launch"]
    lib.destroy()
    del lib
    if rank == 0:
        # diagnostics pass with per-launch events (not part of any reported rate above): engine and kernel
        # rates inside a step, beside attention; the events themselves slow this pass down
        plib = fresh_ctx(B.PS_FLAG_PROFILE)
        swap_workload_step(torch, B, plib, w, q, out, q_res, out_res, budget)
        prof = plib.get_profile(reset=True)
        result["swap"].update({
            "d2h_engine_gbs": prof["d2h_bytes"] / prof["d2h_ms"] / 1e6 if prof["d2h_ms"] > 0 else None,
            "h2d_engine_gbs": prof["h2d_bytes"] / prof["h2d_ms"] / 1e6 if prof["h2d_ms"] > 0 else None,
            "gather_in_step_gbs_rw": 2 * prof["gather_bytes"] / prof["gather_ms"] / 1e6 if prof["gather_ms"] > 0 else None,
            "scatter_in_step_gbs_rw": 2 * prof["scatter_bytes"] / prof["scatter_ms"] / 1e6 if prof["scatter_ms"] > 0 else None,
            "gather_launches": prof["gather_launches"], "scatter_launches": prof["scatter_launches"],
        })
        flat["gather_beside_attention_gbs_rw"] = result["swap"]["gather_in_step_gbs_rw"]
        flat["scatter_beside_attention_gbs_rw"] = result["swap"]["scatter_in_step_gbs_rw"]
        plib.destroy()
        del plib
    if rank == 0 and not args.no_overlap:
        ov = overlap_sweep(torch, B, K, V, hbm_peak)
        result["overlap"] = ov
        flat["overlap_attn_gbs"] = ov["attn_gbs"]
        flat["overlap_hideable_budget_mib"] = ov["hideable_budget_mib"]
        for key, tag in (("pipelined_16MiB", "16mib"), ("pipelined_64MiB", "64mib"), ("pipelined_256MiB", "256mib"),
                         ("pipelined_adaptive", "adaptive"), ("pipelined_unlimited", "unlimited"),
                         ("sync_reload_256MiB", "sync256mib")):
            if key in ov:
                row = ov[key]
                flat[f"overlap_{tag}_hidden_frac"] = row["hidden_frac"]
                flat[f"overlap_{tag}_step_us_with_reload"] = row["step_us_with_reload"]
                flat[f"overlap_{tag}_step_us_no_reload"] = row["step_us_no_reload"]
                flat[f"overlap_{tag}_reload_alone_gbs"] = row["reload_alone_gbs"]
                flat[f"overlap_{tag}_reload_alone_frac_of_link"] = row["reload_alone_gbs"] / link["h2d_gbs"]
    del K, V
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_extra:
        # the two other full-size workloads, compact: long context (70B shape) and priority churn (32B shape)
        try:
            lc = long_context_leg(torch, B, hbm_peak, compact=True)
            result["long_context"] = lc
            flat.update({"longctx_offload_under_decode_gbs": lc["offload_under_decode_gbs"],
                         "longctx_offload_alone_gbs": lc["offload_alone_gbs"],
                         "longctx_adaptive_hidden_frac": lc["pipelined_adaptive"]["hidden_frac"],
                         "longctx_adaptive_reload_gbs": lc["pipelined_adaptive"]["reload_under_decode_gbs"],
                         "longctx_adaptive_step_us_with_reload": lc["pipelined_adaptive"]["step_us_with_reload"],
                         "longctx_step_us_no_reload": lc["pipelined_adaptive"]["step_us_no_reload"],
                         "longctx_256mib_hidden_frac": lc["pipelined_256MiB"]["hidden_frac"]})
        except Exception as e:                       # e.g. the box cannot pin 10 GiB
            result["long_context"] = {"skipped": repr(e)[:200]}
        torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_extra:
        try:
            cl = churn_loop_leg(torch, B, hbm_peak, 80)
            result["churn_closed_loop"] = cl
            flat.update({"churn_reload_gbs_sustained": cl["reload_gbs_sustained"],
                         "churn_offload_gbs_sustained": cl["offload_gbs_sustained"],
                         "churn_step_ms_mean": cl["step_ms_mean"], "churn_no_swap_step_ms_model": cl["no_swap_step_ms_model"],
                         "churn_hidden_frac_estimate": cl["hidden_frac_estimate"], "churn_evicted": cl["evicted"],
                         "churn_readmitted": cl["readmitted"], "churn_rule_skips": cl["skipped"]})
        except Exception as e:
            result["churn_closed_loop"] = {"skipped": repr(e)[:200]}
        torch.cuda.empty_cache()
    if rank == 0 and "roofline" in result:
        result["roofline"].update(flat)
    if rank == 0 and world == 1:
        result["cpu_baseline"] = time_oracle(args.cpu_seconds, sh.num_layers, sum(w.ctx_lens))
    group.close()
    if rank == 0:
        print(json.dumps(result))


def spawn_replicas(args):
    """`python bench.py --gpus N` outside a launcher: starts the N replicas itself (rank 0 prints the line)."""
    from paper_2512_12928_b200 import replicas
    rcs = replicas.spawn([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], args.gpus)
    sys.exit(max(abs(rc) for rc in rcs))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--budget-mib", type=int, default=-1, help="copy budget per step in MiB for phase B (-1 = unlimited)")
    ap.add_argument("--staging-mib", type=int, default=0, help="device staging per direction in MiB (0 = library default)")
    ap.add_argument("--no-overlap", action="store_true", help="skip the overlap budget sweep")
    ap.add_argument("--no-extra", action="store_true", help="skip the compact long-context and churn legs")
    ap.add_argument("--cpu-seconds", type=float, default=10.0)
    ap.add_argument("--workload", default="llama8b_swap", choices=["llama8b_swap", "long_context", "churn", "decode_shapes"],
                    help="llama8b_swap is the headline line; the others print a line of their own (one GPU)")
    ap.add_argument("--churn-steps", type=int, default=100)
    ap.add_argument("--churn-rounds", type=int, default=200, help="rounds of the closed loop (--workload churn)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_replicas(args)
    elif args.workload != "llama8b_swap":
        run_extra(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
