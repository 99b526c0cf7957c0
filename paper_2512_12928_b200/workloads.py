"""Seeded synthetic workloads: shapes, context lengths, victims, free orders, raw bf16 bit patterns.

This module only *draws inputs*.  It holds none of the method's arithmetic (no block copy, no
budget rule, no attention) so that both the CUDA path and the CPU checker can take their inputs
from it without sharing any of the computation under test.

The five workloads mirror the serving situations the paper's block management is built for
(Section 4.3: preemption spills a request's KV blocks to host memory, readmission reloads them
layer by layer under a copy budget).  The paper's traces (ShareGPT, Azure, BurstGPT, QwenTrace,
an industrial trace) are not available offline; these inputs stand in for them with the KV shapes
of the model families the paper serves and context-length ranges of the same kind.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

SEED_BASE = 251212928
MiB = 1 << 20
GiB = 1 << 30


@dataclass
class KVShape:
    """Geometry of a paged KV cache (notation of Section 4.3: s_blk = block_size)."""
    num_layers: int
    num_kv_heads: int
    num_q_heads: int
    head_dim: int
    block_size: int
    num_gpu_blocks: int

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def slab_elems(self) -> int:
        """Elements of one K (or V) slab: one block of one layer."""
        return self.block_size * self.num_kv_heads * self.head_dim

    @property
    def slab_bytes(self) -> int:
        return self.slab_elems * 2

    @property
    def layer_block_bytes(self) -> int:
        """K slab + V slab of one block in one layer."""
        return 2 * self.slab_bytes

    @property
    def block_bytes(self) -> int:
        """One block across all layers: the unit the copy budget counts."""
        return self.num_layers * self.layer_block_bytes

    def blocks_for(self, n_tokens: int) -> int:
        return (n_tokens + self.block_size - 1) // self.block_size


@dataclass
class Workload:
    name: str
    index: int
    shape: KVShape
    seed: int
    ctx_lens: List[int]                 # context length of every live request, request id = position
    victims: List[int]                  # request ids preempted (swapped out, later reloaded)
    free_order: np.ndarray              # seeded permutation: order in which block ids are handed out
    decode_batch: Optional[int] = None  # number of requests that decode each step
    budgets: List[int] = field(default_factory=list)   # copy budgets in bytes (per step)
    notes: str = ""

    @property
    def total_blocks_needed(self) -> int:
        return sum(self.shape.blocks_for(c) for c in self.ctx_lens)


def _rng(index: int, stream: int = 0) -> np.random.Generator:
    return np.random.default_rng([SEED_BASE + index, stream])


def _free_order(index: int, num_blocks: int) -> np.ndarray:
    return _rng(index, 1).permutation(num_blocks).astype(np.int32)


def lognormal_ctx(rng: np.random.Generator, n: int, mean: float, sigma: float, cap: int, floor: int = 16):
    mu = math.log(mean) - 0.5 * sigma * sigma
    x = rng.lognormal(mu, sigma, size=n)
    return [int(min(cap, max(floor, round(v)))) for v in x]


def tiny(num_requests: int = 8) -> Workload:
    shape = KVShape(2, 4, 8, 64, 16, 256)
    rng = _rng(0)
    ctx = [int(v) for v in rng.integers(16, 257, size=num_requests)]
    victims = sorted(int(v) for v in rng.choice(num_requests, size=num_requests // 2, replace=False))
    return Workload("tiny", 0, shape, SEED_BASE, ctx, victims, _free_order(0, 256), decode_batch=num_requests,
                    budgets=[-1])


def llama8b_swap(num_requests: int = 64, num_victims: int = 16, num_gpu_blocks: int = 20480,
                 ctx_lo: int = 1024, ctx_hi: int = 4096) -> Workload:
    """32 layers, 8 KV heads, head_dim 128, block 16; 64 residents 1k-4k tokens; preempt 16."""
    shape = KVShape(32, 8, 32, 128, 16, num_gpu_blocks)
    rng = _rng(1)
    ctx = [int(v) for v in rng.integers(ctx_lo, ctx_hi + 1, size=num_requests)]
    victims = sorted(int(v) for v in rng.choice(num_requests, size=num_victims, replace=False))
    return Workload("llama8b_swap", 1, shape, SEED_BASE + 1, ctx, victims, _free_order(1, num_gpu_blocks),
                    decode_batch=num_requests, budgets=[-1])


def overlap(decode_batch: int = 128, num_preempted: int = 8, num_gpu_blocks: int = 24576,
            mean: float = 2048.0, sigma: float = 0.8, cap: int = 8192) -> Workload:
    """Same 8B shape, GQA 4, decode batch 128 lognormal contexts; 8 preempted requests reload."""
    shape = KVShape(32, 8, 32, 128, 16, num_gpu_blocks)
    rng = _rng(2)
    ctx = lognormal_ctx(rng, decode_batch + num_preempted, mean, sigma, cap)
    victims = list(range(decode_batch, decode_batch + num_preempted))
    return Workload("overlap", 2, shape, SEED_BASE + 2, ctx, victims, _free_order(2, num_gpu_blocks),
                    decode_batch=decode_batch, budgets=[16 * MiB, 64 * MiB, 256 * MiB],
                    notes="sigma of the lognormal is this build's choice; the paper gives none")


def churn(num_requests: int = 256, num_gpu_blocks: int = 24576, steps: int = 200,
          ctx_lo: int = 512, ctx_hi: int = 16384) -> Workload:
    """Qwen3-32B-shaped KV (64 layers), two priority classes, per-step swap-out/in of 2-16 requests.

    The literal configuration (256 live requests of mean 8448 tokens at 256 KiB per token) needs
    about 528 GiB and cannot be resident at once; it is read as an oversubscribed instance: a fixed
    device pool, a pinned host pool, and a waiting set with no KV.
    """
    shape = KVShape(64, 8, 64, 128, 16, num_gpu_blocks)
    rng = _rng(3)
    ctx = [int(v) for v in rng.integers(ctx_lo, ctx_hi + 1, size=num_requests)]
    w = Workload("churn", 3, shape, SEED_BASE + 3, ctx, [], _free_order(3, num_gpu_blocks),
                 decode_batch=num_requests, budgets=[256 * MiB])
    w.priority = [int(v) for v in rng.integers(0, 2, size=num_requests)]   # 0 = high, 1 = low (50/50)
    w.steps = steps
    return w


def long_context(decode_batch: int = 64, ctx: int = 4096, long_ctx: int = 32768,
                 num_gpu_blocks: int = 9344) -> Workload:
    """70B-shaped KV (80 layers, block 32): one 32k-token request swapped out and reloaded."""
    shape = KVShape(80, 8, 64, 128, 32, num_gpu_blocks)
    ctxs = [ctx] * decode_batch + [long_ctx]
    return Workload("long_context", 4, shape, SEED_BASE + 4, ctxs, [decode_batch],
                    _free_order(4, num_gpu_blocks), decode_batch=decode_batch, budgets=[256 * MiB])


def churn_script(w: Workload, host_pool_bytes: int, fill_frac: float = 0.90, host_fill_frac: float = 0.75):
    """Deterministic per-step action list for the churn workload.

    Pure bookkeeping over block *counts* (no KV bytes, no budget rule): decides, from the seed, which
    requests start resident, which start on host, and for each step which low-priority residents
    are asked out and which host-resident requests are asked in, clipped to capacity so that every
    action is legal.  Capacity is tracked conservatively (blocks of a request leaving this step do
    not count as free until the next step).
    """
    sh = w.shape
    rng = _rng(w.index, 7)
    nblk = [sh.blocks_for(c) for c in w.ctx_lens]
    order = [int(v) for v in rng.permutation(len(w.ctx_lens))]
    resident, host, waiting = [], [], []
    used = 0
    host_used = 0
    for r in order:
        if used + nblk[r] <= fill_frac * sh.num_gpu_blocks:
            resident.append(r)
            used += nblk[r]
        elif host_used + nblk[r] * sh.block_bytes <= host_fill_frac * host_pool_bytes:
            host.append(r)
            host_used += nblk[r] * sh.block_bytes
        else:
            waiting.append(r)
    init = dict(resident=list(resident), host=list(host), waiting=list(waiting))
    steps = []
    free_blocks = sh.num_gpu_blocks - used
    host_free = host_pool_bytes - host_used
    pending_free = 0          # blocks leaving in the previous step: usable from this step on
    pending_host_free = 0
    for _ in range(w.steps):
        free_blocks += pending_free
        host_free += pending_host_free
        pending_free = 0
        pending_host_free = 0
        n_out = int(rng.integers(2, 17))
        n_in = int(rng.integers(2, 17))
        low = [r for r in resident if w.priority[r] == 1]
        outs = []
        for r in [low[int(i)] for i in rng.permutation(len(low))][:n_out]:
            need = nblk[r] * sh.block_bytes
            if need <= host_free:
                outs.append(r)
                host_free -= need
        ins = []
        for r in [host[int(i)] for i in rng.permutation(len(host))][:n_in]:
            if nblk[r] <= free_blocks:
                ins.append(r)
                free_blocks -= nblk[r]
        for r in outs:
            resident.remove(r)
            pending_free += nblk[r]
        for r in ins:
            host.remove(r)
            pending_host_free += nblk[r] * sh.block_bytes
        # requests that finish loading become resident; requests that left become host-resident
        steps.append(dict(out=outs, inn=ins))
        resident.extend(ins)
        host.extend(outs)
    return init, steps


def by_index(index: int, **kw) -> Workload:
    return [tiny, llama8b_swap, overlap, churn, long_context][index](**kw)


# ---------------------------------------------------------------------------------------------
# raw values
# ---------------------------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bfloat16 (ties to even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def randn_bf16_bits(rng: np.random.Generator, shape) -> np.ndarray:
    """N(0,1) samples as bf16 bit patterns (uint16)."""
    return f32_to_bf16_bits(rng.standard_normal(size=shape, dtype=np.float32))


def make_pools_numpy(w: Workload, stream: int = 11):
    """K and V pools as uint16 [L][num_blocks][S][Hkv][D], N(0,1) bf16 (small workloads only)."""
    sh = w.shape
    rng = _rng(w.index, stream)
    dims = (sh.num_layers, sh.num_gpu_blocks, sh.block_size, sh.num_kv_heads, sh.head_dim)
    return randn_bf16_bits(rng, dims), randn_bf16_bits(rng, dims)


def make_queries_numpy(w: Workload, batch: int, stream: int = 13) -> np.ndarray:
    """Decode queries as uint16 bf16 bits [L][batch][Hq][D], N(0,1)."""
    sh = w.shape
    return randn_bf16_bits(_rng(w.index, stream), (sh.num_layers, batch, sh.num_q_heads, sh.head_dim))


def build_order_round_robin(w: Workload):
    """Allocation script that fragments the tables: one block per request per turn.

    Returns a list of (request id, n_tokens_total) calls for kv_alloc, in issue order.
    """
    sh = w.shape
    calls = []
    remaining = {r: c for r, c in enumerate(w.ctx_lens)}
    have = {r: 0 for r in remaining}
    while remaining:
        for r in sorted(remaining):
            have[r] = min(w.ctx_lens[r], have[r] + sh.block_size)
            calls.append((r, have[r]))
            if have[r] >= w.ctx_lens[r]:
                del remaining[r]
    return calls
