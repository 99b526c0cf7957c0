"""Plain CPU checker for KV-block swap, copy-budget consumption and paged decode attention.

TEST INFRASTRUCTURE ONLY.  Nothing in the product path may import this module: it exists so that
the tests, the smoke check and the benchmark's CPU-baseline leg have an independent, slow,
obviously-correct statement of what the hot path computes.  It shares no code with the CUDA
library and imports nothing from it.

What it follows (ProServe, Section 4.3 "Efficient Block Management", and Appendix B):

* Eviction spills a request's KV blocks to host memory instead of dropping them; the device
  blocks can be reclaimed only after the transfer has completed ("Asynchronous Offloading").
  -> `swap_out` copies the blocks byte for byte into a host image; `reap` gives the blocks back.
* Offloading can also run ahead of eviction: a copy for every n_off newly filled blocks of a request
  ("Asynchronous Offloading").  -> `offload_progress`; `swap_out` then copies only the rest.  (The paper
  drops the not-yet-copied tail at eviction and recomputes it; without recomputation it is copied.)
* A readmitted request gets its KV restored layer by layer ("Pipelined Reloading"; Appendix B:
  one completion event per layer chunk).  -> `swap_in_begin`, `swap_in_layer`.
* A per-step host-to-device copy budget B_copy (in blocks) is consumed in queue order at request
  granularity: all missing blocks b_miss of a request if they fit, otherwise a partial copy with
  the residual budget ("Put it Together"; Alg. 1: GetCopyBudget, ConsumeCopyBudget).  -> `step_plan`, `step`.
  The beta admission test of that paragraph (SatisfyCopyCondition) depends on the scheduler's
  computable-token count: `step_plan` applies it to the requests for which the caller supplies that
  count and always allows the partial copy for the others; a request decodes only once complete.
* The number of blocks to reload per step, B_copy, follows the three-case procedure of "Adaptive
  Copy-Budget Control" with the decode latency model of Section 4.1.  -> `copy_budget`.
* The computation the reload overlaps with is the decode forward; its KV-consuming part is
  attention over the paged cache.  The paper gives no formula; the textbook definition
  softmax(q K^T / sqrt(d)) V is used, in float64, over KV gathered through the block table.

Parity pins (tests/test_oracle_*.py): brute-force loops on tiny inputs, torch's own fp64
scaled-dot-product attention on contiguous KV, scipy's logsumexp, closed forms (one token, equal
keys, two-token sigmoid mix), masking and permutation invariants, hand-worked budget schedules,
round-trip and ownership invariants.  The adaptive budget is pinned by hand-worked cases and an
exhaustive scan (tests/test_adaptive_budget.py), proactive offloading by element loops and equality
with on-demand offloading (tests/test_proactive_offload.py), the eviction policy, the partial-copy
rule and the queue ordering by hand-worked cases and properties (tests/test_eviction_policy.py), the
batch latency estimator and the reload-versus-recompute cost by hand-worked values and the identity that
chunking leaves a causal prefill's cost unchanged (tests/test_resume_cost.py).
No function here is "parity unpinned".

Layouts (this build's reading; the paper is silent): per layer a K pool and a V pool,
uint16[num_blocks][S][Hkv][D] holding bf16 bit patterns; host image of a request
uint16[L][n_blk][2][S][Hkv][D] (layer-major, K slab then V slab per block).
"""
from __future__ import annotations

import math
from collections import deque
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

# status codes (same numeric contract as the C header; restated here, not imported)
OK = 0
ERR_INVALID = -1
ERR_NOMEM = -2
ERR_HOST_NOMEM = -3
ERR_STATE = -4
ERR_BUSY = -5

# request states
ST_RESIDENT = 1
ST_SWAPPING_OUT = 2
ST_HOST = 3
ST_SWAPPING_IN = 4


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of bfloat16 bit patterns as float64 (bf16 is the top half of a float32)."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


class _Req:
    __slots__ = ("n_tokens", "table", "state", "image", "image_bytes", "layer_done", "old_table", "segs")

    def __init__(self):
        self.n_tokens = 0
        self.table: List[int] = []
        self.state = ST_RESIDENT
        self.image: Optional[np.ndarray] = None
        self.image_bytes = 0
        self.layer_done: List[int] = []
        self.old_table: List[int] = []
        # host image: segments (blk_lo, blk_hi, array [L][hi - lo][2][S][Hkv][D] or None without pools);
        # `image` is the array of the only segment when there is exactly one
        self.segs: List[Tuple[int, int, Optional[np.ndarray]]] = []


class PsOracle:
    def __init__(self, num_layers: int, num_kv_heads: int, num_q_heads: int, head_dim: int, block_size: int,
                 num_gpu_blocks: int, initial_free_order: Optional[Sequence[int]] = None,
                 kpool: Optional[np.ndarray] = None, vpool: Optional[np.ndarray] = None,
                 host_pool_bytes: Optional[int] = None):
        self.L, self.Hkv, self.Hq, self.D, self.S = num_layers, num_kv_heads, num_q_heads, head_dim, block_size
        self.num_blocks = num_gpu_blocks
        assert num_q_heads % num_kv_heads == 0
        self.G = num_q_heads // num_kv_heads
        order = list(range(num_gpu_blocks)) if initial_free_order is None else [int(v) for v in initial_free_order]
        assert sorted(order) == list(range(num_gpu_blocks)), "initial_free_order must be a permutation"
        # the stack's top is its last element; order[0] is handed out first
        self.free: List[int] = order[::-1]
        self.reqs: Dict[int, _Req] = {}
        self.K = kpool
        self.V = vpool
        if kpool is not None:
            want = (self.L, self.num_blocks, self.S, self.Hkv, self.D)
            assert kpool.shape == want and vpool.shape == want and kpool.dtype == np.uint16
        self.out_fifo: deque = deque()       # swap-outs whose blocks are not yet reclaimed, issue order
        self.in_fifo: deque = deque()        # reload queue, issue order
        self.host_pool_bytes = host_pool_bytes
        self.host_used = 0

    # ------------------------------------------------------------------ sizes
    @property
    def block_bytes(self) -> int:
        """Bytes of one block across all layers (K and V): the copy budget's unit."""
        return self.L * 2 * self.S * self.Hkv * self.D * 2

    def blocks_for(self, n_tokens: int) -> int:
        return -(-n_tokens // self.S)

    # ------------------------------------------------------------------ allocation
    def kv_alloc(self, req: int, n_tokens_total: int) -> int:
        """Grow request `req` to hold n_tokens_total tokens; all-or-nothing; pops ids one at a time."""
        if n_tokens_total < 0:
            return ERR_INVALID
        r = self.reqs.get(req)
        if r is not None and r.state != ST_RESIDENT:
            return ERR_STATE
        have = 0 if r is None else len(r.table)
        if r is not None and n_tokens_total < r.n_tokens:
            return ERR_INVALID
        need = self.blocks_for(n_tokens_total) - have
        if need > len(self.free):
            return ERR_NOMEM
        if r is None:
            r = self.reqs[req] = _Req()
        for _ in range(need):
            r.table.append(self.free.pop())
        r.n_tokens = n_tokens_total
        return OK

    def kv_free(self, req: int) -> int:
        r = self.reqs.get(req)
        if r is None:
            return ERR_INVALID
        if r.state in (ST_SWAPPING_OUT, ST_SWAPPING_IN):
            return ERR_BUSY
        if r.state == ST_RESIDENT:
            self.free.extend(r.table)            # pushed in table order: last entry ends on top
        self._release_image(r)
        del self.reqs[req]
        return OK

    def block_table(self, req: int) -> Tuple[List[int], int]:
        r = self.reqs[req]
        return list(r.table), r.state

    def num_free_blocks(self) -> int:
        return len(self.free)

    # ------------------------------------------------------------------ swap-out
    def _image_bytes(self, n_blk: int) -> int:
        return n_blk * self.block_bytes

    def _release_image(self, r: _Req) -> None:
        self.host_used -= r.image_bytes
        r.image_bytes = 0
        r.image = None
        r.segs = []

    def _host_issued(self, r: _Req) -> int:
        return r.segs[-1][1] if r.segs else 0

    def _offload_segment(self, r: _Req, lo: int, hi: int) -> int:
        """Byte-for-byte copy of logical blocks [lo, hi), every layer, into a new image segment."""
        nbytes = self._image_bytes(hi - lo)
        if self.host_pool_bytes is not None and self.host_used + nbytes > self.host_pool_bytes:
            return ERR_HOST_NOMEM
        r.image_bytes += nbytes
        self.host_used += nbytes
        img = None
        if self.K is not None:
            img = np.empty((self.L, hi - lo, 2, self.S, self.Hkv, self.D), dtype=np.uint16)
            for l in range(self.L):
                for j in range(lo, hi):
                    img[l, j - lo, 0] = self.K[l, r.table[j]]
                    img[l, j - lo, 1] = self.V[l, r.table[j]]
        r.segs.append((lo, hi, img))
        r.image = img if len(r.segs) == 1 else None
        return OK

    def offload_progress(self, req: int, n_off: int):
        """Proactive incremental offloading ("Asynchronous Offloading"): a copy for every n_off newly filled
        blocks.  Copies the largest whole number of groups of n_off completely filled, not yet offloaded
        blocks; the request stays resident.  Returns (status, blocks copied)."""
        r = self.reqs.get(req)
        if n_off <= 0 or r is None:
            return ERR_INVALID, 0
        if r.state != ST_RESIDENT:
            return ERR_STATE, 0
        lo = self._host_issued(r)
        groups = (r.n_tokens // self.S - lo) // n_off
        if groups <= 0:
            return OK, 0
        rc = self._offload_segment(r, lo, lo + groups * n_off)
        return rc, (groups * n_off if rc == OK else 0)

    def offload_sweep(self, reqs: Sequence[int], n_off: Sequence[int]):
        """The same trigger over a batch, request r with its own threshold n_off^r ("Asynchronous Offloading":
        lower-priority requests get smaller thresholds).  Requests that are not resident are skipped; stops at
        the first failure.  Returns (status, blocks copied)."""
        if any(n <= 0 for n in n_off):
            return ERR_INVALID, 0
        total = 0
        for req, n in zip(reqs, n_off):
            r = self.reqs.get(req)
            if r is None or r.state != ST_RESIDENT:
                continue
            rc, issued = self.offload_progress(req, n)
            total += issued
            if rc != OK:
                return rc, total
        return OK, total

    def host_blocks(self, req: int) -> int:
        """b_host of Section 4.3: blocks of the request that have a copy on host."""
        return self._host_issued(self.reqs[req])

    def swap_out(self, req: int) -> int:
        """Spill the request's blocks to a host image; blocks stay owned until `reap`."""
        r = self.reqs.get(req)
        if r is None:
            return ERR_INVALID
        if r.state != ST_RESIDENT:
            return ERR_STATE
        n = len(r.table)
        lo = self._host_issued(r)
        if lo < n or not r.segs:                 # what proactive offloading has not covered goes out now
            rc = self._offload_segment(r, lo, n)
            if rc != OK:
                return rc
        r.state = ST_SWAPPING_OUT
        self.out_fifo.append(req)
        return OK

    def reap(self, count: Optional[int] = None) -> int:
        """Transfers complete in issue order; give the blocks of the first `count` back (all if None)."""
        done = 0
        while self.out_fifo and (count is None or done < count):
            r = self.reqs[self.out_fifo.popleft()]
            self.free.extend(r.table)
            r.old_table = r.table
            r.table = []
            r.state = ST_HOST
            done += 1
        return done

    # ------------------------------------------------------------------ swap-in
    def swap_in_begin(self, req: int) -> int:
        """Queue a host-resident request for reload and give it fresh blocks (all-or-nothing)."""
        r = self.reqs.get(req)
        if r is None:
            return ERR_INVALID
        if r.state != ST_HOST:
            return ERR_STATE
        n = self.blocks_for(r.n_tokens)
        if n > len(self.free):
            return ERR_NOMEM
        r.table = [self.free.pop() for _ in range(n)]
        r.layer_done = [0] * self.L
        r.state = ST_SWAPPING_IN
        self.in_fifo.append(req)
        if n == 0:                               # nothing to restore: resident at once
            r.state = ST_RESIDENT
            self._release_image(r)
            r.old_table = []
            self.in_fifo.remove(req)
        return OK

    def swap_in_cancel(self, req: int) -> int:
        """Withdraw a queued reload that has not started; the fresh blocks go back in table order."""
        r = self.reqs.get(req)
        if r is None:
            return ERR_INVALID
        if r.state != ST_SWAPPING_IN:
            return ERR_STATE
        if any(r.layer_done):
            return ERR_BUSY
        self.free.extend(r.table)
        r.table = []
        r.state = ST_HOST
        self.in_fifo.remove(req)
        return OK

    def swap_in_layer(self, req: int, layer: int, blk_lo: int, blk_hi: int) -> int:
        """Restore logical blocks [blk_lo, blk_hi) of one layer from the host image into the fresh blocks."""
        r = self.reqs.get(req)
        if r is None:
            return ERR_INVALID
        if r.state != ST_SWAPPING_IN:
            return ERR_STATE
        n = len(r.table)
        if not (0 <= layer < self.L) or not (0 <= blk_lo <= blk_hi <= n) or blk_lo != r.layer_done[layer]:
            return ERR_INVALID
        if self.K is not None:
            for j in range(blk_lo, blk_hi):
                b = r.table[j]
                lo, hi, img = next(sg for sg in r.segs if sg[0] <= j < sg[1])
                self.K[layer, b] = img[layer, j - lo, 0]
                self.V[layer, b] = img[layer, j - lo, 1]
        r.layer_done[layer] = blk_hi
        if all(d == n for d in r.layer_done):
            r.state = ST_RESIDENT
            self._release_image(r)
            r.old_table = []
            self.in_fifo.remove(req)
        return OK

    # ------------------------------------------------------------------ copy budget
    def missing_blocks(self, req: int) -> int:
        """b_miss of Section 4.3: blocks on host that are not yet on the device."""
        r = self.reqs[req]
        if r.state != ST_SWAPPING_IN:
            return 0
        return len(r.table) - min(r.layer_done)

    def step_plan(self, copy_budget_bytes: int, rule: Optional[Dict[int, Tuple[int, int]]] = None,
                  beta: Optional[float] = None) -> List[Tuple[int, int, int]]:
        """Consume the budget over the reload queue in order; returns (req, blk_lo, blk_hi) per request.

        Budget in blocks = floor(bytes / block_bytes) with a block spanning all layers; negative
        means unlimited.  A request whose missing blocks fit is copied whole.  The first one that does
        not fit gets what is left -- always, when `rule` does not list it; when rule[req] =
        (l_comp, l_comp_max) is given, only if the partial-copy test of "Put it Together" passes
        (`copy_condition` with the residual budget), otherwise the request is skipped this round and
        the scheduler proceeds to the next request with the budget unchanged (Alg. 1: `continue`
        after SatisfyCopyCondition fails).
        """
        left = None if copy_budget_bytes < 0 else copy_budget_bytes // self.block_bytes
        plan = []
        for req in self.in_fifo:
            r = self.reqs[req]
            lo = min(r.layer_done)
            miss = len(r.table) - lo
            if miss == 0:
                continue
            if left is not None and left == 0:
                break
            take = miss
            if left is not None and miss > left:
                if rule is not None and req in rule:
                    l_comp, l_comp_max = rule[req]
                    if not copy_condition(l_comp, l_comp_max, miss, left, self.S, beta):
                        continue
                take = left
            plan.append((req, lo, lo + take))
            if left is not None:
                left -= take
        return plan

    def step(self, copy_budget_bytes: int, reqs: Optional[Sequence[int]] = None,
             q_bits: Optional[np.ndarray] = None, rule: Optional[Dict[int, Tuple[int, int]]] = None,
             beta: Optional[float] = None):
        """One engine step: reload under the budget (every layer), then decode the complete requests.

        Returns (plan, decoded mask, out) with out float64 [L][B][Hq][D] (rows of requests that
        did not decode are NaN) or None when no queries were given.
        """
        plan = self.step_plan(copy_budget_bytes, rule, beta)
        for req, lo, hi in plan:
            for l in range(self.L):
                rc = self.swap_in_layer(req, l, lo, hi)
                assert rc == OK, rc
        if reqs is None:
            return plan, None, None
        mask = [1 if (q in self.reqs and self.reqs[q].state == ST_RESIDENT) else 0 for q in reqs]
        out = None
        if q_bits is not None:
            out = np.full((self.L, len(reqs), self.Hq, self.D), np.nan)
            live = [i for i, m in enumerate(mask) if m]
            for l in range(self.L):
                if live:
                    o, _ = self.decode_attn(l, q_bits[l][live], [reqs[i] for i in live])
                    out[l, live] = o
        return plan, mask, out

    # ------------------------------------------------------------------ adaptive copy budget
    def step_latency_after(self, reqs: Sequence[int], n_blocks: int, a_d: float, b_d: float, t_c: float) -> float:
        """Estimated time of the decode step (Section 4.1: sum over decode requests of a_d * l_kv + b_d, plus
        t_c) if the reload queue consumed `n_blocks` blocks in order first: the requests of `reqs` that are
        resident now decode, and so do the queued ones whose last missing block is among those blocks."""
        done = set()
        left = n_blocks
        for q in self.in_fifo:
            miss = self.missing_blocks(q)
            if miss == 0:
                continue
            if miss > left:
                break
            left -= miss
            done.add(q)
        t = t_c
        seen = set()
        for q in reqs:
            r = self.reqs.get(q)
            if r is None or q in seen:
                continue
            seen.add(q)
            if r.state == ST_RESIDENT or (r.state == ST_SWAPPING_IN and q in done):
                t += a_d * r.n_tokens + b_d
        return t

    def copy_budget(self, reqs: Sequence[int], a_d: float, b_d: float, t_c: float, t_block: float,
                    t_budget: float) -> Tuple[int, int]:
        """B_copy by the decision procedure of Section 4.3, "Adaptive Copy-Budget Control".

        T_fwd_min: estimated forward time with all host-resident blocks of the queue copied;
        T_trans_max = sum of b_miss * t_block.  (1) T_fwd_min > t_budget: floor(t_budget / t_block).
        (2) otherwise, (i) T_fwd_min > T_trans_max: all missing blocks; (ii) else the largest B_copy whose
        transfer time does not exceed the estimated batch latency.  The paper finds it by binary search,
        relying on a latency that falls monotonically as more is copied (its engine recomputes what is
        missing).  Reading for this decode-only path (no recomputation): the batch latency after copying B
        blocks is `step_latency_after`, a step function that jumps up whenever a queued request becomes
        complete, so "B * t_block <= latency(B)" can turn false and true again; the definition itself is
        taken instead: every B from 0 to B_missing is tried and the largest feasible one returned.
        Returns (B_copy, case) with case 1, 21 or 22.
        """
        b_missing = sum(self.missing_blocks(q) for q in self.in_fifo)
        t_fwd_min = self.step_latency_after(reqs, b_missing, a_d, b_d, t_c)
        t_trans_max = b_missing * t_block
        if t_fwd_min > t_budget:
            return int(math.floor(t_budget / t_block)), 1
        if t_fwd_min > t_trans_max:
            return b_missing, 21
        best = 0
        for b in range(b_missing + 1):
            if b * t_block <= self.step_latency_after(reqs, b, a_d, b_d, t_c):
                best = b
        return best, 22

    # ------------------------------------------------------------------ eviction policy, partial-copy rule
    def select_victims(self, queue: Sequence[int], waited: Sequence[float], tau: float, near_frac: float,
                       blocks_needed: int) -> Tuple[List[int], int]:
        """"Eviction Policy": requests near the tail of the sorted queue are evicted first, except those whose
        waiting time is close to the starvation threshold (reading: waited >= near_frac * tau).  Returns the
        victims in eviction order and the blocks they free (stops once blocks_needed is reached)."""
        victims: List[int] = []
        freed = 0
        for pos in range(len(queue) - 1, -1, -1):
            if freed >= blocks_needed:
                break
            r = self.reqs.get(queue[pos])
            if r is None or r.state != ST_RESIDENT or not r.table or queue[pos] in victims:
                continue
            if waited[pos] >= near_frac * tau:
                continue
            victims.append(queue[pos])
            freed += len(r.table)
        return victims, freed

    # ------------------------------------------------------------------ attention
    def gather_kv(self, layer: int, req: int) -> Tuple[np.ndarray, np.ndarray]:
        """Contiguous K, V of a request for one layer: float64 [ctx][Hkv][D]."""
        r = self.reqs[req]
        ks = np.concatenate([self.K[layer, b] for b in r.table], axis=0)[: r.n_tokens]
        vs = np.concatenate([self.V[layer, b] for b in r.table], axis=0)[: r.n_tokens]
        return bf16_bits_to_f64(ks), bf16_bits_to_f64(vs)

    def decode_attn(self, layer: int, q_bits: np.ndarray, reqs: Sequence[int]):
        """o = softmax(q K^T / sqrt(D)) V per request and query head, float64.

        q_bits: uint16 bf16 patterns [B][Hq][D].  Query head h reads KV head h // G.
        Returns (o [B][Hq][D], lse [B][Hq]) with lse = log sum exp of the scaled logits.
        A request with no tokens gives o = 0 and lse = -inf.
        """
        B = len(reqs)
        q = bf16_bits_to_f64(q_bits).reshape(B, self.Hq, self.D)
        o = np.zeros((B, self.Hq, self.D))
        lse = np.full((B, self.Hq), -np.inf)
        for i, req in enumerate(reqs):
            r = self.reqs[req]
            assert r.state == ST_RESIDENT, "only complete, resident requests decode"
            if r.n_tokens == 0:
                continue
            k, v = self.gather_kv(layer, req)                       # [T][Hkv][D]
            for h in range(self.Hq):
                g = h // self.G
                s = (k[:, g, :] @ q[i, h]) / math.sqrt(self.D)      # [T]
                m = s.max()
                e = np.exp(s - m)
                z = e.sum()
                o[i, h] = (e / z) @ v[:, g, :]
                lse[i, h] = m + math.log(z)
        return o, lse

    def attn_probs(self, layer: int, q_bits: np.ndarray, req: int) -> np.ndarray:
        """Attention weights p [Hq][ctx] of one request (for the rows-sum-to-one pin)."""
        q = bf16_bits_to_f64(q_bits).reshape(self.Hq, self.D)
        k, _ = self.gather_kv(layer, req)
        out = []
        for h in range(self.Hq):
            s = (k[:, h // self.G, :] @ q[h]) / math.sqrt(self.D)
            e = np.exp(s - s.max())
            out.append(e / e.sum())
        return np.stack(out)

    # ------------------------------------------------------------------ invariants
    def check_invariants(self) -> None:
        """free list and all tables partition the block ids; sizes and states are legal."""
        owned: List[int] = list(self.free)
        for rid, r in self.reqs.items():
            assert r.state in (ST_RESIDENT, ST_SWAPPING_OUT, ST_HOST, ST_SWAPPING_IN), (rid, r.state)
            if r.state == ST_HOST:
                assert r.table == [], rid
            else:
                assert len(r.table) == self.blocks_for(r.n_tokens), (rid, len(r.table), r.n_tokens)
            owned.extend(r.table)
        assert len(owned) == self.num_blocks, (len(owned), self.num_blocks)
        assert sorted(owned) == list(range(self.num_blocks)), "a block id is owned twice or lost"


# -------------------------------------------------------------------------------------------------
# Brute-force restatements for tiny inputs (pure Python loops and floats)
# -------------------------------------------------------------------------------------------------

def order_queue(exec_t: Sequence[float], remain: Sequence[float], weight: Sequence[float], eta: float, gamma: float,
                t_c: float, waited: Optional[Sequence[float]] = None, tau: float = 0.0):
    """The request ordering of the SlideBatching algorithm (Section 4.2) with the co-located load judgment.

    The latency budget is the smallest remaining deadline, bounded below by eta.  A request is URGENT if its
    remaining time is below gamma * phi(Q), phi(Q) = t_budget / (t_budget - t_c) * sum of exec.  URGENT requests
    come first in descending density (weight / exec), the others in ascending remaining time; a request whose
    waiting time exceeds the starvation threshold tau is promoted to the head.  Returns (order as indices,
    class per index: 2 starving / 1 urgent / 0 normal, t_budget)."""
    n = len(exec_t)
    t_budget = max(min(remain), eta) if n else eta
    if n == 0:
        return [], [], t_budget
    phi = t_budget / (t_budget - t_c) * sum(exec_t)
    cls = []
    for i in range(n):
        if waited is not None and waited[i] > tau:
            cls.append(2)
        else:
            cls.append(1 if remain[i] < gamma * phi else 0)
    starving = [i for i in range(n) if cls[i] == 2]
    urgent = sorted((i for i in range(n) if cls[i] == 1), key=lambda i: -(weight[i] / exec_t[i]))   # stable
    normal = sorted((i for i in range(n) if cls[i] == 0), key=lambda i: remain[i])
    return starving + urgent + normal, cls, t_budget


def estimate_batch(model: Dict[str, float], prefill: Sequence[Tuple[int, int]], decode: Sequence[int]) -> float:
    """Section 4.1, "Batch Latency Estimator": a prefill request costs a_p l_q^2 + b_p l_q l_kv + c_p l_q, a
    decode request a_d l_kv + b_d, and a batch the sum over its requests plus the constant overhead t_c.
    prefill holds (l_q, l_kv) pairs, decode holds l_kv values."""
    total = 0.0
    for l_q, l_kv in prefill:
        total += model["a_p"] * l_q ** 2 + model["b_p"] * l_q * l_kv + model["c_p"] * l_q
    for l_kv in decode:
        total += model["a_d"] * l_kv + model["b_d"]
    return total + model["t_c"]


def resume_cost(model: Dict[str, float], n_tokens: int, chunk_tokens: int, s_blk: int, t_block: float):
    """Cost of bringing an evicted request back, both ways (Section 4.3 "Eviction Policy" spills and restores;
    the ablation arm "Recompute" of the evaluation discards blocks at eviction).  Reload: every block of the
    context is missing, T_trans = b_miss * t_block.  Recompute (no formula is printed; the estimator's own
    prefill model is used): the context is prefilled again in chunks, chunk k being a batch of one prefill
    request with l_q tokens on the k * chunk tokens already rebuilt.  Returns (reload, recompute)."""
    b_miss = -(-n_tokens // s_blk)
    reload_t = b_miss * t_block
    chunk = chunk_tokens if chunk_tokens > 0 else n_tokens
    recompute_t = 0.0
    done = 0
    while done < n_tokens:
        l_q = min(chunk, n_tokens - done)
        recompute_t += estimate_batch(model, [(l_q, done)], [])
        done += l_q
    return reload_t, recompute_t


def copy_condition(l_comp: int, l_comp_max: int, b_miss: int, b_rem: int, s_blk: int, beta: float) -> bool:
    """"Put it Together": all missing blocks are copied if the remaining budget covers them; otherwise partial
    copying is enabled only when l_comp reaches the maximum computable-token limit of the round, or the ratio
    l_comp / ((b_miss - B_rem) * s_blk) exceeds beta (beta > 1); else the request is skipped this round."""
    if b_rem >= b_miss:
        return True
    if l_comp >= l_comp_max:
        return True
    return l_comp / ((b_miss - b_rem) * s_blk) > beta


def _bf16_to_float(b: int) -> float:
    """One bf16 pattern to a Python float via its sign / exponent / mantissa fields."""
    sign = -1.0 if (b >> 15) & 1 else 1.0
    exp = (b >> 7) & 0xFF
    man = b & 0x7F
    if exp == 0:
        return sign * man * 2.0 ** (-126 - 7)
    if exp == 0xFF:
        return sign * math.inf if man == 0 else math.nan
    return sign * (1.0 + man / 128.0) * 2.0 ** (exp - 127)


def brute_force_attn(K, V, table, n_tokens, q_bits, S, G):
    """Loop-by-loop decode attention for one request and one layer.

    K, V: uint16 [num_blocks][S][Hkv][D]; q_bits uint16 [Hq][D].  Returns nested lists o[Hq][D].
    """
    Hq, D = len(q_bits), len(q_bits[0])
    out = []
    for h in range(Hq):
        g = h // G
        logits = []
        for t in range(n_tokens):
            blk, slot = table[t // S], t % S
            acc = 0.0
            for d in range(D):
                acc += _bf16_to_float(int(q_bits[h][d])) * _bf16_to_float(int(K[blk][slot][g][d]))
            logits.append(acc / math.sqrt(D))
        m = max(logits)
        w = [math.exp(x - m) for x in logits]
        z = sum(w)
        row = []
        for d in range(D):
            acc = 0.0
            for t in range(n_tokens):
                blk, slot = table[t // S], t % S
                acc += (w[t] / z) * _bf16_to_float(int(V[blk][slot][g][d]))
            row.append(acc)
        out.append(row)
    return out


def brute_force_image(K, V, table, L, S, Hkv, D):
    """Element-by-element host image of a request: flat list in [L][n_blk][K|V][S][Hkv][D] order."""
    flat = []
    for l in range(L):
        for b in table:
            for pool in (K, V):
                for s in range(S):
                    for h in range(Hkv):
                        for d in range(D):
                            flat.append(int(pool[l][b][s][h][d]))
    return flat
