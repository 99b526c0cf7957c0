"""A scheduler stub that drives the library in the paper's closed loop.

Section 4.3 "Put it Together": every round the local scheduler exports the ordered queue and the latency
budget, block management answers with the host-to-device copy budget, and the budget is consumed in queue
order under the partial-copy test.  Under memory pressure requests near the tail of the ordered queue are
evicted (their KV spilled to host memory), and a request that comes back to the head is readmitted and
reloaded layer by layer under the running decode steps.

This module is the *driver* of that loop, not the method: every decision is one call into the library
(`ps_order_queue`, `ps_select_victims`, `ps_copy_budget`, `ps_step_ruled` with its partial-copy rule) through a
small backend interface, so that a test can put a backend in its place that makes every call twice, on the
library and on a checker, and compares.  What the stub adds is the synthetic traffic around the calls: seeded
arrivals with two priority classes, per-token deadlines, requests that finish after a number of generated
tokens.  The model forward is not run: a "step" is the KV-consuming part (attention of every layer over the
paged cache), and simulated time advances by the decode latency model of Section 4.1.

Requests are of two kinds.  A *decoding* request can compute nothing before its whole KV is back, so the
partial-copy test sees l_comp = 0 of a limit of 1 token for it and it is reloaded only in a round whose
residual budget covers it whole -- until it has missed its deadline: from then on the stub reports its one
token as reachable (l_comp = l_comp_max = 1), i.e. it takes whatever residual there is, round after round,
rather than starve behind requests that fit.  A *prefilling* request was evicted in the middle of a chunked
prefill and still has prompt tokens to process: its l_comp is what is left of the prompt, capped by the chunk
limit of a round, which is also its l_comp_max.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

from . import binding as B


@dataclass
class LoopParams:
    """Knobs of the stub (the paper's symbols where it has one)."""
    eta_us: float = 20000.0          # lower bound of the latency budget (eta)
    gamma: float = 0.9               # aggressiveness coefficient (gamma)
    tau_us: float = 2.0e6            # starvation threshold (tau)
    near_frac: float = 0.8           # "close to" the threshold for the eviction policy
    beta: float = 1.5                # partial-copy threshold (beta > 1)
    chunk_tokens: int = 512          # a round's computable-token limit for a prefilling request
    a_d_us: float = 0.034            # decode latency model of Section 4.1: a_d * l_kv + b_d per request,
    b_d_us: float = 2.0              # t_c per batch
    t_c_us: float = 300.0
    t_block_us: float = 80.0         # profiled copy time of one block (all layers)
    tpot_us: Tuple[float, float] = (50000.0, 200000.0)     # per-token deadline of the two classes (high, low)
    ttft_us: Tuple[float, float] = (500000.0, 5.0e6)       # first-token deadline of a request without KV
    weight: Tuple[float, float] = (2.0, 1.0)               # token-level gain of the two classes
    gen_tokens: Tuple[int, int] = (30, 120)                # tokens a request generates before it finishes
    prefilling_frac: float = 0.3     # share of arrivals that still have prompt chunks to process
    max_admit: int = 1               # admissions (arrival or readmission) per round
    fill_frac: float = 0.9           # device pool share filled before the first round
    host_budget_bytes: int = 12 << 30   # host images the stub plans with
    max_batch: int = 256
    subtract_backlog: bool = True    # take reload copies still in flight off the next step's budget


def config4_params(**over) -> LoopParams:
    """Knobs for the priority-churn workload at its full shape (64 layers, 4 MiB blocks, steps of about 13 ms):
    a starvation threshold and lifetimes short enough that evicted requests come back within tens of rounds,
    which offers the host link a sustained load of about half its rate in each direction."""
    kw = dict(tau_us=150e3, max_admit=2, gen_tokens=(20, 60), host_budget_bytes=12 << 30)
    kw.update(over)
    return LoopParams(**kw)


@dataclass
class StubRequest:
    rid: int
    tokens: int
    cls: int                # 0 = high priority, 1 = low
    arrived_us: float
    last_run_us: Optional[float] = None
    todo: int = 0           # tokens still to generate
    prefill_left: int = 0   # prompt tokens still to process (0 = decoding)


class LibBackend:
    """The library behind the stub's interface (argument marshalling only)."""

    def __init__(self, lib: B.KVSwap):
        self.lib = lib

    def order_queue(self, exec_us, remain_us, weight, waited_us, p: LoopParams):
        rc, order, cls, t_budget = B.ps_order_queue(exec_us, remain_us, weight, eta=p.eta_us, gamma=p.gamma,
                                                     t_c=p.t_c_us, waited_us=waited_us, tau=p.tau_us)
        if rc != B.PS_OK:
            raise B.PsError(rc, "ps_order_queue")
        return order, cls, t_budget

    def select_victims(self, queue, waited_us, p: LoopParams, blocks_needed: int):
        rc, victims, freed = self.lib.select_victims(queue, waited_us, p.tau_us, p.near_frac, blocks_needed)
        if rc != B.PS_OK:
            raise B.PsError(rc, "ps_select_victims", self.lib.last_error())
        return victims, freed

    def copy_budget(self, reqs, p: LoopParams, t_budget_us: float):
        rc, blocks, nbytes, case = self.lib.copy_budget(reqs, a_d=p.a_d_us, b_d=p.b_d_us, t_c=p.t_c_us,
                                                        t_block=p.t_block_us, t_budget=t_budget_us)
        if rc != B.PS_OK:
            raise B.PsError(rc, "ps_copy_budget", self.lib.last_error())
        return blocks, nbytes, case

    def kv_alloc(self, rid, n_tokens):
        return self.lib.kv_alloc(rid, n_tokens)

    def kv_free(self, rid):
        return self.lib.kv_free(rid)

    def swap_out(self, rid):
        return self.lib.swap_out(rid)

    def swap_in_begin(self, rid):
        return self.lib.swap_in_begin(rid)

    def poll(self) -> int:
        return self.lib.poll()

    def step(self, q, out, reqs, budget_bytes, beta, rule: Dict[int, Tuple[int, int]]):
        rr = sorted(rule)
        rc, mask, st = self.lib.step_ruled(q, out, reqs, budget_bytes, beta, rr, [rule[r][0] for r in rr],
                                           [rule[r][1] for r in rr])
        if rc != B.PS_OK:
            raise B.PsError(rc, "ps_step_ruled", self.lib.last_error())
        return mask, st

    def state(self, rid) -> int:
        """ps_req_state of the request; PS_REQ_NONE for one the library does not know."""
        return self.lib.req_state(rid)

    def missing(self, rid) -> int:
        return self.lib.missing_blocks(rid)

    def free_blocks(self) -> int:
        return self.lib.num_free_blocks()

    def reload_backlog(self) -> int:
        return self.lib.reload_backlog()


@dataclass
class RoundReport:
    now_us: float
    t_budget_us: float
    budget_blocks: int
    budget_case: int
    batch: List[int]
    mask: List[int]
    stats: dict
    evicted: List[int] = field(default_factory=list)
    admitted: List[int] = field(default_factory=list)
    readmitted: List[int] = field(default_factory=list)
    finished: List[int] = field(default_factory=list)
    skipped_by_rule: int = 0
    decode_tokens: int = 0
    model_step_us: float = 0.0


class SchedulerStub:
    """Seeded traffic + the closed loop of Section 4.3 over a backend (the library, or library and checker)."""

    def __init__(self, backend, ctx_lens: Sequence[int], priority: Sequence[int], block_size: int, block_bytes: int,
                 num_gpu_blocks: int, params: LoopParams, seed: int):
        self.be = backend
        self.p = params
        self.S = block_size
        self.block_bytes = block_bytes
        self.num_gpu_blocks = num_gpu_blocks
        self.rng = np.random.default_rng(seed)
        self.ctx_pool = [int(c) for c in ctx_lens]            # contexts of later arrivals are drawn from these
        self.now = 0.0
        self.next_id = 0
        self.live: Dict[int, StubRequest] = {}
        for c, pr in zip(ctx_lens, priority):
            self._arrive(int(c), int(pr), spread=True)
        self.rounds = 0

    # ---- traffic
    def _arrive(self, ctx: int, cls: int, spread: bool = False) -> StubRequest:
        p = self.p
        r = StubRequest(self.next_id, ctx, cls, self.now)
        if spread:                      # the first population did not arrive all at once
            r.arrived_us = self.now - float(self.rng.uniform(0.0, p.ttft_us[cls]))
        r.todo = int(self.rng.integers(p.gen_tokens[0], p.gen_tokens[1] + 1))
        if self.rng.random() < p.prefilling_frac:
            r.prefill_left = int(self.rng.integers(1, 5)) * p.chunk_tokens // 2
        self.live[r.rid] = r
        self.next_id += 1
        return r

    def blocks_for(self, tokens: int) -> int:
        return (tokens + self.S - 1) // self.S

    def _deadline(self, r: StubRequest) -> float:
        p = self.p
        if r.last_run_us is None:
            return r.arrived_us + p.ttft_us[r.cls]
        return r.last_run_us + p.tpot_us[r.cls]

    # ---- set-up: the device pool is filled in queue order before the first round (no transfer involved)
    def fill(self) -> List[int]:
        order, _, _ = self._ordered()
        used = 0
        placed = []
        for rid in order:
            need = self.blocks_for(self.live[rid].tokens)
            if used + need > self.p.fill_frac * self.num_gpu_blocks:
                continue
            if len(placed) >= self.p.max_batch - 8:
                break
            rc = self.be.kv_alloc(rid, self.live[rid].tokens)
            if rc != B.PS_OK:
                raise B.PsError(rc, "ps_kv_alloc")
            used += need
            placed.append(rid)
        return placed

    def _ordered(self):
        p = self.p
        ids = sorted(self.live)
        exec_us = [p.a_d_us * self.live[r].tokens + p.b_d_us for r in ids]
        remain = [self._deadline(self.live[r]) - self.now for r in ids]
        weight = [p.weight[self.live[r].cls] for r in ids]
        waited = [self.now - (self.live[r].last_run_us if self.live[r].last_run_us is not None
                              else self.live[r].arrived_us) for r in ids]
        order, cls, t_budget = self.be.order_queue(exec_us, remain, weight, waited, p)
        return [ids[i] for i in order], [waited[i] for i in order], t_budget

    # ---- one round of the closed loop
    def round(self, q_all, out_all, on_step=None) -> RoundReport:
        """One round.  q_all / out_all: device bf16 [L][max_batch][Hq][D] (their first len(batch) rows are used) or
        None on a context without a device.  on_step(batch, mask, q, out), if given, is called right after the
        step, before the decoded requests grow by their new token."""
        p, be = self.p, self.be
        be.poll()                                             # finished offloads give their blocks back
        queue, waited, t_budget = self._ordered()
        pos = {r: i for i, r in enumerate(queue)}
        states = {r: be.state(r) for r in queue}
        nblk = {r: self.blocks_for(self.live[r].tokens) for r in queue}
        host_used = sum(nblk[r] for r, st in states.items()
                        if st in (B.PS_REQ_SWAPPING_OUT, B.PS_REQ_HOST, B.PS_REQ_SWAPPING_IN)) * self.block_bytes
        # blocks on their way back to the pool (offloads in flight) are counted as coming
        pending_out = sum(nblk[r] for r, st in states.items() if st == B.PS_REQ_SWAPPING_OUT)
        evicted, admitted, readmitted = [], [], []
        holders = sum(1 for st in states.values() if st in (B.PS_REQ_RESIDENT, B.PS_REQ_SWAPPING_IN))

        def evict_from_tail(short: int, ahead_of: int):
            """Memory is saturated: requests near the tail give up their blocks (never one ahead of `ahead_of`)."""
            nonlocal host_used, pending_out, holders
            victims, _ = be.select_victims(queue, waited, p, short)
            for v in victims:
                if pos[v] <= ahead_of:
                    continue
                vb = nblk[v]
                if host_used + vb * self.block_bytes > p.host_budget_bytes:
                    continue
                rc = be.swap_out(v)
                if rc != B.PS_OK:
                    raise B.PsError(rc, "ps_swap_out")
                states[v] = B.PS_REQ_SWAPPING_OUT
                host_used += vb * self.block_bytes
                pending_out += vb
                holders -= 1
                evicted.append(v)

        # residents whose next token opens a new block must find one: they come before any admission
        grow_need = sum(1 for r, st in states.items()
                        if st == B.PS_REQ_RESIDENT and self.live[r].prefill_left == 0 and self.live[r].tokens % self.S == 0)
        if be.free_blocks() + pending_out < grow_need:
            evict_from_tail(grow_need - be.free_blocks() - pending_out, -1)
        for rid in queue:                                     # head first: admit or readmit
            st = states[rid]
            if st in (B.PS_REQ_RESIDENT, B.PS_REQ_SWAPPING_IN, B.PS_REQ_SWAPPING_OUT):
                continue
            if len(admitted) + len(readmitted) >= p.max_admit or holders >= p.max_batch:
                break
            r = self.live[rid]
            need = self.blocks_for(r.tokens)
            free = be.free_blocks() - grow_need            # blocks the residents' growth will take are not counted
            if free < need:
                short = need - free - pending_out
                if short > 0:
                    evict_from_tail(short, pos[rid])
                break                                         # the head waits for its blocks; nobody overtakes it
            if st == B.PS_REQ_HOST:
                rc = be.swap_in_begin(rid)
                readmitted.append(rid)
            else:
                rc = be.kv_alloc(rid, r.tokens)               # an arrival: its prompt's KV (the prefill is not run)
                admitted.append(rid)
            if rc != B.PS_OK:
                raise B.PsError(rc, "admission")
            states[rid] = B.PS_REQ_SWAPPING_IN if st == B.PS_REQ_HOST else B.PS_REQ_RESIDENT
            holders += 1
        # GetCopyBudget, then the step: ConsumeCopyBudget under SatisfyCopyCondition, reload, attention
        blocks, nbytes, case = be.copy_budget(queue, p, t_budget)
        if p.subtract_backlog:
            # GetCopyBudget assumes the previous steps' transfers have ended; what is still in flight (the link ran
            # below the profiled t_block) comes off this step's budget, so the copy queue cannot grow without bound
            backlog_blocks = -(-be.reload_backlog() // self.block_bytes)
            blocks = max(0, blocks - backlog_blocks)
            nbytes = blocks * self.block_bytes
        batch = [r for r in queue if states[r] in (B.PS_REQ_RESIDENT, B.PS_REQ_SWAPPING_IN)][: p.max_batch]
        rule = {}
        for rid in batch:
            if states[rid] == B.PS_REQ_SWAPPING_IN:
                r = self.live[rid]
                if r.prefill_left > 0:
                    rule[rid] = (min(r.prefill_left, p.chunk_tokens), p.chunk_tokens)
                else:
                    rule[rid] = (1, 1) if self._deadline(r) < self.now else (0, 1)
        n = len(batch)
        before = {rid: be.missing(rid) for rid in rule}
        mask, stats = be.step(_front(q_all, n), _front(out_all, n), batch, nbytes, p.beta, rule)
        rep = RoundReport(self.now, t_budget, blocks, case, batch, mask, stats, evicted, admitted, readmitted)
        if on_step is not None:
            on_step(batch, mask, _front(q_all, n), _front(out_all, n))
        if stats["blocks_copied"] < blocks:                   # budget left over: who was passed over by the rule?
            rep.skipped_by_rule = sum(1 for rid, m in before.items() if m > 0 and be.missing(rid) == m)
        # what the step did to the traffic
        step_us = p.t_c_us
        for rid, m in zip(batch, mask):
            if not m:
                continue
            r = self.live[rid]
            step_us += p.a_d_us * r.tokens + p.b_d_us
            rep.decode_tokens += r.tokens
            r.last_run_us = self.now
            if r.prefill_left > 0:
                r.prefill_left = max(0, r.prefill_left - p.chunk_tokens)
                continue
            if be.kv_alloc(rid, r.tokens + 1) == B.PS_OK:     # the new token's slot (a new block every s_blk tokens)
                r.tokens += 1
                r.todo -= 1
            if r.todo <= 0:
                rc = be.kv_free(rid)
                if rc != B.PS_OK:
                    raise B.PsError(rc, "ps_kv_free")
                cls = r.cls
                del self.live[rid]
                rep.finished.append(rid)
                self._arrive(self.ctx_pool[int(self.rng.integers(0, len(self.ctx_pool)))], cls)
        rep.model_step_us = step_us
        self.now += step_us
        self.rounds += 1
        return rep


def _front(t, n):
    """A contiguous [L][n][Hq][D] view over the front of t's storage, or None (bookkeeping runs pass None)."""
    if t is None:
        return None
    L, _, Hq, D = t.shape
    return t.flatten()[: L * n * Hq * D].view(L, n, Hq, D)
