"""A backend for the scheduler stub that makes every call on the library and on the CPU checker(s) and
compares: decisions (queue order, victims, copy budget, plans under the partial-copy rule), status codes,
states, free-block counts.  `book` is a checker without pool bytes over all layers; `data` (optional) holds
the bytes of some layers over the full block-id space and replays the same block movements."""
from oracle import ps_oracle as po
from paper_2512_12928_b200 import binding as B


class PairedBackend:
    def __init__(self, lib, book, data=None, n_layers=None):
        self.lib, self.book, self.data = lib, book, data
        self.L = n_layers if n_layers is not None else book.L
        self.plans = []                      # the last step's plan (for the test's own checks)
        self.counts = dict(order=0, victims=0, budget=0, steps=0, cases=set(), rule_skips=0, partial=0)

    def _all(self, name, *args):
        a = getattr(self.lib, name)(*args)
        b = getattr(self.book, name)(*args)
        assert a == b, (name, args, a, b, self.lib.last_error())
        if self.data is not None and a == B.PS_OK:
            c = getattr(self.data, name)(*args)
            assert c == a, (name, args, a, c)
        return a

    def order_queue(self, exec_us, remain_us, weight, waited_us, p):
        rc, order, cls, t_budget = B.ps_order_queue(exec_us, remain_us, weight, eta=p.eta_us, gamma=p.gamma,
                                                     t_c=p.t_c_us, waited_us=waited_us, tau=p.tau_us)
        want = po.order_queue(exec_us, remain_us, weight, p.eta_us, p.gamma, p.t_c_us, waited=waited_us, tau=p.tau_us)
        assert rc == B.PS_OK and (order, cls, t_budget) == want
        self.counts["order"] += 1
        return order, cls, t_budget

    def select_victims(self, queue, waited_us, p, blocks_needed):
        rc, victims, freed = self.lib.select_victims(queue, waited_us, p.tau_us, p.near_frac, blocks_needed)
        want = self.book.select_victims(queue, waited_us, p.tau_us, p.near_frac, blocks_needed)
        assert rc == B.PS_OK and (victims, freed) == want, (victims, freed, want)
        self.counts["victims"] += 1
        return victims, freed

    def copy_budget(self, reqs, p, t_budget_us):
        rc, blocks, nbytes, case = self.lib.copy_budget(reqs, a_d=p.a_d_us, b_d=p.b_d_us, t_c=p.t_c_us,
                                                        t_block=p.t_block_us, t_budget=t_budget_us)
        want = self.book.copy_budget(reqs, p.a_d_us, p.b_d_us, p.t_c_us, p.t_block_us, t_budget_us)
        assert rc == B.PS_OK and (blocks, case) == want, (blocks, case, want)
        assert nbytes == blocks * self.book.block_bytes
        self.counts["budget"] += 1
        self.counts["cases"].add(case)
        return blocks, nbytes, case

    def kv_alloc(self, rid, n_tokens):
        return self._all("kv_alloc", rid, n_tokens)

    def kv_free(self, rid):
        return self._all("kv_free", rid)

    def swap_out(self, rid):
        return self._all("swap_out", rid)

    def swap_in_begin(self, rid):
        return self._all("swap_in_begin", rid)

    def _reap(self, n):
        if n:
            self.book.reap(n)
            if self.data is not None:
                self.data.reap(n)

    def poll(self):
        n = self.lib.poll()
        self._reap(n)
        return n

    def step(self, q, out, reqs, budget_bytes, beta, rule):
        rr = sorted(rule)
        rc, mask, st = self.lib.step_ruled(q, out, reqs, budget_bytes, beta, rr, [rule[r][0] for r in rr],
                                           [rule[r][1] for r in rr])
        assert rc == B.PS_OK, self.lib.last_error()
        self._reap(st["swapouts_reaped"])
        plan = self.book.step_plan(budget_bytes, rule, beta)
        plain = self.book.step_plan(budget_bytes)
        self.counts["rule_skips"] += plan != plain
        for req, lo, hi in plan:
            self.counts["partial"] += hi < len(self.book.reqs[req].table)
            for l in range(self.book.L):
                assert self.book.swap_in_layer(req, l, lo, hi) == po.OK
            if self.data is not None:
                for l in range(self.data.L):
                    assert self.data.swap_in_layer(req, l, lo, hi) == po.OK
        omask = [1 if (r in self.book.reqs and self.book.reqs[r].state == po.ST_RESIDENT) else 0 for r in reqs]
        assert mask == omask, (mask, omask)
        assert st["blocks_copied"] == sum(hi - lo for _, lo, hi in plan)
        self.plans = plan
        self.counts["steps"] += 1
        return mask, st

    def state(self, rid):
        a = self.lib.req_state(rid)
        b = self.book.reqs[rid].state if rid in self.book.reqs else 0
        assert a == b, (rid, a, b)
        return a

    def missing(self, rid):
        a = self.lib.missing_blocks(rid)
        assert a == self.book.missing_blocks(rid)
        return a

    def reload_backlog(self):
        return self.lib.reload_backlog()                  # timing information: an input to both sides, not compared

    def free_blocks(self):
        a = self.lib.num_free_blocks()
        assert a == self.book.num_free_blocks()
        return a
