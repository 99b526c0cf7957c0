"""Eviction policy and the partial-copy admission rule (Section 4.3): hand-worked cases for the checker, and
the library against the checker."""
import numpy as np
import pytest

from oracle import ps_oracle as po
from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import build as ps_build
from paper_2512_12928_b200 import workloads as wl


@pytest.fixture(scope="module", autouse=True)
def built_library():
    ps_build.build()
    return B.load()


def pair(nb=64, S=4):
    sh = wl.KVShape(2, 1, 1, 8, S, nb)
    lib = B.KVSwap(num_layers=2, num_kv_heads=1, num_q_heads=1, head_dim=8, block_size=S, num_gpu_blocks=nb,
                   max_blocks_per_req=nb, host_pool_bytes=1 << 30, flags=B.PS_FLAG_BOOKKEEPING_ONLY)
    return lib, po.PsOracle(2, 1, 1, 8, S, nb)


def test_victims_come_from_the_tail_and_near_starving_requests_are_spared():
    lib, orc = pair()
    tokens = {1: 16, 2: 8, 3: 12, 4: 20, 5: 4}          # blocks: 4, 2, 3, 5, 1
    for x in (lib, orc):
        for r, n in tokens.items():
            assert x.kv_alloc(r, n) == 0
        assert x.swap_out(2) == 0                      # request 2 is not resident: never a victim
    queue = [1, 2, 3, 4, 5, 99]                        # head first; 99 is unknown
    waited = [0.0, 0.0, 50.0, 95.0, 10.0, 0.0]
    # tau = 100, "close" = 80 %: request 4 (waited 95) is spared; from the tail: 5 (1 block), then 3 (3 blocks)
    assert orc.select_victims(queue, waited, 100.0, 0.8, 4) == ([5, 3], 4)
    assert orc.select_victims(queue, waited, 100.0, 0.8, 1) == ([5], 1)
    assert orc.select_victims(queue, waited, 100.0, 0.8, 5) == ([5, 3, 1], 8)
    assert orc.select_victims(queue, waited, 100.0, 0.8, 100) == ([5, 3, 1], 8)     # not enough to free
    assert orc.select_victims(queue, waited, 100.0, 1.0, 4) == ([5, 4], 6)          # 95 < 100: not starving yet
    assert orc.select_victims(queue, waited, 100.0, 0.8, 0) == ([], 0)
    for near, need in [(0.8, 4), (0.8, 1), (0.8, 5), (0.8, 100), (1.0, 4), (0.8, 0), (0.05, 3)]:
        rc, victims, freed = lib.select_victims(queue, waited, 100.0, near, need)
        assert (rc, (victims, freed)) == (B.PS_OK, orc.select_victims(queue, waited, 100.0, near, need))
    assert lib.select_victims(queue, waited, 100.0, 0.0, 1)[0] == B.PS_ERR_INVALID


def test_victim_selection_matches_checker_on_random_queues():
    rng = np.random.default_rng(99)
    lib, orc = pair(nb=512)
    ids = list(range(40))
    for x in (lib, orc):
        for r in ids:
            assert x.kv_alloc(r, int(np.random.default_rng(r).integers(0, 40))) == 0
        for r in ids[::7]:
            assert x.swap_out(r) == 0
    for _ in range(200):
        queue = [int(v) for v in rng.permutation(ids)[: int(rng.integers(1, 40))]]
        if rng.random() < 0.3:
            queue.append(queue[0])                                  # a duplicate entry is taken once
        waited = [float(v) for v in rng.uniform(0, 120, size=len(queue))]
        need = int(rng.integers(0, 80))
        near = float(rng.uniform(0.1, 1.0))
        rc, victims, freed = lib.select_victims(queue, waited, 100.0, near, need)
        assert (rc, (victims, freed)) == (B.PS_OK, orc.select_victims(queue, waited, 100.0, near, need))
        # properties: victims are resident, spared ones stay, and the walk stops as soon as enough is freed
        for v in victims:
            assert orc.reqs[v].state == po.ST_RESIDENT
        if victims and need > 0:
            assert freed - len(orc.reqs[victims[-1]].table) < need


def test_partial_copy_condition_hand_worked():
    # b_miss = 10 blocks of 16 tokens, residual budget 4 blocks: 6 blocks = 96 tokens stay missing
    assert po.copy_condition(l_comp=200, l_comp_max=512, b_miss=10, b_rem=4, s_blk=16, beta=2.0) is True    # 200/96 = 2.08 > 2
    assert po.copy_condition(l_comp=192, l_comp_max=512, b_miss=10, b_rem=4, s_blk=16, beta=2.0) is False   # exactly 2.0
    assert po.copy_condition(l_comp=100, l_comp_max=100, b_miss=10, b_rem=4, s_blk=16, beta=2.0) is True    # reaches the round's limit
    assert po.copy_condition(l_comp=0, l_comp_max=512, b_miss=10, b_rem=10, s_blk=16, beta=2.0) is True     # the budget covers everything
    assert po.copy_condition(l_comp=0, l_comp_max=512, b_miss=10, b_rem=0, s_blk=16, beta=1.5) is False
    rng = np.random.default_rng(5)
    for _ in range(500):
        a = [int(rng.integers(0, 600)), int(rng.integers(0, 600)), int(rng.integers(0, 30)), int(rng.integers(0, 30)),
             int(rng.choice([4, 16, 32]))]
        beta = float(rng.uniform(1.01, 4.0))
        rc, allowed = B.ps_copy_condition(*a, beta)
        assert rc == B.PS_OK and allowed == po.copy_condition(*a, beta)
    assert B.ps_copy_condition(1, 1, 1, 0, 16, 1.0)[0] == B.PS_ERR_INVALID
    assert B.ps_copy_condition(1, 1, 1, 0, 0, 2.0)[0] == B.PS_ERR_INVALID


def test_queue_order_hand_worked_and_against_the_library():
    # five requests; t_c = 10; eta = 50.  min remain = 100 -> t_budget = 100; phi = 100/90 * (20+30+10+40+50) = 166.67
    exec_t = [20.0, 30.0, 10.0, 40.0, 50.0]
    remain = [100.0, 400.0, 150.0, 165.0, 900.0]
    weight = [2.0, 1.0, 2.0, 1.0, 2.0]
    # gamma = 1: urgent = remain < 166.67 -> requests 0, 2, 3; densities 0.1, 0.2, 0.025 -> 2, 0, 3; normal by remain: 1, 4
    assert po.order_queue(exec_t, remain, weight, eta=50.0, gamma=1.0, t_c=10.0) == ([2, 0, 3, 1, 4], [1, 0, 1, 1, 0], 100.0)
    # gamma = 0.5: threshold 83.3 -> nobody urgent: pure deadline order
    assert po.order_queue(exec_t, remain, weight, eta=50.0, gamma=0.5, t_c=10.0)[0] == [0, 2, 3, 1, 4]
    # starvation: request 4 waited longer than tau and goes to the head
    got = po.order_queue(exec_t, remain, weight, eta=50.0, gamma=1.0, t_c=10.0, waited=[0, 0, 0, 0, 999.0], tau=500.0)
    assert got[0] == [4, 2, 0, 3, 1] and got[1][4] == 2
    # eta bounds the budget from below: min remain 100 < eta 200 -> t_budget 200, phi = 200/190 * 150 = 157.9
    got = po.order_queue(exec_t, remain, weight, eta=200.0, gamma=1.0, t_c=10.0)
    assert got[2] == 200.0 and got[1] == [1, 0, 1, 0, 0]
    rng = np.random.default_rng(17)
    for _ in range(300):
        n = int(rng.integers(0, 12))
        e = [float(v) for v in rng.uniform(1, 100, n)]
        r = [float(v) for v in rng.uniform(20, 2000, n)]
        w = [float(v) for v in rng.choice([1.0, 2.0], n)]
        waited = [float(v) for v in rng.uniform(0, 1000, n)] if rng.random() < 0.5 else None
        kw = dict(eta=float(rng.uniform(20, 300)), gamma=float(rng.uniform(0.3, 1.5)), t_c=float(rng.uniform(0, 15)))
        want = po.order_queue(e, r, w, waited=waited, tau=700.0, **kw)
        rc, order, cls, tb = B.ps_order_queue(e, r, w, waited_us=waited, tau=700.0, **kw)
        assert rc == B.PS_OK and (order, cls, tb) == want
    assert B.ps_order_queue([1.0], [5.0], [1.0], eta=1.0, gamma=1.0, t_c=10.0)[0] == B.PS_ERR_INVALID     # t_budget <= t_c


def test_closed_loop_of_scheduler_order_eviction_budget_and_reload():
    """The paper's loop on a small instance: order the queue, evict from its tail when the pool is short,
    readmit from its head, choose the copy budget, step.  Library (bookkeeping context) and checker take the
    same decisions and end with the same tables."""
    rng = np.random.default_rng(23)
    lib, orc = pair(nb=64, S=4)
    ids = list(range(14))
    tokens = {r: int(rng.integers(8, 60)) for r in ids}
    weight = {r: float(rng.choice([1.0, 2.0])) for r in ids}
    deadline = {r: float(rng.uniform(200, 3000)) for r in ids}
    arrived = {r: 0.0 for r in ids}
    now = 0.0
    model = dict(a_d=0.5, b_d=2.0, t_c=5.0, t_block=9.0)
    decoded_total = evicted_total = 0
    for rnd in range(40):
        now += 60.0
        # requests arrive over time and are admitted when blocks are free; otherwise someone is evicted
        queue = [r for r in ids if r in orc.reqs or r <= rnd]
        exec_t = [model["a_d"] * tokens[r] + model["b_d"] for r in queue]
        remain = [deadline[r] - now for r in queue]
        w = [weight[r] for r in queue]
        waited = [now - arrived[r] for r in queue]
        kw = dict(eta=40.0, gamma=0.9, t_c=model["t_c"])
        o_order, o_cls, o_tb = po.order_queue(exec_t, remain, w, waited=waited, tau=1500.0, **kw)
        rc, l_order, l_cls, l_tb = B.ps_order_queue(exec_t, remain, w, waited_us=waited, tau=1500.0, **kw)
        assert rc == B.PS_OK and (l_order, l_cls, l_tb) == (o_order, o_cls, o_tb)
        sorted_q = [queue[i] for i in o_order]
        sorted_waited = [waited[i] for i in o_order]
        for r in sorted_q:                                           # head first: admit or readmit
            need = orc.blocks_for(tokens[r])
            st = orc.reqs[r].state if r in orc.reqs else None
            if st in (po.ST_RESIDENT, po.ST_SWAPPING_IN, po.ST_SWAPPING_OUT):
                continue
            if orc.num_free_blocks() < need:
                want_v = orc.select_victims(sorted_q, sorted_waited, 1500.0, 0.8, need - orc.num_free_blocks())
                rc, victims, freed = lib.select_victims(sorted_q, sorted_waited, 1500.0, 0.8, need - lib.num_free_blocks())
                assert (victims, freed) == want_v
                victims = [v for v in victims if sorted_q.index(v) > sorted_q.index(r)]   # never evict for a later request
                for v in victims:
                    assert lib.swap_out(v) == orc.swap_out(v) == 0
                    evicted_total += 1
                lib.sync(); orc.reap()
            if orc.num_free_blocks() < need:
                continue
            if st is None:
                assert lib.kv_alloc(r, tokens[r]) == orc.kv_alloc(r, tokens[r]) == 0
            else:
                assert lib.swap_in_begin(r) == orc.swap_in_begin(r) == 0
        budget_o = orc.copy_budget(sorted_q, t_budget=o_tb, **model)
        rc, blocks, nbytes, case = lib.copy_budget(sorted_q, t_budget=o_tb, **model)
        assert rc == B.PS_OK and (blocks, case) == budget_o
        rc, mask, st = lib.step(None, None, sorted_q, nbytes)
        plan, omask, _ = orc.step(nbytes, sorted_q)
        assert rc == B.PS_OK and mask == omask
        decoded_total += sum(mask)
        for r in sorted_q:                                           # decode appends a token to whoever ran
            if r in orc.reqs and orc.reqs[r].state == po.ST_RESIDENT:
                tokens[r] += 1
                a, b = lib.kv_alloc(r, tokens[r]), orc.kv_alloc(r, tokens[r])
                assert a == b
                if a != 0:
                    tokens[r] -= 1
        for r in sorted_q:
            if r in orc.reqs:
                assert lib.block_table(r) == orc.block_table(r)
        orc.check_invariants()
    assert decoded_total > 100 and evicted_total > 3
