"""Pins for the CPU checker's block bookkeeping, swap and copy-budget rule (no GPU)."""
import json
import os

import numpy as np
import pytest

from oracle import ps_oracle as po
from paper_2512_12928_b200 import workloads as wl


def small_oracle(seed=0, L=2, Hkv=2, Hq=4, D=8, S=4, nb=24, with_data=True, host_pool_bytes=None):
    rng = np.random.default_rng(seed)
    order = rng.permutation(nb)
    K = V = None
    if with_data:
        K = rng.integers(0, 65536, size=(L, nb, S, Hkv, D), dtype=np.uint16)
        V = rng.integers(0, 65536, size=(L, nb, S, Hkv, D), dtype=np.uint16)
    return po.PsOracle(L, Hkv, Hq, D, S, nb, order, K, V, host_pool_bytes=host_pool_bytes), order


def logical_kv(o, req):
    t, _ = o.block_table(req)
    return np.stack([o.K[:, b] for b in t], 1).copy(), np.stack([o.V[:, b] for b in t], 1).copy()


def test_alloc_order_is_the_free_order():
    o, order = small_oracle(with_data=False)
    assert o.kv_alloc(7, 9) == po.OK          # ceil(9/4) = 3 blocks
    assert o.block_table(7)[0] == [int(v) for v in order[:3]]
    assert o.kv_alloc(8, 4) == po.OK
    assert o.block_table(8)[0] == [int(order[3])]
    assert o.kv_alloc(7, 13) == po.OK         # grows by one block: next id in order
    assert o.block_table(7)[0] == [int(v) for v in order[:3]] + [int(order[4])]
    o.check_invariants()


def test_free_pushes_in_table_order_lifo():
    o, order = small_oracle(with_data=False)
    o.kv_alloc(1, 12)
    t = o.block_table(1)[0]
    assert o.kv_free(1) == po.OK
    o.kv_alloc(2, 12)
    assert o.block_table(2)[0] == t[::-1]     # last pushed id is handed out first
    o.check_invariants()


def test_alloc_all_or_nothing_and_errors():
    o, _ = small_oracle(with_data=False, nb=4)
    assert o.kv_alloc(1, 8) == po.OK
    before = o.num_free_blocks()
    assert o.kv_alloc(2, 100) == po.ERR_NOMEM
    assert o.num_free_blocks() == before and 2 not in o.reqs
    assert o.kv_alloc(1, 100) == po.ERR_NOMEM and len(o.block_table(1)[0]) == 2
    assert o.kv_alloc(1, 4) == po.ERR_INVALID          # cannot shrink
    assert o.kv_free(99) == po.ERR_INVALID
    assert o.swap_out(99) == po.ERR_INVALID
    assert o.swap_in_begin(1) == po.ERR_STATE
    o.check_invariants()


def test_host_image_matches_element_loops():
    o, _ = small_oracle(seed=3)
    o.kv_alloc(0, 5); o.kv_alloc(1, 11); o.kv_alloc(0, 9)
    table = o.block_table(1)[0]
    want = po.brute_force_image(o.K.tolist(), o.V.tolist(), table, o.L, o.S, o.Hkv, o.D)
    assert o.swap_out(1) == po.OK
    assert o.reqs[1].image.reshape(-1).tolist() == want
    assert o.reqs[1].image.shape == (o.L, len(table), 2, o.S, o.Hkv, o.D)


def test_round_trip_restores_logical_kv_and_touches_nothing_else():
    o, _ = small_oracle(seed=5, nb=40)
    for r, n in [(0, 13), (1, 30), (2, 7), (3, 22)]:
        assert o.kv_alloc(r, n) == po.OK
    before = {r: logical_kv(o, r) for r in range(4)}
    K0, V0 = o.K.copy(), o.V.copy()
    old_tables = {r: o.block_table(r)[0] for r in range(4)}
    assert o.swap_out(1) == po.OK and o.swap_out(3) == po.OK
    assert o.block_table(1)[1] == po.ST_SWAPPING_OUT
    assert o.kv_free(1) == po.ERR_BUSY
    free_before = o.num_free_blocks()
    assert o.reap() == 2
    assert o.num_free_blocks() == free_before + len(old_tables[1]) + len(old_tables[3])
    assert o.block_table(1) == ([], po.ST_HOST)
    o.check_invariants()
    # a new request grabs (and dirties) some of the reclaimed blocks
    assert o.kv_alloc(9, 10) == po.OK
    for b in o.block_table(9)[0]:
        o.K[:, b] = 0xABCD
        o.V[:, b] = 0x1234
    K1, V1 = o.K.copy(), o.V.copy()
    assert o.swap_in_begin(3) == po.OK and o.swap_in_begin(1) == po.OK
    new3 = o.block_table(3)[0]
    assert set(new3).isdisjoint(o.block_table(9)[0])
    plan, _, _ = o.step(-1)
    assert plan == [(3, 0, len(new3)), (1, 0, len(o.block_table(1)[0]))]
    assert o.block_table(1)[1] == po.ST_RESIDENT and o.block_table(3)[1] == po.ST_RESIDENT
    for r in (1, 3):
        k, v = logical_kv(o, r)
        assert np.array_equal(k, before[r][0]) and np.array_equal(v, before[r][1])
    # blocks outside the two reloaded tables are untouched by the reload
    touched = set(o.block_table(1)[0]) | set(o.block_table(3)[0])
    others = [b for b in range(o.num_blocks) if b not in touched]
    assert np.array_equal(o.K[:, others], K1[:, others]) and np.array_equal(o.V[:, others], V1[:, others])
    # swap-out itself wrote nothing to the pools
    untouched_by_9 = [b for b in range(o.num_blocks) if b not in o.block_table(9)[0] and b not in touched]
    assert np.array_equal(o.K[:, untouched_by_9], K0[:, untouched_by_9])
    assert o.host_used == 0
    o.check_invariants()


def test_partial_reload_is_a_growing_prefix():
    o, _ = small_oracle(seed=8, nb=30)
    o.kv_alloc(0, 37)                        # 10 blocks
    k0, v0 = logical_kv(o, 0)
    o.swap_out(0); o.reap()
    o.K[:] = 0; o.V[:] = 0
    o.swap_in_begin(0)
    bb = o.block_bytes
    assert o.step(3 * bb + 5)[0] == [(0, 0, 3)]
    assert o.block_table(0)[1] == po.ST_SWAPPING_IN and o.missing_blocks(0) == 7
    k, v = logical_kv(o, 0)
    assert np.array_equal(k[:, :3], k0[:, :3]) and not k[:, 3:].any()
    assert o.swap_in_cancel(0) == po.ERR_BUSY
    assert o.step(3 * bb)[0] == [(0, 3, 6)]
    assert o.step(100 * bb)[0] == [(0, 6, 10)]
    k, v = logical_kv(o, 0)
    assert np.array_equal(k, k0) and np.array_equal(v, v0)
    assert o.step(100 * bb)[0] == []


def test_swap_in_layer_checks_prefix_order():
    o, _ = small_oracle(seed=2)
    o.kv_alloc(0, 16); o.swap_out(0); o.reap(); o.swap_in_begin(0)
    assert o.swap_in_layer(0, 0, 1, 2) == po.ERR_INVALID    # must start at the layer's progress
    assert o.swap_in_layer(0, 5, 0, 1) == po.ERR_INVALID
    assert o.swap_in_layer(0, 0, 0, 9) == po.ERR_INVALID
    assert o.swap_in_layer(0, 0, 0, 4) == po.OK
    assert o.block_table(0)[1] == po.ST_SWAPPING_IN          # layer 1 still missing
    assert o.swap_in_layer(0, 1, 0, 4) == po.OK
    assert o.block_table(0)[1] == po.ST_RESIDENT


def test_cancel_queued_reload_returns_blocks():
    o, _ = small_oracle(with_data=False)
    o.kv_alloc(0, 16); o.swap_out(0); o.reap()
    free = list(o.free)
    assert o.swap_in_begin(0) == po.OK
    assert o.swap_in_cancel(0) == po.OK
    assert o.block_table(0) == ([], po.ST_HOST)
    assert sorted(o.free) == sorted(free)
    o.check_invariants()


def test_swap_in_nomem_and_host_pool_limit():
    o, _ = small_oracle(with_data=False, nb=8, host_pool_bytes=None)
    o.kv_alloc(0, 24); o.swap_out(0); o.reap()
    o.kv_alloc(1, 20)
    assert o.swap_in_begin(0) == po.ERR_NOMEM
    assert o.block_table(0) == ([], po.ST_HOST)
    o2, _ = small_oracle(with_data=False, nb=8, host_pool_bytes=3 * 2 * 2 * 4 * 2 * 8 * 2)
    o2.kv_alloc(0, 8); o2.kv_alloc(1, 8)
    assert o2.swap_out(0) == po.OK
    assert o2.swap_out(1) == po.ERR_HOST_NOMEM
    assert o2.block_table(1)[1] == po.ST_RESIDENT


def test_budget_schedule_golden(repo_root):
    g = json.load(open(os.path.join(repo_root, "tests", "golden", "budget_schedule.json")))
    for case in g["cases"]:
        o = po.PsOracle(**g["shape"])
        assert o.block_bytes == g["block_bytes"]
        for req, n in g["queue_tokens"]:
            assert o.kv_alloc(req, n) == po.OK
        for req, _ in g["queue_tokens"]:
            assert o.swap_out(req) == po.OK
        o.reap()
        for req, _ in g["queue_tokens"]:
            assert o.swap_in_begin(req) == po.OK
        for want in case["steps"]:
            plan, _, _ = o.step(case["budget_bytes"])
            assert [list(p) for p in plan] == want, (case["budget_bytes"], plan, want)
        o.check_invariants()


def test_swap_in_begin_of_a_request_without_blocks_is_resident_at_once():
    """Section 4.3 "Pipelined Reloading": a readmitted request's KV must be restored before computation can
    proceed; a request with no tokens has nothing to restore, so it is RESIDENT as soon as it is readmitted:
    it never sits in the reload queue (where no budget could ever complete it) and holds no host bytes."""
    o, _ = small_oracle(with_data=True, host_pool_bytes=1 << 20)
    assert o.kv_alloc(0, 0) == po.OK and o.kv_alloc(1, 9) == po.OK
    assert o.swap_out(0) == po.OK and o.swap_out(1) == po.OK
    o.reap()
    assert o.block_table(0) == ([], po.ST_HOST)
    used_by_1 = o.host_used
    assert used_by_1 == 3 * o.block_bytes                 # the empty image of request 0 holds nothing
    free_before = o.num_free_blocks()
    assert o.swap_in_begin(1) == po.OK and o.swap_in_begin(0) == po.OK
    assert o.block_table(0) == ([], po.ST_RESIDENT)
    assert list(o.in_fifo) == [1]                          # FIFO unchanged by the empty request
    assert o.host_used == used_by_1 and o.num_free_blocks() == free_before - 3
    assert o.missing_blocks(0) == 0
    assert o.step_plan(-1) == [(1, 0, 3)]
    assert o.swap_in_begin(0) == po.ERR_STATE              # already resident
    assert o.kv_alloc(0, 5) == po.OK                       # and it can grow like any resident request
    o.step(-1)
    assert o.host_used == 0
    o.check_invariants()


def test_ruled_budget_schedule_golden(repo_root):
    """The partial-copy admission test while the budget is consumed: hand-worked schedules."""
    g = json.load(open(os.path.join(repo_root, "tests", "golden", "budget_schedule.json")))
    for case in g["ruled_cases"]:
        o = po.PsOracle(**g["shape"])
        for req, n in g["queue_tokens"]:
            assert o.kv_alloc(req, n) == po.OK
        for req, _ in g["queue_tokens"]:
            assert o.swap_out(req) == po.OK
        o.reap()
        for req, _ in g["queue_tokens"]:
            assert o.swap_in_begin(req) == po.OK
        rule = {int(k): tuple(v) for k, v in case["rule"].items()}
        for want in case["steps"]:
            plan, _, _ = o.step(case["budget_bytes"], rule=rule, beta=case["beta"])
            assert [list(p) for p in plan] == want, (case["_derivation"], plan, want)
        o.check_invariants()


def test_ruled_plan_equals_plain_plan_when_every_partial_copy_is_allowed():
    """With l_comp at the round's limit for every request the rule never bites: same plans as without it."""
    rng = np.random.default_rng(5)
    for trial in range(20):
        a, _ = small_oracle(with_data=False, nb=64)
        b, _ = small_oracle(with_data=False, nb=64)
        ids = list(range(5))
        for r in ids:
            n = int(rng.integers(1, 40))
            for o in (a, b):
                assert o.kv_alloc(r, n) == po.OK
        for o in (a, b):
            for r in ids:
                assert o.swap_out(r) == po.OK
            o.reap()
            for r in ids:
                assert o.swap_in_begin(r) == po.OK
        budget = int(rng.integers(1, 6)) * a.block_bytes
        rule = {r: (7, 7) for r in ids}
        for _ in range(12):
            assert a.step(budget)[0] == b.step(budget, rule=rule, beta=2.0)[0]


def test_tiny_workload_script_round_trip():
    w = wl.tiny()
    K, V = wl.make_pools_numpy(w)
    sh = w.shape
    o = po.PsOracle(sh.num_layers, sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size,
                    sh.num_gpu_blocks, w.free_order, K, V)
    for r, n in wl.build_order_round_robin(w):
        assert o.kv_alloc(r, n) == po.OK
    # round-robin growth interleaves the requests' blocks
    t0 = o.block_table(0)[0]
    assert len(t0) == sh.blocks_for(w.ctx_lens[0])
    before = {r: logical_kv(o, r) for r in w.victims}
    for r in w.victims:
        assert o.swap_out(r) == po.OK
    o.reap()
    for r in w.victims:
        assert o.swap_in_begin(r) == po.OK
    o.step(-1)
    for r in w.victims:
        k, v = logical_kv(o, r)
        assert np.array_equal(k, before[r][0]) and np.array_equal(v, before[r][1])
    o.check_invariants()


def test_invariant_checker_catches_a_double_owner():
    o, _ = small_oracle(with_data=False)
    o.kv_alloc(0, 8); o.kv_alloc(1, 8)
    o.reqs[1].table[0] = o.reqs[0].table[0]
    with pytest.raises(AssertionError):
        o.check_invariants()


def test_workload_generators_are_seeded_and_sized():
    a, b = wl.llama8b_swap(), wl.llama8b_swap()
    assert a.ctx_lens == b.ctx_lens and a.victims == b.victims and np.array_equal(a.free_order, b.free_order)
    assert len(a.ctx_lens) == 64 and len(a.victims) == 16 and min(a.ctx_lens) >= 1024 and max(a.ctx_lens) <= 4096
    assert a.shape.block_bytes == 2 * wl.MiB and a.shape.slab_bytes == 32 * 1024
    assert a.total_blocks_needed <= a.shape.num_gpu_blocks
    o = wl.overlap()
    assert len(o.ctx_lens) == 136 and max(o.ctx_lens) <= 8192 and 1200 < np.mean(o.ctx_lens) < 3000
    assert o.total_blocks_needed <= o.shape.num_gpu_blocks
    lc = wl.long_context()
    assert lc.shape.block_bytes == 10 * wl.MiB and lc.total_blocks_needed == 64 * 128 + 1024
    c = wl.churn()
    init, steps = wl.churn_script(c, 48 * wl.GiB)
    assert len(steps) == 200 and len(init["resident"]) + len(init["host"]) + len(init["waiting"]) == 256
    assert wl.tiny().shape.block_bytes == 32 * 1024
