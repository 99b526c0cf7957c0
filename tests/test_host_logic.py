"""The library's host side on a machine without a GPU: exports, block tables, states, error codes and
copy-budget plans, id for id against the CPU checker (bookkeeping-only contexts move no bytes)."""
import json
import os
import re

import numpy as np
import pytest

from oracle import ps_oracle as po
from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import build as ps_build
from paper_2512_12928_b200 import workloads as wl


@pytest.fixture(scope="session", autouse=True)
def built_library():
    ps_build.build()
    return B.load()


def make_pair(sh: wl.KVShape, free_order, host_pool_bytes=1 << 40, max_blocks=None):
    lib = B.KVSwap(num_layers=sh.num_layers, num_kv_heads=sh.num_kv_heads, num_q_heads=sh.num_q_heads,
                   head_dim=sh.head_dim, block_size=sh.block_size, num_gpu_blocks=sh.num_gpu_blocks,
                   max_blocks_per_req=max_blocks or sh.num_gpu_blocks, host_pool_bytes=host_pool_bytes,
                   initial_free_order=free_order, flags=B.PS_FLAG_BOOKKEEPING_ONLY)
    orc = po.PsOracle(sh.num_layers, sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size,
                      sh.num_gpu_blocks, free_order, host_pool_bytes=None)
    return lib, orc


def same_tables(lib, orc, reqs):
    for r in reqs:
        assert lib.block_table(r) == orc.block_table(r), r
    assert lib.num_free_blocks() == orc.num_free_blocks()


def test_library_exports_every_declared_symbol(repo_root, built_library):
    header = open(os.path.join(repo_root, "include", "ps_kvswap.h")).read()
    declared = set(re.findall(r"^(?:int32_t|const char\*)\s+(ps_[a-z_0-9]+)\s*\(", header, re.M))
    assert declared == set(B.EXPORTS), declared ^ set(B.EXPORTS)
    for name in declared:
        assert hasattr(built_library, name), name


def test_status_codes_match_the_checker():
    assert (B.PS_OK, B.PS_ERR_INVALID, B.PS_ERR_NOMEM, B.PS_ERR_HOST_NOMEM, B.PS_ERR_STATE, B.PS_ERR_BUSY) == \
           (po.OK, po.ERR_INVALID, po.ERR_NOMEM, po.ERR_HOST_NOMEM, po.ERR_STATE, po.ERR_BUSY)
    assert (B.PS_REQ_RESIDENT, B.PS_REQ_SWAPPING_OUT, B.PS_REQ_HOST, B.PS_REQ_SWAPPING_IN) == \
           (po.ST_RESIDENT, po.ST_SWAPPING_OUT, po.ST_HOST, po.ST_SWAPPING_IN)


def test_create_rejects_bad_config():
    with pytest.raises(B.PsError) as e:
        B.KVSwap(num_layers=2, num_kv_heads=2, num_q_heads=4, head_dim=64, block_size=16, num_gpu_blocks=4,
                 max_blocks_per_req=4, initial_free_order=[0, 1, 1, 3], flags=B.PS_FLAG_BOOKKEEPING_ONLY)
    assert e.value.code == B.PS_ERR_INVALID and "permutation" in str(e.value)
    with pytest.raises(B.PsError):
        B.KVSwap(num_layers=2, num_kv_heads=3, num_q_heads=4, head_dim=64, block_size=16, num_gpu_blocks=4,
                 max_blocks_per_req=4, flags=B.PS_FLAG_BOOKKEEPING_ONLY)


def test_tiny_script_tables_match_id_for_id():
    w = wl.tiny()
    lib, orc = make_pair(w.shape, w.free_order)
    for r, n in wl.build_order_round_robin(w):
        assert lib.kv_alloc(r, n) == orc.kv_alloc(r, n) == B.PS_OK
    reqs = list(range(len(w.ctx_lens)))
    same_tables(lib, orc, reqs)
    for r in w.victims:
        assert lib.swap_out(r) == orc.swap_out(r) == B.PS_OK
        assert lib.block_table(r)[1] == B.PS_REQ_SWAPPING_OUT
    assert lib.kv_free(w.victims[0]) == orc.kv_free(w.victims[0]) == B.PS_ERR_BUSY
    assert lib.sync() == B.PS_OK
    orc.reap()
    same_tables(lib, orc, reqs)
    for r in reversed(w.victims):
        assert lib.swap_in_begin(r) == orc.swap_in_begin(r) == B.PS_OK
    same_tables(lib, orc, reqs)
    rc, mask, st = lib.step(None, None, reqs, -1)
    plan, omask, _ = orc.step(-1, reqs)
    assert rc == B.PS_OK and mask == omask == [1] * len(reqs)
    assert st["blocks_copied"] == sum(hi - lo for _, lo, hi in plan)
    assert st["reloads_completed"] == len(w.victims)
    same_tables(lib, orc, reqs)
    orc.check_invariants()


def test_budget_schedule_golden_through_the_library(repo_root):
    g = json.load(open(os.path.join(repo_root, "tests", "golden", "budget_schedule.json")))
    sh = wl.KVShape(**g["shape"])
    for case in g["cases"]:
        lib, _ = make_pair(sh, None)
        for req, n in g["queue_tokens"]:
            assert lib.kv_alloc(req, n) == B.PS_OK
        for req, _ in g["queue_tokens"]:
            assert lib.swap_out(req) == B.PS_OK
        assert lib.sync() == B.PS_OK
        for req, _ in g["queue_tokens"]:
            assert lib.swap_in_begin(req) == B.PS_OK
        ids = [r for r, _ in g["queue_tokens"]]
        for want in case["steps"]:
            before = {r: lib.missing_blocks(r) for r in ids}
            rc, mask, st = lib.step(None, None, ids, case["budget_bytes"])
            assert rc == B.PS_OK
            after = {r: lib.missing_blocks(r) for r in ids}
            got = {r: before[r] - after[r] for r in ids if before[r] != after[r]}
            assert got == {r: hi - lo for r, lo, hi in want}, (case["budget_bytes"], got, want)
            assert st["h2d_bytes"] == sum(hi - lo for _, lo, hi in want) * g["block_bytes"]


def test_ruled_budget_schedule_golden_through_the_library(repo_root):
    """ps_step_ruled: the partial-copy admission test applied while the budget is consumed."""
    g = json.load(open(os.path.join(repo_root, "tests", "golden", "budget_schedule.json")))
    sh = wl.KVShape(**g["shape"])
    for case in g["ruled_cases"]:
        lib, orc = make_pair(sh, None)
        for req, n in g["queue_tokens"]:
            assert lib.kv_alloc(req, n) == orc.kv_alloc(req, n) == B.PS_OK
        for req, _ in g["queue_tokens"]:
            assert lib.swap_out(req) == orc.swap_out(req) == B.PS_OK
        assert lib.sync() == B.PS_OK
        orc.reap()
        for req, _ in g["queue_tokens"]:
            assert lib.swap_in_begin(req) == orc.swap_in_begin(req) == B.PS_OK
        ids = [r for r, _ in g["queue_tokens"]]
        rule = {int(k): tuple(v) for k, v in case["rule"].items()}
        rr = sorted(rule)
        for want in case["steps"]:
            before = {r: lib.missing_blocks(r) for r in ids}
            rc, mask, st = lib.step_ruled(None, None, ids, case["budget_bytes"], case["beta"], rr,
                                          [rule[r][0] for r in rr], [rule[r][1] for r in rr])
            assert rc == B.PS_OK, lib.last_error()
            plan, omask, _ = orc.step(case["budget_bytes"], ids, rule=rule, beta=case["beta"])
            got = {r: before[r] - lib.missing_blocks(r) for r in ids if before[r] != lib.missing_blocks(r)}
            assert got == {r: hi - lo for r, lo, hi in want} == {r: hi - lo for r, lo, hi in plan}
            assert mask == omask
            same_tables(lib, orc, ids)
    lib, _ = make_pair(sh, None)
    assert lib.step_ruled(None, None, [], 0, 1.0, [], [], [])[0] == B.PS_ERR_INVALID      # beta must exceed 1
    assert lib.step_ruled(None, None, [], 0, 2.0, [1], [-1], [0])[0] == B.PS_ERR_INVALID


def test_kernel_status_word_is_reported_with_its_own_code_and_text():
    """What a kernel writes into the status word surfaces from the next poll: a bad block id as
    PS_ERR_BOUNDS, a wait that ran out inside the attention kernel as PS_ERR_TIMEOUT.  The word is written
    by a test hook: no kernel is made to fail."""
    sh = wl.KVShape(2, 2, 4, 64, 16, 8)
    lib, _ = make_pair(sh, None)
    assert lib.poll() == 0
    for value, code, text in ((1, B.PS_ERR_BOUNDS, "copy kernel"), (2, B.PS_ERR_BOUNDS, "attention kernel met"),
                              (3, B.PS_ERR_TIMEOUT, "bounded wait")):
        assert lib.inject_status(value) == B.PS_OK
        with pytest.raises(B.PsError) as e:
            lib.poll()
        assert e.value.code == code and text in str(e.value), str(e.value)
        assert lib.poll() == 0                      # reported once, then clear
    assert lib.inject_status(3) == B.PS_OK
    assert lib.step(None, None, [], 0)[0] == B.PS_ERR_TIMEOUT
    assert lib.sync() == B.PS_OK
    assert lib.inject_status(0) == B.PS_ERR_INVALID and lib.inject_status(4) == B.PS_ERR_INVALID


def test_random_script_against_checker():
    """A long seeded mix of alloc / grow / free / swap-out / reap / swap-in / cancel / budgeted steps."""
    sh = wl.KVShape(3, 2, 4, 64, 8, 96)
    rng = np.random.default_rng(1234)
    order = rng.permutation(sh.num_gpu_blocks)
    lib, orc = make_pair(sh, order, host_pool_bytes=1 << 40, max_blocks=40)
    live = set()
    next_id = 100
    for it in range(3000):
        op = rng.integers(0, 10)
        if op <= 1:
            r, n = next_id, int(rng.integers(0, 200))
            next_id += 1
            a, b = lib.kv_alloc(r, n), orc.kv_alloc(r, n)
            assert a == b, (it, "alloc", a, b)
            if a == B.PS_OK:
                live.add(r)
        elif op == 2 and live:
            r = int(rng.choice(sorted(live)))
            n = lib.n_tokens(r) + int(rng.integers(0, 40))
            assert lib.kv_alloc(r, n) == orc.kv_alloc(r, n), (it, "grow")
        elif op == 3 and live:
            r = int(rng.choice(sorted(live)))
            a, b = lib.kv_free(r), orc.kv_free(r)
            assert a == b, (it, "free", a, b)
            if a == B.PS_OK:
                live.discard(r)
        elif op == 4 and live:
            r = int(rng.choice(sorted(live)))
            assert lib.swap_out(r) == orc.swap_out(r), (it, "out")
        elif op == 5:
            assert lib.sync() == B.PS_OK
            orc.reap()
        elif op == 6 and live:
            r = int(rng.choice(sorted(live)))
            assert lib.swap_in_begin(r) == orc.swap_in_begin(r), (it, "in_begin")
        elif op == 7 and live:
            r = int(rng.choice(sorted(live)))
            assert lib.swap_in_cancel(r) == orc.swap_in_cancel(r), (it, "cancel")
        elif op >= 8:
            budget = int(rng.choice([-1, 0, 1, 3, 7, 20])) * (sh.block_bytes if rng.integers(0, 2) else sh.block_bytes + 17)
            ids = sorted(live)
            # in bookkeeping mode every offload completes at once: the checker reaps before the step too
            orc.reap()
            rc, mask, st = lib.step(None, None, ids, budget)
            plan, omask, _ = orc.step(budget, ids)
            assert rc == B.PS_OK and mask == omask, (it, "step")
            assert st["blocks_copied"] == sum(hi - lo for _, lo, hi in plan)
        if it % 50 == 0:
            lib.sync(); orc.reap()
            same_tables(lib, orc, sorted(live))
            orc.check_invariants()
    lib.sync(); orc.reap()
    same_tables(lib, orc, sorted(live))
    # partition property checked on the library's own answers
    owned = []
    for r in live:
        t, st = lib.block_table(r)
        owned += t
        assert (st == B.PS_REQ_HOST) == (t == []) or lib.n_tokens(r) == 0
    assert len(owned) == len(set(owned)) == sh.num_gpu_blocks - lib.num_free_blocks()


def test_swap_in_layer_prefix_rule_and_states():
    sh = wl.KVShape(2, 2, 4, 64, 4, 16)
    lib, orc = make_pair(sh, None)
    for x in (lib, orc):
        assert x.kv_alloc(0, 16) == B.PS_OK and x.swap_out(0) == B.PS_OK
    lib.sync(); orc.reap()
    for x in (lib, orc):
        assert x.swap_in_layer(0, 0, 0, 1) == B.PS_ERR_STATE
        assert x.swap_in_begin(0) == B.PS_OK
        assert x.swap_in_layer(0, 0, 1, 2) == B.PS_ERR_INVALID
        assert x.swap_in_layer(0, 7, 0, 1) == B.PS_ERR_INVALID
        assert x.swap_in_layer(0, 0, 0, 9) == B.PS_ERR_INVALID
        assert x.swap_in_layer(0, 0, 0, 4) == B.PS_OK
        assert x.block_table(0)[1] == B.PS_REQ_SWAPPING_IN
        assert x.swap_in_cancel(0) == B.PS_ERR_BUSY
        assert x.swap_in_layer(0, 1, 0, 2) == B.PS_OK
        assert x.missing_blocks(0) == 2
        assert x.swap_in_layer(0, 1, 2, 4) == B.PS_OK
        assert x.block_table(0)[1] == B.PS_REQ_RESIDENT


def test_host_pool_exhaustion_and_reuse():
    sh = wl.KVShape(2, 1, 1, 64, 4, 32)
    bb = sh.block_bytes
    lib = B.KVSwap(num_layers=2, num_kv_heads=1, num_q_heads=1, head_dim=64, block_size=4, num_gpu_blocks=32,
                   max_blocks_per_req=32, host_pool_bytes=8 * bb, flags=B.PS_FLAG_BOOKKEEPING_ONLY)
    for r in range(3):
        assert lib.kv_alloc(r, 16) == B.PS_OK           # 4 blocks each
    assert lib.swap_out(0) == B.PS_OK and lib.swap_out(1) == B.PS_OK
    assert lib.swap_out(2) == B.PS_ERR_HOST_NOMEM
    assert lib.block_table(2)[1] == B.PS_REQ_RESIDENT
    lib.sync()
    assert lib.kv_free(0) == B.PS_OK                    # releases its host image
    assert lib.swap_out(2) == B.PS_OK
    assert lib.swap_out(2) == B.PS_ERR_STATE
    assert lib.decode_attn(0, _Fake(), _Fake(), [1]) == B.PS_ERR_INVALID   # no device in this mode


class _Fake:
    def data_ptr(self):
        return 0


def test_churn_script_same_answers_as_the_checker():
    """The seeded churn script (60 steps) gets the same status codes, masks and tables from both sides.

    The script's own capacity clipping is approximate (a budgeted reload can take several steps), so
    some requests are refused; what is pinned is that library and checker refuse the same ones.  The
    host pool is twice the script's figure so that the library's contiguous images never fail on
    fragmentation, which the checker does not model.
    """
    w = wl.churn(num_requests=64, num_gpu_blocks=6144, steps=60)
    sh = w.shape
    host_bytes = 12 * wl.GiB
    init, steps = wl.churn_script(w, host_bytes)
    lib, orc = make_pair(sh, w.free_order, host_pool_bytes=2 * host_bytes, max_blocks=1024)
    orc.host_pool_bytes = 2 * host_bytes
    for r in init["host"]:                       # host-resident requests pass through the device first
        for x in (lib, orc):
            assert x.kv_alloc(r, w.ctx_lens[r]) == B.PS_OK
            assert x.swap_out(r) == B.PS_OK
        lib.sync(); orc.reap()
    for r in init["resident"]:
        for x in (lib, orc):
            assert x.kv_alloc(r, w.ctx_lens[r]) == B.PS_OK
    moved = ok_out = ok_in = 0
    for i, stp in enumerate(steps):
        for r in stp["out"]:
            a, b = lib.swap_out(r), orc.swap_out(r)
            assert a == b, (i, "out", r, a, b)
            ok_out += a == B.PS_OK
        for r in stp["inn"]:
            a, b = lib.swap_in_begin(r), orc.swap_in_begin(r)
            assert a == b, (i, "in", r, a, b)
            ok_in += a == B.PS_OK
        live = sorted(orc.reqs)
        orc.reap()
        rc, mask, st = lib.step(None, None, live, 256 * wl.MiB)
        plan, omask, _ = orc.step(256 * wl.MiB, live)
        assert rc == B.PS_OK and mask == omask
        assert st["blocks_copied"] == sum(hi - lo for _, lo, hi in plan)
        moved += st["blocks_copied"]
    same_tables(lib, orc, sorted(orc.reqs))
    orc.check_invariants()
    assert moved > 0 and ok_out > 10 and ok_in > 10
