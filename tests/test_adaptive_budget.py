"""Adaptive copy-budget control (Section 4.3): the checker against hand-worked cases, brute force and
properties, and the library (bookkeeping contexts, no GPU) against the checker, decision for decision."""
import json
import math
import os

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


def make_pair(sh, host_pool_bytes=1 << 40):
    lib = B.KVSwap(num_layers=sh.num_layers, num_kv_heads=sh.num_kv_heads, num_q_heads=sh.num_q_heads,
                   head_dim=sh.head_dim, block_size=sh.block_size, num_gpu_blocks=sh.num_gpu_blocks,
                   max_blocks_per_req=sh.num_gpu_blocks, host_pool_bytes=host_pool_bytes,
                   flags=B.PS_FLAG_BOOKKEEPING_ONLY)
    orc = po.PsOracle(sh.num_layers, sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size, sh.num_gpu_blocks)
    return lib, orc


def golden_setup(g):
    sh = wl.KVShape(**g["shape"])
    lib, orc = make_pair(sh)
    for x in (lib, orc):
        for r, n in g["resident_tokens"] + g["queued_tokens"]:
            assert x.kv_alloc(r, n) == 0
        for r, _ in g["queued_tokens"]:
            assert x.swap_out(r) == 0
    lib.sync(); orc.reap()
    for x in (lib, orc):
        for r, _ in g["queued_tokens"]:
            assert x.swap_in_begin(r) == 0
    reqs = [r for r, _ in g["resident_tokens"] + g["queued_tokens"]]
    return sh, lib, orc, reqs


def test_hand_worked_cases_checker_and_library(repo_root):
    g = json.load(open(os.path.join(repo_root, "tests", "golden", "adaptive_budget.json")))
    sh, lib, orc, reqs = golden_setup(g)
    for c in g["cases"]:
        kw = dict(a_d=c["a_d"], b_d=c["b_d"], t_c=c["t_c"], t_block=c["t_block"], t_budget=c["t_budget"])
        assert orc.copy_budget(reqs, **kw) == (c["blocks"], c["case"]), c
        rc, blocks, nbytes, case = lib.copy_budget(reqs, **kw)
        assert (rc, blocks, case) == (B.PS_OK, c["blocks"], c["case"]), c
        assert nbytes == blocks * sh.block_bytes


def brute_largest_feasible(orc, reqs, b_missing, a_d, b_d, t_c, t_block):
    best = 0
    for b in range(b_missing + 1):
        if b * t_block <= orc.step_latency_after(reqs, b, a_d, b_d, t_c):
            best = b
    return best


def test_search_equals_exhaustive_scan_and_library_matches_on_random_queues():
    rng = np.random.default_rng(4321)
    sh = wl.KVShape(2, 2, 4, 64, 8, 4096)
    for trial in range(40):
        lib, orc = make_pair(sh)
        n_res, n_q = int(rng.integers(0, 6)), int(rng.integers(1, 7))
        ids = list(range(n_res + n_q))
        for x in (lib, orc):
            for r in ids:
                assert x.kv_alloc(r, int(np.random.default_rng([trial, r]).integers(1, 900))) == 0
            for r in ids[n_res:]:
                assert x.swap_out(r) == 0
        lib.sync(); orc.reap()
        for x in (lib, orc):
            for r in ids[n_res:]:
                assert x.swap_in_begin(r) == 0
        # a partial step so that the head of the queue has some blocks already
        part = int(rng.integers(0, 20)) * sh.block_bytes
        lib.step(None, None, ids, part); orc.step(part, ids)
        batch = [r for r in ids if rng.random() < 0.8] + [999]           # an unknown id is ignored
        a_d = float(rng.uniform(0.001, 0.05)); b_d = float(rng.uniform(0, 3)); t_c = float(rng.uniform(0, 50))
        if trial % 2:                                    # large per-request constants: the test is far from monotone
            b_d = float(rng.uniform(20, 200))
        t_block = float(rng.uniform(0.05, 5.0))
        b_missing = sum(orc.missing_blocks(r) for r in ids)
        for t_budget in (0.0, float(rng.uniform(0, 200)), 1e9):
            want = orc.copy_budget(batch, a_d, b_d, t_c, t_block, t_budget)
            rc, blocks, nbytes, case = lib.copy_budget(batch, a_d=a_d, b_d=b_d, t_c=t_c, t_block=t_block, t_budget=t_budget)
            assert (rc, blocks, case) == (B.PS_OK,) + want, (trial, t_budget)
            if want[1] == 22:
                assert want[0] == brute_largest_feasible(orc, batch, b_missing, a_d, b_d, t_c, t_block)
            if want[1] == 21:
                assert want[0] == b_missing
            if want[1] == 1:
                assert want[0] == math.floor(t_budget / t_block)
        # the chosen budget, fed to the step, copies no more than B_copy blocks
        want = orc.copy_budget(batch, a_d, b_d, t_c, t_block, 1e9)
        rc, mask, st = lib.step(None, None, ids, want[0] * sh.block_bytes)
        assert st["blocks_copied"] == min(want[0], b_missing)


def test_transfer_of_the_chosen_budget_is_hidden_under_the_estimated_step():
    """Property of case 2: B_copy * t_block <= estimated step time after the copy (the reason for the rule)."""
    g_sh = wl.KVShape(2, 1, 1, 8, 4, 256)
    lib, orc = make_pair(g_sh)
    for r, n in [(0, 100), (1, 60), (2, 333), (3, 47)]:
        assert orc.kv_alloc(r, n) == 0
    for r in (2, 3):
        assert orc.swap_out(r) == 0
    orc.reap()
    for r in (2, 3):
        assert orc.swap_in_begin(r) == 0
    reqs = [0, 1, 2, 3]
    for t_block in (0.5, 1.0, 3.0, 9.0):
        blocks, case = orc.copy_budget(reqs, 0.1, 1.0, 5.0, t_block, 1e9)
        assert case in (21, 22)
        assert blocks * t_block <= orc.step_latency_after(reqs, blocks, 0.1, 1.0, 5.0)
        if case == 22:
            assert (blocks + 1) * t_block > orc.step_latency_after(reqs, blocks + 1, 0.1, 1.0, 5.0)
    # more link time per block never raises the budget
    picks = [orc.copy_budget(reqs, 0.1, 1.0, 5.0, tb, 1e9)[0] for tb in (0.5, 1.0, 3.0, 9.0, 30.0)]
    assert picks == sorted(picks, reverse=True)
    # a planted mistake (forgetting the constant overhead t_c) changes an answer
    assert orc.copy_budget(reqs, 0.1, 1.0, 5.0, 3.0, 1e9) != orc.copy_budget(reqs, 0.1, 1.0, 0.0, 3.0, 1e9)


def test_library_rejects_bad_models():
    sh = wl.KVShape(2, 1, 1, 8, 4, 32)
    lib, _ = make_pair(sh)
    assert lib.kv_alloc(0, 40) == 0 and lib.swap_out(0) == 0
    lib.sync()
    assert lib.swap_in_begin(0) == 0
    assert lib.copy_budget([0], a_d=1.0, b_d=0.0, t_c=0.0, t_block=0.0, t_budget=10.0)[0] == B.PS_ERR_INVALID
    assert lib.copy_budget([0], a_d=-1.0, b_d=0.0, t_c=0.0, t_block=1.0, t_budget=10.0)[0] == B.PS_ERR_INVALID
    # a block that copies as fast as it is attended to is no longer refused: every interval is scanned
    rc, blocks, _, case = lib.copy_budget([0], a_d=1.0, b_d=0.0, t_c=0.0, t_block=4.0, t_budget=1e9)
    assert (rc, blocks, case) == (B.PS_OK, 10, 22)          # 10 blocks * 4 = 40 <= 40 tokens * 1


def test_largest_feasible_budget_beyond_a_first_failure(repo_root):
    """The hand-worked queue on which the feasibility test fails and holds again (a binary search answers 2)."""
    g = json.load(open(os.path.join(repo_root, "tests", "golden", "adaptive_budget.json")))["non_monotone_case"]
    lib, orc = make_pair(wl.KVShape(**g["shape"]))
    for x in (lib, orc):
        for r, n in g["resident_tokens"] + g["queued_tokens"]:
            assert x.kv_alloc(r, n) == 0
        for r, _ in g["queued_tokens"]:
            assert x.swap_out(r) == 0
    lib.sync(); orc.reap()
    for x in (lib, orc):
        for r, _ in g["queued_tokens"]:
            assert x.swap_in_begin(r) == 0
    kw = dict(a_d=g["a_d"], b_d=g["b_d"], t_c=g["t_c"], t_block=g["t_block"], t_budget=g["t_budget"])
    assert orc.copy_budget(g["batch"], **kw) == (g["blocks"], g["case"])
    rc, blocks, _, case = lib.copy_budget(g["batch"], **kw)
    assert (rc, blocks, case) == (B.PS_OK, g["blocks"], g["case"])
