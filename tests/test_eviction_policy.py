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
