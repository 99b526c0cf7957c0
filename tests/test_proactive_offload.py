"""Proactive incremental offloading (Section 4.3, "Asynchronous Offloading"): a copy for every n_off newly
filled blocks, so that eviction only has the tail left to move.

CPU part: the checker against element loops and invariants, the library's host logic against the checker.
GPU part (marked gpu): segments, pools and attention through the C ABI against the checker."""
import ctypes as C

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


def small_oracle(seed=3, L=2, nb=48, S=4, Hkv=2, D=8):
    rng = np.random.default_rng(seed)
    K = rng.integers(0, 65536, size=(L, nb, S, Hkv, D), dtype=np.uint16)
    V = rng.integers(0, 65536, size=(L, nb, S, Hkv, D), dtype=np.uint16)
    order = rng.permutation(nb)
    return po.PsOracle(L, Hkv, Hkv, D, S, nb, order, K, V), K.copy(), V.copy()


def test_checker_segments_cover_filled_blocks_in_groups_and_match_element_loops():
    orc, K0, V0 = small_oracle()
    assert orc.kv_alloc(7, 4 * 5 + 3) == po.OK                  # 5 full blocks + a partial one
    assert orc.offload_progress(7, 2) == (po.OK, 4)            # two groups of 2; the fifth full block waits
    assert orc.host_blocks(7) == 4
    assert orc.offload_progress(7, 2) == (po.OK, 0)            # nothing new
    assert orc.kv_alloc(7, 4 * 8) == po.OK                     # grows to 8 full blocks
    assert orc.offload_progress(7, 3) == (po.OK, 3)            # blocks 4..6; block 7 waits for a group of 3
    assert [(lo, hi) for lo, hi, _ in orc.reqs[7].segs] == [(0, 4), (4, 7)]
    assert orc.reqs[7].state == po.ST_RESIDENT
    table = list(orc.reqs[7].table)
    assert orc.swap_out(7) == po.OK                            # only the tail [7, 8) goes out now
    assert [(lo, hi) for lo, hi, _ in orc.reqs[7].segs] == [(0, 4), (4, 7), (7, 8)]
    for lo, hi, img in orc.reqs[7].segs:                       # each segment against the element-by-element image
        want = po.brute_force_image(K0, V0, table[lo:hi], orc.L, orc.S, orc.Hkv, orc.D)
        assert img.reshape(-1).tolist() == want
    assert orc.host_used == 8 * orc.block_bytes
    orc.reap()
    orc.check_invariants()
    # reload through the segments under a budget of 3 blocks per step: a growing prefix, then identical logical KV
    assert orc.swap_in_begin(7) == po.OK
    steps = 0
    while orc.missing_blocks(7):
        orc.step(3 * orc.block_bytes)
        steps += 1
    assert steps == 3 and orc.host_used == 0
    new = orc.reqs[7].table
    for l in range(orc.L):
        for j in range(8):
            assert np.array_equal(orc.K[l, new[j]], K0[l, table[j]]) and np.array_equal(orc.V[l, new[j]], V0[l, table[j]])


def test_checker_proactive_and_on_demand_offload_restore_the_same_bytes():
    a, _, _ = small_oracle(seed=9)
    b, _, _ = small_oracle(seed=9)
    for x in (a, b):
        assert x.kv_alloc(1, 30) == po.OK and x.kv_alloc(2, 17) == po.OK
    assert a.offload_progress(1, 1) == (po.OK, 7) and a.offload_progress(2, 4) == (po.OK, 4)
    for x in (a, b):
        for r in (1, 2):
            assert x.swap_out(r) == po.OK
        x.reap()
        for r in (2, 1):
            assert x.swap_in_begin(r) == po.OK
        x.step(-1)
    assert a.block_table(1) == b.block_table(1) and a.block_table(2) == b.block_table(2)
    assert np.array_equal(a.K, b.K) and np.array_equal(a.V, b.V)


def test_checker_errors_and_free_of_a_resident_request_with_copies():
    orc, _, _ = small_oracle()
    assert orc.offload_progress(5, 2) == (po.ERR_INVALID, 0)
    assert orc.kv_alloc(5, 16) == po.OK
    assert orc.offload_progress(5, 0) == (po.ERR_INVALID, 0)
    assert orc.offload_progress(5, 2) == (po.OK, 4)
    assert orc.kv_free(5) == po.OK and orc.host_used == 0       # the copies go with the request
    assert orc.kv_alloc(6, 16) == po.OK and orc.swap_out(6) == po.OK
    assert orc.offload_progress(6, 2) == (po.ERR_STATE, 0)


def test_library_host_logic_matches_checker_on_a_random_script():
    sh = wl.KVShape(3, 2, 4, 64, 8, 128)
    rng = np.random.default_rng(77)
    order = rng.permutation(sh.num_gpu_blocks)
    lib = B.KVSwap(num_layers=sh.num_layers, num_kv_heads=sh.num_kv_heads, num_q_heads=sh.num_q_heads,
                   head_dim=sh.head_dim, block_size=sh.block_size, num_gpu_blocks=sh.num_gpu_blocks,
                   max_blocks_per_req=64, host_pool_bytes=1 << 40, initial_free_order=order,
                   flags=B.PS_FLAG_BOOKKEEPING_ONLY)
    orc = po.PsOracle(sh.num_layers, sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size, sh.num_gpu_blocks, order)
    live = []
    for it in range(1500):
        op = int(rng.integers(0, 8))
        if op == 0 and len(live) < 10:
            r = 1000 + it
            a, b = lib.kv_alloc(r, int(rng.integers(0, 60))), None
            b = orc.kv_alloc(r, lib.n_tokens(r) if a == 0 else 0) if a == 0 else a
            assert a == b
            if a == 0:
                live.append(r)
        elif op == 1 and live:                                   # decode appends tokens
            r = int(rng.choice(live))
            n = lib.n_tokens(r) + int(rng.integers(1, 30))
            assert lib.kv_alloc(r, n) == orc.kv_alloc(r, n)
        elif op in (2, 3) and live:
            r = int(rng.choice(live))
            n_off = int(rng.integers(1, 5))
            assert lib.offload_progress(r, n_off) == orc.offload_progress(r, n_off), (it, r)
        elif op == 4 and live:
            r = int(rng.choice(live))
            assert lib.swap_out(r) == orc.swap_out(r)
        elif op == 5:
            assert lib.sync() == 0
            orc.reap()
        elif op == 6 and live:
            r = int(rng.choice(live))
            assert lib.swap_in_begin(r) == orc.swap_in_begin(r)
        elif op == 7 and live:
            if rng.random() < 0.3:
                r = int(rng.choice(live))
                a, b = lib.kv_free(r), orc.kv_free(r)
                assert a == b
                if a == 0:
                    live.remove(r)
            else:
                budget = int(rng.choice([-1, 0, 2, 5])) * sh.block_bytes
                orc.reap()
                rc, mask, st = lib.step(None, None, live, budget)
                plan, omask, _ = orc.step(budget, live)
                assert rc == 0 and mask == omask and st["blocks_copied"] == sum(hi - lo for _, lo, hi in plan)
        for r in live:
            assert lib.host_blocks(r)[0] == orc.host_blocks(r)
            segs = [(lo, hi) for _, _, lo, hi in lib.host_segments(r)]
            assert segs == [(lo, hi) for lo, hi, _ in orc.reqs[r].segs]
    lib.sync(); orc.reap()
    for r in live:
        assert lib.block_table(r) == orc.block_table(r)
    orc.check_invariants()


def test_batch_sweep_with_per_request_thresholds_equals_the_single_calls():
    """A sweep with thresholds n_off^r is the per-request trigger applied in order; requests that are not
    resident are skipped; a host pool that fills up stops the sweep where it stands."""
    sh = wl.KVShape(2, 2, 4, 64, 8, 128)
    order = np.random.default_rng(5).permutation(sh.num_gpu_blocks)
    mk = lambda host: B.KVSwap(num_layers=2, num_kv_heads=2, num_q_heads=4, head_dim=64, block_size=8, num_gpu_blocks=128,
                               max_blocks_per_req=64, host_pool_bytes=host, initial_free_order=order,
                               flags=B.PS_FLAG_BOOKKEEPING_ONLY)
    lib, ref = mk(1 << 40), mk(1 << 40)
    orc = po.PsOracle(2, 2, 4, 64, 8, 128, order)
    tokens = {1: 100, 2: 37, 3: 8, 4: 64, 5: 90}
    for x in (lib, ref, orc):
        for r, n in tokens.items():
            assert x.kv_alloc(r, n) == 0
        assert x.swap_out(4) == 0                                  # request 4 is not resident during the sweep
    reqs, thr = [1, 2, 99, 3, 4, 5], [5, 2, 1, 1, 1, 3]              # 99 is unknown
    # hand count: 100 tokens = 12 full blocks -> 2 groups of 5 = 10; 37 -> 4 full -> 4; 8 -> 1 full -> 1; 90 -> 11 -> 9
    assert orc.offload_sweep(reqs, thr) == (po.OK, 24)
    assert lib.offload_sweep(reqs, thr) == (B.PS_OK, 24)
    singles = sum(ref.offload_progress(r, n)[1] for r, n in zip(reqs, thr) if r in (1, 2, 3, 5))
    assert singles == 24
    for r in (1, 2, 3, 5):
        assert lib.host_blocks(r)[0] == ref.host_blocks(r)[0] == orc.host_blocks(r)
        assert lib.host_segments(r)[0][2:] == ref.host_segments(r)[0][2:]
    assert lib.offload_sweep(reqs, thr) == (B.PS_OK, 0) and orc.offload_sweep(reqs, thr) == (po.OK, 0)   # nothing new
    for x in (lib, orc):                                           # decode goes on: more blocks fill up
        assert x.kv_alloc(2, 37 + 16) == 0
    assert lib.offload_sweep([2], [2]) == (B.PS_OK, 2) and orc.offload_sweep([2], [2]) == (po.OK, 2)
    assert lib.offload_sweep([1], [0])[0] == B.PS_ERR_INVALID and orc.offload_sweep([1], [0])[0] == po.ERR_INVALID
    # a host pool of 12 blocks: the first request's 10 blocks fit, the second one's 4 do not
    small = mk(12 * sh.block_bytes)
    for r, n in tokens.items():
        assert small.kv_alloc(r, n) == 0
    assert small.offload_sweep([1, 2, 3], [5, 2, 1]) == (B.PS_ERR_HOST_NOMEM, 10)
    assert small.host_blocks(1)[0] == 10 and small.host_blocks(2)[0] == 0 and small.host_blocks(3)[0] == 0


# ------------------------------------------------------------------------------------------------- GPU

@pytest.mark.gpu
def test_gpu_proactive_offload_segments_round_trip_and_attention():
    import torch
    from gpu_util import Pair, bits_to_dev, check_attn
    L, Hkv, Hq, D, S, nb = 3, 8, 32, 128, 16, 200
    sh = wl.KVShape(L, Hkv, Hq, D, S, nb)
    rng = np.random.default_rng(2024)
    K = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    V = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    p = Pair(sh, rng.permutation(nb), K, V, max_batch=4, staging_bytes=1 << 20)
    lens = {0: 9 * S + 5, 1: 30 * S, 2: 3}
    for r, n in lens.items():
        assert p.both("kv_alloc", r, n) == B.PS_OK
    assert p.both("offload_progress", 0, 4) == (B.PS_OK, 8)
    assert p.both("offload_progress", 1, 7) == (B.PS_OK, 28)
    assert p.both("offload_progress", 2, 1) == (B.PS_OK, 0)
    # request 0 decodes on: new blocks are allocated and filled on the compute stream, then offloaded further
    assert p.both("kv_alloc", 0, 20 * S + 1) == B.PS_OK
    table = p.orc.block_table(0)[0]
    fresh = table[10:]
    newk = wl.randn_bf16_bits(rng, (L, len(fresh), S, Hkv, D))
    p.Kd[:, fresh] = bits_to_dev(newk)
    p.orc.K[:, fresh] = newk
    assert p.both("offload_progress", 0, 4) == (B.PS_OK, 12)
    assert p.lib.sync() == B.PS_OK
    assert p.lib.host_blocks(0) == (20, 20) and p.orc.host_blocks(0) == 20
    assert p.lib.block_table(0)[1] == B.PS_REQ_RESIDENT
    for r in (0, 1, 2):
        assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    p.assert_tables_equal([0, 1, 2])
    for r in (0, 1, 2):
        segs = p.lib.host_segments(r)
        want = p.orc.reqs[r].segs
        assert [(lo, hi) for _, _, lo, hi in segs] == [(lo, hi) for lo, hi, _ in want]
        for (ptr, nbytes, lo, hi), (_, _, img) in zip(segs, want):
            got = np.ctypeslib.as_array((C.c_uint16 * (nbytes // 2)).from_address(ptr))
            assert np.array_equal(got, img.reshape(-1)), (r, lo, hi)
    free_ids = sorted(p.orc.free)
    p.Kd[:, free_ids] = 0; p.Vd[:, free_ids] = 0
    p.orc.K[:, free_ids] = 0; p.orc.V[:, free_ids] = 0
    for r in (1, 0, 2):
        assert p.both("swap_in_begin", r) == B.PS_OK
    reqs = [0, 1, 2]
    q = wl.randn_bf16_bits(rng, (L, 3, Hq, D))
    qd = bits_to_dev(q)
    budget = 9 * sh.block_bytes                                   # runs of blocks cross segment borders
    steps = 0
    while any(p.orc.missing_blocks(r) for r in reqs):
        out = torch.zeros_like(qd)
        rc, mask, st = p.lib.step(qd, out, reqs, budget)
        assert rc == B.PS_OK, p.lib.last_error()
        plan, omask, want = p.orc.step(budget, reqs, q)
        assert mask == omask
        p.sync()
        p.assert_pools_equal()
        live = [i for i, m in enumerate(mask) if m]
        if live:
            check_attn(out[:, live], want[:, live])
        steps += 1
        assert steps < 20
    assert steps == -(-(21 + 30 + 1) // 9)
    p.assert_tables_equal(reqs)
    assert p.lib.host_segments(0) == []
