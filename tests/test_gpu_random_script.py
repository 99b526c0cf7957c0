"""A seeded random mix of every state-changing call on the GPU (tensor-core attention shape), driven side by
side with the CPU checker over identical pools: allocation and growth with fresh KV written on the compute
stream, proactive and on-demand offloading, budgeted and unbudgeted reloads (with and without the
partial-copy rule, in layer chunks of several sizes) that interleave with decode steps, frees and cancels.
No host synchronisation is placed between dependent calls: offloads are still in flight when steps run, and
the checker is told how many of them each step reaped (the library reports it), so that any missing stream
ordering in the library (a block reused while a kernel still reads it, a gather racing a write) shows up as a
byte or attention mismatch."""
import numpy as np
import pytest
import torch

from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_util import Pair, bits_to_dev, check_attn


@pytest.mark.parametrize("seed,Hkv,Hq,S", [(1, 8, 32, 16), (2, 8, 64, 32), (3, 8, 8, 16), (4, 8, 16, 48), (5, 4, 28, 16),
                                           (6, 2, 8, 32), (7, 1, 8, 16)])
def test_random_script_with_data(seed, Hkv, Hq, S):
    L, D, nb = 2, 128, 160
    sh = wl.KVShape(L, Hkv, Hq, D, S, nb)
    rng = np.random.default_rng([2512, seed])
    K = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    V = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    # host pool of twice what 8 live requests of 64 blocks can hold (proactive copies of residents included):
    # the checker has no host limit, so the library's must never bind here
    p = Pair(sh, rng.permutation(nb), K, V, max_batch=12, staging_bytes=2 << 20, max_blocks_per_req=64,
             host_pool_bytes=1024 * sh.block_bytes,
             layer_chunk_bytes=[0, -1, 96 * 1024, 1 << 30][seed % 4])
    live, next_id = [], 0
    decoded_steps = reloaded = ruled_steps = reaped_by_steps = 0

    def write_fresh_kv(r, old_blocks):
        """New tokens of a growing request: random KV into its new blocks, enqueued on the compute stream."""
        table = p.orc.block_table(r)[0]
        fresh = table[old_blocks:]
        if not fresh:
            return
        for pool_d, pool_o in ((p.Kd, p.orc.K), (p.Vd, p.orc.V)):
            bits = wl.randn_bf16_bits(rng, (L, len(fresh), S, Hkv, D))
            pool_d[:, fresh] = bits_to_dev(bits)
            pool_o[:, fresh] = bits

    for it in range(140):
        op = int(rng.integers(0, 10))
        if op == 0 and len(live) < 8:
            r, n = next_id, int(rng.integers(0, 500))
            next_id += 1
            rc = p.both("kv_alloc", r, n)
            if rc == B.PS_OK:
                live.append(r)
                write_fresh_kv(r, 0)
        elif op == 1 and live:
            r = int(rng.choice(live))
            if p.orc.reqs[r].state == 1:
                old = len(p.orc.block_table(r)[0])
                if p.both("kv_alloc", r, p.lib.n_tokens(r) + int(rng.integers(1, 120))) == B.PS_OK:
                    write_fresh_kv(r, old)
        elif op == 2 and live:
            p.both("offload_progress", int(rng.choice(live)), int(rng.integers(1, 6)))
        elif op == 3 and live:
            p.both("swap_out", int(rng.choice(live)))
        elif op == 4:
            p.sync()                                             # offloads complete; blocks go back to the pool
        elif op == 5 and live:
            p.both("swap_in_begin", int(rng.choice(live)))
        elif op == 6 and live:
            r = int(rng.choice(live))
            if rng.random() < 0.5:
                p.both("swap_in_cancel", r)
            else:
                a = p.lib.kv_free(r)
                if a == B.PS_ERR_BUSY and p.orc.reqs[r].state == 1:
                    p.sync()                                     # its reload or proactive copy had not been seen complete
                    a = p.lib.kv_free(r)
                b = p.orc.kv_free(r)
                assert a == b, (it, a, b)
                if a == B.PS_OK:
                    live.remove(r)
        elif op >= 7 and live:
            budget = int(rng.choice([-1, 0, 3, 8, 20])) * sh.block_bytes
            q = wl.randn_bf16_bits(rng, (L, len(live), Hq, D))
            qd = bits_to_dev(q)
            out = torch.full_like(qd, 3.0)
            rule, beta = None, None
            if rng.random() < 0.5:                               # the partial-copy test for the queued reloads
                beta = 1.5
                rule = {r: [(0, 1), (1, 1), (40, 64), (200, 64)][int(rng.integers(0, 4))]
                        for r in live if p.orc.reqs[r].state == 4}
                rr = sorted(rule)
                rc, mask, st = p.lib.step_ruled(qd, out, live, budget, beta, rr, [rule[r][0] for r in rr],
                                                [rule[r][1] for r in rr])
                ruled_steps += 1
            else:
                rc, mask, st = p.lib.step(qd, out, live, budget)
            assert rc == B.PS_OK, p.lib.last_error()
            p.orc.reap(st["swapouts_reaped"])                    # offloads the step found complete, in issue order
            reaped_by_steps += st["swapouts_reaped"]
            plan, omask, want = p.orc.step(budget, live, q, rule=rule, beta=beta)
            assert mask == omask, it
            assert st["blocks_copied"] == sum(hi - lo for _, lo, hi in plan)
            reloaded += st["reloads_completed"]
            rows = [i for i, m in enumerate(mask) if m]
            if rows:
                decoded_steps += 1
                check_attn(out[:, rows], want[:, rows])
            idle = [i for i, m in enumerate(mask) if not m]
            if idle:
                assert (out[:, idle].float() == 3.0).all()
        if it % 20 == 19:
            p.sync()
            p.assert_pools_equal()
            p.assert_tables_equal(live)
            p.orc.check_invariants()
    p.sync()
    p.assert_pools_equal()
    p.assert_tables_equal(live)
    assert decoded_steps > 10 and reloaded > 0 and ruled_steps > 5
