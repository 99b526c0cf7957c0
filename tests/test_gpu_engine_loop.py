"""The block management driven the way a serving engine drives it, on the GPU with real bytes.

Two loops.  (1) A caller-driven layer loop (Appendix B): reload chunks issued per layer, and before each layer's
attention the forward pass appends the new token's K and V to every request, the readmitted ones included,
which is what ps_reload_fence is for.  (2) The paper's closed loop (Sections 4.2-4.3): the queue is ordered,
victims are taken from its tail when the pool is short, requests are readmitted from its head, the copy
budget is chosen per step, ps_step reloads and decodes, decoding appends tokens, filled blocks are offloaded
ahead of eviction.  In both, the CPU checker
replays the same calls; block tables, pool bytes and attention outputs must agree.
"""
import numpy as np
import pytest
import torch

from oracle import ps_oracle as po
from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_util import Pair, bits_to_dev, check_attn


def make_pair(L, nb, S, rng, **kw):
    sh = wl.KVShape(L, 8, 32, 128, S, nb)
    K = wl.randn_bf16_bits(rng, (L, nb, S, 8, 128))
    V = wl.randn_bf16_bits(rng, (L, nb, S, 8, 128))
    return sh, Pair(sh, rng.permutation(nb).astype(np.int32), K, V, **kw)


def append_token(p, layer, req, n_tokens, k_bits, v_bits):
    """What a decode forward does before a layer's attention: the new token's K and V rows go into the slot
    of token n_tokens - 1.  Device side on the compute stream (a plain indexed write, not the path under
    test); checker side in its arrays."""
    S = p.sh.block_size
    table = p.orc.reqs[req].table
    blk, slot = table[(n_tokens - 1) // S], (n_tokens - 1) % S
    p.Kd[layer, blk, slot] = bits_to_dev(k_bits)
    p.Vd[layer, blk, slot] = bits_to_dev(v_bits)
    p.orc.K[layer][blk][slot] = k_bits
    p.orc.V[layer][blk][slot] = v_bits


def test_caller_driven_layer_loop_appends_into_reloaded_blocks():
    rng = np.random.default_rng(20251214)
    L, S = 4, 16
    sh, p = make_pair(L, 256, S, rng, max_batch=8)
    tokens = {0: 100, 1: 333, 2: 16, 3: 47, 4: 512, 5: 129}
    grown = {r: 0 for r in tokens}
    while any(grown[r] < tokens[r] for r in tokens):                  # interleaved growth: scattered tables
        for r in tokens:
            if grown[r] < tokens[r]:
                grown[r] = min(tokens[r], grown[r] + S)
                assert p.both("kv_alloc", r, grown[r]) == B.PS_OK
    reqs = sorted(tokens)
    for round_no, victims in enumerate([[1, 4], [3], [1, 5, 0]]):
        for v in victims:
            assert p.both("swap_out", v) == B.PS_OK
        p.sync()
        # readmission: every layer's reload is issued up front on the copy streams ...
        for v in victims:
            assert p.both("swap_in_begin", v) == B.PS_OK
            n = p.orc.blocks_for(tokens[v])
            for l in range(L):
                assert p.both("swap_in_layer", v, l, 0, n) == B.PS_OK
        # ... and the forward pass runs under it: a new token for everyone, layer by layer
        for r in reqs:
            tokens[r] += 1
            assert p.both("kv_alloc", r, tokens[r]) == B.PS_OK
        q_bits = wl.randn_bf16_bits(rng, (L, len(reqs), sh.num_q_heads, sh.head_dim))
        qd = bits_to_dev(q_bits)
        out = torch.zeros_like(qd)
        for l in range(L):
            assert p.lib.reload_fence(l) == B.PS_OK, p.lib.last_error()
            for r in reqs:
                append_token(p, l, r, tokens[r], wl.randn_bf16_bits(rng, (8, 128)), wl.randn_bf16_bits(rng, (8, 128)))
            assert p.lib.decode_attn(l, qd[l], out[l], reqs) == B.PS_OK, p.lib.last_error()
        p.sync()
        for l in range(L):
            want, _ = p.orc.decode_attn(l, q_bits[l], reqs)
            check_attn(out[l], want)
        p.assert_tables_equal(reqs)
        p.assert_pools_equal()
        p.orc.check_invariants()
    assert p.lib.reload_fence(-1) == B.PS_OK
    assert p.lib.reload_fence(L) == B.PS_ERR_INVALID
    assert p.lib.reload_fence(-2) == B.PS_ERR_INVALID


def test_fence_orders_an_append_behind_a_long_reload():
    """A reload of ~400 MB is still in flight when the forward pass wants to append to the reloaded request's
    last block; the write of each layer must land after that layer's scatter."""
    rng = np.random.default_rng(20251215)
    L, S, nb = 4, 16, 2048
    sh, p = make_pair(L, nb, S, rng, max_batch=4)
    tokens = {0: 200, 1: 1500 * S - 9}                                # request 1: 1500 blocks, last one partly filled
    for r, n in tokens.items():
        assert p.both("kv_alloc", r, n) == B.PS_OK
    assert p.both("swap_out", 1) == B.PS_OK
    p.sync()
    new_kv = [(wl.randn_bf16_bits(rng, (8, 128)), wl.randn_bf16_bits(rng, (8, 128))) for _ in range(L)]
    q_bits = wl.randn_bf16_bits(rng, (L, 2, sh.num_q_heads, sh.head_dim))
    qd = bits_to_dev(q_bits)
    out = torch.zeros_like(qd)
    torch.cuda.synchronize()
    # the library first, with nothing slow on the host in between (the checker replays afterwards): the
    # appends are enqueued while most of the reload is still on the link
    assert p.lib.swap_in_begin(1) == B.PS_OK
    for l in range(L):
        assert p.lib.swap_in_layer(1, l, 0, 1500) == B.PS_OK
    assert p.lib.kv_alloc(1, tokens[1] + 1) == B.PS_OK
    blk, slot = p.lib.block_table(1)[0][tokens[1] // S], tokens[1] % S
    kv_dev = [(bits_to_dev(k), bits_to_dev(v)) for k, v in new_kv]
    for l in range(L):
        assert p.lib.reload_fence(l) == B.PS_OK, p.lib.last_error()
        p.Kd[l, blk, slot] = kv_dev[l][0]
        p.Vd[l, blk, slot] = kv_dev[l][1]
        assert p.lib.decode_attn(l, qd[l], out[l], [0, 1]) == B.PS_OK, p.lib.last_error()
    assert p.orc.swap_in_begin(1) == po.OK
    for l in range(L):
        assert p.orc.swap_in_layer(1, l, 0, 1500) == po.OK
    tokens[1] += 1
    assert p.orc.kv_alloc(1, tokens[1]) == po.OK
    assert p.orc.reqs[1].table[(tokens[1] - 1) // S] == blk
    for l in range(L):
        p.orc.K[l][blk][slot], p.orc.V[l][blk][slot] = new_kv[l]
    p.sync()
    p.assert_pools_equal()
    for l in (0, L - 1):
        want, _ = p.orc.decode_attn(l, q_bits[l], [0, 1])
        check_attn(out[l], want)


def test_closed_loop_with_real_bytes():
    rng = np.random.default_rng(31)             # the script's decisions
    drng = np.random.default_rng(32)            # queries and appended K, V
    L, S, nb = 2, 16, 64
    # host pool: every request could be on the host at once (the checker has no host limit)
    sh, p = make_pair(L, nb, S, rng, max_batch=16, host_pool_bytes=4 * nb * L * 2 * S * 8 * 128 * 2)
    lib, orc = p.lib, p.orc
    ids = list(range(14))
    tokens = {r: int(rng.integers(30, 240)) for r in ids}
    weight = {r: float(rng.choice([1.0, 2.0])) for r in ids}
    deadline = {r: float(rng.uniform(200, 3000)) for r in ids}
    now = 0.0
    model = dict(a_d=0.1, b_d=2.0, t_c=5.0, t_block=16.0)    # both branches of case 2 of the budget rule occur
    born = dict(tokens)
    next_id = 100
    cases = set()
    last_run = {}
    decoded_total = evicted_total = reloaded_total = finished_total = ahead_total = 0
    for rnd in range(36):
        now += 60.0
        queue = [r for r in ids if r in orc.reqs or r <= rnd or r >= 100]
        exec_t = [model["a_d"] * tokens[r] + model["b_d"] for r in queue]
        remain = [deadline[r] - now for r in queue]
        w = [weight[r] for r in queue]
        waited = [now - last_run.setdefault(r, now - 60.0) for r in queue]    # since arrival or the last decode
        kw = dict(eta=150.0, gamma=0.9, t_c=model["t_c"])
        o_order, o_cls, o_tb = po.order_queue(exec_t, remain, w, waited=waited, tau=1500.0, **kw)
        rc, l_order, l_cls, l_tb = B.ps_order_queue(exec_t, remain, w, waited_us=waited, tau=1500.0, **kw)
        assert rc == B.PS_OK and (l_order, l_cls, l_tb) == (o_order, o_cls, o_tb)
        sorted_q = [queue[i] for i in o_order]
        sorted_waited = [waited[i] for i in o_order]
        for r in sorted_q:                                             # head first: admit or readmit
            need = orc.blocks_for(tokens[r])
            st = orc.reqs[r].state if r in orc.reqs else None
            if st in (po.ST_RESIDENT, po.ST_SWAPPING_IN, po.ST_SWAPPING_OUT):
                continue
            if orc.num_free_blocks() < need:
                short = need - orc.num_free_blocks()
                want_v = orc.select_victims(sorted_q, sorted_waited, 1500.0, 0.8, short)
                rc, victims, freed = lib.select_victims(sorted_q, sorted_waited, 1500.0, 0.8, short)
                assert (victims, freed) == want_v
                victims = [v for v in victims if sorted_q.index(v) > sorted_q.index(r)]
                for v in victims:
                    ahead_total += len(lib.host_segments(v)) > 0      # proactive copies: only the tail is left to move
                    assert p.both("swap_out", v) == B.PS_OK
                    evicted_total += 1
                p.sync()
            if orc.num_free_blocks() < need:
                continue
            if st is None:
                assert p.both("kv_alloc", r, tokens[r]) == B.PS_OK
            else:
                assert p.both("swap_in_begin", r) == B.PS_OK
                reloaded_total += 1
        budget_o = orc.copy_budget(sorted_q, t_budget=o_tb, **model)
        rc, blocks, nbytes, case = lib.copy_budget(sorted_q, t_budget=o_tb, **model)
        assert rc == B.PS_OK and (blocks, case) == budget_o
        cases.add(case)
        q_bits = wl.randn_bf16_bits(drng, (L, len(sorted_q), sh.num_q_heads, sh.head_dim))
        qd = bits_to_dev(q_bits)
        out = torch.zeros_like(qd)
        rc, mask, st = lib.step(qd, out, sorted_q, nbytes)
        assert rc == B.PS_OK, lib.last_error()
        plan, omask, want = orc.step(nbytes, sorted_q, q_bits)
        assert mask == omask
        live = [i for i, m in enumerate(mask) if m]
        decoded_total += len(live)
        torch.cuda.synchronize()
        if live:
            check_attn(out[:, live], want[:, live])
        for i in live:                                                 # decoding appends a token and its K, V
            r = sorted_q[i]
            last_run[r] = now
            a, b = lib.kv_alloc(r, tokens[r] + 1), orc.kv_alloc(r, tokens[r] + 1)
            assert a == b
            if a == B.PS_OK:
                tokens[r] += 1
                for l in range(L):
                    append_token(p, l, r, tokens[r], wl.randn_bf16_bits(drng, (8, 128)), wl.randn_bf16_bits(drng, (8, 128)))
            if tokens[r] - born[r] >= 10:                              # the request is done; another arrives
                assert p.both("kv_free", r) == B.PS_OK
                finished_total += 1
                ids[ids.index(r)] = next_id
                tokens[next_id] = born[next_id] = int(rng.integers(30, 240))
                weight[next_id] = float(rng.choice([1.0, 2.0]))
                deadline[next_id] = now + float(rng.uniform(200, 3000))
                next_id += 1
        # proactive offloading after the step: low-weight requests, the likelier victims, copy more often
        holders = [r for r in sorted_q if r in orc.reqs]
        assert p.both("offload_sweep", holders, [2 if weight[r] == 1.0 else 4 for r in holders])[0] == B.PS_OK
        p.assert_tables_equal(holders)
        orc.check_invariants()
    p.sync()
    p.assert_pools_equal()
    assert decoded_total > 100 and evicted_total > 5 and reloaded_total > 5 and finished_total > 5 and ahead_total > 3
    assert {21, 22} <= cases
