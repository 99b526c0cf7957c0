"""GPU parity at the edges of the path: empty and maximal batches, budgets of zero and of less than one
block, requests without blocks, a request at the table limit, a pool used to its last block."""
import numpy as np
import pytest
import torch

from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_util import Pair, bits_to_dev, check_attn


def make_pair(L, Hkv, Hq, D, S, nb, seed, **kw):
    sh = wl.KVShape(L, Hkv, Hq, D, S, nb)
    rng = np.random.default_rng(seed)
    K = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    V = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    return sh, rng, Pair(sh, rng.permutation(nb), K, V, **kw)


def test_empty_batch_and_budgets_below_one_block():
    sh, rng, p = make_pair(3, 8, 32, 128, 16, 96, 11, max_batch=8)
    for r, n in ((0, 40), (1, 16), (2, 100)):
        assert p.both("kv_alloc", r, n) == B.PS_OK
    assert p.both("swap_out", 2) == B.PS_OK
    p.sync()
    assert p.both("swap_in_begin", 2) == B.PS_OK
    # an empty decode batch is legal: the step only moves the reload forward
    q0 = torch.zeros((3, 0, 32, 128), dtype=torch.bfloat16, device="cuda")
    assert p.lib.decode_attn(0, q0[0], q0[0], []) == B.PS_OK
    for budget in (0, 1, sh.block_bytes - 1):            # floor(bytes / block bytes) = 0 blocks
        rc, mask, st = p.lib.step(q0, q0, [], budget)
        plan, omask, _ = p.orc.step(budget, [], None)
        assert rc == B.PS_OK and mask == omask == [] and plan == [] and st["blocks_copied"] == 0
    assert p.lib.missing_blocks(2) == p.orc.missing_blocks(2) == 7
    # exactly one block per step, no decode rows: 7 steps bring the request back
    for k in range(7):
        rc, mask, st = p.lib.step(q0, q0, [], sh.block_bytes)
        plan, _, _ = p.orc.step(sh.block_bytes, [], None)
        assert rc == B.PS_OK and st["blocks_copied"] == 1 and plan == [(2, k, k + 1)]
        assert st["reloads_completed"] == (1 if k == 6 else 0)
    p.sync()
    p.assert_pools_equal()
    p.assert_tables_equal([0, 1, 2])
    # a budget of zero with a decode batch: the queued request does not decode, the others do
    assert p.both("swap_out", 1) == B.PS_OK
    p.sync()
    assert p.both("swap_in_begin", 1) == B.PS_OK
    q = wl.randn_bf16_bits(rng, (3, 3, 32, 128))
    qd = bits_to_dev(q)
    out = torch.full_like(qd, 5.0)
    rc, mask, st = p.lib.step(qd, out, [0, 1, 2], 0)
    plan, omask, want = p.orc.step(0, [0, 1, 2], q)
    assert rc == B.PS_OK and mask == omask == [1, 0, 1] and st["decoded"] == 2
    p.sync()
    check_attn(out[:, [0, 2]], want[:, [0, 2]])
    assert (out[:, 1].float() == 5.0).all()
    p.orc.check_invariants()


def test_requests_without_blocks_go_out_and_come_back():
    sh, rng, p = make_pair(2, 4, 8, 64, 16, 32, 12, max_batch=8)
    assert p.both("kv_alloc", 0, 0) == B.PS_OK
    assert p.both("kv_alloc", 1, 33) == B.PS_OK
    assert p.both("swap_out", 0) == B.PS_OK              # nothing to copy
    p.sync()
    assert p.lib.block_table(0) == p.orc.block_table(0)
    assert p.both("swap_in_begin", 0) == B.PS_OK         # nothing to restore: resident at once
    assert p.lib.block_table(0) == p.orc.block_table(0)
    assert p.lib.missing_blocks(0) == p.orc.missing_blocks(0) == 0
    q = wl.randn_bf16_bits(rng, (2, 2, 8, 64))
    qd = bits_to_dev(q)
    out = torch.full_like(qd, 9.0)
    rc, mask, st = p.lib.step(qd, out, [0, 1], -1)
    plan, omask, want = p.orc.step(-1, [0, 1], q)
    assert rc == B.PS_OK and mask == omask == [1, 1] and plan == []
    p.sync()
    check_attn(out, want)                                # the row without tokens is all zeros on both sides
    assert (out[:, 0].float() == 0.0).all()
    assert p.both("kv_free", 0) == B.PS_OK
    p.orc.check_invariants()


def test_request_at_the_table_limit_and_pool_used_to_the_last_block():
    S, nb, cap = 16, 72, 40
    sh, rng, p = make_pair(2, 8, 64, 128, S, nb, 13, max_batch=4, max_blocks_per_req=cap)
    assert p.lib.kv_alloc(0, cap * S + 1) == B.PS_ERR_INVALID       # one token beyond the table limit
    assert p.both("kv_alloc", 0, cap * S) == B.PS_OK                 # exactly at the limit
    assert p.both("kv_alloc", 1, (nb - cap) * S) == B.PS_OK          # the pool's last block
    assert p.lib.num_free_blocks() == p.orc.num_free_blocks() == 0
    assert p.both("kv_alloc", 2, 1) == B.PS_ERR_NOMEM
    q = wl.randn_bf16_bits(rng, (2, 2, 64, 128))
    qd = bits_to_dev(q)
    out = torch.zeros_like(qd)
    rc, mask, _ = p.lib.step(qd, out, [0, 1], -1)
    _, omask, want = p.orc.step(-1, [0, 1], q)
    assert rc == B.PS_OK and mask == omask == [1, 1]
    p.sync()
    check_attn(out, want)
    # with no free block a readmission is refused and changes nothing; after an eviction it goes through
    assert p.both("swap_out", 0) == B.PS_OK
    p.sync()
    assert p.both("kv_alloc", 2, (cap - 1) * S) == B.PS_OK
    assert p.both("swap_in_begin", 0) == B.PS_ERR_NOMEM
    p.assert_tables_equal([0, 1, 2])
    assert p.both("kv_free", 2) == B.PS_OK
    assert p.both("swap_in_begin", 0) == B.PS_OK
    out2 = torch.zeros_like(qd)
    rc, mask, st = p.lib.step(qd, out2, [0, 1], -1)
    _, omask, want2 = p.orc.step(-1, [0, 1], q)
    assert rc == B.PS_OK and mask == omask == [1, 1] and st["blocks_copied"] == cap
    p.sync()
    p.assert_pools_equal()
    check_attn(out2, want2)
    assert torch.equal(out, out2)                                    # the same bytes in other blocks
    p.orc.check_invariants()


@pytest.mark.parametrize("Hkv,Hq,D,kernel", [(8, 32, 128, B.PS_ATTN_MMA), (4, 8, 64, B.PS_ATTN_SIMT)])
def test_batch_of_the_maximum_size_with_one_token_rows(Hkv, Hq, D, kernel):
    """256 rows (the largest batch a context takes), most of one token: more rows than work items per CTA."""
    S, nbatch = 16, 256
    sh, rng, p = make_pair(1, Hkv, Hq, D, S, 400, [14, Hkv], max_batch=nbatch, attn_kernel=kernel)
    ctxs = [1] * nbatch
    ctxs[7], ctxs[100], ctxs[255] = 5 * S + 3, 2 * S, 64 * S - 1
    for r, c in enumerate(ctxs):
        assert p.both("kv_alloc", r, c) == B.PS_OK
    reqs = list(range(nbatch))
    q = wl.randn_bf16_bits(rng, (1, nbatch, Hq, D))
    qd = bits_to_dev(q)
    out = torch.zeros_like(qd)
    rc, mask, st = p.lib.step(qd, out, reqs, -1)
    _, omask, want = p.orc.step(-1, reqs, q)
    assert rc == B.PS_OK and mask == omask and st["decoded"] == nbatch
    p.sync()
    check_attn(out, want)
    # one row more than the context was created for is refused before any launch
    big = torch.zeros((1, nbatch + 1, Hq, D), dtype=torch.bfloat16, device="cuda")
    assert p.lib.decode_attn(0, big[0], big[0], reqs + [0]) == B.PS_ERR_INVALID


def test_two_contexts_of_different_shapes_interleaved():
    """Two live contexts (different shapes, kernels and staging sizes) driven in turn: nothing is shared."""
    sh_a, rng_a, a = make_pair(3, 8, 32, 128, 16, 128, 21, max_batch=8, staging_bytes=1 << 20)
    sh_b, rng_b, b = make_pair(2, 4, 8, 64, 16, 96, 22, max_batch=8)
    ctx_a, ctx_b = [300, 77, 512, 16], [40, 200, 129]
    for r, n in enumerate(ctx_a):
        assert a.both("kv_alloc", r, n) == B.PS_OK
    for r, n in enumerate(ctx_b):
        assert b.both("kv_alloc", r, n) == B.PS_OK
    qa = wl.randn_bf16_bits(rng_a, (3, 4, 32, 128))
    qb = wl.randn_bf16_bits(rng_b, (2, 3, 8, 64))
    qa_d, qb_d = bits_to_dev(qa), bits_to_dev(qb)
    assert a.both("swap_out", 2) == B.PS_OK
    assert b.both("swap_out", 1) == B.PS_OK
    assert a.both("swap_out", 0) == B.PS_OK
    a.sync()
    b.sync()
    for r in (2, 0):
        assert a.both("swap_in_begin", r) == B.PS_OK
    assert b.both("swap_in_begin", 1) == B.PS_OK
    budget_a, budget_b = 9 * sh_a.block_bytes, 4 * sh_b.block_bytes
    for _ in range(8):
        oa = torch.full_like(qa_d, 2.0)
        ob = torch.full_like(qb_d, 2.0)
        rc_a, mask_a, _ = a.lib.step(qa_d, oa, [0, 1, 2, 3], budget_a)      # both steps in flight together
        rc_b, mask_b, _ = b.lib.step(qb_d, ob, [0, 1, 2], budget_b)
        assert rc_a == B.PS_OK and rc_b == B.PS_OK
        _, want_mask_a, want_a = a.orc.step(budget_a, [0, 1, 2, 3], qa)
        _, want_mask_b, want_b = b.orc.step(budget_b, [0, 1, 2], qb)
        assert mask_a == want_mask_a and mask_b == want_mask_b
        a.sync()
        b.sync()
        la = [i for i, m in enumerate(mask_a) if m]
        lb = [i for i, m in enumerate(mask_b) if m]
        check_attn(oa[:, la], want_a[:, la])
        check_attn(ob[:, lb], want_b[:, lb])
    assert mask_a == [1, 1, 1, 1] and mask_b == [1, 1, 1]
    a.assert_pools_equal()
    b.assert_pools_equal()
    a.assert_tables_equal([0, 1, 2, 3])
    b.assert_tables_equal([0, 1, 2])
    a.lib.destroy()                                   # one context goes, the other keeps working
    ob = torch.zeros_like(qb_d)
    rc_b, mask_b, _ = b.lib.step(qb_d, ob, [0, 1, 2], 0)
    _, _, want_b = b.orc.step(0, [0, 1, 2], qb)
    assert rc_b == B.PS_OK
    b.sync()
    check_attn(ob, want_b)


@pytest.mark.parametrize("Hkv,Hq,D,S,kernel", [(8, 32, 128, 16, B.PS_ATTN_MMA), (8, 64, 128, 32, B.PS_ATTN_MMA_ROWS),
                                               (4, 28, 128, 32, B.PS_ATTN_MMA), (1, 8, 128, 48, B.PS_ATTN_MMA),
                                               (4, 8, 64, 16, B.PS_ATTN_SIMT), (8, 32, 128, 16, B.PS_ATTN_SIMT)])
def test_non_finite_leftovers_past_a_context_end_do_not_reach_the_output(Hkv, Hq, D, S, kernel):
    """Slots of a request's last block beyond its context, and every block it does not own, hold NaN and
    infinity patterns in K and V: the output must be what the checker computes from the first ctx tokens."""
    L, nb = 1, 96
    sh, rng, p = make_pair(L, Hkv, Hq, D, S, nb, [15, Hkv, S], max_batch=8, attn_kernel=kernel, kv_split_tokens=3 * S)
    ctxs = [1, S - 1, S + 1, 5 * S + 7, 9 * S - 1, 2 * S]
    for r, c in enumerate(ctxs):
        assert p.both("kv_alloc", r, c) == B.PS_OK
    poison = np.array([0x7FC0, 0x7F80, 0xFF80, 0xFFC1], np.uint16)        # NaN, +inf, -inf, another NaN
    owned = set()
    for r, c in enumerate(ctxs):
        table = p.orc.block_table(r)[0]
        owned.update(table)
        used = c - (len(table) - 1) * S                                     # tokens in the last block
        if used < S:
            fill = poison[rng.integers(0, 4, size=(S - used, Hkv, D))]
            for pool_d, pool_o in ((p.Kd, p.orc.K), (p.Vd, p.orc.V)):
                pool_o[0, table[-1], used:] = fill
                pool_d[0, table[-1], used:] = bits_to_dev(fill)
    foreign = [b for b in range(nb) if b not in owned]
    fill = poison[rng.integers(0, 4, size=(len(foreign), S, Hkv, D))]
    for pool_d, pool_o in ((p.Kd, p.orc.K), (p.Vd, p.orc.V)):
        pool_o[0, foreign] = fill
        pool_d[0, foreign] = bits_to_dev(fill)
    reqs = list(range(len(ctxs)))
    q = wl.randn_bf16_bits(rng, (L, len(reqs), Hq, D))
    qd = bits_to_dev(q)
    out = torch.zeros_like(qd)
    lse = torch.zeros((len(reqs), Hq), dtype=torch.float32, device="cuda")
    assert p.lib.decode_attn(0, qd[0], out[0], reqs, lse) == B.PS_OK, p.lib.last_error()
    assert p.lib.sync() == B.PS_OK, p.lib.last_error()
    want, wlse = p.orc.decode_attn(0, q[0], reqs)
    assert np.isfinite(want).all()
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()
    check_attn(out[0], want)
    assert np.max(np.abs(lse.double().cpu().numpy() - wlse)) < 1e-3


@pytest.mark.parametrize("Hkv,Hq,D,S,kernel,split", [(8, 32, 128, 16, B.PS_ATTN_MMA, 0), (8, 64, 128, 32, B.PS_ATTN_MMA_ROWS, 0),
                                                     (2, 16, 128, 16, B.PS_ATTN_MMA, 0), (4, 8, 64, 16, B.PS_ATTN_SIMT, 48),
                                                     (8, 32, 128, 16, B.PS_ATTN_SIMT, 64)])
def test_peaked_and_flat_softmax_with_large_logits(Hkv, Hq, D, S, kernel, split):
    """Logits of magnitude in the hundreds.  Request 0: q and K eight times the usual scale, so each head's
    weights collapse onto a few tokens and the running maximum jumps by hundreds between tiles and between
    the parts of a split row.  Request 1: every key equals -6 q of its head's first query, so that query's
    logits are one large negative constant and its output is the plain mean of V."""
    L, nb = 1, 128
    sh, rng, p = make_pair(L, Hkv, Hq, D, S, nb, [16, Hkv, D], max_batch=4, attn_kernel=kernel, kv_split_tokens=split)
    G = Hq // Hkv
    n0, n1 = 37 * S + 5, 21 * S - 2
    assert p.both("kv_alloc", 0, n0) == B.PS_OK
    assert p.both("kv_alloc", 1, n1) == B.PS_OK
    from oracle.ps_oracle import bf16_bits_to_f64
    q = wl.randn_bf16_bits(rng, (L, 2, Hq, D))
    q[0, 0] = wl.f32_to_bf16_bits((8.0 * bf16_bits_to_f64(q[0, 0])).astype(np.float32))
    t0 = p.orc.block_table(0)[0]
    big = wl.f32_to_bf16_bits((8.0 * rng.standard_normal((len(t0), S, Hkv, D))).astype(np.float32))
    p.orc.K[0, t0] = big
    p.Kd[0, t0] = bits_to_dev(big)
    t1 = p.orc.block_table(1)[0]
    qf = bf16_bits_to_f64(q[0, 1])
    for h in range(Hkv):
        kb = wl.f32_to_bf16_bits((-6.0 * qf[h * G]).astype(np.float32))
        p.orc.K[0, t1, :, h] = kb
        p.Kd[0, t1, :, h] = bits_to_dev(kb)
    qd = bits_to_dev(q)
    out = torch.zeros_like(qd)
    lse = torch.zeros((2, Hq), dtype=torch.float32, device="cuda")
    assert p.lib.decode_attn(0, qd[0], out[0], [0, 1], lse) == B.PS_OK, p.lib.last_error()
    assert p.lib.sync() == B.PS_OK
    want, wlse = p.orc.decode_attn(0, q[0], [0, 1])
    check_attn(out[0], want, rel_l2=2e-2)
    got_lse = lse.double().cpu().numpy()
    assert np.max(np.abs(got_lse - wlse) / np.maximum(1.0, np.abs(wlse))) < 2e-3
    assert np.abs(wlse[0]).max() > 100 and wlse[1].min() < -30          # the logits really are large
    Vf = bf16_bits_to_f64(p.orc.V[0])
    for h in range(Hkv):                                                 # flat rows: the mean of the value rows
        rows = np.concatenate([Vf[b, :, h] for b in t1])[:n1]
        assert np.max(np.abs(want[1, h * G] - rows.mean(0))) < 1e-9


def test_destroy_with_an_offload_and_a_reload_in_flight():
    """ps_destroy right behind ps_swap_out / a budgeted step, without a sync in between: it waits for the
    transfers itself, the pools stay intact, and a new context over the same pools works at once."""
    L, Hkv, Hq, D, S, nb = 8, 8, 32, 128, 16, 1200
    sh = wl.KVShape(L, Hkv, Hq, D, S, nb)
    g = torch.Generator(device="cuda"); g.manual_seed(17)
    K = torch.empty((L, nb, S, Hkv, D), dtype=torch.bfloat16, device="cuda").normal_(generator=g)
    V = torch.empty_like(K).normal_(generator=g)
    K0, V0 = K.clone(), V.clone()

    def ctx():
        return B.KVSwap(num_layers=L, num_kv_heads=Hkv, num_q_heads=Hq, head_dim=D, block_size=S, num_gpu_blocks=nb,
                        max_blocks_per_req=1024, max_batch=4, host_pool_bytes=(1024 + 64) * sh.block_bytes,
                        k_pools=[K[l] for l in range(L)], v_pools=[V[l] for l in range(L)])

    lib = ctx()
    assert lib.kv_alloc(1, 1000 * S) == B.PS_OK            # 1000 blocks x 512 KiB = 500 MiB of KV
    assert lib.kv_alloc(2, 100 * S) == B.PS_OK
    assert lib.swap_out(1) == B.PS_OK
    lib.destroy()                                           # offload in flight
    lib = ctx()
    assert lib.kv_alloc(1, 1000 * S) == B.PS_OK
    old = torch.tensor(lib.block_table(1)[0], device="cuda", dtype=torch.long)
    assert lib.swap_out(1) == B.PS_OK
    assert lib.sync() == B.PS_OK
    assert torch.equal(K, K0) and torch.equal(V, V0)        # offloading reads the pools only
    assert lib.swap_in_begin(1) == B.PS_OK
    new = torch.tensor(lib.block_table(1)[0], device="cuda", dtype=torch.long)
    K[:, new] = 0                                           # the fresh blocks hold nothing yet
    V[:, new] = 0
    rc, _, st = lib.step(None, None, [], 600 * sh.block_bytes)
    assert rc == B.PS_OK and st["blocks_copied"] == 600
    lib.destroy()                                           # reload in flight: destroy waits for it
    torch.cuda.synchronize()
    assert torch.equal(K[:, new[:600]], K0[:, old[:600]]) and torch.equal(V[:, new[:600]], V0[:, old[:600]])
    assert not K[:, new[600:]].any() and not V[:, new[600:]].any()       # nothing written beyond the budget
    rest = torch.ones(nb, dtype=torch.bool, device="cuda")
    rest[new] = False
    assert torch.equal(K[:, rest], K0[:, rest]) and torch.equal(V[:, rest], V0[:, rest])
    lib = ctx()
    assert lib.kv_alloc(5, 300 * S + 3) == B.PS_OK
    q = torch.randn((Hq, D), generator=g, device="cuda").to(torch.bfloat16).unsqueeze(0)
    out = torch.zeros_like(q)
    assert lib.decode_attn(0, q, out, [5]) == B.PS_OK
    assert lib.sync() == B.PS_OK
    ids = torch.tensor(lib.block_table(5)[0], device="cuda", dtype=torch.long)
    kk = K[0][ids].reshape(-1, Hkv, D)[: 300 * S + 3].float()
    vv = V[0][ids].reshape(-1, Hkv, D)[: 300 * S + 3].float()
    G = Hq // Hkv
    sc = torch.einsum("hd,thd->ht", q[0].float(), kk.repeat_interleave(G, dim=1)) / D ** 0.5
    ref = torch.einsum("ht,thd->hd", torch.softmax(sc, dim=-1), vv.repeat_interleave(G, dim=1))
    assert (out[0].float() - ref).abs().max() < 2e-2
    lib.destroy()
