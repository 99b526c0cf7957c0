"""GPU parity: the CUDA path through the C ABI against the CPU checker on identical seeded inputs.

Byte, id and index results must be identical; attention must be within max-abs 2e-2 of the fp64
checker (bf16 inputs, fp32 accumulation, bf16 output) and within 1e-2 relative L2 per (request, head).
"""
import numpy as np
import pytest
import torch

from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_util import Pair, bits_to_dev, check_attn, dev_to_bits


def tiny_pair(**kw):
    w = wl.tiny()
    K, V = wl.make_pools_numpy(w)
    p = Pair(w.shape, w.free_order, K, V, max_batch=16, **kw)
    for r, n in wl.build_order_round_robin(w):
        assert p.both("kv_alloc", r, n) == B.PS_OK
    return w, p


@pytest.mark.parametrize("staging", [0, 64 * 1024])
def test_tiny_swap_out_image_and_round_trip(staging):
    """Config 1: swap 4 of 8 out, compare host images and tables, reload, compare every pool byte, decode."""
    w, p = tiny_pair(staging_bytes=staging)      # 64 KiB staging = 16 KiB slots: many segments per request
    reqs = list(range(len(w.ctx_lens)))
    for r in w.victims:
        assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    p.assert_tables_equal(reqs)
    for r in w.victims:
        assert np.array_equal(p.host_image_bits(r), p.orc.reqs[r].image.reshape(-1)), r
    # dirty the reclaimed blocks on both sides so that a missing write cannot hide
    free_ids = sorted(p.orc.free)
    p.Kd[:, free_ids] = 0
    p.Vd[:, free_ids] = 0
    p.orc.K[:, free_ids] = 0
    p.orc.V[:, free_ids] = 0
    for r in reversed(w.victims):
        assert p.both("swap_in_begin", r) == B.PS_OK
    p.assert_tables_equal(reqs)
    q = wl.make_queries_numpy(w, len(reqs))
    qd = bits_to_dev(q)
    out = torch.zeros_like(qd)
    rc, mask, st = p.lib.step(qd, out, reqs, -1)
    assert rc == B.PS_OK, p.lib.last_error()
    plan, omask, want = p.orc.step(-1, reqs, q)
    assert mask == omask == [1] * len(reqs)
    assert st["reloads_completed"] == len(w.victims) and st["gated"] == len(w.victims)
    assert st["blocks_copied"] == sum(hi - lo for _, lo, hi in plan)
    p.sync()
    p.assert_pools_equal()
    p.assert_tables_equal(reqs)
    check_attn(out, want)
    p.orc.check_invariants()
    # a second step: nothing to reload, nobody gated, same answer
    out2 = torch.zeros_like(qd)
    rc, mask, st = p.lib.step(qd, out2, reqs, -1)
    assert rc == B.PS_OK and st["gated"] == 0 and st["blocks_copied"] == 0
    p.sync()
    assert torch.equal(out, out2)


def test_budgeted_partial_reload_matches_every_step():
    w, p = tiny_pair()
    reqs = list(range(len(w.ctx_lens)))
    for r in w.victims:
        assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    free_ids = sorted(p.orc.free)
    p.Kd[:, free_ids] = 0; p.Vd[:, free_ids] = 0
    p.orc.K[:, free_ids] = 0; p.orc.V[:, free_ids] = 0
    for r in w.victims:
        assert p.both("swap_in_begin", r) == B.PS_OK
    q = wl.make_queries_numpy(w, len(reqs))
    qd = bits_to_dev(q)
    budget = 5 * w.shape.block_bytes + 100
    steps = 0
    while any(p.orc.missing_blocks(r) for r in w.victims):
        out = torch.full_like(qd, 7.0)
        rc, mask, st = p.lib.step(qd, out, reqs, budget)
        assert rc == B.PS_OK, p.lib.last_error()
        plan, omask, want = p.orc.step(budget, reqs, q)
        assert mask == omask
        assert st["blocks_copied"] == sum(hi - lo for _, lo, hi in plan) <= 5
        p.sync()
        p.assert_pools_equal()
        for r in w.victims:
            assert p.lib.missing_blocks(r) == p.orc.missing_blocks(r)
        live = [i for i, m in enumerate(mask) if m]
        dead = [i for i, m in enumerate(mask) if not m]
        check_attn(out[:, live], want[:, live])
        assert (out[:, dead].float() == 7.0).all()          # rows that do not decode are left untouched
        steps += 1
        assert steps < 100
    assert steps > 3
    p.assert_tables_equal(reqs)


SHAPES = [
    # (Hkv, Hq, D, S, kernel, split)
    (4, 8, 64, 16, B.PS_ATTN_SIMT, 0),
    (2, 2, 64, 8, B.PS_ATTN_SIMT, 64),
    (2, 8, 64, 16, B.PS_ATTN_SIMT, 32),
    (1, 8, 64, 16, B.PS_ATTN_SIMT, 0),
    (8, 8, 128, 16, B.PS_ATTN_SIMT, 64),
    (2, 4, 128, 32, B.PS_ATTN_SIMT, 0),
    (8, 32, 128, 16, B.PS_ATTN_SIMT, 128),
    (8, 32, 128, 16, B.PS_ATTN_SIMT, 0),
    (2, 16, 128, 16, B.PS_ATTN_SIMT, 48),
    (2, 4, 128, 24, B.PS_ATTN_SIMT, 100),      # block size that is not a power of two, ragged split
    # tensor-core kernel (head_dim 128, 8 KV heads): every group size, block sizes 16 / 32 / 48
    (8, 8, 128, 16, B.PS_ATTN_MMA, 0),
    (8, 16, 128, 16, B.PS_ATTN_MMA, 0),
    (8, 32, 128, 16, B.PS_ATTN_MMA, 0),
    (8, 64, 128, 16, B.PS_ATTN_MMA, 0),
    (8, 64, 128, 32, B.PS_ATTN_MMA, 0),
    (8, 32, 128, 48, B.PS_ATTN_MMA, 0),
    # group sizes that are not powers of two (28 query heads over 4 KV heads is Qwen2-7B's shape)
    (4, 28, 128, 16, B.PS_ATTN_SIMT, 0),
    (2, 10, 64, 16, B.PS_ATTN_SIMT, 40),
    (8, 24, 128, 16, B.PS_ATTN_MMA, 0),
    (8, 56, 128, 32, B.PS_ATTN_MMA, 0),
    (8, 40, 128, 16, B.PS_ATTN_MMA_ROWS, 0),
    # fewer than 8 KV heads: a stage holds 8 / Hkv sub-tiles, the warps of a head combine their states
    (4, 16, 128, 16, B.PS_ATTN_MMA, 0),
    (4, 28, 128, 32, B.PS_ATTN_MMA, 0),
    (2, 16, 128, 16, B.PS_ATTN_MMA, 0),
    (2, 2, 128, 48, B.PS_ATTN_MMA, 0),
    (1, 8, 128, 16, B.PS_ATTN_MMA, 0),
    (1, 5, 128, 32, B.PS_ATTN_MMA, 0),
    # the same kernel fed by one bulk copy per token row instead of tensor-map boxes
    (8, 32, 128, 16, B.PS_ATTN_MMA_ROWS, 0),
    (8, 64, 128, 32, B.PS_ATTN_MMA_ROWS, 0),
    (8, 8, 128, 48, B.PS_ATTN_MMA_ROWS, 0),
]


@pytest.mark.parametrize("Hkv,Hq,D,S,kernel,split", SHAPES)
def test_decode_attn_shapes_ragged_contexts(Hkv, Hq, D, S, kernel, split):
    L, nb = 2, 160
    sh = wl.KVShape(L, Hkv, Hq, D, S, nb)
    rng = np.random.default_rng([Hkv, Hq, D, S, split, kernel])
    K = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    V = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    p = Pair(sh, rng.permutation(nb), K, V, max_batch=16, attn_kernel=kernel, kv_split_tokens=split)
    ctxs = [0, 1, S - 1, S, S + 1, 3 * S, 3 * S + 1, 7 * S + 5, 40 * S - 3, 2, 19 * S]
    grown = [0] * len(ctxs)
    assert p.both("kv_alloc", 0, 0) == B.PS_OK
    while any(g < c for g, c in zip(grown, ctxs)):
        for r, c in enumerate(ctxs):
            if grown[r] < c:
                grown[r] = min(c, grown[r] + S)
                assert p.both("kv_alloc", r, grown[r]) == B.PS_OK
    reqs = list(range(len(ctxs)))
    q = wl.randn_bf16_bits(rng, (L, len(ctxs), Hq, D))
    qd = bits_to_dev(q)
    for layer in range(L):
        out = torch.full((len(ctxs), Hq, D), 3.0, dtype=torch.bfloat16, device="cuda")
        lse = torch.zeros((len(ctxs), Hq), dtype=torch.float32, device="cuda")
        assert p.lib.decode_attn(layer, qd[layer], out, reqs, lse) == B.PS_OK, p.lib.last_error()
        assert p.lib.sync() == B.PS_OK, p.lib.last_error()
        want, wlse = p.orc.decode_attn(layer, q[layer], reqs)
        check_attn(out, want)
        got_lse = lse.double().cpu().numpy()
        assert np.isneginf(got_lse[0]).all() and np.isneginf(wlse[0]).all()
        assert np.max(np.abs(got_lse[1:] - wlse[1:])) < 1e-3
    # a permuted / repeated batch addresses q and out rows by position
    order = [5, 5, 1, 10, 0, 8]
    out = torch.zeros((len(order), Hq, D), dtype=torch.bfloat16, device="cuda")
    qsub = qd[0][order].contiguous()
    assert p.lib.decode_attn(0, qsub, out, order) == B.PS_OK
    p.lib.sync()
    want, _ = p.orc.decode_attn(0, q[0][order], order)
    check_attn(out, want)


@pytest.mark.parametrize("Hkv,Hq,D,S", [(4, 8, 64, 16), (8, 32, 128, 16), (8, 64, 128, 32), (4, 16, 128, 16),
                                        (1, 4, 128, 16)])
def test_decode_attn_index_coded_values_and_equal_keys(Hkv, Hq, D, S):
    """Outputs of magnitude ~1..100: a read from a wrong block, slot or head cannot hide under 2e-2."""
    L, nb = 1, 64
    G = Hq // Hkv
    sh = wl.KVShape(L, Hkv, Hq, D, S, nb)
    rng = np.random.default_rng([7, Hkv, D])

    def code(b, s, h):
        # integers of magnitude <= 256 are exact in bf16; the sign carries the head parity
        return (1 + (b % 16) * 16 + s % 16) * (1 if h % 2 == 0 else -1)

    K = np.zeros((L, nb, S, Hkv, D), np.uint16)
    V = np.zeros_like(K)
    for b in range(nb):
        for s in range(S):
            for h in range(Hkv):
                V[0, b, s, h] = wl.f32_to_bf16_bits(np.full(D, code(b, s, h), np.float32))
    p = Pair(sh, rng.permutation(nb), K, V, max_batch=4, kv_split_tokens=4 * S)
    n_tok = 13 * S + 3
    assert p.both("kv_alloc", 0, n_tok) == B.PS_OK
    assert p.both("kv_alloc", 1, 5 * S) == B.PS_OK
    table = p.orc.block_table(0)[0]
    q = wl.randn_bf16_bits(rng, (1, 2, Hq, D))
    from oracle.ps_oracle import bf16_bits_to_f64
    qf = bf16_bits_to_f64(q[0][0])
    picks = [int(v) for v in rng.integers(0, n_tok, size=Hkv)]
    for h in range(Hkv):                       # each KV head gets one dominant key aligned with its first q head
        t = picks[h]
        kb = wl.f32_to_bf16_bits((48.0 * qf[h * G]).astype(np.float32))
        p.orc.K[0, table[t // S], t % S, h] = kb
        p.Kd[0, table[t // S], t % S, h] = bits_to_dev(kb)
    qd = bits_to_dev(q)
    out = torch.zeros((2, Hq, D), dtype=torch.bfloat16, device="cuda")
    assert p.lib.decode_attn(0, qd[0], out, [0, 1]) == B.PS_OK
    p.lib.sync()
    want, _ = p.orc.decode_attn(0, q[0], [0, 1])
    got = out.double().cpu().numpy()
    for h in range(Hkv):
        t = picks[h]
        coded = code(table[t // S], t % S, h)
        assert np.max(np.abs(want[0, h * G] - coded)) < 1e-6          # the checker itself selects that row
        assert np.max(np.abs(got[0, h * G] - coded)) <= 0.5           # an exactly representable value
    # request 1: all keys zero (equal) -> output is the mean of its value rows
    t1 = p.orc.block_table(1)[0]
    for h in range(Hkv):
        mean = np.mean([code(b, s, h) for b in t1 for s in range(S)])
        assert np.max(np.abs(got[1, h * G:(h + 1) * G] - mean)) <= 1.0   # bf16 rounding at magnitude <= 256
        assert np.max(np.abs(want[1, h * G] - mean)) < 1e-9


def test_copy_blocks_gather_scatter_bit_exact():
    sh = wl.KVShape(3, 8, 8, 128, 16, 96)
    rng = np.random.default_rng(5)
    K = wl.randn_bf16_bits(rng, (3, 96, 16, 8, 128))
    V = wl.randn_bf16_bits(rng, (3, 96, 16, 8, 128))
    p = Pair(sh, None, K, V, max_batch=1)
    ids = [int(v) for v in rng.permutation(96)[:37]]
    stage = torch.zeros((37, 2, 16, 8, 128), dtype=torch.bfloat16, device="cuda")
    assert p.lib.copy_blocks(1, ids, stage, 0) == B.PS_OK
    p.lib.sync()
    got = dev_to_bits(stage)
    assert np.array_equal(got[:, 0], K[1][ids]) and np.array_equal(got[:, 1], V[1][ids])
    # scatter the same staging into other blocks of layer 2
    dst = [int(v) for v in rng.permutation(96)[:37]]
    assert p.lib.copy_blocks(2, dst, stage, 1) == B.PS_OK
    p.lib.sync()
    K2, V2 = K.copy(), V.copy()
    K2[2][dst] = K[1][ids]
    V2[2][dst] = V[1][ids]
    assert np.array_equal(dev_to_bits(p.Kd), K2) and np.array_equal(dev_to_bits(p.Vd), V2)
    assert p.lib.copy_blocks(0, [96], stage, 0) == B.PS_ERR_INVALID
    assert p.lib.copy_blocks(0, [], stage, 0) == B.PS_OK


def test_manual_layer_loop_with_gated_attention():
    """A caller driving the layer loop itself: swap_in_layer per layer, then decode_attn of that layer."""
    w, p = tiny_pair()
    r = w.victims[0]
    assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    free_ids = sorted(p.orc.free)
    p.Kd[:, free_ids] = 0; p.Vd[:, free_ids] = 0
    p.orc.K[:, free_ids] = 0; p.orc.V[:, free_ids] = 0
    assert p.both("swap_in_begin", r) == B.PS_OK
    n = len(p.orc.block_table(r)[0])
    q = wl.make_queries_numpy(w, 2)
    qd = bits_to_dev(q)
    other = [x for x in range(len(w.ctx_lens)) if x not in w.victims][0]
    mid = max(1, n // 2)
    for layer in range(w.shape.num_layers):
        assert p.both("swap_in_layer", r, layer, 0, mid) == B.PS_OK
    assert p.lib.decode_attn(0, qd[0], torch.zeros_like(qd[0]), [r, other]) == B.PS_ERR_STATE
    for layer in range(w.shape.num_layers):
        assert p.both("swap_in_layer", r, layer, mid, n) == B.PS_OK
    assert p.lib.block_table(r)[1] == B.PS_REQ_RESIDENT
    for layer in range(w.shape.num_layers):
        out = torch.zeros_like(qd[layer])
        assert p.lib.decode_attn(layer, qd[layer], out, [r, other]) == B.PS_OK, p.lib.last_error()
        p.lib.sync()
        want, _ = p.orc.decode_attn(layer, q[layer], [r, other])
        check_attn(out, want)
    p.assert_pools_equal()
    # swap the same request out again right away (its reload events are honoured) and compare the image
    assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    assert np.array_equal(p.host_image_bits(r), p.orc.reqs[r].image.reshape(-1))


def test_swap_out_is_ordered_after_compute_stream_writes():
    """KV written on the compute stream just before swap_out must be what lands in the host image."""
    w, p = tiny_pair()
    r = w.victims[1]
    table = p.orc.block_table(r)[0]
    torch.cuda._sleep(200_000_000)                      # keep the compute stream busy for a while
    newk = wl.randn_bf16_bits(np.random.default_rng(99), p.orc.K[:, table].shape)
    p.Kd[:, table] = bits_to_dev(newk)                  # enqueued behind the sleep
    p.orc.K[:, table] = newk
    assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    assert np.array_equal(p.host_image_bits(r), p.orc.reqs[r].image.reshape(-1))


def test_errors_on_device_context():
    w, p = tiny_pair()
    r = w.victims[0]
    assert p.both("swap_out", r) == B.PS_OK
    assert p.both("swap_out", r) == B.PS_ERR_STATE
    assert p.both("kv_free", r) == B.PS_ERR_BUSY
    p.sync()
    assert p.both("swap_in_begin", r) == B.PS_OK
    assert p.both("swap_in_begin", r) == B.PS_ERR_STATE
    assert p.both("swap_in_cancel", r) == B.PS_OK
    assert p.both("kv_free", r) == B.PS_OK
    assert p.both("kv_alloc", 1000, 250 * 16) == B.PS_ERR_NOMEM
    p.assert_tables_equal([x for x in range(len(w.ctx_lens)) if x != r])
    q = torch.zeros((1, 8, 64), dtype=torch.bfloat16, device="cuda")
    assert p.lib.decode_attn(5, q, q, [0]) == B.PS_ERR_INVALID
    assert p.lib.decode_attn(0, q, q, [12345]) == B.PS_ERR_INVALID


def test_sync_reload_flag_gives_identical_results():
    w, p = tiny_pair(flags=B.PS_FLAG_SYNC_RELOAD | B.PS_FLAG_PROFILE)
    reqs = list(range(len(w.ctx_lens)))
    for r in w.victims:
        assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    for r in w.victims:
        assert p.both("swap_in_begin", r) == B.PS_OK
    q = wl.make_queries_numpy(w, len(reqs))
    qd = bits_to_dev(q)
    out = torch.zeros_like(qd)
    rc, mask, st = p.lib.step(qd, out, reqs, -1)
    assert rc == B.PS_OK
    _, _, want = p.orc.step(-1, reqs, q)
    p.sync()
    p.assert_pools_equal()
    check_attn(out, want)
    prof = p.lib.get_profile()
    assert prof["attn_launches"] >= w.shape.num_layers and prof["attn_ms"] > 0
    assert prof["gather_bytes"] == prof["d2h_bytes"] == prof["h2d_bytes"] == prof["scatter_bytes"] > 0
    assert p.lib.launch_count() > 0


def test_sync_times_out_while_the_compute_stream_is_busy_and_recovers():
    """Bounded host wait: PS_ERR_TIMEOUT leaves everything in flight; a later wait succeeds."""
    w, p = tiny_pair()
    torch.cuda._sleep(400_000_000)                      # a kernel that ends by itself after ~0.2 s
    assert p.lib.sync(timeout_ms=1) == B.PS_ERR_TIMEOUT
    assert "timed out" in p.lib.last_error()
    assert p.lib.sync(timeout_ms=-1) == B.PS_OK
    r = w.victims[0]
    assert p.both("swap_out", r) == B.PS_OK             # the context is fully usable afterwards
    p.sync()
    assert np.array_equal(p.host_image_bits(r), p.orc.reqs[r].image.reshape(-1))


def test_kernel_skips_a_block_id_outside_the_pool_and_reports_it():
    """A table entry outside [0, num_blocks) is never dereferenced: the kernel records status 2 and goes on;
    rows with valid tables are unaffected."""
    Hkv, Hq, D, S, nb = 2, 4, 64, 16, 32
    rng = np.random.default_rng(31)
    K = wl.randn_bf16_bits(rng, (1, nb, S, Hkv, D))
    V = wl.randn_bf16_bits(rng, (1, nb, S, Hkv, D))
    p = Pair(wl.KVShape(1, Hkv, Hq, D, S, nb), None, K, V, max_batch=2)
    assert p.both("kv_alloc", 0, 3 * S) == B.PS_OK and p.both("kv_alloc", 1, 2 * S) == B.PS_OK
    tables = torch.tensor([p.lib.block_table(0)[0], p.lib.block_table(1)[0] + [0]], dtype=torch.int32, device="cuda")
    bad = tables.clone()
    bad[1, 1] = nb + 5                                   # out of range, in the second request only
    q = wl.randn_bf16_bits(rng, (2, Hq, D))
    qd = bits_to_dev(q)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.zeros_like(qd)
    kw = dict(num_kv_heads=Hkv, num_q_heads=Hq, head_dim=D, block_size=S, num_gpu_blocks=nb, status_word=status)
    rc, text = B.ps_decode_attn_static(p.Kd[0], p.Vd[0], qd, out, bad, [3 * S, 2 * S], **kw)
    assert rc == B.PS_OK, text
    torch.cuda.synchronize()
    assert int(status.item()) == 2
    want, _ = p.orc.decode_attn(0, q, [0, 1])
    check_attn(out[0:1], want[0:1])                      # the request with a valid table is exact
    status.zero_()
    rc, text = B.ps_decode_attn_static(p.Kd[0], p.Vd[0], qd, out, tables, [3 * S, 2 * S], **kw)
    torch.cuda.synchronize()
    assert rc == B.PS_OK and int(status.item()) == 0
    check_attn(out, want)
