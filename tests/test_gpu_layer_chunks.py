"""GPU parity of the reload's layer chunks, of the step with host buffers, of the swap kernels alone over
several layers, and of the recovery after a kernel-side wait that ran out.

A layer chunk (Appendix B: one completion event per layer chunk) groups consecutive layers into one strided
host copy, one scatter launch and one event when a single layer's share of the step's copy budget is small.
Whatever the grouping, pools, tables and attention must equal the CPU checker's, which knows nothing of
chunks: it restores block by block, layer by layer.
"""
import numpy as np
import pytest
import torch

from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_util import Pair, bits_to_dev, check_attn, dev_to_bits


def build_pair(L, nb, seed, *, Hkv=4, Hq=8, D=64, S=16, **kw):
    sh = wl.KVShape(L, Hkv, Hq, D, S, nb)
    rng = np.random.default_rng(seed)
    K = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    V = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    return sh, rng, Pair(sh, rng.permutation(nb), K, V, **kw)


@pytest.mark.parametrize("chunk_bytes,staging", [(-1, 0), (0, 0), (40 * 1024, 0), (100 * 1024, 0), (1 << 30, 0),
                                                 (0, 256 * 1024), (100 * 1024, 128 * 1024)])
def test_budgeted_reload_in_layer_chunks_matches_the_checker(chunk_bytes, staging):
    """Six layers of 16 KiB per block; budgets of 1 to 5 blocks per step; images in one or several segments
    (proactive offloading), so a chunk's strided copies meet different layer strides."""
    L = 6
    sh, rng, p = build_pair(L, 160, 41, max_batch=8, layer_chunk_bytes=chunk_bytes, staging_bytes=staging)
    tokens = [200, 37, 333, 16, 129, 250]
    reqs = list(range(len(tokens)))
    grown = 0
    while grown < max(tokens):                           # interleaved growth: fragmented tables
        grown += sh.block_size
        for r, n in enumerate(tokens):
            if grown - sh.block_size < n:
                assert p.both("kv_alloc", r, min(n, grown)) == B.PS_OK
    assert p.both("offload_progress", 0, 3) == (B.PS_OK, 12)       # request 0: segments [0,12) and the tail
    assert p.both("offload_progress", 2, 5) == (B.PS_OK, 20)
    victims = [0, 2, 3, 4]
    for r in victims:
        assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    free_ids = sorted(p.orc.free)
    p.Kd[:, free_ids] = 0; p.Vd[:, free_ids] = 0
    p.orc.K[:, free_ids] = 0; p.orc.V[:, free_ids] = 0
    for r in victims:
        assert p.both("swap_in_begin", r) == B.PS_OK
    q = wl.randn_bf16_bits(rng, (L, len(reqs), sh.num_q_heads, sh.head_dim))
    qd = bits_to_dev(q)
    steps = 0
    while any(p.orc.missing_blocks(r) for r in victims):
        budget = int(rng.integers(1, 6)) * sh.block_bytes
        out = torch.full_like(qd, 3.0)
        rc, mask, st = p.lib.step(qd, out, reqs, budget)
        assert rc == B.PS_OK, p.lib.last_error()
        plan, omask, want = p.orc.step(budget, reqs, q)
        assert mask == omask and st["blocks_copied"] == sum(hi - lo for _, lo, hi in plan)
        torch.cuda.synchronize()
        live = [i for i, m in enumerate(mask) if m]
        check_attn(out[:, live], want[:, live])
        if steps % 3 == 0:
            p.sync()
            p.assert_pools_equal()
        steps += 1
        assert steps < 200
    p.sync()
    p.assert_pools_equal()
    p.assert_tables_equal(reqs)
    # copy-only steps (no attention) take the same chunks
    for r in victims:
        assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    for r in victims:
        assert p.both("swap_in_begin", r) == B.PS_OK
    while any(p.orc.missing_blocks(r) for r in victims):
        rc, _, st = p.lib.step(None, None, [], 7 * sh.block_bytes)
        assert rc == B.PS_OK, p.lib.last_error()
        p.orc.step(7 * sh.block_bytes)
    p.sync()
    p.assert_pools_equal()
    p.orc.check_invariants()


def test_layer_chunks_at_the_8b_shape_with_the_tensor_core_kernel():
    """8 KV heads, head_dim 128 (64 KiB per block and layer), 8 layers: 2 MiB chunks group 1 to 8 layers
    depending on the step's budget; the requests completed by a step run on the reload lane behind the chunk
    events."""
    L = 8
    sh, rng, p = build_pair(L, 400, 43, Hkv=8, Hq=32, D=128, max_batch=8, max_blocks_per_req=64)
    tokens = [700, 512, 90, 333, 1000, 260]
    reqs = list(range(len(tokens)))
    for r, n in enumerate(tokens):
        assert p.both("kv_alloc", r, n) == B.PS_OK
    victims = [1, 3, 4]
    for r in victims:
        assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    for r in victims:
        assert p.both("swap_in_begin", r) == B.PS_OK
    q = wl.randn_bf16_bits(rng, (L, len(reqs), sh.num_q_heads, sh.head_dim))
    qd = bits_to_dev(q)
    gated_seen = 0
    for budget_blocks in (2, 9, 40, 3, 17, 64, 64, 64):
        if not any(p.orc.missing_blocks(r) for r in victims):
            break
        out = torch.zeros_like(qd)
        rc, mask, st = p.lib.step(qd, out, reqs, budget_blocks * sh.block_bytes)
        assert rc == B.PS_OK, p.lib.last_error()
        plan, omask, want = p.orc.step(budget_blocks * sh.block_bytes, reqs, q)
        assert mask == omask
        gated_seen += st["gated"]
        torch.cuda.synchronize()
        live = [i for i, m in enumerate(mask) if m]
        check_attn(out[:, live], want[:, live])
    assert gated_seen == len(victims) and not any(p.orc.missing_blocks(r) for r in victims)
    p.sync()
    p.assert_pools_equal()


def test_step_with_host_buffers_matches_the_checker():
    """ps_step_host: queries and outputs in pinned host memory, the copies made by the library."""
    w = wl.tiny()
    K, V = wl.make_pools_numpy(w)
    p = Pair(w.shape, w.free_order, K, V, max_batch=16)
    for r, n in wl.build_order_round_robin(w):
        assert p.both("kv_alloc", r, n) == B.PS_OK
    reqs = list(range(len(w.ctx_lens)))
    for r in w.victims:
        assert p.both("swap_out", r) == B.PS_OK
    p.sync()
    for r in w.victims:
        assert p.both("swap_in_begin", r) == B.PS_OK
    q = wl.make_queries_numpy(w, len(reqs))
    q_host = torch.from_numpy(q.view(np.int16)).view(torch.bfloat16).pin_memory()
    out_host = torch.full_like(q_host, 9.0).pin_memory()
    budget = 4 * w.shape.block_bytes
    steps = 0
    while True:
        rc, mask, st = p.lib.step_host(q_host, out_host, reqs, budget)
        assert rc == B.PS_OK, p.lib.last_error()
        plan, omask, want = p.orc.step(budget, reqs, q)
        assert mask == omask
        torch.cuda.synchronize()
        live = [i for i, m in enumerate(mask) if m]
        dead = [i for i, m in enumerate(mask) if not m]
        check_attn(out_host[:, live].cuda(), want[:, live])
        assert (out_host[:, dead].float() == 0).all()          # rows that do not decode come back as zeros
        steps += 1
        if all(mask):
            break
        assert steps < 50
    assert steps > 2
    p.sync()
    p.assert_pools_equal()
    assert p.lib.step_host(q_host, out_host, [], budget)[0] == B.PS_ERR_INVALID


def test_copy_blocks_over_a_layer_chunk_is_bit_exact():
    """The swap path's gather and scatter kernels alone, three layers per launch."""
    sh, rng, p = build_pair(4, 96, 47, Hkv=8, Hq=8, D=128, max_batch=1)
    K, V = p.orc.K.copy(), p.orc.V.copy()
    ids = [int(v) for v in rng.permutation(96)[:29]]
    stage = torch.zeros((3, 29, 2, 16, 8, 128), dtype=torch.bfloat16, device="cuda")
    assert p.lib.copy_blocks(1, ids, stage, 0, n_layers=3) == B.PS_OK
    p.lib.sync()
    got = dev_to_bits(stage)
    for i, l in enumerate((1, 2, 3)):
        assert np.array_equal(got[i, :, 0], K[l][ids]) and np.array_equal(got[i, :, 1], V[l][ids])
    dst = [int(v) for v in rng.permutation(96)[:29]]
    assert p.lib.copy_blocks(0, dst, stage, 1, n_layers=3) == B.PS_OK
    p.lib.sync()
    K2, V2 = K.copy(), V.copy()
    for i, l in enumerate((0, 1, 2)):
        K2[l][dst] = K[i + 1][ids]
        V2[l][dst] = V[i + 1][ids]
    assert np.array_equal(dev_to_bits(p.Kd), K2) and np.array_equal(dev_to_bits(p.Vd), V2)
    assert p.lib.copy_blocks(2, ids, stage, 0, n_layers=3) == B.PS_ERR_INVALID      # layers 2..4 do not exist


def test_attention_recovers_after_a_kernel_side_timeout_report():
    """Status 3 (a bounded wait inside the attention kernel ran out) is written by a test hook that also
    leaves the kernel's chunk and arrival counters dirty, as CTAs that gave up would.  The next poll reports
    PS_ERR_TIMEOUT and resets the counters: split rows are combined correctly again afterwards.  No kernel is
    made to wait or fail."""
    sh, rng, p = build_pair(2, 420, 53, Hkv=8, Hq=32, D=128, max_batch=8, max_blocks_per_req=64,
                            attn_kernel=B.PS_ATTN_MMA)
    tokens = [700, 650, 720, 512, 690, 705]               # rows longer than a CTA's share: several parts each
    reqs = list(range(len(tokens)))
    for r, n in enumerate(tokens):
        assert p.both("kv_alloc", r, n) == B.PS_OK
    q = wl.randn_bf16_bits(rng, (2, len(reqs), sh.num_q_heads, sh.head_dim))
    qd = bits_to_dev(q)
    out = torch.zeros_like(qd)
    want = [p.orc.decode_attn(l, q[l], reqs)[0] for l in range(2)]
    for l in range(2):
        assert p.lib.decode_attn(l, qd[l], out[l], reqs) == B.PS_OK
    torch.cuda.synchronize()
    for l in range(2):
        check_attn(out[l], want[l])
    assert p.lib.inject_status(3) == B.PS_OK
    with pytest.raises(B.PsError) as e:
        p.lib.poll()
    assert e.value.code == B.PS_ERR_TIMEOUT
    out.zero_()
    rc, mask, st = p.lib.step(qd, out, reqs, 0)
    assert rc == B.PS_OK and all(mask), p.lib.last_error()
    for l in range(2):
        assert p.lib.decode_attn(l, qd[l], out[l], reqs) == B.PS_OK
    torch.cuda.synchronize()
    for l in range(2):
        check_attn(out[l], want[l])
    assert p.lib.sync() == B.PS_OK


@pytest.mark.parametrize("flags", [0, B.PS_FLAG_ATTN_PLAIN_LAUNCH])
def test_attention_with_early_set_up_matches_after_any_predecessor(flags):
    """One-layer-per-call launches are by default programmatically dependent on the kernel before them and wait
    for it before reading any input (PS_FLAG_ATTN_PLAIN_LAUNCH: ordinary launches).  Back to back (the predecessor is the same kernel, which lets
    dependents start early), after another library's kernel that produces the queries, and after a table
    change (the predecessor is the metadata upload): results equal the checker's every time."""
    sh, rng, p = build_pair(4, 420, 59, Hkv=8, Hq=32, D=128, max_batch=8, max_blocks_per_req=64,
                            attn_kernel=B.PS_ATTN_MMA, flags=flags)
    tokens = [700, 33, 720, 512, 1, 705]
    reqs = list(range(len(tokens)))
    for r, n in enumerate(tokens):
        assert p.both("kv_alloc", r, n) == B.PS_OK
    q = wl.randn_bf16_bits(rng, (4, len(reqs), sh.num_q_heads, sh.head_dim))
    qd = bits_to_dev(q)
    out = torch.zeros_like(qd)
    for rounds in range(3):
        for l in range(4):                                   # back to back: every launch follows the same kernel
            assert p.lib.decode_attn(l, qd[l], out[l], reqs) == B.PS_OK
    torch.cuda.synchronize()
    for l in range(4):
        check_attn(out[l], p.orc.decode_attn(l, q[l], reqs)[0])
    # the queries are produced on the stream right before the launch that reads them
    q2 = wl.randn_bf16_bits(rng, (4, len(reqs), sh.num_q_heads, sh.head_dim))
    src = bits_to_dev(q2)
    big = torch.empty(64 << 20, dtype=torch.uint8, device="cuda")
    for l in range(4):
        big.fill_(l)                                         # some work in front, so the copy below is not instant
        qd[l].copy_(src[l])
        assert p.lib.decode_attn(l, qd[l], out[l], reqs) == B.PS_OK
    torch.cuda.synchronize()
    for l in range(4):
        check_attn(out[l], p.orc.decode_attn(l, q2[l], reqs)[0])
    # a table change: the batch metadata is uploaded by a kernel right before the attention launch
    assert p.both("kv_alloc", 1, 400) == B.PS_OK
    assert p.lib.decode_attn(2, qd[2], out[2], reqs) == B.PS_OK
    torch.cuda.synchronize()
    check_attn(out[2], p.orc.decode_attn(2, q2[2], reqs)[0])


def test_small_device_to_host_copies_do_not_wait_for_a_whole_offload():
    """The copy engine serves device-to-host copies in submission order, whatever their stream.  The library's
    offload worker therefore hands it two staging slots at a time: a small copy the caller makes right after
    ps_swap_out (a step's result, sampled tokens) completes after those, not after the whole image.  The image
    itself is byte-exact as ever."""
    import time
    L, nb = 16, 2200                                       # 16 layers x 64 KiB: 1 MiB per block
    sh = wl.KVShape(L, 8, 8, 128, 16, nb)
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    K = torch.empty((L, nb, 16, 8, 128), dtype=torch.bfloat16, device="cuda").normal_(generator=g)
    V = torch.empty_like(K).normal_(generator=g)
    lib = B.KVSwap(num_layers=L, num_kv_heads=8, num_q_heads=8, head_dim=128, block_size=16, num_gpu_blocks=nb,
                   max_blocks_per_req=2100, max_batch=1, host_pool_bytes=(2048 + 64) << 20,
                   k_pools=[K[l] for l in range(L)], v_pools=[V[l] for l in range(L)])
    assert lib.kv_alloc(7, 2048 * 16) == B.PS_OK           # 2048 blocks = 2 GiB of KV: about 36 ms of host link
    table = torch.tensor(lib.block_table(7)[0], device="cuda", dtype=torch.long)
    small = torch.arange(4096, device="cuda", dtype=torch.int32)
    host = torch.empty(4096, dtype=torch.int32).pin_memory()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    assert lib.swap_out(7) == B.PS_OK
    host.copy_(small, non_blocking=True)
    torch.cuda.current_stream().synchronize()
    t_small = time.perf_counter() - t0
    assert lib.sync() == B.PS_OK
    t_all = time.perf_counter() - t0
    assert torch.equal(host, small.cpu())
    assert t_all > 0.025, t_all                            # the offload really took its tens of milliseconds
    assert t_small < 0.5 * t_all, (t_small, t_all)         # and the small copy did not wait for it
    # the image: layer-major, block by block through the table
    ptr, nbytes = lib.host_image(7)
    import ctypes as C
    img = np.ctypeslib.as_array((C.c_uint16 * (nbytes // 2)).from_address(ptr)).reshape(L, 2048, 2, -1)
    for l in (0, 7, L - 1):
        assert np.array_equal(img[l][:, 0], dev_to_bits(K[l][table]).reshape(2048, -1))
        assert np.array_equal(img[l][:, 1], dev_to_bits(V[l][table]).reshape(2048, -1))
    lib.destroy()
