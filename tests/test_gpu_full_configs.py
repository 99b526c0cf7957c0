"""GPU parity at the full sizes of the five workloads, in the launch configuration the benchmark times.

Pools of tens of GiB cannot be mirrored on the host, so each test drives three parties (see
gpu_util.FullSizePair): the library, a checker for tables / states / plans over all layers, and a
checker holding the bytes of two sampled layers (first and last) over the full block-id space.  What
the sampled checker cannot see is covered by properties that hold at any size: every swapped request's
logical KV, all layers, is bit-identical after the round trip; no block outside the reloaded tables
changes (per-block sums); attention on sampled rows stays within tolerance of the fp64 checker.
"""
import numpy as np
import pytest
import torch

from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_util import FullSizePair
    from loop_util import PairedBackend
    from paper_2512_12928_b200 import engine_loop as el


def _queries(sh, n, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    q = torch.randn((sh.num_layers, n, sh.num_q_heads, sh.head_dim), generator=g, device="cuda").to(torch.bfloat16)
    return q, torch.zeros_like(q)


def _need_memory(gib):
    import gc
    gc.collect()
    torch.cuda.empty_cache()                      # the previous test's pools sit in torch's cache
    free, _ = torch.cuda.mem_get_info()
    if free < gib * (1 << 30):
        pytest.skip(f"needs {gib} GiB of free device memory")


def test_config2_llama8b_swap_round_trip_full_size():
    """64 residents of 1k-4k tokens, a seeded 16 preempted (about 6 GiB) and reloaded; then one decode step."""
    _need_memory(60)
    w = wl.llama8b_swap()
    sh = w.shape
    victim_blocks = sum(sh.blocks_for(w.ctx_lens[r]) for r in w.victims)
    p = FullSizePair(w, [0, sh.num_layers - 1], max_batch=len(w.ctx_lens), max_blocks_per_req=257,
                     host_pool_bytes=victim_blocks * sh.block_bytes + (256 << 20))
    reqs = list(range(len(w.ctx_lens)))
    for r, n in wl.build_order_round_robin(w):
        assert p.all3("kv_alloc", r, n) == B.PS_OK
    p.assert_tables_equal(reqs)
    saved = {r: p.logical_kv(r) for r in w.victims}
    for r in w.victims:
        assert p.all3("swap_out", r) == B.PS_OK
    p.sync()
    p.assert_tables_equal(reqs)
    for r in w.victims:
        p.assert_image_matches(r, extra_layers=[sh.num_layers // 2] if r == w.victims[0] else ())
    # dirty the reclaimed blocks everywhere so that a missing write cannot hide
    freed = torch.tensor(sorted(p.book.free), device="cuda")
    p.Kd[:, freed] = 0
    p.Vd[:, freed] = 0
    p.data.K[:, sorted(p.book.free)] = 0
    p.data.V[:, sorted(p.book.free)] = 0
    sums_before = p.block_sums()
    for r in reversed(w.victims):
        assert p.all3("swap_in_begin", r) == B.PS_OK
    q, out = _queries(sh, len(reqs), 7)
    mask, st, plan = p.step(q, out, reqs, -1)
    assert mask == [1] * len(reqs) and st["reloads_completed"] == len(w.victims) and st["gated"] == len(w.victims)
    p.sync()
    p.assert_tables_equal(reqs)
    p.assert_sampled_pools_equal()
    touched = set()
    for r in w.victims:
        k, v = p.logical_kv(r)
        assert torch.equal(k, saved[r][0]) and torch.equal(v, saved[r][1]), f"request {r} changed in the round trip"
        touched.update(p.lib.block_table(r)[0])
    untouched = torch.tensor(sorted(set(range(sh.num_gpu_blocks)) - touched), device="cuda")
    assert torch.equal(p.block_sums()[:, :, untouched], sums_before[:, :, untouched]), "a foreign block was written"
    p.check_attention(out, q, reqs, mask, sample_reqs=w.victims[:4] + [r for r in reqs if r not in w.victims][:4])
    p.book.check_invariants()
    p.destroy()


def test_config3_overlap_budgeted_reload_under_decode_full_size():
    """Decode batch 128 (lognormal contexts) while 8 preempted requests reload under 64 MiB per step."""
    _need_memory(70)
    w = wl.overlap()
    sh = w.shape
    reload_blocks = sum(sh.blocks_for(w.ctx_lens[r]) for r in w.victims)
    p = FullSizePair(w, [0, sh.num_layers - 1], max_batch=len(w.ctx_lens), max_blocks_per_req=513,
                     host_pool_bytes=reload_blocks * sh.block_bytes + (64 << 20))
    reqs = list(range(len(w.ctx_lens)))
    for r, n in wl.build_order_round_robin(w):
        assert p.all3("kv_alloc", r, n) == B.PS_OK
    saved = {r: p.logical_kv(r) for r in w.victims}
    for r in w.victims:
        assert p.all3("swap_out", r) == B.PS_OK
    p.sync()
    for r in w.victims:
        p.assert_image_matches(r)
        assert p.all3("swap_in_begin", r) == B.PS_OK
    q, out = _queries(sh, len(reqs), 11)
    budget = 64 * wl.MiB
    steps = 0
    sample = [0, 17, 64, 127] + list(range(128, 136))
    while any(p.book.missing_blocks(r) for r in w.victims):
        out.fill_(5.0)
        mask, st, plan = p.step(q, out, reqs, budget)
        assert st["blocks_copied"] <= budget // sh.block_bytes == 32
        steps += 1
        if steps % 6 == 1 or st["reloads_completed"]:
            assert p.lib.sync() == B.PS_OK
            p.check_attention(out, q, reqs, mask, sample)
            dead = [i for i, m in enumerate(mask) if not m]
            if dead:
                assert (out[:, dead].float() == 5.0).all()      # rows that do not decode are left untouched
        assert steps < 200
    assert steps == -(-reload_blocks // 32)
    p.sync()
    p.assert_tables_equal(reqs)
    p.assert_sampled_pools_equal()
    for r in w.victims:
        k, v = p.logical_kv(r)
        assert torch.equal(k, saved[r][0]) and torch.equal(v, saved[r][1])
    p.destroy()


def test_config5_long_context_offload_and_budgeted_reload_full_size():
    """70B-shaped KV, one 32k-token request (10 GiB) offloaded under decode and reloaded at 256 MiB per step."""
    _need_memory(120)
    w = wl.long_context()
    sh = w.shape
    long_req = w.victims[0]
    n_long = sh.blocks_for(w.ctx_lens[long_req])
    try:
        p = FullSizePair(w, [0, sh.num_layers - 1], max_batch=len(w.ctx_lens), max_blocks_per_req=n_long + 1,
                         host_pool_bytes=n_long * sh.block_bytes + (64 << 20))
    except B.PsError as e:                       # the box would not pin 10 GiB
        pytest.skip(str(e))
    reqs = list(range(len(w.ctx_lens)))
    batch = [r for r in reqs if r != long_req]
    for r, n in wl.build_order_round_robin(w):
        assert p.all3("kv_alloc", r, n) == B.PS_OK
    saved = p.logical_kv(long_req)
    q, out = _queries(sh, len(reqs), 13)
    assert p.all3("swap_out", long_req) == B.PS_OK
    # decode keeps running while the offload drains (no reload queued: the checkers have nothing to replay)
    for _ in range(3):
        rc, mask, st = p.lib.step(q[:, : len(batch)].contiguous(), out[:, : len(batch)].contiguous(), batch, 0)
        assert rc == B.PS_OK and all(mask)
    p.sync()
    p.assert_tables_equal(reqs)
    p.assert_image_matches(long_req, extra_layers=[40])
    freed = sorted(p.book.free)
    p.Kd[:, torch.tensor(freed, device="cuda")] = 0
    p.data.K[:, freed] = 0
    assert p.all3("swap_in_begin", long_req) == B.PS_OK
    budget = 256 * wl.MiB
    per_step = budget // sh.block_bytes
    steps = 0
    while p.book.missing_blocks(long_req):
        mask, st, plan = p.step(q, out, reqs, budget)
        steps += 1
        assert st["blocks_copied"] <= per_step
        if steps in (1, 20) or st["reloads_completed"]:
            assert p.lib.sync() == B.PS_OK
            p.check_attention(out, q, reqs, mask, [0, 31, 63, 64])
    assert steps == -(-n_long // per_step)
    p.sync()
    p.assert_sampled_pools_equal()
    k, v = p.logical_kv(long_req)
    assert torch.equal(k, saved[0]) and torch.equal(v, saved[1])
    p.assert_tables_equal(reqs)
    p.destroy()


def test_config4_priority_churn_full_shape():
    """Qwen3-32B-shaped KV (64 layers), 256 live requests of 512-16k tokens on an oversubscribed instance:
    200 seeded steps, each swapping out 2-16 low-priority requests and swapping in 2-16 others (clipped
    to capacity by the seeded script), decode over the resident set.
    The literal configuration (about 528 GiB of KV) does not fit one GPU: the device pool is 24 576
    blocks (96 GiB), the script plans with 12 GiB of host images, and requests that fit neither wait
    without KV (about 45 requests hold KV at any time).  The copy budget is unlimited: the configuration
    states none and asks for the swaps of a step to happen in that step; under a 256 MiB budget the
    reload queue of this script grows without bound (2 GiB per request against 64 blocks per step).
    The library's host pool is twice the script's figure because its images are contiguous, which the
    checker does not model."""
    _need_memory(130)
    host_bytes = 12 * wl.GiB
    w = wl.churn()
    sh = w.shape
    init, script = wl.churn_script(w, host_bytes)
    try:
        p = FullSizePair(w, [0, sh.num_layers - 1], max_batch=len(w.ctx_lens), max_blocks_per_req=1025,
                         host_pool_bytes=2 * host_bytes)
    except B.PsError as e:
        pytest.skip(str(e))
    p.book.host_pool_bytes = 2 * host_bytes
    for r in init["host"]:                       # host-resident requests pass through the device first
        assert p.all3("kv_alloc", r, w.ctx_lens[r]) == B.PS_OK
        assert p.all3("swap_out", r) == B.PS_OK
        p.sync()
    for r in init["resident"]:
        assert p.all3("kv_alloc", r, w.ctx_lens[r]) == B.PS_OK
    nreq = len(w.ctx_lens)
    q, out = _queries(sh, nreq, 17)
    budget = -1
    moved = ok_out = ok_in = decoded = 0
    for i, stp in enumerate(script):
        p.sync()                                  # the previous step's reloads have landed: their images are released
        for r in stp["out"]:
            rc = p.all3("swap_out", r)
            ok_out += rc == B.PS_OK
        for r in stp["inn"]:
            rc = p.all3("swap_in_begin", r)
            ok_in += rc == B.PS_OK
        p.sync()                                  # offloads complete in the step that issues them
        live = sorted(p.book.reqs)
        q_live = q[:, : len(live)].contiguous()
        out_live = torch.zeros_like(q_live)
        mask, st, plan = p.step(q_live, out_live, live, budget)
        moved += st["blocks_copied"]
        decoded += st["decoded"]
        if i % 40 == 0 or i == len(script) - 1:
            assert p.lib.sync() == B.PS_OK
            rows = [k for k, m in enumerate(mask) if m]
            p.check_attention(out_live, q_live, live, mask, rows[:2] + rows[-2:])
            p.assert_tables_equal(live)
            p.book.check_invariants()
    p.sync()
    p.assert_tables_equal(sorted(p.book.reqs))
    p.assert_sampled_pools_equal()
    for r, rq in p.data.reqs.items():             # every image still on host equals the checker's
        if rq.state == 3:
            p.assert_image_matches(r)
    assert moved > 0 and ok_out > 50 and ok_in > 50 and decoded > 0
    p.destroy()


def test_config4_closed_loop_driven_by_the_scheduler_stub_full_shape():
    """Config 4 at its shape (64 layers, 24 576 blocks of 4 MiB, 256 live requests of 512-16k tokens, two
    priority classes) driven by the paper's closed loop instead of a seeded script: every round the queue is
    ordered (ps_order_queue), memory pressure evicts from the tail (ps_select_victims, asynchronous offloads
    reaped when their transfers complete), the head is readmitted, ps_copy_budget sets the step's budget and
    ps_step_ruled consumes it under the partial-copy rule while the resident set decodes.  A backend makes
    every call on the library and on the checkers and compares decisions, codes, states and plans; bytes of
    two sampled layers and attention on sampled rows are compared as in the other full-size tests."""
    _need_memory(130)
    w = wl.churn()
    sh = w.shape
    params = el.config4_params()
    try:
        p = FullSizePair(w, [0, sh.num_layers - 1], max_batch=params.max_batch, max_blocks_per_req=1040,
                         host_pool_bytes=30 * wl.GiB)
    except B.PsError as e:
        pytest.skip(str(e))
    be = PairedBackend(p.lib, p.book, p.data)
    stub = el.SchedulerStub(be, w.ctx_lens, w.priority, sh.block_size, sh.block_bytes, sh.num_gpu_blocks, params,
                            seed=w.seed)
    placed = stub.fill()
    assert len(placed) > 30
    q, out = _queries(sh, params.max_batch, 19)
    checked = []

    def on_step(batch, mask, qv, ov):
        if stub.rounds % 12 == 0 or stub.rounds >= 58:
            torch.cuda.synchronize()
            rows = [k for k, m in enumerate(mask) if m]
            gated_rows = [k for k in rows if batch[k] in {r for r, _, _ in be.plans}]
            p.check_attention(ov, qv, batch, mask, (rows[:2] + rows[-1:] + gated_rows[:2]))
            checked.append(len(rows))

    tot = dict(evicted=0, readmitted=0, admitted=0, finished=0, copied=0, decoded=0)
    for _ in range(60):
        rep = stub.round(q, out, on_step)
        tot["evicted"] += len(rep.evicted)
        tot["readmitted"] += len(rep.readmitted)
        tot["admitted"] += len(rep.admitted)
        tot["finished"] += len(rep.finished)
        tot["copied"] += rep.stats["blocks_copied"]
        tot["decoded"] += sum(rep.mask)
        if stub.rounds % 20 == 0:
            p.book.check_invariants()
    p.sync()
    p.assert_tables_equal(sorted(p.book.reqs))
    p.assert_sampled_pools_equal()
    for r, rq in p.data.reqs.items():             # every image still on host equals the checker's
        if rq.state == 3:
            p.assert_image_matches(r)
    assert tot["evicted"] >= 3 and tot["readmitted"] >= 2 and tot["copied"] > 500 and tot["decoded"] > 1500, tot
    assert be.counts["victims"] >= 1 and be.counts["budget"] == 60 and len(checked) >= 5
    p.destroy()
