"""The scheduler stub's closed loop on a bookkeeping-only library context against the checker (no GPU):
queue ordering, eviction from the tail, readmission from the head, the adaptive copy budget and its
consumption under the partial-copy rule, round after round, decisions and tables identical on both sides."""
import numpy as np

from loop_util import PairedBackend
from oracle import ps_oracle as po
from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import engine_loop as el
from paper_2512_12928_b200 import workloads as wl


def small_loop(seed, rounds, **over):
    sh = wl.KVShape(2, 2, 4, 64, 16, 600)
    rng = np.random.default_rng(seed)
    order = rng.permutation(sh.num_gpu_blocks)
    lib = B.KVSwap(num_layers=sh.num_layers, num_kv_heads=sh.num_kv_heads, num_q_heads=sh.num_q_heads,
                   head_dim=sh.head_dim, block_size=sh.block_size, num_gpu_blocks=sh.num_gpu_blocks,
                   max_blocks_per_req=80, host_pool_bytes=1 << 40, initial_free_order=order,
                   flags=B.PS_FLAG_BOOKKEEPING_ONLY)
    book = po.PsOracle(sh.num_layers, sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size,
                       sh.num_gpu_blocks, order)
    be = PairedBackend(lib, book)
    ctx = [int(v) for v in rng.integers(64, 1025, size=64)]
    prio = [int(v) for v in rng.integers(0, 2, size=64)]
    kw = dict(t_block_us=80.0, host_budget_bytes=400 * sh.block_bytes, max_batch=64, tau_us=60000.0,
              tpot_us=(3000.0, 12000.0), ttft_us=(20000.0, 200000.0), eta_us=1500.0, gen_tokens=(5, 30))
    kw.update(over)
    stub = el.SchedulerStub(be, ctx, prio, sh.block_size, sh.block_bytes, sh.num_gpu_blocks, el.LoopParams(**kw), seed)
    stub.fill()
    tot = dict(evicted=0, readmitted=0, admitted=0, finished=0, decoded=0, copied=0, skipped=0)
    for _ in range(rounds):
        rep = stub.round(None, None)
        tot["evicted"] += len(rep.evicted)
        tot["readmitted"] += len(rep.readmitted)
        tot["admitted"] += len(rep.admitted)
        tot["finished"] += len(rep.finished)
        tot["decoded"] += sum(rep.mask)
        tot["copied"] += rep.stats["blocks_copied"]
        tot["skipped"] += rep.skipped_by_rule
        book.check_invariants()
    for r in sorted(book.reqs):
        assert lib.block_table(r) == book.block_table(r)
    return stub, be, tot


def test_closed_loop_decisions_match_the_checker_round_for_round():
    stub, be, tot = small_loop(seed=7, rounds=400)
    assert len(stub.live) == 64
    assert tot["evicted"] > 20 and tot["readmitted"] > 20 and tot["finished"] > 40 and tot["decoded"] > 2000
    assert tot["copied"] > 200
    assert be.counts["victims"] > 10 and {21, 22} & be.counts["cases"]
    # the partial-copy rule was consulted and did change plans (requests skipped or held back)
    assert be.counts["rule_skips"] > 0 and tot["skipped"] > 0


def test_closed_loop_of_prefilling_requests_takes_partial_copies():
    """Every arrival still has prompt chunks to process: while a request's backlog reaches the chunk limit its
    l_comp reaches the round's limit and it takes the residual budget, so plans carry partial copies."""
    stub, be, tot = small_loop(seed=11, rounds=250, prefilling_frac=1.0, chunk_tokens=64)
    assert be.counts["partial"] > 30 and tot["readmitted"] > 5 and tot["copied"] > 200
