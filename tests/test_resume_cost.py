"""Batch latency estimator (Section 4.1) and the reload-versus-recompute cost of an evicted request: the checker
against hand-worked values and identities, and the library against the checker."""
import json
import os

import numpy as np
import pytest

from oracle import ps_oracle as po
from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import build as ps_build

GOLDEN = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "latency_estimator.json")))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    ps_build.build()
    return B.load()


def c_model(m):
    return B.PsLatencyModel(m["a_p"], m["b_p"], m["c_p"], m["a_d"], m["b_d"], m["t_c"])


def test_checker_reproduces_the_hand_worked_estimates():
    m = GOLDEN["model"]
    for case in GOLDEN["batches"]:
        got = po.estimate_batch(m, [tuple(p) for p in case["prefill"]], case["decode"])
        assert got == pytest.approx(case["us"], rel=1e-12, abs=1e-9), case["work"]
    for case in GOLDEN["resume"]:
        reload_t, recompute_t = po.resume_cost(m, case["n_tokens"], case["chunk_tokens"], case["s_blk"], case["t_block"])
        assert reload_t == pytest.approx(case["reload_us"], rel=1e-12, abs=1e-9), case["work"]
        assert recompute_t == pytest.approx(case["recompute_us"], rel=1e-12, abs=1e-9), case["work"]


def test_decode_only_batch_agrees_with_the_step_estimate_of_the_budget_rule():
    """The adaptive budget's step-time estimate is the same batch equation restricted to decode requests."""
    orc = po.PsOracle(2, 1, 1, 8, 4, 64)
    ctxs = [5, 16, 33, 1]
    for r, n in enumerate(ctxs):
        assert orc.kv_alloc(r, n) == 0
    m = dict(a_p=0.0, b_p=0.0, c_p=0.0, a_d=0.7, b_d=3.0, t_c=11.0)
    assert po.estimate_batch(m, [], ctxs) == pytest.approx(orc.step_latency_after(range(4), 0, 0.7, 3.0, 11.0), rel=1e-14)


def test_chunking_a_causal_prefill_leaves_its_cost_unchanged():
    """With b_p = 2 a_p (a token attends to each cached token at twice the cost per pair of the a_p term, which
    counts the causal half of the chunk's own square) and no per-batch overhead, the chunks' costs telescope:
    sum_k a (l_k^2 + 2 l_k s_k) = a n^2 where s_k is the prefix before chunk k.  So any chunk size, ragged or
    not, must return a n^2 + c n."""
    rng = np.random.default_rng(4128)
    for _ in range(50):
        a, c = float(rng.uniform(1e-4, 1e-2)), float(rng.uniform(1.0, 20.0))
        n = int(rng.integers(1, 5000))
        chunk = int(rng.integers(1, n + 50))
        m = dict(a_p=a, b_p=2 * a, c_p=c, a_d=0.0, b_d=0.0, t_c=0.0)
        _, got = po.resume_cost(m, n, chunk, 16, 1.0)
        assert got == pytest.approx(a * n * n + c * n, rel=1e-10)


def test_every_chunk_is_a_batch_and_pays_the_constant_overhead():
    m0 = dict(GOLDEN["model"], t_c=0.0)
    m1 = dict(GOLDEN["model"], t_c=37.5)
    for n, chunk in [(100, 0), (100, 100), (100, 33), (1, 7), (4096, 512), (4097, 512)]:
        chunks = 1 if chunk == 0 else -(-n // chunk)
        d = po.resume_cost(m1, n, chunk, 16, 1.0)[1] - po.resume_cost(m0, n, chunk, 16, 1.0)[1]
        assert d == pytest.approx(chunks * 37.5, rel=1e-9)


def test_reload_counts_whole_blocks_and_grows_with_the_context():
    m = GOLDEN["model"]
    prev = (-1.0, -1.0)
    for n in range(0, 200):
        cur = po.resume_cost(m, n, 64, 16, 40.0)
        assert cur[0] == 40.0 * ((n + 15) // 16)
        assert cur[0] >= prev[0] and cur[1] >= prev[1]
        prev = cur


def test_library_estimates_equal_the_checker():
    rng = np.random.default_rng(97)
    for _ in range(200):
        m = dict(a_p=float(rng.uniform(0, 1e-2)), b_p=float(rng.uniform(0, 1e-2)), c_p=float(rng.uniform(0, 30)),
                 a_d=float(rng.uniform(0, 0.1)), b_d=float(rng.uniform(0, 50)), t_c=float(rng.uniform(0, 200)))
        prefill = [(int(rng.integers(0, 4096)), int(rng.integers(0, 32768))) for _ in range(int(rng.integers(0, 5)))]
        decode = [int(v) for v in rng.integers(0, 32768, size=int(rng.integers(0, 9)))]
        rc, got = B.ps_estimate_batch(c_model(m), prefill, decode)
        assert rc == B.PS_OK
        assert got == pytest.approx(po.estimate_batch(m, prefill, decode), rel=1e-12, abs=1e-9)
        n, chunk = int(rng.integers(0, 40000)), int(rng.choice([0, 1, 17, 256, 512, 2048, 50000]))
        if chunk == 1:
            n = min(n, 3000)
        s_blk, t_block = int(rng.choice([1, 16, 32])), float(rng.uniform(0, 100))
        rc, reload_us, recompute_us = B.ps_resume_cost(c_model(m), n, chunk, s_blk, t_block)
        assert rc == B.PS_OK
        want = po.resume_cost(m, n, chunk, s_blk, t_block)
        assert reload_us == pytest.approx(want[0], rel=1e-12, abs=1e-9)
        assert recompute_us == pytest.approx(want[1], rel=1e-12, abs=1e-9)
    for case in GOLDEN["resume"]:
        rc, reload_us, recompute_us = B.ps_resume_cost(c_model(GOLDEN["model"]), case["n_tokens"], case["chunk_tokens"],
                                                       case["s_blk"], case["t_block"])
        assert (rc, reload_us) == (B.PS_OK, case["reload_us"])
        assert recompute_us == pytest.approx(case["recompute_us"], rel=1e-12, abs=1e-9)


def test_library_rejects_bad_arguments():
    m = GOLDEN["model"]
    assert B.ps_estimate_batch(c_model(dict(m, a_p=-1.0)), [], [])[0] == B.PS_ERR_INVALID
    assert B.ps_estimate_batch(c_model(m), [(-1, 0)], [])[0] == B.PS_ERR_INVALID
    assert B.ps_estimate_batch(c_model(m), [], [-5])[0] == B.PS_ERR_INVALID
    assert B.ps_resume_cost(c_model(m), -1, 0, 16, 1.0)[0] == B.PS_ERR_INVALID
    assert B.ps_resume_cost(c_model(m), 10, -1, 16, 1.0)[0] == B.PS_ERR_INVALID
    assert B.ps_resume_cost(c_model(m), 10, 0, 0, 1.0)[0] == B.PS_ERR_INVALID
    assert B.ps_resume_cost(c_model(m), 10, 0, 16, -1.0)[0] == B.PS_ERR_INVALID
    assert B.ps_resume_cost(c_model(dict(m, t_c=-1.0)), 10, 0, 16, 1.0)[0] == B.PS_ERR_INVALID
