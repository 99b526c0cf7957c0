"""ps_decode_attn_static, the entry point for callers that may not allocate device memory.

An engine that gave every byte of the GPU to its own pool allocator at start-up, a plug-in bound
to another program's memory budget, or a loop in which an allocation (a possible device-wide
synchronisation) is forbidden cannot use ps_create, whose context allocates the split-KV scratch.
For them the library carries one fixed scratch array in its own image.  This test calls that entry
point through the C ABI twice in a row (the second call sees the first call's leftovers in the
shared array) and checks each output against ps_decode_attn on the same inputs, and against the
CPU checker.  It is collected last so that a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import workloads as wl

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from gpu_util import Pair, bits_to_dev, check_attn


def _tables_on_device(p, reqs):
    tabs = [p.lib.block_table(r)[0] for r in reqs]
    stride = max(1, max(len(t) for t in tabs))
    arr = np.zeros((len(reqs), stride), np.int32)
    for i, t in enumerate(tabs):
        arr[i, : len(t)] = t
    return torch.from_numpy(arr).cuda()


def test_static_scratch_attention_matches_context_attention_twice():
    Hkv, Hq, D, S, L, nb = 8, 32, 128, 16, 1, 700
    sh = wl.KVShape(L, Hkv, Hq, D, S, nb)
    rng = np.random.default_rng(20251212)
    K = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    V = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    p = Pair(sh, rng.permutation(nb), K, V, max_batch=16, attn_kernel=B.PS_ATTN_SIMT)
    ctxs = [3000, 1, 0, S, 5 * S + 7, 2049, 777, 1500]
    grown = [0] * len(ctxs)
    assert p.both("kv_alloc", 2, 0) == B.PS_OK
    while any(g < c for g, c in zip(grown, ctxs)):                 # interleaved growth: scattered tables
        for r, c in enumerate(ctxs):
            if grown[r] < c:
                grown[r] = min(c, grown[r] + S)
                assert p.both("kv_alloc", r, grown[r]) == B.PS_OK
    q_bits = wl.randn_bf16_bits(rng, (2, len(ctxs), Hq, D))
    qd = bits_to_dev(q_bits)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    # two different batches back to back: long split contexts first, then a short, reordered one
    calls = [(list(range(len(ctxs))), 0, 256), ([6, 1, 4, 0], 1, 0)]
    for reqs, qi, split in calls:
        q = qd[qi][: len(reqs)].contiguous()
        want_dev = torch.zeros_like(q)
        want_lse = torch.zeros((len(reqs), Hq), dtype=torch.float32, device="cuda")
        assert p.lib.decode_attn(0, q, want_dev, reqs, want_lse) == B.PS_OK, p.lib.last_error()
        assert p.lib.sync() == B.PS_OK
        tables = _tables_on_device(p, reqs)
        out = torch.full_like(q, 9.0)
        lse = torch.zeros_like(want_lse)
        rc, text = B.ps_decode_attn_static(p.Kd[0], p.Vd[0], q, out, tables, [ctxs[r] for r in reqs],
                                           num_kv_heads=Hkv, num_q_heads=Hq, head_dim=D, block_size=S,
                                           num_gpu_blocks=nb, kv_split_tokens=split, lse=lse, status_word=status)
        assert rc == B.PS_OK, text
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        diff = (out.double() - want_dev.double()).abs().max().item()
        assert diff <= 2e-2, diff
        finite = torch.isfinite(want_lse)
        assert torch.equal(finite, torch.isfinite(lse))
        assert (lse[finite] - want_lse[finite]).abs().max().item() < 1e-3
        want, _ = p.orc.decode_attn(0, q_bits[qi][: len(reqs)], reqs)
        check_attn(out, want)

    # sizes beyond the fixed scratch are refused with a message, and nothing is launched
    rc, text = B.ps_decode_attn_static(p.Kd[0], p.Vd[0], qd[0], torch.zeros_like(qd[0]), _tables_on_device(p, [0]),
                                       [1] * (B.PS_STATIC_MAX_BATCH + 1), num_kv_heads=Hkv, num_q_heads=Hq,
                                       head_dim=D, block_size=S, num_gpu_blocks=nb)
    assert rc == B.PS_ERR_INVALID and "maximum" in text
    rc, text = B.ps_decode_attn_static(p.Kd[0], p.Vd[0], qd[0], torch.zeros_like(qd[0]), _tables_on_device(p, [0]),
                                       [3000], num_kv_heads=Hkv, num_q_heads=Hq, head_dim=D, block_size=S,
                                       num_gpu_blocks=nb, kv_split_tokens=1)
    assert rc == B.PS_ERR_INVALID and "scratch" in text
    torch.cuda.synchronize()
