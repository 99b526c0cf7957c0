"""Pins for the CPU checker's paged decode attention (no GPU).

Each test fixes the fp64 attention to something other than itself: explicit loops, a library's
own attention / logsumexp routines on contiguous KV, closed forms, or invariants a correct
softmax-attention over a block table must have.
"""
import math

import numpy as np
import pytest
import scipy.special
import torch

from oracle import ps_oracle as po
from paper_2512_12928_b200 import workloads as wl


def make(seed=0, L=2, Hkv=2, Hq=4, D=16, S=4, nb=32, ctxs=(5, 16, 1, 23)):
    rng = np.random.default_rng(seed)
    K = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    V = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    o = po.PsOracle(L, Hkv, Hq, D, S, nb, rng.permutation(nb), K, V)
    turn = 0
    grown = [0] * len(ctxs)
    while any(g < c for g, c in zip(grown, ctxs)):          # interleave to fragment the tables
        for r, c in enumerate(ctxs):
            if grown[r] < c:
                grown[r] = min(c, grown[r] + S)
                assert o.kv_alloc(r, grown[r]) == po.OK
        turn += 1
    q = wl.randn_bf16_bits(rng, (L, len(ctxs), Hq, D))
    return o, q


def test_bf16_decode_matches_field_by_field_and_torch():
    bits = np.array([0x0000, 0x8000, 0x3F80, 0xBF80, 0x4049, 0x0001, 0x7F7F, 0x3DCC, 0x0080], dtype=np.uint16)
    got = po.bf16_bits_to_f64(bits)
    want = [po._bf16_to_float(int(b)) for b in bits]
    assert got.tolist() == want
    t = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).double().numpy()
    assert got.tolist() == t.tolist()
    assert got[2] == 1.0 and got[3] == -1.0 and got[4] == 3.140625


def test_bf16_rounding_of_generator_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, -2.5, 3.14159, 1e-3], dtype=np.float32)  # 1+2^-8 is a tie
    got = wl.f32_to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert got.tolist() == want.tolist()


def test_matches_brute_force_loops():
    o, q = make(seed=1)
    for layer in range(o.L):
        got, _ = o.decode_attn(layer, q[layer], [0, 1, 2, 3])
        for i in range(4):
            t, _ = o.block_table(i)
            want = po.brute_force_attn(o.K[layer].tolist(), o.V[layer].tolist(), t, o.reqs[i].n_tokens,
                                       q[layer][i].tolist(), o.S, o.G)
            assert np.max(np.abs(got[i] - np.array(want))) < 1e-12


def test_matches_torch_sdpa_fp64_on_contiguous_kv():
    o, q = make(seed=2, Hkv=2, Hq=8, D=32, S=8, nb=40, ctxs=(17, 64, 9))
    for layer in range(o.L):
        got, lse = o.decode_attn(layer, q[layer], [0, 1, 2])
        for i in range(3):
            t, _ = o.block_table(i)
            n = o.reqs[i].n_tokens
            # contiguous KV built here, independently of the checker's gather
            kb = torch.from_numpy(o.K[layer][t].reshape(-1, o.Hkv, o.D)[:n].view(np.int16)).view(torch.bfloat16).double()
            vb = torch.from_numpy(o.V[layer][t].reshape(-1, o.Hkv, o.D)[:n].view(np.int16)).view(torch.bfloat16).double()
            qq = torch.from_numpy(q[layer][i].view(np.int16)).view(torch.bfloat16).double()       # [Hq][D]
            kk = kb.permute(1, 0, 2).repeat_interleave(o.G, dim=0)                              # [Hq][T][D]
            vv = vb.permute(1, 0, 2).repeat_interleave(o.G, dim=0)
            want = torch.nn.functional.scaled_dot_product_attention(qq[:, None, :], kk, vv)[:, 0, :]
            assert np.max(np.abs(got[i] - want.numpy())) < 1e-12
            logits = torch.einsum("hd,htd->ht", qq, kk).numpy() / math.sqrt(o.D)
            assert np.max(np.abs(lse[i] - scipy.special.logsumexp(logits, axis=1))) < 1e-12


def test_probabilities_sum_to_one_and_reproduce_output():
    o, q = make(seed=3)
    for i in range(4):
        p = o.attn_probs(0, q[0][i], i)
        assert p.shape == (o.Hq, o.reqs[i].n_tokens)
        assert np.max(np.abs(p.sum(axis=1) - 1.0)) < 1e-12 and (p >= 0).all()
        _, v = o.gather_kv(0, i)
        got, _ = o.decode_attn(0, q[0][i:i + 1], [i])
        for h in range(o.Hq):
            assert np.max(np.abs(p[h] @ v[:, h // o.G, :] - got[0, h])) < 1e-12


def test_single_token_returns_its_value_row():
    o, q = make(seed=4)
    got, lse = o.decode_attn(1, q[1][2:3], [2])              # request 2 has one token
    b = o.block_table(2)[0][0]
    for h in range(o.Hq):
        assert np.array_equal(got[0, h], po.bf16_bits_to_f64(o.V[1, b, 0, h // o.G]))
        s = float(po.bf16_bits_to_f64(o.K[1, b, 0, h // o.G]) @ po.bf16_bits_to_f64(q[1][2][h])) / math.sqrt(o.D)
        assert abs(lse[0, h] - s) < 1e-12


def test_equal_keys_give_mean_of_values():
    o, q = make(seed=5)
    t = o.block_table(3)[0]
    n = o.reqs[3].n_tokens
    for b in t:
        o.K[0, b] = o.K[0, t[0], 0][None]                     # every token's key = first token's key
    got, _ = o.decode_attn(0, q[0][3:4], [3])
    _, v = o.gather_kv(0, 3)
    for h in range(o.Hq):
        assert np.max(np.abs(got[0, h] - v[:n, h // o.G].mean(axis=0))) < 1e-12


def test_two_token_closed_form_pins_the_scale():
    """o = sigma(delta) v0 + (1 - sigma(delta)) v1 with delta = q.(k0 - k1)/sqrt(D)."""
    L, Hkv, Hq, D, S, nb = 1, 1, 1, 64, 2, 4
    K = np.zeros((L, nb, S, Hkv, D), np.uint16); V = np.zeros_like(K)
    one, two, mone = 0x3F80, 0x4000, 0xBF80
    o = po.PsOracle(L, Hkv, Hq, D, S, nb, [2, 0, 1, 3], K, V)
    o.kv_alloc(0, 2)
    b = o.block_table(0)[0][0]
    assert b == 2
    K[0, b, 0, 0, :] = one           # k0 = 1s
    K[0, b, 1, 0, :] = mone          # k1 = -1s
    V[0, b, 0, 0, :] = two           # v0 = 2s
    V[0, b, 1, 0, :] = mone          # v1 = -1s
    q = np.zeros((1, Hq, D), np.uint16); q[0, 0, :16] = one   # q.(k0-k1) = 32, /sqrt(64) = 4
    got, lse = o.decode_attn(0, q, [0])
    sig = 1.0 / (1.0 + math.exp(-4.0))
    assert np.max(np.abs(got[0, 0] - (sig * 2.0 + (1 - sig) * -1.0))) < 1e-14
    assert abs(lse[0, 0] - math.log(math.exp(2.0) + math.exp(-2.0))) < 1e-14


def test_dominant_key_selects_its_value_row_through_the_table():
    o, q = make(seed=6, ctxs=(23,), nb=16)
    t = o.block_table(0)[0]
    # V rows encode (block id, slot): a read from the wrong block or slot shows in the output
    for b in range(o.num_blocks):
        for s in range(o.S):
            o.V[:, b, s] = wl.f32_to_bf16_bits(np.full((o.Hkv, o.D), b * o.S + s, np.float32))
    o.K[:] = 0
    tok = 13
    qf = po.bf16_bits_to_f64(q[0][0])                          # [Hq][D]
    for g in range(o.Hkv):
        o.K[0, t[tok // o.S], tok % o.S, g] = wl.f32_to_bf16_bits((64.0 * qf[g * o.G]).astype(np.float32))
    got, _ = o.decode_attn(0, q[0], [0])
    want = t[tok // o.S] * o.S + tok % o.S
    assert np.max(np.abs(got[0, ::o.G] - want)) < 1e-6        # heads g*G see their own scaled key


def test_tokens_beyond_ctx_len_are_masked():
    o, q = make(seed=7)
    got0, lse0 = o.decode_attn(0, q[0], [0, 1, 2, 3])
    for r in range(4):
        n = o.reqs[r].n_tokens
        t = o.block_table(r)[0]
        if n % o.S:
            o.K[0, t[-1], n % o.S:] = 0x7F80                   # +inf in the unused tail slots
            o.V[0, t[-1], n % o.S:] = 0x7FC0                   # NaN
    got1, lse1 = o.decode_attn(0, q[0], [0, 1, 2, 3])
    assert np.array_equal(got0, got1) and np.array_equal(lse0, lse1)


def test_output_independent_of_physical_block_placement():
    o, q = make(seed=8, ctxs=(19, 8))
    got0, _ = o.decode_attn(1, q[1], [0, 1])
    # move request 0 to other physical blocks: swap out, disturb the free list, swap in
    assert o.swap_out(0) == po.OK
    o.reap()
    assert o.kv_alloc(5, 7) == po.OK
    assert o.swap_in_begin(0) == po.OK
    o.step(-1)
    got1, _ = o.decode_attn(1, q[1], [0, 1])
    assert np.array_equal(got0, got1)


def test_gqa_head_mapping():
    o, q = make(seed=9, Hkv=2, Hq=4)
    qq = q[0].copy()
    qq[:, 1] = qq[:, 0]; qq[:, 3] = qq[:, 2]                   # heads sharing a KV head get equal queries
    got, _ = o.decode_attn(0, qq, [0, 1, 2, 3])
    assert np.array_equal(got[:, 0], got[:, 1]) and np.array_equal(got[:, 2], got[:, 3])
    assert not np.allclose(got[:, 0], got[:, 2])
    # zeroing KV head 1 changes only query heads 2 and 3
    o.V[0, :, :, 1] = 0
    got2, _ = o.decode_attn(0, qq, [0, 1, 2, 3])
    assert np.array_equal(got2[:, :2], got[:, :2]) and not got2[:, 2:].any()


def test_empty_context_gives_zero_and_minus_inf():
    o, q = make(seed=10)
    assert o.kv_alloc(9, 0) == po.OK
    got, lse = o.decode_attn(0, q[0][:1], [9])
    assert not got.any() and np.isneginf(lse).all()


def test_step_decodes_only_complete_requests():
    o, q = make(seed=11, ctxs=(9, 14, 6))
    o.swap_out(1); o.reap(); o.swap_in_begin(1)
    bb = o.block_bytes
    plan, mask, out = o.step(2 * bb, [0, 1, 2], q)
    assert plan == [(1, 0, 2)] and mask == [1, 0, 1]
    assert np.isnan(out[:, 1]).all() and not np.isnan(out[:, [0, 2]]).any()
    plan, mask, out = o.step(2 * bb, [0, 1, 2], q)
    assert plan == [(1, 2, 4)] and mask == [1, 1, 1] and not np.isnan(out).any()
    want, _ = o.decode_attn(1, q[1], [0, 1, 2])
    assert np.array_equal(out[1], want)


@pytest.mark.parametrize("mistake", ["no_scale", "wrong_head", "off_by_one_mask"])
def test_pins_catch_planted_mistakes(mistake):
    """A broken variant of the checker must fail at least one pin (the mistake lives on the CPU)."""
    class Broken(po.PsOracle):
        def decode_attn(self, layer, q_bits, reqs):
            q = po.bf16_bits_to_f64(q_bits).reshape(len(reqs), self.Hq, self.D)
            o = np.zeros((len(reqs), self.Hq, self.D))
            for i, req in enumerate(reqs):
                k, v = self.gather_kv(layer, req)
                if mistake == "off_by_one_mask":
                    k, v = k[:-1] if len(k) > 1 else k, v[:-1] if len(v) > 1 else v
                for h in range(self.Hq):
                    g = (h % self.Hkv) if mistake == "wrong_head" else h // self.G
                    s = k[:, g] @ q[i, h]
                    if mistake != "no_scale":
                        s = s / math.sqrt(self.D)
                    e = np.exp(s - s.max())
                    o[i, h] = (e / e.sum()) @ v[:, g]
            return o, None
    rng = np.random.default_rng(0)
    L, Hkv, Hq, D, S, nb = 1, 2, 4, 16, 4, 8
    K = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D)); V = wl.randn_bf16_bits(rng, (L, nb, S, Hkv, D))
    good = po.PsOracle(L, Hkv, Hq, D, S, nb, None, K, V)
    bad = Broken(L, Hkv, Hq, D, S, nb, None, K, V)
    for x in (good, bad):
        x.kv_alloc(0, 11)
    q = wl.randn_bf16_bits(rng, (1, Hq, D))
    ref = np.array(po.brute_force_attn(K[0].tolist(), V[0].tolist(), good.block_table(0)[0], 11, q[0].tolist(), S, 2))
    assert np.max(np.abs(good.decode_attn(0, q, [0])[0][0] - ref)) < 1e-12
    assert np.max(np.abs(bad.decode_attn(0, q, [0])[0][0] - ref)) > 1e-3
