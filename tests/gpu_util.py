"""Helpers for the GPU parity tests: device pools from the seeded bit patterns, a paired driver."""
import ctypes as C

import numpy as np
import torch

from oracle import ps_oracle as po
from paper_2512_12928_b200 import binding as B
from paper_2512_12928_b200 import workloads as wl


def bits_to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 patterns -> bf16 tensor on the GPU, same shape."""
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def dev_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bf16_dev_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().double().cpu().numpy()


class Pair:
    """The library on the GPU and the CPU checker over identical pools, driven side by side."""

    def __init__(self, sh: wl.KVShape, free_order, K: np.ndarray, V: np.ndarray, *, max_batch=64,
                 host_pool_bytes=None, staging_bytes=0, flags=0, attn_kernel=B.PS_ATTN_AUTO, kv_split_tokens=0,
                 max_blocks_per_req=None, layer_chunk_bytes=0):
        self.sh = sh
        self.Kd = bits_to_dev(K)           # [L][nb][S][Hkv][D]
        self.Vd = bits_to_dev(V)
        torch.cuda.synchronize()
        if host_pool_bytes is None:
            host_pool_bytes = sh.num_gpu_blocks * sh.block_bytes + (1 << 20)
        self.lib = B.KVSwap(num_layers=sh.num_layers, num_kv_heads=sh.num_kv_heads, num_q_heads=sh.num_q_heads,
                            head_dim=sh.head_dim, block_size=sh.block_size, num_gpu_blocks=sh.num_gpu_blocks,
                            max_blocks_per_req=max_blocks_per_req or sh.num_gpu_blocks, max_batch=max_batch,
                            host_pool_bytes=host_pool_bytes, staging_bytes=staging_bytes,
                            initial_free_order=free_order, k_pools=[self.Kd[l] for l in range(sh.num_layers)],
                            v_pools=[self.Vd[l] for l in range(sh.num_layers)], flags=flags,
                            attn_kernel=attn_kernel, kv_split_tokens=kv_split_tokens,
                            layer_chunk_bytes=layer_chunk_bytes)
        self.orc = po.PsOracle(sh.num_layers, sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size,
                               sh.num_gpu_blocks, free_order, K.copy(), V.copy())

    def both(self, name, *args):
        a = getattr(self.lib, name)(*args)
        b = getattr(self.orc, name)(*args)
        assert a == b, (name, args, a, b)
        return a

    def sync(self):
        assert self.lib.sync() == B.PS_OK, self.lib.last_error()
        self.orc.reap()

    def host_image_bits(self, req) -> np.ndarray:
        ptr, nbytes = self.lib.host_image(req)
        buf = (C.c_uint16 * (nbytes // 2)).from_address(ptr)
        return np.ctypeslib.as_array(buf).copy()

    def assert_tables_equal(self, reqs):
        for r in reqs:
            assert self.lib.block_table(r) == self.orc.block_table(r), r
        assert self.lib.num_free_blocks() == self.orc.num_free_blocks()

    def assert_pools_equal(self):
        torch.cuda.synchronize()
        assert np.array_equal(dev_to_bits(self.Kd), self.orc.K), "K pool differs from the checker"
        assert np.array_equal(dev_to_bits(self.Vd), self.orc.V), "V pool differs from the checker"


def check_attn(got_bf16: torch.Tensor, want: np.ndarray, max_abs=2e-2, rel_l2=1e-2):
    """got: device bf16 [..., D]; want: float64 same shape.  Max-abs contract plus per-row relative L2."""
    got = bf16_dev_to_f64(got_bf16)
    assert got.shape == want.shape
    err = np.abs(got - want)
    assert err.max() <= max_abs, f"max abs err {err.max()}"
    num = np.sqrt(((got - want) ** 2).sum(-1))
    den = np.sqrt((want ** 2).sum(-1))
    ok = den > 0
    if ok.any():
        worst = (num[ok] / den[ok]).max()
        assert worst <= rel_l2, f"relative L2 err {worst}"
    return float(err.max())


class FullSizePair:
    """The library at a workload's full size, checked against the CPU checker on what it can hold.

    Three parties are driven side by side with the same calls:
      lib   the library on the GPU over the full pools (all layers),
      book  a checker without pool bytes (all layers): block tables, states, budget plans, id for id,
      data  a checker over the full block-id space but only `sample_layers` of the pools (copied from the
            device with plain tensor.cpu(), which is not the path under test): host images, pool bytes and
            attention of those layers, byte for byte / within tolerance.
    Bytes of the other layers are checked by properties computed with torch on the device (round trip of
    the logical KV, per-block sums of untouched blocks)."""

    def __init__(self, w: wl.Workload, sample_layers, *, max_batch, host_pool_bytes, max_blocks_per_req, flags=0):
        sh = self.sh = w.shape
        self.w = w
        self.sample_layers = list(sample_layers)
        L, nb = sh.num_layers, sh.num_gpu_blocks
        g = torch.Generator(device="cuda")
        g.manual_seed(w.seed)
        self.Kd = torch.empty((L, nb, sh.block_size, sh.num_kv_heads, sh.head_dim), dtype=torch.bfloat16, device="cuda")
        self.Vd = torch.empty_like(self.Kd)
        for l in range(L):
            self.Kd[l].normal_(generator=g)
            self.Vd[l].normal_(generator=g)
        torch.cuda.synchronize()
        self.lib = B.KVSwap(num_layers=L, num_kv_heads=sh.num_kv_heads, num_q_heads=sh.num_q_heads,
                            head_dim=sh.head_dim, block_size=sh.block_size, num_gpu_blocks=nb,
                            max_blocks_per_req=max_blocks_per_req, max_batch=max_batch, host_pool_bytes=host_pool_bytes,
                            initial_free_order=w.free_order, k_pools=[self.Kd[l] for l in range(L)],
                            v_pools=[self.Vd[l] for l in range(L)], flags=flags)
        self.book = po.PsOracle(L, sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size, nb, w.free_order)
        Ks = np.stack([dev_to_bits(self.Kd[l]) for l in self.sample_layers])
        Vs = np.stack([dev_to_bits(self.Vd[l]) for l in self.sample_layers])
        self.data = po.PsOracle(len(self.sample_layers), sh.num_kv_heads, sh.num_q_heads, sh.head_dim, sh.block_size,
                                nb, w.free_order, Ks, Vs)

    def all3(self, name, *args):
        a = getattr(self.lib, name)(*args)
        b = getattr(self.book, name)(*args)
        assert a == b, (name, args, a, b)
        if a == B.PS_OK:                     # a refused call changed nothing; the data checker has no host-pool limit
            c = getattr(self.data, name)(*args)
            assert c == a, (name, args, a, c)
        return a

    def sync(self):
        assert self.lib.sync() == B.PS_OK, self.lib.last_error()
        self.book.reap()
        self.data.reap()

    def step(self, q_all, out_all, reqs, budget):
        """One ps_step on the library; the checkers replay the same plan (the data checker layer by layer)."""
        rc, mask, st = self.lib.step(q_all, out_all, reqs, budget)
        assert rc == B.PS_OK, self.lib.last_error()
        plan = self.book.step_plan(budget)
        for req, lo, hi in plan:
            for l in range(self.sh.num_layers):
                assert self.book.swap_in_layer(req, l, lo, hi) == po.OK
            for l in range(len(self.sample_layers)):
                assert self.data.swap_in_layer(req, l, lo, hi) == po.OK
        omask = [1 if (r in self.book.reqs and self.book.reqs[r].state == po.ST_RESIDENT) else 0 for r in reqs]
        assert mask == omask
        assert st["blocks_copied"] == sum(hi - lo for _, lo, hi in plan)
        return mask, st, plan

    def assert_tables_equal(self, reqs):
        for r in reqs:
            assert self.lib.block_table(r) == self.book.block_table(r) == self.data.block_table(r), r
        assert self.lib.num_free_blocks() == self.book.num_free_blocks()

    def image_view(self, req) -> np.ndarray:
        """The library's host image as uint16 [L][n_blk][2][slab elements] (a view, no copy)."""
        ptr, nbytes = self.lib.host_image(req)
        n_blk = nbytes // self.sh.block_bytes
        buf = (C.c_uint16 * (nbytes // 2)).from_address(ptr)
        return np.ctypeslib.as_array(buf).reshape(self.sh.num_layers, n_blk, 2, self.sh.slab_elems)

    def assert_image_matches(self, req, extra_layers=()):
        """Sampled layers against the data checker byte for byte; extra layers against the device pools."""
        img = self.image_view(req)
        want = self.data.reqs[req].image
        for i, l in enumerate(self.sample_layers):
            assert np.array_equal(img[l].reshape(-1), want[i].reshape(-1)), (req, l)
        table = self.data.reqs[req].table or self.data.reqs[req].old_table
        for l in extra_layers:
            idx = torch.tensor(table, device="cuda")
            k = dev_to_bits(self.Kd[l][idx]).reshape(len(table), -1)
            v = dev_to_bits(self.Vd[l][idx]).reshape(len(table), -1)
            assert np.array_equal(img[l][:, 0], k) and np.array_equal(img[l][:, 1], v), (req, l)

    def assert_sampled_pools_equal(self):
        torch.cuda.synchronize()
        for i, l in enumerate(self.sample_layers):
            assert np.array_equal(dev_to_bits(self.Kd[l]), self.data.K[i]), f"K pool of layer {l} differs"
            assert np.array_equal(dev_to_bits(self.Vd[l]), self.data.V[i]), f"V pool of layer {l} differs"

    def logical_kv(self, req):
        """Device copy of a request's KV through its current table, all layers: (K, V) [L][n_blk][...]."""
        idx = torch.tensor(self.lib.block_table(req)[0], device="cuda")
        return self.Kd[:, idx].clone(), self.Vd[:, idx].clone()

    def block_sums(self):
        """Per (layer, block) 64-bit sums of the raw 16-bit patterns of K and V: [2][L][num_blocks]."""
        nb = self.sh.num_gpu_blocks
        out = torch.empty((2, self.sh.num_layers, nb), dtype=torch.int64, device="cuda")
        for t, pool in enumerate((self.Kd, self.Vd)):
            for l in range(self.sh.num_layers):
                out[t, l] = pool[l].view(torch.int16).view(nb, -1).sum(dim=1, dtype=torch.int64)
        return out

    def check_attention(self, out_all, q_all, reqs, mask, sample_reqs):
        """Rows of `sample_reqs` (positions in reqs) of the sampled layers against the fp64 checker."""
        rows = [i for i in sample_reqs if mask[i]]
        if not rows:
            return
        for i, l in enumerate(self.sample_layers):
            qb = dev_to_bits(q_all[l][rows])
            want, _ = self.data.decode_attn(i, qb, [reqs[r] for r in rows])
            check_attn(out_all[l][rows], want)

    def destroy(self):
        self.lib.destroy()
