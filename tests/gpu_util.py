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
                 max_blocks_per_req=None):
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
                            attn_kernel=attn_kernel, kv_split_tokens=kv_split_tokens)
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
