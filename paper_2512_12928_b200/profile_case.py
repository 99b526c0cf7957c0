"""Small, self-contained cases of the three kernels for profilers and quick timing.

    python -m paper_2512_12928_b200.profile_case attn    [--iters N] [--batch B] [--ctx T] [--q-heads H] [--kv-heads H] [--simt | --rows]
    python -m paper_2512_12928_b200.profile_case gather  [--iters N] [--blocks K] [--layers L] [--chunk-layers G]
    python -m paper_2512_12928_b200.profile_case scatter [--iters N] [--blocks K] [--layers L] [--chunk-layers G]

gather / scatter launch the kernels of the swap path (gather_image_kernel, scatter_image_kernel) through
ps_copy_blocks: K blocks of G consecutive layers per launch, the shape of a staging slot (large K) or of a
reload's layer chunk under a small copy budget (small K, G > 1).

The cases keep the Llama-3-8B KV shape (8 KV heads, head_dim 128, block 16) but only two layers and
a pool of a few GiB, so that a profiler that saves and restores device memory between passes stays
cheap, while one launch still moves more bytes than the 126 MB L2 holds.  Each run prints the
CUDA-event time per launch (launches are enqueued back to back so the GPU never waits for the host).
"""
from __future__ import annotations

import argparse
import ctypes as C
import json

import numpy as np
import torch

from . import binding as B
from . import workloads as wl


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["attn", "gather", "scatter"])
    ap.add_argument("--iters", type=int, default=6)
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--ctx", type=int, default=2048)
    ap.add_argument("--q-heads", type=int, default=32)
    ap.add_argument("--kv-heads", type=int, default=8)
    ap.add_argument("--blocks", type=int, default=2048)
    ap.add_argument("--layers", type=int, default=2, help="layers of the case's pools")
    ap.add_argument("--chunk-layers", type=int, default=1, help="gather / scatter: layers moved by one launch")
    ap.add_argument("--simt", action="store_true")
    ap.add_argument("--rows", action="store_true", help="tensor-core kernel fed by per-row bulk copies")
    args = ap.parse_args()

    L, Hkv, D, S = max(args.layers, args.chunk_layers), args.kv_heads, 128, 16
    nblk_req = (args.ctx + S - 1) // S
    nb = max(args.batch * nblk_req + 64, 2 * args.blocks + 64)
    sh = wl.KVShape(L, Hkv, args.q_heads, D, S, nb)
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    K = torch.empty((L, nb, S, Hkv, D), dtype=torch.bfloat16, device="cuda").normal_(generator=g)
    V = torch.empty_like(K).normal_(generator=g)
    order = np.random.default_rng(1).permutation(nb)
    lib = B.KVSwap(num_layers=L, num_kv_heads=Hkv, num_q_heads=args.q_heads, head_dim=D, block_size=S,
                   num_gpu_blocks=nb, max_blocks_per_req=nblk_req + 1, max_batch=args.batch, host_pool_bytes=1 << 20,
                   initial_free_order=order, k_pools=[K[l] for l in range(L)], v_pools=[V[l] for l in range(L)],
                   attn_kernel=B.PS_ATTN_SIMT if args.simt else B.PS_ATTN_MMA_ROWS if args.rows else B.PS_ATTN_AUTO)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    res = {"case": args.case}
    if args.case == "attn":
        grown = 0
        while grown < args.ctx:                       # interleaved growth: fragmented block tables
            grown = min(args.ctx, grown + S)
            for r in range(args.batch):
                assert lib.kv_alloc(r, grown) == 0, lib.last_error()
        reqs = list(range(args.batch))
        q = torch.randn((L, args.batch, args.q_heads, D), generator=g, device="cuda").to(torch.bfloat16)
        out = torch.zeros_like(q)
        for i in range(3):
            assert lib.decode_attn(i % L, q[i % L], out[i % L], reqs) == 0, lib.last_error()
        torch.cuda.synchronize()
        e0.record()
        for i in range(args.iters):
            assert lib.decode_attn(i % L, q[i % L], out[i % L], reqs) == 0, lib.last_error()
        e1.record()
        e1.synchronize()
        ms = e0.elapsed_time(e1) / args.iters
        kv_bytes = args.batch * args.ctx * 2 * Hkv * D * 2
        res.update(us_per_launch=ms * 1e3, kv_bytes_per_launch=kv_bytes, gb_per_s=kv_bytes / ms / 1e6,
                   batch=args.batch, ctx=args.ctx, q_heads=args.q_heads, kv_heads=Hkv, kernel="simt" if args.simt else "mma_rows" if args.rows else "auto")
    else:
        direction = 0 if args.case == "gather" else 1
        ids = np.random.default_rng(2).permutation(nb)[: args.blocks].astype(np.int32)
        arr = (C.c_int32 * args.blocks)(*[int(v) for v in ids])
        nl = args.chunk_layers
        stage = torch.zeros((nl, args.blocks, 2, S, Hkv, D), dtype=torch.bfloat16, device="cuda")
        for i in range(3):
            assert lib.lib.ps_copy_blocks(lib.h, (i % (L - nl + 1)), nl, arr, args.blocks, C.c_void_p(stage.data_ptr()), direction) == 0
        torch.cuda.synchronize()
        e0.record()
        for i in range(args.iters):
            assert lib.lib.ps_copy_blocks(lib.h, (i % (L - nl + 1)), nl, arr, args.blocks, C.c_void_p(stage.data_ptr()), direction) == 0
        e1.record()
        e1.synchronize()
        ms = e0.elapsed_time(e1) / args.iters
        payload = nl * args.blocks * sh.layer_block_bytes
        res.update(us_per_launch=ms * 1e3, payload_bytes_per_launch=payload, gb_per_s_read_plus_write=2 * payload / ms / 1e6,
                   blocks=args.blocks, chunk_layers=nl,
                   kernel="gather_image_kernel" if direction == 0 else "scatter_image_kernel")
    assert lib.sync() == 0, lib.last_error()
    lib.destroy()
    print(json.dumps(res))


if __name__ == "__main__":
    main()
