"""Thin ctypes binding of libps_kvswap.so: argument marshalling only, same names as the C ABI.

Every step of the hot path (block bookkeeping, gather/scatter, transfers, attention, the step loop)
runs inside the library; this module converts Python values to pointers and sizes.  PyTorch appears
only as the owner of device memory and of the compute stream (`tensor.data_ptr()`,
`torch.cuda.current_stream().cuda_stream`).

The library must have been built (`python -m paper_2512_12928_b200.build`); loading fails loudly
otherwise.  There is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

_PKG = os.path.dirname(os.path.abspath(__file__))
# PS_KVSWAP_LIB selects another build of the same library (e.g. one with -G or extra checks)
LIB_PATH = os.environ.get("PS_KVSWAP_LIB") or os.path.join(_PKG, "lib", "libps_kvswap.so")

# status codes / states / flags (values fixed by include/ps_kvswap.h)
PS_OK, PS_ERR_INVALID, PS_ERR_NOMEM, PS_ERR_HOST_NOMEM = 0, -1, -2, -3
PS_ERR_STATE, PS_ERR_BUSY, PS_ERR_TIMEOUT, PS_ERR_CUDA, PS_ERR_BOUNDS = -4, -5, -6, -7, -8
PS_REQ_NONE, PS_REQ_RESIDENT, PS_REQ_SWAPPING_OUT, PS_REQ_HOST, PS_REQ_SWAPPING_IN = 0, 1, 2, 3, 4
PS_FLAG_BOOKKEEPING_ONLY, PS_FLAG_PROFILE, PS_FLAG_SYNC_RELOAD, PS_FLAG_ATTN_PLAIN_LAUNCH = 1, 2, 4, 8
PS_ATTN_AUTO, PS_ATTN_SIMT, PS_ATTN_MMA, PS_ATTN_MMA_ROWS = 0, 1, 2, 3

EXPORTS = [
    "ps_create", "ps_destroy", "ps_last_error", "ps_kv_alloc", "ps_kv_free", "ps_block_table",
    "ps_num_free_blocks", "ps_swap_out", "ps_host_image", "ps_swap_in_begin", "ps_swap_in_cancel",
    "ps_swap_in_layer", "ps_missing_blocks", "ps_decode_attn", "ps_step", "ps_poll", "ps_sync",
    "ps_launch_count", "ps_get_profile", "ps_link_probe", "ps_copy_blocks", "ps_trace", "ps_trace_read",
    "ps_decode_attn_static", "ps_copy_budget", "ps_offload_progress", "ps_host_blocks", "ps_host_segment",
    "ps_select_victims", "ps_copy_condition", "ps_order_queue", "ps_estimate_batch", "ps_resume_cost",
    "ps_reload_fence", "ps_offload_sweep", "ps_step_ruled", "ps_step_host", "ps_inject_status", "ps_hbm_probe", "ps_reload_backlog",
]


class PsConfig(C.Structure):
    _fields_ = [
        ("num_layers", C.c_int32), ("num_kv_heads", C.c_int32), ("num_q_heads", C.c_int32),
        ("head_dim", C.c_int32), ("block_size", C.c_int32), ("num_gpu_blocks", C.c_int32),
        ("max_blocks_per_req", C.c_int32), ("max_batch", C.c_int32), ("flags", C.c_int32),
        ("attn_kernel", C.c_int32), ("kv_split_tokens", C.c_int32), ("layer_chunk_bytes", C.c_int32),
        ("host_pool_bytes", C.c_int64), ("staging_bytes", C.c_int64),
        ("initial_free_order", C.POINTER(C.c_int32)),
    ]


class PsStepStats(C.Structure):
    _fields_ = [
        ("h2d_bytes", C.c_int64), ("blocks_copied", C.c_int64), ("reloads_completed", C.c_int32),
        ("swapouts_reaped", C.c_int32), ("decoded", C.c_int32), ("gated", C.c_int32),
        ("kernel_launches", C.c_int32), ("reserved0", C.c_int32),
    ]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_ if k != "reserved0"}


class PsProfile(C.Structure):
    _fields_ = [
        ("attn_ms", C.c_double), ("attn_launches", C.c_int64), ("attn_kv_bytes", C.c_int64),
        ("merge_ms", C.c_double), ("merge_launches", C.c_int64),
        ("gather_ms", C.c_double), ("gather_launches", C.c_int64), ("gather_bytes", C.c_int64),
        ("scatter_ms", C.c_double), ("scatter_launches", C.c_int64), ("scatter_bytes", C.c_int64),
        ("d2h_ms", C.c_double), ("d2h_copies", C.c_int64), ("d2h_bytes", C.c_int64),
        ("h2d_ms", C.c_double), ("h2d_copies", C.c_int64), ("h2d_bytes", C.c_int64),
    ]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class PsBudgetModel(C.Structure):
    _fields_ = [("a_d_us_per_token", C.c_double), ("b_d_us", C.c_double), ("t_c_us", C.c_double),
                ("t_block_us", C.c_double), ("t_budget_us", C.c_double)]


class PsCopyRule(C.Structure):
    _fields_ = [("beta", C.c_double), ("n", C.c_int32), ("reserved0", C.c_int32), ("reqs", C.POINTER(C.c_int64)),
                ("l_comp", C.POINTER(C.c_int32)), ("l_comp_max", C.POINTER(C.c_int32))]


class PsSchedParams(C.Structure):
    _fields_ = [("eta_us", C.c_double), ("gamma", C.c_double), ("t_c_us", C.c_double), ("tau_us", C.c_double)]


class PsLatencyModel(C.Structure):
    _fields_ = [("a_p_us", C.c_double), ("b_p_us", C.c_double), ("c_p_us", C.c_double),
                ("a_d_us", C.c_double), ("b_d_us", C.c_double), ("t_c_us", C.c_double)]


class PsTraceSpan(C.Structure):
    _fields_ = [("kind", C.c_int32), ("tag", C.c_int32), ("start_us", C.c_float), ("end_us", C.c_float)]


TRACE_KINDS = ["attn", "merge", "gather", "scatter", "d2h", "h2d"]


class PsError(RuntimeError):
    def __init__(self, code: int, where: str, text: str = ""):
        super().__init__(f"{where} failed with status {code}" + (f": {text}" if text else ""))
        self.code = code


_lib = None


def load() -> C.CDLL:
    """Loads the shared library and declares the prototypes.  Raises if it is not built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2512_12928_b200.build` "
            "(there is no fallback implementation)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    p32, p64 = C.POINTER(C.c_int32), C.POINTER(C.c_int64)
    proto = {
        "ps_create": (i32, [C.POINTER(PsConfig), C.POINTER(vp), C.POINTER(vp), vp, vp, C.POINTER(vp)]),
        "ps_destroy": (i32, [vp]),
        "ps_last_error": (C.c_char_p, [vp]),
        "ps_kv_alloc": (i32, [vp, i64, i32]),
        "ps_kv_free": (i32, [vp, i64]),
        "ps_block_table": (i32, [vp, i64, p32, i32, p32, p32, p32]),
        "ps_num_free_blocks": (i32, [vp, p32]),
        "ps_swap_out": (i32, [vp, i64]),
        "ps_host_image": (i32, [vp, i64, C.POINTER(vp), p64]),
        "ps_swap_in_begin": (i32, [vp, i64]),
        "ps_swap_in_cancel": (i32, [vp, i64]),
        "ps_swap_in_layer": (i32, [vp, i64, i32, i32, i32]),
        "ps_missing_blocks": (i32, [vp, i64, p32]),
        "ps_reload_fence": (i32, [vp, i32]),
        "ps_decode_attn": (i32, [vp, i32, vp, vp, vp, p64, i32]),
        "ps_step": (i32, [vp, vp, vp, p64, i32, i64, p32, C.POINTER(PsStepStats)]),
        "ps_poll": (i32, [vp, p32]),
        "ps_sync": (i32, [vp, i32]),
        "ps_launch_count": (i32, [vp, p64]),
        "ps_get_profile": (i32, [vp, C.POINTER(PsProfile), i32]),
        "ps_link_probe": (i32, [i64, i32, i32, C.POINTER(C.c_double)]),
        "ps_hbm_probe": (i32, [i64, i32, i32, C.POINTER(C.c_double)]),
        "ps_copy_blocks": (i32, [vp, i32, i32, p32, i32, vp, i32]),
        "ps_inject_status": (i32, [vp, i32]),
        "ps_reload_backlog": (i32, [vp, p64]),
        "ps_step_ruled": (i32, [vp, vp, vp, p64, i32, i64, C.POINTER(PsCopyRule), p32, C.POINTER(PsStepStats)]),
        "ps_step_host": (i32, [vp, vp, vp, p64, i32, i64, p32, C.POINTER(PsStepStats)]),
        "ps_trace": (i32, [vp, i32]),
        "ps_trace_read": (i32, [vp, C.POINTER(PsTraceSpan), i32, p32]),
        "ps_offload_progress": (i32, [vp, i64, i32, p32]),
        "ps_host_blocks": (i32, [vp, i64, p32, p32]),
        "ps_offload_sweep": (i32, [vp, p64, p32, i32, p64]),
        "ps_host_segment": (i32, [vp, i64, i32, C.POINTER(vp), p64, p32, p32, p32]),
        "ps_select_victims": (i32, [vp, p64, i32, C.POINTER(C.c_double), C.c_double, C.c_double, i32, p64, i32, p32, p32]),
        "ps_copy_condition": (i32, [i32, i32, i32, i32, i32, C.c_double, p32]),
        "ps_order_queue": (i32, [i32, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_double),
                                 C.POINTER(C.c_double), C.POINTER(PsSchedParams), p32, p32, C.POINTER(C.c_double)]),
        "ps_copy_budget": (i32, [vp, p64, i32, C.POINTER(PsBudgetModel), p64, p64, p32]),
        "ps_estimate_batch": (i32, [C.POINTER(PsLatencyModel), i32, p32, p32, i32, p32, C.POINTER(C.c_double)]),
        "ps_resume_cost": (i32, [C.POINTER(PsLatencyModel), i32, i32, i32, C.c_double, C.POINTER(C.c_double),
                                 C.POINTER(C.c_double)]),
        "ps_decode_attn_static": (i32, [vp, vp, vp, vp, vp, vp, i32, p32, i32, i32, i32, i32, i32, i32, i32, vp, vp,
                                        C.c_char_p, i32]),
    }
    for name, (res, args) in proto.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def ps_link_probe(nbytes: int, direction: int, iters: int = 10) -> float:
    """Pinned-copy host link rate in GB/s (1e9): 0 = H2D, 1 = D2H, 2 = both at once (sum)."""
    out = C.c_double(0.0)
    rc = load().ps_link_probe(nbytes, direction, iters, C.byref(out))
    if rc != PS_OK:
        raise PsError(rc, "ps_link_probe", load().ps_last_error(None).decode())
    return out.value


def ps_hbm_probe(nbytes: int, mode: int, iters: int = 5) -> float:
    """Device-memory rate of a plain streaming kernel in GB/s (1e9): 0 = read only, 1 = copy (read + written)."""
    out = C.c_double(0.0)
    rc = load().ps_hbm_probe(nbytes, mode, iters, C.byref(out))
    if rc != PS_OK:
        raise PsError(rc, "ps_hbm_probe", load().ps_last_error(None).decode())
    return out.value


PS_STATIC_MAX_BATCH = 256
PS_STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


def ps_decode_attn_static(kpool, vpool, q, out, block_tables, ctx_lens: Sequence[int], *, num_kv_heads: int,
                          num_q_heads: int, head_dim: int, block_size: int, num_gpu_blocks: int,
                          kv_split_tokens: int = 0, lse=None, status_word=None, stream: Optional[int] = None):
    """Decode attention with no context and no allocation (scratch is a fixed array inside the library).

    kpool, vpool, q, out, block_tables (int32 [batch][stride]), lse, status_word: device tensors;
    ctx_lens: host integers.  Returns (status, error text).  See ps_decode_attn_static in the header:
    calls on one device share the scratch, so overlapping calls on unordered streams race."""
    if stream is None:
        import torch
        stream = torch.cuda.current_stream().cuda_stream
    batch = len(ctx_lens)
    arr = (C.c_int32 * max(batch, 1))(*[int(v) for v in ctx_lens])
    err = C.create_string_buffer(512)
    ptr = lambda t: C.c_void_p(t.data_ptr()) if t is not None else None
    stride = int(block_tables.shape[-1]) if block_tables is not None and block_tables.dim() > 1 else 1
    rc = load().ps_decode_attn_static(ptr(kpool), ptr(vpool), ptr(q), ptr(out), ptr(lse), ptr(block_tables), stride,
                                      arr, batch, num_kv_heads, num_q_heads, head_dim, block_size, num_gpu_blocks,
                                      kv_split_tokens, ptr(status_word), C.c_void_p(stream or None), err, 512)
    return rc, err.value.decode()


def ps_order_queue(exec_us, remain_us, weight, *, eta: float, gamma: float, t_c: float, waited_us=None, tau: float = 0.0):
    """SlideBatching's queue order: (status, order as indices head first, classes per index, t_budget)."""
    n = len(exec_us)
    arr = lambda v: (C.c_double * max(n, 1))(*[float(x) for x in v])
    params = PsSchedParams(eta, gamma, t_c, tau)
    order, cls, tb = (C.c_int32 * max(n, 1))(), (C.c_int32 * max(n, 1))(), C.c_double()
    rc = load().ps_order_queue(n, arr(exec_us), arr(remain_us), arr(weight), arr(waited_us) if waited_us is not None else None,
                               C.byref(params), order, cls, C.byref(tb))
    return rc, list(order[:n]), list(cls[:n]), tb.value


def ps_copy_condition(l_comp: int, l_comp_max: int, b_miss: int, b_rem: int, s_blk: int, beta: float):
    """Partial-copy admission rule of Section 4.3: (status, allowed)."""
    out = C.c_int32()
    rc = load().ps_copy_condition(l_comp, l_comp_max, b_miss, b_rem, s_blk, beta, C.byref(out))
    return rc, bool(out.value)


def ps_estimate_batch(model: PsLatencyModel, prefill: Sequence[Tuple[int, int]], decode: Sequence[int]):
    """Batch latency estimate of Section 4.1: prefill = (l_q, l_kv) pairs, decode = l_kv values.  (status, us)."""
    i32s = lambda v: (C.c_int32 * max(len(v), 1))(*[int(x) for x in v])
    out = C.c_double()
    rc = load().ps_estimate_batch(C.byref(model), len(prefill), i32s([p[0] for p in prefill]),
                                  i32s([p[1] for p in prefill]), len(decode), i32s(decode), C.byref(out))
    return rc, out.value


def ps_resume_cost(model: PsLatencyModel, n_tokens: int, chunk_tokens: int, s_blk: int, t_block_us: float):
    """Reload versus recompute of an evicted request: (status, reload_us, recompute_us)."""
    reload_us, recompute_us = C.c_double(), C.c_double()
    rc = load().ps_resume_cost(C.byref(model), n_tokens, chunk_tokens, s_blk, t_block_us, C.byref(reload_us),
                               C.byref(recompute_us))
    return rc, reload_us.value, recompute_us.value


def _i64_array(vals: Sequence[int]):
    return (C.c_int64 * max(len(vals), 1))(*[int(v) for v in vals])


class KVSwap:
    """One library context.  Methods carry the C entry points' names without the `ps_` prefix and
    return the raw status code where the call can legitimately fail (so a test script can drive the
    library and a checker side by side); `check=True` variants raise instead."""

    def __init__(self, *, num_layers: int, num_kv_heads: int, num_q_heads: int, head_dim: int, block_size: int,
                 num_gpu_blocks: int, max_blocks_per_req: int, max_batch: int = 0, host_pool_bytes: int = 0,
                 staging_bytes: int = 0, initial_free_order=None, k_pools=None, v_pools=None, flags: int = 0,
                 attn_kernel: int = PS_ATTN_AUTO, kv_split_tokens: int = 0, host_pool_ptr: int = 0,
                 compute_stream: Optional[int] = None, layer_chunk_bytes: int = 0):
        self.lib = load()
        self.L = num_layers
        self.Hq, self.D = num_q_heads, head_dim
        cfg = PsConfig()
        cfg.num_layers, cfg.num_kv_heads, cfg.num_q_heads = num_layers, num_kv_heads, num_q_heads
        cfg.head_dim, cfg.block_size, cfg.num_gpu_blocks = head_dim, block_size, num_gpu_blocks
        cfg.max_blocks_per_req, cfg.max_batch, cfg.flags = max_blocks_per_req, max_batch, flags
        cfg.attn_kernel, cfg.kv_split_tokens = attn_kernel, kv_split_tokens
        cfg.layer_chunk_bytes = layer_chunk_bytes
        cfg.host_pool_bytes, cfg.staging_bytes = host_pool_bytes, staging_bytes
        self._order = None
        if initial_free_order is not None:
            self._order = (C.c_int32 * num_gpu_blocks)(*[int(v) for v in initial_free_order])
            cfg.initial_free_order = C.cast(self._order, C.POINTER(C.c_int32))
        self._pools = (k_pools, v_pools)      # keep the tensors alive
        kp = vp = None
        if not (flags & PS_FLAG_BOOKKEEPING_ONLY):
            if k_pools is None or v_pools is None or len(k_pools) != num_layers or len(v_pools) != num_layers:
                raise ValueError("k_pools and v_pools must be lists of num_layers device tensors")
            kp = (C.c_void_p * num_layers)(*[t.data_ptr() for t in k_pools])
            vp = (C.c_void_p * num_layers)(*[t.data_ptr() for t in v_pools])
            if compute_stream is None:
                import torch
                compute_stream = torch.cuda.current_stream().cuda_stream
        self.compute_stream = compute_stream or 0
        handle = C.c_void_p()
        rc = self.lib.ps_create(C.byref(cfg), kp, vp, C.c_void_p(host_pool_ptr or None),
                                C.c_void_p(self.compute_stream or None), C.byref(handle))
        if rc != PS_OK:
            raise PsError(rc, "ps_create", self.lib.ps_last_error(None).decode())
        self.h = handle

    # ---- lifetime
    def destroy(self) -> None:
        if getattr(self, "h", None):
            self.lib.ps_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def last_error(self) -> str:
        return self.lib.ps_last_error(self.h).decode()

    def _ck(self, rc: int, where: str) -> int:
        if rc != PS_OK:
            raise PsError(rc, where, self.last_error())
        return rc

    # ---- pool
    def kv_alloc(self, req: int, n_tokens_total: int) -> int:
        return self.lib.ps_kv_alloc(self.h, req, n_tokens_total)

    def kv_free(self, req: int) -> int:
        return self.lib.ps_kv_free(self.h, req)

    def block_table(self, req: int) -> Tuple[List[int], int]:
        n, st, nt = C.c_int32(), C.c_int32(), C.c_int32()
        self._ck(self.lib.ps_block_table(self.h, req, None, 0, C.byref(n), C.byref(st), C.byref(nt)), "ps_block_table")
        ids = (C.c_int32 * max(n.value, 1))()
        self._ck(self.lib.ps_block_table(self.h, req, ids, n.value, None, None, None), "ps_block_table")
        return list(ids[: n.value]), st.value

    def req_state(self, req: int) -> int:
        """ps_req_state of the request, PS_REQ_NONE for an unknown one (no table is copied)."""
        st = C.c_int32()
        rc = self.lib.ps_block_table(self.h, req, None, 0, None, C.byref(st), None)
        return st.value if rc == PS_OK else PS_REQ_NONE

    def n_tokens(self, req: int) -> int:
        nt = C.c_int32()
        self._ck(self.lib.ps_block_table(self.h, req, None, 0, None, None, C.byref(nt)), "ps_block_table")
        return nt.value

    def num_free_blocks(self) -> int:
        out = C.c_int32()
        self._ck(self.lib.ps_num_free_blocks(self.h, C.byref(out)), "ps_num_free_blocks")
        return out.value

    # ---- swap
    def swap_out(self, req: int) -> int:
        return self.lib.ps_swap_out(self.h, req)

    def host_image(self, req: int) -> Tuple[int, int]:
        ptr, nbytes = C.c_void_p(), C.c_int64()
        self._ck(self.lib.ps_host_image(self.h, req, C.byref(ptr), C.byref(nbytes)), "ps_host_image")
        return ptr.value or 0, nbytes.value

    def offload_progress(self, req: int, n_off: int):
        """Proactive offload of whole groups of n_off filled blocks: (status, blocks issued)."""
        n = C.c_int32()
        rc = self.lib.ps_offload_progress(self.h, req, n_off, C.byref(n))
        return rc, n.value

    def offload_sweep(self, reqs: Sequence[int], n_off: Sequence[int]):
        """Proactive offload over a batch with per-request thresholds: (status, blocks issued)."""
        total = C.c_int64()
        thr = (C.c_int32 * max(len(n_off), 1))(*[int(v) for v in n_off])
        rc = self.lib.ps_offload_sweep(self.h, _i64_array(reqs), thr, len(reqs), C.byref(total))
        return rc, total.value

    def host_blocks(self, req: int) -> Tuple[int, int]:
        a, b = C.c_int32(), C.c_int32()
        self._ck(self.lib.ps_host_blocks(self.h, req, C.byref(a), C.byref(b)), "ps_host_blocks")
        return a.value, b.value

    def host_segments(self, req: int):
        """List of (address, bytes, blk_lo, blk_hi) of the request's image segments."""
        n = C.c_int32()
        self._ck(self.lib.ps_host_segment(self.h, req, -1, None, None, None, None, C.byref(n)), "ps_host_segment")
        out = []
        for i in range(n.value):
            ptr, nbytes, lo, hi = C.c_void_p(), C.c_int64(), C.c_int32(), C.c_int32()
            self._ck(self.lib.ps_host_segment(self.h, req, i, C.byref(ptr), C.byref(nbytes), C.byref(lo), C.byref(hi),
                                              None), "ps_host_segment")
            out.append((ptr.value or 0, nbytes.value, lo.value, hi.value))
        return out

    def swap_in_begin(self, req: int) -> int:
        return self.lib.ps_swap_in_begin(self.h, req)

    def swap_in_cancel(self, req: int) -> int:
        return self.lib.ps_swap_in_cancel(self.h, req)

    def swap_in_layer(self, req: int, layer: int, blk_lo: int, blk_hi: int) -> int:
        return self.lib.ps_swap_in_layer(self.h, req, layer, blk_lo, blk_hi)

    def reload_fence(self, layer: int = -1) -> int:
        return self.lib.ps_reload_fence(self.h, layer)

    def missing_blocks(self, req: int) -> int:
        out = C.c_int32()
        self._ck(self.lib.ps_missing_blocks(self.h, req, C.byref(out)), "ps_missing_blocks")
        return out.value

    # ---- attention / step
    def decode_attn(self, layer: int, q, out, reqs: Sequence[int], lse=None) -> int:
        """q, out: device bf16 tensors [B][Hq][D]; lse: device fp32 [B][Hq] or None."""
        arr = _i64_array(reqs)
        return self.lib.ps_decode_attn(self.h, layer, C.c_void_p(q.data_ptr()), C.c_void_p(out.data_ptr()),
                                       C.c_void_p(lse.data_ptr()) if lse is not None else None, arr, len(reqs))

    def step(self, q_all, out_all, reqs: Sequence[int], copy_budget_bytes: int):
        """Returns (status, decoded mask list, stats dict).  q_all/out_all: device bf16 [L][B][Hq][D] or None."""
        arr = _i64_array(reqs)
        mask = (C.c_int32 * max(len(reqs), 1))()
        st = PsStepStats()
        rc = self.lib.ps_step(self.h, C.c_void_p(q_all.data_ptr()) if q_all is not None else None,
                              C.c_void_p(out_all.data_ptr()) if out_all is not None else None, arr, len(reqs),
                              copy_budget_bytes, mask, C.byref(st))
        return rc, list(mask[: len(reqs)]), st.as_dict()

    def step_ruled(self, q_all, out_all, reqs: Sequence[int], copy_budget_bytes: int, beta: float,
                   rule_reqs: Sequence[int], l_comp: Sequence[int], l_comp_max: Sequence[int]):
        """ps_step with the partial-copy admission test: (status, decoded mask list, stats dict)."""
        arr = _i64_array(reqs)
        mask = (C.c_int32 * max(len(reqs), 1))()
        st = PsStepStats()
        n = len(rule_reqs)
        rr = _i64_array(rule_reqs)
        lc = (C.c_int32 * max(n, 1))(*[int(v) for v in l_comp])
        lm = (C.c_int32 * max(n, 1))(*[int(v) for v in l_comp_max])
        rule = PsCopyRule(beta, n, 0, C.cast(rr, C.POINTER(C.c_int64)), C.cast(lc, C.POINTER(C.c_int32)),
                          C.cast(lm, C.POINTER(C.c_int32)))
        rc = self.lib.ps_step_ruled(self.h, C.c_void_p(q_all.data_ptr()) if q_all is not None else None,
                                    C.c_void_p(out_all.data_ptr()) if out_all is not None else None, arr, len(reqs),
                                    copy_budget_bytes, C.byref(rule), mask, C.byref(st))
        return rc, list(mask[: len(reqs)]), st.as_dict()

    def step_host(self, q_host, out_host, reqs: Sequence[int], copy_budget_bytes: int):
        """ps_step with queries and outputs in host memory (tensors with data_ptr(), e.g. pinned CPU tensors):
        (status, decoded mask list, stats dict).  Asynchronous: synchronise the compute stream before reading."""
        arr = _i64_array(reqs)
        mask = (C.c_int32 * max(len(reqs), 1))()
        st = PsStepStats()
        rc = self.lib.ps_step_host(self.h, C.c_void_p(q_host.data_ptr()), C.c_void_p(out_host.data_ptr()), arr,
                                   len(reqs), copy_budget_bytes, mask, C.byref(st))
        return rc, list(mask[: len(reqs)]), st.as_dict()

    def reload_backlog(self) -> int:
        """Reload bytes issued by earlier steps whose copies have not been seen complete."""
        out = C.c_int64()
        self._ck(self.lib.ps_reload_backlog(self.h, C.byref(out)), "ps_reload_backlog")
        return out.value

    def inject_status(self, value: int) -> int:
        return self.lib.ps_inject_status(self.h, value)

    def copy_budget(self, reqs: Sequence[int], *, a_d: float, b_d: float, t_c: float, t_block: float, t_budget: float):
        """Adaptive copy budget for the coming step: (status, blocks, bytes, case 1 / 21 / 22); times in us."""
        m = PsBudgetModel(a_d, b_d, t_c, t_block, t_budget)
        blocks, nbytes, case = C.c_int64(), C.c_int64(), C.c_int32()
        rc = self.lib.ps_copy_budget(self.h, _i64_array(reqs), len(reqs), C.byref(m), C.byref(blocks), C.byref(nbytes),
                                     C.byref(case))
        return rc, blocks.value, nbytes.value, case.value

    def select_victims(self, queue: Sequence[int], waited_us: Sequence[float], tau_us: float, near_frac: float,
                       blocks_needed: int):
        """Eviction policy: (status, victims in eviction order, blocks they free)."""
        n = len(queue)
        w = (C.c_double * max(n, 1))(*[float(v) for v in waited_us])
        out = (C.c_int64 * max(n, 1))()
        cnt, freed = C.c_int32(), C.c_int32()
        rc = self.lib.ps_select_victims(self.h, _i64_array(queue), n, w, tau_us, near_frac, blocks_needed, out, n,
                                        C.byref(cnt), C.byref(freed))
        return rc, list(out[: cnt.value]), freed.value

    # ---- completion
    def poll(self) -> int:
        n = C.c_int32()
        self._ck(self.lib.ps_poll(self.h, C.byref(n)), "ps_poll")
        return n.value

    def sync(self, timeout_ms: int = 120000) -> int:
        return self.lib.ps_sync(self.h, timeout_ms)

    # ---- measurement
    def launch_count(self) -> int:
        out = C.c_int64()
        self._ck(self.lib.ps_launch_count(self.h, C.byref(out)), "ps_launch_count")
        return out.value

    def get_profile(self, reset: bool = False) -> dict:
        p = PsProfile()
        self._ck(self.lib.ps_get_profile(self.h, C.byref(p), 1 if reset else 0), "ps_get_profile")
        return p.as_dict()

    def trace(self, enable: bool) -> int:
        return self.lib.ps_trace(self.h, 1 if enable else 0)

    def trace_read(self):
        """List of (kind name, tag, start_us, end_us), call after sync()."""
        n = C.c_int32()
        self._ck(self.lib.ps_trace_read(self.h, None, 0, C.byref(n)), "ps_trace_read")
        buf = (PsTraceSpan * max(n.value, 1))()
        self._ck(self.lib.ps_trace_read(self.h, buf, n.value, C.byref(n)), "ps_trace_read")
        return [(TRACE_KINDS[s.kind], s.tag, s.start_us, s.end_us) for s in buf[: n.value]]

    def copy_blocks(self, layer: int, ids: Sequence[int], staging, direction: int, n_layers: int = 1) -> int:
        arr = (C.c_int32 * max(len(ids), 1))(*[int(v) for v in ids])
        return self.lib.ps_copy_blocks(self.h, layer, n_layers, arr, len(ids), C.c_void_p(staging.data_ptr()), direction)
