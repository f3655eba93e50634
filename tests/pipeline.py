"""Helpers for the parity tests: run one stage through the C-ABI binding on the
GPU, and the same stage through the fp64 oracle on the CPU, on the same seeded
host arrays.  Nothing flows from the GPU side into the oracle side."""
from __future__ import annotations

import numpy as np
import torch

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl


def f64(t):
    if isinstance(t, torch.Tensor):
        return t.detach().to("cpu").to(torch.float64).numpy()
    return np.asarray(t, dtype=np.float64)


def dev(x, dtype=None):
    if isinstance(x, np.ndarray):
        x = torch.from_numpy(np.ascontiguousarray(x))
    x = x.to("cuda")
    return x.to(dtype) if dtype is not None else x.contiguous()


def make_ctx(shape: wl.Shape, max_pos=8192):
    from paper_2608_19662_b200 import ReCache
    return ReCache(shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.rope_theta, shape.dtype,
                   max_pos=max_pos, page_tokens=wl.PAGE_TOKENS)


# ------------------------------------------------------------------ GPU side --
def gpu_encode(rc, pool: wl.ResourceBatch, out_dtype=torch.float32, caches=None, nan_fill=True):
    sh = pool.shape
    if caches is None:
        kc = torch.empty((sh.n_kv_heads, pool.pool_tokens, sh.head_dim), dtype=sh.torch_dtype, device="cuda")
        vc = torch.empty_like(kc)
        if nan_fill:       # unwritten cache rows must never reach a result
            kc.fill_(float("nan")); vc.fill_(float("nan"))
    else:
        kc, vc = caches
    o = rc.encode_resources(dev(pool.q), dev(pool.k), dev(pool.v), dev(pool.cu_seqlens), pool.max_len,
                            dev(pool.dst_slot), kc, vc, out_dtype=out_dtype)
    return o, kc, vc


def gpu_compact(rc, pool, req, kc, vc, mode=0, capacity=None, n_pool_pages=None, free_pages=None,
                max_pages=None):
    from paper_2608_19662_b200 import PAGED
    sh = pool.shape
    n_routes = req.n_requests * sh.n_kv_heads
    if capacity is None:
        capacity = int(req.res_len.sum()) * 1 + 1      # a route can never hold more than its request lists
        capacity = max(capacity * sh.n_kv_heads, 1)
    route_cu = torch.full((n_routes + 1,), -7, dtype=torch.int32, device="cuda")
    route_len = torch.full((n_routes,), -7, dtype=torch.int32, device="cuda")
    route_idx = torch.full((capacity,), -7, dtype=torch.int32, device="cuda")
    out = dict(route_cu=route_cu, route_len=route_len, route_idx=route_idx)
    if mode == PAGED:
        pt = wl.PAGE_TOKENS
        k_out = torch.full((n_pool_pages, pt, sh.head_dim), float("nan"), dtype=sh.torch_dtype, device="cuda")
        v_out = torch.full_like(k_out, float("nan"))
        page_table = torch.full((n_routes, max_pages), -7, dtype=torch.int32, device="cuda")
        fp = dev(np.asarray(free_pages, dtype=np.int32))
        rc.compact_routes(kc, vc, dev(pool.keep), dev(req.res_off), dev(req.res_slot), dev(req.res_len),
                          dev(req.vis), mode, route_cu, route_idx, k_out, v_out, route_len=route_len,
                          page_table=page_table, free_pages=fp)
        out.update(page_table=page_table)
    else:
        k_out = torch.full((capacity, sh.head_dim), float("nan"), dtype=sh.torch_dtype, device="cuda")
        v_out = torch.full_like(k_out, float("nan"))
        rc.compact_routes(kc, vc, dev(pool.keep), dev(req.res_off), dev(req.res_slot), dev(req.res_len),
                          dev(req.vis), mode, route_cu, route_idx, k_out, v_out, route_len=route_len)
    out.update(k_out=k_out, v_out=v_out)
    return out


def gpu_prefill(rc, req, k_route, v_route, route_cu, out_dtype=torch.float32):
    return rc.attend_prefill(dev(req.q), dev(req.k_conv), dev(req.v_conv), dev(req.cu_q), dev(req.q_pos0),
                             req.max_q, k_route, v_route, route_cu, out_dtype=out_dtype)


# --------------------------------------------------------------- oracle side --
def oracle_encode(pool: wl.ResourceBatch, round_q: bool = True):
    sh = pool.shape
    o, k_hat, v = orc.encode_resources(f64(pool.q), f64(pool.k), f64(pool.v), pool.cu_seqlens, sh.rope_theta,
                                       storage=sh.dtype, round_q=round_q)
    kc = np.full((sh.n_kv_heads, pool.pool_tokens, sh.head_dim), np.nan)
    vc = np.full_like(kc, np.nan)
    orc.write_cache(kc, vc, k_hat, v, pool.cu_seqlens, pool.dst_slot)
    return o, kc, vc


def oracle_cache_only(pool: wl.ResourceBatch):
    """Rotated keys / values in cache layout without the attention (cheap)."""
    sh = pool.shape
    k_hat = np.zeros(tuple(pool.k.shape))
    kk = f64(pool.k)
    for i in range(len(pool.lens)):
        a, b = int(pool.cu_seqlens[i]), int(pool.cu_seqlens[i + 1])
        if b > a:
            k_hat[a:b] = orc.rope(kk[a:b], np.arange(b - a), sh.rope_theta)
    k_hat = orc.round_storage(k_hat, sh.dtype)
    kc = np.full((sh.n_kv_heads, pool.pool_tokens, sh.head_dim), np.nan)
    vc = np.full_like(kc, np.nan)
    orc.write_cache(kc, vc, k_hat, f64(pool.v), pool.cu_seqlens, pool.dst_slot)
    return kc, vc


def oracle_rows(pool, req):
    return orc.compact_routes(pool.keep, req.res_off, req.res_slot, req.res_len, req.vis)


def oracle_prefill(req, rows, kc, vc, round_q: bool = True):
    sh = req.shape
    return orc.attend_prefill(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0, rows, kc, vc,
                              sh.rope_theta, storage=sh.dtype, round_q=round_q)


# ---------------------------------------------------------------- comparisons --
def report_readings(case: str, stage: str, gated: float, unrounded: float):
    """The parity gate compares with the oracle whose rotated query is rounded to
    the storage dtype (what the kernels compute).  Beside it, the error against
    the oracle that keeps the rotated query exact (cached keys as stored) is
    printed, and appended to the file RECACHE_PARITY_REPORT names, so that the
    share of the tolerance the reading consumes is on record per case."""
    import os
    line = f"{case:28s} {stage:8s} max|gpu-oracle| = {gated:.3e}   vs oracle with unrounded query = {unrounded:.3e}"
    print(line)
    path = os.environ.get("RECACHE_PARITY_REPORT")
    if path:
        with open(path, "a") as f:
            f.write(line + "\n")


def max_abs(a, b):
    a, b = f64(a), f64(b)
    return float(np.abs(a - b).max()) if a.size else 0.0


def bf16_ulp_distance(a: torch.Tensor, b64: np.ndarray) -> np.ndarray:
    """|a - b| in units of bf16 ulps of b (a is a bf16 tensor, b exact bf16 values as fp64)."""
    a64 = f64(a)
    _, e = np.frexp(np.where(b64 == 0, 1.0, b64))
    ulp = np.ldexp(1.0, e - 8)
    return np.abs(a64 - b64) / ulp


def sample_rows(rng, cu, n_heads, n_samples, extra_tokens=()):
    """Seeded (token, head) sample that always holds every sequence's first and last row."""
    cu = np.asarray(cu)
    toks = set(int(t) for t in extra_tokens)
    for i in range(len(cu) - 1):
        if cu[i + 1] > cu[i]:
            toks.update([int(cu[i]), int(cu[i + 1] - 1)])
    rows = [(t, int(rng.integers(0, n_heads))) for t in sorted(toks)]
    total = int(cu[-1])
    while len(rows) < n_samples:
        rows.append((int(rng.integers(0, total)), int(rng.integers(0, n_heads))))
    return rows
