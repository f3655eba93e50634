"""Seeded synthetic inputs for resource-routed attention.

This module holds no arithmetic of the method: it only draws lengths, masks,
route tables and N(0,1) tensors from seeded generators and hands the same host
arrays to whoever asks (the CUDA binding, the tests, the benchmark).  It imports
neither the CUDA extension nor the CPU oracle.

Shapes follow the five workloads the build is measured on (Qwen3-class
attention shapes: 32 query heads, 8 KV-head groups, head_dim 128; a tiny fp32
case with 4/2 heads and head_dim 64).  Nothing here comes from a dataset.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

PAGE_TOKENS = 64


@dataclass
class Shape:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    rope_theta: float
    dtype: str  # "f32" | "bf16"

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def group_size(self) -> int:
        return self.n_q_heads // self.n_kv_heads


QWEN3_4B = Shape(32, 8, 128, 1.0e6, "bf16")
TINY_F32 = Shape(4, 2, 64, 1.0e4, "f32")


def _tgen(seed: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def normal(seed: int, shape, dtype: torch.dtype) -> torch.Tensor:
    """N(0,1) drawn in fp32 on the host, rounded once to the storage dtype."""
    return torch.randn(*shape, generator=_tgen(seed), dtype=torch.float32).to(dtype)


def uniform_lengths(rng: np.random.Generator, n: int, lo: int, hi: int) -> np.ndarray:
    return rng.integers(lo, hi + 1, size=n).astype(np.int32)


def keep_mask_bernoulli(rng, lens, p: float, force: str = "first") -> List[np.ndarray]:
    out = []
    for n in lens:
        m = (rng.random(int(n)) < p).astype(np.uint8)
        if n > 0:
            m[0 if force == "first" else -1] = 1
        out.append(m)
    return out


def keep_mask_spans(rng, lens, span=(4, 32), gap=(10, 74), force_last=True) -> List[np.ndarray]:
    """Kept tokens come as contiguous field spans separated by dropped gaps.

    Mean span 18 against mean gap 42 gives a keep ratio near 30 %.  The final
    token of every resource is kept (the suffix-token rule)."""
    out = []
    for n in lens:
        n = int(n)
        m = np.zeros(n, dtype=np.uint8)
        pos = int(rng.integers(0, gap[1] + 1))  # start somewhere inside a gap
        while pos < n:
            ln = int(rng.integers(span[0], span[1] + 1))
            m[pos:pos + ln] = 1
            pos += ln + int(rng.integers(gap[0], gap[1] + 1))
        if force_last and n > 0:
            m[-1] = 1
        out.append(m)
    return out


def routes_random(rng, n_groups: int, n_res: int, frac: float) -> np.ndarray:
    """vis[g][r] = 1 for exactly max(1, round(frac * n_res)) resources per group."""
    k = max(1, int(np.floor(frac * n_res + 0.5)))
    vis = np.zeros((n_groups, n_res), dtype=np.uint8)
    for g in range(n_groups):
        vis[g, rng.choice(n_res, size=min(k, n_res), replace=False)] = 1
    return vis


def routes_product(n_layers: int, n_groups: int, layers, groups) -> np.ndarray:
    """The structured case: a route (l, g) sees every resource or none."""
    om = np.zeros((n_layers, n_groups), dtype=np.uint8)
    for l in layers:
        for g in groups:
            om[l, g] = 1
    return om


# --------------------------------------------------------------------------
# Resource pool: what gets encoded once and cached.
# --------------------------------------------------------------------------
@dataclass
class ResourceBatch:
    """N resources packed back to back, pre-RoPE projections of one layer."""
    shape: Shape
    lens: np.ndarray            # [N] int32
    cu_seqlens: np.ndarray      # [N+1] int32
    dst_slot: np.ndarray        # [N] int32 first cache row of each resource
    pool_tokens: int
    q: torch.Tensor             # [T, Hq, d]
    k: torch.Tensor             # [T, G, d]
    v: torch.Tensor             # [T, G, d]
    keep: np.ndarray            # [pool_tokens] uint8 (by cache row)

    @property
    def total_tokens(self) -> int:
        return int(self.cu_seqlens[-1])

    @property
    def max_len(self) -> int:
        return int(self.lens.max()) if len(self.lens) else 0


def resource_tensors(seed: int, res_id: int, length: int, shape: Shape, layer: int = 0):
    """q/k/v of ONE pool resource; a function of (seed, layer, res_id) only, so
    the same resource carries the same data in every composition."""
    base = (seed * 1000003 + layer * 7919 + res_id) * 4
    q = normal(base + 0, (length, shape.n_q_heads, shape.head_dim), shape.torch_dtype)
    k = normal(base + 1, (length, shape.n_kv_heads, shape.head_dim), shape.torch_dtype)
    v = normal(base + 2, (length, shape.n_kv_heads, shape.head_dim), shape.torch_dtype)
    return q, k, v


def pack_resources(shape: Shape, seed: int, lens, keep_masks, res_ids=None, layer: int = 0,
                   slot_gap: int = 0, bulk: bool = False) -> ResourceBatch:
    """Pack resources back to back.  Cache slots follow the same order with an
    optional gap of unused rows between resources.  `bulk=True` draws the whole
    batch from one stream (fast, for the large benchmark shapes); otherwise each
    resource has its own stream keyed by res_id."""
    lens = np.asarray(lens, dtype=np.int32)
    n = len(lens)
    res_ids = list(range(n)) if res_ids is None else list(res_ids)
    cu = np.zeros(n + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    t = int(cu[-1])
    slot = np.zeros(n, dtype=np.int32)
    cur = 0
    for i in range(n):
        slot[i] = cur
        cur += int(lens[i]) + slot_gap
    pool = max(cur, 1)
    if bulk:
        q = normal(seed * 4 + 0, (t, shape.n_q_heads, shape.head_dim), shape.torch_dtype)
        k = normal(seed * 4 + 1, (t, shape.n_kv_heads, shape.head_dim), shape.torch_dtype)
        v = normal(seed * 4 + 2, (t, shape.n_kv_heads, shape.head_dim), shape.torch_dtype)
    else:
        parts = [resource_tensors(seed, rid, int(l), shape, layer) for rid, l in zip(res_ids, lens)]
        cat = lambda j, h: (torch.cat([p[j] for p in parts], 0) if parts else
                            torch.zeros(0, h, shape.head_dim, dtype=shape.torch_dtype))
        q, k, v = cat(0, shape.n_q_heads), cat(1, shape.n_kv_heads), cat(2, shape.n_kv_heads)
    keep = np.zeros(pool, dtype=np.uint8)
    for i in range(n):
        keep[slot[i]:slot[i] + lens[i]] = keep_masks[i]
    return ResourceBatch(shape, lens, cu, slot, pool, q, k, v, keep)


# --------------------------------------------------------------------------
# Requests: which cached resources a conversation sees, through which routes.
# --------------------------------------------------------------------------
@dataclass
class RequestBatch:
    """B requests over a cache pool (one layer's routes)."""
    shape: Shape
    res_off: np.ndarray         # [B+1] int32 into the listed-resource arrays
    res_slot: np.ndarray        # [R] int32 first cache row of each listed resource
    res_len: np.ndarray         # [R] int32
    vis: np.ndarray             # [G][R] uint8
    cu_q: np.ndarray            # [B+1] int32
    q_pos0: np.ndarray          # [B] int32 position of each request's first query token
    q: torch.Tensor             # [sum Tq, Hq, d]
    k_conv: torch.Tensor        # [sum Tq, G, d]
    v_conv: torch.Tensor        # [sum Tq, G, d]
    res_ids: Optional[List[List[int]]] = None

    @property
    def n_requests(self) -> int:
        return len(self.cu_q) - 1

    @property
    def total_q(self) -> int:
        return int(self.cu_q[-1])

    @property
    def max_q(self) -> int:
        return int(np.diff(self.cu_q).max()) if self.n_requests else 0


def make_requests(shape: Shape, seed: int, pool: ResourceBatch, res_lists: List[List[int]],
                  vis_per_request: List[np.ndarray], tq: List[int],
                  q_pos0: Optional[List[int]] = None) -> RequestBatch:
    """res_lists[b] = indices into `pool` in request order; vis_per_request[b] is
    [G][len(res_lists[b])]."""
    b = len(res_lists)
    res_off = np.zeros(b + 1, dtype=np.int32)
    res_off[1:] = np.cumsum([len(r) for r in res_lists])
    flat = [r for lst in res_lists for r in lst]
    res_slot = pool.dst_slot[flat].astype(np.int32) if flat else np.zeros(0, np.int32)
    res_len = pool.lens[flat].astype(np.int32) if flat else np.zeros(0, np.int32)
    g = shape.n_kv_heads
    vis = (np.concatenate(vis_per_request, axis=1).astype(np.uint8) if flat
           else np.zeros((g, 0), np.uint8))
    cu_q = np.zeros(b + 1, dtype=np.int32)
    cu_q[1:] = np.cumsum(tq)
    if q_pos0 is None:  # conversation keeps the positions it would have after the resources
        q_pos0 = [int(pool.lens[lst].sum()) if len(lst) else 0 for lst in res_lists]
    tot = int(cu_q[-1])
    q = normal(seed * 4 + 100, (tot, shape.n_q_heads, shape.head_dim), shape.torch_dtype)
    kc = normal(seed * 4 + 101, (tot, shape.n_kv_heads, shape.head_dim), shape.torch_dtype)
    vc = normal(seed * 4 + 102, (tot, shape.n_kv_heads, shape.head_dim), shape.torch_dtype)
    return RequestBatch(shape, res_off, res_slot, res_len, np.ascontiguousarray(vis), cu_q,
                        np.asarray(q_pos0, dtype=np.int32), q, kc, vc, [list(r) for r in res_lists])


# --------------------------------------------------------------------------
# The five workloads (full size by default; every size is a parameter so the
# parity tests can run the same recipe at sizes the oracle finishes quickly).
# --------------------------------------------------------------------------
SEED0 = 0x5EED0000


def config1():
    """Tiny fp32 case: 3 resources of 17/40/23 tokens, 32 query tokens from
    position 64, group 0 sees {0,2}, group 1 sees {1}, Bernoulli(0.5) keep
    mask with each resource's first token kept."""
    rng = np.random.default_rng(SEED0 + 1)
    lens = [17, 40, 23]
    pool = pack_resources(TINY_F32, SEED0 + 1, lens, keep_mask_bernoulli(rng, lens, 0.5, "first"))
    vis = np.array([[1, 0, 1], [0, 1, 0]], dtype=np.uint8)
    req = make_requests(TINY_F32, SEED0 + 1, pool, [[0, 1, 2]], [vis], [32], q_pos0=[64])
    return pool, req


def config2(n_res=8, len_range=(200, 800), tq=512, route_frac=0.25, seed=SEED0 + 2,
            shape: Shape = QWEN3_4B):
    """One Qwen3-4B-shaped layer: 8 resources U[200,800], 512 query tokens,
    each group sees 25 % of the resources, ~30 % of tokens kept as spans."""
    rng = np.random.default_rng(seed)
    lens = uniform_lengths(rng, n_res, *len_range)
    pool = pack_resources(shape, seed, lens, keep_mask_spans(rng, lens))
    vis = routes_random(rng, shape.n_kv_heads, n_res, route_frac)
    req = make_requests(shape, seed, pool, [list(range(n_res))], [vis], [tq])
    return pool, req


def config3_pool(n_pool=64, len_range=(150, 1200), seed=SEED0 + 3, layer=0,
                 shape: Shape = QWEN3_4B):
    rng = np.random.default_rng(seed)  # lengths and masks do not depend on the layer
    lens = uniform_lengths(rng, n_pool, *len_range)
    masks = keep_mask_spans(rng, lens)
    return pack_resources(shape, seed, lens, masks, layer=layer)


def config3_compositions(n_pool: int, n_requests=16, draw=(4, 12), tq_range=(256, 1024), seed=SEED0 + 3):
    """The requests of the composition-reuse workload: each draws 4-12 distinct pool
    resources in random order and has 256-1024 query tokens.  The same for every layer."""
    rng = np.random.default_rng(seed + 17)
    lists, tqs = [], []
    for _ in range(n_requests):
        k = int(rng.integers(draw[0], min(draw[1], n_pool) + 1))
        lists.append([int(x) for x in rng.choice(n_pool, size=k, replace=False)])
        tqs.append(int(rng.integers(tq_range[0], tq_range[1] + 1)))
    return lists, tqs


def config3_layer_routes(shape: Shape, lists, layer: int, seed=SEED0 + 3, route_frac=0.25):
    """Routes of one layer: redrawn per layer (the compositions are not)."""
    rng_l = np.random.default_rng(seed + 1000 + layer)
    return [routes_random(rng_l, shape.n_kv_heads, len(l), route_frac) for l in lists]


def config3_requests(pool: ResourceBatch, n_requests=16, draw=(4, 12), tq_range=(256, 1024),
                     seed=SEED0 + 3, layer=0, route_frac=0.25):
    """Requests drawing 4-12 distinct pool resources in random order; routes are
    redrawn per layer, the compositions are not."""
    shape = pool.shape
    lists, tqs = config3_compositions(len(pool.lens), n_requests, draw, tq_range, seed)
    vis = config3_layer_routes(shape, lists, layer, seed, route_frac)
    return make_requests(shape, seed + 31 * layer, pool, lists, vis, tqs)


@dataclass
class DecodeBatch:
    """Paged decode step.  Page pools are [n_pages][PAGE_TOKENS][d] per tensor;
    a (sequence, group) item owns a resource table and a history table."""
    shape: Shape
    q: torch.Tensor               # [B, Hq, d] pre-RoPE
    q_pos: np.ndarray             # [B]
    k_pages: torch.Tensor         # [n_pages, 64, d]
    v_pages: torch.Tensor
    res_page_table: np.ndarray    # [B*G, max_res_pages] int32 (-1 = unused)
    res_len: np.ndarray           # [B*G]
    hist_page_table: np.ndarray   # [B*G, max_hist_pages]
    hist_len: np.ndarray          # [B*G]


def config4_decode(batch=64, n_res=16, res_len=(500, 700), keep_ratio=0.3, route_frac=0.25,
                   hist=2048, seed=SEED0 + 4, shape: Shape = QWEN3_4B, shuffle_pages=True,
                   ragged=True):
    """Decode step over already-materialised pages.  Per (sequence, group):
    round(route_frac*n_res) resources of U[res_len] tokens at `keep_ratio`
    kept, then `hist` history rows (the current token is the last of them).
    Page contents are N(0,1) stand-ins for rotated keys / values; every item
    has its own pages, so logical bytes equal HBM bytes.  Pages are handed out
    in shuffled order."""
    rng = np.random.default_rng(seed)
    g = shape.n_kv_heads
    items = batch * g
    k_vis = max(1, int(np.floor(route_frac * n_res + 0.5)))
    rlen = np.zeros(items, np.int32)
    for it in range(items):
        ls = uniform_lengths(rng, k_vis, *res_len)
        rlen[it] = int(sum(max(1, int(round(l * keep_ratio))) for l in ls)) if ragged else \
            int(k_vis * round(0.5 * (res_len[0] + res_len[1]) * keep_ratio))
    hlen = np.full(items, hist, np.int32)
    rp = (rlen + PAGE_TOKENS - 1) // PAGE_TOKENS
    hp = (hlen + PAGE_TOKENS - 1) // PAGE_TOKENS
    n_pages = int(rp.sum() + hp.sum())
    order = rng.permutation(n_pages).astype(np.int32) if shuffle_pages else np.arange(n_pages, dtype=np.int32)
    rpt = np.full((items, max(1, int(rp.max()))), -1, np.int32)
    hpt = np.full((items, max(1, int(hp.max()))), -1, np.int32)
    c = 0
    for it in range(items):
        rpt[it, :rp[it]] = order[c:c + rp[it]]; c += int(rp[it])
        hpt[it, :hp[it]] = order[c:c + hp[it]]; c += int(hp[it])
    d = shape.head_dim
    kp = normal(seed * 4 + 0, (n_pages, PAGE_TOKENS, d), shape.torch_dtype)
    vp = normal(seed * 4 + 1, (n_pages, PAGE_TOKENS, d), shape.torch_dtype)
    q = normal(seed * 4 + 2, (batch, shape.n_q_heads, d), shape.torch_dtype)
    q_pos = np.full(batch, int(n_res * 0.5 * (res_len[0] + res_len[1])) + hist - 1, np.int32)
    return DecodeBatch(shape, q, q_pos, kp, vp, rpt, rlen, hpt, hlen)


def config5(n_res=64, len_range=(1000, 2000), tq=2048, route_frac=0.25, seed=SEED0 + 5,
            shape: Shape = QWEN3_4B, bulk=True):
    """Long tool set: 64 resources U[1000,2000] encoded in one launch, then a
    2048-token prefill at ~8 % retained KV (25 % routes x 30 % kept)."""
    rng = np.random.default_rng(seed)
    lens = uniform_lengths(rng, n_res, *len_range)
    pool = pack_resources(shape, seed, lens, keep_mask_spans(rng, lens), bulk=bulk)
    vis = routes_random(rng, shape.n_kv_heads, n_res, route_frac)
    req = make_requests(shape, seed, pool, [list(range(n_res))], [vis], [tq])
    return pool, req


def all_visible(req: RequestBatch) -> RequestBatch:
    """The dense comparison point: every route sees every listed resource."""
    r = RequestBatch(**{**req.__dict__})
    r.vis = np.ones_like(req.vis)
    return r


def keep_all(pool: ResourceBatch) -> ResourceBatch:
    p = ResourceBatch(**{**pool.__dict__})
    keep = np.zeros_like(pool.keep)
    for s, l in zip(pool.dst_slot, pool.lens):
        keep[s:s + l] = 1
    p.keep = keep
    return p


# --------------------------------------------------------------------------
# Decode composed from a resource pool (paged compaction feeds the decode).
# --------------------------------------------------------------------------
@dataclass
class DecodeCompose:
    """Config-4-shaped decode where the resource pages are materialised from a
    cache pool by paged compaction.  Only index data lives here; the cache and
    history contents are N(0,1) tensors drawn by `seeded_normal`."""
    shape: Shape
    batch: int
    lens: np.ndarray              # [batch * n_res] pool resource lengths
    dst_slot: np.ndarray
    pool_tokens: int
    keep: np.ndarray              # [pool_tokens]
    res_off: np.ndarray           # [batch + 1]
    vis: np.ndarray               # [G][batch * n_res]
    hist_len: np.ndarray          # [batch * G]
    hist_page_table: np.ndarray   # [batch * G, hist_pages]
    free_pages: np.ndarray        # page ids handed to compaction (shuffled)
    n_pages: int
    max_res_pages: int
    q_pos: np.ndarray             # [batch]


def config4_compose(batch=64, n_res=16, res_len=(500, 700), route_frac=0.25, hist=2048,
                    seed=SEED0 + 4, shape: Shape = QWEN3_4B) -> DecodeCompose:
    rng = np.random.default_rng(seed + 7)
    g = shape.n_kv_heads
    lens = uniform_lengths(rng, batch * n_res, *res_len)
    masks = keep_mask_spans(rng, lens)
    slot = np.zeros(len(lens), np.int32)
    slot[1:] = np.cumsum(lens)[:-1]
    pool_tokens = int(lens.sum())
    keep = np.concatenate(masks).astype(np.uint8)
    res_off = (np.arange(batch + 1) * n_res).astype(np.int32)
    vis = np.concatenate([routes_random(rng, g, n_res, route_frac) for _ in range(batch)], axis=1)
    kept = np.array([int(m.sum()) for m in masks])
    route_len = np.array([[int((vis[kg, b * n_res:(b + 1) * n_res] * kept[b * n_res:(b + 1) * n_res]).sum())
                           for kg in range(g)] for b in range(batch)]).reshape(-1)
    res_pages = (route_len + PAGE_TOKENS - 1) // PAGE_TOKENS
    hist_pages = (hist + PAGE_TOKENS - 1) // PAGE_TOKENS
    n_res_pages = int(res_pages.sum())
    n_pages = n_res_pages + batch * g * hist_pages
    order = rng.permutation(n_pages).astype(np.int32)
    free_pages = order[:n_res_pages].copy()
    hpt = order[n_res_pages:].reshape(batch * g, hist_pages).copy()
    q_pos = np.full(batch, int(lens[:n_res].sum()) + hist - 1, np.int32)
    return DecodeCompose(shape, batch, lens, slot, pool_tokens, keep, res_off, np.ascontiguousarray(vis),
                         np.full(batch * g, hist, np.int32), hpt, free_pages, n_pages,
                         int(res_pages.max()) if len(res_pages) else 1, q_pos)


def seeded_normal(seed: int, shape, dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """N(0,1) from a seeded generator on `device` (cache / page contents that
    stand in for earlier encode results; drawn where they are used)."""
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return torch.randn(*shape, generator=g, dtype=torch.float32 if device == "cpu" else dtype,
                       device=device).to(dtype)
