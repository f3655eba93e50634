"""fp64 CPU oracle for resource-routed attention.  TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's cpu_baseline /
reference arm may import this file.  It shares no code with the CUDA path and
imports nothing from the package.  Everything is the plain definition written
out: ordinary softmax attention under the visibility mask and position
assignment the paper defines, evaluated in numpy float64 with one matrix
product per (resource | request, head) and no blocking, fusion or reordering.

What follows which passage of the paper ("Section ReCache"):
  rope / encode_resources   "Resource-Wise Attention": no pair crosses two
                            resources; positions restart inside every resource.
  compact_routes            "Structural Pruning" (routes with M_resource /
                            M_context) and "Semantic Pruning" (retained
                            subsequence of each resource); "Efficiency" metric
                            paragraph (request-local KV materialisation).
  attend_prefill / decode   the final mask of the architecture figure:
                            conversation tokens attend to the retained fields
                            of the resources their route exposes, plus their
                            own causal context, in one softmax.

Readings taken where the paper is silent (all parameters here, none hidden):
positions start at 0; RoPE pairs element i with i + d/2; scale 1/sqrt(d);
query head h reads KV group h // (Hq/G); a route's rows are ordered by request
order then ascending token; rotated queries and keys are materialised in the
storage dtype (`storage`: "bf16", "f32" or None = keep fp64) before the score
product, as a transformer running in that dtype does, so the key a resource's
own tokens attend to is the very key the cache holds for every later reader.
Rounding the rotated KEY is forced by the method (a cached block is reused as
stored); rounding the rotated QUERY is a reading, and `round_q=False` evaluates
the other one (query kept in fp64 after the rotation) so that the tests can say
what the reading is worth.

Pins (tests/test_oracle_*.py): hand-computed RoPE values, brute-force masked
attention in pure Python, torch's fp64 scaled_dot_product_attention on the
special cases that reduce to it, the closed-form route/keep counting identities
and the sparsity figures the paper prints, and the invariances the method
rests on.  No function in this file is "parity unpinned".
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# ---------------------------------------------------------------- storage --
def round_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bfloat16 (8 significant bits, ties to even), returned as fp64.
    Direct from fp64, so there is no double rounding through fp32.  Normal
    range only (the data here is unit-variance)."""
    x = np.asarray(x, dtype=F64)
    m, e = np.frexp(x)                      # x = m * 2**e, 0.5 <= |m| < 1
    return np.ldexp(np.rint(m * 256.0), e - 8)


def round_storage(x: np.ndarray, storage: Optional[str]) -> np.ndarray:
    if storage is None:
        return np.asarray(x, dtype=F64)
    if storage == "bf16":
        return round_bf16(x)
    if storage == "f32":
        return np.asarray(x, dtype=F64).astype(np.float32).astype(F64)
    raise ValueError(storage)


# ------------------------------------------------------------------- RoPE --
def rope(x: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, half-split pairing.  x: [n, H, d]; positions: [n].
    out[i]       = x[i] cos(p phi_i) - x[i+d/2] sin(p phi_i)
    out[i+d/2]   = x[i+d/2] cos(p phi_i) + x[i] sin(p phi_i),  phi_i = theta^(-2i/d)."""
    x = np.asarray(x, dtype=F64)
    n, _, d = x.shape
    half = d // 2
    phi = F64(theta) ** (-2.0 * np.arange(half, dtype=F64) / d)
    ang = np.asarray(positions, dtype=F64).reshape(n, 1) * phi.reshape(1, half)
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


# ---------------------------------------------------------------- softmax --
def _softmax_rows(s: np.ndarray) -> np.ndarray:
    """Row softmax; -inf entries are masked keys.  Every row must have a key."""
    m = s.max(axis=-1, keepdims=True)
    p = np.exp(s - m)
    return p / p.sum(axis=-1, keepdims=True)


# ----------------------------------------------------------------- encode --
def encode_resources(q, k, v, cu_seqlens, theta: float, storage: Optional[str] = None,
                     pos_offset: Optional[Sequence[int]] = None, prefix_k=None, prefix_v=None,
                     round_q: bool = True):
    """Resource-wise encoding.  q: [T,Hq,d]; k, v: [T,G,d] (pre-RoPE), resource
    i = rows cu_seqlens[i]..cu_seqlens[i+1]-1 at positions pos_offset[i] + 0..D_i-1
    (pos_offset = None: resource-local positions from 0; one common offset P: the
    layout after a shared prefix of P tokens; global offsets: the "Block"
    variant, which drops cross-resource attention but keeps original positions).
    prefix_k / prefix_v [G][P][d]: rotated keys / values of a shared prefix as a
    cache holds them; every resource token sees all of them besides its own
    resource's tokens j' <= j (the shared-prefix form of resource-wise attention,
    Section "Resource-Wise Attention").
    Returns (o [T,Hq,d], k_hat [T,G,d] in storage precision, v [T,G,d])."""
    q = np.asarray(q, F64); k = np.asarray(k, F64); v = np.asarray(v, F64)
    t, hq, d = q.shape
    g = k.shape[1]
    s = hq // g
    o = np.zeros_like(q)
    k_hat = np.zeros_like(k)
    for i in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[i]), int(cu_seqlens[i + 1])
        n = b - a
        if n == 0:
            continue
        pos = np.arange(n) + (0 if pos_offset is None else int(pos_offset[i]))
        qh = round_storage(rope(q[a:b], pos, theta), storage if round_q else None)
        kh = round_storage(rope(k[a:b], pos, theta), storage)
        k_hat[a:b] = kh
        causal = np.tril(np.ones((n, n), dtype=bool))
        for h in range(hq):
            kg = h // s
            sc = qh[:, h, :] @ kh[:, kg, :].T / math.sqrt(d)
            sc = np.where(causal, sc, -np.inf)
            vals = v[a:b, kg, :]
            if prefix_k is not None and np.asarray(prefix_k).shape[1] > 0:
                pk, pv = np.asarray(prefix_k[kg], F64), np.asarray(prefix_v[kg], F64)
                sc = np.concatenate([qh[:, h, :] @ pk.T / math.sqrt(d), sc], axis=1)
                vals = np.concatenate([pv, vals], axis=0)
            o[a:b, h, :] = _softmax_rows(sc) @ vals
    return o, k_hat, v.copy()


def encode_rows(q, k, v, cu_seqlens, theta: float, rows: Sequence[Tuple[int, int]],
                storage: Optional[str] = None, round_q: bool = True):
    """The same definition for a chosen set of output rows (token, head) only,
    one at a time; for sizes where the full table takes minutes.  q/k/v may be
    fp32 arrays holding bf16 values: only the rows a sample needs are widened."""
    t, hq, d = q.shape
    g = k.shape[1]
    s = hq // g
    cu = np.asarray(cu_seqlens)
    out = np.zeros((len(rows), d), F64)
    for n, (tok, h) in enumerate(rows):
        i = int(np.searchsorted(cu, tok, side="right") - 1)
        a = int(cu[i])
        j = tok - a
        kg = h // s
        qh = round_storage(rope(np.asarray(q[tok:tok + 1, h:h + 1], F64), np.array([j]), theta),
                           storage if round_q else None)[0, 0]
        kh = round_storage(rope(np.asarray(k[a:tok + 1, kg:kg + 1], F64), np.arange(j + 1), theta), storage)[:, 0, :]
        sc = kh @ qh / math.sqrt(d)
        out[n] = _softmax_rows(sc[None, :])[0] @ np.asarray(v[a:tok + 1, kg, :], F64)
    return out


def write_cache(k_cache, v_cache, k_hat, v, cu_seqlens, dst_slot):
    """Cache layout [G][pool_tokens][d]; resource i goes to rows dst_slot[i]+j."""
    for i in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[i]), int(cu_seqlens[i + 1])
        s0 = int(dst_slot[i])
        k_cache[:, s0:s0 + (b - a), :] = np.transpose(k_hat[a:b], (1, 0, 2))
        v_cache[:, s0:s0 + (b - a), :] = np.transpose(v[a:b], (1, 0, 2))


# -------------------------------------------------------------- compaction --
def compact_routes(keep, res_off, res_slot, res_len, vis) -> List[List[np.ndarray]]:
    """rows[b][g] = cache rows route (b, g) exposes: the request's resources in
    request order, those with vis[g][r] = 1, their kept tokens ascending."""
    keep = np.asarray(keep)
    n_groups = vis.shape[0]
    out = []
    for b in range(len(res_off) - 1):
        per_group = []
        for g in range(n_groups):
            rows = []
            for r in range(int(res_off[b]), int(res_off[b + 1])):
                if vis[g][r]:
                    s0, n = int(res_slot[r]), int(res_len[r])
                    for j in range(n):
                        if keep[s0 + j]:
                            rows.append(s0 + j)
            per_group.append(np.asarray(rows, dtype=np.int32))
        out.append(per_group)
    return out


def route_prefix(rows: List[List[np.ndarray]]) -> np.ndarray:
    """Exclusive prefix of route lengths in (request-major, group-minor) order."""
    lens = [len(r) for per in rows for r in per]
    cu = np.zeros(len(lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    return cu


def gather_packed(cache, rows: List[List[np.ndarray]]) -> np.ndarray:
    """Packed layout [sum route rows][d]: route (b, g) holds cache[g][rows[b][g]]."""
    d = cache.shape[-1]
    parts = [cache[g][r] for per in rows for g, r in enumerate(per)]
    return np.concatenate(parts, axis=0) if parts else np.zeros((0, d), cache.dtype)


def page_layout(rows: List[List[np.ndarray]], free_pages, page_tokens: int, max_pages: int):
    """Paged layout: route i (request-major) takes ceil(len_i / page_tokens)
    consecutive entries of free_pages, starting where route i-1 stopped.
    Returns (page_table [routes][max_pages] with -1 padding, pages used)."""
    flat = [r for per in rows for r in per]
    table = np.full((len(flat), max_pages), -1, dtype=np.int32)
    cur = 0
    for i, r in enumerate(flat):
        n = (len(r) + page_tokens - 1) // page_tokens
        table[i, :n] = np.asarray(free_pages[cur:cur + n], dtype=np.int32)
        cur += n
    return table, cur


def gather_paged(cache, rows, page_table, n_pages: int, page_tokens: int, fill=0.0):
    """Page pool [n_pages][page_tokens][d] holding each route's rows; slots no
    route writes keep `fill`."""
    d = cache.shape[-1]
    pool = np.full((n_pages, page_tokens, d), fill, dtype=cache.dtype)
    i = 0
    for per in rows:
        for g, r in enumerate(per):
            for n, row in enumerate(r):
                pool[page_table[i, n // page_tokens], n % page_tokens] = cache[g][row]
            i += 1
    return pool


# ------------------------------------------------------- routed attention --
def attend_prefill(q, k_conv, v_conv, cu_q, q_pos0, rows, k_cache, v_cache, theta: float,
                   storage: Optional[str] = None, hist_k=None, hist_v=None, round_q: bool = True):
    """Conversation tokens of request b (positions q_pos0[b] + t) attend, in one
    softmax with scale 1/sqrt(d), to (i) every row of their route's compacted
    resource KV (cached rotated keys used as stored) and (ii) conversation
    tokens t' <= t.  A route without rows is the context-only mask.
    hist_k[b] / hist_v[b] ([G][H_b][d], rotated keys as stored): earlier turns of
    request b, all visible to every new token (multi-turn history).
    Returns (o [sum Tq,Hq,d], k_conv_hat [sum Tq,G,d] in storage precision)."""
    q = np.asarray(q, F64); k_conv = np.asarray(k_conv, F64); v_conv = np.asarray(v_conv, F64)
    tq, hq, d = q.shape
    g = k_conv.shape[1]
    s = hq // g
    o = np.zeros_like(q)
    kc_hat = np.zeros_like(k_conv)
    for b in range(len(cu_q) - 1):
        a, e = int(cu_q[b]), int(cu_q[b + 1])
        n = e - a
        if n == 0:
            continue
        pos = int(q_pos0[b]) + np.arange(n)
        qh = round_storage(rope(q[a:e], pos, theta), storage if round_q else None)
        kh = round_storage(rope(k_conv[a:e], pos, theta), storage)
        kc_hat[a:e] = kh
        causal = np.tril(np.ones((n, n), dtype=bool))
        for h in range(hq):
            kg = h // s
            r = rows[b][kg]
            kr = np.asarray(k_cache[kg][r], F64).reshape(len(r), d)
            vr = np.asarray(v_cache[kg][r], F64).reshape(len(r), d)
            if hist_k is not None and hist_k[b] is not None:     # earlier turns: more all-visible rows
                kr = np.concatenate([kr, np.asarray(hist_k[b][kg], F64)], axis=0)
                vr = np.concatenate([vr, np.asarray(hist_v[b][kg], F64)], axis=0)
            s_res = qh[:, h, :] @ kr.T / math.sqrt(d)
            s_conv = np.where(causal, qh[:, h, :] @ kh[:, kg, :].T / math.sqrt(d), -np.inf)
            p = _softmax_rows(np.concatenate([s_res, s_conv], axis=1))
            o[a:e, h, :] = p @ np.concatenate([vr, v_conv[a:e, kg, :]], axis=0)
    return o, kc_hat


def prefill_rows(q, k_conv, v_conv, cu_q, q_pos0, rows, k_cache, v_cache, theta: float,
                 out_rows: Sequence[Tuple[int, int]], storage: Optional[str] = None, round_q: bool = True):
    """attend_prefill for chosen (query token, head) rows only."""
    cu = np.asarray(cu_q)
    tq, hq, d = q.shape
    g = k_conv.shape[1]
    s = hq // g
    out = np.zeros((len(out_rows), d), F64)
    for n, (tok, h) in enumerate(out_rows):
        b = int(np.searchsorted(cu, tok, side="right") - 1)
        a = int(cu[b])
        t = tok - a
        kg = h // s
        p0 = int(q_pos0[b])
        qh = round_storage(rope(np.asarray(q[tok:tok + 1, h:h + 1], F64), np.array([p0 + t]), theta),
                           storage if round_q else None)[0, 0]
        kh = round_storage(rope(np.asarray(k_conv[a:tok + 1, kg:kg + 1], F64), p0 + np.arange(t + 1), theta),
                           storage)[:, 0, :]
        r = rows[b][kg]
        keys = np.concatenate([np.asarray(k_cache[kg][r], F64).reshape(len(r), d), kh], axis=0)
        vals = np.concatenate([np.asarray(v_cache[kg][r], F64).reshape(len(r), d),
                               np.asarray(v_conv[a:tok + 1, kg, :], F64)], axis=0)
        out[n] = _softmax_rows((keys @ qh / math.sqrt(d))[None, :])[0] @ vals
    return out


def append_decode_kv(k_pages, v_pages, hist_page_table, hist_len, k_new, v_new, q_pos,
                     theta: float, page_tokens: int, storage: Optional[str] = None):
    """The current token's rotated key and its value become the LAST history
    row (index hist_len - 1) of every (sequence, group) item."""
    b, g, d = k_new.shape
    kh = round_storage(rope(np.asarray(k_new, F64), np.asarray(q_pos), theta), storage)
    for i in range(b):
        for kg in range(g):
            it = i * g + kg
            n = int(hist_len[it]) - 1
            pg = int(hist_page_table[it, n // page_tokens])
            k_pages[pg, n % page_tokens] = kh[i, kg]
            v_pages[pg, n % page_tokens] = np.asarray(v_new[i, kg], F64)


def attend_decode(q, q_pos, k_pages, v_pages, res_page_table, res_len, hist_page_table,
                  hist_len, theta: float, page_tokens: int, items: Optional[Sequence[int]] = None,
                  storage: Optional[str] = None, round_q: bool = True):
    """One query token per sequence over its route's paged resource rows and its
    paged history (whose last row is the current token).  q: [B,Hq,d] pre-RoPE.
    `items` restricts the work to chosen (sequence*G + group) items; other
    output rows stay zero."""
    q = np.asarray(q, F64)
    b, hq, d = q.shape
    g = len(res_len) // b
    s = hq // g
    qh = round_storage(rope(q, np.asarray(q_pos), theta), storage if round_q else None)
    o = np.zeros_like(q)

    def rows_of(table, n):
        idx = np.arange(n)
        return table[idx // page_tokens], idx % page_tokens

    todo = range(b * g) if items is None else items
    for it in todo:
        i, kg = divmod(int(it), g)
        pr, sr = rows_of(res_page_table[it], int(res_len[it]))
        ph, sh = rows_of(hist_page_table[it], int(hist_len[it]))
        keys = np.concatenate([np.asarray(k_pages[pr, sr], F64).reshape(-1, d),
                               np.asarray(k_pages[ph, sh], F64).reshape(-1, d)], axis=0)
        vals = np.concatenate([np.asarray(v_pages[pr, sr], F64).reshape(-1, d),
                               np.asarray(v_pages[ph, sh], F64).reshape(-1, d)], axis=0)
        for h in range(kg * s, (kg + 1) * s):
            sc = keys @ qh[i, h] / math.sqrt(d)
            o[i, h] = _softmax_rows(sc[None, :])[0] @ vals
    return o


# ---------------------------------------------------------- route selection --
def routes_from_contributions(s_layers, s_groups, k_layers: int, k_groups: int):
    """Omega* = TopK_{K_L}(w_l) x TopK_{K_G}(w_g) with w_i = max(s_i, 0) / sum_j max(s_j, 0)
    ("Structural Pruning"); ties go to the lower index.  Returns (omega [L][G],
    kept layers, kept groups, CC of the kept layers, CC of the kept groups)."""
    def top(s, k):
        w = np.maximum(np.asarray(s, F64), 0.0)
        w = w / w.sum() if w.sum() > 0 else w
        order = sorted(range(len(w)), key=lambda i: (-w[i], i))[:k]
        return order, float(sum(w[i] for i in order))
    kl, ccl = top(s_layers, k_layers)
    kg, ccg = top(s_groups, k_groups)
    omega = np.zeros((len(s_layers), len(s_groups)), dtype=np.uint8)
    for l in kl:
        for g in kg:
            omega[l, g] = 1
    return omega, kl, kg, ccl, ccg


# ------------------------------------------------------------ bookkeeping --
def structural_sparsity(n_layers_kept: int, n_groups_kept: int, n_layers: int, n_groups: int) -> float:
    """rho(Omega) = 1 - |L*||G*| / (L G) for a product route set."""
    return 1.0 - (n_layers_kept * n_groups_kept) / (n_layers * n_groups)


def useful_pairs_encode(lens) -> int:
    """Unmasked (query, key) pairs per query head in resource-wise encoding."""
    return int(sum(int(n) * (int(n) + 1) // 2 for n in lens))


def useful_pairs_prefill(tq: int, route_len: int) -> int:
    """Unmasked pairs per query head for one request on one route."""
    return tq * route_len + tq * (tq + 1) // 2
