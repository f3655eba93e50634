"""Pins for the fp64 oracle: everything here runs on the CPU.

Each test ties a function of oracle/recache_oracle.py to something other than
itself: hand-computed values, a brute-force masked attention written with
Python scalars, torch's fp64 scaled_dot_product_attention on the special cases
that reduce to it, closed-form counting identities with the figures the paper
prints, or an invariance the method rests on.
"""
import cmath
import math
import os

import numpy as np
import pytest
import torch

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f64(t):
    return t.to(torch.float64).numpy()


# ------------------------------------------------------------ brute force --
def brute_rope(vec, p, theta):
    """Rotation of the pair (x[i], x[i+d/2]) as a complex multiplication."""
    d = len(vec)
    out = [0.0] * d
    for i in range(d // 2):
        z = complex(vec[i], vec[i + d // 2]) * cmath.exp(1j * p * theta ** (-2.0 * i / d))
        out[i], out[i + d // 2] = z.real, z.imag
    return out


def brute_attention(queries, keys, values, visible):
    """queries/keys/values: lists of Python-float vectors; visible(i, j) -> bool."""
    d = len(queries[0])
    out = []
    for i, qv in enumerate(queries):
        sc = [sum(a * b for a, b in zip(qv, kv)) / math.sqrt(d) if visible(i, j) else None
              for j, kv in enumerate(keys)]
        m = max(s for s in sc if s is not None)
        w = [math.exp(s - m) if s is not None else 0.0 for s in sc]
        z = sum(w)
        out.append([sum(w[j] * values[j][c] for j in range(len(keys))) / z for c in range(d)])
    return out


# ------------------------------------------------------------------- RoPE --
def test_rope_hand_values():
    # d = 4, theta = 1e4: phi = (1, 0.01).  x = (1, 2, 3, 4), p = 3.
    x = np.array([[[1.0, 2.0, 3.0, 4.0]]])
    y = orc.rope(x, np.array([3]), 1.0e4)[0, 0]
    want = [1 * math.cos(3) - 3 * math.sin(3), 2 * math.cos(0.03) - 4 * math.sin(0.03),
            3 * math.cos(3) + 1 * math.sin(3), 4 * math.cos(0.03) + 2 * math.sin(0.03)]
    assert np.allclose(y, want, rtol=0, atol=1e-15)
    # d = 2: phi_0 = 1 for any theta, so (1, 0) at position p is (cos p, sin p).
    y2 = orc.rope(np.array([[[1.0, 0.0]]]), np.array([0.5]), 123.0)[0, 0]
    assert np.allclose(y2, [math.cos(0.5), math.sin(0.5)], atol=1e-16)


def test_rope_identity_norm_relative():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 3, 64))
    assert np.array_equal(orc.rope(x, np.zeros(5), 1e6), x)          # position 0 is the identity
    y = orc.rope(x, np.arange(5) * 977, 1e6)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)
    # <rope(q,a), rope(k,b)> depends on a - b only
    q = rng.standard_normal((1, 1, 64)); k = rng.standard_normal((1, 1, 64))
    d1 = (orc.rope(q, [70], 1e4) * orc.rope(k, [13], 1e4)).sum()
    d2 = (orc.rope(q, [1057], 1e4) * orc.rope(k, [1000], 1e4)).sum()
    assert abs(d1 - d2) < 1e-11


def test_rope_matches_complex_form():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((4, 2, 8))
    y = orc.rope(x, np.array([0, 1, 17, 300]), 1e4)
    for n, p in enumerate([0, 1, 17, 300]):
        for h in range(2):
            assert np.allclose(y[n, h], brute_rope(list(x[n, h]), p, 1e4), atol=1e-13)


def test_round_bf16():
    # exact bf16 values stay; ties go to even; agrees with torch away from fp32 double rounding
    assert orc.round_bf16(np.array([1.0, -2.5, 0.15625]))[2] == 0.15625
    assert orc.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0            # tie -> even (1.0)
    assert orc.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6  # tie -> even
    x = np.random.default_rng(2).standard_normal(20000)
    want = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    got = orc.round_bf16(x.astype(np.float32).astype(np.float64))
    assert np.array_equal(got, want)


# ----------------------------------------------------------------- encode --
def _c1():
    pool, req = wl.config1()
    return pool, req


def test_encode_matches_bruteforce_block_mask():
    """C1: dense T x T attention with an explicit mask (same resource and
    j' <= j) and explicit per-token local positions."""
    pool, _ = _c1()
    sh = pool.shape
    q, k, v = f64(pool.q), f64(pool.k), f64(pool.v)
    o, k_hat, v_out = orc.encode_resources(q, k, v, pool.cu_seqlens, sh.rope_theta)
    t = pool.total_tokens
    res_of = np.searchsorted(pool.cu_seqlens, np.arange(t), side="right") - 1
    local = np.arange(t) - pool.cu_seqlens[res_of]
    assert local[pool.cu_seqlens[1]] == 0 and local[pool.cu_seqlens[1] - 1] == 16
    s = sh.group_size
    for h in range(sh.n_q_heads):
        g = h // s
        qs = [brute_rope(list(q[n, h]), int(local[n]), sh.rope_theta) for n in range(t)]
        ks = [brute_rope(list(k[n, g]), int(local[n]), sh.rope_theta) for n in range(t)]
        vs = [list(v[n, g]) for n in range(t)]
        want = brute_attention(qs, ks, vs, lambda i, j: res_of[i] == res_of[j] and j <= i)
        assert np.allclose(o[:, h, :], np.array(want), atol=1e-12)
        assert np.allclose(k_hat[:, g, :], np.array(ks), atol=1e-13)
    assert np.array_equal(v_out, v)


def test_single_resource_is_causal_sdpa():
    """One resource encoded resource-wise == standard causal attention at
    positions 0..L-1 (torch fp64 SDPA, RoPE applied via torch.polar)."""
    sh = wl.Shape(4, 2, 32, 1e4, "f32")
    L = 29
    q, k, v = wl.resource_tensors(7, 0, L, sh)
    o, _, _ = orc.encode_resources(f64(q), f64(k), f64(v), [0, L], sh.rope_theta)

    def trope(x):  # [L, H, d] torch fp64, independent formulation
        x = x.to(torch.float64)
        half = sh.head_dim // 2
        phi = sh.rope_theta ** (-2.0 * torch.arange(half, dtype=torch.float64) / sh.head_dim)
        rot = torch.polar(torch.ones(L, half, dtype=torch.float64),
                          torch.arange(L, dtype=torch.float64)[:, None] * phi[None, :])
        z = torch.complex(x[..., :half], x[..., half:]) * rot[:, None, :]
        return torch.cat([z.real, z.imag], -1)

    qh = trope(q).permute(1, 0, 2)[None]
    kh = trope(k).permute(1, 0, 2).repeat_interleave(2, 0)[None]
    vh = v.to(torch.float64).permute(1, 0, 2).repeat_interleave(2, 0)[None]
    want = torch.nn.functional.scaled_dot_product_attention(qh, kh, vh, is_causal=True)[0]
    assert np.allclose(o, want.permute(1, 0, 2).numpy(), atol=1e-12)


def test_encode_degenerate_rows():
    sh = wl.TINY_F32
    q, k, v = wl.resource_tensors(3, 0, 6, sh)
    # lengths 1, 0, 5: a one-token resource returns its own value; an empty one is skipped
    o, k_hat, _ = orc.encode_resources(f64(q), f64(k), f64(v), [0, 1, 1, 6], sh.rope_theta)
    s = sh.group_size
    for h in range(sh.n_q_heads):
        assert np.allclose(o[0, h], f64(v)[0, h // s], atol=1e-15)
        assert np.allclose(o[1, h], f64(v)[1, h // s], atol=1e-15)      # first row of resource 2
    assert np.array_equal(k_hat[0], f64(k)[0]) and np.array_equal(k_hat[1], f64(k)[1])


def test_resource_kv_independent_of_neighbours_and_order():
    """A resource's output, rotated keys and values are EXACTLY the same alone,
    between other resources, or in another order."""
    sh = wl.TINY_F32
    lens = [17, 40, 23]
    parts = [wl.resource_tensors(11, r, n, sh) for r, n in enumerate(lens)]

    def run(order):
        q = np.concatenate([f64(parts[r][0]) for r in order]); k = np.concatenate([f64(parts[r][1]) for r in order])
        v = np.concatenate([f64(parts[r][2]) for r in order])
        cu = np.concatenate([[0], np.cumsum([lens[r] for r in order])])
        o, kh, vv = orc.encode_resources(q, k, v, cu, sh.rope_theta)
        return {r: (o[cu[i]:cu[i + 1]], kh[cu[i]:cu[i + 1]], vv[cu[i]:cu[i + 1]]) for i, r in enumerate(order)}

    base = run([0, 1, 2])
    for order in ([2, 0, 1], [1], [1, 2]):
        got = run(order)
        for r in order:
            for a, b in zip(got[r], base[r]):
                assert np.array_equal(a, b)


def test_position_shift_changes_keys_not_outputs():
    """Shifting every local position of a resource by a constant leaves its
    outputs unchanged (only relative positions enter) but changes the keys:
    global positions and local positions differ only in what is cached."""
    pool, _ = _c1()
    sh = pool.shape
    q, k, v = f64(pool.q), f64(pool.k), f64(pool.v)
    o0, k0, _ = orc.encode_resources(q, k, v, pool.cu_seqlens, sh.rope_theta)
    o1, k1, _ = orc.encode_resources(q, k, v, pool.cu_seqlens, sh.rope_theta, pos_offset=[5, 22, 62])
    assert np.allclose(o0, o1, atol=1e-11)
    assert np.abs(k0 - k1).max() > 0.1


def test_encode_rows_agrees_with_table():
    pool, _ = _c1()
    q, k, v = f64(pool.q), f64(pool.k), f64(pool.v)
    o, _, _ = orc.encode_resources(q, k, v, pool.cu_seqlens, 1e4)
    rows = [(0, 0), (16, 3), (17, 1), (56, 2), (79, 3)]
    got = orc.encode_rows(q, k, v, pool.cu_seqlens, 1e4, rows)
    for n, (tok, h) in enumerate(rows):
        assert np.allclose(got[n], o[tok, h], atol=1e-13)


# -------------------------------------------------------------- compaction --
def test_compaction_bruteforce_and_order():
    rng = np.random.default_rng(5)
    lens = [5, 1, 9, 4]
    slot = [3, 0, 20, 9]                     # slots not in list order, with gaps
    keep = (rng.random(40) < 0.5).astype(np.uint8)
    res_off = [0, 3, 3, 4]                   # request 1 lists nothing
    vis = np.array([[1, 0, 1, 1], [0, 1, 1, 0]], dtype=np.uint8)
    rows = orc.compact_routes(keep, res_off, slot, lens, vis)
    # written out by hand for request 0, group 0: resources 0 and 2 in that order
    want = [3 + j for j in range(5) if keep[3 + j]] + [20 + j for j in range(9) if keep[20 + j]]
    assert rows[0][0].tolist() == want
    assert rows[0][1].tolist() == [j for j in [0] if keep[0]] + [20 + j for j in range(9) if keep[20 + j]]
    assert rows[1][0].size == 0 and rows[1][1].size == 0
    assert rows[2][0].tolist() == [9 + j for j in range(4) if keep[9 + j]] and rows[2][1].size == 0
    assert orc.route_prefix(rows).tolist() == np.concatenate(
        [[0], np.cumsum([len(r) for per in rows for r in per])]).tolist()


def test_compaction_keep_all_is_identity_ranges():
    pool, req = wl.config2(n_res=5, len_range=(10, 30), tq=8)
    pool = wl.keep_all(pool); req = wl.all_visible(req)
    rows = orc.compact_routes(pool.keep, req.res_off, req.res_slot, req.res_len, req.vis)
    want = np.concatenate([np.arange(s, s + n) for s, n in zip(req.res_slot, req.res_len)])
    for g in range(pool.shape.n_kv_heads):
        assert np.array_equal(rows[0][g], want)


def _golden():
    budgets, mem = [], {}
    for line in open(os.path.join(GOLDEN, "structural_budget.txt")):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "budget":
            budgets.append((f[1], int(f[2]), int(f[3]), int(f[4]), int(f[5]), float(f[6])))
        else:
            mem[f[0]] = float(f[1])
    return budgets, mem


def test_retained_rows_match_printed_sparsity():
    """Product routes Omega = L* x G*: the retained share of resource KV rows,
    counted by compaction over all layers and groups, equals 1 - rho with the
    rho the paper prints for both backbones, and (1 - rho) * keep ratio once
    tokens are pruned too; the paper's memory figures compose the same way."""
    budgets, mem = _golden()
    for _, kl, nl, kg, ng, rho_pct in budgets:
        assert round(100 * orc.structural_sparsity(kl, kg, nl, ng), 1) == rho_pct
        lens = [12, 7, 30]
        rng = np.random.default_rng(nl)
        masks = wl.keep_mask_bernoulli(rng, lens, 0.4)
        shape = wl.Shape(2 * ng, ng, 8, 1e4, "f32")
        pool = wl.pack_resources(shape, 1, lens, masks)
        omega = wl.routes_product(nl, ng, range(kl), range(kg))
        kept_rows = 0
        for layer in range(nl):
            vis = np.repeat(omega[layer][:, None], len(lens), axis=1)
            rows = orc.compact_routes(pool.keep, [0, 3], pool.dst_slot, pool.lens, vis)
            kept_rows += sum(len(r) for r in rows[0])
        total = nl * ng * sum(lens)
        kappa = sum(int(m.sum()) for m in masks) / sum(lens)
        assert abs(kept_rows / total - (1 - rho_pct / 100) * kappa) < 1e-3 * kappa
        assert kept_rows == kl * kg * sum(int(m.sum()) for m in masks)
    composite = 100 * (1 - (1 - mem["mem_structural"] / 100) * (1 - mem["mem_semantic"] / 100))
    assert abs(composite - mem["mem_recache"]) < 0.05


def test_page_layout_and_paged_equals_packed():
    pool, req = wl.config2(n_res=4, len_range=(60, 200), tq=4, shape=wl.Shape(4, 2, 8, 1e4, "f32"))
    rows = orc.compact_routes(pool.keep, req.res_off, req.res_slot, req.res_len, req.vis)
    cache = np.random.default_rng(0).standard_normal((2, pool.pool_tokens, 8))
    free = [9, 3, 7, 1, 0, 5, 11, 2, 4, 6, 8, 10]
    table, used = orc.page_layout(rows, free, 64, 6)
    assert used == sum((len(r) + 63) // 64 for r in rows[0])
    assert table[0, 0] == 9
    pages = orc.gather_paged(cache, rows, table, 12, 64)
    packed = orc.gather_packed(cache, rows)
    cu = orc.route_prefix(rows)
    for i in range(2):
        n = cu[i + 1] - cu[i]
        flat = np.concatenate([pages[p] for p in table[i] if p >= 0])[:n]
        assert np.array_equal(flat, packed[cu[i]:cu[i + 1]])


# ------------------------------------------------------- routed attention --
def _c1_pipeline():
    pool, req = _c1()
    sh = pool.shape
    q, k, v = f64(pool.q), f64(pool.k), f64(pool.v)
    o, k_hat, vv = orc.encode_resources(q, k, v, pool.cu_seqlens, sh.rope_theta)
    kc = np.zeros((sh.n_kv_heads, pool.pool_tokens, sh.head_dim)); vc = np.zeros_like(kc)
    orc.write_cache(kc, vc, k_hat, vv, pool.cu_seqlens, pool.dst_slot)
    rows = orc.compact_routes(pool.keep, req.res_off, req.res_slot, req.res_len, req.vis)
    return pool, req, kc, vc, rows


def test_prefill_matches_bruteforce_mask():
    """C1: dense attention of the 32 query tokens over [all 80 resource tokens ;
    32 conversation tokens] with an explicit boolean mask built from the route
    table and the keep mask, positions assigned per token."""
    pool, req, kc, vc, rows = _c1_pipeline()
    sh = pool.shape
    assert rows[0][0].size > 0 and set(rows[0][0]) <= set(range(0, 17)) | set(range(57, 80))
    o, kconv_hat = orc.attend_prefill(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0,
                                      rows, kc, vc, sh.rope_theta)
    t = pool.total_tokens
    res_of = np.searchsorted(pool.cu_seqlens, np.arange(t), side="right") - 1
    local = np.arange(t) - pool.cu_seqlens[res_of]
    tq = req.total_q
    s = sh.group_size
    for h in range(sh.n_q_heads):
        g = h // s
        qs = [brute_rope(list(f64(req.q)[n, h]), 64 + n, sh.rope_theta) for n in range(tq)]
        ks = [brute_rope(list(f64(pool.k)[n, g]), int(local[n]), sh.rope_theta) for n in range(t)] + \
             [brute_rope(list(f64(req.k_conv)[n, g]), 64 + n, sh.rope_theta) for n in range(tq)]
        vs = [list(f64(pool.v)[n, g]) for n in range(t)] + [list(f64(req.v_conv)[n, g]) for n in range(tq)]

        def visible(i, j):
            if j < t:
                return bool(req.vis[g][res_of[j]]) and bool(pool.keep[pool.dst_slot[res_of[j]] + local[j]])
            return (j - t) <= i

        want = brute_attention(qs, ks, vs, visible)
        assert np.allclose(o[:, h, :], np.array(want), atol=1e-12)


def test_all_visible_keep_all_is_dense_block_mask_sdpa():
    """Every route sees everything and nothing is pruned: dense attention over
    the concatenated KV; checked with torch fp64 SDPA and an attn_mask."""
    pool, req, kc, vc, _ = _c1_pipeline()
    sh = pool.shape
    pool_all = wl.keep_all(pool); req_all = wl.all_visible(req)
    rows = orc.compact_routes(pool_all.keep, req_all.res_off, req_all.res_slot, req_all.res_len, req_all.vis)
    o, kconv_hat = orc.attend_prefill(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0,
                                      rows, kc, vc, sh.rope_theta)
    t, tq = pool.total_tokens, req.total_q
    qh = torch.from_numpy(orc.rope(f64(req.q), 64 + np.arange(tq), sh.rope_theta)).permute(1, 0, 2)[None]
    keys = np.concatenate([np.transpose(kc[:, :t], (1, 0, 2)), kconv_hat], 0)   # slots are contiguous in C1
    vals = np.concatenate([np.transpose(vc[:, :t], (1, 0, 2)), f64(req.v_conv)], 0)
    kh = torch.from_numpy(keys).permute(1, 0, 2).repeat_interleave(sh.group_size, 0)[None]
    vh = torch.from_numpy(vals).permute(1, 0, 2).repeat_interleave(sh.group_size, 0)[None]
    mask = torch.cat([torch.ones(tq, t, dtype=torch.bool), torch.tril(torch.ones(tq, tq, dtype=torch.bool))], 1)
    want = torch.nn.functional.scaled_dot_product_attention(qh, kh, vh, attn_mask=mask)[0]
    assert np.allclose(o, want.permute(1, 0, 2).numpy(), atol=1e-12)


def test_resource_order_permutation_invariance():
    pool, req, kc, vc, rows = _c1_pipeline()
    sh = pool.shape
    o, _ = orc.attend_prefill(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0, rows, kc, vc, sh.rope_theta)
    perm = [2, 0, 1]
    rows_p = orc.compact_routes(pool.keep, req.res_off, req.res_slot[perm], req.res_len[perm], req.vis[:, perm])
    assert rows_p[0][0].tolist() != rows[0][0].tolist() and sorted(rows_p[0][0]) == sorted(rows[0][0])
    o_p, _ = orc.attend_prefill(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0, rows_p, kc, vc, sh.rope_theta)
    assert np.allclose(o, o_p, atol=1e-12)


def test_empty_route_is_causal_self_attention():
    pool, req, kc, vc, _ = _c1_pipeline()
    sh = pool.shape
    vis0 = np.zeros_like(req.vis)
    rows = orc.compact_routes(pool.keep, req.res_off, req.res_slot, req.res_len, vis0)
    o, kconv_hat = orc.attend_prefill(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0, rows, kc, vc, sh.rope_theta)
    tq = req.total_q
    qh = torch.from_numpy(orc.rope(f64(req.q), 64 + np.arange(tq), sh.rope_theta)).permute(1, 0, 2)[None]
    kh = torch.from_numpy(kconv_hat).permute(1, 0, 2).repeat_interleave(sh.group_size, 0)[None]
    vh = req.v_conv.to(torch.float64).permute(1, 0, 2).repeat_interleave(sh.group_size, 0)[None]
    want = torch.nn.functional.scaled_dot_product_attention(qh, kh, vh, is_causal=True)[0]
    assert np.allclose(o, want.permute(1, 0, 2).numpy(), atol=1e-12)


def test_constant_values_give_constant_output():
    pool, req, kc, vc, rows = _c1_pipeline()
    vc[:] = 0.75
    vconv = np.full(tuple(req.v_conv.shape), 0.75)
    o, _ = orc.attend_prefill(f64(req.q), f64(req.k_conv), vconv, req.cu_q, req.q_pos0, rows, kc, vc, 1e4)
    assert np.allclose(o, 0.75, atol=1e-14)


def test_prefill_rows_agrees_with_table():
    pool, req, kc, vc, rows = _c1_pipeline()
    o, _ = orc.attend_prefill(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0, rows, kc, vc, 1e4)
    pick = [(0, 0), (31, 3), (7, 2)]
    got = orc.prefill_rows(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0, rows, kc, vc, 1e4, pick)
    for n, (tok, h) in enumerate(pick):
        assert np.allclose(got[n], o[tok, h], atol=1e-13)


def test_decode_equals_last_prefill_row_and_paged_equals_packed():
    """Decoding the last conversation token over paged KV (resource pages from
    the compaction layout, history pages from the rotated conversation keys)
    gives the last row of the prefill over the same tokens."""
    pool, req, kc, vc, rows = _c1_pipeline()
    sh = pool.shape
    g, d, pt = sh.n_kv_heads, sh.head_dim, 16
    o, kconv_hat = orc.attend_prefill(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0, rows, kc, vc, sh.rope_theta)
    tq = req.total_q
    n_res_pages = [(len(rows[0][kg]) + pt - 1) // pt for kg in range(g)]
    n_hist_pages = (tq + pt - 1) // pt
    total = sum(n_res_pages) + g * n_hist_pages
    free = list(np.random.default_rng(3).permutation(total))
    res_pt, used = orc.page_layout(rows, free, pt, max(n_res_pages))
    k_pages = orc.gather_paged(kc, rows, res_pt, total, pt, fill=np.nan)
    v_pages = orc.gather_paged(vc, rows, res_pt, total, pt, fill=np.nan)
    hist_pt = np.array(free[used:used + g * n_hist_pages], dtype=np.int32).reshape(g, n_hist_pages)
    for kg in range(g):                       # history without the current token ...
        for n in range(tq - 1):
            k_pages[hist_pt[kg, n // pt], n % pt] = kconv_hat[n, kg]
            v_pages[hist_pt[kg, n // pt], n % pt] = f64(req.v_conv)[n, kg]
    hist_len = np.full(g, tq, np.int32)
    q_pos = np.array([64 + tq - 1])
    orc.append_decode_kv(k_pages, v_pages, hist_pt, hist_len, f64(req.k_conv)[tq - 1:tq], f64(req.v_conv)[tq - 1:tq],
                         q_pos, sh.rope_theta, pt)   # ... then the current token is appended
    res_len = np.array([len(rows[0][kg]) for kg in range(g)], np.int32)
    od = orc.attend_decode(f64(req.q)[tq - 1:tq], q_pos, k_pages, v_pages, res_pt, res_len, hist_pt, hist_len,
                           sh.rope_theta, pt)
    assert np.allclose(od[0], o[tq - 1], atol=1e-12)
    assert not np.isnan(od).any()             # never touched an unwritten page slot


def test_pair_counts():
    assert orc.useful_pairs_encode([1, 2, 3]) == 1 + 3 + 6
    assert orc.useful_pairs_prefill(4, 10) == 40 + 10


# ------------------------------------------- shared prefix / global positions --
def test_prefixed_encode_is_causal_attention_over_prefix_plus_resource():
    """One resource behind a shared prefix of P tokens, positions P..P+L-1, equals
    the resource rows of standard causal attention over [prefix ; resource]
    (torch fp64 SDPA); without a prefix the extended call is the plain one."""
    sh = wl.Shape(4, 2, 32, 1e4, "f32")
    P, L = 11, 23
    qp, kp, vp = wl.resource_tensors(5, 100, P, sh)
    q, k, v = wl.resource_tensors(5, 0, L, sh)
    pk = np.transpose(orc.rope(f64(kp), np.arange(P), sh.rope_theta), (1, 0, 2))       # [G][P][d], as a cache holds it
    pv = np.transpose(f64(vp), (1, 0, 2))
    o, k_hat, _ = orc.encode_resources(f64(q), f64(k), f64(v), [0, L], sh.rope_theta, pos_offset=[P],
                                       prefix_k=pk, prefix_v=pv)
    qa = torch.from_numpy(orc.rope(np.concatenate([f64(qp), f64(q)]), np.arange(P + L), sh.rope_theta))
    ka = torch.from_numpy(orc.rope(np.concatenate([f64(kp), f64(k)]), np.arange(P + L), sh.rope_theta))
    va = torch.from_numpy(np.concatenate([f64(vp), f64(v)]))
    want = torch.nn.functional.scaled_dot_product_attention(
        qa.permute(1, 0, 2)[None], ka.permute(1, 0, 2).repeat_interleave(2, 0)[None],
        va.permute(1, 0, 2).repeat_interleave(2, 0)[None], is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.allclose(o, want[P:], atol=1e-12)
    assert np.allclose(k_hat, ka.numpy()[P:], atol=1e-13)
    o0, _, _ = orc.encode_resources(f64(q), f64(k), f64(v), [0, L], sh.rope_theta)
    o1, _, _ = orc.encode_resources(f64(q), f64(k), f64(v), [0, L], sh.rope_theta, pos_offset=[0],
                                    prefix_k=np.zeros((2, 0, 32)), prefix_v=np.zeros((2, 0, 32)))
    assert np.array_equal(o0, o1)


def test_block_variant_no_cross_resource_attention_with_global_positions():
    """Global position offsets ("Block"): still no pair across resources, so each
    resource equals its own causal attention; with a prefix the offsets matter
    (the relative position to the prefix changes) and the result is the masked
    dense attention over [prefix ; all resources] with original positions."""
    sh = wl.TINY_F32
    lens = [9, 14, 6]
    P = 5
    parts = [wl.resource_tensors(13, r, n, sh) for r, n in enumerate(lens)]
    qp, kp, vp = wl.resource_tensors(13, 50, P, sh)
    q = np.concatenate([f64(p[0]) for p in parts]); k = np.concatenate([f64(p[1]) for p in parts])
    v = np.concatenate([f64(p[2]) for p in parts])
    cu = np.concatenate([[0], np.cumsum(lens)])
    offs = [P + int(cu[i]) for i in range(3)]                      # original positions after the prefix
    pk = np.transpose(orc.rope(f64(kp), np.arange(P), sh.rope_theta), (1, 0, 2)); pv = np.transpose(f64(vp), (1, 0, 2))
    o, _, _ = orc.encode_resources(q, k, v, cu, sh.rope_theta, pos_offset=offs, prefix_k=pk, prefix_v=pv)
    t = int(cu[-1])
    res_of = np.searchsorted(cu, np.arange(t), side="right") - 1
    s = sh.group_size
    for h in range(sh.n_q_heads):
        g = h // s
        qs = [brute_rope(list(q[n, h]), P + n, sh.rope_theta) for n in range(t)]
        ks = [brute_rope(list(f64(kp)[n, g]), n, sh.rope_theta) for n in range(P)] + \
             [brute_rope(list(k[n, g]), P + n, sh.rope_theta) for n in range(t)]
        vs = [list(f64(vp)[n, g]) for n in range(P)] + [list(v[n, g]) for n in range(t)]
        want = brute_attention(qs, ks, vs, lambda i, j: j < P or (res_of[j - P] == res_of[i] and j - P <= i))
        assert np.allclose(o[:, h, :], np.array(want), atol=1e-12)
    o_local, _, _ = orc.encode_resources(q, k, v, cu, sh.rope_theta, pos_offset=[P] * 3, prefix_k=pk, prefix_v=pv)
    assert np.abs(o_local - o)[cu[1]:].max() > 1e-3                # offsets do matter once there is a prefix
    assert np.allclose(o_local[:cu[1]], o[:cu[1]], atol=1e-12)     # ... except for the first resource (same offset)


# ------------------------------------------------------- multi-turn history --
def test_second_turn_with_history_equals_rows_of_one_long_prefill():
    """Turn 1 (20 tokens) then turn 2 (12 tokens) with turn 1 as all-visible
    history, positions continuing, gives the turn-2 rows of a single 32-token
    prefill (already pinned against brute force)."""
    pool, req, kc, vc, rows = _c1_pipeline()
    sh = pool.shape
    q, k, v = f64(req.q), f64(req.k_conv), f64(req.v_conv)
    o_all, kh_all = orc.attend_prefill(q, k, v, req.cu_q, req.q_pos0, rows, kc, vc, sh.rope_theta)
    n1 = 20
    o1, kh1 = orc.attend_prefill(q[:n1], k[:n1], v[:n1], [0, n1], [64], rows, kc, vc, sh.rope_theta)
    assert np.allclose(o1, o_all[:n1], atol=1e-12)
    hist_k = [np.transpose(kh1, (1, 0, 2))]; hist_v = [np.transpose(v[:n1], (1, 0, 2))]
    o2, _ = orc.attend_prefill(q[n1:], k[n1:], v[n1:], [0, 32 - n1], [64 + n1], rows, kc, vc, sh.rope_theta,
                               hist_k=hist_k, hist_v=hist_v)
    assert np.allclose(o2, o_all[n1:], atol=1e-12)
