"""Attention-only scaling sweeps on one GPU, through the library's public calls.

`python -m paper_2608_19662_b200.sweep buckets` — the paper's scaling study
(Section "Scalability", requests bucketed by total resource length D_R) restated
for the attention path alone: for each D_R, one layer's time to first token
analogue (dense causal prefill over resources + conversation; cache hit with
every route and every token visible; routed and pruned, materialised or
zero-copy) and one decode step (dense history against routed pages), plus the
resource KV bytes each variant materialises.

`python -m paper_2608_19662_b200.sweep budgets` — structural budgets
Omega_{K_L,K_G} (Section "Structural routing", the appendix's contribution
weights): sparsity rho against the prefill attention time summed over all layers,
for the 36-layer / 4-heads-per-group and the 28-layer / 2-heads-per-group shape.

Every line printed is one JSON object.  Inputs are seeded N(0,1) tensors drawn on
the device (stand-ins for activations and for an earlier encode's cache); times are
CUDA-event means over `--iters` runs after 3 warm-up runs, L2 not flushed (the
small buckets fit in L2: that is what a serving loop would see too)."""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import PACKED, ReCache, binding
from . import workloads as wl


def _timed(fn, iters):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def _dev(a, device):
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


class _Pool:
    """Index data of B requests x N resources of equal length (the tensors live on the device only)."""

    def __init__(self, sh, batch, n_res, res_len, keep_ratio_spans, rng):
        self.lens = np.full(batch * n_res, res_len, np.int32)
        self.slot = (np.arange(batch * n_res, dtype=np.int64) * res_len).astype(np.int32)
        self.pool_tokens = int(batch * n_res * res_len)
        masks = wl.keep_mask_spans(rng, self.lens) if keep_ratio_spans else [np.ones(res_len, np.uint8)] * (batch * n_res)
        self.keep = np.concatenate(masks).astype(np.uint8)
        self.res_off = (np.arange(batch + 1) * n_res).astype(np.int32)


def _prefill_variant(rc, sh, pool, vis, tq, batch, device, gather, iters):
    """compaction (+ materialisation unless `gather`) and the prefill of `tq` tokens per request."""
    g, d, dt = sh.n_kv_heads, sh.head_dim, sh.torch_dtype
    kc = wl.seeded_normal(11, (g, pool.pool_tokens, d), dt, device=device)
    vc = wl.seeded_normal(12, (g, pool.pool_tokens, d), dt, device=device)
    keep, res_off = _dev(pool.keep, device), _dev(pool.res_off, device)
    res_slot, res_len, dvis = _dev(pool.slot, device), _dev(pool.lens, device), _dev(vis, device)
    n_routes = batch * g
    kept = np.array([int(pool.keep[s:s + n].sum()) for s, n in zip(pool.slot, pool.lens)])
    cap = int((vis.astype(np.int64) * kept[None, :]).sum()) + 64
    route_cu = torch.empty(n_routes + 1, dtype=torch.int32, device=device)
    route_idx = torch.empty(cap, dtype=torch.int32, device=device)
    k_route = v_route = None
    if not gather:
        k_route, v_route = torch.empty((cap, d), dtype=dt, device=device), torch.empty((cap, d), dtype=dt, device=device)
    tot = batch * tq
    q = wl.seeded_normal(13, (tot, sh.n_q_heads, d), dt, device=device)
    kq = wl.seeded_normal(14, (tot, g, d), dt, device=device)
    vq = wl.seeded_normal(15, (tot, g, d), dt, device=device)
    cu_q = _dev((np.arange(batch + 1) * tq).astype(np.int32), device)
    n_res = len(pool.lens) // batch
    q_pos0 = _dev(np.full(batch, n_res * int(pool.lens[0]), np.int32), device)
    out = torch.empty((tot, sh.n_q_heads, d), dtype=dt, device=device)
    ko, vo = torch.empty((g, tot, d), dtype=dt, device=device), torch.empty((g, tot, d), dtype=dt, device=device)

    def run():
        rc.compact_routes(kc, vc, keep, res_off, res_slot, res_len, dvis, PACKED, route_cu, route_idx, k_route, v_route)
        if gather:
            rc.attend_prefill_gather(q, kq, vq, cu_q, q_pos0, tq, kc, vc, route_idx, route_cu, k_conv_out=ko, v_conv_out=vo, out=out)
        else:
            rc.attend_prefill(q, kq, vq, cu_q, q_pos0, tq, k_route, v_route, route_cu, k_conv_out=ko, v_conv_out=vo, out=out)

    ms = _timed(run, iters)
    rows = int(route_cu[-1].item())
    return ms, rows, (0 if gather else rows * d * 2 * 2)


def _dense_prefill(rc, sh, total_len, batch, device, iters):
    """One causal sequence of resources + conversation per request: what a model without a resource cache does."""
    g, d, dt = sh.n_kv_heads, sh.head_dim, sh.torch_dtype
    tot = batch * total_len
    q = wl.seeded_normal(21, (tot, sh.n_q_heads, d), dt, device=device)
    k = wl.seeded_normal(22, (tot, g, d), dt, device=device)
    v = wl.seeded_normal(23, (tot, g, d), dt, device=device)
    cu = _dev((np.arange(batch + 1) * total_len).astype(np.int32), device)
    slot = _dev((np.arange(batch) * total_len).astype(np.int32), device)
    kc, vc = torch.empty((g, tot, d), dtype=dt, device=device), torch.empty((g, tot, d), dtype=dt, device=device)
    out = torch.empty((tot, sh.n_q_heads, d), dtype=dt, device=device)
    return _timed(lambda: rc.encode_resources(q, k, v, cu, total_len, slot, kc, vc, out=out), iters), tot * g * d * 2 * 2


def _decode(rc, sh, batch, route_rows, hist_rows, device, iters):
    """One decode step: `route_rows` resource rows and `hist_rows` history rows per (sequence, group)."""
    g, d, dt, pt = sh.n_kv_heads, sh.head_dim, sh.torch_dtype, wl.PAGE_TOKENS
    items = batch * g
    rp, hp = (route_rows + pt - 1) // pt, (hist_rows + pt - 1) // pt
    n_pages = items * (rp + hp) + 1
    kp = wl.seeded_normal(31, (n_pages, pt, d), dt, device=device)
    vp = wl.seeded_normal(32, (n_pages, pt, d), dt, device=device)
    ids = np.random.default_rng(7).permutation(n_pages - 1).astype(np.int32)
    rpt = ids[:items * rp].reshape(items, rp) if rp else np.zeros((items, 1), np.int32)
    hpt = ids[items * rp:items * (rp + hp)].reshape(items, hp)
    q = wl.seeded_normal(33, (batch, sh.n_q_heads, d), dt, device=device)
    q_pos = _dev(np.full(batch, route_rows + hist_rows, np.int32), device)
    rlen, hlen = _dev(np.full(items, route_rows, np.int32), device), _dev(np.full(items, hist_rows, np.int32), device)
    d_rpt, d_hpt = _dev(rpt, device), _dev(hpt, device)
    out = torch.empty((batch, sh.n_q_heads, d), dtype=dt, device=device)
    return _timed(lambda: rc.attend_decode(q, q_pos, kp, vp, d_rpt, rlen, d_hpt, hlen, out=out), iters)


def sweep_buckets(args):
    sh = wl.QWEN3_4B
    device = torch.device("cuda", args.device)
    g = sh.n_kv_heads
    for d_r in args.lengths:
        n_res, batch, tq = args.n_res, args.batch, args.tq
        res_len = max(1, d_r // n_res)
        rng = np.random.default_rng(d_r)
        rc = ReCache(sh.n_q_heads, g, sh.head_dim, sh.rope_theta, sh.dtype, max_pos=n_res * res_len + tq + 2,
                     page_tokens=wl.PAGE_TOKENS, device=args.device)
        full = _Pool(sh, batch, n_res, res_len, False, rng)
        pruned = _Pool(sh, batch, n_res, res_len, True, rng)
        vis_all = np.ones((g, batch * n_res), np.uint8)
        vis_routed = np.concatenate([wl.routes_random(rng, g, n_res, args.route_frac) for _ in range(batch)], axis=1)
        ms_dense, kv_dense = _dense_prefill(rc, sh, n_res * res_len + tq, batch, device, args.iters)
        ms_full, rows_full, kv_full = _prefill_variant(rc, sh, full, vis_all, tq, batch, device, False, args.iters)
        ms_rc, rows_rc, kv_rc = _prefill_variant(rc, sh, pruned, vis_routed, tq, batch, device, False, args.iters)
        ms_zc, _, _ = _prefill_variant(rc, sh, pruned, vis_routed, tq, batch, device, True, args.iters)
        route_rows = rows_rc // (batch * g)
        ms_dec_dense = _decode(rc, sh, batch, 0, n_res * res_len + tq + 1, device, args.iters)
        ms_dec_rc = _decode(rc, sh, batch, route_rows, tq + 1, device, args.iters)
        if rc.poll_status() != 0:
            raise SystemExit("device status after bucket %d: %s" % (d_r, rc.last_error()))
        rc.close()
        print(json.dumps({
            "sweep": "buckets", "resource_tokens_per_request": n_res * res_len, "requests": batch, "query_tokens": tq,
            "layer_prefill_ms": {"dense_causal": round(ms_dense, 4), "cache_hit_all_visible": round(ms_full, 4),
                                 "routed_pruned": round(ms_rc, 4), "routed_pruned_zero_copy": round(ms_zc, 4)},
            "prefill_speedup_vs_dense": {"cache_hit_all_visible": round(ms_dense / ms_full, 2),
                                         "routed_pruned": round(ms_dense / ms_rc, 2)},
            "layer_decode_ms": {"dense_history": round(ms_dec_dense, 4), "routed_pruned": round(ms_dec_rc, 4),
                                "speedup": round(ms_dec_dense / ms_dec_rc, 2)},
            "retained_rows_per_route": route_rows, "retained_fraction": round(rows_rc / max(rows_full, 1), 4),
            "resource_kv_bytes_materialised": {"dense_causal": kv_dense, "cache_hit_all_visible": kv_full,
                                               "routed_pruned": kv_rc, "routed_pruned_zero_copy": 0}}), flush=True)


def _load_weights(path):
    """{(model, "layer" | "group"): {unit (1-based): weight in percent}} from the text fixture of printed weights."""
    w = {}
    for line in open(path):
        f = line.split()
        if not f or f[0].startswith("#") or f[0] == "budget":
            continue
        w.setdefault((f[0], f[1]), {})[int(f[2])] = float(f[3])
    return w


def sweep_budgets(args):
    device = torch.device("cuda", args.device)
    path = args.weights
    models = [("Ql", wl.QWEN3_4B, 36), ("Qs", wl.Shape(16, 8, 128, 1e6, "bf16"), 28)]
    for tag, sh, n_layers in models:
        g = sh.n_kv_heads
        if path and os.path.exists(path):
            w = _load_weights(path)
            s_l = np.array([w[(tag, "layer")][i + 1] for i in range(n_layers)])
            s_g = np.array([w[(tag, "group")][i + 1] for i in range(g)])
            src = "printed contribution weights"
        else:
            rng = np.random.default_rng(n_layers)
            s_l, s_g = rng.exponential(1.0, n_layers), rng.exponential(1.0, g)
            src = "seeded exponential scores (no weight file given)"
        batch, n_res, res_len, tq = args.batch, args.n_res, args.res_len, args.tq
        rng = np.random.default_rng(99)
        pool = _Pool(sh, batch, n_res, res_len, True, rng)
        rc = ReCache(sh.n_q_heads, g, sh.head_dim, sh.rope_theta, sh.dtype, max_pos=n_res * res_len + tq + 2,
                     page_tokens=wl.PAGE_TOKENS, device=args.device)
        seen = set()
        for k_l, k_g in args.budgets:
            k_l, k_g = min(k_l, n_layers), min(k_g, g)
            if (k_l, k_g) in seen:      # two budgets that clamp to the same one for this model
                continue
            seen.add((k_l, k_g))
            omega, cc_l, cc_g, rho = binding.build_routes(s_l, s_g, k_l, k_g)
            # a layer's time depends only on how many of its groups have a route (all or none of the resources)
            per_count = {}
            total = 0.0
            for layer in range(n_layers):
                n_on = int(omega[layer].sum())
                if n_on not in per_count:
                    vis = np.zeros((g, batch * n_res), np.uint8)
                    vis[np.flatnonzero(omega[layer])] = 1
                    per_count[n_on] = _prefill_variant(rc, sh, pool, vis, tq, batch, device, False, args.iters)[0]
                total += per_count[n_on]
            print(json.dumps({"sweep": "budgets", "model": tag, "scores": src, "layers": n_layers, "groups": g,
                              "heads_per_group": sh.group_size, "k_layers": k_l, "k_groups": k_g,
                              "rho": round(rho, 4), "coverage_layers": round(cc_l, 4), "coverage_groups": round(cc_g, 4),
                              "prefill_attention_ms_all_layers": round(total, 3),
                              "workload": "%d requests x %d resources of %d tokens (30%% kept), %d query tokens" % (
                                  batch, n_res, res_len, tq)}), flush=True)
        if rc.poll_status() != 0:
            raise SystemExit("device status after the budget sweep: " + rc.last_error())
        rc.close()


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    sub = ap.add_subparsers(dest="what", required=True)
    b = sub.add_parser("buckets")
    b.add_argument("--lengths", type=int, nargs="+", default=[1024, 2048, 4096, 8192, 16384, 32768])
    b.add_argument("--n-res", type=int, default=16)
    b.add_argument("--batch", type=int, default=8)
    b.add_argument("--tq", type=int, default=256)
    b.add_argument("--route-frac", type=float, default=0.25)
    u = sub.add_parser("budgets")
    u.add_argument("--weights", default=os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "tests", "golden",
                                                     "contribution_weights.txt"))
    u.add_argument("--budgets", type=lambda s: tuple(int(x) for x in s.split(",")), nargs="+",
                   default=[(36, 8), (28, 8), (20, 8), (20, 5), (20, 3), (12, 3), (20, 7), (4, 1)])
    u.add_argument("--n-res", type=int, default=16)
    u.add_argument("--res-len", type=int, default=1024)
    u.add_argument("--batch", type=int, default=8)
    u.add_argument("--tq", type=int, default=512)
    for p in (b, u):
        p.add_argument("--iters", type=int, default=20)
        p.add_argument("--device", type=int, default=0)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("the sweeps need a CUDA device")
    (sweep_buckets if args.what == "buckets" else sweep_budgets)(args)


if __name__ == "__main__":
    main()
