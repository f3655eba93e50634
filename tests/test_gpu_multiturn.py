"""Multi-turn path on the GPU: a first turn, a second turn that sees the first
as history, then a short decode loop whose history pages ARE the conversation
cache the prefills wrote (64-aligned slots), all against the oracle."""
import numpy as np
import pytest
import torch

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl

from pipeline import dev, f64, gpu_compact, gpu_encode, make_ctx, max_abs, oracle_encode, oracle_rows

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,tol", [(wl.QWEN3_4B, 1e-2), (wl.TINY_F32, 1e-5)])
def test_two_turns_then_decode_loop(shape, tol):
    from paper_2608_19662_b200 import PAGED
    sh = shape
    g, d, s, pt = sh.n_kv_heads, sh.head_dim, sh.group_size, wl.PAGE_TOKENS
    rng = np.random.default_rng(77)
    lens = [90, 150, 40, 200]
    pool = wl.pack_resources(sh, 77, lens, wl.keep_mask_spans(rng, lens))
    res_lists = [[0, 2, 3], [1], [3, 0]]
    vis = [wl.routes_random(rng, g, len(l), 0.5) for l in res_lists]
    len1, len2, n_dec = [70, 33, 130], [64, 64, 10], 3
    B = len(res_lists)
    pos_first = [int(pool.lens[l].sum()) for l in res_lists]
    rc = make_ctx(sh, max_pos=2048)
    _, kc_ref, vc_ref = oracle_encode(pool)
    _, kc, vc = gpu_encode(rc, pool)

    # one page pool: [resource pages | conversation cache]; request b owns 256 cache rows per group
    slot_rows = 256
    cache_rows = B * slot_rows
    conv_slot = np.arange(B, dtype=np.int32) * slot_rows
    req1 = wl.make_requests(sh, 5, pool, res_lists, vis, len1, q_pos0=pos_first)
    rows = oracle_rows(pool, req1)
    n_res_pages = [[(len(r) + pt - 1) // pt for r in per] for per in rows]
    R = sum(sum(x) for x in n_res_pages) + 2
    n_pages = R + g * cache_rows // pt
    k_pool = torch.full((n_pages, pt, d), float("nan"), dtype=sh.torch_dtype, device="cuda")
    v_pool = torch.full_like(k_pool, float("nan"))
    k_conv_cache = k_pool[R:].view(g, cache_rows, d)
    v_conv_cache = v_pool[R:].view(g, cache_rows, d)

    # packed route KV for the prefills, paged route KV (same rows) for the decode steps
    packed = gpu_compact(rc, pool, req1, kc, vc)
    max_rp = max(max(x) for x in n_res_pages) + 1
    n_routes = B * g
    d_cu = torch.empty(n_routes + 1, dtype=torch.int32, device="cuda"); d_len = torch.empty(n_routes, dtype=torch.int32, device="cuda")
    d_idx = torch.empty(int(packed["route_cu"][-1]) + 8, dtype=torch.int32, device="cuda")
    d_pt = torch.empty((n_routes, max_rp), dtype=torch.int32, device="cuda")
    free = dev(np.random.default_rng(1).permutation(R).astype(np.int32))
    rc.compact_routes(kc, vc, dev(pool.keep), dev(req1.res_off), dev(req1.res_slot), dev(req1.res_len), dev(req1.vis), PAGED,
                      d_cu, d_idx, k_pool, v_pool, route_len=d_len, page_table=d_pt, free_pages=free)

    # ---- turn 1 (no history yet) ----
    zeros = np.zeros(B, np.int32)
    o1 = rc.attend_prefill_history(dev(req1.q), dev(req1.k_conv), dev(req1.v_conv), dev(req1.cu_q), dev(req1.q_pos0),
                                   req1.max_q, packed["k_out"], packed["v_out"], packed["route_cu"], k_conv_cache,
                                   v_conv_cache, dev(conv_slot), dev(zeros), out_dtype=torch.float32)
    r1, kh1 = orc.attend_prefill(f64(req1.q), f64(req1.k_conv), f64(req1.v_conv), req1.cu_q, req1.q_pos0, rows,
                                 kc_ref, vc_ref, sh.rope_theta, storage=sh.dtype)
    assert max_abs(o1, r1) < tol
    hist_k = [np.transpose(kh1[req1.cu_q[b]:req1.cu_q[b + 1]], (1, 0, 2)) for b in range(B)]
    hist_v = [np.transpose(f64(req1.v_conv)[req1.cu_q[b]:req1.cu_q[b + 1]], (1, 0, 2)) for b in range(B)]

    # ---- turn 2: sees turn 1 as history, positions continue ----
    req2 = wl.make_requests(sh, 6, pool, res_lists, vis, len2, q_pos0=[p + n for p, n in zip(pos_first, len1)])
    o2 = rc.attend_prefill_history(dev(req2.q), dev(req2.k_conv), dev(req2.v_conv), dev(req2.cu_q), dev(req2.q_pos0),
                                   req2.max_q, packed["k_out"], packed["v_out"], packed["route_cu"], k_conv_cache,
                                   v_conv_cache, dev(conv_slot), dev(np.asarray(len1, np.int32)), out_dtype=torch.float32)
    r2, kh2 = orc.attend_prefill(f64(req2.q), f64(req2.k_conv), f64(req2.v_conv), req2.cu_q, req2.q_pos0, rows,
                                 kc_ref, vc_ref, sh.rope_theta, storage=sh.dtype, hist_k=hist_k, hist_v=hist_v)
    assert max_abs(o2, r2) < tol
    for b in range(B):
        hist_k[b] = np.concatenate([hist_k[b], np.transpose(kh2[req2.cu_q[b]:req2.cu_q[b + 1]], (1, 0, 2))], 1)
        hist_v[b] = np.concatenate([hist_v[b], np.transpose(f64(req2.v_conv)[req2.cu_q[b]:req2.cu_q[b + 1]], (1, 0, 2))], 1)
    # the cache now holds both turns, contiguous per request: values are byte copies
    for b in range(B):
        n = len1[b] + len2[b]
        got_v = f64(v_conv_cache[:, conv_slot[b]:conv_slot[b] + n])
        assert np.array_equal(got_v, hist_v[b])
        assert torch.isnan(v_conv_cache[:, conv_slot[b] + n:conv_slot[b] + slot_rows]).all()

    # ---- decode loop: history pages = the conversation cache, viewed as 64-token pages ----
    hist_pt = np.zeros((n_routes, slot_rows // pt), np.int32)
    for b in range(B):
        for kg in range(g):
            hist_pt[b * g + kg] = R + (kg * cache_rows + conv_slot[b]) // pt + np.arange(slot_rows // pt)
    cur = np.asarray([a + c for a, c in zip(len1, len2)], np.int32)
    for step in range(n_dec):
        qd = wl.normal(300 + step, (B, sh.n_q_heads, d), sh.torch_dtype)
        kn = wl.normal(400 + step, (B, g, d), sh.torch_dtype)
        vn = wl.normal(500 + step, (B, g, d), sh.torch_dtype)
        q_pos = np.asarray([p + int(c) for p, c in zip(pos_first, cur)], np.int32)
        hist_len = np.repeat(cur + 1, g).astype(np.int32)
        od = rc.attend_decode(dev(qd), dev(q_pos), k_pool, v_pool, d_pt, d_len, dev(hist_pt), dev(hist_len),
                              k_new=dev(kn), v_new=dev(vn), out_dtype=torch.float32)
        # oracle: a one-token "turn" with everything before it as history
        cu1 = np.arange(B + 1, dtype=np.int32)
        rd, khd = orc.attend_prefill(f64(qd), f64(kn), f64(vn), cu1, q_pos, rows, kc_ref, vc_ref, sh.rope_theta,
                                     storage=sh.dtype, hist_k=hist_k, hist_v=hist_v)
        assert max_abs(od, rd) < tol, step
        for b in range(B):
            hist_k[b] = np.concatenate([hist_k[b], np.transpose(khd[b:b + 1], (1, 0, 2))], 1)
            hist_v[b] = np.concatenate([hist_v[b], np.transpose(f64(vn)[b:b + 1], (1, 0, 2))], 1)
        cur = cur + 1
    assert rc.poll_status() == 0
