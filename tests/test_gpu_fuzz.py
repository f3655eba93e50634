"""Seeded random small cases through the whole bf16 path (encode, compaction,
prefill with and without history, decode over paged and gathered rows) against
the oracle: lengths, routes, masks and request shapes nobody hand-picked."""
import numpy as np
import pytest
import torch

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl

from pipeline import dev, f64, gpu_compact, gpu_encode, make_ctx, max_abs, oracle_encode, oracle_rows

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", list(range(8)))
def test_random_case(seed):
    from paper_2608_19662_b200 import PACKED
    rng = np.random.default_rng(1000 + seed)
    sh = [wl.QWEN3_4B, wl.Shape(16, 8, 128, 1e6, "bf16"), wl.Shape(16, 2, 128, 1e4, "bf16")][seed % 3]
    g, d, pt = sh.n_kv_heads, sh.head_dim, wl.PAGE_TOKENS
    n_res = int(rng.integers(1, 7))
    lens = [int(x) for x in rng.integers(1, 330, n_res)]
    if seed % 4 == 0:
        lens[0] = 0 if n_res > 1 else lens[0]                       # an empty resource now and then
    masks = wl.keep_mask_bernoulli(rng, lens, float(rng.uniform(0.05, 0.9)), "last")
    pool = wl.pack_resources(sh, 2000 + seed, lens, masks, slot_gap=int(rng.integers(0, 9)))
    B = int(rng.integers(1, 4))
    res_lists = [[int(x) for x in rng.permutation(n_res)[:int(rng.integers(0, n_res + 1))]] for _ in range(B)]
    vis = [(rng.random((g, len(l))) < 0.5).astype(np.uint8) for l in res_lists]
    tq = [int(x) for x in rng.integers(1, 160, B)]
    hist = [int(x) for x in rng.integers(0, 150, B)]
    pos0 = [int(x) for x in rng.integers(0, 3000, B)]
    rc = make_ctx(sh, max_pos=4096)

    o_ref, kc_ref, vc_ref = oracle_encode(pool)
    o, kc, vc = gpu_encode(rc, pool)
    assert max_abs(o, o_ref) < 1e-2
    req = wl.make_requests(sh, 3000 + seed, pool, res_lists, vis, tq, q_pos0=[p + h for p, h in zip(pos0, hist)])
    rows = oracle_rows(pool, req)
    out = gpu_compact(rc, pool, req, kc, vc)
    cu = orc.route_prefix(rows)
    assert np.array_equal(out["route_cu"].cpu().numpy(), cu)
    if cu[-1]:
        assert np.array_equal(out["route_idx"].cpu().numpy()[:cu[-1]], np.concatenate([r for per in rows for r in per]))

    # earlier turns: random rotated keys / values already in the conversation cache (64-aligned slots)
    slot_rows = 384
    conv_slot = (np.arange(B) * slot_rows).astype(np.int32)
    hk = [orc.round_bf16(rng.standard_normal((g, h, d))) for h in hist]
    hv = [orc.round_bf16(rng.standard_normal((g, h, d))) for h in hist]
    n_res_pages = 8 * B * g
    k_pool = torch.full((n_res_pages + g * B * slot_rows // pt, pt, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    v_pool = torch.full_like(k_pool, float("nan"))
    kcache = k_pool[n_res_pages:].view(g, B * slot_rows, d); vcache = v_pool[n_res_pages:].view(g, B * slot_rows, d)
    for b in range(B):
        if hist[b]:
            kcache[:, conv_slot[b]:conv_slot[b] + hist[b]] = dev(hk[b]).to(torch.bfloat16)
            vcache[:, conv_slot[b]:conv_slot[b] + hist[b]] = dev(hv[b]).to(torch.bfloat16)
    p = rc.attend_prefill_history(dev(req.q), dev(req.k_conv), dev(req.v_conv), dev(req.cu_q), dev(req.q_pos0), req.max_q,
                                  out["k_out"], out["v_out"], out["route_cu"], kcache, vcache, dev(conv_slot),
                                  dev(np.asarray(hist, np.int32)), out_dtype=torch.float32)
    p_ref, kh = orc.attend_prefill(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0, rows, kc_ref, vc_ref,
                                   sh.rope_theta, storage="bf16", hist_k=hk, hist_v=hv)
    assert max_abs(p, p_ref) < 1e-2

    # one decode step on top (gathered resource rows, history = the conversation cache as pages)
    for b in range(B):
        hk[b] = np.concatenate([hk[b], np.transpose(kh[req.cu_q[b]:req.cu_q[b + 1]], (1, 0, 2))], 1)
        hv[b] = np.concatenate([hv[b], np.transpose(f64(req.v_conv)[req.cu_q[b]:req.cu_q[b + 1]], (1, 0, 2))], 1)
    cur = np.asarray([h + t for h, t in zip(hist, tq)], np.int32)
    hist_pt = np.stack([n_res_pages + (kg * B * slot_rows + conv_slot[b]) // pt + np.arange(slot_rows // pt)
                        for b in range(B) for kg in range(g)]).astype(np.int32)
    qd = wl.normal(4000 + seed, (B, sh.n_q_heads, d), torch.bfloat16)
    kn = wl.normal(4100 + seed, (B, g, d), torch.bfloat16); vn = wl.normal(4200 + seed, (B, g, d), torch.bfloat16)
    q_pos = np.asarray([pp + int(c) for pp, c in zip(pos0, cur)], np.int32)
    max_rp = max(1, max((len(r) + pt - 1) // pt for per in rows for r in per))
    od = rc.attend_decode_gather(dev(qd), dev(q_pos), kc, vc, out["route_idx"], out["route_cu"], max_rp, k_pool, v_pool,
                                 dev(hist_pt), dev(np.repeat(cur + 1, g).astype(np.int32)), k_new=dev(kn), v_new=dev(vn),
                                 out_dtype=torch.float32)
    rd, _ = orc.attend_prefill(f64(qd), f64(kn), f64(vn), np.arange(B + 1), q_pos, rows, kc_ref, vc_ref, sh.rope_theta,
                               storage="bf16", hist_k=hk, hist_v=hv)
    assert max_abs(od, rd) < 1e-2
    assert rc.poll_status() == 0


@pytest.mark.parametrize("seed", list(range(6)))
def test_random_multi_tile_case(seed):
    """The same idea at sizes that span many K/V tiles: resources of up to 1600 tokens, up to 700 query
    tokens per request, 2 / 4 / 8 query heads per KV group, span-shaped keep masks, gaps between cache slots;
    encode, compaction, packed prefill and the zero-copy prefill (which must agree bit for bit)."""
    from pipeline import gpu_prefill, oracle_prefill
    rng = np.random.default_rng(7000 + seed)
    sh = [wl.QWEN3_4B, wl.Shape(16, 8, 128, 1e6, "bf16"), wl.Shape(16, 2, 128, 1e4, "bf16")][seed % 3]
    g = sh.n_kv_heads
    n_res = int(rng.integers(2, 6))
    lens = [int(x) for x in rng.integers(100, 1600, n_res)]
    pool = wl.pack_resources(sh, 8000 + seed, lens, wl.keep_mask_spans(rng, lens), slot_gap=int(rng.integers(0, 70)))
    B = int(rng.integers(1, 4))
    res_lists = [[int(x) for x in rng.permutation(n_res)[:int(rng.integers(1, n_res + 1))]] for _ in range(B)]
    vis = [(rng.random((g, len(l))) < 0.6).astype(np.uint8) for l in res_lists]
    tq = [int(x) for x in rng.integers(1, 700, B)]
    rc = make_ctx(sh, max_pos=16384)
    o_ref, kc_ref, vc_ref = oracle_encode(pool)
    o, kc, vc = gpu_encode(rc, pool)
    assert max_abs(o, o_ref) < 1e-2
    req = wl.make_requests(sh, 9000 + seed, pool, res_lists, vis, tq)
    rows = oracle_rows(pool, req)
    out = gpu_compact(rc, pool, req, kc, vc)
    assert np.array_equal(out["route_cu"].cpu().numpy(), orc.route_prefix(rows))
    p, _, _ = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"])
    p_ref, _ = oracle_prefill(req, rows, kc_ref, vc_ref)
    assert max_abs(p, p_ref) < 1e-2
    p_g, _, _ = rc.attend_prefill_gather(dev(req.q), dev(req.k_conv), dev(req.v_conv), dev(req.cu_q), dev(req.q_pos0),
                                         req.max_q, kc, vc, out["route_idx"], out["route_cu"], out_dtype=torch.float32)
    assert torch.equal(p_g, p)
    assert rc.poll_status() == 0
