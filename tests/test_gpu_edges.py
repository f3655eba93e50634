"""Edge cases of the CUDA path against the oracle: ragged and empty inputs, tile
boundaries, degenerate routes and masks, other head layouts, and the error
reporting that must never trap (device status word, host status codes)."""
import numpy as np
import pytest
import torch

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl

from pipeline import (dev, f64, gpu_compact, gpu_encode, gpu_prefill, make_ctx, max_abs, oracle_encode,
                      oracle_prefill, oracle_rows)

pytestmark = pytest.mark.gpu

TOL_BF16 = 1e-2


def _pool(shape, lens, seed=21, slot_gap=0, keep="spans"):
    rng = np.random.default_rng(seed)
    masks = wl.keep_mask_spans(rng, lens) if keep == "spans" else keep
    return wl.pack_resources(shape, seed, lens, masks, slot_gap=slot_gap)


def test_encode_lengths_around_tile_boundaries_and_empty_resources():
    """Lengths 0, 1 and every boundary of the 32/64-token query tiles and the
    128-row key tiles, with gaps of unwritten (NaN) cache rows in between."""
    sh = wl.QWEN3_4B
    lens = [1, 0, 31, 32, 33, 63, 64, 65, 127, 128, 129, 0, 255, 256, 257, 385]
    pool = _pool(sh, lens, slot_gap=5)
    rc = make_ctx(sh, max_pos=4096)
    o_ref, kc_ref, vc_ref = oracle_encode(pool)
    o, kc, vc = gpu_encode(rc, pool)
    assert max_abs(o, o_ref) < TOL_BF16
    s = sh.group_size
    assert torch.equal(o[0].cpu(), pool.v[0].repeat_interleave(s, 0).float())     # one-token resource: O = v
    written = ~np.isnan(kc_ref)
    assert np.array_equal(np.isnan(f64(kc)), ~written)
    assert rc.poll_status() == 0


@pytest.mark.parametrize("hq,g,d", [(16, 8, 128), (32, 4, 128), (8, 8, 128), (8, 2, 64)])
def test_other_head_layouts(hq, g, d):
    """2 and 8 query heads per group (tensor-core path), 1 per group and head_dim 64 (row kernels)."""
    sh = wl.Shape(hq, g, d, 1e6, "bf16")
    pool = _pool(sh, [70, 130, 33])
    rng = np.random.default_rng(3)
    vis = wl.routes_random(rng, g, 3, 0.4)
    req = wl.make_requests(sh, 5, pool, [[2, 0, 1]], [vis], [77])
    rc = make_ctx(sh, max_pos=2048)
    o_ref, kc_ref, vc_ref = oracle_encode(pool)
    o, kc, vc = gpu_encode(rc, pool)
    assert max_abs(o, o_ref) < TOL_BF16
    rows = oracle_rows(pool, req)
    out = gpu_compact(rc, pool, req, kc, vc)
    assert np.array_equal(out["route_cu"].cpu().numpy(), orc.route_prefix(rows))
    p_ref, _ = oracle_prefill(req, rows, kc_ref, vc_ref)
    p, _, _ = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"])
    assert max_abs(p, p_ref) < TOL_BF16
    assert rc.poll_status() == 0


def test_degenerate_routes_masks_and_ragged_requests():
    """Empty route (context-only mask), a resource whose mask keeps nothing, a
    request that lists no resource, the paper's product routes (a group sees
    all resources or none), requests of 1 / 31 / 65 / 200 tokens."""
    sh = wl.QWEN3_4B
    lens = [90, 40, 150, 64]
    rng = np.random.default_rng(8)
    masks = wl.keep_mask_spans(rng, lens)
    masks[1][:] = 0                                   # nothing retained from resource 1
    pool = wl.pack_resources(sh, 31, lens, masks)
    g = sh.n_kv_heads
    omega_row = np.array([1, 0, 1, 1, 0, 0, 1, 0], np.uint8)              # product routes: groups in / out
    vis_a = np.repeat(omega_row[:, None], 3, axis=1)
    vis_b = np.zeros((g, 0), np.uint8)                                    # request 1 lists nothing
    vis_c = np.zeros((g, 2), np.uint8); vis_c[0, 0] = 1; vis_c[3, :] = 1  # only resource 1 (empty mask) on group 0
    vis_d = np.ones((g, 4), np.uint8)
    req = wl.make_requests(sh, 9, pool, [[0, 1, 2], [], [1, 3], [3, 2, 1, 0]], [vis_a, vis_b, vis_c, vis_d],
                           [31, 1, 65, 200], q_pos0=[300, 0, 7, 1000])
    rc = make_ctx(sh, max_pos=4096)
    _, kc_ref, vc_ref = oracle_encode(pool)
    _, kc, vc = gpu_encode(rc, pool)
    rows = oracle_rows(pool, req)
    assert len(rows[0][1]) == 0 and len(rows[1][0]) == 0 and len(rows[2][0]) == 0 and len(rows[2][3]) > 0
    out = gpu_compact(rc, pool, req, kc, vc)
    cu = orc.route_prefix(rows)
    assert np.array_equal(out["route_cu"].cpu().numpy(), cu)
    flat = np.concatenate([r for per in rows for r in per])
    assert np.array_equal(out["route_idx"].cpu().numpy()[:cu[-1]], flat)
    p_ref, _ = oracle_prefill(req, rows, kc_ref, vc_ref)
    p, _, _ = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"])
    assert max_abs(p, p_ref) < TOL_BF16
    assert rc.poll_status() == 0


def test_paged_compaction_many_routes_bit_exact():
    """More routes than one scan block (B*G > 1024), paged layout, shuffled free list."""
    from paper_2608_19662_b200 import PAGED
    sh = wl.Shape(8, 8, 128, 1e6, "bf16")
    dc = wl.config4_compose(batch=140, n_res=3, res_len=(20, 150), hist=64, shape=sh)
    rc = make_ctx(sh, max_pos=4096)
    g, d = sh.n_kv_heads, sh.head_dim
    kc = wl.seeded_normal(5, (g, dc.pool_tokens, d), torch.bfloat16, device="cuda")
    vc = wl.seeded_normal(6, (g, dc.pool_tokens, d), torch.bfloat16, device="cuda")
    n_routes = dc.batch * g
    assert n_routes > 1024
    route_cu = torch.empty(n_routes + 1, dtype=torch.int32, device="cuda")
    route_len = torch.empty(n_routes, dtype=torch.int32, device="cuda")
    rows = orc.compact_routes(dc.keep, dc.res_off, dc.dst_slot, dc.lens, dc.vis)
    cu = orc.route_prefix(rows)
    route_idx = torch.full((int(cu[-1]) + 8,), -7, dtype=torch.int32, device="cuda")
    kp = torch.full((dc.n_pages, wl.PAGE_TOKENS, d), float("nan"), dtype=torch.bfloat16, device="cuda")
    vp = torch.full_like(kp, float("nan"))
    pt = torch.empty((n_routes, dc.max_res_pages), dtype=torch.int32, device="cuda")
    rc.compact_routes(kc, vc, dev(dc.keep), dev(dc.res_off), dev(dc.dst_slot), dev(dc.lens), dev(dc.vis), PAGED, route_cu,
                      route_idx, kp, vp, route_len=route_len, page_table=pt, free_pages=dev(dc.free_pages))
    assert np.array_equal(route_cu.cpu().numpy(), cu)
    flat = np.concatenate([r for per in rows for r in per])
    assert np.array_equal(route_idx.cpu().numpy()[:cu[-1]], flat) and (route_idx.cpu().numpy()[cu[-1]:] == -7).all()
    table_ref, used = orc.page_layout(rows, dc.free_pages, wl.PAGE_TOKENS, dc.max_res_pages)
    assert np.array_equal(pt.cpu().numpy(), table_ref)
    # every compacted row landed, byte for byte, in its page slot; nothing else was written
    kc_h, kp_h = kc.cpu().view(torch.int16).numpy(), kp.cpu().view(torch.int16).numpy()
    vc_h, vp_h = vc.cpu().view(torch.int16).numpy(), vp.cpu().view(torch.int16).numpy()
    written = np.zeros((dc.n_pages, wl.PAGE_TOKENS), bool)
    i = 0
    for per in rows:
        for kg, r in enumerate(per):
            n = np.arange(len(r))
            pg, sl = table_ref[i, n // wl.PAGE_TOKENS], n % wl.PAGE_TOKENS
            assert np.array_equal(kp_h[pg, sl], kc_h[kg][r]) and np.array_equal(vp_h[pg, sl], vc_h[kg][r])
            written[pg, sl] = True
            i += 1
    assert torch.isnan(kp.cpu()[torch.from_numpy(~written)]).all()
    assert rc.poll_status() == 0


def test_device_status_codes_instead_of_faults():
    """Out-of-range indices are skipped and reported, the context stays usable."""
    sh = wl.QWEN3_4B
    pool = _pool(sh, [50, 60])
    rc = make_ctx(sh, max_pos=1024)
    bad = wl.ResourceBatch(**{**pool.__dict__})
    bad.dst_slot = np.array([0, 100], np.int32)          # second resource would end past the pool (110 rows)
    gpu_encode(rc, bad, nan_fill=False)
    assert rc.poll_status() == 2
    assert rc.poll_status() == 0              # cleared by the poll
    # compaction into too small a buffer: rows that fit are written, the overflow is reported
    o, kc, vc = gpu_encode(rc, pool)
    vis = np.ones((sh.n_kv_heads, 2), np.uint8)
    req = wl.make_requests(sh, 3, wl.keep_all(pool), [[0, 1]], [vis], [8])
    out = gpu_compact(rc, wl.keep_all(pool), req, kc, vc, capacity=100)
    assert rc.poll_status() == 3
    assert int(out["route_cu"][-1]) == 110 * sh.n_kv_heads
    # a prefill handed that prefix (ranges beyond the 100 packed rows) reports it and skips those routes,
    # on the tensor-core path and on the exact row-per-warp path alike
    gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"])
    assert rc.poll_status() == 3
    sh32 = wl.Shape(4, 2, 64, 1e4, "f32")
    pool32 = wl.keep_all(_pool(sh32, [50, 60]))
    rc32 = make_ctx(sh32, max_pos=1024)
    _, kc32, vc32 = gpu_encode(rc32, pool32)
    vis32 = np.ones((sh32.n_kv_heads, 2), np.uint8)
    req32 = wl.make_requests(sh32, 3, pool32, [[0, 1]], [vis32], [8])
    out32 = gpu_compact(rc32, pool32, req32, kc32, vc32, capacity=100)
    assert rc32.poll_status() == 3
    gpu_prefill(rc32, req32, out32["k_out"], out32["v_out"], out32["route_cu"])
    assert rc32.poll_status() == 3
    # conversation positions running past the rotary table (1000 + 64 > 1024)
    req_far = wl.make_requests(sh, 4, wl.keep_all(pool), [[0, 1]], [vis], [64], q_pos0=[1000])
    big = gpu_compact(rc, wl.keep_all(pool), req_far, kc, vc)
    gpu_prefill(rc, req_far, big["k_out"], big["v_out"], big["route_cu"])
    assert rc.poll_status() == 6
    # decode with a page id outside the pool
    dec = wl.config4_decode(batch=2, n_res=4, res_len=(60, 100), hist=70)
    rpt = dec.res_page_table.copy(); rpt[0, 0] = 10 ** 6
    rc.attend_decode(dev(dec.q), dev(dec.q_pos), dev(dec.k_pages), dev(dec.v_pages), dev(rpt), dev(dec.res_len),
                     dev(dec.hist_page_table), dev(dec.hist_len))
    assert rc.poll_status() == 4
    # and the context still computes correctly afterwards
    od = rc.attend_decode(dev(dec.q), dev(dec.q_pos), dev(dec.k_pages), dev(dec.v_pages), dev(dec.res_page_table),
                          dev(dec.res_len), dev(dec.hist_page_table), dev(dec.hist_len), out_dtype=torch.float32)
    ref = orc.attend_decode(f64(dec.q), dec.q_pos, f64(dec.k_pages), f64(dec.v_pages), dec.res_page_table, dec.res_len,
                            dec.hist_page_table, dec.hist_len, sh.rope_theta, wl.PAGE_TOKENS, storage="bf16")
    assert max_abs(od, ref) < TOL_BF16 and rc.poll_status() == 0


def test_host_side_errors_are_returned_before_any_launch():
    from paper_2608_19662_b200 import ReCacheError
    sh = wl.QWEN3_4B
    rc = make_ctx(sh, max_pos=1024)
    pool = _pool(sh, [40])
    q, k, v = dev(pool.q), dev(pool.k), dev(pool.v)
    kc = torch.empty((sh.n_kv_heads, 40, sh.head_dim), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ReCacheError, match="max_len exceeds"):
        rc.encode_resources(q, k, v, dev(pool.cu_seqlens), 5000, dev(pool.dst_slot), kc, kc.clone())
    with pytest.raises(ReCacheError, match="workspace too small"):
        rc.encode_resources(q, k, v, dev(pool.cu_seqlens), 40, dev(pool.dst_slot), kc, kc.clone(),
                            workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    n = 40 * sh.n_q_heads * sh.head_dim
    q_off = torch.empty(n + 8, dtype=torch.bfloat16, device="cuda")[1:1 + n].view(40, sh.n_q_heads, sh.head_dim)
    with pytest.raises(ReCacheError, match="16-byte aligned"):
        rc.encode_resources(q_off, k, v, dev(pool.cu_seqlens), 40, dev(pool.dst_slot), kc, kc.clone())
    i32 = lambda *a: torch.zeros(a, dtype=torch.int32, device="cuda")
    with pytest.raises(ReCacheError, match="bad mode"):
        rc.compact_routes(kc, kc, torch.ones(40, dtype=torch.uint8, device="cuda"), i32(2), i32(1), i32(1),
                          torch.ones((sh.n_kv_heads, 1), dtype=torch.uint8, device="cuda"), 7, i32(9), i32(64),
                          torch.empty((64, 128), dtype=torch.bfloat16, device="cuda"),
                          torch.empty((64, 128), dtype=torch.bfloat16, device="cuda"))
    assert rc.poll_status() == 0


def test_bounded_wait_runs_out_sets_status_and_context_stays_usable():
    """The failure path of the TMA kernels' barrier waits, exercised by the library's
    self-test kernel (same wait and drain helpers, small probe bound, a barrier nobody
    arrives at): it must give up within milliseconds, report RECACHE_DEV_TIMEOUT with
    its location, and leave the context clean for the next ordinary call."""
    sh = wl.QWEN3_4B
    rc = make_ctx(sh, max_pos=1024)
    gave_up, kcycles = rc.selftest_wait_timeout()
    assert gave_up
    assert 100 < kcycles < 100_000                 # ~2^10 suspended probes: around a millisecond, never seconds
    assert rc.poll_status() == 7                   # RECACHE_DEV_TIMEOUT
    assert "wait self-test" in rc.last_error()
    assert rc.poll_status() == 0                   # cleared by the poll
    pool = _pool(sh, [70, 200])
    o_ref, _, _ = oracle_encode(pool)
    o, _, _ = gpu_encode(rc, pool)
    assert max_abs(o, o_ref) < TOL_BF16 and rc.poll_status() == 0


@pytest.mark.parametrize("hq,g", [(16, 8), (32, 8), (32, 4)])
def test_thousands_of_tiny_resources(hq, g):
    """Many resources no longer than one query tile (1 .. 128/s tokens, so the
    second tile of every work item is empty and every item has a single K/V
    tile): each CTA runs dozens of such items back to back, the case in which a
    role that is idle in an item could run ahead of the others."""
    sh = wl.Shape(hq, g, 128, 1e6, "bf16")
    tq = 128 // sh.group_size
    rng = np.random.default_rng(hq + g)
    n = 2000
    lens = rng.integers(1, tq + 1, n)
    lens[::7] = rng.integers(tq + 1, 2 * tq + 1, len(lens[::7]))     # some with a second tile in between
    pool = _pool(sh, [int(x) for x in lens], keep=[np.ones(int(x), np.uint8) for x in lens])
    rc = make_ctx(sh, max_pos=1024)
    o_ref, kc_ref, vc_ref = oracle_encode(pool)
    o, kc, vc = gpu_encode(rc, pool)
    assert rc.poll_status() == 0
    assert max_abs(o, o_ref) < TOL_BF16
    assert np.array_equal(f64(vc)[~np.isnan(vc_ref)], vc_ref[~np.isnan(vc_ref)])
    # many short requests with empty routes through the prefill entry point
    nreq = 600
    tqs = [int(x) for x in rng.integers(1, tq + 1, nreq)]
    vis0 = np.zeros((g, 1), np.uint8)
    req = wl.make_requests(sh, 9, pool, [[0]] * nreq, [vis0] * nreq, tqs)
    rows = oracle_rows(pool, req)
    out = gpu_compact(rc, pool, req, kc, vc)
    p_ref, _ = oracle_prefill(req, rows, kc_ref, vc_ref)
    p, _, _ = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"])
    assert rc.poll_status() == 0
    assert max_abs(p, p_ref) < TOL_BF16
