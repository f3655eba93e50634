"""Parity at the full benchmark sizes, in the launch configuration bench.py
times: integer outputs (routes, indices, page tables, gathered bytes) are
checked in full; attention outputs on seeded samples of rows that the oracle
computes one by one.  Oracle inputs are the seeded host inputs and the seeded
device-drawn cache / page contents (inputs, not results of the CUDA path)."""
import os
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl

from pipeline import (f64, gpu_compact, gpu_encode, gpu_prefill, make_ctx, oracle_cache_only, report_readings,
                      sample_rows)
from test_gpu_parity import assert_rotated_close

pytestmark = pytest.mark.gpu

TOL = 1e-2
HALF_ULP = 2.0 ** -8     # outputs are bf16 here: half a unit in the last place of the reference on top


def _close(got, ref):
    return (np.abs(got - ref) <= TOL + HALF_ULP * np.abs(ref)).all()


def test_bench_step_full_size():
    import bench
    w = bench.Workload("full")
    run = bench.Runner(w, 0)
    run.step()
    torch.cuda.synchronize()
    assert run.rc.poll_status() == 0
    sh, pool, req, dc = w.shape, w.pool, w.req, w.dc
    assert len(pool.lens) == 64 and pool.lens.min() >= 1000 and req.total_q == 2048 and dc.batch == 64
    rng = np.random.default_rng(123)

    # ---- encode: cache in full, outputs on sampled rows (tile-boundary tokens included) ----
    kc_ref, vc_ref = oracle_cache_only(pool)
    assert np.array_equal(f64(run.v_cache), vc_ref)
    assert_rotated_close(sh, run.k_cache, kc_ref)
    extra = [int(pool.cu_seqlens[i]) + t for i in (0, 17, 63) for t in (31, 32, 63, 64, 127, 128, 129, 999)]
    rows = sample_rows(rng, pool.cu_seqlens, sh.n_q_heads, 260, extra_tokens=extra)
    f32 = lambda t: t.float().numpy()            # bf16 values are exact in fp32; the oracle widens what it samples
    ref = orc.encode_rows(f32(pool.q), f32(pool.k), f32(pool.v), pool.cu_seqlens, sh.rope_theta, rows, storage="bf16")
    o = run.o_enc.cpu()
    got = np.stack([f64(o[t, h]) for t, h in rows])
    assert _close(got, ref)
    ref_u = orc.encode_rows(f32(pool.q), f32(pool.k), f32(pool.v), pool.cu_seqlens, sh.rope_theta, rows[:64],
                            storage="bf16", round_q=False)
    report_readings("config5 full (bf16 out)", "encode", float(np.abs(got - ref).max()),
                    float(np.abs(got[:64] - ref_u).max()))

    # ---- packed compaction: exact ----
    rt = orc.compact_routes(pool.keep, req.res_off, req.res_slot, req.res_len, req.vis)
    cu = orc.route_prefix(rt)
    assert np.array_equal(run.route_cu.cpu().numpy(), cu)
    flat = np.concatenate([r for per in rt for r in per])
    assert np.array_equal(run.route_idx.cpu().numpy()[:cu[-1]], flat)
    g_of = np.concatenate([np.full(len(r), kg) for per in rt for kg, r in enumerate(per)])
    gi, ri = torch.from_numpy(g_of).cuda().long(), torch.from_numpy(flat).cuda().long()
    assert torch.equal(run.k_route.view(torch.int16)[:cu[-1]], run.k_cache.view(torch.int16)[gi, ri])
    assert torch.equal(run.v_route.view(torch.int16)[:cu[-1]], run.v_cache.view(torch.int16)[gi, ri])
    assert 0.05 < cu[-1] / (sh.n_kv_heads * pool.total_tokens) < 0.11          # ~8 % of the KV is retained

    # ---- prefill: sampled rows ----
    prow = sample_rows(rng, req.cu_q, sh.n_q_heads, 160, extra_tokens=[31, 32, 63, 64, 1023, 1024])
    pref = orc.prefill_rows(f32(req.q), f32(req.k_conv), f32(req.v_conv), req.cu_q, req.q_pos0, rt, kc_ref, vc_ref,
                            sh.rope_theta, prow, storage="bf16")
    op = run.o_pre.cpu()
    gotp = np.stack([f64(op[t, h]) for t, h in prow])
    assert _close(gotp, pref)
    pref_u = orc.prefill_rows(f32(req.q), f32(req.k_conv), f32(req.v_conv), req.cu_q, req.q_pos0, rt, kc_ref, vc_ref,
                              sh.rope_theta, prow[:64], storage="bf16", round_q=False)
    report_readings("config5 full (bf16 out)", "prefill", float(np.abs(gotp - pref).max()),
                    float(np.abs(gotp[:64] - pref_u).max()))

    # ---- paged compaction for the decode batch: exact ----
    rows4 = orc.compact_routes(dc.keep, dc.res_off, dc.dst_slot, dc.lens, dc.vis)
    cu4 = orc.route_prefix(rows4)
    assert np.array_equal(run.d_route_cu.cpu().numpy(), cu4)
    assert np.array_equal(run.d_route_len.cpu().numpy(), np.diff(cu4))
    flat4 = np.concatenate([r for per in rows4 for r in per])
    assert np.array_equal(run.d_route_idx.cpu().numpy()[:cu4[-1]], flat4)
    table_ref, used = orc.page_layout(rows4, dc.free_pages, wl.PAGE_TOKENS, dc.max_res_pages)
    assert used == len(dc.free_pages)
    assert np.array_equal(run.d_page_table.cpu().numpy(), table_ref)

    # ---- decode: sampled (sequence, group) items from the seeded cache / history contents ----
    g, d, pt, s = sh.n_kv_heads, sh.head_dim, wl.PAGE_TOKENS, sh.group_size
    kc4, vc4 = run.d_k_cache.cpu(), run.d_v_cache.cpu()            # seeded inputs drawn on the device
    kp_in = wl.seeded_normal(79, (dc.n_pages, pt, d), sh.torch_dtype, device="cuda").cpu()   # history contents, as drawn
    vp_in = wl.seeded_normal(80, (dc.n_pages, pt, d), sh.torch_dtype, device="cuda").cpu()
    od = run.o_dec.cpu()
    items = sorted(set([0, dc.batch * g - 1] + [int(v) for v in rng.integers(0, dc.batch * g, 22)]))
    flat_rows = [r for per in rows4 for r in per]
    for it in items:
        b, kg = divmod(it, g)
        r = flat_rows[it]
        n_rp = (len(r) + pt - 1) // pt
        hp = dc.hist_page_table[it]
        # a private little page pool for this item: its resource pages, then its history pages
        kpool = np.zeros((n_rp + len(hp), pt, d)); vpool = np.zeros_like(kpool)
        ridx, hidx = torch.from_numpy(r).long(), torch.from_numpy(hp).long()
        kpool[:n_rp].reshape(-1, d)[:len(r)] = f64(kc4[kg][ridx]); vpool[:n_rp].reshape(-1, d)[:len(r)] = f64(vc4[kg][ridx])
        kpool[n_rp:] = f64(kp_in[hidx]); vpool[n_rp:] = f64(vp_in[hidx])
        res_t = np.arange(n_rp, dtype=np.int32)[None, :]
        hist_t = (n_rp + np.arange(len(hp), dtype=np.int32))[None, :]
        hl = np.array([dc.hist_len[it]], np.int32)
        qp = np.array([dc.q_pos[b]], np.int32)
        orc.append_decode_kv(kpool, vpool, hist_t, hl, f64(w.dec_k_new[b:b + 1, kg:kg + 1]),
                             f64(w.dec_v_new[b:b + 1, kg:kg + 1]), qp, sh.rope_theta, pt, storage="bf16")
        ref_o = orc.attend_decode(f64(w.dec_q[b:b + 1, kg * s:(kg + 1) * s]), qp, kpool, vpool, res_t,
                                  np.array([len(r)], np.int32), hist_t, hl, sh.rope_theta, pt, storage="bf16")
        assert _close(f64(od[b, kg * s:(kg + 1) * s]), ref_o[0])


@pytest.mark.parametrize("layer", [0, 7, 35])
def test_composition_reuse_full_size_layer(layer):
    """Layers of the composition-reuse workload at full size (the first, one in
    the middle, the last of the 36): a pool of 64 resources U[150,1200] encoded
    once, 16 requests of 4-12 pool resources in random order with 256-1024 query
    tokens; sampled rows against the oracle and exact compaction.  (The layers
    differ in their inputs and routes.)"""
    pool = wl.config3_pool(layer=layer)
    sh = pool.shape
    req = wl.config3_requests(pool, layer=layer)
    assert len(pool.lens) == 64 and req.n_requests == 16 and 256 <= np.diff(req.cu_q).min()
    rc = make_ctx(sh, max_pos=16384)
    o, kc, vc = gpu_encode(rc, pool, out_dtype=torch.bfloat16)
    kc_ref, vc_ref = oracle_cache_only(pool)
    assert_rotated_close(sh, kc, kc_ref)
    rng = np.random.default_rng(layer)
    rows = sample_rows(rng, pool.cu_seqlens, sh.n_q_heads, 200)
    f32 = lambda t: t.float().numpy()
    ref = orc.encode_rows(f32(pool.q), f32(pool.k), f32(pool.v), pool.cu_seqlens, sh.rope_theta, rows, storage="bf16")
    oc = o.cpu()
    assert _close(np.stack([f64(oc[t, h]) for t, h in rows]), ref)
    rt = orc.compact_routes(pool.keep, req.res_off, req.res_slot, req.res_len, req.vis)
    out = gpu_compact(rc, pool, req, kc, vc)
    cu = orc.route_prefix(rt)
    assert np.array_equal(out["route_cu"].cpu().numpy(), cu)
    assert np.array_equal(out["route_idx"].cpu().numpy()[:cu[-1]], np.concatenate([r for per in rt for r in per]))
    p, _, _ = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"], out_dtype=torch.bfloat16)
    prow = sample_rows(rng, req.cu_q, sh.n_q_heads, 200)
    pref = orc.prefill_rows(f32(req.q), f32(req.k_conv), f32(req.v_conv), req.cu_q, req.q_pos0, rt, kc_ref, vc_ref,
                            sh.rope_theta, prow, storage="bf16")
    pc = p.cpu()
    assert _close(np.stack([f64(pc[t, h]) for t, h in prow]), pref)
    assert rc.poll_status() == 0


def test_long_resource_bit_identical_across_work_list_orders():
    """The encode launch orders its work two ways: the whole pool of 64 resources
    makes thousands of work items and is walked sequence by sequence, a launch of
    three resources is sorted heaviest-first.  A resource of more than 1000
    tokens encoded in both gives the same output and cache rows, bit for bit."""
    layer = 3
    pool = wl.config3_pool(layer=layer)
    sh = pool.shape
    long_ids = [int(i) for i in np.argsort(-pool.lens)[:2]]
    assert pool.lens[long_ids[1]] >= 1000
    tpi = 2 * 128 // sh.group_size                      # tokens per work item
    assert sum((int(n) + tpi - 1) // tpi for n in pool.lens) * sh.n_kv_heads > 1024      # sequence-major order
    rc = make_ctx(sh, max_pos=16384)
    o_all, kc, vc = gpu_encode(rc, pool, out_dtype=torch.bfloat16)
    sub = [long_ids[0], int(np.argmin(pool.lens)), long_ids[1]]
    assert sum((int(pool.lens[r]) + tpi - 1) // tpi for r in sub) * sh.n_kv_heads <= 1024  # sorted order
    masks = [pool.keep[pool.dst_slot[r]:pool.dst_slot[r] + pool.lens[r]] for r in sub]
    pool_b = wl.pack_resources(sh, wl.SEED0 + 3, pool.lens[sub], masks, res_ids=sub, layer=layer, slot_gap=11)
    o_b, kc_b, vc_b = gpu_encode(rc, pool_b, out_dtype=torch.bfloat16)
    for n, r in enumerate(sub):
        a, e = pool.cu_seqlens[r], pool.cu_seqlens[r + 1]
        a2, e2 = pool_b.cu_seqlens[n], pool_b.cu_seqlens[n + 1]
        assert torch.equal(pool.q[a:e], pool_b.q[a2:e2])
        assert torch.equal(o_all[a:e].view(torch.int16), o_b[a2:e2].view(torch.int16))
        s1, s2, ln = pool.dst_slot[r], pool_b.dst_slot[n], pool.lens[r]
        assert torch.equal(kc[:, s1:s1 + ln].view(torch.int16), kc_b[:, s2:s2 + ln].view(torch.int16))
        assert torch.equal(vc[:, s1:s1 + ln].view(torch.int16), vc_b[:, s2:s2 + ln].view(torch.int16))
    assert rc.poll_status() == 0


def test_dense_comparison_full_size_sampled_rows():
    """The comparison point of the long-tool-set workload at full size: every
    route sees every token of all 64 resources (keep-all masks), 2048 query
    tokens over ~95k rows per group.  Exact compaction (identity ranges) and
    sampled prefill rows against the oracle."""
    pool, req = wl.config5()
    pool, req = wl.keep_all(pool), wl.all_visible(req)
    sh = pool.shape
    g, d = sh.n_kv_heads, sh.head_dim
    rc = make_ctx(sh, max_pos=int(req.q_pos0.max() + req.max_q) + 1)
    kc = wl.seeded_normal(91, (g, pool.pool_tokens, d), sh.torch_dtype, device="cuda")    # stand-in for an earlier encode
    vc = wl.seeded_normal(92, (g, pool.pool_tokens, d), sh.torch_dtype, device="cuda")
    out = gpu_compact(rc, pool, req, kc, vc)
    cu = out["route_cu"].cpu().numpy()
    n = pool.total_tokens
    assert np.array_equal(cu, np.arange(g + 1) * n)                       # every group holds every token
    want = np.concatenate([np.arange(s0, s0 + ln) for s0, ln in zip(req.res_slot, req.res_len)])
    idx = out["route_idx"].cpu().numpy()
    for kg in range(g):
        assert np.array_equal(idx[kg * n:(kg + 1) * n], want)
    p, _, _ = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"], out_dtype=torch.bfloat16)
    rng = np.random.default_rng(55)
    prow = sample_rows(rng, req.cu_q, sh.n_q_heads, 48, extra_tokens=[31, 32, 63, 64, 1023, 1024])
    rows = [[want.astype(np.int32) for _ in range(g)]]
    f32 = lambda t: t.float().numpy()
    kc_h, vc_h = kc.cpu().float().numpy(), vc.cpu().float().numpy()        # bf16 values are exact in fp32
    pref = orc.prefill_rows(f32(req.q), f32(req.k_conv), f32(req.v_conv), req.cu_q, req.q_pos0, rows, kc_h, vc_h,
                            sh.rope_theta, prow, storage="bf16")
    pc = p.cpu()
    assert _close(np.stack([f64(pc[t, h]) for t, h in prow]), pref)
    assert rc.poll_status() == 0


def test_bench_composition_reuse_stack_runs():
    """The benchmark's 36-layer composition-reuse stack, cut to two layers: runs through the public calls with
    a clean status word and reports plausible work and rates."""
    import bench
    peaks, _ = bench.load_peaks()
    r = bench.other_workload_config3_stack(0, peaks, n_layers=2, reps=1)
    assert r["useful_tflop_per_stack"] > 0.5 and r["ms_per_stack"] > 0
    assert 50 < r["encode_attn"]["tflops"] < 2300 and 50 < r["prefill_attn"]["tflops"] < 2300
