"""Parity of the CUDA path (through the C ABI) with the fp64 oracle, element by
element on the same seeded inputs.  Tolerances: indices / routes / gathered
bytes bit-exact; fp32 path max-abs 1e-5; bf16 inputs with fp32 accumulation
max-abs 1e-2 on unit-variance data (gate on fp32 outputs; bf16 outputs may add
half a bf16 ulp of the reference on top)."""
import numpy as np
import pytest
import torch

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl

from pipeline import (bf16_ulp_distance, dev, f64, gpu_compact, gpu_encode, gpu_prefill, make_ctx, max_abs,
                      oracle_cache_only, oracle_encode, oracle_prefill, oracle_rows, report_readings, sample_rows)

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-5
TOL_BF16 = 1e-2


def assert_status_ok(rc):
    assert rc.poll_status() == 0


def check_cache(shape, kc_gpu, vc_gpu, kc_ref, vc_ref):
    """Values are byte copies; rotated keys are the fp32 rotation of the oracle's
    fp64 one: equal up to the last place of the storage type."""
    written = ~np.isnan(kc_ref)
    assert np.array_equal(np.isnan(f64(kc_gpu)), ~written)       # only the resources' rows are written
    assert np.array_equal(f64(vc_gpu)[written], vc_ref[written])
    assert_rotated_close(shape, kc_gpu, np.where(written, kc_ref, 0.0), written)


def assert_rotated_close(shape, got, ref, mask=None):
    """fp32 rotation on the GPU against the fp64 one: equal up to one unit in the
    last place of the storage type (plus the fp32 rounding of the two products,
    which matters only where they cancel), and different in few places."""
    mask = np.ones(ref.shape, bool) if mask is None else mask
    diff = np.abs(f64(got) - ref)[mask]
    if shape.dtype == "bf16":
        ulps = bf16_ulp_distance(got, ref)[mask]
        assert ((ulps <= 1.0) | (diff < 2e-6)).all()
        assert (diff > 0).mean() < 0.01
    else:
        assert diff.max() < 2e-6


def check_compaction(out, rows, kc_gpu, vc_gpu, shape):
    cu = orc.route_prefix(rows)
    assert np.array_equal(out["route_cu"].cpu().numpy(), cu)
    assert np.array_equal(out["route_len"].cpu().numpy(), np.diff(cu))
    flat = np.concatenate([r for per in rows for r in per]) if cu[-1] else np.zeros(0, np.int32)
    n = int(cu[-1])
    idx = out["route_idx"].cpu().numpy()
    assert np.array_equal(idx[:n], flat)
    assert (idx[n:] == -7).all()                                  # nothing written past the end
    return cu, flat


def check_packed_bytes(out, rows, kc_gpu, vc_gpu):
    """Packed rows are byte copies of the GPU's own cache rows at the oracle's indices."""
    cu = orc.route_prefix(rows)
    g_of = np.concatenate([np.full(len(r), g) for per in rows for g, r in enumerate(per)]) if cu[-1] else np.zeros(0, int)
    flat = np.concatenate([r for per in rows for r in per]) if cu[-1] else np.zeros(0, int)
    n = int(cu[-1])
    kw = kc_gpu.view(torch.int16 if kc_gpu.dtype == torch.bfloat16 else torch.int32)
    vw = vc_gpu.view(kw.dtype)
    gi, ri = torch.from_numpy(g_of).cuda().long(), torch.from_numpy(flat).cuda().long()
    assert torch.equal(out["k_out"].view(kw.dtype)[:n], kw[gi, ri])
    assert torch.equal(out["v_out"].view(kw.dtype)[:n], vw[gi, ri])
    assert torch.isnan(out["k_out"][n:]).all()


# ---------------------------------------------------------------- config 1 --
def test_config1_fp32_whole_path():
    pool, req = wl.config1()
    sh = pool.shape
    rc = make_ctx(sh, max_pos=256)
    o_ref, kc_ref, vc_ref = oracle_encode(pool)
    o, kc, vc = gpu_encode(rc, pool)
    assert max_abs(o, o_ref) < TOL_F32
    report_readings("config1 fp32", "encode", max_abs(o, o_ref), max_abs(o, oracle_encode(pool, round_q=False)[0]))
    check_cache(sh, kc, vc, kc_ref, vc_ref)
    # position 0 is the identity: the first cached key row of every resource is its input, bitwise
    for i, s0 in enumerate(pool.dst_slot):
        assert torch.equal(kc[:, s0].cpu(), pool.k[pool.cu_seqlens[i]])

    rows = oracle_rows(pool, req)
    out = gpu_compact(rc, pool, req, kc, vc)
    check_compaction(out, rows, kc, vc, sh)
    check_packed_bytes(out, rows, kc, vc)

    p_ref, kconv_ref = oracle_prefill(req, rows, kc_ref, vc_ref)
    p, kconv, vconv = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"])
    assert max_abs(p, p_ref) < TOL_F32
    report_readings("config1 fp32", "prefill", max_abs(p, p_ref),
                    max_abs(p, oracle_prefill(req, rows, kc_ref, vc_ref, round_q=False)[0]))
    assert_rotated_close(sh, kconv, np.transpose(kconv_ref, (1, 0, 2)))
    assert torch.equal(vconv.cpu(), req.v_conv.permute(1, 0, 2))
    assert_status_ok(rc)


def test_config1_decode_equals_last_prefill_row():
    """Paged compaction + decode of the last conversation token (appended by the
    call) reproduces the oracle's decode and the last row of the prefill."""
    from paper_2608_19662_b200 import PAGED
    pool, req = wl.config1()
    sh = pool.shape
    g, d, pt = sh.n_kv_heads, sh.head_dim, wl.PAGE_TOKENS
    rc = make_ctx(sh, max_pos=256)
    _, kc_ref, vc_ref = oracle_encode(pool)
    _, kc, vc = gpu_encode(rc, pool)
    rows = oracle_rows(pool, req)
    n_res_pages = [(len(r) + pt - 1) // pt for r in rows[0]]
    tq = req.total_q
    n_hist_pages = (tq + pt - 1) // pt
    total = sum(n_res_pages) + g * n_hist_pages + 3
    free = np.random.default_rng(9).permutation(total).astype(np.int32)
    out = gpu_compact(rc, pool, req, kc, vc, mode=PAGED, n_pool_pages=total, free_pages=free,
                      max_pages=max(n_res_pages) + 1)
    check_compaction(out, rows, kc, vc, sh)
    table_ref, used = orc.page_layout(rows, free, pt, max(n_res_pages) + 1)
    assert np.array_equal(out["page_table"].cpu().numpy(), table_ref)
    kp_ref = orc.gather_paged(kc_ref, rows, table_ref, total, pt, fill=np.nan)
    vp_ref = orc.gather_paged(vc_ref, rows, table_ref, total, pt, fill=np.nan)
    got = f64(out["k_out"])
    assert np.array_equal(np.isnan(got), np.isnan(kp_ref))       # exactly the routes' slots are written
    assert np.array_equal(f64(out["v_out"])[~np.isnan(vp_ref)], vp_ref[~np.isnan(vp_ref)])

    # history = rotated conversation keys 0..tq-2 (from the oracle), the call appends token tq-1
    p_ref, kconv_ref = oracle_prefill(req, rows, kc_ref, vc_ref)
    hist_pt = free[used:used + g * n_hist_pages].reshape(g, n_hist_pages)
    vconv = f64(req.v_conv)
    res_mask = ~np.isnan(kp_ref)
    for kg in range(g):
        for n in range(tq - 1):
            kp_ref[hist_pt[kg, n // pt], n % pt] = kconv_ref[n, kg]
            vp_ref[hist_pt[kg, n // pt], n % pt] = vconv[n, kg]
    k_pages, v_pages = out["k_out"], out["v_out"]
    hmask = ~np.isnan(kp_ref) & ~res_mask          # history slots only; resource rows stay the GPU's own
    k_pages[torch.from_numpy(hmask).cuda()] = torch.from_numpy(kp_ref[hmask]).to(sh.torch_dtype).cuda()
    v_pages[torch.from_numpy(hmask).cuda()] = torch.from_numpy(vp_ref[hmask]).to(sh.torch_dtype).cuda()
    hist_len = np.full(g, tq, np.int32)
    q_pos = np.array([64 + tq - 1], np.int32)
    od = rc.attend_decode(dev(req.q[tq - 1:tq]), dev(q_pos), k_pages, v_pages, out["page_table"], out["route_len"],
                          dev(hist_pt), dev(hist_len), k_new=dev(req.k_conv[tq - 1:tq]),
                          v_new=dev(req.v_conv[tq - 1:tq]), out_dtype=torch.float32)
    orc.append_decode_kv(kp_ref, vp_ref, hist_pt, hist_len, f64(req.k_conv)[tq - 1:tq], vconv[tq - 1:tq], q_pos,
                         sh.rope_theta, pt, storage=sh.dtype)
    res_len = np.array([len(r) for r in rows[0]], np.int32)
    od_ref = orc.attend_decode(f64(req.q)[tq - 1:tq], q_pos, kp_ref, vp_ref, table_ref, res_len, hist_pt, hist_len,
                               sh.rope_theta, pt, storage=sh.dtype)
    assert max_abs(od, od_ref) < TOL_F32
    assert max_abs(od, p_ref[tq - 1:tq]) < TOL_F32
    assert_status_ok(rc)


# ---------------------------------------------------------------- config 2 --
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_config2_bf16_whole_path(out_dtype):
    pool, req = wl.config2()
    sh = pool.shape
    rc = make_ctx(sh, max_pos=8192)
    o_ref, kc_ref, vc_ref = oracle_encode(pool)
    o, kc, vc = gpu_encode(rc, pool, out_dtype=out_dtype)
    slack = 0.0 if out_dtype == torch.float32 else 2.0 ** -8      # half a bf16 ulp of the reference
    assert (np.abs(f64(o) - o_ref) <= TOL_BF16 + slack * np.abs(o_ref)).all()
    tag = "config2 bf16 out=" + ("f32" if out_dtype == torch.float32 else "bf16")
    report_readings(tag, "encode", max_abs(o, o_ref), max_abs(o, oracle_encode(pool, round_q=False)[0]))
    check_cache(sh, kc, vc, kc_ref, vc_ref)
    rows = oracle_rows(pool, req)
    lens = [len(r) for r in rows[0]]
    assert 0.2 < pool.keep.sum() / pool.total_tokens < 0.4 and min(lens) > 0
    out = gpu_compact(rc, pool, req, kc, vc)
    check_compaction(out, rows, kc, vc, sh)
    check_packed_bytes(out, rows, kc, vc)
    p_ref, kconv_ref = oracle_prefill(req, rows, kc_ref, vc_ref)
    p, kconv, vconv = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"], out_dtype=out_dtype)
    assert (np.abs(f64(p) - p_ref) <= TOL_BF16 + slack * np.abs(p_ref)).all()
    report_readings(tag, "prefill", max_abs(p, p_ref),
                    max_abs(p, oracle_prefill(req, rows, kc_ref, vc_ref, round_q=False)[0]))
    assert_rotated_close(sh, kconv, np.transpose(kconv_ref, (1, 0, 2)))
    assert torch.equal(vconv.cpu(), req.v_conv.permute(1, 0, 2))
    assert_status_ok(rc)


# ---------------------------------------------------------------- config 3 --
def test_config3_reuse_bit_identical_kv_and_permutation_invariance():
    """A pool resource encoded alone, inside the whole pool, or next to other
    neighbours in another order gives bit-identical cache rows AND outputs;
    permuting a request's resource order leaves its outputs unchanged."""
    n_layers = 2
    for layer in range(n_layers):
        pool = wl.config3_pool(n_pool=10, len_range=(150, 420), layer=layer)
        sh = pool.shape
        rc = make_ctx(sh, max_pos=8192)
        o_all, kc, vc = gpu_encode(rc, pool, out_dtype=torch.bfloat16)
        # another composition: a subset, reversed, with gaps between the slots
        sub = [7, 2, 5]
        masks = [pool.keep[pool.dst_slot[r]:pool.dst_slot[r] + pool.lens[r]] for r in sub]
        pool_b = wl.pack_resources(sh, wl.SEED0 + 3, pool.lens[sub], masks, res_ids=sub, layer=layer, slot_gap=37)
        o_b, kc_b, vc_b = gpu_encode(rc, pool_b, out_dtype=torch.bfloat16)
        for n, r in enumerate(sub):
            a, e = pool.cu_seqlens[r], pool.cu_seqlens[r + 1]
            a2, e2 = pool_b.cu_seqlens[n], pool_b.cu_seqlens[n + 1]
            assert torch.equal(pool.q[a:e], pool_b.q[a2:e2])        # same resource, same data
            assert torch.equal(o_all[a:e].view(torch.int16), o_b[a2:e2].view(torch.int16))
            s1, s2, ln = pool.dst_slot[r], pool_b.dst_slot[n], pool.lens[r]
            assert torch.equal(kc[:, s1:s1 + ln].view(torch.int16), kc_b[:, s2:s2 + ln].view(torch.int16))
            assert torch.equal(vc[:, s1:s1 + ln].view(torch.int16), vc_b[:, s2:s2 + ln].view(torch.int16))

        req = wl.config3_requests(pool, n_requests=3, draw=(3, 6), tq_range=(60, 200), layer=layer)
        rows = oracle_rows(pool, req)
        out = gpu_compact(rc, pool, req, kc, vc)
        check_compaction(out, rows, kc, vc, sh)
        check_packed_bytes(out, rows, kc, vc)
        p, _, _ = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"])
        kc_ref, vc_ref = oracle_cache_only(pool)
        p_ref, _ = oracle_prefill(req, rows, kc_ref, vc_ref)
        assert max_abs(p, p_ref) < TOL_BF16
        report_readings(f"config3 small layer {layer}", "prefill", max_abs(p, p_ref),
                        max_abs(p, oracle_prefill(req, rows, kc_ref, vc_ref, round_q=False)[0]))
        # same requests with every resource list reversed (and the route table permuted with it)
        perm = np.concatenate([np.arange(req.res_off[b], req.res_off[b + 1])[::-1] for b in range(req.n_requests)])
        req_p = wl.RequestBatch(**{**req.__dict__})
        req_p.res_slot, req_p.res_len = req.res_slot[perm].copy(), req.res_len[perm].copy()
        req_p.vis = np.ascontiguousarray(req.vis[:, perm])
        out_p = gpu_compact(rc, pool, req_p, kc, vc)
        check_compaction(out_p, oracle_rows(pool, req_p), kc, vc, sh)
        p_perm, _, _ = gpu_prefill(rc, req_p, out_p["k_out"], out_p["v_out"], out_p["route_cu"])
        assert max_abs(p_perm, p_ref) < TOL_BF16
        assert max_abs(p_perm, p) < 2e-3          # same math, other summation order
        assert rc.poll_status() == 0


# ---------------------------------------------------------------- config 4 --
def test_config4_decode_small_batch():
    dec = wl.config4_decode(batch=3, n_res=8, res_len=(100, 260), hist=300)
    sh = dec.shape
    rc = make_ctx(sh, max_pos=8192)
    od = rc.attend_decode(dev(dec.q), dev(dec.q_pos), dev(dec.k_pages), dev(dec.v_pages), dev(dec.res_page_table),
                          dev(dec.res_len), dev(dec.hist_page_table), dev(dec.hist_len), out_dtype=torch.float32)
    ref = orc.attend_decode(f64(dec.q), dec.q_pos, f64(dec.k_pages), f64(dec.v_pages), dec.res_page_table,
                            dec.res_len, dec.hist_page_table, dec.hist_len, sh.rope_theta, wl.PAGE_TOKENS,
                            storage=sh.dtype)
    assert max_abs(od, ref) < TOL_BF16
    ref_u = orc.attend_decode(f64(dec.q), dec.q_pos, f64(dec.k_pages), f64(dec.v_pages), dec.res_page_table,
                              dec.res_len, dec.hist_page_table, dec.hist_len, sh.rope_theta, wl.PAGE_TOKENS,
                              storage=sh.dtype, round_q=False)
    report_readings("config4 small", "decode", max_abs(od, ref), max_abs(od, ref_u))
    assert_status_ok(rc)


def test_config4_decode_full_size_sampled_items():
    dec = wl.config4_decode()
    sh = dec.shape
    assert dec.q.shape[0] == 64 and int(dec.hist_len[0]) == 2048
    rc = make_ctx(sh, max_pos=16384)
    od = rc.attend_decode(dev(dec.q), dev(dec.q_pos), dev(dec.k_pages), dev(dec.v_pages), dev(dec.res_page_table),
                          dev(dec.res_len), dev(dec.hist_page_table), dev(dec.hist_len), out_dtype=torch.float32)
    items = sorted(set([0, 511] + [int(x) for x in np.random.default_rng(4).integers(0, 512, 30)]))
    # bf16 values are exact in fp32; the oracle widens the rows it gathers to fp64
    ref = orc.attend_decode(f64(dec.q), dec.q_pos, dec.k_pages.float().numpy(), dec.v_pages.float().numpy(),
                            dec.res_page_table,
                            dec.res_len, dec.hist_page_table, dec.hist_len, sh.rope_theta, wl.PAGE_TOKENS, items=items,
                            storage=sh.dtype)
    ref_u = orc.attend_decode(f64(dec.q), dec.q_pos, dec.k_pages.float().numpy(), dec.v_pages.float().numpy(),
                              dec.res_page_table, dec.res_len, dec.hist_page_table, dec.hist_len, sh.rope_theta,
                              wl.PAGE_TOKENS, items=items, storage=sh.dtype, round_q=False)
    g, s = sh.n_kv_heads, sh.group_size
    worst = worst_u = 0.0
    for it in items:
        b, kg = divmod(it, g)
        assert max_abs(od[b, kg * s:(kg + 1) * s], ref[b, kg * s:(kg + 1) * s]) < TOL_BF16
        worst = max(worst, max_abs(od[b, kg * s:(kg + 1) * s], ref[b, kg * s:(kg + 1) * s]))
        worst_u = max(worst_u, max_abs(od[b, kg * s:(kg + 1) * s], ref_u[b, kg * s:(kg + 1) * s]))
    report_readings("config4 full (32 items)", "decode", worst, worst_u)
    assert_status_ok(rc)


# ---------------------------------------------------------------- config 5 --
def test_config5_scaled_routed_and_dense_comparison():
    pool, req = wl.config5(n_res=6, len_range=(300, 700), tq=300, bulk=False)
    sh = pool.shape
    rc = make_ctx(sh, max_pos=8192)
    o_ref, kc_ref, vc_ref = oracle_encode(pool)
    o, kc, vc = gpu_encode(rc, pool)
    assert max_abs(o, o_ref) < TOL_BF16
    report_readings("config5 scaled", "encode", max_abs(o, o_ref), max_abs(o, oracle_encode(pool, round_q=False)[0]))
    for pl, rq in ((pool, req), (wl.keep_all(pool), wl.all_visible(req))):
        rows = oracle_rows(pl, rq)
        out = gpu_compact(rc, pl, rq, kc, vc)
        check_compaction(out, rows, kc, vc, sh)
        check_packed_bytes(out, rows, kc, vc)
        p_ref, _ = oracle_prefill(rq, rows, kc_ref, vc_ref)
        p, _, _ = gpu_prefill(rc, rq, out["k_out"], out["v_out"], out["route_cu"])
        assert max_abs(p, p_ref) < TOL_BF16
        report_readings("config5 scaled " + ("routed" if pl is pool else "dense"), "prefill", max_abs(p, p_ref),
                        max_abs(p, oracle_prefill(rq, rows, kc_ref, vc_ref, round_q=False)[0]))
    assert_status_ok(rc)
