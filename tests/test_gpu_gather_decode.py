"""Zero-copy routed decode: the resource rows are read from the cache through the
compaction's index list (index-only compaction, no row moved).  Same results as
the materialised (paged) path, bit for bit, and as the oracle."""
import numpy as np
import pytest
import torch

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl

from pipeline import dev, f64, make_ctx

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("batch,n_res,res_len,hist", [(3, 6, (40, 200), 130), (20, 16, (300, 700), 1000)])
def test_gather_decode_equals_paged_decode_and_oracle(batch, n_res, res_len, hist):
    from paper_2608_19662_b200 import PACKED, PAGED
    sh = wl.QWEN3_4B
    dc = wl.config4_compose(batch=batch, n_res=n_res, res_len=res_len, hist=hist)
    g, d, pt, s = sh.n_kv_heads, sh.head_dim, wl.PAGE_TOKENS, sh.group_size
    rc = make_ctx(sh, max_pos=32768)
    kc = wl.seeded_normal(5, (g, dc.pool_tokens, d), torch.bfloat16, device="cuda")
    vc = wl.seeded_normal(6, (g, dc.pool_tokens, d), torch.bfloat16, device="cuda")
    k_pages = wl.seeded_normal(7, (dc.n_pages, pt, d), torch.bfloat16, device="cuda")
    v_pages = wl.seeded_normal(8, (dc.n_pages, pt, d), torch.bfloat16, device="cuda")
    n_items = batch * g
    q = wl.normal(9, (batch, sh.n_q_heads, d), torch.bfloat16)
    kn = wl.normal(10, (batch, g, d), torch.bfloat16); vn = wl.normal(11, (batch, g, d), torch.bfloat16)
    args = (dev(dc.keep), dev(dc.res_off), dev(dc.dst_slot), dev(dc.lens), dev(dc.vis))
    rows = orc.compact_routes(dc.keep, dc.res_off, dc.dst_slot, dc.lens, dc.vis)
    cu = orc.route_prefix(rows)

    # index-only compaction: route_cu / route_idx, no key or value row is touched
    r_cu = torch.empty(n_items + 1, dtype=torch.int32, device="cuda")
    r_idx = torch.full((int(cu[-1]) + 4,), -7, dtype=torch.int32, device="cuda")
    rc.compact_routes(kc, vc, args[0], args[1], args[2], args[3], args[4], PACKED, r_cu, r_idx, None, None)
    assert np.array_equal(r_cu.cpu().numpy(), cu)
    assert np.array_equal(r_idx.cpu().numpy()[:cu[-1]], np.concatenate([r for per in rows for r in per]))
    kp1, vp1 = k_pages.clone(), v_pages.clone()
    o_g = rc.attend_decode_gather(dev(q), dev(dc.q_pos), kc, vc, r_idx, r_cu, dc.max_res_pages, kp1, vp1,
                                  dev(dc.hist_page_table), dev(dc.hist_len), k_new=dev(kn), v_new=dev(vn),
                                  out_dtype=torch.float32)

    # the materialised path on the same routes
    p_cu = torch.empty(n_items + 1, dtype=torch.int32, device="cuda"); p_len = torch.empty(n_items, dtype=torch.int32, device="cuda")
    p_idx = torch.empty(int(cu[-1]) + 4, dtype=torch.int32, device="cuda")
    p_pt = torch.empty((n_items, dc.max_res_pages), dtype=torch.int32, device="cuda")
    kp2, vp2 = k_pages.clone(), v_pages.clone()
    rc.compact_routes(kc, vc, args[0], args[1], args[2], args[3], args[4], PAGED, p_cu, p_idx, kp2, vp2, route_len=p_len,
                      page_table=p_pt, free_pages=dev(dc.free_pages))
    o_p = rc.attend_decode(dev(q), dev(dc.q_pos), kp2, vp2, p_pt, p_len, dev(dc.hist_page_table), dev(dc.hist_len),
                           k_new=dev(kn), v_new=dev(vn), out_dtype=torch.float32)
    assert torch.equal(o_g, o_p)                      # same rows, same order, same arithmetic
    # the gather path wrote nothing but the appended history row
    hist_pages = torch.from_numpy(np.unique(dc.hist_page_table)).cuda().long()
    mask = torch.ones(dc.n_pages, dtype=torch.bool, device="cuda"); mask[hist_pages] = False
    assert torch.equal(kp1[mask].view(torch.int16), k_pages[mask].view(torch.int16))

    # oracle on sampled items
    rng = np.random.default_rng(3)
    kch, vch, kph, vph = kc.cpu(), vc.cpu(), k_pages.cpu(), v_pages.cpu()
    flat = [r for per in rows for r in per]
    for it in sorted(set([0, n_items - 1] + [int(x) for x in rng.integers(0, n_items, 6)])):
        b, kg = divmod(it, g)
        r = flat[it]
        n_rp = (len(r) + pt - 1) // pt
        hp = dc.hist_page_table[it]
        kpool = np.zeros((n_rp + len(hp), pt, d)); vpool = np.zeros_like(kpool)
        ridx, hidx = torch.from_numpy(r).long(), torch.from_numpy(hp).long()
        kpool[:n_rp].reshape(-1, d)[:len(r)] = f64(kch[kg][ridx]); vpool[:n_rp].reshape(-1, d)[:len(r)] = f64(vch[kg][ridx])
        kpool[n_rp:] = f64(kph[hidx]); vpool[n_rp:] = f64(vph[hidx])
        res_t = np.arange(n_rp, dtype=np.int32)[None, :]; hist_t = (n_rp + np.arange(len(hp), dtype=np.int32))[None, :]
        hl = np.array([dc.hist_len[it]], np.int32); qp = np.array([dc.q_pos[b]], np.int32)
        orc.append_decode_kv(kpool, vpool, hist_t, hl, f64(kn[b:b + 1, kg:kg + 1]), f64(vn[b:b + 1, kg:kg + 1]), qp,
                             sh.rope_theta, pt, storage="bf16")
        ref = orc.attend_decode(f64(q[b:b + 1, kg * s:(kg + 1) * s]), qp, kpool, vpool, res_t, np.array([len(r)], np.int32),
                                hist_t, hl, sh.rope_theta, pt, storage="bf16")
        assert np.abs(f64(o_g[b, kg * s:(kg + 1) * s]) - ref[0]).max() < 1e-2
    assert rc.poll_status() == 0
    # an index list shorter than the prefix says: the items past its end are reported and read as empty
    # routes (history only), nothing is read outside the list
    short = r_idx[:int(cu[n_items // 2])].clone()
    rc.attend_decode_gather(dev(q), dev(dc.q_pos), kc, vc, short, r_cu, dc.max_res_pages, kp1, vp1,
                            dev(dc.hist_page_table), dev(dc.hist_len), out_dtype=torch.float32)
    assert rc.poll_status() == 3
