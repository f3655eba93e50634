"""Cache rows beyond 2^31 elements and 2^32 bytes: two resources whose cache slots
are nine million rows apart in a 4.6 GB key cache (and as much for the values), so
that every address the kernels form for the second one (rotate-and-store, the
compaction gather, the tensor maps of the attention kernel, the per-row gather of
the zero-copy prefill) needs 64-bit arithmetic.  The oracle runs on the same
resources packed back to back: rotated keys, values and attention outputs do not
depend on where a resource sits in the cache."""
import numpy as np
import pytest
import torch

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl

from pipeline import (dev, f64, gpu_compact, gpu_encode, gpu_prefill, make_ctx, max_abs, oracle_encode, oracle_prefill,
                      oracle_rows)

pytestmark = pytest.mark.gpu

GAP = 9_000_000


def test_slots_past_two_to_the_31_elements():
    free, _ = torch.cuda.mem_get_info()
    if free < 16 * 2**30:
        pytest.skip("needs about 10 GB of device memory for the two caches")
    sh = wl.Shape(8, 2, 128, 1e6, "bf16")            # 4 query heads per group: the tensor-core path
    g = sh.n_kv_heads
    lens = [300, 200]
    rng = np.random.default_rng(77)
    masks = wl.keep_mask_spans(rng, lens)
    near = wl.pack_resources(sh, 77, lens, masks)
    far = wl.pack_resources(sh, 77, lens, masks, slot_gap=GAP)
    # the far resource's rows of the last group: element index past 2^31, byte offset past 2^32
    assert (far.pool_tokens * (g - 1) + int(far.dst_slot[1])) * sh.head_dim > 2**31 and torch.equal(near.q, far.q)
    vis = wl.routes_random(rng, g, 2, 1.0)            # both groups see both resources
    req_near = wl.make_requests(sh, 78, near, [[1, 0]], [vis], [150])
    req_far = wl.make_requests(sh, 78, far, [[1, 0]], [vis], [150])
    assert torch.equal(req_near.q, req_far.q)

    o_ref, kc_ref, vc_ref = oracle_encode(near)
    p_ref, _ = oracle_prefill(req_near, oracle_rows(near, req_near), kc_ref, vc_ref)

    rc = make_ctx(sh, max_pos=2048)
    o, kc, vc = gpu_encode(rc, far)                  # caches are NaN-filled first: 2 x 4.6 GB
    assert max_abs(o, o_ref) < 1e-2
    for i in range(2):
        a, b, n = int(far.dst_slot[i]), int(near.dst_slot[i]), int(lens[i])
        assert np.array_equal(f64(vc[:, a:a + n]), vc_ref[:, b:b + n])
        assert max_abs(kc[:, a:a + n], kc_ref[:, b:b + n]) < 2.0 ** -6      # one bf16 ulp of a rotated key at most
    # nothing was written around the far resource
    a = int(far.dst_slot[1])
    assert torch.isnan(kc[:, a - 64:a]).all() and torch.isnan(kc[:, a + lens[1]:a + lens[1] + 64]).all()

    out = gpu_compact(rc, far, req_far, kc, vc)
    rows_far = oracle_rows(far, req_far)
    assert np.array_equal(out["route_cu"].cpu().numpy(), orc.route_prefix(rows_far))
    n_rows = int(out["route_cu"][-1])
    assert np.array_equal(out["route_idx"][:n_rows].cpu().numpy(), np.concatenate([np.asarray(r) for per in rows_far for r in per]))
    p, _, _ = gpu_prefill(rc, req_far, out["k_out"], out["v_out"], out["route_cu"])
    assert max_abs(p, p_ref) < 1e-2
    p_g, _, _ = rc.attend_prefill_gather(dev(req_far.q), dev(req_far.k_conv), dev(req_far.v_conv), dev(req_far.cu_q),
                                         dev(req_far.q_pos0), req_far.max_q, kc, vc, out["route_idx"], out["route_cu"],
                                         out_dtype=torch.float32)
    assert torch.equal(p_g, p)
    assert rc.poll_status() == 0


def test_pages_past_two_to_the_31_elements():
    """Split-KV decode over a page pool of 300,000 pages (4.9 GB of keys, as much of values): the pages of a
    small decode batch are moved behind page 270,000, where a row's element index no longer fits 31 bits."""
    free, _ = torch.cuda.mem_get_info()
    if free < 16 * 2**30:
        pytest.skip("needs about 10 GB of device memory for the two page pools")
    dec = wl.config4_decode(batch=3, n_res=8, res_len=(100, 260), hist=300)
    sh = dec.shape
    n_small = dec.k_pages.shape[0]
    shift, n_big = 270_000, 300_000
    assert shift * wl.PAGE_TOKENS * sh.head_dim > 2**31 and shift + n_small <= n_big
    k_big = torch.full((n_big, wl.PAGE_TOKENS, sh.head_dim), float("nan"), dtype=sh.torch_dtype, device="cuda")
    v_big = torch.full_like(k_big, float("nan"))
    k_big[shift:shift + n_small] = dev(dec.k_pages)
    v_big[shift:shift + n_small] = dev(dec.v_pages)
    far = lambda t: np.where(t >= 0, t + shift, t).astype(np.int32)
    rc = make_ctx(sh, max_pos=8192)
    od = rc.attend_decode(dev(dec.q), dev(dec.q_pos), k_big, v_big, dev(far(dec.res_page_table)), dev(dec.res_len),
                          dev(far(dec.hist_page_table)), dev(dec.hist_len), out_dtype=torch.float32)
    ref = orc.attend_decode(f64(dec.q), dec.q_pos, f64(dec.k_pages), f64(dec.v_pages), dec.res_page_table,
                            dec.res_len, dec.hist_page_table, dec.hist_len, sh.rope_theta, wl.PAGE_TOKENS,
                            storage=sh.dtype)
    assert max_abs(od, ref) < 1e-2
    assert rc.poll_status() == 0


def test_positions_near_the_end_of_a_long_rotary_table():
    """A conversation that starts at position 130,000 of a 131,072-row cos/sin table (angles of up to 1.3e5
    radians for the fastest frequency: the table is built in double precision on the host); the last query
    token sits on the table's last row."""
    sh = wl.QWEN3_4B
    g = sh.n_kv_heads
    max_pos = 131072
    rng = np.random.default_rng(5)
    lens = [200, 90]
    pool = wl.pack_resources(sh, 55, lens, wl.keep_mask_spans(rng, lens))
    vis = wl.routes_random(rng, g, 2, 0.5)
    tq = 300
    req = wl.make_requests(sh, 56, pool, [[0, 1]], [vis], [tq], q_pos0=[max_pos - tq])
    rc = make_ctx(sh, max_pos=max_pos)
    _, kc_ref, vc_ref = oracle_encode(pool)
    _, kc, vc = gpu_encode(rc, pool)
    out = gpu_compact(rc, pool, req, kc, vc)
    p, k_hat, _ = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"])
    p_ref, k_hat_ref = oracle_prefill(req, oracle_rows(pool, req), kc_ref, vc_ref)
    assert max_abs(p, p_ref) < 1e-2
    # rotated conversation keys at these positions: one bf16 ulp at most (values up to ~4: ulp 2^-6)
    assert max_abs(k_hat.transpose(0, 1) if k_hat.shape[0] == g else k_hat, k_hat_ref) <= 2.0 ** -6
    assert rc.poll_status() == 0
