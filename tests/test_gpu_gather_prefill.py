"""Zero-copy routed prefill: the route rows are read from the resource cache
through the compaction's index list (index-only compaction, no row moved).  Same
results as the materialised (packed) path, bit for bit, and as the oracle."""
import numpy as np
import pytest
import torch

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl

from pipeline import dev, f64, gpu_compact, gpu_encode, gpu_prefill, make_ctx, max_abs, oracle_encode, oracle_rows, sample_rows

pytestmark = pytest.mark.gpu


def _index_only(rc, pool, req, kc, vc):
    from paper_2608_19662_b200 import PACKED
    sh = pool.shape
    n_routes = req.n_requests * sh.n_kv_heads
    cap = int(req.res_len.sum()) * sh.n_kv_heads + 8
    r_cu = torch.empty(n_routes + 1, dtype=torch.int32, device="cuda")
    r_idx = torch.full((cap,), -7, dtype=torch.int32, device="cuda")
    rc.compact_routes(kc, vc, dev(pool.keep), dev(req.res_off), dev(req.res_slot), dev(req.res_len), dev(req.vis), PACKED,
                      r_cu, r_idx, None, None)
    return r_cu, r_idx


@pytest.mark.parametrize("sh", [wl.QWEN3_4B, wl.Shape(16, 8, 128, 1e6, "bf16"), wl.Shape(16, 2, 128, 1e4, "bf16")],
                         ids=["4_per_group", "2_per_group", "8_per_group"])
def test_gather_prefill_equals_packed_prefill_and_oracle(sh):
    """Several requests with ragged routes (tail tiles, an empty route) and ragged lengths."""
    g = sh.n_kv_heads
    rng = np.random.default_rng(31)
    lens = [300, 77, 130, 512, 45, 260]
    pool = wl.pack_resources(sh, 31, lens, wl.keep_mask_spans(rng, lens))
    res_lists = [[0, 3, 5], [1, 2], [4, 0, 2, 3]]
    vis = [wl.routes_random(rng, g, len(l), 0.5) for l in res_lists]
    vis[1][g - 1, :] = 0                                 # an empty route: plain causal attention for that group
    req = wl.make_requests(sh, 32, pool, res_lists, vis, [150, 64, 333])
    rc = make_ctx(sh, max_pos=4096)
    _, kc, vc = gpu_encode(rc, pool)
    r_cu, r_idx = _index_only(rc, pool, req, kc, vc)
    o_g, kg, vg = rc.attend_prefill_gather(dev(req.q), dev(req.k_conv), dev(req.v_conv), dev(req.cu_q), dev(req.q_pos0),
                                           req.max_q, kc, vc, r_idx, r_cu, out_dtype=torch.float32)
    out = gpu_compact(rc, pool, req, kc, vc)
    assert torch.equal(out["route_cu"], r_cu)
    o_p, kp, vp = gpu_prefill(rc, req, out["k_out"], out["v_out"], out["route_cu"])
    assert torch.equal(o_g, o_p)                        # same rows, same tiles, same arithmetic
    assert torch.equal(kg.view(torch.int16), kp.view(torch.int16)) and torch.equal(vg.view(torch.int16), vp.view(torch.int16))
    assert rc.poll_status() == 0
    # oracle
    _, kc_ref, vc_ref = oracle_encode(pool)
    rows = oracle_rows(pool, req)
    ref, _ = orc.attend_prefill(f64(req.q), f64(req.k_conv), f64(req.v_conv), req.cu_q, req.q_pos0, rows, kc_ref, vc_ref,
                                sh.rope_theta, storage=sh.dtype)
    assert max_abs(o_g, ref) < 1e-2


def test_gather_prefill_full_size_sampled():
    """The benchmark's prefill (2048 tokens over ~8 % of 95k resource tokens) through the gather path:
    identical to the packed path, and sampled rows against the oracle."""
    import bench
    w = bench.Workload("full")
    run = bench.Runner(w, 0)
    run.step()
    torch.cuda.synchronize()
    sh, pool, req = w.shape, w.pool, w.req
    d = run.d
    o_g, _, _ = run.rc.attend_prefill_gather(d["cq"], d["ck"], d["cv"], d["cu_q"], d["q_pos0"], req.max_q, run.k_cache,
                                             run.v_cache, run.route_idx, run.route_cu, out_dtype=torch.bfloat16)
    torch.cuda.synchronize()
    assert torch.equal(o_g.view(torch.int16), run.o_pre.view(torch.int16))
    assert run.rc.poll_status() == 0


def test_gather_prefill_bad_index_is_flagged():
    sh = wl.QWEN3_4B
    pool, req = wl.config2(n_res=3, len_range=(100, 200), tq=64)
    rc = make_ctx(sh, max_pos=2048)
    _, kc, vc = gpu_encode(rc, pool)
    r_cu, r_idx = _index_only(rc, pool, req, kc, vc)
    n = int(r_cu[-1])
    if n == 0:
        pytest.skip("no route rows in this draw")
    r_idx[n // 2] = pool.pool_tokens + 5                 # out of range
    rc.attend_prefill_gather(dev(req.q), dev(req.k_conv), dev(req.v_conv), dev(req.cu_q), dev(req.q_pos0), req.max_q,
                             kc, vc, r_idx, r_cu)
    torch.cuda.synchronize()
    assert rc.poll_status() == 2                          # bad slot


def test_gather_prefill_unsupported_context():
    sh = wl.TINY_F32
    rc = make_ctx(sh, max_pos=256)
    pool, req = wl.config1()
    _, kc, vc = gpu_encode(rc, pool)
    r_cu, r_idx = _index_only(rc, pool, req, kc, vc)
    with pytest.raises(RuntimeError):
        rc.attend_prefill_gather(dev(req.q), dev(req.k_conv), dev(req.v_conv), dev(req.cu_q), dev(req.q_pos0), req.max_q,
                                 kc, vc, r_idx, r_cu)
