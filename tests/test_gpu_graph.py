"""The hot-path calls are plain stream work: a whole small step (encode,
compaction, prefill, paged compaction, decode) can be captured in a CUDA graph
and replayed with bit-identical results.  (The allocation-free decode entry
point is not part of this test.)"""
import numpy as np
import pytest
import torch

from paper_2608_19662_b200 import workloads as wl

from pipeline import dev, make_ctx

pytestmark = pytest.mark.gpu


def test_step_replays_from_a_cuda_graph():
    from paper_2608_19662_b200 import PACKED
    pool, req = wl.config2()
    sh = pool.shape
    g, d = sh.n_kv_heads, sh.head_dim
    rc = make_ctx(sh, max_pos=8192)
    t = {k: dev(v) for k, v in dict(q=pool.q, k=pool.k, v=pool.v, cu=pool.cu_seqlens, slot=pool.dst_slot, keep=pool.keep,
                                    res_off=req.res_off, res_slot=req.res_slot, res_len=req.res_len, vis=req.vis,
                                    cq=req.q, ck=req.k_conv, cv=req.v_conv, cu_q=req.cu_q, pos0=req.q_pos0).items()}
    E = lambda *s, dtype=torch.bfloat16: torch.zeros(s, dtype=dtype, device="cuda")
    kc, vc = E(g, pool.pool_tokens, d), E(g, pool.pool_tokens, d)
    o_enc = E(pool.total_tokens, sh.n_q_heads, d)
    cap = int(pool.keep.sum()) * g + 8
    r_cu, r_idx = E(g + 1, dtype=torch.int32), E(cap, dtype=torch.int32)
    kr, vr = E(cap, d), E(cap, d)
    o_pre = E(req.total_q, sh.n_q_heads, d)
    kco, vco = E(g, req.total_q, d), E(g, req.total_q, d)
    ws = torch.empty(max(rc.encode_workspace_bytes(len(pool.lens), pool.total_tokens, pool.max_len),
                         rc.compact_workspace_bytes(1, len(req.res_slot)),
                         rc.prefill_workspace_bytes(1, req.total_q, req.max_q), 256), dtype=torch.uint8, device="cuda")

    def step():
        rc.encode_resources(t["q"], t["k"], t["v"], t["cu"], pool.max_len, t["slot"], kc, vc, out=o_enc, workspace=ws)
        rc.compact_routes(kc, vc, t["keep"], t["res_off"], t["res_slot"], t["res_len"], t["vis"], PACKED, r_cu, r_idx, kr, vr,
                          workspace=ws)
        rc.attend_prefill(t["cq"], t["ck"], t["cv"], t["cu_q"], t["pos0"], req.max_q, kr, vr, r_cu, k_conv_out=kco,
                          v_conv_out=vco, out=o_pre, workspace=ws)

    step()                                   # eager: also does every one-time set-up
    torch.cuda.synchronize()
    want = [x.clone() for x in (o_enc, o_pre, r_idx, kr)]
    for x in (o_enc, o_pre, r_idx, kr, kc, vc):
        x.zero_()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    graph.replay()
    torch.cuda.synchronize()
    for a, b in zip((o_enc, o_pre, r_idx, kr), want):
        assert torch.equal(a, b)
    # timing: launch-bound small workload, eager vs replay
    def timed(fn, n=50):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fn(); torch.cuda.synchronize()
        e0.record()
        for _ in range(n):
            fn()
        e1.record(); torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n * 1e3
    print(f"config-2 step: eager {timed(step):.1f} us, graph replay {timed(graph.replay):.1f} us")
    assert rc.poll_status() == 0
