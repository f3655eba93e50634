"""Two contexts driven from two streams at the same time give the same results
as one after the other, and back-to-back calls that reuse one workspace on one
stream stay ordered: the work list of the tensor-core attention is built on a
second stream of the context (forked from and joined to the caller's stream by
events), which must not be visible from outside."""
import numpy as np
import pytest
import torch

from paper_2608_19662_b200 import workloads as wl

from pipeline import dev, make_ctx

pytestmark = pytest.mark.gpu


def _state(seed):
    from paper_2608_19662_b200 import PACKED
    pool, req = wl.config2(seed=wl.SEED0 + 50 + seed)
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
    ws = torch.empty(max(rc.encode_workspace_bytes(len(pool.lens), pool.total_tokens, pool.max_len),
                         rc.compact_workspace_bytes(1, len(req.res_slot)),
                         rc.prefill_workspace_bytes(1, req.total_q, req.max_q), 256), dtype=torch.uint8, device="cuda")

    def step():
        # one workspace for all three calls: the second call's work list overwrites the first one's
        rc.encode_resources(t["q"], t["k"], t["v"], t["cu"], pool.max_len, t["slot"], kc, vc, out=o_enc, workspace=ws)
        rc.compact_routes(kc, vc, t["keep"], t["res_off"], t["res_slot"], t["res_len"], t["vis"], PACKED, r_cu, r_idx, kr, vr,
                          workspace=ws)
        rc.attend_prefill(t["cq"], t["ck"], t["cv"], t["cu_q"], t["pos0"], req.max_q, kr, vr, r_cu, out=o_pre, workspace=ws)

    return rc, step, (o_enc, o_pre, r_idx, kr)


def test_two_contexts_on_two_streams():
    a, b = _state(0), _state(1)
    for _, step, _ in (a, b):                 # one after the other, default stream
        step()
    torch.cuda.synchronize()
    want = [[x.clone() for x in s[2]] for s in (a, b)]
    for s in (a, b):
        for x in s[2]:
            x.zero_()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for st in streams:
        st.wait_stream(torch.cuda.current_stream())
    for rep in range(6):                      # interleaved launches from both streams, several steps deep
        for s, st in zip((a, b), streams):
            with torch.cuda.stream(st):
                s[1]()
    torch.cuda.synchronize()
    for s, w in zip((a, b), want):
        for x, y in zip(s[2], w):
            assert torch.equal(x, y)
        assert s[0].poll_status() == 0
