"""The allocation-free decode entry point gives the same results as the regular
one.  It exists for callers that cannot allocate device memory at the point where
they decode (a frozen memory plan, a plugin in a process that owns all device
memory): its scratch is a fixed array inside the library.  Collected last, so a
run that stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

from paper_2608_19662_b200 import workloads as wl

from pipeline import dev, make_ctx

pytestmark = pytest.mark.gpu


def _run_both(rc, dec, out_dtype):
    args = (dev(dec.q), dev(dec.q_pos), dev(dec.k_pages), dev(dec.v_pages), dev(dec.res_page_table),
            dev(dec.res_len), dev(dec.hist_page_table), dev(dec.hist_len))
    want = rc.attend_decode(*args, out_dtype=out_dtype)
    out = torch.full(tuple(dec.q.shape), float("nan"), dtype=out_dtype, device="cuda")   # allocated by the test
    got = rc.attend_decode_noalloc(*args, out=out)
    torch.cuda.synchronize()
    return got, want


def test_noalloc_decode_matches_regular_entry_point_twice_in_a_row():
    sh = wl.QWEN3_4B
    rc = make_ctx(sh, max_pos=8192)
    # two different batches back to back: the second reuses the scratch the first one dirtied
    first = wl.config4_decode(batch=6, n_res=8, res_len=(100, 400), hist=700, seed=11)
    second = wl.config4_decode(batch=3, n_res=4, res_len=(60, 200), hist=130, seed=12)
    # the first batch really goes through the scratch: its partials (520 B per split, sequence, group
    # and query head of the group) need more than one split per (sequence, group)
    one_split = first.q.shape[0] * sh.n_q_heads * 520
    assert rc.decode_workspace_bytes(first.q.shape[0], first.res_page_table.shape[1],
                                     first.hist_page_table.shape[1]) > one_split
    for dec, dt in ((first, torch.float32), (second, torch.bfloat16), (first, torch.bfloat16)):
        got, want = _run_both(rc, dec, dt)
        assert not torch.isnan(got.float()).any()
        # same kernels, same split plan, same arithmetic order: identical, well inside the 1e-2 bf16 bound
        assert (got.float() - want.float()).abs().max().item() <= 1e-2
        assert torch.equal(got, want)
    assert rc.poll_status() == 0


def test_noalloc_decode_appends_the_current_token_like_the_regular_entry_point():
    """With k_new / v_new the call first writes the current token's rotated key and its
    value into the last history row: same pages and same outputs as the regular call."""
    sh = wl.QWEN3_4B
    rc = make_ctx(sh, max_pos=8192)
    dec = wl.config4_decode(batch=5, n_res=8, res_len=(100, 300), hist=333, seed=13)
    k_new = dev(wl.normal(71, (5, sh.n_kv_heads, sh.head_dim), sh.torch_dtype))
    v_new = dev(wl.normal(72, (5, sh.n_kv_heads, sh.head_dim), sh.torch_dtype))
    tables = (dev(dec.res_page_table), dev(dec.res_len), dev(dec.hist_page_table), dev(dec.hist_len))
    q, q_pos = dev(dec.q), dev(dec.q_pos)
    kp_a, vp_a, kp_b, vp_b = dev(dec.k_pages), dev(dec.v_pages), dev(dec.k_pages), dev(dec.v_pages)
    want = rc.attend_decode(q, q_pos, kp_a, vp_a, *tables, k_new=k_new, v_new=v_new, out_dtype=torch.float32)
    out = torch.full(tuple(dec.q.shape), float("nan"), dtype=torch.float32, device="cuda")
    got = rc.attend_decode_noalloc(q, q_pos, kp_b, vp_b, *tables, out=out, k_new=k_new, v_new=v_new)
    torch.cuda.synchronize()
    assert torch.equal(kp_a.view(torch.int16), kp_b.view(torch.int16))
    assert torch.equal(vp_a.view(torch.int16), vp_b.view(torch.int16))
    assert not torch.equal(kp_b.view(torch.int16), dev(dec.k_pages).view(torch.int16))     # the append did write
    assert torch.equal(got, want)
    assert rc.poll_status() == 0


def test_noalloc_decode_rejects_what_does_not_fit():
    from paper_2608_19662_b200 import ReCacheError
    sh = wl.QWEN3_4B
    rc = make_ctx(sh, max_pos=8192)
    big = 1024                                            # 1024 x 8 groups x splits x 4 heads x 520 B > 4 MiB
    q = torch.zeros((big, sh.n_q_heads, sh.head_dim), dtype=torch.bfloat16, device="cuda")
    pages = torch.zeros((4, wl.PAGE_TOKENS, sh.head_dim), dtype=torch.bfloat16, device="cuda")
    tbl = torch.zeros((big * sh.n_kv_heads, 1), dtype=torch.int32, device="cuda")
    ln = torch.ones(big * sh.n_kv_heads, dtype=torch.int32, device="cuda")
    with pytest.raises(ReCacheError, match="exceeds the 4 MiB"):
        rc.attend_decode_noalloc(q, torch.zeros(big, dtype=torch.int32, device="cuda"), pages, pages, tbl, ln, tbl, ln,
                                 out=torch.empty_like(q))
    rc32 = make_ctx(wl.TINY_F32, max_pos=256)
    with pytest.raises(ReCacheError, match="EUNSUPPORTED"):
        rc32.attend_decode_noalloc(q[:1, :4, :64].float().contiguous(), torch.zeros(1, dtype=torch.int32, device="cuda"),
                                   pages.float()[:, :, :64].contiguous(), pages.float()[:, :, :64].contiguous(),
                                   tbl[:2], ln[:2], tbl[:2], ln[:2], out=torch.empty((1, 4, 64), device="cuda"))
