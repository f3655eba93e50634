"""Encoding behind a shared prefix and with global position offsets (the
"Block" ablation) on the GPU against the oracle, fp32 and bf16 paths."""
import numpy as np
import pytest
import torch

from oracle import recache_oracle as orc
from paper_2608_19662_b200 import workloads as wl

from pipeline import dev, f64, make_ctx, max_abs
from test_gpu_parity import assert_rotated_close

pytestmark = pytest.mark.gpu


def _case(sh, lens, P, seed):
    rng = np.random.default_rng(seed)
    pool = wl.pack_resources(sh, seed, lens, wl.keep_mask_spans(rng, lens), slot_gap=3)
    _, kp, vp = wl.resource_tensors(seed, 900, P, sh)
    return pool, kp, vp


@pytest.mark.parametrize("shape,tol,lens,P", [
    (wl.TINY_F32, 1e-5, [17, 40, 23], 9),
    (wl.QWEN3_4B, 1e-2, [130, 64, 257, 33, 200], 150),      # prefix longer than one key tile
    (wl.Shape(16, 8, 128, 1e6, "bf16"), 1e-2, [70, 190], 37),
])
def test_prefixed_and_block_encode(shape, tol, lens, P):
    sh = shape
    pool, kp, vp = _case(sh, lens, P, 41)
    rc = make_ctx(sh, max_pos=4096)
    g, d = sh.n_kv_heads, sh.head_dim
    # the prefix as a cache holds it: keys rotated at 0..P-1 in the storage dtype (from the oracle)
    pk = orc.round_storage(np.transpose(orc.rope(f64(kp), np.arange(P), sh.rope_theta), (1, 0, 2)), sh.dtype)
    pv = np.transpose(f64(vp), (1, 0, 2))
    pk_d, pv_d = dev(pk).to(sh.torch_dtype).contiguous(), dev(pv).to(sh.torch_dtype).contiguous()
    for name, offs in (("local", [P] * len(lens)), ("block", [P + int(c) for c in pool.cu_seqlens[:-1]])):
        ref_o, ref_k, ref_v = orc.encode_resources(f64(pool.q), f64(pool.k), f64(pool.v), pool.cu_seqlens, sh.rope_theta,
                                                   storage=sh.dtype, pos_offset=offs, prefix_k=pk, prefix_v=pv)
        kc = torch.full((g, pool.pool_tokens, d), float("nan"), dtype=sh.torch_dtype, device="cuda")
        vc = torch.full_like(kc, float("nan"))
        o = rc.encode_resources_prefixed(dev(pool.q), dev(pool.k), dev(pool.v), dev(pool.cu_seqlens), pool.max_len,
                                         dev(pool.dst_slot), kc, vc, k_prefix=pk_d, v_prefix=pv_d,
                                         pos_offset=dev(np.asarray(offs, np.int32)), out_dtype=torch.float32)
        assert max_abs(o, ref_o) < tol, name
        kc_ref = np.full((g, pool.pool_tokens, d), np.nan); vc_ref = np.full_like(kc_ref, np.nan)
        orc.write_cache(kc_ref, vc_ref, ref_k, ref_v, pool.cu_seqlens, pool.dst_slot)
        written = ~np.isnan(kc_ref)
        assert np.array_equal(np.isnan(f64(kc)), ~written)
        assert_rotated_close(sh, kc, np.where(written, kc_ref, 0.0), written)
    # no prefix, no offsets: the extended call is the plain one, bit for bit
    kc1 = torch.zeros((g, pool.pool_tokens, d), dtype=sh.torch_dtype, device="cuda"); vc1 = torch.zeros_like(kc1)
    kc2, vc2 = torch.zeros_like(kc1), torch.zeros_like(kc1)
    a = rc.encode_resources(dev(pool.q), dev(pool.k), dev(pool.v), dev(pool.cu_seqlens), pool.max_len, dev(pool.dst_slot), kc1, vc1)
    b = rc.encode_resources_prefixed(dev(pool.q), dev(pool.k), dev(pool.v), dev(pool.cu_seqlens), pool.max_len,
                                     dev(pool.dst_slot), kc2, vc2)
    assert torch.equal(a, b) and torch.equal(kc1, kc2)
    assert rc.poll_status() == 0
