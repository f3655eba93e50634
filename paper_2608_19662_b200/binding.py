"""Thin ctypes binding over librecache.so: argument marshalling only.

Every step of the hot path runs in the library's CUDA kernels; torch provides
device memory and the current stream.  There is no CPU fallback: loading fails
loudly when the shared library has not been built (run
`python -m paper_2608_19662_b200.build`).
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "librecache.so")

F32, BF16 = 0, 1
PACKED, PAGED = 0, 1
STATUS_NAMES = {0: "OK", 1: "EINVAL", 2: "ESHAPE", 3: "EUNSUPPORTED", 4: "ENOMEM", 5: "ECUDA"}
DEVICE_CODES = {0: "ok", 1: "bad seqlens", 2: "bad slot", 3: "row capacity overflow", 4: "bad page",
                5: "free pages exhausted", 6: "position outside rotary table"}


class Desc(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("dtype", C.c_int32), ("max_pos", C.c_int32), ("page_tokens", C.c_int32),
                ("rope_theta", C.c_double)]


_P, _I32, _I64 = C.c_void_p, C.c_int32, C.c_int64
SIGNATURES = {
    "recache_create": (C.c_int, [C.POINTER(_P), C.POINTER(Desc), C.c_int]),
    "recache_destroy": (None, [_P]),
    "recache_last_error": (C.c_char_p, [_P]),
    "recache_poll_status": (C.c_int, [_P, _P, C.POINTER(_I32)]),
    "recache_kernel_count": (_I32, []),
    "recache_kernel_name": (C.c_char_p, [_I32]),
    "recache_selftest_wait_timeout": (C.c_int, [_P, _P, _P]),
    "recache_kernel_timer": (C.c_int, [_P, _I32]),
    "recache_kernel_times": (C.c_int, [_P, C.POINTER(C.c_float), C.POINTER(_I64)]),
    "recache_encode_workspace_bytes": (_I64, [_P, _I32, _I32, _I32]),
    "recache_compact_workspace_bytes": (_I64, [_P, _I32, _I32]),
    "recache_prefill_workspace_bytes": (_I64, [_P, _I32, _I32, _I32]),
    "recache_decode_workspace_bytes": (_I64, [_P, _I32, _I32, _I32]),
    "recache_encode_resources": (C.c_int, [_P, _P, _P, _P, _P, _I32, _I32, _I32, _P, _P, _P, _I64, _P, _I32,
                                           _P, _I64, _P]),
    "recache_encode_resources_prefixed": (C.c_int, [_P, _P, _P, _P, _P, _I32, _I32, _I32, _P, _P, _P, _I64, _P, _P,
                                                    _I32, _P, _P, _I32, _P, _I64, _P]),
    "recache_compact_routes": (C.c_int, [_P, _P, _P, _I64, _P, _P, _P, _P, _I32, _I32, _P, _I32, _P, _P, _P,
                                         _I64, _P, _P, _P, _I32, _P, _I64, _I64, _P, _I64, _P]),
    "recache_attend_prefill": (C.c_int, [_P, _P, _P, _P, _P, _P, _I32, _I32, _I32, _P, _P, _P, _I64, _P, _P,
                                         _P, _I32, _P, _I64, _P]),
    "recache_attend_prefill_gather": (C.c_int, [_P, _P, _P, _P, _P, _P, _I32, _I32, _I32, _P, _P, _I64, _P, _P, _I64,
                                                _P, _P, _P, _I32, _P, _I64, _P]),
    "recache_attend_prefill_history": (C.c_int, [_P, _P, _P, _P, _P, _P, _I32, _I32, _I32, _P, _P, _P, _I64, _P, _P,
                                                 _I64, _P, _P, _P, _I32, _P, _I64, _P]),
    "recache_attend_decode": (C.c_int, [_P, _P, _P, _I32, _P, _P, _P, _P, _I64, _P, _I32, _P, _P, _I32, _P,
                                        _P, _I32, _P, _I64, _P]),
    "recache_attend_decode_gather": (C.c_int, [_P, _P, _P, _I32, _P, _P, _P, _P, _I64, _P, _P, _I64, _I32, _P, _P, _I64,
                                               _P, _I32, _P, _P, _I32, _P, _I64, _P]),
    "recache_build_routes": (C.c_int, [C.POINTER(C.c_double), _I32, C.POINTER(C.c_double), _I32, _I32, _I32,
                                       C.POINTER(C.c_uint8), C.POINTER(C.c_double), C.POINTER(C.c_double),
                                       C.POINTER(C.c_double)]),
    "recache_attend_decode_noalloc": (C.c_int, [_P, _P, _P, _I32, _P, _P, _P, _P, _I64, _P, _I32, _P, _P, _I32, _P,
                                                _P, _I32, _P]),
}

_lib = None


def load_library() -> C.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_19662_b200.build` "
                               "(there is no fallback path)")
        lib = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


class ReCacheError(RuntimeError):
    pass


def build_routes(s_layers, s_groups, k_layers: int, k_groups: int):
    """recache_build_routes (host only): returns (omega [L][G] uint8 numpy array, cc_layers, cc_groups, rho)."""
    import numpy as np
    lib = load_library()
    sl = np.ascontiguousarray(s_layers, dtype=np.float64)
    sg = np.ascontiguousarray(s_groups, dtype=np.float64)
    omega = np.zeros((len(sl), len(sg)), dtype=np.uint8)
    ccl, ccg, rho = C.c_double(), C.c_double(), C.c_double()
    dp = lambda a: a.ctypes.data_as(C.POINTER(C.c_double))
    st = lib.recache_build_routes(dp(sl), len(sl), dp(sg), len(sg), int(k_layers), int(k_groups),
                                  omega.ctypes.data_as(C.POINTER(C.c_uint8)), C.byref(ccl), C.byref(ccg), C.byref(rho))
    if st != 0:
        raise ReCacheError(f"recache_build_routes: {STATUS_NAMES.get(st, st)}")
    return omega, ccl.value, ccg.value, rho.value


class ReCache:
    """One context = one attention shape (heads, head_dim, dtype, rotary table) on one device."""

    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, rope_theta: float, dtype: str = "bf16",
                 max_pos: int = 8192, page_tokens: int = 64, device: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("resource-routed attention needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.desc = Desc(n_q_heads, n_kv_heads, head_dim, BF16 if dtype == "bf16" else F32, max_pos,
                         page_tokens, float(rope_theta))
        self.device = torch.device("cuda", device)
        self.torch_dtype = torch.bfloat16 if dtype == "bf16" else torch.float32
        self.dtype_code = self.desc.dtype
        h = _P()
        st = self.lib.recache_create(C.byref(h), C.byref(self.desc), device)
        if st != 0:
            raise ReCacheError(f"recache_create failed: {STATUS_NAMES.get(st, st)}")
        self.h = h
        self._ws = None

    def close(self):
        if getattr(self, "h", None):
            self.lib.recache_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---------------------------------------------------------------- helpers --
    def _check(self, st: int, what: str):
        if st != 0:
            msg = self.lib.recache_last_error(self.h).decode()
            raise ReCacheError(f"{what}: {STATUS_NAMES.get(st, st)}: {msg}")

    def workspace(self, nbytes: int) -> torch.Tensor:
        """A cached scratch tensor of at least nbytes (torch owns the memory)."""
        nbytes = max(int(nbytes), 256)
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        return self._ws

    def _out_code(self, out_dtype: Optional[torch.dtype]):
        od = self.torch_dtype if out_dtype is None else out_dtype
        return od, (F32 if od == torch.float32 else BF16)

    def poll_status(self) -> int:
        code = _I32(0)
        self._check(self.lib.recache_poll_status(self.h, _stream(), C.byref(code)), "recache_poll_status")
        return int(code.value)

    def selftest_wait_timeout(self):
        """Runs the bounded-wait self-test kernel (a wait on a barrier nobody arrives at); returns
        (gave_up, kilo-cycles waited).  poll_status() afterwards reports the time-out once."""
        report = torch.zeros(2, dtype=torch.int32, device=self.device)
        self._check(self.lib.recache_selftest_wait_timeout(self.h, _ptr(report), _stream()),
                    "recache_selftest_wait_timeout")
        r = report.cpu().tolist()
        return bool(r[0]), int(r[1])

    def last_error(self) -> str:
        """Text of the context's last error (after a device time-out: which wait ran out)."""
        return self.lib.recache_last_error(self.h).decode()

    def kernel_timer(self, enable):
        """False / 0: off; True / 1: an event pair around every launch; 2: around the attention launches only."""
        self._check(self.lib.recache_kernel_timer(self.h, int(enable)), "recache_kernel_timer")

    def kernel_times(self):
        """{kernel name: (total ms, launches)} since the last call; clears the counters."""
        n = self.lib.recache_kernel_count()
        ms = (C.c_float * n)()
        cnt = (_I64 * n)()
        self._check(self.lib.recache_kernel_times(self.h, ms, cnt), "recache_kernel_times")
        return {self.lib.recache_kernel_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n)}

    # -------------------------------------------------------------- hot path --
    def encode_workspace_bytes(self, n_resources, total_tokens, max_len) -> int:
        return int(self.lib.recache_encode_workspace_bytes(self.h, n_resources, total_tokens, max_len))

    def compact_workspace_bytes(self, n_requests, total_listed) -> int:
        return int(self.lib.recache_compact_workspace_bytes(self.h, n_requests, total_listed))

    def prefill_workspace_bytes(self, n_requests, total_q, max_q) -> int:
        return int(self.lib.recache_prefill_workspace_bytes(self.h, n_requests, total_q, max_q))

    def decode_workspace_bytes(self, batch, max_res_pages, max_hist_pages) -> int:
        return int(self.lib.recache_decode_workspace_bytes(self.h, batch, max_res_pages, max_hist_pages))

    def encode_resources(self, q, k, v, cu_seqlens, max_len, dst_slot, k_cache, v_cache, out=None,
                         out_dtype=None, workspace=None):
        """recache_encode_resources: q [T,Hq,d], k/v [T,G,d], caches [G,pool,d]. Returns o [T,Hq,d]."""
        n_res = cu_seqlens.numel() - 1
        total = q.shape[0]
        od, oc = self._out_code(out_dtype)
        if out is None:
            out = torch.empty(q.shape, dtype=od, device=q.device)
        ws = workspace if workspace is not None else self.workspace(self.encode_workspace_bytes(n_res, total, max_len))
        st = self.lib.recache_encode_resources(self.h, _ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens), n_res, total,
                                               int(max_len), _ptr(dst_slot), _ptr(k_cache), _ptr(v_cache),
                                               k_cache.shape[1], _ptr(out), oc, _ptr(ws), ws.numel(), _stream())
        self._check(st, "recache_encode_resources")
        return out

    def encode_resources_prefixed(self, q, k, v, cu_seqlens, max_len, dst_slot, k_cache, v_cache, k_prefix=None,
                                  v_prefix=None, pos_offset=None, out=None, out_dtype=None, workspace=None):
        """recache_encode_resources_prefixed: encode behind a shared prefix [G,P,d] and / or with a first
        position per resource (pos_offset [N]).  Returns o [T,Hq,d]."""
        n_res = cu_seqlens.numel() - 1
        total = q.shape[0]
        od, oc = self._out_code(out_dtype)
        if out is None:
            out = torch.empty(q.shape, dtype=od, device=q.device)
        ws = workspace if workspace is not None else self.workspace(self.encode_workspace_bytes(n_res, total, max_len))
        st = self.lib.recache_encode_resources_prefixed(
            self.h, _ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens), n_res, total, int(max_len), _ptr(dst_slot),
            _ptr(k_cache), _ptr(v_cache), k_cache.shape[1], _ptr(k_prefix), _ptr(v_prefix),
            0 if k_prefix is None else k_prefix.shape[1], _ptr(pos_offset), _ptr(out), oc, _ptr(ws), ws.numel(), _stream())
        self._check(st, "recache_encode_resources_prefixed")
        return out

    def compact_routes(self, k_cache, v_cache, keep, res_off, res_slot, res_len, vis, mode, route_cu, route_idx,
                       k_out, v_out, route_len=None, page_table=None, free_pages=None, workspace=None):
        """recache_compact_routes.  All outputs are caller-allocated tensors:
        route_cu [B*G+1], route_idx [capacity], k_out/v_out packed [capacity,d] or page pools
        [n_pages,page_tokens,d]; paged mode also needs page_table [B*G,max_pages] and free_pages."""
        n_req = res_off.numel() - 1
        total_listed = res_slot.numel()
        ws = workspace if workspace is not None else self.workspace(self.compact_workspace_bytes(n_req, total_listed))
        paged = mode == PAGED
        st = self.lib.recache_compact_routes(
            self.h, _ptr(k_cache), _ptr(v_cache), k_cache.shape[1], _ptr(keep), _ptr(res_off), _ptr(res_slot),
            _ptr(res_len), n_req, total_listed, _ptr(vis), mode, _ptr(route_cu), _ptr(route_len), _ptr(route_idx),
            route_idx.numel() if (paged or k_out is None) else min(route_idx.numel(), k_out.shape[0]), _ptr(k_out),
            _ptr(v_out),
            _ptr(page_table),
            page_table.shape[1] if paged else 0, _ptr(free_pages), free_pages.numel() if paged else 0,
            k_out.shape[0] if paged else 0, _ptr(ws), ws.numel(), _stream())
        self._check(st, "recache_compact_routes")

    def attend_prefill(self, q, k_conv, v_conv, cu_q, q_pos0, max_q, k_route, v_route, route_cu, k_conv_out=None,
                       v_conv_out=None, out=None, out_dtype=None, workspace=None):
        """recache_attend_prefill.  Returns (o [Tq,Hq,d], k_conv_out [G,Tq,d], v_conv_out [G,Tq,d])."""
        n_req = cu_q.numel() - 1
        total_q = q.shape[0]
        g, d = k_conv.shape[1], k_conv.shape[2]
        od, oc = self._out_code(out_dtype)
        if out is None:
            out = torch.empty(q.shape, dtype=od, device=q.device)
        if k_conv_out is None:
            k_conv_out = torch.empty((g, total_q, d), dtype=k_conv.dtype, device=q.device)
        if v_conv_out is None:
            v_conv_out = torch.empty((g, total_q, d), dtype=k_conv.dtype, device=q.device)
        ws = workspace if workspace is not None else self.workspace(self.prefill_workspace_bytes(n_req, total_q, max_q))
        st = self.lib.recache_attend_prefill(self.h, _ptr(q), _ptr(k_conv), _ptr(v_conv), _ptr(cu_q), _ptr(q_pos0),
                                             n_req, total_q, int(max_q), _ptr(k_route), _ptr(v_route), _ptr(route_cu),
                                             k_route.shape[0], _ptr(k_conv_out), _ptr(v_conv_out), _ptr(out), oc,
                                             _ptr(ws), ws.numel(), _stream())
        self._check(st, "recache_attend_prefill")
        return out, k_conv_out, v_conv_out

    def attend_prefill_gather(self, q, k_conv, v_conv, cu_q, q_pos0, max_q, k_cache, v_cache, route_idx, route_cu,
                              k_conv_out=None, v_conv_out=None, out=None, out_dtype=None, workspace=None):
        """recache_attend_prefill_gather: the route rows are read from the resource cache [G,pool,d]
        through route_idx (index-only compaction).  Returns (o, k_conv_out, v_conv_out)."""
        n_req = cu_q.numel() - 1
        total_q = q.shape[0]
        g, d = k_conv.shape[1], k_conv.shape[2]
        od, oc = self._out_code(out_dtype)
        if out is None:
            out = torch.empty(q.shape, dtype=od, device=q.device)
        if k_conv_out is None:
            k_conv_out = torch.empty((g, total_q, d), dtype=k_conv.dtype, device=q.device)
        if v_conv_out is None:
            v_conv_out = torch.empty((g, total_q, d), dtype=k_conv.dtype, device=q.device)
        ws = workspace if workspace is not None else self.workspace(self.prefill_workspace_bytes(n_req, total_q, max_q))
        st = self.lib.recache_attend_prefill_gather(
            self.h, _ptr(q), _ptr(k_conv), _ptr(v_conv), _ptr(cu_q), _ptr(q_pos0), n_req, total_q, int(max_q),
            _ptr(k_cache), _ptr(v_cache), k_cache.shape[1], _ptr(route_idx), _ptr(route_cu), route_idx.numel(),
            _ptr(k_conv_out), _ptr(v_conv_out), _ptr(out), oc, _ptr(ws), ws.numel(), _stream())
        self._check(st, "recache_attend_prefill_gather")
        return out, k_conv_out, v_conv_out

    def attend_prefill_history(self, q, k_conv, v_conv, cu_q, q_pos0, max_q, k_route, v_route, route_cu,
                               k_conv_cache, v_conv_cache, conv_slot, hist_len, out=None, out_dtype=None, workspace=None):
        """recache_attend_prefill_history: a later turn over caches [G,rows,d] that already hold hist_len[b]
        rows per request from conv_slot[b]; appends the new rotated keys / values there.  Returns o."""
        n_req = cu_q.numel() - 1
        total_q = q.shape[0]
        od, oc = self._out_code(out_dtype)
        if out is None:
            out = torch.empty(q.shape, dtype=od, device=q.device)
        ws = workspace if workspace is not None else self.workspace(self.prefill_workspace_bytes(n_req, total_q, max_q))
        st = self.lib.recache_attend_prefill_history(
            self.h, _ptr(q), _ptr(k_conv), _ptr(v_conv), _ptr(cu_q), _ptr(q_pos0), n_req, total_q, int(max_q),
            _ptr(k_route), _ptr(v_route), _ptr(route_cu), k_route.shape[0], _ptr(k_conv_cache), _ptr(v_conv_cache),
            k_conv_cache.shape[1], _ptr(conv_slot), _ptr(hist_len), _ptr(out), oc, _ptr(ws), ws.numel(), _stream())
        self._check(st, "recache_attend_prefill_history")
        return out

    def attend_decode(self, q, q_pos, k_pages, v_pages, res_page_table, res_len, hist_page_table, hist_len,
                      k_new=None, v_new=None, out=None, out_dtype=None, workspace=None):
        """recache_attend_decode.  q [B,Hq,d]; tables [B*G,max_pages]. Returns o [B,Hq,d]."""
        batch = q.shape[0]
        od, oc = self._out_code(out_dtype)
        if out is None:
            out = torch.empty(q.shape, dtype=od, device=q.device)
        mr, mh = res_page_table.shape[1], hist_page_table.shape[1]
        ws = workspace if workspace is not None else self.workspace(self.decode_workspace_bytes(batch, mr, mh))
        st = self.lib.recache_attend_decode(self.h, _ptr(q), _ptr(q_pos), batch, _ptr(k_new), _ptr(v_new),
                                            _ptr(k_pages), _ptr(v_pages), k_pages.shape[0], _ptr(res_page_table), mr,
                                            _ptr(res_len), _ptr(hist_page_table), mh, _ptr(hist_len), _ptr(out), oc,
                                            _ptr(ws), ws.numel(), _stream())
        self._check(st, "recache_attend_decode")
        return out

    def attend_decode_gather(self, q, q_pos, k_cache, v_cache, route_idx, route_cu, max_res_pages, k_pages, v_pages,
                             hist_page_table, hist_len, k_new=None, v_new=None, out=None, out_dtype=None, workspace=None):
        """recache_attend_decode_gather: decode whose resource rows are read from the cache through the
        compaction's index list (nothing materialised).  Returns o [B,Hq,d]."""
        batch = q.shape[0]
        od, oc = self._out_code(out_dtype)
        if out is None:
            out = torch.empty(q.shape, dtype=od, device=q.device)
        mh = hist_page_table.shape[1]
        ws = workspace if workspace is not None else self.workspace(self.decode_workspace_bytes(batch, max_res_pages, mh))
        st = self.lib.recache_attend_decode_gather(
            self.h, _ptr(q), _ptr(q_pos), batch, _ptr(k_new), _ptr(v_new), _ptr(k_cache), _ptr(v_cache), k_cache.shape[1],
            _ptr(route_idx), _ptr(route_cu), route_idx.numel(), int(max_res_pages), _ptr(k_pages), _ptr(v_pages),
            k_pages.shape[0],
            _ptr(hist_page_table), mh, _ptr(hist_len), _ptr(out), oc, _ptr(ws), ws.numel(), _stream())
        self._check(st, "recache_attend_decode_gather")
        return out

    def attend_decode_noalloc(self, q, q_pos, k_pages, v_pages, res_page_table, res_len, hist_page_table, hist_len,
                              out, k_new=None, v_new=None):
        """recache_attend_decode_noalloc: decode for callers that must not allocate where they decode.
        `out` [B,Hq,d] (bf16 or fp32) is caller-provided; the split partials live in the library's own
        4 MiB scratch, so neither the library nor this wrapper allocates anything.  Calls on one device
        share that scratch: do not overlap them on different streams."""
        oc = F32 if out.dtype == torch.float32 else BF16
        st = self.lib.recache_attend_decode_noalloc(
            self.h, _ptr(q), _ptr(q_pos), q.shape[0], _ptr(k_new), _ptr(v_new), _ptr(k_pages), _ptr(v_pages),
            k_pages.shape[0], _ptr(res_page_table), res_page_table.shape[1], _ptr(res_len), _ptr(hist_page_table),
            hist_page_table.shape[1], _ptr(hist_len), _ptr(out), oc, _stream())
        self._check(st, "recache_attend_decode_noalloc")
        return out
