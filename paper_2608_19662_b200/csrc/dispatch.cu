// Chooses the kernel for each attention call and sizes its scratch.
#include "common.cuh"

int64_t rc_encode_workspace_bytes(const recache_ctx*, int, int, int) { return 0; }
int64_t rc_prefill_workspace_bytes(const recache_ctx*, int, int, int) { return 0; }
int64_t rc_decode_workspace_bytes(const recache_ctx*, int, int, int) { return 0; }

cudaError_t rc_launch_encode_attn(const recache_ctx* ctx, const EncodeArgs& a, cudaStream_t st) {
  AttnRowsArgs r{a.q, a.o, a.out_dtype, a.cu, a.n_res, a.total, nullptr, a.slot, a.k_cache, a.v_cache,
                 a.pool_tokens, nullptr, nullptr, nullptr};
  return rc_launch_attn_rows(ctx, r, st);
}

cudaError_t rc_launch_prefill_attn(const recache_ctx* ctx, const PrefillArgs& a, cudaStream_t st) {
  AttnRowsArgs r{a.q, a.o, a.out_dtype, a.cu_q, a.n_req, a.total_q, a.pos0, nullptr, a.k_conv, a.v_conv,
                 (int64_t)a.total_q, a.k_route, a.v_route, a.route_cu};
  return rc_launch_attn_rows(ctx, r, st);
}

cudaError_t rc_launch_decode(const recache_ctx* ctx, const DecodeArgs& a, cudaStream_t st) {
  return rc_launch_decode_rows(ctx, a, st);
}
