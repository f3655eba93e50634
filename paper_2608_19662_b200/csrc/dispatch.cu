// Chooses the kernel for each attention call and sizes its scratch.
//   fp32 contexts, and bf16 shapes the tensor-core kernel does not cover
//   (head_dim 64, one or more than eight query heads per group): exact row kernels.
//   bf16, head_dim 128, 2/4/8 query heads per group: tcgen05 kernel.
//   bf16 decode, head_dim 128, 64-token pages, <= 8 heads per group: split-KV kernel.
#include "common.cuh"

int64_t rc_encode_workspace_bytes(const recache_ctx* ctx, int n_res, int total, int max_len) {
  return rc_tc_supported(ctx) ? rc_tc_workspace_bytes(ctx, n_res, total, max_len) : 0;
}
int64_t rc_prefill_workspace_bytes(const recache_ctx* ctx, int n_req, int total_q, int max_q) {
  return rc_tc_supported(ctx) ? rc_tc_workspace_bytes(ctx, n_req, total_q, max_q) : 0;
}
int64_t rc_decode_workspace_bytes(const recache_ctx* ctx, int batch, int max_res_pages, int max_hist_pages) {
  return rc_decode_split_supported(ctx) ? rc_decode_split_workspace_bytes(ctx, batch, max_res_pages, max_hist_pages) : 0;
}

cudaError_t rc_launch_encode_attn(const recache_ctx* ctx, const EncodeArgs& a, cudaStream_t st) {
  if (rc_tc_supported(ctx)) {
    TcAttnArgs t{a.q, a.o, a.out_dtype, a.cu, a.n_res, a.total, a.max_len, a.pos_offset, a.slot, a.k_cache, a.v_cache,
                 a.pool_tokens, a.k_prefix, a.v_prefix, nullptr, (int64_t)ctx->desc.n_kv_heads * a.prefix_len,
                 a.workspace, a.prefix_len};
    return rc_launch_attn_tc(ctx, t, st);
  }
  AttnRowsArgs r{a.q, a.o, a.out_dtype, a.cu, a.n_res, a.total, a.pos_offset, a.slot, a.k_cache, a.v_cache,
                 a.pool_tokens, a.k_prefix, a.v_prefix, nullptr, a.prefix_len};
  r.route_rows = (int64_t)ctx->desc.n_kv_heads * a.prefix_len;
  return rc_launch_attn_rows(ctx, r, st);
}

cudaError_t rc_launch_prefill_attn(const recache_ctx* ctx, const PrefillArgs& a, cudaStream_t st) {
  if (rc_tc_supported(ctx)) {
    TcAttnArgs t{a.q, a.o, a.out_dtype, a.cu_q, a.n_req, a.total_q, a.max_q, a.pos0, a.conv_slot, a.k_conv, a.v_conv,
                 a.conv_rows, a.k_route, a.v_route, a.route_cu, a.route_rows, a.workspace, 0, a.hist};
    t.k_cache = a.k_cache; t.v_cache = a.v_cache; t.pool_tokens = a.pool_tokens; t.route_idx = a.route_idx;
    return rc_launch_attn_tc(ctx, t, st);
  }
  AttnRowsArgs r{a.q, a.o, a.out_dtype, a.cu_q, a.n_req, a.total_q, a.pos0, a.conv_slot, a.k_conv, a.v_conv,
                 a.conv_rows, a.k_route, a.v_route, a.route_cu, 0, a.hist};
  r.route_rows = a.route_rows;
  return rc_launch_attn_rows(ctx, r, st);
}

cudaError_t rc_launch_decode(const recache_ctx* ctx, const DecodeArgs& a, cudaStream_t st) {
  if (rc_decode_split_supported(ctx)) return rc_launch_decode_split(ctx, a, st);
  return rc_launch_decode_rows(ctx, a, st);
}
