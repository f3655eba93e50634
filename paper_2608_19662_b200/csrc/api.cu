// C ABI of librecache.so: context management, host-side validation, dispatch.
#include <cmath>
#include <cstdio>
#include <vector>

#include "common.cuh"

namespace {

recache_status fail(recache_ctx* ctx, recache_status st, const char* what) {
  if (ctx) ctx->err = what;
  return st;
}
recache_status cuda_fail(recache_ctx* ctx, cudaError_t e, const char* where) {
  if (ctx) ctx->err = std::string(where) + ": " + cudaGetErrorString(e);
  return RECACHE_ECUDA;
}
bool dtype_ok(int dt) { return dt == RECACHE_F32 || dt == RECACHE_BF16; }
bool out_dtype_ok(const recache_ctx* ctx, int out_dtype) {
  return out_dtype == RECACHE_F32 || out_dtype == ctx->desc.dtype;
}
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

void clear_timer(recache_ctx* ctx) {
  for (auto& t : ctx->timed) { cudaEventDestroy(t.start); cudaEventDestroy(t.stop); }
  ctx->timed.clear();
  for (int i = 0; i < RC_K_COUNT; ++i) ctx->launches[i] = 0;
}

#define RC_REQUIRE(cond, st, msg) do { if (!(cond)) return fail(ctx, st, msg); } while (0)
#define RC_CUDA(expr, where) do { cudaError_t e_ = (expr); if (e_ != cudaSuccess) return cuda_fail(ctx, e_, where); } while (0)

}  // namespace

extern "C" {

recache_status recache_create(recache_ctx** out, const recache_desc* desc, int device) {
  if (!out || !desc) return RECACHE_EINVAL;
  *out = nullptr;
  if (!dtype_ok(desc->dtype) || desc->max_pos <= 0 || desc->page_tokens <= 0 || !(desc->rope_theta > 0.0))
    return RECACHE_EINVAL;
  if (desc->n_q_heads <= 0 || desc->n_kv_heads <= 0 || desc->n_q_heads % desc->n_kv_heads != 0 ||
      desc->n_q_heads / desc->n_kv_heads > 8)
    return RECACHE_ESHAPE;
  if (desc->head_dim != 64 && desc->head_dim != 128) return RECACHE_ESHAPE;
  if (cudaSetDevice(device) != cudaSuccess) return RECACHE_ECUDA;
  recache_ctx* ctx = new recache_ctx();
  ctx->desc = *desc;
  ctx->device = device;
  ctx->cos_tab = ctx->sin_tab = nullptr;
  ctx->status = nullptr;
  cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device);

  const int half = desc->head_dim / 2;
  const size_t n = (size_t)desc->max_pos * half;
  std::vector<float> c(n), s(n);
  std::vector<double> inv(half);
  for (int i = 0; i < half; ++i) inv[i] = std::pow(desc->rope_theta, -2.0 * i / desc->head_dim);
  for (int p = 0; p < desc->max_pos; ++p)
    for (int i = 0; i < half; ++i) {
      const double a = (double)p * inv[i];
      c[(size_t)p * half + i] = (float)std::cos(a);
      s[(size_t)p * half + i] = (float)std::sin(a);
    }
  bool ok = cudaMalloc(&ctx->cos_tab, n * sizeof(float)) == cudaSuccess &&
            cudaMalloc(&ctx->sin_tab, n * sizeof(float)) == cudaSuccess &&
            cudaMalloc(&ctx->status, 256) == cudaSuccess &&
            cudaMemcpy(ctx->cos_tab, c.data(), n * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess &&
            cudaMemcpy(ctx->sin_tab, s.data(), n * sizeof(float), cudaMemcpyHostToDevice) == cudaSuccess &&
            cudaMemset(ctx->status, 0, 256) == cudaSuccess &&
            cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    recache_destroy(ctx);
    return RECACHE_ENOMEM;
  }
  *out = ctx;
  return RECACHE_OK;
}

void recache_destroy(recache_ctx* ctx) {
  if (!ctx) return;
  cudaFree(ctx->cos_tab);
  cudaFree(ctx->sin_tab);
  cudaFree(ctx->status);
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
  if (ctx->side) cudaStreamDestroy(ctx->side);
  clear_timer(ctx);
  delete ctx;
}

const char* recache_last_error(const recache_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

recache_status recache_poll_status(recache_ctx* ctx, void* stream, int32_t* device_code) {
  if (!ctx || !device_code) return RECACHE_EINVAL;
  cudaStream_t st = (cudaStream_t)stream;
  int32_t code[2] = {0, 0};   // the code, and where a wait ran out
  RC_CUDA(cudaMemcpyAsync(code, ctx->status, sizeof(code), cudaMemcpyDeviceToHost, st), "poll copy");
  RC_CUDA(cudaMemsetAsync(ctx->status, 0, sizeof(code), st), "poll clear");
  RC_CUDA(cudaStreamSynchronize(st), "poll sync");
  *device_code = code[0];
  if (code[0] == RECACHE_DEV_TIMEOUT) {
    const uint32_t w = (uint32_t)code[1];
    char msg[160];
    if ((w >> 28) == 2)
      snprintf(msg, sizeof(msg), "a kernel gave up waiting: split-KV decode, block %u, barrier slot %u, warp %u", (w >> 16) & 0xfffu,
               (w >> 8) & 0xffu, w & 0xffu);
    else if ((w >> 28) == 3)
      snprintf(msg, sizeof(msg), "a kernel gave up waiting: wait self-test, block %u, warp %u", (w >> 16) & 0xfffu, w & 0xffu);
    else
      snprintf(msg, sizeof(msg), "a kernel gave up waiting: tensor-core attention (records no location)");
    ctx->err = msg;
  }
  return RECACHE_OK;
}

recache_status recache_selftest_wait_timeout(recache_ctx* ctx, int32_t* report, void* stream) {
  if (!ctx || !report) return RECACHE_EINVAL;
  RC_CUDA(cudaSetDevice(ctx->device), "selftest: set device");
  RC_CUDA(rc_launch_wait_selftest(ctx, report, (cudaStream_t)stream), "selftest launch");
  return RECACHE_OK;
}

static const char* kKernelNames[RC_K_COUNT] = {
    "rope_store", "tile_plan", "encode_attn", "prefill_attn", "compact_count", "compact_plan",
    "compact_gather", "decode_append", "decode_attn", "decode_merge"};

int32_t recache_kernel_count(void) { return RC_K_COUNT; }
const char* recache_kernel_name(int32_t id) { return (id >= 0 && id < RC_K_COUNT) ? kKernelNames[id] : ""; }

recache_status recache_kernel_timer(recache_ctx* ctx, int32_t enable) {
  if (!ctx) return RECACHE_EINVAL;
  clear_timer(ctx);
  ctx->timer_on = enable != 0;
  ctx->timer_attn_only = enable == 2;
  return RECACHE_OK;
}

recache_status recache_kernel_times(recache_ctx* ctx, float* ms_total, int64_t* launches) {
  if (!ctx || !ms_total || !launches) return RECACHE_EINVAL;
  for (int i = 0; i < RC_K_COUNT; ++i) { ms_total[i] = 0.f; launches[i] = ctx->launches[i]; }
  for (auto& t : ctx->timed) {
    RC_CUDA(cudaEventSynchronize(t.stop), "kernel_times: event sync");
    float ms = 0.f;
    RC_CUDA(cudaEventElapsedTime(&ms, t.start, t.stop), "kernel_times: elapsed");
    ms_total[t.id] += ms;
  }
  clear_timer(ctx);
  return RECACHE_OK;
}

int64_t recache_encode_workspace_bytes(const recache_ctx* ctx, int32_t n_resources, int32_t total_tokens,
                                       int32_t max_len) {
  if (!ctx || n_resources < 0 || total_tokens < 0 || max_len < 0) return -1;
  return rc_encode_workspace_bytes(ctx, n_resources, total_tokens, max_len);
}
int64_t recache_compact_workspace_bytes(const recache_ctx* ctx, int32_t n_requests, int32_t total_listed) {
  if (!ctx || n_requests < 0 || total_listed < 0) return -1;
  return rc_compact_workspace_bytes(ctx, n_requests, total_listed);
}
int64_t recache_prefill_workspace_bytes(const recache_ctx* ctx, int32_t n_requests, int32_t total_q, int32_t max_q) {
  if (!ctx || n_requests < 0 || total_q < 0 || max_q < 0) return -1;
  return rc_prefill_workspace_bytes(ctx, n_requests, total_q, max_q);
}
int64_t recache_decode_workspace_bytes(const recache_ctx* ctx, int32_t batch, int32_t max_res_pages,
                                       int32_t max_hist_pages) {
  if (!ctx || batch < 0 || max_res_pages < 0 || max_hist_pages < 0) return -1;
  return rc_decode_workspace_bytes(ctx, batch, max_res_pages, max_hist_pages);
}

static recache_status encode_impl(recache_ctx* ctx, const void* q, const void* k, const void* v,
                                  const int32_t* cu_seqlens, int32_t n_resources, int32_t total_tokens,
                                  int32_t max_len, const int32_t* dst_slot, void* k_cache, void* v_cache,
                                  int64_t pool_tokens, const void* k_prefix, const void* v_prefix,
                                  int32_t prefix_len, const int32_t* pos_offset, void* out_o, int32_t out_dtype,
                                  void* workspace, int64_t workspace_bytes, void* stream) {
  if (!ctx) return RECACHE_EINVAL;
  RC_REQUIRE(prefix_len >= 0, RECACHE_EINVAL, "encode: negative prefix_len");
  RC_REQUIRE(prefix_len == 0 || (k_prefix && v_prefix && aligned16(k_prefix) && aligned16(v_prefix)), RECACHE_EINVAL,
             "encode: prefix tensors missing or not 16-byte aligned");
  RC_REQUIRE(n_resources >= 0 && total_tokens >= 0 && max_len >= 0 && pool_tokens >= 0, RECACHE_EINVAL,
             "encode: negative size");
  RC_REQUIRE(out_dtype_ok(ctx, out_dtype), RECACHE_EINVAL, "encode: out_dtype must be f32 or the context dtype");
  if (n_resources == 0 || total_tokens == 0) return RECACHE_OK;
  RC_REQUIRE(q && k && v && cu_seqlens && dst_slot && k_cache && v_cache && out_o, RECACHE_EINVAL,
             "encode: null pointer");
  RC_REQUIRE(aligned16(q) && aligned16(k) && aligned16(v) && aligned16(k_cache) && aligned16(v_cache) &&
                 aligned16(out_o), RECACHE_EINVAL, "encode: tensors must be 16-byte aligned");
  RC_REQUIRE(max_len <= ctx->desc.max_pos, RECACHE_ESHAPE, "encode: max_len exceeds the rotary table (max_pos)");
  const int64_t need = rc_encode_workspace_bytes(ctx, n_resources, total_tokens, max_len);
  RC_REQUIRE(need == 0 || (workspace && workspace_bytes >= need), RECACHE_ENOMEM, "encode: workspace too small");
  cudaStream_t st = (cudaStream_t)stream;
  RC_CUDA(cudaSetDevice(ctx->device), "encode: set device");

  RopeStoreArgs ra{k, v, k_cache, v_cache, cu_seqlens, n_resources, total_tokens, dst_slot, pos_offset,
                   pool_tokens, 0};
  rc_fork_point(ctx, st);
  RC_CUDA(rc_launch_rope_store(ctx, ra, st), "encode: rope/store launch");
  EncodeArgs ea{q, out_o, out_dtype, cu_seqlens, n_resources, total_tokens, max_len, dst_slot,
                k_cache, v_cache, pool_tokens, workspace, workspace_bytes, k_prefix, v_prefix, prefix_len, pos_offset};
  RC_CUDA(rc_launch_encode_attn(ctx, ea, st), "encode: attention launch");
  return RECACHE_OK;
}

recache_status recache_encode_resources(recache_ctx* ctx, const void* q, const void* k, const void* v,
                                        const int32_t* cu_seqlens, int32_t n_resources, int32_t total_tokens,
                                        int32_t max_len, const int32_t* dst_slot, void* k_cache, void* v_cache,
                                        int64_t pool_tokens, void* out_o, int32_t out_dtype, void* workspace,
                                        int64_t workspace_bytes, void* stream) {
  return encode_impl(ctx, q, k, v, cu_seqlens, n_resources, total_tokens, max_len, dst_slot, k_cache, v_cache,
                     pool_tokens, nullptr, nullptr, 0, nullptr, out_o, out_dtype, workspace, workspace_bytes, stream);
}

recache_status recache_encode_resources_prefixed(recache_ctx* ctx, const void* q, const void* k, const void* v,
                                                 const int32_t* cu_seqlens, int32_t n_resources,
                                                 int32_t total_tokens, int32_t max_len, const int32_t* dst_slot,
                                                 void* k_cache, void* v_cache, int64_t pool_tokens,
                                                 const void* k_prefix, const void* v_prefix, int32_t prefix_len,
                                                 const int32_t* pos_offset, void* out_o, int32_t out_dtype,
                                                 void* workspace, int64_t workspace_bytes, void* stream) {
  return encode_impl(ctx, q, k, v, cu_seqlens, n_resources, total_tokens, max_len, dst_slot, k_cache, v_cache,
                     pool_tokens, k_prefix, v_prefix, prefix_len, pos_offset, out_o, out_dtype, workspace,
                     workspace_bytes, stream);
}

recache_status recache_compact_routes(recache_ctx* ctx, const void* k_cache, const void* v_cache,
                                      int64_t pool_tokens, const uint8_t* keep, const int32_t* res_off,
                                      const int32_t* res_slot, const int32_t* res_len, int32_t n_requests,
                                      int32_t total_listed, const uint8_t* vis, int32_t mode, int32_t* route_cu,
                                      int32_t* route_len, int32_t* route_idx, int64_t row_capacity, void* k_out,
                                      void* v_out, int32_t* page_table, int32_t max_pages_per_route,
                                      const int32_t* free_pages, int64_t n_free_pages, int64_t n_pool_pages,
                                      void* workspace, int64_t workspace_bytes, void* stream) {
  if (!ctx) return RECACHE_EINVAL;
  RC_REQUIRE(n_requests >= 0 && total_listed >= 0 && pool_tokens >= 0 && row_capacity >= 0, RECACHE_EINVAL,
             "compact: negative size");
  RC_REQUIRE(mode == RECACHE_PACKED || mode == RECACHE_PAGED, RECACHE_EINVAL, "compact: bad mode");
  RC_REQUIRE(route_cu && res_off, RECACHE_EINVAL, "compact: null route_cu / res_off");
  if (total_listed > 0) {
    RC_REQUIRE(keep && res_slot && res_len && vis && route_idx, RECACHE_EINVAL, "compact: null pointer");
    RC_REQUIRE((k_out == nullptr) == (v_out == nullptr), RECACHE_EINVAL, "compact: k_out and v_out go together");
    RC_REQUIRE(!k_out || (k_cache && v_cache), RECACHE_EINVAL, "compact: null cache");
    RC_REQUIRE(k_out || mode == RECACHE_PACKED, RECACHE_EINVAL, "compact: index-only compaction is a packed-mode call");
  }
  if (mode == RECACHE_PAGED)
    RC_REQUIRE(page_table && free_pages && max_pages_per_route > 0 && n_free_pages >= 0 && n_pool_pages > 0,
               RECACHE_EINVAL, "compact: paged mode needs page_table, free_pages and pool sizes");
  RC_REQUIRE(aligned16(k_cache) && aligned16(v_cache) && aligned16(k_out) && aligned16(v_out), RECACHE_EINVAL,
             "compact: tensors must be 16-byte aligned");
  const int64_t need = rc_compact_workspace_bytes(ctx, n_requests, total_listed);
  RC_REQUIRE(workspace && workspace_bytes >= need, RECACHE_ENOMEM, "compact: workspace too small");
  cudaStream_t st = (cudaStream_t)stream;
  RC_CUDA(cudaSetDevice(ctx->device), "compact: set device");
  CompactArgs a{k_cache, v_cache, pool_tokens, keep, res_off, res_slot, res_len, n_requests, total_listed,
                vis, mode, route_cu, route_len, route_idx, row_capacity, k_out, v_out, page_table,
                max_pages_per_route, free_pages, n_free_pages, n_pool_pages, workspace};
  RC_CUDA(rc_launch_compact(ctx, a, st), "compact: launch");
  return RECACHE_OK;
}

static recache_status prefill_impl(recache_ctx* ctx, const void* q, const void* k_conv, const void* v_conv,
                                   const int32_t* cu_q, const int32_t* q_pos0, int32_t n_requests, int32_t total_q,
                                   int32_t max_q, const void* k_route, const void* v_route, const int32_t* route_cu,
                                   int64_t route_rows, void* k_conv_out, void* v_conv_out, int64_t conv_rows,
                                   const int32_t* conv_slot, const int32_t* hist_len, void* out_o, int32_t out_dtype,
                                   void* workspace, int64_t workspace_bytes, void* stream,
                                   const void* k_cache = nullptr, const void* v_cache = nullptr,
                                   int64_t pool_tokens = 0, const int32_t* route_idx = nullptr) {
  if (!ctx) return RECACHE_EINVAL;
  RC_REQUIRE(n_requests >= 0 && total_q >= 0 && max_q >= 0 && route_rows >= 0 && conv_rows >= 0, RECACHE_EINVAL,
             "prefill: negative size");
  RC_REQUIRE(out_dtype_ok(ctx, out_dtype), RECACHE_EINVAL, "prefill: out_dtype must be f32 or the context dtype");
  if (n_requests == 0 || total_q == 0) return RECACHE_OK;
  RC_REQUIRE(q && k_conv && v_conv && cu_q && q_pos0 && route_cu && k_conv_out && v_conv_out && out_o,
             RECACHE_EINVAL, "prefill: null pointer");
  RC_REQUIRE(route_rows == 0 || (k_route && v_route) || route_idx, RECACHE_EINVAL, "prefill: null route KV");
  RC_REQUIRE(aligned16(q) && aligned16(k_conv) && aligned16(v_conv) && aligned16(k_route) && aligned16(v_route) &&
                 aligned16(k_conv_out) && aligned16(v_conv_out) && aligned16(out_o), RECACHE_EINVAL,
             "prefill: tensors must be 16-byte aligned");
  const int64_t need = rc_prefill_workspace_bytes(ctx, n_requests, total_q, max_q);
  RC_REQUIRE(need == 0 || (workspace && workspace_bytes >= need), RECACHE_ENOMEM, "prefill: workspace too small");
  cudaStream_t st = (cudaStream_t)stream;
  RC_CUDA(cudaSetDevice(ctx->device), "prefill: set device");

  RopeStoreArgs ra{k_conv, v_conv, k_conv_out, v_conv_out, cu_q, n_requests, total_q, conv_slot, q_pos0,
                   conv_rows, conv_slot ? 2 : 1};
  ra.hist = hist_len;
  rc_fork_point(ctx, st);
  RC_CUDA(rc_launch_rope_store(ctx, ra, st), "prefill: rope/store launch");
  PrefillArgs pa{q, out_o, out_dtype, cu_q, q_pos0, n_requests, total_q, max_q, k_route, v_route, route_cu,
                 route_rows, k_conv_out, v_conv_out, workspace, workspace_bytes, conv_rows, conv_slot, hist_len};
  pa.k_cache = k_cache; pa.v_cache = v_cache; pa.pool_tokens = pool_tokens; pa.route_idx = route_idx;
  RC_CUDA(rc_launch_prefill_attn(ctx, pa, st), "prefill: attention launch");
  return RECACHE_OK;
}

recache_status recache_attend_prefill(recache_ctx* ctx, const void* q, const void* k_conv, const void* v_conv,
                                      const int32_t* cu_q, const int32_t* q_pos0, int32_t n_requests,
                                      int32_t total_q, int32_t max_q, const void* k_route, const void* v_route,
                                      const int32_t* route_cu, int64_t route_rows, void* k_conv_out,
                                      void* v_conv_out, void* out_o, int32_t out_dtype, void* workspace,
                                      int64_t workspace_bytes, void* stream) {
  return prefill_impl(ctx, q, k_conv, v_conv, cu_q, q_pos0, n_requests, total_q, max_q, k_route, v_route, route_cu,
                      route_rows, k_conv_out, v_conv_out, (int64_t)total_q, nullptr, nullptr, out_o, out_dtype,
                      workspace, workspace_bytes, stream);
}

recache_status recache_attend_prefill_history(recache_ctx* ctx, const void* q, const void* k_conv, const void* v_conv,
                                              const int32_t* cu_q, const int32_t* q_pos0, int32_t n_requests,
                                              int32_t total_q, int32_t max_q, const void* k_route,
                                              const void* v_route, const int32_t* route_cu, int64_t route_rows,
                                              void* k_conv_cache, void* v_conv_cache, int64_t cache_rows,
                                              const int32_t* conv_slot, const int32_t* hist_len, void* out_o,
                                              int32_t out_dtype, void* workspace, int64_t workspace_bytes,
                                              void* stream) {
  if (!ctx) return RECACHE_EINVAL;
  RC_REQUIRE(conv_slot && hist_len, RECACHE_EINVAL, "prefill_history: null conv_slot / hist_len");
  return prefill_impl(ctx, q, k_conv, v_conv, cu_q, q_pos0, n_requests, total_q, max_q, k_route, v_route, route_cu,
                      route_rows, k_conv_cache, v_conv_cache, cache_rows, conv_slot, hist_len, out_o, out_dtype,
                      workspace, workspace_bytes, stream);
}

recache_status recache_attend_prefill_gather(recache_ctx* ctx, const void* q, const void* k_conv, const void* v_conv,
                                             const int32_t* cu_q, const int32_t* q_pos0, int32_t n_requests,
                                             int32_t total_q, int32_t max_q, const void* k_cache,
                                             const void* v_cache, int64_t pool_tokens, const int32_t* route_idx,
                                             const int32_t* route_cu, int64_t route_rows, void* k_conv_out,
                                             void* v_conv_out, void* out_o, int32_t out_dtype, void* workspace,
                                             int64_t workspace_bytes, void* stream) {
  if (!ctx) return RECACHE_EINVAL;
  RC_REQUIRE(rc_tc_supported(ctx), RECACHE_EUNSUPPORTED,
             "prefill_gather: needs a bf16 context with head_dim 128 and 2, 4 or 8 query heads per KV head");
  RC_REQUIRE(pool_tokens >= 0 && route_rows >= 0, RECACHE_EINVAL, "prefill_gather: negative size");
  RC_REQUIRE(n_requests == 0 || total_q == 0 || (k_cache && v_cache && route_idx), RECACHE_EINVAL,
             "prefill_gather: null cache / route_idx");
  RC_REQUIRE(aligned16(k_cache) && aligned16(v_cache), RECACHE_EINVAL, "prefill_gather: caches must be 16-byte aligned");
  return prefill_impl(ctx, q, k_conv, v_conv, cu_q, q_pos0, n_requests, total_q, max_q, nullptr, nullptr, route_cu,
                      route_rows, k_conv_out, v_conv_out, (int64_t)total_q, nullptr, nullptr, out_o, out_dtype,
                      workspace, workspace_bytes, stream, k_cache, v_cache, pool_tokens, route_idx);
}

recache_status recache_attend_decode(recache_ctx* ctx, const void* q, const int32_t* q_pos, int32_t batch,
                                     const void* k_new, const void* v_new, void* k_pages, void* v_pages,
                                     int64_t n_pages, const int32_t* res_page_table, int32_t max_res_pages,
                                     const int32_t* res_len, const int32_t* hist_page_table,
                                     int32_t max_hist_pages, const int32_t* hist_len, void* out_o,
                                     int32_t out_dtype, void* workspace, int64_t workspace_bytes, void* stream) {
  if (!ctx) return RECACHE_EINVAL;
  RC_REQUIRE(batch >= 0 && n_pages >= 0 && max_res_pages >= 0 && max_hist_pages > 0, RECACHE_EINVAL,
             "decode: bad size");
  RC_REQUIRE(out_dtype_ok(ctx, out_dtype), RECACHE_EINVAL, "decode: out_dtype must be f32 or the context dtype");
  if (batch == 0) return RECACHE_OK;
  RC_REQUIRE(q && q_pos && k_pages && v_pages && res_len && hist_page_table && hist_len && out_o, RECACHE_EINVAL,
             "decode: null pointer");
  RC_REQUIRE(max_res_pages == 0 || res_page_table, RECACHE_EINVAL, "decode: null resource page table");
  RC_REQUIRE((k_new == nullptr) == (v_new == nullptr), RECACHE_EINVAL, "decode: k_new and v_new go together");
  RC_REQUIRE(aligned16(q) && aligned16(k_pages) && aligned16(v_pages) && aligned16(out_o), RECACHE_EINVAL,
             "decode: tensors must be 16-byte aligned");
  const int64_t need = rc_decode_workspace_bytes(ctx, batch, max_res_pages, max_hist_pages);
  RC_REQUIRE(need == 0 || (workspace && workspace_bytes >= need), RECACHE_ENOMEM, "decode: workspace too small");
  cudaStream_t st = (cudaStream_t)stream;
  RC_CUDA(cudaSetDevice(ctx->device), "decode: set device");
  DecodeArgs a{q, q_pos, batch, k_new, v_new, k_pages, v_pages, n_pages, res_page_table, max_res_pages, res_len,
               hist_page_table, max_hist_pages, hist_len, out_o, out_dtype, workspace, workspace_bytes};
  if (k_new) RC_CUDA(rc_launch_decode_append(ctx, a, st), "decode: append launch");
  RC_CUDA(rc_launch_decode(ctx, a, st), "decode: attention launch");
  return RECACHE_OK;
}

recache_status recache_attend_decode_gather(recache_ctx* ctx, const void* q, const int32_t* q_pos, int32_t batch,
                                            const void* k_new, const void* v_new, const void* k_cache,
                                            const void* v_cache, int64_t pool_tokens, const int32_t* route_idx,
                                            const int32_t* route_cu, int64_t route_rows, int32_t max_res_pages, void* k_pages,
                                            void* v_pages, int64_t n_pages, const int32_t* hist_page_table,
                                            int32_t max_hist_pages, const int32_t* hist_len, void* out_o,
                                            int32_t out_dtype, void* workspace, int64_t workspace_bytes,
                                            void* stream) {
  if (!ctx) return RECACHE_EINVAL;
  RC_REQUIRE(batch >= 0 && n_pages >= 0 && max_res_pages >= 0 && max_hist_pages > 0 && pool_tokens >= 0 && route_rows >= 0,
             RECACHE_EINVAL, "decode_gather: bad size");
  RC_REQUIRE(batch == 0 || pool_tokens > 0, RECACHE_EINVAL, "decode_gather: an index list needs a cache with at least one row");
  RC_REQUIRE(out_dtype_ok(ctx, out_dtype), RECACHE_EINVAL, "decode_gather: out_dtype must be f32 or the context dtype");
  RC_REQUIRE(rc_decode_split_supported(ctx), RECACHE_EUNSUPPORTED,
             "decode_gather: needs a bf16 context with head_dim 128 and 64-token pages");
  if (batch == 0) return RECACHE_OK;
  RC_REQUIRE(q && q_pos && k_cache && v_cache && route_idx && route_cu && k_pages && v_pages && hist_page_table &&
                 hist_len && out_o, RECACHE_EINVAL, "decode_gather: null pointer");
  RC_REQUIRE((k_new == nullptr) == (v_new == nullptr), RECACHE_EINVAL, "decode_gather: k_new and v_new go together");
  RC_REQUIRE(aligned16(q) && aligned16(k_cache) && aligned16(v_cache) && aligned16(k_pages) && aligned16(v_pages) &&
                 aligned16(out_o), RECACHE_EINVAL, "decode_gather: tensors must be 16-byte aligned");
  const int64_t need = rc_decode_workspace_bytes(ctx, batch, max_res_pages, max_hist_pages);
  RC_REQUIRE(need == 0 || (workspace && workspace_bytes >= need), RECACHE_ENOMEM, "decode_gather: workspace too small");
  cudaStream_t st = (cudaStream_t)stream;
  RC_CUDA(cudaSetDevice(ctx->device), "decode_gather: set device");
  DecodeArgs a{q, q_pos, batch, k_new, v_new, k_pages, v_pages, n_pages, nullptr, max_res_pages, nullptr,
               hist_page_table, max_hist_pages, hist_len, out_o, out_dtype, workspace, workspace_bytes};
  a.k_cache = k_cache; a.v_cache = v_cache; a.pool_tokens = pool_tokens; a.route_idx = route_idx; a.route_cu = route_cu;
  a.route_rows = route_rows;
  if (k_new) RC_CUDA(rc_launch_decode_append(ctx, a, st), "decode_gather: append launch");
  RC_CUDA(rc_launch_decode_split(ctx, a, st), "decode_gather: attention launch");
  return RECACHE_OK;
}

}  // extern "C"
