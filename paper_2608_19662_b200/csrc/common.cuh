// Internal declarations shared by the translation units of librecache.so.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <string>
#include <vector>

#include "recache.h"

// Kernels of the library, for launch counting and optional per-kernel timing.
enum RcKernel {
  RC_K_ROPE_STORE = 0, RC_K_TILE_PLAN, RC_K_ENCODE_ATTN, RC_K_PREFILL_ATTN,
  RC_K_COMPACT_COUNT, RC_K_COMPACT_PLAN, RC_K_COMPACT_GATHER,
  RC_K_DECODE_APPEND, RC_K_DECODE_ATTN, RC_K_DECODE_MERGE, RC_K_COUNT
};

struct RcTimedLaunch { int id; cudaEvent_t start, stop; };

struct recache_ctx {
  recache_desc desc;
  int device;
  float* cos_tab;     // [max_pos][d/2]
  float* sin_tab;     // [max_pos][d/2]
  int32_t* status;    // device status word
  int sm_count;
  std::string err;
  // A second stream for small set-up kernels that do not depend on the call's first kernel (the work
  // list of the tensor-core attention beside the rotate-and-store pass): forked from and joined to
  // the caller's stream with the two events, so the caller sees one stream's ordering.
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  mutable bool forked = false;   // ev_fork was recorded for the call in progress
  // launch accounting (host side only)
  mutable bool timer_on = false;
  mutable bool timer_attn_only = false;   // bracket the two attention launches only
  mutable int64_t launches[RC_K_COUNT] = {0};
  mutable std::vector<RcTimedLaunch> timed;
};

// Brackets one kernel launch: counts it, and when the timer is enabled records
// a CUDA event pair around it on the launch stream.
struct RcLaunchScope {
  const recache_ctx* ctx; cudaStream_t st; cudaEvent_t stop = nullptr;
  RcLaunchScope(const recache_ctx* c, int id, cudaStream_t s) : ctx(c), st(s) {
    ctx->launches[id]++;
    if (ctx->timer_on && (!ctx->timer_attn_only || id == RC_K_ENCODE_ATTN || id == RC_K_PREFILL_ATTN)) {
      RcTimedLaunch t{id, nullptr, nullptr};
      if (cudaEventCreate(&t.start) == cudaSuccess && cudaEventCreate(&t.stop) == cudaSuccess) {
        cudaEventRecord(t.start, st);
        stop = t.stop;
        ctx->timed.push_back(t);
      }
    }
  }
  ~RcLaunchScope() { if (stop) cudaEventRecord(stop, st); }
};

// Marks the point of the caller's stream that the side stream may start from (everything enqueued
// before the call): record it before the call's first kernel.
// (Not while the timer brackets every kernel: its event pairs are meant for kernels that run alone.)
inline void rc_fork_point(const recache_ctx* ctx, cudaStream_t st) {
  ctx->forked = ctx->side && (!ctx->timer_on || ctx->timer_attn_only) && cudaEventRecord(ctx->ev_fork, st) == cudaSuccess;
}

// First device-side error wins.
__device__ __forceinline__ void rc_set_status(int32_t* status, int32_t code) {
  atomicCAS(status, 0, code);
}
// A bounded wait of the split-KV decode kernel that ran out also says where (second status word, first one wins):
// kernel tag << 28 | (block & 0xfff) << 16 | (barrier's shared address / 8 & 0xff) << 8 | warp.
constexpr uint32_t RC_WHERE_DECODE_SPLIT = 2;
constexpr uint32_t RC_WHERE_SELFTEST = 3;
__device__ __forceinline__ void rc_set_timeout(int32_t* status, uint32_t kernel_tag, uint32_t bar) {
  atomicCAS(status, 0, (int32_t)RECACHE_DEV_TIMEOUT);
  const uint32_t where = kernel_tag << 28 | (blockIdx.x & 0xfffu) << 16 | ((bar >> 3) & 0xffu) << 8 | (threadIdx.x >> 5);
  atomicCAS(status + 1, 0, (int32_t)where);
}

// ---- bounded mbarrier wait, shared by the TMA kernels ----
__device__ __forceinline__ bool rc_mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Gives up after PROBES unsuccessful probes (or as soon as another thread of the CTA has given
// up), records RECACHE_DEV_TIMEOUT in the device status word and returns, so that the kernel runs
// to its end and releases what it holds.  The bound is a probe count, not a clock reading: a probe
// that fails has suspended the thread for about 1.3 us (measured), and the loop then holds no
// 64-bit start time across it (the 32-register warps of the attention kernel are sensitive to every
// register and instruction around their waits).  WHERE_TAG != 0 also records where the wait ran
// out (second status word); the attention kernel passes 0: one more instruction on this cold path
// cost it 6 %.
template <uint32_t PROBES, uint32_t WHERE_TAG>
__device__ __forceinline__ void rc_mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  if (rc_mbar_try(bar, parity)) return;
  for (uint32_t it = 1;; ++it) {
    if (rc_mbar_try(bar, parity)) return;
    if ((it & 1023u) == 0u) {
      if (*abort_flag) return;
      if (it >= PROBES) {
        *abort_flag = 1;
        if constexpr (WHERE_TAG != 0) rc_set_timeout(status, WHERE_TAG, bar);
        else rc_set_status(status, RECACHE_DEV_TIMEOUT);
        return;
      }
    }
  }
}
// After a wait ran out the roles fall through their loops with loads, copies and MMAs possibly
// still in flight.  Let them land (none depends on another CTA; ~100 us is far more than any of
// them takes) before shared and tensor memory go away under them.
__device__ __forceinline__ void rc_timeout_drain() {
  asm volatile("cp.async.wait_all;" ::: "memory");
  const long long t0 = clock64();
  while (clock64() - t0 < 200000ll) { }
}

// Largest i with cu[i] <= x, for cu[0..n] non-decreasing (n >= 1).
__device__ __forceinline__ int rc_find_segment(const int32_t* __restrict__ cu, int n, int x) {
  int lo = 0, hi = n;  // answer in [lo, hi)
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= x) lo = mid; else hi = mid;
  }
  return lo;
}

template <typename T> __device__ __forceinline__ float rc_to_float(T x);
template <> __device__ __forceinline__ float rc_to_float<float>(float x) { return x; }
template <> __device__ __forceinline__ float rc_to_float<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T rc_from_float(float x);
template <> __device__ __forceinline__ float rc_from_float<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 rc_from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// ---- launchers (one per translation unit) -------------------------------
// All return the cudaError_t of the launch (cudaGetLastError).

// Rotates keys at their positions and stores keys/values head-major.
//  mode 0 (encode): token t of resource i -> position pos0[i] + t - cu[i] (pos0 may be null = 0),
//                   row slot[i] + (t - cu[i])
//  mode 1 (prefill): token t of request b -> position pos0[b] + (t - cu[b]), row t
//  mode 2 (prefill into a conversation cache): same position, row slot[b] + hist[b] + (t - cu[b])
struct RopeStoreArgs {
  const void* k; const void* v;       // [total][G][d]
  void* k_dst; void* v_dst;           // [G][dst_rows][d]
  const int32_t* cu; int n_seq; int total;
  const int32_t* slot;                // mode 0, 2
  const int32_t* pos0;                // mode 1, 2; optional in mode 0
  int64_t dst_rows;
  int mode;
  const int32_t* hist = nullptr;      // mode 2: rows already in each sequence's region; new rows follow them
};
cudaError_t rc_launch_rope_store(const recache_ctx* ctx, const RopeStoreArgs& a, cudaStream_t st);

// Generic row-per-warp attention (exact fp32 arithmetic; the fp32 path and the
// small-shape path of bf16).
struct AttnRowsArgs {
  const void* q; void* o; int out_dtype;   // [total][Hq][d]
  const int32_t* cu; int n_seq; int total; // sequences (resources or requests)
  const int32_t* pos0;                     // null: positions start at 0
  const int32_t* slot;                     // causal segment base row per sequence; null: cu[b]
  const void* k_self; const void* v_self;  // [G][self_rows][d] rotated keys / values
  int64_t self_rows;
  const void* k_route; const void* v_route; const int32_t* route_cu;  // null for encode
  int prefix_len;   // > 0 (with route_cu null): every sequence sees rows g*prefix_len .. +prefix_len of k_route/v_route
  const int32_t* hist = nullptr;   // rows that precede each sequence's own tokens in the self part, all visible
  int64_t route_rows = 0;          // rows of k_route / v_route: a route_cu range outside them is reported and skipped
};
cudaError_t rc_launch_attn_rows(const recache_ctx* ctx, const AttnRowsArgs& a, cudaStream_t st);

struct CompactArgs {
  const void* k_cache; const void* v_cache; int64_t pool_tokens;
  const uint8_t* keep;
  const int32_t* res_off; const int32_t* res_slot; const int32_t* res_len;
  int n_requests; int total_listed;
  const uint8_t* vis; int mode;
  int32_t* route_cu; int32_t* route_len; int32_t* route_idx; int64_t row_capacity;
  void* k_out; void* v_out;
  int32_t* page_table; int max_pages_per_route;
  const int32_t* free_pages; int64_t n_free_pages; int64_t n_pool_pages;
  void* workspace;
};
int64_t rc_compact_workspace_bytes(const recache_ctx* ctx, int n_requests, int total_listed);
cudaError_t rc_launch_compact(const recache_ctx* ctx, const CompactArgs& a, cudaStream_t st);

struct DecodeArgs {
  const void* q; const int32_t* q_pos; int batch;
  const void* k_new; const void* v_new;
  void* k_pages; void* v_pages; int64_t n_pages;
  const int32_t* res_pt; int max_res_pages; const int32_t* res_len;
  const int32_t* hist_pt; int max_hist_pages; const int32_t* hist_len;
  void* o; int out_dtype;
  void* workspace; int64_t workspace_bytes;
  // gather variant (route_idx != null): the resource part of item `it` is rows
  // route_idx[route_cu[it] .. route_cu[it+1]) of the cache; res_pt / res_len are unused
  const void* k_cache = nullptr; const void* v_cache = nullptr; int64_t pool_tokens = 0;
  const int32_t* route_idx = nullptr; const int32_t* route_cu = nullptr;
  int64_t route_rows = 0;   // entries of route_idx
};
cudaError_t rc_launch_decode_append(const recache_ctx* ctx, const DecodeArgs& a, cudaStream_t st);
cudaError_t rc_launch_decode_rows(const recache_ctx* ctx, const DecodeArgs& a, cudaStream_t st);

// ---- dispatch between the exact-fp32 kernels and the bf16 tensor-core ones ----
struct EncodeArgs {
  const void* q; void* o; int out_dtype;
  const int32_t* cu; int n_res; int total; int max_len;
  const int32_t* slot; const void* k_cache; const void* v_cache; int64_t pool_tokens;
  void* workspace; int64_t workspace_bytes;
  const void* k_prefix; const void* v_prefix; int prefix_len;   // shared prefix [G][prefix_len][d], or null / 0
  const int32_t* pos_offset;                                      // first position of each resource, or null
};
struct PrefillArgs {
  const void* q; void* o; int out_dtype;
  const int32_t* cu_q; const int32_t* pos0; int n_req; int total_q; int max_q;
  const void* k_route; const void* v_route; const int32_t* route_cu; int64_t route_rows;
  const void* k_conv; const void* v_conv;   // rotated, [G][conv_rows][d]
  void* workspace; int64_t workspace_bytes;
  int64_t conv_rows;                        // rows per group of k_conv / v_conv
  const int32_t* conv_slot = nullptr;       // first row of each request's region (null: cu_q[b])
  const int32_t* hist = nullptr;            // earlier-turn rows at the start of that region (null: 0)
  // gather mode: see TcAttnArgs
  const void* k_cache = nullptr; const void* v_cache = nullptr; int64_t pool_tokens = 0; const int32_t* route_idx = nullptr;
};
int64_t rc_encode_workspace_bytes(const recache_ctx* ctx, int n_res, int total, int max_len);
int64_t rc_prefill_workspace_bytes(const recache_ctx* ctx, int n_req, int total_q, int max_q);
int64_t rc_decode_workspace_bytes(const recache_ctx* ctx, int batch, int max_res_pages, int max_hist_pages);
cudaError_t rc_launch_encode_attn(const recache_ctx* ctx, const EncodeArgs& a, cudaStream_t st);
cudaError_t rc_launch_prefill_attn(const recache_ctx* ctx, const PrefillArgs& a, cudaStream_t st);
cudaError_t rc_launch_decode(const recache_ctx* ctx, const DecodeArgs& a, cudaStream_t st);

// ---- bf16 tensor-core attention (tcgen05 / TMEM / TMA) ----
struct TcAttnArgs {
  const void* q; void* o; int out_dtype;
  const int32_t* cu; int n_seq; int total; int max_len;
  const int32_t* pos0;                     // null: positions start at 0
  const int32_t* slot;                     // null: causal rows start at cu[b]
  const void* k_self; const void* v_self; int64_t self_rows;   // [G][self_rows][128]
  const void* k_route; const void* v_route; const int32_t* route_cu; int64_t route_rows;
  void* workspace;
  int prefix_len;   // > 0 (route_cu null): all sequences see rows g*prefix_len .. of k_route/v_route ([G*prefix_len][128])
  const int32_t* hist = nullptr;   // rows preceding each sequence's own tokens in the self part (earlier turns), all visible
  // gather mode (route_idx != null): route rows are rows route_idx[.] of group g in k_cache / v_cache
  // ([G][pool_tokens][128]); k_route / v_route are unused
  const void* k_cache = nullptr; const void* v_cache = nullptr; int64_t pool_tokens = 0; const int32_t* route_idx = nullptr;
};
bool rc_tc_supported(const recache_ctx* ctx);
int64_t rc_tc_workspace_bytes(const recache_ctx* ctx, int n_seq, int total, int max_len);
cudaError_t rc_launch_attn_tc(const recache_ctx* ctx, const TcAttnArgs& a, cudaStream_t st);

// ---- self-test of the bounded barrier wait (report: 2 ints on the device) ----
cudaError_t rc_launch_wait_selftest(const recache_ctx* ctx, int32_t* report, cudaStream_t st);

// ---- bf16 split-KV paged decode (TMA + mma.sync, persistent) ----
bool rc_decode_split_supported(const recache_ctx* ctx);
int64_t rc_decode_split_workspace_bytes(const recache_ctx* ctx, int batch, int max_res_pages, int max_hist_pages);
cudaError_t rc_launch_decode_split(const recache_ctx* ctx, const DecodeArgs& a, cudaStream_t st);
