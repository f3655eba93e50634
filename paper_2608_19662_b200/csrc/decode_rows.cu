// Routed decode, exact-fp32 path: one warp per (sequence, query head) walks the
// item's paged resource rows and paged history rows with an online softmax.
// Also the append step shared by every decode path: the current token's key is
// rotated at q_pos and stored, with its value, as history row hist_len - 1.
#include "common.cuh"

namespace {

template <typename T>
__global__ void __launch_bounds__(128) decode_append_kernel(
    const T* __restrict__ k_new, const T* __restrict__ v_new, const int32_t* __restrict__ q_pos,
    T* __restrict__ k_pages, T* __restrict__ v_pages, int64_t n_pages,
    const int32_t* __restrict__ hist_pt, int max_hist_pages, const int32_t* __restrict__ hist_len,
    int G, int d, int page_tokens, const float* __restrict__ cos_tab, const float* __restrict__ sin_tab,
    int max_pos, int32_t* status) {
  const int it = blockIdx.x;                 // b * G + g
  const int b = it / G;
  const int n = hist_len[it] - 1;
  const int pos = q_pos[b];
  if (n < 0 || n / page_tokens >= max_hist_pages) { if (threadIdx.x == 0) rc_set_status(status, RECACHE_DEV_BAD_PAGE); return; }
  if (pos < 0 || pos >= max_pos) { if (threadIdx.x == 0) rc_set_status(status, RECACHE_DEV_BAD_POS); return; }
  const int pg = hist_pt[(int64_t)it * max_hist_pages + n / page_tokens];
  if (pg < 0 || pg >= n_pages) { if (threadIdx.x == 0) rc_set_status(status, RECACHE_DEV_BAD_PAGE); return; }
  const int half = d / 2;
  const T* ks = k_new + (int64_t)it * d;
  const T* vs = v_new + (int64_t)it * d;
  T* kd = k_pages + ((int64_t)pg * page_tokens + n % page_tokens) * d;
  T* vd = v_pages + ((int64_t)pg * page_tokens + n % page_tokens) * d;
  for (int i = threadIdx.x; i < half; i += blockDim.x) {
    const float lo = rc_to_float<T>(ks[i]), hi = rc_to_float<T>(ks[i + half]);
    const float c = cos_tab[(int64_t)pos * half + i], s = sin_tab[(int64_t)pos * half + i];
    kd[i] = rc_from_float<T>(__fmaf_rn(lo, c, -__fmul_rn(hi, s)));
    kd[i + half] = rc_from_float<T>(__fmaf_rn(hi, c, __fmul_rn(lo, s)));
    vd[i] = vs[i];
    vd[i + half] = vs[i + half];
  }
}

constexpr int WARPS = 4;

template <typename T, typename TO, int D>
__global__ void __launch_bounds__(WARPS * 32) decode_rows_kernel(
    const T* __restrict__ q, const int32_t* __restrict__ q_pos, int batch,
    const T* __restrict__ k_pages, const T* __restrict__ v_pages, int64_t n_pages,
    const int32_t* __restrict__ res_pt, int max_res_pages, const int32_t* __restrict__ res_len,
    const int32_t* __restrict__ hist_pt, int max_hist_pages, const int32_t* __restrict__ hist_len,
    TO* __restrict__ o, int Hq, int G, int page_tokens, const float* __restrict__ cos_tab,
    const float* __restrict__ sin_tab, int max_pos, float scale, int32_t* status) {
  __shared__ float q_s[WARPS][D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row = blockIdx.x * WARPS + warp;
  if (row >= batch * Hq) return;
  const int b = row / Hq, h = row % Hq, g = h / (Hq / G);
  const int it = b * G + g;
  const int pos = q_pos[b];
  if (pos < 0 || pos >= max_pos) { if (lane == 0) rc_set_status(status, RECACHE_DEV_BAD_POS); return; }
  constexpr int HALF = D / 2;
  const T* qrow = q + (int64_t)row * D;
  for (int i = lane; i < HALF; i += 32) {
    const float lo = rc_to_float<T>(qrow[i]), hi = rc_to_float<T>(qrow[i + HALF]);
    const float c = cos_tab[(int64_t)pos * HALF + i], s = sin_tab[(int64_t)pos * HALF + i];
    // the rotated query is a tensor of the storage dtype, like the cached keys
    q_s[warp][i] = rc_to_float<T>(rc_from_float<T>(__fmaf_rn(lo, c, -__fmul_rn(hi, s))));
    q_s[warp][i + HALF] = rc_to_float<T>(rc_from_float<T>(__fmaf_rn(hi, c, __fmul_rn(lo, s))));
  }
  __syncwarp();
  constexpr int CPL = D / 32;
  float acc[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
  float m = -INFINITY, l = 0.f;
  for (int seg = 0; seg < 2; ++seg) {
    const int32_t* pt = seg == 0 ? res_pt + (int64_t)it * max_res_pages : hist_pt + (int64_t)it * max_hist_pages;
    const int n = seg == 0 ? res_len[it] : hist_len[it];
    const int maxp = seg == 0 ? max_res_pages : max_hist_pages;
    for (int k0 = 0; k0 < n; k0 += 32) {
      const int kk = k0 + lane;
      float s = -INFINITY;
      int64_t my_row = -1;
      if (kk < n) {
        const int pi = kk / page_tokens;
        const int pg = pi < maxp ? pt[pi] : -1;
        if (pg < 0 || pg >= n_pages) rc_set_status(status, RECACHE_DEV_BAD_PAGE);
        else {
          my_row = (int64_t)pg * page_tokens + kk % page_tokens;
          const T* kr = k_pages + my_row * D;
          float a = 0.f;
          for (int i = 0; i < D; ++i) a = fmaf(rc_to_float<T>(kr[i]), q_s[warp][i], a);
          s = a * scale;
        }
      }
      float mx = s;
#pragma unroll
      for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      const float m_new = fmaxf(m, mx);
      if (m_new == -INFINITY) continue;          // nothing readable in this chunk
      const float corr = (m == -INFINITY) ? 0.f : expf(m - m_new);
      const float p = (my_row >= 0) ? expf(s - m_new) : 0.f;
      float ps = p;
#pragma unroll
      for (int off = 16; off; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
      l = l * corr + ps;
      m = m_new;
#pragma unroll
      for (int c = 0; c < CPL; ++c) acc[c] *= corr;
      const int cnt = min(32, n - k0);
      for (int jj = 0; jj < cnt; ++jj) {
        const float pj = __shfl_sync(0xffffffffu, p, jj);
        const int64_t vr = __shfl_sync(0xffffffffu, my_row, jj);
        if (vr < 0) continue;
        const T* vrow = v_pages + vr * D;
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] = fmaf(pj, rc_to_float<T>(vrow[lane + 32 * c]), acc[c]);
      }
    }
  }
  const float inv = l > 0.f ? 1.f / l : 0.f;
  TO* orow = o + (int64_t)row * D;
#pragma unroll
  for (int c = 0; c < CPL; ++c) orow[lane + 32 * c] = rc_from_float<TO>(acc[c] * inv);
}

template <typename T, typename TO>
cudaError_t launch_rows(const recache_ctx* ctx, const DecodeArgs& a, cudaStream_t st) {
  const int d = ctx->desc.head_dim, Hq = ctx->desc.n_q_heads, G = ctx->desc.n_kv_heads;
  const int rows = a.batch * Hq;
  const unsigned blocks = (unsigned)((rows + WARPS - 1) / WARPS);
  const float scale = (float)(1.0 / sqrt((double)d));
  RcLaunchScope scope(ctx, RC_K_DECODE_ATTN, st);
#define RC_ARGS (const T*)a.q, a.q_pos, a.batch, (const T*)a.k_pages, (const T*)a.v_pages, a.n_pages, a.res_pt, \
    a.max_res_pages, a.res_len, a.hist_pt, a.max_hist_pages, a.hist_len, (TO*)a.o, Hq, G,                       \
    ctx->desc.page_tokens, ctx->cos_tab, ctx->sin_tab, ctx->desc.max_pos, scale, ctx->status
  if (d == 64) decode_rows_kernel<T, TO, 64><<<blocks, WARPS * 32, 0, st>>>(RC_ARGS);
  else         decode_rows_kernel<T, TO, 128><<<blocks, WARPS * 32, 0, st>>>(RC_ARGS);
#undef RC_ARGS
  return cudaGetLastError();
}

}  // namespace

cudaError_t rc_launch_decode_append(const recache_ctx* ctx, const DecodeArgs& a, cudaStream_t st) {
  const int d = ctx->desc.head_dim, G = ctx->desc.n_kv_heads;
  RcLaunchScope scope(ctx, RC_K_DECODE_APPEND, st);
  if (ctx->desc.dtype == RECACHE_BF16)
    decode_append_kernel<__nv_bfloat16><<<a.batch * G, 64, 0, st>>>(
        (const __nv_bfloat16*)a.k_new, (const __nv_bfloat16*)a.v_new, a.q_pos, (__nv_bfloat16*)a.k_pages,
        (__nv_bfloat16*)a.v_pages, a.n_pages, a.hist_pt, a.max_hist_pages, a.hist_len, G, d,
        ctx->desc.page_tokens, ctx->cos_tab, ctx->sin_tab, ctx->desc.max_pos, ctx->status);
  else
    decode_append_kernel<float><<<a.batch * G, 64, 0, st>>>(
        (const float*)a.k_new, (const float*)a.v_new, a.q_pos, (float*)a.k_pages, (float*)a.v_pages,
        a.n_pages, a.hist_pt, a.max_hist_pages, a.hist_len, G, d, ctx->desc.page_tokens, ctx->cos_tab,
        ctx->sin_tab, ctx->desc.max_pos, ctx->status);
  return cudaGetLastError();
}

cudaError_t rc_launch_decode_rows(const recache_ctx* ctx, const DecodeArgs& a, cudaStream_t st) {
  if (ctx->desc.dtype == RECACHE_F32) return launch_rows<float, float>(ctx, a, st);
  if (a.out_dtype == RECACHE_F32) return launch_rows<__nv_bfloat16, float>(ctx, a, st);
  return launch_rows<__nv_bfloat16, __nv_bfloat16>(ctx, a, st);
}
