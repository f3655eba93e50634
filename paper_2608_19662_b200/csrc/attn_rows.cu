// Row-per-warp attention in exact fp32 arithmetic (no tensor cores, accurate
// expf): the fp32 path of encode and prefill.  One warp owns one (token, head)
// output row, walks its keys 32 at a time with an online softmax (warp-shuffle
// max / sum) and accumulates d / 32 output columns per lane.
//
// Key set of a row (token t of sequence b at local index j, head h, group g):
//   route part : rows route_cu[b*G+g] .. route_cu[b*G+g+1]-1 of k_route/v_route,
//                all visible (prefill only)
//   self part  : rows base(b) .. base(b)+j of k_self[g]/v_self[g] (causal);
//                base = slot[b] for encoding (cache rows of the resource),
//                cu[b] for prefill (rotated conversation keys).
// The query is rotated on load at position pos0[b] + j (0 + j for encoding).
#include "common.cuh"

namespace {

template <typename T>
__device__ __forceinline__ float dot_row(const T* __restrict__ krow, const float* __restrict__ qs, int d);

template <>
__device__ __forceinline__ float dot_row<float>(const float* __restrict__ krow, const float* __restrict__ qs, int d) {
  float acc = 0.f;
  for (int i = 0; i < d; i += 4) {
    const float4 kv = *reinterpret_cast<const float4*>(krow + i);
    acc = fmaf(kv.x, qs[i], acc); acc = fmaf(kv.y, qs[i + 1], acc);
    acc = fmaf(kv.z, qs[i + 2], acc); acc = fmaf(kv.w, qs[i + 3], acc);
  }
  return acc;
}
template <>
__device__ __forceinline__ float dot_row<__nv_bfloat16>(const __nv_bfloat16* __restrict__ krow,
                                                        const float* __restrict__ qs, int d) {
  float acc = 0.f;
  for (int i = 0; i < d; i += 8) {
    const uint4 u = *reinterpret_cast<const uint4*>(krow + i);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      acc = fmaf(__uint_as_float(w[c] << 16), qs[i + 2 * c], acc);
      acc = fmaf(__uint_as_float(w[c] & 0xffff0000u), qs[i + 2 * c + 1], acc);
    }
  }
  return acc;
}

constexpr int WARPS = 4;

template <typename T, typename TO, int D>
__global__ void __launch_bounds__(WARPS * 32) attn_rows_kernel(
    const T* __restrict__ q, TO* __restrict__ o, const int32_t* __restrict__ cu, int n_seq, int total,
    const int32_t* __restrict__ pos0, const int32_t* __restrict__ slot,
    const T* __restrict__ k_self, const T* __restrict__ v_self, int64_t self_rows,
    const T* __restrict__ k_route, const T* __restrict__ v_route, const int32_t* __restrict__ route_cu,
    int prefix_len, const int32_t* __restrict__ hist, int64_t route_rows, int Hq, int G, const float* __restrict__ cos_tab, const float* __restrict__ sin_tab, int max_pos,
    float scale, int32_t* status) {
  __shared__ float q_s[WARPS][D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * WARPS + warp;
  if (row >= (int64_t)total * Hq) return;
  const int t = (int)(row / Hq), h = (int)(row % Hq);
  const int g = h / (Hq / G);
  const int b = rc_find_segment(cu, n_seq, t);
  const int j = t - cu[b];
  if (t >= cu[n_seq] || j < 0) { if (lane == 0) rc_set_status(status, RECACHE_DEV_BAD_SEQLENS); return; }
  const int pos = (pos0 ? pos0[b] : 0) + j;
  const int64_t base = slot ? (int64_t)slot[b] : (int64_t)cu[b];
  const int H = hist ? hist[b] : 0;      // earlier-turn rows at the start of the self part, all visible
  if (pos < 0 || pos >= max_pos) { if (lane == 0) rc_set_status(status, RECACHE_DEV_BAD_POS); return; }
  if (base < 0 || H < 0 || base + H + j >= self_rows) { if (lane == 0) rc_set_status(status, RECACHE_DEV_BAD_SLOT); return; }

  // rotate the query row into shared memory
  constexpr int HALF = D / 2;
  const T* qrow = q + ((int64_t)t * Hq + h) * D;
  for (int i = lane; i < HALF; i += 32) {
    const float lo = rc_to_float<T>(qrow[i]), hi = rc_to_float<T>(qrow[i + HALF]);
    const float c = cos_tab[(int64_t)pos * HALF + i], s = sin_tab[(int64_t)pos * HALF + i];
    // the rotated query is a tensor of the storage dtype, like the cached keys
    q_s[warp][i] = rc_to_float<T>(rc_from_float<T>(__fmaf_rn(lo, c, -__fmul_rn(hi, s))));
    q_s[warp][i + HALF] = rc_to_float<T>(rc_from_float<T>(__fmaf_rn(hi, c, __fmul_rn(lo, s))));
  }
  __syncwarp();

  constexpr int CPL = D / 32;   // output columns per lane
  float acc[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
  float m = -INFINITY, l = 0.f;

  // two key segments: route rows (all visible), then the causal self rows
  for (int seg = 0; seg < 2; ++seg) {
    const T* kb; const T* vb; int n;
    if (seg == 0) {
      if (!route_cu && prefix_len <= 0) continue;
      // the route's packed rows, or (encoding behind a shared prefix) the group's prefix rows
      const int r0 = route_cu ? route_cu[b * G + g] : g * prefix_len;
      const int r1 = route_cu ? route_cu[b * G + g + 1] : r0 + prefix_len;
      // a range outside the route tensors (e.g. after a compaction that overflowed its capacity)
      // is reported and read as an empty route
      if (r0 < 0 || r1 < r0 || (int64_t)r1 > route_rows) {
        if (lane == 0) rc_set_status(status, RECACHE_DEV_OVERFLOW);
        continue;
      }
      kb = k_route + (int64_t)r0 * D; vb = v_route + (int64_t)r0 * D; n = r1 - r0;
    } else {
      kb = k_self + ((int64_t)g * self_rows + base) * D;
      vb = v_self + ((int64_t)g * self_rows + base) * D;
      n = H + j + 1;
    }
    for (int k0 = 0; k0 < n; k0 += 32) {
      const int kk = k0 + lane;
      float s = -INFINITY;
      if (kk < n) s = dot_row<T>(kb + (int64_t)kk * D, q_s[warp], D) * scale;
      float mx = s;
#pragma unroll
      for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
      const float m_new = fmaxf(m, mx);
      const float corr = (m == -INFINITY) ? 0.f : expf(m - m_new);
      const float p = (kk < n) ? expf(s - m_new) : 0.f;
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
        const T* vrow = vb + (int64_t)(k0 + jj) * D;
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] = fmaf(pj, rc_to_float<T>(vrow[lane + 32 * c]), acc[c]);
      }
    }
  }
  const float inv = 1.f / l;   // the self part always holds the token itself
  TO* orow = o + ((int64_t)t * Hq + h) * D;
#pragma unroll
  for (int c = 0; c < CPL; ++c) orow[lane + 32 * c] = rc_from_float<TO>(acc[c] * inv);
}

template <typename T, typename TO>
cudaError_t launch(const recache_ctx* ctx, const AttnRowsArgs& a, cudaStream_t st) {
  const int d = ctx->desc.head_dim, Hq = ctx->desc.n_q_heads, G = ctx->desc.n_kv_heads;
  const int64_t rows = (int64_t)a.total * Hq;
  if (rows == 0) return cudaSuccess;
  const unsigned blocks = (unsigned)((rows + WARPS - 1) / WARPS);
  const float scale = (float)(1.0 / sqrt((double)d));
  RcLaunchScope scope(ctx, a.route_cu ? RC_K_PREFILL_ATTN : RC_K_ENCODE_ATTN, st);
#define RC_ARGS (const T*)a.q, (TO*)a.o, a.cu, a.n_seq, a.total, a.pos0, a.slot, (const T*)a.k_self, \
    (const T*)a.v_self, a.self_rows, (const T*)a.k_route, (const T*)a.v_route, a.route_cu, a.prefix_len, a.hist, a.route_rows, Hq, G, \
    ctx->cos_tab, ctx->sin_tab, ctx->desc.max_pos, scale, ctx->status
  if (d == 64) attn_rows_kernel<T, TO, 64><<<blocks, WARPS * 32, 0, st>>>(RC_ARGS);
  else         attn_rows_kernel<T, TO, 128><<<blocks, WARPS * 32, 0, st>>>(RC_ARGS);
#undef RC_ARGS
  return cudaGetLastError();
}

}  // namespace

cudaError_t rc_launch_attn_rows(const recache_ctx* ctx, const AttnRowsArgs& a, cudaStream_t st) {
  if (ctx->desc.dtype == RECACHE_F32) return launch<float, float>(ctx, a, st);
  if (a.out_dtype == RECACHE_F32) return launch<__nv_bfloat16, float>(ctx, a, st);
  return launch<__nv_bfloat16, __nv_bfloat16>(ctx, a, st);
}
