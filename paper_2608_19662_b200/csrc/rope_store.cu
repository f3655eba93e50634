// Rotary embedding of keys + head-major store of keys and values.
//
// Encoding: token t of resource i has local position t - cu[i] (plus the
// resource's position offset when one is given) and goes to cache row slot[i] +
// local position (section "Resource-Wise Attention": positions restart inside
// every resource).  Prefill: token t of request b has position
// pos0[b] + (t - cu[b]) and goes to row t of the conversation KV.
// Memory-bound: reads k, v once, writes both once; 16-byte accesses.
#include "common.cuh"

namespace {

template <typename T> struct Vec16;               // 16-byte vector of T
template <> struct Vec16<float> { static constexpr int N = 4; };
template <> struct Vec16<__nv_bfloat16> { static constexpr int N = 8; };

template <typename T>
__device__ __forceinline__ void unpack16(const uint4& u, float* f);
template <> __device__ __forceinline__ void unpack16<float>(const uint4& u, float* f) {
  f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y);
  f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
}
template <> __device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4& u, float* f) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
template <typename T>
__device__ __forceinline__ uint4 pack16(const float* f);
template <> __device__ __forceinline__ uint4 pack16<float>(const float* f) {
  return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
template <> __device__ __forceinline__ uint4 pack16<__nv_bfloat16>(const float* f) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&p);
  }
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// One thread handles one 16-byte chunk of the low half of a key row together
// with the matching chunk of the high half (the rotation pairs i with i + d/2),
// and the two matching chunks of the value row.
template <typename T>
__global__ void __launch_bounds__(256) rope_store_kernel(
    const T* __restrict__ k, const T* __restrict__ v, T* __restrict__ k_dst, T* __restrict__ v_dst,
    const int32_t* __restrict__ cu, int n_seq, int total, const int32_t* __restrict__ slot,
    const int32_t* __restrict__ pos0, const int32_t* __restrict__ hist, int64_t dst_rows, int mode, int G, int d,
    const float* __restrict__ cos_tab, const float* __restrict__ sin_tab, int max_pos,
    int32_t* status) {
  constexpr int N = Vec16<T>::N;
  const int half = d / 2;
  const int chunks = half / N;                  // 16-byte chunks per half row
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t n_work = (int64_t)total * G * chunks;
  if (gid >= n_work) return;
  const int c = (int)(gid % chunks);
  const int g = (int)((gid / chunks) % G);
  const int t = (int)(gid / ((int64_t)chunks * G));

  const int b = rc_find_segment(cu, n_seq, t);
  const int local = t - cu[b];
  // position = the sequence's first position (0 when none is given) + index inside the sequence;
  // row = the sequence's first cache row + that index (encode) or the token index itself (prefill)
  const int pos = (pos0 ? pos0[b] : 0) + local;
  const int64_t row = mode == 0 ? (int64_t)slot[b] + local
                    : mode == 2 ? (int64_t)slot[b] + (hist ? hist[b] : 0) + local : (int64_t)t;
  if (t >= cu[n_seq] || cu[b + 1] < cu[b]) { rc_set_status(status, RECACHE_DEV_BAD_SEQLENS); return; }
  if (row < 0 || row >= dst_rows) { rc_set_status(status, RECACHE_DEV_BAD_SLOT); return; }
  if (pos < 0 || pos >= max_pos) { rc_set_status(status, RECACHE_DEV_BAD_POS); return; }

  const T* ksrc = k + ((int64_t)t * G + g) * d;
  const T* vsrc = v + ((int64_t)t * G + g) * d;
  T* kd = k_dst + ((int64_t)g * dst_rows + row) * d;
  T* vd = v_dst + ((int64_t)g * dst_rows + row) * d;

  float lo[N], hi[N], cs[N], sn[N], olo[N], ohi[N];
  unpack16<T>(*reinterpret_cast<const uint4*>(ksrc + c * N), lo);
  unpack16<T>(*reinterpret_cast<const uint4*>(ksrc + half + c * N), hi);
  const float* cp = cos_tab + (int64_t)pos * half + c * N;
  const float* sp = sin_tab + (int64_t)pos * half + c * N;
#pragma unroll
  for (int i = 0; i < N; i += 4) {
    *reinterpret_cast<float4*>(cs + i) = *reinterpret_cast<const float4*>(cp + i);
    *reinterpret_cast<float4*>(sn + i) = *reinterpret_cast<const float4*>(sp + i);
  }
#pragma unroll
  for (int i = 0; i < N; ++i) {
    // fixed operation order: the stored key depends on (k, position) only
    olo[i] = __fmaf_rn(lo[i], cs[i], -__fmul_rn(hi[i], sn[i]));
    ohi[i] = __fmaf_rn(hi[i], cs[i], __fmul_rn(lo[i], sn[i]));
  }
  *reinterpret_cast<uint4*>(kd + c * N) = pack16<T>(olo);
  *reinterpret_cast<uint4*>(kd + half + c * N) = pack16<T>(ohi);
  *reinterpret_cast<uint4*>(vd + c * N) = *reinterpret_cast<const uint4*>(vsrc + c * N);
  *reinterpret_cast<uint4*>(vd + half + c * N) = *reinterpret_cast<const uint4*>(vsrc + half + c * N);
}

}  // namespace

cudaError_t rc_launch_rope_store(const recache_ctx* ctx, const RopeStoreArgs& a, cudaStream_t st) {
  const int d = ctx->desc.head_dim, G = ctx->desc.n_kv_heads;
  if (a.total == 0) return cudaSuccess;
  const bool bf = ctx->desc.dtype == RECACHE_BF16;
  const int chunks = (d / 2) / (bf ? 8 : 4);
  const int64_t n_work = (int64_t)a.total * G * chunks;
  const int threads = 256;
  const unsigned blocks = (unsigned)((n_work + threads - 1) / threads);
  RcLaunchScope scope(ctx, RC_K_ROPE_STORE, st);
  if (bf)
    rope_store_kernel<__nv_bfloat16><<<blocks, threads, 0, st>>>(
        (const __nv_bfloat16*)a.k, (const __nv_bfloat16*)a.v, (__nv_bfloat16*)a.k_dst, (__nv_bfloat16*)a.v_dst,
        a.cu, a.n_seq, a.total, a.slot, a.pos0, a.hist, a.dst_rows, a.mode, G, d, ctx->cos_tab, ctx->sin_tab,
        ctx->desc.max_pos, ctx->status);
  else
    rope_store_kernel<float><<<blocks, threads, 0, st>>>(
        (const float*)a.k, (const float*)a.v, (float*)a.k_dst, (float*)a.v_dst,
        a.cu, a.n_seq, a.total, a.slot, a.pos0, a.hist, a.dst_rows, a.mode, G, d, ctx->cos_tab, ctx->sin_tab,
        ctx->desc.max_pos, ctx->status);
  return cudaGetLastError();
}
