// Tensor-core attention for encode and prefill (bf16, head_dim 128, Hq/G in {2,4,8}).
//
// One CTA owns one work item = (sequence, KV group, pair of query tiles).  A
// query tile is 128 rows = (128 / s) consecutive tokens x the s query heads of
// the group, so every K/V tile is shared by all heads of the group and the
// causal granularity is 128 / s tokens.  The two tiles of a CTA are consecutive
// and share each K/V tile, read once from L2/HBM by TMA.
//
//   warps 0-3  softmax of tile A      warps 4-7  softmax of tile B
//   warp  8    TMA producer           warp  9    tcgen05.mma issuer (+ TMEM alloc)
//   warps 10-11 idle: they complete the third warpgroup so that setmaxnreg can
//   move registers from it to the two softmax warpgroups (128 scores per thread).
//
// Tensor memory (512 columns): S_A | S_B | O_A | O_B, 128 fp32 columns each.
// S = Q K^T (both operands in 128B-swizzled shared memory, K-major); the softmax
// warps read S with tcgen05.ld, keep a running maximum with lazy rescaling of O,
// and write P = exp2(.) as bf16 over the first 64 columns of S; O += P V takes P
// from tensor memory and V (MN-major) from shared memory.  While one tile's
// softmax runs, the tensor core works on the other tile.
//
// Key tiles of an item: first the route's packed rows (all visible), then the
// causal rows of the sequence itself up to the tile pair's last token.  The
// query rows are rotated in shared memory after the TMA load (position = pos0 +
// token index) and rounded to bf16, so no rotated copy of Q ever touches HBM.
// Tiles are aligned to the sequence start, never to the batch: a resource gives
// bit-identical outputs whatever else is in the launch.
#include <cuda.h>

#include "common.cuh"

namespace {

constexpr int D = 128;
constexpr int TILE_N = 128;
constexpr int NSTAGE = 2;
constexpr int BOX_BYTES = 16384;   // [128 rows][64 bf16], 128-byte swizzle
constexpr int TILE_BYTES = 32768;  // two boxes: head_dim halves
constexpr int NTHREADS = 384;
constexpr int REGS_SOFTMAX = 224, REGS_AUX = 56;   // 256*224 + 128*56 = 384*168

constexpr int SM_Q = 0;                              // 2 query tiles
constexpr int SM_K = SM_Q + 2 * TILE_BYTES;          // NSTAGE key tiles
constexpr int SM_V = SM_K + NSTAGE * TILE_BYTES;     // NSTAGE value tiles
constexpr int SM_BAR = SM_V + NSTAGE * TILE_BYTES;   // mbarriers
constexpr int SM_MISC = SM_BAR + 32 * 8;             // tmem base, abort flag
constexpr int SM_TOTAL = SM_MISC + 64;
constexpr int SM_ALLOC = SM_TOTAL + 1024;            // slack for 1024-byte alignment

enum { B_QFULL = 0, B_QREADY, B_KFULL, B_KEMPTY = B_KFULL + NSTAGE, B_VFULL = B_KEMPTY + NSTAGE,
       B_VEMPTY = B_VFULL + NSTAGE, B_SFULL = B_VEMPTY + NSTAGE, B_PREADY = B_SFULL + 2, B_ODONE = B_PREADY + 2,
       B_COUNT = B_ODONE + 2 };

constexpr uint32_t COL_S = 0, COL_O = 256;           // + 128 * tile

constexpr long long WAIT_CYCLES = 4000000000ll;      // ~2 s: a wait this long is a bug, not load

struct TcParams {
  const int2* items; const int32_t* n_items;
  const int32_t* cu; const int32_t* pos0; const int32_t* slot; const int32_t* route_cu;
  int n_seq, G, Hq, s;
  int64_t self_rows;
  void* out;
  const float* cos_tab; const float* sin_tab; int max_pos;
  float scale_log2;
  int32_t* status;
};

// ------------------------------------------------------------------ PTX --
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after WAIT_CYCLES (or as soon as another thread of the
// CTA has given up), records the failure in the device status word and lets the
// kernel run to its end so that tensor memory is released.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  if (mbar_try(bar, parity)) return;
  const long long t0 = clock64();
  for (uint32_t it = 0;; ++it) {
    if (mbar_try(bar, parity)) return;
    if ((it & 63) == 63) {
      if (*abort_flag) return;
      if (clock64() - t0 > WAIT_CYCLES) {
        *abort_flag = 1;
        rc_set_status(status, RECACHE_DEV_TIMEOUT);
        return;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
               ::"r"(d), "r"(a), "l"(bdesc), "r"(idesc), "r"(acc) : "memory");
}

#define RC_R32(r, o) "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), \
    "=r"(r[o + 6]), "=r"(r[o + 7]), "=r"(r[o + 8]), "=r"(r[o + 9]), "=r"(r[o + 10]), "=r"(r[o + 11]),               \
    "=r"(r[o + 12]), "=r"(r[o + 13]), "=r"(r[o + 14]), "=r"(r[o + 15]), "=r"(r[o + 16]), "=r"(r[o + 17]),           \
    "=r"(r[o + 18]), "=r"(r[o + 19]), "=r"(r[o + 20]), "=r"(r[o + 21]), "=r"(r[o + 22]), "=r"(r[o + 23]),           \
    "=r"(r[o + 24]), "=r"(r[o + 25]), "=r"(r[o + 26]), "=r"(r[o + 27]), "=r"(r[o + 28]), "=r"(r[o + 29]),           \
    "=r"(r[o + 30]), "=r"(r[o + 31])
#define RC_W32(r, o) "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]),       \
    "r"(r[o + 6]), "r"(r[o + 7]), "r"(r[o + 8]), "r"(r[o + 9]), "r"(r[o + 10]), "r"(r[o + 11]), "r"(r[o + 12]),      \
    "r"(r[o + 13]), "r"(r[o + 14]), "r"(r[o + 15]), "r"(r[o + 16]), "r"(r[o + 17]), "r"(r[o + 18]), "r"(r[o + 19]),  \
    "r"(r[o + 20]), "r"(r[o + 21]), "r"(r[o + 22]), "r"(r[o + 23]), "r"(r[o + 24]), "r"(r[o + 25]), "r"(r[o + 26]),  \
    "r"(r[o + 27]), "r"(r[o + 28]), "r"(r[o + 29]), "r"(r[o + 30]), "r"(r[o + 31])
#define RC_LIST32_OUT "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}"
#define RC_LIST32_IN "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32}"

// 32 consecutive columns of this thread's lane
#define TMEM_LD32(taddr, r, o) \
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 " RC_LIST32_OUT ", [%32];" : RC_R32(r, o) : "r"(taddr) : "memory")
#define TMEM_ST32(taddr, r, o) \
  asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], " RC_LIST32_IN ";" ::"r"(taddr), RC_W32(r, o) : "memory")

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory matrix descriptors, 128-byte swizzle, 8-row groups 1024 bytes apart.
//  K-major operand (rows = M or N index, 64 bf16 of K per 128-byte row): SBO = 1024.
//  MN-major operand (rows = K index, 64 bf16 of N per row): SBO = 1024 between 8-row
//  K groups, LBO = distance between 64-wide N chunks.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32) | (1ull << 46) | (2ull << 61);
}
// kind::f16 instruction descriptor: fp32 accumulate, bf16 A and B, M = 128, N = 128
constexpr uint32_t IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t IDESC_QK = IDESC_BASE;               // A, B K-major
constexpr uint32_t IDESC_PV = IDESC_BASE | (1u << 16);  // B (= V) MN-major

__device__ __forceinline__ void unpack8(const uint4& u, float* f) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { f[2 * i] = __uint_as_float(w[i] << 16); f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}

// ------------------------------------------------------------- work list --
// Items = (sequence, tile-pair index), heaviest causal range first: all
// sequences' last tile pairs, then the ones before, and so on.  One CTA.
__global__ void __launch_bounds__(1024) tile_plan_kernel(const int32_t* __restrict__ cu, int n_seq, int tok_per_cta,
                                                         int n_levels, int32_t* __restrict__ header,
                                                         int2* __restrict__ items, int32_t* __restrict__ level_off,
                                                         int max_items, int32_t* status) {
  for (int l = threadIdx.x; l < n_levels; l += blockDim.x) {
    int cnt = 0;
    for (int b = 0; b < n_seq; ++b) {
      const int len = cu[b + 1] - cu[b];
      if (len < 0) rc_set_status(status, RECACHE_DEV_BAD_SEQLENS);
      const int nt = (len + tok_per_cta - 1) / tok_per_cta;
      if (nt > n_levels) rc_set_status(status, RECACHE_DEV_BAD_SEQLENS);   // longer than the max_len given
      cnt += nt > l;
    }
    level_off[l] = cnt;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    for (int l = n_levels - 1; l >= 0; --l) { const int c = level_off[l]; level_off[l] = run; run += c; }
    header[0] = run < max_items ? run : max_items;
  }
  __syncthreads();
  for (int l = threadIdx.x; l < n_levels; l += blockDim.x) {
    int k = level_off[l];
    for (int b = 0; b < n_seq; ++b) {
      const int nt = (cu[b + 1] - cu[b] + tok_per_cta - 1) / tok_per_cta;
      if (nt > l) { if (k < max_items) items[k] = make_int2(b, l); ++k; }
    }
  }
}

// ---------------------------------------------------------------- kernel --
template <typename TO>
__global__ void __launch_bounds__(NTHREADS, 1) attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                              const __grid_constant__ CUtensorMap tm_ks,
                                                              const __grid_constant__ CUtensorMap tm_vs,
                                                              const __grid_constant__ CUtensorMap tm_kr,
                                                              const __grid_constant__ CUtensorMap tm_vr,
                                                              const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const int item_idx = blockIdx.x / p.G, g = blockIdx.x % p.G;
  if (item_idx >= *p.n_items) return;
  const int2 item = p.items[item_idx];
  const int b = item.x, qt = item.y;
  const int s = p.s, TQ = 128 / s;
  const int seq0 = p.cu[b], L = p.cu[b + 1] - seq0;
  const int tok0 = qt * 2 * TQ;                    // first token of tile A (local index)
  const bool b_valid = tok0 + TQ < L;              // tile B holds at least one real token
  const int kv_end = min(L, tok0 + 2 * TQ);        // causal keys needed by the pair
  const int64_t base = p.slot ? (int64_t)p.slot[b] : (int64_t)seq0;
  const int pos0 = p.pos0 ? p.pos0[b] : 0;
  int rA0 = 0, lenA = 0;
  if (p.route_cu) { rA0 = p.route_cu[b * p.G + g]; lenA = p.route_cu[b * p.G + g + 1] - rA0; }
  if (L <= 0 || tok0 >= L || lenA < 0 || base < 0 || base + L > p.self_rows || seq0 < 0) {
    if (threadIdx.x == 0) rc_set_status(p.status, RECACHE_DEV_BAD_SLOT);
    return;
  }
  const int nA = (lenA + TILE_N - 1) / TILE_N, nB = (kv_end + TILE_N - 1) / TILE_N;
  const int n_tiles = nA + nB;

  const uint32_t sm = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sm_gen = smem_raw + (sm - smem_u32(smem_raw));
  const uint32_t bars = sm + SM_BAR;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm_gen + SM_MISC + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm_gen + SM_MISC);
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bar(B_QFULL), 1);
    mbar_init(bar(B_QREADY), 256);
    for (int i = 0; i < NSTAGE; ++i) {
      mbar_init(bar(B_KFULL + i), 1); mbar_init(bar(B_KEMPTY + i), 1);
      mbar_init(bar(B_VFULL + i), 1); mbar_init(bar(B_VEMPTY + i), 1);
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(bar(B_SFULL + x), 1); mbar_init(bar(B_PREADY + x), 128); mbar_init(bar(B_ODONE + x), 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8 && lane == 0) {
    prefetch_tmap(&tm_q); prefetch_tmap(&tm_ks); prefetch_tmap(&tm_vs);
    if (nA) { prefetch_tmap(&tm_kr); prefetch_tmap(&tm_vr); }
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sm + SM_MISC), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp >= 8) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_AUX));
  if (warp == 8) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      mbar_expect_tx(bar(B_QFULL), 2 * TILE_BYTES);
      for (int x = 0; x < 2; ++x)
        for (int kc = 0; kc < 2; ++kc)
          tma_load_3d(sm + SM_Q + x * TILE_BYTES + kc * BOX_BYTES, &tm_q, bar(B_QFULL), kc * 64, g * s,
                      seq0 + tok0 + x * TQ);
      for (int i = 0; i < n_tiles; ++i) {
        const int st = i % NSTAGE;
        const uint32_t ph = (uint32_t)(i / NSTAGE) & 1u;
        const bool route = i < nA;
        const int row = route ? rA0 + i * TILE_N : (int)((int64_t)g * p.self_rows + base) + (i - nA) * TILE_N;
        mbar_wait(bar(B_KEMPTY + st), ph ^ 1u, abort_flag, p.status);
        mbar_expect_tx(bar(B_KFULL + st), TILE_BYTES);
        for (int kc = 0; kc < 2; ++kc)
          tma_load_2d(sm + SM_K + st * TILE_BYTES + kc * BOX_BYTES, route ? &tm_kr : &tm_ks, bar(B_KFULL + st), kc * 64, row);
        mbar_wait(bar(B_VEMPTY + st), ph ^ 1u, abort_flag, p.status);
        mbar_expect_tx(bar(B_VFULL + st), TILE_BYTES);
        for (int kc = 0; kc < 2; ++kc)
          tma_load_2d(sm + SM_V + st * TILE_BYTES + kc * BOX_BYTES, route ? &tm_vr : &tm_vs, bar(B_VFULL + st), kc * 64, row);
      }
    }
    __syncwarp();
  } else if (warp == 9) {
    // ===================== MMA issuer =====================
    auto issue_qk = [&](int x, int st) {
      const uint32_t qa = sm + SM_Q + x * TILE_BYTES, ka = sm + SM_K + st * TILE_BYTES;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t off = (j >> 2) * BOX_BYTES + (j & 3) * 32;
        mma_ss(tmem + COL_S + 128 * x, smem_desc(qa + off, 16, 1024), smem_desc(ka + off, 16, 1024), IDESC_QK, j > 0);
      }
    };
    auto issue_pv = [&](int x, int st, int ksteps, bool first) {
      const uint32_t va = sm + SM_V + st * TILE_BYTES;
      for (int j = 0; j < ksteps; ++j)
        mma_ts(tmem + COL_O + 128 * x, tmem + COL_S + 128 * x + 8 * j, smem_desc(va + j * 2048, BOX_BYTES, 1024),
               IDESC_PV, (!first || j > 0) ? 1u : 0u);
    };
    mbar_wait(bar(B_QREADY), 0, abort_flag, p.status);
    mbar_wait(bar(B_KFULL + 0), 0, abort_flag, p.status);
    tc_fence_after();
    if (lane == 0) {
      issue_qk(0, 0); tc_commit(bar(B_SFULL + 0));
      if (b_valid) { issue_qk(1, 0); tc_commit(bar(B_SFULL + 1)); }
      tc_commit(bar(B_KEMPTY + 0));
    }
    __syncwarp();
    for (int i = 0; i < n_tiles; ++i) {
      const int st = i % NSTAGE;
      const uint32_t ph = (uint32_t)(i / NSTAGE) & 1u;
      // rows of this tile that really belong to the segment; keys the pair can see
      const int seg_rows = i < nA ? lenA - i * TILE_N : L - (i - nA) * TILE_N;
      const int vis_rows = i < nA ? seg_rows : kv_end - (i - nA) * TILE_N;
      const int ksteps = (min(vis_rows, TILE_N) + 15) >> 4;
      mbar_wait(bar(B_VFULL + st), ph, abort_flag, p.status);
      if (seg_rows < ksteps * 16) {
        // rows past the segment hold whatever follows it in memory: zero them, 0 * NaN would poison O
        uint8_t* vb = sm_gen + SM_V + st * TILE_BYTES;
        const int n_rows = ksteps * 16 - seg_rows;
        for (int e = lane; e < n_rows * 16; e += 32) {
          const int r = seg_rows + (e >> 4), c = e & 15;
          *reinterpret_cast<uint4*>(vb + (c >> 3) * BOX_BYTES + r * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
        }
        fence_async_smem();
      }
      __syncwarp();
      const int st1 = (i + 1) % NSTAGE;
      const uint32_t ph1 = (uint32_t)((i + 1) / NSTAGE) & 1u;
      mbar_wait(bar(B_PREADY + 0), (uint32_t)i & 1u, abort_flag, p.status);
      tc_fence_after();
      if (lane == 0) { issue_pv(0, st, ksteps, i == 0); tc_commit(bar(B_ODONE + 0)); }
      if (i + 1 < n_tiles) {
        mbar_wait(bar(B_KFULL + st1), ph1, abort_flag, p.status);
        tc_fence_after();
        if (lane == 0) { issue_qk(0, st1); tc_commit(bar(B_SFULL + 0)); }
      }
      if (b_valid) {
        mbar_wait(bar(B_PREADY + 1), (uint32_t)i & 1u, abort_flag, p.status);
        tc_fence_after();
        if (lane == 0) { issue_pv(1, st, ksteps, i == 0); tc_commit(bar(B_ODONE + 1)); }
      }
      if (lane == 0) tc_commit(bar(B_VEMPTY + st));
      if (i + 1 < n_tiles && lane == 0) {
        if (b_valid) { issue_qk(1, st1); tc_commit(bar(B_SFULL + 1)); }
        tc_commit(bar(B_KEMPTY + st1));
      }
      __syncwarp();
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX));
    // ===================== softmax warpgroups =====================
    const int x = warp >> 2;                       // tile A or B
    const int row = threadIdx.x & 127;             // row of the tile = TMEM lane
    const uint32_t lane_addr = ((uint32_t)(32 * (warp & 3)) << 16);
    const int t_row = tok0 + x * TQ + row / s;     // token (local index)
    const bool row_valid = t_row < L;
    const int t_eff = min(t_row, L - 1);
    const int head = g * s + row % s;

    // ---- rotate this row of Q in shared memory (swizzled 16-byte chunks) ----
    mbar_wait(bar(B_QFULL), 0, abort_flag, p.status);
    {
      const int pos = min(max(pos0 + t_eff, 0), p.max_pos - 1);
      if (pos0 + t_eff >= p.max_pos) rc_set_status(p.status, RECACHE_DEV_BAD_POS);
      const float* cp = p.cos_tab + (int64_t)pos * 64;
      const float* sp = p.sin_tab + (int64_t)pos * 64;
      uint8_t* qb = sm_gen + SM_Q + x * TILE_BYTES + row * 128;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const int off = ((c ^ (row & 7)) << 4);
        uint4 ulo = *reinterpret_cast<uint4*>(qb + off), uhi = *reinterpret_cast<uint4*>(qb + BOX_BYTES + off);
        float lo[8], hi[8], cs[8], sn[8];
        unpack8(ulo, lo); unpack8(uhi, hi);
        *reinterpret_cast<float4*>(cs) = *reinterpret_cast<const float4*>(cp + 8 * c);
        *reinterpret_cast<float4*>(cs + 4) = *reinterpret_cast<const float4*>(cp + 8 * c + 4);
        *reinterpret_cast<float4*>(sn) = *reinterpret_cast<const float4*>(sp + 8 * c);
        *reinterpret_cast<float4*>(sn + 4) = *reinterpret_cast<const float4*>(sp + 8 * c + 4);
        uint32_t wl[4], wh[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float a0 = __fmaf_rn(lo[2 * i], cs[2 * i], -__fmul_rn(hi[2 * i], sn[2 * i]));
          const float a1 = __fmaf_rn(lo[2 * i + 1], cs[2 * i + 1], -__fmul_rn(hi[2 * i + 1], sn[2 * i + 1]));
          const float b0 = __fmaf_rn(hi[2 * i], cs[2 * i], __fmul_rn(lo[2 * i], sn[2 * i]));
          const float b1 = __fmaf_rn(hi[2 * i + 1], cs[2 * i + 1], __fmul_rn(lo[2 * i + 1], sn[2 * i + 1]));
          wl[i] = pack2(a0, a1); wh[i] = pack2(b0, b1);
        }
        *reinterpret_cast<uint4*>(qb + off) = make_uint4(wl[0], wl[1], wl[2], wl[3]);
        *reinterpret_cast<uint4*>(qb + BOX_BYTES + off) = make_uint4(wh[0], wh[1], wh[2], wh[3]);
      }
      fence_async_smem();
      mbar_arrive(bar(B_QREADY));
    }

    if (x == 0 || b_valid) {
      const uint32_t t_s = tmem + lane_addr + COL_S + 128 * x;
      const uint32_t t_o = tmem + lane_addr + COL_O + 128 * x;
      const float c2 = p.scale_log2;
      float m_ref = -INFINITY, l_sum = 0.f;
      for (int i = 0; i < n_tiles; ++i) {
        mbar_wait(bar(B_SFULL + x), (uint32_t)i & 1u, abort_flag, p.status);
        tc_fence_after();
        uint32_t sr[128];
        TMEM_LD32(t_s + 0, sr, 0); TMEM_LD32(t_s + 32, sr, 32); TMEM_LD32(t_s + 64, sr, 64); TMEM_LD32(t_s + 96, sr, 96);
        tmem_wait_ld();
        // keys this row may see in this tile: columns [0, lim)
        const int lim = i < nA ? lenA - i * TILE_N : t_eff - (i - nA) * TILE_N + 1;
        if (lim < TILE_N) {
#pragma unroll
          for (int c = 0; c < 128; ++c) if (c >= lim) sr[c] = 0xff800000u;   // -inf
        }
        float mx4[4] = {__uint_as_float(sr[0]), __uint_as_float(sr[1]), __uint_as_float(sr[2]), __uint_as_float(sr[3])};
#pragma unroll
        for (int c = 4; c < 128; c += 4) {
#pragma unroll
          for (int u = 0; u < 4; ++u) mx4[u] = fmaxf(mx4[u], __uint_as_float(sr[c + u]));
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        const float m_new = fmaxf(m_ref, mx);
        bool need = false;
        if (i == 0) m_ref = m_new;                       // O is overwritten by the first P V
        else need = (m_new - m_ref) * c2 > 8.f;          // lazy: P stays below 2^8 otherwise
        if (__any_sync(0xffffffffu, need)) {
          mbar_wait(bar(B_ODONE + x), (uint32_t)(i - 1) & 1u, abort_flag, p.status);
          tc_fence_after();
          const float f = need ? ex2((m_ref - m_new) * c2) : 1.f;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            uint32_t orr[32];
            TMEM_LD32(t_o + 32 * ch, orr, 0);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) orr[c] = __float_as_uint(__uint_as_float(orr[c]) * f);
            TMEM_ST32(t_o + 32 * ch, orr, 0);
          }
          tmem_wait_st();
          if (need) { l_sum *= f; m_ref = m_new; }
        }
        const float neg_m = -m_ref * c2;
        uint32_t pr[64];
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int c = 0; c < 64; c += 2) {
          const float p0 = ex2(fmaf(__uint_as_float(sr[2 * c]), c2, neg_m));
          const float p1 = ex2(fmaf(__uint_as_float(sr[2 * c + 1]), c2, neg_m));
          const float p2 = ex2(fmaf(__uint_as_float(sr[2 * c + 2]), c2, neg_m));
          const float p3 = ex2(fmaf(__uint_as_float(sr[2 * c + 3]), c2, neg_m));
          acc[0] += p0; acc[1] += p1; acc[2] += p2; acc[3] += p3;
          pr[c] = pack2(p0, p1);
          pr[c + 1] = pack2(p2, p3);
          if (c == 30) TMEM_ST32(t_s + 0, pr, 0);        // first half of P goes out while the second is computed
        }
        l_sum += (acc[0] + acc[1]) + (acc[2] + acc[3]);
        TMEM_ST32(t_s + 32, pr, 32);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(B_PREADY + x));
      }
      // ---- epilogue: O / l -> global ----
      mbar_wait(bar(B_ODONE + x), (uint32_t)(n_tiles - 1) & 1u, abort_flag, p.status);
      tc_fence_after();
      const float inv = 1.f / l_sum;
      TO* orow = reinterpret_cast<TO*>(p.out) + ((int64_t)(seq0 + t_row) * p.Hq + head) * D;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t orr[32];
        TMEM_LD32(t_o + 32 * ch, orr, 0);
        tmem_wait_ld();
        if (row_valid) {
          if constexpr (sizeof(TO) == 4) {
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              *reinterpret_cast<float4*>(reinterpret_cast<float*>(orow) + 32 * ch + c) =
                  make_float4(__uint_as_float(orr[c]) * inv, __uint_as_float(orr[c + 1]) * inv,
                              __uint_as_float(orr[c + 2]) * inv, __uint_as_float(orr[c + 3]) * inv);
          } else {
#pragma unroll
            for (int c = 0; c < 32; c += 8)
              *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(orow) + 32 * ch + c) =
                  make_uint4(pack2(__uint_as_float(orr[c]) * inv, __uint_as_float(orr[c + 1]) * inv),
                             pack2(__uint_as_float(orr[c + 2]) * inv, __uint_as_float(orr[c + 3]) * inv),
                             pack2(__uint_as_float(orr[c + 4]) * inv, __uint_as_float(orr[c + 5]) * inv),
                             pack2(__uint_as_float(orr[c + 6]) * inv, __uint_as_float(orr[c + 7]) * inv));
          }
        }
      }
    }
  }
  // ---- teardown: every thread is done with tensor memory before it is freed ----
  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

// ------------------------------------------------------------------ host --
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)ptr;
  }
  return fn;
}

// rows x 128 bf16, row-major; box = 128 rows x 64 columns
bool map_rows(CUtensorMap* m, const void* base, uint64_t rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  if (rows == 0) rows = 1;
  cuuint64_t dims[2] = {128, rows};
  cuuint64_t strides[1] = {256};
  cuuint32_t box[2] = {64, 128};
  cuuint32_t es[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// q [tokens][Hq][128]; box = (128/s tokens) x (s heads) x 64 columns -> 128 rows ordered (token, head)
bool map_q(CUtensorMap* m, const void* base, uint64_t tokens, int Hq, int s) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {128, (cuuint64_t)Hq, tokens};
  cuuint64_t strides[2] = {256, (cuuint64_t)Hq * 256};
  cuuint32_t box[3] = {64, (cuuint32_t)s, (cuuint32_t)(128 / s)};
  cuuint32_t es[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int64_t align256(int64_t x) { return (x + 255) & ~(int64_t)255; }

}  // namespace

bool rc_tc_supported(const recache_ctx* ctx) {
  const int s = ctx->desc.n_q_heads / ctx->desc.n_kv_heads;
  return ctx->desc.dtype == RECACHE_BF16 && ctx->desc.head_dim == 128 && (s == 2 || s == 4 || s == 8);
}

static int tc_tok_per_cta(const recache_ctx* ctx) { return 2 * 128 / (ctx->desc.n_q_heads / ctx->desc.n_kv_heads); }
static int64_t tc_max_items(const recache_ctx* ctx, int n_seq, int total) {
  return (int64_t)total / tc_tok_per_cta(ctx) + n_seq;
}
static int tc_levels(const recache_ctx* ctx, int max_len) {
  const int t = tc_tok_per_cta(ctx);
  return (max_len + t - 1) / t + 1;
}

int64_t rc_tc_workspace_bytes(const recache_ctx* ctx, int n_seq, int total, int max_len) {
  return 256 + align256(tc_max_items(ctx, n_seq, total) * 8) + align256((int64_t)tc_levels(ctx, max_len) * 4);
}

cudaError_t rc_launch_attn_tc(const recache_ctx* ctx, const TcAttnArgs& a, cudaStream_t st) {
  const int G = ctx->desc.n_kv_heads, Hq = ctx->desc.n_q_heads, s = Hq / G;
  if (a.total == 0 || a.n_seq == 0) return cudaSuccess;
  const int64_t max_items = tc_max_items(ctx, a.n_seq, a.total);
  const int n_levels = tc_levels(ctx, a.max_len);
  uint8_t* ws = (uint8_t*)a.workspace;
  int32_t* header = (int32_t*)ws;
  int2* items = (int2*)(ws + 256);
  int32_t* level_off = (int32_t*)(ws + 256 + align256(max_items * 8));

  CUtensorMap tq, tks, tvs, tkr, tvr;
  const uint64_t self_total = (uint64_t)G * (uint64_t)a.self_rows;
  if (!map_q(&tq, a.q, (uint64_t)a.total, Hq, s) || !map_rows(&tks, a.k_self, self_total) ||
      !map_rows(&tvs, a.v_self, self_total))
    return cudaErrorInvalidValue;
  const bool has_route = a.route_cu != nullptr && a.route_rows > 0;
  if (!map_rows(&tkr, has_route ? a.k_route : a.k_self, has_route ? (uint64_t)a.route_rows : self_total) ||
      !map_rows(&tvr, has_route ? a.v_route : a.v_self, has_route ? (uint64_t)a.route_rows : self_total))
    return cudaErrorInvalidValue;

  {
    RcLaunchScope scope(ctx, RC_K_TILE_PLAN, st);
    tile_plan_kernel<<<1, 1024, 0, st>>>(a.cu, a.n_seq, tc_tok_per_cta(ctx), n_levels, header, items, level_off,
                                         (int)max_items, ctx->status);
  }
  TcParams p;
  p.items = items; p.n_items = header; p.cu = a.cu; p.pos0 = a.pos0; p.slot = a.slot; p.route_cu = a.route_cu;
  p.n_seq = a.n_seq; p.G = G; p.Hq = Hq; p.s = s; p.self_rows = a.self_rows; p.out = a.o;
  p.cos_tab = ctx->cos_tab; p.sin_tab = ctx->sin_tab; p.max_pos = ctx->desc.max_pos;
  p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)ctx->desc.head_dim));
  p.status = ctx->status;
  const unsigned grid = (unsigned)(max_items * G);
  RcLaunchScope scope(ctx, a.route_cu ? RC_K_PREFILL_ATTN : RC_K_ENCODE_ATTN, st);
  if (a.out_dtype == RECACHE_F32) {
    static bool attr_f = false;
    if (!attr_f) { cudaFuncSetAttribute(attn_tc_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM_ALLOC); attr_f = true; }
    attn_tc_kernel<float><<<grid, NTHREADS, SM_ALLOC, st>>>(tq, tks, tvs, tkr, tvr, p);
  } else {
    static bool attr_b = false;
    if (!attr_b) { cudaFuncSetAttribute(attn_tc_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM_ALLOC); attr_b = true; }
    attn_tc_kernel<__nv_bfloat16><<<grid, NTHREADS, SM_ALLOC, st>>>(tq, tks, tvs, tkr, tvr, p);
  }
  return cudaGetLastError();
}
