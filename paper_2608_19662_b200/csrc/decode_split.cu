// Routed split-KV decode for bf16, head_dim 128, 64-token pages: memory-bound.
//
// Persistent kernel, one CTA per SM.  A work unit is (item = sequence x KV group,
// split) = a contiguous range of the item's logical pages (resource pages first,
// then history pages).  Units are dealt round-robin to the CTAs.  Inside a CTA
//   warp 3     : TMA producer.  Walks its units' pages in order and keeps a ring
//                of NSTAGE (K page + V page) buffers full; it runs ahead across
//                unit boundaries, so the HBM stream never drains.
//   warps 0-2  : consumers.  The page at ring position n belongs to warp n % 3
//                and stage n % 6, so a stage is always consumed by the same warp
//                and that warp sees every phase of its stages' barriers in
//                order (a parity wait is only valid one phase ahead).  The s
//                query heads of the group are the first s rows of a 16-row
//                mma.sync tile, so each K/V byte is read once for all heads.
//                Scores: m16n8k16 over ldmatrix fragments of the swizzled K page;
//                online softmax in registers (quad shuffles); O += P V with
//                transposed ldmatrix fragments of the V page.
// The consumer warps' partial (max, sum, O) are merged through shared memory; with
// more than one split the unit's partial goes to the workspace and a second
// small kernel merges the splits.
// Every K/V byte crosses HBM once; the roofline is bytes / HBM bandwidth.
#include <cuda.h>

#include <atomic>

#include "common.cuh"

namespace {

constexpr int D = 128;
constexpr int PT = 64;                 // tokens per page
constexpr int NSTAGE = 6;
constexpr int PAGE_BYTES = PT * D * 2; // 16 KB
constexpr int BOX_BYTES = 8192;        // [64 tokens][64 bf16], 128-byte swizzle
constexpr int STAGE_BYTES = 2 * PAGE_BYTES;
// Gather variant: the resource rows of a chunk come straight from the cache with 16-byte cp.async
// copies (half a warp per 256-byte row) written at the swizzled positions a TMA page load would use,
// so the consumers see one layout.  Four producer warps share a chunk (16 rows each): one warp alone
// cannot issue the 2048 copies of a chunk fast enough.  A full barrier then takes 128 arrivals: every
// producer lane's copies (gathered chunk), or the expect-tx arrival plus 127 plain ones (TMA page).
constexpr int NCW = 3;                 // consumer warps; NSTAGE % NCW == 0
static_assert(NSTAGE % NCW == 0, "a stage must always be consumed by the same warp");
constexpr int NPW_GATHER = 4;           // producer warps of the gather variant (the paged variant has one)
constexpr int NTHREADS = (NCW + 1) * 32;
constexpr int NTHREADS_GATHER = (NCW + NPW_GATHER) * 32;
constexpr int SM_STAGES = 0;
template <bool GATHER> struct Lay {
  static constexpr int STAGE = STAGE_BYTES;
  static constexpr int VOFF = PAGE_BYTES;                               // V half inside a stage
  static constexpr int BAR = NSTAGE * STAGE;                            // full[NSTAGE], empty[NSTAGE]
  static constexpr int Q = BAR + 2 * NSTAGE * 8 + 32;                   // per-warp rotated q: NCW x 8 x 128 bf16
  static constexpr int MERGE = Q + NCW * 8 * D * 2;                     // NCW x 8 x (2 + 128) floats
  static constexpr int MISC = MERGE + NCW * 8 * 130 * 4;
  static constexpr int TOTAL = MISC + 64;
  static constexpr int ALLOC = TOTAL + 1024;
};
static_assert(Lay<true>::ALLOC <= 232448, "shared memory");
constexpr uint32_t WAIT_PROBES = 1u << 21;   // ~2.8 s

struct DecParams {
  const __nv_bfloat16* q; const int32_t* q_pos;
  const int32_t* res_pt; int max_res_pages; const int32_t* res_len;
  const int32_t* hist_pt; int max_hist_pages; const int32_t* hist_len;
  int n_items, n_splits, G, Hq, s;
  int64_t n_pages;
  void* out; float* part_o; float* part_ml;      // partials: [unit][s][128], [unit][s][2]
  const float* cos_tab; const float* sin_tab; int max_pos;
  float scale_log2;
  int32_t* status;
  // gather variant: the resource part of item `it` is rows route_idx[route_cu[it] .. route_cu[it+1]) of the cache
  const __nv_bfloat16* k_cache; const __nv_bfloat16* v_cache; int64_t pool_tokens;
  const int32_t* route_idx; const int32_t* route_cu; int64_t route_rows;   // entries of route_idx
};

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
// Bounded wait: see rc_mbar_wait; this kernel also records where a wait ran out.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  rc_mbar_wait<WAIT_PROBES, RC_WHERE_DECODE_SPLIT>(bar, parity, abort_flag, status);
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)) : "memory");
}
// the barrier gets one (pre-counted) arrival when all earlier cp.async of this thread have landed
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ void mma_bf16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ void bar_consumers() { asm volatile("bar.sync 1, %0;" ::"n"(NCW * 32) : "memory"); }

// Pages of item `it` and the range split `sp` owns.
struct UnitPages { int n_res_pages, n_hist_pages, p0, p1, res_len, hist_len; };
template <bool GATHER>
__device__ __forceinline__ UnitPages unit_pages(const DecParams& p, int it, int sp) {
  UnitPages u;
  if (GATHER) {
    // the item's slice of the index list must lie inside it; otherwise the route is treated as empty
    const int r0 = p.route_cu[it], r1 = p.route_cu[it + 1];
    const bool ok = r0 >= 0 && r1 >= r0 && (int64_t)r1 <= p.route_rows;
    if (!ok) rc_set_status(p.status, RECACHE_DEV_OVERFLOW);
    u.res_len = ok ? r1 - r0 : 0;
  } else {
    u.res_len = max(p.res_len[it], 0);
  }
  u.hist_len = max(p.hist_len[it], 0);
  u.n_res_pages = GATHER ? (u.res_len + PT - 1) / PT : min((u.res_len + PT - 1) / PT, p.max_res_pages);
  u.n_hist_pages = min((u.hist_len + PT - 1) / PT, p.max_hist_pages);
  const int total = u.n_res_pages + u.n_hist_pages;
  u.p0 = (int)((int64_t)total * sp / p.n_splits);
  u.p1 = (int)((int64_t)total * (sp + 1) / p.n_splits);
  return u;
}

template <typename TO, bool GATHER>
__global__ void __launch_bounds__(GATHER ? NTHREADS_GATHER : NTHREADS, 1) decode_split_kernel(const __grid_constant__ CUtensorMap tm_k,
                                                                   const __grid_constant__ CUtensorMap tm_v,
                                                                   const DecParams p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sm = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sm_gen = smem_raw + (sm - smem_u32(smem_raw));
  using L = Lay<GATHER>;
  constexpr int SM_BAR = L::BAR, SM_Q = L::Q, SM_MERGE = L::MERGE, SM_MISC = L::MISC, STAGE = L::STAGE, VOFF = L::VOFF;
  const uint32_t bars = sm + SM_BAR;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm_gen + SM_MISC);
  auto full = [&](int i) { return bars + 8u * (uint32_t)i; };
  auto empty = [&](int i) { return bars + 8u * (uint32_t)(NSTAGE + i); };
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_units = p.n_items * p.n_splits;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int i = 0; i < NSTAGE; ++i) { mbar_init(full(i), GATHER ? 32 * NPW_GATHER : 1); mbar_init(empty(i), 1); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp >= NCW) {
    // ===================== producer(s) =====================
    const int pw = warp - NCW;                         // producer warp index (0 in the paged variant)
    int64_t idx_next = 0;                              // gather variant: row index prefetched for the next chunk
    uint32_t n = 0;   // pages issued so far (ring position)
    for (int unit = blockIdx.x; unit < n_units; unit += gridDim.x) {
      const int it = unit / p.n_splits, sp = unit % p.n_splits;
      const UnitPages u = unit_pages<GATHER>(p, it, sp);
      for (int lp = u.p0; lp < u.p1; ++lp, ++n) {
        const int st = n % NSTAGE;
        const uint32_t dst = sm + SM_STAGES + st * STAGE;
        if (GATHER && lp < u.n_res_pages) {
          // 64 route rows straight from the cache: half a warp copies one 256-byte row, 16 bytes per lane
          const int g = it % p.G;
          const int r0 = p.route_cu[it] + lp * PT;
          const int valid = min(PT, u.res_len - lp * PT);
          constexpr int RPW = PT / NPW_GATHER;                 // rows per producer warp (16)
          // cache row of chunk row pw * 16 + lane (lanes 0..15): fetched one chunk ahead inside a unit
          auto load_idx = [&](int chunk) -> int64_t {
            const int rr = chunk * PT + pw * RPW + lane;
            return (lane < RPW && rr < u.res_len) ? (int64_t)p.route_idx[p.route_cu[it] + rr] : 0;
          };
          int64_t idx_l = (lp == u.p0) ? load_idx(lp) : idx_next;
          if (lp + 1 < u.p1 && lp + 1 < u.n_res_pages) idx_next = load_idx(lp + 1);
          if (idx_l < 0 || idx_l >= p.pool_tokens) {
            rc_set_status(p.status, RECACHE_DEV_BAD_SLOT);
            idx_l = min(max(idx_l, (int64_t)0), p.pool_tokens - 1);
          }
          if (lane == 0) mbar_wait(empty(st), ((n / NSTAGE) & 1u) ^ 1u, abort_flag, p.status);
          __syncwarp();
          const int c = lane & 15;
#pragma unroll
          for (int rr = 0; rr < RPW; rr += 2) {
            const int lrow = rr + (lane >> 4);
            const int row = pw * RPW + lrow;
            const int64_t idx = __shfl_sync(0xffffffffu, idx_l, lrow);
            if (row < valid) {
              const int64_t off = ((int64_t)g * p.pool_tokens + idx) * D + c * 8;
              const uint32_t d0 = dst + (c >> 3) * BOX_BYTES + row * 128 + (((c & 7) ^ (row & 7)) << 4);
              cp_async16(d0, p.k_cache + off);
              cp_async16(d0 + VOFF, p.v_cache + off);
            }
          }
          cp_async_arrive(full(st));
        } else {
          if (lane == 0 && pw == 0) {
            int pg = (!GATHER && lp < u.n_res_pages) ? p.res_pt[(int64_t)it * p.max_res_pages + lp]
                                                     : p.hist_pt[(int64_t)it * p.max_hist_pages + (lp - u.n_res_pages)];
            if (pg < 0 || pg >= p.n_pages) { rc_set_status(p.status, RECACHE_DEV_BAD_PAGE); pg = 0; }
            mbar_wait(empty(st), ((n / NSTAGE) & 1u) ^ 1u, abort_flag, p.status);
            mbar_expect_tx(full(st), STAGE_BYTES);
            tma_load_2d(dst, &tm_k, full(st), 0, pg * PT);
            tma_load_2d(dst + BOX_BYTES, &tm_k, full(st), 64, pg * PT);
            tma_load_2d(dst + VOFF, &tm_v, full(st), 0, pg * PT);
            tma_load_2d(dst + VOFF + BOX_BYTES, &tm_v, full(st), 64, pg * PT);
          }
          if (GATHER) {           // the other 127 of the 128 arrivals a full barrier takes in this variant
            if (lane == 0 && pw != 0) mbar_wait(empty(st), ((n / NSTAGE) & 1u) ^ 1u, abort_flag, p.status);
            __syncwarp();         // (not before this warp has seen the stage released)
            if (lane != 0 || pw != 0) mbar_arrive(full(st));
          }
        }
        __syncwarp();
      }
    }
  } else {
    // ===================== consumers =====================
    const int gq = lane >> 2, tq = lane & 3;           // fragment row (query head) and column pair
    const int s = p.s;
    uint32_t n_base = 0;                                // ring position of the unit's first page
    __nv_bfloat16* q_sm = reinterpret_cast<__nv_bfloat16*>(sm_gen + SM_Q) + warp * 8 * D;
    float* mrg = reinterpret_cast<float*>(sm_gen + SM_MERGE);
    for (int unit = blockIdx.x; unit < n_units; unit += gridDim.x) {
      const int it = unit / p.n_splits, sp = unit % p.n_splits;
      const int b = it / p.G, g = it % p.G;
      const UnitPages u = unit_pages<GATHER>(p, it, sp);
      if (sp == 0 && lane == 0 && warp == 0) {
        if (u.hist_len < 1 || (!GATHER && (u.res_len + PT - 1) / PT > p.max_res_pages) ||
            (u.hist_len + PT - 1) / PT > p.max_hist_pages)
          rc_set_status(p.status, RECACHE_DEV_BAD_PAGE);
      }
      // ---- rotated query heads of the group -> A fragments (rows >= s are zero) ----
      {
        int pos = p.q_pos[b];
        if (pos < 0 || pos >= p.max_pos) { rc_set_status(p.status, RECACHE_DEV_BAD_POS); pos = min(max(pos, 0), p.max_pos - 1); }
        const __nv_bfloat16* qg = p.q + ((int64_t)b * p.Hq + g * s) * D;
        for (int e = lane; e < 8 * 64; e += 32) {
          const int h = e >> 6, i = e & 63;
          float olo = 0.f, ohi = 0.f;
          if (h < s) {
            const float lo = __bfloat162float(qg[h * D + i]), hi = __bfloat162float(qg[h * D + i + 64]);
            const float c = p.cos_tab[(int64_t)pos * 64 + i], sn = p.sin_tab[(int64_t)pos * 64 + i];
            olo = __fmaf_rn(lo, c, -__fmul_rn(hi, sn));
            ohi = __fmaf_rn(hi, c, __fmul_rn(lo, sn));
          }
          q_sm[h * D + i] = __float2bfloat16_rn(olo);
          q_sm[h * D + i + 64] = __float2bfloat16_rn(ohi);
        }
        __syncwarp();
      }
      uint32_t qa[8][2];   // per k-step: a0 (cols 2tq,+1) and a2 (cols 8+2tq,+1) of row gq; rows 8..15 are zero
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        qa[kk][0] = *reinterpret_cast<const uint32_t*>(q_sm + gq * D + kk * 16 + tq * 2);
        qa[kk][1] = *reinterpret_cast<const uint32_t*>(q_sm + gq * D + kk * 16 + 8 + tq * 2);
      }
      __syncwarp();

      float o[16][4];
#pragma unroll
      for (int nt = 0; nt < 16; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
      float m_run = -INFINITY, l_run = 0.f;      // row gq (replicated over the quad), log2 domain

      // first page of the unit whose ring position belongs to this warp
      const int first = (int)(((uint32_t)warp + NCW - n_base % NCW) % NCW);
      for (int lp = u.p0 + first; lp < u.p1; lp += NCW) {
        const uint32_t n = n_base + (uint32_t)(lp - u.p0);
        const int st = n % NSTAGE;
        // tokens of this page that exist
        int valid = PT;
        if (lp < u.n_res_pages) valid = min(PT, u.res_len - lp * PT);
        else valid = min(PT, u.hist_len - (lp - u.n_res_pages) * PT);
        mbar_wait(full(st), (n / NSTAGE) & 1u, abort_flag, p.status);
        const uint32_t kb = sm + SM_STAGES + st * STAGE, vb = kb + VOFF;
        if (valid < PT) {
          // slots past the end of the part were never written: clear their values (0 * NaN would poison O)
          uint8_t* vg = sm_gen + SM_STAGES + st * STAGE + VOFF;
          const int v0 = max(valid, 0);
          for (int e = lane; e < (PT - v0) * 16; e += 32) {
            const int r = v0 + (e >> 4), c = e & 15;
            *reinterpret_cast<uint4*>(vg + (c >> 3) * BOX_BYTES + r * 128 + (c & 7) * 16) = make_uint4(0, 0, 0, 0);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // a later TMA load overwrites these bytes
          __syncwarp();
        }
        // ---- S = q K^T : 8 token tiles x 8 k-steps ----
        float sc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
          const int tok = nt * 8 + (lane & 7);
#pragma unroll
          for (int kq = 0; kq < 4; ++kq) {
            const int c = 4 * kq + (lane >> 3);
            const uint32_t addr = kb + (c >> 3) * BOX_BYTES + tok * 128 + (((c & 7) ^ (tok & 7)) << 4);
            uint32_t b0, b1, b2, b3;
            ldsm_x4(addr, b0, b1, b2, b3);
            mma_bf16(sc[nt], qa[2 * kq][0], 0u, qa[2 * kq][1], 0u, b0, b1);
            mma_bf16(sc[nt], qa[2 * kq + 1][0], 0u, qa[2 * kq + 1][1], 0u, b2, b3);
          }
        }
        // ---- online softmax of row gq (columns nt*8 + 2tq, +1) ----
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          const int c0 = nt * 8 + tq * 2;
          sc[nt][0] = c0 < valid ? sc[nt][0] * p.scale_log2 : -INFINITY;
          sc[nt][1] = c0 + 1 < valid ? sc[nt][1] * p.scale_log2 : -INFINITY;
          mx = fmaxf(mx, fmaxf(sc[nt][0], sc[nt][1]));
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run, mx);
        const float m_use = m_new == -INFINITY ? 0.f : m_new;    // a page with no valid token
        const float corr = ex2(m_run - m_use);                   // 0 on the first page
        float ps = 0.f;
        uint32_t pa[4][2];   // P as A fragments: per 16-token k-step, a0 / a2 of row gq
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
          const float p0 = ex2(sc[nt][0] - m_use), p1 = ex2(sc[nt][1] - m_use);
          ps += p0 + p1;
          pa[nt >> 1][nt & 1] = pack2(p0, p1);
        }
        ps += __shfl_xor_sync(0xffffffffu, ps, 1);
        ps += __shfl_xor_sync(0xffffffffu, ps, 2);
        l_run = l_run * corr + ps;
        m_run = m_new;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) { o[nt][0] *= corr; o[nt][1] *= corr; }
        // ---- O += P V : 4 k-steps (16 tokens) x 16 d tiles ----
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const int tok = kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7);
#pragma unroll
          for (int np = 0; np < 8; ++np) {
            const int c = 2 * np + (lane >> 4);
            const uint32_t addr = vb + (c >> 3) * BOX_BYTES + tok * 128 + (((c & 7) ^ (tok & 7)) << 4);
            uint32_t b0, b1, b2, b3;
            ldsm_x4_t(addr, b0, b1, b2, b3);
            mma_bf16(o[2 * np], pa[kk][0], 0u, pa[kk][1], 0u, b0, b1);
            mma_bf16(o[2 * np + 1], pa[kk][0], 0u, pa[kk][1], 0u, b2, b3);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty(st));
      }
      n_base += (uint32_t)(u.p1 - u.p0);

      // ---- merge the consumer warps' partials (rows gq < s) ----
      if (gq < s) {
        float* mine = mrg + (warp * 8 + gq) * 130;
        if (tq == 0) { mine[0] = m_run; mine[1] = l_run; }
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
          mine[2 + nt * 8 + tq * 2] = o[nt][0];
          mine[2 + nt * 8 + tq * 2 + 1] = o[nt][1];
        }
      }
      bar_consumers();
      {
        const int t = threadIdx.x;               // head t/32 (+NCW ...), dims (t%32)*4..+3
        for (int h = t >> 5; h < s; h += NCW) {
          float mw[NCW], M = -INFINITY;
#pragma unroll
          for (int w = 0; w < NCW; ++w) { mw[w] = mrg[(w * 8 + h) * 130]; M = fmaxf(M, mw[w]); }
          float Lsum = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int w = 0; w < NCW; ++w) {
            const float f = mw[w] == -INFINITY ? 0.f : ex2(mw[w] - M);
            Lsum += mrg[(w * 8 + h) * 130 + 1] * f;
            const float* ow = mrg + (w * 8 + h) * 130 + 2 + (t & 31) * 4;
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[c] += ow[c] * f;
          }
          if (p.n_splits == 1) {
            const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
            TO* orow = reinterpret_cast<TO*>(p.out) + ((int64_t)b * p.Hq + g * s + h) * D + (t & 31) * 4;
            if constexpr (sizeof(TO) == 4) {
              *reinterpret_cast<float4*>(orow) = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
            } else {
              *reinterpret_cast<uint2*>(orow) = make_uint2(pack2(acc[0] * inv, acc[1] * inv), pack2(acc[2] * inv, acc[3] * inv));
            }
          } else {
            float* po = p.part_o + ((int64_t)unit * s + h) * D + (t & 31) * 4;
            *reinterpret_cast<float4*>(po) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            if ((t & 31) == 0) { p.part_ml[((int64_t)unit * s + h) * 2] = M; p.part_ml[((int64_t)unit * s + h) * 2 + 1] = Lsum; }
          }
        }
      }
      bar_consumers();
    }
  }
  if (*abort_flag) rc_timeout_drain();   // a wait ran out: let the loads in flight land before the CTA ends
}

// Combines the splits of every (sequence, head): one warp per output row (32 lanes x 4 dims), eight
// rows per CTA.
constexpr int MERGE_ROWS = 8;
template <typename TO>
__global__ void __launch_bounds__(32 * MERGE_ROWS) decode_merge_kernel(const float* __restrict__ part_o,
                                                                       const float* __restrict__ part_ml,
                                                                       TO* __restrict__ out, int n_rows, int n_splits, int G, int Hq, int s) {
  const int row = blockIdx.x * MERGE_ROWS + (threadIdx.x >> 5);   // b * Hq + head
  if (row >= n_rows) return;
  const int b = row / Hq, head = row % Hq, g = head / s, h = head % s;
  const int it = b * G + g;
  const int t = threadIdx.x & 31;
  float M = -INFINITY;
  for (int sp = 0; sp < n_splits; ++sp) M = fmaxf(M, part_ml[((int64_t)(it * n_splits + sp) * s + h) * 2]);
  float L = 0.f, acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int sp = 0; sp < n_splits; ++sp) {
    const int64_t u = ((int64_t)(it * n_splits + sp) * s + h);
    const float mw = part_ml[u * 2];
    const float f = mw == -INFINITY ? 0.f : ex2(mw - M);
    L += part_ml[u * 2 + 1] * f;
    const float4 v = *reinterpret_cast<const float4*>(part_o + u * D + t * 4);
    acc[0] += v.x * f; acc[1] += v.y * f; acc[2] += v.z * f; acc[3] += v.w * f;
  }
  const float inv = L > 0.f ? 1.f / L : 0.f;
  TO* orow = out + (int64_t)row * D + t * 4;
  if constexpr (sizeof(TO) == 4) {
    *reinterpret_cast<float4*>(orow) = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
  } else {
    *reinterpret_cast<uint2*>(orow) = make_uint2(pack2(acc[0] * inv, acc[1] * inv), pack2(acc[2] * inv, acc[3] * inv));
  }
}

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
// page pool viewed as [n_pages * 64 rows][128 bf16]; box = one page x 64 columns
bool map_pages(CUtensorMap* m, const void* base, uint64_t n_pages) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {128, n_pages * PT};
  cuuint64_t strides[1] = {256};
  cuuint32_t box[2] = {64, PT};
  cuuint32_t es[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int64_t align256(int64_t x) { return (x + 255) & ~(int64_t)255; }

}  // namespace

bool rc_decode_split_supported(const recache_ctx* ctx) {
  const int s = ctx->desc.n_q_heads / ctx->desc.n_kv_heads;
  return ctx->desc.dtype == RECACHE_BF16 && ctx->desc.head_dim == 128 && ctx->desc.page_tokens == PT && s <= 8;
}

// Splits per item: the smallest count that fills the persistent grid evenly
// (units / SMs close to an integer from below) while a split keeps >= 4 pages.
int rc_decode_n_splits(const recache_ctx* ctx, int batch, int max_res_pages, int max_hist_pages) {
  const int items = batch * ctx->desc.n_kv_heads, sms = ctx->sm_count > 0 ? ctx->sm_count : 148;
  const int pages = max_res_pages + max_hist_pages;
  int best = 1; double best_eff = 0.0;
  for (int ns = 1; ns <= 16; ++ns) {
    if (ns > 1 && pages / ns < 4) break;
    const int units = items * ns;
    const double eff = (double)units / ((double)((units + sms - 1) / sms) * sms);
    if (eff > best_eff + 0.02) { best_eff = eff; best = ns; }
  }
  return best;
}

int64_t rc_decode_split_workspace_bytes(const recache_ctx* ctx, int batch, int max_res_pages, int max_hist_pages) {
  const int ns = rc_decode_n_splits(ctx, batch, max_res_pages, max_hist_pages);
  const int s = ctx->desc.n_q_heads / ctx->desc.n_kv_heads;
  const int64_t units = (int64_t)batch * ctx->desc.n_kv_heads * ns;
  return align256(units * s * D * 4) + align256(units * s * 2 * 4);
}

cudaError_t rc_launch_decode_split(const recache_ctx* ctx, const DecodeArgs& a, cudaStream_t st) {
  const int G = ctx->desc.n_kv_heads, Hq = ctx->desc.n_q_heads, s = Hq / G;
  const int ns = rc_decode_n_splits(ctx, a.batch, a.max_res_pages, a.max_hist_pages);
  const int64_t units = (int64_t)a.batch * G * ns;
  if ((uint64_t)a.n_pages * PT > 0x7fffffffull) return cudaErrorInvalidValue;   // TMA coordinates are 32-bit row indices
  CUtensorMap tk, tv;
  if (!map_pages(&tk, a.k_pages, (uint64_t)a.n_pages) || !map_pages(&tv, a.v_pages, (uint64_t)a.n_pages))
    return cudaErrorInvalidValue;
  DecParams p;
  p.q = (const __nv_bfloat16*)a.q; p.q_pos = a.q_pos;
  p.res_pt = a.res_pt; p.max_res_pages = a.max_res_pages; p.res_len = a.res_len;
  p.hist_pt = a.hist_pt; p.max_hist_pages = a.max_hist_pages; p.hist_len = a.hist_len;
  p.n_items = a.batch * G; p.n_splits = ns; p.G = G; p.Hq = Hq; p.s = s; p.n_pages = a.n_pages;
  p.out = a.o;
  p.part_o = (float*)a.workspace;
  p.part_ml = (float*)((uint8_t*)a.workspace + align256(units * s * D * 4));
  p.cos_tab = ctx->cos_tab; p.sin_tab = ctx->sin_tab; p.max_pos = ctx->desc.max_pos;
  p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)D));
  p.status = ctx->status;
  p.k_cache = (const __nv_bfloat16*)a.k_cache; p.v_cache = (const __nv_bfloat16*)a.v_cache;
  p.pool_tokens = a.pool_tokens; p.route_idx = a.route_idx; p.route_cu = a.route_cu; p.route_rows = a.route_rows;
  const int sms = ctx->sm_count > 0 ? ctx->sm_count : 148;
  const unsigned grid = (unsigned)(units < sms ? units : sms);
  const bool f32 = a.out_dtype == RECACHE_F32, gather = a.route_idx != nullptr;
  {
    RcLaunchScope scope(ctx, RC_K_DECODE_ATTN, st);
    auto launch = [&](auto kernel, int smem) {
      cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      kernel<<<grid, gather ? NTHREADS_GATHER : NTHREADS, smem, st>>>(tk, tv, p);
    };
    if (gather) {
      if (f32) launch(decode_split_kernel<float, true>, Lay<true>::ALLOC);
      else launch(decode_split_kernel<__nv_bfloat16, true>, Lay<true>::ALLOC);
    } else {
      if (f32) launch(decode_split_kernel<float, false>, Lay<false>::ALLOC);
      else launch(decode_split_kernel<__nv_bfloat16, false>, Lay<false>::ALLOC);
    }
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || ns == 1) return e;
  RcLaunchScope scope(ctx, RC_K_DECODE_MERGE, st);
  const int n_rows = a.batch * Hq, blocks = (n_rows + MERGE_ROWS - 1) / MERGE_ROWS;
  if (f32) decode_merge_kernel<float><<<blocks, 32 * MERGE_ROWS, 0, st>>>(p.part_o, p.part_ml, (float*)a.o, n_rows, ns, G, Hq, s);
  else decode_merge_kernel<__nv_bfloat16><<<blocks, 32 * MERGE_ROWS, 0, st>>>(p.part_o, p.part_ml, (__nv_bfloat16*)a.o, n_rows, ns, G, Hq, s);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// Allocation-free decode.
//
// recache_attend_decode needs a scratch buffer for the split partials, which the
// caller normally gets from its allocator.  Some callers cannot allocate at the
// point where they decode: code running inside a region where the CUDA allocator
// must not be touched (a serving loop that has pinned down its memory plan, a
// plugin loaded into a host process that owns all device memory, a signal-safe
// or real-time path).  For them the scratch lives in this file-scope device
// array, reserved by every GPU that loads the library until the process exits.
// ---------------------------------------------------------------------------
namespace {

constexpr int64_t NOALLOC_SCRATCH_BYTES = 4ll << 20;   // 4 MiB per device
static __device__ __align__(256) unsigned char g_decode_scratch[NOALLOC_SCRATCH_BYTES];

constexpr int NOALLOC_MAX_DEVICES = 64;
// Device address of g_decode_scratch, per device.  Host threads may make the first call on a
// device at the same time: each looks the address up and stores the same value, through an atomic
// so that the concurrent store and load are well defined.
std::atomic<void*> g_scratch_addr[NOALLOC_MAX_DEVICES];

}  // namespace

extern "C" RECACHE_API recache_status recache_attend_decode_noalloc(
    recache_ctx* ctx, const void* q, const int32_t* q_pos, int32_t batch, const void* k_new, const void* v_new,
    void* k_pages, void* v_pages, int64_t n_pages, const int32_t* res_page_table, int32_t max_res_pages,
    const int32_t* res_len, const int32_t* hist_page_table, int32_t max_hist_pages, const int32_t* hist_len,
    void* out_o, int32_t out_dtype, void* stream) {
  if (!ctx) return RECACHE_EINVAL;
  auto fail = [&](recache_status st, const char* msg) { ctx->err = msg; return st; };
  if (batch < 0 || n_pages < 0 || max_res_pages < 0 || max_hist_pages <= 0)
    return fail(RECACHE_EINVAL, "decode_noalloc: bad size");
  if (out_dtype != RECACHE_F32 && out_dtype != ctx->desc.dtype)
    return fail(RECACHE_EINVAL, "decode_noalloc: out_dtype must be f32 or the context dtype");
  if (batch == 0) return RECACHE_OK;
  if (!q || !q_pos || !k_pages || !v_pages || !res_len || !hist_page_table || !hist_len || !out_o ||
      (max_res_pages > 0 && !res_page_table) || ((k_new == nullptr) != (v_new == nullptr)))
    return fail(RECACHE_EINVAL, "decode_noalloc: null pointer");
  if (((uintptr_t)q | (uintptr_t)k_pages | (uintptr_t)v_pages | (uintptr_t)out_o) & 15)
    return fail(RECACHE_EINVAL, "decode_noalloc: tensors must be 16-byte aligned");
  if (!rc_decode_split_supported(ctx))
    return fail(RECACHE_EUNSUPPORTED, "decode_noalloc: needs a bf16 context with head_dim 128 and 64-token pages");
  if (ctx->timer_on)
    return fail(RECACHE_EINVAL, "decode_noalloc: the kernel timer creates event objects; disable it first");
  const int64_t need = rc_decode_split_workspace_bytes(ctx, batch, max_res_pages, max_hist_pages);
  if (need > NOALLOC_SCRATCH_BYTES)
    return fail(RECACHE_ENOMEM, "decode_noalloc: batch x groups x splits exceeds the 4 MiB built-in scratch; "
                                "use recache_attend_decode with a caller workspace");
  if (ctx->device < 0 || ctx->device >= NOALLOC_MAX_DEVICES)
    return fail(RECACHE_EUNSUPPORTED, "decode_noalloc: device index out of range");
  if (cudaSetDevice(ctx->device) != cudaSuccess) return fail(RECACHE_ECUDA, "decode_noalloc: set device");
  // In host code the array's name is only a handle; the kernel needs its device
  // address, looked up once per device with that device current.
  void* scratch = g_scratch_addr[ctx->device].load(std::memory_order_relaxed);
  if (!scratch) {
    cudaError_t e = cudaGetSymbolAddress(&scratch, g_decode_scratch);
    if (e != cudaSuccess || !scratch) {
      ctx->err = std::string("decode_noalloc: cudaGetSymbolAddress: ") + cudaGetErrorString(e);
      return RECACHE_ECUDA;
    }
    g_scratch_addr[ctx->device].store(scratch, std::memory_order_relaxed);
  }
  cudaStream_t st = (cudaStream_t)stream;
  DecodeArgs a{q, q_pos, batch, k_new, v_new, k_pages, v_pages, n_pages, res_page_table, max_res_pages, res_len,
               hist_page_table, max_hist_pages, hist_len, out_o, out_dtype, scratch, NOALLOC_SCRATCH_BYTES};
  cudaError_t e = cudaSuccess;
  if (k_new) e = rc_launch_decode_append(ctx, a, st);
  if (e == cudaSuccess) e = rc_launch_decode_split(ctx, a, st);
  if (e != cudaSuccess) {
    ctx->err = std::string("decode_noalloc: launch: ") + cudaGetErrorString(e);
    return RECACHE_ECUDA;
  }
  return RECACHE_OK;
}
