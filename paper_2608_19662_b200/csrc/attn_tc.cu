// Tensor-core attention for encode and prefill (bf16, head_dim 128, Hq/G in {2,4,8}).
//
// Persistent kernel, one CTA per SM; a work item = (sequence, KV group, pair of
// query tiles).  A query tile is 128 rows = (128 / s) consecutive tokens x the s query heads of
// the group, so every K/V tile is shared by all heads of the group and the
// causal granularity is 128 / s tokens.  The two tiles of a CTA are consecutive
// and share each K/V tile, read once from L2/HBM by TMA.
//
//   warps 0-3    softmax of tile A    warps 4-7  softmax of tile B
//   warp  8      TMA producer         warp  9    tcgen05.mma issuer (+ TMEM alloc)
//   warp  10     scheduler: draws work items from a global counter and publishes
//                them through a two-slot ring in shared memory
//   warp  11     idle (completes the third warpgroup)
//   warps 12-15  epilogue: O of a finished tile goes from tensor memory to HBM
//                while the softmax warps already rotate the next item's Q; in
//                gather mode (route rows read from the resource cache through an
//                index list) the same 128 lanes also fill the route's K/V tiles
// setmaxnreg moves registers from warps 8-15 to the two softmax warpgroups,
// which hold 128 scores per thread.
//
// Tensor memory (512 columns): S_A | S_B | O_A | O_B, 128 fp32 columns each.
// S = Q K^T (both operands in 128B-swizzled shared memory, K-major); the softmax
// warps read S with tcgen05.ld, keep a running maximum with lazy rescaling of O,
// and write P = exp2(.) as bf16 over the first 64 columns of S; O += P V takes P
// from tensor memory and V (MN-major) from shared memory, the first 64 keys as
// soon as their half of P is stored.  While one tile's softmax runs, the tensor
// core works on the other tile.
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
constexpr int NTHREADS = 512;
constexpr int REGS_SOFTMAX = 224, REGS_AUX = 32, REGS_EPI = 32;   // 256*224 + 128*(32 + 32) = 65536

constexpr int SM_Q = 0;                              // 2 query tiles
constexpr int SM_K = SM_Q + 2 * TILE_BYTES;          // NSTAGE key tiles
constexpr int SM_V = SM_K + NSTAGE * TILE_BYTES;     // NSTAGE value tiles
constexpr int ROT_BYTES = 16384;                     // cos (and sin) rows of 64 positions, fp32
constexpr int SM_ROT = SM_V + NSTAGE * TILE_BYTES;   // cos | sin of the item's positions
constexpr int SM_BAR = SM_ROT + 2 * ROT_BYTES;       // mbarriers
constexpr int SM_MISC = SM_BAR + 32 * 8;             // tmem base, abort flag
constexpr int SM_ITEM = SM_MISC + 64;                // two published work items
constexpr int SM_INVL = SM_ITEM + 2 * 64;            // 1 / row sum of each query tile's rows, for the epilogue warps
constexpr int SM_TOTAL = SM_INVL + 2 * 128 * 4;
constexpr int SM_ALLOC = SM_TOTAL + 1024;            // slack for 1024-byte alignment

enum { B_QFULL = 0, B_QREADY, B_QEMPTY = B_QREADY + 2, B_KFULL, B_KEMPTY = B_KFULL + NSTAGE, B_VFULL = B_KEMPTY + NSTAGE,
       B_VEMPTY = B_VFULL + NSTAGE, B_SFULL = B_VEMPTY + NSTAGE, B_PREADY = B_SFULL + 2, B_ODONE = B_PREADY + 2,
       B_IFULL = B_ODONE + 2, B_IEMPTY = B_IFULL + 2, B_LREADY = B_IEMPTY + 2, B_ODRAIN = B_LREADY + 2,
       B_PHALF = B_ODRAIN + 2, B_COUNT = B_PHALF + 2 };
static_assert(B_COUNT <= 32, "barrier area");

constexpr uint32_t COL_S = 0, COL_O = 256;           // + 128 * tile

constexpr int SORT_MAX = 4096;                      // work items up to which the plan sorts a prefill by weight (encode: a quarter)

constexpr uint32_t WAIT_PROBES = 1u << 21;           // ~2.8 s of suspended probes: a wait this long is a bug, not load

struct TcParams {
  const int2* items; int32_t* header;   // header[0] = number of items, header[1] = work counter, header[2] = order[] is valid
  const int32_t* order;                 // work indices, heaviest first (launches of at most SORT_MAX work items)
  // gather mode: route row n of group g is row route_idx[n] of gather_k / gather_v ([G][pool_tokens][128] bf16)
  const uint8_t* gather_k; const uint8_t* gather_v; const int32_t* route_idx; int64_t pool_tokens;
  const int32_t* cu; const int32_t* pos0; const int32_t* slot; const int32_t* route_cu; const int32_t* hist;
  int n_seq, G, Hq, s;
  int prefix_len;   // > 0: every sequence sees rows g*prefix_len .. of the "route" tensors (shared prefix)
  int64_t self_rows;
  int64_t route_rows;   // rows of the packed route tensors / entries of route_idx
  void* out;
  const float* cos_tab; const float* sin_tab; int max_pos;
  float scale_log2;
  int32_t* status;
};

// Optional in-kernel timeline (build with -DRC_TRACE; never part of the shipped library): CTA 0
// stamps %clock64 at the hand-overs of its first TR_ITEMS work items, one row of 16 stamps per
// (role, item).  Without the flag the macro is empty.
#ifdef RC_TRACE
constexpr int TR_ITEMS = 192, TR_ROLES = 5;   // roles: softmax A, softmax B, MMA, epilogue, producer
__device__ long long g_trace[TR_ROLES * TR_ITEMS * 16];
#ifndef RC_TRACE_ROLES
#define RC_TRACE_ROLES 31   // bit per role: stamping the 32-register roles disturbs them most
#endif
#define TR(role, item, k) do { if (((RC_TRACE_ROLES >> (role)) & 1) && blockIdx.x == 0 && (item) < (uint32_t)TR_ITEMS) g_trace[((role) * TR_ITEMS + (item)) * 16 + (k)] = clock64(); } while (0)
#define TRV(role, item, k, v) do { if (((RC_TRACE_ROLES >> (role)) & 1) && blockIdx.x == 0 && (item) < (uint32_t)TR_ITEMS) g_trace[((role) * TR_ITEMS + (item)) * 16 + (k)] = (v); } while (0)
#else
#define TR(role, item, k) do {} while (0)
#define TRV(role, item, k, v) do {} while (0)
#endif
// A second, non-intrusive form (-DRC_OBSERVE): the otherwise idle warp 11 of CTA 0 polls the CTA's
// barriers with test_wait and logs (clock, barrier) whenever one completes a phase, so the timeline
// of the hand-overs is seen without a single extra instruction in the working roles.
#ifdef RC_OBSERVE
constexpr int OBS_PER = 2048;                 // events per barrier
__device__ long long g_observe[32 * OBS_PER];   // row 31, entry 0: start time
__device__ int g_observe_n[32];
#endif

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
// Bounded wait: see rc_mbar_wait (no location word here).
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
  rc_mbar_wait<WAIT_PROBES, 0>(bar, parity, abort_flag, status);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros instead
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(src_bytes) : "memory");
}
// one arrival on the barrier once all earlier cp.async of this thread have landed (the barrier's
// expected count already includes it)
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
// plain bulk copy global -> shared (16-byte aligned, size a multiple of 16)
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
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
// D[tmem] (+)= A * B with A in shared memory (mma_ss) or tensor memory (mma_ts); the 64-bit shared
// memory descriptors advance by adds on their address field.
__device__ __forceinline__ void mma_ss(uint32_t d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(d), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d, uint32_t a, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
               ::"r"(d), "r"(a), "l"(db), "r"(idesc), "r"(acc) : "memory");
}
// one lane of a fully converged warp, chosen by the hardware
__device__ __forceinline__ bool elect_one() {
  uint32_t e;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(e));
  return e != 0;
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

#define TMEM_LD16(taddr, r) \
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];" \
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), \
                 "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]) : "r"(taddr) : "memory")

// one 32-byte store (the address is 32-byte aligned)
__device__ __forceinline__ void st_global_v8(void* ptr, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t e, uint32_t f,
                                             uint32_t g, uint32_t h) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(ptr), "r"(a), "r"(b), "r"(c), "r"(d), "r"(e),
               "r"(f), "r"(g), "r"(h) : "memory");
}
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

// Packed fp32 pairs (one instruction, two lanes of the FMA pipe).
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b, float c) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %5};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1) {
  asm("{\n\t.reg .b64 ra, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rd, {%0, %1};\n\tadd.rn.f32x2 rd, rd, ra;\n\t"
      "mov.b64 {%0, %1}, rd;\n\t}"
      : "+f"(d0), "+f"(d1) : "f"(a0), "f"(a1));
}
// d = a * b + c and d = a * b on pairs (one instruction each; same rounding as the scalar forms)
__device__ __forceinline__ void fma2v(float& d0, float& d1, float a0, float a1, float b0, float b1, float c0, float c1) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}
__device__ __forceinline__ void mul2v(float& d0, float& d1, float a0, float a1, float b0, float b1) {
  asm("{\n\t.reg .b64 ra, rb, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
      "mul.rn.f32x2 rd, ra, rb;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}

// One work item as published by the scheduler warp (16 ints in shared memory).
struct Item {
  int n_tiles;      // -1: no more work
  int g, seq0, L, tok0, kv_end, pos0, rA0, lenA, nA, b_valid;
  int H;            // rows that precede the sequence's own tokens in the self part (earlier turns), all visible
  int64_t base;
};
enum { IT_NTILES = 0, IT_G, IT_SEQ0, IT_L, IT_TOK0, IT_KVEND, IT_POS0, IT_RA0, IT_LENA, IT_NA, IT_BVALID, IT_BASE_LO,
       IT_BASE_HI, IT_H, IT_WORDS = 16 };

// Work index w -> item; false when the caller's index arrays are inconsistent
// (flagged in the status word; the scheduler skips the item).
__device__ __forceinline__ bool load_item(const TcParams& p, int w, Item& it) {
  const int2 e = p.items[w / p.G];
  it.g = w % p.G;
  const int b = e.x;
  const int TQ = 128 / p.s;
  it.seq0 = p.cu[b];
  it.L = p.cu[b + 1] - it.seq0;
  it.tok0 = e.y * 2 * TQ;
  it.b_valid = it.tok0 + TQ < it.L;
  it.H = p.hist ? p.hist[b] : 0;
  it.kv_end = it.H + min(it.L, it.tok0 + 2 * TQ);   // self rows the pair can see: the history, then its causal range
  it.base = p.slot ? (int64_t)p.slot[b] : (int64_t)it.seq0;
  it.pos0 = p.pos0 ? p.pos0[b] : 0;
  it.rA0 = 0; it.lenA = 0;
  bool route_ok = true;
  if (p.route_cu) {
    it.rA0 = p.route_cu[b * p.G + it.g]; it.lenA = p.route_cu[b * p.G + it.g + 1] - it.rA0;
    route_ok = (int64_t)it.rA0 + it.lenA <= p.route_rows;   // e.g. after a compaction that overflowed its capacity
  }
  else if (p.prefix_len > 0) { it.rA0 = it.g * p.prefix_len; it.lenA = p.prefix_len; }
  it.nA = (it.lenA + TILE_N - 1) / TILE_N;
  it.n_tiles = it.nA + (it.kv_end + TILE_N - 1) / TILE_N;
  const bool ok = it.L > 0 && it.tok0 < it.L && it.lenA >= 0 && it.rA0 >= 0 && it.base >= 0 && it.H >= 0 &&
                  it.base + it.H + it.L <= p.self_rows && it.seq0 >= 0 && route_ok;
  if (!ok) rc_set_status(p.status, route_ok ? RECACHE_DEV_BAD_SLOT : RECACHE_DEV_OVERFLOW);
  return ok;
}

// ------------------------------------------------------------- work list --
// Items = (sequence, tile-pair index): sequence by sequence, the longest sequences
// first, and inside a sequence the last (heaviest) tile pair first, so that the
// launch ends on the light items of short sequences.  With the KV group as the
// fastest index of the flattened work list, the CTAs that run at the same time
// share one sequence's K/V, which then stays in L2 instead of being streamed
// from HBM once per tile pair.  One CTA.  (Sequences of equal length land in an
// order that may differ between launches; no result depends on it.)
__global__ void __launch_bounds__(1024) tile_plan_kernel(const TcParams p, int tok_per_cta, int n_levels,
                                                         int2* __restrict__ items, int32_t* __restrict__ level_off,
                                                         int32_t* __restrict__ order, int max_items) {
  __shared__ int warp_sum[32];
  __shared__ int hist[1025];
  const int n_seq = p.n_seq;
  const int32_t* cu = p.cu;
  // each thread owns a contiguous chunk of sequences: local sums, block scan of the chunk sums, then the items
  const int per = (n_seq + blockDim.x - 1) / blockDim.x;
  const int b0 = min(n_seq, (int)threadIdx.x * per), b1 = min(n_seq, b0 + per);
  int sum = 0;
  for (int b = b0; b < b1; ++b) {
    const int len = cu[b + 1] - cu[b];
    if (len < 0) rc_set_status(p.status, RECACHE_DEV_BAD_SEQLENS);
    int nt = len > 0 ? (len + tok_per_cta - 1) / tok_per_cta : 0;
    if (nt > n_levels) { rc_set_status(p.status, RECACHE_DEV_BAD_SEQLENS); nt = n_levels; }   // longer than the max_len given
    sum += nt;
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = sum;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += v;
  }
  if (lane == 31) warp_sum[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = warp_sum[lane], wi = w;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, wi, off);
      if (lane >= off) wi += v;
    }
    warp_sum[lane] = wi - w;   // exclusive
    if (lane == 31) {
      p.header[0] = wi < max_items ? wi : max_items;
      p.header[1] = 0;         // dynamic work counter of the attention kernel
    }
  }
  __syncthreads();
  // (an encode launch shares K/V between the items of a sequence only: beyond a thousand items the
  // sequence-major order, which keeps a sequence's K/V in L2, is worth more than the balance)
  const int n_work = p.header[0] * p.G;
  const bool sorted = n_work <= (p.route_cu ? SORT_MAX : SORT_MAX / 4);
  if (sorted) {
    // few work items: they are sorted one by one below, so the sequences keep their order here
    int k = warp_sum[warp] + incl - sum;
    for (int b = b0; b < b1; ++b) {
      const int len = cu[b + 1] - cu[b];
      int nt = len > 0 ? (len + tok_per_cta - 1) / tok_per_cta : 0;
      if (nt > n_levels) nt = n_levels;
      level_off[b] = k;
      for (int l = nt - 1; l >= 0; --l, ++k)
        if (k < max_items) items[k] = make_int2(b, l);
    }
  } else {
    // counting sort of the sequences by their number of tile pairs, longest first: hist[bin] = items of
    // that bin, then (scanned from the top bin down) the first item index of the bin
    for (int i = threadIdx.x; i < 1025; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (int b = b0; b < b1; ++b) {
      const int len = cu[b + 1] - cu[b];
      int nt = len > 0 ? (len + tok_per_cta - 1) / tok_per_cta : 0;
      if (nt > n_levels) nt = n_levels;
      if (nt > 0) atomicAdd(&hist[min(nt, 1024)], nt);
    }
    __syncthreads();
    if (warp == 0) {
      int carry = 0;
      for (int c0 = 1024; c0 >= 0; c0 -= 32) {      // lane 0 takes the highest bin of the chunk
        const int bin_i = c0 - lane;
        const int v = bin_i >= 0 ? hist[bin_i] : 0;
        int vi = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const int u = __shfl_up_sync(0xffffffffu, vi, off);
          if (lane >= off) vi += u;
        }
        if (bin_i >= 0) hist[bin_i] = carry + vi - v;
        carry += __shfl_sync(0xffffffffu, vi, 31);
      }
    }
    __syncthreads();
    for (int b = b0; b < b1; ++b) {
      const int len = cu[b + 1] - cu[b];
      int nt = len > 0 ? (len + tok_per_cta - 1) / tok_per_cta : 0;
      if (nt > n_levels) nt = n_levels;
      if (nt == 0) continue;
      int k = atomicAdd(&hist[min(nt, 1024)], nt);
      level_off[b] = k;
      for (int l = nt - 1; l >= 0; --l, ++k)
        if (k < max_items) items[k] = make_int2(b, l);
    }
  }
  // Few work items (a prefill of a handful of requests): one CTA gets one or two of them, so their
  // order decides the tail.  Sort them by weight (K/V tiles), heaviest first, with a counting sort.
  __syncthreads();
  if (threadIdx.x == 0) p.header[2] = sorted ? 1 : 0;
  if (!sorted) return;
  for (int i = threadIdx.x; i < 1025; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  int bin[SORT_MAX / 1024];
#pragma unroll
  for (int j = 0; j < SORT_MAX / 1024; ++j) {
    const int w = threadIdx.x + j * 1024;
    bin[j] = -1;
    if (w < n_work) {
      Item it;
      const bool ok = load_item(p, w, it);
      bin[j] = 1024 - (ok ? min(it.n_tiles, 1024) : 0);   // heaviest first
      atomicAdd(&hist[bin[j]], 1);
    }
  }
  __syncthreads();
  if (warp == 0) {   // exclusive scan of the 1025 bins
    int carry = 0;
    for (int c0 = 0; c0 < 1025; c0 += 32) {
      const int v = c0 + lane < 1025 ? hist[c0 + lane] : 0;
      int vi = v;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, vi, off);
        if (lane >= off) vi += u;
      }
      if (c0 + lane < 1025) hist[c0 + lane] = carry + vi - v;
      carry += __shfl_sync(0xffffffffu, vi, 31);
    }
  }
  __syncthreads();
#pragma unroll
  for (int j = 0; j < SORT_MAX / 1024; ++j)
    if (bin[j] >= 0) order[atomicAdd(&hist[bin[j]], 1)] = threadIdx.x + j * 1024;
}

// ---------------------------------------------------------------- kernel --
// Persistent: a scheduler warp draws work indices from a global counter (the
// list is heavy-first inside each sequence, or heavy-first overall when the plan
// sorted it, so the tail of the launch is made of light items) and publishes
// items through a two-slot ring in shared memory.
// The next item's Q load, Q rotation and first K/V tiles overlap the current
// item's last tiles and its epilogue.  Barrier phases run on across items.
template <typename TO, bool ROT_SMEM, bool GATHER>
__global__ void __launch_bounds__(NTHREADS, 1) attn_tc_kernel(const __grid_constant__ CUtensorMap tm_q,
                                                              const __grid_constant__ CUtensorMap tm_ks,
                                                              const __grid_constant__ CUtensorMap tm_vs,
                                                              const __grid_constant__ CUtensorMap tm_kr,
                                                              const __grid_constant__ CUtensorMap tm_vr,
                                                              const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  const int total = p.header[0] * p.G;
  if ((int)blockIdx.x >= total) return;
  const int s = p.s, TQ = 128 / s;

  const uint32_t sm = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sm_gen = smem_raw + (sm - smem_u32(smem_raw));
  const uint32_t bars = sm + SM_BAR;
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sm_gen + SM_MISC + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm_gen + SM_MISC);
  volatile int* item_ring = reinterpret_cast<volatile int*>(sm_gen + SM_ITEM);
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(bar(B_QFULL), 1);
    mbar_init(bar(B_QREADY + 0), 128); mbar_init(bar(B_QREADY + 1), 128);
    mbar_init(bar(B_QEMPTY), 1);
    for (int i = 0; i < NSTAGE; ++i) {   // gather mode: the 128 epilogue lanes and the TMA producer arrive on every stage
      mbar_init(bar(B_KFULL + i), GATHER ? 129 : 1); mbar_init(bar(B_KEMPTY + i), 1);
      mbar_init(bar(B_VFULL + i), GATHER ? 129 : 1); mbar_init(bar(B_VEMPTY + i), 1);
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(bar(B_SFULL + x), 1); mbar_init(bar(B_PREADY + x), 128); mbar_init(bar(B_ODONE + x), 1);
      // producer + MMA + 256 softmax + 128 epilogue threads
      mbar_init(bar(B_IFULL + x), 1); mbar_init(bar(B_IEMPTY + x), 386);
      mbar_init(bar(B_LREADY + x), 128); mbar_init(bar(B_ODRAIN + x), 128); mbar_init(bar(B_PHALF + x), 128);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8 && lane == 0) {
    prefetch_tmap(&tm_q); prefetch_tmap(&tm_ks); prefetch_tmap(&tm_vs);
    if (p.route_cu || p.prefix_len > 0) { prefetch_tmap(&tm_kr); prefetch_tmap(&tm_vr); }
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sm + SM_MISC), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  // Item n of this CTA lives in ring slot n & 1; every consumer copies it to
  // registers and then releases the slot.
  auto fetch_item = [&](uint32_t n, Item& it, bool release) {
    const int sl = n & 1u;
    mbar_wait(bar(B_IFULL + sl), (n >> 1) & 1u, abort_flag, p.status);
    const int* r = const_cast<const int*>(item_ring) + sl * IT_WORDS;   // (ordered by the barrier wait above and the arrive below)
    it.n_tiles = r[IT_NTILES]; it.g = r[IT_G]; it.seq0 = r[IT_SEQ0]; it.L = r[IT_L]; it.tok0 = r[IT_TOK0];
    it.kv_end = r[IT_KVEND]; it.pos0 = r[IT_POS0]; it.rA0 = r[IT_RA0]; it.lenA = r[IT_LENA]; it.nA = r[IT_NA];
    it.b_valid = r[IT_BVALID]; it.H = r[IT_H];
    it.base = (int64_t)(((uint64_t)(uint32_t)r[IT_BASE_HI] << 32) | (uint32_t)r[IT_BASE_LO]);
    if (*abort_flag) it.n_tiles = -1;
    if (release) mbar_arrive(bar(B_IEMPTY + sl));
  };

  if (warp >= 12) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_EPI));
    // ===================== epilogue warps =====================
    // O of a finished query tile leaves tensor memory here, so that the softmax warps can go
    // straight to the next item's Q.  Warp 12 + q reads lanes 32 q .. 32 q + 31.
    const int row = threadIdx.x & 127;
    const uint32_t lane_addr = ((uint32_t)(32 * (warp & 3)) << 16);
    const float* inv_l = reinterpret_cast<const float*>(sm_gen + SM_INVL);
    Item it, nx;
    uint32_t done[2] = {0, 0};
    fetch_item(0, it, true);
    uint32_t kv_n = 0;
    for (uint32_t item_n = 0; it.n_tiles > 0; ++item_n) {
      if (GATHER) {
        // Gather mode: these 128 lanes also fill the route tiles of the item.  Row n of the route is
        // row route_idx[n] of the resource cache: warp w takes rows 32 w .. 32 w + 31 of a tile, one
        // index per lane handed round by shuffles, 16 16-byte asynchronous copies per lane straight
        // to the swizzled positions of a TMA tile (zero-fill past the route's end).  A lane's arrival
        // fires when its copies have landed; the MMA warp puts a proxy fence before the reads.
        const int w = warp & 3, hi = lane >> 4, c = lane & 15;
        uint32_t sw[4];
#pragma unroll
        for (int m = 0; m < 4; ++m) sw[m] = (uint32_t)(((c & 7) ^ ((2 * m + hi) & 7)) << 4);
        for (int i = 0; i < it.n_tiles; ++i) {
          const uint32_t n = kv_n + (uint32_t)i;
          const int st = n % NSTAGE;
          const uint32_t ph = (n / NSTAGE) & 1u;
          const bool route = i < it.nA;
          int idx = -1;
          if (route) {
            const int r = 32 * w + lane, cnt = min(TILE_N, it.lenA - i * TILE_N);
            if (r < cnt) {
              idx = p.route_idx[it.rA0 + i * TILE_N + r];
              if (idx < 0 || idx >= p.pool_tokens) { rc_set_status(p.status, RECACHE_DEV_BAD_SLOT); idx = -1; }
            }
          }
#pragma unroll
          for (int kv = 0; kv < 2; ++kv) {
            const int b_full = kv ? B_VFULL : B_KFULL, b_empty = kv ? B_VEMPTY : B_KEMPTY;
            mbar_wait(bar(b_empty + st), ph ^ 1u, abort_flag, p.status);
            if (route) {
              const uint8_t* src_l = (kv ? p.gather_v : p.gather_k) + (int64_t)it.g * p.pool_tokens * 256 + c * 16;
              const uint32_t dst_l = sm + (kv ? SM_V : SM_K) + st * TILE_BYTES + (c >> 3) * BOX_BYTES + (32 * w + hi) * 128;
#pragma unroll
              for (int kk = 0; kk < 16; ++kk) {
                const int ix = __shfl_sync(0xffffffffu, idx, 2 * kk + hi);
                cp_async16(dst_l + 2 * kk * 128 + sw[kk & 3], src_l + (int64_t)max(ix, 0) * 256, ix >= 0 ? 16u : 0u);
              }
              cp_async_arrive(bar(b_full + st));
            } else {
              mbar_arrive(bar(b_full + st));
            }
          }
        }
        kv_n += (uint32_t)it.n_tiles;
      }
      fetch_item(item_n + 1, nx, true);
      if (row == 0) { TR(3, item_n, 0); TRV(3, item_n, 15, it.n_tiles * 2 + it.b_valid); }
      // The stores below and the rotation of the next item's Q go through the same load/store
      // path, and the rotation is the urgent one: a tile's O is written back once the same tile's
      // next Q has been rotated.  (O is not needed back before the next item's first P V, a whole
      // softmax later; tile B's rotation finishes after tile A's, so tile A is not held up by it.)
      // This wait is a matter of priority only, so it is taken only where the rotating warpgroup
      // cannot complete a second phase before it: tile A's warpgroup is active in every item and
      // stops at the end of the next item for this item's O-drained arrival, which comes after the
      // wait.  Tile B's warpgroup rotates Q even in items where its tile is empty and is held back by
      // nothing there, so with an empty tile B in this item or the next (short sequences) it could
      // pass two phases while tile A is being drained here, and a parity wait would then sleep
      // through the phase it wants.
      for (int x = 0; x < 2; ++x) {
        if (nx.n_tiles > 0 && (x == 0 || (it.b_valid && nx.b_valid)))
          mbar_wait(bar(B_QREADY + x), (item_n + 1u) & 1u, abort_flag, p.status);
        if (row == 0) TR(3, item_n, 1 + 5 * x);
        if (x == 1 && !it.b_valid) continue;
        mbar_wait(bar(B_LREADY + x), done[x] & 1u, abort_flag, p.status);
        if (row == 0) TR(3, item_n, 2 + 5 * x);
        mbar_wait(bar(B_ODONE + x), done[x] & 1u, abort_flag, p.status);
        if (row == 0) TR(3, item_n, 3 + 5 * x);
        ++done[x];
        tc_fence_after();
        const float inv = inv_l[x * 128 + row];
        const int t_row = it.tok0 + x * TQ + row / s;
        const bool row_valid = t_row < it.L;
        TO* orow = reinterpret_cast<TO*>(p.out) + ((int64_t)(it.seq0 + t_row) * p.Hq + it.g * s + row % s) * D;
        const uint32_t t_o = tmem + lane_addr + COL_O + 128 * x;
#pragma unroll 1
        for (int ch = 0; ch < 8; ++ch) {
          uint32_t orr[16];
          TMEM_LD16(t_o + 16 * ch, orr);
          tmem_wait_ld();
          if (row_valid) {
            if constexpr (sizeof(TO) == 4) {
#pragma unroll
              for (int c = 0; c < 16; c += 8)
                st_global_v8(reinterpret_cast<float*>(orow) + 16 * ch + c,
                             __float_as_uint(__uint_as_float(orr[c]) * inv), __float_as_uint(__uint_as_float(orr[c + 1]) * inv),
                             __float_as_uint(__uint_as_float(orr[c + 2]) * inv), __float_as_uint(__uint_as_float(orr[c + 3]) * inv),
                             __float_as_uint(__uint_as_float(orr[c + 4]) * inv), __float_as_uint(__uint_as_float(orr[c + 5]) * inv),
                             __float_as_uint(__uint_as_float(orr[c + 6]) * inv), __float_as_uint(__uint_as_float(orr[c + 7]) * inv));
            } else {
              st_global_v8(reinterpret_cast<__nv_bfloat16*>(orow) + 16 * ch,
                           pack2(__uint_as_float(orr[0]) * inv, __uint_as_float(orr[1]) * inv),
                           pack2(__uint_as_float(orr[2]) * inv, __uint_as_float(orr[3]) * inv),
                           pack2(__uint_as_float(orr[4]) * inv, __uint_as_float(orr[5]) * inv),
                           pack2(__uint_as_float(orr[6]) * inv, __uint_as_float(orr[7]) * inv),
                           pack2(__uint_as_float(orr[8]) * inv, __uint_as_float(orr[9]) * inv),
                           pack2(__uint_as_float(orr[10]) * inv, __uint_as_float(orr[11]) * inv),
                           pack2(__uint_as_float(orr[12]) * inv, __uint_as_float(orr[13]) * inv),
                           pack2(__uint_as_float(orr[14]) * inv, __uint_as_float(orr[15]) * inv));
            }
          }
        }
        // the next item's first P V overwrites O, its softmax overwrites 1 / l: both wait for this
        tc_fence_before();
        mbar_arrive(bar(B_ODRAIN + x));
        if (row == 0) TR(3, item_n, 4 + 5 * x);
      }
      it = nx;
    }
  } else if (warp >= 8) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_AUX));
#ifdef RC_OBSERVE
  if (warp == 11 && blockIdx.x == 0) {
    // lane b watches barrier b (lanes past the last barrier watch barrier 0 and log nothing)
    const bool logs = lane < B_COUNT;
    const uint32_t my = bar(logs ? lane : 0);
    uint32_t par = 0;
    int n = 0;
    const long long start = clock64();
    if (lane == 0) g_observe[OBS_PER * 31] = start;
    uint32_t last = (uint32_t)start;
    for (uint32_t iter = 0;; ++iter) {
      uint32_t ok, now;
      asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%2], %3;\n\tselp.u32 %0, 1, 0, p;\n\tmov.u32 %1, %%clock;\n\t}"
                   : "=r"(ok), "=r"(now) : "r"(my), "r"(par) : "memory");
      if (ok) {
        par ^= 1u; last = now;
        if (logs && n < OBS_PER) g_observe[lane * OBS_PER + n++] = start + (long long)(uint32_t)(now - (uint32_t)start);
      }
      if ((iter & 63u) == 63u) {
        const uint32_t newest = __reduce_max_sync(0xffffffffu, last - (uint32_t)start);
        if ((now - (uint32_t)start) - newest > 60000u) break;
      }
    }
    if (logs) g_observe_n[lane] = n;
  }
#endif
  if (warp == 10) {
    // ===================== scheduler =====================
    if (lane == 0) {
      bool first = true;
      for (uint32_t n = 0;; ++n) {
        const int sl = n & 1u;
        mbar_wait(bar(B_IEMPTY + sl), ((n >> 1) & 1u) ^ 1u, abort_flag, p.status);
        Item it;
        for (;;) {   // CTA c starts with index c; every later index comes from the shared counter
          const int w = first ? (int)blockIdx.x : (int)gridDim.x + atomicAdd(p.header + 1, 1);
          first = false;
          if (w >= total || *abort_flag) { it.n_tiles = -1; break; }
          if (load_item(p, p.header[2] ? p.order[w] : w, it)) break;
        }
        volatile int* r = item_ring + sl * IT_WORDS;
        r[IT_NTILES] = it.n_tiles;
        if (it.n_tiles > 0) {
          r[IT_G] = it.g; r[IT_SEQ0] = it.seq0; r[IT_L] = it.L; r[IT_TOK0] = it.tok0; r[IT_KVEND] = it.kv_end;
          r[IT_POS0] = it.pos0; r[IT_RA0] = it.rA0; r[IT_LENA] = it.lenA; r[IT_NA] = it.nA; r[IT_BVALID] = it.b_valid;
          r[IT_H] = it.H;
          r[IT_BASE_LO] = (int)(uint32_t)(it.base & 0xffffffffll); r[IT_BASE_HI] = (int)(uint32_t)((uint64_t)it.base >> 32);
        }
        mbar_arrive(bar(B_IFULL + sl));
        if (it.n_tiles < 0) break;
      }
    }
    __syncwarp();
  } else if (warp == 8) {
    // ===================== TMA producer =====================
    if (lane == 0) {
      Item it;
      uint32_t kv_n = 0;
      for (uint32_t item_n = 0;; ++item_n) {
        fetch_item(item_n, it, true);
        if (it.n_tiles < 0) break;
        // Q tiles: free once the previous item's last S = Q K^T has completed
        TR(4, item_n, 0);
        mbar_wait(bar(B_QEMPTY), (item_n & 1u) ^ 1u, abort_flag, p.status);
        TR(4, item_n, 1);
        uint32_t rot_bytes = 0;
        const int pos_start = it.pos0 + it.tok0;
        if (ROT_SMEM) {
          const int rows = min(2 * TQ, p.max_pos - pos_start);
          if (pos_start >= 0 && rows > 0) rot_bytes = (uint32_t)rows * 256u;
        }
        mbar_expect_tx(bar(B_QFULL), 2 * TILE_BYTES + 2 * rot_bytes);
        for (int x = 0; x < 2; ++x)
          for (int kc = 0; kc < 2; ++kc)
            tma_load_3d(sm + SM_Q + x * TILE_BYTES + kc * BOX_BYTES, &tm_q, bar(B_QFULL), kc * 64, it.g * s,
                        it.seq0 + it.tok0 + x * TQ);
        if (rot_bytes) {   // cos / sin rows of the item's positions (contiguous in the table)
          bulk_load(sm + SM_ROT, p.cos_tab + (int64_t)pos_start * 64, rot_bytes, bar(B_QFULL));
          bulk_load(sm + SM_ROT + ROT_BYTES, p.sin_tab + (int64_t)pos_start * 64, rot_bytes, bar(B_QFULL));
        }
        for (int i = 0; i < it.n_tiles; ++i, ++kv_n) {
          const int st = kv_n % NSTAGE;
          const uint32_t ph = (kv_n / NSTAGE) & 1u;
          const bool route = i < it.nA;
          const int row = route ? it.rA0 + i * TILE_N
                                : (int)((int64_t)it.g * p.self_rows + it.base) + (i - it.nA) * TILE_N;
          // (gather mode: a route tile is filled by the epilogue warps; every stage barrier expects
          // their 128 arrivals plus one from here, whoever brings the data)
          mbar_wait(bar(B_KEMPTY + st), ph ^ 1u, abort_flag, p.status);
          if (i == 0) TR(4, item_n, 2);
          if (GATHER && route) {
            mbar_arrive(bar(B_KFULL + st));
          } else {
            mbar_expect_tx(bar(B_KFULL + st), TILE_BYTES);
            for (int kc = 0; kc < 2; ++kc)
              tma_load_2d(sm + SM_K + st * TILE_BYTES + kc * BOX_BYTES, route ? &tm_kr : &tm_ks, bar(B_KFULL + st), kc * 64, row);
          }
          mbar_wait(bar(B_VEMPTY + st), ph ^ 1u, abort_flag, p.status);
          if (GATHER && route) {
            mbar_arrive(bar(B_VFULL + st));
          } else {
            mbar_expect_tx(bar(B_VFULL + st), TILE_BYTES);
            for (int kc = 0; kc < 2; ++kc)
              tma_load_2d(sm + SM_V + st * TILE_BYTES + kc * BOX_BYTES, route ? &tm_vr : &tm_vs, bar(B_VFULL + st), kc * 64, row);
          }
          if (i == 0) TR(4, item_n, 3);
          if (i == it.n_tiles - 1) TR(4, item_n, 4);
        }
      }
    }
    __syncwarp();
  } else if (warp == 9) {
    // ===================== MMA issuer =====================
    // descriptor words: low = (address >> 4) | (LBO >> 4) << 16, high = (SBO >> 4) | version | swizzle
    // The issuing lane is elected once: every MMA and every commit comes from that one thread
    // (a commit tracks the MMAs of the thread that executes it).
    const bool issuer = elect_one();
    const uint64_t d_q = smem_desc(0, 16, 1024) + ((sm + SM_Q) >> 4), d_k = smem_desc(0, 16, 1024) + ((sm + SM_K) >> 4);
    const uint64_t d_v = smem_desc(0, BOX_BYTES, 1024) + ((sm + SM_V) >> 4);
    auto issue_qk = [&](int x, int st) {
      const uint64_t qa = d_q + x * (TILE_BYTES >> 4), ka = d_k + st * (TILE_BYTES >> 4);
      const uint32_t dst = tmem + COL_S + 128 * x;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t off = ((j >> 2) * BOX_BYTES + (j & 3) * 32) >> 4;
        mma_ss(dst, qa + off, ka + off, IDESC_QK, j > 0);
      }
    };
    // K steps k0 .. ksteps-1 of O += P V (16 keys each); a full half (4 steps) is the common case
    auto issue_pv = [&](int x, int st, int k0, int ksteps, bool first) {
      const uint64_t va = d_v + st * (TILE_BYTES >> 4);
      const uint32_t dst = tmem + COL_O + 128 * x, src = tmem + COL_S + 128 * x;
      if (ksteps - k0 == 4) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
          mma_ts(dst, src + 8 * (k0 + j), va + (k0 + j) * (2048 >> 4), IDESC_PV, (!first || j > 0) ? 1u : 0u);
      } else {
#pragma unroll 1
        for (int j = k0; j < ksteps; ++j)
          mma_ts(dst, src + 8 * j, va + j * (2048 >> 4), IDESC_PV, (!first || j > k0) ? 1u : 0u);
      }
    };
    Item it;
    uint32_t kv_n = 0, cnt[2] = {0, 0};   // K/V tiles, tiles per query tile so far
    uint32_t items_x[2] = {0, 0};         // items each query tile has taken part in
    for (uint32_t item_n = 0;; ++item_n) {
      fetch_item(item_n, it, false);
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_IEMPTY + (item_n & 1u)));
      if (it.n_tiles < 0) break;
      const int n_tiles = it.n_tiles, nA = it.nA, lenA = it.lenA, L = it.H + it.L, kv_end = it.kv_end;
      const bool b_valid = it.b_valid != 0;
      if (issuer) TR(2, item_n, 0);
      // each query tile starts as soon as its own half of Q has been rotated
      mbar_wait(bar(B_QREADY + 0), item_n & 1u, abort_flag, p.status);
      if (issuer) TR(2, item_n, 1);
      mbar_wait(bar(B_KFULL + kv_n % NSTAGE), (kv_n / NSTAGE) & 1u, abort_flag, p.status);
      if (issuer) TR(2, item_n, 2);
      if (GATHER) fence_async_smem();   // the tile may have been written by cp.async (generic proxy)
      tc_fence_after();
      const int st0 = kv_n % NSTAGE;
      if (issuer) { issue_qk(0, st0); tc_commit(bar(B_SFULL + 0)); }
      // (waited for even when the second tile is empty: its warps still rewrite that half of Q,
      // and the Q-empty commit below lets the next load overwrite it)
      if (issuer) TR(2, item_n, 3);
      mbar_wait(bar(B_QREADY + 1), item_n & 1u, abort_flag, p.status);
      if (issuer) TR(2, item_n, 4);
      tc_fence_after();
      if (issuer) {
        if (b_valid) { issue_qk(1, st0); tc_commit(bar(B_SFULL + 1)); }
        if (n_tiles == 1) tc_commit(bar(B_QEMPTY));
      }
      __syncwarp();
      for (int i = 0; i < n_tiles; ++i) {
        const uint32_t n = kv_n + (uint32_t)i;
        const int st = n % NSTAGE;
        const uint32_t ph = (n / NSTAGE) & 1u;
        // rows of this tile that really belong to the segment; keys the pair can see
        const int seg_rows = i < nA ? lenA - i * TILE_N : L - (i - nA) * TILE_N;
        const int vis_rows = i < nA ? seg_rows : kv_end - (i - nA) * TILE_N;
        const int ksteps = (min(vis_rows, TILE_N) + 15) >> 4;
        mbar_wait(bar(B_VFULL + st), ph, abort_flag, p.status);
        if (issuer && i == 0) TR(2, item_n, 5);
        if (GATHER) fence_async_smem();
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
        const int st1 = (n + 1) % NSTAGE;
        const uint32_t ph1 = ((n + 1) / NSTAGE) & 1u;
        const bool more = i + 1 < n_tiles;
        // P of keys 0..63 arrives first: half of P V runs while the softmax finishes the other half
        mbar_wait(bar(B_PHALF + 0), cnt[0] & 1u, abort_flag, p.status);
        if (issuer && i == 0) TR(2, item_n, 6);
        if (i == 0 && items_x[0] > 0) mbar_wait(bar(B_ODRAIN + 0), (items_x[0] - 1u) & 1u, abort_flag, p.status);
        if (issuer && i == 0) TR(2, item_n, 7);
        tc_fence_after();
        if (issuer) issue_pv(0, st, 0, min(ksteps, 4), i == 0);
        mbar_wait(bar(B_PREADY + 0), cnt[0]++ & 1u, abort_flag, p.status);
        tc_fence_after();
        if (issuer) { issue_pv(0, st, 4, ksteps, false); if (!more) tc_commit(bar(B_ODONE + 0)); }
        if (more) {
          mbar_wait(bar(B_KFULL + st1), ph1, abort_flag, p.status);
          if (GATHER) fence_async_smem();
          tc_fence_after();
          if (issuer) { issue_qk(0, st1); tc_commit(bar(B_SFULL + 0)); }
        }
        if (b_valid) {
          if (issuer && i == 0) TR(2, item_n, 8);
          mbar_wait(bar(B_PHALF + 1), cnt[1] & 1u, abort_flag, p.status);
          if (issuer && i == 0) TR(2, item_n, 9);
          if (i == 0 && items_x[1] > 0) mbar_wait(bar(B_ODRAIN + 1), (items_x[1] - 1u) & 1u, abort_flag, p.status);
          if (issuer && i == 0) TR(2, item_n, 10);
          tc_fence_after();
          if (issuer) issue_pv(1, st, 0, min(ksteps, 4), i == 0);
          mbar_wait(bar(B_PREADY + 1), cnt[1]++ & 1u, abort_flag, p.status);
          tc_fence_after();
          if (issuer) { issue_pv(1, st, 4, ksteps, false); if (!more) tc_commit(bar(B_ODONE + 1)); }
        }
        if (issuer) {
          if (more) {
            if (b_valid) { issue_qk(1, st1); tc_commit(bar(B_SFULL + 1)); }
            if (i + 2 == n_tiles) tc_commit(bar(B_QEMPTY));   // the item's last S has been issued
          } else {
            tc_commit(bar(B_VEMPTY + st));                    // the item's last V tile (earlier ones: see the softmax side)
          }
        }
        __syncwarp();
        if (issuer && i == 0) TR(2, item_n, 11);
        if (issuer && i == n_tiles - 2) TR(2, item_n, 12);
      }
      if (issuer) { TR(2, item_n, 13); TRV(2, item_n, 15, n_tiles * 2 + (b_valid ? 1 : 0)); }
      kv_n += (uint32_t)n_tiles;
      ++items_x[0];
      if (b_valid) ++items_x[1];
    }
  }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_SOFTMAX));
    // ===================== softmax warpgroups =====================
    const int x = warp >> 2;                       // tile A or B
    const int row = threadIdx.x & 127;             // row of the tile = TMEM lane
    const uint32_t lane_addr = ((uint32_t)(32 * (warp & 3)) << 16);
    const uint32_t t_s = tmem + lane_addr + COL_S + 128 * x;
    const uint32_t t_o = tmem + lane_addr + COL_O + 128 * x;
    const float c2 = p.scale_log2;
    uint32_t item_n = 0, cnt = 0;                  // items seen; tiles this query tile has gone through
    uint32_t kv_n = 0, done_n = 0;                 // K/V tiles of all items so far; items this query tile took part in

    // Rotates this query tile of the freshly loaded Q in shared memory (swizzled 16-byte chunks;
    // element i pairs with i + 64 in the other box).  A thread takes one (token, chunk) pair at a
    // time and goes through the token's s heads, so that cos / sin are read once per token, not
    // once per row; the 8 lanes of a token cover whole 128-byte rows of Q.
    auto rotate_q = [&](const Item& it, uint32_t n_item) {
      if (row == 0) TR(x, n_item, 0);
      mbar_wait(bar(B_QFULL), n_item & 1u, abort_flag, p.status);
      if (row == 0) TR(x, n_item, 1);
      uint8_t* qt = sm_gen + SM_Q + x * TILE_BYTES;
      for (int u = row; u < TQ * 8; u += 128) {
        const int tok = u >> 3, c = u & 7;
        const int t_eff = min(it.tok0 + x * TQ + tok, it.L - 1);
        const int pos = it.pos0 + t_eff;
        if (pos < 0 || pos >= p.max_pos) rc_set_status(p.status, RECACHE_DEV_BAD_POS);
        const float *cp, *sp;
        if (ROT_SMEM) {   // staged by the producer: row = token index inside the tile pair
          const int ri = min(max(t_eff - it.tok0, 0), 2 * TQ - 1);
          cp = reinterpret_cast<const float*>(sm_gen + SM_ROT + ri * 256) + c * 8;
          sp = reinterpret_cast<const float*>(sm_gen + SM_ROT + ROT_BYTES + ri * 256) + c * 8;
        } else {
          const int pc = min(max(pos, 0), p.max_pos - 1);
          cp = p.cos_tab + (int64_t)pc * 64 + c * 8;
          sp = p.sin_tab + (int64_t)pc * 64 + c * 8;
        }
        // lanes c and c + 4 would hit the same banks: they take the two halves in opposite order
        const int first = (c & 4) ? 4 : 0;
        const float4 ca = *reinterpret_cast<const float4*>(cp + first), cb = *reinterpret_cast<const float4*>(cp + 4 - first);
        const float4 sa = *reinterpret_cast<const float4*>(sp + first), sb = *reinterpret_cast<const float4*>(sp + 4 - first);
        const float4 c0 = first ? cb : ca, c1 = first ? ca : cb, s0 = first ? sb : sa, s1 = first ? sa : sb;
        const float cs[8] = {c0.x, c0.y, c0.z, c0.w, c1.x, c1.y, c1.z, c1.w};
        const float sn[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll 2
        for (int h = 0; h < s; ++h) {
          const int r = tok * s + h;
          uint8_t* qb = qt + r * 128 + ((c ^ (r & 7)) << 4);
          const uint4 ulo = *reinterpret_cast<uint4*>(qb), uhi = *reinterpret_cast<uint4*>(qb + BOX_BYTES);
          const uint32_t wlo[4] = {ulo.x, ulo.y, ulo.z, ulo.w}, whi[4] = {uhi.x, uhi.y, uhi.z, uhi.w};
          uint32_t ol[4], oh[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float l0 = __uint_as_float(wlo[i] << 16), l1 = __uint_as_float(wlo[i] & 0xffff0000u);
            const float h0 = __uint_as_float(whi[i] << 16), h1 = __uint_as_float(whi[i] & 0xffff0000u);
            // lo' = lo cos - hi sin, hi' = hi cos + lo sin: the products with sin are rounded first
            // (hi * (-sin) is exactly -(hi * sin)), as in the scalar form of the other kernels
            float t0, t1, u0, u1, a0, a1, b0, b1;
            mul2v(t0, t1, h0, h1, -sn[2 * i], -sn[2 * i + 1]);
            mul2v(u0, u1, l0, l1, sn[2 * i], sn[2 * i + 1]);
            fma2v(a0, a1, l0, l1, cs[2 * i], cs[2 * i + 1], t0, t1);
            fma2v(b0, b1, h0, h1, cs[2 * i], cs[2 * i + 1], u0, u1);
            ol[i] = pack2(a0, a1);
            oh[i] = pack2(b0, b1);
          }
          *reinterpret_cast<uint4*>(qb) = make_uint4(ol[0], ol[1], ol[2], ol[3]);
          *reinterpret_cast<uint4*>(qb + BOX_BYTES) = make_uint4(oh[0], oh[1], oh[2], oh[3]);
        }
      }
      fence_async_smem();
      mbar_arrive(bar(B_QREADY + x));
      if (row == 0) TR(x, n_item, 2);
    };

    Item it, nx;
    fetch_item(0, it, true);
    if (it.n_tiles > 0) rotate_q(it, 0);
    while (it.n_tiles > 0) {
      const bool active = x == 0 || it.b_valid;
      const bool releaser = row == 0 && x == (it.b_valid ? 1 : 0);   // the tile whose S = Q K^T is issued last
      const int t_row = it.tok0 + x * TQ + row / s;     // token (local index)
      const int t_eff = min(t_row, it.L - 1);
      const int n_tiles = it.n_tiles, nA = it.nA, lenA = it.lenA, H = it.H;
      float m_ref = -INFINITY, l_sum = 0.f;
      if (active) {
        for (int i = 0; i < n_tiles; ++i, ++cnt) {
          mbar_wait(bar(B_SFULL + x), cnt & 1u, abort_flag, p.status);
          if (row == 0 && i == 0) TR(x, item_n, 3);
          if (row == 0 && i == 1) TR(x, item_n, 5);
          if (row == 0 && i == n_tiles - 1) TR(x, item_n, 6);
          tc_fence_after();
          if (releaser) {
            // S of tile i is complete: so is every earlier MMA, i.e. the last reader of K tile i
            // and of V tile i - 1.  Hand both stages back to the producer.
            mbar_arrive(bar(B_KEMPTY + (kv_n + i) % NSTAGE));
            if (i > 0) mbar_arrive(bar(B_VEMPTY + (kv_n + i - 1) % NSTAGE));
          }
          uint32_t sr[128];
          TMEM_LD32(t_s + 0, sr, 0); TMEM_LD32(t_s + 32, sr, 32); TMEM_LD32(t_s + 64, sr, 64); TMEM_LD32(t_s + 96, sr, 96);
          tmem_wait_ld();
          // keys this row may see in this tile: columns [0, lim)
          const int lim = i < nA ? lenA - i * TILE_N : H + t_eff - (i - nA) * TILE_N + 1;
          if (lim < TILE_N) {
#pragma unroll
            for (int c = 0; c < 128; ++c) if (c >= lim) sr[c] = 0xff800000u;   // -inf
          }
          float mx4[4] = {__uint_as_float(sr[0]), __uint_as_float(sr[1]), __uint_as_float(sr[2]), __uint_as_float(sr[3])};
#pragma unroll
          for (int c = 4; c < 124; c += 8) {     // three-input max: 4 chains, 2 new values per step
#pragma unroll
            for (int u = 0; u < 4; ++u) mx4[u] = fmax3(mx4[u], __uint_as_float(sr[c + 2 * u]), __uint_as_float(sr[c + 2 * u + 1]));
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) mx4[u] = fmaxf(mx4[u], __uint_as_float(sr[124 + u]));
          const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
          const float m_new = fmaxf(m_ref, mx);
          bool need = false;
          if (i == 0) m_ref = m_new;                       // O is overwritten by the first P V
          else need = (m_new - m_ref) * c2 > 8.f;          // lazy: P stays below 2^8 otherwise
          if (__any_sync(0xffffffffu, need)) {
            // the previous P V of this tile was issued before this S, so it is complete as well
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
            float x0, x1, x2, x3;
            fma2(x0, x1, __uint_as_float(sr[2 * c]), __uint_as_float(sr[2 * c + 1]), c2, neg_m);
            fma2(x2, x3, __uint_as_float(sr[2 * c + 2]), __uint_as_float(sr[2 * c + 3]), c2, neg_m);
            const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
            add2(acc[0], acc[1], p0, p1);
            add2(acc[2], acc[3], p2, p3);
            pr[c] = pack2(p0, p1);
            pr[c + 1] = pack2(p2, p3);
            if (c == 30) {   // first half of P goes out, and into P V, while the second is computed
              TMEM_ST32(t_s + 0, pr, 0);
              tmem_wait_st();
              tc_fence_before();
              mbar_arrive(bar(B_PHALF + x));
            }
          }
          l_sum += (acc[0] + acc[1]) + (acc[2] + acc[3]);
          TMEM_ST32(t_s + 32, pr, 32);
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(bar(B_PREADY + x));
          if (row == 0 && i == 0) TR(x, item_n, 4);
          if (row == 0 && i == n_tiles - 1) TR(x, item_n, 7);
        }
      }
      // ---- hand the finished tile to the epilogue warps (they wait for its last P V themselves) ----
      if (active) {
        if (done_n > 0) mbar_wait(bar(B_ODRAIN + x), (done_n - 1u) & 1u, abort_flag, p.status);   // 1 / l of the item before was read
        if (row == 0) TR(x, item_n, 8);
        reinterpret_cast<float*>(sm_gen + SM_INVL)[x * 128 + row] = 1.f / l_sum;
        mbar_arrive(bar(B_LREADY + x));
        ++done_n;
      }
      kv_n += (uint32_t)n_tiles;
      // ---- next item's Q (its load was issued a tile ago) ----
      fetch_item(item_n + 1, nx, true);
      if (row == 0) { TR(x, item_n, 9); TRV(x, item_n, 15, n_tiles * 2 + it.b_valid); }
      if (nx.n_tiles > 0) rotate_q(nx, item_n + 1);
      it = nx; ++item_n;
    }
  }
  // ---- teardown: every thread is done with tensor memory before it is freed ----
  if (*abort_flag) rc_timeout_drain();   // a wait ran out: let what is in flight land first
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

#ifdef RC_OBSERVE
extern "C" __attribute__((visibility("default"))) int recache_debug_observe(long long* host, int* counts) {
  if (cudaMemcpyFromSymbol(counts, g_observe_n, sizeof(int) * 32) != cudaSuccess) return -1;
  return cudaMemcpyFromSymbol(host, g_observe, sizeof(long long) * 32 * OBS_PER) == cudaSuccess ? 32 * OBS_PER : -1;
}
#endif
#ifdef RC_TRACE
extern "C" __attribute__((visibility("default"))) int recache_debug_trace(long long* host, int n) {
  const int m = TR_ROLES * TR_ITEMS * 16;
  if (n < m) return -m;
  return cudaMemcpyFromSymbol(host, g_trace, sizeof(long long) * m) == cudaSuccess ? m : -1;
}
#endif

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
  return 256 + align256(tc_max_items(ctx, n_seq, total) * 8) + align256((int64_t)(n_seq + 1) * 4) + align256(SORT_MAX * 4);
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
  int32_t* order = (int32_t*)(ws + 256 + align256(max_items * 8) + align256((int64_t)(a.n_seq + 1) * 4));

  CUtensorMap tq, tks, tvs, tkr, tvr;
  const uint64_t self_total = (uint64_t)G * (uint64_t)a.self_rows;
  // TMA coordinates are 32-bit row indices
  if (self_total + TILE_N > 0x7fffffffull || (uint64_t)a.route_rows + TILE_N > 0x7fffffffull) return cudaErrorInvalidValue;
  if (!map_q(&tq, a.q, (uint64_t)a.total, Hq, s) || !map_rows(&tks, a.k_self, self_total) ||
      !map_rows(&tvs, a.v_self, self_total))
    return cudaErrorInvalidValue;
  const bool has_route = (a.route_cu != nullptr || a.prefix_len > 0) && a.route_rows > 0 && a.route_idx == nullptr;
  if (!map_rows(&tkr, has_route ? a.k_route : a.k_self, has_route ? (uint64_t)a.route_rows : self_total) ||
      !map_rows(&tvr, has_route ? a.v_route : a.v_self, has_route ? (uint64_t)a.route_rows : self_total))
    return cudaErrorInvalidValue;

  TcParams p;
  p.items = items; p.header = header; p.cu = a.cu; p.pos0 = a.pos0; p.slot = a.slot; p.route_cu = a.route_cu;
  p.n_seq = a.n_seq; p.G = G; p.Hq = Hq; p.s = s; p.self_rows = a.self_rows; p.route_rows = a.route_rows; p.out = a.o;
  p.prefix_len = a.route_cu ? 0 : a.prefix_len;
  p.hist = a.hist;
  p.cos_tab = ctx->cos_tab; p.sin_tab = ctx->sin_tab; p.max_pos = ctx->desc.max_pos;
  p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)ctx->desc.head_dim));
  p.status = ctx->status;
  p.order = order;
  const bool gather = a.route_idx != nullptr;
  p.gather_k = (const uint8_t*)a.k_cache; p.gather_v = (const uint8_t*)a.v_cache; p.route_idx = a.route_idx;
  p.pool_tokens = a.pool_tokens;
  {
    // The work list only depends on the index arrays: when the caller marked a fork point before the
    // rotate-and-store pass, it is built on the side stream beside that pass.
    const bool fork = ctx->forked && cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) == cudaSuccess;
    ctx->forked = false;
    cudaStream_t ps = fork ? ctx->side : st;
    {
      RcLaunchScope scope(ctx, RC_K_TILE_PLAN, ps);
      tile_plan_kernel<<<1, 1024, 0, ps>>>(p, tc_tok_per_cta(ctx), n_levels, items, level_off, order, (int)max_items);
    }
    if (fork && (cudaEventRecord(ctx->ev_join, ctx->side) != cudaSuccess ||
                 cudaStreamWaitEvent(st, ctx->ev_join, 0) != cudaSuccess))
      return cudaErrorUnknown;
  }
  const int sms = ctx->sm_count > 0 ? ctx->sm_count : 148;
  const unsigned grid = (unsigned)(max_items * G < sms ? max_items * G : sms);
  RcLaunchScope scope(ctx, a.route_cu ? RC_K_PREFILL_ATTN : RC_K_ENCODE_ATTN, st);
  auto launch = [&](auto kernel) {
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SM_ALLOC);
    kernel<<<grid, NTHREADS, SM_ALLOC, st>>>(tq, tks, tvs, tkr, tvr, p);
  };
  const bool f32 = a.out_dtype == RECACHE_F32, rot = s >= 4;   // 2 * 128 / s <= 64 positions fit the staging area
  if (gather) {
    if (f32) { if (rot) launch(attn_tc_kernel<float, true, true>); else launch(attn_tc_kernel<float, false, true>); }
    else { if (rot) launch(attn_tc_kernel<__nv_bfloat16, true, true>); else launch(attn_tc_kernel<__nv_bfloat16, false, true>); }
  } else {
    if (f32) { if (rot) launch(attn_tc_kernel<float, true, false>); else launch(attn_tc_kernel<float, false, false>); }
    else { if (rot) launch(attn_tc_kernel<__nv_bfloat16, true, false>); else launch(attn_tc_kernel<__nv_bfloat16, false, false>); }
  }
  return cudaGetLastError();
}

