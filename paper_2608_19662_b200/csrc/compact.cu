// Route / keep-mask compaction: the request-local KV materialisation step.
//
// Three launches, all integer work plus byte copies:
//   1. count : kept[r]   = number of retained tokens of listed resource r
//   2. plan  : route lengths, their exclusive prefix (route_cu), the offset of
//              every visible resource inside its route, the page prefix and
//              the page table (one CTA; a few thousand integers)
//   3. gather: one CTA per (listed resource, group) that the route table marks
//              visible: stable stream compaction of the keep mask (one block
//              scan per 2048 tokens), the row indices, and 16-byte-vectorised
//              copies of the kept key and value rows into the packed or paged
//              destination, eight pieces in flight per thread.
// Order inside a route = request order, then ascending token (stable), so the
// indices are unique and can be compared bit for bit.
#include "common.cuh"

namespace {

constexpr int TPB = 256;

__device__ __forceinline__ int warp_incl_scan(int v, int lane) {
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, v, off);
    if (lane >= off) v += n;
  }
  return v;
}

// Block-wide exclusive scan of one int per thread; returns the exclusive prefix
// and writes the block total to *total.  `ws` holds blockDim/32 + 1 ints.
__device__ __forceinline__ int block_excl_scan(int v, int* ws, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int incl = warp_incl_scan(v, lane);
  __syncthreads();                      // ws may still be read from the previous call
  if (lane == 31) ws[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = lane < nw ? ws[lane] : 0;
    const int wi = warp_incl_scan(w, lane);
    if (lane < nw) ws[lane] = wi - w;
    if (lane == nw - 1) ws[nw] = wi;
  }
  __syncthreads();
  *total = ws[nw];
  return incl - v + ws[warp];
}

__global__ void __launch_bounds__(TPB) compact_count_kernel(
    const uint8_t* __restrict__ keep, const int32_t* __restrict__ res_slot,
    const int32_t* __restrict__ res_len, int total_listed, int64_t pool_tokens,
    int32_t* __restrict__ kept, int32_t* status) {
  __shared__ int red[TPB / 32];
  for (int r = blockIdx.x; r < total_listed; r += gridDim.x) {
    const int64_t s0 = res_slot[r];
    const int n = res_len[r];
    int cnt = 0;
    if (n < 0 || s0 < 0 || s0 + n > pool_tokens) {
      if (threadIdx.x == 0) rc_set_status(status, RECACHE_DEV_BAD_SLOT);
    } else {
      for (int j = threadIdx.x; j < n; j += TPB) cnt += keep[s0 + j] != 0;
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) {
      int s = 0;
      for (int w = 0; w < TPB / 32; ++w) s += red[w];
      kept[r] = s;
    }
  }
}

__global__ void __launch_bounds__(1024) compact_plan_kernel(
    const int32_t* __restrict__ kept, const int32_t* __restrict__ res_off, int n_requests,
    int total_listed, const uint8_t* __restrict__ vis, int G, int mode, int page_tokens,
    int32_t* __restrict__ route_cu, int32_t* __restrict__ route_len_out,
    int32_t* __restrict__ res_route_off,   // [G][total_listed]
    int32_t* __restrict__ page_cu,         // [n_routes + 1]
    int64_t row_capacity, int32_t* __restrict__ page_table, int max_pages_per_route,
    const int32_t* __restrict__ free_pages, int64_t n_free_pages, int64_t n_pool_pages,
    int32_t* status) {
  __shared__ int ws[1024 / 32 + 1];
  __shared__ int wlen_sh[32];
  __shared__ int carry_rows, carry_pages;
  const int n_routes = n_requests * G;
  const bool warp_per_route = n_routes <= 32;
  if (threadIdx.x == 0) { carry_rows = 0; carry_pages = 0; }
  __syncthreads();
  for (int r0 = 0; r0 < n_routes; r0 += blockDim.x) {
    const int route = r0 + threadIdx.x;
    int len = 0;
    if (route < n_routes) {
      const int b = route / G, g = route % G;
      const int a = res_off[b], e = res_off[b + 1];
      if (a < 0 || e < a || e > total_listed) {
        rc_set_status(status, RECACHE_DEV_BAD_SEQLENS);
      } else if (!warp_per_route) {
        for (int r = a; r < e; ++r) {
          res_route_off[(int64_t)g * total_listed + r] = len;
          if (vis[(int64_t)g * total_listed + r]) len += kept[r];
        }
      }
    }
    if (warp_per_route) {
      // few routes, many resources each (a prefill): warp w walks route w's list 32 resources at a
      // time (independent loads, one warp scan per chunk), then hands the length to thread w
      const int lane = threadIdx.x & 31, wr = r0 + (threadIdx.x >> 5);
      int wlen = 0;
      if (wr < n_routes) {
        const int b = wr / G, g = wr % G;
        const int a = res_off[b], e = res_off[b + 1];
        if (a >= 0 && e >= a && e <= total_listed) {
          for (int c0 = a; c0 < e; c0 += 32) {
            const int r = c0 + lane;
            int v = 0;
            if (r < e && vis[(int64_t)g * total_listed + r]) v = kept[r];
            int incl = v;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
              const int u = __shfl_up_sync(0xffffffffu, incl, off);
              if (lane >= off) incl += u;
            }
            if (r < e) res_route_off[(int64_t)g * total_listed + r] = wlen + incl - v;
            wlen += __shfl_sync(0xffffffffu, incl, 31);
          }
        }
      }
      if (lane == 0) wlen_sh[threadIdx.x >> 5] = wlen;
      __syncthreads();
      if (route < n_routes && threadIdx.x < 32) len = wlen_sh[threadIdx.x];
      __syncthreads();
    }
    const int pages = (mode == RECACHE_PAGED) ? (len + page_tokens - 1) / page_tokens : 0;
    int tot_rows, tot_pages;
    const int ex_rows = block_excl_scan(len, ws, &tot_rows);
    const int ex_pages = block_excl_scan(pages, ws, &tot_pages);
    const int base_rows = carry_rows, base_pages = carry_pages;
    if (route < n_routes) {
      route_cu[route] = base_rows + ex_rows;
      if (route_len_out) route_len_out[route] = len;
      page_cu[route] = base_pages + ex_pages;
      if (mode == RECACHE_PAGED) {
        if (pages > max_pages_per_route) rc_set_status(status, RECACHE_DEV_BAD_PAGE);
        for (int p = 0; p < max_pages_per_route; ++p) {
          int id = -1;
          const int64_t fi = (int64_t)base_pages + ex_pages + p;
          if (p < pages && fi < n_free_pages) {
            id = free_pages[fi];
            if (id < 0 || id >= n_pool_pages) { rc_set_status(status, RECACHE_DEV_BAD_PAGE); id = -1; }
          }
          page_table[(int64_t)route * max_pages_per_route + p] = id;
        }
      }
    }
    __syncthreads();
    if (threadIdx.x == 0) { carry_rows = base_rows + tot_rows; carry_pages = base_pages + tot_pages; }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    route_cu[n_routes] = carry_rows;
    page_cu[n_routes] = carry_pages;
    if (carry_rows > row_capacity) rc_set_status(status, RECACHE_DEV_OVERFLOW);
    if (mode == RECACHE_PAGED && carry_pages > n_free_pages) rc_set_status(status, RECACHE_DEV_NO_PAGES);
  }
}

constexpr int TOK_PER_THREAD = 8;
constexpr int SUPER = TPB * TOK_PER_THREAD;   // tokens scanned per pass (2048)

// One CTA per (listed resource, group) that the route table marks visible.
// Pass = up to 2048 tokens: every thread reads 8 mask bytes, one block scan ranks
// the kept tokens, their (source row, destination row) pairs go to shared memory,
// and then all threads stream the rows with eight 16-byte pieces in flight each.
__global__ void __launch_bounds__(TPB) compact_gather_kernel(
    const uint8_t* __restrict__ k_cache, const uint8_t* __restrict__ v_cache, int64_t pool_tokens,
    const uint8_t* __restrict__ keep, const int32_t* __restrict__ res_off,
    const int32_t* __restrict__ res_slot, const int32_t* __restrict__ res_len, int n_requests,
    int total_listed, const uint8_t* __restrict__ vis, int G, int mode, int page_tokens,
    const int32_t* __restrict__ route_cu, const int32_t* __restrict__ res_route_off,
    const int32_t* __restrict__ page_cu, int32_t* __restrict__ route_idx, int64_t row_capacity,
    uint8_t* __restrict__ k_out, uint8_t* __restrict__ v_out, const int32_t* __restrict__ free_pages,
    int64_t n_free_pages, int64_t n_pool_pages, int row_bytes) {
  __shared__ int ws[TPB / 32 + 1];
  __shared__ int32_t src_tok[SUPER];   // token offset (inside the resource) of the pass's n-th kept token
  __shared__ int32_t dst_row[SUPER];   // destination row (packed row, or page * page_tokens + slot); -1 = skip
  const int r = blockIdx.x, g = blockIdx.y;
  if (!vis[(int64_t)g * total_listed + r]) return;
  const int64_t s0 = res_slot[r];
  const int n = res_len[r];
  if (n <= 0 || s0 < 0 || s0 + n > pool_tokens) return;   // flagged by the count kernel
  const int b = rc_find_segment(res_off, n_requests, r);
  const int route = b * G + g;
  const int in_route = res_route_off[(int64_t)g * total_listed + r];
  const int64_t route_base = route_cu[route];
  const int64_t page_base = page_cu[route];
  const int segs = row_bytes / 16;
  const uint8_t* kc = k_cache + ((int64_t)g * pool_tokens + s0) * row_bytes;
  const uint8_t* vc = v_cache + ((int64_t)g * pool_tokens + s0) * row_bytes;

  int run = 0;
  for (int j0 = 0; j0 < n; j0 += SUPER) {
    const int jt = j0 + threadIdx.x * TOK_PER_THREAD;
    uint32_t flags = 0;
#pragma unroll
    for (int u = 0; u < TOK_PER_THREAD; ++u)
      if (jt + u < n && keep[s0 + jt + u] != 0) flags |= 1u << u;
    int tot;
    int rank = in_route + run + block_excl_scan(__popc(flags), ws, &tot);   // row inside the route
    const int list0 = rank - in_route - run;
    int k = 0;
#pragma unroll
    for (int u = 0; u < TOK_PER_THREAD; ++u) {
      if (flags & (1u << u)) {
        const int64_t packed = route_base + rank;
        if (packed < row_capacity && blockIdx.z == 0) route_idx[packed] = (int32_t)(s0 + jt + u);
        int64_t dst = -1;
        if (mode == RECACHE_PACKED) {
          if (packed < row_capacity) dst = packed;
        } else {
          const int64_t fi = page_base + rank / page_tokens;
          if (fi < n_free_pages) {
            const int pg = free_pages[fi];
            if (pg >= 0 && pg < n_pool_pages) dst = (int64_t)pg * page_tokens + rank % page_tokens;
          }
        }
        src_tok[list0 + k] = jt + u;
        dst_row[list0 + k] = (int32_t)dst;
        ++k; ++rank;
      }
    }
    __syncthreads();
    // with few (resource, group) pairs the copy is shared by gridDim.z CTAs that all ran the (cheap) scan
    const int n_piece = k_out ? tot * segs : 0;   // index-only compaction moves no rows
    for (int e0 = threadIdx.x + blockIdx.z * TPB * 4; e0 < n_piece; e0 += TPB * 4 * gridDim.z) {
      uint4 kx[4], vx[4];
      int64_t dof[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = e0 + u * TPB;
        dof[u] = -1;
        if (e < n_piece) {
          const int rr = e / segs, sg = e - rr * segs;
          const int d = dst_row[rr];
          if (d >= 0) {
            const int64_t so = (int64_t)src_tok[rr] * row_bytes + sg * 16;
            dof[u] = (int64_t)d * row_bytes + sg * 16;
            kx[u] = *reinterpret_cast<const uint4*>(kc + so);
            vx[u] = *reinterpret_cast<const uint4*>(vc + so);
          }
        }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        if (dof[u] >= 0) {
          *reinterpret_cast<uint4*>(k_out + dof[u]) = kx[u];
          *reinterpret_cast<uint4*>(v_out + dof[u]) = vx[u];
        }
      }
    }
    run += tot;
    __syncthreads();
  }
}

struct Ws { int32_t* kept; int32_t* res_route_off; int32_t* page_cu; };
__host__ int64_t align256(int64_t x) { return (x + 255) & ~(int64_t)255; }

Ws carve(void* base, int n_routes, int total_listed, int G) {
  uint8_t* p = (uint8_t*)base;
  Ws w;
  w.kept = (int32_t*)p; p += align256((int64_t)total_listed * 4 + 4);
  w.res_route_off = (int32_t*)p; p += align256((int64_t)total_listed * G * 4 + 4);
  w.page_cu = (int32_t*)p;
  return w;
}

}  // namespace

int64_t rc_compact_workspace_bytes(const recache_ctx* ctx, int n_requests, int total_listed) {
  const int G = ctx->desc.n_kv_heads;
  return align256((int64_t)total_listed * 4 + 4) + align256((int64_t)total_listed * G * 4 + 4) +
         align256(((int64_t)n_requests * G + 1) * 4);
}

cudaError_t rc_launch_compact(const recache_ctx* ctx, const CompactArgs& a, cudaStream_t st) {
  const int G = ctx->desc.n_kv_heads, d = ctx->desc.head_dim;
  const int n_routes = a.n_requests * G;
  const int row_bytes = d * (ctx->desc.dtype == RECACHE_BF16 ? 2 : 4);
  Ws w = carve(a.workspace, n_routes, a.total_listed, G);
  if (a.total_listed > 0) {
    const int blocks = a.total_listed < 4096 ? a.total_listed : 4096;
    RcLaunchScope scope(ctx, RC_K_COMPACT_COUNT, st);
    compact_count_kernel<<<blocks, TPB, 0, st>>>(a.keep, a.res_slot, a.res_len, a.total_listed,
                                                 a.pool_tokens, w.kept, ctx->status);
  }
  {
    RcLaunchScope scope(ctx, RC_K_COMPACT_PLAN, st);
    compact_plan_kernel<<<1, 1024, 0, st>>>(w.kept, a.res_off, a.n_requests, a.total_listed, a.vis, G, a.mode,
                                            ctx->desc.page_tokens, a.route_cu, a.route_len, w.res_route_off,
                                            w.page_cu, a.row_capacity, a.page_table, a.max_pages_per_route,
                                            a.free_pages, a.n_free_pages, a.n_pool_pages, ctx->status);
  }
  if (a.total_listed > 0) {
    const int64_t pairs = (int64_t)a.total_listed * G;
    const unsigned z = (unsigned)(pairs >= 2048 ? 1 : (2048 + pairs - 1) / pairs > 8 ? 8 : (2048 + pairs - 1) / pairs);
    dim3 grid((unsigned)a.total_listed, (unsigned)G, z);
    RcLaunchScope scope(ctx, RC_K_COMPACT_GATHER, st);
    compact_gather_kernel<<<grid, TPB, 0, st>>>(
        (const uint8_t*)a.k_cache, (const uint8_t*)a.v_cache, a.pool_tokens, a.keep, a.res_off, a.res_slot,
        a.res_len, a.n_requests, a.total_listed, a.vis, G, a.mode, ctx->desc.page_tokens, a.route_cu,
        w.res_route_off, w.page_cu, a.route_idx, a.row_capacity, (uint8_t*)a.k_out, (uint8_t*)a.v_out,
        a.free_pages, a.n_free_pages, a.n_pool_pages, row_bytes);
  }
  return cudaGetLastError();
}
