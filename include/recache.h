/*
 * recache.h - C ABI of the resource-routed attention library (sm_100a).
 *
 * The four hot-path calls follow the problem statement of the ReCache paper
 * (section "ReCache"): resources are encoded one by one with positions that
 * restart inside each resource ("Resource-Wise Attention"); at request time the
 * conversation sees, on every (layer, KV-head-group) route, only the resources
 * that route exposes ("Structural Pruning", masks M_resource / M_context) and
 * only their retained token fields ("Semantic Pruning"); the gather of those
 * rows is the request-local materialisation of KV that the paper counts inside TTFT
 * (section "Evaluation Metrics", paragraph "Efficiency").
 *
 * Conventions that hold for every call
 *  - Every tensor pointer is CALLER-OWNED DEVICE memory of the context's dtype
 *    (float or bfloat16) unless the comment says otherwise.  The library keeps
 *    no pointer past the call and frees nothing it was given.
 *  - int32 index arrays (cu_seqlens, slots, tables ...) are DEVICE pointers.
 *    Plain int arguments are host values: exact sizes or upper bounds used to
 *    size launches.
 *  - `stream` is a cudaStream_t passed as void*.  Calls enqueue work and return
 *    without synchronising.
 *  - `workspace` is caller-owned device scratch of at least the number of bytes
 *    the matching recache_*_workspace_bytes() query returns (256-byte aligned).
 *    Its contents are undefined after the call.
 *  - Return value: RECACHE_OK, or an error detected on the host BEFORE any
 *    launch (null pointer, unsupported shape, capacity too small, CUDA launch
 *    failure).  recache_last_error() gives the text.
 *  - Errors only the device can see (an index outside its buffer, a position
 *    past the rotary table, a route longer than the capacity given) never trap:
 *    the offending access is skipped and a code is stored in the context's
 *    device status word, read (and cleared) by recache_poll_status().
 *
 * Layouts (d = head_dim, G = n_kv_heads, Hq = n_q_heads, s = Hq / G; query head
 * h reads KV group h / s)
 *  - token-major activations:  q [tokens][Hq][d];  k, v [tokens][G][d]
 *  - resource cache (one layer): k_cache, v_cache [G][pool_tokens][d]; resource
 *    i occupies rows dst_slot[i] .. dst_slot[i] + D_i - 1 of every group
 *  - packed route KV: [rows][d]; route r = request * G + group owns rows
 *    route_cu[r] .. route_cu[r+1]-1
 *  - paged KV: k_pages, v_pages [n_pages][page_tokens][d]; a page belongs to
 *    one (sequence, group) item
 *  - rotary embedding pairs element i with i + d/2; angle = pos * theta^(-2i/d)
 */
#ifndef RECACHE_H
#define RECACHE_H

#include <stdint.h>

#if defined(__GNUC__)
#define RECACHE_API __attribute__((visibility("default")))
#else
#define RECACHE_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RECACHE_OK = 0,
  RECACHE_EINVAL = 1,       /* null pointer, negative size, bad enum */
  RECACHE_ESHAPE = 2,       /* head counts / head_dim / sizes inconsistent */
  RECACHE_EUNSUPPORTED = 3, /* valid but not implemented for this dtype/shape */
  RECACHE_ENOMEM = 4,       /* workspace or capacity too small, allocation failed */
  RECACHE_ECUDA = 5         /* a CUDA runtime/driver call failed */
} recache_status;

enum { RECACHE_F32 = 0, RECACHE_BF16 = 1 };
enum { RECACHE_PACKED = 0, RECACHE_PAGED = 1 };

/* Codes stored in the device status word (first error wins). */
enum {
  RECACHE_DEV_OK = 0,
  RECACHE_DEV_BAD_SEQLENS = 1,  /* cu_seqlens / cu_q not monotone or past total */
  RECACHE_DEV_BAD_SLOT = 2,     /* cache row outside [0, pool_tokens) */
  RECACHE_DEV_OVERFLOW = 3,     /* route rows exceed row_capacity */
  RECACHE_DEV_BAD_PAGE = 4,     /* page id outside [0, n_pages) or table too short */
  RECACHE_DEV_NO_PAGES = 5,     /* free page list exhausted */
  RECACHE_DEV_BAD_POS = 6,      /* position outside [0, max_pos) */
  RECACHE_DEV_TIMEOUT = 7       /* a kernel gave up waiting on one of its own barriers */
};

typedef struct recache_ctx recache_ctx;

typedef struct {
  int32_t n_q_heads;   /* Hq */
  int32_t n_kv_heads;  /* G; Hq % G == 0, Hq / G <= 8 */
  int32_t head_dim;    /* 64 or 128 */
  int32_t dtype;       /* RECACHE_F32 or RECACHE_BF16: storage of q/k/v/caches */
  int32_t max_pos;     /* rotary table rows: every position must be < max_pos */
  int32_t page_tokens; /* tokens per KV page (64) */
  double rope_theta;
} recache_desc;

/* Creates a context on `device`: builds the cos/sin table (computed in double on
 * the host, stored as float, max_pos * head_dim * 4 bytes on the device) and the
 * device status word.  The only call that allocates device memory. */
RECACHE_API recache_status recache_create(recache_ctx** out, const recache_desc* desc, int device);
RECACHE_API void recache_destroy(recache_ctx* ctx);
/* Text of the last host-side error of this context ("" if none). Host pointer,
 * owned by the context. */
RECACHE_API const char* recache_last_error(const recache_ctx* ctx);
/* Synchronises `stream`, returns the device status word in *device_code and
 * clears it.  After RECACHE_DEV_TIMEOUT, recache_last_error() names the kernel
 * (and, for the split-KV decode kernel, the block, barrier and warp that gave up first). */
RECACHE_API recache_status recache_poll_status(recache_ctx* ctx, void* stream, int32_t* device_code);

/* Self-test of the failure path (no paper counterpart).  Every barrier wait inside the TMA kernels
 * is bounded: a wait that runs out sets RECACHE_DEV_TIMEOUT, releases the CTA's other waits, lets
 * the copies in flight land and the kernel end normally.  This call enqueues one small CTA that
 * runs exactly that code (the same wait and drain helpers, probe bound 2^10, about a millisecond)
 * on a barrier nobody arrives at.  report: DEVICE pointer to two int32: [0] = 1 if the wait gave
 * up, [1] = thousands of SM cycles it waited.  Afterwards recache_poll_status() returns
 * RECACHE_DEV_TIMEOUT once and recache_last_error() names the self-test; the context stays usable.
 * Nothing hangs or faults. */
RECACHE_API recache_status recache_selftest_wait_timeout(recache_ctx* ctx, int32_t* report, void* stream);

/*
 * Launch accounting.  The library counts every kernel it launches; with the
 * timer enabled it also records a CUDA event pair around each launch on the
 * launch stream (a few microseconds of host time per launch).
 *   recache_kernel_count()      number of distinct kernels K
 *   recache_kernel_name(id)     static string, id in [0, K)
 *   recache_kernel_timer(ctx,e) 0 = off, 1 = every launch, 2 = the two attention launches only (light
 *       enough to leave on inside a timed region); clears counters and pending events.
 *       With 0 or 2 the small set-up kernel of the tensor-core attention runs on a
 *       second stream of the context beside the call's first kernel (forked from and
 *       joined to the caller's stream by events); with 1 everything stays on one stream.
 *   recache_kernel_times(ctx, ms_total[K], launches[K])  waits for the recorded
 *       events, returns per-kernel summed device time in ms (0 when the timer
 *       was off) and launch counts since the last clear, then clears both.
 * Host arrays; no paper counterpart (measurement aid).
 */
RECACHE_API int32_t recache_kernel_count(void);
RECACHE_API const char* recache_kernel_name(int32_t id);
RECACHE_API recache_status recache_kernel_timer(recache_ctx* ctx, int32_t enable);
RECACHE_API recache_status recache_kernel_times(recache_ctx* ctx, float* ms_total, int64_t* launches);

/* Scratch sizes in bytes for the calls below (same size arguments). */
RECACHE_API int64_t recache_encode_workspace_bytes(const recache_ctx* ctx, int32_t n_resources,
                                       int32_t total_tokens, int32_t max_len);
RECACHE_API int64_t recache_compact_workspace_bytes(const recache_ctx* ctx, int32_t n_requests,
                                        int32_t total_listed);
RECACHE_API int64_t recache_prefill_workspace_bytes(const recache_ctx* ctx, int32_t n_requests,
                                        int32_t total_q, int32_t max_q);
RECACHE_API int64_t recache_decode_workspace_bytes(const recache_ctx* ctx, int32_t batch,
                                       int32_t max_res_pages, int32_t max_hist_pages);

/*
 * Resource-wise encoding (paper: "Resource-Wise Attention"; figure panel (a)).
 * N resources are packed back to back; resource i is rows cu_seqlens[i] ..
 * cu_seqlens[i+1]-1 and its token j has position j (0-based).  For every token
 * j of resource i and query head h:
 *     o[i,j,h] = sum_{j' <= j} softmax_j'( rope(q,j) . rope(k,j') / sqrt(d) ) v[j']
 * with keys/values of the same resource only.  The rotated keys and the values
 * are written to the cache rows dst_slot[i] + j.  Nothing computed for a
 * resource depends on the other resources of the batch, their order or the
 * launch: outputs and cache rows are bit-identical across compositions.
 *   q [T][Hq][d], k/v [T][G][d] pre-rotation;  T = total_tokens (exact);
 *   max_len >= every D_i;  dst_slot [N];  caches [G][pool_tokens][d];
 *   out_o [T][Hq][d] of out_dtype (RECACHE_F32 or the context dtype).
 * Empty resources (D_i = 0) are allowed.
 */
RECACHE_API recache_status recache_encode_resources(recache_ctx* ctx,
    const void* q, const void* k, const void* v,
    const int32_t* cu_seqlens, int32_t n_resources, int32_t total_tokens, int32_t max_len,
    const int32_t* dst_slot, void* k_cache, void* v_cache, int64_t pool_tokens,
    void* out_o, int32_t out_dtype,
    void* workspace, int64_t workspace_bytes, void* stream);

/*
 * Encoding variants of the paper's ablation (section "Cache Reuse"): resources
 * encoded behind a prefix they all share, and the Block configuration, which
 * has no attention between resources but leaves every token at its global position.
 * Same as recache_encode_resources, plus
 *   k_prefix / v_prefix [G][prefix_len][d]: rotated keys and values of a shared
 *       prefix, as a cache holds them (e.g. written by an earlier encode call);
 *       every resource token also attends to all of them (the shared-prefix form
 *       of section "Resource-Wise Attention").  NULL / 0: no prefix.
 *   pos_offset [N] (device, may be NULL = all 0): position of each resource's
 *       first token.  One common value P = the resource-local layout behind a
 *       prefix of P tokens (still composition-independent); global offsets = the
 *       "Block" variant.  Positions pos_offset[i] + D_i must stay below max_pos.
 * The cache receives keys rotated at those positions.
 */
RECACHE_API recache_status recache_encode_resources_prefixed(recache_ctx* ctx,
    const void* q, const void* k, const void* v,
    const int32_t* cu_seqlens, int32_t n_resources, int32_t total_tokens, int32_t max_len,
    const int32_t* dst_slot, void* k_cache, void* v_cache, int64_t pool_tokens,
    const void* k_prefix, const void* v_prefix, int32_t prefix_len, const int32_t* pos_offset,
    void* out_o, int32_t out_dtype,
    void* workspace, int64_t workspace_bytes, void* stream);

/*
 * Route / keep-mask compaction = request-local KV materialisation (paper:
 * "Structural Pruning", "Semantic Pruning", and the TTFT definition).
 * Request b lists resources res_off[b] .. res_off[b+1]-1 (entries of res_slot /
 * res_len, in request order).  Route r = b * G + g exposes, in this order, the
 * listed resources with vis[g][listed index] != 0, and of each the cache rows
 * slot + j (j ascending) with keep[slot + j] != 0.
 *   keep [pool_tokens] uint8;  vis [G][total_listed] uint8 (this layer's routes)
 * Outputs
 *   route_cu  [B*G+1]  exclusive prefix of route lengths
 *   route_len [B*G]    (optional, may be NULL) the lengths themselves
 *   route_idx [row_capacity] cache row of every compacted row, packed order
 *   mode RECACHE_PACKED: k_out/v_out [row_capacity][d] packed route KV; both may be
 *        NULL: indices and prefix only, no row is copied (see recache_attend_decode_gather)
 *   mode RECACHE_PAGED : k_out/v_out are page pools [n_pool_pages][page_tokens][d];
 *        route r takes ceil(len_r / page_tokens) consecutive entries of
 *        free_pages [n_free_pages], starting where route r-1 stopped; row n of
 *        the route goes to page_table[r][n / page_tokens], slot n % page_tokens;
 *        page_table [B*G][max_pages_per_route] is padded with -1.
 * Indices are exact (stable order); gathered rows are byte copies.  A route with
 * no visible resource or no kept token has length 0.
 */
RECACHE_API recache_status recache_compact_routes(recache_ctx* ctx,
    const void* k_cache, const void* v_cache, int64_t pool_tokens,
    const uint8_t* keep,
    const int32_t* res_off, const int32_t* res_slot, const int32_t* res_len,
    int32_t n_requests, int32_t total_listed,
    const uint8_t* vis, int32_t mode,
    int32_t* route_cu, int32_t* route_len, int32_t* route_idx, int64_t row_capacity,
    void* k_out, void* v_out,
    int32_t* page_table, int32_t max_pages_per_route,
    const int32_t* free_pages, int64_t n_free_pages, int64_t n_pool_pages,
    void* workspace, int64_t workspace_bytes, void* stream);

/*
 * Routed prefill (paper: final mask of the architecture figure; routes in Omega
 * use M_resource, the others M_context).  Query token t of request b has
 * position q_pos0[b] + t.  For head h in group g, ONE softmax (scale 1/sqrt(d))
 * runs over (i) all rows of route b*G+g in k_route/v_route (keys used as cached,
 * no causal restriction) and (ii) conversation tokens t' <= t of the same
 * request (keys rotated at their own positions).  A route of length 0 is plain
 * causal self-attention of the conversation.
 *   q [total_q][Hq][d], k_conv/v_conv [total_q][G][d] pre-rotation;
 *   cu_q [B+1], q_pos0 [B];  max_q >= every request's length;
 *   k_route/v_route packed [route_rows][d] with route_cu [B*G+1] (from compaction)
 * Outputs
 *   k_conv_out/v_conv_out [G][total_q][d]: rotated conversation keys / values,
 *       head-major (the rows a later decode step keeps as history); required
 *   out_o [total_q][Hq][d] of out_dtype.
 */
RECACHE_API recache_status recache_attend_prefill(recache_ctx* ctx,
    const void* q, const void* k_conv, const void* v_conv,
    const int32_t* cu_q, const int32_t* q_pos0,
    int32_t n_requests, int32_t total_q, int32_t max_q,
    const void* k_route, const void* v_route, const int32_t* route_cu, int64_t route_rows,
    void* k_conv_out, void* v_conv_out,
    void* out_o, int32_t out_dtype,
    void* workspace, int64_t workspace_bytes, void* stream);

/*
 * Routed prefill of a later turn (paper, problem setup: in a multi-turn
 * interaction the input also carries the turns that came before).
 * Same as recache_attend_prefill, with the conversation's rotated keys / values
 * kept in a cache [G][cache_rows][d]: request b owns rows conv_slot[b] ..., of
 * which the first hist_len[b] hold its earlier turns.  The new tokens attend to
 * (i) the route's rows, (ii) ALL hist_len[b] earlier rows, (iii) new tokens
 * t' <= t, in one softmax; their rotated keys / values are appended at rows
 * conv_slot[b] + hist_len[b] + t.  q_pos0[b] is the position of the first NEW
 * token.  With 64-aligned slots the cache doubles as the decode history pages
 * (page id = (g * cache_rows + conv_slot[b]) / 64 + n).
 */
RECACHE_API recache_status recache_attend_prefill_history(recache_ctx* ctx,
    const void* q, const void* k_conv, const void* v_conv,
    const int32_t* cu_q, const int32_t* q_pos0,
    int32_t n_requests, int32_t total_q, int32_t max_q,
    const void* k_route, const void* v_route, const int32_t* route_cu, int64_t route_rows,
    void* k_conv_cache, void* v_conv_cache, int64_t cache_rows,
    const int32_t* conv_slot, const int32_t* hist_len,
    void* out_o, int32_t out_dtype,
    void* workspace, int64_t workspace_bytes, void* stream);

/*
 * Routed prefill without materialising the route rows (zero-copy; the paper's
 * request-local KV materialisation replaced by an index list): route b*G+g is
 * rows route_idx[route_cu[r] .. route_cu[r+1]) of group g of the resource cache
 * k_cache / v_cache [G][pool_tokens][d] - what recache_compact_routes writes when
 * called with k_out = v_out = NULL in packed mode.  route_rows = entries of
 * route_idx.  Same mask, same softmax, same tiles as recache_attend_prefill on
 * the packed rows: the results are bit-identical to it.
 * bf16 contexts with head_dim 128 and 2, 4 or 8 query heads per KV head only
 * (RECACHE_EUNSUPPORTED otherwise).  An index outside [0, pool_tokens) sets the
 * device status (bad slot) and its row is read as zeros.
 */
RECACHE_API recache_status recache_attend_prefill_gather(recache_ctx* ctx,
    const void* q, const void* k_conv, const void* v_conv,
    const int32_t* cu_q, const int32_t* q_pos0,
    int32_t n_requests, int32_t total_q, int32_t max_q,
    const void* k_cache, const void* v_cache, int64_t pool_tokens,
    const int32_t* route_idx, const int32_t* route_cu, int64_t route_rows,
    void* k_conv_out, void* v_conv_out,
    void* out_o, int32_t out_dtype,
    void* workspace, int64_t workspace_bytes, void* stream);

/*
 * Routed decode (paper: the final mask also holds while decoding; the Attn. latency of
 * the efficiency study).  One query token per sequence at position q_pos[b].
 * Item it = b * G + g reads res_len[it] rows through res_page_table[it][*] and
 * hist_len[it] rows through hist_page_table[it][*] (row n lives in page
 * table[n / page_tokens], slot n % page_tokens); one softmax over both parts.
 * If k_new/v_new ([B][G][d], pre-rotation) are given, the current token's
 * rotated key and value are first written as history row hist_len[it]-1; pass
 * NULL when the caller has appended them already.  hist_len >= 1 always.
 *   q [B][Hq][d] pre-rotation;  out_o [B][Hq][d] of out_dtype.
 */
RECACHE_API recache_status recache_attend_decode(recache_ctx* ctx,
    const void* q, const int32_t* q_pos, int32_t batch,
    const void* k_new, const void* v_new,
    void* k_pages, void* v_pages, int64_t n_pages,
    const int32_t* res_page_table, int32_t max_res_pages, const int32_t* res_len,
    const int32_t* hist_page_table, int32_t max_hist_pages, const int32_t* hist_len,
    void* out_o, int32_t out_dtype,
    void* workspace, int64_t workspace_bytes, void* stream);

/*
 * Routed decode without materialising the resource rows (zero-copy): the
 * resource part of item it = b * G + g is read straight from the resource cache,
 * rows route_idx[route_cu[it] .. route_cu[it+1]) of group g - the index list that
 * recache_compact_routes writes (call it with k_out = v_out = NULL, packed mode,
 * to get the indices only: no key / value byte is moved, and requests that share
 * a resource share its cache rows).  History stays paged as in
 * recache_attend_decode; same softmax, same results.
 *   route_rows: number of entries of route_idx (an item whose route_cu range does
 *   not lie inside it is reported as RECACHE_DEV_OVERFLOW and read as an empty route);
 *   pool_tokens > 0;
 *   max_res_pages: upper bound of ceil(route length / page_tokens), used to size
 *   the split plan and the workspace (recache_decode_workspace_bytes).
 * bf16 contexts with head_dim 128 and 64-token pages only.
 */
RECACHE_API recache_status recache_attend_decode_gather(recache_ctx* ctx,
    const void* q, const int32_t* q_pos, int32_t batch,
    const void* k_new, const void* v_new,
    const void* k_cache, const void* v_cache, int64_t pool_tokens,
    const int32_t* route_idx, const int32_t* route_cu, int64_t route_rows, int32_t max_res_pages,
    void* k_pages, void* v_pages, int64_t n_pages,
    const int32_t* hist_page_table, int32_t max_hist_pages, const int32_t* hist_len,
    void* out_o, int32_t out_dtype,
    void* workspace, int64_t workspace_bytes, void* stream);

/*
 * Route table from contribution scores (paper: "Structural Pruning", the
 * weights w_i = max(s_i,0) / sum_j max(s_j,0), TopK and Omega* = L* x G*;
 * sparsity rho of "Structural Budget Analysis").  Host-only helper, all
 * pointers are HOST memory.
 *   s_layers [n_layers], s_groups [n_groups]: leave-one-in contributions (or
 *       already-normalised weights); negative values count as 0
 *   k_layers, k_groups: budgets K_L, K_G; ties go to the lower index
 *   omega [n_layers][n_groups] (out): 1 where route (l, g) exposes the resources;
 *       a layer's row, repeated over the request's resources, is that layer's
 *       `vis` table for recache_compact_routes
 *   cc_layers, cc_groups (out, optional): contribution coverage of the kept units
 *   rho (out, optional): 1 - K_L K_G / (L G)
 */
RECACHE_API recache_status recache_build_routes(const double* s_layers, int32_t n_layers,
    const double* s_groups, int32_t n_groups, int32_t k_layers, int32_t k_groups,
    uint8_t* omega, double* cc_layers, double* cc_groups, double* rho);

/*
 * Decode without any allocation.  (The paper has no counterpart: this is a
 * deployment variant of recache_attend_decode, same arguments minus the
 * workspace, same results.)
 *
 * Who needs it: callers that may not allocate device memory where they decode -
 * a serving loop that has frozen its memory plan, a plugin inside a host process
 * that owns all device memory, a latency-critical path that must not enter the
 * allocator.  The split-KV partials go to a 4 MiB scratch array that is part of
 * the library image on every GPU that loads it (held until the process exits),
 * so nothing is allocated or freed, here or in any library this call uses.
 *
 * Limits and rules
 *  - bf16 contexts with head_dim 128 and 64-token pages only (RECACHE_EUNSUPPORTED
 *    otherwise); the kernel timer must be off (it creates event objects).
 *  - batch * n_kv_heads * splits * heads-per-group * 520 bytes must fit in 4 MiB
 *    (e.g. batch 64 with 8 KV groups of 4 heads uses 2.1 MiB); beyond that the
 *    call returns RECACHE_ENOMEM with a message and launches nothing.
 *  - The first call on a device looks up the scratch array's device address
 *    (once per device, with that device current).  Make that first call outside
 *    any stream capture.
 *  - All calls on a device share the one array, which keeps the previous call's
 *    contents; every slot a call reads it has written first, so nothing needs
 *    clearing.  Two calls that overlap on the GPU (different streams) race on
 *    it: serialise them.
 */
RECACHE_API recache_status recache_attend_decode_noalloc(recache_ctx* ctx,
    const void* q, const int32_t* q_pos, int32_t batch,
    const void* k_new, const void* v_new,
    void* k_pages, void* v_pages, int64_t n_pages,
    const int32_t* res_page_table, int32_t max_res_pages, const int32_t* res_len,
    const int32_t* hist_page_table, int32_t max_hist_pages, const int32_t* hist_len,
    void* out_o, int32_t out_dtype, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RECACHE_H */
