// CSR SpMM kernels of the sat_b200 library (aggregation with the propagation matrix P),
// row gather and row scatter.  All of them are bandwidth-bound: every feature row is moved
// with 128-bit loads, one group of lanes per work item, warp shuffles broadcast the column
// ids, and nothing is accumulated with floating-point atomics (results are reproducible).
#include "sat_internal.h"

#include <algorithm>
#include <cstdlib>

__device__ __forceinline__ float4 ld4(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ void fma4(float4 &a, float w, const float4 &x)
{
    a.x = fmaf(w, x.x, a.x);
    a.y = fmaf(w, x.y, a.y);
    a.z = fmaf(w, x.z, a.z);
    a.w = fmaf(w, x.w, a.w);
}

// zero the components of float4 column `idx` of a row whose bits in the row's bit mask (word_base = row * words) are 0
__device__ __forceinline__ void mask4(float4 &r, const uint32_t *__restrict__ omask, int64_t word_base, int idx)
{
    const uint32_t m = __ldg(omask + word_base + (idx >> 3)) >> ((idx & 7) * 4);
    if (!(m & 1u)) r.x = 0.f;
    if (!(m & 2u)) r.y = 0.f;
    if (!(m & 4u)) r.z = 0.f;
    if (!(m & 8u)) r.w = 0.f;
}

template <int G>
__device__ __forceinline__ unsigned group_mask(int lane_in_warp)
{
    return G == 32 ? 0xffffffffu : (((1u << (G & 31)) - 1u) << (lane_in_warp & ~(G - 1)));
}

// -------------------------------------------------------------------------------------
// One group of G lanes per work item (a row, or a chunk of SAT_SPMM_CHUNK entries of a
// long row).  Lane l owns float4 columns l, l+G, ..., l+(NV-1)G of the feature row.
//   single-chunk rows write  out[row] = dinv[row] * sum_e dinv[col_e] * src[col_e]
//   chunks of long rows write their un-scaled partial sum to `partial`; k_spmm_fixup adds
//   them in chunk order.
// -------------------------------------------------------------------------------------
template <int G, int NV>
__global__ void __launch_bounds__(256, NV <= 2 ? 8 : 4)
k_spmm_items(const int64_t *__restrict__ lrowptr, const int32_t *__restrict__ inner_cnt, const int32_t *__restrict__ lenc,
             const float *__restrict__ lw, const float *__restrict__ dinv_enc, const int32_t *__restrict__ item_row, const int32_t *__restrict__ first_item,
             const int32_t *__restrict__ item_mslot, int32_t item0, int32_t n_items, int32_t mitem0, int inner_only, int32_t n,
             int32_t d4, const float *__restrict__ in_base, int64_t ld_in, const float *__restrict__ halo_base, int64_t ld_halo,
             float *__restrict__ out_base, int64_t ld_out, float *__restrict__ partial, const uint32_t *__restrict__ omask, int32_t omask_words,
             DbgLimits dbg)
{
    // (Several consecutive work items per lane group — fewer, longer-lived blocks — were measured: neutral on the large
    // workload, 40 % slower on the medium one, where the chunks of a hub row then land in one warp.)
    const int lane = threadIdx.x & (G - 1);
    const int64_t gid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    if (gid >= n_items) return;
    const unsigned mask = group_mask<G>(threadIdx.x & 31);
    const int col0 = blockIdx.y * (G * NV);  // first float4 column of this block column
    const int32_t item = item0 + (int32_t)gid;
    const int32_t row = (int32_t)SAT_IDX(item_row[item], dbg.out_lo, dbg.out_hi, dbg.status);
    const int32_t k = item - first_item[row];
    const int64_t rb = lrowptr[row];
    // inner_only: 0 = all entries, 1 = the inner prefix of the row, 2 = its halo suffix
    const int64_t re = inner_only == 1 ? rb + inner_cnt[row] : lrowptr[row + 1];
    int64_t e0 = rb + (int64_t)k * SAT_SPMM_CHUNK;
    const int64_t e1 = (e0 + SAT_SPMM_CHUNK < re) ? e0 + SAT_SPMM_CHUNK : re;
    if (inner_only == 2 && e0 < rb + inner_cnt[row]) e0 = rb + inner_cnt[row];
    float4 acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    // (Cheaper row addressing was measured twice and was slower both times: 32 x 32 -> 64-bit multiplies in float4 units for the
    // two matrices, and a single-matrix form — one multiply-add, no select — for launches whose columns all index one matrix
    // (inner-only, halo-only, a halo matrix right behind the inner one, both read from a matrix over all nodes).  Either way
    // the kernel executes a third fewer instructions and runs 4-10 % slower on every workload: it is bound by memory
    // latency and DRAM, not by instruction issue, and at 32 registers the leaner loop spills more.)
    for (int64_t eb = e0; eb < e1; eb += G) {
        const int64_t e = eb + lane;
        int32_t c = 0;
        float w = 0.f;
        if (e < e1) {
            c = __ldg(lenc + e);
            w = __ldg(lw + e);
        }
        const int cnt = (e1 - eb) < G ? (int)(e1 - eb) : G;
#pragma unroll 4
        for (int j = 0; j < cnt; ++j) {
            const int32_t cj = __shfl_sync(mask, c, j, G);
            const float wj = __shfl_sync(mask, w, j, G);
            const float *src = cj < n ? in_base + SAT_IDX((int64_t)cj, dbg.src_lo, dbg.src_hi, dbg.status) * ld_in
                                      : halo_base + SAT_IDX((int64_t)(cj - n), dbg.halo_lo, dbg.halo_hi, dbg.status) * ld_halo;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int idx = col0 + lane + v * G;
                if (idx < d4) fma4(acc[v], wj, ld4(src + 4 * idx));
            }
        }
    }
    const int32_t ms = item_mslot[item];
    if (ms < 0) {
        const float s = __ldg(dinv_enc + row);
        float *o = out_base + (int64_t)row * ld_out;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int idx = col0 + lane + v * G;
            if (idx < d4) {
                float4 r = make_float4(s * acc[v].x, s * acc[v].y, s * acc[v].z, s * acc[v].w);
                if (omask) mask4(r, omask, (int64_t)row * omask_words, idx);
                *reinterpret_cast<float4 *>(o + 4 * idx) = r;
            }
        }
    } else {
        float *o = partial + (int64_t)(ms - mitem0) * (4 * (int64_t)d4);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int idx = col0 + lane + v * G;
            if (idx < d4) *reinterpret_cast<float4 *>(o + 4 * idx) = acc[v];
        }
    }
}

// rows cut into several chunks: add the partial sums in chunk order, scale, store
__global__ void k_spmm_fixup(const int32_t *__restrict__ mrows, int32_t mrow0, int32_t n_mrows, const int32_t *__restrict__ first_item,
                             const int32_t *__restrict__ item_mslot, int32_t mitem0, const float *__restrict__ dinv_enc, int32_t d4,
                             const float *__restrict__ partial, float *__restrict__ out_base, int64_t ld_out,
                             const uint32_t *__restrict__ omask, int32_t omask_words, DbgLimits dbg)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d4;
    const int c = (int)(t - i * d4);
    if (i >= n_mrows) return;
    const int32_t row = (int32_t)SAT_IDX(mrows[mrow0 + i], dbg.out_lo, dbg.out_hi, dbg.status);
    const int32_t it0 = first_item[row], it1 = first_item[row + 1];
    const int32_t ms0 = item_mslot[it0] - mitem0;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int32_t q = 0; q < it1 - it0; ++q) {
        const float4 x = *reinterpret_cast<const float4 *>(partial + ((int64_t)(ms0 + q) * d4 + c) * 4);
        a.x += x.x;
        a.y += x.y;
        a.z += x.z;
        a.w += x.w;
    }
    const float s = dinv_enc[row];
    float4 r = make_float4(s * a.x, s * a.y, s * a.z, s * a.w);
    if (omask) mask4(r, omask, (int64_t)row * omask_words, c);
    *reinterpret_cast<float4 *>(out_base + (int64_t)row * ld_out + 4 * c) = r;
}

// -------------------------------------------------------------------------------------
// Source-blocked forward SpMM.  When the sources of a partition (inner + halo rows) are several times the L2, a row-major
// walk re-reads most of them from DRAM: every source row is used by ~10-20 rows spread over the whole partition and is
// evicted between two uses.  The blocked work list walks the partition once per block of sources instead (the entries of a
// row are sorted by source, so a row meets a block in one contiguous run); the rows gathered at any one time then belong to
// one or two blocks, which the L2 holds.  The price is one partial sum per (row, block) and the pass that adds them.
// -------------------------------------------------------------------------------------
__device__ __forceinline__ int64_t lower_bound_col(const int32_t *__restrict__ lenc, int64_t lo, int64_t hi, int64_t key)
{
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if ((int64_t)lenc[mid] < key) lo = mid + 1;
        else hi = mid;
    }
    return lo;
}

// encoded column of source p of a partition whose sources are [n_rows inner rows from row0 ; halo rows from halo0]
__device__ __forceinline__ int64_t sb_source_col(int64_t p, int32_t row0, int32_t n_rows, int32_t n, int64_t halo0)
{
    return p < n_rows ? (int64_t)row0 + p : (int64_t)n + halo0 + (p - n_rows);
}

// The run of entries [lo, hi) of `row` that is walked with block j, or an empty run.  A row of `len` entries is cut into
// G = min(blocks, len / min_run) groups of consecutive blocks (a short row would otherwise leave a partial sum per block for
// a handful of entries each): group g covers blocks [ceil(g B / G), ceil((g + 1) B / G)) and its run is walked with the
// first of them.
__device__ __forceinline__ void sb_run(const int64_t *__restrict__ lrowptr, const int32_t *__restrict__ lenc,
                                       const int32_t *__restrict__ inner_cnt, int32_t row, int32_t j, int32_t n_blocks, int64_t block_rows,
                                       int32_t min_run, int32_t row0, int32_t n_rows, int32_t n, int64_t halo0, int64_t *lo, int64_t *hi)
{
    // inner_cnt given: the list covers the inner prefix of every row only (the backward product P_in^T)
    const int64_t rb = lrowptr[row], re = inner_cnt ? rb + inner_cnt[row] : lrowptr[row + 1];
    int64_t G = min_run > 0 ? (re - rb) / min_run : n_blocks;
    G = G < 1 ? 1 : G > n_blocks ? n_blocks : G;
    const int64_t g = (int64_t)j * G / n_blocks;
    const int64_t j_first = (g * n_blocks + G - 1) / G, j_next = ((g + 1) * n_blocks + G - 1) / G;
    if (j != j_first) {
        *lo = *hi = rb;
        return;
    }
    *lo = j == 0 ? rb : lower_bound_col(lenc, rb, re, sb_source_col((int64_t)j * block_rows, row0, n_rows, n, halo0));
    *hi = j_next >= n_blocks ? re : lower_bound_col(lenc, *lo, re, sb_source_col(j_next * block_rows, row0, n_rows, n, halo0));
}

// count[j * n_rows + r] = items of row row0 + r in block j
__global__ void k_sb_count(const int64_t *__restrict__ lrowptr, const int32_t *__restrict__ lenc, const int32_t *__restrict__ inner_cnt,
                           int32_t row0, int32_t n_rows, int32_t n, int64_t halo0, int32_t n_blocks, int64_t block_rows, int32_t min_run, int32_t *__restrict__ count)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (int64_t)n_rows * n_blocks) return;
    const int32_t j = (int32_t)(t / n_rows), r = (int32_t)(t - (int64_t)j * n_rows);
    int64_t lo, hi;
    sb_run(lrowptr, lenc, inner_cnt, row0 + r, j, n_blocks, block_rows, min_run, row0, n_rows, n, halo0, &lo, &hi);
    count[t] = (int32_t)((hi - lo + SAT_SPMM_CHUNK - 1) / SAT_SPMM_CHUNK);
}

__global__ void k_sb_row_totals(const int32_t *__restrict__ count, int32_t row0, int32_t n_rows, int32_t n_blocks, int32_t *__restrict__ tot,
                                int32_t *__restrict__ slots, int32_t *__restrict__ multi)
{
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n_rows) return;
    int32_t s = 0;
    for (int32_t j = 0; j < n_blocks; ++j) s += count[(int64_t)j * n_rows + r];
    tot[row0 + r] = s;
    slots[row0 + r] = s > 1 ? s : 0;
    multi[row0 + r] = s > 1 ? 1 : 0;
}

__global__ void k_sb_fill(const int64_t *__restrict__ lrowptr, const int32_t *__restrict__ lenc, const int32_t *__restrict__ inner_cnt,
                          int32_t row0, int32_t n_rows, int32_t n, int64_t halo0, int32_t n_blocks, int64_t block_rows, int32_t min_run, const int32_t *__restrict__ count,
                          const int64_t *__restrict__ item_off, const int32_t *__restrict__ tot, const int64_t *__restrict__ slot_off,
                          int4 *__restrict__ item)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (int64_t)n_rows * n_blocks) return;
    const int32_t j = (int32_t)(t / n_rows), r = (int32_t)(t - (int64_t)j * n_rows);
    const int32_t c = count[t];
    if (c == 0) return;
    const int32_t row = row0 + r;
    int64_t lo, hi;
    sb_run(lrowptr, lenc, inner_cnt, row, j, n_blocks, block_rows, min_run, row0, n_rows, n, halo0, &lo, &hi);
    int32_t before = 0;
    for (int32_t q = 0; q < j; ++q) before += count[(int64_t)q * n_rows + r];
    const bool multi = tot[row] > 1;
    for (int32_t q = 0; q < c; ++q) {
        const int64_t e0 = lo + (int64_t)q * SAT_SPMM_CHUNK;
        const int32_t len = (int32_t)((hi - e0) < SAT_SPMM_CHUNK ? (hi - e0) : SAT_SPMM_CHUNK);
        item[item_off[t] + q] = make_int4(row, multi ? (int32_t)(slot_off[row] + before + q) : -1, (int32_t)(uint32_t)(e0 & 0xffffffffll),
                                          (int32_t)((e0 >> 32) & 0xffff) | (len << 16));
    }
}

__global__ void k_sb_rows(const int64_t *__restrict__ slot_off, const int32_t *__restrict__ multi, const int64_t *__restrict__ mrow_off,
                          int32_t n, int32_t *__restrict__ slot0, int32_t *__restrict__ mrows)
{
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n) return;
    slot0[r] = (int32_t)slot_off[r];
    if (multi[r]) mrows[mrow_off[r]] = (int32_t)r;
}

static sat_status sb_read_i64(sat_ctx *ctx, const int64_t *d, int64_t *h)
{
    SAT_CUDA(ctx, cudaMemcpyAsync(h, d, sizeof(int64_t), cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return SAT_OK;
}

// partitions whose sources fit `fit_rows` rows keep one block (their items are then the row chunks of the plain list)
static int64_t sb_blocks_of(const sat_ctx *ctx, int m, int64_t block_rows, int64_t fit_rows, int64_t min_run)
{
    const int64_t rows = ctx->h_inner_off[m + 1] - ctx->h_inner_off[m];
    const int64_t T = rows + (ctx->h_halo_off[m + 1] - ctx->h_halo_off[m]);
    if (T <= fit_rows || rows == 0) return 1;
    int64_t B = cdiv64(T, block_rows);
    if (B > 4096) B = 4096;
    // blocking pays where a row meets a block with a run of entries long enough to carry the extra partial sum
    const int64_t entries = ctx->h_lnnz_off[m + 1] - ctx->h_lnnz_off[m];
    return entries / (rows * B) >= min_run ? B : 1;
}

static sat_status sb_build(sat_ctx *ctx, int64_t block_rows, int64_t fit_rows, int64_t min_run, int64_t row_run, int mode, SrcBlockedItems **out)
{
    for (SrcBlockedItems &sb : ctx->src_blocked)
        if (sb.mode == mode && (mode == 1 || (sb.block_rows == block_rows && sb.min_run == min_run && sb.fit_rows == fit_rows && sb.row_run == row_run))) {
            *out = &sb;
            return SAT_OK;
        }
    const int32_t M = ctx->M, n = ctx->n;
    std::vector<int32_t> nb((size_t)M);
    std::vector<int64_t> br((size_t)M), cbase((size_t)M + 1, 0);
    for (int m = 0; m < M; ++m) {
        const int64_t rows = ctx->h_inner_off[m + 1] - ctx->h_inner_off[m];
        const int64_t T = rows + (ctx->h_halo_off[m + 1] - ctx->h_halo_off[m]);
        const int64_t B = mode == 1 ? 1 : sb_blocks_of(ctx, m, block_rows, fit_rows, min_run);   // the inner prefix is never cut
        nb[m] = (int32_t)B;
        br[m] = cdiv64(T > 0 ? T : 1, B);  // equal blocks
        cbase[m + 1] = cbase[m] + rows * B;
    }
    const int64_t total = cbase[M];
    const int32_t row_min_run = (int32_t)(row_run < 0 ? 0 : row_run > (1 << 20) ? (1 << 20) : row_run);   // per-row grouping of blocks (sb_run)
    int32_t *count = nullptr, *slots = nullptr, *multi = nullptr;
    int64_t *item_off = nullptr, *slot_off = nullptr, *mrow_off = nullptr;
    SrcBlockedItems sb;
    sb.block_rows = block_rows;
    sb.min_run = min_run;
    sb.fit_rows = fit_rows;
    sb.row_run = row_run;
    sb.mode = mode;
    auto cleanup = [&](bool all) {
        cudaFree(count); cudaFree(slots); cudaFree(multi); cudaFree(item_off); cudaFree(slot_off); cudaFree(mrow_off);
        if (all) { cudaFree(sb.item); cudaFree(sb.slot0); cudaFree(sb.tot); cudaFree(sb.mrows); }
    };
#define SB_TRY(expr)                       \
    do {                                   \
        sat_status s_ = (expr);            \
        if (s_ != SAT_OK) {                \
            cleanup(true);                 \
            return s_;                     \
        }                                  \
    } while (0)
#define SB_CUDA(call)                                                     \
    do {                                                                  \
        cudaError_t e_ = (call);                                          \
        if (e_ != cudaSuccess) {                                          \
            cleanup(true);                                                \
            return sat_check_cuda(ctx, e_, #call);                        \
        }                                                                 \
    } while (0)
    SB_CUDA(cudaMalloc((void **)&count, (size_t)(total + 1) * sizeof(int32_t)));
    SB_CUDA(cudaMalloc((void **)&item_off, (size_t)(total + 2) * sizeof(int64_t)));
    SB_CUDA(cudaMalloc((void **)&slots, (size_t)(n + 1) * sizeof(int32_t)));
    SB_CUDA(cudaMalloc((void **)&multi, (size_t)(n + 1) * sizeof(int32_t)));
    SB_CUDA(cudaMalloc((void **)&slot_off, (size_t)(n + 2) * sizeof(int64_t)));
    SB_CUDA(cudaMalloc((void **)&mrow_off, (size_t)(n + 2) * sizeof(int64_t)));
    SB_CUDA(cudaMalloc((void **)&sb.slot0, (size_t)(n + 1) * sizeof(int32_t)));
    SB_CUDA(cudaMalloc((void **)&sb.tot, (size_t)(n + 1) * sizeof(int32_t)));
    for (int m = 0; m < M; ++m) {
        const int32_t row0 = ctx->h_inner_off[m], rows = ctx->h_inner_off[m + 1] - row0;
        if (rows == 0) continue;
        k_sb_count<<<(unsigned)cdiv64((int64_t)rows * nb[m], 256), 256, 0, ctx->stream>>>(ctx->lrowptr, ctx->lenc, mode == 1 ? ctx->inner_cnt : nullptr, row0, rows, n, ctx->h_halo_off[m],
                                                                                         nb[m], br[m], row_min_run, count + cbase[m]);
        k_sb_row_totals<<<(unsigned)cdiv64(rows, 256), 256, 0, ctx->stream>>>(count + cbase[m], row0, rows, nb[m], sb.tot, slots, multi);
    }
    SAT_LAUNCHED(ctx);
    SB_TRY(sat_scan_i32(ctx, count, total, item_off));
    SB_TRY(sat_scan_i32(ctx, slots, n, slot_off));
    SB_TRY(sat_scan_i32(ctx, multi, n, mrow_off));
    int64_t n_items = 0, n_mrows = 0;
    SB_TRY(sb_read_i64(ctx, item_off + total, &n_items));
    SB_TRY(sb_read_i64(ctx, slot_off + n, &sb.n_slots));
    SB_TRY(sb_read_i64(ctx, mrow_off + n, &n_mrows));
    if (n_items >= ((int64_t)1 << 31) || sb.n_slots >= ((int64_t)1 << 31)) {
        cleanup(true);
        return sat_fail(ctx, SAT_EINVAL, "sat_spmm: too many source-blocked work items");
    }
    sb.n_items = (int32_t)n_items;
    sb.n_mrows = (int32_t)n_mrows;
    SB_CUDA(cudaMalloc((void **)&sb.item, (size_t)(n_items > 0 ? n_items : 1) * sizeof(int4)));
    SB_CUDA(cudaMalloc((void **)&sb.mrows, (size_t)(n_mrows > 0 ? n_mrows : 1) * sizeof(int32_t)));
    for (int m = 0; m < M; ++m) {
        const int32_t row0 = ctx->h_inner_off[m], rows = ctx->h_inner_off[m + 1] - row0;
        if (rows == 0) continue;
        k_sb_fill<<<(unsigned)cdiv64((int64_t)rows * nb[m], 256), 256, 0, ctx->stream>>>(ctx->lrowptr, ctx->lenc, mode == 1 ? ctx->inner_cnt : nullptr, row0, rows, n, ctx->h_halo_off[m],
                                                                                        nb[m], br[m], row_min_run, count + cbase[m], item_off + cbase[m], sb.tot,
                                                                                        slot_off, sb.item);
    }
    k_sb_rows<<<(unsigned)cdiv64(n > 0 ? n : 1, 256), 256, 0, ctx->stream>>>(slot_off, multi, mrow_off, n, sb.slot0, sb.mrows);
    SAT_LAUNCHED(ctx);
    sb.h_item_off.assign((size_t)M + 1, 0);
    sb.h_mrow_off.assign((size_t)M + 1, 0);
    sb.h_slot_off.assign((size_t)M + 1, 0);
    for (int m = 0; m <= M; ++m) {
        int64_t a = 0, b = 0, c = 0;
        SB_TRY(sb_read_i64(ctx, item_off + cbase[m], &a));
        SB_TRY(sb_read_i64(ctx, slot_off + ctx->h_inner_off[m], &b));
        SB_TRY(sb_read_i64(ctx, mrow_off + ctx->h_inner_off[m], &c));
        sb.h_item_off[m] = (int32_t)a;
        sb.h_slot_off[m] = b;
        sb.h_mrow_off[m] = (int32_t)c;
    }
    SB_CUDA(cudaStreamSynchronize(ctx->stream));
#undef SB_TRY
#undef SB_CUDA
    cleanup(false);
    ctx->src_blocked.push_back(std::move(sb));
    *out = &ctx->src_blocked.back();
    return SAT_OK;
}

// Source blocking is used for partitions whose sources exceed `fit` bytes and whose rows meet a block with a run of at least
// `min_run` entries on average; inside such a partition a row of `len` entries is cut into at most len / row_run groups of
// blocks (sb_run).  Defaults: blocks of 64 MiB; partitions from 192 MiB whose rows meet a block with 8 entries on average;
// row groups of at least 32 entries (measured on the 2.4 M-row graph: 0 / 8 / 16 / 32 / 64 entries give 6.47 / 6.26 / 6.11 /
// 6.06 / 6.13 ms per d = 100 launch; work items 4.39 M -> 3.53 M, partial-sum rows 2.37 M -> 1.30 M).  The environment variable SAT_SPMM_SRC_BLOCK = "<block bytes>[,<fit bytes>[,<min run>[,<row run>]]]" overrides them for a
// process (block bytes 0 = never blocked; row run 0 = every row cut at every block).
struct SbConfig {
    int64_t block_rows, fit_rows, min_run, row_run;
};
static SbConfig sb_config(int32_t d4)
{
    int64_t block_bytes = (int64_t)64 << 20, fit_bytes = (int64_t)192 << 20, min_run = 8, row_run = 32;
    if (const char *e = getenv("SAT_SPMM_SRC_BLOCK")) {
        char *end = nullptr;
        block_bytes = strtoll(e, &end, 10);
        fit_bytes = 3 * block_bytes;
        if (end && *end == ',') fit_bytes = strtoll(end + 1, &end, 10);
        if (end && *end == ',') min_run = strtoll(end + 1, &end, 10);
        row_run = min_run;
        if (end && *end == ',') row_run = strtoll(end + 1, &end, 10);
    }
    SbConfig c{0, 0, min_run, row_run};
    if (block_bytes > 0) {
        c.block_rows = std::max<int64_t>(64, block_bytes / ((int64_t)d4 * 16) / 64 * 64);
        c.fit_rows = fit_bytes / ((int64_t)d4 * 16);
    }
    return c;
}

// partitions [a, b) of a view that covers whole partitions (false for any other view)
static bool sb_view_parts(const sat_ctx *ctx, const PartView &v, int *a, int *b)
{
    *a = (int)(std::lower_bound(ctx->h_inner_off.begin(), ctx->h_inner_off.end(), v.row0) - ctx->h_inner_off.begin());
    *b = (int)(std::lower_bound(ctx->h_inner_off.begin(), ctx->h_inner_off.end(), v.row0 + v.n_rows) - ctx->h_inner_off.begin());
    return *b <= ctx->M && *a <= *b && ctx->h_inner_off[*a] == v.row0 && ctx->h_inner_off[*b] == v.row0 + v.n_rows;
}

// true when at least one partition of the view is source-blocked
static bool sb_view_blocked(const sat_ctx *ctx, const PartView &v, const SbConfig &cfg, int *a, int *b)
{
    if (cfg.block_rows <= 0 || !sb_view_parts(ctx, v, a, b)) return false;
    for (int m = *a; m < *b; ++m)
        if (sb_blocks_of(ctx, m, cfg.block_rows, cfg.fit_rows, cfg.min_run) > 1) return true;
    return false;
}

template <int G, int NV>
__global__ void __launch_bounds__(256, NV <= 2 ? 8 : 4)
k_spmm_sb(const int4 *__restrict__ items, int32_t item0, int32_t n_items, int64_t slot_base, const int32_t *__restrict__ lenc,
          const float *__restrict__ lw, const float *__restrict__ dinv_enc, int32_t n, int32_t d4, const float *__restrict__ in_base, int64_t ld_in,
          const float *__restrict__ halo_base, int64_t ld_halo, float *__restrict__ out_base, int64_t ld_out, float *__restrict__ partial,
          const uint32_t *__restrict__ omask, int32_t omask_words, DbgLimits dbg)
{
    const int lane = threadIdx.x & (G - 1);
    const int64_t gid = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
    if (gid >= n_items) return;
    const unsigned mask = group_mask<G>(threadIdx.x & 31);
    const int col0 = blockIdx.y * (G * NV);
    const int4 it = __ldg(items + item0 + gid);
    const int32_t row = (int32_t)SAT_IDX(it.x, dbg.out_lo, dbg.out_hi, dbg.status);
    const int64_t e0 = (int64_t)(uint32_t)it.z | ((int64_t)(it.w & 0xffff) << 32);
    const int64_t e1 = e0 + (it.w >> 16);
    float4 acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t eb = e0; eb < e1; eb += G) {
        const int64_t e = eb + lane;
        int32_t c = 0;
        float w = 0.f;
        if (e < e1) {
            c = __ldg(lenc + e);
            w = __ldg(lw + e);
        }
        const int cnt = (e1 - eb) < G ? (int)(e1 - eb) : G;
#pragma unroll 4
        for (int j = 0; j < cnt; ++j) {
            const int32_t cj = __shfl_sync(mask, c, j, G);
            const float wj = __shfl_sync(mask, w, j, G);
            const float *src = cj < n ? in_base + SAT_IDX((int64_t)cj, dbg.src_lo, dbg.src_hi, dbg.status) * ld_in
                                      : halo_base + SAT_IDX((int64_t)(cj - n), dbg.halo_lo, dbg.halo_hi, dbg.status) * ld_halo;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int idx = col0 + lane + v * G;
                if (idx < d4) fma4(acc[v], wj, ld4(src + 4 * idx));
            }
        }
    }
    if (it.y < 0) {
        const float s = __ldg(dinv_enc + row);
        float *o = out_base + (int64_t)row * ld_out;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int idx = col0 + lane + v * G;
            if (idx < d4) {
                float4 r = make_float4(s * acc[v].x, s * acc[v].y, s * acc[v].z, s * acc[v].w);
                if (omask) mask4(r, omask, (int64_t)row * omask_words, idx);
                *reinterpret_cast<float4 *>(o + 4 * idx) = r;
            }
        }
    } else {
        float *o = partial + ((int64_t)it.y - slot_base) * (4 * (int64_t)d4);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int idx = col0 + lane + v * G;
            if (idx < d4) *reinterpret_cast<float4 *>(o + 4 * idx) = acc[v];
        }
    }
}

// rows with several source-blocked items: add the partial sums in item order (block by block), scale, store
__global__ void k_spmm_sb_fixup(const int32_t *__restrict__ mrows, int32_t mrow0, int32_t n_mrows, const int32_t *__restrict__ slot0,
                                const int32_t *__restrict__ tot, int64_t slot_base, const float *__restrict__ dinv_enc, int32_t d4,
                                const float *__restrict__ partial, float *__restrict__ out_base, int64_t ld_out,
                                const uint32_t *__restrict__ omask, int32_t omask_words, DbgLimits dbg)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d4;
    const int c = (int)(t - i * d4);
    if (i >= n_mrows) return;
    const int32_t row = (int32_t)SAT_IDX(mrows[mrow0 + i], dbg.out_lo, dbg.out_hi, dbg.status);
    const int64_t s0 = (int64_t)slot0[row] - slot_base;
    const int32_t cnt = tot[row];
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int32_t q = 0; q < cnt; ++q) {
        const float4 x = *reinterpret_cast<const float4 *>(partial + ((s0 + q) * d4 + c) * 4);
        a.x += x.x;
        a.y += x.y;
        a.z += x.z;
        a.w += x.w;
    }
    const float s = dinv_enc[row];
    float4 r = make_float4(s * a.x, s * a.y, s * a.z, s * a.w);
    if (omask) mask4(r, omask, (int64_t)row * omask_words, c);
    *reinterpret_cast<float4 *>(out_base + (int64_t)row * ld_out + 4 * c) = r;
}

template <int G, int NV>
static void launch_sb(sat_ctx *ctx, const PartView &v, const SrcBlockedItems &sb, int32_t item0, int32_t n_items, int64_t slot_base, int32_t d4,
                      const float *in_base, int32_t ld_in, const float *halo_base, int32_t ld_halo, float *out_base, int32_t ld_out, float *partial,
                      const uint32_t *omask, int32_t omask_words, const int32_t *cols, DbgRange halo_range, DbgRange src_range)
{
    dim3 grid((unsigned)cdiv64((int64_t)n_items * G, 256), (unsigned)cdiv64(d4, G * NV));
    k_spmm_sb<G, NV><<<grid, 256, 0, ctx->stream>>>(sb.item, item0, n_items, slot_base, cols, ctx->lw, ctx->dinv_enc, ctx->n, d4, in_base, ld_in,
                                                     halo_base, ld_halo, out_base, ld_out, partial, omask, omask_words,
                                                     dbg_limits(src_range, halo_range, DbgRange{v.row0, (int64_t)v.row0 + v.n_rows}, ctx->d_flag + 1));
}

template <int G, int NV>
static void launch_items(sat_ctx *ctx, const PartView &v, int inner_only, int32_t d4, const float *in_base, int32_t ld_in,
                         const float *halo_base, int32_t ld_halo, float *out_base, int32_t ld_out, float *partial, const uint32_t *omask,
                         int32_t omask_words, const int32_t *cols, DbgRange halo_range, DbgRange src_range)
{
    dim3 grid((unsigned)cdiv64((int64_t)v.n_items * G, 256), (unsigned)cdiv64(d4, G * NV));
    k_spmm_items<G, NV><<<grid, 256, 0, ctx->stream>>>(ctx->lrowptr, ctx->inner_cnt, cols, ctx->lw, ctx->dinv_enc, ctx->item_row, ctx->first_item,
                                                        ctx->item_mslot, v.item0, v.n_items, v.mitem0, inner_only, ctx->n, d4, in_base, ld_in, halo_base,
                                                        ld_halo, out_base, ld_out, partial, omask, omask_words,
                                                        dbg_limits(src_range, halo_range, DbgRange{v.row0, (int64_t)v.row0 + v.n_rows}, ctx->d_flag + 1));
}

// halo columns as global node ids (for a halo source that is a matrix over all nodes)
__global__ void k_cols_by_gid(const int32_t *__restrict__ lenc, const int32_t *__restrict__ halo_gid, int64_t count, int32_t n,
                              int32_t *__restrict__ out)
{
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= count) return;
    const int32_t c = lenc[e];
    out[e] = c < n ? c : n + halo_gid[c - n];
}

// all columns as global node ids (inner columns through the partition-major order, halo columns through the halo list)
__global__ void k_cols_all_gid(const int32_t *__restrict__ lenc, const int32_t *__restrict__ perm, const int32_t *__restrict__ halo_gid,
                               int64_t count, int32_t n, int32_t *__restrict__ out)
{
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= count) return;
    const int32_t c = lenc[e];
    out[e] = c < n ? perm[c] : halo_gid[c - n];
}

sat_status sat_spmm(sat_ctx *ctx, const PartView &v, int inner_only, int32_t d, const float *in_base, int32_t ld_in,
                    const float *halo_base, int32_t ld_halo, float *out_base, int32_t ld_out, const uint32_t *omask, int32_t omask_words,
                    bool halo_global, bool in_global)
{
    if (v.n_items == 0) return SAT_OK;
    const int32_t d4 = (d + 3) / 4;
    const int32_t *cols = ctx->lenc;
    DbgRange halo_range{v.halo0, v.halo0 + v.n_halo};
    DbgRange src_range{v.row0, (int64_t)v.row0 + v.n_rows};
    if (in_global) {
        // inner and halo rows both come from one matrix over all nodes (`in_base`, global id order): every column becomes a
        // node id (all below n, so the kernel takes its inner branch for each of them)
        if (!ctx->lenc_all_gid) {
            const int64_t lnnz = ctx->nnz + ctx->n;
            SAT_CUDA(ctx, cudaMalloc((void **)&ctx->lenc_all_gid, (size_t)lnnz * sizeof(int32_t)));
            k_cols_all_gid<<<(unsigned)cdiv64(lnnz, 256), 256, 0, ctx->stream>>>(ctx->lenc, ctx->perm, ctx->halo_gid, lnnz, ctx->n, ctx->lenc_all_gid);
            SAT_LAUNCHED(ctx);
        }
        cols = ctx->lenc_all_gid;
        src_range = DbgRange{0, ctx->n};
        halo_range = DbgRange{0, 0};
    }
    if (!in_global && halo_global) {
        if (!ctx->lenc_gid) {
            const int64_t lnnz = ctx->nnz + ctx->n;
            SAT_CUDA(ctx, cudaMalloc((void **)&ctx->lenc_gid, (size_t)lnnz * sizeof(int32_t)));
            k_cols_by_gid<<<(unsigned)cdiv64(lnnz, 256), 256, 0, ctx->stream>>>(ctx->lenc, ctx->halo_gid, lnnz, ctx->n, ctx->lenc_gid);
            SAT_LAUNCHED(ctx);
        }
        cols = ctx->lenc_gid;
        halo_range = DbgRange{0, ctx->n};
    }
    // algorithmic bytes: column ids + row offsets + dinv, every source row once, every output row once (a halo source over
    // all nodes holds at most n distinct rows)
    const double n_halo_src = halo_global && v.n_halo > ctx->n ? (double)ctx->n : (double)v.n_halo;
    double n_src = inner_only == 1 ? (double)v.n_rows : inner_only == 2 ? n_halo_src : (double)v.n_rows + n_halo_src;
    if (in_global && n_src > ctx->n) n_src = ctx->n;
    // the backward reads the inner prefix of every row, the transposed predictor convolution the halo suffix
    const double n_ent = (double)(inner_only == 1 ? v.lnnz - v.hnnz : inner_only == 2 ? v.hnnz : v.lnnz);
    ProfScope prof(ctx, inner_only ? SATK_SPMM_BWD : SATK_SPMM_FWD,
                   4.0 * n_ent + 12.0 * v.n_rows + 4.0 * n_src + 4.0 * d * (n_src + v.n_rows), 2.0 * n_ent * d);
    if (inner_only == 0 || inner_only == 1) {
        const SbConfig cfg = sb_config(d4);
        int a = 0, b = 0;
        // forward: the source-blocked list where a partition calls for it.  Backward (inner prefix of every row): a list of
        // its own with one descriptor per 256-entry chunk of the prefix — the plain list cuts whole rows, so a long row whose
        // inner entries fit one chunk still ran one (empty) work item per further chunk and went through the partial sums
        // (SAT_SPMM_SRC_BLOCK=0 in the environment sends both back to the plain list.)  Measured, descriptor list against
        // plain list: backward 7.02 -> 6.08 ms per epoch on the 2.4 M-row graph, 5.02 -> 4.60 on the 717 k-row one, 0.40 -> 0.38
        // on the 169 k-row one; forward, where no partition is blocked: 0.735 -> 0.721 ms on the 169 k-row graph.
        const bool blocked = cfg.block_rows > 0 && sb_view_parts(ctx, v, &a, &b);
        const int64_t block_rows = cfg.block_rows, fit_rows = cfg.fit_rows, min_run = cfg.min_run;
        if (blocked) {
            SrcBlockedItems *sb = nullptr;
            SAT_TRY(sb_build(ctx, block_rows, fit_rows, min_run, cfg.row_run, inner_only, &sb));
            const int32_t item0 = sb->h_item_off[a], n_items = sb->h_item_off[b] - item0;
            const int32_t mrow0 = sb->h_mrow_off[a], n_mrows = sb->h_mrow_off[b] - mrow0;
            const int64_t slot_base = sb->h_slot_off[a], n_slots = sb->h_slot_off[b] - slot_base;
            float *partial = nullptr;
            if (n_slots > 0) {
                SAT_TRY(sat_ensure(ctx, ctx->buf_sbpartial, (size_t)n_slots * d4 * 16));
                partial = (float *)ctx->buf_sbpartial.p;
            }
#define ARGS ctx, v, *sb, item0, n_items, slot_base, d4, in_base, ld_in, halo_base, ld_halo, out_base, ld_out, partial, omask, omask_words, cols, halo_range, src_range
            if (d4 <= 4) launch_sb<4, 1>(ARGS);
            else if (d4 <= 8) launch_sb<8, 1>(ARGS);
            else if (d4 <= 16) launch_sb<16, 1>(ARGS);
            else if (d4 <= 32) launch_sb<16, 2>(ARGS);
            else if (d4 <= 64) launch_sb<32, 2>(ARGS);   // 8 resident blocks per SM; 6 / 5 blocks (38-40 registers, no spills, loop unrolled 4-8x): 10-20 % slower here too
            else if (d4 <= 96) launch_sb<32, 3>(ARGS);
            else if (d4 <= 128) launch_sb<32, 4>(ARGS);
            else if (d4 <= 160) launch_sb<32, 5>(ARGS);
            else if (d4 <= 192) launch_sb<32, 6>(ARGS);
            else launch_sb<32, 8>(ARGS);
#undef ARGS
            SAT_LAUNCHED(ctx);
            if (n_mrows > 0) {
                k_spmm_sb_fixup<<<(unsigned)cdiv64((int64_t)n_mrows * d4, 256), 256, 0, ctx->stream>>>(
                    sb->mrows, mrow0, n_mrows, sb->slot0, sb->tot, slot_base, ctx->dinv_enc, d4, partial, out_base, ld_out, omask, omask_words,
                    dbg_limits(DbgRange{0, 0}, DbgRange{0, 0}, DbgRange{v.row0, (int64_t)v.row0 + v.n_rows}, ctx->d_flag + 1));
                SAT_LAUNCHED(ctx);
            }
            return SAT_OK;
        }
    }
    float *partial = nullptr;
    if (v.n_mitems > 0) {
        SAT_TRY(sat_ensure(ctx, ctx->buf_partial, (size_t)v.n_mitems * d4 * 16));
        partial = (float *)ctx->buf_partial.p;
    }
#define ARGS ctx, v, inner_only, d4, in_base, ld_in, halo_base, ld_halo, out_base, ld_out, partial, omask, omask_words, cols, halo_range, src_range
    if (d4 <= 4) launch_items<4, 1>(ARGS);
    else if (d4 <= 8) launch_items<8, 1>(ARGS);
    else if (d4 <= 16) launch_items<16, 1>(ARGS);
    else if (d4 <= 32) launch_items<16, 2>(ARGS);   // 16 lanes x 2 vectors: 16-18 % faster than 8 x 4 on the 2.4 M-row graph (d = 100, 128), equal on the 169 k-row one
    else if (d4 <= 64) launch_items<32, 2>(ARGS);   // compiled for 8 resident blocks per SM (32 registers): 6 / 5 / 4 blocks (40-44 registers, no spills) measured 3 / 12 / 11 % slower
    else if (d4 <= 96) launch_items<32, 3>(ARGS);
    else if (d4 <= 128) launch_items<32, 4>(ARGS);
    else if (d4 <= 160) launch_items<32, 5>(ARGS);
    else if (d4 <= 192) launch_items<32, 6>(ARGS);
    else launch_items<32, 8>(ARGS);
#undef ARGS
    SAT_LAUNCHED(ctx);
    if (v.n_mrows > 0) {
        k_spmm_fixup<<<(unsigned)cdiv64((int64_t)v.n_mrows * d4, 256), 256, 0, ctx->stream>>>(
            ctx->mrows, v.mrow0, v.n_mrows, ctx->first_item, ctx->item_mslot, v.mitem0, ctx->dinv_enc, d4, partial, out_base, ld_out, omask, omask_words,
            dbg_limits(DbgRange{0, 0}, DbgRange{0, 0}, DbgRange{v.row0, (int64_t)v.row0 + v.n_rows}, ctx->d_flag + 1));
        SAT_LAUNCHED(ctx);
    }
    return SAT_OK;
}

extern "C" sat_status sat_spmm_plan(sat_ctx *ctx, int32_t part, int32_t d, int32_t *n_blocks, int64_t *n_items, int64_t *n_partial_rows)
{
    CHECK_CTX(ctx);
    PartView v;
    SAT_TRY(sat_part_view(ctx, part, &v));
    if (d < 1) return sat_fail(ctx, SAT_EINVAL, "sat_spmm_plan: d = %d", d);
    const SbConfig cfg = sb_config((d + 3) / 4);
    int a = 0, b = 0;
    int32_t nb = 1;
    int64_t items = v.n_items, slots = v.n_mitems;
    if (sb_view_blocked(ctx, v, cfg, &a, &b)) {
        SrcBlockedItems *sb = nullptr;
        SAT_TRY(sb_build(ctx, cfg.block_rows, cfg.fit_rows, cfg.min_run, cfg.row_run, 0, &sb));
        for (int m = a; m < b; ++m) nb = std::max<int32_t>(nb, (int32_t)sb_blocks_of(ctx, m, cfg.block_rows, cfg.fit_rows, cfg.min_run));
        items = sb->h_item_off[b] - sb->h_item_off[a];
        slots = sb->h_slot_off[b] - sb->h_slot_off[a];
    }
    if (n_blocks) *n_blocks = nb;
    if (n_items) *n_items = items;
    if (n_partial_rows) *n_partial_rows = slots;
    return SAT_OK;
}

// -------------------------------------------------------------------------------------
// Halo-row products (rows = halo entries of the partition, columns = their neighbours
// inside the partition):
//   out[j] = dinv[u_j] * ( [self] dinv[u_j] * self_src[halo_slot_j] + sum_e dinv[v_e] * src[idx_e] )
// idx_e is the partition-major row of v_e (by_slot = 0) or its cache slot (by_slot = 1).
// Used for the predictor's graph convolution on the LSTM state (self term, by slot) and for
// the optional halo gradient P_out^T G_AGG (no self term, by row).
// -------------------------------------------------------------------------------------
// One thread block per chunk of SAT_HROW_CHUNK entries of a long halo row (the first blocks of the grid, so that they start
// first and the short rows fill the other SMs meanwhile): the 256 / G lane groups take the chunk's entries round-robin, their
// partial sums are added in group order through shared memory (fixed order: reproducible) and written, un-scaled and
// without the self term, to the chunk's row of `partial`; k_hrow_long_fixup adds the chunks of a row in chunk order.
template <int G, int NV>
__device__ __forceinline__ void hrow_chunk_block(int32_t chunk, const int32_t *__restrict__ hlong, const int64_t *__restrict__ hchunk_first,
                                                 const int32_t *__restrict__ hchunk_row, int32_t hchunk0, const int64_t *__restrict__ hrow_ptr,
                                                 const int32_t *__restrict__ hrow_pos, const int32_t *__restrict__ hrow_slot,
                                                 const float *__restrict__ hrow_w, int by_slot, int32_t d4, const float *__restrict__ src_base,
                                                 int64_t ld_src, float *__restrict__ partial, const DbgLimits &dbg)
{
    constexpr int NG = 256 / G;
    __shared__ float4 red[NG][G * NV];
    const int lane = threadIdx.x & (G - 1), grp = threadIdx.x / G;
    const int col0 = blockIdx.y * (G * NV);
    const int32_t li = hchunk_row[chunk];
    const int64_t j = SAT_IDX((int64_t)hlong[li], dbg.halo_lo, dbg.halo_hi, dbg.status);
    const int64_t k = chunk - hchunk_first[li];
    float4 acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    const int64_t e0 = hrow_ptr[j] + k * SAT_HROW_CHUNK;
    const int64_t e1 = e0 + SAT_HROW_CHUNK < hrow_ptr[j + 1] ? e0 + SAT_HROW_CHUNK : hrow_ptr[j + 1];
    const float4 *src4 = reinterpret_cast<const float4 *>(src_base) + (col0 + lane);
    const uint32_t lds4 = (uint32_t)(ld_src >> 2);
    const int32_t *__restrict__ ecol = by_slot ? hrow_slot : hrow_pos;
    for (int64_t e = e0 + grp; e < e1; e += NG) {
        const float w = __ldg(hrow_w + e);
        const int32_t c = (int32_t)SAT_IDX(__ldg(ecol + e), dbg.src_lo, dbg.src_hi, dbg.status);
        const float4 *src = src4 + (uint64_t)(uint32_t)c * lds4;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            if (col0 + lane + v * G < d4) fma4(acc[v], w, __ldg(src + v * G));
        }
    }
#pragma unroll
    for (int v = 0; v < NV; ++v) red[grp][lane + v * G] = acc[v];
    __syncthreads();
    if (grp == 0) {
        float *o = partial + (int64_t)(chunk - hchunk0) * (4 * (int64_t)d4);
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int idx = col0 + lane + v * G;
            if (idx >= d4) continue;
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int g = 0; g < NG; ++g) {
                const float4 x = red[g][lane + v * G];
                a.x += x.x; a.y += x.y; a.z += x.z; a.w += x.w;
            }
            *reinterpret_cast<float4 *>(o + 4 * idx) = a;
        }
    }
}

// long halo rows: out[j] = dinv[u_j] * ( [self] dinv[u_j] * self_src[halo_slot_j] + sum over the row's chunks, in chunk order )
__global__ void k_hrow_long_fixup(const int32_t *__restrict__ hlong, int32_t hlong0, int32_t n_hlong, const int64_t *__restrict__ hchunk_first,
                                  int32_t hchunk0, const int32_t *__restrict__ halo_slot, const float *__restrict__ dinv_enc, int32_t n,
                                  int32_t d4, const float *__restrict__ partial, const float *__restrict__ self_src, int64_t ld_src,
                                  float *__restrict__ out_base, int64_t ld_out, DbgLimits dbg)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d4;
    const int c = (int)(t - i * d4);
    if (i >= n_hlong) return;
    const int64_t j = SAT_IDX((int64_t)hlong[hlong0 + i], dbg.halo_lo, dbg.halo_hi, dbg.status);
    const float du = __ldg(dinv_enc + n + j);
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    if (self_src) fma4(a, du, ld4(self_src + SAT_IDX((int64_t)halo_slot[j], dbg.src_lo, dbg.src_hi, dbg.status) * ld_src + 4 * c));
    for (int64_t q = hchunk_first[hlong0 + i]; q < hchunk_first[hlong0 + i + 1]; ++q) {
        const float4 x = *reinterpret_cast<const float4 *>(partial + ((q - hchunk0) * d4 + c) * 4);
        a.x += x.x; a.y += x.y; a.z += x.z; a.w += x.w;
    }
    *reinterpret_cast<float4 *>(out_base + j * ld_out + 4 * c) = make_float4(du * a.x, du * a.y, du * a.z, du * a.w);
}

template <int G, int NV>
__global__ void __launch_bounds__(256)
k_spmm_hrow(const int64_t *__restrict__ hrow_ptr, const int32_t *__restrict__ hrow_pos, const int32_t *__restrict__ hrow_slot,
            const float *__restrict__ hrow_w, const int32_t *__restrict__ halo_slot, const float *__restrict__ dinv_enc, int32_t n, int64_t halo0, int64_t n_halo,
            int by_slot, int32_t d4, const float *__restrict__ src_base, int64_t ld_src, const float *__restrict__ self_src,
            float *__restrict__ out_base, int64_t ld_out, const int32_t *__restrict__ hlong, const int64_t *__restrict__ hchunk_first,
            const int32_t *__restrict__ hchunk_row, int32_t hchunk0, int32_t n_hchunks, float *__restrict__ hpartial, int32_t ipg, DbgLimits dbg)
{
    if ((int32_t)blockIdx.x < n_hchunks) {
        hrow_chunk_block<G, NV>(hchunk0 + (int32_t)blockIdx.x, hlong, hchunk_first, hchunk_row, hchunk0, hrow_ptr, hrow_pos, hrow_slot, hrow_w, by_slot,
                                d4, src_base, ld_src, hpartial, dbg);
        return;
    }
    const int lane = threadIdx.x & (G - 1);
    const int64_t gid = ((int64_t)(blockIdx.x - n_hchunks) * blockDim.x + threadIdx.x) / G;
    const int col0 = blockIdx.y * (G * NV);
    // a lane group walks `ipg` consecutive halo rows (fewer, longer-lived blocks; the header loads of a row overlap the
    // gathers of the one before)
    const int64_t g0 = gid * ipg;
    if (g0 >= n_halo) return;
    const int64_t g1 = g0 + ipg < n_halo ? g0 + ipg : n_halo;
    const int32_t *__restrict__ ecol = by_slot ? hrow_slot : hrow_pos;
    // row addresses in float4 units: one 32 x 32 -> 64-bit multiply per gathered row
    const float4 *src4 = reinterpret_cast<const float4 *>(src_base) + (col0 + lane);
    const float4 *self4 = reinterpret_cast<const float4 *>(self_src) + (col0 + lane);
    const uint32_t lds4 = (uint32_t)(ld_src >> 2);
    for (int64_t g = g0; g < g1; ++g) {
        const int64_t j = halo0 + g;
        const int64_t e0 = hrow_ptr[j], e1 = hrow_ptr[j + 1];
        if (e1 - e0 > SAT_HROW_LONG) continue;  // cut into chunks, a block each (hrow_chunk_block), combined by k_hrow_long_fixup
        const float du = __ldg(dinv_enc + n + j);
        float4 acc[NV];
#pragma unroll
        for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (self_src) {
            const float4 *src = self4 + (uint64_t)(uint32_t)SAT_IDX((int64_t)halo_slot[j], dbg.src_lo, dbg.src_hi, dbg.status) * lds4;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                if (col0 + lane + v * G < d4) fma4(acc[v], du, __ldg(src + v * G));
            }
        }
        // Halo rows are short (a handful of cut edges): every lane reads the entry's column and weight itself (one broadcast
        // transaction per group) instead of sharing them through shuffles, four entries in flight; entries in order, so the
        // sum has the same order as the long-row path's per-group partial sums.
        for (int64_t e = e0; e < e1; e += 4) {
            int32_t c[4];
            float w[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const bool ok = e + u < e1;
                c[u] = ok ? (int32_t)SAT_IDX(__ldg(ecol + e + u), dbg.src_lo, dbg.src_hi, dbg.status) : -1;
                w[u] = ok ? __ldg(hrow_w + e + u) : 0.f;
            }
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                if (col0 + lane + v * G >= d4) continue;
                float4 x[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    x[u] = c[u] >= 0 ? __ldg(src4 + (uint64_t)(uint32_t)c[u] * lds4 + v * G) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (c[u] >= 0) fma4(acc[v], w[u], x[u]);
            }
        }
        float *o = out_base + j * ld_out;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int idx = col0 + lane + v * G;
            if (idx < d4) *reinterpret_cast<float4 *>(o + 4 * idx) = make_float4(du * acc[v].x, du * acc[v].y, du * acc[v].z, du * acc[v].w);
        }
    }
}

template <int G, int NV>
static void launch_hrow(sat_ctx *ctx, const PartView &v, int by_slot, int32_t d4, const float *src_base, int32_t ld_src,
                        const float *self_src, float *out_base, int32_t ld_out, float *hpartial)
{
    // rows per lane group: launches of millions of halo rows (hundreds of thousands of short-lived blocks at one row per
    // group) run 18 % faster at four rows per group; smaller launches need every block they can get (measured: 263 k rows
    // are 25 % slower at four)
    const int32_t ipg = v.n_halo >= ((int64_t)4 << 20) ? 4 : v.n_halo >= ((int64_t)2 << 20) ? 2 : 1;
    dim3 grid((unsigned)(cdiv64(cdiv64(v.n_halo, ipg) * G, 256) + v.n_hchunks), (unsigned)cdiv64(d4, G * NV));
    k_spmm_hrow<G, NV><<<grid, 256, 0, ctx->stream>>>(ctx->hrow_ptr, ctx->hrow_pos, ctx->hrow_slot, ctx->hrow_w, ctx->halo_slot, ctx->dinv_enc, ctx->n,
                                                       v.halo0, v.n_halo, by_slot, d4, src_base, ld_src, self_src, out_base, ld_out,
                                                       ctx->hlong, ctx->hchunk_first, ctx->hchunk_row, v.hchunk0, v.n_hchunks, hpartial, ipg,
                                                       dbg_limits(by_slot ? DbgRange{0, ctx->n_slots} : DbgRange{v.row0, (int64_t)v.row0 + v.n_rows}, DbgRange{v.halo0, v.halo0 + v.n_halo}, DbgRange{v.halo0, v.halo0 + v.n_halo}, ctx->d_flag + 1));
}

sat_status sat_spmm_hrow(sat_ctx *ctx, const PartView &v, int32_t d, const float *src_base, int32_t ld_src, int by_slot,
                         const float *self_src, float *out_base, int32_t ld_out)
{
    if (v.n_halo == 0) return SAT_OK;
    const int32_t d4 = (d + 3) / 4;
    // algorithmic bytes: column + weight per entry, row offsets / slot / dinv per halo row, every source row once (the
    // boundary rows of the selection, plus the halo nodes' own rows for the self term), every output row once
    const double n_src = (double)v.n_push + (self_src ? (double)v.n_halo : 0.0);
    ProfScope prof(ctx, SATK_SPMM_HROW, 8.0 * (double)v.hnnz + 12.0 * (double)v.n_halo + 4.0 * d * (n_src + (double)v.n_halo),
                   2.0 * d * ((double)v.hnnz + (self_src ? (double)v.n_halo : 0.0)));
    float *hpartial = nullptr;
    if (v.n_hchunks > 0) {
        SAT_TRY(sat_ensure(ctx, ctx->buf_hpartial, (size_t)v.n_hchunks * d4 * 16));
        hpartial = (float *)ctx->buf_hpartial.p;
    }
#define ARGS ctx, v, by_slot, d4, src_base, ld_src, self_src, out_base, ld_out, hpartial
    if (d4 <= 4) launch_hrow<4, 1>(ARGS);
    else if (d4 <= 8) launch_hrow<8, 1>(ARGS);
    else if (d4 <= 16) launch_hrow<16, 1>(ARGS);   // at h = 64: 8 x 2, 4 x 4 and 32 x 1 measured 25-50 % slower (169 k- and 2.4 M-row graphs)
    else if (d4 <= 32) launch_hrow<32, 1>(ARGS);
    else if (d4 <= 64) launch_hrow<32, 2>(ARGS);
    else if (d4 <= 128) launch_hrow<32, 4>(ARGS);
    else launch_hrow<32, 8>(ARGS);
#undef ARGS
    SAT_LAUNCHED(ctx);
    if (v.n_hlong > 0) {
        k_hrow_long_fixup<<<(unsigned)cdiv64((int64_t)v.n_hlong * d4, 256), 256, 0, ctx->stream>>>(
            ctx->hlong, v.hlong0, v.n_hlong, ctx->hchunk_first, v.hchunk0, ctx->halo_slot, ctx->dinv_enc, ctx->n, d4, hpartial, self_src, ld_src,
            out_base, ld_out,
            dbg_limits(by_slot ? DbgRange{0, ctx->n_slots} : DbgRange{v.row0, (int64_t)v.row0 + v.n_rows}, DbgRange{v.halo0, v.halo0 + v.n_halo},
                       DbgRange{v.halo0, v.halo0 + v.n_halo}, ctx->d_flag + 1));
        SAT_LAUNCHED(ctx);
    }
    return SAT_OK;
}

// -------------------------------------------------------------------------------------
// row gather / scatter (pull of raw features, push into the cache, identity predictor)
// -------------------------------------------------------------------------------------
__global__ void k_gather_rows(const int32_t *__restrict__ idx, int64_t count, int32_t d4, const float *__restrict__ src, int64_t ld_src,
                              float *__restrict__ out, int64_t ld_out, DbgLimits dbg)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d4;
    const int c = (int)(t - i * d4);
    if (i >= count) return;
    const float4 x = ld4(src + SAT_IDX((int64_t)idx[i], dbg.src_lo, dbg.src_hi, dbg.status) * ld_src + 4 * c);
    *reinterpret_cast<float4 *>(out + i * ld_out + 4 * c) = x;
}

sat_status sat_gather(sat_ctx *ctx, const int32_t *idx, int64_t count, int32_t d, const float *src, int32_t ld_src, float *out,
                      int32_t ld_out, DbgRange src_rows)
{
    if (count == 0) return SAT_OK;
    const int32_t d4 = (d + 3) / 4;
    ProfScope prof(ctx, SATK_GATHER, (8.0 * d + 4.0) * (double)count, 0.0);
    k_gather_rows<<<(unsigned)cdiv64(count * d4, 256), 256, 0, ctx->stream>>>(idx, count, d4, src, ld_src, out, ld_out,
                                                                              dbg_limits(src_rows, DbgRange{0, 0}, DbgRange{0, count}, ctx->d_flag + 1));
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

__global__ void k_scatter_rows(const int32_t *__restrict__ src_row, const int32_t *__restrict__ dst_row, int64_t count, int32_t d4,
                               const float *__restrict__ src_base, int64_t ld_src, float *__restrict__ dst, int64_t ld_dst, DbgLimits dbg)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d4;
    const int c = (int)(t - i * d4);
    if (i >= count) return;
    const float4 x = ld4(src_base + SAT_IDX((int64_t)src_row[i], dbg.src_lo, dbg.src_hi, dbg.status) * ld_src + 4 * c);
    *reinterpret_cast<float4 *>(dst + SAT_IDX((int64_t)dst_row[i], dbg.out_lo, dbg.out_hi, dbg.status) * ld_dst + 4 * c) = x;
}

sat_status sat_scatter(sat_ctx *ctx, const int32_t *src_row, const int32_t *dst_row, int64_t count, int32_t d, const float *src_base,
                       int32_t ld_src, float *dst, int32_t ld_dst, DbgRange src_rows, DbgRange dst_rows)
{
    if (count == 0) return SAT_OK;
    const int32_t d4 = (d + 3) / 4;
    ProfScope prof(ctx, SATK_SCATTER, (8.0 * d + 8.0) * (double)count, 0.0);
    k_scatter_rows<<<(unsigned)cdiv64(count * d4, 256), 256, 0, ctx->stream>>>(src_row, dst_row, count, d4, src_base, ld_src, dst, ld_dst,
                                                                               dbg_limits(src_rows, DbgRange{0, 0}, dst_rows, ctx->d_flag + 1));
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

__global__ void k_scatter_add_rows(const int32_t *__restrict__ src_row, const int32_t *__restrict__ dst_row, int64_t count, int32_t d4,
                                   const float *__restrict__ src_base, int64_t ld_src, float *__restrict__ dst, int64_t ld_dst,
                                   const uint32_t *__restrict__ mask, int32_t mask_words, DbgLimits dbg)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d4;
    const int c = (int)(t - i * d4);
    if (i >= count) return;
    float4 x = ld4(src_base + (src_row ? SAT_IDX((int64_t)src_row[i], dbg.src_lo, dbg.src_hi, dbg.status) : i) * ld_src + 4 * c);
    const int64_t r = SAT_IDX((int64_t)dst_row[i], dbg.out_lo, dbg.out_hi, dbg.status);
    if (mask) mask4(x, mask, r * mask_words, c);
    float4 *o = reinterpret_cast<float4 *>(dst + r * ld_dst + 4 * c);
    float4 y = *o;
    y.x += x.x;
    y.y += x.y;
    y.z += x.z;
    y.w += x.w;
    *o = y;
}

sat_status sat_scatter_add(sat_ctx *ctx, const int32_t *src_row, const int32_t *dst_row, int64_t count, int32_t d, const float *src_base,
                           int32_t ld_src, float *dst, int32_t ld_dst, const uint32_t *mask, int32_t mask_words, DbgRange src_rows, DbgRange dst_rows)
{
    if (count == 0) return SAT_OK;
    const int32_t d4 = (d + 3) / 4;
    ProfScope prof(ctx, SATK_SCATTER, (12.0 * d + 8.0) * (double)count, 0.0);
    k_scatter_add_rows<<<(unsigned)cdiv64(count * d4, 256), 256, 0, ctx->stream>>>(src_row, dst_row, count, d4, src_base, ld_src, dst, ld_dst, mask,
                                                                                   mask_words, dbg_limits(src_rows, DbgRange{0, 0}, dst_rows, ctx->d_flag + 1));
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

// -------------------------------------------------------------------------------------
// Halo positions by cache slot: the inverse of halo_slot[].  A boundary node is a halo node of every other partition it has
// a neighbour in; reductions over "all copies of a node" (gradient-side history, transposed predictor convolution) read
// their terms through this index, one writer per slot, in ascending partition order.
// -------------------------------------------------------------------------------------
__global__ void k_hs_count(const int32_t *__restrict__ halo_slot, int64_t nb, int32_t *__restrict__ cnt)
{
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p < nb) atomicAdd(cnt + halo_slot[p], 1);   // integer counts: the result does not depend on the order
}

// the halo slots of one partition are distinct, so the cursor of a slot is touched by one thread per launch; the partitions
// are launched in ascending order
__global__ void k_hs_fill(const int32_t *__restrict__ halo_slot, int64_t p0, int64_t count, const int64_t *__restrict__ hs_ptr,
                          int32_t *__restrict__ cursor, int32_t *__restrict__ hs_pos)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    const int32_t s = halo_slot[p0 + i];
    const int32_t k = cursor[s];
    cursor[s] = k + 1;
    hs_pos[hs_ptr[s] + k] = (int32_t)(p0 + i);
}

static sat_status build_halo_by_slot(sat_ctx *ctx)
{
    if (ctx->hs_ptr) return SAT_OK;
    const int64_t ns = ctx->n_slots, nb = ctx->nb;
    int32_t *cnt = nullptr;
    SAT_CUDA(ctx, cudaMalloc(&cnt, (size_t)(ns + 1) * sizeof(int32_t)));
    cudaError_t e = cudaMalloc(&ctx->hs_ptr, (size_t)(ns + 1) * sizeof(int64_t));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->hs_pos, (size_t)(nb > 0 ? nb : 1) * sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemsetAsync(cnt, 0, (size_t)(ns + 1) * sizeof(int32_t), ctx->stream);
    sat_status rc = SAT_OK;
    if (e == cudaSuccess && nb > 0) {
        k_hs_count<<<(unsigned)cdiv64(nb, 256), 256, 0, ctx->stream>>>(ctx->halo_slot, nb, cnt);
        ctx->launches++;
    }
    if (e == cudaSuccess) rc = sat_scan_i32(ctx, cnt, ns, ctx->hs_ptr);
    if (e == cudaSuccess && rc == SAT_OK) e = cudaMemsetAsync(cnt, 0, (size_t)(ns + 1) * sizeof(int32_t), ctx->stream);
    for (int32_t m = 0; e == cudaSuccess && rc == SAT_OK && m < ctx->M; ++m) {
        const int64_t p0 = ctx->h_halo_off[m], count = ctx->h_halo_off[m + 1] - p0;
        if (count == 0) continue;
        k_hs_fill<<<(unsigned)cdiv64(count, 256), 256, 0, ctx->stream>>>(ctx->halo_slot, p0, count, ctx->hs_ptr, cnt, ctx->hs_pos);
        ctx->launches++;
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    cudaFree(cnt);
    if (e != cudaSuccess || rc != SAT_OK) {
        cudaFree(ctx->hs_ptr);
        cudaFree(ctx->hs_pos);
        ctx->hs_ptr = nullptr;
        ctx->hs_pos = nullptr;
        return rc != SAT_OK ? rc : sat_check_cuda(ctx, e, "halo positions by slot");
    }
    return SAT_OK;
}

__global__ void __launch_bounds__(256)
k_sum_by_slot(const int64_t *__restrict__ hs_ptr, const int32_t *__restrict__ hs_pos, int32_t n_slots, const float *__restrict__ dinv_enc,
              int32_t n, int32_t d4, const float *__restrict__ src, int64_t ld_src, int self_scale, int add, float *__restrict__ out, int64_t ld_out,
              DbgLimits dbg)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t s = t / d4;
    const int c = (int)(t - s * d4);
    if (s >= n_slots) return;
    const int64_t b = hs_ptr[s], e = hs_ptr[s + 1];
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t i = b; i < e; ++i) {
        const float4 x = ld4(src + SAT_IDX((int64_t)__ldg(hs_pos + i), dbg.src_lo, dbg.src_hi, dbg.status) * ld_src + 4 * c);
        acc.x += x.x;
        acc.y += x.y;
        acc.z += x.z;
        acc.w += x.w;
    }
    if (self_scale && e > b) {
        const float du = __ldg(dinv_enc + n + hs_pos[b]);
        const float p = du * du;
        acc.x *= p;
        acc.y *= p;
        acc.z *= p;
        acc.w *= p;
    }
    float4 *o = reinterpret_cast<float4 *>(out + s * ld_out + 4 * c);
    if (add) {
        const float4 y = *o;
        acc.x += y.x;
        acc.y += y.y;
        acc.z += y.z;
        acc.w += y.w;
    }
    *o = acc;
}

sat_status sat_sum_by_slot(sat_ctx *ctx, int32_t d, const float *src, int32_t ld_src, int self_scale, int add, float *out, int32_t ld_out)
{
    if (ctx->n_slots == 0) return SAT_OK;
    SAT_TRY(build_halo_by_slot(ctx));
    const int32_t d4 = (d + 3) / 4;
    ProfScope prof(ctx, SATK_SCATTER, 8.0 * (double)ctx->nb + 4.0 * d * ((double)ctx->nb + (add ? 2.0 : 1.0) * ctx->n_slots), 0.0);
    k_sum_by_slot<<<(unsigned)cdiv64((int64_t)ctx->n_slots * d4, 256), 256, 0, ctx->stream>>>(ctx->hs_ptr, ctx->hs_pos, ctx->n_slots, ctx->dinv_enc,
                                                                                              ctx->n, d4, src, ld_src, self_scale, add, out, ld_out,
                                                                                              dbg_limits(DbgRange{0, ctx->nb}, DbgRange{0, 0}, DbgRange{0, ctx->n_slots}, ctx->d_flag + 1));
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}


// -------------------------------------------------------------------------------------
// Measurement aid: what the L2 -> SM path of this GPU delivers, measured in the run that quotes it.
//   stream: every thread block reads a contiguous 128-bit-per-lane stream of a buffer that fits in L2;
//   gather: one warp per item reads `row_floats`-wide rows of that buffer in a seeded pseudo-random order with the
//           access shape of the SpMM (lanes own 128-bit column slices, several rows in flight), accumulating them.
// Results are kept live through a predicated store that never fires for finite data.
// -------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_l2_stream(const float4 *__restrict__ buf, int64_t n_vec, int reps, float *__restrict__ sink)
{
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int r = 0; r < reps; ++r) {
        int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
        for (; i + 3 * stride < n_vec; i += 4 * stride) {
            const float4 a = __ldg(buf + i), b = __ldg(buf + i + stride), c = __ldg(buf + i + 2 * stride), d = __ldg(buf + i + 3 * stride);
            acc.x += a.x + b.x + c.x + d.x;
            acc.y += a.y + b.y + c.y + d.y;
            acc.z += a.z + b.z + c.z + d.z;
            acc.w += a.w + b.w + c.w + d.w;
        }
        for (; i < n_vec; i += stride) {
            const float4 a = __ldg(buf + i);
            acc.x += a.x; acc.y += a.y; acc.z += a.z; acc.w += a.w;
        }
    }
    if (acc.x + acc.y + acc.z + acc.w == 12345.678f) sink[0] = acc.x;   // never true for the zero-filled buffer
}

template <int NV>
__global__ void __launch_bounds__(256, NV <= 2 ? 8 : 4)
k_l2_gather(const float *__restrict__ buf, uint32_t row_mask, int32_t d4, int64_t n_items, int per_item, float *__restrict__ sink)
{
    const int lane = threadIdx.x & 31;
    const int64_t item = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (item >= n_items) return;
    float4 acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    uint64_t state = 0x9E3779B97F4A7C15ull * (uint64_t)(item + 1);
    for (int e = 0; e < per_item; e += 4) {
        int64_t r[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            state = state * 6364136223846793005ull + 1442695040888963407ull;   // the same sequence in every lane of the warp
            r[u] = (int64_t)((uint32_t)(state >> 24) & row_mask);   // the row count is a power of two
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float *src = buf + r[u] * (4 * (int64_t)d4);
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int idx = lane + 32 * v;
                if (idx < d4) fma4(acc[v], 0.5f, ld4(src + 4 * idx));
            }
        }
    }
    float t = 0.f;
#pragma unroll
    for (int v = 0; v < NV; ++v) t += acc[v].x + acc[v].y + acc[v].z + acc[v].w;
    if (t == 12345.678f) sink[0] = t;
}

extern "C" sat_status sat_profile_l2_rates(sat_ctx *ctx, int32_t row_floats, double *stream_gbs, double *gather_gbs)
{
    CHECK_CTX(ctx);
    if (row_floats < 4 || row_floats > 1024 || (row_floats & 3)) return sat_fail(ctx, SAT_EINVAL, "sat_profile_l2_rates: row width must be a multiple of 4 in [4, 1024]");
    const size_t bytes = (size_t)64 << 20;                        // well inside the 126 MB L2
    const int32_t d4 = row_floats / 4;
    int64_t n_rows = 1;                                           // the largest power of two of rows that fits the buffer
    while (2 * n_rows * (int64_t)row_floats * 4 <= (int64_t)bytes) n_rows *= 2;
    float *buf = nullptr, *sink = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaMalloc((void **)&buf, bytes);
    if (e == cudaSuccess) e = cudaMalloc((void **)&sink, 256);
    if (e == cudaSuccess) e = cudaMemsetAsync(buf, 0, bytes, ctx->stream);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    float ms_stream = 0.f, ms_gather = 0.f;
    const int reps = 8, per_item = 64;
    const int64_t n_items = (int64_t)1 << 20;                      // 64 rows each: 64 Mi row reads per launch
    if (e == cudaSuccess) {
        const int64_t n_vec = (int64_t)(bytes / 16);
        for (int pass = 0; pass < 2 && e == cudaSuccess; ++pass) {  // first pass warms the L2 and the instruction cache
            cudaEventRecord(e0, ctx->stream);
            k_l2_stream<<<148 * 8, 256, 0, ctx->stream>>>((const float4 *)buf, n_vec, reps, sink);
            cudaEventRecord(e1, ctx->stream);
            ctx->launches++;
            e = cudaEventSynchronize(e1);
            if (e == cudaSuccess) e = cudaEventElapsedTime(&ms_stream, e0, e1);
        }
        for (int pass = 0; pass < 2 && e == cudaSuccess; ++pass) {
            cudaEventRecord(e0, ctx->stream);
            const unsigned grid = (unsigned)cdiv64(n_items * 32, 256);
            if (d4 <= 32) k_l2_gather<1><<<grid, 256, 0, ctx->stream>>>(buf, (uint32_t)(n_rows - 1), d4, n_items, per_item, sink);
            else if (d4 <= 64) k_l2_gather<2><<<grid, 256, 0, ctx->stream>>>(buf, (uint32_t)(n_rows - 1), d4, n_items, per_item, sink);
            else if (d4 <= 128) k_l2_gather<4><<<grid, 256, 0, ctx->stream>>>(buf, (uint32_t)(n_rows - 1), d4, n_items, per_item, sink);
            else k_l2_gather<8><<<grid, 256, 0, ctx->stream>>>(buf, (uint32_t)(n_rows - 1), d4, n_items, per_item, sink);
            cudaEventRecord(e1, ctx->stream);
            ctx->launches++;
            e = cudaEventSynchronize(e1);
            if (e == cudaSuccess) e = cudaEventElapsedTime(&ms_gather, e0, e1);
        }
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(buf);
    cudaFree(sink);
    if (e != cudaSuccess) return sat_check_cuda(ctx, e, "sat_profile_l2_rates");
    if (stream_gbs) *stream_gbs = (double)bytes * reps / (ms_stream * 1e-3) / 1e9;
    if (gather_gbs) *gather_gbs = (double)n_items * per_item * row_floats * 4.0 / (ms_gather * 1e-3) / 1e9;
    return SAT_OK;
}
