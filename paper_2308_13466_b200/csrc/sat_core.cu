// Context, graph load and partition construction of the sat_b200 library.
// All graph structures are integer and are built by the kernels below on the device.
#include <new>

#include "sat_internal.h"

// =====================================================================================
// errors, buffers
// =====================================================================================
sat_status sat_fail(sat_ctx *ctx, sat_status code, const char *fmt, ...)
{
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

sat_status sat_check_cuda(sat_ctx *ctx, cudaError_t e, const char *what)
{
    if (e == cudaSuccess) return SAT_OK;
    if (e == cudaErrorMemoryAllocation) {
        cudaGetLastError();
        return sat_fail(ctx, SAT_ENOMEM, "out of memory in %s", what);
    }
    if (ctx) ctx->cuda_failed = true;
    return sat_fail(ctx, SAT_ECUDA, "CUDA error %d (%s) in %s", (int)e, cudaGetErrorString(e), what);
}

sat_status sat_ensure(sat_ctx *ctx, DevBuf &b, size_t bytes)
{
    if (bytes <= b.bytes && b.p) return SAT_OK;
    if (b.p) {
        // the buffer may still be in use by enqueued work
        SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        cudaFree(b.p);
        b.p = nullptr;
        b.bytes = 0;
    }
    size_t want = bytes < 256 ? 256 : bytes;
    SAT_CUDA(ctx, cudaMalloc(&b.p, want));
    b.bytes = want;
    return SAT_OK;
}

void sat_free_buf(DevBuf &b)
{
    if (b.p) cudaFree(b.p);
    b.p = nullptr;
    b.bytes = 0;
}

template <typename T>
static sat_status dev_alloc(sat_ctx *ctx, T **p, int64_t count)
{
    if (*p) {
        cudaFree(*p);
        *p = nullptr;
    }
    size_t bytes = (size_t)(count > 0 ? count : 1) * sizeof(T);
    SAT_CUDA(ctx, cudaMalloc((void **)p, bytes));
    return SAT_OK;
}

template <typename T>
static void dev_free(T **p)
{
    if (*p) cudaFree(*p);
    *p = nullptr;
}

static sat_status read_flag(sat_ctx *ctx, int *value)
{
    SAT_CUDA(ctx, cudaMemcpyAsync(ctx->h_flag, ctx->d_flag, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    *value = *ctx->h_flag;
    return SAT_OK;
}

static void prof_clear(sat_ctx *ctx);

// =====================================================================================
// context
// =====================================================================================
extern "C" sat_status sat_create(sat_ctx **out, int device, void *cuda_stream)
{
    if (!out) return SAT_EINVAL;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return SAT_EINVAL;
    if (cudaSetDevice(device) != cudaSuccess) return SAT_ECUDA;
    sat_ctx *ctx = new (std::nothrow) sat_ctx();
    if (!ctx) return SAT_ENOMEM;
    ctx->device = device;
    ctx->stream = (cudaStream_t)cuda_stream;
    if (cudaMalloc((void **)&ctx->d_flag, 2 * sizeof(int)) != cudaSuccess ||
        cudaMallocHost((void **)&ctx->h_flag, sizeof(int)) != cudaSuccess) {
        delete ctx;
        return SAT_ENOMEM;
    }
    cudaMemsetAsync(ctx->d_flag, 0, 2 * sizeof(int), ctx->stream);  // [0] validation flags, [1] kernel wait time-outs
    *out = ctx;
    return SAT_OK;
}

static void free_partition(sat_ctx *ctx)
{
    dev_free(&ctx->part);
    dev_free(&ctx->perm);
    dev_free(&ctx->pos);
    dev_free(&ctx->halo_gid);
    dev_free(&ctx->halo_slot);
    dev_free(&ctx->slot);
    dev_free(&ctx->push_row);
    dev_free(&ctx->push_slot);
    dev_free(&ctx->row_slot);
    dev_free(&ctx->hs_ptr);
    dev_free(&ctx->hs_pos);
    dev_free(&ctx->lrowptr);
    dev_free(&ctx->lenc);
    dev_free(&ctx->lenc_gid);
    dev_free(&ctx->lenc_all_gid);
    for (SrcBlockedItems &sb : ctx->src_blocked) {
        dev_free(&sb.item);
        dev_free(&sb.slot0);
        dev_free(&sb.tot);
        dev_free(&sb.mrows);
    }
    ctx->src_blocked.clear();
    dev_free(&ctx->inner_cnt);
    dev_free(&ctx->dinv_enc);
    dev_free(&ctx->lw);
    dev_free(&ctx->hrow_ptr);
    dev_free(&ctx->hrow_pos);
    dev_free(&ctx->hrow_slot);
    dev_free(&ctx->hrow_w);
    dev_free(&ctx->hlong);
    dev_free(&ctx->hchunk_first);
    dev_free(&ctx->hchunk_row);
    dev_free(&ctx->halo_tile_order);
    ctx->n_hchunks = 0;
    dev_free(&ctx->first_item);
    dev_free(&ctx->item_row);
    dev_free(&ctx->item_mslot);
    dev_free(&ctx->mrows);
    ctx->part_ok = false;
}

static void free_cache(sat_ctx *ctx)
{
    for (int i = 0; i < SAT_MAX_LAYERS; ++i) {
        dev_free(&ctx->cache[i].buf);
        dev_free(&ctx->cache[i].S);
        dev_free(&ctx->cache[i].proj);
        sat_free_buf(ctx->cache[i].pk_wx);
        sat_free_buf(ctx->cache[i].pk_uh);
        sat_free_buf(ctx->cache[i].pk_wg);
        sat_free_buf(ctx->cache[i].pk_b);
        sat_free_buf(ctx->cache[i].pk_bg);
        ctx->cache[i] = CacheLayer();
    }
    ctx->cache_ok = false;
    ctx->n_cached = 0;
}

static void free_layers(sat_ctx *ctx)
{
    for (int i = 0; i <= SAT_MAX_LAYERS; ++i) {
        dev_free(&ctx->layers[i].agg);
        dev_free(&ctx->layers[i].mask);
        ctx->layers[i] = LayerState();
        dev_free(&ctx->ghist[i].buf);
        ctx->ghist[i] = GradHist();
        sat_free_buf(ctx->gat[i].z_in);
        sat_free_buf(ctx->gat[i].z_halo);
        sat_free_buf(ctx->gat[i].scal);
        ctx->gat[i].d_out = 0;
        ctx->gat[i].valid.clear();
    }
}

extern "C" sat_status sat_destroy(sat_ctx *ctx)
{
    if (!ctx) return SAT_EINVAL;
    cudaSetDevice(ctx->device);
    cudaStreamSynchronize(ctx->stream);
    prof_clear(ctx);
    free_partition(ctx);
    free_cache(ctx);
    free_layers(ctx);
    dev_free(&ctx->rowptr);
    dev_free(&ctx->col);
    dev_free(&ctx->dinv);
    sat_free_buf(ctx->buf_partial);
    sat_free_buf(ctx->buf_hpartial);
    sat_free_buf(ctx->buf_sbpartial);
    sat_free_buf(ctx->buf_gagg);
    sat_free_buf(ctx->buf_splitk);
    sat_free_buf(ctx->buf_lstm_c);
    sat_free_buf(ctx->buf_codec_sizes);
    sat_free_buf(ctx->buf_codec_off);
    sat_free_buf(ctx->buf_codec_bytes);
    sat_free_buf(ctx->buf_lstm_s);
    sat_free_buf(ctx->buf_lstm_w);
    sat_free_buf(ctx->buf_pred_a);
    sat_free_buf(ctx->buf_misc);
    sat_free_buf(ctx->buf_colsum);
    sat_free_buf(ctx->buf_dmask);
    sat_free_buf(ctx->buf_wsplit);
    sat_free_buf(ctx->buf_wsplit2);
    sat_free_buf(ctx->buf_wsplit3);
    sat_free_buf(ctx->buf_bias);
    sat_free_buf(ctx->buf_pred_train);
    sat_free_buf(ctx->buf_ghist_halo);
    sat_free_buf(ctx->buf_ghist_rows);
    sat_free_buf(ctx->buf_ghist_out);
    sat_free_buf(ctx->buf_gat);
    sat_free_buf(ctx->buf_gat_items);
    if (ctx->d_flag) cudaFree(ctx->d_flag);
    if (ctx->h_flag) cudaFreeHost(ctx->h_flag);
    delete ctx;
    return SAT_OK;
}

extern "C" const char *sat_last_error(const sat_ctx *ctx) { return ctx ? ctx->err : "null context"; }

extern "C" sat_status sat_sync_status(sat_ctx *ctx)
{
    if (!ctx) return SAT_EINVAL;
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (ctx->cuda_failed) return SAT_ECUDA;
    SAT_CUDA(ctx, cudaMemcpyAsync(ctx->h_flag, ctx->d_flag + 1, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (*ctx->h_flag & 1) {
        ctx->cuda_failed = true;
        return sat_fail(ctx, SAT_ECUDA, "a tensor-core kernel gave up waiting on a barrier (status %d)", *ctx->h_flag);
    }
    if (*ctx->h_flag & 4) {  // debug build only: an index outside its matrix was met (and replaced by 0); reported once
        SAT_CUDA(ctx, cudaMemsetAsync(ctx->d_flag + 1, 0, sizeof(int), ctx->stream));
        return sat_fail(ctx, SAT_EDATA, "bounds check of the debug build: a graph kernel loaded an index outside the matrix it addresses");
    }
    if (*ctx->h_flag & 2) {  // malformed codec input: reported once, the context stays usable
        SAT_CUDA(ctx, cudaMemsetAsync(ctx->d_flag + 1, 0, sizeof(int), ctx->stream));
        return sat_fail(ctx, SAT_EDATA, "sat_codec_decode: a row does not hold exactly d well-formed values");
    }
    return SAT_OK;
}

// Debug build only: overwrite one entry of an internal index array, so that a test can show the bounds checks at work.
extern "C" sat_status sat_debug_poke_index(sat_ctx *ctx, int which, int64_t pos, int32_t value, int32_t *old_value)
{
    CHECK_CTX(ctx);
#if SAT_DBG
    if (!ctx->part_ok) return sat_fail(ctx, SAT_ESTATE, "sat_debug_poke_index: call sat_partition first");
    int32_t *arr = which == 0 ? ctx->lenc : which == 1 ? ctx->halo_slot : nullptr;
    const int64_t len = which == 0 ? ctx->nnz + ctx->n : ctx->nb;
    if (!arr || pos < 0 || pos >= len) return sat_fail(ctx, SAT_EINVAL, "sat_debug_poke_index: unknown array or position outside it");
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (old_value) SAT_CUDA(ctx, cudaMemcpy(old_value, arr + pos, sizeof(int32_t), cudaMemcpyDeviceToHost));
    SAT_CUDA(ctx, cudaMemcpy(arr + pos, &value, sizeof(int32_t), cudaMemcpyHostToDevice));
    return SAT_OK;
#else
    (void)which; (void)pos; (void)value; (void)old_value;
    return sat_fail(ctx, SAT_ESTATE, "sat_debug_poke_index: only in the bounds-checking debug build of the library");
#endif
}

extern "C" sat_status sat_launch_count(sat_ctx *ctx, int64_t *count)
{
    if (!ctx || !count) return SAT_EINVAL;
    *count = ctx->launches;
    return SAT_OK;
}

// =====================================================================================
// per-family device timing
// =====================================================================================
static const char *k_family_names[SATK_COUNT] = {"spmm_fwd", "spmm_bwd", "spmm_hrow", "gemm_nn", "gemm_nt", "gemm_tn",
                                                 "lstm_cell", "gather", "scatter", "loss", "mask", "gemm_side", "codec", "pred_train", "gat"};

static void prof_clear(sat_ctx *ctx)
{
    for (auto &r : ctx->prof) {
        cudaEventDestroy(r.a);
        cudaEventDestroy(r.b);
    }
    ctx->prof.clear();
}

extern "C" int32_t sat_profile_families(void) { return SATK_COUNT; }

extern "C" sat_status sat_profile_enable(sat_ctx *ctx, int enable)
{
    if (!ctx) return SAT_EINVAL;
    if (enable) {
        SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        prof_clear(ctx);
    }
    ctx->prof_on = enable != 0;
    return SAT_OK;
}

extern "C" sat_status sat_profile_select(sat_ctx *ctx, uint64_t family_mask)
{
    if (!ctx) return SAT_EINVAL;
    ctx->prof_mask = family_mask;
    return SAT_OK;
}

extern "C" sat_status sat_profile_read(sat_ctx *ctx, int32_t family, const char **name, int64_t *calls, double *ms, double *bytes,
                                       double *flops)
{
    if (!ctx || family < 0 || family >= SATK_COUNT) return SAT_EINVAL;
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    int64_t c = 0;
    double t = 0, by = 0, fl = 0;
    for (auto &r : ctx->prof) {
        if (r.family != family) continue;
        float e = 0.f;
        SAT_CUDA(ctx, cudaEventElapsedTime(&e, r.a, r.b));
        c++;
        t += e;
        by += r.bytes;
        fl += r.flops;
    }
    if (name) *name = k_family_names[family];
    if (calls) *calls = c;
    if (ms) *ms = t;
    if (bytes) *bytes = by;
    if (flops) *flops = fl;
    return SAT_OK;
}

// =====================================================================================
// exclusive scan (int32 counts -> int64 offsets), three plain passes
// =====================================================================================
#define SCAN_TILE 2048
#define SCAN_THREADS 256

__global__ void k_scan_tile_sums(const int32_t *__restrict__ in, int64_t count, int64_t *__restrict__ tile_sum)
{
    __shared__ long long red[SCAN_THREADS];
    int64_t base = (int64_t)blockIdx.x * SCAN_TILE;
    long long s = 0;
    for (int i = threadIdx.x; i < SCAN_TILE; i += SCAN_THREADS) {
        int64_t idx = base + i;
        if (idx < count) s += in[idx];
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = SCAN_THREADS / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) tile_sum[blockIdx.x] = red[0];
}

// single block: exclusive scan of the tile sums in place (serial over chunks, tiny)
__global__ void k_scan_tile_offsets(int64_t *tile_sum, int64_t n_tiles, int64_t *total)
{
    __shared__ long long sh[SCAN_THREADS];
    __shared__ long long carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int64_t c0 = 0; c0 < n_tiles; c0 += SCAN_THREADS) {
        int64_t idx = c0 + threadIdx.x;
        long long v = idx < n_tiles ? tile_sum[idx] : 0;
        sh[threadIdx.x] = v;
        __syncthreads();
        for (int o = 1; o < SCAN_THREADS; o <<= 1) {
            long long t = threadIdx.x >= o ? sh[threadIdx.x - o] : 0;
            __syncthreads();
            sh[threadIdx.x] += t;
            __syncthreads();
        }
        long long incl = sh[threadIdx.x];
        if (idx < n_tiles) tile_sum[idx] = carry + incl - v;
        __syncthreads();
        if (threadIdx.x == SCAN_THREADS - 1) carry += incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) *total = carry;
}

__global__ void k_scan_write(const int32_t *__restrict__ in, int64_t count, const int64_t *__restrict__ tile_off,
                             int64_t *__restrict__ out)
{
    // each thread owns SCAN_TILE / SCAN_THREADS consecutive elements
    const int PER = SCAN_TILE / SCAN_THREADS;
    __shared__ long long sh[SCAN_THREADS];
    int64_t base = (int64_t)blockIdx.x * SCAN_TILE + (int64_t)threadIdx.x * PER;
    long long loc[PER];
    long long s = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        int64_t idx = base + i;
        long long v = idx < count ? in[idx] : 0;
        loc[i] = s;
        s += v;
    }
    sh[threadIdx.x] = s;
    __syncthreads();
    for (int o = 1; o < SCAN_THREADS; o <<= 1) {
        long long t = threadIdx.x >= o ? sh[threadIdx.x - o] : 0;
        __syncthreads();
        sh[threadIdx.x] += t;
        __syncthreads();
    }
    long long excl = sh[threadIdx.x] - s + tile_off[blockIdx.x];
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        int64_t idx = base + i;
        if (idx < count) out[idx] = excl + loc[i];
    }
}

sat_status sat_scan_i32(sat_ctx *ctx, const int32_t *in, int64_t count, int64_t *out)
{
    int64_t n_tiles = cdiv64(count > 0 ? count : 1, SCAN_TILE);
    SAT_TRY(sat_ensure(ctx, ctx->buf_misc, (size_t)(n_tiles + 1) * sizeof(int64_t)));
    int64_t *tiles = (int64_t *)ctx->buf_misc.p;
    k_scan_tile_sums<<<(unsigned)n_tiles, SCAN_THREADS, 0, ctx->stream>>>(in, count, tiles);
    SAT_LAUNCHED(ctx);
    k_scan_tile_offsets<<<1, SCAN_THREADS, 0, ctx->stream>>>(tiles, n_tiles, out + count);
    SAT_LAUNCHED(ctx);
    k_scan_write<<<(unsigned)n_tiles, SCAN_THREADS, 0, ctx->stream>>>(in, count, tiles, out);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

// =====================================================================================
// sat_graph_load
// =====================================================================================
enum { BAD_ROWPTR = 1, BAD_COL_RANGE = 2, BAD_COL_ORDER = 4, BAD_SELF_LOOP = 8, BAD_ASYM = 16, BAD_PART = 32 };

__global__ void k_check_rowptr(const int64_t *rowptr, int32_t n, int64_t nnz, int *flag)
{
    int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v == 0 && (rowptr[0] != 0 || rowptr[n] != nnz)) atomicOr(flag, BAD_ROWPTR);
    if (v < n && (rowptr[v + 1] < rowptr[v] || rowptr[v] < 0 || rowptr[v + 1] > nnz)) atomicOr(flag, BAD_ROWPTR);
}

// one warp per row: range, order, self-loop and symmetry (binary search of v in row u)
__global__ void k_check_cols(const int64_t *__restrict__ rowptr, const int32_t *__restrict__ col, int32_t n, int *flag)
{
    int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (w >= n) return;
    int32_t v = (int32_t)w;
    int64_t b = rowptr[v], e = rowptr[v + 1];
    int bad = 0;
    for (int64_t i = b + lane; i < e; i += 32) {
        int32_t u = col[i];
        if (u < 0 || u >= n) {
            bad |= BAD_COL_RANGE;
            continue;
        }
        if (u == v) bad |= BAD_SELF_LOOP;
        if (i > b && col[i - 1] >= u) bad |= BAD_COL_ORDER;
        int64_t lo = rowptr[u], hi = rowptr[u + 1];
        bool found = false;
        while (lo < hi) {
            int64_t mid = (lo + hi) >> 1;
            int32_t c = col[mid];
            if (c == v) {
                found = true;
                break;
            }
            if (c < v) lo = mid + 1;
            else hi = mid;
        }
        if (!found) bad |= BAD_ASYM;
    }
    if (bad) atomicOr(flag, bad);
}

__global__ void k_dinv(const int64_t *__restrict__ rowptr, int32_t n, float *__restrict__ dinv)
{
    int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v < n) dinv[v] = rsqrtf((float)(rowptr[v + 1] - rowptr[v] + 1));
}

extern "C" sat_status sat_graph_load(sat_ctx *ctx, int32_t n, int64_t nnz, const int64_t *rowptr, const int32_t *col,
                                     int ptr_space)
{
    SatRange sat_range__(__func__);
    if (!ctx) return SAT_EINVAL;
    if (ctx->cuda_failed) return sat_fail(ctx, SAT_ECUDA, "context has a sticky CUDA error");
    if (n <= 0 || nnz < 0 || !rowptr || (nnz > 0 && !col)) return sat_fail(ctx, SAT_EINVAL, "sat_graph_load: bad n / nnz / null array");
    if (nnz + (int64_t)n >= ((int64_t)1 << 31) * 8) return sat_fail(ctx, SAT_EINVAL, "sat_graph_load: graph too large");
    if (ptr_space != SAT_HOST && ptr_space != SAT_DEVICE) return sat_fail(ctx, SAT_EINVAL, "sat_graph_load: bad ptr_space");
    SAT_CUDA(ctx, cudaSetDevice(ctx->device));
    // The new graph is copied and validated in buffers of its own; the context's graph, partition, cache and layer state
    // are replaced only once it has passed, so a rejected graph leaves the context as it was.
    int64_t *t_rowptr = nullptr;
    int32_t *t_col = nullptr;
    float *t_dinv = nullptr;
    auto drop = [&]() {
        dev_free(&t_rowptr);
        dev_free(&t_col);
        dev_free(&t_dinv);
    };
    sat_status rc = dev_alloc(ctx, &t_rowptr, (int64_t)n + 1);
    if (rc == SAT_OK) rc = dev_alloc(ctx, &t_col, nnz);
    if (rc == SAT_OK) rc = dev_alloc(ctx, &t_dinv, n);
    if (rc != SAT_OK) {
        drop();
        return rc;
    }
    cudaMemcpyKind kind = ptr_space == SAT_HOST ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice;
    cudaError_t e = cudaMemcpyAsync(t_rowptr, rowptr, sizeof(int64_t) * ((size_t)n + 1), kind, ctx->stream);
    if (e == cudaSuccess && nnz) e = cudaMemcpyAsync(t_col, col, sizeof(int32_t) * (size_t)nnz, kind, ctx->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->d_flag, 0, sizeof(int), ctx->stream);
    if (e != cudaSuccess) {
        drop();
        return sat_check_cuda(ctx, e, "sat_graph_load: copy of the graph arrays");
    }
    int flag = 0;
    k_check_rowptr<<<(unsigned)cdiv64(n, 256), 256, 0, ctx->stream>>>(t_rowptr, n, nnz, ctx->d_flag);
    ctx->launches++;
    rc = read_flag(ctx, &flag);
    if (rc == SAT_OK && flag) rc = sat_fail(ctx, SAT_EDATA, "sat_graph_load: rowptr is not a monotone offset array ending at nnz");
    if (rc == SAT_OK) {
        k_check_cols<<<(unsigned)cdiv64((int64_t)n * 32, 256), 256, 0, ctx->stream>>>(t_rowptr, t_col, n, ctx->d_flag);
        ctx->launches++;
        rc = read_flag(ctx, &flag);
        if (rc == SAT_OK && flag)
            rc = sat_fail(ctx, SAT_EDATA, "sat_graph_load: malformed graph:%s%s%s%s",
                          (flag & BAD_COL_RANGE) ? " column out of range;" : "",
                          (flag & BAD_COL_ORDER) ? " columns unsorted or duplicated;" : "",
                          (flag & BAD_SELF_LOOP) ? " self-loop stored;" : "", (flag & BAD_ASYM) ? " not symmetric;" : "");
    }
    if (rc == SAT_OK) {
        k_dinv<<<(unsigned)cdiv64(n, 256), 256, 0, ctx->stream>>>(t_rowptr, n, t_dinv);
        ctx->launches++;
        e = cudaGetLastError();
        if (e != cudaSuccess) rc = sat_check_cuda(ctx, e, "kernel launch");
    }
    if (rc != SAT_OK) {
        cudaStreamSynchronize(ctx->stream);
        drop();
        return rc;
    }
    // accepted: the old graph and everything derived from it go
    ctx->graph_ok = false;
    free_partition(ctx);
    free_cache(ctx);
    free_layers(ctx);
    dev_free(&ctx->rowptr);
    dev_free(&ctx->col);
    dev_free(&ctx->dinv);
    ctx->rowptr = t_rowptr;
    ctx->col = t_col;
    ctx->dinv = t_dinv;
    ctx->n = n;
    ctx->nnz = nnz;
    ctx->graph_ok = true;
    return SAT_OK;
}

extern "C" sat_status sat_graph_dinv(sat_ctx *ctx, float *dinv_host)
{
    if (!ctx || !dinv_host) return SAT_EINVAL;
    if (!ctx->graph_ok) return sat_fail(ctx, SAT_ESTATE, "sat_graph_dinv: no graph loaded");
    SAT_CUDA(ctx, cudaMemcpyAsync(dinv_host, ctx->dinv, sizeof(float) * (size_t)ctx->n, cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return SAT_OK;
}

// =====================================================================================
// sat_partition kernels
// =====================================================================================
__global__ void k_part_contig(int32_t n, int32_t M, int32_t *part)
{
    int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v < n) part[v] = (int32_t)((v * (int64_t)M) / n);
}

__global__ void k_part_check(const int32_t *part, int32_t n, int32_t M, int *flag)
{
    int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v < n && (part[v] < 0 || part[v] >= M)) atomicOr(flag, BAD_PART);
}

// histogram of partitions per block of 256 nodes; layout hist[m * n_blk + blk]
__global__ void k_part_hist(const int32_t *__restrict__ part, int32_t n, int32_t M, int32_t n_blk, int32_t *__restrict__ hist)
{
    extern __shared__ int sh_hist[];
    for (int i = threadIdx.x; i < M; i += blockDim.x) sh_hist[i] = 0;
    __syncthreads();
    int64_t v = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (v < n) atomicAdd(&sh_hist[part[v]], 1);
    __syncthreads();
    for (int i = threadIdx.x; i < M; i += blockDim.x) hist[(int64_t)i * n_blk + blockIdx.x] = sh_hist[i];
}

// stable multi-split: position of v = offset(part, block) + number of earlier nodes of the block in the same part
__global__ void k_part_place(const int32_t *__restrict__ part, int32_t n, int32_t n_blk, const int64_t *__restrict__ hist_off,
                             int32_t *__restrict__ perm, int32_t *__restrict__ pos)
{
    __shared__ int sp[256];
    int64_t v = (int64_t)blockIdx.x * 256 + threadIdx.x;
    int p = v < n ? part[v] : -1;
    sp[threadIdx.x] = p;
    __syncthreads();
    if (v >= n) return;
    int rank = 0;
    for (int j = 0; j < (int)threadIdx.x; ++j) rank += (sp[j] == p);
    int32_t r = (int32_t)(hist_off[(int64_t)p * n_blk + blockIdx.x] + rank);
    perm[r] = (int32_t)v;
    pos[v] = r;
}

// halo bitmap: bits[m * nw + (u >> 5)] bit (u & 31) set iff u is adjacent to partition m and not in it
__global__ void k_mark_halo(const int64_t *__restrict__ rowptr, const int32_t *__restrict__ col, const int32_t *__restrict__ part,
                            int32_t n, int32_t nw, uint32_t *__restrict__ bits)
{
    int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (w >= n) return;
    int32_t v = (int32_t)w;
    int32_t m = part[v];
    for (int64_t i = rowptr[v] + lane; i < rowptr[v + 1]; i += 32) {
        int32_t u = col[i];
        if (part[u] != m) atomicOr(&bits[(int64_t)m * nw + (u >> 5)], 1u << (u & 31));
    }
}

__global__ void k_popc(const uint32_t *__restrict__ bits, int64_t count, int32_t *__restrict__ cnt)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) cnt[i] = __popc(bits[i]);
}

// union over partitions of the halo bitmaps = boundary set C
__global__ void k_or_parts(const uint32_t *__restrict__ bits, int32_t M, int32_t nw, uint32_t *__restrict__ cbits)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nw) return;
    uint32_t x = 0;
    for (int m = 0; m < M; ++m) x |= bits[(int64_t)m * nw + i];
    cbits[i] = x;
}

// expand bitmap words into ascending id lists: list[off[word] + k] = 32 * (word % nw) + bit
__global__ void k_expand_bits(const uint32_t *__restrict__ bits, int64_t count, int32_t nw, const int64_t *__restrict__ off,
                              int32_t *__restrict__ list)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    uint32_t x = bits[i];
    int64_t o = off[i];
    int32_t base = (int32_t)(i % nw) * 32;
    while (x) {
        int b = __ffs(x) - 1;
        list[o++] = base + b;
        x &= x - 1;
    }
}

__global__ void k_slot(const uint32_t *__restrict__ cbits, const int64_t *__restrict__ coff, int32_t n, int32_t *__restrict__ slot)
{
    int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n) return;
    uint32_t x = cbits[v >> 5];
    uint32_t bit = 1u << (v & 31);
    slot[v] = (x & bit) ? (int32_t)(coff[v >> 5] + __popc(x & (bit - 1))) : -1;
}

__global__ void k_gather_i32(const int32_t *__restrict__ src, const int32_t *__restrict__ idx, int64_t count, int32_t *__restrict__ out)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) out[i] = src[idx[i]];
}

__global__ void k_push_flag(const int32_t *__restrict__ perm, const int32_t *__restrict__ slot, int32_t n, int32_t *__restrict__ flag)
{
    int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < n) flag[r] = slot[perm[r]] >= 0 ? 1 : 0;
}

__global__ void k_push_fill(const int32_t *__restrict__ perm, const int32_t *__restrict__ slot, int32_t n,
                            const int64_t *__restrict__ off, int32_t *__restrict__ push_row, int32_t *__restrict__ push_slot)
{
    int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n) return;
    int32_t s = slot[perm[r]];
    if (s >= 0) {
        push_row[off[r]] = (int32_t)r;
        push_slot[off[r]] = s;
    }
}

__global__ void k_row_len(const int64_t *__restrict__ rowptr, const int32_t *__restrict__ perm, int32_t n, int32_t *__restrict__ len)
{
    int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < n) {
        int32_t v = perm[r];
        len[r] = (int32_t)(rowptr[v + 1] - rowptr[v]) + 1;
    }
}

// position of halo node u inside the concatenated halo list of partition m
__device__ __forceinline__ int64_t halo_position(const uint32_t *bits, const int64_t *woff, int32_t m, int32_t nw, int32_t u)
{
    int64_t wi = (int64_t)m * nw + (u >> 5);
    return woff[wi] + __popc(bits[wi] & ((1u << (u & 31)) - 1u));
}

// one warp per partition-major row r (node v = perm[r]): local CSR row =
//   [inner neighbours and v itself, ascending]  then  [halo neighbours, ascending]
__global__ void k_fill_local(const int64_t *__restrict__ rowptr, const int32_t *__restrict__ col, const int32_t *__restrict__ part,
                             const int32_t *__restrict__ perm, const int32_t *__restrict__ pos, const uint32_t *__restrict__ bits,
                             const int64_t *__restrict__ woff, int32_t n, int32_t nw, const int64_t *__restrict__ lrowptr,
                             int32_t *__restrict__ lenc, int32_t *__restrict__ inner_cnt)
{
    int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (w >= n) return;
    int32_t r = (int32_t)w;
    int32_t v = perm[r];
    int32_t m = part[v];
    int64_t b = rowptr[v], e = rowptr[v + 1];
    // pass 1: number of inner neighbours, and of those with id < v
    int n_in = 0, n_lt = 0;
    for (int64_t i0 = b; i0 < e; i0 += 32) {
        int64_t i = i0 + lane;
        bool in = false, lt = false;
        if (i < e) {
            int32_t u = col[i];
            in = part[u] == m;
            lt = in && u < v;
        }
        n_in += __popc(__ballot_sync(0xffffffffu, in));
        n_lt += __popc(__ballot_sync(0xffffffffu, lt));
    }
    int64_t o = lrowptr[r];
    if (lane == 0) {
        lenc[o + n_lt] = r;  // self-loop in its sorted place
        inner_cnt[r] = n_in + 1;
    }
    // pass 2: write
    int run_in = 0, run_h = 0;
    for (int64_t i0 = b; i0 < e; i0 += 32) {
        int64_t i = i0 + lane;
        bool valid = i < e;
        int32_t u = valid ? col[i] : 0;
        bool in = valid && part[u] == m;
        bool ha = valid && !in;
        unsigned bi = __ballot_sync(0xffffffffu, in), bh = __ballot_sync(0xffffffffu, ha);
        unsigned lt_mask = (1u << lane) - 1u;
        if (in) {
            int k = run_in + __popc(bi & lt_mask);
            lenc[o + k + (u > v ? 1 : 0)] = pos[u];
        } else if (ha) {
            int k = run_h + __popc(bh & lt_mask);
            lenc[o + n_in + 1 + k] = n + (int32_t)halo_position(bits, woff, m, nw, u);
        }
        run_in += __popc(bi);
        run_h += __popc(bh);
    }
}

__global__ void k_dinv_enc(const float *__restrict__ dinv, const int32_t *__restrict__ perm, const int32_t *__restrict__ halo_gid,
                           int32_t n, int64_t nb, float *__restrict__ out)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = dinv[perm[i]];
    else if (i < n + nb) out[i] = dinv[halo_gid[i - n]];
}

__global__ void k_entry_weights(const int32_t *__restrict__ lenc, const float *__restrict__ dinv_enc, int64_t lnnz, float *__restrict__ lw)
{
    int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e < lnnz) lw[e] = dinv_enc[lenc[e]];
}

// partition of each halo entry: largest m with halo_off[m] <= j
__device__ __forceinline__ int32_t find_part(const int64_t *off, int32_t M, int64_t j)
{
    int lo = 0, hi = M;  // invariant off[lo] <= j < off[hi]
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (off[mid] <= j) lo = mid;
        else hi = mid;
    }
    return lo;
}

// one warp per halo entry j: count / fill its neighbours inside the partition
__global__ void k_hrow(const int64_t *__restrict__ rowptr, const int32_t *__restrict__ col, const int32_t *__restrict__ part,
                       const int32_t *__restrict__ pos, const int32_t *__restrict__ slot, const int32_t *__restrict__ halo_gid,
                       const int64_t *__restrict__ halo_off, int32_t M, int64_t nb, int32_t *__restrict__ cnt,
                       const int64_t *__restrict__ hrow_ptr, int32_t *__restrict__ hrow_pos, int32_t *__restrict__ hrow_slot,
                       const float *__restrict__ dinv, float *__restrict__ hrow_w)
{
    int64_t j = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (j >= nb) return;
    int32_t u = halo_gid[j];
    int32_t m = find_part(halo_off, M, j);
    int64_t b = rowptr[u], e = rowptr[u + 1];
    int run = 0;
    int64_t o = hrow_ptr ? hrow_ptr[j] : 0;
    for (int64_t i0 = b; i0 < e; i0 += 32) {
        int64_t i = i0 + lane;
        int32_t v = i < e ? col[i] : 0;
        bool in = i < e && part[v] == m;
        unsigned bi = __ballot_sync(0xffffffffu, in);
        if (in && hrow_ptr) {
            int k = run + __popc(bi & ((1u << lane) - 1u));
            hrow_pos[o + k] = pos[v];
            hrow_slot[o + k] = slot[v];
            hrow_w[o + k] = dinv[v];
        }
        run += __popc(bi);
    }
    if (lane == 0 && !hrow_ptr) cnt[j] = run;
}

__global__ void k_hlong_flag(const int64_t *__restrict__ hrow_ptr, int64_t nb, int32_t *__restrict__ flag)
{
    int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j < nb) flag[j] = (hrow_ptr[j + 1] - hrow_ptr[j]) > SAT_HROW_LONG ? 1 : 0;
}

__global__ void k_hlong_fill(const int32_t *__restrict__ flag, const int64_t *__restrict__ off, int64_t nb, int32_t *__restrict__ out)
{
    int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (j < nb && flag[j]) out[off[j]] = (int32_t)j;
}

// chunks of the long halo rows
__global__ void k_hchunk_count(const int32_t *__restrict__ hlong, const int64_t *__restrict__ hrow_ptr, int32_t n_hlong, int32_t *__restrict__ nch)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_hlong) {
        const int64_t j = hlong[i];
        nch[i] = (int32_t)((hrow_ptr[j + 1] - hrow_ptr[j] + SAT_HROW_CHUNK - 1) / SAT_HROW_CHUNK);
    }
}

__global__ void k_hchunk_fill(const int64_t *__restrict__ first, int32_t n_hlong, int32_t *__restrict__ chunk_row)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_hlong)
        for (int64_t c = first[i]; c < first[i + 1]; ++c) chunk_row[c] = (int32_t)i;
}

__global__ void k_chunks(const int64_t *__restrict__ lrowptr, int32_t n, int32_t *__restrict__ nch)
{
    int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < n) nch[r] = (int32_t)((lrowptr[r + 1] - lrowptr[r] + SAT_SPMM_CHUNK - 1) / SAT_SPMM_CHUNK);
}

__global__ void k_items(const int64_t *__restrict__ item_off, int32_t n, int32_t *__restrict__ first_item, int32_t *__restrict__ item_row,
                        int32_t *__restrict__ item_multi)
{
    int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r > n) return;
    first_item[r] = (int32_t)item_off[r];
    if (r == n) return;
    int32_t a = (int32_t)item_off[r], b = (int32_t)item_off[r + 1];
    for (int32_t i = a; i < b; ++i) {
        item_row[i] = (int32_t)r;
        item_multi[i] = (b - a) > 1 ? 1 : 0;
    }
}

__global__ void k_item_mslot(const int32_t *__restrict__ item_multi, const int64_t *__restrict__ moff, int32_t n_items,
                             int32_t *__restrict__ item_mslot)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_items) item_mslot[i] = item_multi[i] ? (int32_t)moff[i] : -1;
}

__global__ void k_mrow_flag(const int32_t *__restrict__ first_item, int32_t n, int32_t *__restrict__ flag)
{
    int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < n) flag[r] = (first_item[r + 1] - first_item[r]) > 1 ? 1 : 0;
}

__global__ void k_mrow_fill(const int32_t *__restrict__ flag, const int64_t *__restrict__ off, int32_t n, int32_t *__restrict__ mrows)
{
    int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < n && flag[r]) mrows[off[r]] = (int32_t)r;
}

// =====================================================================================
// sat_partition
// =====================================================================================
static sat_status copy_i64(sat_ctx *ctx, const int64_t *dev, int64_t *host)
{
    SAT_CUDA(ctx, cudaMemcpyAsync(host, dev, sizeof(int64_t), cudaMemcpyDeviceToHost, ctx->stream));
    return SAT_OK;
}

#define GRID1(count) (unsigned)cdiv64((count) > 0 ? (count) : 1, 256), 256, 0, ctx->stream
#define GRIDW(count) (unsigned)cdiv64(((count) > 0 ? (int64_t)(count) : 1) * 32, 256), 256, 0, ctx->stream

// SAT_PART_BFS_BLOCKS: breadth-first visit order of the loaded graph (first-in first-out queue, start at node 0, the
// neighbours of a node taken in ascending id, restart at the smallest unvisited id when the queue runs empty);
// part[v] = floor(rank[v] * M / n).  The visit order of a FIFO traversal is inherently sequential, and this is set-up work
// done once per graph: it runs on the host over a copy of the CSR arrays, and only part[] goes back to the device.
static sat_status bfs_block_partition(sat_ctx *ctx, int32_t M, int32_t *part_dev)
{
    const int32_t n = ctx->n;
    const int64_t nnz = ctx->nnz;
    std::vector<int64_t> rp;
    std::vector<int32_t> cl, order, part;
    std::vector<uint8_t> seen;
    try {
        rp.resize((size_t)n + 1);
        cl.resize((size_t)(nnz > 0 ? nnz : 1));
        order.reserve((size_t)n);
        part.resize((size_t)n);
        seen.assign((size_t)n, 0);
    } catch (const std::bad_alloc &) {
        return sat_fail(ctx, SAT_ENOMEM, "sat_partition: host memory for the breadth-first ordering");
    }
    SAT_CUDA(ctx, cudaMemcpyAsync(rp.data(), ctx->rowptr, sizeof(int64_t) * ((size_t)n + 1), cudaMemcpyDeviceToHost, ctx->stream));
    if (nnz) SAT_CUDA(ctx, cudaMemcpyAsync(cl.data(), ctx->col, sizeof(int32_t) * (size_t)nnz, cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    int32_t next_start = 0;
    size_t head = 0;
    while ((int32_t)order.size() < n) {
        while (seen[next_start]) ++next_start;
        seen[next_start] = 1;
        order.push_back(next_start);
        while (head < order.size()) {
            const int32_t u = order[head++];
            for (int64_t e = rp[u]; e < rp[u + 1]; ++e) {
                const int32_t w = cl[e];
                if (!seen[w]) {
                    seen[w] = 1;
                    order.push_back(w);
                }
            }
        }
    }
    for (int32_t r = 0; r < n; ++r) part[order[r]] = (int32_t)(((int64_t)r * M) / n);
    SAT_CUDA(ctx, cudaMemcpyAsync(part_dev, part.data(), sizeof(int32_t) * (size_t)n, cudaMemcpyHostToDevice, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return SAT_OK;
}

extern "C" sat_status sat_partition(sat_ctx *ctx, int32_t M, int method, const int32_t *part_of_node, int ptr_space)
{
    SatRange sat_range__(__func__);
    if (!ctx) return SAT_EINVAL;
    if (ctx->cuda_failed) return sat_fail(ctx, SAT_ECUDA, "context has a sticky CUDA error");
    if (!ctx->graph_ok) return sat_fail(ctx, SAT_ESTATE, "sat_partition: call sat_graph_load first");
    if (M <= 0 || M > SAT_MAX_PARTS || M > ctx->n) return sat_fail(ctx, SAT_EINVAL, "sat_partition: M must be in [1, min(n, %d)]", SAT_MAX_PARTS);
    if (method != SAT_PART_GIVEN && method != SAT_PART_CONTIG_BLOCKS && method != SAT_PART_BFS_BLOCKS)
        return sat_fail(ctx, SAT_EINVAL, "sat_partition: unknown method");
    if (method == SAT_PART_GIVEN && (!part_of_node || (ptr_space != SAT_HOST && ptr_space != SAT_DEVICE)))
        return sat_fail(ctx, SAT_EINVAL, "sat_partition: SAT_PART_GIVEN needs part_of_node and a valid ptr_space");
    SAT_CUDA(ctx, cudaSetDevice(ctx->device));
    free_partition(ctx);
    free_cache(ctx);
    free_layers(ctx);
    const int32_t n = ctx->n;
    const int32_t nw = (n + 31) / 32;
    const int32_t n_blk = (n + 255) / 256;
    cudaStream_t st = ctx->stream;

    // ---- part[] ----
    SAT_TRY(dev_alloc(ctx, &ctx->part, n));
    if (method == SAT_PART_GIVEN) {
        SAT_CUDA(ctx, cudaMemcpyAsync(ctx->part, part_of_node, sizeof(int32_t) * (size_t)n,
                                      ptr_space == SAT_HOST ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice, st));
        SAT_CUDA(ctx, cudaMemsetAsync(ctx->d_flag, 0, sizeof(int), st));
        k_part_check<<<GRID1(n)>>>(ctx->part, n, M, ctx->d_flag);
        SAT_LAUNCHED(ctx);
        int flag = 0;
        SAT_TRY(read_flag(ctx, &flag));
        if (flag) return sat_fail(ctx, SAT_EINVAL, "sat_partition: part_of_node has a value outside [0, M)");
    } else if (method == SAT_PART_BFS_BLOCKS) {
        SAT_TRY(bfs_block_partition(ctx, M, ctx->part));
    } else {
        k_part_contig<<<GRID1(n)>>>(n, M, ctx->part);
        SAT_LAUNCHED(ctx);
    }

    // temporaries (freed at the end of this function)
    int32_t *t_hist = nullptr, *t_cnt = nullptr, *t_flag = nullptr, *t_item_multi = nullptr;
    int64_t *t_hist_off = nullptr, *t_woff = nullptr, *t_coff = nullptr, *t_off = nullptr, *t_item_off = nullptr, *t_moff = nullptr;
    uint32_t *t_bits = nullptr, *t_cbits = nullptr;
    sat_status rc = SAT_OK;
    auto cleanup = [&]() {
        cudaStreamSynchronize(st);
        dev_free(&t_hist); dev_free(&t_cnt); dev_free(&t_flag); dev_free(&t_item_multi);
        dev_free(&t_hist_off); dev_free(&t_woff); dev_free(&t_coff); dev_free(&t_off); dev_free(&t_item_off); dev_free(&t_moff);
        dev_free(&t_bits); dev_free(&t_cbits);
    };
#define P_TRY(expr)             \
    do {                        \
        rc = (expr);            \
        if (rc != SAT_OK) {     \
            cleanup();          \
            free_partition(ctx);\
            return rc;          \
        }                       \
    } while (0)
#define P_LAUNCHED()                                                   \
    do {                                                               \
        ctx->launches++;                                               \
        cudaError_t e__ = cudaGetLastError();                          \
        if (e__ != cudaSuccess) P_TRY(sat_check_cuda(ctx, e__, "kernel launch")); \
    } while (0)
#define P_CUDA(call)                                                   \
    do {                                                               \
        cudaError_t e__ = (call);                                      \
        if (e__ != cudaSuccess) P_TRY(sat_check_cuda(ctx, e__, #call)); \
    } while (0)

    // ---- I_m: stable multi-split of the node ids by partition ----
    const int64_t n_hist = (int64_t)M * n_blk;
    P_TRY(dev_alloc(ctx, &t_hist, n_hist));
    P_TRY(dev_alloc(ctx, &t_hist_off, n_hist + 1));
    P_TRY(dev_alloc(ctx, &ctx->perm, n));
    P_TRY(dev_alloc(ctx, &ctx->pos, n));
    k_part_hist<<<n_blk, 256, (size_t)M * sizeof(int), st>>>(ctx->part, n, M, n_blk, t_hist);
    P_LAUNCHED();
    P_TRY(sat_scan_i32(ctx, t_hist, n_hist, t_hist_off));
    k_part_place<<<n_blk, 256, 0, st>>>(ctx->part, n, n_blk, t_hist_off, ctx->perm, ctx->pos);
    P_LAUNCHED();
    std::vector<int64_t> tmp64((size_t)M + 1);
    for (int m = 0; m <= M; ++m) {
        if (m < M) P_TRY(copy_i64(ctx, t_hist_off + (int64_t)m * n_blk, &tmp64[m]));
        else tmp64[m] = n;
    }
    P_CUDA(cudaStreamSynchronize(st));
    ctx->h_inner_off.assign(M + 1, 0);
    for (int m = 0; m <= M; ++m) ctx->h_inner_off[m] = (int32_t)tmp64[m];

    // ---- B_m: halo bitmaps -> ascending lists ----
    const int64_t n_words = (int64_t)M * nw;
    P_TRY(dev_alloc(ctx, &t_bits, n_words));
    P_TRY(dev_alloc(ctx, &t_cnt, n_words > n ? n_words : (int64_t)n + 1));
    P_TRY(dev_alloc(ctx, &t_woff, n_words + 1));
    P_CUDA(cudaMemsetAsync(t_bits, 0, sizeof(uint32_t) * (size_t)n_words, st));
    k_mark_halo<<<GRIDW(n)>>>(ctx->rowptr, ctx->col, ctx->part, n, nw, t_bits);
    P_LAUNCHED();
    k_popc<<<GRID1(n_words)>>>(t_bits, n_words, t_cnt);
    P_LAUNCHED();
    P_TRY(sat_scan_i32(ctx, t_cnt, n_words, t_woff));
    ctx->h_halo_off.assign(M + 1, 0);
    for (int m = 0; m <= M; ++m) P_TRY(copy_i64(ctx, t_woff + (int64_t)m * nw, &ctx->h_halo_off[m]));
    P_CUDA(cudaStreamSynchronize(st));
    ctx->nb = ctx->h_halo_off[M];
    if (ctx->nb + (int64_t)n >= ((int64_t)1 << 31)) P_TRY(sat_fail(ctx, SAT_EINVAL, "sat_partition: n + sum of halo sizes exceeds 2^31"));
    P_TRY(dev_alloc(ctx, &ctx->halo_gid, ctx->nb));
    P_TRY(dev_alloc(ctx, &ctx->halo_slot, ctx->nb));
    k_expand_bits<<<GRID1(n_words)>>>(t_bits, n_words, nw, t_woff, ctx->halo_gid);
    P_LAUNCHED();

    // ---- C and slot[] ----
    P_TRY(dev_alloc(ctx, &t_cbits, nw));
    P_TRY(dev_alloc(ctx, &t_coff, (int64_t)nw + 1));
    P_TRY(dev_alloc(ctx, &ctx->slot, n));
    k_or_parts<<<GRID1(nw)>>>(t_bits, M, nw, t_cbits);
    P_LAUNCHED();
    k_popc<<<GRID1(nw)>>>(t_cbits, nw, t_cnt);
    P_LAUNCHED();
    P_TRY(sat_scan_i32(ctx, t_cnt, nw, t_coff));
    int64_t n_slots64 = 0;
    P_TRY(copy_i64(ctx, t_coff + nw, &n_slots64));
    k_slot<<<GRID1(n)>>>(t_cbits, t_coff, n, ctx->slot);
    P_LAUNCHED();
    k_gather_i32<<<GRID1(ctx->nb)>>>(ctx->slot, ctx->halo_gid, ctx->nb, ctx->halo_slot);
    P_LAUNCHED();
    P_CUDA(cudaStreamSynchronize(st));
    ctx->n_slots = (int32_t)n_slots64;

    // ---- push lists ----
    P_TRY(dev_alloc(ctx, &t_flag, (int64_t)n + 1));
    P_TRY(dev_alloc(ctx, &t_off, (int64_t)n + 2));
    P_TRY(dev_alloc(ctx, &ctx->push_row, ctx->n_slots));
    P_TRY(dev_alloc(ctx, &ctx->push_slot, ctx->n_slots));
    k_push_flag<<<GRID1(n)>>>(ctx->perm, ctx->slot, n, t_flag);
    P_LAUNCHED();
    P_TRY(sat_scan_i32(ctx, t_flag, n, t_off));
    k_push_fill<<<GRID1(n)>>>(ctx->perm, ctx->slot, n, t_off, ctx->push_row, ctx->push_slot);
    P_LAUNCHED();
    for (int m = 0; m <= M; ++m) P_TRY(copy_i64(ctx, t_off + ctx->h_inner_off[m], &tmp64[m]));
    P_CUDA(cudaStreamSynchronize(st));
    ctx->h_push_off.assign(M + 1, 0);
    for (int m = 0; m <= M; ++m) ctx->h_push_off[m] = (int32_t)tmp64[m];

    // ---- local CSR ----
    const int64_t lnnz = ctx->nnz + n;
    P_TRY(dev_alloc(ctx, &ctx->lrowptr, (int64_t)n + 1));
    P_TRY(dev_alloc(ctx, &ctx->lenc, lnnz));
    P_TRY(dev_alloc(ctx, &ctx->inner_cnt, n));
    k_row_len<<<GRID1(n)>>>(ctx->rowptr, ctx->perm, n, t_flag);
    P_LAUNCHED();
    P_TRY(sat_scan_i32(ctx, t_flag, n, ctx->lrowptr));
    k_fill_local<<<GRIDW(n)>>>(ctx->rowptr, ctx->col, ctx->part, ctx->perm, ctx->pos, t_bits, t_woff, n, nw, ctx->lrowptr,
                               ctx->lenc, ctx->inner_cnt);
    P_LAUNCHED();
    ctx->h_lnnz_off.assign(M + 1, 0);
    for (int m = 0; m <= M; ++m) P_TRY(copy_i64(ctx, ctx->lrowptr + ctx->h_inner_off[m], &ctx->h_lnnz_off[m]));
    P_TRY(dev_alloc(ctx, &ctx->dinv_enc, (int64_t)n + ctx->nb));
    k_dinv_enc<<<GRID1((int64_t)n + ctx->nb)>>>(ctx->dinv, ctx->perm, ctx->halo_gid, n, ctx->nb, ctx->dinv_enc);
    P_LAUNCHED();
    P_TRY(dev_alloc(ctx, &ctx->lw, lnnz));
    k_entry_weights<<<GRID1(lnnz)>>>(ctx->lenc, ctx->dinv_enc, lnnz, ctx->lw);
    P_LAUNCHED();

    // ---- halo-row CSR ----
    {
        int64_t *d_halo_off = nullptr;
        P_TRY(dev_alloc(ctx, &d_halo_off, (int64_t)M + 1));
        cudaError_t e = cudaMemcpyAsync(d_halo_off, ctx->h_halo_off.data(), sizeof(int64_t) * ((size_t)M + 1), cudaMemcpyHostToDevice, st);
        int32_t *t_hcnt = nullptr;
        if (e == cudaSuccess) rc = dev_alloc(ctx, &t_hcnt, ctx->nb + 1);
        if (e == cudaSuccess && rc == SAT_OK) rc = dev_alloc(ctx, &ctx->hrow_ptr, ctx->nb + 1);
        if (e == cudaSuccess && rc == SAT_OK) {
            k_hrow<<<GRIDW(ctx->nb)>>>(ctx->rowptr, ctx->col, ctx->part, ctx->pos, ctx->slot, ctx->halo_gid, d_halo_off, M, ctx->nb,
                                       t_hcnt, nullptr, nullptr, nullptr, nullptr, nullptr);
            ctx->launches++;
            rc = sat_scan_i32(ctx, t_hcnt, ctx->nb, ctx->hrow_ptr);
        }
        if (e == cudaSuccess && rc == SAT_OK) rc = copy_i64(ctx, ctx->hrow_ptr + ctx->nb, &ctx->nnz_cut);
        if (e == cudaSuccess && rc == SAT_OK) e = cudaStreamSynchronize(st);
        if (e == cudaSuccess && rc == SAT_OK) rc = dev_alloc(ctx, &ctx->hrow_pos, ctx->nnz_cut);
        if (e == cudaSuccess && rc == SAT_OK) rc = dev_alloc(ctx, &ctx->hrow_slot, ctx->nnz_cut);
        if (e == cudaSuccess && rc == SAT_OK) rc = dev_alloc(ctx, &ctx->hrow_w, ctx->nnz_cut);
        if (e == cudaSuccess && rc == SAT_OK) {
            k_hrow<<<GRIDW(ctx->nb)>>>(ctx->rowptr, ctx->col, ctx->part, ctx->pos, ctx->slot, ctx->halo_gid, d_halo_off, M, ctx->nb,
                                       nullptr, ctx->hrow_ptr, ctx->hrow_pos, ctx->hrow_slot, ctx->dinv, ctx->hrow_w);
            ctx->launches++;
            e = cudaGetLastError();
        }
        ctx->h_hrow_off.assign(M + 1, 0);
        for (int m = 0; m <= M && e == cudaSuccess && rc == SAT_OK; ++m) rc = copy_i64(ctx, ctx->hrow_ptr + ctx->h_halo_off[m], &ctx->h_hrow_off[m]);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        dev_free(&d_halo_off);
        dev_free(&t_hcnt);
        if (e != cudaSuccess) P_TRY(sat_check_cuda(ctx, e, "halo-row CSR"));
        P_TRY(rc);
    }

    // ---- long halo rows (hubs adjacent to many nodes of one partition) get their own list ----
    {
        int32_t *t_hf = nullptr;
        int64_t *t_ho = nullptr;
        P_TRY(dev_alloc(ctx, &t_hf, ctx->nb + 1));
        rc = dev_alloc(ctx, &t_ho, ctx->nb + 2);
        if (rc == SAT_OK) {
            k_hlong_flag<<<GRID1(ctx->nb)>>>(ctx->hrow_ptr, ctx->nb, t_hf);
            ctx->launches++;
            rc = sat_scan_i32(ctx, t_hf, ctx->nb, t_ho);
        }
        int64_t n_hl = 0;
        std::vector<int64_t> off_h((size_t)M + 1, 0);
        if (rc == SAT_OK) rc = copy_i64(ctx, t_ho + ctx->nb, &n_hl);
        for (int m = 0; m <= M && rc == SAT_OK; ++m) rc = copy_i64(ctx, t_ho + ctx->h_halo_off[m], &off_h[m]);
        cudaError_t e = cudaStreamSynchronize(st);
        if (rc == SAT_OK && e == cudaSuccess) {
            ctx->n_hlong = (int32_t)n_hl;
            ctx->h_hlong_off.assign(M + 1, 0);
            for (int m = 0; m <= M; ++m) ctx->h_hlong_off[m] = (int32_t)off_h[m];
            rc = dev_alloc(ctx, &ctx->hlong, ctx->n_hlong);
        }
        if (rc == SAT_OK && e == cudaSuccess) {
            k_hlong_fill<<<GRID1(ctx->nb)>>>(t_hf, t_ho, ctx->nb, ctx->hlong);
            ctx->launches++;
            e = cudaStreamSynchronize(st);
        }
        dev_free(&t_hf);
        dev_free(&t_ho);
        if (e != cudaSuccess) P_TRY(sat_check_cuda(ctx, e, "long halo rows"));
        P_TRY(rc);
        // ... and are cut into chunks of SAT_HROW_CHUNK entries
        ctx->h_hchunk_off.assign(M + 1, 0);
        ctx->n_hchunks = 0;
        if (ctx->n_hlong > 0) {
            int32_t *t_nch = nullptr;
            P_TRY(dev_alloc(ctx, &t_nch, ctx->n_hlong + 1));
            rc = dev_alloc(ctx, &ctx->hchunk_first, (int64_t)ctx->n_hlong + 2);
            if (rc == SAT_OK) {
                k_hchunk_count<<<GRID1(ctx->n_hlong)>>>(ctx->hlong, ctx->hrow_ptr, ctx->n_hlong, t_nch);
                ctx->launches++;
                rc = sat_scan_i32(ctx, t_nch, ctx->n_hlong, ctx->hchunk_first);
            }
            std::vector<int64_t> off_c((size_t)M + 1, 0);
            for (int m = 0; m <= M && rc == SAT_OK; ++m) rc = copy_i64(ctx, ctx->hchunk_first + ctx->h_hlong_off[m], &off_c[m]);
            e = cudaStreamSynchronize(st);
            if (rc == SAT_OK && e == cudaSuccess) {
                for (int m = 0; m <= M; ++m) ctx->h_hchunk_off[m] = (int32_t)off_c[m];
                ctx->n_hchunks = (int32_t)off_c[M];
                rc = dev_alloc(ctx, &ctx->hchunk_row, ctx->n_hchunks);
            }
            if (rc == SAT_OK && e == cudaSuccess) {
                k_hchunk_fill<<<GRID1(ctx->n_hlong)>>>(ctx->hchunk_first, ctx->n_hlong, ctx->hchunk_row);
                ctx->launches++;
                e = cudaStreamSynchronize(st);
            }
            dev_free(&t_nch);
            if (e != cudaSuccess) P_TRY(sat_check_cuda(ctx, e, "chunks of the long halo rows"));
            P_TRY(rc);
        }
    }

    // ---- SpMM work items ----
    P_TRY(dev_alloc(ctx, &t_item_off, (int64_t)n + 2));
    P_TRY(dev_alloc(ctx, &ctx->first_item, (int64_t)n + 1));
    k_chunks<<<GRID1(n)>>>(ctx->lrowptr, n, t_flag);
    P_LAUNCHED();
    P_TRY(sat_scan_i32(ctx, t_flag, n, t_item_off));
    int64_t n_items64 = 0;
    P_TRY(copy_i64(ctx, t_item_off + n, &n_items64));
    P_CUDA(cudaStreamSynchronize(st));
    if (n_items64 >= ((int64_t)1 << 31)) P_TRY(sat_fail(ctx, SAT_EINVAL, "sat_partition: too many work items"));
    ctx->n_items = (int32_t)n_items64;
    P_TRY(dev_alloc(ctx, &ctx->item_row, ctx->n_items));
    P_TRY(dev_alloc(ctx, &ctx->item_mslot, ctx->n_items));
    P_TRY(dev_alloc(ctx, &t_item_multi, (int64_t)ctx->n_items + 1));
    P_TRY(dev_alloc(ctx, &t_moff, (int64_t)ctx->n_items + 2));
    k_items<<<GRID1((int64_t)n + 1)>>>(t_item_off, n, ctx->first_item, ctx->item_row, t_item_multi);
    P_LAUNCHED();
    P_TRY(sat_scan_i32(ctx, t_item_multi, ctx->n_items, t_moff));
    k_item_mslot<<<GRID1(ctx->n_items)>>>(t_item_multi, t_moff, ctx->n_items, ctx->item_mslot);
    P_LAUNCHED();
    int64_t n_mitems64 = 0;
    P_TRY(copy_i64(ctx, t_moff + ctx->n_items, &n_mitems64));
    ctx->h_item_off.assign(M + 1, 0);
    ctx->h_mitem_off.assign(M + 1, 0);
    ctx->h_mrow_off.assign(M + 1, 0);
    std::vector<int64_t> item_off_h((size_t)M + 1), mitem_off_h((size_t)M + 1), mrow_off_h((size_t)M + 1);
    for (int m = 0; m <= M; ++m) P_TRY(copy_i64(ctx, t_item_off + ctx->h_inner_off[m], &item_off_h[m]));
    P_CUDA(cudaStreamSynchronize(st));
    for (int m = 0; m <= M; ++m) {
        ctx->h_item_off[m] = (int32_t)item_off_h[m];
        P_TRY(copy_i64(ctx, t_moff + ctx->h_item_off[m], &mitem_off_h[m]));
    }
    // multi-chunk rows
    k_mrow_flag<<<GRID1(n)>>>(ctx->first_item, n, t_flag);
    P_LAUNCHED();
    P_TRY(sat_scan_i32(ctx, t_flag, n, t_off));
    int64_t n_mrows64 = 0;
    P_TRY(copy_i64(ctx, t_off + n, &n_mrows64));
    for (int m = 0; m <= M; ++m) P_TRY(copy_i64(ctx, t_off + ctx->h_inner_off[m], &mrow_off_h[m]));
    P_CUDA(cudaStreamSynchronize(st));
    ctx->n_mitems = (int32_t)n_mitems64;
    ctx->n_mrows = (int32_t)n_mrows64;
    for (int m = 0; m <= M; ++m) {
        ctx->h_mitem_off[m] = (int32_t)mitem_off_h[m];
        ctx->h_mrow_off[m] = (int32_t)mrow_off_h[m];
    }
    P_TRY(dev_alloc(ctx, &ctx->mrows, ctx->n_mrows));
    k_mrow_fill<<<GRID1(n)>>>(t_flag, t_off, n, ctx->mrows);
    P_LAUNCHED();

    cleanup();
    if (ctx->cuda_failed) return SAT_ECUDA;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return sat_check_cuda(ctx, e, "sat_partition");
    ctx->M = M;
    ctx->part_ok = true;
    return SAT_OK;
}

sat_status sat_part_view(sat_ctx *ctx, int32_t part, PartView *v)
{
    if (!ctx->part_ok) return sat_fail(ctx, SAT_ESTATE, "no partition: call sat_partition first");
    if (part != SAT_ALL_PARTS && (part < 0 || part >= ctx->M)) return sat_fail(ctx, SAT_EINVAL, "partition index %d out of range", part);
    int a = part == SAT_ALL_PARTS ? 0 : part, b = part == SAT_ALL_PARTS ? ctx->M : part + 1;
    v->row0 = ctx->h_inner_off[a];
    v->n_rows = ctx->h_inner_off[b] - v->row0;
    v->halo0 = ctx->h_halo_off[a];
    v->n_halo = ctx->h_halo_off[b] - v->halo0;
    v->item0 = ctx->h_item_off[a];
    v->n_items = ctx->h_item_off[b] - v->item0;
    v->mrow0 = ctx->h_mrow_off[a];
    v->n_mrows = ctx->h_mrow_off[b] - v->mrow0;
    v->mitem0 = ctx->h_mitem_off[a];
    v->n_mitems = ctx->h_mitem_off[b] - v->mitem0;
    v->push0 = ctx->h_push_off[a];
    v->n_push = ctx->h_push_off[b] - v->push0;
    v->lnnz = ctx->h_lnnz_off[b] - ctx->h_lnnz_off[a];
    v->hnnz = ctx->h_hrow_off.empty() ? 0 : ctx->h_hrow_off[b] - ctx->h_hrow_off[a];
    v->hlong0 = ctx->h_hlong_off[a];
    v->n_hlong = ctx->h_hlong_off[b] - v->hlong0;
    v->hchunk0 = ctx->h_hchunk_off.empty() ? 0 : ctx->h_hchunk_off[a];
    v->n_hchunks = ctx->h_hchunk_off.empty() ? 0 : ctx->h_hchunk_off[b] - v->hchunk0;
    return SAT_OK;
}

// =====================================================================================
// queries
// =====================================================================================
extern "C" sat_status sat_part_sizes(sat_ctx *ctx, int32_t m, int32_t *n_inner, int32_t *n_halo, int64_t *nnz_local,
                                     int32_t *n_push, int64_t *nnz_hrow)
{
    if (!ctx) return SAT_EINVAL;
    PartView v;
    SAT_TRY(sat_part_view(ctx, m, &v));
    int a = m == SAT_ALL_PARTS ? 0 : m, b = m == SAT_ALL_PARTS ? ctx->M : m + 1;
    if (n_inner) *n_inner = v.n_rows;
    if (n_halo) *n_halo = (int32_t)v.n_halo;
    if (nnz_local) *nnz_local = ctx->h_lnnz_off[b] - ctx->h_lnnz_off[a];
    if (n_push) *n_push = v.n_push;
    if (nnz_hrow) *nnz_hrow = ctx->h_hrow_off[b] - ctx->h_hrow_off[a];
    return SAT_OK;
}

// local column id from the encoded column
__global__ void k_decode_cols(const int32_t *__restrict__ lenc, int64_t count, int32_t n, int32_t row0, int32_t n_rows, int64_t halo0,
                              int32_t *__restrict__ out)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    int32_t c = lenc[i];
    out[i] = c < n ? c - row0 : n_rows + (int32_t)((int64_t)(c - n) - halo0);
}

__global__ void k_sub_i32(const int32_t *__restrict__ in, int64_t count, int32_t delta, int32_t *__restrict__ out)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) out[i] = in[i] - delta;
}

__global__ void k_sub_i64(const int64_t *__restrict__ in, int64_t count, int64_t delta, int64_t *__restrict__ out)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) out[i] = in[i] - delta;
}

extern "C" sat_status sat_part_lists(sat_ctx *ctx, int32_t m, int32_t *inner_gid, int32_t *halo_gid, int32_t *halo_slot,
                                     int32_t *push_local, int32_t *push_slot, int64_t *loc_rowptr, int32_t *loc_col,
                                     int64_t *hrow_ptr, int32_t *hrow_col)
{
    if (!ctx) return SAT_EINVAL;
    if (m == SAT_ALL_PARTS) return sat_fail(ctx, SAT_EINVAL, "sat_part_lists: needs a single partition");
    PartView v;
    SAT_TRY(sat_part_view(ctx, m, &v));
    cudaStream_t st = ctx->stream;
    const int64_t lnnz = ctx->h_lnnz_off[m + 1] - ctx->h_lnnz_off[m];
    const int64_t hnnz = ctx->h_hrow_off[m + 1] - ctx->h_hrow_off[m];
    size_t need = sizeof(int64_t) * (size_t)((lnnz > hnnz ? lnnz : hnnz) + v.n_rows + v.n_halo + 8);
    SAT_TRY(sat_ensure(ctx, ctx->buf_gagg, need));
    void *tmp = ctx->buf_gagg.p;
#define D2H(dst, src, bytes) SAT_CUDA(ctx, cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, st))
    if (inner_gid) D2H(inner_gid, ctx->perm + v.row0, sizeof(int32_t) * (size_t)v.n_rows);
    if (halo_gid) D2H(halo_gid, ctx->halo_gid + v.halo0, sizeof(int32_t) * (size_t)v.n_halo);
    if (halo_slot) D2H(halo_slot, ctx->halo_slot + v.halo0, sizeof(int32_t) * (size_t)v.n_halo);
    if (push_slot) D2H(push_slot, ctx->push_slot + v.push0, sizeof(int32_t) * (size_t)v.n_push);
    if (push_local) {
        k_sub_i32<<<GRID1(v.n_push)>>>(ctx->push_row + v.push0, v.n_push, v.row0, (int32_t *)tmp);
        SAT_LAUNCHED(ctx);
        D2H(push_local, tmp, sizeof(int32_t) * (size_t)v.n_push);
        SAT_CUDA(ctx, cudaStreamSynchronize(st));
    }
    if (loc_rowptr) {
        k_sub_i64<<<GRID1((int64_t)v.n_rows + 1)>>>(ctx->lrowptr + v.row0, (int64_t)v.n_rows + 1, ctx->h_lnnz_off[m], (int64_t *)tmp);
        SAT_LAUNCHED(ctx);
        D2H(loc_rowptr, tmp, sizeof(int64_t) * ((size_t)v.n_rows + 1));
        SAT_CUDA(ctx, cudaStreamSynchronize(st));
    }
    if (loc_col) {
        k_decode_cols<<<GRID1(lnnz)>>>(ctx->lenc + ctx->h_lnnz_off[m], lnnz, ctx->n, v.row0, v.n_rows, v.halo0, (int32_t *)tmp);
        SAT_LAUNCHED(ctx);
        D2H(loc_col, tmp, sizeof(int32_t) * (size_t)lnnz);
        SAT_CUDA(ctx, cudaStreamSynchronize(st));
    }
    if (hrow_ptr) {
        k_sub_i64<<<GRID1(v.n_halo + 1)>>>(ctx->hrow_ptr + v.halo0, v.n_halo + 1, ctx->h_hrow_off[m], (int64_t *)tmp);
        SAT_LAUNCHED(ctx);
        D2H(hrow_ptr, tmp, sizeof(int64_t) * ((size_t)v.n_halo + 1));
        SAT_CUDA(ctx, cudaStreamSynchronize(st));
    }
    if (hrow_col) {
        k_sub_i32<<<GRID1(hnnz)>>>(ctx->hrow_pos + ctx->h_hrow_off[m], hnnz, v.row0, (int32_t *)tmp);
        SAT_LAUNCHED(ctx);
        D2H(hrow_col, tmp, sizeof(int32_t) * (size_t)hnnz);
        SAT_CUDA(ctx, cudaStreamSynchronize(st));
    }
#undef D2H
    SAT_CUDA(ctx, cudaStreamSynchronize(st));
    return SAT_OK;
}

extern "C" sat_status sat_slot_map(sat_ctx *ctx, int32_t *part_host, int32_t *slot_host, int32_t *n_slots)
{
    if (!ctx) return SAT_EINVAL;
    if (!ctx->part_ok) return sat_fail(ctx, SAT_ESTATE, "sat_slot_map: call sat_partition first");
    if (part_host) SAT_CUDA(ctx, cudaMemcpyAsync(part_host, ctx->part, sizeof(int32_t) * (size_t)ctx->n, cudaMemcpyDeviceToHost, ctx->stream));
    if (slot_host) SAT_CUDA(ctx, cudaMemcpyAsync(slot_host, ctx->slot, sizeof(int32_t) * (size_t)ctx->n, cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (n_slots) *n_slots = ctx->n_slots;
    return SAT_OK;
}
