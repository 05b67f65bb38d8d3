// Entry points of the per-epoch steps: halo pull, predictor, layer forward / backward,
// cache push / commit, loss seed and parameter step.
#include <cstdlib>

#include "sat_internal.h"

#include <algorithm>
#include <cstdlib>
#include <vector>


template <typename T>
static sat_status dev_realloc(sat_ctx *ctx, T **p, int64_t count)
{
    if (*p) {
        SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        cudaFree(*p);
        *p = nullptr;
    }
    SAT_CUDA(ctx, cudaMalloc((void **)p, (size_t)(count > 0 ? count : 1) * sizeof(T)));
    return SAT_OK;
}

// =====================================================================================
// sat_gather_rows
// =====================================================================================
extern "C" sat_status sat_gather_rows(sat_ctx *ctx, int32_t part, int which, const float *x, int32_t ld_x, int32_t d, float *out,
                                      int32_t ld_out)
{
    CHECK_CTX(ctx);
    PartView v;
    SAT_TRY(sat_part_view(ctx, part, &v));
    if (which != SAT_ROWS_INNER && which != SAT_ROWS_HALO) return sat_fail(ctx, SAT_EINVAL, "sat_gather_rows: bad row selector");
    const int64_t count = which == SAT_ROWS_INNER ? v.n_rows : v.n_halo;
    if (count == 0) return SAT_OK;
    if (!x || !out || d <= 0 || !ok_ld(ld_x, d) || !ok_ld(ld_out, d) || !aligned16(x) || !aligned16(out))
        return sat_fail(ctx, SAT_EINVAL, "sat_gather_rows: null / misaligned tensor or bad leading dimension");
    const int32_t *idx = which == SAT_ROWS_INNER ? ctx->perm + v.row0 : ctx->halo_gid + v.halo0;
    return sat_gather(ctx, idx, count, d, x, ld_x, out, ld_out, DbgRange{0, ctx->n});
}

// =====================================================================================
// cache ring
// =====================================================================================
extern "C" sat_status sat_cache_init(sat_ctx *ctx, int32_t n_cached_layers, const int32_t *width, int32_t tau, int mode,
                                     const float *const *init)
{
    CHECK_CTX(ctx);
    if (!ctx->part_ok) return sat_fail(ctx, SAT_ESTATE, "sat_cache_init: call sat_partition first");
    if (n_cached_layers < 0 || n_cached_layers > SAT_MAX_LAYERS || tau < 1 || (n_cached_layers > 0 && !width))
        return sat_fail(ctx, SAT_EINVAL, "sat_cache_init: bad layer count / tau");
    if (mode != SAT_CACHE_ZERO && mode != SAT_CACHE_COPY) return sat_fail(ctx, SAT_EINVAL, "sat_cache_init: bad mode");
    if (mode == SAT_CACHE_COPY && !init) return sat_fail(ctx, SAT_EINVAL, "sat_cache_init: SAT_CACHE_COPY needs init");
    for (int i = 0; i < n_cached_layers; ++i)
        if (width[i] <= 0 || (mode == SAT_CACHE_COPY && (!init[i] || !aligned16(init[i]))))
            return sat_fail(ctx, SAT_EINVAL, "sat_cache_init: bad width or init pointer for layer %d", i + 1);
    for (int i = 0; i < SAT_MAX_LAYERS; ++i) {
        if (ctx->cache[i].buf) cudaFree(ctx->cache[i].buf);
        if (ctx->cache[i].S) cudaFree(ctx->cache[i].S);
        if (ctx->cache[i].proj) cudaFree(ctx->cache[i].proj);
        ctx->cache[i] = CacheLayer();
    }
    ctx->cache_ok = false;
    for (int i = 0; i < n_cached_layers; ++i) {
        CacheLayer &c = ctx->cache[i];
        c.width = width[i];
        c.ld = round_up4(width[i]);
        const size_t bytes = (size_t)(tau + 1) * (size_t)ctx->n_slots * c.ld * sizeof(float);
        SAT_CUDA(ctx, cudaMalloc((void **)&c.buf, bytes ? bytes : 16));
        SAT_CUDA(ctx, cudaMemsetAsync(c.buf, 0, bytes, ctx->stream));
        if (mode == SAT_CACHE_COPY && ctx->n_slots > 0)
            SAT_CUDA(ctx, cudaMemcpyAsync(c.buf, init[i], (size_t)ctx->n_slots * c.ld * sizeof(float), cudaMemcpyDeviceToDevice, ctx->stream));
    }
    ctx->n_cached = n_cached_layers;
    ctx->tau = tau;
    ctx->write_idx = mode == SAT_CACHE_COPY ? 1 : 0;
    ctx->n_valid = mode == SAT_CACHE_COPY ? 1 : 0;
    ctx->cache_ok = true;
    return SAT_OK;
}

static sat_status cache_layer(sat_ctx *ctx, int32_t layer, CacheLayer **c, const char *who)
{
    if (!ctx->cache_ok) return sat_fail(ctx, SAT_ESTATE, "%s: call sat_cache_init first", who);
    if (layer < 1 || layer > ctx->n_cached) return sat_fail(ctx, SAT_EINVAL, "%s: cached layer %d out of range [1, %d]", who, layer, ctx->n_cached);
    *c = &ctx->cache[layer - 1];
    return SAT_OK;
}

// buffer index of the snapshot of a given age (0 = newest committed)

extern "C" sat_status sat_cache_update(sat_ctx *ctx, int32_t part, int32_t layer, const float *h_out, int32_t ld)
{
    CHECK_CTX(ctx);
    CacheLayer *c;
    SAT_TRY(cache_layer(ctx, layer, &c, "sat_cache_update"));
    PartView v;
    SAT_TRY(sat_part_view(ctx, part, &v));
    if (v.n_push == 0) return SAT_OK;
    if (!h_out || !ok_ld(ld, c->width) || !aligned16(h_out)) return sat_fail(ctx, SAT_EINVAL, "sat_cache_update: null / misaligned h_out or bad ld");
    if (!c->proj_tag.empty()) c->proj_tag[ctx->write_idx] = 0;  // the buffer changes: its cached input projection is stale
    const float *src_base = h_out - (int64_t)v.row0 * ld;
    return sat_scatter(ctx, ctx->push_row + v.push0, ctx->push_slot + v.push0, v.n_push, c->width, src_base, ld,
                       ring_buf(ctx, c, ctx->write_idx), c->ld, DbgRange{v.row0, (int64_t)v.row0 + v.n_rows}, DbgRange{0, ctx->n_slots});
}

extern "C" sat_status sat_cache_commit(sat_ctx *ctx)
{
    CHECK_CTX(ctx);
    if (!ctx->cache_ok) return sat_fail(ctx, SAT_ESTATE, "sat_cache_commit: call sat_cache_init first");
    ctx->write_idx = (ctx->write_idx + 1) % (ctx->tau + 1);
    ctx->n_valid = ctx->n_valid + 1 < ctx->tau ? ctx->n_valid + 1 : ctx->tau;
    for (int i = 0; i < ctx->n_cached; ++i) ctx->cache[i].S_valid = false;
    // gradient-side history: what the epoch collected becomes readable, the other buffer starts the next epoch at zero
    for (int l = 0; l <= SAT_MAX_LAYERS; ++l) {
        GradHist &GH = ctx->ghist[l];
        if (!GH.buf) continue;
        const size_t plane = (size_t)ctx->n_slots * GH.ld;
        GH.read_idx = 1 - GH.read_idx;
        GH.has_read = true;
        SAT_CUDA(ctx, cudaMemsetAsync(GH.buf + (size_t)(1 - GH.read_idx) * plane, 0, plane * sizeof(float), ctx->stream));
    }
    return SAT_OK;
}

extern "C" sat_status sat_grad_history_read(sat_ctx *ctx, int32_t layer, int which, float *out_host)
{
    CHECK_CTX(ctx);
    if (layer < 2 || layer > SAT_MAX_LAYERS || !out_host || (which != 0 && which != 1))
        return sat_fail(ctx, SAT_EINVAL, "sat_grad_history_read: layer must be in [2, %d], which 0 or 1, output non-null", SAT_MAX_LAYERS);
    GradHist &GH = ctx->ghist[layer];
    if (!GH.buf || (which == 0 && !GH.has_read)) return sat_fail(ctx, SAT_ESTATE, "sat_grad_history_read: no such history for layer %d", layer);
    const size_t plane = (size_t)ctx->n_slots * GH.ld;
    const float *src = GH.buf + (size_t)(which == 0 ? GH.read_idx : 1 - GH.read_idx) * plane;
    SAT_CUDA(ctx, cudaMemcpy2DAsync(out_host, (size_t)GH.width * 4, src, (size_t)GH.ld * 4, (size_t)GH.width * 4, (size_t)ctx->n_slots,
                                    cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return SAT_OK;
}

extern "C" sat_status sat_grad_history_write(sat_ctx *ctx, int32_t layer, int32_t width, const float *in_host)
{
    CHECK_CTX(ctx);
    if (!ctx->part_ok) return sat_fail(ctx, SAT_ESTATE, "sat_grad_history_write: call sat_partition first");
    if (layer < 2 || layer > SAT_MAX_LAYERS || width <= 0) return sat_fail(ctx, SAT_EINVAL, "sat_grad_history_write: bad layer or width");
    GradHist &GH = ctx->ghist[layer];
    const int32_t ld_q = round_up4(width);
    const size_t plane = (size_t)ctx->n_slots * ld_q;
    if (!GH.buf || GH.width != width) {
        SAT_TRY(dev_realloc(ctx, &GH.buf, (int64_t)(2 * plane > 0 ? 2 * plane : 1)));
        GH.width = width;
        GH.ld = ld_q;
        GH.read_idx = 0;
    }
    SAT_CUDA(ctx, cudaMemsetAsync(GH.buf, 0, 2 * plane * sizeof(float), ctx->stream));
    GH.has_read = in_host != nullptr;
    if (in_host && ctx->n_slots > 0)
        SAT_CUDA(ctx, cudaMemcpy2DAsync(GH.buf + (size_t)GH.read_idx * plane, (size_t)ld_q * 4, in_host, (size_t)width * 4, (size_t)width * 4,
                                        (size_t)ctx->n_slots, cudaMemcpyHostToDevice, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return SAT_OK;
}

extern "C" sat_status sat_cache_requantise(sat_ctx *ctx, int32_t layer, int32_t age, int32_t precision, int64_t *bytes)
{
    CHECK_CTX(ctx);
    CacheLayer *c;
    SAT_TRY(cache_layer(ctx, layer, &c, "sat_cache_requantise"));
    if (age < 0 || age >= (ctx->n_valid < ctx->tau ? ctx->n_valid : ctx->tau))
        return sat_fail(ctx, SAT_EINVAL, "sat_cache_requantise: age %d outside the %d committed snapshots", age, ctx->n_valid < ctx->tau ? ctx->n_valid : ctx->tau);
    if (precision < 0 || precision > 7) return sat_fail(ctx, SAT_EINVAL, "sat_cache_requantise: precision outside 0..7");
    const int32_t idx = ring_index(ctx, age);
    SAT_TRY(sat_codec_roundtrip(ctx, ring_buf(ctx, c, idx), c->ld, ctx->n_slots, c->width, precision, bytes));
    if (!c->proj_tag.empty()) c->proj_tag[idx] = 0;  // the cached projection was made from the unquantised snapshot
    c->S_valid = false;
    return SAT_OK;
}

extern "C" sat_status sat_cache_state(sat_ctx *ctx, int32_t *write_idx, int32_t *n_valid)
{
    if (!ctx) return SAT_EINVAL;
    if (!ctx->cache_ok) return sat_fail(ctx, SAT_ESTATE, "sat_cache_state: call sat_cache_init first");
    if (write_idx) *write_idx = ctx->write_idx;
    if (n_valid) *n_valid = ctx->n_valid;
    return SAT_OK;
}

extern "C" sat_status sat_cache_set_state(sat_ctx *ctx, int32_t write_idx, int32_t n_valid)
{
    if (!ctx) return SAT_EINVAL;
    if (!ctx->cache_ok) return sat_fail(ctx, SAT_ESTATE, "sat_cache_set_state: call sat_cache_init first");
    if (write_idx < 0 || write_idx > ctx->tau || n_valid < 0 || n_valid > ctx->tau) return sat_fail(ctx, SAT_EINVAL, "sat_cache_set_state: out of range");
    ctx->write_idx = write_idx;
    ctx->n_valid = n_valid;
    for (int i = 0; i < ctx->n_cached; ++i) {
        ctx->cache[i].S_valid = false;
        ctx->cache[i].proj_tag.assign(ctx->cache[i].proj_tag.size(), 0);
    }
    return SAT_OK;
}

extern "C" sat_status sat_cache_read(sat_ctx *ctx, int32_t layer, int32_t age, float *out_host)
{
    CHECK_CTX(ctx);
    CacheLayer *c;
    SAT_TRY(cache_layer(ctx, layer, &c, "sat_cache_read"));
    if (!out_host || age < -1 || age >= ctx->n_valid) return sat_fail(ctx, SAT_EINVAL, "sat_cache_read: null output or age outside [-1, n_valid)");
    if (ctx->n_slots == 0) return SAT_OK;
    const int32_t idx = age < 0 ? ctx->write_idx : ring_index(ctx, age);
    SAT_CUDA(ctx, cudaMemcpy2DAsync(out_host, (size_t)c->width * 4, ring_buf(ctx, c, idx), (size_t)c->ld * 4, (size_t)c->width * 4,
                                    (size_t)ctx->n_slots, cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return SAT_OK;
}

extern "C" sat_status sat_cache_export(sat_ctx *ctx, int32_t layer, float *out_host)
{
    CHECK_CTX(ctx);
    CacheLayer *c;
    SAT_TRY(cache_layer(ctx, layer, &c, "sat_cache_export"));
    if (!out_host) return sat_fail(ctx, SAT_EINVAL, "sat_cache_export: null output");
    const size_t rows = (size_t)(ctx->tau + 1) * ctx->n_slots;
    if (rows == 0) return SAT_OK;
    SAT_CUDA(ctx, cudaMemcpy2DAsync(out_host, (size_t)c->width * 4, c->buf, (size_t)c->ld * 4, (size_t)c->width * 4, rows,
                                    cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return SAT_OK;
}

extern "C" sat_status sat_cache_import(sat_ctx *ctx, int32_t layer, const float *in_host)
{
    CHECK_CTX(ctx);
    CacheLayer *c;
    SAT_TRY(cache_layer(ctx, layer, &c, "sat_cache_import"));
    if (!in_host) return sat_fail(ctx, SAT_EINVAL, "sat_cache_import: null input");
    const size_t rows = (size_t)(ctx->tau + 1) * ctx->n_slots;
    c->S_valid = false;
    c->proj_tag.assign(c->proj_tag.size(), 0);
    if (rows == 0) return SAT_OK;
    SAT_CUDA(ctx, cudaMemcpy2DAsync(c->buf, (size_t)c->ld * 4, in_host, (size_t)c->width * 4, (size_t)c->width * 4, rows,
                                    cudaMemcpyHostToDevice, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return SAT_OK;
}

// =====================================================================================
// sat_predict
// =====================================================================================
// a = x Wx (+ s Uh) + b computed by the dense path into `gates` [rows x 4h] (gate blocks i | f | g | o);
// this kernel applies the cell:  c = f c + i g ; s = o tanh(c).
__global__ void k_lstm_cell(const float *__restrict__ gates, int64_t rows, int32_t h, int first, float *__restrict__ c, float *__restrict__ s)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= rows * h) return;
    const int64_t r = t / h;
    const int j = (int)(t - r * h);
    const float *a = gates + r * 4 * (int64_t)h;
    const float gi = 1.f / (1.f + expf(-a[j]));
    const float gf = 1.f / (1.f + expf(-a[h + j]));
    const float gg = tanhf(a[2 * h + j]);
    const float go = 1.f / (1.f + expf(-a[3 * h + j]));
    const float cp = first ? 0.f : c[t];
    const float cn = gf * cp + gi * gg;
    c[t] = cn;
    s[t] = go * tanhf(cn);
}

// dual-operand NN product (defined in sat_gemm.cu): C = [A1 | A2] [B1 ; B2] + bias
sat_status sat_gemm_nn_dual(sat_ctx *ctx, int64_t m, int32_t n, int32_t k1, const float *A1, int32_t lda1, const float *B1, int32_t ldb1,
                            int32_t k2, const float *A2, int32_t lda2, const float *B2, int32_t ldb2, const float *bias, float *C,
                            int32_t ldc);

// first LSTM step from a cached input projection (gate-interleaved columns 4 j + gate): previous state is zero
__global__ void k_lstm_cell_first(const float *__restrict__ proj, int64_t rows, int32_t h, float *__restrict__ c, float *__restrict__ s)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= rows * h) return;
    const float4 a = __ldg(reinterpret_cast<const float4 *>(proj) + t);  // (i, f, g, o) of unit t % h of row t / h
    const float gi = sigmoid_fast(a.x);   // same gate arithmetic as the fused cell of the later steps
    const float gg = tanh_fast(a.z);
    const float go = sigmoid_fast(a.w);
    const float cn = gi * gg;
    c[sat_cell_offset(t / h, (int32_t)(t % h), h)] = cn;
    s[t] = go * tanh_fast(cn);
}

// LSTM with cached input projections (parameter version promised by the caller).  A snapshot whose projection x Wx + b is
// cached runs its step as a contraction over h only, with the projection added in the epilogue.  A missing projection is
// computed (and kept) only for the newest snapshot, which has tau - 1 further epochs of use ahead; an older snapshot
// without one (after a version bump) runs its step as the contraction over [x | s] instead, which costs less than
// projecting it for the one or two epochs it has left.
static sat_status run_lstm_cached(sat_ctx *ctx, CacheLayer *c, const sat_pred_params *p, int32_t k, float *cell)
{
    const int32_t h = p->h, d = c->width;
    const int64_t rows = ctx->n_slots;
    const int64_t plane = rows * 4 * h;
    if (!c->proj || c->proj_h != h) {
        SAT_TRY(dev_realloc(ctx, &c->proj, (int64_t)(ctx->tau + 1) * plane));
        c->proj_h = h;
        c->proj_tag.assign(ctx->tau + 1, 0);
    }
    TcWeights Wp, Wxu, Up;   // Wx alone, [Wx ; Uh], Uh alone (all gate-interleaved)
    bool have_wp = false, have_wxu = false, have_up = false;
    if (c->pk_h != h) {      // another predictor width: nothing packed fits
        c->tag_wx = c->tag_uh = c->tag_wg = c->tag_b = c->tag_bg = 0;
        c->pk_h = h;
    }
    // the packed weight planes live in the cache layer and are made once per parameter version
    auto pack_wx = [&]() -> sat_status {
        if (have_wp) return SAT_OK;
        if (c->tag_wx == p->version) {
            SAT_TRY(sat_tc_weights_layout(d, 4 * h, c->pk_wx, &Wp));
        } else {
            SAT_TRY(sat_tc_weights(ctx, p->Wx, 4 * h, d, nullptr, 0, 0, 4 * h, 1, c->pk_wx, &Wp, h));
            c->tag_wx = p->version;
        }
        have_wp = true;
        return SAT_OK;
    };
    const int32_t newest = ring_index(ctx, 0);
    if (c->proj_tag[newest] != p->version) {
        SAT_TRY(pack_wx());
        TcEpilogueHost eh;
        eh.C = c->proj + (int64_t)newest * plane;
        eh.ldc = 4 * h;
        eh.bias = p->b;
        eh.pack_gate_h = h;
        eh.bias_home = &c->pk_b;
        eh.bias_ready = c->tag_b == p->version;
        c->tag_b = p->version;
        SAT_TRY(sat_gemm_tc(ctx, rows, 4 * h, ring_buf(ctx, c, newest), c->ld, d, nullptr, 0, 0, Wp, eh, SATK_GEMM_NN));
        c->proj_tag[newest] = p->version;
    }
    // (Running the steps row block by row block, so that a block's state stays in L2 between two steps, was measured and
    // was slower: the smaller launches cost more than the state traffic they save.)
    for (int32_t t = 0; t < k; ++t) {
        const int32_t idx = ring_index(ctx, k - 1 - t);  // oldest first
        const bool cached = c->proj_tag[idx] == p->version;
        const float *pr = c->proj + (int64_t)idx * plane;
        TcEpilogueHost eh;
        eh.C = c->S;
        eh.ldc = h;
        eh.lstm_h = h;
        eh.lstm_c = cell;
        if (cached && t == 0) {
            ProfScope prof(ctx, SATK_LSTM_CELL, 4.0 * (double)rows * h * 6.0, 0.0);
            k_lstm_cell_first<<<(unsigned)cdiv64(rows * h, 256), 256, 0, ctx->stream>>>(pr, rows, h, cell, c->S);
            SAT_LAUNCHED(ctx);
        } else if (cached) {
            if (!have_up) {
                if (c->tag_uh == p->version) {
                    SAT_TRY(sat_tc_weights_layout(h, 4 * h, c->pk_uh, &Up));
                } else {
                    SAT_TRY(sat_tc_weights(ctx, p->Uh, 4 * h, h, nullptr, 0, 0, 4 * h, 1, c->pk_uh, &Up, h));
                    c->tag_uh = p->version;
                }
            }
            have_up = true;
            eh.addend = pr;
            eh.ld_addend = 4 * h;
            SAT_TRY(sat_gemm_tc(ctx, rows, 4 * h, c->S, h, h, nullptr, 0, 0, Up, eh, SATK_GEMM_SIDE));
        } else if (t == 0) {
            SAT_TRY(pack_wx());
            eh.bias = p->b;
            eh.lstm_first = 1;
            SAT_TRY(sat_gemm_tc(ctx, rows, 4 * h, ring_buf(ctx, c, idx), c->ld, d, nullptr, 0, 0, Wp, eh, SATK_GEMM_NN));
        } else {
            if (!have_wxu) SAT_TRY(sat_tc_weights(ctx, p->Wx, 4 * h, d, p->Uh, 4 * h, h, 4 * h, 1, ctx->buf_wsplit3, &Wxu, h));
            have_wxu = true;
            eh.bias = p->b;
            SAT_TRY(sat_gemm_tc(ctx, rows, 4 * h, ring_buf(ctx, c, idx), c->ld, d, c->S, h, h, Wxu, eh, SATK_GEMM_NN));
        }
    }
    c->S_valid = true;
    return SAT_OK;
}

// GRU cell on the two pre-activation matrices gx = x Wx + (b_r | b_z | b_n) and gh = s Uh (null at the first step, where the
// state is zero), gate blocks r | z | n:  n = tanh(gx_n + r (gh_n + b_hn)),  s = (1 - z) n + z s.
__global__ void k_gru_cell(const float *__restrict__ gx, const float *__restrict__ gh, const float *__restrict__ b_hn, int64_t rows, int32_t h,
                           float *__restrict__ s)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= rows * h) return;
    const int64_t r0 = t / h;
    const int j = (int)(t - r0 * h);
    const float *ax = gx + r0 * 3 * (int64_t)h;
    float hr = 0.f, hz = 0.f, hn = 0.f, sp = 0.f;
    if (gh) {
        const float *ah = gh + r0 * 3 * (int64_t)h;
        hr = ah[j];
        hz = ah[h + j];
        hn = ah[2 * h + j];
        sp = s[t];
    }
    const float r = 1.f / (1.f + expf(-(ax[j] + hr)));
    const float z = 1.f / (1.f + expf(-(ax[h + j] + hz)));
    const float n = tanhf(ax[2 * h + j] + r * (hn + b_hn[j]));
    s[t] = (1.f - z) * n + z * sp;
}

// GRU-GCN variant: two plain contractions per step (input side with the bias, hidden side) and the cell kernel
static sat_status run_gru(sat_ctx *ctx, CacheLayer *c, const sat_pred_params *p)
{
    const int32_t h = p->h, d = c->width;
    const int64_t rows = ctx->n_slots;
    if (rows == 0) {   // a single partition: nothing is cached, the state table is empty
        c->S_h = h;
        c->S_valid = true;
        return SAT_OK;
    }
    if (!c->S || c->S_h != h) {
        SAT_TRY(dev_realloc(ctx, &c->S, rows * h));
        c->S_h = h;
    }
    const int32_t k = ctx->n_valid < ctx->tau ? ctx->n_valid : ctx->tau;
    if (k == 0 || rows == 0) {
        SAT_CUDA(ctx, cudaMemsetAsync(c->S, 0, (size_t)(rows > 0 ? rows : 1) * h * sizeof(float), ctx->stream));
        c->S_valid = true;
        return SAT_OK;
    }
    const int64_t plane = rows * 3 * h;
    SAT_TRY(sat_ensure(ctx, ctx->buf_lstm_w, (size_t)2 * plane * sizeof(float)));
    float *gx = (float *)ctx->buf_lstm_w.p, *gh = gx + plane;
    const bool tc_x = sat_use_tc(3 * h, d), tc_h = sat_use_tc(3 * h, h);
    TcWeights Wxp, Uhp;
    if (tc_x) SAT_TRY(sat_tc_weights(ctx, p->Wx, 3 * h, d, nullptr, 0, 0, 3 * h, 1, ctx->buf_wsplit, &Wxp));
    if (tc_h && k > 1) SAT_TRY(sat_tc_weights(ctx, p->Uh, 3 * h, h, nullptr, 0, 0, 3 * h, 1, ctx->buf_wsplit2, &Uhp));
    for (int32_t t = 0; t < k; ++t) {
        const float *x = ring_buf(ctx, c, ring_index(ctx, k - 1 - t));  // oldest first
        if (tc_x) {
            TcEpilogueHost eh;
            eh.C = gx;
            eh.ldc = 3 * h;
            eh.bias = p->b;
            SAT_TRY(sat_gemm_tc(ctx, rows, 3 * h, x, c->ld, d, nullptr, 0, 0, Wxp, eh, SATK_GEMM_NN));
        } else {
            GemmEpilogue ep;
            ep.bias = p->b;
            SAT_TRY(sat_gemm_nn(ctx, rows, 3 * h, d, x, c->ld, p->Wx, 3 * h, gx, 3 * h, ep));
        }
        if (t > 0) {
            if (tc_h) {
                TcEpilogueHost eh;
                eh.C = gh;
                eh.ldc = 3 * h;
                SAT_TRY(sat_gemm_tc(ctx, rows, 3 * h, c->S, h, h, nullptr, 0, 0, Uhp, eh, SATK_GEMM_SIDE));
            } else {
                GemmEpilogue ep;
                SAT_TRY(sat_gemm_nn(ctx, rows, 3 * h, h, c->S, h, p->Uh, 3 * h, gh, 3 * h, ep));
            }
        }
        ProfScope prof(ctx, SATK_LSTM_CELL, 4.0 * (double)rows * h * 8.0, 0.0);
        k_gru_cell<<<(unsigned)cdiv64(rows * h, 256), 256, 0, ctx->stream>>>(gx, t > 0 ? gh : nullptr, p->b + 3 * h, rows, h, c->S);
        SAT_LAUNCHED(ctx);
    }
    c->S_valid = true;
    return SAT_OK;
}

static sat_status run_lstm(sat_ctx *ctx, CacheLayer *c, const sat_pred_params *p)
{
    if (p->cell == SAT_CELL_GRU) return run_gru(ctx, c, p);
    const int32_t h = p->h, d = c->width;
    const int64_t rows = ctx->n_slots;
    if (rows == 0) {   // a single partition: nothing is cached, the state table is empty
        c->S_h = h;
        c->S_valid = true;
        return SAT_OK;
    }
    if (!c->S || c->S_h != h) {
        SAT_TRY(dev_realloc(ctx, &c->S, rows * h));
        c->S_h = h;
    }
    const int32_t k = ctx->n_valid < ctx->tau ? ctx->n_valid : ctx->tau;
    if (k == 0 || rows == 0) {
        SAT_CUDA(ctx, cudaMemsetAsync(c->S, 0, (size_t)(rows > 0 ? rows : 1) * h * sizeof(float), ctx->stream));
        c->S_valid = true;
        return SAT_OK;
    }
    if (!(sat_use_tc(4 * h, d) && 4 * h <= 256)) SAT_TRY(sat_ensure(ctx, ctx->buf_lstm_w, (size_t)rows * 4 * h * sizeof(float)));
    SAT_TRY(sat_ensure(ctx, ctx->buf_lstm_c, sat_cell_floats(rows, h) * sizeof(float)));
    float *gates = (float *)ctx->buf_lstm_w.p;
    float *cell = (float *)ctx->buf_lstm_c.p;
    const bool tc = sat_use_tc(4 * h, d);
    // the cell update can be fused into the epilogue (s and c updated in place) when one tile spans all 4h gate columns:
    // then a tile reads only its own rows of s, and does so before its epilogue overwrites them
    const bool fused = tc && 4 * h <= 256;
    if (fused && p->version != 0 && sat_use_tc(4 * h, h)) return run_lstm_cached(ctx, c, p, k, cell);
    TcWeights W1, W2;   // packed weights for the first step (x only) and the later steps ([x | s])
    if (tc) {
        SAT_TRY(sat_tc_weights(ctx, p->Wx, 4 * h, d, nullptr, 0, 0, 4 * h, 1, ctx->buf_wsplit, &W1, fused ? h : 0));
        if (k > 1) SAT_TRY(sat_tc_weights(ctx, p->Wx, 4 * h, d, p->Uh, 4 * h, h, 4 * h, 1, ctx->buf_wsplit2, &W2, fused ? h : 0));
    }
    for (int32_t t = 0; t < k; ++t) {
        const float *x = ring_buf(ctx, c, ring_index(ctx, k - 1 - t));  // oldest first
        if (tc) {
            TcEpilogueHost eh;
            eh.bias = p->b;
            if (fused) {
                eh.C = c->S;
                eh.ldc = h;
                eh.lstm_h = h;
                eh.lstm_first = t == 0;
                eh.lstm_c = cell;
            } else {
                eh.C = gates;
                eh.ldc = 4 * h;
            }
            if (t == 0) SAT_TRY(sat_gemm_tc(ctx, rows, 4 * h, x, c->ld, d, nullptr, 0, 0, W1, eh, SATK_GEMM_NN));
            else SAT_TRY(sat_gemm_tc(ctx, rows, 4 * h, x, c->ld, d, c->S, h, h, W2, eh, SATK_GEMM_NN));
        } else {
            SAT_TRY(sat_gemm_nn_dual(ctx, rows, 4 * h, d, x, c->ld, p->Wx, 4 * h, t == 0 ? 0 : h, c->S, h, p->Uh, 4 * h, p->b, gates, 4 * h));
        }
        if (!fused) {
            ProfScope prof(ctx, SATK_LSTM_CELL, 4.0 * (double)rows * h * 7.0, 0.0);
            k_lstm_cell<<<(unsigned)cdiv64(rows * h, 256), 256, 0, ctx->stream>>>(gates, rows, h, t == 0, cell, c->S);
            SAT_LAUNCHED(ctx);
        }
    }
    c->S_valid = true;
    return SAT_OK;
}

// Schedule of the predictor-output contraction over the halo rows of all partitions: tiles of 128 rows ordered by the
// cache slot of their first row.  Every partition's halo list is sorted by node id, hence by slot, so a tile covers a
// narrow slot range; walking the tiles of all partitions in slot order puts the (on average 3-4) halo copies of a cached
// node in flight together, and its newest-snapshot row — the skip connection the epilogue gathers — is read from DRAM once
// instead of once per copy.
__global__ void k_tile_keys(const int32_t *__restrict__ halo_slot, int64_t n_halo, int64_t n_tiles, int32_t *__restrict__ keys)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < n_tiles) keys[t] = halo_slot[t * 128 < n_halo ? t * 128 : n_halo - 1];
}

static sat_status halo_tile_order(sat_ctx *ctx, int64_t n_halo, const int32_t **out)
{
    if (!ctx->halo_tile_order) {
        const int64_t n_tiles = cdiv64(n_halo, 128);
        int32_t *d = nullptr;
        SAT_CUDA(ctx, cudaMalloc((void **)&d, (size_t)n_tiles * sizeof(int32_t)));
        k_tile_keys<<<(unsigned)cdiv64(n_tiles, 256), 256, 0, ctx->stream>>>(ctx->halo_slot, n_halo, n_tiles, d);
        std::vector<int32_t> keys((size_t)n_tiles), order((size_t)n_tiles);
        cudaError_t e = cudaMemcpyAsync(keys.data(), d, (size_t)n_tiles * sizeof(int32_t), cudaMemcpyDeviceToHost, ctx->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
        if (e == cudaSuccess) {
            for (int64_t t = 0; t < n_tiles; ++t) order[(size_t)t] = (int32_t)t;
            std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return keys[(size_t)x] < keys[(size_t)y]; });
            e = cudaMemcpyAsync(d, order.data(), (size_t)n_tiles * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->stream);
        }
        if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
        if (e != cudaSuccess) {
            cudaFree(d);
            return sat_check_cuda(ctx, e, "halo_tile_order");
        }
        SAT_LAUNCHED(ctx);
        ctx->halo_tile_order = d;
    }
    *out = ctx->halo_tile_order;
    return SAT_OK;
}

extern "C" sat_status sat_predict(sat_ctx *ctx, int32_t layer, int32_t part, const sat_pred_params *params, int reuse_state,
                                  float *halo_out, int32_t ld_out)
{
    CHECK_CTX(ctx);
    CacheLayer *c;
    SAT_TRY(cache_layer(ctx, layer, &c, "sat_predict"));
    PartView v;
    SAT_TRY(sat_part_view(ctx, part, &v));
    const int32_t d = c->width;
    if (v.n_halo > 0 && (!halo_out || !ok_ld(ld_out, d) || !aligned16(halo_out)))
        return sat_fail(ctx, SAT_EINVAL, "sat_predict: null / misaligned halo_out or bad ld_out");
    const float *newest = ctx->n_valid > 0 ? ring_buf(ctx, c, ring_index(ctx, 0)) : nullptr;
    if (!params) {  // identity predictor: plain historical embeddings
        if (v.n_halo == 0) return SAT_OK;
        if (!newest) {
            SAT_CUDA(ctx, cudaMemset2DAsync(halo_out, (size_t)ld_out * 4, 0, (size_t)d * 4, (size_t)v.n_halo, ctx->stream));
            return SAT_OK;
        }
        return sat_gather(ctx, ctx->halo_slot + v.halo0, v.n_halo, d, newest, c->ld, halo_out, ld_out, DbgRange{0, ctx->n_slots});
    }
    if (params->h <= 0 || !params->Wx || !params->Uh || !params->b || !params->Wg || !params->bg)
        return sat_fail(ctx, SAT_EINVAL, "sat_predict: incomplete predictor parameters");
    if (params->cell != SAT_CELL_LSTM && params->cell != SAT_CELL_GRU) return sat_fail(ctx, SAT_EINVAL, "sat_predict: unknown recurrent cell %d", params->cell);
    // the state table S uses ld = h, and its rows must be 16-byte aligned; checked before any state is touched
    if (params->h & 3) return sat_fail(ctx, SAT_EINVAL, "sat_predict: predictor width h must be a multiple of 4");
    if (reuse_state) {
        if (!c->S_valid || c->S_h != params->h) return sat_fail(ctx, SAT_ESTATE, "sat_predict: no LSTM state table to reuse for layer %d", layer);
    } else {
        SAT_TRY(run_lstm(ctx, c, params));
    }
    if (v.n_halo == 0) return SAT_OK;
    const int32_t h = params->h;
    const int32_t ld_a = round_up4(h);
    SAT_TRY(sat_ensure(ctx, ctx->buf_pred_a, (size_t)v.n_halo * ld_a * sizeof(float)));
    float *a = (float *)ctx->buf_pred_a.p;
    // graph convolution on the LSTM state: a_u = p_uu S_u + sum_{v in N(u) cap V_m} p_uv S_v
    SAT_TRY(sat_spmm_hrow(ctx, v, h, c->S, h, 1, c->S, a - v.halo0 * ld_a, ld_a));
    if (sat_use_tc(d, h)) {
        TcWeights Wg;
        TcEpilogueHost eh;
        if (params->version != 0 && params->cell == SAT_CELL_LSTM) {   // packed output weights and bias kept per parameter version
            if (c->pk_h != h) {
                c->tag_wx = c->tag_uh = c->tag_wg = c->tag_b = c->tag_bg = 0;
                c->pk_h = h;
            }
            if (c->tag_wg == params->version) {
                SAT_TRY(sat_tc_weights_layout(h, d, c->pk_wg, &Wg));
            } else {
                SAT_TRY(sat_tc_weights(ctx, params->Wg, d, h, nullptr, 0, 0, d, 1, c->pk_wg, &Wg));
                c->tag_wg = params->version;
            }
            eh.bias_home = &c->pk_bg;
            eh.bias_ready = c->tag_bg == params->version;
            c->tag_bg = params->version;
        } else {
            SAT_TRY(sat_tc_weights(ctx, params->Wg, d, h, nullptr, 0, 0, d, 1, ctx->buf_wsplit, &Wg));
        }
        eh.C = halo_out;
        eh.ldc = ld_out;
        eh.bias = params->bg;
        if (newest) {
            eh.resid = newest;
            eh.resid_idx = ctx->halo_slot + v.halo0;
            eh.ld_resid = c->ld;
            // all partitions at once and a snapshot several times the L2: walk the row tiles in slot order
            const bool all = v.halo0 == 0 && v.n_halo == ctx->h_halo_off[ctx->M];
            // (SAT_PRED_TILE_ORDER in the environment: 0 = never, 1 = whenever all partitions run at once)
            const char *force = getenv("SAT_PRED_TILE_ORDER");
            const bool pays = v.n_halo > ctx->n_slots && (size_t)ctx->n_slots * c->ld * sizeof(float) > ((size_t)128 << 20);
            if (all && v.n_halo > 0 && (force ? atoi(force) != 0 : pays)) SAT_TRY(halo_tile_order(ctx, v.n_halo, &eh.tile_order));
        }
        return sat_gemm_tc(ctx, v.n_halo, d, a, ld_a, h, nullptr, 0, 0, Wg, eh, SATK_GEMM_SIDE);
    }
    GemmEpilogue ep;
    ep.bias = params->bg;
    if (newest) {
        ep.resid = newest;
        ep.resid_idx = ctx->halo_slot + v.halo0;
        ep.ld_resid = c->ld;
    }
    return sat_gemm_nn(ctx, v.n_halo, d, h, a, ld_a, params->Wg, d, halo_out, ld_out, ep);
}

extern "C" sat_status sat_predict_state(sat_ctx *ctx, int32_t layer, float *S_host, int32_t h)
{
    CHECK_CTX(ctx);
    CacheLayer *c;
    SAT_TRY(cache_layer(ctx, layer, &c, "sat_predict_state"));
    if (!S_host) return sat_fail(ctx, SAT_EINVAL, "sat_predict_state: null output");
    if (!c->S_valid || c->S_h != h) return sat_fail(ctx, SAT_ESTATE, "sat_predict_state: no state table of width %d for layer %d", h, layer);
    SAT_CUDA(ctx, cudaMemcpyAsync(S_host, c->S, (size_t)ctx->n_slots * h * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return SAT_OK;
}

// =====================================================================================
// sat_layer_fwd / sat_layer_bwd
// =====================================================================================
__global__ void k_row_slot(const int32_t *__restrict__ perm, const int32_t *__restrict__ slot, int32_t n, int32_t *__restrict__ row_slot)
{
    const int64_t r = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (r < n) row_slot[r] = slot[perm[r]];
}

extern "C" sat_status sat_layer_fwd(sat_ctx *ctx, int32_t part, int32_t layer, int32_t d_in, int32_t d_out, const float *h_in,
                                    int32_t ld_in, const float *h_halo, int32_t ld_halo, const float *W, const float *bias, int act,
                                    float *h_out, int32_t ld_out)
{
    CHECK_CTX(ctx);
    PartView v;
    SAT_TRY(sat_part_view(ctx, part, &v));
    if (layer < 1 || layer > SAT_MAX_LAYERS) return sat_fail(ctx, SAT_EINVAL, "sat_layer_fwd: layer must be in [1, %d]", SAT_MAX_LAYERS);
    const bool push = (act & SAT_FWD_PUSH) != 0;
    const bool in_global = (act & SAT_FWD_INPUT_GLOBAL) != 0;
    const bool halo_global = in_global || (act & SAT_FWD_HALO_GLOBAL) != 0;
    act &= ~(SAT_FWD_PUSH | SAT_FWD_HALO_GLOBAL | SAT_FWD_INPUT_GLOBAL);
    if (d_in <= 0 || d_out <= 0 || !W || (act != SAT_ACT_NONE && act != SAT_ACT_RELU)) return sat_fail(ctx, SAT_EINVAL, "sat_layer_fwd: bad dims / W / act");
    CacheLayer *pc = nullptr;
    if (push) {
        SAT_TRY(cache_layer(ctx, layer, &pc, "sat_layer_fwd"));
        if (pc->width != d_out) return sat_fail(ctx, SAT_EINVAL, "sat_layer_fwd: cached layer %d has width %d, not %d", layer, pc->width, d_out);
    }
    if (v.n_rows > 0 && (!h_in || !h_out || !ok_ld(ld_in, d_in) || !ok_ld(ld_out, d_out) || !aligned16(h_in) || !aligned16(h_out)))
        return sat_fail(ctx, SAT_EINVAL, "sat_layer_fwd: null / misaligned h_in / h_out or bad leading dimension");
    if (!in_global && v.n_halo > 0 && (!h_halo || !ok_ld(ld_halo, d_in) || !aligned16(h_halo)))
        return sat_fail(ctx, SAT_EINVAL, "sat_layer_fwd: null / misaligned h_halo or bad ld_halo");
    LayerState &L = ctx->layers[layer];
    const int32_t ld_agg = round_up4(d_in), words = (d_out + 31) / 32;
    if (!L.agg || L.d_in != d_in || L.d_out != d_out) {
        SAT_TRY(dev_realloc(ctx, &L.agg, (int64_t)ctx->n * ld_agg));
        SAT_TRY(dev_realloc(ctx, &L.mask, (int64_t)ctx->n * words));
        L.d_in = d_in;
        L.d_out = d_out;
        L.ld_in = ld_agg;
        L.mask_words = words;
        L.valid.assign(ctx->M, 0);
    }
    L.act = act;
    if (v.n_rows == 0) return SAT_OK;
    // the inner source is the partition-major matrix (addressed from its virtual first row) or, like the halo source, a matrix
    // over all nodes; the halo source is the concatenated halo matrix (virtual first row) or a matrix over all nodes
    const float *in_base = in_global ? h_in : h_in - (int64_t)v.row0 * ld_in;
    const float *halo_base = in_global || !h_halo ? nullptr : halo_global ? h_halo : h_halo - v.halo0 * (int64_t)ld_halo;
    SAT_TRY(sat_spmm(ctx, v, 0, d_in, in_base, ld_in, halo_base, ld_halo, L.agg, ld_agg, nullptr, 0, halo_global, in_global));
    uint32_t *mask_out = act == SAT_ACT_RELU ? L.mask + (int64_t)v.row0 * words : nullptr;
    const float *agg = L.agg + (int64_t)v.row0 * ld_agg;
    if (sat_use_tc(d_out, d_in)) {
        TcWeights Wp;
        SAT_TRY(sat_tc_weights(ctx, W, d_out, d_in, nullptr, 0, 0, d_out, 1, ctx->buf_wsplit, &Wp));
        TcEpilogueHost eh;
        eh.C = h_out;
        eh.ldc = ld_out;
        eh.bias = bias;
        eh.relu = act == SAT_ACT_RELU;
        eh.mask_out = mask_out;
        eh.mask_words = words;
        if (push && ctx->n_slots > 0) {   // the boundary rows go to the ring's write buffer from the epilogue
            if (!ctx->row_slot) {
                SAT_TRY(dev_realloc(ctx, &ctx->row_slot, (int64_t)ctx->n));
                k_row_slot<<<(unsigned)cdiv64(ctx->n, 256), 256, 0, ctx->stream>>>(ctx->perm, ctx->slot, ctx->n, ctx->row_slot);
                SAT_LAUNCHED(ctx);
            }
            eh.push_dst = ring_buf(ctx, pc, ctx->write_idx);
            eh.push_slot = ctx->row_slot + v.row0;
            eh.ld_push = pc->ld;
            if (!pc->proj_tag.empty()) pc->proj_tag[ctx->write_idx] = 0;
        }
        SAT_TRY(sat_gemm_tc(ctx, v.n_rows, d_out, agg, ld_agg, d_in, nullptr, 0, 0, Wp, eh, SATK_GEMM_NN));
    } else {
        GemmEpilogue ep;
        ep.bias = bias;
        ep.relu = act == SAT_ACT_RELU;
        ep.mask_out = mask_out;
        ep.mask_words = words;
        SAT_TRY(sat_gemm_nn(ctx, v.n_rows, d_out, d_in, agg, ld_agg, W, d_out, h_out, ld_out, ep));
    }
    if (part == SAT_ALL_PARTS) L.valid.assign(ctx->M, 1);
    else L.valid[part] = 1;
    // widths the tensor-core path does not take: the push as its own step
    if (push && !sat_use_tc(d_out, d_in)) return sat_cache_update(ctx, part, layer, h_out, ld_out);
    return SAT_OK;
}

extern "C" sat_status sat_layer_bwd(sat_ctx *ctx, int32_t part, int32_t layer, const float *g_out, int32_t ld_g, const float *W,
                                    float *g_W, float *g_b, int accumulate, float *g_in, int32_t ld_gin, float *g_halo, int32_t ld_gh)
{
    CHECK_CTX(ctx);
    PartView v;
    SAT_TRY(sat_part_view(ctx, part, &v));
    if (layer < 1 || layer > SAT_MAX_LAYERS) return sat_fail(ctx, SAT_EINVAL, "sat_layer_bwd: layer must be in [1, %d]", SAT_MAX_LAYERS);
    LayerState &L = ctx->layers[layer];
    if (!L.agg) return sat_fail(ctx, SAT_ESTATE, "sat_layer_bwd: sat_layer_fwd has not run for layer %d", layer);
    for (int m = (part == SAT_ALL_PARTS ? 0 : part); m < (part == SAT_ALL_PARTS ? ctx->M : part + 1); ++m)
        if (!L.valid[m]) return sat_fail(ctx, SAT_ESTATE, "sat_layer_bwd: sat_layer_fwd has not run for partition %d of layer %d", m, layer);
    const int32_t d_in = L.d_in, d_out = L.d_out;
    if (!W || !g_W) return sat_fail(ctx, SAT_EINVAL, "sat_layer_bwd: null W / g_W");
    if (v.n_rows > 0 && (!g_out || !ok_ld(ld_g, d_out) || !aligned16(g_out))) return sat_fail(ctx, SAT_EINVAL, "sat_layer_bwd: null / misaligned g_out or bad ld_g");
    if (g_in && v.n_rows > 0 && (!ok_ld(ld_gin, d_in) || !aligned16(g_in))) return sat_fail(ctx, SAT_EINVAL, "sat_layer_bwd: misaligned g_in or bad ld_gin");
    if (g_halo && v.n_halo > 0 && (!ok_ld(ld_gh, d_in) || !aligned16(g_halo))) return sat_fail(ctx, SAT_EINVAL, "sat_layer_bwd: misaligned g_halo or bad ld_gh");
    const int flags = accumulate;
    accumulate = flags & SAT_BWD_ACCUMULATE;
    if (flags & ~(SAT_BWD_ACCUMULATE | SAT_BWD_MASK_G_IN | SAT_BWD_G_OUT_MASKED | SAT_BWD_GRAD_HISTORY))
        return sat_fail(ctx, SAT_EINVAL, "sat_layer_bwd: unknown flag bits");
    const bool hist = (flags & SAT_BWD_GRAD_HISTORY) && layer >= 2 && ctx->n_slots > 0;
    const uint32_t *mask = (L.act == SAT_ACT_RELU && !(flags & SAT_BWD_G_OUT_MASKED)) ? L.mask + (int64_t)v.row0 * L.mask_words : nullptr;
    // ReLU mask of the layer below, applied to g_in on request (indexed by partition-major row like g_in)
    const uint32_t *mask_in = nullptr;
    int32_t mask_in_words = 0;
    if ((flags & SAT_BWD_MASK_G_IN) && layer > 1) {
        LayerState &Lp = ctx->layers[layer - 1];
        bool ok = Lp.agg && Lp.act == SAT_ACT_RELU && Lp.mask && Lp.d_out == L.d_in;
        for (int m = (part == SAT_ALL_PARTS ? 0 : part); ok && m < (part == SAT_ALL_PARTS ? ctx->M : part + 1); ++m) ok = Lp.valid[m];
        if (ok) {
            mask_in = Lp.mask;
            mask_in_words = Lp.mask_words;
        }
    }
    const float *agg = L.agg + (int64_t)v.row0 * L.ld_in;
    const bool want_dx = (g_in || g_halo) && v.n_rows > 0;
    const bool tc_w = sat_use_tc(d_out, d_in) && v.n_rows >= 256;   // weight gradient on the tensor cores
    // input gradient on the tensor cores, except when the halo gradient is wanted: that output sums thousands of signed
    // cut-edge terms, and the truncating fp32 accumulation of the tensor cores would be amplified by the cancellation
    const bool tc_x = want_dx && !g_halo && sat_use_tc(d_in, d_out);
    const float *D = g_out;  // D = g_out o [Z > 0]: materialised once for the tensor-core contractions
    int32_t ld_d = ld_g;
    if (tc_w || tc_x || (hist && mask)) {
        float *dm = nullptr;
        if (mask) {
            ld_d = round_up4(d_out);
            SAT_TRY(sat_ensure(ctx, ctx->buf_dmask, (size_t)v.n_rows * ld_d * sizeof(float)));
            dm = (float *)ctx->buf_dmask.p;
            D = dm;
        }
        SAT_TRY(sat_mask_rows(ctx, g_out, ld_g, v.n_rows, d_out, mask, L.mask_words, dm, ld_d, tc_w ? g_b : nullptr, accumulate));
    }
    // G_W (+)= AGG^T D, G_b (+)= 1^T D
    if (tc_w && d_out <= 64) SAT_TRY(sat_gemm_tn_narrow(ctx, v.n_rows, d_in, d_out, agg, L.ld_in, D, ld_d, g_W, d_out, accumulate));
    else if (tc_w) SAT_TRY(sat_gemm_tc_tn(ctx, v.n_rows, d_in, d_out, agg, L.ld_in, D, ld_d, g_W, d_out, accumulate));
    else SAT_TRY(sat_gemm_tn(ctx, v.n_rows, d_in, d_out, agg, L.ld_in, g_out, ld_g, mask, L.mask_words, g_W, d_out, g_b, accumulate));
    // gradient-side history, this epoch's contribution: Q_write[slot(u)] += (P_out^T D)[u] for the halo nodes u of the
    // selected partitions, one partition after the other (the halo slots of one partition are distinct)
    GradHist &GH = ctx->ghist[layer];
    if (hist) {
        const int32_t ld_q = round_up4(d_out);
        const size_t plane = (size_t)ctx->n_slots * ld_q;
        if (!GH.buf || GH.width != d_out) {
            SAT_TRY(dev_realloc(ctx, &GH.buf, (int64_t)(2 * plane)));
            SAT_CUDA(ctx, cudaMemsetAsync(GH.buf, 0, 2 * plane * sizeof(float), ctx->stream));
            GH.width = d_out;
            GH.ld = ld_q;
            GH.read_idx = 0;
            GH.has_read = false;
        }
        if (v.n_halo > 0 && v.n_rows > 0) {
            SAT_TRY(sat_ensure(ctx, ctx->buf_ghist_halo, (size_t)v.n_halo * ld_q * sizeof(float)));
            float *qh = (float *)ctx->buf_ghist_halo.p;
            SAT_TRY(sat_spmm_hrow(ctx, v, d_out, D - (int64_t)v.row0 * ld_d, ld_d, 0, nullptr, qh - v.halo0 * (int64_t)ld_q, ld_q));
            float *qw = GH.buf + (size_t)(1 - GH.read_idx) * plane;
            if (part == SAT_ALL_PARTS) {
                // all copies of every boundary node are in qh: one gather-sum per slot, copies taken in partition order
                SAT_TRY(sat_sum_by_slot(ctx, d_out, qh, ld_q, 0, 1, qw, ld_q));
            } else {
                const int64_t h0 = ctx->h_halo_off[part], cnt = ctx->h_halo_off[part + 1] - h0;
                SAT_TRY(sat_scatter_add(ctx, nullptr, ctx->halo_slot + h0, cnt, d_out, qh, ld_q, qw, ld_q, nullptr, 0));
            }
        }
    }
    if (!want_dx) return SAT_OK;
    // G_AGG = D W^T
    const int32_t ld_ga = round_up4(d_in);
    SAT_TRY(sat_ensure(ctx, ctx->buf_gagg, (size_t)v.n_rows * ld_ga * sizeof(float)));
    float *gagg = (float *)ctx->buf_gagg.p;
    if (tc_x) {
        TcWeights Wp;
        SAT_TRY(sat_tc_weights(ctx, W, d_out, d_out, nullptr, 0, 0, d_in, 0, ctx->buf_wsplit, &Wp));
        TcEpilogueHost eh;
        eh.C = gagg;
        eh.ldc = ld_ga;
        SAT_TRY(sat_gemm_tc(ctx, v.n_rows, d_in, D, ld_d, d_out, nullptr, 0, 0, Wp, eh, SATK_GEMM_NT));
    } else {
        SAT_TRY(sat_gemm_nt(ctx, v.n_rows, d_in, d_out, g_out, ld_g, mask, L.mask_words, W, d_out, gagg, ld_ga));
    }
    const float *ga_base = gagg - (int64_t)v.row0 * ld_ga;
    // G_in = P_in^T G_AGG: the inner block of P is symmetric, so P_in^T = P_in (inner prefix of every local row)
    if (g_in) SAT_TRY(sat_spmm(ctx, v, 1, d_in, ga_base, ld_ga, nullptr, 0, g_in - (int64_t)v.row0 * ld_gin, ld_gin, mask_in, mask_in_words));
    // gradient-side history, the stale term: G_in[v] += (Q_read[slot(v)] W^T) o mask for the boundary rows v of the selection
    if (hist && GH.has_read && g_in && v.n_push > 0) {
        const size_t plane = (size_t)ctx->n_slots * GH.ld;
        const float *qr = GH.buf + (size_t)GH.read_idx * plane;
        SAT_TRY(sat_ensure(ctx, ctx->buf_ghist_rows, (size_t)v.n_push * GH.ld * sizeof(float)));
        SAT_TRY(sat_ensure(ctx, ctx->buf_ghist_out, (size_t)v.n_push * ld_ga * sizeof(float)));
        float *rows = (float *)ctx->buf_ghist_rows.p, *stale = (float *)ctx->buf_ghist_out.p;
        SAT_TRY(sat_gather(ctx, ctx->push_slot + v.push0, v.n_push, d_out, qr, GH.ld, rows, GH.ld, DbgRange{0, ctx->n_slots}));
        if (sat_use_tc(d_in, d_out)) {
            TcWeights Wp;
            SAT_TRY(sat_tc_weights(ctx, W, d_out, d_out, nullptr, 0, 0, d_in, 0, ctx->buf_wsplit, &Wp));
            TcEpilogueHost eh;
            eh.C = stale;
            eh.ldc = ld_ga;
            SAT_TRY(sat_gemm_tc(ctx, v.n_push, d_in, rows, GH.ld, d_out, nullptr, 0, 0, Wp, eh, SATK_GEMM_NT));
        } else {
            SAT_TRY(sat_gemm_nt(ctx, v.n_push, d_in, d_out, rows, GH.ld, nullptr, 0, W, d_out, stale, ld_ga));
        }
        SAT_TRY(sat_scatter_add(ctx, nullptr, ctx->push_row + v.push0, v.n_push, d_in, stale, ld_ga, g_in - (int64_t)v.row0 * ld_gin, ld_gin,
                                mask_in, mask_in_words));
    }
    // G_halo = P_out^T G_AGG over the halo-row CSR
    if (g_halo) SAT_TRY(sat_spmm_hrow(ctx, v, d_in, ga_base, ld_ga, 0, nullptr, g_halo - v.halo0 * (int64_t)ld_gh, ld_gh));
    return SAT_OK;
}

// =====================================================================================
// dense contractions on caller tensors
// =====================================================================================
extern "C" sat_status sat_dense_nn(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const float *W,
                                   const float *bias, float *C, int32_t ldc)
{
    CHECK_CTX(ctx);
    if (m < 0 || n <= 0 || k <= 0 || !A || !W || !C || !ok_ld(lda, k) || !ok_ld(ldc, n) || !aligned16(A) || !aligned16(C))
        return sat_fail(ctx, SAT_EINVAL, "sat_dense_nn: null / misaligned tensor or bad shape");
    if (sat_use_tc(n, k)) {
        TcWeights Wp;
        SAT_TRY(sat_tc_weights(ctx, W, n, k, nullptr, 0, 0, n, 1, ctx->buf_wsplit, &Wp));
        TcEpilogueHost eh;
        eh.C = C;
        eh.ldc = ldc;
        eh.bias = bias;
        return sat_gemm_tc(ctx, m, n, A, lda, k, nullptr, 0, 0, Wp, eh, SATK_GEMM_NN);
    }
    GemmEpilogue ep;
    ep.bias = bias;
    return sat_gemm_nn(ctx, m, n, k, A, lda, W, n, C, ldc, ep);
}

extern "C" sat_status sat_dense_nt(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const float *W, float *C,
                                   int32_t ldc)
{
    CHECK_CTX(ctx);
    if (m < 0 || n <= 0 || k <= 0 || !A || !W || !C || !ok_ld(lda, k) || !ok_ld(ldc, n) || !aligned16(A) || !aligned16(C))
        return sat_fail(ctx, SAT_EINVAL, "sat_dense_nt: null / misaligned tensor or bad shape");
    if (sat_use_tc(n, k)) {
        TcWeights Wp;
        SAT_TRY(sat_tc_weights(ctx, W, k, k, nullptr, 0, 0, n, 0, ctx->buf_wsplit, &Wp));
        TcEpilogueHost eh;
        eh.C = C;
        eh.ldc = ldc;
        return sat_gemm_tc(ctx, m, n, A, lda, k, nullptr, 0, 0, Wp, eh, SATK_GEMM_NT);
    }
    return sat_gemm_nt(ctx, m, n, k, A, lda, nullptr, 0, W, k, C, ldc);
}

extern "C" sat_status sat_dense_tn(sat_ctx *ctx, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B,
                                   int32_t ldb, float *C)
{
    CHECK_CTX(ctx);
    if (rows < 0 || n <= 0 || m <= 0 || !A || !B || !C || !ok_ld(lda, m) || !ok_ld(ldb, n) || !aligned16(A) || !aligned16(B))
        return sat_fail(ctx, SAT_EINVAL, "sat_dense_tn: null / misaligned tensor or bad shape");
    if (sat_use_tc(n, m) && rows >= 256) return sat_gemm_tc_tn(ctx, rows, m, n, A, lda, B, ldb, C, n, 0);
    return sat_gemm_tn(ctx, rows, m, n, A, lda, B, ldb, nullptr, 0, C, n, nullptr, 0);
}

// =====================================================================================
// loss seed, parameter step
// =====================================================================================
// one warp per row
// Loss kernels: one warp per row, LOSS_ROWS_PER_BLOCK consecutive rows per block (each warp walks its share in order).
// The row losses are summed in double per warp, the warps of a block in fixed order, and k_loss_sum adds the block
// partials in fixed order: the total does not depend on scheduling.
#define LOSS_ROWS_PER_BLOCK 256

__device__ __forceinline__ void loss_block_partial(double warp_sum, double *__restrict__ block_partial)
{
    __shared__ double red[8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) red[warp] = warp_sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += red[w];
        block_partial[blockIdx.x] = s;
    }
}

// softmax cross-entropy: the row (up to 32 CPL classes) is held in registers, one exponential per class
template <int CPL>
__global__ void __launch_bounds__(256)
k_loss_ce(int64_t rows, int32_t C, const float *__restrict__ z, int64_t ld_z, const int32_t *__restrict__ y, float scale,
          float *__restrict__ g, int64_t ld_g, double *__restrict__ block_partial)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t r0 = (int64_t)blockIdx.x * LOSS_ROWS_PER_BLOCK;
    double acc = 0.0;
    for (int i = warp; i < LOSS_ROWS_PER_BLOCK; i += 8) {
        const int64_t r = r0 + i;
        if (r >= rows) break;
        const float *zr = z + r * ld_z;
        float v[CPL];
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < CPL; ++j) {
            const int c = lane + 32 * j;
            v[j] = c < C ? zr[c] : -INFINITY;
            mx = fmaxf(mx, v[j]);
        }
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float se = 0.f;
#pragma unroll
        for (int j = 0; j < CPL; ++j) {
            v[j] = lane + 32 * j < C ? expf(v[j] - mx) : 0.f;
            se += v[j];
        }
        for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
        const float inv = 1.f / se;
        const int32_t yr = y[r];
#pragma unroll
        for (int j = 0; j < CPL; ++j) {
            const int c = lane + 32 * j;
            if (c < C) g[r * ld_g + c] = scale * (v[j] * inv - (c == yr ? 1.f : 0.f));
        }
        if (lane == 0) acc += (double)(scale * (mx + logf(se) - zr[yr]));
    }
    loss_block_partial(acc, block_partial);
}

// any number of classes: three passes over the row
__global__ void __launch_bounds__(256)
k_loss_ce_wide(int64_t rows, int32_t C, const float *__restrict__ z, int64_t ld_z, const int32_t *__restrict__ y, float scale,
               float *__restrict__ g, int64_t ld_g, double *__restrict__ block_partial)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t r0 = (int64_t)blockIdx.x * LOSS_ROWS_PER_BLOCK;
    double acc = 0.0;
    for (int i = warp; i < LOSS_ROWS_PER_BLOCK; i += 8) {
        const int64_t r = r0 + i;
        if (r >= rows) break;
        const float *zr = z + r * ld_z;
        float mx = -INFINITY;
        for (int c = lane; c < C; c += 32) mx = fmaxf(mx, zr[c]);
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float se = 0.f;
        for (int c = lane; c < C; c += 32) se += expf(zr[c] - mx);
        for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
        const float inv = 1.f / se;
        const int32_t yr = y[r];
        for (int c = lane; c < C; c += 32) g[r * ld_g + c] = scale * (expf(zr[c] - mx) * inv - (c == yr ? 1.f : 0.f));
        if (lane == 0) acc += (double)(scale * (mx + logf(se) - zr[yr]));
    }
    loss_block_partial(acc, block_partial);
}

__global__ void __launch_bounds__(256)
k_loss_bce(int64_t rows, int32_t C, const float *__restrict__ z, int64_t ld_z, const uint8_t *__restrict__ y, float scale,
           float *__restrict__ g, int64_t ld_g, double *__restrict__ block_partial)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t r0 = (int64_t)blockIdx.x * LOSS_ROWS_PER_BLOCK;
    const float inv_c = 1.f / (float)C;
    double acc = 0.0;
    for (int i = warp; i < LOSS_ROWS_PER_BLOCK; i += 8) {
        const int64_t r = r0 + i;
        if (r >= rows) break;
        const float *zr = z + r * ld_z;
        float a = 0.f;
        for (int c = lane; c < C; c += 32) {
            const float x = zr[c], yv = (float)y[r * C + c];
            a += fmaxf(x, 0.f) + log1pf(expf(-fabsf(x))) - yv * x;
            g[r * ld_g + c] = scale * inv_c * (1.f / (1.f + expf(-x)) - yv);
        }
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (lane == 0) acc += (double)(scale * inv_c * a);
    }
    loss_block_partial(acc, block_partial);
}

// single block, fixed order: *total += sum(block_partial)
__global__ void k_loss_sum(const double *__restrict__ block_partial, int64_t count, double *total)
{
    __shared__ double red[256];
    double s = 0.0;
    for (int64_t i = threadIdx.x; i < count; i += 256) s += block_partial[i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *total += red[0];
}

extern "C" sat_status sat_loss_grad(sat_ctx *ctx, int32_t part, int kind, int32_t n_classes, const float *z, int32_t ld_z,
                                    const void *labels, double *loss_sum, float *g, int32_t ld_g)
{
    CHECK_CTX(ctx);
    PartView v;
    SAT_TRY(sat_part_view(ctx, part, &v));
    if (kind != SAT_LOSS_SOFTMAX_CE && kind != SAT_LOSS_SIGMOID_BCE) return sat_fail(ctx, SAT_EINVAL, "sat_loss_grad: unknown loss");
    if (v.n_rows == 0) return SAT_OK;
    if (n_classes <= 0 || !z || !labels || !g || ld_z < n_classes || ld_g < n_classes) return sat_fail(ctx, SAT_EINVAL, "sat_loss_grad: null tensor or bad shape");
    const unsigned blocks = (unsigned)cdiv64(v.n_rows, LOSS_ROWS_PER_BLOCK);
    SAT_TRY(sat_ensure(ctx, ctx->buf_misc, (size_t)blocks * sizeof(double)));
    double *block_partial = (double *)ctx->buf_misc.p;
    const float scale = 1.0f / (float)ctx->n;
    ProfScope prof(ctx, SATK_LOSS, 8.0 * (double)v.n_rows * n_classes, 0.0);
    if (kind == SAT_LOSS_SOFTMAX_CE) {
        const int32_t *yl = (const int32_t *)labels;
        if (n_classes <= 32) k_loss_ce<1><<<blocks, 256, 0, ctx->stream>>>(v.n_rows, n_classes, z, ld_z, yl, scale, g, ld_g, block_partial);
        else if (n_classes <= 64) k_loss_ce<2><<<blocks, 256, 0, ctx->stream>>>(v.n_rows, n_classes, z, ld_z, yl, scale, g, ld_g, block_partial);
        else if (n_classes <= 128) k_loss_ce<4><<<blocks, 256, 0, ctx->stream>>>(v.n_rows, n_classes, z, ld_z, yl, scale, g, ld_g, block_partial);
        else k_loss_ce_wide<<<blocks, 256, 0, ctx->stream>>>(v.n_rows, n_classes, z, ld_z, yl, scale, g, ld_g, block_partial);
    } else {
        k_loss_bce<<<blocks, 256, 0, ctx->stream>>>(v.n_rows, n_classes, z, ld_z, (const uint8_t *)labels, scale, g, ld_g, block_partial);
    }
    SAT_LAUNCHED(ctx);
    if (loss_sum) {
        k_loss_sum<<<1, 256, 0, ctx->stream>>>(block_partial, (int64_t)blocks, loss_sum);
        SAT_LAUNCHED(ctx);
    }
    return SAT_OK;
}

// staleness diagnostic: one warp per halo row, fp64 accumulation, block partials added in fixed order by k_loss_sum
__global__ void __launch_bounds__(256)
k_staleness(const int32_t *__restrict__ halo_gid, const int32_t *__restrict__ pos, int64_t halo0, int64_t n_halo, int32_t d,
            const float *__restrict__ fresh, int64_t ld, const float *__restrict__ used, int64_t ld_used, double *__restrict__ block_partial)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t j0 = (int64_t)blockIdx.x * LOSS_ROWS_PER_BLOCK;
    double acc = 0.0;
    for (int i = warp; i < LOSS_ROWS_PER_BLOCK; i += 8) {
        const int64_t j = j0 + i;
        if (j >= n_halo) break;
        const float *a = fresh + (int64_t)pos[halo_gid[halo0 + j]] * ld;
        const float *b = used + j * ld_used;
        double s = 0.0;
        for (int c = lane; c < d; c += 32) {
            const double t = (double)a[c] - (double)b[c];
            s += t * t;
        }
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        acc += s;
    }
    loss_block_partial(acc, block_partial);
}

extern "C" sat_status sat_staleness(sat_ctx *ctx, int32_t part, int32_t d, const float *h_fresh, int32_t ld, const float *h_used_halo,
                                    int32_t ld_halo, double *sq_sum)
{
    CHECK_CTX(ctx);
    PartView v;
    SAT_TRY(sat_part_view(ctx, part, &v));
    if (!sq_sum || d <= 0) return sat_fail(ctx, SAT_EINVAL, "sat_staleness: null result or bad width");
    SAT_CUDA(ctx, cudaMemsetAsync(sq_sum, 0, sizeof(double), ctx->stream));
    if (v.n_halo == 0) return SAT_OK;
    if (!h_fresh || !h_used_halo || ld < d || ld_halo < d) return sat_fail(ctx, SAT_EINVAL, "sat_staleness: null tensor or bad leading dimension");
    const unsigned blocks = (unsigned)cdiv64(v.n_halo, LOSS_ROWS_PER_BLOCK);
    SAT_TRY(sat_ensure(ctx, ctx->buf_misc, (size_t)blocks * sizeof(double)));
    double *block_partial = (double *)ctx->buf_misc.p;
    k_staleness<<<blocks, 256, 0, ctx->stream>>>(ctx->halo_gid, ctx->pos, v.halo0, v.n_halo, d, h_fresh, ld,
                                                 h_used_halo, ld_halo, block_partial);
    SAT_LAUNCHED(ctx);
    k_loss_sum<<<1, 256, 0, ctx->stream>>>(block_partial, (int64_t)blocks, sq_sum);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

__global__ void k_sgd(int64_t count, float *__restrict__ w, const float *__restrict__ g, float lr)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) w[i] = w[i] - lr * g[i];
}

extern "C" sat_status sat_sgd_step(sat_ctx *ctx, int64_t count, float *w, const float *g, float lr)
{
    CHECK_CTX(ctx);
    if (count < 0 || (count > 0 && (!w || !g))) return sat_fail(ctx, SAT_EINVAL, "sat_sgd_step: null tensor");
    if (count == 0) return SAT_OK;
    k_sgd<<<(unsigned)cdiv64(count, 256), 256, 0, ctx->stream>>>(count, w, g, lr);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

// the same step on up to SAT_SGD_MAX arrays in one launch (the parameter arrays of a model are many and small)
#define SAT_SGD_MAX 16
struct SgdBatch {
    float *w[SAT_SGD_MAX];
    const float *g[SAT_SGD_MAX];
    int64_t end[SAT_SGD_MAX];   // running totals of the element counts
    int32_t n;
};

__global__ void k_sgd_many(SgdBatch b, float lr)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= b.end[b.n - 1]) return;
    int t = 0;
    while (i >= b.end[t]) ++t;
    const int64_t j = i - (t ? b.end[t - 1] : 0);
    b.w[t][j] = b.w[t][j] - lr * b.g[t][j];
}

extern "C" sat_status sat_sgd_steps(sat_ctx *ctx, int32_t n_arrays, const int64_t *counts, float *const *w, const float *const *g, float lr)
{
    CHECK_CTX(ctx);
    if (n_arrays < 0 || (n_arrays > 0 && (!counts || !w || !g))) return sat_fail(ctx, SAT_EINVAL, "sat_sgd_steps: null argument");
    for (int32_t a0 = 0; a0 < n_arrays; a0 += SAT_SGD_MAX) {
        SgdBatch b;
        b.n = 0;
        int64_t total = 0;
        for (int32_t a = a0; a < n_arrays && a < a0 + SAT_SGD_MAX; ++a) {
            if (counts[a] < 0 || (counts[a] > 0 && (!w[a] || !g[a]))) return sat_fail(ctx, SAT_EINVAL, "sat_sgd_steps: null tensor %d", a);
            if (counts[a] == 0) continue;
            total += counts[a];
            b.w[b.n] = w[a];
            b.g[b.n] = g[a];
            b.end[b.n] = total;
            ++b.n;
        }
        if (b.n == 0) continue;
        k_sgd_many<<<(unsigned)cdiv64(total, 256), 256, 0, ctx->stream>>>(b, lr);
        SAT_LAUNCHED(ctx);
    }
    return SAT_OK;
}
