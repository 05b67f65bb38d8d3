// Objective and gradient of the embedding predictor (Eq. "predictor loss", Eq. "mini-batch training", Algorithm 1
// "Embedding predictor update"): forward pass of the LSTM + graph convolution + skip connection with the gate values kept,
// squared-error loss against the embeddings pushed in the running epoch, and the backward pass through the output layer,
// the transposed graph convolution and the LSTM (back-propagation through time).  The dense contractions run on the same
// GEMM kernels as the layer steps; this file holds the element-wise and sparse kernels around them.
#include "sat_internal.h"

#define CHECK_CTX(ctx)                                                                             \
    do {                                                                                           \
        if (!(ctx)) return SAT_EINVAL;                                                             \
        if ((ctx)->cuda_failed) return sat_fail(ctx, SAT_ECUDA, "context has a sticky CUDA error"); \
        SAT_CUDA(ctx, cudaSetDevice((ctx)->device));                                               \
    } while (0)

static bool aligned16(const void *p) { return (((uintptr_t)p) & 15u) == 0; }
static int32_t ring_index(const sat_ctx *ctx, int32_t age) { return ((ctx->write_idx - 1 - age) % (ctx->tau + 1) + (ctx->tau + 1)) % (ctx->tau + 1); }
static float *ring_buf(const sat_ctx *ctx, const CacheLayer *c, int32_t idx) { return c->buf + (size_t)idx * ctx->n_slots * c->ld; }

// -------------------------------------------------------------------------------------
// LSTM cell, forward with everything the backward needs: z [rows x 4h] holds the gate pre-activations (blocks i | f | g | o)
// and is overwritten with the gate values; c_out = f c_prev + i g; h_out = o tanh(c_out).
// -------------------------------------------------------------------------------------
__global__ void k_pt_cell_fwd(float *__restrict__ z, int64_t rows, int32_t h, const float *__restrict__ c_prev, float *__restrict__ c_out,
                              float *__restrict__ h_out)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= rows * h) return;
    const int64_t r = t / h;
    const int j = (int)(t - r * h);
    float *a = z + r * 4 * (int64_t)h;
    const float gi = 1.f / (1.f + expf(-a[j]));
    const float gf = 1.f / (1.f + expf(-a[h + j]));
    const float gg = tanhf(a[2 * h + j]);
    const float go = 1.f / (1.f + expf(-a[3 * h + j]));
    const float cn = gf * (c_prev ? c_prev[t] : 0.f) + gi * gg;
    a[j] = gi;
    a[h + j] = gf;
    a[2 * h + j] = gg;
    a[3 * h + j] = go;
    c_out[t] = cn;
    h_out[t] = go * tanhf(cn);
}

// LSTM cell, backward: gz [rows x 4h] holds the gate values of the step and is overwritten with the gradient of the loss
// with respect to the gate pre-activations; dc carries the gradient of the cell state from the later steps (null at the
// last step) and leaves as the gradient with respect to the previous cell state.
__global__ void k_pt_cell_bwd(float *__restrict__ gz, int64_t rows, int32_t h, const float *__restrict__ c_prev, const float *__restrict__ c_cur,
                              const float *__restrict__ dh, const float *dc_in, float *dc_out)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= rows * h) return;
    const int64_t r = t / h;
    const int j = (int)(t - r * h);
    float *a = gz + r * 4 * (int64_t)h;
    const float gi = a[j], gf = a[h + j], gg = a[2 * h + j], go = a[3 * h + j];
    const float tc = tanhf(c_cur[t]);
    const float g_h = dh[t];
    const float g_c = (dc_in ? dc_in[t] : 0.f) + g_h * go * (1.f - tc * tc);
    a[j] = g_c * gg * gi * (1.f - gi);
    a[h + j] = g_c * (c_prev ? c_prev[t] : 0.f) * gf * (1.f - gf);
    a[2 * h + j] = g_c * gi * (1.f - gg * gg);
    a[3 * h + j] = g_h * tc * go * (1.f - go);
    dc_out[t] = g_c * gf;
}

// -------------------------------------------------------------------------------------
// Error rows and loss: one warp per halo row u (all partitions concatenated).  E[u] = (w_u / M) (pred[u] - target[slot(u)])
// written over pred; the row's loss w_u / M * 1/2 |pred - target|^2 is summed in double per warp, the warps of a block in
// fixed order, the blocks by k_pt_sum in fixed order.
// -------------------------------------------------------------------------------------
#define PT_ROWS_PER_BLOCK 64

__global__ void __launch_bounds__(256)
k_pt_error(float *__restrict__ pred, int64_t ld, int64_t n_halo, int32_t d, const float *__restrict__ target, int64_t ld_t,
           const int32_t *__restrict__ halo_slot, const float *__restrict__ row_weight, const int64_t *__restrict__ halo_off, int32_t M,
           double *__restrict__ block_partial)
{
    __shared__ double red[8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t r0 = (int64_t)blockIdx.x * PT_ROWS_PER_BLOCK;
    double sum = 0.0;
    for (int i = warp; i < PT_ROWS_PER_BLOCK; i += 8) {
        const int64_t u = r0 + i;
        if (u >= n_halo) break;
        float w;
        if (row_weight) {
            w = row_weight[u];
        } else {
            int lo = 0, hi = M;   // halo_off[lo] <= u < halo_off[hi]
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (halo_off[mid] <= u) lo = mid;
                else hi = mid;
            }
            w = 1.f / (float)(halo_off[lo + 1] - halo_off[lo]);
        }
        w /= (float)M;
        float *p = pred + u * ld;
        const float *t = target + (int64_t)halo_slot[u] * ld_t;
        float acc = 0.f;
        for (int c = lane; c < d; c += 32) {
            const float df = p[c] - t[c];
            acc = fmaf(df, df, acc);
            p[c] = w * df;
        }
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        sum += 0.5 * (double)w * (double)acc;
    }
    if (lane == 0) red[warp] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += red[w];
        block_partial[blockIdx.x] = s;
    }
}

__global__ void k_pt_sum(const double *__restrict__ block_partial, int64_t count, double *total)
{
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    double s = 0.0;
    for (int64_t i = 0; i < count; ++i) s += block_partial[i];
    *total = s;
}

// -------------------------------------------------------------------------------------
// Transposed graph convolution, G_S = sum_m (conv_m)^T G_a^(m), in two parts that never write the same element twice
// within a launch, so the result does not depend on scheduling:
//  (1) neighbour terms: boundary node v (inner row `row` of its partition, cache slot s) receives
//      sum over its out-of-partition neighbours u of p_uv G_a[halo position of u in v's partition] — the halo entries of
//      v's local CSR row; every slot is written exactly once (overwrite);
//  (2) self terms: halo row u of partition m adds p_uu G_a[u] to the slot of u; the halo slots of one partition are
//      distinct, and the partitions are launched one after the other.
// A group of 16 lanes per row, float4 per lane and pass.
// -------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
k_pt_gs_neighbours(const int32_t *__restrict__ push_row, const int32_t *__restrict__ push_slot, int32_t n_slots,
                   const int64_t *__restrict__ lrowptr, const int32_t *__restrict__ inner_cnt, const int32_t *__restrict__ lenc,
                   const float *__restrict__ dinv_enc, int32_t n, int32_t h4, const float *__restrict__ g_a, int64_t ld_a,
                   float *__restrict__ g_s, int64_t ld_s)
{
    const int lane = threadIdx.x & 15;
    const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 4;
    if (i >= n_slots) return;
    const int32_t row = push_row[i];
    const int64_t e0 = lrowptr[row] + inner_cnt[row], e1 = lrowptr[row + 1];
    const float dv = dinv_enc[row];
    for (int c0 = 0; c0 < h4; c0 += 16) {
        const int c = c0 + lane;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < h4) {
            for (int64_t e = e0; e < e1; ++e) {
                const int32_t enc = __ldg(lenc + e);
                const float w = __ldg(dinv_enc + enc);
                const float4 x = __ldg(reinterpret_cast<const float4 *>(g_a + (int64_t)(enc - n) * ld_a) + c);
                acc.x = fmaf(w, x.x, acc.x);
                acc.y = fmaf(w, x.y, acc.y);
                acc.z = fmaf(w, x.z, acc.z);
                acc.w = fmaf(w, x.w, acc.w);
            }
            reinterpret_cast<float4 *>(g_s + (int64_t)push_slot[i] * ld_s)[c] = make_float4(dv * acc.x, dv * acc.y, dv * acc.z, dv * acc.w);
        }
    }
}

__global__ void __launch_bounds__(256)
k_pt_gs_self(const int32_t *__restrict__ halo_slot, const float *__restrict__ dinv_enc, int32_t n, int64_t halo0, int64_t n_halo,
             int32_t h4, const float *__restrict__ g_a, int64_t ld_a, float *__restrict__ g_s, int64_t ld_s)
{
    const int lane = threadIdx.x & 15;
    const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 4;
    if (i >= n_halo) return;
    const int64_t u = halo0 + i;
    const float du = dinv_enc[n + u];
    const float p = du * du;
    float4 *dst = reinterpret_cast<float4 *>(g_s + (int64_t)halo_slot[u] * ld_s);
    const float4 *src = reinterpret_cast<const float4 *>(g_a + u * ld_a);
    for (int c = lane; c < h4; c += 16) {
        float4 o = dst[c];
        const float4 x = src[c];
        o.x = fmaf(p, x.x, o.x);
        o.y = fmaf(p, x.y, o.y);
        o.z = fmaf(p, x.z, o.z);
        o.w = fmaf(p, x.w, o.w);
        dst[c] = o;
    }
}

// -------------------------------------------------------------------------------------
// host side
// -------------------------------------------------------------------------------------
sat_status sat_gemm_nn_dual(sat_ctx *ctx, int64_t m, int32_t n, int32_t k1, const float *A1, int32_t lda1, const float *B1, int32_t ldb1,
                            int32_t k2, const float *A2, int32_t lda2, const float *B2, int32_t ldb2, const float *bias, float *C,
                            int32_t ldc);

// C[m x n] (+)= A^T B over `rows` rows, colsum[n] (+)= 1^T B: the same choice of kernel as the weight gradient of a layer
static sat_status pt_tn(sat_ctx *ctx, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B, int32_t ldb, float *C,
                        float *colsum, int accumulate)
{
    if (sat_use_tc(n, m) && rows >= 256) {
        if (colsum) SAT_TRY(sat_mask_rows(ctx, B, ldb, rows, n, nullptr, 0, nullptr, 0, colsum, accumulate));
        if (n <= 64) return sat_gemm_tn_narrow(ctx, rows, m, n, A, lda, B, ldb, C, n, accumulate);
        return sat_gemm_tc_tn(ctx, rows, m, n, A, lda, B, ldb, C, n, accumulate);
    }
    return sat_gemm_tn(ctx, rows, m, n, A, lda, B, ldb, nullptr, 0, C, n, colsum, accumulate);
}

// C[m x n] = A[m x k] W^T, W stored [n x k] row-major
static sat_status pt_nt(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const float *W, float *C, int32_t ldc)
{
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

static size_t pt_round(size_t floats) { return (floats + 63) & ~(size_t)63; }

extern "C" sat_status sat_pred_grad(sat_ctx *ctx, int32_t layer, const sat_pred_params *params, const float *row_weight, float *g_Wx,
                                    float *g_Uh, float *g_b, float *g_Wg, float *g_bg, double *loss_host)
{
    CHECK_CTX(ctx);
    if (!ctx->cache_ok) return sat_fail(ctx, SAT_ESTATE, "sat_pred_grad: sat_cache_init has not run");
    if (layer < 1 || layer > ctx->n_cached) return sat_fail(ctx, SAT_EINVAL, "sat_pred_grad: cached layer must be in [1, %d]", ctx->n_cached);
    CacheLayer *c = &ctx->cache[layer - 1];
    if (!params || params->h <= 0 || (params->h & 3) || !params->Wx || !params->Uh || !params->b || !params->Wg || !params->bg)
        return sat_fail(ctx, SAT_EINVAL, "sat_pred_grad: incomplete predictor parameters or h not a multiple of 4");
    if (!g_Wx || !g_Uh || !g_b || !g_Wg || !g_bg) return sat_fail(ctx, SAT_EINVAL, "sat_pred_grad: null gradient array");
    if (!aligned16(g_Wx) || !aligned16(g_Uh) || !aligned16(g_Wg)) return sat_fail(ctx, SAT_EINVAL, "sat_pred_grad: misaligned gradient array");
    PartView v;
    SAT_TRY(sat_part_view(ctx, SAT_ALL_PARTS, &v));
    const int32_t h = params->h, d = c->width, M = ctx->M;
    const int64_t R = ctx->n_slots, nb = v.n_halo;
    const int32_t k = ctx->n_valid < ctx->tau ? ctx->n_valid : ctx->tau;
    const int32_t ld_d = round_up4(d);
    SAT_CUDA(ctx, cudaMemsetAsync(g_Wx, 0, (size_t)d * 4 * h * sizeof(float), ctx->stream));
    SAT_CUDA(ctx, cudaMemsetAsync(g_Uh, 0, (size_t)h * 4 * h * sizeof(float), ctx->stream));
    SAT_CUDA(ctx, cudaMemsetAsync(g_b, 0, (size_t)4 * h * sizeof(float), ctx->stream));
    SAT_CUDA(ctx, cudaMemsetAsync(g_Wg, 0, (size_t)h * d * sizeof(float), ctx->stream));
    SAT_CUDA(ctx, cudaMemsetAsync(g_bg, 0, (size_t)d * sizeof(float), ctx->stream));
    if (nb == 0 || R == 0) {   // no halo row anywhere: the objective is empty
        if (loss_host) {
            SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
            *loss_host = 0.0;
        }
        return SAT_OK;
    }
    // ---- scratch ----
    const int64_t n_blocks = cdiv64(nb, PT_ROWS_PER_BLOCK);
    const size_t f_gates = pt_round((size_t)(k > 0 ? k : 1) * R * 4 * h), f_state = pt_round((size_t)(k > 0 ? k : 1) * R * h);
    const size_t f_a = pt_round((size_t)nb * h), f_e = pt_round((size_t)nb * ld_d), f_rh = pt_round((size_t)R * h);
    const size_t f_off = pt_round(2 * (size_t)(M + 1)), f_part = pt_round(2 * (size_t)(n_blocks + 1));
    SAT_TRY(sat_ensure(ctx, ctx->buf_pred_train, (f_gates + 2 * f_state + 2 * f_a + f_e + 2 * f_rh + f_off + f_part) * sizeof(float)));
    float *gates = (float *)ctx->buf_pred_train.p;
    float *hs = gates + f_gates, *cs = hs + f_state;
    float *a = cs + f_state, *g_a = a + f_a, *E = g_a + f_a;
    float *dh = E + f_e, *dc = dh + f_rh;
    int64_t *halo_off = (int64_t *)(dc + f_rh);
    double *partial = (double *)((float *)halo_off + f_off);
    SAT_CUDA(ctx, cudaMemcpyAsync(halo_off, ctx->h_halo_off.data(), (size_t)(M + 1) * sizeof(int64_t), cudaMemcpyHostToDevice, ctx->stream));
    const int64_t plane_g = R * 4 * (int64_t)h, plane_s = R * (int64_t)h;
    const unsigned cell_grid = (unsigned)cdiv64(plane_s, 256);
    // ---- LSTM forward over the snapshots, oldest first, gate values kept ----
    const bool tc_z = sat_use_tc(4 * h, d);
    TcWeights W1, W2;
    if (tc_z && k > 0) SAT_TRY(sat_tc_weights(ctx, params->Wx, 4 * h, d, nullptr, 0, 0, 4 * h, 1, ctx->buf_wsplit, &W1));
    if (tc_z && k > 1) SAT_TRY(sat_tc_weights(ctx, params->Wx, 4 * h, d, params->Uh, 4 * h, h, 4 * h, 1, ctx->buf_wsplit2, &W2));
    for (int32_t t = 0; t < k; ++t) {
        const float *x = ring_buf(ctx, c, ring_index(ctx, k - 1 - t));
        float *z = gates + t * plane_g;
        const float *h_prev = t ? hs + (t - 1) * plane_s : nullptr;
        if (tc_z) {
            TcEpilogueHost eh;
            eh.C = z;
            eh.ldc = 4 * h;
            eh.bias = params->b;
            SAT_TRY(sat_gemm_tc(ctx, R, 4 * h, x, c->ld, d, h_prev, h, t ? h : 0, t ? W2 : W1, eh, SATK_GEMM_NN));
        } else {
            SAT_TRY(sat_gemm_nn_dual(ctx, R, 4 * h, d, x, c->ld, params->Wx, 4 * h, t ? h : 0, h_prev, h, params->Uh, 4 * h, params->b, z, 4 * h));
        }
        ProfScope prof(ctx, SATK_PRED_TRAIN, 4.0 * (double)plane_s * 11.0, 0.0);
        k_pt_cell_fwd<<<cell_grid, 256, 0, ctx->stream>>>(z, R, h, t ? cs + (t - 1) * plane_s : nullptr, cs + t * plane_s, hs + t * plane_s);
        SAT_LAUNCHED(ctx);
    }
    // ---- graph convolution on the final state, output layer, skip connection ----
    const float *newest = k > 0 ? ring_buf(ctx, c, ring_index(ctx, 0)) : nullptr;
    if (k > 0) SAT_TRY(sat_spmm_hrow(ctx, v, h, hs + (k - 1) * plane_s, h, 1, hs + (k - 1) * plane_s, a, h));
    else SAT_CUDA(ctx, cudaMemsetAsync(a, 0, (size_t)nb * h * sizeof(float), ctx->stream));
    if (sat_use_tc(d, h)) {
        TcWeights Wg;
        SAT_TRY(sat_tc_weights(ctx, params->Wg, d, h, nullptr, 0, 0, d, 1, ctx->buf_wsplit, &Wg));
        TcEpilogueHost eh;
        eh.C = E;
        eh.ldc = ld_d;
        eh.bias = params->bg;
        if (newest) {
            eh.resid = newest;
            eh.resid_idx = ctx->halo_slot;
            eh.ld_resid = c->ld;
        }
        SAT_TRY(sat_gemm_tc(ctx, nb, d, a, h, h, nullptr, 0, 0, Wg, eh, SATK_GEMM_SIDE));
    } else {
        GemmEpilogue ep;
        ep.bias = params->bg;
        if (newest) {
            ep.resid = newest;
            ep.resid_idx = ctx->halo_slot;
            ep.ld_resid = c->ld;
        }
        SAT_TRY(sat_gemm_nn(ctx, nb, d, h, a, h, params->Wg, d, E, ld_d, ep));
    }
    // ---- loss and error rows ----
    {
        ProfScope prof(ctx, SATK_PRED_TRAIN, 4.0 * (double)nb * d * 3.0, 0.0);
        k_pt_error<<<(unsigned)n_blocks, 256, 0, ctx->stream>>>(E, ld_d, nb, d, ring_buf(ctx, c, ctx->write_idx), c->ld, ctx->halo_slot, row_weight,
                                                                halo_off, M, partial);
        SAT_LAUNCHED(ctx);
        k_pt_sum<<<1, 32, 0, ctx->stream>>>(partial, n_blocks, partial + n_blocks);
        SAT_LAUNCHED(ctx);
    }
    // ---- output layer: G_Wg = a^T E, G_bg = 1^T E, G_a = E Wg^T ----
    SAT_TRY(pt_tn(ctx, nb, h, d, a, h, E, ld_d, g_Wg, g_bg, 0));
    if (k > 0) {
        SAT_TRY(pt_nt(ctx, nb, h, d, E, ld_d, params->Wg, g_a, h));
        // ---- transposed graph convolution: gradient of the final hidden state ----
        {
            ProfScope prof(ctx, SATK_PRED_TRAIN, 0.0, 0.0);
            k_pt_gs_neighbours<<<(unsigned)cdiv64(R * 16, 256), 256, 0, ctx->stream>>>(ctx->push_row, ctx->push_slot, (int32_t)R, ctx->lrowptr,
                                                                                     ctx->inner_cnt, ctx->lenc, ctx->dinv_enc, ctx->n, h / 4, g_a, h,
                                                                                     dh, h);
            SAT_LAUNCHED(ctx);
            for (int32_t m = 0; m < M; ++m) {
                const int64_t h0 = ctx->h_halo_off[m], cnt = ctx->h_halo_off[m + 1] - h0;
                if (cnt == 0) continue;
                k_pt_gs_self<<<(unsigned)cdiv64(cnt * 16, 256), 256, 0, ctx->stream>>>(ctx->halo_slot, ctx->dinv_enc, ctx->n, h0, cnt, h / 4, g_a, h,
                                                                                      dh, h);
                SAT_LAUNCHED(ctx);
            }
        }
        // ---- back-propagation through time ----
        for (int32_t t = k - 1; t >= 0; --t) {
            const float *x = ring_buf(ctx, c, ring_index(ctx, k - 1 - t));
            float *z = gates + t * plane_g;
            {
                ProfScope prof(ctx, SATK_PRED_TRAIN, 4.0 * (double)plane_s * 13.0, 0.0);
                k_pt_cell_bwd<<<cell_grid, 256, 0, ctx->stream>>>(z, R, h, t ? cs + (t - 1) * plane_s : nullptr, cs + t * plane_s, dh,
                                                                  t == k - 1 ? nullptr : dc, dc);
                SAT_LAUNCHED(ctx);
            }
            const int acc = t != k - 1;
            SAT_TRY(pt_tn(ctx, R, d, 4 * h, x, c->ld, z, 4 * h, g_Wx, g_b, acc));
            if (t > 0) {
                SAT_TRY(pt_tn(ctx, R, h, 4 * h, hs + (t - 1) * plane_s, h, z, 4 * h, g_Uh, nullptr, acc));
                SAT_TRY(pt_nt(ctx, R, h, 4 * h, z, 4 * h, params->Uh, dh, h));
            }
        }
    }
    if (loss_host) {
        SAT_CUDA(ctx, cudaMemcpyAsync(loss_host, partial + n_blocks, sizeof(double), cudaMemcpyDeviceToHost, ctx->stream));
        SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    }
    return SAT_OK;
}
