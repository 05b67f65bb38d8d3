// Objective and gradient of the embedding predictor (Eq. "predictor loss", Eq. "mini-batch training", Algorithm 1
// "Embedding predictor update"): forward pass of the LSTM + graph convolution + skip connection with the gate values kept,
// squared-error loss against the embeddings pushed in the running epoch, and the backward pass through the output layer,
// the transposed graph convolution and the LSTM (back-propagation through time).  The dense contractions run on the same
// GEMM kernels as the layer steps; this file holds the element-wise and sparse kernels around them.
#include "sat_internal.h"


// -------------------------------------------------------------------------------------
// LSTM cell kernels.  A thread owns four consecutive hidden units of a row (one 16-byte access per gate block and state
// array); h / 4 threads cover a row, 256 / (h / 4) rows are in flight per pass, and a block walks PT_TILE_ROWS rows.
// Forward, with everything the backward needs: z [rows x 4h] holds the gate pre-activations (blocks i | f | g | o) and is
// overwritten with the gate values; c_out = f c_prev + i g; h_out = o tanh(c_out).
// -------------------------------------------------------------------------------------
#define PT_TILE_ROWS 128

__device__ __forceinline__ float4 ld4s(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ void st4s(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
#define PT_MAP4(out, expr)                   \
    do {                                     \
        { const int e = 0; (out).x = (expr); } \
        { const int e = 1; (out).y = (expr); } \
        { const int e = 2; (out).z = (expr); } \
        { const int e = 3; (out).w = (expr); } \
    } while (0)
__device__ __forceinline__ float el(const float4 &v, int e) { return e == 0 ? v.x : e == 1 ? v.y : e == 2 ? v.z : v.w; }

__global__ void __launch_bounds__(256)
k_pt_cell_fwd(float *__restrict__ z, int64_t rows, int32_t h, const float *__restrict__ c_prev, float *__restrict__ c_out,
              float *__restrict__ h_out)
{
    const int h4 = h >> 2, rpp = 256 / h4;
    const int q = threadIdx.x % h4, rr = threadIdx.x / h4;
    if (rr >= rpp) return;
    const int64_t r_end = min(rows, ((int64_t)blockIdx.x + 1) * PT_TILE_ROWS);
    for (int64_t r = (int64_t)blockIdx.x * PT_TILE_ROWS + rr; r < r_end; r += rpp) {
        float *a = z + r * 4 * (int64_t)h + 4 * q;
        const float4 zi = ld4s(a), zf = ld4s(a + h), zg = ld4s(a + 2 * h), zo = ld4s(a + 3 * h);
        const float4 cp = c_prev ? ld4s(c_prev + r * h + 4 * q) : make_float4(0.f, 0.f, 0.f, 0.f);
        float4 gi, gf, gg, go, cn, hn;
        PT_MAP4(gi, sigmoid_fast(el(zi, e)));
        PT_MAP4(gf, sigmoid_fast(el(zf, e)));
        PT_MAP4(gg, tanh_fast(el(zg, e)));
        PT_MAP4(go, sigmoid_fast(el(zo, e)));
        PT_MAP4(cn, fmaf(el(gf, e), el(cp, e), el(gi, e) * el(gg, e)));
        PT_MAP4(hn, el(go, e) * tanh_fast(el(cn, e)));
        st4s(a, gi);
        st4s(a + h, gf);
        st4s(a + 2 * h, gg);
        st4s(a + 3 * h, go);
        st4s(c_out + r * h + 4 * q, cn);
        st4s(h_out + r * h + 4 * q, hn);
    }
}

// Backward: gz [rows x 4h] holds the gate values of the step and is overwritten with the gradient of the loss with respect
// to the gate pre-activations; dc carries the gradient of the cell state from the later steps (null at the last step) and
// leaves as the gradient with respect to the previous cell state.  The column sums of the written gradients (the bias
// gradient of the step) are accumulated on the way: per thread over its rows, then over the row groups of the block in
// fixed order into colsum_part [gridDim.x x 4h].
__global__ void __launch_bounds__(256)
k_pt_cell_bwd(float *__restrict__ gz, int64_t rows, int32_t h, const float *__restrict__ c_prev, const float *__restrict__ c_cur,
              const float *__restrict__ dh, const float *dc_in, float *dc_out, float *__restrict__ colsum_part)
{
    extern __shared__ float red[];   // [rpp][4h]
    const int h4 = h >> 2, rpp = 256 / h4;
    const int q = threadIdx.x % h4, rr = threadIdx.x / h4;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 si = zero, sf = zero, sg = zero, so = zero;
    if (rr < rpp) {
        // the block's tiles: blockIdx.x, blockIdx.x + gridDim.x, ... (fixed order, one partial column sum per block)
        for (int64_t tile = blockIdx.x; tile * PT_TILE_ROWS < rows; tile += gridDim.x)
        for (int64_t r = tile * PT_TILE_ROWS + rr; r < min(rows, (tile + 1) * PT_TILE_ROWS); r += rpp) {
            float *a = gz + r * 4 * (int64_t)h + 4 * q;
            const int64_t o = r * h + 4 * q;
            const float4 gi = ld4s(a), gf = ld4s(a + h), gg = ld4s(a + 2 * h), go = ld4s(a + 3 * h);
            const float4 cc = ld4s(c_cur + o), g_h = ld4s(dh + o);
            const float4 cp = c_prev ? ld4s(c_prev + o) : zero;
            const float4 dci = dc_in ? ld4s(dc_in + o) : zero;
            float4 tc, g_c, di, df, dg, dd, dcp;
            PT_MAP4(tc, tanh_fast(el(cc, e)));
            PT_MAP4(g_c, fmaf(el(g_h, e) * el(go, e), 1.f - el(tc, e) * el(tc, e), el(dci, e)));
            PT_MAP4(di, el(g_c, e) * el(gg, e) * el(gi, e) * (1.f - el(gi, e)));
            PT_MAP4(df, el(g_c, e) * el(cp, e) * el(gf, e) * (1.f - el(gf, e)));
            PT_MAP4(dg, el(g_c, e) * el(gi, e) * (1.f - el(gg, e) * el(gg, e)));
            PT_MAP4(dd, el(g_h, e) * el(tc, e) * el(go, e) * (1.f - el(go, e)));
            PT_MAP4(dcp, el(g_c, e) * el(gf, e));
            st4s(a, di);
            st4s(a + h, df);
            st4s(a + 2 * h, dg);
            st4s(a + 3 * h, dd);
            st4s(dc_out + o, dcp);
            PT_MAP4(si, el(si, e) + el(di, e));
            PT_MAP4(sf, el(sf, e) + el(df, e));
            PT_MAP4(sg, el(sg, e) + el(dg, e));
            PT_MAP4(so, el(so, e) + el(dd, e));
        }
        float *mine = red + (size_t)rr * 4 * h + 4 * q;
        st4s(mine, si);
        st4s(mine + h, sf);
        st4s(mine + 2 * h, sg);
        st4s(mine + 3 * h, so);
    }
    __syncthreads();
    for (int c = threadIdx.x; c < 4 * h; c += 256) {
        float s = 0.f;
        for (int g = 0; g < rpp; ++g) s += red[(size_t)g * 4 * h + c];
        colsum_part[(size_t)blockIdx.x * 4 * h + c] = s;
    }
}

// -------------------------------------------------------------------------------------
// Error rows and loss: one warp per halo row u (all partitions concatenated), 8 warps x 8 rows per tile, a block walking every gridDim.x-th tile.
// E[u] = (w_u / M) (pred[u] - target[slot(u)]) written over pred; the row's loss w_u / M * 1/2 |pred - target|^2 is summed in
// double per warp, the warps of a block in fixed order, the blocks by k_pt_sum in fixed order.  The column sums of E (the
// gradient of the output bias) are accumulated per warp in shared memory over its rows, then over the warps in fixed
// order, into colsum_part [gridDim.x x d].
// -------------------------------------------------------------------------------------
#define PT_ROWS_PER_BLOCK 64

__global__ void __launch_bounds__(256)
k_pt_error(float *__restrict__ pred, int64_t ld, int64_t n_halo, int32_t d, const float *__restrict__ target, int64_t ld_t,
           const int32_t *__restrict__ halo_slot, const float *__restrict__ row_weight, const int64_t *__restrict__ halo_off, int32_t M,
           double *__restrict__ block_partial, float *__restrict__ colsum_part)
{
    extern __shared__ float4 cs4[];   // [8 warps][d rounded up to 4]
    float *cs = reinterpret_cast<float *>(cs4);
    __shared__ double red[8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int d4 = (d + 3) >> 2;
    float *mine = cs + (size_t)warp * 4 * d4;
    for (int c = lane; c < 4 * d4; c += 32) mine[c] = 0.f;
    double sum = 0.0;
    // the block's row tiles: blockIdx.x, blockIdx.x + gridDim.x, ... in order
    for (int64_t r0 = (int64_t)blockIdx.x * PT_ROWS_PER_BLOCK; r0 < n_halo; r0 += (int64_t)gridDim.x * PT_ROWS_PER_BLOCK)
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
        float4 *p4 = reinterpret_cast<float4 *>(pred + u * ld);
        const float4 *t4 = reinterpret_cast<const float4 *>(target + (int64_t)halo_slot[u] * ld_t);
        float4 *m4 = reinterpret_cast<float4 *>(mine);
        float acc = 0.f;
#pragma unroll 2
        for (int c4 = lane; c4 < d4; c4 += 32) {
            const float4 pv = p4[c4], tv = __ldg(t4 + c4);
            float4 df = make_float4(pv.x - tv.x, pv.y - tv.y, pv.z - tv.z, pv.w - tv.w);
            if (4 * c4 + 3 >= d) {   // the padding columns of the last vector hold no data
                if (4 * c4 + 1 >= d) df.y = 0.f;
                if (4 * c4 + 2 >= d) df.z = 0.f;
                df.w = 0.f;
            }
            acc = fmaf(df.x, df.x, fmaf(df.y, df.y, fmaf(df.z, df.z, fmaf(df.w, df.w, acc))));
            const float4 ev = make_float4(w * df.x, w * df.y, w * df.z, w * df.w);
            p4[c4] = ev;
            float4 mv = m4[c4];
            mv.x += ev.x;
            mv.y += ev.y;
            mv.z += ev.z;
            mv.w += ev.w;
            m4[c4] = mv;
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
    for (int c = threadIdx.x; c < d; c += 256) {
        float s = 0.f;
        for (int w = 0; w < 8; ++w) s += cs[(size_t)w * 4 * d4 + c];
        colsum_part[(size_t)blockIdx.x * d + c] = s;
    }
}

// total = sum of the block partials: thread t adds the partials t, t + 256, ... in order, then the 256 thread sums are added
// in index order; the association is fixed, so the total does not depend on scheduling
__global__ void __launch_bounds__(256) k_pt_sum(const double *__restrict__ block_partial, int64_t count, double *total)
{
    __shared__ double part[256];
    double s = 0.0;
    for (int64_t i = threadIdx.x; i < count; i += 256) s += block_partial[i];
    part[threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int i = 0; i < 256; ++i) t += part[i];
        *total = t;
    }
}

// -------------------------------------------------------------------------------------
// Transposed graph convolution, G_S = sum_m (conv_m)^T G_a^(m), in two parts that never write the same element twice
// within a launch, so the result does not depend on scheduling:
//  (1) neighbour terms: boundary node v (inner row of its partition) receives the sum over its out-of-partition
//      neighbours u of p_uv G_a[halo position of u in v's partition] — the halo suffix of v's local CSR row, i.e. the
//      layer SpMM restricted to halo columns (rows cut into chunks like there, so hub nodes do not serialise); the rows of
//      the boundary nodes are then copied to their cache slots, every slot exactly once;
//  (2) self terms: the slot of u receives p_uu times the sum of G_a over the copies of u (its halo positions in the other
//      partitions), taken in partition order through the halo-positions-by-slot index (sat_sum_by_slot).
// -------------------------------------------------------------------------------------
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
    if (params->cell != SAT_CELL_LSTM) return sat_fail(ctx, SAT_EINVAL, "sat_pred_grad: only the LSTM predictor is differentiated");
    if (params->h > 1024 || c->width > 1536) return sat_fail(ctx, SAT_EINVAL, "sat_pred_grad: supports h <= 1024 and cached widths <= 1536");
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
    const int64_t n_tiles = cdiv64(nb, PT_ROWS_PER_BLOCK);
    const int64_t n_blocks = n_tiles < 8 * 148 ? n_tiles : 8 * 148;   // error kernel: the resident blocks of all SMs, each walking its tiles
    const size_t f_gates = pt_round((size_t)(k > 0 ? k : 1) * R * 4 * h), f_state = pt_round((size_t)(k > 0 ? k : 1) * R * h);
    const size_t f_a = pt_round((size_t)nb * h), f_e = pt_round((size_t)nb * ld_d), f_rh = pt_round((size_t)R * h);
    const size_t f_off = pt_round(2 * (size_t)(M + 1)), f_part = pt_round(2 * (size_t)(n_blocks + 1)), f_nh = pt_round((size_t)ctx->n * h);
    SAT_TRY(sat_ensure(ctx, ctx->buf_pred_train, (f_gates + 2 * f_state + 2 * f_a + f_e + 2 * f_rh + f_off + f_part + f_nh) * sizeof(float)));
    float *gates = (float *)ctx->buf_pred_train.p;
    float *hs = gates + f_gates, *cs = hs + f_state;
    float *a = cs + f_state, *g_a = a + f_a, *E = g_a + f_a;
    float *dh = E + f_e, *dc = dh + f_rh;
    int64_t *halo_off = (int64_t *)(dc + f_rh);
    double *partial = (double *)((float *)halo_off + f_off);
    float *g_rows = (float *)partial + f_part;   // [n x h] neighbour terms of the transposed convolution by inner row
    SAT_CUDA(ctx, cudaMemcpyAsync(halo_off, ctx->h_halo_off.data(), (size_t)(M + 1) * sizeof(int64_t), cudaMemcpyHostToDevice, ctx->stream));
    const int64_t plane_g = R * 4 * (int64_t)h, plane_s = R * (int64_t)h;
    const unsigned cell_grid = (unsigned)cdiv64(R, PT_TILE_ROWS);
    const unsigned bwd_grid = cell_grid < 8 * 148 ? cell_grid : 8 * 148;
    const size_t cell_smem = (size_t)(256 / (h / 4)) * 4 * h * sizeof(float);
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
        SAT_TRY(sat_ensure(ctx, ctx->buf_colsum, (size_t)n_blocks * d * sizeof(float)));
        k_pt_error<<<(unsigned)n_blocks, 256, (size_t)8 * ld_d * sizeof(float), ctx->stream>>>(E, ld_d, nb, d, ring_buf(ctx, c, ctx->write_idx), c->ld,
                                                                                           ctx->halo_slot, row_weight, halo_off, M, partial,
                                                                                           (float *)ctx->buf_colsum.p);
        SAT_LAUNCHED(ctx);
        k_pt_sum<<<1, 256, 0, ctx->stream>>>(partial, n_blocks, partial + n_blocks);
        SAT_LAUNCHED(ctx);
    }
    SAT_TRY(sat_splitk_reduce(ctx, (const float *)ctx->buf_colsum.p, d, (int32_t)n_blocks, 0, g_bg, d, d));
    // ---- output layer: G_Wg = a^T E, G_bg = 1^T E, G_a = E Wg^T ----
    SAT_TRY(pt_tn(ctx, nb, h, d, a, h, E, ld_d, g_Wg, nullptr, 0));
    if (k > 0) {
        SAT_TRY(pt_nt(ctx, nb, h, d, E, ld_d, params->Wg, g_a, h));
        // ---- transposed graph convolution: gradient of the final hidden state ----
        SAT_TRY(sat_spmm(ctx, v, 2, h, nullptr, 0, g_a, h, g_rows, h));
        SAT_TRY(sat_scatter(ctx, ctx->push_row, ctx->push_slot, R, h, g_rows, h, dh, h));
        SAT_TRY(sat_sum_by_slot(ctx, h, g_a, h, 1, 1, dh, h));
        // ---- back-propagation through time ----
        for (int32_t t = k - 1; t >= 0; --t) {
            const float *x = ring_buf(ctx, c, ring_index(ctx, k - 1 - t));
            float *z = gates + t * plane_g;
            {
                ProfScope prof(ctx, SATK_PRED_TRAIN, 4.0 * (double)plane_s * 13.0, 0.0);
                SAT_TRY(sat_ensure(ctx, ctx->buf_colsum, (size_t)bwd_grid * 4 * h * sizeof(float)));
                k_pt_cell_bwd<<<bwd_grid, 256, cell_smem, ctx->stream>>>(z, R, h, t ? cs + (t - 1) * plane_s : nullptr, cs + t * plane_s, dh,
                                                                          t == k - 1 ? nullptr : dc, dc, (float *)ctx->buf_colsum.p);
                SAT_LAUNCHED(ctx);
            }
            const int acc = t != k - 1;
            SAT_TRY(sat_splitk_reduce(ctx, (const float *)ctx->buf_colsum.p, 4 * h, (int32_t)bwd_grid, acc, g_b, 4 * h, 4 * h));
            SAT_TRY(pt_tn(ctx, R, d, 4 * h, x, c->ld, z, 4 * h, g_Wx, nullptr, acc));
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
