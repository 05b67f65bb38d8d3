// Dense contractions of the sat_b200 library on the CUDA cores (fp32 FMA, fp32 accumulate):
// the general-shape path used for every size the tensor-core path does not take.
//   NN: C = A B (+bias, ReLU, sign mask, gathered residual)          layer transform, predictor output
//   NT: C = (A o mask) B^T                                            input gradient  D W^T
//   TN: C (+)= A^T (B o mask), colsum (+)= 1^T (B o mask), split-K    weight / bias gradient
#include "sat_internal.h"

#define BM 64
#define BN 64
#define BK 16
#define TN_ROWS_PER_SPLIT 4096

__device__ __forceinline__ bool mask_bit(const uint32_t *mask, int64_t row, int32_t mask_words, int32_t c)
{
    return (mask[row * mask_words + (c >> 5)] >> (c & 31)) & 1u;
}

// 256 threads, thread (ty, tx) = (t / 16, t % 16) owns rows ty*4.., cols tx*4.. of the 64x64 tile
#define INNER_PRODUCT()                                              \
    _Pragma("unroll") for (int kk = 0; kk < BK; ++kk) {             \
        float a[4], b[4];                                            \
        _Pragma("unroll") for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i]; \
        _Pragma("unroll") for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j]; \
        _Pragma("unroll") for (int i = 0; i < 4; ++i)                \
            _Pragma("unroll") for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]); \
    }

__global__ void __launch_bounds__(256)
k_gemm_nn(int64_t m, int32_t n, int32_t k1, const float *__restrict__ A, int64_t lda, const float *__restrict__ B, int64_t ldb,
          int32_t k2, const float *__restrict__ A2, int64_t lda2, const float *__restrict__ B2, int64_t ldb2,
          float *__restrict__ C, int64_t ldc, const float *__restrict__ bias, int relu, uint32_t *__restrict__ mask_out,
          int32_t mask_words, const float *__restrict__ resid, const int32_t *__restrict__ resid_idx, int64_t ld_resid)
{
    // the contraction runs over the virtual concatenation [A | A2] [B ; B2] (k2 may be 0)
    const int32_t k = k1 + k2;
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
    const int64_t row0 = (int64_t)blockIdx.x * BM;
    const int32_t col0 = blockIdx.y * BN;
    float acc[4][4] = {};
    for (int32_t k0 = 0; k0 < k; k0 += BK) {
        {   // A tile: thread loads 4 consecutive k of one row
            const int r = t >> 2, kq = (t & 3) * 4;
            const int64_t gr = row0 + r;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int32_t gk = k0 + kq + q;
                float x = 0.f;
                if (gr < m && gk < k) x = gk < k1 ? A[gr * lda + gk] : A2[gr * lda2 + (gk - k1)];
                As[kq + q][r] = x;
            }
        }
        {   // B tile: thread loads 4 consecutive n of one k
            const int kk = t >> 4, nq = (t & 15) * 4;
            const int32_t gk = k0 + kk;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int32_t gn = col0 + nq + q;
                float x = 0.f;
                if (gk < k && gn < n) x = gk < k1 ? B[(int64_t)gk * ldb + gn] : B2[(int64_t)(gk - k1) * ldb2 + gn];
                Bs[kk][nq + q] = x;
            }
        }
        __syncthreads();
        INNER_PRODUCT();
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t gr = row0 + ty * 4 + i;
        uint32_t nib = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int32_t gn = col0 + tx * 4 + j;
            if (gr < m && gn < n) {
                float z = acc[i][j] + (bias ? bias[gn] : 0.f);
                if (resid) z += resid[(int64_t)resid_idx[gr] * ld_resid + gn];
                if (z > 0.f) nib |= 1u << j;
                if (relu && !(z > 0.f)) z = 0.f;
                C[gr * ldc + gn] = z;
            }
        }
        if (mask_out) {
            // 8 threads (tx & 7) share one 32-bit word of the row
            uint32_t wbits = nib << (4 * (tx & 7));
            wbits |= __shfl_xor_sync(0xffffffffu, wbits, 1);
            wbits |= __shfl_xor_sync(0xffffffffu, wbits, 2);
            wbits |= __shfl_xor_sync(0xffffffffu, wbits, 4);
            const int32_t word = (col0 >> 5) + (tx >> 3);
            if ((tx & 7) == 0 && gr < m && word < mask_words) mask_out[gr * mask_words + word] = wbits;
        }
    }
}

sat_status sat_gemm_nn(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const float *B, int32_t ldb,
                       float *C, int32_t ldc, const GemmEpilogue &ep)
{
    if (m == 0 || n == 0) return SAT_OK;
    ProfScope prof(ctx, SATK_GEMM_NN, 4.0 * ((double)m * (k + n) + (double)k * n), 2.0 * (double)m * n * k);
    dim3 grid((unsigned)cdiv64(m, BM), (unsigned)cdiv64(n, BN));
    k_gemm_nn<<<grid, 256, 0, ctx->stream>>>(m, n, k, A, lda, B, ldb, 0, nullptr, 0, nullptr, 0, C, ldc, ep.bias, ep.relu, ep.mask_out,
                                             ep.mask_words, ep.resid, ep.resid_idx, ep.ld_resid);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

sat_status sat_gemm_nn_dual(sat_ctx *ctx, int64_t m, int32_t n, int32_t k1, const float *A1, int32_t lda1, const float *B1, int32_t ldb1,
                            int32_t k2, const float *A2, int32_t lda2, const float *B2, int32_t ldb2, const float *bias, float *C,
                            int32_t ldc)
{
    if (m == 0 || n == 0) return SAT_OK;
    ProfScope prof(ctx, SATK_GEMM_NN, 4.0 * ((double)m * (k1 + k2 + n) + (double)(k1 + k2) * n), 2.0 * (double)m * n * (k1 + k2));
    dim3 grid((unsigned)cdiv64(m, BM), (unsigned)cdiv64(n, BN));
    k_gemm_nn<<<grid, 256, 0, ctx->stream>>>(m, n, k1, A1, lda1, B1, ldb1, k2, A2, lda2, B2, ldb2, C, ldc, bias, 0, nullptr, 0, nullptr,
                                             nullptr, 0);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

__global__ void __launch_bounds__(256)
k_gemm_nt(int64_t m, int32_t n, int32_t k, const float *__restrict__ A, int64_t lda, const uint32_t *__restrict__ mask,
          int32_t mask_words, const float *__restrict__ B, int64_t ldb, float *__restrict__ C, int64_t ldc)
{
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
    const int64_t row0 = (int64_t)blockIdx.x * BM;
    const int32_t col0 = blockIdx.y * BN;
    float acc[4][4] = {};
    for (int32_t k0 = 0; k0 < k; k0 += BK) {
        const int r = t >> 2, kq = (t & 3) * 4;
        {
            const int64_t gr = row0 + r;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int32_t gk = k0 + kq + q;
                float x = 0.f;
                if (gr < m && gk < k) {
                    x = A[gr * lda + gk];
                    if (mask && !mask_bit(mask, gr, mask_words, gk)) x = 0.f;
                }
                As[kq + q][r] = x;
            }
        }
        {   // B^T tile: B is [n x k]; thread loads 4 consecutive k of one n
            const int32_t gn = col0 + r;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int32_t gk = k0 + kq + q;
                Bs[kq + q][r] = (gn < n && gk < k) ? B[(int64_t)gn * ldb + gk] : 0.f;
            }
        }
        __syncthreads();
        INNER_PRODUCT();
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t gr = row0 + ty * 4 + i;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int32_t gn = col0 + tx * 4 + j;
            if (gr < m && gn < n) C[gr * ldc + gn] = acc[i][j];
        }
    }
}

sat_status sat_gemm_nt(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const uint32_t *mask,
                       int32_t mask_words, const float *B, int32_t ldb, float *C, int32_t ldc)
{
    if (m == 0 || n == 0) return SAT_OK;
    ProfScope prof(ctx, SATK_GEMM_NT, 4.0 * ((double)m * (k + n) + (double)k * n), 2.0 * (double)m * n * k);
    dim3 grid((unsigned)cdiv64(m, BM), (unsigned)cdiv64(n, BN));
    k_gemm_nt<<<grid, 256, 0, ctx->stream>>>(m, n, k, A, lda, mask, mask_words, B, ldb, C, ldc);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

// split-K over the row dimension: block (x, y, z) computes the [64 x 64] tile (x, y) of A^T (B o mask)
// over rows [z * rows_per_split, ...), and the blocks with x == 0 also the column sums of (B o mask).
__global__ void __launch_bounds__(256)
k_gemm_tn(int64_t rows, int64_t rows_per_split, int32_t m, int32_t n, const float *__restrict__ A, int64_t lda,
          const float *__restrict__ B, int64_t ldb, const uint32_t *__restrict__ mask, int32_t mask_words,
          float *__restrict__ part_C /* [splits x m x n] */, float *__restrict__ part_cs /* [splits x n] or null */)
{
    __shared__ float As[BK][BM + 4];
    __shared__ float Bs[BK][BN + 4];
    const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
    const int32_t m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const int64_t r_begin = (int64_t)blockIdx.z * rows_per_split;
    const int64_t r_end = (r_begin + rows_per_split < rows) ? r_begin + rows_per_split : rows;
    float acc[4][4] = {};
    float cs[4] = {0.f, 0.f, 0.f, 0.f};
    const bool want_cs = part_cs != nullptr && blockIdx.x == 0;
    for (int64_t r0 = r_begin; r0 < r_end; r0 += BK) {
        {   // A^T tile: As[kk][i] = A[r0 + kk][m0 + i]; thread loads 4 consecutive m of one row
            const int kk = t >> 4, iq = (t & 15) * 4;
            const int64_t gr = r0 + kk;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int32_t gm = m0 + iq + q;
                As[kk][iq + q] = (gr < r_end && gm < m) ? A[gr * lda + gm] : 0.f;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int32_t gn = n0 + iq + q;
                float x = 0.f;
                if (gr < r_end && gn < n) {
                    x = B[gr * ldb + gn];
                    if (mask && !mask_bit(mask, gr, mask_words, gn)) x = 0.f;
                }
                Bs[kk][iq + q] = x;
            }
        }
        __syncthreads();
        INNER_PRODUCT();
        if (want_cs && ty == 0) {
#pragma unroll
            for (int kk = 0; kk < BK; ++kk)
#pragma unroll
                for (int j = 0; j < 4; ++j) cs[j] += Bs[kk][tx * 4 + j];
        }
        __syncthreads();
    }
    float *pc = part_C + (int64_t)blockIdx.z * m * n;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int32_t gm = m0 + ty * 4 + i;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int32_t gn = n0 + tx * 4 + j;
            if (gm < m && gn < n) pc[(int64_t)gm * n + gn] = acc[i][j];
        }
    }
    if (want_cs && ty == 0) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int32_t gn = n0 + tx * 4 + j;
            if (gn < n) part_cs[(int64_t)blockIdx.z * n + gn] = cs[j];
        }
    }
}

// out[i] (+)= sum_z part[z][i]: eight lanes take the splits round-robin (four independent loads in flight each), their sums
// are added in lane order (fixed order: reproducible)
__global__ void __launch_bounds__(256)
k_splitk_reduce(const float *__restrict__ part, int64_t count, int32_t splits, int accumulate, float *__restrict__ out,
                int32_t ncols, int64_t ld_out)
{
    __shared__ float red[8][32];
    const int o = threadIdx.x & 31, zl = threadIdx.x >> 5;
    const int64_t i = (int64_t)blockIdx.x * 32 + o;
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    if (i < count) {
        int z = zl;
        for (; z + 24 < splits; z += 32) {
            s0 += part[(int64_t)z * count + i];
            s1 += part[(int64_t)(z + 8) * count + i];
            s2 += part[(int64_t)(z + 16) * count + i];
            s3 += part[(int64_t)(z + 24) * count + i];
        }
        for (; z < splits; z += 8) s0 += part[(int64_t)z * count + i];
    }
    red[zl][o] = (s0 + s1) + (s2 + s3);
    __syncthreads();
    if (zl == 0 && i < count) {
        float s = red[0][o];
#pragma unroll
        for (int g = 1; g < 8; ++g) s += red[g][o];
        const int64_t r = i / ncols, c = i - r * ncols;
        float *dst = out + r * ld_out + c;
        *dst = accumulate ? *dst + s : s;
    }
}

sat_status sat_splitk_reduce(sat_ctx *ctx, const float *part, int64_t count, int32_t splits, int accumulate, float *out, int32_t ncols,
                             int32_t ld_out)
{
    if (count == 0) return SAT_OK;
    k_splitk_reduce<<<(unsigned)cdiv64(count, 32), 256, 0, ctx->stream>>>(part, count, splits, accumulate, out, ncols, ld_out);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

sat_status sat_gemm_tn(sat_ctx *ctx, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B, int32_t ldb,
                       const uint32_t *mask, int32_t mask_words, float *C, int32_t ldc, float *colsum, int accumulate)
{
    if (m == 0 || n == 0) return SAT_OK;
    ProfScope prof(ctx, SATK_GEMM_TN, 4.0 * ((double)rows * (m + n) + (double)m * n), 2.0 * (double)rows * m * n);
    int64_t splits = cdiv64(rows > 0 ? rows : 1, TN_ROWS_PER_SPLIT);
    if (splits > 1024) splits = 1024;
    int64_t rows_per_split = cdiv64(cdiv64(rows > 0 ? rows : 1, splits), BK) * BK;
    splits = cdiv64(rows > 0 ? rows : 1, rows_per_split);
    const size_t bytes = (size_t)splits * ((size_t)m * n + n) * sizeof(float);
    SAT_TRY(sat_ensure(ctx, ctx->buf_splitk, bytes));
    float *part_C = (float *)ctx->buf_splitk.p;
    float *part_cs = colsum ? part_C + (size_t)splits * m * n : nullptr;
    dim3 grid((unsigned)cdiv64(m, BM), (unsigned)cdiv64(n, BN), (unsigned)splits);
    k_gemm_tn<<<grid, 256, 0, ctx->stream>>>(rows, rows_per_split, m, n, A, lda, B, ldb, mask, mask_words, part_C, part_cs);
    SAT_LAUNCHED(ctx);
    SAT_TRY(sat_splitk_reduce(ctx, part_C, (int64_t)m * n, (int32_t)splits, accumulate, C, n, ldc));
    if (colsum) SAT_TRY(sat_splitk_reduce(ctx, part_cs, n, (int32_t)splits, accumulate, colsum, n, n));
    return SAT_OK;
}

// =====================================================================================
// Weight gradient with a narrow output (n <= 64: the classifier layer), fp32 FMA with round-to-nearest.
// C = A^T B sums ~1e5 signed terms per element that cancel to a few 1e-3 of their magnitude (softmax gradients sum to
// zero); the tensor-core contraction, whose accumulation truncates, was measured at 1e-4 relative error there against
// 2e-5 for this kernel, which at this width costs about the same.
//   block (x, y): rows [x * rows_per_block, ...), columns y * 256 .. + 255 of A, two per thread; B rows are
//   staged in shared memory and broadcast; partial sums per row block, added in block order by k_splitk_reduce.
// =====================================================================================
#define TNN_STAGE 32
__device__ __forceinline__ void tnn_cp16(void *smem_dst, const void *gsrc, bool valid)
{
    // src-size 0 writes 16 zero bytes without reading the source
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc),
                 "r"(valid ? 16u : 0u)
                 : "memory");
}
// two stages of [TNN_STAGE x 256] of A and [TNN_STAGE x NT] of B, filled by cp.async while the previous stage is consumed;
// 128 threads, each owning columns t and t + 128 of the block's 256 columns of A (2 NT accumulators: two FMAs per
// broadcast shared-memory load of B)
template <int NT>
__global__ void __launch_bounds__(128)
k_gemm_tn_narrow(int64_t rows, int64_t rows_per_block, int32_t m, int32_t n, const float *__restrict__ A, int64_t lda,
                 const float *__restrict__ B, int64_t ldb, float *__restrict__ part)
{
    extern __shared__ __align__(16) float tnn_smem[];
    constexpr int STAGE_FLOATS = TNN_STAGE * 256 + TNN_STAGE * NT;
    const int32_t m0 = blockIdx.y * 256;
    const int32_t col0 = m0 + threadIdx.x, col1 = col0 + 128;
    const int32_t m4 = (m + 3) & ~3, n4 = (n + 3) & ~3;
    const int64_t r_begin = (int64_t)blockIdx.x * rows_per_block;
    const int64_t r_end = r_begin + rows_per_block < rows ? r_begin + rows_per_block : rows;
    auto load_stage = [&](int s, int64_t r0) {
        float *As = tnn_smem + s * STAGE_FLOATS, *Bs = As + TNN_STAGE * 256;
#pragma unroll
        for (int k = 0; k < TNN_STAGE * 64 / 128; ++k) {
            const int i = threadIdx.x + 128 * k, rr = i >> 6, c4 = i & 63;
            const bool ok = r0 + rr < r_end && m0 + 4 * c4 < m4;
            tnn_cp16(As + rr * 256 + 4 * c4, ok ? A + (r0 + rr) * lda + m0 + 4 * c4 : A, ok);
        }
        for (int i = threadIdx.x; i < TNN_STAGE * (NT / 4); i += 128) {
            const int rr = i / (NT / 4), j4 = i - rr * (NT / 4);
            const bool ok = r0 + rr < r_end && 4 * j4 < n4;
            tnn_cp16(Bs + rr * NT + 4 * j4, ok ? B + (r0 + rr) * ldb + 4 * j4 : B, ok);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // accumulators as pairs: the packed FMA of sm_100 (two IEEE-rounded fp32 FMAs per instruction, same results as fmaf)
    // halves the issue slots of the inner loop, which is bound by FMA issue
    float2 acc0[NT / 2], acc1[NT / 2];
#pragma unroll
    for (int j = 0; j < NT / 2; ++j) acc0[j] = acc1[j] = make_float2(0.f, 0.f);
    int s = 0;
    load_stage(0, r_begin);
    for (int64_t r0 = r_begin; r0 < r_end; r0 += TNN_STAGE, s ^= 1) {
        if (r0 + TNN_STAGE < r_end) {
            load_stage(s ^ 1, r0 + TNN_STAGE);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const float *As = tnn_smem + s * STAGE_FLOATS, *Bs = As + TNN_STAGE * 256;
#pragma unroll 2
        for (int rr = 0; rr < TNN_STAGE; ++rr) {
            const float a0 = As[rr * 256 + threadIdx.x], a1 = As[rr * 256 + 128 + threadIdx.x];
            const float2 a0p = make_float2(a0, a0), a1p = make_float2(a1, a1);
#pragma unroll
            for (int j4 = 0; j4 < NT; j4 += 4) {
                const float4 b = *reinterpret_cast<const float4 *>(Bs + rr * NT + j4);
                const float2 blo = make_float2(b.x, b.y), bhi = make_float2(b.z, b.w);
                acc0[j4 / 2] = __ffma2_rn(a0p, blo, acc0[j4 / 2]);
                acc0[j4 / 2 + 1] = __ffma2_rn(a0p, bhi, acc0[j4 / 2 + 1]);
                acc1[j4 / 2] = __ffma2_rn(a1p, blo, acc1[j4 / 2]);
                acc1[j4 / 2 + 1] = __ffma2_rn(a1p, bhi, acc1[j4 / 2 + 1]);
            }
        }
        __syncthreads();  // the stage is refilled two iterations later
    }
    if (col0 < m) {
        float *o = part + ((int64_t)blockIdx.x * m + col0) * n;
#pragma unroll
        for (int j = 0; j < NT; ++j)
            if (j < n) o[j] = (j & 1) ? acc0[j / 2].y : acc0[j / 2].x;
    }
    if (col1 < m) {
        float *o = part + ((int64_t)blockIdx.x * m + col1) * n;
#pragma unroll
        for (int j = 0; j < NT; ++j)
            if (j < n) o[j] = (j & 1) ? acc1[j / 2].y : acc1[j / 2].x;
    }
}

template <int NT>
static sat_status launch_tn_narrow(sat_ctx *ctx, dim3 grid, int64_t rows, int64_t rpb, int32_t m, int32_t n, const float *A, int32_t lda,
                                   const float *B, int32_t ldb, float *part)
{
    static PerDeviceOnce attr_set;
    const size_t smem = 2 * (size_t)(TNN_STAGE * 256 + TNN_STAGE * NT) * sizeof(float);
    if (attr_set.need(ctx->device)) {
        SAT_CUDA(ctx, cudaFuncSetAttribute(k_gemm_tn_narrow<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        attr_set.mark(ctx->device);
    }
    k_gemm_tn_narrow<NT><<<grid, 128, smem, ctx->stream>>>(rows, rpb, m, n, A, lda, B, ldb, part);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

// C[m x n] (+)= A^T B over `rows` rows for n <= 64 (B already masked)
sat_status sat_gemm_tn_narrow(sat_ctx *ctx, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B, int32_t ldb,
                              float *C, int32_t ldc, int accumulate)
{
    if (m == 0 || n == 0) return SAT_OK;
    if (n > 64 || (lda & 3) || (ldb & 3) || (((uintptr_t)A | (uintptr_t)B) & 15u))
        return sat_fail(ctx, SAT_EINVAL, "sat_gemm_tn_narrow: n must be <= 64, operands 16-byte aligned with leading dimensions in multiples of 4");
    ProfScope prof(ctx, SATK_GEMM_TN, 4.0 * ((double)rows * (m + n) + (double)m * n), 2.0 * (double)rows * m * n);
    // two CTAs fit on an SM (80 KB of shared memory each): one full wave of row blocks
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, ctx->device);
    const int64_t want = (2 * (int64_t)sms) / cdiv64(m, 256) > 0 ? (2 * (int64_t)sms) / cdiv64(m, 256) : 1;
    int64_t rpb = cdiv64(cdiv64(rows > 0 ? rows : 1, want), TNN_STAGE) * TNN_STAGE;
    if (rpb < 4 * TNN_STAGE) rpb = 4 * TNN_STAGE;
    const int64_t blocks = cdiv64(rows > 0 ? rows : 1, rpb);
    SAT_TRY(sat_ensure(ctx, ctx->buf_splitk, (size_t)blocks * m * n * sizeof(float)));
    float *part = (float *)ctx->buf_splitk.p;
    dim3 grid((unsigned)blocks, (unsigned)cdiv64(m, 256));
    if (n <= 16) SAT_TRY(launch_tn_narrow<16>(ctx, grid, rows, rpb, m, n, A, lda, B, ldb, part));
    else if (n <= 32) SAT_TRY(launch_tn_narrow<32>(ctx, grid, rows, rpb, m, n, A, lda, B, ldb, part));
    else if (n <= 48) SAT_TRY(launch_tn_narrow<48>(ctx, grid, rows, rpb, m, n, A, lda, B, ldb, part));
    else SAT_TRY(launch_tn_narrow<64>(ctx, grid, rows, rpb, m, n, A, lda, B, ldb, part));
    return sat_splitk_reduce(ctx, part, (int64_t)m * n, (int32_t)blocks, accumulate, C, n, ldc);
}

// =====================================================================================
// sat_dense_tn_static: the split weight-gradient product without any allocation
// =====================================================================================
// Some callers must not allocate device memory at all: code that runs while another component owns the whole device
// heap (a serving process that pre-reserves every byte), real-time loops where cudaMalloc's implicit device-wide
// synchronisation is not acceptable, and code running inside a region where allocation calls are forbidden.  For them the
// split partial sums of C = A^T B live in this fixed array, which is part of the library image: every GPU that loads the
// library carries it until the process exits.
#define SAT_STATIC_SCRATCH_FLOATS (2 * 1024 * 1024) /* 8 MiB */
static __device__ __align__(256) float sat_static_scratch[SAT_STATIC_SCRATCH_FLOATS];

#include <mutex>

#define SAT_STATIC_MAX_DEVICES 64
static std::mutex g_static_mutex;
static float *g_static_ptr[SAT_STATIC_MAX_DEVICES] = {nullptr};  // device address of sat_static_scratch, per device

static sat_status static_fail(char *errbuf, int32_t errbuf_len, sat_status code, const char *fmt, ...)
{
    if (errbuf && errbuf_len > 0) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(errbuf, (size_t)errbuf_len, fmt, ap);
        va_end(ap);
    }
    return code;
}

extern "C" sat_status sat_dense_tn_static(void *cuda_stream, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda,
                                          const float *B, int32_t ldb, float *C, char *errbuf, int32_t errbuf_len)
{
    if (errbuf && errbuf_len > 0) errbuf[0] = 0;
    if (rows < 0 || m <= 0 || n <= 0 || !A || !B || !C || lda < m || ldb < n)
        return static_fail(errbuf, errbuf_len, SAT_EINVAL, "sat_dense_tn_static: null tensor or bad shape (rows %lld, m %d, n %d, lda %d, ldb %d)",
                           (long long)rows, m, n, lda, ldb);
    if ((int64_t)m * n > SAT_STATIC_SCRATCH_FLOATS)
        return static_fail(errbuf, errbuf_len, SAT_EINVAL,
                           "sat_dense_tn_static: m * n = %lld exceeds the built-in scratch of %d floats (8 MiB); use sat_dense_tn",
                           (long long)m * n, SAT_STATIC_SCRATCH_FLOATS);
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= SAT_STATIC_MAX_DEVICES)
        return static_fail(errbuf, errbuf_len, SAT_ECUDA, "sat_dense_tn_static: no usable current device (%s)", cudaGetErrorString(e));
    float *scratch = nullptr;
    {
        // one-time set-up per device: `sat_static_scratch` named in host code is only a handle, the kernels need the
        // address the symbol has on the current device.  The address is kept for the life of the process, so the device's
        // primary context must not be reset (cudaDeviceReset) while this library is in use: the kept address would
        // then point into a context that no longer exists.
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[dev]) {
            float *p = nullptr;
            e = cudaGetSymbolAddress((void **)&p, sat_static_scratch);
            if (e != cudaSuccess || !p)
                return static_fail(errbuf, errbuf_len, SAT_ECUDA, "sat_dense_tn_static: cudaGetSymbolAddress failed (%s)", cudaGetErrorString(e));
            g_static_ptr[dev] = p;
        }
        scratch = g_static_ptr[dev];
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // as many row splits as the fixed array holds (each split owns an m x n block of partial sums)
    int64_t splits = cdiv64(rows > 0 ? rows : 1, TN_ROWS_PER_SPLIT);
    const int64_t cap = SAT_STATIC_SCRATCH_FLOATS / ((int64_t)m * n);
    if (splits > cap) splits = cap;
    if (splits > 1024) splits = 1024;
    int64_t rows_per_split = cdiv64(cdiv64(rows > 0 ? rows : 1, splits), BK) * BK;
    splits = cdiv64(rows > 0 ? rows : 1, rows_per_split);
    // every element of the `splits` partial blocks is written by exactly one thread block below, so nothing left over from
    // an earlier call is ever read and no clearing is needed
    dim3 grid((unsigned)cdiv64(m, BM), (unsigned)cdiv64(n, BN), (unsigned)splits);
    k_gemm_tn<<<grid, 256, 0, st>>>(rows, rows_per_split, m, n, A, lda, B, ldb, nullptr, 0, scratch, nullptr);
    e = cudaGetLastError();
    if (e != cudaSuccess) return static_fail(errbuf, errbuf_len, SAT_ECUDA, "sat_dense_tn_static: launch failed (%s)", cudaGetErrorString(e));
    k_splitk_reduce<<<(unsigned)cdiv64((int64_t)m * n, 32), 256, 0, st>>>(scratch, (int64_t)m * n, (int32_t)splits, 0, C, n, n);
    e = cudaGetLastError();
    if (e != cudaSuccess) return static_fail(errbuf, errbuf_len, SAT_ECUDA, "sat_dense_tn_static: launch failed (%s)", cudaGetErrorString(e));
    return SAT_OK;
}
