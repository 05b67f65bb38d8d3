// Lossy storage of historical embeddings (Supplement, "Data Compression for Historical Embedding Storage"): the
// encoded-polyline scheme applied to every row of an fp32 matrix.
//   q_j = round-half-away-from-zero(x_j * 10^p)   (fp64: the product of an fp32 value and 10^p, p <= 7, is exact)
//   e_0 = q_0, e_j = q_j - q_{j-1};  v = e << 1, bitwise inverted when e < 0
//   5-bit groups of v, least significant first, bit 0x20 on all but the last, each + 63 -> one byte
// One warp per row in all three kernels.  The code length of an element depends only on x_j and x_{j-1}, so sizes and
// bytes are produced element-parallel (warp prefix sums give the byte positions); decoding takes 128 bytes at a time (a
// byte below 0x20 after the -63 ends a value), lets the lane holding the last byte of a value assemble it, and turns the
// deltas into values with a 64-bit warp prefix sum.  Integer and byte work: HBM-bound.
#include "sat_internal.h"

#define CODEC_MAX_GROUPS 13  /* 64 bits / 5 */

__device__ __forceinline__ int64_t codec_quantise(float x, double scale) { return llround((double)x * scale); }
__device__ __forceinline__ uint64_t codec_fold(int64_t e)
{
    const uint64_t v = (uint64_t)e << 1;
    return e < 0 ? ~v : v;
}
__device__ __forceinline__ int codec_len(uint64_t v) { return v == 0 ? 1 : (64 - __clzll((long long)v) + 4) / 5; }

// folded delta of this lane's element against its predecessor: the predecessor's quantised value comes from the lane
// below, or, for lane 0, from the last element of the previous group of 32 (`carry`, updated here)
__device__ __forceinline__ uint64_t codec_symbol(int64_t q, int lane, int64_t &carry)
{
    const int64_t up = __shfl_up_sync(0xffffffffu, q, 1);
    const int64_t prev = lane == 0 ? carry : up;
    carry = __shfl_sync(0xffffffffu, q, 31);
    return codec_fold(q - prev);
}

__global__ void __launch_bounds__(256)
k_codec_sizes(const float *__restrict__ x, int64_t ld, int64_t rows, int32_t d, double scale, int32_t *__restrict__ row_bytes)
{
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    const float *row = x + r * ld;
    int32_t total = 0;
    int64_t carry = 0;
    for (int32_t j0 = 0; j0 < d; j0 += 32) {
        const int32_t j = j0 + lane;
        const int64_t q = j < d ? codec_quantise(row[j], scale) : 0;
        const uint64_t v = codec_symbol(q, lane, carry);
        if (j < d) total += codec_len(v);
    }
    for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(0xffffffffu, total, o);
    if (lane == 0) row_bytes[r] = total;
}

__global__ void __launch_bounds__(256)
k_codec_encode(const float *__restrict__ x, int64_t ld, int64_t rows, int32_t d, double scale, const int64_t *__restrict__ offsets,
               uint8_t *__restrict__ out)
{
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    const float *row = x + r * ld;
    int64_t run = offsets[r];
    int64_t carry = 0;
    for (int32_t j0 = 0; j0 < d; j0 += 32) {
        const int32_t j = j0 + lane;
        const int64_t q = j < d ? codec_quantise(row[j], scale) : 0;
        const uint64_t v = codec_symbol(q, lane, carry);
        const int len = j < d ? codec_len(v) : 0;
        int incl = len;
        for (int o = 1; o < 32; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        uint8_t *dst = out + run + (incl - len);
        for (int k = 0; k < len; ++k) {
            const uint32_t g = (uint32_t)(v >> (5 * k)) & 0x1fu;
            dst[k] = (uint8_t)((k + 1 < len ? 0x20u : 0u) + g + 63u);
        }
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
}

// status bit 2: a row does not hold exactly d well-formed values.
// 128 bytes per iteration, four consecutive bytes per lane.  A byte below 0x20 (after the -63) ends a value; the lane that
// holds the last byte of a value assembles it (walking back over at most 12 continuation bytes, usually its own), the
// lanes' delta sums go through one 64-bit warp prefix sum per window, and the element index of a value is the number of
// terminators before it (one 32-bit prefix sum per window).
__global__ void __launch_bounds__(256)
k_codec_decode(const uint8_t *__restrict__ in, int64_t in_bytes, const int64_t *__restrict__ offsets, int64_t rows, int32_t d, double scale,
               float *__restrict__ x, int64_t ld, int *__restrict__ status)
{
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    const int64_t b0 = offsets[r], b1 = offsets[r + 1];
    // an offset pair that does not lie inside the byte buffer is a malformed row: flagged and skipped, never dereferenced
    if (b0 < 0 || b1 > in_bytes || b1 < b0) {
        if (lane == 0) atomicOr(status, 2);
        return;
    }
    float *row = x + r * ld;
    int64_t q_run = 0;
    int32_t elem_base = 0;
    bool bad = false;
    for (int64_t pos = b0; pos < b1; pos += 128) {
        const int64_t p0 = pos + 4 * lane;
        uint32_t c[4];
        int n_term = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            c[k] = p0 + k < b1 ? (uint32_t)in[p0 + k] - 63u : 0xffu;
            if (p0 + k < b1 && c[k] > 63u) bad = true;  // outside the alphabet
            if (c[k] < 0x20u) ++n_term;
        }
        // values that end in this lane's bytes
        int64_t e[4];
        int64_t lane_sum = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            e[k] = 0;
            if (c[k] < 0x20u) {
                uint64_t v = c[k] & 0x1fu;
                int groups = 1;
                // continuation bytes before it: first this lane's own, then earlier bytes of the row
                int kk = k - 1;
                int64_t s = p0 + k;  // first byte of the value found so far
                while (groups < CODEC_MAX_GROUPS) {
                    uint32_t cc;
                    if (kk >= 0) cc = c[kk];
                    else if (s > b0) cc = (uint32_t)in[s - 1] - 63u;
                    else break;
                    if (cc < 0x20u) break;
                    v = (v << 5) | (cc & 0x1fu);
                    --kk;
                    --s;
                    ++groups;
                }
                if (groups == CODEC_MAX_GROUPS && s > b0 && (uint32_t)in[s - 1] - 63u >= 0x20u) bad = true;  // longer than 64 bits
                e[k] = (v & 1) ? ~(int64_t)(v >> 1) : (int64_t)(v >> 1);
                lane_sum += e[k];
            }
        }
        // exclusive prefixes over the lanes: element index and running quantised value
        int cnt_incl = n_term;
        int64_t sum_incl = lane_sum;
        for (int o = 1; o < 32; o <<= 1) {
            const int cu = __shfl_up_sync(0xffffffffu, cnt_incl, o);
            const int64_t su = __shfl_up_sync(0xffffffffu, sum_incl, o);
            if (lane >= o) {
                cnt_incl += cu;
                sum_incl += su;
            }
        }
        int32_t elem = elem_base + cnt_incl - n_term;
        int64_t q = q_run + sum_incl - lane_sum;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (c[k] < 0x20u) {
                q += e[k];
                if (elem < d) row[elem] = (float)((double)q / scale);
                else bad = true;
                ++elem;
            }
        }
        q_run += __shfl_sync(0xffffffffu, sum_incl, 31);
        elem_base += __shfl_sync(0xffffffffu, cnt_incl, 31);
    }
    // the last byte of the row must end a value, and the row must hold exactly d values
    if (lane == 0 && b1 > b0 && (uint32_t)in[b1 - 1] - 63u >= 0x20u) bad = true;
    if (elem_base != d) bad = true;
    if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, 2);
}

static double codec_scale(int32_t precision)
{
    double s = 1.0;
    for (int32_t i = 0; i < precision; ++i) s *= 10.0;
    return s;
}

static sat_status codec_check(sat_ctx *ctx, const char *who, const void *x, int32_t ld, int64_t rows, int32_t d, int32_t precision)
{
    if (rows < 0 || d <= 0 || ld < d || precision < 0 || precision > 7 || (rows > 0 && !x))
        return sat_fail(ctx, SAT_EINVAL, "%s: null tensor, bad shape or precision outside 0..7", who);
    return SAT_OK;
}

static sat_status codec_plan(sat_ctx *ctx, const float *x, int32_t ld, int64_t rows, int32_t d, int32_t precision, int64_t *row_offsets,
                             int64_t *total_bytes)
{
    SAT_TRY(sat_ensure(ctx, ctx->buf_codec_sizes, (size_t)(rows > 0 ? rows : 1) * sizeof(int32_t)));
    int32_t *sizes = (int32_t *)ctx->buf_codec_sizes.p;
    if (rows > 0) {
        ProfScope prof(ctx, SATK_CODEC, 4.0 * (double)rows * d + 12.0 * (double)rows, 0.0);
        k_codec_sizes<<<(unsigned)cdiv64(rows * 32, 256), 256, 0, ctx->stream>>>(x, ld, rows, d, codec_scale(precision), sizes);
        SAT_LAUNCHED(ctx);
    }
    SAT_TRY(sat_scan_i32(ctx, sizes, rows, row_offsets));
    if (total_bytes) {
        SAT_CUDA(ctx, cudaMemcpyAsync(total_bytes, row_offsets + rows, sizeof(int64_t), cudaMemcpyDeviceToHost, ctx->stream));
        SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    }
    return SAT_OK;
}

extern "C" sat_status sat_codec_plan(sat_ctx *ctx, const float *x, int32_t ld, int64_t rows, int32_t d, int32_t precision,
                                     int64_t *row_offsets, int64_t *total_bytes)
{
    CHECK_CTX(ctx);
    SAT_TRY(codec_check(ctx, "sat_codec_plan", x, ld, rows, d, precision));
    if (!row_offsets || !total_bytes) return sat_fail(ctx, SAT_EINVAL, "sat_codec_plan: null row_offsets / total_bytes");
    return codec_plan(ctx, x, ld, rows, d, precision, row_offsets, total_bytes);
}

static sat_status codec_encode(sat_ctx *ctx, const float *x, int32_t ld, int64_t rows, int32_t d, int32_t precision,
                               const int64_t *row_offsets, uint8_t *out, int64_t total)
{
    if (rows == 0) return SAT_OK;
    ProfScope prof(ctx, SATK_CODEC, 4.0 * (double)rows * d + 8.0 * (double)rows + (double)total, 0.0);
    k_codec_encode<<<(unsigned)cdiv64(rows * 32, 256), 256, 0, ctx->stream>>>(x, ld, rows, d, codec_scale(precision), row_offsets, out);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

extern "C" sat_status sat_codec_encode(sat_ctx *ctx, const float *x, int32_t ld, int64_t rows, int32_t d, int32_t precision,
                                       const int64_t *row_offsets, uint8_t *out, int64_t out_capacity)
{
    CHECK_CTX(ctx);
    SAT_TRY(codec_check(ctx, "sat_codec_encode", x, ld, rows, d, precision));
    if (!row_offsets || out_capacity < 0 || (rows > 0 && !out)) return sat_fail(ctx, SAT_EINVAL, "sat_codec_encode: null row_offsets / out");
    int64_t total = 0;
    SAT_CUDA(ctx, cudaMemcpyAsync(&total, row_offsets + rows, sizeof(int64_t), cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (total > out_capacity)
        return sat_fail(ctx, SAT_EINVAL, "sat_codec_encode: the rows need %lld bytes, the output holds %lld", (long long)total, (long long)out_capacity);
    return codec_encode(ctx, x, ld, rows, d, precision, row_offsets, out, total);
}

static sat_status codec_decode(sat_ctx *ctx, const uint8_t *in, int64_t in_bytes, const int64_t *row_offsets, int64_t rows, int32_t d,
                               int32_t precision, float *x, int32_t ld)
{
    if (rows == 0) return SAT_OK;
    ProfScope prof(ctx, SATK_CODEC, 4.0 * (double)rows * d + 8.0 * (double)rows + (double)in_bytes, 0.0);
    k_codec_decode<<<(unsigned)cdiv64(rows * 32, 256), 256, 0, ctx->stream>>>(in, in_bytes, row_offsets, rows, d, codec_scale(precision), x, ld,
                                                                             ctx->d_flag + 1);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

extern "C" sat_status sat_codec_decode(sat_ctx *ctx, const uint8_t *in, int64_t in_bytes, const int64_t *row_offsets, int64_t rows, int32_t d,
                                       int32_t precision, float *x, int32_t ld)
{
    CHECK_CTX(ctx);
    SAT_TRY(codec_check(ctx, "sat_codec_decode", x, ld, rows, d, precision));
    if (!row_offsets || in_bytes < 0 || (rows > 0 && in_bytes > 0 && !in)) return sat_fail(ctx, SAT_EINVAL, "sat_codec_decode: null row_offsets / in, or negative in_bytes");
    return codec_decode(ctx, in, in_bytes, row_offsets, rows, d, precision, x, ld);
}

// encode + decode of one matrix in place through context scratch (what a compressed ring would hand back)
sat_status sat_codec_roundtrip(sat_ctx *ctx, float *x, int32_t ld, int64_t rows, int32_t d, int32_t precision, int64_t *bytes)
{
    SAT_TRY(sat_ensure(ctx, ctx->buf_codec_off, (size_t)(rows + 1) * sizeof(int64_t)));
    int64_t *offsets = (int64_t *)ctx->buf_codec_off.p;
    int64_t total = 0;
    SAT_TRY(codec_plan(ctx, x, ld, rows, d, precision, offsets, &total));
    SAT_TRY(sat_ensure(ctx, ctx->buf_codec_bytes, (size_t)(total > 0 ? total : 1)));
    uint8_t *data = (uint8_t *)ctx->buf_codec_bytes.p;
    SAT_TRY(codec_encode(ctx, x, ld, rows, d, precision, offsets, data, total));
    SAT_TRY(codec_decode(ctx, data, total, offsets, rows, d, precision, x, ld));
    if (bytes) *bytes = total;
    return SAT_OK;
}
