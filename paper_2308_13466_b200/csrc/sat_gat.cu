// Graph-attention layer as the local layer of a partition (the paper also evaluates SAT with a GAT backbone; the layer
// itself is the standard single-head graph attention layer).  For inner node v, over the entries u of its local CSR row
// (neighbours inside the partition, v itself, neighbours outside = halo rows with cached / predicted embeddings):
//     z_u = h_u W;  e_vu = LeakyReLU_0.2(a_dst . z_v + a_src . z_u);  alpha_vu = softmax_u(e_vu);
//     o_v = sum_u alpha_vu z_u + bias;  h'_v = ReLU(o_v) or o_v.
// Backward with the halo embeddings constant (their z still depends on W):
//     D = g o [o > 0];  dalpha_vu = D_v . z_u;  t_v = sum_u alpha_vu dalpha_vu;
//     dpre_vu = alpha_vu (dalpha_vu - t_v) LeakyReLU'(pre_vu);  ds_dst[v] = sum_u dpre_vu;  ds_src[u] = sum_v dpre_vu;
//     dZ_u = sum_v alpha_vu D_v + ds_src[u] a_src (+ ds_dst[u] a_dst for inner u);
//     G_W = H^T dZ over inner and halo rows;  G_a_src = Z^T ds_src;  G_a_dst = Z_in^T ds_dst;  G_b = 1^T D;  G_in = dZ_in W^T.
// The sums over v for a fixed u run over the inner prefix of u's own row (the inner block is symmetric) or over the
// halo-row CSR; alpha_vu is recomputed from the per-row scalars (s_dst[v], log-sum-exp of row v), so no per-edge array
// is stored.  One warp per work item of the SpMM (a row, or a 256-entry chunk of a long row), per-item partial sums added in
// item order by small combine kernels: every sum has a single writer and a fixed order.  The halo-node side of the backward
// still walks a halo row with one warp.
#include "sat_internal.h"

#define GAT_SLOPE 0.2f
#define GAT_MAX_NV 8   /* float4 per lane: widths up to 1024 */


__device__ __forceinline__ float warp_sum(float x)
{
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
__device__ __forceinline__ float warp_max(float x)
{
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float4 ldz(const float *row, int c4, int d)
{
    // the padding columns of the last vector of a row are not data: read them as zero
    float4 x = *reinterpret_cast<const float4 *>(row + 4 * c4);
    if (4 * c4 + 3 >= d) {
        if (4 * c4 + 1 >= d) x.y = 0.f;
        if (4 * c4 + 2 >= d) x.z = 0.f;
        x.w = 0.f;
    }
    return x;
}
__device__ __forceinline__ float dot4(const float4 &a, const float4 &b) { return fmaf(a.x, b.x, fmaf(a.y, b.y, fmaf(a.z, b.z, a.w * b.w))); }
__device__ __forceinline__ float lrelu(float x) { return x > 0.f ? x : GAT_SLOPE * x; }
// D_v . z_u feeds differences (dalpha - t_v) that cancel most of their size: the products are summed in double
__device__ __forceinline__ double ddot4(const float4 &a, const float4 &b)
{
    return (double)a.x * (double)b.x + (double)a.y * (double)b.y + (double)a.z * (double)b.z + (double)a.w * (double)b.w;
}
__device__ __forceinline__ double warp_sum_d(double x)
{
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// s_src[r] = a_src . z_r, s_dst[r] = a_dst . z_r (when asked for); one warp per row
__global__ void __launch_bounds__(256)
k_gat_scores(const float *__restrict__ z, int64_t ld, int64_t rows, int32_t d, const float *__restrict__ a_src, const float *__restrict__ a_dst,
             float *__restrict__ s_src, float *__restrict__ s_dst)
{
    const int64_t r = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (r >= rows) return;
    float ps = 0.f, pd = 0.f;
    for (int c = lane; c < d; c += 32) {
        const float x = z[r * ld + c];
        ps = fmaf(x, a_src[c], ps);
        if (a_dst) pd = fmaf(x, a_dst[c], pd);
    }
    ps = warp_sum(ps);
    pd = warp_sum(pd);
    if (lane == 0) {
        s_src[r] = ps;
        if (a_dst) s_dst[r] = pd;
    }
}

// forward over work items: k_gat_lse (a warp per row, lanes over the entries) gives the log-sum-exp of every row; then one warp
// per item accumulates its chunk of the weighted sum.  Rows of a single item are finished here (bias, ReLU); items of
// longer rows write their partial sum to `partial` (row index item_mslot) and k_gat_fwd_fixup adds them in item order.
__global__ void __launch_bounds__(256)
k_gat_lse(const int64_t *__restrict__ lrowptr, const int32_t *__restrict__ lenc, int32_t n, int32_t row0, int32_t n_rows,
          const float *__restrict__ s_in, const float *__restrict__ s_halo, const float *__restrict__ s_dst, float *__restrict__ lse)
{
    const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n_rows) return;
    const int32_t row = row0 + (int32_t)w;
    const int64_t e0 = lrowptr[row], e1 = lrowptr[row + 1];
    const float sd = s_dst[row];
    float mx = -INFINITY;
    for (int64_t e = e0 + lane; e < e1; e += 32) {
        const int32_t c = lenc[e];
        mx = fmaxf(mx, lrelu(sd + (c < n ? s_in[c] : s_halo[c - n])));
    }
    mx = warp_max(mx);
    float den = 0.f;
    for (int64_t e = e0 + lane; e < e1; e += 32) {
        const int32_t c = lenc[e];
        den += expf(lrelu(sd + (c < n ? s_in[c] : s_halo[c - n])) - mx);
    }
    den = warp_sum(den);
    if (lane == 0) lse[row] = mx + logf(den);
}

template <int NV>
__global__ void __launch_bounds__(256)
k_gat_fwd_items(const int64_t *__restrict__ lrowptr, const int32_t *__restrict__ lenc, const int32_t *__restrict__ item_row,
                const int32_t *__restrict__ first_item, const int32_t *__restrict__ item_mslot, int32_t item0, int32_t n_items, int32_t mitem0,
                int32_t n, const float *__restrict__ z_in, const float *__restrict__ z_halo, int64_t ld_z, const float *__restrict__ s_in,
                const float *__restrict__ s_halo, const float *__restrict__ s_dst, const float *__restrict__ lse, int32_t d,
                const float *__restrict__ bias, int relu, float *__restrict__ out_base, int64_t ld_out, float *__restrict__ partial)
{
    const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n_items) return;
    const int32_t item = item0 + (int32_t)w;
    const int32_t row = item_row[item];
    const int64_t re = lrowptr[row + 1];
    const int64_t e0 = lrowptr[row] + (int64_t)(item - first_item[row]) * SAT_SPMM_CHUNK;
    const int64_t e1 = e0 + SAT_SPMM_CHUNK < re ? e0 + SAT_SPMM_CHUNK : re;
    const float sd = s_dst[row], l = lse[row];
    const int d4 = (d + 3) >> 2;
    float4 acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t eb = e0; eb < e1; eb += 32) {
        const int64_t e = eb + lane;
        int32_t c = 0;
        float a = 0.f;
        if (e < e1) {
            c = lenc[e];
            a = expf(lrelu(sd + (c < n ? s_in[c] : s_halo[c - n])) - l);
        }
        const int cnt = (e1 - eb) < 32 ? (int)(e1 - eb) : 32;
#pragma unroll 4
        for (int j = 0; j < cnt; ++j) {
            const int32_t cj = __shfl_sync(0xffffffffu, c, j);
            const float aj = __shfl_sync(0xffffffffu, a, j);
            const float *src = cj < n ? z_in + (int64_t)cj * ld_z : z_halo + (int64_t)(cj - n) * ld_z;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int c4 = lane + 32 * v;
                if (c4 < d4) {
                    const float4 x = *reinterpret_cast<const float4 *>(src + 4 * c4);
                    acc[v].x = fmaf(aj, x.x, acc[v].x);
                    acc[v].y = fmaf(aj, x.y, acc[v].y);
                    acc[v].z = fmaf(aj, x.z, acc[v].z);
                    acc[v].w = fmaf(aj, x.w, acc[v].w);
                }
            }
        }
    }
    const int32_t ms = item_mslot[item];
    if (ms >= 0) {
        float *o = partial + (int64_t)(ms - mitem0) * ld_z;
#pragma unroll
        for (int v = 0; v < NV; ++v) {
            const int c4 = lane + 32 * v;
            if (c4 < d4) *reinterpret_cast<float4 *>(o + 4 * c4) = acc[v];
        }
        return;
    }
    float *o = out_base + (int64_t)row * ld_out;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int c4 = lane + 32 * v;
        if (c4 < d4) {
            float4 r = acc[v];
            const int c = 4 * c4;
            if (bias) {
                r.x += bias[c];
                if (c + 1 < d) r.y += bias[c + 1];
                if (c + 2 < d) r.z += bias[c + 2];
                if (c + 3 < d) r.w += bias[c + 3];
            }
            if (relu) {
                r.x = fmaxf(r.x, 0.f);
                r.y = fmaxf(r.y, 0.f);
                r.z = fmaxf(r.z, 0.f);
                r.w = fmaxf(r.w, 0.f);
            }
            *reinterpret_cast<float4 *>(o + 4 * c4) = r;
        }
    }
}

// rows cut into several items: add the partial sums in item order, then bias and activation
__global__ void k_gat_fwd_fixup(const int32_t *__restrict__ mrows, int32_t mrow0, int32_t n_mrows, const int32_t *__restrict__ first_item,
                                const int32_t *__restrict__ item_mslot, int32_t mitem0, int32_t d, const float *__restrict__ partial, int64_t ld_z,
                                const float *__restrict__ bias, int relu, float *__restrict__ out_base, int64_t ld_out)
{
    const int d4 = (d + 3) >> 2;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d4;
    const int c4 = (int)(t - i * d4);
    if (i >= n_mrows) return;
    const int32_t row = mrows[mrow0 + i];
    const int32_t it0 = first_item[row], it1 = first_item[row + 1];
    const int32_t ms0 = item_mslot[it0] - mitem0;
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int32_t q = 0; q < it1 - it0; ++q) {
        const float4 x = *reinterpret_cast<const float4 *>(partial + (int64_t)(ms0 + q) * ld_z + 4 * c4);
        r.x += x.x;
        r.y += x.y;
        r.z += x.z;
        r.w += x.w;
    }
    const int c = 4 * c4;
    if (bias) {
        r.x += bias[c];
        if (c + 1 < d) r.y += bias[c + 1];
        if (c + 2 < d) r.z += bias[c + 2];
        if (c + 3 < d) r.w += bias[c + 3];
    }
    if (relu) {
        r.x = fmaxf(r.x, 0.f);
        r.y = fmaxf(r.y, 0.f);
        r.z = fmaxf(r.z, 0.f);
        r.w = fmaxf(r.w, 0.f);
    }
    *reinterpret_cast<float4 *>(out_base + (int64_t)row * ld_out + 4 * c4) = r;
}

// D = g o [h_out > 0] (ReLU layer) or g
__global__ void k_gat_dmask(const float *__restrict__ g, int64_t ld_g, const float *__restrict__ h_out, int64_t ld_h, int64_t rows, int32_t d,
                            float *__restrict__ D, int64_t ld_d)
{
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t r = t / d;
    const int c = (int)(t - r * d);
    if (r >= rows) return;
    const float x = g[r * ld_g + c];
    D[r * ld_d + c] = (!h_out || h_out[r * ld_h + c] > 0.f) ? x : 0.f;
}

// Column-side walk shared by the three kernels below: entries e_first, e_first + stride, ... (< e_end) of an index list of
// rows v that hold node u.  The lanes fetch the row scalars of 32 entries at a time — one exponential per entry instead of
// one per lane and entry — and then walk those entries together, lanes over the columns, four rows in flight.
//   acc += alpha_vu D_v,   returns sum_v alpha_vu slope_vu (D_v . z_u - t_v), the same on every lane
// ds_src is linear in the dot products, so every lane keeps its own share and the warp is reduced once at the end (the
// first version reduced every dot product across the warp: ten dependent shuffles per entry).
template <int NV>
__device__ __forceinline__ double gat_cols_walk(const int32_t *__restrict__ idx, int64_t e_first, int64_t e_end, int64_t stride, float su,
                                                const float *__restrict__ s_dst, const float *__restrict__ lse, const double *__restrict__ t_in,
                                                const float *__restrict__ D, int64_t ld_d, int32_t d, int d4, int lane, const float4 (&zu)[NV],
                                                float4 (&acc)[NV])
{
    double dss = 0.0, tss = 0.0;
    for (int64_t eb = e_first; eb < e_end; eb += 32 * stride) {
        const int64_t e = eb + lane * stride;
        int32_t v_row = 0;
        float al = 0.f, as = 0.f;
        if (e < e_end) {
            v_row = idx[e];
            const float pre = s_dst[v_row] + su;
            al = expf(lrelu(pre) - lse[v_row]);
            as = al * (pre > 0.f ? 1.f : GAT_SLOPE);
            tss += (double)as * t_in[v_row];
        }
        const int64_t left = (e_end - eb + stride - 1) / stride;
        const int cnt = left < 32 ? (int)left : 32;
#pragma unroll 4
        for (int j = 0; j < cnt; ++j) {
            const int32_t vj = __shfl_sync(0xffffffffu, v_row, j);
            const float aj = __shfl_sync(0xffffffffu, al, j);
            const float asj = __shfl_sync(0xffffffffu, as, j);
            const float *dr = D + (int64_t)vj * ld_d;
            double p = 0.0;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int c4 = lane + 32 * v;
                if (c4 < d4) {
                    const float4 x = ldz(dr, c4, d);
                    p += ddot4(x, zu[v]);
                    acc[v].x = fmaf(aj, x.x, acc[v].x);
                    acc[v].y = fmaf(aj, x.y, acc[v].y);
                    acc[v].z = fmaf(aj, x.z, acc[v].z);
                    acc[v].w = fmaf(aj, x.w, acc[v].w);
                }
            }
            dss += (double)asj * p;
        }
    }
    return warp_sum_d(dss) - warp_sum_d(tss);
}

// backward, column side: one warp per node u keeps z_u in registers and walks the rows v that have u as an entry:
//   HALO = 0: u is inner row `row0 + w`, the v are the inner prefix of its own row (symmetric block, self entry included);
//   HALO = 1: u is halo position `halo0 + w`, the v are its halo-row CSR entries.
//   dZ_u = sum_v alpha_vu D_v + ds_src[u] a_src (+ ds_dst[u] a_dst),  ds_src[u] = sum_v alpha_vu (D_v . z_u - t_v) slope_vu
template <int NV, int HALO>
__global__ void __launch_bounds__(256)
k_gat_bwd_cols(const int64_t *__restrict__ ptr, const int32_t *__restrict__ idx, const int32_t *__restrict__ inner_cnt, int64_t u0, int64_t n_u,
               const float *__restrict__ z_u_base, int64_t ld_z, const float *__restrict__ s_u, const float *__restrict__ s_dst,
               const float *__restrict__ lse, const double *__restrict__ t_in, const float *__restrict__ ds_dst, int32_t d,
               const float *__restrict__ D, int64_t ld_d, const float *__restrict__ a_src, const float *__restrict__ a_dst,
               float *__restrict__ dz_base, float *__restrict__ ds_src)
{
    const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n_u) return;
    const int64_t u = u0 + w;
    const int d4 = (d + 3) >> 2;
    float4 zu[NV], acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int c4 = lane + 32 * v;
        zu[v] = c4 < d4 ? ldz(z_u_base + u * ld_z, c4, d) : make_float4(0.f, 0.f, 0.f, 0.f);
        acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const int64_t e0 = ptr[u], e1 = HALO ? ptr[u + 1] : e0 + inner_cnt[u];
    if (HALO && e1 - e0 > SAT_HROW_LONG) return;   // long halo rows: k_gat_bwd_cols_long, a thread block each
    const float su = s_u[u];
    const double dss = gat_cols_walk<NV>(idx, e0, e1, 1, su, s_dst, lse, t_in, D, ld_d, d, d4, lane, zu, acc);
    const float dsd = HALO ? 0.f : ds_dst[u];
    const float dssf = (float)dss;
    float *o = dz_base + u * ld_z;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int c4 = lane + 32 * v;
        if (c4 < d4) {
            const int c = 4 * c4;
            float4 r = acc[v];
            r.x += dssf * a_src[c] + (HALO ? 0.f : dsd * a_dst[c]);
            if (c + 1 < d) r.y += dssf * a_src[c + 1] + (HALO ? 0.f : dsd * a_dst[c + 1]);
            if (c + 2 < d) r.z += dssf * a_src[c + 2] + (HALO ? 0.f : dsd * a_dst[c + 2]);
            if (c + 3 < d) r.w += dssf * a_src[c + 3] + (HALO ? 0.f : dsd * a_dst[c + 3]);
            if (c + 1 >= d) r.y = 0.f;
            if (c + 2 >= d) r.z = 0.f;
            if (c + 3 >= d) r.w = 0.f;
            *reinterpret_cast<float4 *>(o + 4 * c4) = r;
        }
    }
    if (lane == 0) ds_src[u] = dssf;
}

// -------------------------------------------------------------------------------------
// The same two sweeps over the SpMM's work items (rows cut into chunks of SAT_SPMM_CHUNK entries), one warp per item, so
// that a hub row is walked by many warps; the per-item partial sums are added per row in item order by the combine kernels.
// -------------------------------------------------------------------------------------
template <int NV>
__global__ void __launch_bounds__(256)
k_gat_bwd_rows_items(const int64_t *__restrict__ lrowptr, const int32_t *__restrict__ lenc, const int32_t *__restrict__ item_row,
                     const int32_t *__restrict__ first_item, int32_t item0, int32_t n_items, int32_t n, const float *__restrict__ z_in,
                     const float *__restrict__ z_halo, int64_t ld_z, const float *__restrict__ s_in, const float *__restrict__ s_halo,
                     const float *__restrict__ s_dst, const float *__restrict__ lse, int32_t d, const float *__restrict__ D, int64_t ld_d,
                     double *__restrict__ part4)
{
    const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n_items) return;
    const int32_t item = item0 + (int32_t)w;
    const int32_t row = item_row[item];
    const int d4 = (d + 3) >> 2;
    float4 dv[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int c4 = lane + 32 * v;
        dv[v] = c4 < d4 ? ldz(D + (int64_t)row * ld_d, c4, d) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const int64_t re = lrowptr[row + 1];
    const int64_t e0 = lrowptr[row] + (int64_t)(item - first_item[row]) * SAT_SPMM_CHUNK;
    const int64_t e1 = e0 + SAT_SPMM_CHUNK < re ? e0 + SAT_SPMM_CHUNK : re;
    const float sd = s_dst[row], l = lse[row];
    // the lanes fetch the scalars of 32 entries at a time (one exponential per entry), then the warp walks those entries
    // together; t_v and ds_dst are linear in the dot products D_v . z_u, so the lanes keep their shares and the warp is reduced
    // once per item
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    for (int64_t eb = e0; eb < e1; eb += 32) {
        const int64_t e = eb + lane;
        int32_t c = 0;
        float al = 0.f, as = 0.f;
        if (e < e1) {
            c = lenc[e];
            const float pre = sd + (c < n ? s_in[c] : s_halo[c - n]);
            const float slope = pre > 0.f ? 1.f : GAT_SLOPE;
            al = expf(lrelu(pre) - l);
            as = al * slope;
            a0 += (double)al;
            a3 += (double)al * (double)slope;
        }
        const int cnt = (e1 - eb) < 32 ? (int)(e1 - eb) : 32;
#pragma unroll 4
        for (int j = 0; j < cnt; ++j) {
            const int32_t cj = __shfl_sync(0xffffffffu, c, j);
            const float aj = __shfl_sync(0xffffffffu, al, j);
            const float asj = __shfl_sync(0xffffffffu, as, j);
            const float *src = cj < n ? z_in + (int64_t)cj * ld_z : z_halo + (int64_t)(cj - n) * ld_z;
            double p = 0.0;
#pragma unroll
            for (int v = 0; v < NV; ++v) {
                const int c4 = lane + 32 * v;
                if (c4 < d4) p += ddot4(dv[v], ldz(src, c4, d));
            }
            a1 += (double)aj * p;
            a2 += (double)asj * p;
        }
    }
    a0 = warp_sum_d(a0);
    a1 = warp_sum_d(a1);
    a2 = warp_sum_d(a2);
    a3 = warp_sum_d(a3);
    if (lane == 0) {
        double *o = part4 + 4 * w;
        o[0] = a0;
        o[1] = a1;
        o[2] = a2;
        o[3] = a3;
    }
}

__global__ void k_gat_rows_combine(const int32_t *__restrict__ first_item, int32_t item0, int32_t row0, int32_t n_rows,
                                   const double *__restrict__ part4, double *__restrict__ t_out, float *__restrict__ ds_dst)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_rows) return;
    const int32_t row = row0 + (int32_t)i;
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    for (int32_t it = first_item[row]; it < first_item[row + 1]; ++it) {
        const double *p = part4 + 4 * (int64_t)(it - item0);
        a0 += p[0];
        a1 += p[1];
        a2 += p[2];
        a3 += p[3];
    }
    t_out[row] = a1 / a0;
    ds_dst[row] = (float)(a2 / a0 - (a1 / a0) * (a3 / a0));
}

// column side for the inner nodes: the item's entries that lie in the inner prefix of the row of u
template <int NV>
__global__ void __launch_bounds__(256)
k_gat_bwd_cols_items(const int64_t *__restrict__ lrowptr, const int32_t *__restrict__ lenc, const int32_t *__restrict__ inner_cnt,
                     const int32_t *__restrict__ item_row, const int32_t *__restrict__ first_item, int32_t item0, int32_t n_items,
                     const float *__restrict__ z_in, int64_t ld_z, const float *__restrict__ s_in, const float *__restrict__ s_dst,
                     const float *__restrict__ lse, const double *__restrict__ t_in, int32_t d, const float *__restrict__ D, int64_t ld_d,
                     float *__restrict__ pdz, double *__restrict__ pdss)
{
    const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n_items) return;
    const int32_t item = item0 + (int32_t)w;
    const int32_t u = item_row[item];
    const int d4 = (d + 3) >> 2;
    float4 zu[NV], acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int c4 = lane + 32 * v;
        zu[v] = c4 < d4 ? ldz(z_in + (int64_t)u * ld_z, c4, d) : make_float4(0.f, 0.f, 0.f, 0.f);
        acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const int64_t rb = lrowptr[u], re = rb + inner_cnt[u];
    const int64_t e0 = rb + (int64_t)(item - first_item[u]) * SAT_SPMM_CHUNK;
    const int64_t e1 = e0 + SAT_SPMM_CHUNK < re ? e0 + SAT_SPMM_CHUNK : re;
    const float su = s_in[u];
    const double dss = gat_cols_walk<NV>(lenc, e0, e1, 1, su, s_dst, lse, t_in, D, ld_d, d, d4, lane, zu, acc);
    float *o = pdz + w * ld_z;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int c4 = lane + 32 * v;
        if (c4 < d4) *reinterpret_cast<float4 *>(o + 4 * c4) = acc[v];
    }
    if (lane == 0) pdss[w] = dss;
}

// dZ_u = sum of the item partials in item order + ds_src[u] a_src + ds_dst[u] a_dst; one thread per (row, float4 column)
__global__ void k_gat_cols_combine(const int32_t *__restrict__ first_item, int32_t item0, int32_t row0, int32_t n_rows, int32_t d,
                                   const float *__restrict__ pdz, int64_t ld_z, const double *__restrict__ pdss, const float *__restrict__ ds_dst,
                                   const float *__restrict__ a_src, const float *__restrict__ a_dst, float *__restrict__ dz_base,
                                   float *__restrict__ ds_src)
{
    const int d4 = (d + 3) >> 2;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / d4;
    const int c4 = (int)(t - i * d4);
    if (i >= n_rows) return;
    const int32_t u = row0 + (int32_t)i;
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    double dss = 0.0;
    for (int32_t it = first_item[u]; it < first_item[u + 1]; ++it) {
        const float4 x = *reinterpret_cast<const float4 *>(pdz + (int64_t)(it - item0) * ld_z + 4 * c4);
        r.x += x.x;
        r.y += x.y;
        r.z += x.z;
        r.w += x.w;
        dss += pdss[it - item0];
    }
    const float s1 = (float)dss, s2 = ds_dst[u];
    const int c = 4 * c4;
    r.x += s1 * a_src[c] + s2 * a_dst[c];
    r.y = c + 1 < d ? r.y + s1 * a_src[c + 1] + s2 * a_dst[c + 1] : 0.f;
    r.z = c + 2 < d ? r.z + s1 * a_src[c + 2] + s2 * a_dst[c + 2] : 0.f;
    r.w = c + 3 < d ? r.w + s1 * a_src[c + 3] + s2 * a_dst[c + 3] : 0.f;
    *reinterpret_cast<float4 *>(dz_base + (int64_t)u * ld_z + 4 * c4) = r;
    if (c4 == 0) ds_src[u] = s1;
}

// column side for the halo rows with more than SAT_HROW_LONG entries (hub nodes seen from another partition): one thread
// block per row, its 8 warps taking the entries round-robin; the warps' partial sums are added in warp order.
template <int NV>
__global__ void __launch_bounds__(256)
k_gat_bwd_cols_long(const int32_t *__restrict__ hlong, int32_t hlong0, const int64_t *__restrict__ ptr, const int32_t *__restrict__ idx,
                    const float *__restrict__ z_halo, int64_t ld_z, const float *__restrict__ s_halo, const float *__restrict__ s_dst,
                    const float *__restrict__ lse, const double *__restrict__ t_in, int32_t d, const float *__restrict__ D, int64_t ld_d,
                    const float *__restrict__ a_src, float *__restrict__ dz_base, float *__restrict__ ds_src)
{
    __shared__ float4 red[8][NV][32];
    __shared__ double red_s[8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t u = hlong[hlong0 + blockIdx.x];
    const int d4 = (d + 3) >> 2;
    float4 zu[NV], acc[NV];
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int c4 = lane + 32 * v;
        zu[v] = c4 < d4 ? ldz(z_halo + u * ld_z, c4, d) : make_float4(0.f, 0.f, 0.f, 0.f);
        acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const int64_t e0 = ptr[u], e1 = ptr[u + 1];
    const float su = s_halo[u];
    const double dss = gat_cols_walk<NV>(idx, e0 + warp, e1, 8, su, s_dst, lse, t_in, D, ld_d, d, d4, lane, zu, acc);
#pragma unroll
    for (int v = 0; v < NV; ++v) red[warp][v][lane] = acc[v];
    if (lane == 0) red_s[warp] = dss;
    __syncthreads();
    if (warp != 0) return;
    double tot = 0.0;
    for (int q = 0; q < 8; ++q) tot += red_s[q];
    const float s1 = (float)tot;
    float *o = dz_base + u * ld_z;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int c4 = lane + 32 * v;
        if (c4 < d4) {
            float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int q = 0; q < 8; ++q) {
                const float4 x = red[q][v][lane];
                r.x += x.x;
                r.y += x.y;
                r.z += x.z;
                r.w += x.w;
            }
            const int c = 4 * c4;
            r.x += s1 * a_src[c];
            r.y = c + 1 < d ? r.y + s1 * a_src[c + 1] : 0.f;
            r.z = c + 2 < d ? r.z + s1 * a_src[c + 2] : 0.f;
            r.w = c + 3 < d ? r.w + s1 * a_src[c + 3] : 0.f;
            *reinterpret_cast<float4 *>(o + 4 * c4) = r;
        }
    }
    if (lane == 0) ds_src[u] = s1;
}

// part[b][c] = sum over the rows r of block b, in order, of w[r] x[r][c]
#define GAT_WSUM_ROWS 256
__global__ void __launch_bounds__(256)
k_gat_wcolsum(const float *__restrict__ x, int64_t ld, int64_t rows, int32_t d, const float *__restrict__ wgt, float *__restrict__ part)
{
    const int64_t r0 = (int64_t)blockIdx.x * GAT_WSUM_ROWS;
    const int64_t r1 = r0 + GAT_WSUM_ROWS < rows ? r0 + GAT_WSUM_ROWS : rows;
    for (int c = threadIdx.x; c < d; c += 256) {
        float s = 0.f;
        for (int64_t r = r0; r < r1; ++r) s = fmaf(wgt[r], x[r * ld + c], s);
        part[(int64_t)blockIdx.x * d + c] = s;
    }
}

// -------------------------------------------------------------------------------------
// host side
// -------------------------------------------------------------------------------------
static sat_status gat_nn(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const float *W, float *C, int32_t ldc)
{
    if (m == 0) return SAT_OK;
    if (sat_use_tc(n, k)) {
        TcWeights Wp;
        SAT_TRY(sat_tc_weights(ctx, W, n, k, nullptr, 0, 0, n, 1, ctx->buf_wsplit, &Wp));
        TcEpilogueHost eh;
        eh.C = C;
        eh.ldc = ldc;
        return sat_gemm_tc(ctx, m, n, A, lda, k, nullptr, 0, 0, Wp, eh, SATK_GEMM_NN);
    }
    GemmEpilogue ep;
    return sat_gemm_nn(ctx, m, n, k, A, lda, W, n, C, ldc, ep);
}

static sat_status gat_nt(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const float *W, float *C, int32_t ldc)
{
    if (m == 0) return SAT_OK;
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

static sat_status gat_tn(sat_ctx *ctx, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B, int32_t ldb, float *C,
                         int accumulate)
{
    if (rows == 0) {
        if (!accumulate) SAT_CUDA(ctx, cudaMemsetAsync(C, 0, (size_t)m * n * sizeof(float), ctx->stream));
        return SAT_OK;
    }
    if (sat_use_tc(n, m) && rows >= 256) {
        if (n <= 64) return sat_gemm_tn_narrow(ctx, rows, m, n, A, lda, B, ldb, C, n, accumulate);
        return sat_gemm_tc_tn(ctx, rows, m, n, A, lda, B, ldb, C, n, accumulate);
    }
    return sat_gemm_tn(ctx, rows, m, n, A, lda, B, ldb, nullptr, 0, C, n, nullptr, accumulate);
}

// out[c] (+)= sum_r w[r] x[r][c]
static sat_status gat_wcolsum(sat_ctx *ctx, const float *x, int32_t ld, int64_t rows, int32_t d, const float *w, float *out, int accumulate)
{
    if (rows == 0) {
        if (!accumulate) SAT_CUDA(ctx, cudaMemsetAsync(out, 0, (size_t)d * sizeof(float), ctx->stream));
        return SAT_OK;
    }
    const int64_t blocks = cdiv64(rows, GAT_WSUM_ROWS);
    SAT_TRY(sat_ensure(ctx, ctx->buf_colsum, (size_t)blocks * d * sizeof(float)));
    k_gat_wcolsum<<<(unsigned)blocks, 256, 0, ctx->stream>>>(x, ld, rows, d, w, (float *)ctx->buf_colsum.p);
    SAT_LAUNCHED(ctx);
    return sat_splitk_reduce(ctx, (const float *)ctx->buf_colsum.p, d, (int32_t)blocks, accumulate, out, d, d);
}

#define GAT_DISPATCH(NVV, CALL)            \
    do {                                   \
        if ((NVV) <= 1) { CALL(1); }       \
        else if ((NVV) <= 2) { CALL(2); }  \
        else if ((NVV) <= 4) { CALL(4); }  \
        else { CALL(8); }                  \
    } while (0)

extern "C" sat_status sat_gat_fwd(sat_ctx *ctx, int32_t part, int32_t layer, int32_t d_in, int32_t d_out, const float *h_in, int32_t ld_in,
                                  const float *h_halo, int32_t ld_halo, const float *W, const float *a_src, const float *a_dst,
                                  const float *bias, int act, float *h_out, int32_t ld_out)
{
    CHECK_CTX(ctx);
    PartView v;
    SAT_TRY(sat_part_view(ctx, part, &v));
    if (layer < 1 || layer > SAT_MAX_LAYERS) return sat_fail(ctx, SAT_EINVAL, "sat_gat_fwd: layer must be in [1, %d]", SAT_MAX_LAYERS);
    if (d_in <= 0 || d_out <= 0 || d_out > 128 * GAT_MAX_NV || !W || !a_src || !a_dst) return sat_fail(ctx, SAT_EINVAL, "sat_gat_fwd: bad widths or null parameters");
    if (act != SAT_ACT_NONE && act != SAT_ACT_RELU) return sat_fail(ctx, SAT_EINVAL, "sat_gat_fwd: unknown activation");
    if (v.n_rows > 0 && (!h_in || !h_out || !ok_ld(ld_in, d_in) || !ok_ld(ld_out, d_out) || !aligned16(h_in) || !aligned16(h_out)))
        return sat_fail(ctx, SAT_EINVAL, "sat_gat_fwd: null / misaligned h_in / h_out or bad leading dimension");
    if (v.n_halo > 0 && (!h_halo || !ok_ld(ld_halo, d_in) || !aligned16(h_halo))) return sat_fail(ctx, SAT_EINVAL, "sat_gat_fwd: null / misaligned h_halo");
    GatState &G = ctx->gat[layer];
    const int32_t ld_z = round_up4(d_out);
    const int64_t n = ctx->n, nb = ctx->nb;
    if (G.d_out != d_out || G.valid.size() != (size_t)ctx->M) {
        // buffers over all rows / halo positions of the graph (any partition may be called); zeroed once so that the padding
        // columns of the z rows, which no kernel writes, read as zero
        SAT_TRY(sat_ensure(ctx, G.z_in, (size_t)(n > 0 ? n : 1) * ld_z * sizeof(float)));
        SAT_TRY(sat_ensure(ctx, G.z_halo, (size_t)(nb > 0 ? nb : 1) * ld_z * sizeof(float)));
        SAT_TRY(sat_ensure(ctx, G.scal, (size_t)(3 * (n > 0 ? n : 1) + (nb > 0 ? nb : 1)) * sizeof(float)));
        SAT_CUDA(ctx, cudaMemsetAsync(G.z_in.p, 0, G.z_in.bytes, ctx->stream));
        SAT_CUDA(ctx, cudaMemsetAsync(G.z_halo.p, 0, G.z_halo.bytes, ctx->stream));
        G.d_out = d_out;
        G.valid.assign(ctx->M, 0);
    }
    G.relu = act == SAT_ACT_RELU;
    float *z_in = (float *)G.z_in.p, *z_halo = (float *)G.z_halo.p;
    float *s_in = (float *)G.scal.p, *s_dst = s_in + n, *lse = s_dst + n, *s_halo = lse + n;
    SAT_TRY(gat_nn(ctx, v.n_rows, d_out, d_in, h_in, ld_in, W, z_in + (int64_t)v.row0 * ld_z, ld_z));
    SAT_TRY(gat_nn(ctx, v.n_halo, d_out, d_in, h_halo, ld_halo, W, z_halo + v.halo0 * ld_z, ld_z));
    ProfScope prof(ctx, SATK_GAT, 0.0, 0.0);
    if (v.n_rows > 0) {
        k_gat_scores<<<(unsigned)cdiv64((int64_t)v.n_rows * 32, 256), 256, 0, ctx->stream>>>(z_in + (int64_t)v.row0 * ld_z, ld_z, v.n_rows, d_out, a_src, a_dst,
                                                                                           s_in + v.row0, s_dst + v.row0);
        SAT_LAUNCHED(ctx);
    }
    if (v.n_halo > 0) {
        k_gat_scores<<<(unsigned)cdiv64(v.n_halo * 32, 256), 256, 0, ctx->stream>>>(z_halo + v.halo0 * ld_z, ld_z, v.n_halo, d_out, a_src, nullptr,
                                                                                  s_halo + v.halo0, nullptr);
        SAT_LAUNCHED(ctx);
    }
    if (v.n_rows > 0) {
        const int nv = ((d_out + 3) / 4 + 31) / 32;
        float *partial = nullptr;
        if (v.n_mitems > 0) {
            SAT_TRY(sat_ensure(ctx, ctx->buf_partial, (size_t)v.n_mitems * ld_z * sizeof(float)));
            partial = (float *)ctx->buf_partial.p;
        }
        k_gat_lse<<<(unsigned)cdiv64((int64_t)v.n_rows * 32, 256), 256, 0, ctx->stream>>>(ctx->lrowptr, ctx->lenc, ctx->n, v.row0, v.n_rows, s_in, s_halo,
                                                                                        s_dst, lse);
        SAT_LAUNCHED(ctx);
        const unsigned grid = (unsigned)cdiv64((int64_t)v.n_items * 32, 256);
        float *out_base = h_out - (int64_t)v.row0 * ld_out;
#define CALL(NV)                                                                                                                                    \
    k_gat_fwd_items<NV><<<grid, 256, 0, ctx->stream>>>(ctx->lrowptr, ctx->lenc, ctx->item_row, ctx->first_item, ctx->item_mslot, v.item0, v.n_items,    \
                                                       v.mitem0, ctx->n, z_in, z_halo, ld_z, s_in, s_halo, s_dst, lse, d_out, bias, G.relu, out_base, \
                                                       ld_out, partial)
        GAT_DISPATCH(nv, CALL);
#undef CALL
        SAT_LAUNCHED(ctx);
        if (v.n_mrows > 0) {
            k_gat_fwd_fixup<<<(unsigned)cdiv64((int64_t)v.n_mrows * ((d_out + 3) / 4), 256), 256, 0, ctx->stream>>>(
                ctx->mrows, v.mrow0, v.n_mrows, ctx->first_item, ctx->item_mslot, v.mitem0, d_out, partial, ld_z, bias, G.relu, out_base, ld_out);
            SAT_LAUNCHED(ctx);
        }
    }
    for (int m = (part == SAT_ALL_PARTS ? 0 : part); m < (part == SAT_ALL_PARTS ? ctx->M : part + 1); ++m) G.valid[m] = 1;
    return SAT_OK;
}

// the attention scores kept by the forward call, for checkpoints and tests
extern "C" sat_status sat_gat_scores(sat_ctx *ctx, int32_t layer, float *s_src_inner_host, float *s_dst_host, float *s_src_halo_host)
{
    CHECK_CTX(ctx);
    if (layer < 1 || layer > SAT_MAX_LAYERS) return sat_fail(ctx, SAT_EINVAL, "sat_gat_scores: layer must be in [1, %d]", SAT_MAX_LAYERS);
    GatState &G = ctx->gat[layer];
    if (G.d_out <= 0 || G.valid.size() != (size_t)ctx->M) return sat_fail(ctx, SAT_ESTATE, "sat_gat_scores: sat_gat_fwd has not run for layer %d", layer);
    for (int m = 0; m < ctx->M; ++m)
        if (!G.valid[m]) return sat_fail(ctx, SAT_ESTATE, "sat_gat_scores: sat_gat_fwd has not run for partition %d of layer %d", m, layer);
    const int64_t n = ctx->n, nb = ctx->nb;
    const float *s_in = (const float *)G.scal.p, *s_dst = s_in + n, *s_halo = s_dst + 2 * n;
    if (s_src_inner_host) SAT_CUDA(ctx, cudaMemcpyAsync(s_src_inner_host, s_in, (size_t)n * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    if (s_dst_host) SAT_CUDA(ctx, cudaMemcpyAsync(s_dst_host, s_dst, (size_t)n * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    if (s_src_halo_host && nb > 0) SAT_CUDA(ctx, cudaMemcpyAsync(s_src_halo_host, s_halo, (size_t)nb * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    SAT_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return SAT_OK;
}

extern "C" sat_status sat_gat_bwd(sat_ctx *ctx, int32_t part, int32_t layer, const float *g_out, int32_t ld_g, const float *h_out, int32_t ld_out,
                                  const float *h_in, int32_t ld_in, const float *h_halo, int32_t ld_halo, int32_t d_in, const float *W,
                                  const float *a_src, const float *a_dst, float *g_W, float *g_a_src, float *g_a_dst, float *g_b,
                                  int accumulate, float *g_in, int32_t ld_gin)
{
    CHECK_CTX(ctx);
    PartView v;
    SAT_TRY(sat_part_view(ctx, part, &v));
    if (layer < 1 || layer > SAT_MAX_LAYERS) return sat_fail(ctx, SAT_EINVAL, "sat_gat_bwd: layer must be in [1, %d]", SAT_MAX_LAYERS);
    GatState &G = ctx->gat[layer];
    if (G.d_out <= 0 || G.valid.size() != (size_t)ctx->M) return sat_fail(ctx, SAT_ESTATE, "sat_gat_bwd: sat_gat_fwd has not run for layer %d", layer);
    for (int m = (part == SAT_ALL_PARTS ? 0 : part); m < (part == SAT_ALL_PARTS ? ctx->M : part + 1); ++m)
        if (!G.valid[m]) return sat_fail(ctx, SAT_ESTATE, "sat_gat_bwd: sat_gat_fwd has not run for partition %d of layer %d", m, layer);
    const int32_t d_out = G.d_out, ld_z = round_up4(d_out);
    if (d_in <= 0 || !W || !a_src || !a_dst || !g_W || !g_a_src || !g_a_dst || !g_b) return sat_fail(ctx, SAT_EINVAL, "sat_gat_bwd: null parameter or gradient array");
    if (accumulate != 0 && accumulate != 1) return sat_fail(ctx, SAT_EINVAL, "sat_gat_bwd: accumulate must be 0 or 1");
    if (v.n_rows > 0 && (!g_out || !h_in || !ok_ld(ld_g, d_out) || !ok_ld(ld_in, d_in) || !aligned16(g_out) || !aligned16(h_in) ||
                         (G.relu && (!h_out || !ok_ld(ld_out, d_out)))))
        return sat_fail(ctx, SAT_EINVAL, "sat_gat_bwd: null / misaligned g_out / h_in / h_out or bad leading dimension");
    if (v.n_halo > 0 && (!h_halo || !ok_ld(ld_halo, d_in) || !aligned16(h_halo))) return sat_fail(ctx, SAT_EINVAL, "sat_gat_bwd: null / misaligned h_halo");
    if (g_in && v.n_rows > 0 && (!ok_ld(ld_gin, d_in) || !aligned16(g_in))) return sat_fail(ctx, SAT_EINVAL, "sat_gat_bwd: misaligned g_in or bad ld_gin");
    const int64_t n = ctx->n, nb = ctx->nb;
    float *z_in = (float *)G.z_in.p, *z_halo = (float *)G.z_halo.p;
    float *s_in = (float *)G.scal.p, *s_dst = s_in + n, *lse = s_dst + n, *s_halo = lse + n;
    // scratch of the call: D, dZ (inner rows of the selection, halo rows of the selection), t, ds_dst, ds_src
    const size_t f_rows = (size_t)(v.n_rows > 0 ? v.n_rows : 1), f_halo = (size_t)(v.n_halo > 0 ? v.n_halo : 1);
    const size_t t_floats = (2 * f_rows + 3) & ~(size_t)3;                  // the doubles first, then 16-byte aligned rows
    SAT_TRY(sat_ensure(ctx, ctx->buf_gat, (t_floats + (2 * f_rows + f_halo) * ld_z + 2 * f_rows + f_halo + 64) * sizeof(float)));
    double *t = (double *)ctx->buf_gat.p;
    float *D = (float *)ctx->buf_gat.p + t_floats, *dz_in = D + f_rows * ld_z, *dz_halo = dz_in + f_rows * ld_z;
    float *ds_dst = dz_halo + f_halo * ld_z, *ds_in = ds_dst + f_rows, *ds_halo = ds_in + f_rows;
    // virtual bases indexed by partition-major row / global halo position
    const float *Db = D - (int64_t)v.row0 * ld_z;
    float *dz_in_b = dz_in - (int64_t)v.row0 * ld_z, *dz_halo_b = dz_halo - v.halo0 * ld_z;
    double *t_b = t - v.row0;
    float *ds_dst_b = ds_dst - v.row0, *ds_in_b = ds_in - v.row0, *ds_halo_b = ds_halo - v.halo0;
    const int nv = ((d_out + 3) / 4 + 31) / 32;
    if (v.n_rows > 0) {
        SAT_CUDA(ctx, cudaMemsetAsync(D, 0, f_rows * ld_z * sizeof(float), ctx->stream));   // padding columns of D read as zero
        {
            ProfScope prof(ctx, SATK_GAT, 0.0, 0.0);
            k_gat_dmask<<<(unsigned)cdiv64((int64_t)v.n_rows * d_out, 256), 256, 0, ctx->stream>>>(g_out, ld_g, G.relu ? h_out : nullptr, ld_out, v.n_rows, d_out,
                                                                                                 D, ld_z);
            SAT_LAUNCHED(ctx);
        }
        SAT_TRY(sat_mask_rows(ctx, D, ld_z, v.n_rows, d_out, nullptr, 0, nullptr, 0, g_b, accumulate));
        // per-item partial sums: 4 doubles for the row side, a dZ row and a double for the column side
        const size_t n_it = (size_t)v.n_items;
        SAT_TRY(sat_ensure(ctx, ctx->buf_gat_items, (5 * n_it * 2 + n_it * ld_z + 64) * sizeof(float)));
        double *part4 = (double *)ctx->buf_gat_items.p, *pdss = part4 + 4 * n_it;
        float *pdz = (float *)(pdss + n_it + (n_it & 1));   // 16-byte aligned rows after an even number of doubles
        ProfScope prof(ctx, SATK_GAT, 0.0, 0.0);
        const unsigned grid = (unsigned)cdiv64((int64_t)v.n_items * 32, 256);
#define CALL(NV)                                                                                                                                 \
    k_gat_bwd_rows_items<NV><<<grid, 256, 0, ctx->stream>>>(ctx->lrowptr, ctx->lenc, ctx->item_row, ctx->first_item, v.item0, v.n_items, ctx->n, z_in, \
                                                            z_halo, ld_z, s_in, s_halo, s_dst, lse, d_out, Db, ld_z, part4)
        GAT_DISPATCH(nv, CALL);
#undef CALL
        SAT_LAUNCHED(ctx);
        k_gat_rows_combine<<<(unsigned)cdiv64(v.n_rows, 256), 256, 0, ctx->stream>>>(ctx->first_item, v.item0, v.row0, v.n_rows, part4, t_b, ds_dst_b);
        SAT_LAUNCHED(ctx);
#define CALL(NV)                                                                                                                                  \
    k_gat_bwd_cols_items<NV><<<grid, 256, 0, ctx->stream>>>(ctx->lrowptr, ctx->lenc, ctx->inner_cnt, ctx->item_row, ctx->first_item, v.item0, v.n_items, \
                                                            z_in, ld_z, s_in, s_dst, lse, t_b, d_out, Db, ld_z, pdz, pdss)
        GAT_DISPATCH(nv, CALL);
#undef CALL
        SAT_LAUNCHED(ctx);
        k_gat_cols_combine<<<(unsigned)cdiv64((int64_t)v.n_rows * ((d_out + 3) / 4), 256), 256, 0, ctx->stream>>>(
            ctx->first_item, v.item0, v.row0, v.n_rows, d_out, pdz, ld_z, pdss, ds_dst_b, a_src, a_dst, dz_in_b, ds_in_b);
        SAT_LAUNCHED(ctx);
    } else if (!accumulate) {
        SAT_CUDA(ctx, cudaMemsetAsync(g_b, 0, (size_t)d_out * sizeof(float), ctx->stream));
    }
    if (v.n_halo > 0 && v.n_rows > 0) {
        ProfScope prof(ctx, SATK_GAT, 0.0, 0.0);
        const unsigned grid = (unsigned)cdiv64(v.n_halo * 32, 256);
#define CALL(NV)                                                                                                                                   \
    k_gat_bwd_cols<NV, 1><<<grid, 256, 0, ctx->stream>>>(ctx->hrow_ptr, ctx->hrow_pos, nullptr, v.halo0, v.n_halo, z_halo, ld_z, s_halo, s_dst, lse, \
                                                         t_b, nullptr, d_out, Db, ld_z, a_src, a_dst, dz_halo_b, ds_halo_b)
        GAT_DISPATCH(nv, CALL);
#undef CALL
        SAT_LAUNCHED(ctx);
        if (v.n_hlong > 0) {
#define CALL(NV)                                                                                                                                  \
    k_gat_bwd_cols_long<NV><<<(unsigned)v.n_hlong, 256, 0, ctx->stream>>>(ctx->hlong, v.hlong0, ctx->hrow_ptr, ctx->hrow_pos, z_halo, ld_z, s_halo, s_dst, \
                                                                          lse, t_b, d_out, Db, ld_z, a_src, dz_halo_b, ds_halo_b)
            GAT_DISPATCH(nv, CALL);
#undef CALL
            SAT_LAUNCHED(ctx);
        }
    }
    const int64_t halo_rows = v.n_rows > 0 ? v.n_halo : 0;
    // parameter gradients
    SAT_TRY(gat_tn(ctx, v.n_rows, d_in, d_out, h_in, ld_in, dz_in, ld_z, g_W, accumulate));
    if (halo_rows > 0) SAT_TRY(gat_tn(ctx, halo_rows, d_in, d_out, h_halo, ld_halo, dz_halo, ld_z, g_W, 1));
    SAT_TRY(gat_wcolsum(ctx, z_in + (int64_t)v.row0 * ld_z, ld_z, v.n_rows, d_out, ds_in, g_a_src, accumulate));
    if (halo_rows > 0) SAT_TRY(gat_wcolsum(ctx, z_halo + v.halo0 * ld_z, ld_z, halo_rows, d_out, ds_halo, g_a_src, 1));
    SAT_TRY(gat_wcolsum(ctx, z_in + (int64_t)v.row0 * ld_z, ld_z, v.n_rows, d_out, ds_dst, g_a_dst, accumulate));
    // input gradient of the inner rows
    if (g_in && v.n_rows > 0) SAT_TRY(gat_nt(ctx, v.n_rows, d_in, d_out, dz_in, ld_z, W, g_in, ld_gin));
    return SAT_OK;
}
