// Dense contractions on the 5th-generation tensor cores (tcgen05.mma kind::tf32, accumulators in TMEM,
// operands staged in shared memory by TMA) with fp32-level accuracy from a two-term TF32 split:
//     x = hi + lo                                               (|x - hi - lo| <= 2^-21 |x|)
//     A B ~= Ah Bh + Ah Bl + Al Bh                              (three MMAs per k-step, fp32 accumulate)
// Activations and weights stay plain fp32 in global memory: TMA brings the fp32 tiles into shared memory and the
// converter warps write the residual tiles next to them, element-wise, so the swizzled layout never has to be decoded
// (see "TF32 split of a shared-memory tile" below for the two variants).  Weights are repacked once per call into the
// K-major operand layout.
//
//   k_gemm_tc_k   C[M x N] = A[M x K] B[N x K]^T   both operands K-major, 64-byte swizzle, BLOCK_K = 16, persistent
//                 (layer transform, LSTM gates with two A operands or a cached projection, predictor output, input gradient)
//   k_gemm_tc_mn  C[M x N] = A[R x M]^T B[R x N]   both operands MN-major, 128-byte swizzle with 32-byte atoms, split over R
//                 (weight gradient)
// Warp roles of k_gemm_tc_k (512 threads): warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, then 6 converter and
// 8 epilogue warps (two per TMEM lane quadrant), or 2 + 12 for the K = h variants with a side operand.  k_gemm_tc_mn:
// warps 0 / 1 as above, warps 2..5 convert during the main loop and then run the epilogue.  Every mbarrier wait is
// bounded; a timeout raises a status word and lets the CTA drain (TMEM is freed, the kernel returns).
#include <cuda.h>

#include "sat_internal.h"

#define TC_BM 128
#define TC_BK 16          /* fp32 elements per k-block: 64-byte rows */
#define TC_THREADS 192
#define TC_WAIT_LIMIT (1u << 22)

// =====================================================================================
// PTX wrappers
// =====================================================================================
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// bounded wait: returns false (and raises *dead) when the limit is hit or another thread already gave up.
// SLEEP_NS > 0 backs off between polls: a spinning warp otherwise takes issue slots from the warps doing the work
// (the epilogue shares its schedulers with the waiting converter warps).
template <int SLEEP_NS = 0>
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *dead, int *status)
{
    const uint32_t addr = smem_u32(bar);
    for (uint32_t it = 0; it < TC_WAIT_LIMIT; ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t"
            "}"
            : "=r"(ok)
            : "r"(addr), "r"(parity)
            : "memory");
        if (ok) return true;
        if (*dead) return false;
        if (SLEEP_NS > 0) __nanosleep(SLEEP_NS);
    }
    *dead = 1;
    atomicOr(status, 1);
    return false;
}
// whole-warp wait: lane 0 polls, then every lane observes the completed phase itself (one immediate try_wait each), so
// that a waiting warp issues one poll per round instead of 32
__device__ __forceinline__ bool mbar_wait_warp(uint64_t *bar, uint32_t parity, volatile int *dead, int *status, int lane)
{
    int ok = 1;
    if (lane == 0) ok = mbar_wait<64>(bar, parity, dead, status) ? 1 : 0;
    ok = __shfl_sync(0xffffffffu, ok, 0);
    if (!ok) return false;
    return mbar_wait(bar, parity, dead, status);
}
__device__ __forceinline__ void tma_load_2d(void *smem_dst, const CUtensorMap *map, uint64_t *bar, int32_t x, int32_t y)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, const void *smem_src, int32_t x, int32_t y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"((uint64_t)map), "r"(smem_u32(smem_src)),
                 "r"(x), "r"(y)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// waits until at most `N` of this thread's bulk stores still read their shared-memory source
template <int N>
__device__ __forceinline__ void tma_store_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t"
        "}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t *r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, "
        "%19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// shared-memory matrix descriptor: start address, leading / stride byte offsets (16-byte units), sm_100 version, swizzle mode
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout_type)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)layout_type << 61;
    return d;
}

// instruction descriptor for kind::tf32 (TF32 operands in 32-bit containers, fp32 accumulation)
__host__ __device__ inline uint32_t make_idesc(int n, int a_mn_major, int b_mn_major)
{
    uint32_t d = 0;
    d |= 1u << 4;   // D format: f32
    d |= 2u << 7;   // A format: tf32
    d |= 2u << 10;  // B format: tf32
    d |= (uint32_t)a_mn_major << 15;
    d |= (uint32_t)b_mn_major << 16;
    d |= (uint32_t)(n >> 3) << 17;
    d |= (uint32_t)(TC_BM >> 4) << 24;
    return d;
}

// =====================================================================================
// TF32 split of a shared-memory tile, element-wise (the swizzled layout never has to be decoded).
//
// The tensor core reads an fp32 container as TF32 by ignoring the low 13 mantissa bits.  split_tile_residual uses that:
// the raw tile already is the "hi" operand (hi = x with those bits cleared) and only lo = tf32_rn(x - hi) is written, to
// the second tile (x - hi is exact; rounding lo to nearest keeps the representation error |x - hi - lo| <= 2^-21 |x|
// free of bias).  split_tile_round rounds hi to nearest as well and rewrites the raw tile in place: hi and lo are then
// symmetric around x, which matters for the weight gradient (a small difference of ~1e5 signed terms per element).
// =====================================================================================
__device__ __forceinline__ float tf32_round(float x)
{
    return __uint_as_float((__float_as_uint(x) + 0x1000u) & 0xFFFFE000u);  // round half away from zero to 10 mantissa bits
}
__device__ __forceinline__ float tf32_residual(float x) { return tf32_round(x - __uint_as_float(__float_as_uint(x) & 0xFFFFE000u)); }
__device__ __forceinline__ float4 residual4(const float4 &x)
{
    return make_float4(tf32_residual(x.x), tf32_residual(x.y), tf32_residual(x.z), tf32_residual(x.w));
}
__device__ __forceinline__ void split4(const float4 &x, float4 &h, float4 &l)
{
    h.x = tf32_round(x.x); l.x = tf32_round(x.x - h.x);
    h.y = tf32_round(x.y); l.y = tf32_round(x.y - h.y);
    h.z = tf32_round(x.z); l.z = tf32_round(x.z - h.z);
    h.w = tf32_round(x.w); l.w = tf32_round(x.w - h.w);
}
// two 16-byte chunks per thread and iteration, loads first (the loops are latency-bound otherwise)
__device__ __forceinline__ void split_tile_residual(const uint8_t *hi_tile, uint8_t *lo_tile, uint32_t bytes, int tid, int nthreads)
{
    const uint32_t step = (uint32_t)nthreads * 16;
    for (uint32_t off = (uint32_t)tid * 16; off < bytes; off += 2 * step) {
        const uint32_t off2 = off + step;
        const bool two = off2 < bytes;
        const float4 x1 = *reinterpret_cast<const float4 *>(hi_tile + off);
        float4 x2 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (two) x2 = *reinterpret_cast<const float4 *>(hi_tile + off2);
        *reinterpret_cast<float4 *>(lo_tile + off) = residual4(x1);
        if (two) *reinterpret_cast<float4 *>(lo_tile + off2) = residual4(x2);
    }
}
__device__ __forceinline__ void split_tile_round(uint8_t *hi_tile, uint8_t *lo_tile, uint32_t bytes, int tid, int nthreads)
{
    const uint32_t step = (uint32_t)nthreads * 16;
    for (uint32_t off = (uint32_t)tid * 16; off < bytes; off += 2 * step) {
        const uint32_t off2 = off + step;
        const bool two = off2 < bytes;
        const float4 x1 = *reinterpret_cast<float4 *>(hi_tile + off);
        float4 x2 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (two) x2 = *reinterpret_cast<float4 *>(hi_tile + off2);
        float4 h1, l1, h2, l2;
        split4(x1, h1, l1);
        split4(x2, h2, l2);
        *reinterpret_cast<float4 *>(hi_tile + off) = h1;
        *reinterpret_cast<float4 *>(lo_tile + off) = l1;
        if (two) {
            *reinterpret_cast<float4 *>(hi_tile + off2) = h2;
            *reinterpret_cast<float4 *>(lo_tile + off2) = l2;
        }
    }
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// make generic-proxy shared-memory writes visible to the tensor-core (async) proxy
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// =====================================================================================
// K-major kernel
// =====================================================================================
struct TcEpilogue {
    float *C;
    int64_t ldc;
    const float *bias;
    int relu;
    uint32_t *mask_out;
    int32_t mask_words;
    const float *resid;  // C += resid[resid_idx[row]]  (row gather)
    const int32_t *resid_idx;
    int64_t ld_resid;
    int32_t lstm_h;      // > 0: fused LSTM cell, C = hidden state [M x lstm_h], lstm_c = cell state
    int lstm_first;
    float *lstm_c;       // cell state in the blocked layout of sat_cell_offset
    const float *addend; // [M x ld_addend] added to the gate pre-activations (cached input projection), or null
    int64_t ld_addend;
    float *push_dst;     // (EPI_PUSH) row i is also written to push_dst + push_slot[i] * ld_push when push_slot[i] >= 0
    const int32_t *push_slot;
    int64_t ld_push;
    const int32_t *tile_order;  // row tile walked at position i of the schedule (null: i itself)
};

// Row tile (of TC_BM rows) of schedule position t: the persistent CTAs walk positions blockIdx.x, blockIdx.x + gridDim.x, ...;
// a permutation lets the caller choose which row tiles run at the same time (results do not depend on it).
__device__ __forceinline__ int64_t tck_row_tile(const TcEpilogue &ep, int64_t t, int32_t n_tiles_n)
{
    const int64_t rt = t / n_tiles_n;
    return ep.tile_order ? (int64_t)__ldg(ep.tile_order + rt) : rt;
}

struct TcShared {
    uint64_t full[4];       // TMA bytes of the stage have landed
    uint64_t conv[4];       // the converter threads have split the stage
    uint64_t empty[4];      // the MMAs reading the stage have completed
    uint64_t accum;         // (MN-major kernel) all MMAs of the tile have completed
    uint64_t acc_full[2];   // (K-major kernel) accumulator buffer holds a finished tile
    uint64_t acc_empty[2];  // (K-major kernel) accumulator buffer has been drained by the epilogue
    uint32_t tmem_base;
    int dead;
};

#define TC_CONV_THREADS 128
#define TC_EPI_THREADS 128
/* 512 threads, 128 registers each: warp 0 TMA, warp 1 MMA, then the converter warps, then the epilogue warps.  The split
 * between converters and epilogue depends on the epilogue variant (TckCfg): the K = h variants with a side operand have
 * four k-blocks per tile and an epilogue bound by instruction issue, so they run 2 + 12 instead of 6 + 8.
 * The converter warps work in two groups on alternate k-blocks, so two stages are being split at any time.  Every stage
 * count is even, hence a stage is always handled by the same group and each group meets the phases of its stages in
 * order (a parity wait must never be more than one phase ahead of its barrier). */
#define TCK_THREADS 512
#define TCK_CONV_GROUPS 2
/* The weights' residual plane is made once by k_split_weights and fetched by TMA next to the raw plane: B is the same for
 * every row tile, and splitting its tile again per k-block cost the converters twice what the A tile costs (measured:
 * K = 256 transform 132 -> 118 us, K = 64 LSTM step 98 -> 85 us) for 16 KB more L2 -> SM traffic per k-block. */
#define TCK_B_PRESPLIT 1

// Epilogue variants.  The ones with a per-row side operand streamed from global memory (gathered residual rows, cached
// LSTM input projection) keep a ring of 32 x 32 side tiles per epilogue warp in shared memory, filled by cp.async ahead of
// the consumer: one chunk in flight per warp left the loads latency-bound at ~2 TB/s.  Those variants contract over a
// small K (the predictor width), so they give up main-loop stages for the ring.
enum { EPI_PLAIN = 0, EPI_RESID = 1, EPI_LSTM = 2, EPI_LSTM_ADD = 3, EPI_PUSH = 4 };   // EPI_PUSH = EPI_PLAIN + a second copy of the rows that have a cache slot
template <int EPI> struct TckCfg { static constexpr int stages = 4, ring = 0, conv_warps = 6, epi_warps = 8, out_bytes = epi_warps * 4096; };
template <> struct TckCfg<EPI_RESID> { static constexpr int stages = 2, ring = 1, conv_warps = 2, epi_warps = 12, out_bytes = epi_warps * 4096; };
template <> struct TckCfg<EPI_LSTM> { static constexpr int stages = 4, ring = 0, conv_warps = 6, epi_warps = 8, out_bytes = 0; };
template <> struct TckCfg<EPI_LSTM_ADD> { static constexpr int stages = 2, ring = 2, conv_warps = 2, epi_warps = 12, out_bytes = 0; };
static_assert(TckCfg<EPI_PLAIN>::stages % TCK_CONV_GROUPS == 0 && TckCfg<EPI_RESID>::stages % TCK_CONV_GROUPS == 0 &&
                  TckCfg<EPI_LSTM>::stages % TCK_CONV_GROUPS == 0 && TckCfg<EPI_LSTM_ADD>::stages % TCK_CONV_GROUPS == 0,
              "a stage must always be split by the same converter group");

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc, bool valid)
{
    // src-size 0 writes 16 zero bytes without reading the source
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(valid ? 16u : 0u) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Persistent: each CTA walks tiles blockIdx.x, blockIdx.x + gridDim.x, ...  The shared-memory ring of k-block stages
// and the two TMEM accumulator buffers let the TMA loads, the TF32 split, the MMAs and the epilogue of consecutive tiles
// overlap.  A and B arrive as raw fp32 tiles, which the tensor core reads as the hi operands; the converters write the
// residual tiles.  The epilogue is a template parameter (plain bias / ReLU / mask, gathered residual, fused LSTM cell)
// and runs on eight or twelve warps, two or three per TMEM lane quadrant taking 32-column chunks in turn: with one warp
// per scheduler the epilogue was bound by instruction issue and load latency (9 - 14 us per 128 x 256 tile, longer than
// the main loop of a K = 256 tile).
template <int EPI>
__global__ void __launch_bounds__(TCK_THREADS, 1)
k_gemm_tc_k(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapA2, const __grid_constant__ CUtensorMap mapB,
            const __grid_constant__ CUtensorMap mapBlo, const __grid_constant__ CUtensorMap mapC, int use_tma_store, int64_t M, int32_t N, int32_t nkb1, int32_t nkb2, int32_t bn, int32_t n_tiles_n, int64_t n_tiles, TcEpilogue ep, int *status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t a_bytes = TC_BM * TC_BK * 4;  // one plane of the A tile: 128 rows x 64 B
    const uint32_t b_bytes = (uint32_t)bn * TC_BK * 4;
    const uint32_t stage_bytes = 2 * a_bytes + 2 * b_bytes;  // [A hi | A lo | B hi | B lo]
    constexpr int STAGES = TckCfg<EPI>::stages;
    constexpr int RING = TckCfg<EPI>::ring;
    uint8_t *out_stage = smem + (size_t)STAGES * stage_bytes;
    uint8_t *ring_base = out_stage + TckCfg<EPI>::out_bytes;
    constexpr int CONV_THREADS = TckCfg<EPI>::conv_warps * 32, CONV_GROUP_THREADS = CONV_THREADS / TCK_CONV_GROUPS;
    constexpr int EPI_WARPS = TckCfg<EPI>::epi_warps, EPI_WARP0 = 2 + TckCfg<EPI>::conv_warps;
    constexpr int CHUNK_STEP = 32 * (EPI_WARPS / 4);  // the EPI_WARPS / 4 warps of a TMEM lane quadrant take 32-column chunks in turn
    static_assert(64 + CONV_THREADS + EPI_WARPS * 32 == TCK_THREADS && EPI_WARP0 % 4 == 0 && EPI_WARPS % 4 == 0, "warp roles");
    TcShared *sh = (TcShared *)(ring_base + (size_t)EPI_WARPS * RING * 4096);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int32_t nkb = nkb1 + nkb2;
    const uint32_t acc_cols = 256;  // column stride between the two accumulator buffers

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&sh->full[s], 1);
            mbar_init(&sh->conv[s], CONV_GROUP_THREADS);
            mbar_init(&sh->empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh->acc_full[i], 1);
            mbar_init(&sh->acc_empty[i], EPI_WARPS * 32);
        }
        sh->dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;
    volatile int *dead = &sh->dead;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t it = 0;
            for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
                const int32_t m0 = (int32_t)tck_row_tile(ep, t, n_tiles_n) * TC_BM;
                const int32_t n0 = (int32_t)(t % n_tiles_n) * bn;
                for (int32_t kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    if (!mbar_wait(&sh->empty[s], ph ^ 1u, dead, status)) goto done;
                    uint8_t *st = smem + (size_t)s * stage_bytes;
                    mbar_expect_tx(&sh->full[s], a_bytes + (TCK_B_PRESPLIT ? 2 * b_bytes : b_bytes));
                    if (kb < nkb1) tma_load_2d(st, &mapA, &sh->full[s], kb * TC_BK, m0);
                    else tma_load_2d(st, &mapA2, &sh->full[s], (kb - nkb1) * TC_BK, m0);
                    tma_load_2d(st + 2 * a_bytes, &mapB, &sh->full[s], kb * TC_BK, n0);
                    if (TCK_B_PRESPLIT) tma_load_2d(st + 2 * a_bytes + b_bytes, &mapBlo, &sh->full[s], kb * TC_BK, n0);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = make_idesc(bn, 0, 0);
            const uint64_t desc0 = make_desc(smem_u32(smem), 16, 512, 4);
            uint32_t it = 0, lt = 0;
            for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++lt) {
                const uint32_t buf = lt & 1u;
                if (!mbar_wait(&sh->acc_empty[buf], ((lt >> 1) & 1u) ^ 1u, dead, status)) goto done;
                tc_fence_after();
                const uint32_t acc = tmem + buf * acc_cols;
                for (int32_t kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1u;
                    // the converters arrive on conv[s] only after they have seen full[s] (the TMA bytes) themselves
                    if (!mbar_wait(&sh->conv[s], ph, dead, status)) goto done;
                    tc_fence_after();
                    // K-major, 64-byte swizzle: rows 64 B apart, 8-row groups 512 B apart; a k-step (8 values) is 32 B inside the
                    // row.  Only the 14-bit start-address field (bytes >> 4) differs between the descriptors of a stage.
                    const uint64_t a_hi0 = desc0 + (uint64_t)(((uint32_t)s * stage_bytes) >> 4);
#pragma unroll
                    for (int ks = 0; ks < TC_BK / 8; ++ks) {
                        const uint64_t a_hi = a_hi0 + (uint64_t)(ks * 2);
                        const uint64_t a_lo = a_hi + (a_bytes >> 4);
                        const uint64_t b_hi = a_hi + (2 * a_bytes >> 4);
                        const uint64_t b_lo = b_hi + (b_bytes >> 4);
                        tc_mma(acc, a_hi, b_hi, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
                        tc_mma(acc, a_hi, b_lo, idesc, 1u);
                        tc_mma(acc, a_lo, b_hi, idesc, 1u);
                    }
                    tc_commit(&sh->empty[s]);  // the stage is free once these MMAs have read it
                }
                tc_commit(&sh->acc_full[buf]);
            }
        }
    } else if (warp < EPI_WARP0) {
        // ---------------- converters: TF32 split of the A and B tiles of every k-block ----------------
        const int grp = (threadIdx.x - 64) / CONV_GROUP_THREADS;
        const int ctid = (threadIdx.x - 64) % CONV_GROUP_THREADS;
        uint32_t it = 0;
        for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
            for (int32_t kb = 0; kb < nkb; ++kb, ++it) {
                if ((int)(it % TCK_CONV_GROUPS) != grp) continue;
                const int s = it % STAGES;
                const uint32_t ph = (it / STAGES) & 1u;
                if (!mbar_wait(&sh->full[s], ph, dead, status)) goto done;
                uint8_t *st = smem + (size_t)s * stage_bytes;
                split_tile_residual(st, st + a_bytes, a_bytes, ctid, CONV_GROUP_THREADS);
                if (!TCK_B_PRESPLIT) split_tile_residual(st + 2 * a_bytes, st + 2 * a_bytes + b_bytes, b_bytes, ctid, CONV_GROUP_THREADS);
                fence_async_smem();
                mbar_arrive(&sh->conv[s]);
            }
        }
    } else {
        // ---------------- epilogue ----------------
        // warp w reads TMEM lanes 32 (w % 4) .. +31 = rows of the tile, one row per thread; the warps of a lane quadrant
        // take alternate 32-column chunks.
        constexpr bool LSTM = EPI == EPI_LSTM || EPI == EPI_LSTM_ADD;
        const int e = warp - EPI_WARP0;
        const int q = warp & 3;
        const int c_first = 32 * (e >> 2);
        uint8_t *obuf = out_stage + e * 4096;
        const bool vec = ((ep.ldc & 3) == 0) && ((((uintptr_t)ep.C) & 15u) == 0);
        const int32_t n4 = (N + 3) & ~3;
        const bool lstm_full = LSTM && (ep.lstm_h & 3) == 0;
        const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);

        // Side-operand ring (RING slots of 32 rows x 128 B, 128-byte swizzle like the store staging tile), private to the
        // warp: cp.async group counting plus __syncwarp is all the synchronisation needed.  The prefetch cursor (pf_*)
        // walks this warp's (tile, chunk) sequence RING chunks ahead of the consumer.
        uint8_t *ring = ring_base + (size_t)e * RING * 4096;
        int64_t pf_t = blockIdx.x;
        int pf_c = c_first;
        const float *pf_srow = nullptr;
        int32_t pf_lim = 0;
        int32_t pf_idx_next = -1;   // (gathered residual) row index for the tile after the cursor's, fetched a tile early
        uint32_t pf_slot = 0, rd_slot = 0;
        auto pf_enter_tile = [&](int32_t idx_now) {
            // called when the cursor enters tile pf_t; idx_now = gathered row index for this thread's row, or -1
            pf_srow = nullptr;
            if (pf_t < n_tiles) {
                const int64_t prow = tck_row_tile(ep, pf_t, n_tiles_n) * TC_BM + q * 32 + lane;
                const int32_t pn0 = (int32_t)(pf_t % n_tiles_n) * bn;
                if (EPI == EPI_RESID) {
                    if (prow < M && idx_now >= 0) pf_srow = ep.resid + (int64_t)idx_now * ep.ld_resid + pn0;  // rows padded to 4 floats
                    pf_lim = n4 - pn0;
                    const int64_t nt = pf_t + gridDim.x;
                    const int64_t nrow = tck_row_tile(ep, nt, n_tiles_n) * TC_BM + q * 32 + lane;
                    pf_idx_next = (nt < n_tiles && nrow < M) ? __ldg(ep.resid_idx + nrow) : -1;
                } else {
                    if (prow < M) pf_srow = ep.addend + prow * ep.ld_addend + pn0;
                    pf_lim = N - pn0;
                }
            }
        };
        auto pf_issue = [&]() {
            // one group per call (possibly empty), so that the consumer's wait count is uniform.  Lane L copies 16-byte
            // piece (L & 7) of rows (L >> 3) + 4 i: an instruction touches 4 rows (4 cache lines) instead of 32, which
            // matters because the load/store unit handles one line per cycle.
            if (pf_t < n_tiles && pf_c < bn) {
                uint8_t *slot = ring + pf_slot * 4096;
                const float *base = EPI == EPI_RESID ? ep.resid : ep.addend;
                const int piece = lane & 7;
                const bool col_ok = pf_c + 4 * piece < pf_lim;
                if (EPI == EPI_RESID) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {  // gathered rows: the row pointer lives in the lane that owns the row
                        const int rr = (lane >> 3) + 4 * i;
                        const float *rowp = reinterpret_cast<const float *>(__shfl_sync(0xffffffffu, (unsigned long long)(uintptr_t)pf_srow, rr));
                        const bool valid = rowp != nullptr && col_ok;
                        cp_async16(slot + rr * 128 + ((piece ^ (rr & 7)) << 4), (valid ? rowp : base) + pf_c + 4 * piece, valid);
                    }
                } else {
                    // dense side operand: rows of the tile are ld_addend apart
                    const int64_t prow0 = tck_row_tile(ep, pf_t, n_tiles_n) * TC_BM + q * 32 + (lane >> 3);
                    const float *p0 = base + prow0 * ep.ld_addend + (int32_t)(pf_t % n_tiles_n) * bn + pf_c + 4 * piece;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int rr = (lane >> 3) + 4 * i;
                        const bool valid = prow0 + 4 * i < M && col_ok;
                        cp_async16(slot + rr * 128 + ((piece ^ (rr & 7)) << 4), valid ? p0 + (int64_t)(4 * i) * ep.ld_addend : base, valid);
                    }
                }
                pf_c += CHUNK_STEP;
                if (pf_c >= bn) {
                    pf_c = c_first;
                    pf_t += gridDim.x;
                    pf_enter_tile(pf_idx_next);
                }
            }
            cp_async_commit();
            pf_slot = pf_slot + 1 == RING ? 0 : pf_slot + 1;
        };
        if (RING > 0 && c_first < bn) {
            int32_t idx0 = -1;
            if (EPI == EPI_RESID && pf_t < n_tiles) {
                const int64_t prow = tck_row_tile(ep, pf_t, n_tiles_n) * TC_BM + q * 32 + lane;
                if (prow < M) idx0 = __ldg(ep.resid_idx + prow);
            }
            pf_enter_tile(idx0);
#pragma unroll
            for (int i = 0; i < RING; ++i) pf_issue();
        }

        uint32_t lt = 0;
        for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x, ++lt) {
            const int64_t m0 = tck_row_tile(ep, t, n_tiles_n) * TC_BM;
            const int32_t n0 = (int32_t)(t % n_tiles_n) * bn;
            const uint32_t buf = lt & 1u;
            const int64_t row = m0 + q * 32 + lane;
            const bool row_ok = row < M;
            float *crow = ep.C + row * ep.ldc;
            float *prow = nullptr;   // (EPI_PUSH) this row's home in the cache ring, if it has one
            // (EPI_PUSH with the staged store) the push goes out of the staging tile, four rows of 128 bytes per warp
            // instruction: lane L writes 16-byte piece L & 7 of rows (L >> 3) + 4 i, so it needs those rows' ring rows
            int32_t ps8[8];
            if (EPI == EPI_PUSH && !use_tma_store && row_ok) {
                const int32_t ps = __ldg(ep.push_slot + row);
                if (ps >= 0) prow = ep.push_dst + (int64_t)ps * ep.ld_push;
            }
            if (EPI == EPI_PUSH && use_tma_store) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int64_t rr = m0 + q * 32 + (lane >> 3) + 4 * i;
                    ps8[i] = rr < M ? __ldg(ep.push_slot + rr) : -1;
                }
            }
            float4 side[8], cside[2];
            // previous cell state of the next chunk, fetched one chunk ahead (two 128-bit loads per thread)
            auto load_cell = [&](int c0) {
                if (LSTM) {
                    cside[0] = cside[1] = zero4;
                    const int32_t j0 = (n0 + c0) >> 2;
                    if (row_ok && lstm_full && !ep.lstm_first && j0 + 7 < ep.lstm_h) {
                        const float *cp = ep.lstm_c + sat_cell_offset(row, j0, ep.lstm_h);
                        cside[0] = *reinterpret_cast<const float4 *>(cp);
                        cside[1] = *reinterpret_cast<const float4 *>(cp + 4);
                    }
                }
            };
            if (c_first < bn) load_cell(c_first);
            if (!mbar_wait_warp(&sh->acc_full[buf], (lt >> 1) & 1u, dead, status, lane)) goto done;
            tc_fence_after();
            for (int c0 = c_first; c0 < bn; c0 += CHUNK_STEP) {
                uint32_t r[32];
                tc_ld32(tmem + buf * acc_cols + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
                if (RING > 0) {
                    cp_async_wait<(RING > 0 ? RING - 1 : 0)>();  // every lane's copies of the oldest chunk in the ring have landed ...
                    __syncwarp();                                // ... and are visible to the lane that owns the row
                    const uint8_t *src = ring + rd_slot * 4096 + lane * 128;
#pragma unroll
                    for (int u = 0; u < 8; ++u) side[u] = *reinterpret_cast<const float4 *>(src + ((u ^ (lane & 7)) << 4));
                    rd_slot = rd_slot + 1 == RING ? 0 : rd_slot + 1;
                    __syncwarp();  // all lanes have read the slot: refill it with the chunk RING steps ahead
                    pf_issue();
                }
                if (LSTM) {
                    // packed columns 4 j .. 4 j + 3 are the (i, f, g, o) pre-activations of hidden unit j
                    if (row_ok) {
                        const int32_t j0 = (n0 + c0) >> 2;
                        const bool full = lstm_full && j0 + 7 < ep.lstm_h;
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            float4 b4 = EPI == EPI_LSTM_ADD ? side[u] : zero4;
                            if (ep.bias) {
                                const float4 bb = __ldg(reinterpret_cast<const float4 *>(ep.bias + n0 + c0) + u);
                                b4.x += bb.x; b4.y += bb.y; b4.z += bb.z; b4.w += bb.w;
                            }
                            r[4 * u] = __float_as_uint(__uint_as_float(r[4 * u]) + b4.x);
                            r[4 * u + 1] = __float_as_uint(__uint_as_float(r[4 * u + 1]) + b4.y);
                            r[4 * u + 2] = __float_as_uint(__uint_as_float(r[4 * u + 2]) + b4.z);
                            r[4 * u + 3] = __float_as_uint(__uint_as_float(r[4 * u + 3]) + b4.w);
                        }
                        float cprev[8];
                        cprev[0] = cside[0].x; cprev[1] = cside[0].y; cprev[2] = cside[0].z; cprev[3] = cside[0].w;
                        cprev[4] = cside[1].x; cprev[5] = cside[1].y; cprev[6] = cside[1].z; cprev[7] = cside[1].w;
                        if (!ep.lstm_first && !full) {
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                if (j0 + u < ep.lstm_h) cprev[u] = ep.lstm_c[sat_cell_offset(row, j0 + u, ep.lstm_h)];
                        }
                        if (c0 + CHUNK_STEP < bn) load_cell(c0 + CHUNK_STEP);
                        float sv[8], cv[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const float gi = sigmoid_fast(__uint_as_float(r[4 * u]));
                            const float gf = sigmoid_fast(__uint_as_float(r[4 * u + 1]));
                            const float gg = tanh_fast(__uint_as_float(r[4 * u + 2]));
                            const float go = sigmoid_fast(__uint_as_float(r[4 * u + 3]));
                            cv[u] = gf * cprev[u] + gi * gg;
                            sv[u] = go * tanh_fast(cv[u]);
                        }
                        if (full) {
                            float4 *cd = reinterpret_cast<float4 *>(ep.lstm_c + sat_cell_offset(row, j0, ep.lstm_h));
                            float4 *sd = reinterpret_cast<float4 *>(ep.C + row * ep.ldc + j0);
                            cd[0] = make_float4(cv[0], cv[1], cv[2], cv[3]);
                            cd[1] = make_float4(cv[4], cv[5], cv[6], cv[7]);
                            sd[0] = make_float4(sv[0], sv[1], sv[2], sv[3]);
                            sd[1] = make_float4(sv[4], sv[5], sv[6], sv[7]);
                        } else {
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                if (j0 + u < ep.lstm_h) {
                                    ep.lstm_c[sat_cell_offset(row, j0 + u, ep.lstm_h)] = cv[u];
                                    ep.C[row * ep.ldc + j0 + u] = sv[u];
                                }
                        }
                    }
                    continue;
                }
                uint32_t bits = 0;
                if (row_ok) {
                    // bias is padded with zeros to the tile width and the accumulators of padded columns are exactly zero,
                    // so no column predicate is needed (the stores clip)
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float4 b4 = EPI == EPI_RESID ? side[j] : zero4;
                        if (ep.bias) {
                            const float4 bb = __ldg(reinterpret_cast<const float4 *>(ep.bias + n0 + c0) + j);
                            b4.x += bb.x; b4.y += bb.y; b4.z += bb.z; b4.w += bb.w;
                        }
                        r[4 * j] = __float_as_uint(__uint_as_float(r[4 * j]) + b4.x);
                        r[4 * j + 1] = __float_as_uint(__uint_as_float(r[4 * j + 1]) + b4.y);
                        r[4 * j + 2] = __float_as_uint(__uint_as_float(r[4 * j + 2]) + b4.z);
                        r[4 * j + 3] = __float_as_uint(__uint_as_float(r[4 * j + 3]) + b4.w);
                    }
                    if ((EPI == EPI_PLAIN || EPI == EPI_PUSH) && ep.mask_out) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) bits |= (__uint_as_float(r[j]) > 0.f ? 1u : 0u) << j;
                    }
                    if (ep.relu) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(fmaxf(__uint_as_float(r[j]), 0.f));
                    }
                }
                if (EPI == EPI_PUSH && prow) {   // one full 128-byte line per thread and chunk
#pragma unroll
                    for (int j4 = 0; j4 < 32; j4 += 4) {
                        const int32_t colb = n0 + c0 + j4;
                        if (colb + 3 < N) {
                            *reinterpret_cast<uint4 *>(prow + colb) = make_uint4(r[j4], r[j4 + 1], r[j4 + 2], r[j4 + 3]);
                        } else {
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj)
                                if (colb + jj < N) prow[colb + jj] = __uint_as_float(r[j4 + jj]);
                        }
                    }
                }
                if (use_tma_store) {
                    // stage the 32 x 32 block (128-byte swizzle: 16-byte chunk j of row r sits at chunk j ^ (r & 7)) and
                    // let the TMA write it as whole 128-byte row segments; rows / columns past the matrix are clipped
                    if (lane == 0) tma_store_wait_read<0>();  // the previous block has left the staging tile
                    __syncwarp();
                    uint8_t *dst = obuf + lane * 128;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<uint4 *>(dst + ((j ^ (lane & 7)) << 4)) = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) tma_store_2d(&mapC, obuf, n0 + c0, (int32_t)(m0 + q * 32));
                    if (EPI == EPI_PUSH) {
                        // the boundary rows also go to the cache ring, read back from the staged block: every instruction
                        // writes whole 128-byte row segments (the per-thread form touches 32 different lines per instruction)
                        const int piece = lane & 7;
                        const int32_t colb = n0 + c0 + 4 * piece;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            if (ps8[i] < 0 || colb >= N) continue;
                            float *pr = ep.push_dst + (int64_t)ps8[i] * ep.ld_push;
                            const int rr = (lane >> 3) + 4 * i;
                            const uint4 x = *reinterpret_cast<const uint4 *>(obuf + rr * 128 + ((piece ^ (rr & 7)) << 4));
                            if (colb + 3 < N) {
                                *reinterpret_cast<uint4 *>(pr + colb) = x;
                            } else {
                                pr[colb] = __uint_as_float(x.x);
                                if (colb + 1 < N) pr[colb + 1] = __uint_as_float(x.y);
                                if (colb + 2 < N) pr[colb + 2] = __uint_as_float(x.z);
                            }
                        }
                    }
                } else if (row_ok) {
#pragma unroll
                    for (int j4 = 0; j4 < 32; j4 += 4) {
                        const int32_t colb = n0 + c0 + j4;
                        if (vec && colb + 3 < N) {
                            *reinterpret_cast<uint4 *>(crow + colb) = make_uint4(r[j4], r[j4 + 1], r[j4 + 2], r[j4 + 3]);
                        } else {
#pragma unroll
                            for (int jj = 0; jj < 4; ++jj)
                                if (colb + jj < N) crow[colb + jj] = __uint_as_float(r[j4 + jj]);
                        }
                    }
                }
                if ((EPI == EPI_PLAIN || EPI == EPI_PUSH) && ep.mask_out && row_ok) {
                    const int32_t word = (n0 + c0) >> 5;
                    if (word < ep.mask_words) ep.mask_out[row * ep.mask_words + word] = bits;
                }
            }
            tc_fence_before();
            mbar_arrive(&sh->acc_empty[buf]);  // the accumulator buffer may be overwritten by the tile after next
        }
        if (use_tma_store && lane == 0) tma_store_wait_all();
        if (RING > 0) cp_async_wait<0>();
    }
done:
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// =====================================================================================
// MN-major kernel (weight gradient): block (x, y, z) = tile (x, y) of A^T B over rows [z * rps, (z + 1) * rps)
// =====================================================================================
__global__ void __launch_bounds__(TC_THREADS, 2)
k_gemm_tc_mn(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB, int32_t Mdim, int32_t N, int64_t rps,
             int32_t bn, int32_t stages, int32_t tmem_cols, float *part_C, int *status)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t blk_bytes = TC_BK * 128;                // one 32-column block of a k-block: 16 rows x 128 B
    const int n_blks_b = (bn + 31) / 32;
    const uint32_t a_bytes = (TC_BM / 32) * blk_bytes;     // one plane of A: 128 columns
    const uint32_t b_bytes = (uint32_t)n_blks_b * blk_bytes;
    const uint32_t stage_bytes = 2 * a_bytes + 2 * b_bytes;  // [A hi | A lo | B hi | B lo]
    TcShared *sh = (TcShared *)(smem + (size_t)stages * stage_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int32_t m0 = blockIdx.x * TC_BM;
    const int32_t n0 = blockIdx.y * bn;
    const int64_t r0 = (int64_t)blockIdx.z * rps;
    const int32_t nkb = (int32_t)(rps / TC_BK);

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&sh->full[s], 1);
            mbar_init(&sh->conv[s], TC_CONV_THREADS);
            mbar_init(&sh->empty[s], 1);
        }
        mbar_init(&sh->accum, 1);
        sh->dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"((uint32_t)tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;
    volatile int *dead = &sh->dead;

    if (warp == 0) {
        if (lane == 0) {
            for (int32_t kb = 0; kb < nkb; ++kb) {
                const int s = kb % stages;
                const uint32_t ph = (uint32_t)(kb / stages) & 1u;
                if (!mbar_wait(&sh->empty[s], ph ^ 1u, dead, status)) break;
                uint8_t *st = smem + (size_t)s * stage_bytes;
                const int32_t r = (int32_t)(r0 + (int64_t)kb * TC_BK);
                mbar_expect_tx(&sh->full[s], a_bytes + b_bytes);
                for (int bl = 0; bl < TC_BM / 32; ++bl) tma_load_2d(st + bl * blk_bytes, &mapA, &sh->full[s], m0 + bl * 32, r);
                for (int bl = 0; bl < n_blks_b; ++bl) tma_load_2d(st + 2 * a_bytes + bl * blk_bytes, &mapB, &sh->full[s], n0 + bl * 32, r);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = make_idesc(bn, 1, 1);
            for (int32_t kb = 0; kb < nkb; ++kb) {
                const int s = kb % stages;
                const uint32_t ph = (uint32_t)(kb / stages) & 1u;
                // the converters arrive on conv[s] only after they have seen full[s] (the TMA bytes) themselves
                if (!mbar_wait(&sh->conv[s], ph, dead, status)) break;
                tc_fence_after();
                const uint32_t st = smem_u32(smem + (size_t)s * stage_bytes);
#pragma unroll
                for (int ks = 0; ks < TC_BK / 8; ++ks) {
                    // MN-major 32-bit operands use the 128-byte swizzle with 32-byte atoms (the only layout the tensor core
                    // accepts for them): 32-column blocks blk_bytes apart (leading offset), groups of 4 k-rows 512 B apart
                    // (stride offset); a k-step is 8 rows = 1024 B
                    const uint32_t koff = ks * 1024;
                    const uint64_t a_hi = make_desc(st + koff, blk_bytes, 512, 1);
                    const uint64_t a_lo = make_desc(st + a_bytes + koff, blk_bytes, 512, 1);
                    const uint64_t b_hi = make_desc(st + 2 * a_bytes + koff, blk_bytes, 512, 1);
                    const uint64_t b_lo = make_desc(st + 2 * a_bytes + b_bytes + koff, blk_bytes, 512, 1);
                    tc_mma(tmem, a_hi, b_hi, idesc, (kb > 0 || ks > 0) ? 1u : 0u);
                    tc_mma(tmem, a_hi, b_lo, idesc, 1u);
                    tc_mma(tmem, a_lo, b_hi, idesc, 1u);
                }
                tc_commit(&sh->empty[s]);
            }
            tc_commit(&sh->accum);
        }
    } else {
        const int ctid = threadIdx.x - 64;
        bool alive = true;
        for (int32_t kb = 0; kb < nkb && alive; ++kb) {
            const int s = kb % stages;
            const uint32_t ph = (uint32_t)(kb / stages) & 1u;
            alive = mbar_wait(&sh->full[s], ph, dead, status);
            if (!alive) break;
            uint8_t *st = smem + (size_t)s * stage_bytes;
            split_tile_round(st, st + a_bytes, a_bytes, ctid, TC_CONV_THREADS);
            split_tile_round(st + 2 * a_bytes, st + 2 * a_bytes + b_bytes, b_bytes, ctid, TC_CONV_THREADS);
            fence_async_smem();
            mbar_arrive(&sh->conv[s]);
        }
        const int q = warp & 3;
        const int32_t row = m0 + q * 32 + lane;
        const bool ok = alive && mbar_wait(&sh->accum, 0, dead, status);
        tc_fence_after();
        if (ok) {
            float *pc = part_C + (int64_t)blockIdx.z * Mdim * N;
            for (int c0 = 0; c0 < bn; c0 += 32) {
                uint32_t r[32];
                tc_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
                if (row >= Mdim) continue;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int32_t col = n0 + c0 + j;
                    if (col < N) pc[(int64_t)row * N + col] = __uint_as_float(r[j]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)tmem_cols) : "memory");
    }
}

// =====================================================================================
// element-wise helpers
// =====================================================================================
// D = src o mask (written only when `dst` is non-null) and per-block column sums of it for the bias gradient.
// A block covers MASK_ROWS_PER_BLOCK rows; TPR threads (a power of two >= d / 4) walk one row with 128-bit accesses,
// 256 / TPR rows per pass; each thread keeps the running sum of its four columns, the row groups are added through
// shared memory in fixed order.
#define MASK_ROWS_PER_BLOCK 256
__global__ void __launch_bounds__(256)
k_mask_rows(const float *__restrict__ src, int64_t ld, int64_t rows, int32_t d, int32_t tpr, const uint32_t *__restrict__ mask,
            int32_t mask_words, float *__restrict__ dst, int64_t ld_dst, float *__restrict__ colsum_part)
{
    __shared__ float4 red[256];
    const int c4 = threadIdx.x % tpr, rg = threadIdx.x / tpr, n_rg = 256 / tpr;
    const int64_t r0 = (int64_t)blockIdx.x * MASK_ROWS_PER_BLOCK;
    const int64_t r1 = (r0 + MASK_ROWS_PER_BLOCK < rows) ? r0 + MASK_ROWS_PER_BLOCK : rows;
    const int d4 = (d + 3) / 4;
    for (int cb = 0; cb < d4; cb += tpr) {  // column blocks (one unless d > 1024)
        const int c = cb + c4;
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < d4) {
            // four rows in flight per thread (the loop is latency-bound otherwise); the sums are taken in row order
            for (int64_t r = r0 + rg; r < r1; r += 4 * n_rg) {
                float4 x[4];
                uint32_t w[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int64_t rr = r + (int64_t)u * n_rg;
                    x[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    w[u] = 0xFu;
                    if (rr < r1) {
                        x[u] = __ldg(reinterpret_cast<const float4 *>(src + rr * ld) + c);
                        if (mask) w[u] = __ldg(mask + rr * mask_words + (c >> 3)) >> ((c & 7) * 4);
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int64_t rr = r + (int64_t)u * n_rg;
                    if (rr >= r1) break;
                    if (!(w[u] & 1u)) x[u].x = 0.f;
                    if (!(w[u] & 2u)) x[u].y = 0.f;
                    if (!(w[u] & 4u)) x[u].z = 0.f;
                    if (!(w[u] & 8u)) x[u].w = 0.f;
                    if (4 * c + 3 >= d) {  // ragged tail: keep the padding columns out of the sums
                        if (4 * c + 1 >= d) x[u].y = 0.f;
                        if (4 * c + 2 >= d) x[u].z = 0.f;
                        x[u].w = 0.f;
                    }
                    if (dst) *(reinterpret_cast<float4 *>(dst + rr * ld_dst) + c) = x[u];
                    s.x += x[u].x; s.y += x[u].y; s.z += x[u].z; s.w += x[u].w;
                }
            }
        }
        if (colsum_part) {
            red[threadIdx.x] = s;
            __syncthreads();
            if (rg == 0 && c < d4) {
                float4 t = red[c4];
                for (int g = 1; g < n_rg; ++g) {
                    const float4 y = red[g * tpr + c4];
                    t.x += y.x; t.y += y.y; t.z += y.z; t.w += y.w;
                }
                float *o = colsum_part + (int64_t)blockIdx.x * d + 4 * c;
                o[0] = t.x;
                if (4 * c + 1 < d) o[1] = t.y;
                if (4 * c + 2 < d) o[2] = t.z;
                if (4 * c + 3 < d) o[3] = t.w;
            }
            __syncthreads();
        }
    }
}

// zero-padded bias for the tile width (optionally with the same gate interleave as the weights)
__global__ void k_pack_bias(const float *__restrict__ bias, int32_t n, int32_t n_pad, int32_t gate_h, float *__restrict__ out)
{
    const int32_t np = blockIdx.x * blockDim.x + threadIdx.x;
    if (np >= n_pad) return;
    const int32_t nn = gate_h > 0 ? (np & 3) * gate_h + (np >> 2) : np;
    out[np] = np < n ? bias[nn] : 0.f;
}

// B operand [n_pad x k_pad] (K-major fp32, zero padded) from fp32 weights; the TF32 split happens in the GEMM kernel.
//   transpose = 1: W is [K x N] row-major (ldw) -> B[n][k] = W[k][n]          (C = A W)
//   transpose = 0: W is [N x K] row-major (ldw) -> B[n][k] = W[n][k]          (C = A W^T)
// A second source W2 (same orientation, k2 rows) continues along K at column offset k1_pad.
__global__ void k_split_weights(const float *__restrict__ W, int64_t ldw, int32_t k1, int32_t k1_pad, const float *__restrict__ W2,
                                int64_t ldw2, int32_t k2, int32_t n, int32_t n_pad, int32_t k_pad, int transpose, int32_t gate_h,
                                float *__restrict__ hi, float *__restrict__ lo)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)n_pad * k_pad) return;
    const int32_t np = (int32_t)(i / k_pad), kk = (int32_t)(i - (int64_t)np * k_pad);
    const int32_t nn = gate_h > 0 ? (np & 3) * gate_h + (np >> 2) : np;  // packed row -> logical column
    float x = 0.f;
    if (np < n) {
        if (kk < k1) x = transpose ? W[(int64_t)kk * ldw + nn] : W[(int64_t)nn * ldw + kk];
        else if (kk >= k1_pad && kk - k1_pad < k2) x = transpose ? W2[(int64_t)(kk - k1_pad) * ldw2 + nn] : W2[(int64_t)nn * ldw2 + (kk - k1_pad)];
    }
    hi[i] = x;
    lo[i] = tf32_residual(x);  // second plane: read by the variants that do not split B in the kernel
}

// =====================================================================================
// host side
// =====================================================================================
typedef CUresult (*PFN_encodeTiled)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                    const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static PFN_encodeTiled get_encode()
{
    static PFN_encodeTiled fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (PFN_encodeTiled)p;
    }
    return fn;
}

// 2-D fp32 tensor map: `inner` contiguous elements per row, `outer` rows `ld` elements apart
static sat_status make_map(sat_ctx *ctx, CUtensorMap *map, const void *base, int64_t inner, int64_t outer, int64_t ld, int box_inner,
                           int box_outer, CUtensorMapSwizzle swz)
{
    PFN_encodeTiled enc = get_encode();
    if (!enc) return sat_fail(ctx, SAT_ECUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t gdim[2] = {(cuuint64_t)(inner > 0 ? inner : 1), (cuuint64_t)(outer > 0 ? outer : 1)};
    cuuint64_t gstr[1] = {(cuuint64_t)ld * 4};
    cuuint32_t box[2] = {(cuuint32_t)box_inner, (cuuint32_t)box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void *>(base), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return sat_fail(ctx, SAT_EINVAL, "cuTensorMapEncodeTiled failed (%d): base %p inner %lld outer %lld ld %lld", (int)r, base,
                                           (long long)inner, (long long)outer, (long long)ld);
    return SAT_OK;
}

static int tmem_cols_for(int bn) { return bn <= 32 ? 32 : bn <= 64 ? 64 : bn <= 128 ? 128 : 256; }
static int tile_n_for(int n) { return n >= 256 ? 256 : (n + 31) / 32 * 32; }

bool sat_use_tc(int32_t n, int32_t k)
{
    static int no_tc = -1;
    if (no_tc < 0) {
        const char *e = getenv("SAT_NO_TC");
        no_tc = (e && e[0] == '1') ? 1 : 0;
    }
    return !no_tc && k >= 16 && n >= 16;
}

sat_status sat_mask_rows(sat_ctx *ctx, const float *src, int32_t ld, int64_t rows, int32_t d, const uint32_t *mask, int32_t mask_words,
                         float *dst, int32_t ld_dst, float *colsum, int accumulate)
{
    if (rows == 0 || d == 0) return SAT_OK;
    if (!dst && !colsum) return SAT_OK;
    ProfScope prof(ctx, SATK_SPLIT, (dst ? 8.0 : 4.0) * (double)rows * d, 0.0);
    const int64_t blocks = cdiv64(rows, MASK_ROWS_PER_BLOCK);
    float *part = nullptr;
    if (colsum) {
        SAT_TRY(sat_ensure(ctx, ctx->buf_colsum, (size_t)blocks * d * sizeof(float)));
        part = (float *)ctx->buf_colsum.p;
    }
    int tpr = 1;
    while (tpr < (d + 3) / 4 && tpr < 256) tpr <<= 1;
    k_mask_rows<<<(unsigned)blocks, 256, 0, ctx->stream>>>(src, ld, rows, d, tpr, mask, mask_words, dst, ld_dst, part);
    SAT_LAUNCHED(ctx);
    if (colsum) SAT_TRY(sat_splitk_reduce(ctx, part, d, (int32_t)blocks, accumulate, colsum, d, d));
    return SAT_OK;
}

sat_status sat_tc_weights(sat_ctx *ctx, const float *W, int32_t ldw, int32_t k1, const float *W2, int32_t ldw2, int32_t k2, int32_t n,
                          int transpose, DevBuf &buf, TcWeights *out, int32_t gate_h)
{
    const int32_t k1_pad = W2 ? (k1 + TC_BK - 1) / TC_BK * TC_BK : k1;
    const int32_t k_tot = k1_pad + (W2 ? k2 : 0);
    const int32_t k_pad = (k_tot + TC_BK - 1) / TC_BK * TC_BK;
    const int32_t bn = tile_n_for(n);
    const int32_t n_pad = (n + bn - 1) / bn * bn;
    const size_t plane = ((size_t)n_pad * k_pad * sizeof(float) + 255) & ~(size_t)255;
    SAT_TRY(sat_ensure(ctx, buf, 2 * plane));
    out->hi = (float *)buf.p;
    out->lo = (float *)((char *)buf.p + plane);
    out->ld = k_pad;
    out->n_pad = n_pad;
    k_split_weights<<<(unsigned)cdiv64((int64_t)n_pad * k_pad, 256), 256, 0, ctx->stream>>>(W, ldw, k1, k1_pad, W2, ldw2, k2, n, n_pad, k_pad,
                                                                                          transpose, gate_h, out->hi, out->lo);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

// the description of planes that an earlier sat_tc_weights call (single source, k terms, n outputs) left in `buf`
sat_status sat_tc_weights_layout(int32_t k, int32_t n, const DevBuf &buf, TcWeights *out)
{
    const int32_t k_pad = (k + TC_BK - 1) / TC_BK * TC_BK;
    const int32_t bn = tile_n_for(n);
    const int32_t n_pad = (n + bn - 1) / bn * bn;
    const size_t plane = ((size_t)n_pad * k_pad * sizeof(float) + 255) & ~(size_t)255;
    if (!buf.p || buf.bytes < 2 * plane) return SAT_ESTATE;
    out->hi = (float *)buf.p;
    out->lo = (float *)((char *)buf.p + plane);
    out->ld = k_pad;
    out->n_pad = n_pad;
    return SAT_OK;
}

static PerDeviceOnce g_attr_mn;
#define TC_SMEM_BUDGET (100 * 1024)

struct TckLaunch {
    CUtensorMap mA, mA2, mB, mBlo, mC;
    int use_tma_store;
    int64_t m;
    int32_t n, nkb1, nkb2, bn, n_tiles_n;
    int64_t n_tiles;
    unsigned grid;
    uint32_t stage_bytes;
};

template <int EPI>
static sat_status launch_tck(sat_ctx *ctx, const TckLaunch &L, const TcEpilogue &ep)
{
    static PerDeviceOnce attr_set;
    const size_t smem = (size_t)TckCfg<EPI>::stages * L.stage_bytes + TckCfg<EPI>::out_bytes + (size_t)TckCfg<EPI>::epi_warps * TckCfg<EPI>::ring * 4096 +
                        sizeof(TcShared) + 1024;
    if (smem > 227 * 1024) return sat_fail(ctx, SAT_EINVAL, "tensor-core GEMM: shared-memory layout of %zu bytes does not fit", smem);
    if (attr_set.need(ctx->device)) {
        SAT_CUDA(ctx, cudaFuncSetAttribute(k_gemm_tc_k<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        attr_set.mark(ctx->device);
    }
    k_gemm_tc_k<EPI><<<L.grid, TCK_THREADS, smem, ctx->stream>>>(L.mA, L.mA2, L.mB, L.mBlo, L.mC, L.use_tma_store, L.m, L.n, L.nkb1, L.nkb2, L.bn, L.n_tiles_n,
                                                                L.n_tiles, ep, ctx->d_flag + 1);
    SAT_LAUNCHED(ctx);
    return SAT_OK;
}

// C[m x n] = [A | A2] B^T with B = packed weights [n_pad x k_pad]
sat_status sat_gemm_tc(sat_ctx *ctx, int64_t m, int32_t n, const float *A, int32_t lda, int32_t k1, const float *A2, int32_t lda2, int32_t k2,
                       const TcWeights &Bw, const TcEpilogueHost &eh, int family)
{
    if (m == 0 || n == 0) return SAT_OK;
    const int32_t nkb1 = (k1 + TC_BK - 1) / TC_BK, nkb2 = A2 ? (k2 + TC_BK - 1) / TC_BK : 0;
    const int32_t bn = tile_n_for(n);
    const uint32_t stage_bytes = 2 * (TC_BM * TC_BK * 4) + 2 * (uint32_t)bn * TC_BK * 4;
    // algorithmic bytes: operands once, results once.  Plain: A, B, C.  Gathered residual: + the residual rows.  LSTM cell:
    // the output is the hidden state [m x h] plus the cell state read and written, and the cached projection if it is added.
    double alg_bytes = 4.0 * ((double)m * (k1 + k2) + (double)(k1 + k2) * n);
    if (eh.lstm_h > 0) alg_bytes += 4.0 * (double)m * eh.lstm_h * (eh.lstm_first ? 2.0 : 3.0) + (eh.addend ? 4.0 * (double)m * n : 0.0);
    else alg_bytes += 4.0 * (double)m * n * (eh.resid_idx ? 2.0 : 1.0);
    ProfScope prof(ctx, family, alg_bytes, 2.0 * (double)m * n * (k1 + k2));
    CUtensorMap mA, mA2, mB, mBlo, mC;
    const int use_tma_store = eh.lstm_h == 0 && ((eh.ldc & 3) == 0) && ((((uintptr_t)eh.C) & 15u) == 0);
    if (use_tma_store) SAT_TRY(make_map(ctx, &mC, eh.C, n, m, eh.ldc, 32, 32, CU_TENSOR_MAP_SWIZZLE_128B));
    else memset(&mC, 0, sizeof(mC));
    SAT_TRY(make_map(ctx, &mA, A, k1, m, lda, TC_BK, TC_BM, CU_TENSOR_MAP_SWIZZLE_64B));
    if (A2) SAT_TRY(make_map(ctx, &mA2, A2, k2, m, lda2, TC_BK, TC_BM, CU_TENSOR_MAP_SWIZZLE_64B));
    else mA2 = mA;
    SAT_TRY(make_map(ctx, &mB, Bw.hi, Bw.ld, Bw.n_pad, Bw.ld, TC_BK, bn, CU_TENSOR_MAP_SWIZZLE_64B));
    SAT_TRY(make_map(ctx, &mBlo, Bw.lo, Bw.ld, Bw.n_pad, Bw.ld, TC_BK, bn, CU_TENSOR_MAP_SWIZZLE_64B));
    TcEpilogue ep;
    ep.C = eh.C;
    ep.ldc = eh.ldc;
    ep.bias = nullptr;
    if (eh.bias) {  // zero-padded copy so that the epilogue can read whole 128-bit vectors
        const size_t padded = (size_t)cdiv64(n, bn) * bn;
        DevBuf &home = eh.bias_home ? *eh.bias_home : ctx->buf_bias;
        if (!(eh.bias_home && eh.bias_ready && home.bytes >= padded * sizeof(float))) {
            SAT_TRY(sat_ensure(ctx, home, padded * sizeof(float)));
            k_pack_bias<<<(unsigned)cdiv64(padded, 256), 256, 0, ctx->stream>>>(eh.bias, n, (int32_t)padded, eh.lstm_h > 0 ? eh.lstm_h : eh.pack_gate_h,
                                                                                (float *)home.p);
            SAT_LAUNCHED(ctx);
        }
        ep.bias = (const float *)home.p;
    }
    ep.push_dst = eh.push_dst;
    ep.push_slot = eh.push_slot;
    ep.ld_push = eh.ld_push;
    if (eh.push_dst && (eh.lstm_h > 0 || eh.resid_idx || !eh.push_slot || (eh.ld_push & 3) || (((uintptr_t)eh.push_dst) & 15u)))
        return sat_fail(ctx, SAT_EINVAL, "push epilogue needs a slot map, an aligned destination and the plain epilogue");
    ep.lstm_h = eh.lstm_h;
    ep.lstm_first = eh.lstm_first;
    ep.lstm_c = eh.lstm_c;
    ep.addend = eh.addend;
    ep.ld_addend = eh.ld_addend;
    if (eh.lstm_h > 0 && ((!eh.bias && !eh.addend) || !eh.lstm_c || n != 4 * eh.lstm_h || (eh.addend && (eh.ld_addend & 3))))
        return sat_fail(ctx, SAT_EINVAL, "fused LSTM epilogue needs bias or addend, cell state and n = 4h");
    if (eh.resid_idx && (eh.mask_out || eh.lstm_h > 0))
        return sat_fail(ctx, SAT_EINVAL, "gathered-residual epilogue cannot be combined with a mask output or the LSTM cell");
    ep.relu = eh.relu;
    ep.mask_out = eh.mask_out;
    ep.mask_words = eh.mask_words;
    ep.resid = eh.resid;
    ep.resid_idx = eh.resid_idx;
    ep.ld_resid = eh.ld_resid;
    ep.tile_order = eh.tile_order;
    const int32_t n_tiles_n = (int32_t)cdiv64(n, bn);
    const int64_t n_tiles = cdiv64(m, TC_BM) * n_tiles_n;
    int sms = 148;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, ctx->device);
    const unsigned grid = (unsigned)(n_tiles < sms ? n_tiles : sms);
    TckLaunch L;
    L.mA = mA; L.mA2 = mA2; L.mB = mB; L.mBlo = mBlo; L.mC = mC;
    L.use_tma_store = use_tma_store;
    L.m = m; L.n = n; L.nkb1 = nkb1; L.nkb2 = nkb2; L.bn = bn; L.n_tiles_n = n_tiles_n; L.n_tiles = n_tiles;
    L.grid = grid;
    L.stage_bytes = stage_bytes;
    if (ep.lstm_h > 0) return ep.addend ? launch_tck<EPI_LSTM_ADD>(ctx, L, ep) : launch_tck<EPI_LSTM>(ctx, L, ep);
    if (ep.resid_idx) return launch_tck<EPI_RESID>(ctx, L, ep);
    if (ep.push_dst) return launch_tck<EPI_PUSH>(ctx, L, ep);
    return launch_tck<EPI_PLAIN>(ctx, L, ep);
}

// C[m x n] (+)= A^T B over `rows` rows: A fp32 [rows x m] (lda), B fp32 [rows x n] (ldb)
sat_status sat_gemm_tc_tn(sat_ctx *ctx, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B, int32_t ldb, float *C,
                          int32_t ldc, int accumulate)
{
    if (m == 0 || n == 0) return SAT_OK;
    ProfScope prof(ctx, SATK_GEMM_TN, 4.0 * ((double)rows * (m + n) + (double)m * n), 2.0 * (double)rows * m * n);
    const int32_t bn = tile_n_for(n);
    const int n_blks_b = (bn + 31) / 32;
    const uint32_t stage_bytes = 2 * ((TC_BM / 32) * TC_BK * 128) + 2 * (uint32_t)n_blks_b * TC_BK * 128;
    int stages = (int)(TC_SMEM_BUDGET / stage_bytes);
    if (stages > 4) stages = 4;
    if (stages < 2) stages = 2;
    const size_t smem = (size_t)stages * stage_bytes + sizeof(TcShared) + 1024;
    const int64_t tiles = cdiv64(m, TC_BM) * cdiv64(n, bn);
    int64_t splits = (2 * 148 + tiles - 1) / tiles;
    const int64_t max_splits = cdiv64(rows > 0 ? rows : 1, 8 * TC_BK);
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    const int64_t rps = cdiv64(cdiv64(rows > 0 ? rows : 1, splits), TC_BK) * TC_BK;
    splits = cdiv64(rows > 0 ? rows : 1, rps);
    SAT_TRY(sat_ensure(ctx, ctx->buf_splitk, (size_t)splits * m * n * sizeof(float)));
    float *part = (float *)ctx->buf_splitk.p;
    CUtensorMap mA, mB;
    SAT_TRY(make_map(ctx, &mA, A, m, rows, lda, 32, TC_BK, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B));
    SAT_TRY(make_map(ctx, &mB, B, n, rows, ldb, 32, TC_BK, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B));
    if (g_attr_mn.need(ctx->device)) {
        SAT_CUDA(ctx, cudaFuncSetAttribute(k_gemm_tc_mn, cudaFuncAttributeMaxDynamicSharedMemorySize, 110 * 1024));
        g_attr_mn.mark(ctx->device);
    }
    dim3 grid((unsigned)cdiv64(m, TC_BM), (unsigned)cdiv64(n, bn), (unsigned)splits);
    k_gemm_tc_mn<<<grid, TC_THREADS, smem, ctx->stream>>>(mA, mB, m, n, rps, bn, stages, tmem_cols_for(bn), part, ctx->d_flag + 1);
    SAT_LAUNCHED(ctx);
    return sat_splitk_reduce(ctx, part, (int64_t)m * n, (int32_t)splits, accumulate, C, n, ldc);
}
