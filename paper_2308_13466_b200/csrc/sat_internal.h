// Internal declarations of the sat_b200 library (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <stdint.h>

#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <vector>

#include "../../include/sat_b200.h"

#define SAT_MAX_LAYERS 16
#define SAT_MAX_PARTS 4096
#define SAT_SPMM_CHUNK 256 /* edges per SpMM work item */
#define SAT_HROW_LONG 256  /* halo rows with more entries than this are cut into chunks, a thread block per chunk */
#define SAT_HROW_CHUNK 2048 /* entries per chunk of a long halo row */

// Debug build (-DSAT_DEBUG_BOUNDS, libsat_b200_dbg.so): every index the graph kernels load from an index array (column ids,
// row lists, cache slots) is checked against the extent of the matrix it addresses; an index outside it raises bit 4 of
// the device status word (reported by sat_sync_status as SAT_EDATA) and is replaced by the first valid index, so the access that
// follows stays inside the matrix: no trap, no assert, the context stays usable.  The stand-in for a memory checker on these kernels.
#ifdef SAT_DEBUG_BOUNDS
#define SAT_DBG 1
#ifdef __CUDACC__
__device__ __forceinline__ int64_t sat_bound(int64_t i, int64_t lo, int64_t hi, int *status)
{
    if (i < lo || i >= hi) {
        atomicOr(status, 4);
        return lo;    // a row that exists (the kernels are not launched on empty matrices)
    }
    return i;
}
#endif
#define SAT_IDX(i, lo, hi, status) sat_bound((i), (lo), (hi), (status))
#else
#define SAT_DBG 0
#define SAT_IDX(i, lo, hi, status) (i)
#endif
// valid row indices [lo, hi) of a matrix as a kernel addresses it (a per-partition view starts above 0)
struct DbgRange {
    int64_t lo, hi;
};
// index ranges handed to the graph kernels for those checks (unused, and optimised away, in the regular build)
struct DbgLimits {
    int64_t src_lo, src_hi;     // rows of the first source matrix (inner rows / cache slots / generic source)
    int64_t halo_lo, halo_hi;   // rows of the halo source matrix
    int64_t out_lo, out_hi;     // rows of the output
    int *status;                // device status word
};
static inline DbgLimits dbg_limits(DbgRange src, DbgRange halo, DbgRange out, int *status)
{
    return DbgLimits{src.lo, src.hi, halo.lo, halo.hi, out.lo, out.hi, status};
}

// A growable device buffer owned by the context.
struct DevBuf {
    void *p = nullptr;
    size_t bytes = 0;
};

struct LayerState {
    float *agg = nullptr;      // [N x ld_in]  saved aggregation (rows in partition-major order)
    uint32_t *mask = nullptr;  // [N x mask_words] bit j of word w: Z[row][32w + j] > 0
    int32_t d_in = 0, d_out = 0, ld_in = 0, mask_words = 0;
    int act = 0;
    std::vector<uint8_t> valid;  // per partition: forward state present
};

struct CacheLayer {
    float *buf = nullptr;  // [(tau+1) x n_slots x ld]
    int32_t width = 0, ld = 0;
    float *S = nullptr;  // LSTM state table [n_slots x h]
    int32_t S_h = 0;
    bool S_valid = false;
    // input projections x Wx + b of the ring buffers (gate-interleaved columns), reused while the caller's parameter
    // version stays the same: [(tau+1) x n_slots x 4 proj_h]; proj_tag[i] = version the projection of buffer i was made with
    float *proj = nullptr;
    int32_t proj_h = 0;
    std::vector<uint64_t> proj_tag;
    // packed (TF32 hi / lo planes, padded) copies of the predictor's weights and biases, reused while the caller's
    // parameter version stays the same: input weights Wx, recurrent weights Uh, output weights Wg, gate bias b, output bias bg
    DevBuf pk_wx, pk_uh, pk_wg, pk_b, pk_bg;
    uint64_t tag_wx = 0, tag_uh = 0, tag_wg = 0, tag_b = 0, tag_bg = 0;
    int32_t pk_h = 0;
};

// Gradient-side history of one layer j >= 2 (Appendix, back-propagation of SAT): Q^(j) = sum_m P_out^(m)T D^(m, j) over the
// boundary nodes, two buffers [n_slots x ld]: buf + read_idx * plane is the previous epoch's, the other one collects the
// running epoch (zeroed at commit).
struct GradHist {
    float *buf = nullptr;
    int32_t width = 0, ld = 0, read_idx = 0;
    bool has_read = false;
};

// Saved forward state of a graph-attention layer: z = h W for all inner rows and halo positions of the graph, the attention
// scores s_src (inner, halo), s_dst and the log-sum-exp of every inner row (scal = [s_in | s_dst | lse | s_halo]).
struct GatState {
    DevBuf z_in, z_halo, scal;
    int32_t d_out = 0;
    int relu = 0;
    std::vector<uint8_t> valid;
};

// kernel families for the optional per-family device timing (sat_profile_*)
enum {
    SATK_SPMM_FWD = 0, SATK_SPMM_BWD, SATK_SPMM_HROW, SATK_GEMM_NN, SATK_GEMM_NT, SATK_GEMM_TN, SATK_LSTM_CELL,
    SATK_GATHER, SATK_SCATTER, SATK_LOSS, SATK_SPLIT, SATK_GEMM_SIDE, SATK_CODEC, SATK_PRED_TRAIN, SATK_GAT, SATK_COUNT
};

struct ProfRec {
    int family;
    cudaEvent_t a, b;
    double bytes, flops;
};

// Forward SpMM work list in source-block-major order (sat_spmm.cu).  The sources of a partition (its inner rows, then its
// halo rows) are cut into blocks of at most `block_rows` rows; the entries of every local-CSR row are sorted by source, so a
// row meets each block in one contiguous run of entries.  An item is such a run (cut further at SAT_SPMM_CHUNK entries);
// within a partition items are ordered by block, then by row, so that the rows gathered at any one time come from one or
// two blocks.  Rows with more than one item add their partial sums in item order (k_spmm_sb_fixup).
struct SrcBlockedItems {
    int64_t block_rows = 0, fit_rows = 0, min_run = 0, row_run = 0;  // key
    int mode = 0;              // key: 0 = all entries of a row, 1 = its inner prefix only (one block per partition)
    int32_t n_items = 0, n_mrows = 0;
    int64_t n_slots = 0;
    int4 *item = nullptr;      // {row, partial slot or -1, first entry: low 32 bits, first entry: high 16 bits | entries << 16}
    int32_t *slot0 = nullptr;  // [n] first partial slot of a row with several items
    int32_t *tot = nullptr;    // [n] items of the row
    int32_t *mrows = nullptr;  // [n_mrows] rows with several items
    std::vector<int32_t> h_item_off, h_mrow_off;  // [M+1] per partition
    std::vector<int64_t> h_slot_off;              // [M+1]
};

struct sat_ctx {
    bool prof_on = false;
    uint64_t prof_mask = ~0ull;  // families that are bracketed while prof_on
    std::vector<ProfRec> prof;
    int device = 0;
    cudaStream_t stream = nullptr;
    char err[512] = {0};
    bool cuda_failed = false;
    int64_t launches = 0;
    int *d_flag = nullptr;  // device status word used by validation kernels
    int *h_flag = nullptr;  // pinned host mirror

    // ---- graph ----
    bool graph_ok = false;
    int32_t n = 0;
    int64_t nnz = 0;  // stored directed edges (no self-loops)
    int64_t *rowptr = nullptr;
    int32_t *col = nullptr;
    float *dinv = nullptr;

    // ---- partition ----
    bool part_ok = false;
    int32_t M = 0;
    int32_t *part = nullptr;      // [n]
    int32_t *perm = nullptr;      // [n]   inner global ids, partition-major (= concatenated I_m)
    int32_t *pos = nullptr;       // [n]   inverse of perm
    int32_t *halo_gid = nullptr;  // [nb]  concatenated B_m
    int32_t *halo_slot = nullptr; // [nb]
    int32_t *slot = nullptr;      // [n]
    int32_t n_slots = 0;
    int64_t nb = 0;               // sum_m b_m
    int32_t *push_row = nullptr;  // [n_slots] partition-major row index of every boundary node
    int32_t *push_slot = nullptr; // [n_slots]
    int32_t *row_slot = nullptr;  // [n] cache slot of every partition-major row, -1 for interior nodes (built on first use)
    int64_t *lrowptr = nullptr;   // [n+1] local CSR, rows partition-major
    int32_t *lenc = nullptr;      // [nnz+n] encoded column: < n: partition-major row of an inner node; >= n: n + halo position
    int32_t *lenc_gid = nullptr;  // [nnz+n] the same with halo columns as n + global node id (built on first use: SAT_FWD_HALO_GLOBAL)
    int32_t *lenc_all_gid = nullptr; // [nnz+n] every column as a global node id (built on first use: SAT_FWD_INPUT_GLOBAL)
    std::vector<SrcBlockedItems> src_blocked;  // source-blocked forward work lists, one per block size (built on first use)
    int32_t *inner_cnt = nullptr; // [n] number of inner entries (incl. self-loop) at the front of each row
    float *dinv_enc = nullptr;    // [n + nb] dinv of the node behind each encoded column
    float *lw = nullptr;          // [nnz+n] dinv_enc[lenc[e]] stored per entry (read with the column instead of gathered)
    int64_t *hrow_ptr = nullptr;  // [nb+1] halo-row CSR
    int32_t *hrow_pos = nullptr;  // [nnz_cut] partition-major row of the inner neighbour
    int32_t *hrow_slot = nullptr; // [nnz_cut] its cache slot
    float *hrow_w = nullptr;      // [nnz_cut] its dinv (the entry's weight up to the row's own dinv)
    int64_t nnz_cut = 0;
    int64_t *hs_ptr = nullptr;    // [n_slots+1] halo positions by cache slot (built on first use): slot s is the halo node at
    int32_t *hs_pos = nullptr;    // [nb]        positions hs_pos[hs_ptr[s] .. hs_ptr[s+1]), in ascending partition order
    int32_t *hlong = nullptr;     // [n_hlong] halo positions of the halo rows longer than SAT_HROW_LONG
    int32_t n_hlong = 0;
    std::vector<int32_t> h_hlong_off;
    // the long halo rows cut into chunks of SAT_HROW_CHUNK entries (a hub next to most of a partition has tens of thousands)
    int64_t *hchunk_first = nullptr; // [n_hlong+1] first chunk of every long row
    int32_t *hchunk_row = nullptr;   // [n_hchunks] index into hlong[] of the row a chunk belongs to
    int32_t *halo_tile_order = nullptr;  // [ceil(n_halo / 128)] tiles of 128 halo rows ordered by the cache slot of their first row (built on first use)
    int32_t n_hchunks = 0;
    std::vector<int32_t> h_hchunk_off;  // [M+1] first chunk of every partition
    // SpMM work items (rows cut into chunks of SAT_SPMM_CHUNK edges)
    int32_t *first_item = nullptr; // [n+1]
    int32_t *item_row = nullptr;   // [n_items]
    int32_t *item_mslot = nullptr; // [n_items] index of the partial-sum row for items of multi-chunk rows, else -1
    int32_t *mrows = nullptr;      // [n_mrows] rows with more than one chunk
    int32_t n_items = 0, n_mrows = 0, n_mitems = 0;
    std::vector<int32_t> h_inner_off, h_push_off, h_item_off, h_mrow_off, h_mitem_off;
    std::vector<int64_t> h_halo_off, h_lnnz_off, h_hrow_off;

    // ---- cache ----
    bool cache_ok = false;
    int32_t n_cached = 0, tau = 0, write_idx = 0, n_valid = 0;
    CacheLayer cache[SAT_MAX_LAYERS];

    // ---- layers ----
    LayerState layers[SAT_MAX_LAYERS + 1];
    GradHist ghist[SAT_MAX_LAYERS + 1];
    GatState gat[SAT_MAX_LAYERS + 1];

    // ---- scratch ----
    DevBuf buf_codec_sizes, buf_codec_off, buf_codec_bytes;  // embedding codec scratch
    DevBuf buf_hpartial, buf_sbpartial;
    DevBuf buf_partial, buf_gagg, buf_splitk, buf_lstm_c, buf_lstm_s, buf_lstm_w, buf_pred_a, buf_misc, buf_colsum, buf_dmask,
        buf_wsplit, buf_wsplit2, buf_wsplit3, buf_bias, buf_pred_train, buf_ghist_halo, buf_ghist_rows, buf_ghist_out, buf_gat, buf_gat_items;
};

sat_status sat_fail(sat_ctx *ctx, sat_status code, const char *fmt, ...);
sat_status sat_check_cuda(sat_ctx *ctx, cudaError_t e, const char *what);
sat_status sat_ensure(sat_ctx *ctx, DevBuf &b, size_t bytes);
void sat_free_buf(DevBuf &b);

#define SAT_CUDA(ctx, call)                                          \
    do {                                                             \
        cudaError_t e__ = (call);                                    \
        if (e__ != cudaSuccess) return sat_check_cuda(ctx, e__, #call); \
    } while (0)

#define SAT_TRY(expr)                   \
    do {                                \
        sat_status s__ = (expr);        \
        if (s__ != SAT_OK) return s__;  \
    } while (0)

// Counts the launch and checks the launch error.
#define SAT_LAUNCHED(ctx)                                                     \
    do {                                                                      \
        (ctx)->launches++;                                                    \
        cudaError_t e__ = cudaGetLastError();                                 \
        if (e__ != cudaSuccess) return sat_check_cuda(ctx, e__, "kernel launch"); \
    } while (0)

// Brackets the launches of one kernel family with CUDA events on the context's stream when profiling is on.
struct ProfScope {
    sat_ctx *ctx;
    ProfRec rec;
    bool on;
    ProfScope(sat_ctx *c, int family, double bytes, double flops) : ctx(c), on(c->prof_on && ((c->prof_mask >> family) & 1ull))
    {
        if (!on) return;
        rec.family = family;
        rec.bytes = bytes;
        rec.flops = flops;
        if (cudaEventCreate(&rec.a) != cudaSuccess || cudaEventCreate(&rec.b) != cudaSuccess) {
            on = false;
            return;
        }
        cudaEventRecord(rec.a, ctx->stream);
    }
    ~ProfScope()
    {
        if (!on) return;
        cudaEventRecord(rec.b, ctx->stream);
        ctx->prof.push_back(rec);
    }
};

// NVTX range around an entry point (named after the function): shows the library's calls on a profiler's timeline; costs
// a few nanoseconds when no tool is attached
struct SatRange {
    explicit SatRange(const char *name) { nvtxRangePushA(name); }
    ~SatRange() { nvtxRangePop(); }
    SatRange(const SatRange &) = delete;
    SatRange &operator=(const SatRange &) = delete;
};

// entry-point prologue: an NVTX range for the call, and a usable context on its device
#define CHECK_CTX(ctx)                                                                             \
    SatRange sat_range__(__func__);                                                                \
    do {                                                                                           \
        if (!(ctx)) return SAT_EINVAL;                                                             \
        if ((ctx)->cuda_failed) return sat_fail(ctx, SAT_ECUDA, "context has a sticky CUDA error"); \
        SAT_CUDA(ctx, cudaSetDevice((ctx)->device));                                               \
    } while (0)

// argument checks of the entry points: 16-byte aligned base, leading dimension >= width and a multiple of 4 floats
static inline bool aligned16(const void *p) { return (((uintptr_t)p) & 15u) == 0; }
static inline bool ok_ld(int32_t ld, int32_t d) { return ld >= d && (ld & 3) == 0; }
// ring buffer `age` epochs back from the newest committed snapshot (age 0), and its base address
static inline int32_t ring_index(const sat_ctx *ctx, int32_t age) { return ((ctx->write_idx - 1 - age) % (ctx->tau + 1) + (ctx->tau + 1)) % (ctx->tau + 1); }
static inline float *ring_buf(const sat_ctx *ctx, const CacheLayer *c, int32_t idx) { return c->buf + (size_t)idx * ctx->n_slots * c->ld; }

static inline int64_t cdiv64(int64_t a, int64_t b) { return (a + b - 1) / b; }

// One-time per-device set-up of a kernel (cudaFuncSetAttribute applies to the current device only): a bit per device
// ordinal; devices beyond 63 simply repeat the (idempotent) set-up on every launch.
struct PerDeviceOnce {
    std::atomic<uint64_t> done{0};
    bool need(int dev) const { return dev < 0 || dev >= 64 || !((done.load(std::memory_order_acquire) >> dev) & 1ull); }
    void mark(int dev)
    {
        if (dev >= 0 && dev < 64) done.fetch_or(1ull << dev, std::memory_order_release);
    }
};
static inline int32_t round_up4(int32_t x) { return (x + 3) & ~3; }

// ---- device-side helpers implemented in the .cu files ----
// exclusive scan: out[i] = sum_{j<i} in[j], i = 0..count (count+1 outputs), int64 results
sat_status sat_scan_i32(sat_ctx *ctx, const int32_t *in, int64_t count, int64_t *out);

// embedding codec (sat_codec.cu): encode + decode of one matrix in place; *bytes (host, nullable) = encoded size
sat_status sat_codec_roundtrip(sat_ctx *ctx, float *x, int32_t ld, int64_t rows, int32_t d, int32_t precision, int64_t *bytes);

// row range / bases of a partition selector
struct PartView {
    int32_t row0, n_rows;     // partition-major rows
    int64_t halo0, n_halo;    // halo positions
    int32_t item0, n_items;   // SpMM work items
    int32_t mrow0, n_mrows;   // multi-chunk rows
    int32_t mitem0, n_mitems; // partial-sum rows
    int32_t push0, n_push;
    int32_t hlong0, n_hlong;  // long halo rows
    int32_t hchunk0, n_hchunks; // their chunks
    int64_t lnnz;             // local non-zeros (entries of A + I) of the selected rows
    int64_t hnnz;             // of which entries with a halo column (= entries of the halo-row CSR)
};
sat_status sat_part_view(sat_ctx *ctx, int32_t part, PartView *v);

// SpMM family (sat_spmm.cu)
//   out[row] = dinv[row] * sum_e dinv[col_e] * src(col_e), over all entries of the row (inner_only = 0)
//   or over its inner prefix (inner_only = 1), or over its halo suffix (inner_only = 2; in_base is not read).  `in_base` / `halo_base` are the virtual bases of the
//   partition-major inner matrix and of the concatenated halo matrix (already offset for a single
//   partition); `out_base` likewise.
// omask (or null): bit mask [rows x omask_words] indexed like out_base; output components whose bit is 0 are written as 0
// halo_global: the halo columns address a matrix over all n nodes in global id order (halo_base = its first row);
// in_global: inner and halo columns both address such a matrix (in_base = its first row; halo_base is not used)
sat_status sat_spmm(sat_ctx *ctx, const PartView &v, int inner_only, int32_t d, const float *in_base, int32_t ld_in,
                    const float *halo_base, int32_t ld_halo, float *out_base, int32_t ld_out, const uint32_t *omask = nullptr,
                    int32_t omask_words = 0, bool halo_global = false, bool in_global = false);
//   halo-row products: out[j] = sum_{e in hrow(j)} dinv[halo j] dinv[inner e] * src[pos_e]   (+ self term if self_src)
sat_status sat_spmm_hrow(sat_ctx *ctx, const PartView &v, int32_t d, const float *src_base, int32_t ld_src,
                         int by_slot, const float *self_src, float *out_base, int32_t ld_out);
// src_rows / dst_rows: valid row indices of the source / destination matrices, used by the debug build's index checks
// (SAT_ANY_ROW: unknown, not checked)
static const DbgRange SAT_ANY_ROW = {INT64_MIN, INT64_MAX};
sat_status sat_gather(sat_ctx *ctx, const int32_t *idx, int64_t count, int32_t d, const float *src, int32_t ld_src,
                      float *out, int32_t ld_out, DbgRange src_rows = SAT_ANY_ROW);
sat_status sat_scatter(sat_ctx *ctx, const int32_t *src_row, const int32_t *dst_row, int64_t count, int32_t d,
                       const float *src_base, int32_t ld_src, float *dst, int32_t ld_dst, DbgRange src_rows = SAT_ANY_ROW,
                       DbgRange dst_rows = SAT_ANY_ROW);
// out[s] (+)= scale_s * sum over the halo positions p of cache slot s, in ascending partition order, of src[p]; scale_s = p_ss
// (the self-loop weight of the node behind the slot) when self_scale, else 1.  One writer per slot: no atomics, fixed order.
sat_status sat_sum_by_slot(sat_ctx *ctx, int32_t d, const float *src, int32_t ld_src, int self_scale, int add, float *out, int32_t ld_out);
// dst[dst_row[i]] += src[src_row ? src_row[i] : i] (o mask bits of the destination row, when given); the dst_row[i] of one
// call must be distinct
sat_status sat_scatter_add(sat_ctx *ctx, const int32_t *src_row, const int32_t *dst_row, int64_t count, int32_t d, const float *src_base,
                           int32_t ld_src, float *dst, int32_t ld_dst, const uint32_t *mask, int32_t mask_words, DbgRange src_rows = SAT_ANY_ROW,
                           DbgRange dst_rows = SAT_ANY_ROW);

// GEMM family (sat_gemm.cu)
// C[m x n] = A[m x k] B[k x n] (+ bias) with optional ReLU, sign-mask output, row-gathered residual add.
struct GemmEpilogue {
    const float *bias = nullptr;       // [n]
    int relu = 0;
    uint32_t *mask_out = nullptr;      // [m x mask_words] bit = (z > 0)
    int32_t mask_words = 0;
    const float *resid = nullptr;      // C += resid[resid_idx[i]] (row gather), ld_resid
    const int32_t *resid_idx = nullptr;
    int32_t ld_resid = 0;
};
sat_status sat_gemm_nn(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const float *B,
                       int32_t ldb, float *C, int32_t ldc, const GemmEpilogue &ep);
// C[m x n] = (A o mask)[m x k] B^T, B stored [n x k] row-major (ldb); mask may be null
sat_status sat_gemm_nt(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const uint32_t *mask,
                       int32_t mask_words, const float *B, int32_t ldb, float *C, int32_t ldc);
// C[m x n] (+)= A^T (B o mask): A [rows x m] (lda), B [rows x n] (ldb); colsum[n] (+)= 1^T (B o mask) if non-null.
sat_status sat_gemm_tn(sat_ctx *ctx, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B,
                       int32_t ldb, const uint32_t *mask, int32_t mask_words, float *C, int32_t ldc, float *colsum,
                       int accumulate);

// out[r][c] (+)= sum_z part[z][r * ncols + c], z ascending (fixed order: reproducible)
sat_status sat_gemm_tn_narrow(sat_ctx *ctx, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B, int32_t ldb,
                              float *C, int32_t ldc, int accumulate);
sat_status sat_splitk_reduce(sat_ctx *ctx, const float *part, int64_t count, int32_t splits, int accumulate, float *out, int32_t ncols,
                             int32_t ld_out);

// GEMM family on the tensor cores (sat_gemm_tc.cu): TF32 two-term split, fp32 operands in global memory
// Cell state of the fused LSTM (internal scratch, never exposed): blocks of [32 rows x 8 units] = 1 KB, block index
// (row / 32) * ceil(h / 8) + unit / 8.  A warp of the GEMM epilogue (one row per lane, 8 units per chunk) then reads and
// writes one contiguous KB instead of 32 separate cache lines.
__host__ __device__ inline int64_t sat_cell_offset(int64_t row, int32_t j, int32_t h)
{
    return (((row >> 5) * ((h + 7) >> 3) + (j >> 3)) << 8) + ((row & 31) << 3) + (j & 7);
}
inline size_t sat_cell_floats(int64_t rows, int32_t h) { return (size_t)((rows + 31) / 32) * ((h + 7) / 8) * 256; }

#ifdef __CUDACC__
// logistic and tanh from the hardware base-2 exponential and reciprocal (ex2.approx / rcp.approx, flush-to-zero forms:
// one instruction each): absolute error of a few 1e-7, which is what matters for gate values in [0, 1] / [-1, 1].  Four and
// five instructions per value; the LSTM epilogue is bound by instruction issue, so the libm versions (and even __expf /
// __fdividef, which carry range handling) cost more than the memory traffic of the step.
__device__ __forceinline__ float ex2_fast(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcp_fast(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float sigmoid_fast(float x) { return rcp_fast(1.f + ex2_fast(-1.4426950408889634f * x)); }
// tanh x = 1 - 2 / (1 + e^{2x}); saturates correctly (e -> inf gives 1, e -> 0 gives -1)
__device__ __forceinline__ float tanh_fast(float x) { return fmaf(-2.f, rcp_fast(1.f + ex2_fast(2.8853900817779268f * x)), 1.f); }
#endif

struct TcWeights {         // weight operand as two fp32 planes [n_pad x ld] holding the TF32 hi / lo terms, K-major
    float *hi = nullptr, *lo = nullptr;
    int32_t ld = 0, n_pad = 0;
};
struct TcEpilogueHost {
    float *C = nullptr;
    int32_t ldc = 0;
    const float *bias = nullptr;
    int relu = 0;
    uint32_t *mask_out = nullptr;
    int32_t mask_words = 0;
    const float *resid = nullptr;      // C += resid[resid_idx[i]] (row gather)
    const int32_t *resid_idx = nullptr;
    int32_t ld_resid = 0;
    // order in which the persistent kernel walks the tiles of 128 rows: [ceil(m / 128)] row-tile indices, a permutation
    // (null: ascending).  Results do not depend on it; it decides which rows are in flight together.
    const int32_t *tile_order = nullptr;
    // fused LSTM cell (the weights must have been packed with gate interleave): the n = 4h outputs of a row are the gate
    // pre-activations; the epilogue applies c = f c + i g, s = o tanh(c) and writes s to C [m x h] and c to lstm_c [m x h]
    int32_t lstm_h = 0;
    int lstm_first = 0;                // first step: previous cell state is zero
    float *lstm_c = nullptr;
    const float *addend = nullptr;     // dense [m x ld_addend], added to the accumulators before the LSTM cell (row-aligned)
    int32_t ld_addend = 0;
    int32_t pack_gate_h = 0;           // > 0: the bias is interleaved like weights packed with gate_h (without the LSTM epilogue)
    // second destination of the rows that have a cache slot (the push of Algorithm 1 fused into the layer transform):
    // row i also goes to push_dst + push_slot[i] * ld_push when push_slot[i] >= 0
    float *push_dst = nullptr;
    const int32_t *push_slot = nullptr;
    int32_t ld_push = 0;
    // optional home of the padded bias copy (default: a scratch buffer of the context, repacked by every call); with
    // bias_ready the copy in *bias_home is current and is used as it is
    DevBuf *bias_home = nullptr;
    bool bias_ready = false;
};
// tensor-core path on / off for a contraction with n outputs and k terms (SAT_NO_TC=1 in the environment forces the CUDA cores)
bool sat_use_tc(int32_t n, int32_t k);
// dst = src o mask (skipped when dst is null) and colsum (+)= 1^T (src o mask) (skipped when colsum is null)
sat_status sat_mask_rows(sat_ctx *ctx, const float *src, int32_t ld, int64_t rows, int32_t d, const uint32_t *mask, int32_t mask_words,
                         float *dst, int32_t ld_dst, float *colsum, int accumulate);
// weight planes in `buf`; transpose = 1 for W given as [K x N], 0 for [N x K]; optional second source continuing along K
// gate_h > 0: the n = 4 gate_h columns (gate blocks i | f | g | o) are interleaved so that packed column 4 j + gate is gate `gate`
// of hidden unit j (what the fused LSTM epilogue expects)
sat_status sat_tc_weights(sat_ctx *ctx, const float *W, int32_t ldw, int32_t k1, const float *W2, int32_t ldw2, int32_t k2, int32_t n,
                          int transpose, DevBuf &buf, TcWeights *out, int32_t gate_h = 0);
sat_status sat_tc_weights_layout(int32_t k, int32_t n, const DevBuf &buf, TcWeights *out);
// C[m x n] = [A | A2] B^T (+ epilogue)
sat_status sat_gemm_tc(sat_ctx *ctx, int64_t m, int32_t n, const float *A, int32_t lda, int32_t k1, const float *A2, int32_t lda2, int32_t k2,
                       const TcWeights &Bw, const TcEpilogueHost &eh, int family);
// C[m x n] (+)= A^T B over `rows` rows
sat_status sat_gemm_tc_tn(sat_ctx *ctx, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B, int32_t ldb, float *C,
                          int32_t ldc, int accumulate);
