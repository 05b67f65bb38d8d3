/*
 * sat_b200 — C ABI of the SAT (staleness-alleviated training, arXiv 2308.13466) hot path
 * for one NVIDIA B200 (sm_100a).
 *
 * The library holds M graph partitions of one graph on one GPU and runs, per partition
 * or for all partitions at once, the GCN layer step of historical-value training:
 * pull predicted out-of-subgraph ("halo") embeddings from the historical-embedding cache
 * (Algorithm 1, "Pull"), run the local layer forward (Eq. "sat forward"; Appendix,
 * forward of SAT), push the fresh boundary embeddings (Algorithm 1, "Push"), and run the
 * local backward (Appendix, backward equations).
 *
 * General rules
 *   - Plain C types only.  Every pointer argument says HOST or DEVICE.  Device tensors
 *     are caller-owned (allocated by the caller, e.g. through PyTorch), are never
 *     retained after the call, and must be 16-byte aligned with a leading dimension
 *     (`ld`, in floats) that is a multiple of 4 and >= the row width.
 *   - All floating tensors are fp32, row-major.
 *   - All work is enqueued on the stream given to sat_create (borrowed, not owned) and
 *     is asynchronous; argument and state errors are reported synchronously and leave
 *     the outputs untouched.
 *   - Every function returns a sat_status (0 = ok, < 0 = error) and never throws,
 *     aborts, traps or blocks indefinitely.  sat_last_error() gives a message.
 *   - `part` selects a partition m in [0, M) or SAT_ALL_PARTS (-1): all partitions in one
 *     launch, operands being the per-partition tensors concatenated in partition order
 *     (inner rows: N rows; halo rows: sum_m b_m rows).  Results are identical to the M
 *     per-partition calls.
 *   - Layer index convention: GNN layer l in 1..L consumes H^(l-1) and produces H^(l);
 *     cached layer l in 1..L-1 stores H^(l); sat_predict(layer = l) yields the halo input
 *     of GNN layer l+1.
 */
#ifndef SAT_B200_H
#define SAT_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sat_ctx sat_ctx; /* opaque; owns only library-internal device / host memory */
typedef int32_t sat_status;

enum {
    SAT_OK = 0,
    SAT_EINVAL = -1, /* bad argument: null pointer, shape, alignment, index out of range   */
    SAT_ESTATE = -2, /* call order: e.g. sat_partition before sat_graph_load                */
    SAT_ENOMEM = -3, /* device or host allocation failed                                    */
    SAT_ECUDA = -4,  /* CUDA runtime error (sticky for the context)                         */
    SAT_EDATA = -5   /* malformed graph: rowptr not monotone, column out of range, columns   */
                     /* unsorted or duplicated, self-loop stored, or graph not symmetric     */
};

enum { SAT_HOST = 0, SAT_DEVICE = 1 };                   /* where an index array lives           */
enum { SAT_ALL_PARTS = -1 };
enum { SAT_PART_GIVEN = 0, SAT_PART_CONTIG_BLOCKS = 1, SAT_PART_BFS_BLOCKS = 2 }; /* sat_partition methods */
enum { SAT_ACT_NONE = 0, SAT_ACT_RELU = 1 };
/* Flag for the `act` argument of sat_layer_fwd (act = SAT_ACT_* | SAT_FWD_PUSH): the rows of h_out that belong to boundary
 * nodes are also written into the write buffer of cached layer `layer`, exactly what sat_cache_update(part, layer, h_out)
 * does afterwards (Algorithm 1 "Push"), from the epilogue of the layer transform instead of a second pass over h_out.
 * Needs sat_cache_init with that layer cached at width d_out (SAT_ESTATE / SAT_EINVAL otherwise). */
#define SAT_FWD_PUSH 0x100
/* Flag for the `act` argument of sat_layer_fwd: h_halo is not the [b_m x ld_halo] matrix of the partition's halo rows but a
 * matrix over ALL n nodes in global id order ([n x ld_halo], e.g. the raw feature matrix for layer 1, whose out-of-subgraph
 * rows are exact and need no cache: Eq. "mini-batch" with h^(0) = x); the layer reads the halo nodes' rows from it directly,
 * which saves the sat_gather_rows pull and its [sum_m b_m x d] copy.  Same result, bit for bit, as the gathered call. */
#define SAT_FWD_HALO_GLOBAL 0x200
/* ... and SAT_FWD_INPUT_GLOBAL: h_in too is that matrix over all n nodes in global id order ([n x ld_in]; h_halo is ignored
 * and may be NULL): the in-subgraph rows are read through the partition's inner list, the out-of-subgraph rows through its
 * halo list.  For layer 1 the caller then needs neither the partition-major copy of the features nor the halo pull.  Same
 * result, bit for bit, as the call on gathered rows. */
#define SAT_FWD_INPUT_GLOBAL 0x400
enum { SAT_LOSS_SOFTMAX_CE = 0, SAT_LOSS_SIGMOID_BCE = 1 };
enum { SAT_ROWS_INNER = 0, SAT_ROWS_HALO = 1 };          /* sat_gather_rows                      */
enum { SAT_CACHE_ZERO = 0, SAT_CACHE_COPY = 1 };         /* sat_cache_init                       */

/* ---------------------------------------------------------------------------------------
 * Context
 * ------------------------------------------------------------------------------------- */

/* Creates a context on CUDA device `device`.  `cuda_stream` is a cudaStream_t (may be 0 for
 * the default stream); it is borrowed for the lifetime of the context. */
sat_status sat_create(sat_ctx **ctx, int device, void *cuda_stream);
sat_status sat_destroy(sat_ctx *ctx);
/* Message of the most recent error on this context (valid until the next call). */
const char *sat_last_error(const sat_ctx *ctx);
/* Waits for the stream and reads the device status word: SAT_ECUDA if any enqueued work failed or a tensor-core kernel
 * gave up waiting on one of its (bounded) barrier waits (sticky: the context is unusable afterwards); SAT_EDATA if
 * sat_codec_decode met a malformed row (reported once, the context stays usable). */
sat_status sat_sync_status(sat_ctx *ctx);

/* ---------------------------------------------------------------------------------------
 * sat_graph_load — the input graph G(V, E) (Preliminaries) and GCN's propagation matrix
 * P = D~^{-1/2} (A + I) D~^{-1/2}, d~_v = deg(v) + 1 (Appendix, Preliminaries: "P is the
 * propagation matrix following the definition of GCN").
 *
 *   n        number of nodes
 *   nnz      number of stored directed edges (both directions of every undirected edge;
 *            self-loops must NOT be stored — the library adds I itself)
 *   rowptr   int64 [n+1], col int32 [nnz]; HOST or DEVICE as `ptr_space` says; columns
 *            sorted ascending and unique inside a row.  The graph must be symmetric.
 * The arrays are copied; the caller may free them after the call.  The graph is validated
 * on the device (SAT_EDATA on failure; this call synchronises the stream).  Computes
 * dinv[v] = (deg(v)+1)^{-1/2}; P is never stored: p_vu = dinv[v] * dinv[u].
 * ------------------------------------------------------------------------------------- */
sat_status sat_graph_load(sat_ctx *ctx, int32_t n, int64_t nnz, const int64_t *rowptr, const int32_t *col,
                          int ptr_space);
/* Copies dinv (fp32 [n]) to HOST memory. */
sat_status sat_graph_dinv(sat_ctx *ctx, float *dinv_host);

/* ---------------------------------------------------------------------------------------
 * sat_partition — split G into M non-overlapping subgraphs G_m(V_m, E_m) (Algorithm 1,
 * "Partitioning the raw graph"; Preliminaries, "Distributed Training for GNNs") and build,
 * per partition, the 1-hop extended subgraph of Section "Embedding Predictor":
 *   I_m  inner nodes, ascending global id
 *   B_m  halo nodes = sorted unique  U_{v in V_m} N(v) \ V_m   (Eq. "communication
 *        complexity", second term)
 *   local CSR over rows I_m with entries N(v) + {v}; local column id = rank in I_m for an
 *        inner node, n_m + rank in B_m for a halo node; columns ascending (P_in | P_out of
 *        the Appendix: P = P_in + P_out)
 *   halo-row CSR: for u in B_m its neighbours inside V_m as local inner ids, ascending
 *        (= P_out^T)
 *   C = sorted union of all B_m = the nodes the cache stores; slot[v] = rank of v in C or -1
 *   push list of m: local ids (ascending) and slots of the inner nodes of m that are in C.
 * Methods: SAT_PART_GIVEN uses part_of_node (int32 [n], values in [0, M), HOST or DEVICE
 * per `ptr_space`); SAT_PART_CONTIG_BLOCKS ignores it and uses part[v] = floor(v*M/n);
 * SAT_PART_BFS_BLOCKS ignores it too: rank[v] = position of v in a breadth-first traversal (FIFO queue, start at node 0,
 * neighbours in ascending id, restart at the smallest unvisited id when the queue is empty) and part[v] =
 * floor(rank[v]*M/n); the graph is not relabelled.  That traversal runs on the host over a copy of the graph (set-up work).
 * (The paper partitions with METIS, which is a third-party tool and not part of this
 * library: pass its output through SAT_PART_GIVEN.)
 * All structures are integer and are built on the device; this call synchronises.
 * ------------------------------------------------------------------------------------- */
sat_status sat_partition(sat_ctx *ctx, int32_t M, int method, const int32_t *part_of_node, int ptr_space);

/* Sizes of partition m (any output pointer may be NULL).  m = SAT_ALL_PARTS gives totals:
 * n, sum_m b_m, nnz(A+I), |C|, number of cut-edge entries. */
sat_status sat_part_sizes(sat_ctx *ctx, int32_t m, int32_t *n_inner, int32_t *n_halo, int64_t *nnz_local,
                          int32_t *n_push, int64_t *nnz_hrow);
/* Copies the lists of partition m to HOST arrays sized by sat_part_sizes (any may be NULL):
 * inner_gid [n_inner], halo_gid [n_halo], halo_slot [n_halo], push_local [n_push],
 * push_slot [n_push], loc_rowptr int64 [n_inner+1] (starting at 0), loc_col [nnz_local],
 * hrow_ptr int64 [n_halo+1] (starting at 0), hrow_col [nnz_hrow]. */
sat_status sat_part_lists(sat_ctx *ctx, int32_t m, int32_t *inner_gid, int32_t *halo_gid, int32_t *halo_slot,
                          int32_t *push_local, int32_t *push_slot, int64_t *loc_rowptr, int32_t *loc_col,
                          int64_t *hrow_ptr, int32_t *hrow_col);
/* Copies part[] (int32 [n], may be NULL) and slot[] (int32 [n], may be NULL) to HOST memory
 * and returns |C|. */
sat_status sat_slot_map(sat_ctx *ctx, int32_t *part_host, int32_t *slot_host, int32_t *n_slots);

/* ---------------------------------------------------------------------------------------
 * sat_gather_rows — out[i, :] = x[gid(i), :] for the inner (SAT_ROWS_INNER) or halo
 * (SAT_ROWS_HALO) nodes of `part`, x being a DEVICE matrix over all n nodes in global id
 * order.  With SAT_ROWS_HALO on the raw features this is the layer-1 pull: H_halo^(0) =
 * X[B_m] (out-of-subgraph term of Eq. "mini-batch" with h^(0) = x).
 * ------------------------------------------------------------------------------------- */
sat_status sat_gather_rows(sat_ctx *ctx, int32_t part, int which, const float *x, int32_t ld_x, int32_t d,
                           float *out, int32_t ld_out);

/* ---------------------------------------------------------------------------------------
 * sat_cache_init — the offline memory of historical embeddings (Section "Problem
 * Formulation": H~_out) as a ring, per cached layer, of tau readable snapshots plus one
 * write buffer over the |C| boundary nodes; tau is the sliding window of Eq. "problem
 * formulation".  width[i] is the embedding width of cached layer i+1.
 * mode SAT_CACHE_ZERO: all zeros, no valid snapshot.  SAT_CACHE_COPY: init[i] (DEVICE,
 * [|C| x width[i]], ld = width rounded up to 4) becomes the single valid snapshot of layer
 * i+1.  Memory: sum_i (tau+1) * |C| * ld_i * 4 bytes, owned by the context.
 * ------------------------------------------------------------------------------------- */
sat_status sat_cache_init(sat_ctx *ctx, int32_t n_cached_layers, const int32_t *width, int32_t tau, int mode,
                          const float *const *init);

/* Predictor parameters g_omega (Section "Embedding Predictor": LSTM + GCN), all DEVICE,
 * dense row-major without padding: Wx [d x 4h], Uh [h x 4h], b [4h] (gate order i, f, g, o),
 * Wg [h x d], bg [d].  d = width of the cached layer.
 * version: 0 = no promise.  A non-zero version promises that the VALUES of all five arrays are the same as in every earlier
 * call that passed the same version for this cached layer (the paper updates the predictor only every Delta-T epochs,
 * Algorithm 1 "Embedding predictor update"; bump the version after each update).  The library then keeps the input
 * projection x Wx + b of every new snapshot and reuses it in the following epochs — the result is the same LSTM, one of
 * tau input projections per epoch instead of tau.  After a version bump the older snapshots are not re-projected: their
 * steps contract over [x | s] as without a version, until they have left the window.  The library also keeps its packed
 * copies of the weights and biases (a few hundred KB per cached layer) for as long as the version stays the same.  Costs (tau+1) * |C| * 4h * 4 bytes per
 * cached layer. */
typedef struct sat_pred_params {
    const float *Wx, *Uh, *b, *Wg, *bg;
    int32_t h;
    int32_t cell;      /* SAT_CELL_LSTM (0) or SAT_CELL_GRU (1) */
    uint64_t version;
} sat_pred_params;
/* cell = SAT_CELL_GRU selects the GRU-GCN variant of the RNN-GNN predictor (Section "Embedding Predictor" names it; the
 * standard gated recurrent unit): Wx [d x 3h] and Uh [h x 3h] in gate order (r, z, n), b [4h] = (b_r, b_z, b_n, b_hn),
 *     r = sigm(x W_r + s U_r + b_r), z = sigm(x W_z + s U_z + b_z), n = tanh(x W_n + b_n + r o (s U_n + b_hn)),
 *     s = (1 - z) o n + z o s.
 * The graph convolution and the skip connection are the same.  version is ignored for the GRU (no projections are kept),
 * and sat_pred_grad supports the LSTM only (SAT_EINVAL otherwise). */
#define SAT_CELL_LSTM 0
#define SAT_CELL_GRU 1

/* ---------------------------------------------------------------------------------------
 * sat_predict — predicted out-of-subgraph embeddings Hhat_out^(l, m) = g_omega over the
 * temporal graph of the last min(n_valid, tau) cached snapshots (Eq. "sat forward",
 * Eq. "problem formulation", Section "Embedding Predictor"):
 *   LSTM over the snapshots (oldest first, zero initial state) for every cached node -> S;
 *   for halo node u of partition m:  a_u = p_uu S_u + sum_{v in N(u), v in V_m} p_uv S_v,
 *   Hhat_u = H~_u(newest snapshot) + a_u Wg + bg     (graph convolution + skip connection).
 * params == NULL is the identity predictor: Hhat_u = H~_u(newest) (plain historical
 * embeddings).  With no valid snapshot H~ = 0 and S = 0.
 *   reuse_state  0: run the LSTM now (for all |C| cached nodes; the table S is kept in the
 *                context per cached layer);  1: reuse the table of the previous call for
 *                this layer (caller guarantees parameters and ring are unchanged;
 *                SAT_ESTATE if there is none since the last commit).
 *   halo_out     DEVICE [b_m x ld_out] (part = SAT_ALL_PARTS: [sum_m b_m x ld_out]).
 * Every predicted row is computed independently of the others, so the order in which the rows are worked on does not
 * change a bit of the result; with part = SAT_ALL_PARTS and a snapshot above 128 MiB the output step walks its tiles of
 * 128 rows in the order of their cache slots (the halo copies of a node then read its newest row together).  The
 * environment variable SAT_PRED_TILE_ORDER=0 / 1 forces that order off / on for the process.
 * ------------------------------------------------------------------------------------- */
sat_status sat_predict(sat_ctx *ctx, int32_t layer, int32_t part, const sat_pred_params *params, int reuse_state,
                       float *halo_out, int32_t ld_out);
/* Copies the LSTM state table S of cached layer `layer` (fp32 [|C| x h]) to HOST memory. */
sat_status sat_predict_state(sat_ctx *ctx, int32_t layer, float *S_host, int32_t h);

/* ---------------------------------------------------------------------------------------
 * sat_pred_grad — objective of the embedding predictor of cached layer `layer` and its gradient with respect to the
 * predictor's parameters (Eq. "predictor loss" with the squared Euclidean norm; Eq. "mini-batch training" through
 * row_weight; Algorithm 1 "Embedding predictor update": omega <- omega - eta_2 grad, e.g. with sat_sgd_step per array).
 *   input   the temporal graph: the min(n_valid, tau) valid snapshots of the layer (oldest first);
 *   target  the embeddings pushed in the RUNNING epoch (the ring's write buffer): call it after every partition's
 *           sat_cache_update for this layer and before sat_cache_commit;
 *   Hhat_u  as in sat_predict (LSTM -> S, graph convolution on S, skip connection), recomputed here with the
 *           intermediate gate values kept for the backward pass;
 *   L = (1/M) sum_m sum_{u in B_m} w_u * 1/2 |Hhat_u^(m) - target_u|^2,   w_u = 1/b_m, or row_weight[u] when given
 *       (1/|batch| on the rows of a sampled batch, 0 elsewhere);
 *   gradient: through the output layer (Wg, bg), the transposed graph convolution and back through time in the LSTM.
 * params      DEVICE arrays as for sat_predict (version is ignored: nothing is reused from earlier calls)
 * row_weight  DEVICE [sum_m b_m] (halo rows of all partitions, concatenated in partition order) or NULL
 * g_Wx [d x 4h], g_Uh [h x 4h], g_b [4h], g_Wg [h x d], g_bg [d]   DEVICE, dense row-major, overwritten
 * loss_host   HOST, may be NULL; when given the call synchronises the stream
 * Scratch (owned by the context, kept): about k * |C| * 6h + sum_m b_m * (d + 2h) floats.
 * Errors: SAT_ESTATE without a cache, SAT_EINVAL for null / misaligned arrays or h not a multiple of 4.
 * ------------------------------------------------------------------------------------- */
sat_status sat_pred_grad(sat_ctx *ctx, int32_t layer, const sat_pred_params *params, const float *row_weight, float *g_Wx,
                         float *g_Uh, float *g_b, float *g_Wg, float *g_bg, double *loss_host);

/* ---------------------------------------------------------------------------------------
 * sat_layer_fwd — local GCN layer forward (Appendix, forward of SAT):
 *     AGG = P_in h_in + P_out h_halo ;  Z = AGG W + bias ;  h_out = ReLU(Z) or Z.
 *   h_in   DEVICE [n_m x ld_in]   in-subgraph embeddings H_in^(l-1, m), rows in I_m order
 *   h_halo DEVICE [b_m x ld_halo] out-of-subgraph embeddings (raw features for layer 1,
 *          sat_predict output otherwise); may be NULL when b_m = 0
 *   W      DEVICE [d_in x d_out] dense row-major;  bias DEVICE [d_out] or NULL
 *   h_out  DEVICE [n_m x ld_out]
 * What the backward needs (AGG and the sign of Z) is kept inside the context per layer,
 * for the rows of `part`; a later sat_layer_fwd of the same (part, layer) overwrites it.
 * ------------------------------------------------------------------------------------- */
sat_status sat_layer_fwd(sat_ctx *ctx, int32_t part, int32_t layer, int32_t d_in, int32_t d_out,
                         const float *h_in, int32_t ld_in, const float *h_halo, int32_t ld_halo,
                         const float *W, const float *bias, int act, float *h_out, int32_t ld_out);

/* ---------------------------------------------------------------------------------------
 * sat_layer_bwd — local backward of the same layer (Appendix, backward equations):
 *     D = g_out o [Z > 0] (ReLU layer) or g_out ;  g_W (+)= AGG^T D ;  g_b (+)= 1^T D ;
 *     G_AGG = D W^T ;  g_in = P_in^T G_AGG ;  g_halo = P_out^T G_AGG.
 * The predicted halo embeddings are constants of the epoch (Section "Optimization
 * Algorithm"), so g_halo is an optional by-product and is not propagated.
 *   g_out  DEVICE [n_m x ld_g]  gradient w.r.t. this layer's output h_out
 *   g_W    DEVICE [d_in x d_out] dense; g_b DEVICE [d_out] or NULL
 *   accumulate  bit set of SAT_BWD_* flags (0 and 1 keep their plain meaning):
 *               SAT_BWD_ACCUMULATE (1)   add to g_W / g_b instead of overwriting them (summing partitions gives the
 *                                        gradient of the global loss, Eq. "global loss")
 *               SAT_BWD_MASK_G_IN (2)    write g_in already multiplied by the ReLU mask that sat_layer_fwd recorded for
 *                                        layer - 1 on these rows, i.e. g_in = D of layer - 1 instead of the gradient w.r.t.
 *                                        h_in (no-op when layer - 1 has no ReLU or has not run): saves the separate
 *                                        masking pass over the activations' gradient
 *               SAT_BWD_G_OUT_MASKED (4) g_out is such a pre-masked gradient (D of this layer): the mask is not applied again
 *               SAT_BWD_GRAD_HISTORY (8) the stale-gradient term of SAT's back-propagation (Appendix):
 *                                        G_H^(t, l-1) = P_in^T D^(t, l) W^T + P_out^T D^(t-1, l) W^T.  For layer >= 2 the call
 *                                        (a) adds (P_out^T D)[u] of the selected partitions' halo nodes u to the running
 *                                        epoch's history Q^(l) [|C| x d_out] at the cache slot of u, and (b) when a
 *                                        committed history exists and g_in is wanted, adds Q_prev^(l)[slot(v)] W^T (with
 *                                        this call's W) to g_in for the boundary rows v, under the same mask as g_in.
 *                                        sat_cache_commit turns the running history into the committed one.  The history
 *                                        buffers (2 x |C| x d_out floats per layer) are allocated on first use and dropped
 *                                        on re-partitioning.  Partitions add to the history in call order (all partitions
 *                                        of a SAT_ALL_PARTS call in index order).
 *   g_in   DEVICE [n_m x ld_gin] or NULL (layer 1);  g_halo DEVICE [b_m x ld_gh] or NULL
 * Requires the matching sat_layer_fwd to have run (SAT_ESTATE otherwise).  Results are
 * bit-reproducible from run to run (no floating-point atomics).
 * ------------------------------------------------------------------------------------- */
#define SAT_BWD_ACCUMULATE 1
#define SAT_BWD_MASK_G_IN 2
#define SAT_BWD_G_OUT_MASKED 4
#define SAT_BWD_GRAD_HISTORY 8
sat_status sat_layer_bwd(sat_ctx *ctx, int32_t part, int32_t layer, const float *g_out, int32_t ld_g,
                         const float *W, float *g_W, float *g_b, int accumulate,
                         float *g_in, int32_t ld_gin, float *g_halo, int32_t ld_gh);

/* ---------------------------------------------------------------------------------------
 * sat_cache_update — push (Algorithm 1, "Push computed embeddings to the server"): rows of
 * h_out (DEVICE [n_m x ld], the output of GNN layer `layer` < L) that belong to boundary
 * nodes are written into the write buffer of cached layer `layer`.  Invisible to
 * sat_predict until sat_cache_commit.  Every boundary node must be pushed once per epoch
 * (rows not pushed keep whatever the buffer held tau+1 epochs earlier).
 * sat_cache_commit — end of epoch: the write buffer becomes the newest snapshot, the oldest
 * one is dropped, n_valid = min(n_valid + 1, tau); LSTM state tables are invalidated.
 * ------------------------------------------------------------------------------------- */
sat_status sat_cache_update(sat_ctx *ctx, int32_t part, int32_t layer, const float *h_out, int32_t ld);
sat_status sat_cache_commit(sat_ctx *ctx);

/* ---------------------------------------------------------------------------------------
 * sat_gat_fwd / sat_gat_bwd — graph-attention layer in place of the GCN layer (the paper reports SAT with a GAT backbone as
 * well, Table "performance comparison"; it gives no equations: this is the standard single-head graph attention layer).
 * For inner node v of the partition, over the entries u of its local row (neighbours inside the partition, v itself, and
 * neighbours outside, whose embeddings come from the cache / predictor exactly as for sat_layer_fwd):
 *     z_u = h_u W ;  e_vu = LeakyReLU_0.2(a_dst . z_v + a_src . z_u) ;  alpha_vu = softmax_u(e_vu) ;
 *     h_out_v = act( sum_u alpha_vu z_u + bias ).
 * The GCN normalisation is not used.  W [d_in x d_out], a_src [d_out], a_dst [d_out], bias [d_out] or NULL: DEVICE, dense.
 * sat_gat_fwd keeps z, the attention scores and the log-sum-exp of every row for sat_gat_bwd (memory: (n + sum_m b_m) *
 * d_out floats per layer, owned by the context).  d_out <= 1024.
 * sat_gat_bwd: g_out [n_m x ld_g] gradient w.r.t. h_out; h_out as written by sat_gat_fwd (used for the ReLU mask; may be
 * NULL for SAT_ACT_NONE); h_in / h_halo the same inputs as in the forward call.  The halo embeddings are constants of the
 * epoch, W acts on them as on the inner rows:  g_W [d_in x d_out], g_a_src [d_out], g_a_dst [d_out], g_b [d_out] are
 * overwritten (accumulate = 0) or added to (accumulate = 1); g_in [n_m x ld_gin] (or NULL) = gradient w.r.t. h_in.
 * Results are bit-reproducible (no floating-point atomics).  SAT_ESTATE without the matching forward call.
 * ------------------------------------------------------------------------------------- */
sat_status sat_gat_fwd(sat_ctx *ctx, int32_t part, int32_t layer, int32_t d_in, int32_t d_out, const float *h_in, int32_t ld_in,
                       const float *h_halo, int32_t ld_halo, const float *W, const float *a_src, const float *a_dst,
                       const float *bias, int act, float *h_out, int32_t ld_out);
sat_status sat_gat_bwd(sat_ctx *ctx, int32_t part, int32_t layer, const float *g_out, int32_t ld_g, const float *h_out, int32_t ld_out,
                       const float *h_in, int32_t ld_in, const float *h_halo, int32_t ld_halo, int32_t d_in, const float *W,
                       const float *a_src, const float *a_dst, float *g_W, float *g_a_src, float *g_a_dst, float *g_b,
                       int accumulate, float *g_in, int32_t ld_gin);

/* The attention scores sat_gat_fwd kept for layer `layer` (all partitions must have run), copied to HOST memory (any pointer may
 * be NULL): s_src of the inner rows (a_src . z_u, fp32 [n], partition-major rows), s_dst (a_dst . z_v, fp32 [n]) and s_src of
 * the halo positions (fp32 [sum_m b_m]).  The logit of entry (v, u) before the LeakyReLU is the fp32 sum s_dst[v] + s_src[u],
 * which is what decides its slope in sat_gat_bwd.  For tests and diagnostics (the paper has no counterpart).  Synchronises. */
sat_status sat_gat_scores(sat_ctx *ctx, int32_t layer, float *s_src_inner_host, float *s_dst_host, float *s_src_halo_host);

/* Gradient-side history of layer `layer` >= 2 (see SAT_BWD_GRAD_HISTORY), for checkpoints and tests.
 * sat_grad_history_read: copies the committed history (which = 0; SAT_ESTATE before the first commit) or the running
 * epoch's (which = 1) to HOST memory, dense [|C| x d_out].
 * sat_grad_history_write: makes in_host (HOST, dense [|C| x width]) the committed history and clears the running one;
 * in_host = NULL clears both and marks the committed one absent. */
sat_status sat_grad_history_read(sat_ctx *ctx, int32_t layer, int which, float *out_host);
sat_status sat_grad_history_write(sat_ctx *ctx, int32_t layer, int32_t width, const float *in_host);
/* Ring bookkeeping: index of the write buffer in [0, tau] and number of valid snapshots. */
sat_status sat_cache_state(sat_ctx *ctx, int32_t *write_idx, int32_t *n_valid);
/* Copies snapshot `age` (0 = newest committed, ..., n_valid-1 = oldest; -1 = the write
 * buffer) of cached layer `layer` to HOST memory as dense [|C| x width]. */
sat_status sat_cache_read(sat_ctx *ctx, int32_t layer, int32_t age, float *out_host);
/* Checkpoint / resume of the whole ring of one cached layer: raw [(tau+1) x |C| x width]
 * HOST array in buffer-index order, plus write_idx / n_valid via sat_cache_state and
 * sat_cache_set_state. */
sat_status sat_cache_export(sat_ctx *ctx, int32_t layer, float *out_host);
sat_status sat_cache_import(sat_ctx *ctx, int32_t layer, const float *in_host);
sat_status sat_cache_set_state(sat_ctx *ctx, int32_t write_idx, int32_t n_valid);

/* ---------------------------------------------------------------------------------------
 * Auxiliary steps of the epoch (Algorithm 1, "Local GNN update" / "Global GNN update").
 * sat_loss_grad — local loss (Eq. "local loss") weighted by w_m = |V_m| / N (Eq. "global
 * loss"), i.e. every node carries weight 1/N:  *loss_sum (DEVICE double, += ) receives
 * sum_v Loss_v / N over the rows of `part`; g = (1/N) dLoss_v/dz (DEVICE [n_m x ld_g]).
 *   SAT_LOSS_SOFTMAX_CE:  labels int32 [n_m] DEVICE;  Loss_v = -log softmax(z_v)[y_v]
 *   SAT_LOSS_SIGMOID_BCE: labels uint8 [n_m x n_classes] DEVICE;
 *                         Loss_v = (1/C) sum_c softplus(z_c) - y_c z_c
 * sat_sgd_step — w <- w - lr * g over `count` floats (the parameter step on the summed
 * gradient; all partitions share theta within an epoch, so AGG is the identity here).
 * ------------------------------------------------------------------------------------- */
sat_status sat_loss_grad(sat_ctx *ctx, int32_t part, int kind, int32_t n_classes, const float *z, int32_t ld_z,
                         const void *labels, double *loss_sum, float *g, int32_t ld_g);
sat_status sat_sgd_step(sat_ctx *ctx, int64_t count, float *w, const float *g, float lr);
/* The same step on n_arrays arrays at once: counts[i] floats of w[i] and g[i] (HOST arrays of sizes and of DEVICE pointers);
 * one launch per 16 arrays. */
sat_status sat_sgd_steps(sat_ctx *ctx, int32_t n_arrays, const int64_t *counts, float *const *w, const float *const *g, float lr);

/* ---------------------------------------------------------------------------------------
 * The dense contractions of the layer step on caller tensors (all DEVICE fp32; the paper has no counterpart:
 * they are the matrix products inside the forward / backward formulas of the Appendix, exposed so that the
 * kernels can be exercised and measured in isolation).  Same kernels and same path selection as inside
 * sat_layer_fwd / sat_layer_bwd / sat_predict.
 *   sat_dense_nn: C[m x n] = A[m x k] W[k x n] + bias        (W dense row-major, bias [n] or NULL)
 *   sat_dense_nt: C[m x n] = A[m x k] W[n x k]^T
 *   sat_dense_tn: C[m x n] = A[rows x m]^T B[rows x n]        (C dense row-major)
 * ------------------------------------------------------------------------------------- */
sat_status sat_dense_nn(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const float *W, const float *bias,
                        float *C, int32_t ldc);
sat_status sat_dense_nt(sat_ctx *ctx, int64_t m, int32_t n, int32_t k, const float *A, int32_t lda, const float *W, float *C, int32_t ldc);
sat_status sat_dense_tn(sat_ctx *ctx, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B, int32_t ldb,
                        float *C);

/* ---------------------------------------------------------------------------------------
 * sat_dense_tn_static — C[m x n] = A[rows x m]^T B[rows x n] like sat_dense_tn, for callers that cannot allocate.
 * (The paper has no counterpart; this is a deployment variant of the weight-gradient product.)
 *
 * Who needs it: code that must not call cudaMalloc — a process whose device heap is fully owned by another component,
 * latency-critical loops that cannot take the device-wide synchronisation an allocation implies, or a host region in which
 * allocation calls are forbidden.  This entry point needs no context, calls no cudaMalloc / cudaFree and no allocating
 * library routine: the partial sums of the row splits live in an 8 MiB array that is part of the library image (every
 * GPU that loads the library holds it until the process exits).
 *
 *   cuda_stream  cudaStream_t to enqueue on (may be 0); the device must be current
 *   A, B, C      DEVICE fp32, caller-owned; A [rows x lda], B [rows x ldb], C dense [m x n] (overwritten)
 *   errbuf       HOST buffer (may be NULL) that receives a message when the status is not SAT_OK
 * Limit: m * n <= 2,097,152 (the array holds at least one m x n block of partial sums); larger shapes are rejected with
 * SAT_EINVAL and a message naming the limit — use sat_dense_tn then.  Fewer splits fit for larger m * n, so very tall
 * inputs run slower here than through sat_dense_tn.
 * Set-up: the first call on each device looks up the device address of the array (once per device, kept for the
 * process); make that first call outside any stream capture, and do not reset the device (cudaDeviceReset) afterwards:
 * the kept address belongs to the device's primary context.
 * Sharing: all calls on a device use the same array.  It keeps whatever the previous call left; nothing has to be
 * cleared because each call overwrites every partial block it later reads.  Two calls that overlap on the GPU (different
 * streams, or concurrent threads) race on the array: serialise them.
 * The result is bit-reproducible from call to call (fixed split sizes and summation order).
 * ------------------------------------------------------------------------------------- */
sat_status sat_dense_tn_static(void *cuda_stream, int64_t rows, int32_t m, int32_t n, const float *A, int32_t lda, const float *B,
                               int32_t ldb, float *C, char *errbuf, int32_t errbuf_len);

/* ---------------------------------------------------------------------------------------
 * sat_staleness — staleness of the out-of-subgraph embeddings of a partition (Eq. "staleness def"):
 *     sq_sum = sum over the halo rows j of `part` of || h_fresh[row of halo node j] - h_used_halo[j] ||^2 ,
 * the squared Frobenius norm the equation takes the root of (squared, so that partitions can be added up).
 *   h_fresh      DEVICE [n x ld]  this epoch's embeddings of ALL nodes in partition-major row order (the h_out of
 *                sat_layer_fwd called with SAT_ALL_PARTS, or the per-partition outputs side by side)
 *   h_used_halo  DEVICE [b_m x ld_halo]  what the partition used for its halo: the identity predictor's output for the
 *                historical embeddings, sat_predict's output for the predicted ones
 *   sq_sum       DEVICE double, overwritten.  Accumulation in fp64, fixed order (reproducible).
 * A diagnostic: not part of the training step.
 * ------------------------------------------------------------------------------------- */
sat_status sat_staleness(sat_ctx *ctx, int32_t part, int32_t d, const float *h_fresh, int32_t ld, const float *h_used_halo,
                         int32_t ld_halo, double *sq_sum);

/* ---------------------------------------------------------------------------------------
 * Embedding codec — lossy storage of historical embeddings (Supplement, "Data Compression for
 * Historical Embedding Storage": the encoded-polyline scheme at a configurable decimal precision).
 * Every row of an fp32 matrix is one delta-coded sequence:
 *     q_j = round-half-away-from-zero(x_j * 10^p)      (evaluated in fp64, where the product is exact for p <= 7)
 *     e_0 = q_0, e_j = q_j - q_{j-1};  v = e << 1, bitwise inverted when e < 0
 *     5-bit groups of v, least significant first, bit 0x20 on every group but the last, each + 63 -> one ASCII byte
 * Row r occupies bytes [row_offsets[r], row_offsets[r+1]).  Decoding: x_j = (float)((double)q_j / 10^p).
 * The paper fixes neither the rounding of ties nor what the deltas run over; this is the reading taken here.
 *
 *   sat_codec_plan    sizes: writes row_offsets (DEVICE int64 [rows + 1], exclusive prefix sums of the row sizes) and
 *                     returns the total in *total_bytes (HOST); synchronises the context's stream
 *   sat_codec_encode  writes the bytes (DEVICE uint8, capacity >= the planned total) for the same x / precision
 *   sat_codec_decode  inverse; `in` holds in_bytes bytes.  Rows whose bytes do not hold exactly d values, and rows whose
 *                     offsets do not lie inside [0, in_bytes] in ascending order (such a row is skipped: nothing outside
 *                     the buffer is read), raise the device status word (sat_sync_status returns SAT_EDATA); a row with
 *                     malformed bytes is left partly written
 *   sat_cache_requantise  stores the committed snapshot `age` (0 = newest) of cached layer `layer` the way a compressed
 *                     ring would hold it: encode + decode in place (context scratch); *bytes (HOST, nullable) = size
 *                     of the encoded snapshot.  Cached input projections of that snapshot are dropped.
 * x: DEVICE [rows x ld] fp32, ld >= d; precision in 0..7.  SAT_EINVAL on bad arguments.
 * ------------------------------------------------------------------------------------- */
sat_status sat_codec_plan(sat_ctx *ctx, const float *x, int32_t ld, int64_t rows, int32_t d, int32_t precision,
                          int64_t *row_offsets, int64_t *total_bytes);
sat_status sat_codec_encode(sat_ctx *ctx, const float *x, int32_t ld, int64_t rows, int32_t d, int32_t precision,
                            const int64_t *row_offsets, uint8_t *out, int64_t out_capacity);
sat_status sat_codec_decode(sat_ctx *ctx, const uint8_t *in, int64_t in_bytes, const int64_t *row_offsets, int64_t rows, int32_t d,
                            int32_t precision, float *x, int32_t ld);
sat_status sat_cache_requantise(sat_ctx *ctx, int32_t layer, int32_t age, int32_t precision, int64_t *bytes);

/* Bounds-checking debug build (libsat_b200_dbg.so: the same sources compiled with -DSAT_DEBUG_BOUNDS; the paper has no
 * counterpart).  Every index the graph kernels (SpMM, halo-row products, row gather / scatter, per-slot sums) load from an
 * index array is compared with the extent of the matrix it addresses; an index outside it raises a bit of the device status
 * word — sat_sync_status then returns SAT_EDATA once, the context stays usable — and is replaced by a valid index before use, so
 * nothing outside the matrix is touched: no trap, no device assert.  It stands in for a memory checker on these kernels.
 * sat_debug_poke_index overwrites entry `pos` of an internal index array (which = 0: encoded column ids of the local CSR,
 * length nnz(A+I); 1: cache slots of the halo positions, length sum_m b_m) and returns the old value (HOST, nullable), so
 * that a test can show the checks at work; in the regular build it changes nothing and returns SAT_ESTATE. */
sat_status sat_debug_poke_index(sat_ctx *ctx, int which, int64_t pos, int32_t value, int32_t *old_value);

/* Number of kernels this context has launched since creation (all entry points). */
sat_status sat_launch_count(sat_ctx *ctx, int64_t *count);

/* Optional device timing per kernel family, with CUDA events on the context's stream (measurement aid; the
 * paper has no counterpart).  sat_profile_enable(1) clears the records and starts bracketing every family's
 * launches with an event pair; sat_profile_enable(0) stops.  sat_profile_read waits for the stream and returns,
 * for family f in [0, sat_profile_families()), its name, number of bracketed calls, total milliseconds and the
 * algorithmic bytes / flops those calls moved / performed (each operand read once, each result written once).
 * Every bracketed call costs two event records on the stream (of the order of a microsecond of device time each);
 * sat_profile_select restricts the bracketing to the families whose bit (1 << family) is set in family_mask (default: all),
 * so that a timed run can carry the events of one family only. */
enum { SAT_PROF_SPMM_FWD = 0, SAT_PROF_SPMM_BWD, SAT_PROF_SPMM_HROW, SAT_PROF_GEMM_NN, SAT_PROF_GEMM_NT,
       SAT_PROF_GEMM_TN, SAT_PROF_LSTM_CELL, SAT_PROF_GATHER, SAT_PROF_SCATTER, SAT_PROF_LOSS, SAT_PROF_MASK,
       SAT_PROF_GEMM_SIDE, SAT_PROF_CODEC, SAT_PROF_PRED_TRAIN, SAT_PROF_GAT };
int32_t sat_profile_families(void);
sat_status sat_profile_enable(sat_ctx *ctx, int enable);
sat_status sat_profile_select(sat_ctx *ctx, uint64_t family_mask);
sat_status sat_profile_read(sat_ctx *ctx, int32_t family, const char **name, int64_t *calls, double *ms, double *bytes,
                            double *flops);

/* How the forward aggregation (the `P_in H_in + P_out Hhat` product of sat_layer_fwd; Appendix, forward of SAT) at width `d`
 * walks partition `part` (or SAT_ALL_PARTS).  Where a partition's source rows (inner + out-of-subgraph) are several times
 * the L2 and its rows are long, the library walks it once per block of sources instead of once, row by row: a row then
 * contributes one partial sum per block it has entries in, added in block order afterwards (fixed order: reproducible, and
 * the same whether the partition is run alone or with all others).  HOST outputs, each may be NULL: `n_blocks` = source
 * blocks of the most finely cut partition (1 = plain row-by-row walk), `n_items` = work items of the launch,
 * `n_partial_rows` = partial-sum rows of width d it writes and re-reads.  The cut is chosen per width (blocks of 64 MiB of
 * source rows, for partitions above 192 MiB whose rows meet a block with 8 or more entries on average; inside such a
 * partition a short row is walked in groups of consecutive blocks, at least 32 entries per group, so that it leaves few
 * partial sums); the environment variable SAT_SPMM_SRC_BLOCK="<block bytes>[,<from bytes>[,<entries>[,<entries per row
 * group>]]]" overrides the four figures for the process ("0" = never).  Builds the work list on first use (device memory, freed with the partition); synchronises the stream.
 * Errors: SAT_ESTATE without a partition, SAT_EINVAL for a bad `part` or d < 1. */
sat_status sat_spmm_plan(sat_ctx *ctx, int32_t part, int32_t d, int32_t *n_blocks, int64_t *n_items, int64_t *n_partial_rows);

/* What the L2 -> SM path of the GPU delivers, measured now (measurement aid; the paper has no counterpart): a 64 MiB buffer,
 * resident in L2, read (a) as a contiguous stream by all SMs and (b) as rows of `row_floats` floats (a multiple of 4, at most
 * 1024) in pseudo-random order with the access shape of the SpMM kernels.  Both in GB/s (HOST outputs, either may be NULL).
 * Allocates and frees its buffer; synchronises the stream.  The SpMM's neighbour-row gather comes mostly out of L2, so
 * these are the rates to hold its gather rate against — measured in the same run, on the same GPU, at the same clocks. */
sat_status sat_profile_l2_rates(sat_ctx *ctx, int32_t row_floats, double *stream_gbs, double *gather_gbs);

#ifdef __cplusplus
}
#endif
#endif /* SAT_B200_H */
