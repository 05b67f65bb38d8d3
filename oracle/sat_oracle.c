/*
 * CPU oracle for the SAT (staleness-alleviated training) partition-parallel GCN step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, obviously-correct statement
 * of what the hot path computes; the tests, the smoke check and the benchmark's CPU
 * baseline leg are its only users.  It shares no code with the CUDA library and the
 * CUDA library never calls it.
 *
 * Conventions
 *   - every sum is accumulated in double precision in the order the formula is
 *     written (row by row, neighbour by neighbour, k ascending);
 *   - inputs that the method stores as fp32 (features, cached embeddings, weights,
 *     gradients handed from layer to layer) are read as fp32; results are rounded to
 *     fp32 only where the method itself stores them (layer outputs, cache entries,
 *     predictor state and output, gradients);
 *   - `omp parallel for` appears only over independent output rows / columns, so the
 *     summation order of every output element is fixed.
 *
 * Notation follows the paper: P = propagation matrix of GCN (Appendix, Preliminaries),
 * P = P_in + P_out per partition, H_in / H_out(halo) in- and out-of-subgraph
 * embeddings (Eq. "matrix form forward"), D = G o sigma'(Z), G_W, G_H (Appendix,
 * backward equations), S / C = LSTM hidden state / memory cell and
 * dH = GCN(S, A) (Section "Embedding Predictor").
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------
 * O-1  Propagation matrix of GCN with self-loops (Appendix, Preliminaries: "P is the
 * propagation matrix following the definition of GCN"):
 *     P = D~^{-1/2} (A + I) D~^{-1/2},   d~_v = deg(v) + 1,
 *     p_vu = 1 / sqrt(d~_v d~_u)  for u in N(v) or u == v.
 * `dtil` holds the integers d~_v.
 * ---------------------------------------------------------------------------------- */
static inline double p_entry(int32_t dt_v, int32_t dt_u)
{
    return 1.0 / sqrt((double)dt_v * (double)dt_u);
}

void orc_degrees(int32_t n, const int64_t *rowptr, int32_t *dtil, float *dinv)
{
    for (int32_t v = 0; v < n; ++v) {
        dtil[v] = (int32_t)(rowptr[v + 1] - rowptr[v]) + 1;
        dinv[v] = (float)(1.0 / sqrt((double)dtil[v]));
    }
}

/* ------------------------------------------------------------------------------------
 * O-6  Layer forward for partition m (Appendix, forward of SAT; Eq. "sat forward"):
 *     AGG = P_in H_in + P_out H_halo            (one pass over the local CSR)
 *     Z   = AGG W + b
 *     H   = ReLU(Z)  (act = 1)   or   H = Z  (act = 0)
 * Local CSR: rows = inner nodes of m, columns are local ids: c < n_in is inner node c,
 * c >= n_in is halo node c - n_in; the self-loop is an explicit entry.
 * rows_sel (may be NULL = all rows) restricts the computation to a sample of rows;
 * outputs are always addressed by the full row id.
 * AGG and Z are kept in double (the method never exposes them); H is the fp32 layer
 * output.
 * ---------------------------------------------------------------------------------- */
void orc_layer_fwd(int32_t n_sel, const int32_t *rows_sel,
                   int32_t n_in, const int64_t *lrowptr, const int32_t *lcol,
                   const int32_t *inner_gid, const int32_t *halo_gid, const int32_t *dtil,
                   int32_t d_in, int32_t d_out,
                   const float *H_in, int64_t ld_in, const float *H_halo, int64_t ld_halo,
                   const float *W, const float *bias, int32_t act,
                   double *AGG /* [n_in x d_in] */, double *Z /* [n_in x d_out] */,
                   float *H /* [n_in x ld_h] */, int64_t ld_h)
{
    int32_t count = rows_sel ? n_sel : n_in;
#pragma omp parallel for schedule(dynamic, 16)
    for (int32_t i = 0; i < count; ++i) {
        int32_t v = rows_sel ? rows_sel[i] : i;
        double *agg = AGG + (int64_t)v * d_in;
        for (int32_t k = 0; k < d_in; ++k) agg[k] = 0.0;
        int32_t dt_v = dtil[inner_gid[v]];
        for (int64_t e = lrowptr[v]; e < lrowptr[v + 1]; ++e) {
            int32_t c = lcol[e];
            const float *src;
            int32_t dt_u;
            if (c < n_in) {
                src = H_in + (int64_t)c * ld_in;
                dt_u = dtil[inner_gid[c]];
            } else {
                src = H_halo + (int64_t)(c - n_in) * ld_halo;
                dt_u = dtil[halo_gid[c - n_in]];
            }
            double p = p_entry(dt_v, dt_u);
            for (int32_t k = 0; k < d_in; ++k) agg[k] += p * (double)src[k];
        }
        double *z = Z + (int64_t)v * d_out;
        for (int32_t j = 0; j < d_out; ++j) z[j] = 0.0;
        for (int32_t k = 0; k < d_in; ++k) {
            double a = agg[k];
            const float *wrow = W + (int64_t)k * d_out;
            for (int32_t j = 0; j < d_out; ++j) z[j] += a * (double)wrow[j];
        }
        float *h = H + (int64_t)v * ld_h;
        for (int32_t j = 0; j < d_out; ++j) {
            if (bias) z[j] += (double)bias[j];
            double o = (act == 1 && !(z[j] > 0.0)) ? 0.0 : z[j];
            h[j] = (float)o;
        }
    }
}

/* ------------------------------------------------------------------------------------
 * O-9  Layer backward for partition m (Appendix, backward equations):
 *     D     = G_out o [Z > 0]         (hidden layer; mask supplied as bytes)   or  D = G_out
 *     G_W  += AGG^T D                  (G_W = (P H)^T D)
 *     G_b  += column sums of D
 *     G_AGG = D W^T
 *     G_in  = P_in^T  G_AGG            (G_H = P^T D W^T restricted to inner columns: the
 *                                       predicted halo embeddings are constants)
 *     G_halo= P_out^T G_AGG            (optional; the part a gradient exchange would need)
 * P^T is applied as a scatter over the same local CSR, row by row, so the order of
 * additions into every output element is the row order.
 * ---------------------------------------------------------------------------------- */
void orc_layer_bwd(int32_t n_in, int32_t n_halo, const int64_t *lrowptr, const int32_t *lcol,
                   const int32_t *inner_gid, const int32_t *halo_gid, const int32_t *dtil,
                   int32_t d_in, int32_t d_out,
                   const float *G_out, int64_t ld_g, const uint8_t *mask /* [n_in x d_out] or NULL */,
                   const double *AGG, const float *W,
                   double *G_W /* [d_in x d_out], += */, double *G_b /* [d_out], += */,
                   float *G_in /* [n_in x ld_gin] or NULL */, int64_t ld_gin,
                   float *G_halo /* [n_halo x ld_gh] or NULL */, int64_t ld_gh)
{
    double *D = (double *)malloc(sizeof(double) * (size_t)n_in * d_out);
    double *GA = (double *)malloc(sizeof(double) * (size_t)n_in * d_in);
#pragma omp parallel for
    for (int32_t v = 0; v < n_in; ++v)
        for (int32_t j = 0; j < d_out; ++j) {
            double g = (double)G_out[(int64_t)v * ld_g + j];
            if (mask && !mask[(int64_t)v * d_out + j]) g = 0.0;
            D[(int64_t)v * d_out + j] = g;
        }
    /* G_W[k][j] += sum_v AGG[v][k] D[v][j], v ascending */
#pragma omp parallel for
    for (int32_t k = 0; k < d_in; ++k) {
        double *gw = G_W + (int64_t)k * d_out;
        for (int32_t v = 0; v < n_in; ++v) {
            double a = AGG[(int64_t)v * d_in + k];
            const double *drow = D + (int64_t)v * d_out;
            for (int32_t j = 0; j < d_out; ++j) gw[j] += a * drow[j];
        }
    }
#pragma omp parallel for
    for (int32_t j = 0; j < d_out; ++j) {
        double s = 0.0;
        for (int32_t v = 0; v < n_in; ++v) s += D[(int64_t)v * d_out + j];
        G_b[j] += s;
    }
    /* G_AGG[v][k] = sum_j D[v][j] W[k][j] */
#pragma omp parallel for
    for (int32_t v = 0; v < n_in; ++v)
        for (int32_t k = 0; k < d_in; ++k) {
            double s = 0.0;
            const float *wrow = W + (int64_t)k * d_out;
            const double *drow = D + (int64_t)v * d_out;
            for (int32_t j = 0; j < d_out; ++j) s += drow[j] * (double)wrow[j];
            GA[(int64_t)v * d_in + k] = s;
        }
    if (G_in || G_halo) {
        int32_t n_tot = n_in + n_halo;
        double *T = (double *)calloc((size_t)n_tot * d_in, sizeof(double));
        /* scatter form of P^T: each thread owns a disjoint range of feature columns */
#pragma omp parallel
        {
            int nt = 1, id = 0;
#ifdef _OPENMP
            nt = omp_get_num_threads();
            id = omp_get_thread_num();
#endif
            int32_t k0 = (int32_t)((int64_t)d_in * id / nt), k1 = (int32_t)((int64_t)d_in * (id + 1) / nt);
            if (k1 > k0)
                for (int32_t v = 0; v < n_in; ++v) {
                    int32_t dt_v = dtil[inner_gid[v]];
                    const double *ga = GA + (int64_t)v * d_in;
                    for (int64_t e = lrowptr[v]; e < lrowptr[v + 1]; ++e) {
                        int32_t c = lcol[e];
                        int32_t dt_u = c < n_in ? dtil[inner_gid[c]] : dtil[halo_gid[c - n_in]];
                        double p = p_entry(dt_v, dt_u);
                        double *t = T + (int64_t)c * d_in;
                        for (int32_t k = k0; k < k1; ++k) t[k] += p * ga[k];
                    }
                }
        }
        if (G_in)
            for (int32_t u = 0; u < n_in; ++u)
                for (int32_t k = 0; k < d_in; ++k) G_in[(int64_t)u * ld_gin + k] = (float)T[(int64_t)u * d_in + k];
        if (G_halo)
            for (int32_t u = 0; u < n_halo; ++u)
                for (int32_t k = 0; k < d_in; ++k)
                    G_halo[(int64_t)u * ld_gh + k] = (float)T[(int64_t)(n_in + u) * d_in + k];
        free(T);
    }
    free(D);
    free(GA);
}

/* ------------------------------------------------------------------------------------
 * O-4  LSTM over the cached snapshots (Section "Embedding Predictor": the recurrent
 * part of the RNN-GNN predictor iterates over epochs t-tau .. t-1).
 * For every cached node (slot) w:  s = c = 0; for the k snapshots, oldest first:
 *     a = x W_x + s U_h + b           (4h wide, gate order i, f, g, o)
 *     i = sigm(a_i) f = sigm(a_f) g = tanh(a_g) o = sigm(a_o)
 *     c = f o c + i o g ;  s = o o tanh(c)
 * S_w = final s, stored fp32 (zeros when k == 0).
 * snaps[t] is snapshot t (oldest = 0), each [n_slots x ld].
 * ---------------------------------------------------------------------------------- */
static inline double sigm(double x) { return 1.0 / (1.0 + exp(-x)); }

void orc_lstm(int32_t n_sel, const int32_t *slots_sel, int32_t n_slots, int32_t k,
              const float *const *snaps, int64_t ld, int32_t d, int32_t h,
              const float *Wx /* [d x 4h] */, const float *Uh /* [h x 4h] */, const float *b /* [4h] */,
              float *S /* [n_slots x h] */)
{
    int32_t count = slots_sel ? n_sel : n_slots;
#pragma omp parallel
    {
        double *a = (double *)malloc(sizeof(double) * 4 * (size_t)h);
        double *s = (double *)malloc(sizeof(double) * (size_t)h);
        double *c = (double *)malloc(sizeof(double) * (size_t)h);
#pragma omp for schedule(dynamic, 16)
        for (int32_t idx = 0; idx < count; ++idx) {
            int32_t w = slots_sel ? slots_sel[idx] : idx;
            for (int32_t j = 0; j < h; ++j) s[j] = c[j] = 0.0;
            for (int32_t t = 0; t < k; ++t) {
                const float *x = snaps[t] + (int64_t)w * ld;
                for (int32_t j = 0; j < 4 * h; ++j) a[j] = 0.0;
                for (int32_t q = 0; q < d; ++q) {
                    double xv = (double)x[q];
                    const float *wr = Wx + (int64_t)q * 4 * h;
                    for (int32_t j = 0; j < 4 * h; ++j) a[j] += xv * (double)wr[j];
                }
                for (int32_t q = 0; q < h; ++q) {
                    double sv = s[q];
                    const float *ur = Uh + (int64_t)q * 4 * h;
                    for (int32_t j = 0; j < 4 * h; ++j) a[j] += sv * (double)ur[j];
                }
                for (int32_t j = 0; j < 4 * h; ++j) a[j] += (double)b[j];
                for (int32_t j = 0; j < h; ++j) {
                    double gi = sigm(a[j]), gf = sigm(a[h + j]), gg = tanh(a[2 * h + j]), go = sigm(a[3 * h + j]);
                    c[j] = gf * c[j] + gi * gg;
                    s[j] = go * tanh(c[j]);
                }
            }
            for (int32_t j = 0; j < h; ++j) S[(int64_t)w * h + j] = (float)s[j];
        }
        free(a);
        free(s);
        free(c);
    }
}

/* ------------------------------------------------------------------------------------
 * O-4b  GRU in place of the LSTM (Section "Embedding Predictor" names GRU-GCN as a variant of the RNN-GNN
 * predictor; the paper gives no equations, so this is the standard gated recurrent unit):
 *     r = sigm(x W_r + s U_r + b_r)   z = sigm(x W_z + s U_z + b_z)
 *     n = tanh(x W_n + b_n + r o (s U_n + b_hn))
 *     s = (1 - z) o n + z o s
 * W_x = [W_r | W_z | W_n] is [d x 3h], U_h likewise [h x 3h], b = [b_r | b_z | b_n | b_hn] has 4h entries.
 * Same calling convention as orc_lstm.
 * ---------------------------------------------------------------------------------- */
void orc_gru(int32_t n_sel, const int32_t *slots_sel, int32_t n_slots, int32_t k,
             const float *const *snaps, int64_t ld, int32_t d, int32_t h,
             const float *Wx /* [d x 3h] */, const float *Uh /* [h x 3h] */, const float *b /* [4h] */,
             float *S /* [n_slots x h] */)
{
    int32_t count = slots_sel ? n_sel : n_slots;
#pragma omp parallel
    {
        double *ax = (double *)malloc(sizeof(double) * 3 * (size_t)h);
        double *ah = (double *)malloc(sizeof(double) * 3 * (size_t)h);
        double *s = (double *)malloc(sizeof(double) * (size_t)h);
#pragma omp for schedule(dynamic, 16)
        for (int32_t idx = 0; idx < count; ++idx) {
            int32_t w = slots_sel ? slots_sel[idx] : idx;
            for (int32_t j = 0; j < h; ++j) s[j] = 0.0;
            for (int32_t t = 0; t < k; ++t) {
                const float *x = snaps[t] + (int64_t)w * ld;
                for (int32_t j = 0; j < 3 * h; ++j) ax[j] = ah[j] = 0.0;
                for (int32_t q = 0; q < d; ++q) {
                    double xv = (double)x[q];
                    const float *wr = Wx + (int64_t)q * 3 * h;
                    for (int32_t j = 0; j < 3 * h; ++j) ax[j] += xv * (double)wr[j];
                }
                for (int32_t q = 0; q < h; ++q) {
                    double sv = s[q];
                    const float *ur = Uh + (int64_t)q * 3 * h;
                    for (int32_t j = 0; j < 3 * h; ++j) ah[j] += sv * (double)ur[j];
                }
                for (int32_t j = 0; j < h; ++j) {
                    double r = sigm(ax[j] + ah[j] + (double)b[j]);
                    double z = sigm(ax[h + j] + ah[h + j] + (double)b[h + j]);
                    double n = tanh(ax[2 * h + j] + (double)b[2 * h + j] + r * (ah[2 * h + j] + (double)b[3 * h + j]));
                    ax[j] = (1.0 - z) * n + z * s[j];   /* new state, kept aside until every unit has read the old one */
                }
                for (int32_t j = 0; j < h; ++j) s[j] = ax[j];
            }
            for (int32_t j = 0; j < h; ++j) S[(int64_t)w * h + j] = (float)s[j];
        }
        free(ax);
        free(ah);
        free(s);
    }
}

/* ------------------------------------------------------------------------------------
 * O-5  Graph convolution on the final LSTM state plus skip connection, for the halo
 * rows of partition m (Section "Embedding Predictor": dH = GCN(S, A) on the 1-hop
 * extended subgraph; the prediction corrects the newest cached embedding):
 *     a_u   = p_uu S_u + sum_{v in N(u) cap V_m} p_uv S_v
 *     dH_u  = a_u W_g + b_g
 *     Hhat_u= Htilde_u(newest) + dH_u
 * Halo-row CSR: row j = halo node j of m, columns = local inner ids of its neighbours
 * inside m.  `newest` may be NULL (no committed snapshot: Htilde = 0).
 * ---------------------------------------------------------------------------------- */
void orc_predict_halo(int32_t n_sel, const int32_t *rows_sel,
                      int32_t n_halo, const int64_t *hrow_ptr, const int32_t *hrow_col,
                      const int32_t *inner_gid, const int32_t *halo_gid, const int32_t *slot,
                      const int32_t *dtil, int32_t h, int32_t d,
                      const float *S /* [n_slots x h] */, const float *newest, int64_t ld_new,
                      const float *Wg /* [h x d] */, const float *bg /* [d] */,
                      float *out /* [n_halo x ld_out] */, int64_t ld_out)
{
    int32_t count = rows_sel ? n_sel : n_halo;
#pragma omp parallel
    {
        double *a = (double *)malloc(sizeof(double) * (size_t)h);
#pragma omp for schedule(dynamic, 16)
        for (int32_t idx = 0; idx < count; ++idx) {
            int32_t j = rows_sel ? rows_sel[idx] : idx;
            int32_t u = halo_gid[j];
            int32_t dt_u = dtil[u];
            const float *su = S + (int64_t)slot[u] * h;
            double puu = p_entry(dt_u, dt_u);
            for (int32_t q = 0; q < h; ++q) a[q] = puu * (double)su[q];
            for (int64_t e = hrow_ptr[j]; e < hrow_ptr[j + 1]; ++e) {
                int32_t v = inner_gid[hrow_col[e]];
                double p = p_entry(dt_u, dtil[v]);
                const float *sv = S + (int64_t)slot[v] * h;
                for (int32_t q = 0; q < h; ++q) a[q] += p * (double)sv[q];
            }
            for (int32_t c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int32_t q = 0; q < h; ++q) acc += a[q] * (double)Wg[(int64_t)q * d + c];
                acc += (double)bg[c];
                if (newest) acc += (double)newest[(int64_t)slot[u] * ld_new + c];
                out[(int64_t)j * ld_out + c] = (float)acc;
            }
        }
        free(a);
    }
}

/* ------------------------------------------------------------------------------------
 * O-8  Loss and its gradient with respect to the logits (Eq. "global loss" /
 * Eq. "local loss": L = sum_m w_m (1/|V_m|) sum_{v in V_m} Loss(h_v, y_v); with
 * w_m = |V_m| / N every node carries weight 1/N).
 *   softmax cross-entropy:  Loss_v = -log softmax(z_v)[y_v];  dLoss/dz = softmax(z) - onehot(y)
 *   sigmoid BCE (multi-label): Loss_v = (1/C) sum_c [softplus(z_c) - y_c z_c];
 *                              dLoss/dz_c = (sigm(z_c) - y_c) / C
 * Returns the sum over the given rows of scale * Loss_v; G = scale * dLoss/dz (fp32).
 * ---------------------------------------------------------------------------------- */
double orc_loss_ce(int32_t n, int32_t n_classes, const float *Z, int64_t ld_z, const int32_t *y,
                   double scale, float *G, int64_t ld_g)
{
    double total = 0.0;
    for (int32_t v = 0; v < n; ++v) {
        const float *z = Z + (int64_t)v * ld_z;
        double mx = (double)z[0];
        for (int32_t c = 1; c < n_classes; ++c)
            if ((double)z[c] > mx) mx = (double)z[c];
        double se = 0.0;
        for (int32_t c = 0; c < n_classes; ++c) se += exp((double)z[c] - mx);
        double lse = mx + log(se);
        total += scale * (lse - (double)z[y[v]]);
        if (G)
            for (int32_t c = 0; c < n_classes; ++c) {
                double pr = exp((double)z[c] - lse);
                G[(int64_t)v * ld_g + c] = (float)(scale * (pr - (c == y[v] ? 1.0 : 0.0)));
            }
    }
    return total;
}

double orc_loss_bce(int32_t n, int32_t n_labels, const float *Z, int64_t ld_z, const uint8_t *Y,
                    double scale, float *G, int64_t ld_g)
{
    double total = 0.0;
    for (int32_t v = 0; v < n; ++v) {
        const float *z = Z + (int64_t)v * ld_z;
        double acc = 0.0;
        for (int32_t c = 0; c < n_labels; ++c) {
            double x = (double)z[c], yv = (double)Y[(int64_t)v * n_labels + c];
            double sp = (x > 0.0 ? x : 0.0) + log1p(exp(-fabs(x))); /* softplus */
            acc += sp - yv * x;
            if (G) G[(int64_t)v * ld_g + c] = (float)(scale * (sigm(x) - yv) / (double)n_labels);
        }
        total += scale * acc / (double)n_labels;
    }
    return total;
}

/* ------------------------------------------------------------------------------------------
 * Lossy storage of historical embeddings (Supplement, "Data Compression for Historical Embedding
 * Storage"): the encoded-polyline scheme applied to every row of an embedding matrix.
 *   q_j = round-half-away-from-zero(x_j * 10^p)   (the product of an fp32 value and 10^p, p <= 7, is exact in fp64)
 *   e_0 = q_0,  e_j = q_j - q_{j-1}               (delta against the previous element of the row)
 *   v   = e << 1, bitwise inverted when e < 0     (sign folded into bit 0)
 *   5-bit groups of v, least significant first; every group but the last gets bit 0x20; each + 63 -> one ASCII byte
 * Rows are independent; row r occupies bytes [offset[r], offset[r+1]).
 * Decoding reverses the steps; x_hat_j = (float)((double)q_j / 10^p).
 * ------------------------------------------------------------------------------------------ */
static double pow10_int(int32_t p)
{
    double s = 1.0;
    for (int32_t i = 0; i < p; ++i) s *= 10.0;
    return s;
}

static int64_t codec_quantise(float x, double scale) { return (int64_t)llround((double)x * scale); }

static int32_t codec_put(int64_t e, uint8_t *out) /* writes the bytes of one signed integer, returns their number */
{
    uint64_t v = (uint64_t)e << 1;
    if (e < 0) v = ~v;
    int32_t n = 0;
    while (v >= 0x20) {
        if (out) out[n] = (uint8_t)((0x20 | (v & 0x1f)) + 63);
        ++n;
        v >>= 5;
    }
    if (out) out[n] = (uint8_t)(v + 63);
    return n + 1;
}

/* bytes per row into row_bytes[rows] */
void orc_codec_row_bytes(int64_t rows, int32_t d, const float *X, int64_t ld, int32_t p, int32_t *row_bytes)
{
    const double scale = pow10_int(p);
    for (int64_t r = 0; r < rows; ++r) {
        int64_t prev = 0;
        int32_t total = 0;
        for (int32_t j = 0; j < d; ++j) {
            const int64_t q = codec_quantise(X[r * ld + j], scale);
            total += codec_put(q - prev, (uint8_t *)0);
            prev = q;
        }
        row_bytes[r] = total;
    }
}

/* offsets[rows + 1] must hold the exclusive prefix sums of the row sizes */
void orc_codec_encode(int64_t rows, int32_t d, const float *X, int64_t ld, int32_t p, const int64_t *offsets, uint8_t *out)
{
    const double scale = pow10_int(p);
    for (int64_t r = 0; r < rows; ++r) {
        int64_t prev = 0;
        uint8_t *o = out + offsets[r];
        for (int32_t j = 0; j < d; ++j) {
            const int64_t q = codec_quantise(X[r * ld + j], scale);
            o += codec_put(q - prev, o);
            prev = q;
        }
    }
}

/* returns 0, or 1 + the index of the first malformed row (wrong number of values, or a value that does not end) */
int64_t orc_codec_decode(int64_t rows, int32_t d, const uint8_t *in, const int64_t *offsets, int32_t p, float *X, int64_t ld)
{
    const double scale = pow10_int(p);
    for (int64_t r = 0; r < rows; ++r) {
        int64_t pos = offsets[r], end = offsets[r + 1], q = 0;
        for (int32_t j = 0; j < d; ++j) {
            uint64_t v = 0;
            int shift = 0;
            for (;;) {
                if (pos >= end) return r + 1;
                const uint32_t c = (uint32_t)in[pos++] - 63u;
                v |= (uint64_t)(c & 0x1f) << shift;
                shift += 5;
                if (c < 0x20) break;
            }
            const int64_t e = (v & 1) ? ~(int64_t)(v >> 1) : (int64_t)(v >> 1);
            q += e;
            X[r * ld + j] = (float)((double)q / scale);
        }
        if (pos != end) return r + 1;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------
 * O-2 (partitioner)  Breadth-first visit order with a plain first-in first-out queue: start at node 0, neighbours of the
 * node taken off the queue are visited in ascending id (the CSR rows are sorted), and when the queue runs empty the
 * traversal restarts at the smallest unvisited id.  rank[v] = position of v in the visit order.  The partitioner built on
 * it cuts that order into M equal blocks (Algorithm 1, "Partitioning the raw graph": any non-overlapping partition will do).
 * ------------------------------------------------------------------------------------ */
void orc_bfs_rank(int32_t n, const int64_t *rowptr, const int32_t *col, int32_t *rank)
{
    int32_t *queue = (int32_t *)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
    for (int32_t v = 0; v < n; ++v) rank[v] = -1;
    int32_t head = 0, tail = 0, visited = 0;
    for (int32_t start = 0; start < n; ++start) {
        if (rank[start] >= 0) continue;
        rank[start] = visited++;
        queue[tail++] = start;
        while (head < tail) {
            int32_t u = queue[head++];
            for (int64_t e = rowptr[u]; e < rowptr[u + 1]; ++e) {
                int32_t w = col[e];
                if (rank[w] < 0) {
                    rank[w] = visited++;
                    queue[tail++] = w;
                }
            }
        }
    }
    free(queue);
}
