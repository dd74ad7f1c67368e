/*
 * CPU oracle for the binarized Bi-GCN forward layer (Bi-GCN, Sec. 3 and Sec. 4.1-4.2).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * forward path computes, one loop per definition, so that a reader can hold it
 * against the paper.  It shares nothing with the CUDA library: no header, no
 * helper, no table.  Only the test-suite, the smoke check and the timed CPU
 * baseline of the benchmark may call it; the product never does.
 *
 * Conventions taken where the paper is silent or misprinted:
 *   - sign(x) = +1 iff x >= 0 (so +0.0 and -0.0 give +1), else -1; a NaN gives -1.
 *   - the scalar of a bucket of t values is ||.||_1 / t with t = d_in for both
 *     the weight columns (Eq. "alpha", printed with 1/d_out) and the feature
 *     rows (Eq. "beta", printed with 1/N): the generic rule of Sec. 4.1.
 *   - every scalar sum is accumulated in double and rounded once to float.
 *   - zeta_ij = (beta_i * alpha_j) * (float)dot_ij, two float multiplications.
 *   - aggregation accumulates a row in double over the CSR entries in storage
 *     order and rounds once to float.
 *   - packed layout: element 32*w + k of a bucket is bit k (LSB = bit 0) of
 *     32-bit word w; +1 is stored as 1, -1 as 0; unused bits and words are 0.
 *
 * Parallelism: OpenMP over output rows only; every row is computed by one
 * thread from start to end, so results do not depend on the thread count.
 *
 * Pins (tests marked "not gpu"): brute force over all sign vectors for the
 * optimal (V_B, alpha) of Sec. 4.1; dense +-1 float matrix products for the
 * XNOR/bit-count contraction; dense N x N products and hand-worked star/path
 * graphs for the adjacency and the aggregation; the fp32 GCN layer of Eq. 1 on
 * +-1 inputs for the whole layer; Table 1 and the C.O./M.S./D.S. columns of
 * the result tables for the cost model; the GraphSAGE mean layer on +-1 inputs
 * for the Bi-GraphSAGE layer.  The numerical value of a full forward
 * on the paper's datasets is "parity unpinned": the paper prints no worked
 * numerical example and the datasets are not available.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_num_threads(int t)
{
#ifdef _OPENMP
    if (t > 0) omp_set_num_threads(t);
#else
    (void)t;
#endif
}

/* ------------------------------------------------------------------------- */
/* Sec. 3.1: A_hat = A + I, D_hat its degree matrix;                          */
/* Eq. 1:    A_tilde = D_hat^-1/2 A_hat D_hat^-1/2, kept sparse (CSR here).   */
/* ------------------------------------------------------------------------- */

static int cmp_i32(const void* a, const void* b)
{
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}

/*
 * Input: m ordered pairs (src[e], dst[e]) with ids in [0, n); any mix of
 * directions, duplicates and self pairs.  The graph is undirected (Sec. 3.1),
 * so a pair in either direction makes both a_uv = a_vu = 1; repeated pairs
 * count once; self pairs in the input are ignored and exactly one self-loop
 * per node is added (A_hat = A + I).
 *
 * Output: CSR of A_tilde.  rowptr[n+1]; colidx/val need room for 2*m + n
 * entries; columns ascending within a row; dinv[i] = 1/sqrt(D_hat_ii) computed
 * in double and rounded to float; val = dinv[i] * dinv[j] as a float product.
 * Returns nnz, or -1 on a bad id or failed allocation.
 */
int64_t oracle_normalize_adjacency(int64_t n, int64_t m, const int32_t* src, const int32_t* dst,
                                   int64_t* rowptr, int32_t* colidx, float* val, float* dinv)
{
    int64_t* start = (int64_t*)calloc((size_t)n + 1, sizeof(int64_t));
    if (!start) return -1;
    for (int64_t e = 0; e < m; ++e) {
        int32_t u = src[e], v = dst[e];
        if (u < 0 || u >= n || v < 0 || v >= n) { free(start); return -1; }
        if (u == v) continue;
        start[u + 1] += 1;
        start[v + 1] += 1;
    }
    for (int64_t i = 0; i < n; ++i) start[i + 1] += 1;           /* the self-loop of A + I */
    for (int64_t i = 0; i < n; ++i) start[i + 1] += start[i];
    int64_t total = start[n];
    int32_t* tmp = (int32_t*)malloc((size_t)(total > 0 ? total : 1) * sizeof(int32_t));
    int64_t* fill = (int64_t*)malloc((size_t)(n > 0 ? n : 1) * sizeof(int64_t));
    if (!tmp || !fill) { free(start); free(tmp); free(fill); return -1; }
    for (int64_t i = 0; i < n; ++i) { fill[i] = start[i]; tmp[fill[i]++] = (int32_t)i; }
    for (int64_t e = 0; e < m; ++e) {
        int32_t u = src[e], v = dst[e];
        if (u == v) continue;
        tmp[fill[u]++] = v;
        tmp[fill[v]++] = u;
    }
    /* sort each row and drop repeats; count what is left */
    rowptr[0] = 0;
    for (int64_t i = 0; i < n; ++i) {
        int64_t a = start[i], b = start[i + 1];
        qsort(tmp + a, (size_t)(b - a), sizeof(int32_t), cmp_i32);
        int64_t kept = 0;
        for (int64_t p = a; p < b; ++p)
            if (p == a || tmp[p] != tmp[p - 1]) tmp[a + kept++] = tmp[p];
        rowptr[i + 1] = rowptr[i] + kept;
    }
    for (int64_t i = 0; i < n; ++i) {
        int64_t deg_hat = rowptr[i + 1] - rowptr[i];             /* D_hat_ii = sum_j a_hat_ij */
        dinv[i] = (float)(1.0 / sqrt((double)deg_hat));
        memcpy(colidx + rowptr[i], tmp + start[i], (size_t)deg_hat * sizeof(int32_t));
    }
    for (int64_t i = 0; i < n; ++i)
        for (int64_t p = rowptr[i]; p < rowptr[i + 1]; ++p)
            val[p] = dinv[i] * dinv[colidx[p]];
    free(start); free(tmp); free(fill);
    return rowptr[n];
}

/* ------------------------------------------------------------------------- */
/* Sec. 4.4, step one of the general recipe: batch normalisation of a layer's */
/* input to zero mean and unit variance per feature (column) over the nodes.  */
/* Inference form: shift_j = mean_j, scale_j = 1/sqrt(var_j + eps), biased    */
/* variance, no affine part.                                                  */
/* ------------------------------------------------------------------------- */
void oracle_col_stats(const float* H, int64_t n, int32_t d, int64_t ld, double eps,
                      float* shift, float* scale)
{
#pragma omp parallel for schedule(static)
    for (int32_t j = 0; j < d; ++j) {
        double s = 0.0;
        for (int64_t i = 0; i < n; ++i) s += (double)H[i * ld + j];
        double mean = n > 0 ? s / (double)n : 0.0;
        double q = 0.0;
        for (int64_t i = 0; i < n; ++i) {
            double c = (double)H[i * ld + j] - mean;
            q += c * c;
        }
        double var = n > 0 ? q / (double)n : 0.0;
        shift[j] = (float)mean;
        scale[j] = (float)(1.0 / sqrt(var + eps));
    }
}

/* x_hat = (h - shift) * scale, one float subtraction then one float product */
static inline float bn_apply(float h, const float* shift, const float* scale, int32_t j)
{
    if (!shift) return h;
    volatile float c = h - shift[j];     /* volatile: keep the two roundings separate */
    volatile float r = c * scale[j];
    return r;
}

/* ------------------------------------------------------------------------- */
/* Sec. 4.2.2: F_i = sign(H_i,:), beta_i = ||H_i,:||_1 / d_in  (row buckets)  */
/* applied to the batch-normalised input when shift/scale are given.          */
/* F is a +-1 matrix in int8, row-major n x d.                                */
/* ------------------------------------------------------------------------- */
void oracle_binarize_rows(const float* H, int64_t n, int32_t d, int64_t ld,
                          const float* shift, const float* scale, int8_t* F, float* beta)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        double l1 = 0.0;
        for (int32_t j = 0; j < d; ++j) {
            float x = bn_apply(H[i * ld + j], shift, scale, j);
            F[i * (int64_t)d + j] = (x >= 0.0f) ? 1 : -1;
            l1 += fabs((double)x);
        }
        beta[i] = (float)(l1 / (double)d);
    }
}

/* ------------------------------------------------------------------------- */
/* Sec. 4.2.1: B_j = sign(W_:,j), alpha_j = ||W_:,j||_1 / d_in (column        */
/* buckets).  B is a +-1 matrix in int8, row-major d_in x d_out.              */
/* ------------------------------------------------------------------------- */
void oracle_binarize_cols(const float* W, int32_t d_in, int32_t d_out, int64_t ldw,
                          int8_t* B, float* alpha)
{
    for (int32_t j = 0; j < d_out; ++j) {
        double l1 = 0.0;
        for (int32_t k = 0; k < d_in; ++k) {
            float w = W[k * ldw + j];
            B[(int64_t)k * d_out + j] = (w >= 0.0f) ? 1 : -1;
            l1 += fabs((double)w);
        }
        alpha[j] = (float)(l1 / (double)d_in);
    }
}

/* ------------------------------------------------------------------------- */
/* Storage of Sec. 5.1-5.2: one bit per element plus one float per bucket.    */
/* Row i of F (length d) -> stride 32-bit words, of which ceil(d/32) are used.*/
/* ------------------------------------------------------------------------- */
void oracle_pack_rows(const int8_t* F, int64_t n, int32_t d, uint32_t* bits, int64_t stride)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {
        for (int64_t w = 0; w < stride; ++w) bits[i * stride + w] = 0u;
        for (int32_t j = 0; j < d; ++j)
            if (F[i * (int64_t)d + j] > 0) bits[i * stride + (j >> 5)] |= (1u << (j & 31));
    }
}

/* Column j of B (length d_in) -> row j of the packed, transposed weight matrix */
void oracle_pack_cols(const int8_t* B, int32_t d_in, int32_t d_out, uint32_t* bitsT, int64_t stride)
{
    for (int32_t j = 0; j < d_out; ++j) {
        for (int64_t w = 0; w < stride; ++w) bitsT[j * stride + w] = 0u;
        for (int32_t k = 0; k < d_in; ++k)
            if (B[(int64_t)k * d_out + j] > 0) bitsT[j * stride + (k >> 5)] |= (1u << (k & 31));
    }
}

/* inverse of the two packers: bit -> +-1, for the round-trip pin */
void oracle_unpack_rows(const uint32_t* bits, int64_t stride, int64_t n, int32_t d, int8_t* F)
{
    for (int64_t i = 0; i < n; ++i)
        for (int32_t j = 0; j < d; ++j)
            F[i * (int64_t)d + j] = ((bits[i * stride + (j >> 5)] >> (j & 31)) & 1u) ? 1 : -1;
}

/* ------------------------------------------------------------------------- */
/* Eq. "cdot-op": the inner product F_i,: . B_:,j of two +-1 vectors,         */
/* written out term by term.                                                  */
/* ------------------------------------------------------------------------- */
void oracle_dot_pm1(const int8_t* F, const int8_t* B, int64_t n, int32_t d_in, int32_t d_out,
                    int32_t* dot)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int32_t j = 0; j < d_out; ++j) {
            int32_t s = 0;
            for (int32_t k = 0; k < d_in; ++k)
                s += (int32_t)F[i * (int64_t)d_in + k] * (int32_t)B[(int64_t)k * d_out + j];
            dot[i * (int64_t)d_out + j] = s;
        }
}

/* bit count of a word (the compiler's population-count primitive) */
static inline int32_t count_ones(uint32_t x) { return (int32_t)__builtin_popcount(x); }

/* ------------------------------------------------------------------------- */
/* Eq. "bi-op": the same inner product by XNOR and bit count.  Over the d_in  */
/* valid positions, agreements = d_in - popc(a XOR b), so                     */
/* dot = agreements - disagreements = d_in - 2 * popc(a XOR b).               */
/* Pad bits are 0 in both operands and so never count as disagreements.       */
/* ------------------------------------------------------------------------- */
void oracle_dot_popc(const uint32_t* bits, int64_t stride_a, const uint32_t* bitsT, int64_t stride_b,
                     int64_t n, int32_t d_in, int32_t d_out, int32_t* dot)
{
    int32_t kw = (d_in + 31) / 32;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int32_t j = 0; j < d_out; ++j) {
            int32_t differ = 0;
            for (int32_t w = 0; w < kw; ++w)
                differ += count_ones(bits[i * stride_a + w] ^ bitsT[j * stride_b + w]);
            dot[i * (int64_t)d_out + j] = d_in - 2 * differ;
        }
}

/* zeta_ij = beta_i alpha_j (F_i . B_j)   (Eq. "cdot-op" / "bi-op") */
void oracle_rescale(const int32_t* dot, const float* beta, const float* alpha,
                    int64_t n, int32_t d_out, float* zeta, int64_t ldz)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i)
        for (int32_t j = 0; j < d_out; ++j) {
            volatile float ba = beta[i] * alpha[j];
            zeta[i * ldz + j] = ba * (float)dot[i * (int64_t)d_out + j];
        }
}

/* ------------------------------------------------------------------------- */
/* H_b^(l+1) = A_tilde zeta^(l)  (last equation of Sec. 4.2.3): for each node */
/* the weighted sum of the zeta rows of its neighbours and itself.            */
/* rowptr may be offset to a slice of rows: entries index colidx absolutely.  */
/* ------------------------------------------------------------------------- */
void oracle_spmm(int64_t n_rows, const int64_t* rowptr, const int32_t* colidx, const float* val,
                 const float* zeta, int32_t d_out, int64_t ldz, float* out, int64_t ldo)
{
#pragma omp parallel
    {
        double* acc = (double*)malloc((size_t)(d_out > 0 ? d_out : 1) * sizeof(double));
#pragma omp for schedule(dynamic, 64)
        for (int64_t i = 0; i < n_rows; ++i) {
            for (int32_t j = 0; j < d_out; ++j) acc[j] = 0.0;
            for (int64_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
                double a = (double)val[p];
                const float* z = zeta + (int64_t)colidx[p] * ldz;
                for (int32_t j = 0; j < d_out; ++j) acc[j] += a * (double)z[j];
            }
            for (int32_t j = 0; j < d_out; ++j) out[i * ldo + j] = (float)acc[j];
        }
        free(acc);
    }
}

/* ------------------------------------------------------------------------- */
/* Bi-GraphSAGE (Sec. 4.4.2, Eq. "bisage-conv"): the mean aggregator           */
/*   h_i' = W_theta (*) h_i + (1/|N_i|) sum_{j in N_i} W_n (*) h_j             */
/* needs the neighbourhood matrix with rows scaled by 1/|N_i|: N_i is the set  */
/* of distinct neighbours of i (no self-loop); a node without neighbours gets  */
/* an empty row (its neighbour term is 0).                                     */
/* Same input convention as oracle_normalize_adjacency.  colidx/val need room  */
/* for 2*m entries; inv_deg[i] = (float)(1.0/|N_i|), 0 for isolated nodes;     */
/* val = inv_deg[i] on every entry of row i.  Returns nnz or -1.               */
/* ------------------------------------------------------------------------- */
int64_t oracle_mean_adjacency(int64_t n, int64_t m, const int32_t* src, const int32_t* dst,
                              int64_t* rowptr, int32_t* colidx, float* val, float* inv_deg)
{
    int64_t* start = (int64_t*)calloc((size_t)n + 1, sizeof(int64_t));
    if (!start) return -1;
    for (int64_t e = 0; e < m; ++e) {
        int32_t u = src[e], v = dst[e];
        if (u < 0 || u >= n || v < 0 || v >= n) { free(start); return -1; }
        if (u == v) continue;
        start[u + 1] += 1;
        start[v + 1] += 1;
    }
    for (int64_t i = 0; i < n; ++i) start[i + 1] += start[i];
    int64_t total = start[n];
    int32_t* tmp = (int32_t*)malloc((size_t)(total > 0 ? total : 1) * sizeof(int32_t));
    int64_t* fill = (int64_t*)malloc((size_t)(n > 0 ? n : 1) * sizeof(int64_t));
    if (!tmp || !fill) { free(start); free(tmp); free(fill); return -1; }
    for (int64_t i = 0; i < n; ++i) fill[i] = start[i];
    for (int64_t e = 0; e < m; ++e) {
        int32_t u = src[e], v = dst[e];
        if (u == v) continue;
        tmp[fill[u]++] = v;
        tmp[fill[v]++] = u;
    }
    rowptr[0] = 0;
    for (int64_t i = 0; i < n; ++i) {
        int64_t a = start[i], b = start[i + 1];
        qsort(tmp + a, (size_t)(b - a), sizeof(int32_t), cmp_i32);
        int64_t kept = 0;
        for (int64_t p = a; p < b; ++p)
            if (p == a || tmp[p] != tmp[p - 1]) tmp[a + kept++] = tmp[p];
        rowptr[i + 1] = rowptr[i] + kept;
    }
    for (int64_t i = 0; i < n; ++i) {
        int64_t deg = rowptr[i + 1] - rowptr[i];                  /* |N_i| */
        inv_deg[i] = deg > 0 ? (float)(1.0 / (double)deg) : 0.0f;
        memcpy(colidx + rowptr[i], tmp + start[i], (size_t)deg * sizeof(int32_t));
        for (int64_t p = rowptr[i]; p < rowptr[i + 1]; ++p) val[p] = inv_deg[i];
    }
    free(start); free(tmp); free(fill);
    return rowptr[n];
}

/* out_i,: = self_i,: + sum_{k in row i} val_ik * z_k,:   -- the two terms of Eq. "bisage-conv"      */
/* added in double and rounded once (self may be NULL: then this is oracle_spmm).                   */
void oracle_spmm_add(int64_t n_rows, const int64_t* rowptr, const int32_t* colidx, const float* val,
                     const float* z, int32_t d_out, int64_t ldz, const float* self, int64_t lds,
                     float* out, int64_t ldo)
{
#pragma omp parallel
    {
        double* acc = (double*)malloc((size_t)(d_out > 0 ? d_out : 1) * sizeof(double));
#pragma omp for schedule(dynamic, 64)
        for (int64_t i = 0; i < n_rows; ++i) {
            for (int32_t j = 0; j < d_out; ++j) acc[j] = self ? (double)self[i * lds + j] : 0.0;
            for (int64_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
                double a = (double)val[p];
                const float* zr = z + (int64_t)colidx[p] * ldz;
                for (int32_t j = 0; j < d_out; ++j) acc[j] += a * (double)zr[j];
            }
            for (int32_t j = 0; j < d_out; ++j) out[i * ldo + j] = (float)acc[j];
        }
        free(acc);
    }
}

/* ------------------------------------------------------------------------- */
/* Sec. 5 cost model: storage bits and operation counts of an L-layer GCN and */
/* its binarized form on a graph with n nodes and e edges (as the paper       */
/* counts them).  dims[0..L].  One "cycle operation" = one multiply + one     */
/* add = 64 binary operations (Sec. 5.3).                                     */
/* out[0] = GCN cycle ops, out[1] = Bi-GCN cycle ops,                         */
/* out[2] = GCN model bytes, out[3] = Bi-GCN model bytes,                     */
/* out[4] = GCN data bytes,  out[5] = Bi-GCN data bytes.                      */
/* ------------------------------------------------------------------------- */
void oracle_cost_model(double n, double e, const int32_t* dims, int32_t n_layers, double* out)
{
    double ops_fp = 0.0, ops_bi = 0.0, model_fp_bits = 0.0, model_bi_bits = 0.0;
    for (int32_t l = 0; l < n_layers; ++l) {
        double din = dims[l], dout = dims[l + 1];
        ops_fp += n * din * dout + e * dout;                         /* numerator of Eq. "S-full" */
        ops_bi += n * din * dout / 64.0 + 2.0 * n * dout + e * dout; /* its denominator */
        model_fp_bits += 32.0 * din * dout;                          /* Eq. "pc-l" numerator */
        model_bi_bits += din * dout + 32.0 * dout;                   /* its denominator */
    }
    double d0 = dims[0];
    out[0] = ops_fp;
    out[1] = ops_bi;
    out[2] = model_fp_bits / 8.0;
    out[3] = model_bi_bits / 8.0;
    out[4] = 32.0 * n * d0 / 8.0;                                    /* Eq. "DC" numerator */
    out[5] = (n * d0 + 32.0 * n) / 8.0;                              /* its denominator */
}

/* ------------------------------------------------------------------------- */
/* Sec. 6.2 "Entropy Estimation of Hidden Layers": the binning estimate.      */
/* For neuron (column) i over the N samples (rows): the value range           */
/* [min_i, max_i] is cut into M intervals of equal width, p_{i,m} is the      */
/* fraction of samples in interval m (the empirical distribution), and        */
/*     H_hat(h_i) = - sum_m p_{i,m} log p_{i,m}.                              */
/* The layer estimate is the independent sum H_ind(h) = sum_i H_hat(h_i).     */
/* Readings (the paper fixes neither): equal-width intervals over the         */
/* column's own range; the largest value falls into the last interval; a      */
/* constant column has entropy 0; the logarithm is base 2 (bits), which the   */
/* paper's own table forces (its PubMed value exceeds 16 ln 200).             */
/* The interval index is decided in fp32, in this order:                      */
/*     scale = (float)M / (max - min);  m = (int)((x - min) * scale)          */
/* then clamped to M - 1.  Inputs must be finite.                             */
/* counts: d x M, entropy: d values in bits.  Returns H_ind.                  */
/* ------------------------------------------------------------------------- */
double oracle_entropy_bins(const float* H, int64_t n, int32_t d, int64_t ld, int32_t M,
                           float* col_min, float* col_max, int64_t* counts, double* entropy)
{
    double total = 0.0;
    for (int32_t j = 0; j < d; ++j) {
        float lo = INFINITY, hi = -INFINITY;
        for (int64_t i = 0; i < n; ++i) {
            const float x = H[i * ld + j];
            if (x < lo) lo = x;
            if (x > hi) hi = x;
        }
        col_min[j] = lo;
        col_max[j] = hi;
        int64_t* c = counts + (int64_t)j * M;
        for (int32_t m = 0; m < M; ++m) c[m] = 0;
        if (n > 0) {
            if (hi > lo) {
                const float scale = (float)M / (hi - lo);
                for (int64_t i = 0; i < n; ++i) {
                    const float t = (H[i * ld + j] - lo) * scale;
                    int32_t m = (int32_t)t;
                    if (m > M - 1) m = M - 1;
                    c[m] += 1;
                }
            } else {
                c[0] = n;                      /* every sample has the same value */
            }
        }
        double h = 0.0;
        for (int32_t m = 0; m < M; ++m) {
            if (c[m] > 0) {
                const double p = (double)c[m] / (double)n;
                h -= p * log2(p);
            }
        }
        entropy[j] = h;
        total += h;
    }
    return total;
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1 (Sec. 4.3): back-propagation through one binarized graph       */
/* convolutional layer  H' = A_tilde (H~ W~),  H~_ik = beta_i F_ik,           */
/* W~_kj = alpha_j B_kj.  Given G' = dL/dH' (n x d_out):                      */
/*   step 1:  G_zeta = A_tilde^T G'                                           */
/*            G_W~   = H~^T G_zeta            (d_in x d_out)                  */
/*            G_H~   = G_zeta W~^T            (n x d_in)                      */
/*   step 2 (Eq. bp-H):  G_H = G_H~ where |G_H~| < 1, else 0                  */
/*   step 3 (Eq. bp-W):  G_W_ij = (1/d_in) B_ij sum_k G_W~_kj B_kj            */
/*                               + alpha_j G_W~_ij [ |W_ij| < 1 ]             */
/*            (the last factor is the straight-through estimate of            */
/*             d sign(r)/dr = 1_{|r|<1}).                                     */
/* Step 4 of the algorithm (the parameter update) belongs to the optimiser    */
/* and is not part of this function.  A_tilde^T is applied as a true          */
/* transpose: entry (i, k) of A_tilde sends row i of G' to row k of G_zeta.   */
/* All sums in double; every output rounded to float once.  g_zeta, g_wt,     */
/* g_ht are the intermediate results (nullable).                              */
/* ------------------------------------------------------------------------- */
void oracle_layer_backward(int64_t n, const int64_t* rowptr, const int32_t* colidx, const float* val,
                           int32_t d_in, int32_t d_out, const int8_t* F, const float* beta,
                           const int8_t* B, const float* alpha, const float* W,
                           const float* G_out, float* g_zeta, float* g_wt, float* g_ht,
                           float* g_h, float* g_w)
{
    double* gz = (double*)calloc((size_t)n * d_out, sizeof(double));
    double* gwt = (double*)calloc((size_t)d_in * d_out, sizeof(double));
    /* G_zeta = A_tilde^T G' */
    for (int64_t i = 0; i < n; ++i)
        for (int64_t e = rowptr[i]; e < rowptr[i + 1]; ++e) {
            const int64_t k = colidx[e];
            for (int32_t j = 0; j < d_out; ++j) gz[k * d_out + j] += (double)val[e] * (double)G_out[i * d_out + j];
        }
    /* G_W~ = H~^T G_zeta */
    for (int64_t i = 0; i < n; ++i)
        for (int32_t k = 0; k < d_in; ++k) {
            const double h = (double)beta[i] * (double)F[i * d_in + k];
            for (int32_t j = 0; j < d_out; ++j) gwt[(int64_t)k * d_out + j] += h * gz[i * d_out + j];
        }
    /* G_H~ = G_zeta W~^T, then Eq. bp-H */
    for (int64_t i = 0; i < n; ++i)
        for (int32_t k = 0; k < d_in; ++k) {
            double s = 0.0;
            for (int32_t j = 0; j < d_out; ++j)
                s += gz[i * d_out + j] * ((double)alpha[j] * (double)B[(int64_t)k * d_out + j]);
            if (g_ht) g_ht[i * d_in + k] = (float)s;
            if (g_h) g_h[i * d_in + k] = (fabs(s) < 1.0) ? (float)s : 0.f;
        }
    /* Eq. bp-W */
    for (int32_t j = 0; j < d_out; ++j) {
        double col = 0.0;                                  /* sum_k G_W~_kj B_kj */
        for (int32_t k = 0; k < d_in; ++k) col += gwt[(int64_t)k * d_out + j] * (double)B[(int64_t)k * d_out + j];
        for (int32_t i = 0; i < d_in; ++i) {
            const int64_t at = (int64_t)i * d_out + j;
            double g = (double)B[at] * col / (double)d_in;
            if (fabsf(W[at]) < 1.0f) g += (double)alpha[j] * gwt[at];
            if (g_w) g_w[at] = (float)g;
        }
    }
    if (g_zeta) for (int64_t t = 0; t < n * d_out; ++t) g_zeta[t] = (float)gz[t];
    if (g_wt) for (int64_t t = 0; t < (int64_t)d_in * d_out; ++t) g_wt[t] = (float)gwt[t];
    free(gz);
    free(gwt);
}
