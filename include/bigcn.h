/*
 * bigcn.h - C ABI of the binarized Bi-GCN forward layer for NVIDIA B200 (sm_100a).
 *
 * The library implements the forward path of "Binary Graph Convolutional Network with Capacity
 * Exploration" (Bi-GCN): feature / weight binarization with bit packing (Sec. 4.2.1, 4.2.2), the
 * XNOR + bit-count contraction with its beta_i alpha_j rescale (Sec. 4.2.3, Eq. "cdot-op" and
 * "bi-op"; computed as int8 tensor-core products on the bits expanded to +1 / -1 where the layer is
 * narrow enough, see BIGCN_OPT_CONTRACTION: the same integers), and the floating-point aggregation with A_tilde = D_hat^-1/2 (A + I) D_hat^-1/2
 * (Eq. 1; last equation of Sec. 4.2.3), whose output can be re-binarized for the next layer.
 *
 * General rules
 *   - Every data pointer is a DEVICE pointer owned by the caller unless a comment says "host".
 *     The library allocates no data buffers: scratch comes from the workspace the caller attaches
 *     with bigcn_set_workspace().  A context owns only a few hundred bytes of device status words
 *     and some CUDA events.
 *   - All work is enqueued on the stream given to bigcn_create() (borrowed, not owned).  Calls are
 *     asynchronous unless stated; results are ready once that stream has been synchronised.
 *   - Matrices are row-major; leading dimensions ("ld") are in elements, packed strides in 32-bit
 *     words.  Outputs must not alias inputs.  n = 0 is a valid no-op.
 *   - Arguments are validated on the host before anything is launched; a failing call launches
 *     nothing, returns a status other than BIGCN_OK and leaves a message in bigcn_last_error().
 *   - There is no CPU fallback: without a CUDA device every compute entry point fails.
 *
 * Packed layout (the paper fixes "1 bit per element plus one 32-bit float per bucket", Sec. 5.1-5.2,
 * not the bit order; this is the order used here): element 32*w + k of a bucket is bit k (bit 0 =
 * least significant) of 32-bit word w; +1 is stored as 1 and -1 as 0; bits past the bucket length
 * and words past ceil(len/32) are 0.  A packed row occupies bigcn_packed_stride_words(len) words:
 * ceil(len/32) rounded up to a multiple of 4, so that every row starts on a 16-byte boundary.
 * sign(x) = +1 iff x >= 0 (both zeros give +1; a NaN gives -1).
 */
#ifndef BIGCN_H
#define BIGCN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BIGCN_MAX_LAYERS 16
/* Widest layer the contraction kernels serve: the packed K extent of a tile of feature rows and of the
 * weight panel is kept in shared memory.  A layer with d_in above this, or d_out above
 * BIGCN_MAX_D_OUT, is refused with BIGCN_ERR_UNSUPPORTED before anything is launched. */
#define BIGCN_MAX_D_IN 16384
#define BIGCN_MAX_D_OUT 512

typedef enum {
    BIGCN_OK = 0,
    BIGCN_ERR_NULL = 1,        /* a required pointer is null */
    BIGCN_ERR_SHAPE = 2,       /* a size, leading dimension or stride is out of range */
    BIGCN_ERR_ALIGN = 3,       /* a pointer is not aligned as documented */
    BIGCN_ERR_GRAPH = 4,       /* the sparse structure is malformed */
    BIGCN_ERR_WORKSPACE = 5,   /* no workspace attached, or it is too small */
    BIGCN_ERR_CUDA = 6,        /* a CUDA runtime call failed (message in bigcn_last_error) */
    BIGCN_ERR_UNSUPPORTED = 7, /* a valid request this build does not implement */
    BIGCN_ERR_INTERNAL = 8,    /* a device-side self-check tripped */
    BIGCN_ERR_BUSY = 9         /* every slot of a pipeline holds a step that has not been waited for */
} bigcn_status;

typedef struct bigcn_ctx bigcn_ctx;

/* Options for bigcn_set_option(). */
enum {
    /* Storage of the rescaled contraction zeta between the bit-GEMM and the aggregation.
     * 0 = choose per layer (default: for 129..256 output columns, where the aggregation streams 256-byte
     *     rows, and for 33..64 output columns of a layer whose result is only written out as fp32 (no next
     *     layer) or of a hidden layer on a graph whose rows average at least 8 stored entries (the aggregation
     *     then streams one stored entry per lane), 3 when d_in <= 127 and 5 when 128 <= d_in <= 256 and the
     *     layer has at least 2^20 outputs;
     *     otherwise 4 when d_in <= 2048, else 2);
     * 1 = fp32 zeta_ij = (beta_i alpha_j) dot_ij, exactly Eq. "cdot-op";
     * 2 = the integer dot products as int16, with beta folded into the edge weights and alpha
     *     applied once per output element (same sum, different rounding order);
     * 3 = as 2 but int8 (layers with d_in <= 127 only; others fall back to 4);
     * 4 = as 2 but the integers held as fp16, which is exact for |dot| <= 2048 (layers with
     *     d_in <= 2048 only; others fall back to 2);
     * 5 = signed bytes for 128 <= d_in <= 256 and up to 256 output columns (other layers as 0; the automatic
     *     choice takes it for 129..256 output columns, and for 33..64 as described under 0): the byte is
     *     s = (dot' - 1) / 2, dot' the dot without its first position when d_in is even (so that dot' is
     *     odd and s fits a byte exactly); the aggregation adds back sum_k w_k (1 + f_k0 b_0j), two per-row
     *     sums that ride along with the edge weights.  Exact in the integers; on the tensor-core contraction. */
    BIGCN_OPT_ZETA_FORMAT = 1,
    /* Rows of the sparse matrix with more entries than this are split across thread blocks. 0 = default. */
    BIGCN_OPT_LONG_ROW = 2,
    /* How the binary contraction runs.  0 = default: as int8 tensor-core products (tcgen05, the packed bits
     * expanded to +1 / -1 bytes in shared memory; the same integers) for layers with d_in <= 256 and
     * d_out <= 256 and at least 2^20 outputs, on the XOR / bit-count pipe otherwise; 1 = always on the
     * XOR / bit-count pipe; 2 = tensor cores for every layer with d_in <= 256 and d_out <= 256. */
    BIGCN_OPT_CONTRACTION = 3,
    /* How rows of 129..256 signed bytes (zeta formats 3 and 5) are aggregated.
     * 1 = the fp32 FMA stream (bytes converted to fp32 one by one; with format 5 this stream takes the edge values
     *     as non-negative, as those of the normalized adjacency are);
     * 2 = exact integer products on the tensor cores through mma.sync (s8 x s8 -> s32: the edge weights of up to 32
     *     stored entries of a row in 28..31-bit fixed point against a common power of two, split into four signed
     *     base-256 digits; the digit sums recombined in fp32 when the row ends; edge values of either sign);
     * 3 = the same fixed-point digits on the 5th-generation tensor cores (tcgen05.mma kind::i8: the gathered rows
     *     of 64 stored entries go by asynchronous copies straight into shared memory as the swizzled A operand, the
     *     digits of the edge weights are the B operand, the digit sums are read back from tensor memory once per
     *     row segment; graphs of fewer than 2^31 stored entries, otherwise the FMA stream runs);
     * 0 = default: 3 for a launch that wants only the next layer's sign bits and beta (a hidden layer inside
     *     bigcn_forward) on a graph whose rows average at least 8 stored entries, 1 otherwise.  Measured on the two
     *     256-column layers of a 2.4 M-node, 126 M-entry graph, bits and beta only: 4.9 / 5.2 ms for 3,
     *     5.7-5.9 / 5.9-6.1 ms for 1, 8.0 / 8.3 ms for 2.  All paths meet the same tolerance; their fp32 sums differ
     *     in rounding, so a re-binarized bit at the threshold may differ between them. */
    BIGCN_OPT_BYTE_AGGREGATION = 4
};

/* Context: binds a device and a stream.  `cuda_stream` is a cudaStream_t (0 = default stream). */
bigcn_status bigcn_create(bigcn_ctx** out, int device, void* cuda_stream);
bigcn_status bigcn_destroy(bigcn_ctx* ctx);
/* Message of the last failing call on this context ("" if none).  Host string owned by ctx. */
const char* bigcn_last_error(const bigcn_ctx* ctx);
const char* bigcn_status_string(bigcn_status s);
bigcn_status bigcn_set_option(bigcn_ctx* ctx, int32_t option, int64_t value);
/* Number of kernels this context has launched so far. */
int64_t bigcn_launch_count(const bigcn_ctx* ctx);
/* Synchronises the stream and reports a pending CUDA error or a tripped device self-check. */
bigcn_status bigcn_sync_check(bigcn_ctx* ctx);

/* Words per packed row of `len` elements: ceil(len/32) rounded up to a multiple of 4. */
int64_t bigcn_packed_stride_words(int32_t len);

/* Scratch.  bigcn_workspace_bytes() bounds what bigcn_forward()/bigcn_layer_forward() need for a
 * graph of n nodes and nnz stored entries and the layer widths dims[0..n_layers];
 * with host_io = 1 it adds the staging buffers of bigcn_forward_host(), with host_io = k > 1 those
 * of a pipeline with k slots (bigcn_pipeline_open).
 * bigcn_set_workspace() attaches caller-owned device memory (256-byte aligned) until replaced. */
size_t bigcn_workspace_bytes(int64_t n, int64_t nnz, const int32_t* dims /*host*/, int32_t n_layers,
                             int32_t host_io);
bigcn_status bigcn_set_workspace(bigcn_ctx* ctx, void* workspace, size_t bytes);

/* Sparse normalised adjacency in CSR (Eq. 1: A_tilde = D_hat^-1/2 (A + I) D_hat^-1/2, "a sparse
 * matrix").  rowptr[n+1] int64, colidx[nnz] int32 ascending within a row and including the
 * diagonal, val[nnz] fp32 = dinv[i] * dinv[j], dinv[n] fp32 = D_hat_ii^-1/2.  n < 2^31. */
typedef struct {
    int64_t n;
    int64_t nnz;
    const int64_t* rowptr;
    const int32_t* colidx;
    const float* val;
    const float* dinv;
} bigcn_graph;

/* Set-up from a raw list of node pairs (Sec. 3.1: an undirected graph; A_hat = A + I).  src, dst int32 [m] in DEVICE
 * memory, node ids in [0, n): any order, either or both directions, repeats and self pairs allowed.  Every pair
 * (u, v) with u != v contributes the entries (u, v) and (v, u); repeats and self pairs are dropped (the one self-loop
 * per node is added by bigcn_normalize_adjacency()).  Output: the pattern of A as the CSR that
 * bigcn_normalize_adjacency() takes -- rowptr_A int64 [n + 1], colidx_A int32 with room for 2 m entries (ascending
 * and unique within a row, symmetric, no diagonal); *nnz_out = entries written.  m < 2^30.
 * Needs bigcn_edges_workspace_bytes(n, m) of workspace (about 32 m bytes: two buffers of 64-bit sort keys and the
 * scratch of the CUDA toolkit's device-wide sort and de-duplication, which this set-up step uses).  SYNCHRONOUS.
 * BIGCN_ERR_GRAPH if a node id lies outside [0, n). */
size_t bigcn_edges_workspace_bytes(int64_t n, int64_t m);
bigcn_status bigcn_adjacency_from_edges(bigcn_ctx* ctx, int64_t n, int64_t m, const int32_t* src, const int32_t* dst,
                                        int64_t* rowptr_A, int32_t* colidx_A, int64_t* nnz_out /*host*/);

/* Set-up step, once per graph (Sec. 3.1, Eq. 1).  Input: CSR of the adjacency A of an undirected
 * graph: symmetric pattern, columns ascending and unique within a row; diagonal entries in the
 * input are ignored and exactly one self-loop per node is added (A_hat = A + I).
 * Output arrays must hold nnz_in + n entries (colidx, val), n + 1 (rowptr) and n (dinv).
 * D_hat_ii = number of stored entries of row i of A_hat; dinv = 1/sqrt(D_hat_ii) evaluated in
 * double and rounded to fp32; val = fp32 product dinv[i] * dinv[j].
 * The input is checked on the device (ascending unique columns in [0, n), symmetry); a violation
 * gives BIGCN_ERR_GRAPH.  Needs 16 * (n/1024 + 2) + 64 bytes of workspace.  SYNCHRONOUS: returns after the
 * stream has drained; *nnz_out (host) receives the number of stored entries. */
bigcn_status bigcn_normalize_adjacency(bigcn_ctx* ctx, int64_t n, int64_t nnz_in,
                                       const int64_t* rowptr_A, const int32_t* colidx_A,
                                       int64_t* rowptr, int32_t* colidx, float* val, float* dinv,
                                       int64_t* nnz_out /*host*/);

/* Feature binarization (Sec. 4.2.2, Eq. "beta" and "F"; batch normalisation of the input as in
 * Sec. 4.4).  H fp32 [n x d], leading dimension ld >= d.  With col_shift/col_scale (fp32 [d], both
 * or neither) x_hat_ij = (H_ij - shift_j) * scale_j in fp32, else x_hat = H.
 * bits_out u32 [n x stride_words] gets F_i = sign(x_hat_i,:) in the packed layout (stride_words >=
 * bigcn_packed_stride_words(d), multiple of 4; every word of the row is written); beta_out fp32 [n]
 * gets ||x_hat_i,:||_1 / d (the bucket length; Eq. "beta" prints 1/N, see the generic rule of
 * Sec. 4.1).  bits_out must be 16-byte aligned. */
bigcn_status bigcn_pack_features(bigcn_ctx* ctx, const float* H, int64_t n, int32_t d, int64_t ld,
                                 const float* col_shift, const float* col_scale,
                                 uint32_t* bits_out, int64_t stride_words, float* beta_out);

/* Weight binarization (Sec. 4.2.1, Eq. "B" and "alpha").  W fp32 [d_in x d_out], leading dimension
 * ldw >= d_out.  bitsT_out u32 [d_out x stride_words]: row j holds B_j = sign(W_:,j) packed along
 * d_in; alpha_out fp32 [d_out] = ||W_:,j||_1 / d_in. */
bigcn_status bigcn_pack_weights(bigcn_ctx* ctx, const float* W, int32_t d_in, int32_t d_out, int64_t ldw,
                                uint32_t* bitsT_out, int64_t stride_words, float* alpha_out);

/* One binarized layer's parameters: packed weights from bigcn_pack_weights() with
 * stride bigcn_packed_stride_words(d_in), and the optional batch-norm constants of the layer's
 * INPUT (fp32 [d_in], both or neither; Sec. 4.4).  1 <= d_in <= BIGCN_MAX_D_IN,
 * 1 <= d_out <= BIGCN_MAX_D_OUT. */
typedef struct {
    int32_t d_in;
    int32_t d_out;
    const uint32_t* w_bitsT;
    const float* alpha;
    const float* in_shift;
    const float* in_scale;
} bigcn_layer;

/* One layer (Sec. 4.2.3): dot_ij = F_i (*) B_j = d_in - 2 popc(F_i XOR B_j) (Eq. "bi-op"),
 * zeta_ij = beta_i alpha_j dot_ij (Eq. "cdot-op"), H' = A_tilde zeta.  No bias, no activation.
 *   in_bits  u32 [n x bigcn_packed_stride_words(d_in)], in_beta fp32 [n]: the packed input.
 *   h_out    fp32 [n x ldh] or null: H'.
 *   next     null, or the following layer: then next_bits [n x bigcn_packed_stride_words(d_out)] and
 *            next_beta [n] receive the binarization of H' under next->in_shift/in_scale
 *            (next->d_in must equal layer->d_out).  h_out and next may both be given.
 *   dbg_dot  int32 [n x d_out] or null, dbg_zeta fp32 [n x d_out] or null: taps on the contraction
 *            for testing (dbg_zeta always in the fp32 form of Eq. "cdot-op").
 * Needs workspace (bigcn_workspace_bytes with n_layers = 1). */
bigcn_status bigcn_layer_forward(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layer,
                                 const uint32_t* in_bits, const float* in_beta,
                                 float* h_out, int64_t ldh,
                                 const bigcn_layer* next, uint32_t* next_bits, float* next_beta,
                                 int32_t* dbg_dot, float* dbg_zeta);

/* Per-step device times of one bigcn_forward() call, in milliseconds (CUDA events). */
typedef struct {
    int32_t n_layers;
    int32_t launches;
    float ms_total;
    float ms_pack;                       /* binarize + pack of X */
    float ms_gemm[BIGCN_MAX_LAYERS];     /* binary contraction + rescale */
    float ms_spmm[BIGCN_MAX_LAYERS];     /* aggregation (+ re-binarization) */
} bigcn_stats;

/* L stacked layers from fp32 features to logits (H^(0) = X, Sec. 3.2; every layer binarized, the
 * last one's H' returned as logits [n x ldo]).  `layers` is a HOST array of n_layers structs whose
 * pointers are device pointers.  With stats != null the call records events around every step and
 * synchronises before returning; otherwise it is asynchronous. */
bigcn_status bigcn_forward(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layers /*host*/,
                           int32_t n_layers, const float* X, int64_t ldx,
                           float* logits_out, int64_t ldo, bigcn_stats* stats /*host, nullable*/);

/* As bigcn_forward() from features that are already binarized ("loaded data is binary", Sec. 5.2):
 * x_bits [n x bigcn_packed_stride_words(dims[0])], x_beta [n]. */
bigcn_status bigcn_forward_packed(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layers /*host*/,
                                  int32_t n_layers, const uint32_t* x_bits, const float* x_beta,
                                  float* logits_out, int64_t ldo, bigcn_stats* stats /*host, nullable*/);

/* As bigcn_forward() with HOST buffers for the per-call data: X_host fp32 [n x ldx] (ldx = d_0
 * required) is copied to the device, the forward runs, logits_host fp32 [n x ldo] (ldo = classes)
 * is copied back, and the call returns after the stream has drained.  Graph and layer arrays
 * stay device-resident.  Page-locked host memory makes the copies asynchronous and faster but is
 * not required.  Needs a workspace sized with host_io = 1. */
bigcn_status bigcn_forward_host(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layers /*host*/,
                                int32_t n_layers, const float* X_host, int64_t ldx,
                                float* logits_host, int64_t ldo);

/* Binning estimate of the entropy of a layer's activations (Sec. 6.2, "Entropy Estimation of Hidden
 * Layers"): for every neuron (column j of H, fp32 [n x d], ld >= d) over the n samples (rows), the
 * empirical distribution over n_bins intervals and H_hat(h_j) = -sum_m p_jm log2 p_jm; total =
 * H_ind(h) = sum_j H_hat(h_j), the lower bound the Entropy Cover Hypothesis puts on the width of a
 * binary hidden layer.  The paper fixes neither the intervals nor the logarithm; here: n_bins
 * intervals of equal width over the column's own range [min_j, max_j]; the interval of a value x is
 * decided in fp32 as m = (int)((x - min_j) * ((float)n_bins / (max_j - min_j))), clamped to
 * n_bins - 1 (the maximum falls into the last interval); a constant column puts every sample into
 * interval 0; entropies are in bits.  Values must be finite.
 * Outputs (device): col_min, col_max [d] fp32; counts [d x n_bins] uint32 (overwritten; n < 2^31);
 * entropy [d] and total [1] in double.  1 <= n_bins <= 8192 (BIGCN_ERR_UNSUPPORTED above).  With
 * n = 0 the counts and entropies are zero and col_min / col_max are left untouched.  Needs 8 * d
 * bytes of workspace.  Four launches, two passes over H. */
bigcn_status bigcn_entropy_bins(bigcn_ctx* ctx, const float* H, int64_t n, int32_t d, int64_t ld,
                                int32_t n_bins, float* col_min, float* col_max, uint32_t* counts,
                                double* entropy, double* total);

/* Back-propagation through one binarized layer (Algorithm 1, Sec. 4.3).  The forward pass of the
 * layer was H' = A_tilde (H~ W~) with H~_ik = beta_i F_ik (the packed input in_bits / in_beta of
 * bigcn_layer_forward) and W~_kj = alpha_j sign(W_kj).  Given g_out = dL/dH' (fp32 [n x d_out],
 * ldg >= d_out) the call computes, in the algorithm's order,
 *   G_zeta = A_tilde^T g_out,  G_W~ = H~^T G_zeta,  G_H~ = G_zeta W~^T          (step 1)
 *   g_in   = G_H~ where |G_H~| < 1, else 0                                       (step 2, Eq. bp-H)
 *   g_w_ij = (1/d_in) B_ij sum_k G_W~_kj B_kj + alpha_j G_W~_ij [|W_ij| < 1]     (step 3, Eq. bp-W;
 *            the bracket is the straight-through estimate of the sign's derivative)
 * and leaves step 4, the parameter update, to the caller's optimiser.  W is the latent fp32 weight
 * matrix [d_in x d_out] (ldw >= d_out) from which layer->w_bitsT and layer->alpha were packed.
 * g_in fp32 [n x d_in] (ldgi >= d_in) is nullable (the first layer needs no input gradient);
 * g_w fp32 [d_in x d_out] (ldgw >= d_out).  g_in is the gradient at the input of the binarization,
 * i.e. after the layer's batch normalisation if it has one (the algorithm does not cover that step).
 * A_tilde must be symmetric, as bigcn_normalize_adjacency() produces it: A_tilde^T is applied as
 * A_tilde.  d_out <= 512.  Needs bigcn_backward_workspace_bytes(n, d_in, d_out) of workspace.
 * fp32 throughout, sums over the nodes split into slabs that are added in a fixed order. */
size_t bigcn_backward_workspace_bytes(int64_t n, int32_t d_in, int32_t d_out);
bigcn_status bigcn_layer_backward(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layer,
                                  const float* W, int64_t ldw, const uint32_t* in_bits, const float* in_beta,
                                  const float* g_out, int64_t ldg, float* g_in, int64_t ldgi,
                                  float* g_w, int64_t ldgw);

/* Back-to-back forwards from host buffers, overlapped.  bigcn_forward_host() finishes one step (copy
 * in, forward, copy out) before the next begins, so the link to the host and the GPU take turns.
 * A pipeline keeps `slots` steps in flight on three streams: while step k computes on the context's
 * stream, the input of step k+1 is copied in and the logits of step k-1 are copied out.  The paper
 * has no counterpart of these calls (its costs are operation and byte counts, Sec. 5, not transfers); each
 * step computes exactly what bigcn_forward() computes.
 *   bigcn_pipeline_open   copies the graph and layer descriptions (their device arrays must outlive
 *                         the pipeline) and creates streams and events; allocates no device memory.
 *                         1 <= slots <= BIGCN_MAX_PIPELINE_SLOTS; 3 overlaps all three stages.
 *   bigcn_pipeline_submit enqueues one step and returns without waiting: X_host fp32 [n x d_0] dense,
 *                         logits_host fp32 [n x classes] dense, both HOST memory that must stay valid
 *                         (and, for the copies to overlap, page-locked) until the matching wait.
 *                         BIGCN_ERR_BUSY if `slots` steps are outstanding; BIGCN_ERR_WORKSPACE unless
 *                         the context's workspace was sized with host_io = slots.  The workspace must
 *                         not be replaced, and the context not used for other calls, while steps are
 *                         outstanding.
 *   bigcn_pipeline_submit_packed  the same step from an input that is already binary (Sec. 5.2, Eq. "DC": the
 *                         loaded data is 1 bit per element and one scalar per node, about 31 times less than
 *                         fp32): bits_host u32 [n x bigcn_packed_stride_words(d_0)] and beta_host fp32 [n] in
 *                         HOST memory, as bigcn_pack_features() produces them under the first layer's
 *                         batch-norm constants.  The step computes what bigcn_forward_packed() computes.  Steps
 *                         of both kinds may be mixed in one pipeline.
 *   bigcn_pipeline_wait   blocks until the OLDEST outstanding step has delivered its logits (steps
 *                         complete in submission order); BIGCN_OK at once if none is outstanding.
 *   bigcn_pipeline_close  waits for everything outstanding and frees the streams and events. */
#define BIGCN_MAX_PIPELINE_SLOTS 8
typedef struct bigcn_pipeline bigcn_pipeline;
bigcn_status bigcn_pipeline_open(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layers /*host*/,
                                 int32_t n_layers, int32_t slots, bigcn_pipeline** out);
bigcn_status bigcn_pipeline_submit(bigcn_pipeline* pipe, const float* X_host, float* logits_host);
bigcn_status bigcn_pipeline_submit_packed(bigcn_pipeline* pipe, const uint32_t* bits_host, const float* beta_host,
                                          float* logits_host);
bigcn_status bigcn_pipeline_wait(bigcn_pipeline* pipe);
bigcn_status bigcn_pipeline_close(bigcn_pipeline* pipe);

/* Batch statistics for the batch normalisation of a layer's input (Sec. 4.4: zero mean, unit
 * variance per feature over the nodes): shift_out[j] = mean_j, scale_out[j] = 1/sqrt(var_j + eps),
 * biased variance.  H fp32 [n x d], ld >= d.  Needs 16 * d * 1024 bytes of workspace. */
bigcn_status bigcn_col_stats(bigcn_ctx* ctx, const float* H, int64_t n, int32_t d, int64_t ld,
                             float eps, float* shift_out, float* scale_out);

/* Bi-GraphSAGE with the mean aggregator (Sec. 4.4.2, Eq. "bisage-conv"):
 *   h_i' = W_theta (*) h_i + (1/|N_i|) sum_{j in N_i} W_n (*) h_j,   no activation,
 * both products by XNOR and bit count on the same binarized input.
 *
 * bigcn_mean_adjacency(): set-up, once per graph.  Same input and checks as
 * bigcn_normalize_adjacency(); the output CSR holds, for row i, its distinct neighbours (no
 * self-loop) with val = 1/|N_i| (computed in double, rounded to fp32); inv_deg[n] receives 1/|N_i|
 * (0 for a node without neighbours, whose row is empty).  Outputs need nnz_in entries.  SYNCHRONOUS.
 *
 * bigcn_sage_layer_forward(): one layer.  mean_graph from bigcn_mean_adjacency(); self_layer and
 * nbr_layer hold the packed W_theta and W_n (same d_in and d_out; the batch-norm fields of these two
 * structs are not used: the input arrives already binarized); in_bits / in_beta, h_out, next,
 * next_bits, next_beta as in bigcn_layer_forward().  Needs twice the workspace of
 * bigcn_layer_forward() for the same sizes (bigcn_workspace_bytes with n_layers = 1, times two). */
bigcn_status bigcn_mean_adjacency(bigcn_ctx* ctx, int64_t n, int64_t nnz_in,
                                  const int64_t* rowptr_A, const int32_t* colidx_A,
                                  int64_t* rowptr, int32_t* colidx, float* val, float* inv_deg,
                                  int64_t* nnz_out /*host*/);
bigcn_status bigcn_sage_layer_forward(bigcn_ctx* ctx, const bigcn_graph* mean_graph,
                                      const bigcn_layer* self_layer, const bigcn_layer* nbr_layer,
                                      const uint32_t* in_bits, const float* in_beta,
                                      float* h_out, int64_t ldh,
                                      const bigcn_layer* next, uint32_t* next_bits, float* next_beta);

/* Measurement aid: the rate at which this GPU retires the step the contraction of Eq. "bi-op" is made
 * of (XOR, bit count and add on one 32-bit word per lane), from a register-only loop; the result, in
 * word steps per second, is the denominator of the bit-GEMM's roofline fraction (x 64 = binary ops/s).
 * Needs 1.2 MB of workspace.  SYNCHRONOUS. */
bigcn_status bigcn_measure_popc_peak(bigcn_ctx* ctx, double* word_steps_per_s /*host*/);

/* Measurement aid: the time the memory system alone needs for the access pattern of the aggregation
 * H' = A_tilde zeta (last equation of Sec. 4.2.3) on graph g -- for every stored entry, the row colidx[e] of a
 * row-major matrix of `row_bytes` bytes per row (a power of two, 16..512) is read, 16 bytes per lane, and
 * discarded; no weights, no sums, no output.  *ms (host) receives the best of three runs in milliseconds:
 * the ceiling an aggregation kernel over rows of that size can be held against.  The rows read are the
 * first n * row_bytes bytes of the workspace (contents irrelevant); needs that much workspace + 256 bytes.
 * SYNCHRONOUS. */
bigcn_status bigcn_measure_gather_peak(bigcn_ctx* ctx, const bigcn_graph* g, int32_t row_bytes, double* ms /*host*/);

/* One layer without any allocation (the paper has no counterpart of this call; it is a packaging of
 * bigcn_layer_forward() for callers that must not allocate device memory: a process whose own pool
 * took the whole GPU at start-up, so that cudaMalloc would fail, or a latency-critical loop that
 * cannot afford the device-wide synchronisation an allocation implies).
 * It needs no context and no workspace: the scratch between the bit-GEMM and the aggregation
 * lives in a fixed array of BIGCN_NOALLOC_SCRATCH_BYTES inside the library's device image (held by
 * every GPU that loads the library until the process exits).  It never calls cudaMalloc, cudaFree
 * or any allocating routine.
 *   cuda_stream  the cudaStream_t to enqueue on (0 = default stream); the device that owns it
 *                must be the calling thread's current device.
 *   other arguments and results: as bigcn_layer_forward(), without the debug taps.  The integer
 *   dots are the same; between the contraction and the aggregation they are always kept as 16-bit
 *   values here, whereas bigcn_layer_forward() picks narrower rows for some widths and so adds the
 *   same fp32 terms in another order: H' and next_beta agree with that call within fp32 rounding
 *   (inside the library's tolerance 1e-4 + 1e-5 |x|), and a re-binarized bit can differ where the
 *   value under the sign sits at the threshold within that rounding.
 * Limits and rules:
 *   - n * round_up(d_out, 8) * 2 bytes must not exceed BIGCN_NOALLOC_SCRATCH_BYTES - 256; a larger
 *     problem is refused with BIGCN_ERR_WORKSPACE before anything is launched.
 *   - A bounded wait inside the tensor-core contraction that runs out makes that kernel stop early
 *     and raise a device flag; with no context here, the flag is only reported by
 *     bigcn_sync_check() on some context of the same device.
 *   - The first call on a device looks up the array's device address (once per device); make that
 *     first call before starting any stream capture on that device.
 *   - All calls in a process share the one array, and it keeps what the previous call left; the call
 *     itself rewrites everything it later reads, so a stale content is harmless, but two calls whose
 *     GPU work overlaps (different streams, or different threads) race on it: keep them ordered.
 * Returns a status only (there is no context to hold a message). */
#define BIGCN_NOALLOC_SCRATCH_BYTES (8u * 1024u * 1024u)
bigcn_status bigcn_layer_forward_noalloc(void* cuda_stream, const bigcn_graph* graph, const bigcn_layer* layer,
                                         const uint32_t* in_bits, const float* in_beta,
                                         float* h_out, int64_t ldh,
                                         const bigcn_layer* next, uint32_t* next_bits, float* next_beta);

#ifdef __cplusplus
}
#endif
#endif /* BIGCN_H */
