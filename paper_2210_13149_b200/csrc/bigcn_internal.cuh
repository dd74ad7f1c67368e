// Internal declarations shared by the translation units of libbigcn (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "bigcn.h"

namespace bigcn {

constexpr int kWarp = 32;

// Storage of the contraction result between the bit-GEMM and the aggregation.
// kZetaI8H (128 <= d_in <= 256): signed bytes s = (dot' - 1) / 2 where dot' is the dot without the first position when
// d_in is even (so that dot' is odd and s fits a byte); the aggregation adds the missing terms back (see spmm.cu).
enum ZetaFormat : int { kZetaF32 = 1, kZetaI16 = 2, kZetaI8 = 3, kZetaF16 = 4, kZetaI8H = 5 };

inline __host__ __device__ int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline __host__ __device__ int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }

// Elements per row of the zeta buffer: d_out rounded up so that a row is a whole number of 16-byte vectors.
inline int64_t zeta_ld(int d_out, int fmt)
{
    return round_up(d_out, 16 / (fmt == kZetaF32 ? 4 : ((fmt == kZetaI8 || fmt == kZetaI8H) ? 1 : 2)));
}
inline int zeta_elt_bytes(int fmt) { return fmt == kZetaF32 ? 4 : ((fmt == kZetaI8 || fmt == kZetaI8H) ? 1 : 2); }

// Number of multiprocessors of the calling thread's current device (queried once per device; 1 if the query
// fails, so that a grid derived from it stays valid).  Persistent grids are sized from it.
int sm_count();

// ---- launchers (each returns the launch status; all asynchronous on `s`) ------------------------

cudaError_t launch_pack_rows(cudaStream_t s, const float* H, int64_t n, int d, int64_t ld,
                             const float* shift, const float* scale,
                             uint32_t* bits, int64_t stride, float* beta, int* launches);

cudaError_t launch_pack_weights(cudaStream_t s, const float* W, int d_in, int d_out, int64_t ldw,
                                uint32_t* bitsT, int64_t stride, float* alpha, int* launches);

cudaError_t launch_bitgemm(cudaStream_t s, const uint32_t* A, int64_t stride_a,
                           const uint32_t* BT, int64_t stride_b, int64_t n, int d_in, int d_out,
                           const float* beta, const float* alpha, int fmt, void* zeta, int64_t ldz,
                           int32_t* dbg_dot, float* dbg_zeta, int* launches, int path = 0 /* 0 auto, 1 bit-count pipe, 2 tensor cores wherever covered */,
                           float* nws = nullptr /* kZetaI8H: [n] beta_i times the first sign */, float* col_b0 = nullptr /* kZetaI8H: [d_out] */,
                           int row_tail = 0 /* byte formats on the tensor-core path, ldz = 64: the row's node factor in its last four bytes */);
// Whether launch_bitgemm will take the tensor-core path for these arguments.
bool bitgemm_takes_tc(int fmt, int path, int64_t n, int d_in, int d_out, int64_t stride_a, int64_t stride_b);

struct SpmmArgs {
    int64_t n;
    int64_t nnz = 0;         // stored entries (0 = unknown): the mean row length picks the stream for narrow rows
    const int64_t* rowptr;
    const int32_t* colidx;
    const float* val;
    int fmt;                 // ZetaFormat of `zeta`
    const void* zeta;        // [n x ldz] of float / int16 / int8
    int64_t ldz;
    int d_out;
    const float* node_w;     // integer formats: per-source-node factor (beta), multiplied into the edge weight
    const float* col_w;      // integer formats: per-column factor (alpha), applied once per output
    const float* col_b0 = nullptr;   // half-dot bytes (kZetaI8H): per-column first weight sign (0 when d_in is odd)
    bool half_dots = false;          // zeta holds s = (dot' - 1) / 2 and node_w carries the first feature sign
    int byte_path = 0;               // rows of 129..256 bytes: 0 auto (the fp32 FMA stream), 1 the fp32 FMA stream, 2 integer tensor-core products
    bool row_tail = false;           // byte rows of 64 bytes whose last four bytes hold the source's node factor (see bitgemm_tc.cu)
    const float* add = nullptr;   // optional fp32 [n x ld_add] added to every aggregated row (Bi-GraphSAGE self term)
    int64_t ld_add = 0;
    float* h_out;            // nullable
    int64_t ldh;
    uint32_t* next_bits;     // nullable: fused re-binarization of the output
    int64_t next_stride;
    float* next_beta;
    const float* next_shift; // nullable
    const float* next_scale;
    int64_t long_row;        // rows with more entries are split (0 = never)
    void* scratch;           // partial sums of split rows
    size_t scratch_bytes;
};
cudaError_t launch_spmm(cudaStream_t s, const SpmmArgs& a, int* launches);
size_t spmm_scratch_bytes(int64_t n, int64_t nnz, int d_out);

cudaError_t launch_normalize_adjacency(cudaStream_t s, int64_t n, int64_t nnz_in,
                                       const int64_t* rowptr_A, const int32_t* colidx_A,
                                       int64_t* rowptr, int32_t* colidx, float* val, float* dinv,
                                       void* scratch, int* d_flag, int* launches, bool mean = false);
size_t normalize_scratch_bytes(int64_t n);

// Canonical CSR pattern of A from a raw list of node pairs (edges.cu).
cudaError_t launch_adjacency_from_edges(cudaStream_t s, int64_t n, int64_t m, const int32_t* src, const int32_t* dst,
                                        int64_t* rowptr, int32_t* colidx, void* scratch, int* flag, int* launches);
size_t edges_scratch_bytes(int64_t m);

cudaError_t launch_col_stats(cudaStream_t s, const float* H, int64_t n, int d, int64_t ld, float eps,
                             float* shift, float* scale, void* scratch, int* launches);
size_t col_stats_scratch_bytes(int d);

cudaError_t measure_popc_peak(cudaStream_t s, void* scratch, double* word_steps_per_s, int* launches);
size_t popc_peak_scratch_bytes();
cudaError_t measure_gather_peak(cudaStream_t s, const int32_t* colidx, int64_t nnz, const void* rows, int row_bytes,
                                void* scratch, double* ms_out, int* launches);

// The same contraction as tcgen05 int8 products (bitgemm_tc.cu): shapes with d_in, d_out <= 256.
bool bitgemm_tc_covers(int d_in, int d_out, int64_t stride_a, int64_t stride_b);
cudaError_t launch_bitgemm_tc(cudaStream_t s, const uint32_t* A, int64_t stride_a, const uint32_t* BT, int64_t stride_b,
                              int64_t n, int d_in, int d_out, const float* beta, const float* alpha, int fmt, void* zeta,
                              int64_t ldz, int32_t* dbg_dot, float* dbg_zeta, float* nws = nullptr, float* col_b0 = nullptr, int row_tail = 0);
int bitgemm_tc_timeouts();

// Binning entropy estimate (entropy.cu): scratch = 2 * d uint32.
cudaError_t launch_entropy_bins(cudaStream_t s, const float* H, int64_t n, int d, int64_t ld, int n_bins,
                                float* col_min, float* col_max, uint32_t* counts, double* entropy, double* total,
                                void* scratch, int* launches);
size_t entropy_scratch_bytes(int d);
int entropy_max_bins();

// Back-propagation through one binarized layer (backward.cu).
size_t backward_scratch_bytes(int64_t n, int d_in, int d_out);
int backward_tc_timeouts();
cudaError_t launch_layer_backward(cudaStream_t s, int64_t n, const int64_t* rowptr, const int32_t* colidx,
                                  const float* val, int d_in, int d_out, const float* W, int64_t ldw,
                                  const float* alpha, const uint32_t* in_bits, int64_t stride_in,
                                  const float* in_beta, const float* g_out, int64_t ldg, float* g_in,
                                  int64_t ldgi, float* g_w, int64_t ldgw, int64_t long_row, void* scratch,
                                  int* launches);

}  // namespace bigcn
