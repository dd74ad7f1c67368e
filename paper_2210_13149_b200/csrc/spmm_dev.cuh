// Device-side argument block of the aggregation kernels (spmm.cu, spmm_tc.cu).
#pragma once
#include <stdint.h>

#include <cuda_runtime.h>

namespace bigcn {

struct SpmmDev {
    int64_t n;
    const int64_t* rowptr;
    const int32_t* colidx;
    const float* val;
    const uint4* zeta;       // rows of nv 16-byte vectors
    int nv;                  // vectors per zeta row
    int nv_fin;              // groups of Elt<T>::kPerVec columns the row epilogue covers (nv, unless the epilogue's element type differs)
    int d_out;
    const float* node_w;     // nullable
    const float* col_w;      // nullable
    const float* col_b0;     // half-dot bytes only: per-column first weight sign (0 where none)
    int half_dots;           // zeta holds s = (dot' - 1) / 2; node_w carries the first feature sign
    int byte_path;           // 129..256 byte columns: 0 / 1 the FMA stream, 2 integer tensor-core products
    int row_tail;            // rows of 64 bytes whose last four bytes hold the source's node factor as a float
    const float* add;        // nullable: fp32 [n x ld_add] added to the aggregated row (after col_w)
    int64_t ld_add;
    float* h_out;
    int64_t ldh;
    int h_vec;               // 1: rows of h_out can be stored as float4
    uint32_t* next_bits;
    int64_t next_stride;
    float* next_beta;
    const float* next_shift;
    const float* next_scale;
    int64_t long_row;
    int covered_words;       // packed words of the next layer that the zeta columns cover
    float inv_d_out;
    int* run_counter;        // zeroed before the launch: next run of rows to hand out
};

// The aggregation of 129..256-byte rows as tcgen05 integer products (spmm_tc.cu).
bool spmm_tc_covers(const SpmmDev& p);
cudaError_t launch_spmm_tc(cudaStream_t s, const SpmmDev& p);
int spmm_tc_timeouts();

}  // namespace bigcn
