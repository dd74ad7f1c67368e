// Measures the throughput of the integer pipe on the XOR + bit-count + add step that the
// XNOR/bit-count contraction (Bi-GCN Sec. 4.2.3, Eq. "bi-op") is made of: the denominator of the
// bit-GEMM's roofline fraction.  Register-only loop, no memory traffic inside the timed region.
#include "bigcn_internal.cuh"

namespace bigcn {

namespace {

constexpr int kIndep = 8;          // independent accumulators per lane

__global__ void __launch_bounds__(256)
popc_peak_kernel(uint32_t* out, int iters, uint32_t seed)
{
    uint32_t a[kIndep], acc[kIndep];
#pragma unroll
    for (int i = 0; i < kIndep; ++i) {
        a[i] = seed * (threadIdx.x + 1) * (i + 3) + blockIdx.x;
        acc[i] = i;
    }
    uint32_t b = seed ^ threadIdx.x;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < kIndep; ++i) acc[i] += __popc(a[i] ^ b);
        b = b * 1664525u + 1013904223u;
#pragma unroll
        for (int i = 0; i < kIndep; ++i) a[i] ^= b;       // keeps the operands changing
    }
    uint32_t s = 0;
#pragma unroll
    for (int i = 0; i < kIndep; ++i) s += acc[i];
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

// The aggregation's gather and nothing else: for every stored entry e of a CSR matrix, the row colidx[e] of a
// row-major byte matrix with `row_bytes` per row is read (16 bytes per lane, 16 lanes per row for 256-byte rows, as
// the aggregation kernels fetch it) and folded into a checksum.  No weights, no sums, no row ends: the time of this
// kernel is what the memory system alone needs for the access pattern of Bi-GCN's H' = A_tilde zeta (Sec. 4.2.3) on
// this graph -- the ceiling the aggregation kernels are measured against.
__global__ void __launch_bounds__(256)
gather_peak_kernel(const int32_t* __restrict__ colidx, int64_t nnz, const uint4* __restrict__ rows, int pieces, uint32_t* out)
{
    const int lane = threadIdx.x & 31;
    const int lpr = pieces;                                   // lanes per row: 16-byte pieces of a row (a power of two, <= 32)
    const int epi = 32 / lpr;                                 // entries per warp instruction
    const int sub = lane / lpr, piece = lane % lpr;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5), w0 = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    uint32_t acc = 0u;
    for (int64_t e0 = w0 * 32; e0 < nnz; e0 += warps * 32) {
        const int col = e0 + lane < nnz ? __ldg(colidx + e0 + lane) : 0;
        const int cnt = (int)min((int64_t)32, nnz - e0);
        uint4 v[8];
        for (int j0 = 0; j0 < 32; j0 += 8 * epi) {            // eight loads in flight per lane
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int j = j0 + u * epi + sub;
                const int c = __shfl_sync(0xffffffffu, col, j & 31);
                v[u] = make_uint4(0u, 0u, 0u, 0u);
                if (j < cnt) v[u] = __ldg(rows + (int64_t)c * pieces + piece);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
        }
    }
    if (acc == 0x9e3779b9u) out[0] = acc;                     // keeps the loads alive; practically never taken
}

}  // namespace

// Times the gather of `row_bytes`-byte rows (16, 32, .. 512: a power of two) along the column indices of a matrix
// with nnz stored entries; `rows` is any buffer of n * row_bytes bytes (its contents do not matter).  Best of three
// runs, in milliseconds.  Synchronises the stream.
cudaError_t measure_gather_peak(cudaStream_t s, const int32_t* colidx, int64_t nnz, const void* rows, int row_bytes,
                                void* scratch, double* ms_out, int* launches)
{
    const int pieces = row_bytes / 16;
    const int blocks = sm_count() * 8;
    cudaEvent_t e0, e1;
    cudaError_t e = cudaEventCreate(&e0);
    if (e != cudaSuccess) return e;
    e = cudaEventCreate(&e1);
    if (e != cudaSuccess) { cudaEventDestroy(e0); return e; }
    float best = 1e30f;
    for (int rep = 0; rep < 4 && e == cudaSuccess; ++rep) {   // the first run warms the caches as a forward's earlier layers would
        cudaEventRecord(e0, s);
        gather_peak_kernel<<<blocks, 256, 0, s>>>(colidx, nnz, static_cast<const uint4*>(rows), pieces, static_cast<uint32_t*>(scratch));
        ++*launches;
        cudaEventRecord(e1, s);
        e = cudaEventSynchronize(e1);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
        if (e == cudaSuccess && rep > 0 && ms < best) best = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess) return e;
    *ms_out = (double)best;
    return cudaGetLastError();
}

size_t popc_peak_scratch_bytes() { return (size_t)sm_count() * 8 * 256 * sizeof(uint32_t); }

// Runs the loop three times and returns the best rate in 32-bit word steps (one XOR, one bit count,
// one add on 32 bits) per second.  Synchronises the stream.
cudaError_t measure_popc_peak(cudaStream_t s, void* scratch, double* word_steps_per_s, int* launches)
{
    const int blocks = sm_count() * 8, iters = 20000;
    cudaEvent_t e0, e1;
    cudaError_t e = cudaEventCreate(&e0);
    if (e != cudaSuccess) return e;
    e = cudaEventCreate(&e1);
    if (e != cudaSuccess) { cudaEventDestroy(e0); return e; }
    float best = 1e30f;
    for (int rep = 0; rep < 3 && e == cudaSuccess; ++rep) {
        cudaEventRecord(e0, s);
        popc_peak_kernel<<<blocks, 256, 0, s>>>(static_cast<uint32_t*>(scratch), iters, 12345u);
        ++*launches;
        cudaEventRecord(e1, s);
        e = cudaEventSynchronize(e1);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
        if (e == cudaSuccess && ms < best) best = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (e != cudaSuccess) return e;
    *word_steps_per_s = (double)blocks * 256.0 * iters * kIndep / (best * 1e-3);
    return cudaGetLastError();
}

}  // namespace bigcn
