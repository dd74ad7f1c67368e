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

}  // namespace

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
