// Binning entropy estimate of a layer's activations (Bi-GCN Sec. 6.2): per neuron (column) the range
// over the N samples (rows), an M-interval histogram over that range, H_hat = -sum p log2 p, and the
// independent sum over the neurons.  Two streaming passes over the N x d matrix (range, histogram),
// both bound by HBM reads; the histogram of a strip of columns lives in shared memory.
#include <algorithm>

#include "bigcn_internal.cuh"

namespace bigcn {

namespace {

constexpr int kEntThreads = 256;
constexpr int kEntWarps = kEntThreads / kWarp;

// Order-preserving map from float to unsigned (so that integer atomicMin / atomicMax order floats).
__device__ __forceinline__ uint32_t float_key(float x)
{
    const uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Pass 1.  Block (x, y) scans its share of the rows for columns 32 y .. 32 y + 31: lane = column, the
// warps of a block take rows in turn (each warp load is 128 contiguous bytes), four rows in flight per
// warp.  One atomicMin and one atomicMax per column and block on the order-preserving keys.
__global__ void __launch_bounds__(kEntThreads)
range_kernel(const float* __restrict__ H, int64_t n, int d, int64_t ld, int64_t rows_per_block,
             uint32_t* __restrict__ key_min, uint32_t* __restrict__ key_max)
{
    __shared__ float s_lo[kEntWarps][kWarp], s_hi[kEntWarps][kWarp];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int col = blockIdx.y * 32 + lane;
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_block;
    const int64_t r1 = min(n, r0 + rows_per_block);
    float lo = INFINITY, hi = -INFINITY;
    if (col < d) {
        int64_t r = r0 + warp;
        for (; r + 3 * kEntWarps < r1; r += 4 * kEntWarps) {
            float x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) x[u] = __ldg(H + (r + u * kEntWarps) * ld + col);
#pragma unroll
            for (int u = 0; u < 4; ++u) { lo = fminf(lo, x[u]); hi = fmaxf(hi, x[u]); }
        }
        for (; r < r1; r += kEntWarps) {
            const float x = __ldg(H + r * ld + col);
            lo = fminf(lo, x);
            hi = fmaxf(hi, x);
        }
    }
    s_lo[warp][lane] = lo;
    s_hi[warp][lane] = hi;
    __syncthreads();
    if (warp == 0 && col < d) {
#pragma unroll
        for (int w = 1; w < kEntWarps; ++w) { lo = fminf(lo, s_lo[w][lane]); hi = fmaxf(hi, s_hi[w][lane]); }
        if (lo <= hi) {                                   // the block saw at least one row
            atomicMin(key_min + col, float_key(lo));
            atomicMax(key_max + col, float_key(hi));
        }
    }
}

// Pass 2.  Block (x, y) histograms its share of the rows for the strip of CW columns CW y ..: a warp
// instruction covers 32 / CW rows x CW columns (CW * 4 contiguous bytes per row); the strip's CW x M
// counters sit in shared memory and are added to the global ones once per block.  The interval of a
// value is decided in fp32 exactly as documented for the entry point: (x - min) * (M / (max - min)),
// truncated, clamped to M - 1; a constant column has scale 0 and lands in interval 0.
template <int CW>
__global__ void __launch_bounds__(kEntThreads)
histogram_kernel(const float* __restrict__ H, int64_t n, int d, int64_t ld, int n_bins, int64_t rows_per_block,
                 const uint32_t* __restrict__ key_min, const uint32_t* __restrict__ key_max,
                 float* __restrict__ col_min, float* __restrict__ col_max, uint32_t* __restrict__ counts)
{
    extern __shared__ uint32_t hist[];                    // [CW][n_bins]
    constexpr int RPW = kWarp / CW;                       // rows per warp instruction
    constexpr int RPB = RPW * kEntWarps;                  // rows per block step
    for (int i = threadIdx.x; i < CW * n_bins; i += kEntThreads) hist[i] = 0u;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int cl = lane % CW;                             // column inside the strip
    const int col = blockIdx.y * CW + cl;
    const bool col_in = col < d;
    float lo = 0.f, scale = 0.f;
    if (col_in) {
        lo = key_float(key_min[col]);
        const float hi = key_float(key_max[col]);
        scale = hi > lo ? __fdiv_rn((float)n_bins, __fsub_rn(hi, lo)) : 0.f;
        if (blockIdx.x == 0 && threadIdx.x < CW) { col_min[col] = lo; col_max[col] = hi; }
    }
    __syncthreads();
    const int64_t r0 = (int64_t)blockIdx.x * rows_per_block;
    const int64_t r1 = min(n, r0 + rows_per_block);
    uint32_t* my = hist + cl * n_bins;
    const int last = n_bins - 1;
    if (col_in) {
        int64_t r = r0 + warp * RPW + lane / CW;
        for (; r + 3 * RPB < r1; r += 4 * RPB) {
            float x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) x[u] = __ldg(H + (r + u * RPB) * ld + col);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int m = min((int)__fmul_rn(__fsub_rn(x[u], lo), scale), last);
                atomicAdd(my + m, 1u);
            }
        }
        for (; r < r1; r += RPB) {
            const float x = __ldg(H + r * ld + col);
            const int m = min((int)__fmul_rn(__fsub_rn(x, lo), scale), last);
            atomicAdd(my + m, 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < CW * n_bins; i += kEntThreads) {
        const uint32_t v = hist[i];
        const int c = blockIdx.y * CW + i / n_bins;
        if (v && c < d) atomicAdd(counts + (int64_t)c * n_bins + (i % n_bins), v);
    }
}

// H_hat of one column per warp, in double: lanes take intervals lane, lane + 32, ... and the 32
// partial sums are combined in a fixed order.
__global__ void __launch_bounds__(kEntThreads)
entropy_kernel(const uint32_t* __restrict__ counts, int d, int n_bins, int64_t n, double* __restrict__ entropy)
{
    const int lane = threadIdx.x & 31;
    const int col = blockIdx.x * kEntWarps + (threadIdx.x >> 5);
    if (col >= d) return;
    const uint32_t* c = counts + (int64_t)col * n_bins;
    const double inv_n = 1.0 / (double)n;
    double h = 0.0;
    for (int m = lane; m < n_bins; m += 32) {
        const uint32_t v = c[m];
        if (v) {
            const double p = (double)v * inv_n;
            h -= p * log2(p);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) h += __shfl_xor_sync(0xffffffffu, h, o);
    if (lane == 0) entropy[col] = h;
}

// H_ind = sum over the columns, one warp, fixed order.
__global__ void __launch_bounds__(kWarp)
entropy_total_kernel(const double* __restrict__ entropy, int d, double* __restrict__ total)
{
    double s = 0.0;
    for (int j = threadIdx.x; j < d; j += 32) s += entropy[j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (threadIdx.x == 0) *total = s;
}

template <int CW>
cudaError_t launch_histogram(cudaStream_t s, const float* H, int64_t n, int d, int64_t ld, int n_bins,
                             const uint32_t* key_min, const uint32_t* key_max, float* col_min, float* col_max,
                             uint32_t* counts)
{
    const size_t smem = (size_t)CW * n_bins * sizeof(uint32_t);
    cudaError_t e = cudaFuncSetAttribute(histogram_kernel<CW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const unsigned gy = (unsigned)ceil_div(d, CW);
    const int per_sm = (int)std::max<size_t>(1, std::min<size_t>(8, (200 * 1024) / std::max<size_t>(smem, 1)));
    // about one resident wave of blocks over both grid dimensions; every block takes a contiguous range of rows
    const int64_t gx = std::max<int64_t>(1, std::min<int64_t>(ceil_div(n, 1024), ceil_div((int64_t)sm_count() * per_sm, gy)));
    const int64_t rows_per_block = ceil_div(n, gx);
    histogram_kernel<CW><<<dim3((unsigned)gx, gy), kEntThreads, smem, s>>>(H, n, d, ld, n_bins, rows_per_block, key_min,
                                                                         key_max, col_min, col_max, counts);
    return cudaGetLastError();
}

}  // namespace

size_t entropy_scratch_bytes(int d) { return 2 * (size_t)d * sizeof(uint32_t); }

int entropy_max_bins() { return 8192; }

cudaError_t launch_entropy_bins(cudaStream_t s, const float* H, int64_t n, int d, int64_t ld, int n_bins,
                                float* col_min, float* col_max, uint32_t* counts, double* entropy, double* total,
                                void* scratch, int* launches)
{
    uint32_t* key_min = static_cast<uint32_t*>(scratch);
    uint32_t* key_max = key_min + d;
    cudaError_t e = cudaMemsetAsync(key_min, 0xff, (size_t)d * 4, s);          // larger than every key
    if (e == cudaSuccess) e = cudaMemsetAsync(key_max, 0, (size_t)d * 4, s);   // smaller than every key
    if (e == cudaSuccess) e = cudaMemsetAsync(counts, 0, (size_t)d * n_bins * 4, s);
    if (e != cudaSuccess) return e;
    {
        const unsigned gy = (unsigned)ceil_div(d, 32);
        const int64_t gx = std::max<int64_t>(1, std::min<int64_t>(ceil_div(n, 256), ceil_div((int64_t)sm_count() * 8, gy)));
        range_kernel<<<dim3((unsigned)gx, gy), kEntThreads, 0, s>>>(H, n, d, ld, ceil_div(n, gx), key_min, key_max);
        ++*launches;
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    if (n_bins <= 1024) e = launch_histogram<16>(s, H, n, d, ld, n_bins, key_min, key_max, col_min, col_max, counts);
    else if (n_bins <= 4096) e = launch_histogram<8>(s, H, n, d, ld, n_bins, key_min, key_max, col_min, col_max, counts);
    else e = launch_histogram<4>(s, H, n, d, ld, n_bins, key_min, key_max, col_min, col_max, counts);
    ++*launches;
    if (e != cudaSuccess) return e;
    entropy_kernel<<<(unsigned)ceil_div(d, kEntWarps), kEntThreads, 0, s>>>(counts, d, n_bins, n, entropy);
    ++*launches;
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    entropy_total_kernel<<<1, kWarp, 0, s>>>(entropy, d, total);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace bigcn
