// Set-up kernels: the normalised adjacency A_tilde = D_hat^-1/2 (A + I) D_hat^-1/2 in CSR
// (Bi-GCN Sec. 3.1 and Eq. 1) and the per-feature batch statistics of a layer input (Sec. 4.4).
#include <algorithm>

#include "bigcn_internal.cuh"

namespace bigcn {

namespace {

constexpr int kRowsPerBlock = 8;          // one warp per row
constexpr int kScanBlock = 1024;

// Bits of the device flag word written by the checks below.
constexpr int kFlagOrder = 1;             // columns not ascending / repeated
constexpr int kFlagRange = 2;             // column outside [0, n)
constexpr int kFlagSymmetry = 4;          // (i, j) stored without (j, i)
constexpr int kFlagRowptr = 8;            // rowptr not monotone or not matching nnz

// Pass 1: D_hat_ii = 1 + number of off-diagonal entries of row i; checks order and range.
template <bool kMean>
__global__ void __launch_bounds__(kRowsPerBlock* kWarp)
degree_kernel(int64_t n, int64_t nnz_in, const int64_t* __restrict__ rowptr_A,
              const int32_t* __restrict__ colidx_A, int64_t* __restrict__ rowptr,
              float* __restrict__ dinv, int* __restrict__ flag)
{
    const int lane = threadIdx.x & 31;
    const int64_t i = (int64_t)blockIdx.x * kRowsPerBlock + (threadIdx.x >> 5);
    if (i >= n) return;
    const int64_t a = rowptr_A[i], b = rowptr_A[i + 1];
    int bad = 0;
    if (a > b || a < 0 || b > nnz_in || (i == 0 && a != 0) || (i == n - 1 && b != nnz_in)) {
        bad |= kFlagRowptr;
    } else {
        int off_diag = 0;
        for (int64_t q = a + lane; q < b; q += 32) {
            const int32_t c = colidx_A[q];
            if (c < 0 || c >= n) bad |= kFlagRange;
            if (q > a && colidx_A[q - 1] >= c) bad |= kFlagOrder;
            off_diag += (c != (int32_t)i);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) off_diag += __shfl_xor_sync(0xffffffffu, off_diag, o);
        if (lane == 0) {
            if (kMean) {                                   // mean aggregator: |N_i| entries, factor 1/|N_i|
                rowptr[i + 1] = off_diag;
                dinv[i] = off_diag > 0 ? (float)(1.0 / (double)off_diag) : 0.f;
            } else {
                const int64_t deg_hat = (int64_t)off_diag + 1;
                rowptr[i + 1] = deg_hat;
                dinv[i] = (float)(1.0 / sqrt((double)deg_hat));
            }
        }
    }
    if (i == 0 && lane == 0) rowptr[0] = 0;
    if (bad) atomicOr(flag, bad);
}

// Inclusive scan of x[0..m) in three launches: block totals, scan of the totals, block scans.
__device__ __forceinline__ int64_t block_inclusive_scan(int64_t v, int64_t* warp_tot)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int64_t t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    if (warp == 0) {
        int64_t w = warp_tot[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int64_t t = __shfl_up_sync(0xffffffffu, w, o);
            if (lane >= o) w += t;
        }
        warp_tot[lane] = w;
    }
    __syncthreads();
    if (warp > 0) v += warp_tot[warp - 1];
    return v;
}

__global__ void __launch_bounds__(kScanBlock)
scan_totals_kernel(const int64_t* __restrict__ x, int64_t m, int64_t* __restrict__ totals)
{
    __shared__ int64_t warp_tot[32];
    const int64_t idx = (int64_t)blockIdx.x * kScanBlock + threadIdx.x;
    const int64_t v = block_inclusive_scan(idx < m ? x[idx] : 0, warp_tot);
    if (threadIdx.x == kScanBlock - 1) totals[blockIdx.x] = v;
}

__global__ void __launch_bounds__(kScanBlock)
scan_of_totals_kernel(int64_t* __restrict__ totals, int64_t nb)
{
    __shared__ int64_t warp_tot[32];
    __shared__ int64_t carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int64_t base = 0; base < nb; base += kScanBlock) {
        const int64_t idx = base + threadIdx.x;
        const int64_t v = block_inclusive_scan(idx < nb ? totals[idx] : 0, warp_tot);
        const int64_t c = carry;
        if (idx < nb) totals[idx] = v + c;
        __syncthreads();
        if (threadIdx.x == kScanBlock - 1) carry = v + c;
        __syncthreads();
    }
}

__global__ void __launch_bounds__(kScanBlock)
scan_apply_kernel(int64_t* __restrict__ x, int64_t m, const int64_t* __restrict__ totals)
{
    __shared__ int64_t warp_tot[32];
    const int64_t idx = (int64_t)blockIdx.x * kScanBlock + threadIdx.x;
    int64_t v = block_inclusive_scan(idx < m ? x[idx] : 0, warp_tot);
    if (blockIdx.x > 0) v += totals[blockIdx.x - 1];
    if (idx < m) x[idx] = v;
}

// Pass 2: writes row i of A_tilde (off-diagonal entries in order with the diagonal merged in) and
// checks that every stored (i, c) has its mirror (c, i) by binary search in row c.
template <bool kMean>
__global__ void __launch_bounds__(kRowsPerBlock* kWarp)
fill_kernel(int64_t n, const int64_t* __restrict__ rowptr_A, const int32_t* __restrict__ colidx_A,
            const int64_t* __restrict__ rowptr, int32_t* __restrict__ colidx, float* __restrict__ val,
            const float* __restrict__ dinv, int* __restrict__ flag)
{
    const int lane = threadIdx.x & 31;
    const int64_t i = (int64_t)blockIdx.x * kRowsPerBlock + (threadIdx.x >> 5);
    if (i >= n) return;
    if (*reinterpret_cast<volatile int*>(flag) != 0) return;     // pass 1 rejected the input: touch nothing
    const int64_t a = rowptr_A[i], b = rowptr_A[i + 1];
    const int64_t out0 = rowptr[i];
    const float di = dinv[i];
    // number of off-diagonal entries smaller than i = position of the diagonal in the output row
    int below = 0;
    for (int64_t q = a + lane; q < b; q += 32) below += (colidx_A[q] < (int32_t)i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) below += __shfl_xor_sync(0xffffffffu, below, o);
    if (!kMean && lane == 0) {
        colidx[out0 + below] = (int32_t)i;
        val[out0 + below] = __fmul_rn(di, di);
    }
    const int n_out = (int)(rowptr[i + 1] - out0);            // stored entries of the output row
    const int has_self = (int)(b - a) - (kMean ? n_out : n_out - 1);
    int bad = 0;
    for (int64_t q = a + lane; q < b; q += 32) {
        const int32_t c = colidx_A[q];
        if (c == (int32_t)i) continue;
        // entries before the diagonal keep their rank; the diagonal of the input (if any) is skipped
        int64_t rank = q - a;
        if (c > (int32_t)i) rank = rank - has_self + (kMean ? 0 : 1);
        colidx[out0 + rank] = c;
        val[out0 + rank] = kMean ? di : __fmul_rn(di, dinv[c]);
        int64_t lo = rowptr_A[c], hi = rowptr_A[c + 1];      // mirror entry (c, i)
        bool found = false;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            const int32_t m = colidx_A[mid];
            if (m == (int32_t)i) { found = true; break; }
            if (m < (int32_t)i) lo = mid + 1; else hi = mid;
        }
        if (!found) bad |= kFlagSymmetry;
    }
    if (bad) atomicOr(flag, bad);
}

// ---- batch statistics ---------------------------------------------------------------------------

constexpr int kStatChunksMax = 1024;

__global__ void __launch_bounds__(256)
col_partial_kernel(const float* __restrict__ H, int64_t n, int d, int64_t ld, int64_t rows_per_chunk,
                   double* __restrict__ partial /* [chunks][d][2] */)
{
    __shared__ double s_sum[8][33], s_sq[8][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int j = blockIdx.x * 32 + tx;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_chunk;
    const int64_t r1 = min(n, r0 + rows_per_chunk);
    // sums of (x - pivot) and (x - pivot)^2 around the column's first value: the variance formed from them does
    // not cancel for a column with a large offset, and is exactly 0 for a constant one
    double s = 0.0, q = 0.0;
    if (j < d) {
        const double pivot = (double)__ldg(H + j);
        for (int64_t r = r0 + ty; r < r1; r += 8) {
            const double x = (double)__ldg(H + r * ld + j) - pivot;
            s += x;
            q += x * x;
        }
    }
    s_sum[ty][tx] = s;
    s_sq[ty][tx] = q;
    __syncthreads();
    if (ty == 0 && j < d) {
        double ts = 0.0, tq = 0.0;
        for (int r = 0; r < 8; ++r) { ts += s_sum[r][tx]; tq += s_sq[r][tx]; }
        partial[((int64_t)blockIdx.y * d + j) * 2] = ts;
        partial[((int64_t)blockIdx.y * d + j) * 2 + 1] = tq;
    }
}

__global__ void col_final_kernel(const float* __restrict__ H, const double* __restrict__ partial, int chunks, int d, int64_t n, double eps,
                                 float* __restrict__ shift, float* __restrict__ scale)
{
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= d) return;
    double s = 0.0, q = 0.0;
    for (int c = 0; c < chunks; ++c) {
        s += partial[((int64_t)c * d + j) * 2];
        q += partial[((int64_t)c * d + j) * 2 + 1];
    }
    const double off = n > 0 ? s / (double)n : 0.0;                       // mean of x - pivot
    const double mean = n > 0 ? (double)__ldg(H + j) + off : 0.0;
    double var = n > 0 ? q / (double)n - off * off : 0.0;
    if (var < 0.0) var = 0.0;
    shift[j] = (float)mean;
    scale[j] = (float)(1.0 / sqrt(var + eps));
}

}  // namespace

size_t normalize_scratch_bytes(int64_t n) { return (size_t)(ceil_div(n, kScanBlock) + 2) * 8; }

cudaError_t launch_normalize_adjacency(cudaStream_t s, int64_t n, int64_t nnz_in,
                                       const int64_t* rowptr_A, const int32_t* colidx_A,
                                       int64_t* rowptr, int32_t* colidx, float* val, float* dinv,
                                       void* scratch, int* d_flag, int* launches, bool mean)
{
    cudaError_t e = cudaMemsetAsync(d_flag, 0, sizeof(int), s);
    if (e != cudaSuccess) return e;
    const unsigned row_blocks = (unsigned)ceil_div(n, kRowsPerBlock);
    if (mean) degree_kernel<true><<<row_blocks, kRowsPerBlock * kWarp, 0, s>>>(n, nnz_in, rowptr_A, colidx_A, rowptr, dinv, d_flag);
    else degree_kernel<false><<<row_blocks, kRowsPerBlock * kWarp, 0, s>>>(n, nnz_in, rowptr_A, colidx_A, rowptr, dinv, d_flag);
    ++*launches;
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    int64_t* totals = reinterpret_cast<int64_t*>(scratch);
    const int64_t nb = ceil_div(n, kScanBlock);
    scan_totals_kernel<<<(unsigned)nb, kScanBlock, 0, s>>>(rowptr + 1, n, totals);
    scan_of_totals_kernel<<<1, kScanBlock, 0, s>>>(totals, nb);
    scan_apply_kernel<<<(unsigned)nb, kScanBlock, 0, s>>>(rowptr + 1, n, totals);
    *launches += 3;
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (mean) fill_kernel<true><<<row_blocks, kRowsPerBlock * kWarp, 0, s>>>(n, rowptr_A, colidx_A, rowptr, colidx, val, dinv, d_flag);
    else fill_kernel<false><<<row_blocks, kRowsPerBlock * kWarp, 0, s>>>(n, rowptr_A, colidx_A, rowptr, colidx, val, dinv, d_flag);
    ++*launches;
    return cudaGetLastError();
}

size_t col_stats_scratch_bytes(int d) { return (size_t)kStatChunksMax * (size_t)d * 16; }

cudaError_t launch_col_stats(cudaStream_t s, const float* H, int64_t n, int d, int64_t ld, float eps,
                             float* shift, float* scale, void* scratch, int* launches)
{
    const int64_t rows_per_chunk = std::max<int64_t>(256, ceil_div(n, kStatChunksMax));
    const int chunks = (int)std::max<int64_t>(1, ceil_div(n, rows_per_chunk));
    double* partial = reinterpret_cast<double*>(scratch);
    col_partial_kernel<<<dim3((unsigned)ceil_div(d, 32), (unsigned)chunks), 256, 0, s>>>(H, n, d, ld, rows_per_chunk, partial);
    ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    col_final_kernel<<<(unsigned)ceil_div(d, 128), 128, 0, s>>>(H, partial, chunks, d, n, (double)eps, shift, scale);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace bigcn
