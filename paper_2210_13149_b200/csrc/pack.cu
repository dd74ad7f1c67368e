// Binarization + bit packing of node features (rows) and weights (columns).
// Bi-GCN Sec. 4.2.1 (Eq. "B", "alpha"), Sec. 4.2.2 (Eq. "F", "beta"), Sec. 4.4 (batch-normalised input).
#include "bigcn_internal.cuh"

namespace bigcn {

namespace {

constexpr int kPackWarpsPerBlock = 8;

// One warp per row.  Lane l reads element 32 w + l of the row (128 contiguous bytes per warp load,
// whatever the row's alignment), so the ballot of "x >= 0" IS packed word w.  Up to 32 words are
// kept one per lane and stored with a single coalesced write.
template <bool kNorm>
__global__ void __launch_bounds__(kPackWarpsPerBlock* kWarp)
pack_rows_kernel(const float* __restrict__ H, int64_t n, int d, int64_t ld,
                 const float* __restrict__ shift, const float* __restrict__ scale,
                 uint32_t* __restrict__ bits, int64_t stride, float* __restrict__ beta)
{
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * kPackWarpsPerBlock + (threadIdx.x >> 5);
    if (row >= n) return;
    const float* __restrict__ h = H + row * ld;
    uint32_t* __restrict__ out = bits + row * stride;
    const int kw = (d + 31) >> 5;
    float l1 = 0.f;
    for (int w0 = 0; w0 < stride; w0 += 32) {
        uint32_t mine = 0u;
        const int wend = min(32, kw - w0);
#pragma unroll 4
        for (int ww = 0; ww < wend; ++ww) {
            const int j = ((w0 + ww) << 5) + lane;
            bool pos = false;
            if (j < d) {
                float x = __ldg(h + j);
                if (kNorm) x = __fmul_rn(__fsub_rn(x, __ldg(shift + j)), __ldg(scale + j));
                pos = x >= 0.f;
                l1 += fabsf(x);
            }
            const uint32_t word = __ballot_sync(0xffffffffu, pos);
            if (lane == ww) mine = word;
        }
        if (w0 + lane < stride) out[w0 + lane] = mine;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l1 += __shfl_xor_sync(0xffffffffu, l1, o);
    if (lane == 0) beta[row] = l1 / (float)d;
}

// Weights: W is [d_in x d_out] row-major and the packed output is transposed (one row per output
// channel, packed along d_in).  A 32 x 32 tile is read coalesced along d_out, the sign bits go
// through shared memory, and warp t ballots the 32 k-values of channel j0 + t.
__global__ void __launch_bounds__(1024)
pack_weights_kernel(const float* __restrict__ W, int d_in, int d_out, int64_t ldw,
                    uint32_t* __restrict__ bitsT, int64_t stride)
{
    __shared__ unsigned char sgn[32][33];
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int j0 = blockIdx.x * 32;
    const int w = blockIdx.y;                 // word index along d_in; words >= ceil(d_in/32) are padding
    const int k = w * 32 + ty;
    const int j = j0 + tx;
    bool pos = false;
    if (k < d_in && j < d_out) pos = __ldg(W + (int64_t)k * ldw + j) >= 0.f;
    sgn[ty][tx] = pos ? 1 : 0;
    __syncthreads();
    const uint32_t word = __ballot_sync(0xffffffffu, sgn[tx][ty] != 0);   // lane tx = k offset, channel j0 + ty
    if (tx == 0 && j0 + ty < d_out) bitsT[(int64_t)(j0 + ty) * stride + w] = word;
}

// alpha_j = ||W_:,j||_1 / d_in.  One block per 32 channels; thread (tx, ty) sums rows ty, ty+32, ...
// of column j0 + tx in double, then the 32 partial sums of a column are added in a fixed order.
__global__ void __launch_bounds__(1024)
weight_scale_kernel(const float* __restrict__ W, int d_in, int d_out, int64_t ldw, float* __restrict__ alpha)
{
    __shared__ double part[32][33];
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int j = blockIdx.x * 32 + tx;
    double s = 0.0;
    if (j < d_out)
        for (int k = ty; k < d_in; k += 32) s += (double)fabsf(__ldg(W + (int64_t)k * ldw + j));
    part[ty][tx] = s;
    __syncthreads();
    if (ty == 0 && j < d_out) {
        double t = 0.0;
        for (int r = 0; r < 32; ++r) t += part[r][tx];
        alpha[j] = (float)(t / (double)d_in);
    }
}

}  // namespace

cudaError_t launch_pack_rows(cudaStream_t s, const float* H, int64_t n, int d, int64_t ld,
                             const float* shift, const float* scale,
                             uint32_t* bits, int64_t stride, float* beta, int* launches)
{
    if (n == 0) return cudaSuccess;
    const unsigned grid = (unsigned)ceil_div(n, kPackWarpsPerBlock);
    const dim3 block(kPackWarpsPerBlock * kWarp);
    if (shift)
        pack_rows_kernel<true><<<grid, block, 0, s>>>(H, n, d, ld, shift, scale, bits, stride, beta);
    else
        pack_rows_kernel<false><<<grid, block, 0, s>>>(H, n, d, ld, nullptr, nullptr, bits, stride, beta);
    ++*launches;
    return cudaGetLastError();
}

cudaError_t launch_pack_weights(cudaStream_t s, const float* W, int d_in, int d_out, int64_t ldw,
                                uint32_t* bitsT, int64_t stride, float* alpha, int* launches)
{
    const dim3 block(32, 32);
    const dim3 grid((unsigned)ceil_div(d_out, 32), (unsigned)stride);
    pack_weights_kernel<<<grid, block, 0, s>>>(W, d_in, d_out, ldw, bitsT, stride);
    ++*launches;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    weight_scale_kernel<<<(unsigned)ceil_div(d_out, 32), block, 0, s>>>(W, d_in, d_out, ldw, alpha);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace bigcn
