// Binarization + bit packing of node features (rows) and weights (columns).
// Bi-GCN Sec. 4.2.1 (Eq. "B", "alpha"), Sec. 4.2.2 (Eq. "F", "beta"), Sec. 4.4 (batch-normalised input).
#include <algorithm>

#include "bigcn_internal.cuh"

namespace bigcn {

namespace {

constexpr int kPackWarpsPerBlock = 8;

// A warp packs R rows at a time.  Lane l reads element 32 w + l of a row (128 contiguous bytes per
// warp load, whatever the row's alignment), so the ballot of "x >= 0" IS packed word w.  The loads of
// a chunk of WC words of all R rows are issued before any of them is used (R * WC loads of 128 bytes
// in flight per warp), and warps loop over the rows of the matrix (persistent grid).  Up to 32 words
// per row are kept one per lane and stored with a single coalesced write.  The R row sums of |x| are
// reduced together: each exchange step halves the rows a lane still carries.
template <bool kNorm, int R, int WC>
__global__ void __launch_bounds__(kPackWarpsPerBlock* kWarp)
pack_rows_kernel(const float* __restrict__ H, int64_t n, int d, int64_t ld,
                 const float* __restrict__ shift, const float* __restrict__ scale,
                 uint32_t* __restrict__ bits, int64_t stride, float* __restrict__ beta)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp_id = (int64_t)blockIdx.x * kPackWarpsPerBlock + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * kPackWarpsPerBlock;
    const int kw = (d + 31) >> 5;
    const float inv_d = 1.f / (float)d;
    for (int64_t row0 = warp_id * R; row0 < n; row0 += n_warps * R) {
        float l1[R];
#pragma unroll
        for (int r = 0; r < R; ++r) l1[r] = 0.f;
        for (int w0 = 0; w0 < stride; w0 += 32) {
            uint32_t mine[R];
#pragma unroll
            for (int r = 0; r < R; ++r) mine[r] = 0u;
            const int wlast = min(w0 + 32, kw);
            for (int c0 = w0; c0 < wlast; c0 += WC) {
                float x[R][WC];
#pragma unroll
                for (int r = 0; r < R; ++r)
#pragma unroll
                    for (int q = 0; q < WC; ++q) {
                        const int j = ((c0 + q) << 5) + lane;
                        x[r][q] = (row0 + r < n && j < d) ? __ldg(H + (row0 + r) * ld + j) : 0.f;
                    }
#pragma unroll
                for (int q = 0; q < WC; ++q) {
                    const int j = ((c0 + q) << 5) + lane;
                    const bool in = j < d;
                    float sh = 0.f, sc = 1.f;
                    if (kNorm && in) { sh = __ldg(shift + j); sc = __ldg(scale + j); }
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        float v = x[r][q];
                        if (kNorm) v = __fmul_rn(__fsub_rn(v, sh), sc);
                        const bool pos = in && (v >= 0.f);
                        if (in) l1[r] += fabsf(v);
                        const uint32_t word = __ballot_sync(0xffffffffu, pos);
                        if (lane == c0 + q - w0) mine[r] = word;
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < R; ++r)
                if (row0 + r < n && w0 + lane < stride) bits[(row0 + r) * stride + w0 + lane] = mine[r];
        }
        // reduce the R row sums: after the halving steps lane L carries row L / (32 / R)
        int off = 16;
#pragma unroll
        for (int half = R / 2; half >= 1; half /= 2, off /= 2) {
            const bool upper = (lane & off) != 0;
#pragma unroll
            for (int i = 0; i < half; ++i) {
                const float send = upper ? l1[i] : l1[i + half];
                const float keep = upper ? l1[i + half] : l1[i];
                l1[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
            }
        }
        for (int o = off; o >= 1; o /= 2) l1[0] += __shfl_xor_sync(0xffffffffu, l1[0], o);
        constexpr int kLanesPerRow = 32 / R;
        const int64_t row = row0 + lane / kLanesPerRow;
        if (lane % kLanesPerRow == 0 && row < n) beta[row] = l1[0] * inv_d;
    }
}

// The same packing with 16-byte loads, for matrices whose rows start on 16-byte boundaries
// (ld a multiple of 4, base aligned): lane l of a warp reads columns 128 c + 4 l .. + 3 of chunk c,
// so a row of up to 128 columns costs one load instruction instead of four.  The four sign bits of a
// lane are shifted to their place in the packed word and OR-ed over the 8 lanes that share the word.
// A warp walks over tiles of R rows x one chunk and always has the NEXT tile's loads in flight while
// it works on the current one (two register buffers used in turn), so the memory system is never
// idle behind the arithmetic.  kRagged: d is not a multiple of 4, so one lane of a row holds columns
// past the end that must not count.
template <bool kNorm, bool kRagged, int R>
__global__ void __launch_bounds__(kPackWarpsPerBlock* kWarp, 4)
pack_rows_vec_kernel(const float* __restrict__ H, int64_t n, int d, int64_t ld,
                     const float* __restrict__ shift, const float* __restrict__ scale,
                     uint32_t* __restrict__ bits, int64_t stride, float* __restrict__ beta)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp_id = (int64_t)blockIdx.x * kPackWarpsPerBlock + (threadIdx.x >> 5);
    const int64_t row_step = (int64_t)gridDim.x * kPackWarpsPerBlock * R;
    const int n_chunks = (int)(stride >> 2);      // 4 packed words = 128 columns per chunk
    const int sub = lane & 7;                     // this lane's nibble inside its packed word
    const int shl = 4 * sub;
    const float inv_d = 1.f / (float)d;

    struct Tile { int64_t row0; int ch; };
    auto next_of = [&](Tile t) {
        Tile u = {t.row0, t.ch + 1};
        if (u.ch == n_chunks) { u.ch = 0; u.row0 = t.row0 + row_step; }
        return u;
    };
    auto load_tile = [&](Tile t, float4 (&x)[R]) {
        const int j0 = t.ch * 128 + lane * 4;
        const float* src = H + t.row0 * ld + j0;
        const bool lane_in = j0 < d;
        if (t.row0 + R <= n) {                                    // the usual case: no row checks
#pragma unroll
            for (int r = 0; r < R; ++r)
                x[r] = lane_in ? __ldg(reinterpret_cast<const float4*>(src + r * ld)) : make_float4(0.f, 0.f, 0.f, 0.f);
        } else {
#pragma unroll
            for (int r = 0; r < R; ++r)
                x[r] = (lane_in && t.row0 + r < n) ? __ldg(reinterpret_cast<const float4*>(src + r * ld))
                                                   : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    float sh[4] = {0.f, 0.f, 0.f, 0.f}, sc[4] = {1.f, 1.f, 1.f, 1.f};
    auto load_norm = [&](int ch) {
        const int j0 = ch * 128 + lane * 4;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const bool in = j0 + i < d;
            sh[i] = in ? __ldg(shift + j0 + i) : 0.f;
            sc[i] = in ? __ldg(scale + j0 + i) : 1.f;
        }
    };
    float l1[R];
#pragma unroll
    for (int r = 0; r < R; ++r) l1[r] = 0.f;

    auto process = [&](Tile t, const float4 (&x)[R]) {
        const int j0 = t.ch * 128 + lane * 4;
        const int n_valid = min(max(d - j0, 0), 4);               // columns of this lane that exist
        const uint32_t keep = ((1u << n_valid) - 1u) << shl;      // missing columns pack as 0
        uint32_t* dst = bits + t.row0 * stride + t.ch * 4 + (lane >> 3);
        const bool full = t.row0 + R <= n;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            float v[4] = {x[r].x, x[r].y, x[r].z, x[r].w};
            uint32_t word = 0u;
            float part = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (kRagged && i >= n_valid) v[i] = 0.f;          // whatever lies between d and ld is not data
                if (kNorm) v[i] = __fmul_rn(__fsub_rn(v[i], sh[i]), sc[i]);
                if (v[i] >= 0.f) word |= 1u << i;
                part += fabsf(v[i]);
            }
            l1[r] += part;
            word = (word << shl) & keep;
            word |= __shfl_xor_sync(0xffffffffu, word, 1);
            word |= __shfl_xor_sync(0xffffffffu, word, 2);
            word |= __shfl_xor_sync(0xffffffffu, word, 4);
            if (sub == 0 && (full || t.row0 + r < n)) dst[r * stride] = word;
        }
        if (t.ch == n_chunks - 1) {
            // reduce the R row sums: after the halving steps lane L carries row L / (32 / R)
            int off = 16;
#pragma unroll
            for (int half = R / 2; half >= 1; half /= 2, off /= 2) {
                const bool upper = (lane & off) != 0;
#pragma unroll
                for (int i = 0; i < half; ++i) {
                    const float send = upper ? l1[i] : l1[i + half];
                    const float keep_v = upper ? l1[i + half] : l1[i];
                    l1[i] = keep_v + __shfl_xor_sync(0xffffffffu, send, off);
                }
            }
            for (int o = off; o >= 1; o /= 2) l1[0] += __shfl_xor_sync(0xffffffffu, l1[0], o);
            constexpr int kLanesPerRow = 32 / R;
            const int64_t row = t.row0 + lane / kLanesPerRow;
            if (lane % kLanesPerRow == 0 && row < n) beta[row] = l1[0] * inv_d;
#pragma unroll
            for (int r = 0; r < R; ++r) l1[r] = 0.f;
        }
    };

    Tile ta = {warp_id * R, 0};
    if (ta.row0 >= n) return;
    float4 xa[R], xb[R];
    load_tile(ta, xa);
    if (kNorm) load_norm(0);
    for (;;) {
        const Tile tb = next_of(ta);
        const bool has_b = tb.row0 < n;
        if (has_b) load_tile(tb, xb);
        process(ta, xa);
        if (!has_b) break;
        if (kNorm && n_chunks > 1) load_norm(tb.ch);
        ta = next_of(tb);
        const bool has_a = ta.row0 < n;
        if (has_a) load_tile(ta, xa);
        process(tb, xb);
        if (!has_a) break;
        if (kNorm && n_chunks > 1) load_norm(ta.ch);
    }
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
    if (ld % 4 == 0 && reinterpret_cast<uintptr_t>(H) % 16 == 0) {          // rows start on 16-byte boundaries
        constexpr int R = 4;
        auto kernel = shift ? ((d & 3) ? pack_rows_vec_kernel<true, true, R> : pack_rows_vec_kernel<true, false, R>)
                            : ((d & 3) ? pack_rows_vec_kernel<false, true, R> : pack_rows_vec_kernel<false, false, R>);
        // persistent grid: exactly the blocks that are resident at once, so that no block waits for a slot
        int per_sm = 0, n_sm = 0, dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kPackWarpsPerBlock * kWarp, 0);
        if (e != cudaSuccess) return e;
        const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(n, (int64_t)kPackWarpsPerBlock * R), (int64_t)n_sm * std::max(per_sm, 1));
        kernel<<<grid, kPackWarpsPerBlock * kWarp, 0, s>>>(H, n, d, ld, shift, scale, bits, stride, beta);
        ++*launches;
        return cudaGetLastError();
    }
    const int kw = (d + 31) / 32;
    const int rows = kw <= 4 ? 8 : (kw <= 8 ? 4 : (kw <= 32 ? 2 : 1));     // rows a warp packs at a time
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(n, (int64_t)kPackWarpsPerBlock * rows), 148 * 8);
    const dim3 block(kPackWarpsPerBlock * kWarp);
#define BIGCN_PACK_LAUNCH(NORM, R, WC) \
    pack_rows_kernel<NORM, R, WC><<<grid, block, 0, s>>>(H, n, d, ld, shift, scale, bits, stride, beta)
    if (shift) {
        if (rows == 8) BIGCN_PACK_LAUNCH(true, 8, 4);
        else if (rows == 4) BIGCN_PACK_LAUNCH(true, 4, 8);
        else if (rows == 2) BIGCN_PACK_LAUNCH(true, 2, 8);
        else BIGCN_PACK_LAUNCH(true, 1, 8);
    } else {
        if (rows == 8) BIGCN_PACK_LAUNCH(false, 8, 4);
        else if (rows == 4) BIGCN_PACK_LAUNCH(false, 4, 8);
        else if (rows == 2) BIGCN_PACK_LAUNCH(false, 2, 8);
        else BIGCN_PACK_LAUNCH(false, 1, 8);
    }
#undef BIGCN_PACK_LAUNCH
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
