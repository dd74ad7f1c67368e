// Binarization + bit packing of node features (rows) and weights (columns).
// Bi-GCN Sec. 4.2.1 (Eq. "B", "alpha"), Sec. 4.2.2 (Eq. "F", "beta"), Sec. 4.4 (batch-normalised input).
#include <algorithm>
#include <mutex>

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

// Packing through shared memory, for matrices whose rows start on 16-byte boundaries (ld a multiple
// of 4, base aligned).  In the kernel above a warp instruction handles one element per lane and most
// instructions are bookkeeping per row; here a LANE owns a whole packed word: the warp copies a tile
// of 8 rows x 128 columns into its own shared-memory ring with 16-byte asynchronous copies (coalesced,
// no registers in between), and then lane 4r + w packs word w of row r from 32 consecutive floats, so
// the sign bits need no exchange between lanes and every bookkeeping instruction is shared by 32
// elements.  Three tiles per warp are in flight.  The staged rows are skewed (one 16-byte pad after
// every 8 units, 36 units per row) so that the 16-byte reads of a quarter warp -- 4 words x 2 rows --
// fall into 8 different bank groups; the per-column shift and scale sit in shared memory in the same
// skewed form.  kRagged: d is not a multiple of 4, so the last 16-byte unit of a row holds columns
// past the end that must not count.
constexpr int kStageRows = 8;                         // rows per tile
constexpr int kStageRowUnits = 36;                    // 16-byte units per staged row: 4 words x (8 + 1 pad)
constexpr int kStageTileUnits = kStageRows * kStageRowUnits;
constexpr int kStageTiles = 3;                        // tiles in flight per warp

__device__ __forceinline__ void stage_copy16(float4* smem_dst, const float* gmem_src)
{
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(gmem_src) : "memory");
}

template <bool kNorm, bool kRagged>
__global__ void __launch_bounds__(kPackWarpsPerBlock* kWarp, 2)
pack_rows_staged_kernel(const float* __restrict__ H, int64_t n, int d, int64_t ld,
                        const float* __restrict__ shift, const float* __restrict__ scale,
                        uint32_t* __restrict__ bits, int64_t stride, float* __restrict__ beta)
{
    extern __shared__ __align__(16) unsigned char pack_smem[];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    float4* ring = reinterpret_cast<float4*>(pack_smem) + warp * (kStageTiles * kStageTileUnits);
    float4* tab_shift = reinterpret_cast<float4*>(pack_smem) + kPackWarpsPerBlock * kStageTiles * kStageTileUnits;
    const int tab_units = (int)stride * 9;            // 8 units of data + 1 pad per packed word
    float4* tab_scale = tab_shift + tab_units;
    if (kNorm) {
        for (int col = threadIdx.x; col < (int)stride * 32; col += blockDim.x) {
            const int at = (col >> 5) * 36 + (col & 31);          // float index in the skewed table
            reinterpret_cast<float*>(tab_shift)[at] = col < d ? __ldg(shift + col) : 0.f;
            reinterpret_cast<float*>(tab_scale)[at] = col < d ? __ldg(scale + col) : 1.f;
        }
        __syncthreads();
    }
    const int64_t warp_id = (int64_t)blockIdx.x * kPackWarpsPerBlock + warp;
    const int64_t row_step = (int64_t)gridDim.x * kPackWarpsPerBlock * kStageRows;
    const int n_chunks = (int)(stride >> 2);          // 4 packed words = 128 columns per chunk
    const float inv_d = 1.f / (float)d;
    const int r = lane >> 2, w = lane & 3;            // the (row, word) of a tile this lane packs
    const int copy_unit = 9 * (lane >> 3) + (lane & 7);   // where this lane's 16 bytes of a staged row go

    // issue cursor and consume cursor walk the same sequence of tiles (row group, chunk)
    int64_t i_row0 = warp_id * kStageRows, c_row0 = i_row0;
    int i_ch = 0, c_ch = 0, i_slot = 0, c_slot = 0;
    float l1 = 0.f;
    auto issue = [&]() {
        if (i_row0 < n) {
            float4* dst = ring + i_slot * kStageTileUnits + copy_unit;
            const int col = i_ch * 128 + 4 * lane;
            const float* src = H + i_row0 * ld + col;
            const bool col_in = col < d;
            const int rows_in = (int)min((int64_t)kStageRows, n - i_row0);
#pragma unroll
            for (int q = 0; q < kStageRows; ++q) {
                if (col_in && q < rows_in) stage_copy16(dst + q * kStageRowUnits, src + q * ld);
                else dst[q * kStageRowUnits] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            if (++i_ch == n_chunks) { i_ch = 0; i_row0 += row_step; }
            i_slot = i_slot + 1 == kStageTiles ? 0 : i_slot + 1;
        }
        asm volatile("cp.async.commit_group;\n" ::: "memory");   // one group per call, possibly empty
    };
#pragma unroll
    for (int t = 0; t < kStageTiles - 1; ++t) issue();
    while (c_row0 < n) {
        issue();
        asm volatile("cp.async.wait_group %0;\n" ::"n"(kStageTiles - 1) : "memory");
        __syncwarp();                                 // the other lanes' copies of this tile are visible
        const float4* src = ring + c_slot * kStageTileUnits + r * kStageRowUnits + w * 9;
        const float4* ts = tab_shift + (c_ch * 4 + w) * 9;
        const float4* tc = tab_scale + (c_ch * 4 + w) * 9;
        const int n_valid = min(max(d - (c_ch * 128 + w * 32), 0), 32);      // columns of this word that exist
        uint32_t word = 0u;
        float part = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float4 x = src[k];
            float v[4] = {x.x, x.y, x.z, x.w};
            float sh[4] = {0.f, 0.f, 0.f, 0.f}, sc[4] = {1.f, 1.f, 1.f, 1.f};
            if (kNorm) {
                const float4 a = ts[k], b = tc[k];
                sh[0] = a.x, sh[1] = a.y, sh[2] = a.z, sh[3] = a.w;
                sc[0] = b.x, sc[1] = b.y, sc[2] = b.z, sc[3] = b.w;
            }
            float quad = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (kRagged && 4 * k + j >= n_valid) v[j] = 0.f;  // whatever lies between d and ld is not data
                if (kNorm) v[j] = __fmul_rn(__fsub_rn(v[j], sh[j]), sc[j]);
                if (v[j] >= 0.f) word |= 1u << (4 * k + j);
                quad += fabsf(v[j]);
            }
            part += quad;
        }
        if (n_valid < 32) word &= (1u << n_valid) - 1u;           // columns past d pack as 0 (their staged value is 0)
        l1 += part;
        const int64_t row = c_row0 + r;
        if (row < n) bits[row * stride + c_ch * 4 + w] = word;
        if (c_ch == n_chunks - 1) {                               // the row is complete: its 4 lanes add up
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
            if (w == 0 && row < n) beta[row] = l1 * inv_d;
            l1 = 0.f;
        }
        __syncwarp();                                 // all lanes are done with the slot before it is refilled
        if (++c_ch == n_chunks) { c_ch = 0; c_row0 += row_step; }
        c_slot = c_slot + 1 == kStageTiles ? 0 : c_slot + 1;
    }
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
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
    const size_t staged_smem = (size_t)kPackWarpsPerBlock * kStageTiles * kStageTileUnits * 16 + (shift ? 2 * (size_t)stride * 9 * 16 : 0);
    if (ld % 4 == 0 && reinterpret_cast<uintptr_t>(H) % 16 == 0 && staged_smem <= 200 * 1024) {   // rows start on 16-byte boundaries
        const int variant = (shift ? 2 : 0) + ((d & 3) ? 1 : 0);
        auto kernel = shift ? ((d & 3) ? pack_rows_staged_kernel<true, true> : pack_rows_staged_kernel<true, false>)
                            : ((d & 3) ? pack_rows_staged_kernel<false, true> : pack_rows_staged_kernel<false, false>);
        // persistent grid: exactly the blocks that are resident at once, so that no block waits for a slot.
        // The attribute and the occupancy query cost tens of microseconds of host time each, so their
        // result is kept per kernel variant for the last (device, shared-memory size) seen.
        struct Cached { int dev = -1; size_t smem = 0; int per_sm = 0; int n_sm = 0; };
        static Cached cache[4];
        static std::mutex cache_mutex;
        int per_sm = 0, n_sm = 0, dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        {
            std::lock_guard<std::mutex> lock(cache_mutex);
            Cached& c = cache[variant];
            if (c.dev != dev || c.smem != staged_smem) {
                e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)staged_smem);
                if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
                if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kPackWarpsPerBlock * kWarp, staged_smem);
                if (e != cudaSuccess) return e;
                c.dev = dev, c.smem = staged_smem, c.per_sm = per_sm, c.n_sm = n_sm;
            }
            per_sm = c.per_sm, n_sm = c.n_sm;
        }
        const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(n, (int64_t)kPackWarpsPerBlock * kStageRows), (int64_t)n_sm * std::max(per_sm, 1));
        kernel<<<grid, kPackWarpsPerBlock * kWarp, staged_smem, s>>>(H, n, d, ld, shift, scale, bits, stride, beta);
        ++*launches;
        return cudaGetLastError();
    }
    const int kw = (d + 31) / 32;
    const int rows = kw <= 4 ? 8 : (kw <= 8 ? 4 : (kw <= 32 ? 2 : 1));     // rows a warp packs at a time
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(n, (int64_t)kPackWarpsPerBlock * rows), sm_count() * 8);
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
