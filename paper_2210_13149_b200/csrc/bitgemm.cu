// XNOR / bit-count contraction fused with the beta_i alpha_j rescale.
// Bi-GCN Sec. 4.2.3: dot_ij = F_i (*) B_j = d_in - 2 popc(F_i XOR B_j)   (Eq. "bi-op"),
//                    zeta_ij = beta_i alpha_j dot_ij                     (Eq. "cdot-op").
#include <cuda_fp16.h>

#include <algorithm>

#include "bigcn_internal.cuh"

namespace bigcn {

namespace {

constexpr int kGemmThreads = 256;
constexpr int kGemmWarps = kGemmThreads / kWarp;
constexpr int kRowsPerWarp = 8;
constexpr int kTileRows = kGemmWarps * kRowsPerWarp;   // 64 rows of A per tile
constexpr int kTM = 4;                                  // rows held in registers at a time

// Shared memory: the packed weight panel of this channel block (row pitch ldb words, odd, so that
// the 32 lanes of a warp - 32 consecutive channels - hit 32 different banks) and one tile of packed
// feature rows (read as warp-wide broadcasts).  Each lane owns channels lane, lane+32, ... (TN of
// them) and kTM rows at a time: kTM x TN integer accumulators of popc(a XOR b).
template <int TN, int FMT, bool DBG>
__global__ void __launch_bounds__(kGemmThreads)
bitgemm_kernel(const uint32_t* __restrict__ A, int64_t stride_a,
               const uint32_t* __restrict__ BT, int64_t stride_b,
               int64_t n, int d_in, int d_out, int kw, int ldb,
               const float* __restrict__ beta, const float* __restrict__ alpha,
               void* __restrict__ zeta, int64_t ldz,
               int32_t* __restrict__ dbg_dot, float* __restrict__ dbg_zeta)
{
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t* Bs = smem;                                   // [TN*32][ldb]
    uint32_t* As = smem + (size_t)TN * 32 * ldb;           // [kTileRows][stride_a]  (16-byte aligned: see launcher)
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int jblock = blockIdx.y * (TN * 32);

    for (int idx = threadIdx.x; idx < TN * 32 * kw; idx += kGemmThreads) {
        const int c = idx / kw, k = idx - c * kw;
        const int j = jblock + c;
        Bs[c * ldb + k] = (j < d_out) ? __ldg(BT + (int64_t)j * stride_b + k) : 0u;
    }
    float al[TN];
#pragma unroll
    for (int t = 0; t < TN; ++t) {
        const int j = jblock + lane + 32 * t;
        al[t] = (j < d_out) ? __ldg(alpha + j) : 0.f;
    }

    const int64_t n_tiles = ceil_div(n, kTileRows);
    const int sa4 = (int)(stride_a >> 2);
    const bool small_k = d_in <= 511;
    for (int64_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        const int64_t r0 = tile * kTileRows;
        const int rows_here = (int)min((int64_t)kTileRows, n - r0);
        __syncthreads();                                   // previous tile fully consumed (and Bs visible)
        {
            const uint4* src = reinterpret_cast<const uint4*>(A + r0 * stride_a);
            uint4* dst = reinterpret_cast<uint4*>(As);
            const int total = rows_here * sa4;
            for (int idx = threadIdx.x; idx < total; idx += kGemmThreads) dst[idx] = __ldg(src + idx);
        }
        __syncthreads();
#pragma unroll 1
        for (int pass = 0; pass < kRowsPerWarp / kTM; ++pass) {
            const int lr0 = warp * kRowsPerWarp + pass * kTM;     // first local row of this pass
            if (lr0 >= rows_here) break;
            int acc[kTM][TN];
#pragma unroll
            for (int m = 0; m < kTM; ++m)
#pragma unroll
                for (int t = 0; t < TN; ++t) acc[m][t] = 0;
            const uint32_t* arow = As + (size_t)lr0 * stride_a;
            const uint32_t* brow = Bs + lane * ldb;
#pragma unroll 2
            for (int k = 0; k < kw; ++k) {
                uint32_t a[kTM], b[TN];
#pragma unroll
                for (int m = 0; m < kTM; ++m) a[m] = arow[(size_t)m * stride_a + k];   // rows past the tile read stale but in-bounds smem
#pragma unroll
                for (int t = 0; t < TN; ++t) b[t] = brow[t * 32 * ldb + k];
#pragma unroll
                for (int m = 0; m < kTM; ++m)
#pragma unroll
                    for (int t = 0; t < TN; ++t) acc[m][t] += __popc(a[m] ^ b[t]);
            }
#pragma unroll
            for (int m = 0; m < kTM; ++m) {
                const int lr = lr0 + m;
                if (lr >= rows_here) break;
                const int64_t row = r0 + lr;
                const float be = __ldg(beta + row);
#pragma unroll
                for (int t = 0; t < TN; ++t) {
                    const int j = jblock + lane + 32 * t;
                    const int dot = d_in - 2 * acc[m][t];
                    if (j < d_out) {
                        if constexpr (FMT == kZetaF16) {
                            // exact integer -> fp16; for |dot| <= 511 without the conversion unit (which the bit
                            // counts keep busy): the bit pattern 0x6600 + dot IS the half 1536 + dot
                            __half h;
                            if (small_k) h = __hsub(__ushort_as_half((unsigned short)(0x6600 + dot)), __ushort_as_half((unsigned short)0x6600));
                            else h = __int2half_rn(dot);                                   // exact: |dot| <= 2048
                            reinterpret_cast<__half*>(zeta)[row * ldz + j] = h;
                        } else if constexpr (FMT == kZetaF32) {
                            reinterpret_cast<float*>(zeta)[row * ldz + j] = __fmul_rn(__fmul_rn(be, al[t]), (float)dot);
                        } else if constexpr (FMT == kZetaI16) {
                            reinterpret_cast<int16_t*>(zeta)[row * ldz + j] = (int16_t)dot;
                        } else {
                            reinterpret_cast<int8_t*>(zeta)[row * ldz + j] = (int8_t)dot;
                        }
                        if constexpr (DBG) {
                            if (dbg_dot) dbg_dot[row * (int64_t)d_out + j] = dot;
                            if (dbg_zeta) dbg_zeta[row * (int64_t)d_out + j] = __fmul_rn(__fmul_rn(be, al[t]), (float)dot);
                        }
                    } else if (j < ldz) {                  // padding columns of the zeta row: keep them zero
                        if constexpr (FMT == kZetaF32) reinterpret_cast<float*>(zeta)[row * ldz + j] = 0.f;
                        else if constexpr (FMT == kZetaI8) reinterpret_cast<int8_t*>(zeta)[row * ldz + j] = 0;
                        else reinterpret_cast<int16_t*>(zeta)[row * ldz + j] = 0;          // int16 and fp16 zero alike
                    }
                }
            }
        }
    }
}

template <int TN, int FMT, bool DBG>
cudaError_t launch_inst(cudaStream_t s, const uint32_t* A, int64_t stride_a, const uint32_t* BT,
                        int64_t stride_b, int64_t n, int d_in, int d_out, const float* beta,
                        const float* alpha, void* zeta, int64_t ldz, int32_t* dbg_dot,
                        float* dbg_zeta, size_t smem_bytes, int ldb)
{
    const int kw = (d_in + 31) / 32;
    if (smem_bytes > 48 * 1024) {                          // opt in to large dynamic shared memory
        cudaError_t e = cudaFuncSetAttribute(bitgemm_kernel<TN, FMT, DBG>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem_bytes);
        if (e != cudaSuccess) return e;
    }
    const int64_t n_tiles = ceil_div(n, kTileRows);
    const unsigned gy = (unsigned)ceil_div(d_out, TN * 32);
    const unsigned gx = (unsigned)std::min<int64_t>(n_tiles, sm_count() * 8);
    bitgemm_kernel<TN, FMT, DBG><<<dim3(gx, gy), kGemmThreads, smem_bytes, s>>>(
        A, stride_a, BT, stride_b, n, d_in, d_out, kw, ldb, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta);
    return cudaGetLastError();
}

template <int TN>
cudaError_t launch_tn(cudaStream_t s, const uint32_t* A, int64_t stride_a, const uint32_t* BT,
                      int64_t stride_b, int64_t n, int d_in, int d_out, const float* beta,
                      const float* alpha, int fmt, void* zeta, int64_t ldz, int32_t* dbg_dot,
                      float* dbg_zeta, size_t smem_bytes, int ldb)
{
#define BIGCN_GEMM_CALL(FMT, DBG) \
    launch_inst<TN, FMT, DBG>(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta, smem_bytes, ldb)
    const bool dbg = dbg_dot || dbg_zeta;
    switch (fmt) {
        case kZetaF32: return dbg ? BIGCN_GEMM_CALL(kZetaF32, true) : BIGCN_GEMM_CALL(kZetaF32, false);
        case kZetaF16: return dbg ? BIGCN_GEMM_CALL(kZetaF16, true) : BIGCN_GEMM_CALL(kZetaF16, false);
        case kZetaI16: return dbg ? BIGCN_GEMM_CALL(kZetaI16, true) : BIGCN_GEMM_CALL(kZetaI16, false);
        case kZetaI8: return dbg ? BIGCN_GEMM_CALL(kZetaI8, true) : BIGCN_GEMM_CALL(kZetaI8, false);
        default: return cudaErrorInvalidValue;
    }
#undef BIGCN_GEMM_CALL
}

}  // namespace

bool bitgemm_takes_tc(int fmt, int path, int64_t n, int d_in, int d_out, int64_t stride_a, int64_t stride_b)
{
    if (!bitgemm_tc_covers(d_in, d_out, stride_a, stride_b)) return false;
    if (fmt == kZetaI8H) return true;
    return path != 1 && (path == 2 || n * (int64_t)d_out >= (int64_t(1) << 20));
}

cudaError_t launch_bitgemm(cudaStream_t s, const uint32_t* A, int64_t stride_a,
                           const uint32_t* BT, int64_t stride_b, int64_t n, int d_in, int d_out,
                           const float* beta, const float* alpha, int fmt, void* zeta, int64_t ldz,
                           int32_t* dbg_dot, float* dbg_zeta, int* launches, int path, float* nws, float* col_b0, int row_tail)
{
    if (n == 0) return cudaSuccess;
    if (fmt == kZetaI8H) {                                 // half-dot bytes exist on the tensor-core path only
        if (!bitgemm_tc_covers(d_in, d_out, stride_a, stride_b)) return cudaErrorInvalidValue;
        ++*launches;
        return launch_bitgemm_tc(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, fmt, zeta, ldz, dbg_dot, dbg_zeta, nws, col_b0, row_tail);
    }
    // the int8 tensor-core path: for covered shapes, by default from a million outputs on (below that the two
    // paths are level and the bit-count kernel has less fixed cost)
    const bool big = n * (int64_t)d_out >= (int64_t(1) << 20);
    if (path != 1 && (path == 2 || big) && bitgemm_tc_covers(d_in, d_out, stride_a, stride_b)) {
        ++*launches;
        return launch_bitgemm_tc(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, fmt, zeta, ldz, dbg_dot, dbg_zeta, nullptr, nullptr, row_tail);
    }
    const int kw = (d_in + 31) / 32;
    const int ldb = kw | 1;
    int tn = 8;
    while (tn > 1 && tn * 16 >= d_out) tn >>= 1;           // smallest power of two with tn*32 >= d_out (max 8)
    auto bytes = [&](int t) {
        // the A tile starts at a 16-byte boundary: the panel size is rounded up to 4 words
        return (size_t)(round_up((int64_t)t * 32 * ldb, 4) + (int64_t)kTileRows * stride_a) * 4;
    };
    while (tn > 1 && bytes(tn) > 200 * 1024) tn >>= 1;
    if (bytes(tn) > 200 * 1024) return cudaErrorInvalidConfiguration;
    ++*launches;
    // ldb is odd, so tn*32*ldb is a multiple of 32 words: As is already 16-byte aligned.
    switch (tn) {
        case 8: return launch_tn<8>(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, fmt, zeta, ldz, dbg_dot, dbg_zeta, bytes(8), ldb);
        case 4: return launch_tn<4>(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, fmt, zeta, ldz, dbg_dot, dbg_zeta, bytes(4), ldb);
        case 2: return launch_tn<2>(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, fmt, zeta, ldz, dbg_dot, dbg_zeta, bytes(2), ldb);
        default: return launch_tn<1>(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, fmt, zeta, ldz, dbg_dot, dbg_zeta, bytes(1), ldb);
    }
}

}  // namespace bigcn
