// The binary contraction on the 5th-generation tensor cores (Bi-GCN Sec. 4.2.3, Eq. "bi-op" / "cdot-op").
//
// dot_ij = F_i . B_j over +-1 vectors is a dense contraction.  The paper counts it in XNOR / bit-count
// operations because it targets hardware whose fastest exact path is the integer pipe; on this part
// the int8 tensor-core path is an order of magnitude faster than the bit-count pipe, so the packed
// bits are expanded to +1 / -1 bytes on the way into shared memory and the product runs as
// tcgen05.mma kind::i8 with int32 accumulators in tensor memory: the same integers, bit for bit.
// Padding bits are 0 in both operands and expand to (-1)(-1) = +1 each: the constant K_pad - d_in is
// subtracted in the epilogue.
//
// One CTA per SM walks over tiles of 128 rows.  The expanded weight panel (N x K bytes) stays in
// shared memory; feature tiles (128 x K bytes) and accumulators (N columns of tensor memory) are
// double-buffered, so the tensor cores work on tile i + 1 while the warps read tile i's accumulators
// back (tcgen05.ld), convert them to the storage format of zeta and write them out.  Operands sit in
// shared memory in the K-major no-swizzle canonical form: core matrices of 8 rows x 16 bytes.
// Every wait on an mbarrier is bounded; if one runs out the kernel raises a flag, frees its tensor
// memory and returns.
#include <algorithm>

#include <cuda_fp16.h>

#include "bigcn_internal.cuh"

namespace bigcn {

namespace {

constexpr int kTcThreads = 256;
constexpr int kTcRows = 128;                  // rows per tile = M of the instruction
constexpr int kTcWaitTries = 1 << 22;         // bound of every mbarrier wait

__device__ int g_tc_timeout;                  // set when a wait ran out

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// 4 bits -> 4 bytes of +1 (0x01) / -1 (0xFF): the multiplication spreads bit i to bit 8 i.
__device__ __forceinline__ uint32_t expand4(uint32_t nib)
{
    const uint32_t y = (nib * 0x00204081u) & 0x01010101u;
    return ~(y * 0xFEu);
}
__device__ __forceinline__ void expand_word(uint32_t w, uint4& lo, uint4& hi)
{
    lo = make_uint4(expand4(w & 15u), expand4((w >> 4) & 15u), expand4((w >> 8) & 15u), expand4((w >> 12) & 15u));
    hi = make_uint4(expand4((w >> 16) & 15u), expand4((w >> 20) & 15u), expand4((w >> 24) & 15u), expand4(w >> 28));
}

// Byte offset of (row r, 16-byte K chunk) in a K-major no-swizzle operand of `rows` rows: the core
// matrices (8 rows x 16 bytes = 128 contiguous bytes) of one K chunk follow each other over the row
// groups; K chunks are rows / 8 * 128 bytes apart.
__device__ __forceinline__ uint32_t canon_off(int rows, int r, int kchunk)
{
    return (uint32_t)((kchunk * (rows >> 3) + (r >> 3)) * 128 + (r & 7) * 16);
}

// Shared-memory matrix descriptor: start address, leading (K direction) and stride (row-group
// direction) byte offsets in 16-byte units, descriptor version 1, no swizzle.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    return d;
}

// Expands `rows_valid` packed rows (stride words each, read 16 bytes at a time) into the canonical
// operand of `rows` rows; rows past rows_valid become zero bytes.
__device__ __forceinline__ void stage_operand(unsigned char* dst, int rows, const uint32_t* __restrict__ src,
                                              int64_t stride, int64_t rows_valid)
{
    const int q = (int)(stride >> 2);                       // 16-byte pieces per packed row
    for (int t = threadIdx.x; t < rows * q; t += kTcThreads) {
        const int r = t / q, piece = t - r * q;
        uint4 w = make_uint4(0u, 0u, 0u, 0u);
        const bool in = r < rows_valid;
        if (in) w = __ldg(reinterpret_cast<const uint4*>(src + (int64_t)r * stride) + piece);
        const uint32_t ws[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo;
            if (in) expand_word(ws[i], lo, hi);
            *reinterpret_cast<uint4*>(dst + canon_off(rows, r, 2 * (4 * piece + i))) = lo;
            *reinterpret_cast<uint4*>(dst + canon_off(rows, r, 2 * (4 * piece + i) + 1)) = hi;
        }
    }
}

__device__ __forceinline__ bool wait_barrier(uint64_t* bar, uint32_t parity)
{
    uint32_t done = 0;
    for (int it = 0; it < kTcWaitTries && !done; ++it)
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
                     : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return done != 0;
}

// N: accumulator columns = N of the instruction (a multiple of 16, at most 256).
// kBuf: feature tiles and accumulators per CTA (2 = the CTA overlaps its own tiles, 1 = two CTAs per SM overlap each other).
template <int N, int FMT, int kBuf>
__global__ void __launch_bounds__(kTcThreads, kBuf == 1 ? 2 : 1)
bitgemm_tc_kernel(const uint32_t* __restrict__ A, int64_t stride_a, const uint32_t* __restrict__ BT, int64_t stride_b,
                  int64_t n, int d_in, int d_out, const float* __restrict__ beta, const float* __restrict__ alpha,
                  void* __restrict__ zeta, int64_t ldz, int32_t* __restrict__ dbg_dot, float* __restrict__ dbg_zeta)
{
    extern __shared__ __align__(128) unsigned char tc_smem[];
    __shared__ __align__(8) uint64_t bar[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ float al_s[N];
    constexpr int kCols = N <= 32 ? 32 : (N <= 64 ? 64 : (N <= 128 ? 128 : 256));   // tensor-memory columns per accumulator
    const int K = (int)stride_a * 32;                       // bytes per expanded row (padding included)
    const int pad = K - d_in;                               // padding positions: each contributes +1
    unsigned char* Bs = tc_smem;                            // [N][K]
    unsigned char* As0 = tc_smem + (size_t)N * K;           // two tiles of [128][K]
    const size_t a_bytes = (size_t)kTcRows * K;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_base_s)), "r"(kBuf * kCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(smem_u32(&bar[0])) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(smem_u32(&bar[1])) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    for (int j = threadIdx.x; j < N; j += kTcThreads) al_s[j] = j < d_out ? __ldg(alpha + j) : 0.f;
    stage_operand(Bs, N, BT, stride_b, d_out);

    const int64_t n_tiles = ceil_div(n, kTcRows);
    const int64_t my_tiles = blockIdx.x < n_tiles ? ceil_div(n_tiles - blockIdx.x, (int64_t)gridDim.x) : 0;
    auto tile_row0 = [&](int64_t i) { return (blockIdx.x + i * gridDim.x) * (int64_t)kTcRows; };
    if (kBuf == 2 && my_tiles > 0) stage_operand(As0, kTcRows, A + tile_row0(0) * stride_a, stride_a, n - tile_row0(0));
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;

    // instruction descriptor: D = s32, A = B = s8, both K-major, N, M = 128
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(kTcRows >> 4) << 24);
    const uint32_t a_lbo = (kTcRows >> 3) * 128, b_lbo = (N >> 3) * 128, sbo = 128;
    auto issue_tile = [&](int buf) {                        // one thread: all K steps of a tile, then the commit
        const uint32_t a_base = smem_u32(As0 + buf * a_bytes), b_base = smem_u32(Bs);
        for (int ks = 0; ks < K / 32; ++ks) {
            const uint64_t ad = make_desc(a_base + 2 * ks * a_lbo, a_lbo, sbo);
            const uint64_t bd = make_desc(b_base + 2 * ks * b_lbo, b_lbo, sbo);
            const uint32_t accum = ks > 0 ? 1u : 0u;
            asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}\n"
                         ::"r"(tmem_base + (uint32_t)(buf * kCols)), "l"(ad), "l"(bd), "r"(idesc), "r"(accum) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_u32(&bar[buf])) : "memory");
    };
    if (kBuf == 2 && my_tiles > 0 && threadIdx.x == 0) issue_tile(0);

    constexpr int kVec = FMT == kZetaF32 ? 4 : (FMT == kZetaI8 ? 16 : 8);     // elements per 16-byte store
    const int lane_base = 32 * (warp & 3);                  // a warp reads tensor-memory lanes 32 (warp % 4) .. + 31
    const int c_begin = (warp >> 2) * (N / 2), c_end = c_begin + N / 2;       // warps 0-3: lower half of the columns
    bool ok = true;
    for (int64_t i = 0; i < my_tiles; ++i) {
        const int buf = kBuf == 2 ? (int)(i & 1) : 0;
        if (kBuf == 2) {
            if (i + 1 < my_tiles)                           // next tile's features: its buffer was released by the wait of tile i - 1
                stage_operand(As0 + (buf ^ 1) * a_bytes, kTcRows, A + tile_row0(i + 1) * stride_a, stride_a, n - tile_row0(i + 1));
        } else {
            stage_operand(As0, kTcRows, A + tile_row0(i) * stride_a, stride_a, n - tile_row0(i));   // the wait of tile i - 1 released it
        }
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
        __syncthreads();                                    // staging done; everyone is past the reads of the accumulator to be overwritten
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        if (kBuf == 2) {
            if (i + 1 < my_tiles && threadIdx.x == 0) issue_tile(buf ^ 1);
        } else if (threadIdx.x == 0) {
            issue_tile(0);
        }
        if (!wait_barrier(&bar[buf], (uint32_t)((kBuf == 2 ? (i >> 1) : i) & 1))) {
            atomicExch(&g_tc_timeout, 1);
            ok = false;
        }
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        if (__syncthreads_or(!ok)) break;                   // leave together if any wait ran out
        // ---- epilogue of tile i: a thread owns one row and walks over its half of the columns
        const int64_t row = tile_row0(i) + lane_base + lane;
        const bool row_in = row < n;
        const float be = (row_in && (FMT == kZetaF32 || dbg_zeta)) ? __ldg(beta + row) : 0.f;
        for (int c0 = c_begin; c0 < c_end; c0 += 16) {
            uint32_t v[16];
            const uint32_t taddr = tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)(buf * kCols + c0);
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
                         : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                           "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                         : "r"(taddr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
            if (!row_in) continue;
            int dot[16];
#pragma unroll
            for (int q = 0; q < 16; ++q) dot[q] = (c0 + q < d_out) ? (int)v[q] - pad : 0;      // padding columns of zeta stay 0
            if constexpr (FMT == kZetaF16) {
                // exact integer -> fp16 without the conversion unit: the bit pattern 0x6600 + dot is the half 1536 + dot (|dot| <= 256 here)
                uint32_t h[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const __half2 biased = __halves2half2(__ushort_as_half((unsigned short)(0x6600 + dot[2 * q])), __ushort_as_half((unsigned short)(0x6600 + dot[2 * q + 1])));
                    const __half2 r = __hsub2(biased, __half2half2(__ushort_as_half((unsigned short)0x6600)));
                    h[q] = *reinterpret_cast<const uint32_t*>(&r);
                }
                __half* dst = reinterpret_cast<__half*>(zeta) + row * ldz + c0;
                if (c0 < ldz) *reinterpret_cast<uint4*>(dst) = make_uint4(h[0], h[1], h[2], h[3]);
                if (c0 + 8 < ldz) *reinterpret_cast<uint4*>(dst + 8) = make_uint4(h[4], h[5], h[6], h[7]);
            } else if constexpr (FMT == kZetaI16) {
                uint32_t h[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) h[q] = ((uint32_t)dot[2 * q] & 0xffffu) | ((uint32_t)dot[2 * q + 1] << 16);
                int16_t* dst = reinterpret_cast<int16_t*>(zeta) + row * ldz + c0;
                if (c0 < ldz) *reinterpret_cast<uint4*>(dst) = make_uint4(h[0], h[1], h[2], h[3]);
                if (c0 + 8 < ldz) *reinterpret_cast<uint4*>(dst + 8) = make_uint4(h[4], h[5], h[6], h[7]);
            } else if constexpr (FMT == kZetaI8) {
                uint32_t b[4];
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    b[q] = ((uint32_t)dot[4 * q] & 0xffu) | (((uint32_t)dot[4 * q + 1] & 0xffu) << 8) | (((uint32_t)dot[4 * q + 2] & 0xffu) << 16) | ((uint32_t)dot[4 * q + 3] << 24);
                int8_t* dst = reinterpret_cast<int8_t*>(zeta) + row * ldz + c0;
                if (c0 < ldz) *reinterpret_cast<uint4*>(dst) = make_uint4(b[0], b[1], b[2], b[3]);
            } else {
                float* dst = reinterpret_cast<float*>(zeta) + row * ldz + c0;
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    float f[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int c = c0 + 4 * q4 + q;
                        f[q] = c < d_out ? __fmul_rn(__fmul_rn(be, al_s[c]), (float)dot[4 * q4 + q]) : 0.f;
                    }
                    if (c0 + 4 * q4 < ldz) *reinterpret_cast<float4*>(dst + 4 * q4) = make_float4(f[0], f[1], f[2], f[3]);
                }
            }
            if (dbg_dot || dbg_zeta) {
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const int c = c0 + q;
                    if (c < d_out) {
                        if (dbg_dot) dbg_dot[row * (int64_t)d_out + c] = dot[q];
                        if (dbg_zeta) dbg_zeta[row * (int64_t)d_out + c] = __fmul_rn(__fmul_rn(be, al_s[c]), (float)dot[q]);
                    }
                }
            }
        }
        (void)kVec;
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(kBuf * kCols) : "memory");
}

template <int N, int FMT>
cudaError_t launch_tc_inst(cudaStream_t s, const uint32_t* A, int64_t stride_a, const uint32_t* BT, int64_t stride_b,
                           int64_t n, int d_in, int d_out, const float* beta, const float* alpha, void* zeta, int64_t ldz,
                           int32_t* dbg_dot, float* dbg_zeta)
{
    // two CTAs per SM, each with one feature tile and one accumulator (N <= 256 columns each: 512 in all)
    constexpr int kBuf = 1;
    const size_t smem = (size_t)(N + kBuf * kTcRows) * stride_a * 32;
    cudaError_t e = cudaFuncSetAttribute(bitgemm_tc_kernel<N, FMT, kBuf>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(n, kTcRows), 148 * (kBuf == 1 ? 2 : 1));
    bitgemm_tc_kernel<N, FMT, kBuf><<<grid, kTcThreads, smem, s>>>(A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta);
    return cudaGetLastError();
}

template <int N>
cudaError_t launch_tc_n(cudaStream_t s, int fmt, const uint32_t* A, int64_t stride_a, const uint32_t* BT, int64_t stride_b,
                        int64_t n, int d_in, int d_out, const float* beta, const float* alpha, void* zeta, int64_t ldz,
                        int32_t* dbg_dot, float* dbg_zeta)
{
    switch (fmt) {
        case kZetaF32: return launch_tc_inst<N, kZetaF32>(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta);
        case kZetaF16: return launch_tc_inst<N, kZetaF16>(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta);
        case kZetaI16: return launch_tc_inst<N, kZetaI16>(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta);
        case kZetaI8: return launch_tc_inst<N, kZetaI8>(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace

bool bitgemm_tc_covers(int d_in, int d_out, int64_t stride_a, int64_t stride_b)
{
    return d_in >= 1 && d_in <= 256 && d_out >= 1 && d_out <= 256 && stride_a == stride_b && stride_a * 32 <= 256;
}

cudaError_t launch_bitgemm_tc(cudaStream_t s, const uint32_t* A, int64_t stride_a, const uint32_t* BT, int64_t stride_b,
                              int64_t n, int d_in, int d_out, const float* beta, const float* alpha, int fmt, void* zeta,
                              int64_t ldz, int32_t* dbg_dot, float* dbg_zeta)
{
    // the instruction's N: the output channels rounded up to 64 / 128 / 256 (16 would do; fewer variants to build)
    if (d_out <= 64) return launch_tc_n<64>(s, fmt, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta);
    if (d_out <= 128) return launch_tc_n<128>(s, fmt, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta);
    return launch_tc_n<256>(s, fmt, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta);
}

// Number of waits that ran out since the library was loaded on the current device (0 = none).
int bitgemm_tc_timeouts()
{
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_tc_timeout, sizeof(int)) != cudaSuccess) return -1;
    return v;
}

}  // namespace bigcn
