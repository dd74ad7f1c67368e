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
// Persistent CTAs (two per SM) walk over tiles of 128 rows.  The expanded weight panel (N x K bytes)
// stays in shared memory; each tile's features are expanded into one 128 x K operand, multiplied into
// N columns of tensor memory, read back (tcgen05.ld), converted to the storage format of zeta and
// written out while the other CTA of the SM is in another phase.  Operands sit in shared memory in the
// K-major no-swizzle canonical form: core matrices of 8 rows x 16 bytes.  Every wait on an mbarrier is
// bounded; if one runs out the kernel raises a flag, frees its tensor memory and returns.
#include <algorithm>

#include <cuda_fp16.h>

#include "bigcn_internal.cuh"
#include "tc_common.cuh"

namespace bigcn {

namespace {

constexpr int kTcThreads = 256;
constexpr int kTcRows = 128;                  // rows per tile = M of the instruction

__device__ int g_tc_timeout;                  // set when a wait ran out

using tc::canon_off;
using tc::make_desc;
using tc::smem_u32;
using tc::wait_barrier;

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

// Converts 16 consecutive dots of one row to the storage format: kPieces 16-byte pieces.
template <int FMT>
struct TcOut;
template <> struct TcOut<kZetaF16> {
    static constexpr int kElt = 2;
    static __device__ __forceinline__ void pack(const int (&dot)[16], float, const float*, uint4 (&out)[2])
    {
        // exact integer -> fp16 without the conversion unit: the bit pattern 0x6600 + dot is the half 1536 + dot (|dot| <= 256 here)
        uint32_t h[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const __half2 biased = __halves2half2(__ushort_as_half((unsigned short)(0x6600 + dot[2 * q])), __ushort_as_half((unsigned short)(0x6600 + dot[2 * q + 1])));
            const __half2 r = __hsub2(biased, __half2half2(__ushort_as_half((unsigned short)0x6600)));
            h[q] = *reinterpret_cast<const uint32_t*>(&r);
        }
        out[0] = make_uint4(h[0], h[1], h[2], h[3]);
        out[1] = make_uint4(h[4], h[5], h[6], h[7]);
    }
};
template <> struct TcOut<kZetaI16> {
    static constexpr int kElt = 2;
    static __device__ __forceinline__ void pack(const int (&dot)[16], float, const float*, uint4 (&out)[2])
    {
        uint32_t h[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) h[q] = ((uint32_t)dot[2 * q] & 0xffffu) | ((uint32_t)dot[2 * q + 1] << 16);
        out[0] = make_uint4(h[0], h[1], h[2], h[3]);
        out[1] = make_uint4(h[4], h[5], h[6], h[7]);
    }
};
template <> struct TcOut<kZetaI8> {
    static constexpr int kElt = 1;
    static __device__ __forceinline__ void pack(const int (&dot)[16], float, const float*, uint4 (&out)[1])
    {
        uint32_t b[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {                       // the low bytes of four ints in one word: three byte permutes
            const uint32_t lo = __byte_perm((uint32_t)dot[4 * q], (uint32_t)dot[4 * q + 1], 0x0040);
            const uint32_t hi = __byte_perm((uint32_t)dot[4 * q + 2], (uint32_t)dot[4 * q + 3], 0x0040);
            b[q] = __byte_perm(lo, hi, 0x5410);
        }
        out[0] = make_uint4(b[0], b[1], b[2], b[3]);
    }
};
// half-dot bytes: the dots are replaced by s = (dot' - 1) / 2 before packing (see the epilogue), then stored as bytes
template <> struct TcOut<kZetaI8H> : TcOut<kZetaI8> {};
template <> struct TcOut<kZetaF32> {
    static constexpr int kElt = 4;
    // zeta_ij = (beta_i alpha_j) dot_ij in this order (Eq. "cdot-op"); al points at the chunk's first column
    static __device__ __forceinline__ void pack(const int (&dot)[16], float be, const float* al, uint4 (&out)[4])
    {
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            float f[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) f[q] = __fmul_rn(__fmul_rn(be, al[4 * q4 + q]), (float)dot[4 * q4 + q]);
            out[q4] = make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
        }
    }
};

// N: accumulator columns = N of the instruction (64, 128 or 256).  Two CTAs per SM, each with one
// feature tile and one accumulator; a CTA's steps per tile are: expand the tile's bits (fetched into
// registers during the previous tile) into shared memory, issue the products, fetch the next tile's
// bits, wait for the accumulators, convert them and write them out.  The write goes through shared
// memory (the feature tile's space, free once the products are done): a thread owns one row of the
// accumulators, and rows are far apart in zeta, so each warp first collects 32 rows x 128 bytes and
// then stores them as whole 128-byte row segments.
// kDebug: the debug taps (the integer dots and the literal fp32 zeta of every element) are wanted.
// Blocks per SM: two where the accumulator takes 256 of the 512 tensor-memory columns or the taps are on, three otherwise.
template <int N, int FMT, bool kDebug>
__global__ void __launch_bounds__(kTcThreads, (N > 128 || kDebug) ? 2 : 3)
bitgemm_tc_kernel(const uint32_t* __restrict__ A, int64_t stride_a, const uint32_t* __restrict__ BT, int64_t stride_b,
                  int64_t n, int d_in, int d_out, const float* __restrict__ beta, const float* __restrict__ alpha,
                  void* __restrict__ zeta, int64_t ldz, int32_t* __restrict__ dbg_dot, float* __restrict__ dbg_zeta,
                  float* __restrict__ nws, float* __restrict__ col_b0, int row_tail)
{
    // row_tail (byte formats, N = 64, d_out <= 60): a row of zeta is 64 bytes and its last four bytes hold the row's
    // node factor as a float (beta_i, with the first feature sign for half-dot bytes), so that the aggregation of a
    // last layer fetches an entry's dots and its factor with one pair of 32-byte loads
    using Out = TcOut<FMT>;
    constexpr int kElt = Out::kElt;                         // bytes per stored element = 16-byte pieces per chunk of 16 columns
    extern __shared__ __align__(128) unsigned char tc_smem[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ float al_s[N];
    __shared__ int b0_s[FMT == kZetaI8H ? N : 1];          // half-dot bytes: first sign of every weight column (0 when d_in is odd)
    __shared__ __align__(16) int hd_s[FMT == kZetaI8H ? 3 * N : 4];   // 1 + f b0_j for the row signs f = -1, 0, +1: what a half-dot subtracts
    constexpr int kCols = N <= 32 ? 32 : (N <= 64 ? 64 : (N <= 128 ? 128 : 256));   // tensor-memory columns of the accumulator
    const int K = (int)stride_a * 32;                       // bytes per expanded row (padding included)
    const int pad = K - d_in;                               // padding positions: each contributes +1
    unsigned char* Bs = tc_smem;                            // [N][K]
    unsigned char* As = tc_smem + (size_t)N * K;            // [128][K]; at least 32 KB: also the epilogue's scratch
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&tmem_base_s)), "r"(kCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"(smem_u32(&bar)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    for (int j = threadIdx.x; j < N; j += kTcThreads) al_s[j] = j < d_out ? __ldg(alpha + j) : 0.f;
    if constexpr (FMT == kZetaI8H) {
        const bool even = (d_in & 1) == 0;                  // even d_in: the first position is left out of the stored dot
        for (int j = threadIdx.x; j < N; j += kTcThreads) {
            const int b0 = (even && j < d_out) ? ((__ldg(BT + (int64_t)j * stride_b) & 1u) ? 1 : -1) : 0;
            b0_s[j] = b0;
            hd_s[j] = 1 - b0;
            hd_s[N + j] = 1;
            hd_s[2 * N + j] = 1 + b0;
            if (blockIdx.x == 0 && j < d_out) col_b0[j] = (float)b0;
        }
    }
    stage_operand(Bs, N, BT, stride_b, d_out);

    const int64_t n_tiles = ceil_div(n, kTcRows);
    const int64_t my_tiles = blockIdx.x < n_tiles ? ceil_div(n_tiles - blockIdx.x, (int64_t)gridDim.x) : 0;
    auto tile_row0 = [&](int64_t i) { return (blockIdx.x + i * gridDim.x) * (int64_t)kTcRows; };
    // a feature tile is 128 rows x (stride / 4) 16-byte pieces of packed bits: at most one piece per thread
    const int q = (int)(stride_a >> 2);
    const int my_r = threadIdx.x / q, my_piece = threadIdx.x - my_r * q;
    const bool my_item = threadIdx.x < kTcRows * q;
    auto fetch = [&](int64_t i) {
        uint4 w = make_uint4(0u, 0u, 0u, 0u);
        if (my_item && i < my_tiles && tile_row0(i) + my_r < n)
            w = __ldg(reinterpret_cast<const uint4*>(A + (tile_row0(i) + my_r) * stride_a) + my_piece);
        return w;
    };
    uint4 pre = fetch(0);
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;

    // instruction descriptor: D = s32, A = B = s8, both K-major, N, M = 128
    const uint32_t idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(kTcRows >> 4) << 24);
    const uint32_t a_lbo = (kTcRows >> 3) * 128, b_lbo = (N >> 3) * 128, sbo = 128;
    const int lane_base = 32 * (warp & 3);                  // a warp reads tensor-memory lanes 32 (warp % 4) .. + 31
    const int c_begin = (warp >> 2) * (N / 2);              // warps 0-3: lower half of the columns, 4-7: upper half
    constexpr int kRowBytes = (N / 2) * kElt;               // bytes of a row that one warp produces
    constexpr int kPpr = kRowBytes >= 128 ? 8 : kRowBytes / 16;     // 16-byte pieces per row and pass (128 bytes at most)
    constexpr int kChunksPerPass = kPpr / kElt > 0 ? kPpr / kElt : 1;
    static_assert(kPpr % kElt == 0 && kRowBytes % (16 * kPpr) == 0, "a pass is a whole number of 16-column chunks");
    constexpr int kPasses = kRowBytes / (16 * kPpr);
    unsigned char* scr = As + warp * 4096;                  // 32 rows x 128 bytes; piece p of row r at r * 128 + ((p ^ (r & 7)) * 16)
    bool ok = true;
    for (int64_t i = 0; i < my_tiles; ++i) {
        // ---- expand this tile's bits (in registers since the previous tile) into the operand
        if (my_item) {
            const bool in = tile_row0(i) + my_r < n;
            const uint32_t ws[4] = {pre.x, pre.y, pre.z, pre.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                uint4 lo = make_uint4(0u, 0u, 0u, 0u), hi = lo;
                if (in) expand_word(ws[u], lo, hi);
                *reinterpret_cast<uint4*>(As + canon_off(kTcRows, my_r, 2 * (4 * my_piece + u))) = lo;
                *reinterpret_cast<uint4*>(As + canon_off(kTcRows, my_r, 2 * (4 * my_piece + u) + 1)) = hi;
            }
        }
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
        __syncthreads();                                    // operand complete; everyone is past the previous tile's accumulator reads
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        if (threadIdx.x == 0) {                             // one thread: all K steps of the tile, then the commit
            const uint32_t a_base = smem_u32(As), b_base = smem_u32(Bs);
            for (int ks = 0; ks < K / 32; ++ks) {
                const uint64_t ad = make_desc(a_base + 2 * ks * a_lbo, a_lbo, sbo);
                const uint64_t bd = make_desc(b_base + 2 * ks * b_lbo, b_lbo, sbo);
                const uint32_t accum = ks > 0 ? 1u : 0u;
                asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}\n"
                             ::"r"(tmem_base), "l"(ad), "l"(bd), "r"(idesc), "r"(accum) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(smem_u32(&bar)) : "memory");
        }
        pre = fetch(i + 1);                                 // in flight while the products and the epilogue run
        if (!wait_barrier(&bar, (uint32_t)(i & 1))) {
            atomicExch(&g_tc_timeout, 1);
            ok = false;
        }
        asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory");
        if (__syncthreads_or(!ok)) break;                   // leave together if any wait ran out
        // ---- epilogue: a thread owns row lane_base + lane and walks over its warp's half of the columns
        const int64_t row0 = tile_row0(i) + lane_base;
        const int64_t row = row0 + lane;
        const bool row_in = row < n;
        const float be = (row_in && (FMT == kZetaF32 || FMT == kZetaI8H || (kDebug && dbg_zeta) || row_tail)) ? __ldg(beta + row) : 0.f;
        float row_fac = be;                                 // the node factor the aggregation multiplies the edge value by
        int f0 = 0;                                         // half-dot bytes: the row's first sign (0 when d_in is odd)
        if constexpr (FMT == kZetaI8H) {
            if (row_in) {
                const int sgn = (__ldg(A + row * stride_a) & 1u) ? 1 : -1;
                f0 = (d_in & 1) ? 0 : sgn;
                row_fac = (d_in & 1) ? be : be * (float)sgn;                     // beta_i carrying the first sign
                if (warp < 4) nws[row] = row_fac;
            }
        }
#pragma unroll 1
        for (int pass = 0; pass < kPasses; ++pass) {
#pragma unroll
            for (int ch = 0; ch < kChunksPerPass; ++ch) {
                const int c0 = c_begin + (pass * kChunksPerPass + ch) * 16;
                uint32_t v[16];
                const uint32_t taddr = tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)c0;
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n"
                             : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                               "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                             : "r"(taddr) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
                int dot[16];
                const bool whole = c0 + 16 <= d_out;        // every column of the chunk exists: no per-column tests
                if (whole) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) dot[e] = (int)v[e] - pad;
                } else {
#pragma unroll
                    for (int e = 0; e < 16; ++e) dot[e] = (c0 + e < d_out) ? (int)v[e] - pad : 0;   // padding columns of zeta stay 0
                }
                int full[kDebug ? 16 : 1];                  // the true dots, for the debug taps
                if constexpr (kDebug) {
#pragma unroll
                    for (int e = 0; e < 16; ++e) full[e] = dot[e];
                }
                if constexpr (FMT == kZetaI8H) {            // s = (dot - f0 b0_j - 1) / 2: odd by construction, exact
                    const int4* hd = reinterpret_cast<const int4*>(hd_s + (f0 + 1) * N + c0);
                    int sub[16];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int4 t = hd[q];
                        sub[4 * q] = t.x, sub[4 * q + 1] = t.y, sub[4 * q + 2] = t.z, sub[4 * q + 3] = t.w;
                    }
                    if (whole) {
#pragma unroll
                        for (int e = 0; e < 16; ++e) dot[e] = (dot[e] - sub[e]) >> 1;
                    } else {
#pragma unroll
                        for (int e = 0; e < 16; ++e)
                            if (c0 + e < d_out) dot[e] = (dot[e] - sub[e]) >> 1;
                    }
                }
                uint4 out[kElt];
                Out::pack(dot, be, al_s + c0, out);
                if constexpr (kElt == 1) {
                    if (row_tail && c0 == 48) out[0].w = __float_as_uint(row_fac);
                }
#pragma unroll
                for (int u = 0; u < kElt; ++u) {
                    const int piece = ch * kElt + u;
                    *reinterpret_cast<uint4*>(scr + lane * 128 + ((piece ^ (lane & 7)) * 16)) = out[u];
                }
                if constexpr (kDebug) {
                    if (row_in) {
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const int c = c0 + e;
                            if (c < d_out) {
                                if (dbg_dot) dbg_dot[row * (int64_t)d_out + c] = full[e];
                                if (dbg_zeta) dbg_zeta[row * (int64_t)d_out + c] = __fmul_rn(__fmul_rn(be, al_s[c]), (float)full[e]);
                            }
                        }
                    }
                }
            }
            __syncwarp();
            // write the 32 rows x kPpr pieces out: a warp instruction covers 32 / kPpr whole row segments
            const int64_t byte0 = (int64_t)(c_begin + pass * kChunksPerPass * 16) * kElt;       // first byte of the pass inside a row of zeta
#pragma unroll
            for (int it = 0; it < kPpr; ++it) {
                const int r = it * (32 / kPpr) + lane / kPpr, pc = lane % kPpr;
                const uint4 val = *reinterpret_cast<const uint4*>(scr + r * 128 + ((pc ^ (r & 7)) * 16));
                const int64_t at = byte0 + pc * 16;
                if (row0 + r < n && at < ldz * kElt)
                    *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(zeta) + (row0 + r) * ldz * kElt + at) = val;
            }
            __syncwarp();
        }
        asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
        __syncthreads();                                    // the scratch is the next tile's operand space
    }
    asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem_base), "r"(kCols) : "memory");
}

template <int N, int FMT>
cudaError_t launch_tc_inst(cudaStream_t s, const uint32_t* A, int64_t stride_a, const uint32_t* BT, int64_t stride_b,
                           int64_t n, int d_in, int d_out, const float* beta, const float* alpha, void* zeta, int64_t ldz,
                           int32_t* dbg_dot, float* dbg_zeta, float* nws, float* col_b0, int row_tail)
{
    // operands: weight panel N x K bytes, feature tile 128 x K bytes (at least the 32 KB the epilogue's scratch needs)
    size_t smem = (size_t)N * stride_a * 32 + std::max<size_t>((size_t)kTcRows * stride_a * 32, 32 * 1024);
    // a CTA holds 256 of the SM's 512 tensor-memory columns when N > 128: ask for enough shared memory that a third
    // CTA can never become resident on an SM and sit in tcgen05.alloc until a neighbour leaves
    if (N > 128) smem = std::max<size_t>(smem, 78 * 1024);
    const bool debug = dbg_dot || dbg_zeta;
    auto launch = [&](auto kernel, int blocks_per_sm) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        // persistent blocks: as many as stay resident (tensor-memory columns, registers, and shared memory: 227 KB per SM)
        const int fit = (int)std::max<size_t>(1, std::min<size_t>((size_t)blocks_per_sm, (size_t)(227 * 1024) / (smem + 2048)));
        const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(n, kTcRows), (int64_t)sm_count() * fit);
        kernel<<<grid, kTcThreads, smem, s>>>(A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta, nws, col_b0, row_tail);
        return cudaGetLastError();
    };
    if (debug) return launch(bitgemm_tc_kernel<N, FMT, true>, 2);
    return launch(bitgemm_tc_kernel<N, FMT, false>, N > 128 ? 2 : 3);
}

template <int N>
cudaError_t launch_tc_n(cudaStream_t s, int fmt, const uint32_t* A, int64_t stride_a, const uint32_t* BT, int64_t stride_b,
                        int64_t n, int d_in, int d_out, const float* beta, const float* alpha, void* zeta, int64_t ldz,
                        int32_t* dbg_dot, float* dbg_zeta, float* nws, float* col_b0, int row_tail)
{
#define BIGCN_TC_CALL(FMT) launch_tc_inst<N, FMT>(s, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta, nws, col_b0, (N == 64 && ldz == 64) ? row_tail : 0)
    switch (fmt) {
        case kZetaF32: return BIGCN_TC_CALL(kZetaF32);
        case kZetaF16: return BIGCN_TC_CALL(kZetaF16);
        case kZetaI16: return BIGCN_TC_CALL(kZetaI16);
        case kZetaI8: return BIGCN_TC_CALL(kZetaI8);
        case kZetaI8H: return (nws && col_b0 && d_in <= 256) ? BIGCN_TC_CALL(kZetaI8H) : cudaErrorInvalidValue;
        default: return cudaErrorInvalidValue;
    }
#undef BIGCN_TC_CALL
}

}  // namespace

bool bitgemm_tc_covers(int d_in, int d_out, int64_t stride_a, int64_t stride_b)
{
    return d_in >= 1 && d_in <= 256 && d_out >= 1 && d_out <= 256 && stride_a == stride_b && stride_a * 32 <= 256;
}

cudaError_t launch_bitgemm_tc(cudaStream_t s, const uint32_t* A, int64_t stride_a, const uint32_t* BT, int64_t stride_b,
                              int64_t n, int d_in, int d_out, const float* beta, const float* alpha, int fmt, void* zeta,
                              int64_t ldz, int32_t* dbg_dot, float* dbg_zeta, float* nws, float* col_b0, int row_tail)
{
    // the instruction's N: the output channels rounded up to 64 / 128 / 256 (16 would do; fewer variants to build)
    if (d_out <= 64) return launch_tc_n<64>(s, fmt, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta, nws, col_b0, row_tail);
    if (d_out <= 128) return launch_tc_n<128>(s, fmt, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta, nws, col_b0, 0);
    return launch_tc_n<256>(s, fmt, A, stride_a, BT, stride_b, n, d_in, d_out, beta, alpha, zeta, ldz, dbg_dot, dbg_zeta, nws, col_b0, 0);
}

// Number of waits that ran out since the library was loaded on the current device (0 = none).
int bitgemm_tc_timeouts()
{
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_tc_timeout, sizeof(int)) != cudaSuccess) return -1;
    return v;
}

}  // namespace bigcn
