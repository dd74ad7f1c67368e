// Back-propagation through one binarized graph convolutional layer (Bi-GCN Algorithm 1, Sec. 4.3):
//   G_zeta = A_tilde^T G'            (the aggregation kernel of the forward pass, fp32 rows)
//   G_W~   = H~^T G_zeta             H~_ik = beta_i F_ik from the packed input bits
//   G_H~   = G_zeta W~^T             W~_kj = alpha_j sign(W_kj)
//   G_H    = G_H~ [|G_H~| < 1]       (Eq. bp-H)
//   G_W_ij = (1/d_in) B_ij sum_k G_W~_kj B_kj + alpha_j G_W~_ij [|W_ij| < 1]   (Eq. bp-W)
// The two dense products have one +-1 operand that is expanded from bits (or from the sign of W) into
// shared memory tile by tile as bf16; the fp32 operand is split into three bf16 terms; the products run
// on the tensor cores with fp32 accumulation.
#include <algorithm>

#include <cuda_bf16.h>

#include "bigcn_internal.cuh"
#include "tc_common.cuh"

namespace bigcn {

namespace {

constexpr int kBwThreads = 256;       // 8 warps per block

// Copies rows of d floats into rows of ld_out floats (ld_out >= d, a multiple of 4), zero-filling the tail.
__global__ void pad_rows_kernel(const float* __restrict__ src, int64_t n, int d, int64_t ld_in,
                                float* __restrict__ dst, int64_t ld_out)
{
    const int64_t total = n * ld_out;
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = t / ld_out;
        const int j = (int)(t - i * ld_out);
        dst[t] = j < d ? __ldg(src + i * ld_in + j) : 0.f;
    }
}

// G_W~ = sum of the slabs, in slab order (double accumulation: the slabs can differ by orders of magnitude).
__global__ void grad_wt_reduce_kernel(const float* __restrict__ part, int n_splits, int64_t elems, float* __restrict__ g_wt)
{
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (t >= elems) return;
    double s = 0.0;
    for (int z = 0; z < n_splits; ++z) s += (double)part[(int64_t)z * elems + t];
    g_wt[t] = (float)s;
}

// ---- the two dense products, on the tensor cores ------------------------------------------------------
// Both products have one operand that is exactly +-1 (exact in bf16) and one fp32 operand.  The fp32
// operand x is split into three bf16 terms x = hi + mid + lo (each the rounding of what is left:
// 3 x 8 significant bits cover fp32's 24), so three bf16 tensor-core products with fp32 accumulation
// reproduce the fp32 product to fp32 accuracy.  mma.sync m16n8k16 (row-major A, column-major B):
// with g = lane / 4, t = lane % 4 a thread holds A[g | g+8][2t, 2t+1 | +8], B[2t, 2t+1 | +8][g],
// C[g | g+8][2t, 2t+1].  Tiles are staged in shared memory as bf16 with a row pitch of 40 elements
// (20 words), which makes the fragment reads of a warp hit 32 different banks.
constexpr int kMmaPitch = 40;                    // bf16 elements per staged row (32 + 8 pad)
constexpr int kMmaTile = 128;                    // output tile 128 x 128 per block, 8 warps of 32 x 64
constexpr int kMmaK = 32;                        // reduction elements per staged step

__device__ __forceinline__ void split3(float x, unsigned short& hi, unsigned short& mid, unsigned short& lo)
{
    const __nv_bfloat16 h = __float2bfloat16_rn(x);
    const float r1 = __fsub_rn(x, __bfloat162float(h));
    const __nv_bfloat16 m = __float2bfloat16_rn(r1);
    const float r2 = __fsub_rn(r1, __bfloat162float(m));
    const __nv_bfloat16 l = __float2bfloat16_rn(r2);
    hi = __bfloat16_as_ushort(h);
    mid = __bfloat16_as_ushort(m);
    lo = __bfloat16_as_ushort(l);
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2])
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// One staged step of the block's 128 x 128 tile: As[3][128][pitch] (the three terms of the fp32
// operand, rows = output rows, k contiguous), Bs[128][pitch] (the +-1 operand, rows = output columns,
// k contiguous).  Warp (wr, wc) owns rows 32 wr.., columns 64 wc...
__device__ __forceinline__ void mma_step(const unsigned short* As, const unsigned short* Bs, int wr, int wc, int lane,
                                         float (&acc)[2][8][4])
{
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int kk = 0; kk < kMmaK; kk += 16) {
        uint32_t b[8][2];
#pragma unroll
        for (int nb = 0; nb < 8; ++nb) {
            const unsigned short* p = Bs + (wc * 64 + nb * 8 + g) * kMmaPitch + kk + 2 * t;
            b[nb][0] = *reinterpret_cast<const uint32_t*>(p);
            b[nb][1] = *reinterpret_cast<const uint32_t*>(p + 8);
        }
#pragma unroll
        for (int sp = 0; sp < 3; ++sp) {
#pragma unroll
            for (int mb = 0; mb < 2; ++mb) {
                const unsigned short* p = As + (sp * kMmaTile + wr * 32 + mb * 16 + g) * kMmaPitch + kk + 2 * t;
                uint32_t a[4];
                a[0] = *reinterpret_cast<const uint32_t*>(p);
                a[1] = *reinterpret_cast<const uint32_t*>(p + 8 * kMmaPitch);
                a[2] = *reinterpret_cast<const uint32_t*>(p + 8);
                a[3] = *reinterpret_cast<const uint32_t*>(p + 8 * kMmaPitch + 8);
#pragma unroll
                for (int nb = 0; nb < 8; ++nb) mma_bf16(acc[mb][nb], a, b[nb]);
            }
        }
    }
}

// G_H = clip(G_zeta W~^T) on the tensor cores.  Block (x, y): rows [128 x, +128) x inputs k in
// [128 y, +128); the reduction runs over the output channels j in steps of 32.  A = G_zeta * alpha_j
// (split in three), B[k][j] = sign(W[k][j]).
__global__ void __launch_bounds__(kBwThreads)
grad_h_mma_kernel(const float* __restrict__ gz, int64_t ldz, const float* __restrict__ alpha,
                  const float* __restrict__ W, int64_t ldw, int64_t n, int d_in, int d_out,
                  float* __restrict__ g_h, int64_t ldh)
{
    __shared__ __align__(16) unsigned short As[3 * kMmaTile * kMmaPitch];
    __shared__ __align__(16) unsigned short Bs[kMmaTile * kMmaPitch];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int wr = warp >> 1, wc = warp & 1;
    const int64_t i0 = (int64_t)blockIdx.x * kMmaTile;
    const int k0 = blockIdx.y * kMmaTile;
    const bool vec_ok = (ldz % 4 == 0) && (reinterpret_cast<uintptr_t>(gz) % 16 == 0);
    float acc[2][8][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[a][b][c] = 0.f;
    for (int j0 = 0; j0 < d_out; j0 += kMmaK) {
        __syncthreads();                                   // the previous step's tiles are consumed
        // stage 128 x 32 of each operand: a thread takes 4 consecutive j of one row (16-byte loads where the
        // row allows it) and writes 8 bytes per term
        for (int t = threadIdx.x; t < kMmaTile * (kMmaK / 4); t += kBwThreads) {
            const int jq = (t & 7) * 4, rr = t >> 3;
            const int j = j0 + jq;
            const int64_t row = i0 + rr;
            float x[4] = {0.f, 0.f, 0.f, 0.f};
            if (row < n) {
                if (j + 3 < d_out && vec_ok) {
                    const float4 v = __ldg(reinterpret_cast<const float4*>(gz + row * ldz + j));
                    x[0] = v.x, x[1] = v.y, x[2] = v.z, x[3] = v.w;
                } else {
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        if (j + q < d_out) x[q] = __ldg(gz + row * ldz + j + q);
                }
            }
            unsigned short hi[4], mid[4], lo[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) split3(j + q < d_out ? __fmul_rn(x[q], __ldg(alpha + j + q)) : 0.f, hi[q], mid[q], lo[q]);
            auto pack = [](const unsigned short (&h)[4]) { return make_uint2((uint32_t)h[0] | ((uint32_t)h[1] << 16), (uint32_t)h[2] | ((uint32_t)h[3] << 16)); };
            *reinterpret_cast<uint2*>(&As[(0 * kMmaTile + rr) * kMmaPitch + jq]) = pack(hi);
            *reinterpret_cast<uint2*>(&As[(1 * kMmaTile + rr) * kMmaPitch + jq]) = pack(mid);
            *reinterpret_cast<uint2*>(&As[(2 * kMmaTile + rr) * kMmaPitch + jq]) = pack(lo);
            const int k = k0 + rr;
            unsigned short sg[4] = {0, 0, 0, 0};
            if (k < d_in) {
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (j + q < d_out) sg[q] = __ldg(W + (int64_t)k * ldw + j + q) >= 0.f ? 0x3F80 : 0xBF80;
            }
            *reinterpret_cast<uint2*>(&Bs[rr * kMmaPitch + jq]) = pack(sg);
        }
        __syncthreads();
        mma_step(As, Bs, wr, wc, lane, acc);
    }
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int mb = 0; mb < 2; ++mb)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int64_t row = i0 + wr * 32 + mb * 16 + g + 8 * half;
            if (row >= n) continue;
#pragma unroll
            for (int nb = 0; nb < 8; ++nb)
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int k = k0 + wc * 64 + nb * 8 + 2 * t + q;
                    const float v = acc[mb][nb][2 * half + q];
                    if (k < d_in) g_h[row * ldh + k] = fabsf(v) < 1.f ? v : 0.f;            // Eq. bp-H
                }
        }
}

// G_W~ partial sums on the tensor cores.  The product is taken transposed, C^T[j][k] = sum over nodes
// of (beta_i G_zeta[i][j]) * F[i][k], so that the fp32 operand is again the row operand: A[j][node]
// (split in three), B[node][k] = +-1 from the packed bits.  Both operands are stored node-major in
// global memory and the reduction runs over the nodes, so the staging transposes them: a thread takes
// two consecutive nodes and writes them as one 32-bit pair.  Block (x, y, z): channels j in
// [128 x, +128), inputs k in [128 y, +128), nodes [z * rows_per_split, +rows_per_split); slab z of
// `part` receives the tile as [k][j].
__global__ void __launch_bounds__(kBwThreads)
grad_wt_mma_kernel(const uint32_t* __restrict__ bits, int64_t stride, const float* __restrict__ beta,
                   const float* __restrict__ gz, int64_t ldz, int64_t n, int d_in, int d_out,
                   int64_t rows_per_split, float* __restrict__ part)
{
    __shared__ __align__(16) unsigned short As[3 * kMmaTile * kMmaPitch];   // [term][j][node]
    __shared__ __align__(16) unsigned short Bs[kMmaTile * kMmaPitch];       // [k][node]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int wr = warp >> 1, wc = warp & 1;
    const int j0 = blockIdx.x * kMmaTile, k0 = blockIdx.y * kMmaTile;
    const int64_t r_begin = (int64_t)blockIdx.z * rows_per_split;
    const int64_t r_end = min(n, r_begin + rows_per_split);
    const bool vec_ok = (ldz % 4 == 0) && (reinterpret_cast<uintptr_t>(gz) % 16 == 0);
    float acc[2][8][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[a][b][c] = 0.f;
    for (int64_t r0 = r_begin; r0 < r_end; r0 += kMmaK) {
        __syncthreads();                                   // the previous step's tiles are consumed
        // A: 16 node pairs x 32 quads of channels
        for (int t = threadIdx.x; t < 16 * 32; t += kBwThreads) {
            const int np = t & 15, jq = (t >> 4) * 4;
            float x[2][4];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int64_t row = r0 + 2 * np + h;
                const int j = j0 + jq;
#pragma unroll
                for (int q = 0; q < 4; ++q) x[h][q] = 0.f;
                if (row < r_end) {
                    const float be = __ldg(beta + row);
                    if (j + 3 < d_out && vec_ok) {
                        const float4 v = __ldg(reinterpret_cast<const float4*>(gz + row * ldz + j));
                        x[h][0] = v.x * be, x[h][1] = v.y * be, x[h][2] = v.z * be, x[h][3] = v.w * be;
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            if (j + q < d_out) x[h][q] = __ldg(gz + row * ldz + j + q) * be;
                    }
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                unsigned short h0, m0, l0, h1, m1, l1;
                split3(x[0][q], h0, m0, l0);
                split3(x[1][q], h1, m1, l1);
                const int at = (jq + q) * kMmaPitch + 2 * np;
                *reinterpret_cast<uint32_t*>(&As[0 * kMmaTile * kMmaPitch + at]) = (uint32_t)h0 | ((uint32_t)h1 << 16);
                *reinterpret_cast<uint32_t*>(&As[1 * kMmaTile * kMmaPitch + at]) = (uint32_t)m0 | ((uint32_t)m1 << 16);
                *reinterpret_cast<uint32_t*>(&As[2 * kMmaTile * kMmaPitch + at]) = (uint32_t)l0 | ((uint32_t)l1 << 16);
            }
        }
        // B: 16 node pairs x 4 words of 32 inputs, each word in two halves of 16
        for (int t = threadIdx.x; t < 16 * 8; t += kBwThreads) {
            const int np = t & 15, wd = (t >> 4) >> 1, half = (t >> 4) & 1;
            const int kw = k0 + wd * 32;                   // first input of the word
            uint32_t w0 = 0u, w1 = 0u;
            const int64_t row = r0 + 2 * np;
            if (kw < d_in) {
                if (row < r_end) w0 = __ldg(bits + row * stride + (kw >> 5));
                if (row + 1 < r_end) w1 = __ldg(bits + (row + 1) * stride + (kw >> 5));
            }
            const bool in0 = row < r_end, in1 = row + 1 < r_end;
#pragma unroll
            for (int b = 0; b < 16; ++b) {
                const int kb = half * 16 + b;
                const bool kin = kw + kb < d_in;
                const uint32_t lo = (kin && in0) ? (((w0 >> kb) & 1u) ? 0x3F80u : 0xBF80u) : 0u;
                const uint32_t hi = (kin && in1) ? (((w1 >> kb) & 1u) ? 0x3F80u : 0xBF80u) : 0u;
                *reinterpret_cast<uint32_t*>(&Bs[(wd * 32 + kb) * kMmaPitch + 2 * np]) = lo | (hi << 16);
            }
        }
        __syncthreads();
        mma_step(As, Bs, wr, wc, lane, acc);
    }
    float* slab = part + (int64_t)blockIdx.z * d_in * d_out;
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int mb = 0; mb < 2; ++mb)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int j = j0 + wr * 32 + mb * 16 + g + 8 * half;
            if (j >= d_out) continue;
#pragma unroll
            for (int nb = 0; nb < 8; ++nb)
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int k = k0 + wc * 64 + nb * 8 + 2 * t + q;
                    if (k < d_in) slab[(int64_t)k * d_out + j] = acc[mb][nb][2 * half + q];
                }
        }
}

// ---- G_H on the 5th-generation tensor cores ---------------------------------------------------------------
// The same product as grad_h_mma_kernel with tcgen05.mma kind::f16 (bf16 operands, fp32 accumulators in
// tensor memory): M = 128 rows, N = 64 / 128 / 256 >= d_in, the reduction over the output channels in
// chunks of 64 (128 bytes per operand row: the three terms of the fp32 operand take 48 KB, the +-1
// operand N x 128 bytes).  Two CTAs per SM overlap each other's staging, products and epilogue.  Operands
// are K-major no-swizzle (core matrices of 8 rows x 16 bytes).  The epilogue reads the accumulators back
// (a thread owns one row), clips (Eq. bp-H) and writes through shared memory as 128-byte row segments.
// Needs d_in a multiple of 4 and 16-byte aligned rows of g_h; every mbarrier wait is bounded.
__device__ int g_bw_tc_timeout;

template <int N>
__global__ void __launch_bounds__(kBwThreads, 2)
grad_h_tc_kernel(const float* __restrict__ gz, int64_t ldz, const float* __restrict__ alpha,
                 const float* __restrict__ W, int64_t ldw, int64_t n, int d_in, int d_out,
                 float* __restrict__ g_h, int64_t ldh)
{
    constexpr int kRows = 128, kKc = 64;                   // tile rows; reduction elements per chunk
    constexpr int kCols = N <= 64 ? 64 : (N <= 128 ? 128 : 256);
    extern __shared__ __align__(128) unsigned char bw_smem[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t tmem_base_s;
    unsigned char* As = bw_smem;                            // [3][128][128 bytes]; also the epilogue's scratch (>= 32 KB)
    unsigned char* Bs = bw_smem + 3 * kRows * 128;          // [N][128 bytes]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) tc::tmem_alloc(&tmem_base_s, kCols);
    if (threadIdx.x == 0) tc::barrier_init(&bar);
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem_base = tmem_base_s;
    // instruction descriptor: D = f32, A = B = bf16, both K-major, N, M = 128
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(kRows >> 4) << 24);
    const uint32_t a_lbo = (kRows >> 3) * 128, b_lbo = (N >> 3) * 128, sbo = 128;
    const bool vec_ok = (ldz % 4 == 0) && (reinterpret_cast<uintptr_t>(gz) % 16 == 0);
    const bool w_vec_ok = (ldw % 4 == 0) && (reinterpret_cast<uintptr_t>(W) % 16 == 0);
    const int n_chunks = (d_out + kKc - 1) / kKc;
    const int64_t n_tiles = ceil_div(n, kRows);
    const int lane_base = 32 * (warp & 3);
    const int c_begin = (warp >> 2) * (N / 2);
    unsigned char* scr = As + warp * 4096;                  // 32 rows x 128 bytes, pieces swizzled by (row & 7)
    uint32_t phase = 0;
    bool ok = true;
    for (int64_t tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int64_t i0 = tile * kRows;
        for (int ch = 0; ch < n_chunks; ++ch) {
            const int j0 = ch * kKc;
            // A: 128 rows x 16 quads of channels -> three bf16 terms of G_zeta * alpha.  All of a thread's loads are
            // issued before the first is used (8 independent 16-byte loads in flight per thread).
            {
                constexpr int kItems = kRows * (kKc / 4) / kBwThreads;
                float4 xv[kItems], av[kItems];
#pragma unroll
                for (int it = 0; it < kItems; ++it) {
                    const int t = threadIdx.x + it * kBwThreads;
                    const int jq = (t & 15) * 4, r = t >> 4;
                    const int j = j0 + jq;
                    const int64_t row = i0 + r;
                    xv[it] = make_float4(0.f, 0.f, 0.f, 0.f);
                    av[it] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (row < n) {
                        if (j + 3 < d_out && vec_ok) {
                            xv[it] = __ldg(reinterpret_cast<const float4*>(gz + row * ldz + j));
                        } else {
                            if (j < d_out) xv[it].x = __ldg(gz + row * ldz + j);
                            if (j + 1 < d_out) xv[it].y = __ldg(gz + row * ldz + j + 1);
                            if (j + 2 < d_out) xv[it].z = __ldg(gz + row * ldz + j + 2);
                            if (j + 3 < d_out) xv[it].w = __ldg(gz + row * ldz + j + 3);
                        }
                    }
                    if (j < d_out) av[it].x = __ldg(alpha + j);
                    if (j + 1 < d_out) av[it].y = __ldg(alpha + j + 1);
                    if (j + 2 < d_out) av[it].z = __ldg(alpha + j + 2);
                    if (j + 3 < d_out) av[it].w = __ldg(alpha + j + 3);
                }
#pragma unroll
                for (int it = 0; it < kItems; ++it) {
                    const int t = threadIdx.x + it * kBwThreads;
                    const int jq = (t & 15) * 4, r = t >> 4;
                    const float x[4] = {__fmul_rn(xv[it].x, av[it].x), __fmul_rn(xv[it].y, av[it].y), __fmul_rn(xv[it].z, av[it].z), __fmul_rn(xv[it].w, av[it].w)};
                    unsigned short hi[4], mid[4], lo[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) split3(x[u], hi[u], mid[u], lo[u]);
                    auto pack = [](const unsigned short (&h)[4]) { return make_uint2((uint32_t)h[0] | ((uint32_t)h[1] << 16), (uint32_t)h[2] | ((uint32_t)h[3] << 16)); };
                    const uint32_t off = tc::canon_off(kRows, r, jq >> 3) + (jq & 7) * 2;
                    *reinterpret_cast<uint2*>(As + 0 * kRows * 128 + off) = pack(hi);
                    *reinterpret_cast<uint2*>(As + 1 * kRows * 128 + off) = pack(mid);
                    *reinterpret_cast<uint2*>(As + 2 * kRows * 128 + off) = pack(lo);
                }
            }
            // B: N inputs x 16 quads of channels -> sign of W as +-1 (loads batched in the same way)
            {
                constexpr int kItems = N * (kKc / 4) / kBwThreads;
                float4 wv[kItems];
#pragma unroll
                for (int it = 0; it < kItems; ++it) {
                    const int t = threadIdx.x + it * kBwThreads;
                    const int jq = (t & 15) * 4, k = t >> 4;
                    const int j = j0 + jq;
                    wv[it] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (k < d_in) {
                        if (j + 3 < d_out && w_vec_ok) {
                            wv[it] = __ldg(reinterpret_cast<const float4*>(W + (int64_t)k * ldw + j));
                        } else {
                            if (j < d_out) wv[it].x = __ldg(W + (int64_t)k * ldw + j);
                            if (j + 1 < d_out) wv[it].y = __ldg(W + (int64_t)k * ldw + j + 1);
                            if (j + 2 < d_out) wv[it].z = __ldg(W + (int64_t)k * ldw + j + 2);
                            if (j + 3 < d_out) wv[it].w = __ldg(W + (int64_t)k * ldw + j + 3);
                        }
                    }
                }
#pragma unroll
                for (int it = 0; it < kItems; ++it) {
                    const int t = threadIdx.x + it * kBwThreads;
                    const int jq = (t & 15) * 4, k = t >> 4;
                    const int j = j0 + jq;
                    const bool kin = k < d_in;
                    const float w[4] = {wv[it].x, wv[it].y, wv[it].z, wv[it].w};
                    uint32_t sg[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) sg[u] = (kin && j + u < d_out) ? (w[u] >= 0.f ? 0x3F80u : 0xBF80u) : 0u;
                    const uint32_t off = tc::canon_off(N, k, jq >> 3) + (jq & 7) * 2;
                    *reinterpret_cast<uint2*>(Bs + off) = make_uint2(sg[0] | (sg[1] << 16), sg[2] | (sg[3] << 16));
                }
            }
            tc::fence_async_smem();
            tc::fence_before_sync();
            __syncthreads();                                // operands complete; previous tile's accumulator reads are over
            tc::fence_after_sync();
            if (threadIdx.x == 0) {
                const uint32_t a_base = tc::smem_u32(As), b_base = tc::smem_u32(Bs);
                for (int ks = 0; ks < kKc / 16; ++ks) {
                    const uint64_t bd = tc::make_desc(b_base + 2 * ks * b_lbo, b_lbo, sbo);
#pragma unroll
                    for (int sp = 0; sp < 3; ++sp) {
                        const uint64_t ad = tc::make_desc(a_base + sp * kRows * 128 + 2 * ks * a_lbo, a_lbo, sbo);
                        const uint32_t accum = (ch > 0 || ks > 0 || sp > 0) ? 1u : 0u;
                        asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                                     ::"r"(tmem_base), "l"(ad), "l"(bd), "r"(idesc), "r"(accum) : "memory");
                    }
                }
                tc::commit_to(&bar);
            }
            if (!tc::wait_barrier(&bar, phase)) {
                atomicExch(&g_bw_tc_timeout, 1);
                ok = false;
            }
            phase ^= 1u;
            tc::fence_after_sync();
            if (__syncthreads_or(!ok)) { ok = false; break; }   // the operands may be overwritten; leave together on a timeout
        }
        if (!ok) break;
        // ---- epilogue: clip and write the tile (a thread owns row lane_base + lane, its warp's half of the columns)
        const int64_t row0 = i0 + lane_base;
        constexpr int kPasses = (N / 2) * 4 / 128 > 0 ? (N / 2) * 4 / 128 : 1;    // 32 columns = 128 bytes per pass
        constexpr int kPpr = (N / 2) * 4 >= 128 ? 8 : (N / 2) * 4 / 16;
#pragma unroll 1
        for (int pass = 0; pass < kPasses; ++pass) {
#pragma unroll
            for (int c2 = 0; c2 < kPpr / 4; ++c2) {
                const int c0 = c_begin + pass * 32 + c2 * 16;
                uint32_t v[16];
                tc::tmem_ld16(tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)c0, v);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float f[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float a = __uint_as_float(v[4 * u + e]);
                        f[e] = fabsf(a) < 1.f ? a : 0.f;                                  // Eq. bp-H
                    }
                    const int piece = c2 * 4 + u;
                    *reinterpret_cast<uint4*>(scr + lane * 128 + ((piece ^ (lane & 7)) * 16)) =
                        make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
                }
            }
            __syncwarp();
            const int col0 = c_begin + pass * 32;
#pragma unroll
            for (int it = 0; it < kPpr; ++it) {
                const int r = it * (32 / kPpr) + lane / kPpr, pc = lane % kPpr;
                const uint4 val = *reinterpret_cast<const uint4*>(scr + r * 128 + ((pc ^ (r & 7)) * 16));
                const int col = col0 + pc * 4;
                if (row0 + r < n && col < d_in) *reinterpret_cast<uint4*>(g_h + (row0 + r) * ldh + col) = val;
            }
            __syncwarp();
        }
        tc::fence_before_sync();
        __syncthreads();                                    // the scratch is the next tile's operand space
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_free(tmem_base, kCols);
}

// ---- G_W~ partial sums on the 5th-generation tensor cores -------------------------------------------------
// The product of grad_wt_mma_kernel (transposed: C^T[j][k] = sum over nodes of (beta_i G_zeta[i][j]) F[i][k])
// with tcgen05.mma kind::f16: M = 128 channels j, N = 64 / 128 / 256 >= d_in inputs k, the reduction over
// the CTA's nodes in chunks of 64, all of them accumulated in one fp32 tile of tensor memory that is read
// back once at the end and written as slab blockIdx.y of `part` ([k][j]: consecutive lanes write consecutive
// j).  Both operands are node-major in global memory; the staging transposes them, two nodes per 32-bit store.
template <int N>
__global__ void __launch_bounds__(kBwThreads, 2)
grad_wt_tc_kernel(const uint32_t* __restrict__ bits, int64_t stride, const float* __restrict__ beta,
                  const float* __restrict__ gz, int64_t ldz, int64_t n, int d_in, int d_out,
                  int64_t rows_per_split, float* __restrict__ part)
{
    constexpr int kRows = 128, kKc = 64;                   // channels per tile; nodes per chunk
    constexpr int kCols = N <= 64 ? 64 : (N <= 128 ? 128 : 256);
    extern __shared__ __align__(128) unsigned char bw_smem[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t tmem_base_s;
    unsigned char* As = bw_smem;                            // [3][128 channels][64 nodes] bf16
    unsigned char* Bs = bw_smem + 3 * kRows * 128;          // [N inputs][64 nodes] bf16
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0) tc::tmem_alloc(&tmem_base_s, kCols);
    if (threadIdx.x == 0) tc::barrier_init(&bar);
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem_base = tmem_base_s;
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(kRows >> 4) << 24);
    const uint32_t a_lbo = (kRows >> 3) * 128, b_lbo = (N >> 3) * 128, sbo = 128;
    const bool vec_ok = (ldz % 4 == 0) && (reinterpret_cast<uintptr_t>(gz) % 16 == 0);
    const int j0 = blockIdx.x * kRows;
    const int64_t r_begin = (int64_t)blockIdx.y * rows_per_split;
    const int64_t r_end = min(n, r_begin + rows_per_split);
    uint32_t phase = 0;
    bool ok = true, any = false;
    for (int64_t r0 = r_begin; r0 < r_end; r0 += kKc) {
        // A: 32 node pairs x 32 quads of channels; all of a thread's loads are issued before the first is used
        {
            constexpr int kItems = 32 * 32 / kBwThreads;
            float4 xv[kItems][2];
            float bv[kItems][2];
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
                const int t = threadIdx.x + it * kBwThreads;
                const int np = t & 31, jq = (t >> 5) * 4;
                const int j = j0 + jq;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int64_t row = r0 + 2 * np + h;
                    xv[it][h] = make_float4(0.f, 0.f, 0.f, 0.f);
                    bv[it][h] = 0.f;
                    if (row < r_end) {
                        bv[it][h] = __ldg(beta + row);
                        if (j + 3 < d_out && vec_ok) {
                            xv[it][h] = __ldg(reinterpret_cast<const float4*>(gz + row * ldz + j));
                        } else {
                            if (j < d_out) xv[it][h].x = __ldg(gz + row * ldz + j);
                            if (j + 1 < d_out) xv[it][h].y = __ldg(gz + row * ldz + j + 1);
                            if (j + 2 < d_out) xv[it][h].z = __ldg(gz + row * ldz + j + 2);
                            if (j + 3 < d_out) xv[it][h].w = __ldg(gz + row * ldz + j + 3);
                        }
                    }
                }
            }
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
                const int t = threadIdx.x + it * kBwThreads;
                const int np = t & 31, jq = (t >> 5) * 4;
                const float x0[4] = {xv[it][0].x * bv[it][0], xv[it][0].y * bv[it][0], xv[it][0].z * bv[it][0], xv[it][0].w * bv[it][0]};
                const float x1[4] = {xv[it][1].x * bv[it][1], xv[it][1].y * bv[it][1], xv[it][1].z * bv[it][1], xv[it][1].w * bv[it][1]};
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    unsigned short h0, m0, l0, h1, m1, l1;
                    split3(x0[u], h0, m0, l0);
                    split3(x1[u], h1, m1, l1);
                    const uint32_t off = tc::canon_off(kRows, jq + u, (2 * np) >> 3) + ((2 * np) & 7) * 2;
                    *reinterpret_cast<uint32_t*>(As + 0 * kRows * 128 + off) = (uint32_t)h0 | ((uint32_t)h1 << 16);
                    *reinterpret_cast<uint32_t*>(As + 1 * kRows * 128 + off) = (uint32_t)m0 | ((uint32_t)m1 << 16);
                    *reinterpret_cast<uint32_t*>(As + 2 * kRows * 128 + off) = (uint32_t)l0 | ((uint32_t)l1 << 16);
                }
            }
        }
        // B: 32 node pairs x (N / 32) packed words x 4 groups of 8 inputs (loads batched in the same way)
        {
            constexpr int kItems = 32 * (N / 32) * 4 / kBwThreads;
            uint32_t w0v[kItems], w1v[kItems];
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
                const int t = threadIdx.x + it * kBwThreads;
                const int np = t & 31, wd = (t >> 5) >> 2;
                const int64_t row = r0 + 2 * np;
                w0v[it] = 0u, w1v[it] = 0u;
                if (wd * 32 < d_in) {
                    if (row < r_end) w0v[it] = __ldg(bits + row * stride + wd);
                    if (row + 1 < r_end) w1v[it] = __ldg(bits + (row + 1) * stride + wd);
                }
            }
#pragma unroll
            for (int it = 0; it < kItems; ++it) {
                const int t = threadIdx.x + it * kBwThreads;
                const int np = t & 31, wd = (t >> 5) >> 2, part8 = (t >> 5) & 3;
                const int kw = wd * 32;
                const int64_t row = r0 + 2 * np;
                const bool in0 = row < r_end, in1 = row + 1 < r_end;
#pragma unroll
                for (int b = 0; b < 8; ++b) {
                    const int kb = part8 * 8 + b, k = kw + kb;
                    const bool kin = k < d_in;
                    const uint32_t lo = (kin && in0) ? (((w0v[it] >> kb) & 1u) ? 0x3F80u : 0xBF80u) : 0u;
                    const uint32_t hi = (kin && in1) ? (((w1v[it] >> kb) & 1u) ? 0x3F80u : 0xBF80u) : 0u;
                    const uint32_t off = tc::canon_off(N, k, (2 * np) >> 3) + ((2 * np) & 7) * 2;
                    *reinterpret_cast<uint32_t*>(Bs + off) = lo | (hi << 16);
                }
            }
        }
        tc::fence_async_smem();
        tc::fence_before_sync();
        __syncthreads();
        tc::fence_after_sync();
        if (threadIdx.x == 0) {
            const uint32_t a_base = tc::smem_u32(As), b_base = tc::smem_u32(Bs);
            for (int ks = 0; ks < kKc / 16; ++ks) {
                const uint64_t bd = tc::make_desc(b_base + 2 * ks * b_lbo, b_lbo, sbo);
#pragma unroll
                for (int sp = 0; sp < 3; ++sp) {
                    const uint64_t ad = tc::make_desc(a_base + sp * kRows * 128 + 2 * ks * a_lbo, a_lbo, sbo);
                    const uint32_t accum = (any || ks > 0 || sp > 0) ? 1u : 0u;
                    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                                 ::"r"(tmem_base), "l"(ad), "l"(bd), "r"(idesc), "r"(accum) : "memory");
                }
            }
            tc::commit_to(&bar);
        }
        any = true;
        if (!tc::wait_barrier(&bar, phase)) {
            atomicExch(&g_bw_tc_timeout, 1);
            ok = false;
        }
        phase ^= 1u;
        tc::fence_after_sync();
        if (__syncthreads_or(!ok)) { ok = false; break; }   // the operands may be overwritten; leave together on a timeout
    }
    // ---- the slab: thread = channel j (tensor-memory lane), its warp's half of the inputs k
    if (ok) {
        float* slab = part + (int64_t)blockIdx.y * d_in * d_out;
        const int lane_base = 32 * (warp & 3);
        const int j = j0 + lane_base + lane;
        const int c_begin = (warp >> 2) * (N / 2);
        for (int c0 = c_begin; c0 < c_begin + N / 2; c0 += 16) {
            uint32_t v[16];
            if (any) tc::tmem_ld16(tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)c0, v);
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int k = c0 + e;
                if (j < d_out && k < d_in) slab[(int64_t)k * d_out + j] = any ? __uint_as_float(v[e]) : 0.f;
            }
        }
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_free(tmem_base, kCols);
}

template <int N>
cudaError_t launch_grad_wt_tc(cudaStream_t s, const uint32_t* bits, int64_t stride, const float* beta, const float* gz,
                              int64_t ldz, int64_t n, int d_in, int d_out, int n_splits, int64_t rows_per_split, float* part)
{
    const size_t smem = 3 * 128 * 128 + (size_t)N * 128;
    cudaError_t e = cudaFuncSetAttribute(grad_wt_tc_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)ceil_div(d_out, 128), (unsigned)n_splits);
    grad_wt_tc_kernel<N><<<grid, kBwThreads, smem, s>>>(bits, stride, beta, gz, ldz, n, d_in, d_out, rows_per_split, part);
    return cudaGetLastError();
}

template <int N>
cudaError_t launch_grad_h_tc(cudaStream_t s, const float* gz, int64_t ldz, const float* alpha, const float* W, int64_t ldw,
                             int64_t n, int d_in, int d_out, float* g_h, int64_t ldh)
{
    const size_t smem = 3 * 128 * 128 + (size_t)N * 128;
    cudaError_t e = cudaFuncSetAttribute(grad_h_tc_kernel<N>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)std::min<int64_t>(ceil_div(n, 128), sm_count() * 2);
    grad_h_tc_kernel<N><<<grid, kBwThreads, smem, s>>>(gz, ldz, alpha, W, ldw, n, d_in, d_out, g_h, ldh);
    return cudaGetLastError();
}

// Eq. bp-W.  One block per 32 output channels: thread (tx, ty) sums G_W~_kj B_kj over k = ty, ty + 32, ...
// for channel j0 + tx in double; the 32 partial sums of a channel are added in a fixed order; then
// every element gets (1/d_in) B_ij col_j + alpha_j G_W~_ij [|W_ij| < 1].
__global__ void __launch_bounds__(1024)
grad_w_kernel(const float* __restrict__ g_wt, const float* __restrict__ W, int64_t ldw,
              const float* __restrict__ alpha, int d_in, int d_out, float* __restrict__ g_w, int64_t ldgw)
{
    __shared__ double part[32][33];
    __shared__ double col[32];
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int j = blockIdx.x * 32 + tx;
    double s = 0.0;
    if (j < d_out)
        for (int k = ty; k < d_in; k += 32) {
            const float w = __ldg(W + (int64_t)k * ldw + j);
            const double g = (double)__ldg(g_wt + (int64_t)k * d_out + j);
            s += w >= 0.f ? g : -g;
        }
    part[ty][tx] = s;
    __syncthreads();
    if (ty == 0) {
        double t = 0.0;
        for (int r = 0; r < 32; ++r) t += part[r][tx];
        col[tx] = t;
    }
    __syncthreads();
    if (j < d_out) {
        const double c = col[tx] / (double)d_in;
        const float al = __ldg(alpha + j);
        for (int i = ty; i < d_in; i += 32) {
            const float w = __ldg(W + (int64_t)i * ldw + j);
            double g = w >= 0.f ? c : -c;
            if (fabsf(w) < 1.f) g += (double)al * (double)__ldg(g_wt + (int64_t)i * d_out + j);
            g_w[(int64_t)i * ldgw + j] = (float)g;
        }
    }
}

int64_t pad4(int64_t d) { return (d + 3) / 4 * 4; }

int wt_splits(int64_t n, int d_in, int d_out)
{
    const int64_t tiles = ceil_div(d_in, kMmaTile) * ceil_div(d_out, kMmaTile);
    const int64_t want = std::max<int64_t>(1, (sm_count() * 4) / tiles);               // about four blocks per SM in all
    return (int)std::max<int64_t>(1, std::min<int64_t>(want, ceil_div(n, 4 * kMmaK)));
}

}  // namespace

int backward_tc_timeouts()
{
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_bw_tc_timeout, sizeof(int)) != cudaSuccess) return -1;
    return v;
}

size_t backward_scratch_bytes(int64_t n, int d_in, int d_out)
{
    const size_t a = 256;
    auto up = [&](size_t b) { return (b + a - 1) / a * a; };
    size_t total = up((size_t)n * pad4(d_out) * 4);                              // G' with rows padded to 16 bytes
    total += up((size_t)n * pad4(d_out) * 4);                                    // G_zeta
    total += up((size_t)wt_splits(n, d_in, d_out) * d_in * d_out * 4);           // slabs of G_W~
    total += up((size_t)d_in * d_out * 4);                                       // G_W~
    total += up(spmm_scratch_bytes(n, 0, 0));
    return total;
}

cudaError_t launch_layer_backward(cudaStream_t s, int64_t n, const int64_t* rowptr, const int32_t* colidx,
                                  const float* val, int d_in, int d_out, const float* W, int64_t ldw,
                                  const float* alpha, const uint32_t* in_bits, int64_t stride_in,
                                  const float* in_beta, const float* g_out, int64_t ldg, float* g_in,
                                  int64_t ldgi, float* g_w, int64_t ldgw, int64_t long_row, void* scratch,
                                  int* launches)
{
    const size_t a = 256;
    auto up = [&](size_t b) { return (b + a - 1) / a * a; };
    char* base = static_cast<char*>(scratch);
    const int64_t ldz = pad4(d_out);
    float* g_pad = reinterpret_cast<float*>(base);
    base += up((size_t)n * ldz * 4);
    float* gz = reinterpret_cast<float*>(base);
    base += up((size_t)n * ldz * 4);
    const int n_splits = wt_splits(n, d_in, d_out);
    float* part = reinterpret_cast<float*>(base);
    base += up((size_t)n_splits * d_in * d_out * 4);
    float* g_wt = reinterpret_cast<float*>(base);
    base += up((size_t)d_in * d_out * 4);
    void* counter = base;

    // step 1a: G_zeta = A_tilde^T G' (A_tilde is symmetric: the forward aggregation on fp32 rows)
    const float* g_src = g_out;
    if (ldg != ldz || reinterpret_cast<uintptr_t>(g_out) % 16 != 0) {            // rows must be 16-byte vectors
        pad_rows_kernel<<<(unsigned)std::min<int64_t>(ceil_div(n * ldz, 256), sm_count() * 16), 256, 0, s>>>(g_out, n, d_out, ldg, g_pad, ldz);
        ++*launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        g_src = g_pad;
    }
    SpmmArgs sa;
    sa.n = n;
    sa.rowptr = rowptr;
    sa.colidx = colidx;
    sa.val = val;
    sa.fmt = kZetaF32;
    sa.zeta = g_src;
    sa.ldz = ldz;
    sa.d_out = d_out;
    sa.node_w = nullptr;
    sa.col_w = nullptr;
    sa.add = nullptr;
    sa.ld_add = 0;
    sa.h_out = gz;
    sa.ldh = ldz;
    sa.next_bits = nullptr;
    sa.next_stride = 0;
    sa.next_beta = nullptr;
    sa.next_shift = nullptr;
    sa.next_scale = nullptr;
    sa.long_row = long_row;
    sa.scratch = counter;
    sa.scratch_bytes = spmm_scratch_bytes(n, 0, 0);
    cudaError_t e = launch_spmm(s, sa, launches);
    if (e != cudaSuccess) return e;

    // step 1b: G_W~ = H~^T G_zeta, split over the rows, slabs added in a fixed order
    {
        const int64_t rows_per_split = ceil_div(ceil_div(n, n_splits), 64) * 64;
        ++*launches;
        if (d_in <= 256) {                                  // tcgen05 version: one tile covers all inputs
            if (d_in <= 64) e = launch_grad_wt_tc<64>(s, in_bits, stride_in, in_beta, gz, ldz, n, d_in, d_out, n_splits, rows_per_split, part);
            else if (d_in <= 128) e = launch_grad_wt_tc<128>(s, in_bits, stride_in, in_beta, gz, ldz, n, d_in, d_out, n_splits, rows_per_split, part);
            else e = launch_grad_wt_tc<256>(s, in_bits, stride_in, in_beta, gz, ldz, n, d_in, d_out, n_splits, rows_per_split, part);
            if (e != cudaSuccess) return e;
        } else {
            const dim3 grid((unsigned)ceil_div(d_out, kMmaTile), (unsigned)ceil_div(d_in, kMmaTile), (unsigned)n_splits);
            grad_wt_mma_kernel<<<grid, kBwThreads, 0, s>>>(in_bits, stride_in, in_beta, gz, ldz, n, d_in, d_out, rows_per_split, part);
            if ((e = cudaGetLastError()) != cudaSuccess) return e;
        }
        const int64_t elems = (int64_t)d_in * d_out;
        grad_wt_reduce_kernel<<<(unsigned)ceil_div(elems, 256), 256, 0, s>>>(part, n_splits, elems, g_wt);
        ++*launches;
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    // step 1c + 2: G_H = clip(G_zeta W~^T)
    if (g_in) {
        ++*launches;
        if (d_in <= 256 && d_in % 4 == 0 && ldgi % 4 == 0 && reinterpret_cast<uintptr_t>(g_in) % 16 == 0) {   // tcgen05 version
            if (d_in <= 64) e = launch_grad_h_tc<64>(s, gz, ldz, alpha, W, ldw, n, d_in, d_out, g_in, ldgi);
            else if (d_in <= 128) e = launch_grad_h_tc<128>(s, gz, ldz, alpha, W, ldw, n, d_in, d_out, g_in, ldgi);
            else e = launch_grad_h_tc<256>(s, gz, ldz, alpha, W, ldw, n, d_in, d_out, g_in, ldgi);
            if (e != cudaSuccess) return e;
        } else {
            const dim3 grid((unsigned)ceil_div(n, kMmaTile), (unsigned)ceil_div(d_in, kMmaTile));
            grad_h_mma_kernel<<<grid, kBwThreads, 0, s>>>(gz, ldz, alpha, W, ldw, n, d_in, d_out, g_in, ldgi);
            if ((e = cudaGetLastError()) != cudaSuccess) return e;
        }
    }
    // step 3: Eq. bp-W
    grad_w_kernel<<<(unsigned)ceil_div(d_out, 32), dim3(32, 32), 0, s>>>(g_wt, W, ldw, alpha, d_in, d_out, g_w, ldgw);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace bigcn
