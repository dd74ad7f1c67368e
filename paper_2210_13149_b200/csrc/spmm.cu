// Aggregation H' = A_tilde zeta as a CSR SpMM (Bi-GCN, last equation of Sec. 4.2.3), with the
// optional re-binarization of H' for the next layer (Sec. 4.2.2 applied to the layer output, after
// the next layer's batch-norm constants of Sec. 4.4) fused into the epilogue.
//
// One warp owns one output row.  A row of zeta is read as 16-byte vectors: LPR lanes cover one row
// (NCH vectors per lane when a row has more than 32 vectors) and the 32/LPR lane groups of a warp
// work on different neighbours at the same time; their partial sums are combined with shuffles.
// Rows with more stored entries than `long_row` are processed by all warps of the thread block
// together (each warp a contiguous slice of the row, partial sums combined through shared memory in
// warp order), so results never depend on scheduling.
#include "bigcn_internal.cuh"

namespace bigcn {

namespace {

constexpr int kSpmmWarps = 8;
constexpr int kSpmmThreads = kSpmmWarps * kWarp;
constexpr int kEdgesInFlight = 4;        // independent 16-byte gathers per lane group

template <typename T> struct Elt;
template <> struct Elt<float> {
    static constexpr int kPerVec = 4;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[4])
    {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
};
template <> struct Elt<int16_t> {
    static constexpr int kPerVec = 8;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[8])
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = (float)(int16_t)(w[i] & 0xffffu);
            f[2 * i + 1] = (float)((int32_t)w[i] >> 16);
        }
    }
};
template <> struct Elt<int8_t> {
    static constexpr int kPerVec = 16;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[16])
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[4 * i] = (float)(int8_t)(w[i] & 0xffu);
            f[4 * i + 1] = (float)(int8_t)((w[i] >> 8) & 0xffu);
            f[4 * i + 2] = (float)(int8_t)((w[i] >> 16) & 0xffu);
            f[4 * i + 3] = (float)((int32_t)w[i] >> 24);
        }
    }
};

struct SpmmDev {
    int64_t n;
    const int64_t* rowptr;
    const int32_t* colidx;
    const float* val;
    const uint4* zeta;       // rows of nv 16-byte vectors
    int nv;                  // vectors per zeta row
    int d_out;
    const float* node_w;     // nullable
    const float* col_w;      // nullable
    float* h_out;
    int64_t ldh;
    int h_vec;               // 1: rows of h_out can be stored as float4
    uint32_t* next_bits;
    int64_t next_stride;
    float* next_beta;
    const float* next_shift;
    const float* next_scale;
    int64_t long_row;
};

// acc += sum over stored entries [start, end) of weight * zeta row, for the calling warp.
template <typename T, int NCH, int LPR>
__device__ __forceinline__ void accumulate(const SpmmDev& p, int64_t start, int64_t end, int lane,
                                           float (&acc)[NCH][Elt<T>::kPerVec])
{
    constexpr int EPV = Elt<T>::kPerVec;
    constexpr int G = kWarp / LPR;
    constexpr int U = kEdgesInFlight;
    const int g = lane / LPR, l = lane % LPR;
    bool active[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) active[c] = (c * 32 + l) < p.nv;

    for (int64_t base = start; base < end; base += 32) {
        const int cnt = (int)min((int64_t)32, end - base);
        int my_col = 0;
        float my_w = 0.f;
        if (lane < cnt) {
            my_col = __ldg(p.colidx + base + lane);
            my_w = __ldg(p.val + base + lane);
            if (p.node_w) my_w *= __ldg(p.node_w + my_col);
        }
        for (int e = 0; e < cnt; e += G * U) {
            uint4 v[U][NCH];
            float w[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int idx = e + u * G + g;
                const int k = __shfl_sync(0xffffffffu, my_col, idx & 31);
                w[u] = __shfl_sync(0xffffffffu, my_w, idx & 31);
                const bool ok = idx < cnt;
                if (!ok) w[u] = 0.f;
                const uint4* zrow = p.zeta + (int64_t)k * p.nv + l;
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    if (ok && active[c]) v[u][c] = __ldg(zrow + c * 32);
                    else v[u][c] = make_uint4(0u, 0u, 0u, 0u);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
                    float f[EPV];
                    Elt<T>::unpack(v[u][c], f);
#pragma unroll
                    for (int i = 0; i < EPV; ++i) acc[c][i] = fmaf(w[u], f[i], acc[c][i]);
                }
        }
    }
    // combine the lane groups: afterwards every lane holds the sum for its vector(s)
#pragma unroll
    for (int o = LPR; o < kWarp; o <<= 1)
#pragma unroll
        for (int c = 0; c < NCH; ++c)
#pragma unroll
            for (int i = 0; i < EPV; ++i) acc[c][i] += __shfl_xor_sync(0xffffffffu, acc[c][i], o);
}

// Writes one finished row: optional fp32 store, optional sign/scale packing for the next layer.
// Called by a full warp; every lane holds the totals of vector(s) c*32 + (lane % LPR).
template <typename T, int NCH, int LPR>
__device__ __forceinline__ void finish_row(const SpmmDev& p, int64_t row, int lane,
                                           float (&acc)[NCH][Elt<T>::kPerVec])
{
    constexpr int EPV = Elt<T>::kPerVec;
    constexpr int LW = 32 / EPV;                  // lanes that share one packed word
    const int g = lane / LPR, l = lane % LPR;
    float l1 = 0.f;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        const int vec = c * 32 + l;
        const int col0 = vec * EPV;
        float x[EPV];
#pragma unroll
        for (int i = 0; i < EPV; ++i) {
            x[i] = acc[c][i];
            if (p.col_w) x[i] *= (col0 + i < p.d_out) ? __ldg(p.col_w + col0 + i) : 0.f;
        }
        if (p.h_out && g == 0 && vec < p.nv) {
            float* dst = p.h_out + row * p.ldh + col0;
            if (EPV == 4 && p.h_vec && col0 + 3 < p.d_out) {
                *reinterpret_cast<float4*>(dst) = make_float4(x[0], x[1], x[2], x[3]);
            } else {
#pragma unroll
                for (int i = 0; i < EPV; ++i)
                    if (col0 + i < p.d_out) dst[i] = x[i];
            }
        }
        if (p.next_bits) {
            uint32_t bits = 0u;
#pragma unroll
            for (int i = 0; i < EPV; ++i) {
                const int col = col0 + i;
                if (col < p.d_out) {
                    float xh = x[i];
                    if (p.next_shift)
                        xh = __fmul_rn(__fsub_rn(xh, __ldg(p.next_shift + col)), __ldg(p.next_scale + col));
                    if (xh >= 0.f) bits |= 1u << i;
                    if (g == 0) l1 += fabsf(xh);
                }
            }
            uint32_t word = bits << ((col0) & 31);
#pragma unroll
            for (int o = 1; o < LW; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
            const int widx = col0 >> 5;
            if (g == 0 && (l % LW) == 0 && vec < p.nv && widx < p.next_stride)
                p.next_bits[row * p.next_stride + widx] = word;
        }
    }
    if (p.next_bits) {
        const int covered = (int)ceil_div((int64_t)p.nv * EPV, 32);
        for (int w = covered + lane; w < p.next_stride; w += 32) p.next_bits[row * p.next_stride + w] = 0u;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l1 += __shfl_xor_sync(0xffffffffu, l1, o);
        if (lane == 0) p.next_beta[row] = l1 / (float)p.d_out;
    }
}

template <typename T, int NCH, int LPR>
__global__ void __launch_bounds__(kSpmmThreads)
spmm_kernel(const SpmmDev p)
{
    constexpr int EPV = Elt<T>::kPerVec;
    __shared__ float part[kSpmmWarps][(LPR < 32 ? LPR : NCH * 32) * EPV];
    __shared__ int long_mask;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t row = (int64_t)blockIdx.x * kSpmmWarps + warp;
    if (threadIdx.x == 0) long_mask = 0;
    __syncthreads();

    int64_t start = 0, end = 0;
    if (row < p.n) {
        start = __ldg(p.rowptr + row);
        end = __ldg(p.rowptr + row + 1);
    }
    const bool is_long = p.long_row > 0 && (end - start) > p.long_row;
    if (row < p.n && !is_long) {
        float acc[NCH][EPV];
#pragma unroll
        for (int c = 0; c < NCH; ++c)
#pragma unroll
            for (int i = 0; i < EPV; ++i) acc[c][i] = 0.f;
        accumulate<T, NCH, LPR>(p, start, end, lane, acc);
        finish_row<T, NCH, LPR>(p, row, lane, acc);
    }
    if (is_long && lane == 0) atomicOr(&long_mask, 1 << warp);
    __syncthreads();
    const int mask = long_mask;
    if (mask == 0) return;

    // Long rows of this block, one after the other, each by all warps together.
    for (int wr = 0; wr < kSpmmWarps; ++wr) {
        if (!((mask >> wr) & 1)) continue;
        const int64_t lrow = (int64_t)blockIdx.x * kSpmmWarps + wr;
        const int64_t ls = __ldg(p.rowptr + lrow), le = __ldg(p.rowptr + lrow + 1);
        const int64_t slice = round_up(ceil_div(le - ls, kSpmmWarps), 32);
        const int64_t s0 = min(le, ls + warp * slice), s1 = min(le, s0 + slice);
        float acc[NCH][EPV];
#pragma unroll
        for (int c = 0; c < NCH; ++c)
#pragma unroll
            for (int i = 0; i < EPV; ++i) acc[c][i] = 0.f;
        accumulate<T, NCH, LPR>(p, s0, s1, lane, acc);
        const int l = lane % LPR;
        if (lane < LPR) {
#pragma unroll
            for (int c = 0; c < NCH; ++c)
#pragma unroll
                for (int i = 0; i < EPV; ++i) part[warp][(c * 32 + l) * EPV + i] = acc[c][i];
        }
        __syncthreads();
        if (warp == 0) {
#pragma unroll
            for (int c = 0; c < NCH; ++c)
#pragma unroll
                for (int i = 0; i < EPV; ++i) {
                    float t = 0.f;
                    for (int w = 0; w < kSpmmWarps; ++w) t += part[w][(c * 32 + l) * EPV + i];
                    acc[c][i] = t;
                }
            finish_row<T, NCH, LPR>(p, lrow, lane, acc);
        }
        __syncthreads();
    }
}

template <typename T, int NCH, int LPR>
cudaError_t launch_one(cudaStream_t s, const SpmmDev& p)
{
    const unsigned grid = (unsigned)ceil_div(p.n, kSpmmWarps);
    spmm_kernel<T, NCH, LPR><<<grid, kSpmmThreads, 0, s>>>(p);
    return cudaGetLastError();
}

template <typename T>
cudaError_t dispatch(cudaStream_t s, const SpmmDev& p)
{
    const int nv = p.nv;
    if (nv <= 1) return launch_one<T, 1, 1>(s, p);
    if (nv <= 2) return launch_one<T, 1, 2>(s, p);
    if (nv <= 4) return launch_one<T, 1, 4>(s, p);
    if (nv <= 8) return launch_one<T, 1, 8>(s, p);
    if (nv <= 16) return launch_one<T, 1, 16>(s, p);
    if (nv <= 32) return launch_one<T, 1, 32>(s, p);
    // wider rows: up to 512 columns in any format (128 / 64 / 32 vectors of fp32 / int16 / int8)
    if constexpr (sizeof(T) >= 2) {
        if (nv <= 64) return launch_one<T, 2, 32>(s, p);
    }
    if constexpr (sizeof(T) == 4) {
        if (nv <= 128) return launch_one<T, 4, 32>(s, p);
    }
    return cudaErrorInvalidConfiguration;
}

}  // namespace

size_t spmm_scratch_bytes(int64_t, int64_t, int) { return 0; }

cudaError_t launch_spmm(cudaStream_t s, const SpmmArgs& a, int* launches)
{
    if (a.n == 0) return cudaSuccess;
    SpmmDev p;
    p.n = a.n;
    p.rowptr = a.rowptr;
    p.colidx = a.colidx;
    p.val = a.val;
    p.zeta = reinterpret_cast<const uint4*>(a.zeta);
    p.nv = (int)(a.ldz * zeta_elt_bytes(a.fmt) / 16);
    p.d_out = a.d_out;
    p.node_w = a.fmt == kZetaF32 ? nullptr : a.node_w;
    p.col_w = a.fmt == kZetaF32 ? nullptr : a.col_w;
    p.h_out = a.h_out;
    p.ldh = a.ldh;
    p.h_vec = (a.h_out && (a.ldh % 4 == 0) && (reinterpret_cast<uintptr_t>(a.h_out) % 16 == 0)) ? 1 : 0;
    p.next_bits = a.next_bits;
    p.next_stride = a.next_stride;
    p.next_beta = a.next_beta;
    p.next_shift = a.next_shift;
    p.next_scale = a.next_scale;
    p.long_row = a.long_row;
    ++*launches;
    switch (a.fmt) {
        case kZetaF32: return dispatch<float>(s, p);
        case kZetaI16: return dispatch<int16_t>(s, p);
        case kZetaI8: return dispatch<int8_t>(s, p);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace bigcn
