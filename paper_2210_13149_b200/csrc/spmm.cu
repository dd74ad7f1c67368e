// Aggregation H' = A_tilde zeta as a CSR SpMM (Bi-GCN, last equation of Sec. 4.2.3), with the
// optional re-binarization of H' for the next layer (Sec. 4.2.2 applied to the layer output, after
// the next layer's batch-norm constants of Sec. 4.4) fused into the epilogue.
//
// The kernel is bound by the random gather of zeta rows, so it is built around keeping many row
// fetches in flight at a low instruction cost per stored entry.  A warp owns a run of consecutive
// output rows and treats their stored entries as one stream.  Each stream position is fetched with
// one warp-wide asynchronous copy (cp.async, 16 bytes per lane, global -> shared, bypassing L1 and
// the register file) into a ring of slots private to the warp; positions are issued and retired in
// groups of PB, and NG groups are in flight per warp, across row boundaries.  A row of zeta is nv
// 16-byte vectors: LPR lanes cover one row (NCH vectors per lane when nv > 32) and the G = 32/LPR
// lane groups of a warp fetch G consecutive entries per position; their partial sums are combined
// with shuffles when a row ends.  Column indices and edge weights are prefetched three 32-entry
// chunks ahead in registers.  There is no waiting on other warps or blocks anywhere:
// cp.async.wait_group only waits for the calling thread's own copies.
//
// Runs of rows are handed out to warps through an atomic counter in global memory (zeroed by the
// launcher), so that warps with heavy rows do not hold back the others; which warp computes a row
// does not change how the row is computed, so results never depend on scheduling.
//
// Rows with more stored entries than `long_row` are left out of the streams and processed afterwards
// by all warps of the thread block together (each warp a contiguous slice, partial sums combined
// through shared memory in warp order).
#include <cuda_fp16.h>

#include <algorithm>

#include "bigcn_internal.cuh"
#include "spmm_dev.cuh"

namespace bigcn {

namespace {

constexpr int kSpmmWarps = 8;
constexpr int kSpmmThreads = kSpmmWarps * kWarp;
constexpr int kMaxRowsPerWarp = 16;      // consecutive rows handed to a warp at a time
constexpr int kLongQueue = 96;           // long rows a thread block can queue for cooperative processing

// Element types of a zeta row and their conversion to fp32 (one 16-byte vector at a time).
template <typename T> struct Elt;
template <> struct Elt<float> {
    static constexpr int kPerVec = 4;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[4])
    {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
};
template <> struct Elt<__half> {
    static constexpr int kPerVec = 8;
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[8])
    {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 t = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
            f[2 * i] = t.x;
            f[2 * i + 1] = t.y;
        }
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
    // Without the conversion unit: b ^ 0x80 placed in the low mantissa byte of 2^23 is the float 2^23 + 128 + b;
    // one subtraction gives b exactly.
    static __device__ __forceinline__ void unpack(const uint4& v, float (&f)[16])
    {
        const uint32_t w[4] = {v.x ^ 0x80808080u, v.y ^ 0x80808080u, v.z ^ 0x80808080u, v.w ^ 0x80808080u};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[4 * i] = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7540)) - 8388736.f;
            f[4 * i + 1] = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7541)) - 8388736.f;
            f[4 * i + 2] = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7542)) - 8388736.f;
            f[4 * i + 3] = __uint_as_float(__byte_perm(w[i], 0x4B000000u, 0x7543)) - 8388736.f;
        }
    }
};


__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src)
{
    const unsigned dst = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

template <int NCH, int EPV>
__device__ __forceinline__ void zero_acc(float (&acc)[NCH][EPV])
{
#pragma unroll
    for (int c = 0; c < NCH; ++c)
#pragma unroll
        for (int i = 0; i < EPV; ++i) acc[c][i] = 0.f;
}

// Sum over the lane groups: afterwards every lane holds the total for its vector(s).
template <int NCH, int EPV, int LPR>
__device__ __forceinline__ void reduce_groups(float (&acc)[NCH][EPV])
{
#pragma unroll
    for (int o = LPR; o < kWarp; o <<= 1)
#pragma unroll
        for (int c = 0; c < NCH; ++c)
#pragma unroll
            for (int i = 0; i < EPV; ++i) acc[c][i] += __shfl_xor_sync(0xffffffffu, acc[c][i], o);
}

// Per-column constants of the row epilogue, staged once per thread block: four arrays of kCols
// floats -- the column factor (0 for padding columns, 1 when there is none), the next layer's shift and
// scale (0 and 1 where there are none, so that applying them changes nothing), and the first weight
// sign of the column (half-dot bytes only, else 0).  Inside an array the 16-byte chunks are ordered so that the
// lanes' reads in the row epilogue are contiguous: a lane holds EPV consecutive columns (EPV / 4 chunks) and reads
// its q-th chunk together with the other lanes, so chunk q of vector v sits at position q * (kCols / EPV) + v
// (in column order the reads of 8- and 16-column vectors fall 32 and 64 bytes apart: 2- and 4-way bank conflicts).
template <int kCols, int EPV>
__device__ __forceinline__ int ctab_at(int col)
{
    constexpr int Q = EPV / 4, NVEC = kCols / EPV;
    const int ch = col >> 2;
    return 4 * ((ch % Q) * NVEC + ch / Q) + (col & 3);
}

template <int kCols, int EPV>
__device__ __forceinline__ void fill_col_table(const SpmmDev& p, float* ctab)
{
    for (int col = threadIdx.x; col < kCols; col += blockDim.x) {
        const bool in = col < p.d_out;
        const int at = ctab_at<kCols, EPV>(col);
        ctab[at] = in ? (p.col_w ? __ldg(p.col_w + col) : 1.f) : 0.f;
        ctab[kCols + at] = (in && p.next_shift) ? __ldg(p.next_shift + col) : 0.f;
        ctab[2 * kCols + at] = (in && p.next_shift) ? __ldg(p.next_scale + col) : 1.f;
        ctab[3 * kCols + at] = (in && p.col_b0) ? __ldg(p.col_b0 + col) : 0.f;
    }
}

// Writes one finished row: optional fp32 store, optional sign/scale packing for the next layer.
// Called by a full warp; every lane holds the totals of vector(s) c*32 + (lane % LPR).
// kHalf (half-dot bytes): the accumulators hold sum_k w_k s_kj with s = (dot' - 1) / 2; the row's sum of the
// edge weights `wsum` and their sum signed by the sources' first feature sign `wsgn` give back
// sum_k w_k dot_kj = 2 acc_j + wsum + b0_j wsgn before the column factor is applied.
template <typename T, int NCH, int LPR, bool kHalf = false>
__device__ __forceinline__ void finish_row(const SpmmDev& p, const float* ctab, int64_t row, int lane,
                                           float (&acc)[NCH][Elt<T>::kPerVec], float wsum = 0.f, float wsgn = 0.f)
{
    constexpr int EPV = Elt<T>::kPerVec;
    constexpr int LW = 32 / EPV;                  // lanes that share one packed word
    constexpr int kCols = NCH * (LPR < 32 ? LPR : 32) * EPV;
    const int g = lane / LPR, l = lane % LPR;
    float l1 = 0.f;
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
        const int vec = c * (LPR < 32 ? LPR : 32) + l;
        const int col0 = vec * EPV;
        float x[EPV], sh[EPV], sc[EPV];
#pragma unroll
        for (int q = 0; q < EPV / 4; ++q) {
            const float4 a = *reinterpret_cast<const float4*>(ctab + ctab_at<kCols, EPV>(col0 + 4 * q));
            float t[4] = {acc[c][4 * q], acc[c][4 * q + 1], acc[c][4 * q + 2], acc[c][4 * q + 3]};
            if constexpr (kHalf) {
                const float4 b0 = *reinterpret_cast<const float4*>(ctab + 3 * kCols + ctab_at<kCols, EPV>(col0 + 4 * q));
                t[0] = fmaf(2.f, t[0], fmaf(b0.x, wsgn, wsum));
                t[1] = fmaf(2.f, t[1], fmaf(b0.y, wsgn, wsum));
                t[2] = fmaf(2.f, t[2], fmaf(b0.z, wsgn, wsum));
                t[3] = fmaf(2.f, t[3], fmaf(b0.w, wsgn, wsum));
            }
            x[4 * q] = t[0] * a.x;
            x[4 * q + 1] = t[1] * a.y;
            x[4 * q + 2] = t[2] * a.z;
            x[4 * q + 3] = t[3] * a.w;
        }
        if (p.add) {
#pragma unroll
            for (int i = 0; i < EPV; ++i)
                if (col0 + i < p.d_out) x[i] += __ldg(p.add + row * p.ld_add + col0 + i);
        }
        if (p.h_out && g == 0 && vec < p.nv_fin) {
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
#pragma unroll
            for (int q = 0; q < EPV / 4; ++q) {
                const float4 a = *reinterpret_cast<const float4*>(ctab + kCols + ctab_at<kCols, EPV>(col0 + 4 * q));
                const float4 b = *reinterpret_cast<const float4*>(ctab + 2 * kCols + ctab_at<kCols, EPV>(col0 + 4 * q));
                sh[4 * q] = a.x, sh[4 * q + 1] = a.y, sh[4 * q + 2] = a.z, sh[4 * q + 3] = a.w;
                sc[4 * q] = b.x, sc[4 * q + 1] = b.y, sc[4 * q + 2] = b.z, sc[4 * q + 3] = b.w;
            }
            uint32_t bits = 0u;
            float l1c = 0.f;
#pragma unroll
            for (int i = 0; i < EPV; ++i) {
                const float xh = __fmul_rn(__fsub_rn(x[i], sh[i]), sc[i]);   // padding columns: (0 - 0) * 1
                if (xh >= 0.f) bits |= 1u << i;
                l1c += fabsf(xh);
            }
            if (vec < p.nv_fin) l1 += l1c;            // lanes past the last vector accumulated nothing meaningful
            const int n_valid = min(max(p.d_out - col0, 0), EPV);            // padding columns pack as 0
            bits &= (n_valid >= 32) ? 0xffffffffu : ((1u << n_valid) - 1u);
            uint32_t word = bits << ((col0) & 31);
#pragma unroll
            for (int o = 1; o < LW; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
            const int widx = col0 >> 5;
            if (g == 0 && (l % LW) == 0 && vec < p.nv_fin && widx < p.next_stride)
                p.next_bits[row * p.next_stride + widx] = word;
        }
    }
    if (p.next_bits) {
        for (int w = p.covered_words + lane; w < p.next_stride; w += 32) p.next_bits[row * p.next_stride + w] = 0u;
        if (g != 0) l1 = 0.f;                     // the other lane groups hold copies of the same totals
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) l1 += __shfl_xor_sync(0xffffffffu, l1, o);
        if (lane == 0) p.next_beta[row] = l1 * p.inv_d_out;
    }
}

template <int NCH, int LPR, bool kAligned = false>
struct Pipe {
    static constexpr int G = kWarp / LPR;                       // entries per position
    // positions per group (PB * G divides 32); the aligned stream with two entries per position takes 8
    static constexpr int PB = ((kAligned && G == 2 && NCH == 1) || (LPR == 32 && NCH == 1)) ? 8 : ((4 * G <= 32) ? 4 : 32 / G);
    static constexpr int NG = (NCH > 1 || PB == 8) ? 2 : ((LPR == 32 || kAligned) ? 4 : 3);  // groups in flight per warp (a power of two for the row-aligned streams)
    static constexpr int RING = PB * NG;                        // slots of NCH * 512 bytes
    static constexpr size_t kWarpBytes = (size_t)RING * (NCH * 512 + G * 4);
};

// Streams the stored entries [e0, e0 + n_ent) through the warp's ring.
//   kPartial = false: the entries are those of rows [row_lo, row_hi); `rp_rel` holds, in lane j, the
//                     end of local row j - 1 relative to e0 (shuffled out as rows complete); every
//                     row is written as its last entry is consumed.
//   kPartial = true : the entries are a slice of one long row; the slice's sum is left in `acc`
//                     (already combined over the lane groups).
__device__ __forceinline__ void fma_bytes16(float w, const uint4& v, float (&acc)[16]);

// kHalf (rows of signed bytes only): half-dot bytes -- the weights' sign carries the source's first feature sign; the
// row's plain and signed weight sums ride along and the epilogue reconstructs the dots (see finish_row).
template <typename T, int NCH, int LPR, bool kPartial, bool kHalf = false>
__device__ __forceinline__ void stream_entries(const SpmmDev& p, uint4* ring, float* wfifo, const float* ctab, int lane,
                                               int64_t e0, int n_ent, int64_t warp_row0, int row_lo,
                                               int row_hi, int rp_rel,
                                               float (&acc)[NCH][Elt<T>::kPerVec])
{
    using P = Pipe<NCH, LPR>;
    constexpr int EPV = Elt<T>::kPerVec;
    constexpr int G = P::G, PB = P::PB, NG = P::NG;
    const int g = lane / LPR, l = lane % LPR;
    bool active[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) active[c] = (c * 32 + l) < p.nv;
    const int32_t* cols = p.colidx + e0;
    const float* vals = p.val + e0;

    // metadata chunks of 32 entries: A = ready (column, weight), B = column/value/node factor in
    // flight, C = column/value in flight
    auto load_col = [&](int e) { return e < n_ent ? __ldg(cols + e) : 0; };
    auto load_val = [&](int e) { return e < n_ent ? __ldg(vals + e) : 0.f; };
    int a_col = load_col(lane);
    float a_w = load_val(lane);
    int b_col = load_col(32 + lane);
    float b_val = load_val(32 + lane);
    int c_col = load_col(64 + lane);
    float c_val = load_val(64 + lane);
    if (p.node_w) a_w *= __ldg(p.node_w + a_col);
    float b_nw = p.node_w ? __ldg(p.node_w + b_col) : 1.f;
    int chunk = 0;

    const int n_groups = (n_ent + PB * G - 1) / (PB * G);
    int rt = row_lo;                                          // row being accumulated (local index)
    int row_end = kPartial ? n_ent : __shfl_sync(0xffffffffu, rp_rel, rt + 1);
    zero_acc<NCH, EPV>(acc);
    float wsum = 0.f, wsgn = 0.f;                             // half-dot bytes: sum of the row's weights, plain and signed

    for (int it = 0; it < n_groups + NG; ++it) {
        const int gslot = (it % NG) * PB;                     // first slot of the group handled now
        if (it >= NG) {
            // ---- retire group it - NG (its copies are the oldest outstanding cp.async group)
            cp_async_wait<NG - 1>();
            __syncwarp();
            const int off0 = (it - NG) * (PB * G);            // first entry of the group
            uint4 v[PB][NCH];
            float w[PB];
#pragma unroll
            for (int b = 0; b < PB; ++b) {
#pragma unroll
                for (int c = 0; c < NCH; ++c) v[b][c] = ring[(gslot + b) * (NCH * 32) + c * 32 + lane];
                w[b] = wfifo[(gslot + b) * G + g];
            }
            if (off0 + PB * G < row_end) {
                // the whole group lies inside the current row: no boundary logic
#pragma unroll
                for (int b = 0; b < PB; ++b) {
                    const float wa = kHalf ? fabsf(w[b]) : w[b];
                    if (kHalf) { wsum += wa; wsgn += w[b]; }
#pragma unroll
                    for (int c = 0; c < NCH; ++c) {
                        if constexpr (sizeof(T) == 1) {
                            if (NCH == 1 || active[c]) fma_bytes16(wa, v[b][c], acc[c]);
                        } else {
                            float f[EPV];
                            Elt<T>::unpack(v[b][c], f);
                            if (NCH == 1 || active[c]) {
#pragma unroll
                                for (int i = 0; i < EPV; ++i) acc[c][i] = fmaf(wa, f[i], acc[c][i]);
                            }
                        }
                    }
                }
            } else {
#pragma unroll
                for (int b = 0; b < PB; ++b) {
                    const int eb = off0 + b * G;              // first entry of the position
                    if (eb >= n_ent) break;
                    const int nb = min(G, n_ent - eb);
                    float f[NCH][EPV];
#pragma unroll
                    for (int c = 0; c < NCH; ++c) Elt<T>::unpack(v[b][c], f[c]);
                    int done = 0;
                    for (;;) {
                        const int rem = row_end - eb;         // entries of the position before the row's end
                        const int upto = rem < nb ? rem : nb;
                        if (g >= done && g < upto) {
                            const float wa = kHalf ? fabsf(w[b]) : w[b];
                            if (kHalf) { wsum += wa; wsgn += w[b]; }
#pragma unroll
                            for (int c = 0; c < NCH; ++c)
                                if (active[c]) {
#pragma unroll
                                    for (int i = 0; i < EPV; ++i) acc[c][i] = fmaf(wa, f[c][i], acc[c][i]);
                                }
                        }
                        if (rem > nb) break;                  // the row continues in a later position
                        reduce_groups<NCH, EPV, LPR>(acc);
                        if (kHalf) {
#pragma unroll
                            for (int o = LPR; o < kWarp; o <<= 1) {
                                wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
                                wsgn += __shfl_xor_sync(0xffffffffu, wsgn, o);
                            }
                        }
                        if (kPartial) {                       // slice complete (only at the last position)
                            if (kHalf) {                      // hand back the reconstructed partial sums
                                constexpr int kCols = NCH * LPR * EPV;
#pragma unroll
                                for (int c = 0; c < NCH; ++c)
#pragma unroll
                                    for (int i = 0; i < EPV; ++i)
                                        acc[c][i] = fmaf(2.f, acc[c][i], fmaf(ctab[3 * kCols + ctab_at<kCols, EPV>((c * LPR + l) * EPV + i)], wsgn, wsum));
                            }
                            return;
                        }
                        finish_row<T, NCH, LPR, kHalf>(p, ctab, warp_row0 + rt, lane, acc, wsum, wsgn);
                        zero_acc<NCH, EPV>(acc);
                        wsum = 0.f;
                        wsgn = 0.f;
                        if (upto > done) done = upto;
                        ++rt;
                        if (rt == row_hi) break;
                        row_end = __shfl_sync(0xffffffffu, rp_rel, rt + 1);
                    }
                }
            }
            __syncwarp();                                     // all lanes are done with these slots
        }
        if (it < n_groups) {
            // ---- issue group `it` into the slots just freed
            const int off0 = it * (PB * G);
            if ((off0 >> 5) != chunk) {                       // rotate the metadata chunks
                a_col = b_col;
                a_w = b_val * b_nw;
                b_col = c_col;
                b_val = c_val;
                b_nw = p.node_w ? __ldg(p.node_w + b_col) : 1.f;
                ++chunk;
                c_col = load_col(((chunk + 2) << 5) + lane);
                c_val = load_val(((chunk + 2) << 5) + lane);
            }
            const bool whole = off0 + PB * G <= n_ent;        // no entry of the group is past the end
#pragma unroll
            for (int b = 0; b < PB; ++b) {
                const int idx = (off0 & 31) + b * G + g;
                const int k = __shfl_sync(0xffffffffu, a_col, idx);
                const float wv = __shfl_sync(0xffffffffu, a_w, idx);
                if (whole || off0 + b * G + g < n_ent) {
                    const uint4* src = p.zeta + (int64_t)k * p.nv + l;
                    uint4* dst = ring + (gslot + b) * (NCH * 32) + lane;
#pragma unroll
                    for (int c = 0; c < NCH; ++c)
                        if (active[c]) cp_async16(dst + c * 32, src + c * 32);
                }
                if (l == 0) wfifo[(gslot + b) * G + g] = wv;  // padding entries carry weight 0
            }
        }
        cp_async_commit();                                    // one group per iteration, possibly empty
    }
    cp_async_wait<0>();
    if constexpr (kPartial) {                                 // empty slice
        reduce_groups<NCH, EPV, LPR>(acc);
    } else {
        while (rt < row_hi) {                                 // rows without entries at the end of the run
            reduce_groups<NCH, EPV, LPR>(acc);
            finish_row<T, NCH, LPR>(p, ctab, warp_row0 + rt, lane, acc);
            zero_acc<NCH, EPV>(acc);
            ++rt;
        }
    }
}

// acc[0..EPV) += w * (the EPV elements of one 16-byte vector), using the packed two-lane fp32 FMA
// of sm_100 where the element type converts pairwise.
template <typename T>
__device__ __forceinline__ void fma_vec(float w, const uint4& v, float (&acc)[Elt<T>::kPerVec])
{
    constexpr int EPV = Elt<T>::kPerVec;
    if constexpr (sizeof(T) == 1) {
        float f[EPV];
        Elt<T>::unpack(v, f);
#pragma unroll
        for (int i = 0; i < EPV; ++i) acc[i] = fmaf(w, f[i], acc[i]);
    } else {
        float f[EPV];
        Elt<T>::unpack(v, f);
        const float2 ww = make_float2(w, w);
#pragma unroll
        for (int i = 0; i < EPV; i += 2) {
            const float2 r = __ffma2_rn(ww, make_float2(f[i], f[i + 1]), make_float2(acc[i], acc[i + 1]));
            acc[i] = r.x;
            acc[i + 1] = r.y;
        }
    }
}

__device__ __forceinline__ void cp_async16_s(uint32_t smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}

// The same stream for wide rows (LPR = 32: one stored entry per position, the common hot case), laid
// out so that the inner loop carries no row-boundary logic: a group of PB positions never straddles a
// row.  A row with `deg` entries takes ceil(deg / PB) groups (at least one, so that rows without
// entries are still written); the unused positions of a row's last group are simply not copied and
// not accumulated.  The issue cursor and the retire cursor walk the rows in the same way, NG groups
// apart.  Column indices and weights of the next entries sit in two ready 32-entry chunks (A, B) so
// that a group may reach past a chunk boundary; two more chunks (C, D) are in flight behind them.
// Full groups (the usual case) take straight-line code on both sides.  kFull: every lane of a position
// holds a vector of the row (nv = 32 * NCH), so no lane needs masking.
template <typename T, int NCH, bool kFull, bool kPartial>
__device__ __forceinline__ void stream_rows_wide(const SpmmDev& p, uint4* ring, float* wfifo, const float* ctab, int lane,
                                                 int64_t e0, int n_ent, int64_t warp_row0, int row_lo,
                                                 int row_hi, int rp_rel,
                                                 float (&acc)[NCH][Elt<T>::kPerVec])
{
    using P = Pipe<NCH, 32>;
    constexpr int EPV = Elt<T>::kPerVec;
    constexpr int PB = P::PB, NG = P::NG;
    static_assert(PB % 4 == 0 && (NG & (NG - 1)) == 0, "float4 weight reads; power-of-two group ring");
    constexpr int kSlotVecs = NCH * 32;                       // 16-byte vectors per slot
    bool active[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) active[c] = (c * 32 + lane) < p.nv;
    const int32_t* cols = p.colidx + e0;
    const float* vals = p.val + e0;
    auto load_col = [&](int e) { return e < n_ent ? __ldg(cols + e) : 0; };
    auto load_val = [&](int e) { return e < n_ent ? __ldg(vals + e) : 0.f; };
    auto load_nw = [&](int col) { return p.node_w ? __ldg(p.node_w + col) : 1.f; };
    auto row_end_of = [&](int r) { return kPartial ? n_ent : __shfl_sync(0xffffffffu, rp_rel, r + 1); };
    const uint4* ring_l = ring + lane;                        // this lane's vector of slot 0
    const uint32_t ring_sa = (uint32_t)__cvta_generic_to_shared(ring_l);
    const char* zeta_l = reinterpret_cast<const char*>(p.zeta + lane);
    const uint32_t row_bytes = (uint32_t)p.nv * 16u;

    int a_col = load_col(lane), b_col = load_col(32 + lane), c_col = load_col(64 + lane), d_col = load_col(96 + lane);
    float a_w = load_val(lane), b_w = load_val(32 + lane), c_val = load_val(64 + lane), d_val = load_val(96 + lane);
    a_w *= load_nw(a_col);
    b_w *= load_nw(b_col);
    float c_nw = load_nw(c_col);
    int cbase = 0;                                            // first entry of chunk A

    int ie = 0, ir = row_lo, iend = row_end_of(row_lo);       // issue cursor: entry, row, end of that row
    int re = 0, rr = row_lo, rend = iend;                     // retire cursor
    bool more = row_lo < row_hi;
    int issued = 0, goff = 0;                                 // groups issued; ring position of the current group
    zero_acc<NCH, EPV>(acc);

    for (int it = 0;; ++it) {
        if (it >= NG) {
            if (it - NG >= issued) break;
            // ---- retire the oldest group
            cp_async_wait<NG - 1>();
            __syncwarp();
            const uint4* gp = ring_l + goff * (PB * kSlotVecs);
            const int left = rend - re;
#pragma unroll
            for (int q = 0; q < PB / 4; ++q) {                // four positions at a time
                uint4 v[4][NCH];
#pragma unroll
                for (int b = 0; b < 4; ++b)
#pragma unroll
                    for (int c = 0; c < NCH; ++c) v[b][c] = gp[(4 * q + b) * kSlotVecs + c * 32];
                const float4 w4 = *reinterpret_cast<const float4*>(wfifo + goff * PB + 4 * q);
                const float w[4] = {w4.x, w4.y, w4.z, w4.w};
                if (left >= PB) {
#pragma unroll
                    for (int b = 0; b < 4; ++b)
#pragma unroll
                        for (int c = 0; c < NCH; ++c)
                            if (kFull || active[c]) fma_vec<T>(w[b], v[b][c], acc[c]);
                } else {
#pragma unroll
                    for (int b = 0; b < 4; ++b)
                        if (4 * q + b < left) {
#pragma unroll
                            for (int c = 0; c < NCH; ++c)
                                if (kFull || active[c]) fma_vec<T>(w[b], v[b][c], acc[c]);
                        }
                }
            }
            re = left >= PB ? re + PB : rend;
            if (re == rend) {                                 // the row is complete
                if (kPartial) return;
                finish_row<T, NCH, 32>(p, ctab, warp_row0 + rr, lane, acc);
                zero_acc<NCH, EPV>(acc);
                ++rr;
                if (rr < row_hi) rend = row_end_of(rr);
            }
            __syncwarp();                                     // all lanes are done with these slots
        }
        if (more) {
            // ---- issue the next group of the row under the issue cursor
            const int left = iend - ie;
            const int base = ie - cbase;                      // position of the group in chunk A (< 32)
            const uint32_t dsta = ring_sa + goff * (PB * kSlotVecs * 16);
            // the window of the next 32 entries: lanes below `base` have handed out their chunk-A entry
            // already and present their chunk-B entry instead, so entry base + b sits in lane (base + b) % 32
            const int m_col = lane >= base ? a_col : b_col;
            const float m_w = lane >= base ? a_w : b_w;
            const int rel = (lane - base) & 31;               // entry of the window held by this lane
            if (left >= PB) {
#pragma unroll
                for (int b = 0; b < PB; ++b) {
                    const uint32_t k = (uint32_t)__shfl_sync(0xffffffffu, m_col, base + b);
                    const char* src = zeta_l + (uint64_t)k * row_bytes;
#pragma unroll
                    for (int c = 0; c < NCH; ++c)
                        if (kFull || active[c]) cp_async16_s(dsta + (b * kSlotVecs + c * 32) * 16, src + c * 512);
                }
                if (rel < PB) wfifo[goff * PB + rel] = m_w;
                ie += PB;
            } else {
#pragma unroll
                for (int b = 0; b < PB - 1; ++b) {
                    const uint32_t k = (uint32_t)__shfl_sync(0xffffffffu, m_col, base + b);
                    const char* src = zeta_l + (uint64_t)k * row_bytes;
                    if (b < left) {
#pragma unroll
                        for (int c = 0; c < NCH; ++c)
                            if (kFull || active[c]) cp_async16_s(dsta + (b * kSlotVecs + c * 32) * 16, src + c * 512);
                    }
                }
                if (rel < left) wfifo[goff * PB + rel] = m_w;
                ie += left;
            }
            ++issued;
            if (ie == iend) {
                ++ir;
                if (ir == row_hi) more = false;
                else iend = row_end_of(ir);
            }
            if (ie - cbase >= 32) {                           // rotate the metadata chunks
                a_col = b_col;
                a_w = b_w;
                b_col = c_col;
                b_w = c_val * c_nw;
                c_col = d_col;
                c_val = d_val;
                c_nw = load_nw(c_col);
                cbase += 32;
                d_col = load_col(cbase + 96 + lane);
                d_val = load_val(cbase + 96 + lane);
            }
        }
        cp_async_commit();                                    // one group per iteration, possibly empty
        goff = (goff + 1) & (NG - 1);
    }
    cp_async_wait<0>();
}

// acc[0..16) += w * (the 16 signed bytes of one 16-byte vector).  A byte b becomes the float
// 2^23 + (b + 128) by placing b ^ 0x80 in the low mantissa byte of 0x4B000000 (one byte-permute, no
// conversion unit); subtracting 2^23 + 128 gives b exactly; both steps and the FMA use the packed
// two-lane fp32 instructions.
__device__ __forceinline__ void fma_bytes16(float w, const uint4& v, float (&acc)[16])
{
    const uint32_t x[4] = {v.x ^ 0x80808080u, v.y ^ 0x80808080u, v.z ^ 0x80808080u, v.w ^ 0x80808080u};
    const float2 ww = make_float2(w, w);
    const float2 bias = make_float2(-8388736.f, -8388736.f);   // -(2^23 + 128)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 lo = make_float2(__uint_as_float(__byte_perm(x[i], 0x4B000000u, 0x7540)),
                                      __uint_as_float(__byte_perm(x[i], 0x4B000000u, 0x7541)));
        const float2 hi = make_float2(__uint_as_float(__byte_perm(x[i], 0x4B000000u, 0x7542)),
                                      __uint_as_float(__byte_perm(x[i], 0x4B000000u, 0x7543)));
        const float2 r0 = __ffma2_rn(ww, __fadd2_rn(lo, bias), make_float2(acc[4 * i], acc[4 * i + 1]));
        const float2 r1 = __ffma2_rn(ww, __fadd2_rn(hi, bias), make_float2(acc[4 * i + 2], acc[4 * i + 3]));
        acc[4 * i] = r0.x, acc[4 * i + 1] = r0.y, acc[4 * i + 2] = r1.x, acc[4 * i + 3] = r1.y;
    }
}

// acc += w * (one 16-byte vector of T), whatever T.
template <typename T>
__device__ __forceinline__ void fma_any(float w, const uint4& v, float (&acc)[Elt<T>::kPerVec])
{
    if constexpr (sizeof(T) == 1) fma_bytes16(w, v, acc);
    else fma_vec<T>(w, v, acc);
}

// The row-aligned stream for rows of up to NV * LPR vectors: a position holds G = 32 / LPR stored entries,
// one per group of LPR lanes (lane = LPR g + l fetches and accumulates vectors l, LPR + l, .. (NV of them)
// of entry G b + g of position b), so the per-position bookkeeping is shared by G entries.
// A group is 4 positions = 4 G entries and never straddles a row (a row takes ceil(deg / 4G) groups,
// at least one), which pays when rows are long compared with a group; the launcher picks the general
// stream otherwise.  The lane groups' sums are added when a row completes.  Cursors, metadata chunks
// and the weight ring are those of stream_rows_wide; the weights of a group are stored lane group by
// lane group (index PB g + b) so that a lane reads four of them with one 16-byte load.  kFull: the row has
// exactly LPR vectors, no lane needs masking.
template <typename T, int G, int NV, bool kFull, bool kPartial, bool kHalf = false>
__device__ __forceinline__ void stream_rows_multi(const SpmmDev& p, uint4* ring, float* wfifo, const float* ctab, int lane,
                                                  int64_t e0, int n_ent, int64_t warp_row0, int row_lo,
                                                  int row_hi, int rp_rel, float (&acc)[NV][Elt<T>::kPerVec])
{
    constexpr int LPR = kWarp / G;
    constexpr int EPV = Elt<T>::kPerVec;
    using P = Pipe<NV, LPR, true>;
    constexpr int PB = P::PB, NG = P::NG, EG = G * PB;        // positions and entries per group
    static_assert(PB % 4 == 0 && (NG & (NG - 1)) == 0, "float4 weight reads; power-of-two group ring");
    const int g = lane / LPR, l = lane % LPR;
    bool active[NV];
#pragma unroll
    for (int c = 0; c < NV; ++c) active[c] = (c * LPR + l) < p.nv;
    const int32_t* cols = p.colidx + e0;
    const float* vals = p.val + e0;
    auto load_col = [&](int e) { return e < n_ent ? __ldg(cols + e) : 0; };
    auto load_val = [&](int e) { return e < n_ent ? __ldg(vals + e) : 0.f; };
    auto load_nw = [&](int col) { return p.node_w ? __ldg(p.node_w + col) : 1.f; };
    auto row_end_of = [&](int r) { return kPartial ? n_ent : __shfl_sync(0xffffffffu, rp_rel, r + 1); };
    const uint4* ring_l = ring + lane;                        // this lane's 16 bytes of slot 0
    const uint32_t ring_sa = (uint32_t)__cvta_generic_to_shared(ring_l);
    const char* zeta_l = reinterpret_cast<const char*>(p.zeta + l);
    const uint32_t row_bytes = (uint32_t)p.nv * 16u;

    int a_col = load_col(lane), b_col = load_col(32 + lane), c_col = load_col(64 + lane), d_col = load_col(96 + lane);
    float a_w = load_val(lane), b_w = load_val(32 + lane), c_val = load_val(64 + lane), d_val = load_val(96 + lane);
    a_w *= load_nw(a_col);
    b_w *= load_nw(b_col);
    float c_nw = load_nw(c_col);
    int cbase = 0;                                            // first entry of chunk A

    int ie = 0, ir = row_lo, iend = row_end_of(row_lo);       // issue cursor: entry, row, end of that row
    int re = 0, rr = row_lo, rend = iend;                     // retire cursor
    bool more = row_lo < row_hi;
    int issued = 0, goff = 0;                                 // groups issued; ring position of the current group
    zero_acc<NV, EPV>(acc);
    float wsum = 0.f, wsgn = 0.f;                             // half-dot bytes: sum of the row's weights, plain and signed

    for (int it = 0;; ++it) {
        if (it >= NG) {
            if (it - NG >= issued) break;
            // ---- retire the oldest group
            cp_async_wait<NG - 1>();
            __syncwarp();
            const uint4* gp = ring_l + goff * (PB * 32 * NV);
            const int left = rend - re;
#pragma unroll
            for (int q = 0; q < PB / 4; ++q) {                // four positions at a time
                uint4 v[4][NV];
#pragma unroll
                for (int b = 0; b < 4; ++b)
#pragma unroll
                    for (int c = 0; c < NV; ++c) v[b][c] = gp[((4 * q + b) * NV + c) * 32];
                const float4 w4 = *reinterpret_cast<const float4*>(wfifo + goff * EG + PB * g + 4 * q);
                const float w[4] = {w4.x, w4.y, w4.z, w4.w};
                if (left >= EG) {
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const float wa = kHalf ? fabsf(w[b]) : w[b];      // the sign carries the source's first feature sign
                        if (kHalf) { wsum += wa; wsgn += w[b]; }
#pragma unroll
                        for (int c = 0; c < NV; ++c)
                            if (kFull || active[c]) fma_any<T>(wa, v[b][c], acc[c]);
                    }
                } else {
#pragma unroll
                    for (int b = 0; b < 4; ++b)
                        if (G * (4 * q + b) + g < left) {
                            const float wa = kHalf ? fabsf(w[b]) : w[b];
                            if (kHalf) { wsum += wa; wsgn += w[b]; }
#pragma unroll
                            for (int c = 0; c < NV; ++c)
                                if (kFull || active[c]) fma_any<T>(wa, v[b][c], acc[c]);
                        }
                }
            }
            re = left >= EG ? re + EG : rend;
            if (re == rend) {                                 // the row is complete
                reduce_groups<NV, EPV, LPR>(acc);
                if (kHalf) {
#pragma unroll
                    for (int o = LPR; o < kWarp; o <<= 1) {
                        wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
                        wsgn += __shfl_xor_sync(0xffffffffu, wsgn, o);
                    }
                }
                if (kPartial) {
                    if (kHalf) {                              // a slice of a long row: hand back the reconstructed partial sums
                        constexpr int kCols = NV * LPR * EPV;
#pragma unroll
                        for (int c = 0; c < NV; ++c)
#pragma unroll
                            for (int i = 0; i < EPV; ++i)
                                acc[c][i] = fmaf(2.f, acc[c][i], fmaf(ctab[3 * kCols + ctab_at<kCols, EPV>((c * LPR + l) * EPV + i)], wsgn, wsum));
                    }
                    return;
                }
                finish_row<T, NV, LPR, kHalf>(p, ctab, warp_row0 + rr, lane, acc, wsum, wsgn);
                zero_acc<NV, EPV>(acc);
                wsum = 0.f;
                wsgn = 0.f;
                ++rr;
                if (rr < row_hi) rend = row_end_of(rr);
            }
            __syncwarp();                                     // all lanes are done with these slots
        }
        if (more) {
            // ---- issue the next group of the row under the issue cursor
            const int left = iend - ie;
            const int base = ie - cbase;                      // position of the group in chunk A (< 32)
            const uint32_t dsta = ring_sa + goff * (PB * 512 * NV);
            // the window of the next 32 entries: lanes below `base` present their chunk-B entry, so
            // entry base + e sits in lane (base + e) % 32
            const int m_col = lane >= base ? a_col : b_col;
            const float m_w = lane >= base ? a_w : b_w;
            const int rel = (lane - base) & 31;               // entry of the window held by this lane
            const int cnt = min(EG, left);
            const int src_lane = base + g;                    // lane of the window that holds entry g of the group
            if (cnt == EG) {
#pragma unroll
                for (int b = 0; b < PB; ++b) {
                    const uint32_t k = (uint32_t)__shfl_sync(0xffffffffu, m_col, src_lane + G * b);
                    const char* src = zeta_l + (uint64_t)k * row_bytes;
#pragma unroll
                    for (int c = 0; c < NV; ++c)
                        if (kFull || active[c]) cp_async16_s(dsta + (b * NV + c) * 512, src + c * (LPR * 16));
                }
            } else {
#pragma unroll
                for (int b = 0; b < PB; ++b) {
                    const uint32_t k = (uint32_t)__shfl_sync(0xffffffffu, m_col, src_lane + G * b);
                    const char* src = zeta_l + (uint64_t)k * row_bytes;
                    if (G * b + g < cnt) {
#pragma unroll
                        for (int c = 0; c < NV; ++c)
                            if (kFull || active[c]) cp_async16_s(dsta + (b * NV + c) * 512, src + c * (LPR * 16));
                    }
                }
            }
            if (rel < cnt) wfifo[goff * EG + PB * (rel % G) + rel / G] = m_w;
            ie += cnt;
            ++issued;
            if (ie == iend) {
                ++ir;
                if (ir == row_hi) more = false;
                else iend = row_end_of(ir);
            }
            if (ie - cbase >= 32) {                           // rotate the metadata chunks
                a_col = b_col;
                a_w = b_w;
                b_col = c_col;
                b_w = c_val * c_nw;
                c_col = d_col;
                c_val = d_val;
                c_nw = load_nw(c_col);
                cbase += 32;
                d_col = load_col(cbase + 96 + lane);
                d_val = load_val(cbase + 96 + lane);
            }
        }
        cp_async_commit();                                    // one group per iteration, possibly empty
        goff = (goff + 1) & (NG - 1);
    }
    cp_async_wait<0>();
}

// ---- rows of signed bytes on the integer tensor-core path -------------------------------------------------------
//
// For 129..256 byte columns the aggregation of one output row, sum_e w_e s_e[j], is computed as exact integer
// products: within a segment of a row the weights are written in fixed point against a common power of two S
// (q_e = trunc(w_e 2^31 / S), |q_e| < 2^30, at least 29 significant bits for the largest weight of the segment's
// first window), q_e is split into four balanced base-256 digits, and a window of up to 32 stored entries of ONE row
// becomes one K = 32 step of mma.sync.m16n8k32 (s8 x s8 -> s32): the A operand holds 16 columns of the 32 gathered
// byte rows (16 instructions per window for 256 columns), columns 0..3 of the B operand hold the four digits of the
// 32 weights, columns 0..3 of the accumulator hold the four digit sums of the 16 columns.  When a row (or a segment) ends,
// the digit sums are recombined in fp32 and scaled by S 2^-31.  The gathered rows never pass through a byte -> float
// conversion: per stored entry the kernel issues about a third of the instructions of the FMA stream.
//
// The A fragment wants, in one register, the same column of four consecutive entries; the gathered rows sit in
// shared memory entry by entry, so a lane reads 16 columns of four entries (4 x 16 bytes) and transposes 4 x 4 bytes
// with byte permutes.  Which accumulator a column lands in is a fixed permutation that the recombination undoes.
// A window's slot holds 32 rows of 256 bytes; 16-byte chunk c of entry e sits at chunk c ^ (2 ((e / 4) % 4)), which
// makes both the asynchronous copies and the fragment reads free of bank conflicts.  A new segment starts with every
// row, when a window holds a weight too large for the current S, and every 2,048 windows (so that the 32-bit digit
// sums cannot overflow).
constexpr int kImmaWarps = 8;
constexpr int kImmaThreads = kImmaWarps * kWarp;
constexpr int kImmaNG = 3;                                    // windows in a warp's ring (two in flight while one retires)
constexpr int kWinData = 32 * 256;                            // gathered rows of a window
constexpr int kWinQ = kWinData;                               // uint32[32]: the digits of the window's weights
constexpr int kWinW = kWinData + 128;                         // float[2][32]: the weights, plain and with the first feature sign
constexpr int kWinInfo = kWinData + 384;                      // int4: descriptor, scale bits
constexpr int kWinBytes = kWinData + 384 + 32;
constexpr int kStagePitch = 324;                              // ints per digit in the recombination buffer (16 chunks of 20)
constexpr int kSegHeadroom = 2;                               // S = 2^(2+1) times the power of two below the first window's largest weight
constexpr int kSegMaxWindows = 2048;
enum : int { kWinCnt = 63, kWinLast = 64, kWinFirst = 128, kWinValid = 256, kWinSegEnd = 512 };

__device__ __forceinline__ void mma_s8_k32(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};\n"
        : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// out[c] = (r0.byte c, r1.byte c, r2.byte c, r3.byte c)
__device__ __forceinline__ void transpose_4x4_bytes(uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3, uint32_t* out)
{
    const uint32_t t0 = __byte_perm(r0, r1, 0x5140), t1 = __byte_perm(r2, r3, 0x5140);
    const uint32_t t2 = __byte_perm(r0, r1, 0x7362), t3 = __byte_perm(r2, r3, 0x7362);
    out[0] = __byte_perm(t0, t1, 0x5410);
    out[1] = __byte_perm(t0, t1, 0x7632);
    out[2] = __byte_perm(t2, t3, 0x5410);
    out[3] = __byte_perm(t2, t3, 0x7632);
}

// Streams the stored entries [e0, e0 + n_ent) of rows [row_lo, row_hi) (kPartial: a slice of one long row, whose
// sum is left in `accf`) through the warp's ring of windows.  Lane L ends up with columns 8 L .. 8 L + 7 of a row.
// Per iteration, oldest first: retire window it - 2 - NG (products, and the row epilogue where a row ends), issue
// the gathers of window it - 2 into the slot just freed, fetch the node factors of window it - 1, and lay out
// window `it` (its column indices and values).
template <bool kFull, bool kPartial, bool kHalf>
__device__ __forceinline__ void stream_rows_imma(const SpmmDev& p, unsigned char* ring, const float* ctab, int lane,
                                                 int64_t e0, int n_ent, int64_t warp_row0, int row_lo, int row_hi,
                                                 int rp_rel, float (&accf)[1][8])
{
    constexpr int NG = kImmaNG;
    const int g = lane >> 2, qq = lane & 3;                   // fragment coordinates
    const int h = lane >> 4, l = lane & 15;                   // gather coordinates: entry parity, 16-byte chunk
    const int32_t* cols = p.colidx + e0;
    const float* vals = p.val + e0;
    auto row_end_of = [&](int r) { return kPartial ? n_ent : __shfl_sync(0xffffffffu, rp_rel, r + 1); };
    const uint32_t ring_sa = (uint32_t)__cvta_generic_to_shared(ring);
    const char* zeta_l = reinterpret_cast<const char*>(p.zeta) + l * 16;
    const uint32_t row_bytes = (uint32_t)p.nv * 16u;
    const bool lact = kFull || l < p.nv;
    const uint32_t frag_off = (uint32_t)(4 * qq) * 256u + (uint32_t)((g ^ (2 * qq)) << 4);   // entry 4 qq, chunk g

    // layout cursor
    int ie = 0, ir = row_lo, iend = row_end_of(row_lo);
    bool ifirst = true, more = row_lo < row_hi;
    int nwin = 0;
    // windows between the stages
    int n_desc = 0, n_col = 0, i_desc = 0, i_col = 0;
    float n_val = 0.f, i_val = 0.f, i_nw = 1.f;
    // issue side: the current segment
    int es_lim = 0, seg_windows = 0;
    // retire side
    int rr = row_lo;
    int C[16][4];                                             // tile t: columns 16 x + t; [0], [1]: x = g, [2], [3]: x = g + 8
#pragma unroll
    for (int t = 0; t < 16; ++t) C[t][0] = C[t][1] = C[t][2] = C[t][3] = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) accf[0][i] = 0.f;
    float wsum = 0.f, wsgn = 0.f;

    for (int it = 0;; ++it) {
        const int kr = it - 2 - NG;
        if (!more && kr >= nwin) break;
        const int sl = it % NG;                               // slot retired and refilled in this iteration
        unsigned char* slot = ring + sl * kWinBytes;
        if (kr >= 0) {
            // ---- retire window kr
            cp_async_wait<NG - 1>();
            __syncwarp();
            const int2 info = *reinterpret_cast<const int2*>(slot + kWinInfo);
            uint32_t b_lo, b_hi;                              // B operand: column n = digit n of the 32 weights (n < 4)
            {
                const uint4 q0 = *reinterpret_cast<const uint4*>(slot + kWinQ + 16 * qq);
                const uint4 q1 = *reinterpret_cast<const uint4*>(slot + kWinQ + 64 + 16 * qq);
                const uint32_t sel = (uint32_t)(g & 3) | ((uint32_t)(4 + (g & 3)) << 4);   // digit g of two words
                b_lo = __byte_perm(__byte_perm(q0.x, q0.y, sel), __byte_perm(q0.z, q0.w, sel), 0x5410);
                b_hi = __byte_perm(__byte_perm(q1.x, q1.y, sel), __byte_perm(q1.z, q1.w, sel), 0x5410);
                if (g >= 4) b_lo = b_hi = 0u;
            }
            {
                // A operand (16 columns x 32 entries): row g = a column of chunk g, row g + 8 = a column of chunk g + 8
                uint4 r[2][2][4];                             // [chunk g / g + 8][entries 4 qq.. / 16 + 4 qq..][entry]
#pragma unroll
                for (int hx = 0; hx < 2; ++hx)
#pragma unroll
                    for (int kh = 0; kh < 2; ++kh)
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            r[hx][kh][j] = *reinterpret_cast<const uint4*>(slot + frag_off + hx * 128 + kh * 4096 + j * 256);
#pragma unroll
                for (int c = 0; c < 4; ++c) {                 // four columns of each chunk at a time
                    uint32_t a[2][2][4];
#pragma unroll
                    for (int hx = 0; hx < 2; ++hx)
#pragma unroll
                        for (int kh = 0; kh < 2; ++kh) {
                            const uint4* v = r[hx][kh];
                            if (c == 0) transpose_4x4_bytes(v[0].x, v[1].x, v[2].x, v[3].x, a[hx][kh]);
                            else if (c == 1) transpose_4x4_bytes(v[0].y, v[1].y, v[2].y, v[3].y, a[hx][kh]);
                            else if (c == 2) transpose_4x4_bytes(v[0].z, v[1].z, v[2].z, v[3].z, a[hx][kh]);
                            else transpose_4x4_bytes(v[0].w, v[1].w, v[2].w, v[3].w, a[hx][kh]);
                        }
#pragma unroll
                    for (int tt = 0; tt < 4; ++tt)
                        mma_s8_k32(C[4 * c + tt], a[0][0][tt], a[1][0][tt], a[0][1][tt], a[1][1][tt], b_lo, b_hi);
                }
            }
            if (kHalf) {
                const float* wf = reinterpret_cast<const float*>(slot + kWinW);
                wsum += wf[lane];
                wsgn += wf[32 + lane];
            }
            if (info.x & (kWinLast | kWinSegEnd)) {
                // ---- the segment ends: recombine the digit sums (through the window's data area, free now)
                __syncwarp();
                int* stage = reinterpret_cast<int*>(slot);
                if (qq < 2) {                                 // these lanes hold digits 2 qq and 2 qq + 1
#pragma unroll
                    for (int hx = 0; hx < 2; ++hx)
#pragma unroll
                        for (int b = 0; b < 2; ++b) {
                            int* dst = stage + (2 * qq + b) * kStagePitch + (g + 8 * hx) * 20;
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                *reinterpret_cast<int4*>(dst + 4 * i) =
                                    make_int4(C[4 * i][2 * hx + b], C[4 * i + 1][2 * hx + b], C[4 * i + 2][2 * hx + b], C[4 * i + 3][2 * hx + b]);
                        }
                }
                __syncwarp();
                const float scale = __int_as_float(info.y);
                const int* src = stage + (lane >> 1) * 20 + 8 * (lane & 1);
                int d[4][8];
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int4 u0 = *reinterpret_cast<const int4*>(src + k * kStagePitch);
                    const int4 u1 = *reinterpret_cast<const int4*>(src + k * kStagePitch + 4);
                    d[k][0] = u0.x, d[k][1] = u0.y, d[k][2] = u0.z, d[k][3] = u0.w;
                    d[k][4] = u1.x, d[k][5] = u1.y, d[k][6] = u1.z, d[k][7] = u1.w;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float f = fmaf((float)d[3][i], 16777216.f, (float)d[2][i] * 65536.f) + fmaf((float)d[1][i], 256.f, (float)d[0][i]);
                    accf[0][i] = fmaf(scale, f, accf[0][i]);
                }
#pragma unroll
                for (int t = 0; t < 16; ++t) C[t][0] = C[t][1] = C[t][2] = C[t][3] = 0;
                if (info.x & kWinLast) {                      // the row is complete
                    if (kHalf) {
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
                            wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
                            wsgn += __shfl_xor_sync(0xffffffffu, wsgn, o);
                        }
                    }
                    if (kPartial) {
                        if (kHalf) {                          // a slice of a long row: hand back the reconstructed partial sums
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                accf[0][i] = fmaf(2.f, accf[0][i], fmaf(ctab[3 * 256 + ctab_at<256, 8>(8 * lane + i)], wsgn, wsum));
                        }
                        return;
                    }
                    finish_row<__half, 1, 32, kHalf>(p, ctab, warp_row0 + rr, lane, accf, wsum, wsgn);
#pragma unroll
                    for (int i = 0; i < 8; ++i) accf[0][i] = 0.f;
                    wsum = 0.f;
                    wsgn = 0.f;
                    ++rr;
                }
            }
            __syncwarp();                                     // all lanes are done with this slot
        }
        if (i_desc & kWinValid) {
            // ---- issue window it - 2 into the slot: fixed-point weights, then the gathers
            const int cnt = i_desc & kWinCnt;
            const float wa = i_val * (kHalf ? fabsf(i_nw) : i_nw);            // the weight of the byte row
            const uint32_t mbits = __reduce_max_sync(0xffffffffu, __float_as_uint(fabsf(wa)));
            const int ew = (int)(mbits >> 23);                                // biased exponent of the window's largest weight
            const bool newseg = (i_desc & kWinFirst) || ew >= es_lim || seg_windows >= kSegMaxWindows;
            if (newseg) {
                es_lim = min(max(ew + kSegHeadroom, 31), 254);                // S = 2^(es_lim + 1 - 127)
                seg_windows = 0;
            }
            ++seg_windows;
            const float inv = __int_as_float((284 - es_lim) << 23);           // 2^31 / S
            const int q = __float2int_rz(wa * inv);                           // |q| < 2^30 (2^29 in a segment's first window)
            *reinterpret_cast<uint32_t*>(slot + kWinQ + 4 * lane) = ((uint32_t)q + 0x00808080u) ^ 0x00808080u;   // balanced digits
            if (kHalf) {
                float* wf = reinterpret_cast<float*>(slot + kWinW);
                wf[lane] = wa;
                wf[32 + lane] = i_val * i_nw;                                 // signed by the source's first feature sign
            }
            if (lane == 0) {
                *reinterpret_cast<int2*>(slot + kWinInfo) = make_int2(i_desc, (es_lim - 30) << 23);   // scale = S 2^-31
                if (newseg && !(i_desc & kWinFirst))                          // the window before this one closes its segment
                    *reinterpret_cast<int*>(ring + ((it + NG - 1) % NG) * kWinBytes + kWinInfo) |= kWinSegEnd;
            }
            const uint32_t dsta = ring_sa + sl * kWinBytes + (uint32_t)h * 256u;
            if (cnt == 32) {
#pragma unroll
                for (int b = 0; b < 16; ++b) {
                    const uint32_t k = (uint32_t)__shfl_sync(0xffffffffu, i_col, 2 * b + h);
                    if (lact) cp_async16_s(dsta + b * 512 + ((l ^ (((b >> 1) & 3) << 1)) << 4), zeta_l + (uint64_t)k * row_bytes);
                }
            } else {
#pragma unroll
                for (int b = 0; b < 16; ++b) {
                    const uint32_t k = (uint32_t)__shfl_sync(0xffffffffu, i_col, 2 * b + h);
                    if (lact && 2 * b + h < cnt) cp_async16_s(dsta + b * 512 + ((l ^ (((b >> 1) & 3) << 1)) << 4), zeta_l + (uint64_t)k * row_bytes);
                }
            }
        }
        cp_async_commit();                                    // one group per iteration, possibly empty
        // ---- the node factors of window it - 1
        i_desc = n_desc;
        i_col = n_col;
        i_val = n_val;
        i_nw = (p.node_w && (n_desc & kWinValid)) ? __ldg(p.node_w + n_col) : 1.f;
        // ---- lay out window `it`
        n_desc = 0;
        n_col = 0;
        n_val = 0.f;
        if (more) {
            const int left = iend - ie;
            const int cnt = min(32, left);
            n_desc = cnt | (cnt == left ? kWinLast : 0) | (ifirst ? kWinFirst : 0) | kWinValid;
            if (lane < cnt) {
                n_col = __ldg(cols + ie + lane);
                n_val = __ldg(vals + ie + lane);
            }
            ie += cnt;
            ifirst = false;
            ++nwin;
            if (ie == iend) {
                ifirst = true;
                ++ir;
                if (ir == row_hi) more = false;
                else iend = row_end_of(ir);
            }
        }
    }
    cp_async_wait<0>();
}

// The kernel around stream_rows_imma: the same hand-out of row runs and the same cooperative treatment of long
// rows as spmm_kernel.  One thread block of 8 warps per SM (the rings take most of the shared memory).
template <bool kFull, bool kHalf>
__global__ void __launch_bounds__(kImmaThreads, 1)
spmm_imma_kernel(const SpmmDev p, int rows_per_warp)
{
    constexpr int kCols = 256;
    extern __shared__ __align__(128) unsigned char dsmem[];
    __shared__ int64_t long_rows[kLongQueue];
    __shared__ int n_long;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    unsigned char* ring = dsmem + (size_t)warp * kImmaNG * kWinBytes;
    float* part = reinterpret_cast<float*>(dsmem);           // [kImmaWarps][kCols], reuses the rings
    float* ctab = reinterpret_cast<float*>(dsmem + (size_t)kImmaWarps * kImmaNG * kWinBytes);   // [4][kCols]
    fill_col_table<kCols, 8>(p, ctab);
    if (threadIdx.x == 0) n_long = 0;
    __syncthreads();

    const int64_t n_runs = ceil_div(p.n, rows_per_warp);
    float accf[1][8];
    for (;;) {
        int64_t run = 0;
        if (lane == 0) run = atomicAdd(p.run_counter, 1);
        run = __shfl_sync(0xffffffffu, run, 0);
        if (run >= n_runs) break;
        const int64_t warp_row0 = run * rows_per_warp;
        const int n_rows = (int)min((int64_t)rows_per_warp, p.n - warp_row0);
        const int64_t rp_reg = __ldg(p.rowptr + warp_row0 + min(lane, n_rows));
        const int64_t rp_next = __shfl_down_sync(0xffffffffu, rp_reg, 1);
        bool is_long = lane < n_rows && p.long_row > 0 && (rp_next - rp_reg) > p.long_row;
        if (is_long) {                                        // queue it for the block; if the queue is full, stream it here
            const int slot = atomicAdd(&n_long, 1);
            if (slot < kLongQueue) long_rows[slot] = warp_row0 + lane;
            else is_long = false;
        }
        const unsigned long_mask = __ballot_sync(0xffffffffu, is_long);
        int ra = 0;
        while (ra < n_rows) {                                 // runs of rows between the long ones
            const unsigned rest = long_mask >> ra;
            const int rl = rest ? ra + (__ffs(rest) - 1) : n_rows;
            if (rl > ra) {
                const int64_t e0 = __shfl_sync(0xffffffffu, rp_reg, ra);
                const int64_t e1 = __shfl_sync(0xffffffffu, rp_reg, rl);
                stream_rows_imma<kFull, false, kHalf>(p, ring, ctab, lane, e0, (int)(e1 - e0), warp_row0, ra, rl, (int)(rp_reg - e0), accf);
            }
            ra = rl + 1;
        }
    }
    __syncthreads();
    const int nl = min(n_long, kLongQueue);
    for (int q = 0; q < nl; ++q) {                            // long rows of this block, each by all warps together
        const int64_t lrow = long_rows[q];
        const int64_t ls = __ldg(p.rowptr + lrow), le = __ldg(p.rowptr + lrow + 1);
        const int64_t slice = round_up(ceil_div(le - ls, kImmaWarps), 32);
        const int64_t s0 = min(le, ls + warp * slice), s1 = min(le, s0 + slice);
        stream_rows_imma<kFull, true, kHalf>(p, ring, ctab, lane, s0, (int)(s1 - s0), 0, 0, 1, 0, accf);
        __syncthreads();                                      // every ring is idle: reuse them for the partial sums
#pragma unroll
        for (int i = 0; i < 8; ++i) part[warp * kCols + 8 * lane + i] = accf[0][i];
        __syncthreads();
        if (warp == 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                float t = 0.f;
                for (int w = 0; w < kImmaWarps; ++w) t += part[w * kCols + 8 * lane + i];
                accf[0][i] = t;
            }
            finish_row<__half, 1, 32>(p, ctab, lrow, lane, accf);
        }
        __syncthreads();
    }
}

template <bool kFull, bool kHalf>
cudaError_t launch_imma(cudaStream_t s, SpmmDev p)
{
    constexpr size_t smem = (size_t)kImmaWarps * kImmaNG * kWinBytes + 4 * 256 * sizeof(float);
    p.nv_fin = 2 * p.nv;                                      // the row epilogue works on groups of 8 columns
    const int rows_per_warp = (int)std::min<int64_t>(kMaxRowsPerWarp, std::max<int64_t>(1, p.n / (kImmaWarps * sm_count() * 8)));
    cudaError_t e = cudaFuncSetAttribute(spmm_imma_kernel<kFull, kHalf>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(p.run_counter, 0, sizeof(int), s);
    if (e != cudaSuccess) return e;
    const int64_t wanted = ceil_div(ceil_div(p.n, rows_per_warp), kImmaWarps);
    const unsigned grid = (unsigned)std::min<int64_t>(wanted, sm_count());
    spmm_imma_kernel<kFull, kHalf><<<grid, kImmaThreads, smem, s>>>(p, rows_per_warp);
    return cudaGetLastError();
}

// ---- narrow rows of signed bytes, one stored entry per lane ------------------------------------------------------
//
// For rows of 3 or 4 sixteen-byte vectors (33..64 byte columns): a network's last layer (fp32 out) or, with kNext,
// a hidden layer whose result is re-binarized for the next one (more columns do not fit: a lane holds 16 NV sums).  The streams above give a lane one vector of an entry, so a warp handles 8 entries per
// instruction and every row end costs a reduction over the lane groups; here a lane owns a whole stored entry:
// it loads the entry's column, value and node factor itself (no shuffles), fetches the NV vectors of the operand
// row straight into registers and accumulates all 16 NV columns.  A pass is up to 32 entries of one row; the
// passes of a run of rows form one stream (column indices two passes ahead, gathers one pass ahead), so that the
// latencies of a row's first pass hide behind the previous row.  When a row ends the 32 lanes' partial sums are
// added through a per-warp shared-memory buffer (a lane reads four columns of sixteen lanes, two half-sums meet
// by one shuffle) and lanes 0 .. 4 NV - 1 write four columns each.
constexpr int kLaneWarps = 8;
constexpr int kLaneThreads = kLaneWarps * kWarp;
constexpr int kLanePitch = 68;                                // floats per lane in the reduction buffer (64 + 4: 16-byte stores of 8 lanes fall into distinct banks)

// Streams rows [row_lo, row_hi) of a run (kPartial: the stored entries [e0, e0 + n_ent) as one row, whose sums are
// handed back in `out` / `wsum` / `wsgn` instead of being written).
// kTail: a row of zeta is 64 bytes, 32-byte aligned, and carries its node factor in its last four bytes: an entry's
// dots and factor come with one pair of 32-byte loads (two tag lookups per entry instead of NV + 1).
template <int NV, bool kHalf, bool kPartial, bool kTail = false, bool kNext = false>
__device__ __forceinline__ void stream_rows_lane(const SpmmDev& p, float* red, int lane, int64_t e0, int n_ent,
                                                 int64_t warp_row0, int row_lo, int row_hi, int rp_rel,
                                                 const float (&al)[4], const float (&b0)[4], float4& out, float& wsum_out, float& wsgn_out,
                                                 const float (&al2)[4], const float (&b02)[4])
{
    constexpr int NG4 = 4 * NV;                               // groups of four columns
    const int32_t* cols = p.colidx + e0;
    const float* vals = p.val + e0;
    const char* zeta = reinterpret_cast<const char*>(p.zeta);
    auto row_start = [&](int r) { return kPartial ? 0 : __shfl_sync(0xffffffffu, rp_rel, r); };
    auto row_end = [&](int r) { return kPartial ? n_ent : __shfl_sync(0xffffffffu, rp_rel, r + 1); };

    int ir = row_lo, io = 0;                                  // index cursor: row, offset of the next pass inside it
    auto fetch_indices = [&](int& c, float& w) {
        c = -1;
        w = 0.f;
        if (ir < row_hi) {
            const int rs = row_start(ir), re = row_end(ir);
            const int idx = rs + io + lane;
            if (idx < re) {
                c = __ldg(cols + idx);
                w = __ldg(vals + idx);
            }
            io += 32;
            if (rs + io >= re) {
                ++ir;
                io = 0;
            }
        }
    };
    uint4 vn[NV];
    float nwn = 1.f;
    auto gather = [&](int c) {
        if (c >= 0) {
            if constexpr (kTail) {
                const char* src = zeta + (uint64_t)(uint32_t)c * 64u;
                uint32_t w[16];
                asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n"
                             : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "l"(src));
                asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n"
                             : "=r"(w[8]), "=r"(w[9]), "=r"(w[10]), "=r"(w[11]), "=r"(w[12]), "=r"(w[13]), "=r"(w[14]), "=r"(w[15]) : "l"(src + 32));
#pragma unroll
                for (int q = 0; q < NV; ++q) vn[q] = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
                nwn = __uint_as_float(w[15]);
            } else {
                nwn = p.node_w ? __ldg(p.node_w + c) : 1.f;
                const uint4* src = reinterpret_cast<const uint4*>(zeta + (uint64_t)(uint32_t)c * (uint32_t)(NV * 16));
#pragma unroll
                for (int q = 0; q < NV; ++q) vn[q] = __ldg(src + q);
            }
        }
    };
    int c1, c2;
    float w1, w2;
#pragma unroll
    for (int q = 0; q < NV; ++q) vn[q] = make_uint4(0u, 0u, 0u, 0u);
    fetch_indices(c1, w1);
    fetch_indices(c2, w2);
    gather(c1);

    float acc[NV][16];
    zero_acc<NV, 16>(acc);
    float ws = 0.f, wg = 0.f;
    int cr = row_lo, co = 0;                                  // consume cursor
    while (cr < row_hi) {
        uint4 v[NV];
#pragma unroll
        for (int q = 0; q < NV; ++q) v[q] = vn[q];
        const float wt = c1 >= 0 ? w1 * nwn : 0.f;            // lanes past the row's end add nothing
        c1 = c2;
        w1 = w2;
        gather(c1);                                           // the next pass's operand rows
        fetch_indices(c2, w2);                                // the indices of the pass after that
        const float wa = kHalf ? fabsf(wt) : wt;              // half-dot bytes: the sign carries the source's first feature sign
        if (kHalf) { ws += wa; wg += wt; }
#pragma unroll
        for (int q = 0; q < NV; ++q) fma_bytes16(wa, v[q], acc[q]);
        const int rs = row_start(cr), re = row_end(cr);
        co += 32;
        if (!kPartial && rs + co >= re) {
            // ---- the row is complete: add the 32 lanes' sums in registers.  Five exchange steps, each halving what a
            // lane holds: a lane keeps the half of its columns that its bit of the lane index selects and sends the other
            // half to its partner (16 NV shuffles in all); afterwards lanes 2 j and 2 j + 1 both hold the totals of
            // columns 16 q + j, q < NV.  (Through shared memory the same reduction moved 12 KB per row, more than the
            // row's gathered operands, and kept the L1 data path, not the gathers, the busiest unit.)
            float x[NV];
#pragma unroll
            for (int q = 0; q < NV; ++q) {
                float t8[8], t4[4], t2[2];
                const bool h16 = (lane & 16) != 0, h8 = (lane & 8) != 0, h4 = (lane & 4) != 0, h2 = (lane & 2) != 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float send = h16 ? acc[q][i] : acc[q][8 + i], keep = h16 ? acc[q][8 + i] : acc[q][i];
                    t8[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float send = h8 ? t8[i] : t8[4 + i], keep = h8 ? t8[4 + i] : t8[i];
                    t4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
                }
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const float send = h4 ? t4[i] : t4[2 + i], keep = h4 ? t4[2 + i] : t4[i];
                    t2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
                }
                const float send = h2 ? t2[0] : t2[1], keep = h2 ? t2[1] : t2[0];
                const float t1 = keep + __shfl_xor_sync(0xffffffffu, send, 2);
                x[q] = t1 + __shfl_xor_sync(0xffffffffu, t1, 1);
            }
            if (kHalf) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    ws += __shfl_xor_sync(0xffffffffu, ws, o);
                    wg += __shfl_xor_sync(0xffffffffu, wg, o);
                }
            }
            const int j = lane >> 1;                          // this lane's column inside every group of 16
#pragma unroll
            for (int q = 0; q < NV; ++q) {
                if (kHalf) x[q] = fmaf(2.f, x[q], fmaf(b02[q], wg, ws));
                x[q] *= al2[q];
            }
            if ((!kNext || p.h_out) && (lane & 1) == 0) {
                float* dst = p.h_out + (warp_row0 + cr) * p.ldh + j;
#pragma unroll
                for (int q = 0; q < NV; ++q)
                    if (16 * q + j < p.d_out) dst[16 * q] = x[q];
            }
            if constexpr (kNext) {
                // ---- re-binarization for the next layer: the lanes 2 j and 2 j + 1 hold column 16 q + j; a packed word
                // wants column 32 w + l in lane l, i.e. group 2 w from lane 2 l for l < 16, group 2 w + 1 from lane
                // 2 (l - 16) otherwise: two shuffles and a ballot per word
                const int64_t row = warp_row0 + cr;
                float xh[NV], l1 = 0.f;
#pragma unroll
                for (int q = 0; q < NV; ++q) {
                    const int col = 16 * q + j;
                    const bool in = col < p.d_out;
                    const float sh = (in && p.next_shift) ? __ldg(p.next_shift + col) : 0.f;
                    const float sc = (in && p.next_shift) ? __ldg(p.next_scale + col) : 1.f;
                    xh[q] = in ? __fmul_rn(__fsub_rn(x[q], sh), sc) : -1.f;    // columns past d_out pack as 0
                    if (in && (lane & 1) == 0) l1 += fabsf(xh[q]);
                }
                const int src = 2 * (lane & 15);
#pragma unroll
                for (int w = 0; w < (NV + 1) / 2; ++w) {
                    const float a = __shfl_sync(0xffffffffu, xh[2 * w], src);
                    const float b = (2 * w + 1 < NV) ? __shfl_sync(0xffffffffu, xh[(2 * w + 1 < NV) ? 2 * w + 1 : 0], src) : -1.f;
                    const uint32_t word = __ballot_sync(0xffffffffu, (lane < 16 ? a : b) >= 0.f);
                    if (lane == 0 && w < p.next_stride) p.next_bits[row * p.next_stride + w] = word;
                }
                for (int w = (NV + 1) / 2 + lane; w < p.next_stride; w += 32) p.next_bits[row * p.next_stride + w] = 0u;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) l1 += __shfl_xor_sync(0xffffffffu, l1, o);
                if (lane == 0) p.next_beta[row] = l1 * p.inv_d_out;
            }
            zero_acc<NV, 16>(acc);
            ws = 0.f;
            wg = 0.f;
            ++cr;
            co = 0;
        } else if (kPartial && rs + co >= re) {
            // ---- a slice of a long row is complete: add the lanes' sums through shared memory and hand them back
            float* mine = red + lane * kLanePitch;
#pragma unroll
            for (int q = 0; q < NV; ++q)
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    *reinterpret_cast<float4*>(mine + 16 * q + 4 * i) = make_float4(acc[q][4 * i], acc[q][4 * i + 1], acc[q][4 * i + 2], acc[q][4 * i + 3]);
            __syncwarp();
            const int cg = lane % NG4, jh = lane / NG4;       // four columns, one half of the lanes (jh = 2: idle)
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (jh < 2) {
                const float* src = red + (16 * jh) * kLanePitch + 4 * cg;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float4 u = *reinterpret_cast<const float4*>(src + j * kLanePitch);
                    t.x += u.x, t.y += u.y, t.z += u.z, t.w += u.w;
                }
            }
            __syncwarp();
            t.x += __shfl_down_sync(0xffffffffu, t.x, NG4);
            t.y += __shfl_down_sync(0xffffffffu, t.y, NG4);
            t.z += __shfl_down_sync(0xffffffffu, t.z, NG4);
            t.w += __shfl_down_sync(0xffffffffu, t.w, NG4);
            if (kHalf) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    ws += __shfl_xor_sync(0xffffffffu, ws, o);
                    wg += __shfl_xor_sync(0xffffffffu, wg, o);
                }
            }
            out = t;
            wsum_out = ws;
            wsgn_out = wg;
            return;
        }
    }
    if (kPartial) {                                           // empty slice
        out = make_float4(0.f, 0.f, 0.f, 0.f);
        wsum_out = 0.f;
        wsgn_out = 0.f;
    }
}

template <int NV, bool kHalf, bool kTail = false, bool kNext = false>
__global__ void __launch_bounds__(kLaneThreads, 2)
spmm_lane_kernel(const SpmmDev p, int rows_per_warp)
{
    constexpr int NG4 = 4 * NV;
    extern __shared__ __align__(16) float lsm[];
    __shared__ int64_t long_rows[kLongQueue];
    __shared__ int n_long;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    float* red = lsm + (size_t)warp * 32 * kLanePitch;
    float* part = lsm + (size_t)kLaneWarps * 32 * kLanePitch;       // [kLaneWarps][NG4 * 4 + 4]: slices of a long row
    constexpr int kPartPitch = NG4 * 4 + 4;
    const int cg = lane % NG4;
    float al[4], b0[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int col = 4 * cg + i;
        const bool in = lane < NG4 && col < p.d_out;
        al[i] = in ? (p.col_w ? __ldg(p.col_w + col) : 1.f) : 0.f;
        b0[i] = (in && kHalf && p.col_b0) ? __ldg(p.col_b0 + col) : 0.f;
    }
    float al2[4], b02[4];                                     // the same constants for the columns 16 q + lane / 2 (rows finished in registers)
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const int col = 16 * q + (lane >> 1);
        const bool in = q < NV && col < p.d_out;
        al2[q] = in ? (p.col_w ? __ldg(p.col_w + col) : 1.f) : 0.f;
        b02[q] = (in && kHalf && p.col_b0) ? __ldg(p.col_b0 + col) : 0.f;
    }
    if (threadIdx.x == 0) n_long = 0;
    __syncthreads();

    const int64_t n_runs = ceil_div(p.n, rows_per_warp);
    float4 t;
    float ws, wg;
    for (;;) {
        int64_t run = 0;
        if (lane == 0) run = atomicAdd(p.run_counter, 1);
        run = __shfl_sync(0xffffffffu, run, 0);
        if (run >= n_runs) break;
        const int64_t warp_row0 = run * rows_per_warp;
        const int n_rows = (int)min((int64_t)rows_per_warp, p.n - warp_row0);
        const int64_t rp_reg = __ldg(p.rowptr + warp_row0 + min(lane, n_rows));
        const int64_t rp_next = __shfl_down_sync(0xffffffffu, rp_reg, 1);
        bool is_long = lane < n_rows && p.long_row > 0 && (rp_next - rp_reg) > p.long_row;
        if (is_long) {                                        // queue it for the block; if the queue is full, stream it here
            const int slot = atomicAdd(&n_long, 1);
            if (slot < kLongQueue) long_rows[slot] = warp_row0 + lane;
            else is_long = false;
        }
        const unsigned long_mask = __ballot_sync(0xffffffffu, is_long);
        int ra = 0;
        while (ra < n_rows) {                                 // runs of rows between the long ones
            const unsigned rest = long_mask >> ra;
            const int rl = rest ? ra + (__ffs(rest) - 1) : n_rows;
            if (rl > ra) {
                const int64_t e0 = __shfl_sync(0xffffffffu, rp_reg, ra);
                stream_rows_lane<NV, kHalf, false, kTail, kNext>(p, red, lane, e0, 0, warp_row0, ra, rl, (int)(rp_reg - e0), al, b0, t, ws, wg, al2, b02);
            }
            ra = rl + 1;
        }
    }
    __syncthreads();
    const int nl = min(n_long, kLongQueue);
    for (int q = 0; q < nl; ++q) {                            // long rows of this block, each by all warps together
        const int64_t lrow = long_rows[q];
        const int64_t ls = __ldg(p.rowptr + lrow), le = __ldg(p.rowptr + lrow + 1);
        const int64_t slice = round_up(ceil_div(le - ls, kLaneWarps), 32);
        const int64_t s0 = min(le, ls + warp * slice), s1 = min(le, s0 + slice);
        stream_rows_lane<NV, kHalf, true, kTail>(p, red, lane, s0, (int)(s1 - s0), 0, 0, (s1 > s0) ? 1 : 0, 0, al, b0, t, ws, wg, al2, b02);
        if (lane < NG4) *reinterpret_cast<float4*>(part + warp * kPartPitch + 4 * cg) = t;
        if (lane == 0) {
            part[warp * kPartPitch + NG4 * 4] = ws;
            part[warp * kPartPitch + NG4 * 4 + 1] = wg;
        }
        __syncthreads();
        if (warp == 0) {
            float x[4] = {0.f, 0.f, 0.f, 0.f};
            float sws = 0.f, swg = 0.f;
            if (lane < NG4) {
                for (int w = 0; w < kLaneWarps; ++w) {
                    const float4 u = *reinterpret_cast<const float4*>(part + w * kPartPitch + 4 * cg);
                    x[0] += u.x, x[1] += u.y, x[2] += u.z, x[3] += u.w;
                    sws += part[w * kPartPitch + NG4 * 4];
                    swg += part[w * kPartPitch + NG4 * 4 + 1];
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (kHalf) x[i] = fmaf(2.f, x[i], fmaf(b0[i], swg, sws));
                    x[i] *= al[i];
                    if ((!kNext || p.h_out) && 4 * cg + i < p.d_out) p.h_out[lrow * p.ldh + 4 * cg + i] = x[i];
                }
            }
            if constexpr (kNext) {                            // lane l < NG4 holds columns 4 l .. 4 l + 3: eight lanes per packed word
                uint32_t bits = 0u;
                float l1 = 0.f;
                if (lane < NG4) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int col = 4 * lane + i;
                        if (col < p.d_out) {
                            const float sh = p.next_shift ? __ldg(p.next_shift + col) : 0.f;
                            const float sc = p.next_shift ? __ldg(p.next_scale + col) : 1.f;
                            const float xh = __fmul_rn(__fsub_rn(x[i], sh), sc);
                            if (xh >= 0.f) bits |= 1u << i;
                            l1 += fabsf(xh);
                        }
                    }
                }
                uint32_t word = bits << ((4 * lane) & 31);
#pragma unroll
                for (int o = 1; o < 8; o <<= 1) word |= __shfl_xor_sync(0xffffffffu, word, o);
                if ((lane & 7) == 0 && lane < NG4 && (lane >> 3) < p.next_stride) p.next_bits[lrow * p.next_stride + (lane >> 3)] = word;
                for (int w = (NV + 1) / 2 + lane; w < p.next_stride; w += 32) p.next_bits[lrow * p.next_stride + w] = 0u;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) l1 += __shfl_xor_sync(0xffffffffu, l1, o);
                if (lane == 0) p.next_beta[lrow] = l1 * p.inv_d_out;
            }
        }
        __syncthreads();
    }
}

template <int NV, bool kHalf, bool kTail = false, bool kNext = false>
cudaError_t launch_lane(cudaStream_t s, const SpmmDev& p)
{
    constexpr size_t smem = ((size_t)kLaneWarps * 32 * kLanePitch + (size_t)kLaneWarps * (NV * 16 + 4)) * sizeof(float);
    const int rows_per_warp = (int)std::min<int64_t>(kMaxRowsPerWarp, std::max<int64_t>(1, p.n / (kLaneWarps * sm_count() * 8)));
    cudaError_t e = cudaFuncSetAttribute(spmm_lane_kernel<NV, kHalf, kTail, kNext>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(p.run_counter, 0, sizeof(int), s);
    if (e != cudaSuccess) return e;
    const int64_t wanted = ceil_div(ceil_div(p.n, rows_per_warp), kLaneWarps);
    const unsigned grid = (unsigned)std::min<int64_t>(wanted, sm_count() * 2);
    spmm_lane_kernel<NV, kHalf, kTail, kNext><<<grid, kLaneThreads, smem, s>>>(p, rows_per_warp);
    return cudaGetLastError();
}

// Thread blocks per SM the kernel is compiled for (register budget) and launched with (grid size).
template <int NCH, int LPR, bool kAligned, int kEltBytes>
constexpr int spmm_blocks_per_sm()
{
    // (a lane of the general stream holds 16 accumulators for byte rows, 4 or 8 otherwise)
    return NCH == 1 ? ((LPR == 32 || kAligned || kEltBytes == 1) ? 3 : 4) : (NCH == 2 ? 2 : 1);
}

// kAligned (rows of 8 or 16 vectors only): the row-aligned multi-entry stream instead of the general one.
// kHalf: half-dot bytes (rows of signed bytes; either stream).
template <typename T, int NCH, int LPR, bool kFull, bool kAligned, bool kHalf = false>
__global__ void __launch_bounds__(kSpmmThreads, spmm_blocks_per_sm<NCH, LPR, kAligned, (int)sizeof(T)>())
spmm_kernel(const SpmmDev p, int rows_per_warp)
{
    static_assert(!kHalf || (sizeof(T) == 1 && LPR < 32), "half-dot bytes: rows of up to 256 signed bytes");
    static_assert(!kAligned || ((NCH == 1 || NCH == 2) && (LPR == 4 || LPR == 8 || LPR == 16)), "the multi-entry stream: 4, 8 or 16 lanes per row, one or two vectors per lane");
    using P = Pipe<NCH, LPR, kAligned>;
    constexpr int EPV = Elt<T>::kPerVec;
    constexpr int G = P::G;
    constexpr int kCols = NCH * (LPR < 32 ? LPR : 32) * EPV;  // accumulator columns of one warp
    extern __shared__ __align__(128) unsigned char dsmem[];
    __shared__ int64_t long_rows[kLongQueue];
    __shared__ int n_long;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    uint4* ring = reinterpret_cast<uint4*>(dsmem + (size_t)warp * P::RING * NCH * 512);
    float* wfifo = reinterpret_cast<float*>(dsmem + (size_t)kSpmmWarps * P::RING * NCH * 512) + warp * P::RING * G;
    float* part = reinterpret_cast<float*>(dsmem);           // [kSpmmWarps][kCols], reuses the rings (see below)
    static_assert((size_t)kSpmmWarps * kCols * 4 <= (size_t)kSpmmWarps * P::RING * NCH * 512, "partials must fit the rings");
    float* ctab = reinterpret_cast<float*>(dsmem + (size_t)kSpmmWarps * P::kWarpBytes);   // [3][kCols]
    fill_col_table<kCols, EPV>(p, ctab);
    if (threadIdx.x == 0) n_long = 0;
    __syncthreads();

    const int64_t n_runs = ceil_div(p.n, rows_per_warp);
    float acc[NCH][EPV];
    for (;;) {
        int64_t run = 0;
        if (lane == 0) run = atomicAdd(p.run_counter, 1);
        run = __shfl_sync(0xffffffffu, run, 0);
        if (run >= n_runs) break;
        const int64_t warp_row0 = run * rows_per_warp;
        const int n_rows = (int)min((int64_t)rows_per_warp, p.n - warp_row0);
        const int64_t rp_reg = __ldg(p.rowptr + warp_row0 + min(lane, n_rows));
        const int64_t rp_next = __shfl_down_sync(0xffffffffu, rp_reg, 1);
        bool is_long = lane < n_rows && p.long_row > 0 && (rp_next - rp_reg) > p.long_row;
        if (is_long) {                                        // queue it for the block; if the queue is full, stream it here
            const int slot = atomicAdd(&n_long, 1);
            if (slot < kLongQueue) long_rows[slot] = warp_row0 + lane;
            else is_long = false;
        }
        const unsigned long_mask = __ballot_sync(0xffffffffu, is_long);
        int ra = 0;
        while (ra < n_rows) {                                 // runs of rows between the long ones
            const unsigned rest = long_mask >> ra;
            const int rl = rest ? ra + (__ffs(rest) - 1) : n_rows;
            if (rl > ra) {
                const int64_t e0 = __shfl_sync(0xffffffffu, rp_reg, ra);
                const int64_t e1 = __shfl_sync(0xffffffffu, rp_reg, rl);
                if constexpr (LPR == 32)
                    stream_rows_wide<T, NCH, kFull, false>(p, ring, wfifo, ctab, lane, e0, (int)(e1 - e0), warp_row0, ra, rl,
                                                    (int)(rp_reg - e0), acc);
                else if constexpr (kAligned)
                    stream_rows_multi<T, kWarp / LPR, NCH, kFull, false, kHalf>(p, ring, wfifo, ctab, lane, e0, (int)(e1 - e0), warp_row0, ra, rl,
                                                                    (int)(rp_reg - e0), acc);
                else
                    stream_entries<T, NCH, LPR, false, kHalf>(p, ring, wfifo, ctab, lane, e0, (int)(e1 - e0), warp_row0, ra, rl,
                                                       (int)(rp_reg - e0), acc);
            }
            ra = rl + 1;
        }
    }
    __syncthreads();
    const int nl = min(n_long, kLongQueue);
    // Long rows of this block, one after the other, each by all warps together.
    for (int q = 0; q < nl; ++q) {
        const int64_t lrow = long_rows[q];
        const int64_t ls = __ldg(p.rowptr + lrow), le = __ldg(p.rowptr + lrow + 1);
        const int64_t slice = round_up(ceil_div(le - ls, kSpmmWarps), 32);
        const int64_t s0 = min(le, ls + warp * slice), s1 = min(le, s0 + slice);
        if constexpr (LPR == 32)
            stream_rows_wide<T, NCH, kFull, true>(p, ring, wfifo, ctab, lane, s0, (int)(s1 - s0), 0, 0, 1, 0, acc);
        else if constexpr (kAligned)
            stream_rows_multi<T, kWarp / LPR, NCH, kFull, true, kHalf>(p, ring, wfifo, ctab, lane, s0, (int)(s1 - s0), 0, 0, 1, 0, acc);
        else
            stream_entries<T, NCH, LPR, true, kHalf>(p, ring, wfifo, ctab, lane, s0, (int)(s1 - s0), 0, 0, 1, 0, acc);
        __syncthreads();                                      // every ring is idle: reuse them for the partial sums
        const int l = lane % LPR;
        if (lane < LPR) {
#pragma unroll
            for (int c = 0; c < NCH; ++c)
#pragma unroll
                for (int i = 0; i < EPV; ++i) part[warp * kCols + (c * (LPR < 32 ? LPR : 32) + l) * EPV + i] = acc[c][i];
        }
        __syncthreads();
        if (warp == 0) {
#pragma unroll
            for (int c = 0; c < NCH; ++c)
#pragma unroll
                for (int i = 0; i < EPV; ++i) {
                    float t = 0.f;
                    for (int w = 0; w < kSpmmWarps; ++w) t += part[w * kCols + (c * (LPR < 32 ? LPR : 32) + l) * EPV + i];
                    acc[c][i] = t;
                }
            finish_row<T, NCH, LPR>(p, ctab, lrow, lane, acc);
        }
        __syncthreads();
    }
}

template <typename T, int NCH, int LPR, bool kFull = false, bool kAligned = false, bool kHalf = false>
cudaError_t launch_one(cudaStream_t s, const SpmmDev& p)
{
    constexpr int kCols = NCH * (LPR < 32 ? LPR : 32) * Elt<T>::kPerVec;
    constexpr size_t smem = kSpmmWarps * Pipe<NCH, LPR, kAligned>::kWarpBytes + 4 * kCols * sizeof(float);   // rings, weights, column table
    // enough thread blocks to fill the machine on small graphs, long runs of rows on large ones
    const int rows_per_warp = (int)std::min<int64_t>(kMaxRowsPerWarp, std::max<int64_t>(1, p.n / (kSpmmWarps * sm_count() * 8)));
    if (smem > 40 * 1024) {                                   // above the default limit: opt in
        cudaError_t e = cudaFuncSetAttribute(spmm_kernel<T, NCH, LPR, kFull, kAligned, kHalf>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    cudaError_t e = cudaMemsetAsync(p.run_counter, 0, sizeof(int), s);
    if (e != cudaSuccess) return e;
    // one wave of resident blocks; the warps pull runs of rows until none are left
    const int64_t wanted = ceil_div(ceil_div(p.n, rows_per_warp), kSpmmWarps);
    const unsigned grid = (unsigned)std::min<int64_t>(wanted, sm_count() * spmm_blocks_per_sm<NCH, LPR, kAligned, (int)sizeof(T)>());
    spmm_kernel<T, NCH, LPR, kFull, kAligned, kHalf><<<grid, kSpmmThreads, smem, s>>>(p, rows_per_warp);
    return cudaGetLastError();
}

// mean_row: stored entries per row (0 = unknown).  256-byte rows of signed bytes take the row-aligned
// multi-entry stream (the general stream has no fast unpack for bytes) unless the rows are known to be
// much shorter than its groups of 8 entries.  For 2- and 4-byte elements in rows of 8 or 16 vectors the
// aligned stream was measured level with the general one at best (c5, 96-byte rows: 3.80 vs 3.72 ms; at
// full size those gathers are bound by DRAM access rate, not by instructions), so they keep the general one.
template <typename T>
cudaError_t dispatch(cudaStream_t s, const SpmmDev& p, double mean_row)
{
    const int nv = p.nv;
    if constexpr (sizeof(T) == 1) {
        // 33..64 byte columns, written out as fp32 (a last layer) or re-binarized (a hidden layer), rows not much
        // shorter than a pass: one entry per lane
        if ((nv == 3 || nv == 4) && (p.h_out || p.next_bits) && !p.add && p.byte_path != 2 && !(mean_row > 0.0 && mean_row < 8.0)) {
            if (p.next_bits) {
                if (p.row_tail && nv == 4) {
                    const bool three = p.d_out <= 48;
                    if (p.half_dots) return three ? launch_lane<3, true, true, true>(s, p) : launch_lane<4, true, true, true>(s, p);
                    return three ? launch_lane<3, false, true, true>(s, p) : launch_lane<4, false, true, true>(s, p);
                }
                if (p.half_dots) return nv == 3 ? launch_lane<3, true, false, true>(s, p) : launch_lane<4, true, false, true>(s, p);
                return nv == 3 ? launch_lane<3, false, false, true>(s, p) : launch_lane<4, false, false, true>(s, p);
            }
            if (p.row_tail && nv == 4) {                      // 64-byte rows that carry their node factor: 3 or 4 vectors of columns
                const bool three = p.d_out <= 48;
                if (p.half_dots) return three ? launch_lane<3, true, true>(s, p) : launch_lane<4, true, true>(s, p);
                return three ? launch_lane<3, false, true>(s, p) : launch_lane<4, false, true>(s, p);
            }
            if (p.half_dots) return nv == 3 ? launch_lane<3, true>(s, p) : launch_lane<4, true>(s, p);
            return nv == 3 ? launch_lane<3, false>(s, p) : launch_lane<4, false>(s, p);
        }
        if (p.half_dots && nv <= 8) {                         // narrow rows of half-dot bytes
            if (nv <= 1) return launch_one<T, 1, 1, false, false, true>(s, p);
            if (nv <= 2) return launch_one<T, 1, 2, false, false, true>(s, p);
            // rows of 3..8 vectors: the row-aligned stream (8 or 4 entries per position, groups of 32 or 16 entries)
            // unless the rows are known to be much shorter than a group
            const bool short_rows = mean_row > 0.0 && mean_row < 8.0;
            if (nv <= 4) {
                if (short_rows) return launch_one<T, 1, 4, false, false, true>(s, p);
                return nv == 4 ? launch_one<T, 1, 4, true, true, true>(s, p) : launch_one<T, 1, 4, false, true, true>(s, p);
            }
            if (short_rows) return launch_one<T, 1, 8, false, false, true>(s, p);
            return nv == 8 ? launch_one<T, 1, 8, true, true, true>(s, p) : launch_one<T, 1, 8, false, true, true>(s, p);
        }
    }
    if (nv <= 1) return launch_one<T, 1, 1>(s, p);
    if (nv <= 2) return launch_one<T, 1, 2>(s, p);
    if (nv <= 4) return launch_one<T, 1, 4>(s, p);
    if (nv <= 8) return launch_one<T, 1, 8>(s, p);
    if (nv <= 16) {
        if constexpr (sizeof(T) == 1) {
            if (nv > 8 && p.byte_path == 2) {                  // integer tensor-core products
                if (p.half_dots) return nv == 16 ? launch_imma<true, true>(s, p) : launch_imma<false, true>(s, p);
                return nv == 16 ? launch_imma<true, false>(s, p) : launch_imma<false, false>(s, p);
            }
            if (p.half_dots) return nv == 16 ? launch_one<T, 1, 16, true, true, true>(s, p) : launch_one<T, 1, 16, false, true, true>(s, p);
            // (8 lanes per row with two vectors each, four entries per position -- launch_one<T, 2, 8, .., true> -- halves
            // the bookkeeping per entry again but needs 123 registers: 7.7 ms against 6.4 ms on c5 layer 0; not used)
            if (!(mean_row > 0.0 && mean_row < 8.0))
                return nv == 16 ? launch_one<T, 1, 16, true, true>(s, p) : launch_one<T, 1, 16, false, true>(s, p);
        }
        return launch_one<T, 1, 16>(s, p);
    }
    if (nv == 32) return launch_one<T, 1, 32, true>(s, p);
    if (nv <= 32) return launch_one<T, 1, 32>(s, p);
    // wider rows: up to 512 columns in any format (128 / 64 / 32 vectors of 4- / 2- / 1-byte elements)
    if constexpr (sizeof(T) >= 2) {
        if (nv <= 64) return launch_one<T, 2, 32>(s, p);
    }
    if constexpr (sizeof(T) == 4) {
        if (nv <= 128) return launch_one<T, 4, 32>(s, p);
    }
    return cudaErrorInvalidConfiguration;
}

}  // namespace

size_t spmm_scratch_bytes(int64_t, int64_t, int) { return 256; }

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
    p.nv_fin = p.nv;
    p.d_out = a.d_out;
    p.node_w = a.fmt == kZetaF32 ? nullptr : a.node_w;
    p.col_w = a.fmt == kZetaF32 ? nullptr : a.col_w;
    p.add = a.add;
    p.col_b0 = a.half_dots ? a.col_b0 : nullptr;
    p.half_dots = a.half_dots ? 1 : 0;
    p.byte_path = a.byte_path;
    p.row_tail = (a.row_tail && a.fmt == kZetaI8 && a.ldz == 64 && a.d_out <= 60) ? 1 : 0;
    if (a.half_dots && (a.fmt != kZetaI8 || p.nv > 16 || !a.col_b0 || !a.node_w)) return cudaErrorInvalidValue;   // up to 256 byte columns
    p.ld_add = a.ld_add;
    p.h_out = a.h_out;
    p.ldh = a.ldh;
    p.h_vec = (a.h_out && (a.ldh % 4 == 0) && (reinterpret_cast<uintptr_t>(a.h_out) % 16 == 0)) ? 1 : 0;
    p.next_bits = a.next_bits;
    p.next_stride = a.next_stride;
    p.next_beta = a.next_beta;
    p.next_shift = a.next_shift;
    p.next_scale = a.next_scale;
    p.long_row = a.long_row;
    p.covered_words = (int)ceil_div(a.ldz, 32);
    p.inv_d_out = 1.f / (float)a.d_out;
    if (!a.scratch || a.scratch_bytes < sizeof(int)) return cudaErrorInvalidValue;
    p.run_counter = static_cast<int*>(a.scratch);
    ++*launches;
    const double mean_row = (a.nnz > 0 && a.n > 0) ? (double)a.nnz / (double)a.n : 0.0;
    // rows of 129..256 signed bytes as tcgen05 integer products (a block's rows must hold fewer than 2^31 entries): when
    // asked for, and by default where that kernel measured faster than the FMA stream -- a hidden layer of which only
    // the sign bits and beta are wanted, on a graph whose rows are not much shorter than its chunks' eight segments allow
    const bool tc_default = a.byte_path == 0 && a.next_bits && !a.h_out && !a.add && mean_row >= 8.0;
    if (a.fmt == kZetaI8 && (a.byte_path == 3 || tc_default) && a.nnz > 0 && a.nnz < (int64_t(1) << 31) && spmm_tc_covers(p)) return launch_spmm_tc(s, p);
    switch (a.fmt) {
        case kZetaF32: return dispatch<float>(s, p, mean_row);
        case kZetaF16: return dispatch<__half>(s, p, mean_row);
        case kZetaI16: return dispatch<int16_t>(s, p, mean_row);
        case kZetaI8: return dispatch<int8_t>(s, p, mean_row);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace bigcn
