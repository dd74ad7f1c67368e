// Aggregation H' = A_tilde zeta (Bi-GCN, last equation of Sec. 4.2.3) for rows of 129..256 signed bytes, with the sum
// over a row's stored entries taken as exact integer products on the 5th-generation tensor cores, and the
// re-binarization of H' for the next layer (Sec. 4.2.2 after the batch-norm constants of Sec. 4.4) in the epilogue.
//
// Why.  The fp32 FMA stream (spmm.cu) turns every gathered byte into a float and multiplies it on the fp32 pipe:
// about 38 warp instructions per stored entry, which bounds it below the rate at which the rows can be fetched.
// Here a gathered row never passes through a register.  The rows of a chunk of 64 stored entries are copied
// (cp.async, 16 bytes per lane) straight into shared memory in the layout the tensor core reads as the A operand:
// M = 128 output columns x K = 64 entries, M-major (an entry's 128 bytes are contiguous), 128-byte swizzle; two such
// operands cover 256 columns.  The B operand holds the chunk's edge weights: weight e of row segment s (the part of
// one output row that falls into the chunk; at most 8 per chunk) is written in fixed point against a power of two
// S_s above the segment's largest weight, q_e = round(w_e 2^30 / S_s), split into four balanced base-256 digits that
// fill columns 4 s .. 4 s + 3 of row e; all other columns of that row are 0.  One tcgen05.mma.kind::i8 per operand and
// K = 32 step (N = 32) leaves in tensor memory, for every output column (a lane) and segment, the four digit sums
// sum_e digit_d(q_e) zeta_e,col: exact integers.  They are read back once per segment (tcgen05.ld, four registers),
// recombined in fp32 (sum_d 256^d . S_s 2^-30) and added to the row's fp32 accumulator; when a row ends, the
// thread that owns a column scales it by alpha, stores it and takes part in the packing of sign bits and beta.
// The error this adds to the fp32 sum is at most 2^-31 S_s sum_e |zeta_e| per segment (S_s < 2 max_e |w_e|).
//
// Who does what.  A block is 4 consumer warps, 1 producer warp and 1 issuer warp.  The rows are split over the blocks once, by
// cost (stored entries plus a constant per row).  The producer streams its block's row offsets, column indices, edge
// values and per-source factors (beta_k, with the first feature sign for half-dot bytes) through shared-memory rings
// with asynchronous copies issued several loop iterations ahead, cuts the entries into chunks, derives the segment
// scales, digits and -- for half-dot bytes -- the per-segment weight sums (as exact integer sums of the q_e, so that
// they match the products digit for digit), and publishes a chunk slot.  The consumers (a thread owns one
// tensor-memory lane = output columns t and 128 + t) copy the rows of chunk i + 2 into the operand stage the products
// of chunk i have released -- the copies report to the stage's mbarrier when they have landed, nobody waits for them
// but the issuer -- and read back chunk i; the issuer's one thread issues the products of a chunk as soon as it is
// published, its rows have landed and its accumulator stage has been read back.
// Two operand stages (32 KB), two accumulator stages (128 tensor-memory columns), four chunk slots per block; four
// blocks per multiprocessor (what bounds the kernel is the latency of each block's chain of dependent steps per chunk,
// so the number of blocks that fit counts for more than the depth of one block's pipeline).
// Hand-offs.  Between warps -- chunk published (producer -> consumers, producer -> issuer), chunk read back (consumers
// -> producer), accumulator stage read back (consumers -> issuer) -- through named barriers: the side that hands over
// arrives, the side that takes over syncs (15 of the block's 16 barriers; a hop measured 50 cycles against 190 through
// an mbarrier).  Where an asynchronous unit reports -- the row copies, tcgen05.commit -- through mbarriers, and every
// wait on those is bounded: if one runs out the block raises a flag (reported by bigcn_sync_check) and from then on
// every role only passes its barriers, without copies' results or products, until the stream of chunks has ended;
// nobody is left waiting, the tensor memory is freed.
#include <algorithm>
#include <cstddef>

#include "bigcn_internal.cuh"
#include "spmm_dev.cuh"
#include "tc_common.cuh"

namespace bigcn {

namespace {

constexpr int kConsumers = 128;                 // 4 consumer warps: thread = tensor-memory lane = output columns lane and 128 + lane
constexpr int kThreads = kConsumers + 64;       // + the producer warp and the issuer warp
constexpr int kChunk = 64;                      // stored entries per chunk: two K = 32 steps
constexpr int kSegMax = 8;                      // row segments per chunk, four digit columns each
constexpr int kN = 4 * kSegMax;                 // N of the instruction
constexpr int kEntRing = 512;                   // producer's ring of stored entries (column, value, factor): 2 kLag + 1 blocks of 64 and slack
constexpr int kRowRing = 128;                   // producer's ring of row offsets
constexpr int kLag = 3;                         // producer loop iterations between issuing a copy and using its data
constexpr int kSlots = 4;                       // chunk slots in flight between producer and consumers
constexpr int kAStages = 2;
constexpr int kAStageBytes = kChunk * 256;      // two operands of 64 entries x 128 bytes
constexpr int kBSlotBytes = kChunk * kN;        // 64 entries x 32 digit columns
constexpr int kTmemCols = 128;                  // 2 accumulator stages x 2 operands x N = 32 columns
constexpr int kEbitsMin = 40, kEbitsMax = 253;  // clamp of the scale's biased exponent (keeps 2^30 / S and S 2^-30 normal floats)

constexpr int kTries = 1 << 20;                 // bound of every mbarrier wait: tries of up to kSuspendNs each
constexpr uint32_t kSuspendNs = 1000;

__device__ int g_spmm_tc_timeout;               // set when a wait ran out

using tc::smem_u32;

struct SegRec {                                 // one row segment of a chunk
    float scale;                                // S_s 2^-30
    float wsum, wsgn;                           // half-dot bytes: sum of the segment's weights, plain and signed by the sources' first feature sign
    int32_t row_done;                           // the output row if it ends with this segment, else -1
};
struct ChunkSlot {
    int32_t cols[kChunk];                       // source node of every entry
    SegRec seg[kSegMax];
    int32_t n_ent;                              // entries in the chunk (0..64); -1 = end of the stream
    int32_t nseg;
    int32_t pad[14];
};
static_assert(sizeof(ChunkSlot) == 448 && offsetof(ChunkSlot, seg) % 16 == 0, "slot size");

// dynamic shared memory, relative to a 1024-byte aligned base
constexpr int kOffA = 0;
constexpr int kOffB = kOffA + kAStages * kAStageBytes;
constexpr int kOffSlots = kOffB + kSlots * kBSlotBytes;
constexpr int kOffBetaPart = kOffSlots + kSlots * (int)sizeof(ChunkSlot);          // float [4][kSegMax][4]: per chunk (index & 3) and segment, one partial sum per consumer warp
constexpr int kOffBetaRow = kOffBetaPart + 4 * kSegMax * 4 * 4;                    // int [4][kSegMax]: the row that ended with the segment, or -1; [4]: segments of the chunk
constexpr int kOffEntRing = kOffBetaRow + 4 * kSegMax * 4 + 16;                         // producer: int32 / float / float [kEntRing]
constexpr int kOffRowRing = kOffEntRing + 3 * kEntRing * 4;                        // producer: int64 [kRowRing]
constexpr int kOffBars = kOffRowRing + kRowRing * 8;                               // uint64 mbarriers: products done [2], rows landed [kAStages]
constexpr int kOffMisc = kOffBars + (2 + kAStages) * 8;               // uint32 tmem base, int abort
constexpr int kSmemBytes = kOffMisc + 16 + 1024;                                   // + slack for the alignment

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
// Bounded wait that also gives up when another thread of the block has raised `abort`.  No sleep between tries: the
// try itself parks the thread (measured: next to no failed tries), and every sleep added to it showed up in the chain
// of hand-offs that bounds the kernel.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort)
{
    uint32_t done = 0;
    for (int it = 0; it < kTries && !done; ++it) {
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\nselp.u32 %0, 1, 0, p;\n}\n"
                     : "=r"(done) : "r"(smem_u32(bar)), "r"(parity), "r"(kSuspendNs) : "memory");   // the thread may be parked for up to the hint
        if (done || *abort) break;
    }
    if (!done) {
        atomicExch(&g_spmm_tc_timeout, 1);
        *abort = 1;
    }
    return done != 0;
}
// Hand-offs between the roles go through named barriers (a round trip through two of them was measured at 100 cycles,
// through two mbarriers at 350-400): the side that hands over arrives, the side that takes over syncs; `count` is the
// number of threads of both sides.  Whole warps execute these.
constexpr int kBarPR = 2, kBarPI = 2 + kSlots, kBarRP = 2 + 2 * kSlots, kBarRI = 2 + 3 * kSlots;   // + slot, + slot, + slot, + stage
static_assert(kBarRI + 2 <= 16, "named barriers");
__device__ __forceinline__ void bar_arrive(int id, int count)
{
    asm volatile("barrier.cta.arrive.aligned %0, %1;\n" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_sync(int id, int count)
{
    asm volatile("barrier.cta.sync.aligned %0, %1;\n" ::"r"(id), "r"(count) : "memory");
}
// All consumers meet; returns the OR of their `bad` flags.
__device__ __forceinline__ bool consumers_sync_or(bool bad)
{
    uint32_t r;
    asm volatile("{\n.reg .pred p, q;\nsetp.ne.u32 q, %1, 0;\nbarrier.cta.red.or.pred p, 1, %2, q;\nselp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(r) : "r"((uint32_t)bad), "n"(kConsumers) : "memory");
    return r != 0;
}
__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_dst), "l"(gmem_src) : "memory");
}
// shared-memory matrix descriptor with a layout type (0 = no swizzle, 2 = 128-byte swizzle)
__device__ __forceinline__ uint64_t make_desc_l(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout)
{
    return tc::make_desc(saddr, lbo_bytes, sbo_bytes) | ((uint64_t)layout << 61);
}

// ---- the producer warp ---------------------------------------------------------------------------------------------

// The rows of the matrix are split over the blocks once, by position in a cost scale on which a row counts its stored
// entries plus kRowCost (the row epilogue): block b takes the rows whose cost offsets fall into the b-th of gridDim.x
// equal parts.  Returns the first row whose offset reaches `target` (32 probes per step, all lanes).
constexpr int kRowCost = 8;
__device__ __forceinline__ int64_t first_row_at_cost(const SpmmDev& p, int64_t target, int lane)
{
    int64_t lo = 0, hi = p.n;                                 // answer in [lo, hi]; cost(hi) >= target or hi == n
    while (hi - lo > 0) {
        const int64_t span = hi - lo;
        const int64_t probe = lo + (span * (lane + 1)) / 33;  // lo <= probe <= hi, non-decreasing in lane, probe < hi when span >= 1
        const bool ge = __ldg(p.rowptr + probe) + kRowCost * probe >= target;
        const unsigned m = __ballot_sync(0xffffffffu, ge);
        const int first = m ? __ffs(m) - 1 : 32;              // first lane whose probe is at or above the target
        const int64_t new_hi = first < 32 ? __shfl_sync(0xffffffffu, probe, first) : hi;
        const int64_t new_lo = first > 0 ? __shfl_sync(0xffffffffu, probe, first - 1) + 1 : lo;
        lo = new_lo;
        hi = new_hi;
    }
    return lo;
}

__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}
__device__ __forceinline__ void cp_async8(void* smem_dst, const void* gmem_src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;\n" ::"r"(smem_u32(smem_dst)), "l"(gmem_src) : "memory");
}

// The producer streams its block's part of the matrix -- row offsets, column indices, edge values, and the
// per-source factors the column indices point at -- through rings in shared memory with asynchronous copies issued
// kLag loop iterations before their data is used (the factors are a dependent fetch: their copies are issued once the
// column indices have landed, and used kLag iterations after that).  Every iteration issues at most one block of
// 64 entries of each kind, commits one copy group, and cuts and publishes at most one chunk.
template <bool kHalf>
__device__ __forceinline__ void producer(const SpmmDev& p, unsigned char* sm, volatile int* abort)
{
    const int lane = threadIdx.x & 31;
    int32_t* col_ring = reinterpret_cast<int32_t*>(sm + kOffEntRing);
    float* val_ring = reinterpret_cast<float*>(sm + kOffEntRing + kEntRing * 4);
    float* nw_ring = reinterpret_cast<float*>(sm + kOffEntRing + kEntRing * 8);
    int64_t* row_ring = reinterpret_cast<int64_t*>(sm + kOffRowRing);

    // this block's rows [R0, R1) and stored entries [E0, E0 + total)
    const int64_t cost_all = __ldg(p.rowptr + p.n) + kRowCost * p.n;
    const int64_t R0 = first_row_at_cost(p, (cost_all * blockIdx.x) / gridDim.x, lane);
    const int64_t R1 = blockIdx.x + 1 == gridDim.x ? p.n : first_row_at_cost(p, (cost_all * (blockIdx.x + 1)) / gridDim.x, lane);
    const int nrows = (int)(R1 - R0);
    const int64_t E0 = __ldg(p.rowptr + R0);
    const int total = (int)(__ldg(p.rowptr + R1) - E0);

    int r = 0, e = 0;                                         // the cutter: next row, next entry (relative to R0, E0)
    int ci = 0, ni = 0, ri = 0;                               // entries / rows whose copies have been issued (blocks of 64 / 16)
    int ci_h[kLag], ni_h[kLag], ri_h[kLag];                   // the same counters after each of the last kLag iterations
#pragma unroll
    for (int q = 0; q < kLag; ++q) ci_h[q] = ni_h[q] = ri_h[q] = 0;

    for (uint32_t k = 0;;) {                                  // k: chunks published so far
        asm volatile("cp.async.wait_group %0;\n" ::"n"(kLag - 1) : "memory");
        __syncwarp();
        const int ci_done = ci_h[kLag - 1], ni_done = ni_h[kLag - 1], ri_done = ri_h[kLag - 1];
        // ---- issue: column indices and values of the next block of entries
        if (ci < total && ci + 64 <= e + kEntRing) {
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int x = ci + 32 * h + lane;
                if (x < total) {
                    cp_async4(col_ring + (x % kEntRing), p.colidx + E0 + x);
                    cp_async4(val_ring + (x % kEntRing), p.val + E0 + x);
                }
            }
            ci += 64;
        }
        // ---- issue: the factors of a block whose column indices have landed
        if (ni < ci_done) {
            if (p.node_w) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int x = ni + 32 * h + lane;
                    if (x < total) cp_async4(nw_ring + (x % kEntRing), p.node_w + col_ring[x % kEntRing]);
                }
            }
            ni += 64;
        }
        // ---- issue: row offsets
        if (ri <= nrows && ri + 16 <= r + kRowRing) {
            const int j = ri + lane;
            if (lane < 16 && j <= nrows) cp_async8(row_ring + (j % kRowRing), p.rowptr + R0 + j);
            ri += 16;
        }
        asm volatile("cp.async.commit_group;\n" ::: "memory");
#pragma unroll
        for (int q = kLag - 1; q > 0; --q) { ci_h[q] = ci_h[q - 1]; ni_h[q] = ni_h[q - 1]; ri_h[q] = ri_h[q - 1]; }
        ci_h[0] = ci; ni_h[0] = ni; ri_h[0] = ri;

        // ---- cut the next chunk if everything it can touch has landed
        const bool finished = r == nrows;
        if (!finished && !(min(r + kSegMax + 1, nrows + 1) <= ri_done && min(e + kChunk, total) <= ni_done)) continue;
        const int slot_i = (int)(k % kSlots);
        if (k >= kSlots) bar_sync(kBarRP + slot_i, kConsumers + 32);      // the consumers have read chunk k - kSlots
        ChunkSlot* slot = reinterpret_cast<ChunkSlot*>(sm + kOffSlots) + slot_i;
        unsigned char* Bs = sm + kOffB + slot_i * kBSlotBytes;
        if (finished) {                                       // end of the stream
            if (lane == 0) slot->n_ent = -1;
            __syncwarp();
            bar_arrive(kBarPR + slot_i, kConsumers + 32);
            bar_arrive(kBarPI + slot_i, 64);
            break;
        }
        // segments: the rows r .. r + 7 as far as they start before the chunk's end (or are empty and sit at it)
        const int rp_rel = (lane <= kSegMax && r + lane <= nrows) ? (int)(row_ring[(r + lane) % kRowRing] - E0) : 0x7fffffff;
        const int row_hi = min(r + kSegMax, nrows);
        const int e_cap = min(e + kChunk, __shfl_sync(0xffffffffu, rp_rel, row_hi - r));
        const int a = rp_rel, b = __shfl_down_sync(0xffffffffu, rp_rel, 1);
        const bool in_run = lane < kSegMax && r + lane < nrows;
        const bool part = in_run && (a < e_cap || b <= e_cap);
        const bool last = part && b <= e_cap;
        const int nseg = __popc(__ballot_sync(0xffffffffu, part));
        const int seg_end = part ? (min(b, e_cap) - e) : 255;
        const int seg_row = (int)(R0 + r + lane);
        const int n_ent = e_cap - e;
        // the chunk's entries: two per lane
        const bool in_a = lane < n_ent, in_b = 32 + lane < n_ent;
        const int xa = (e + lane) % kEntRing, xb = (e + 32 + lane) % kEntRing;
        const int col_a = in_a ? col_ring[xa] : 0, col_b = in_b ? col_ring[xb] : 0;
        const float val_a = in_a ? val_ring[xa] : 0.f, val_b = in_b ? val_ring[xb] : 0.f;
        const float nw_a = (in_a && p.node_w) ? nw_ring[xa] : 1.f, nw_b = (in_b && p.node_w) ? nw_ring[xb] : 1.f;
        r += __popc(__ballot_sync(0xffffffffu, last));
        e = e_cap;

        const float w_a = in_a ? val_a * nw_a : 0.f, w_b = in_b ? val_b * nw_b : 0.f;
        // the segment of each of the two entries: how many segments end at or before it
        int sid_a = 0, sid_b = 0;
        for (int s = 0; s < nseg; ++s) {
            const int end_s = __shfl_sync(0xffffffffu, seg_end, s);
            sid_a += lane >= end_s;
            sid_b += 32 + lane >= end_s;
        }
        // per segment: the largest |w| (as float bits: order-preserving for non-negative floats) -> the scale's exponent
        const uint32_t m_a = __float_as_uint(fabsf(w_a)), m_b = __float_as_uint(fabsf(w_b));
        int eb_a = kEbitsMin, eb_b = kEbitsMin, eb_mine = kEbitsMin;
        for (int s = 0; s < nseg; ++s) {
            const uint32_t m = __reduce_max_sync(0xffffffffu, max(sid_a == s ? m_a : 0u, sid_b == s ? m_b : 0u));
            const int eb = min(max((int)(m >> 23), kEbitsMin), kEbitsMax);
            if (sid_a == s) eb_a = eb;
            if (sid_b == s) eb_b = eb;
            if (lane == s) eb_mine = eb;
        }
        // S = 2^(eb + 1 - 127) > |w|; q = round(w 2^30 / S), |q| <= 2^30
        const float f_a = __uint_as_float((uint32_t)(283 - eb_a) << 23), f_b = __uint_as_float((uint32_t)(283 - eb_b) << 23);
        // half-dot bytes: the factor's sign is the source's first feature sign, not part of the weight
        const float u_a = kHalf ? val_a * fabsf(nw_a) : w_a, u_b = kHalf ? val_b * fabsf(nw_b) : w_b;
        const int q_a = in_a ? __float2int_rn(u_a * f_a) : 0, q_b = in_b ? __float2int_rn(u_b * f_b) : 0;
        // four balanced base-256 digits of q, one per byte
        const uint32_t dg_a = ((uint32_t)q_a + 0x80808080u) ^ 0x80808080u, dg_b = ((uint32_t)q_b + 0x80808080u) ^ 0x80808080u;
        // row e of the B operand: 32 digit columns = two 16-byte lines (N-major, no swizzle: line l of entry e at e * 16 + l * 1024)
        for (int l = 0; l < (nseg > 4 ? 2 : 1); ++l) {
            const int wa = (sid_a >> 2) == l ? (sid_a & 3) : -1, wb = (sid_b >> 2) == l ? (sid_b & 3) : -1;
            const uint4 va = make_uint4(wa == 0 ? dg_a : 0u, wa == 1 ? dg_a : 0u, wa == 2 ? dg_a : 0u, wa == 3 ? dg_a : 0u);
            const uint4 vb = make_uint4(wb == 0 ? dg_b : 0u, wb == 1 ? dg_b : 0u, wb == 2 ? dg_b : 0u, wb == 3 ? dg_b : 0u);
            *reinterpret_cast<uint4*>(Bs + lane * 16 + l * 1024) = va;
            *reinterpret_cast<uint4*>(Bs + (32 + lane) * 16 + l * 1024) = vb;
        }
        slot->cols[lane] = col_a;
        slot->cols[32 + lane] = col_b;
        float my_wsum = 0.f, my_wsgn = 0.f;
        const float my_scale = __uint_as_float((uint32_t)(eb_mine + 1 - 30) << 23);   // S 2^-30
        if constexpr (kHalf) {
            // sum_e q_e and sum_e sign_e q_e per segment, exactly, as two 16-bit halves each
            const int g_a = nw_a < 0.f ? -q_a : q_a, g_b = nw_b < 0.f ? -q_b : q_b;
            for (int s = 0; s < nseg; ++s) {
                const int lo = (sid_a == s ? (q_a & 0xffff) : 0) + (sid_b == s ? (q_b & 0xffff) : 0);
                const int hi = (sid_a == s ? (q_a >> 16) : 0) + (sid_b == s ? (q_b >> 16) : 0);
                const int glo = (sid_a == s ? (g_a & 0xffff) : 0) + (sid_b == s ? (g_b & 0xffff) : 0);
                const int ghi = (sid_a == s ? (g_a >> 16) : 0) + (sid_b == s ? (g_b >> 16) : 0);
                const int tlo = __reduce_add_sync(0xffffffffu, lo), thi = __reduce_add_sync(0xffffffffu, hi);
                const int tglo = __reduce_add_sync(0xffffffffu, glo), tghi = __reduce_add_sync(0xffffffffu, ghi);
                if (lane == s) {
                    my_wsum = fmaf((float)thi, 65536.f, (float)tlo) * my_scale;
                    my_wsgn = fmaf((float)tghi, 65536.f, (float)tglo) * my_scale;
                }
            }
        }
        if (lane < kSegMax)
            *reinterpret_cast<float4*>(&slot->seg[lane]) = make_float4(my_scale, my_wsum, my_wsgn, __int_as_float(last ? seg_row : -1));
        if (lane == 0) {
            slot->n_ent = n_ent;
            slot->nseg = nseg;
        }
        tc::fence_async_smem();                               // the digits are read by the tensor core (async proxy)
        __syncwarp();
        bar_arrive(kBarPR + slot_i, kConsumers + 32);
        bar_arrive(kBarPI + slot_i, 64);
        ++k;
    }
    asm volatile("cp.async.wait_all;\n" ::: "memory");
}

// ---- the issuer warp: products ------------------------------------------------------------------------------------

// Lane 0 polls, every lane gets the outcome.
__device__ __forceinline__ bool wait_bcast(uint64_t* bar, uint32_t parity, volatile int* abort, int lane)
{
    int ok = 1;
    if (lane == 0) ok = mbar_wait(bar, parity, abort) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// Chunk after chunk: once the chunk is published, its rows have landed (the consumers' copies report to the stage's
// mbarrier) and its accumulator stage has been read back (chunk c - 2), one thread issues the products.  The warp
// then finishes beta of the rows that ended in chunk c - 2, whose read-back it has just waited for: the four consumer
// warps' partial sums, in warp order (the partials sit in four buffers, chunk index & 3, so that the consumers, who
// cannot be more than two chunks ahead of this warp, never write the one being read here).
__device__ __forceinline__ void issuer(const SpmmDev& p, unsigned char* sm, volatile int* abort, uint32_t tmem_base)
{
    const int lane = threadIdx.x & 31;
    const float* beta_part = reinterpret_cast<const float*>(sm + kOffBetaPart);
    const int* beta_row = reinterpret_cast<const int*>(sm + kOffBetaRow);
    auto finish_beta = [&](uint32_t d) {
        if (!p.next_bits || *abort) return;
        const int bq = (int)(d & 3u);
        if (lane < beta_row[4 * kSegMax + bq]) {
            const int row = beta_row[bq * kSegMax + lane];
            if (row >= 0) {
                const float4 bp = *reinterpret_cast<const float4*>(beta_part + (bq * kSegMax + lane) * 4);
                p.next_beta[row] = (((bp.x + bp.y) + bp.z) + bp.w) * p.inv_d_out;
            }
        }
    };
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + kOffBars);
    uint64_t* mma_done = bars;
    uint64_t* a_full = bars + 2;
    const ChunkSlot* slots = reinterpret_cast<const ChunkSlot*>(sm + kOffSlots);
    const uint32_t a_base = smem_u32(sm + kOffA), b_base = smem_u32(sm + kOffB);
    // instruction descriptor: D = s32, A = B = s8, both M/N-major, N = 32, M = 128
    const uint32_t idesc0 = (2u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(128 >> 4) << 24);
    for (uint32_t c = 0;; ++c) {
        bar_sync(kBarPI + (int)(c % kSlots), 64);             // chunk c is published
        const ChunkSlot* slot = slots + (c % kSlots);
        const int n_ent = slot->n_ent;
        if (n_ent < 0) {                                      // end of the stream: the last two chunks' rows
            for (uint32_t d = c >= 2 ? c - 2 : 0; d < c; ++d) {
                bar_sync(kBarRI + (int)(d & 1u), kConsumers + 32);
                finish_beta(d);
            }
            return;
        }
        // a wait that runs out raises the block's flag; every role then keeps passing its barriers without work
        wait_bcast(&a_full[c % kAStages], (c / kAStages) & 1u, abort, lane);
        if (c >= 2) bar_sync(kBarRI + (int)(c & 1u), kConsumers + 32);     // the accumulator stage has been read back
        if (lane == 0) {
            tc::fence_async_smem();                           // the copied rows become visible to the tensor core
            tc::fence_after_sync();
            const int ksteps = max(1, (n_ent + 31) >> 5);
            const uint32_t idesc = idesc0 | ((uint32_t)((slot->nseg > 4 ? 32 : 16) >> 3) << 17);
            const uint32_t a_stage = a_base + (c % kAStages) * kAStageBytes;
            const uint32_t b_slot = b_base + (c % kSlots) * kBSlotBytes;
            for (int hh = 0; hh < 2; ++hh)
                for (int ks = 0; ks < ksteps; ++ks) {
                    const uint64_t ad = make_desc_l(a_stage + hh * 8192 + ks * 4096, 8192, 1024, 2);
                    const uint64_t bd = make_desc_l(b_slot + ks * 512, 128, 1024, 0);
                    const uint32_t d_addr = tmem_base + (c & 1u) * 64u + (uint32_t)(hh * 32);
                    const uint32_t accum = ks > 0 ? 1u : 0u;
                    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n}\n"
                                 ::"r"(d_addr), "l"(ad), "l"(bd), "r"(idesc), "r"(accum) : "memory");
                }
            tc::commit_to(&mma_done[c & 1u]);
        }
        __syncwarp();
        if (c >= 2) finish_beta(c - 2);
    }
}

// ---- the consumer warps --------------------------------------------------------------------------------------------

// One segment's four digit sums -> sum_e q_e zeta_e: the two low and the two high digits are combined as integers
// (|digit sum| <= 64 * 128 * 128 = 2^20, so each pair fits 32 bits), then two conversions and one FMA.
__device__ __forceinline__ float digits_to_float(uint32_t d0, uint32_t d1, uint32_t d2, uint32_t d3)
{
    const int lo = (int)d0 + ((int)d1 << 8), hi = (int)d2 + ((int)d3 << 8);
    return fmaf((float)hi, 65536.f, (float)lo);
}

// kBitsOnly: the launch wants only the next layer's sign bits and beta (no fp32 output, nothing added to the rows)
// kFull: rows of exactly 256 bytes, all of them columns (no piece of a row and no column needs a test)
template <bool kHalf, bool kBitsOnly, bool kFull>
__device__ __forceinline__ void consumers(const SpmmDev& p, unsigned char* sm, volatile int* abort, uint32_t tmem_base)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;      // warp = tensor-memory lane quarter
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + kOffBars);
    uint64_t* mma_done = bars;
    uint64_t* a_full = bars + 2;
    ChunkSlot* slots = reinterpret_cast<ChunkSlot*>(sm + kOffSlots);
    float* beta_part = reinterpret_cast<float*>(sm + kOffBetaPart);
    int* beta_row = reinterpret_cast<int*>(sm + kOffBetaRow);
    const uint32_t a_base = smem_u32(sm + kOffA);

    // per-column constants of the row epilogue: this thread owns columns tid (operand 0) and 128 + tid (operand 1)
    float alpha[2], shift[2], scale[2], b0[2];
    bool col_in[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int col = 128 * h + tid;
        col_in[h] = kFull || col < p.d_out;
        alpha[h] = col_in[h] ? (p.col_w ? __ldg(p.col_w + col) : 1.f) : 0.f;
        shift[h] = (col_in[h] && p.next_shift) ? __ldg(p.next_shift + col) : 0.f;
        scale[h] = (col_in[h] && p.next_shift) ? __ldg(p.next_scale + col) : 1.f;
        b0[h] = (kHalf && col_in[h] && p.col_b0) ? __ldg(p.col_b0 + col) : 0.f;
    }

    const char* zeta_b = reinterpret_cast<const char*>(p.zeta);
    const uint32_t row_bytes = (uint32_t)p.nv * 16u;
    const int sub = lane >> 3, piece = lane & 7;              // a warp instruction copies 4 entries x 128 contiguous bytes
    const bool lo_in = kFull || piece < p.nv, hi_in = kFull || 8 + piece < p.nv;   // this lane's 16-byte piece exists in operand 0 / 1
    const char* zeta_l = zeta_b + piece * 16;
    uint32_t dst_off[4];                                      // where this lane's piece of entry 16 warp + 4 g + sub goes inside a stage
#pragma unroll
    for (int g = 0; g < 4; ++g) {
        const int j = 16 * warp + 4 * g + sub;
        dst_off[g] = (uint32_t)(j * 128 + ((piece ^ (j & 7)) * 16));
    }
    // copies of chunk c into operand stage c % kAStages: warp w takes the entries 16 w .. 16 w + 15, both operands; they
    // report to the stage's mbarrier when they have landed.  (Chunk counters are 32-bit: a block sees far fewer than 2^31.)
    auto gather = [&](uint32_t c) {
        const ChunkSlot* slot = slots + (c % kSlots);
        const int n_ent = slot->n_ent;
        const uint32_t stage = a_base + (c % kAStages) * kAStageBytes;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const int j = 16 * warp + 4 * g + sub;
            if (j < n_ent) {
                const char* src = zeta_l + (uint64_t)(uint32_t)slot->cols[j] * row_bytes;
                if (lo_in) cp_async16(stage + dst_off[g], src);
                if (hi_in) cp_async16(stage + dst_off[g] + 8192, src + 128);
            }
        }
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(smem_u32(&a_full[c % kAStages])) : "memory");
    };

    uint32_t end_idx = 0xffffffffu;                           // index of the end marker once seen
    bool bad = false;
    // prologue: the rows of the first kAStages chunks (only one thread polls; the others wait at the named barrier)
    for (uint32_t c = 0; c < kAStages && end_idx == 0xffffffffu && !bad; ++c) {
        bar_sync(kBarPR + (int)(c % kSlots), kConsumers + 32);
        if (slots[c % kSlots].n_ent < 0) end_idx = c;
        else gather(c);
    }

    float acc[2] = {0.f, 0.f};                                // the open row: this thread's two column sums
    float rs = 0.f, rg = 0.f;                                 // and the row's weight sums (half-dot bytes)
    for (uint32_t i = 0;; ++i) {
        const bool has_cur = i < end_idx, need_next = end_idx == 0xffffffffu;
        if (need_next) bar_sync(kBarPR + (int)((i + kAStages) % kSlots), kConsumers + 32);   // chunk i + kAStages is published
        if (tid == 0 && has_cur && !mbar_wait(&mma_done[i & 1u], (i >> 1) & 1u, abort)) bad = true;
        tc::fence_before_sync();
        bad = consumers_sync_or(bad || *abort != 0);          // from here on the block only passes its barriers
        tc::fence_after_sync();
        if (!has_cur) break;
        // the rows of chunk i + kAStages go into the stage the products of chunk i have just released
        if (need_next) {
            if (slots[(i + kAStages) % kSlots].n_ent < 0) end_idx = i + kAStages;
            else gather(i + kAStages);
        }
        // read back chunk i: the four digit sums of every segment, both operands
        const ChunkSlot* slot = slots + (i % kSlots);
        const int par = (int)(i & 1u);
        const int nseg = bad ? 0 : slot->nseg;
        const int bq = (int)(i & 3u);                         // beta partials of this chunk: finished by the issuer warp
        if (tid == 0) beta_row[4 * kSegMax + bq] = nseg;
        const uint32_t t_addr = tmem_base + ((uint32_t)(32 * warp) << 16) + (uint32_t)(par * 64);
        for (int s = 0; s < nseg; ++s) {                       // a run-time loop (uniform over the readers): small code, the same for every segment
            int row_done = -1;
            {
                uint32_t a0, a1, a2, a3, c0, c1, c2, c3;
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];\n"
                             : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(t_addr + 4 * s) : "memory");
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];\n"
                             : "=r"(c0), "=r"(c1), "=r"(c2), "=r"(c3) : "r"(t_addr + 32 + 4 * s) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
                const float4 rec = *reinterpret_cast<const float4*>(&slot->seg[s]);
                acc[0] = fmaf(digits_to_float(a0, a1, a2, a3), rec.x, acc[0]);
                acc[1] = fmaf(digits_to_float(c0, c1, c2, c3), rec.x, acc[1]);
                if constexpr (kHalf) {
                    rs += rec.y;
                    rg += rec.z;
                }
                row_done = __float_as_int(rec.w);
            }
            if (tid == 0) beta_row[bq * kSegMax + s] = row_done;
            if (row_done >= 0) {
                const int64_t row = row_done;
                float l1 = 0.f;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float t = acc[h];
                    if constexpr (kHalf) t = fmaf(2.f, t, fmaf(b0[h], rg, rs));   // sum_k w_k dot_kj = 2 acc_j + wsum + b0_j wsgn
                    float x = t * alpha[h];
                    const int col = 128 * h + tid;
                    if constexpr (!kBitsOnly) {
                        if (p.add && col_in[h]) x += __ldg(p.add + row * p.ld_add + col);
                        if (p.h_out && col_in[h]) p.h_out[row * p.ldh + col] = x;
                    }
                    if (kBitsOnly || p.next_bits) {
                        const float xh = __fmul_rn(__fsub_rn(x, shift[h]), scale[h]);
                        const uint32_t word = __ballot_sync(0xffffffffu, col_in[h] && xh >= 0.f);
                        if (lane == 0 && 4 * h + warp < p.next_stride) p.next_bits[row * p.next_stride + 4 * h + warp] = word;
                        l1 += col_in[h] ? fabsf(xh) : 0.f;
                    }
                    acc[h] = 0.f;
                }
                if (kBitsOnly || p.next_bits) {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) l1 += __shfl_xor_sync(0xffffffffu, l1, o);
                    if (lane == 0) beta_part[(bq * kSegMax + s) * 4 + warp] = l1;
                }
                rs = 0.f;
                rg = 0.f;
            }
        }
        tc::fence_before_sync();
        __syncwarp();
        bar_arrive(kBarRI + par, kConsumers + 32);
        bar_arrive(kBarRP + (int)(i % kSlots), kConsumers + 32);
    }
    asm volatile("cp.async.wait_all;\n" ::: "memory");        // nothing of this thread is in flight when the block leaves
}

template <bool kHalf, bool kBitsOnly, bool kFull>
__global__ void __launch_bounds__(kThreads, 4)
spmm_tc_kernel(const SpmmDev p)
{
    extern __shared__ unsigned char tca_raw[];
    unsigned char* sm = tca_raw + ((1024u - (smem_u32(tca_raw) & 1023u)) & 1023u);   // the swizzled operands want 1024-byte alignment
    uint64_t* bars = reinterpret_cast<uint64_t*>(sm + kOffBars);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(sm + kOffMisc);
    volatile int* abort = reinterpret_cast<volatile int*>(sm + kOffMisc + 4);
    const int warp = threadIdx.x >> 5;
    if (warp == 0) tc::tmem_alloc(tmem_slot, kTmemCols);
    if (threadIdx.x == 32) {
        for (int i = 0; i < 2; ++i) mbar_init(&bars[i], 1);                        // products done: tcgen05.commit
        for (int i = 0; i < kAStages; ++i) mbar_init(&bars[2 + i], kConsumers);   // rows landed: every consumer thread's copies
        *abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;
    if (warp == kConsumers / 32) producer<kHalf>(p, sm, abort);
    else if (warp == kConsumers / 32 + 1) issuer(p, sm, abort, tmem_base);
    else consumers<kHalf, kBitsOnly, kFull>(p, sm, abort, tmem_base);
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 0) tc::tmem_free(tmem_base, kTmemCols);
}

}  // namespace

// Rows of 129..256 signed bytes (9..16 vectors), n < 2^31.
bool spmm_tc_covers(const SpmmDev& p)
{
    return p.nv > 8 && p.nv <= 16 && p.d_out <= 256 && p.next_stride <= 8;
}

cudaError_t launch_spmm_tc(cudaStream_t s, const SpmmDev& p)
{
    // one wave of resident blocks (four per multiprocessor: 4 x 128 = all 512 tensor-memory columns); the rows are
    // split over them by cost inside the kernel
    const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>(ceil_div(p.n, 64), (int64_t)sm_count() * 4));
    const bool bits_only = p.next_bits && !p.h_out && !p.add;
    auto launch = [&](auto kernel) -> cudaError_t {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
        if (e != cudaSuccess) return e;
        kernel<<<grid, kThreads, kSmemBytes, s>>>(p);
        return cudaGetLastError();
    };
    const bool full = p.nv == 16 && p.d_out == 256;
    if (p.half_dots) {
        if (bits_only) return full ? launch(spmm_tc_kernel<true, true, true>) : launch(spmm_tc_kernel<true, true, false>);
        return full ? launch(spmm_tc_kernel<true, false, true>) : launch(spmm_tc_kernel<true, false, false>);
    }
    if (bits_only) return full ? launch(spmm_tc_kernel<false, true, true>) : launch(spmm_tc_kernel<false, true, false>);
    return full ? launch(spmm_tc_kernel<false, false, true>) : launch(spmm_tc_kernel<false, false, false>);
}

int spmm_tc_timeouts()
{
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_spmm_tc_timeout, sizeof(int)) != cudaSuccess) return -1;
    return v;
}

}  // namespace bigcn
