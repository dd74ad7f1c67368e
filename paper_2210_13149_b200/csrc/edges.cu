// Set-up from a raw edge list (Bi-GCN Sec. 3.1: an undirected graph G = (V, E); A_hat = A + I).
//
// The paper takes "the adjacency matrix of an undirected graph" as given.  A list of node pairs as it comes out of
// a data set is rarely that matrix: pairs appear in one direction or both, more than once, and sometimes join a node
// to itself.  This step turns such a list into the canonical form the normalisation step wants -- the pattern of A
// as CSR, symmetric, columns ascending and unique within a row, no diagonal: every pair (u, v) with u != v contributes
// the two entries (u, v) and (v, u), repeats are dropped, self pairs are dropped (the one self-loop of A_hat = A + I
// is added by the normalisation step).
//
// How: each pair becomes two 64-bit keys row << 32 | column (self pairs: the all-ones key, which sorts last); the
// keys are radix-sorted and de-duplicated with the CUDA toolkit's device-wide primitives (cub::DeviceRadixSort,
// cub::DeviceSelect::Unique -- a set-up step that runs once per graph, not part of the timed forward); a column index
// is the low half of a key, and a row's start is the position of the first key at or above row << 32.
#include <algorithm>

#include <cub/device/device_radix_sort.cuh>
#include <cub/device/device_select.cuh>

#include "bigcn_internal.cuh"

namespace bigcn {

namespace {

constexpr uint64_t kNoKey = ~uint64_t(0);

__global__ void edge_keys_kernel(const int32_t* __restrict__ src, const int32_t* __restrict__ dst, int64_t m, int64_t n,
                                 uint64_t* __restrict__ keys, int* __restrict__ flag)
{
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < m; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t u = src[e], v = dst[e];
        uint64_t k0 = kNoKey, k1 = kNoKey;
        if (u < 0 || u >= n || v < 0 || v >= n) atomicOr(flag, 2);          // a node id outside [0, n)
        else if (u != v) {
            k0 = ((uint64_t)u << 32) | (uint64_t)v;
            k1 = ((uint64_t)v << 32) | (uint64_t)u;
        }
        keys[2 * e] = k0;
        keys[2 * e + 1] = k1;
    }
}

// rowptr[r] = number of unique keys below r << 32 (binary search in the sorted unique keys); colidx = low halves.
__global__ void csr_from_keys_kernel(const uint64_t* __restrict__ keys, const int* __restrict__ n_unique_p, int64_t n,
                                     int64_t* __restrict__ rowptr, int32_t* __restrict__ colidx)
{
    int64_t cnt = *n_unique_p;
    if (cnt > 0 && keys[cnt - 1] == kNoKey) --cnt;                           // the self pairs' key, if any, is the last one
    const int64_t stride = (int64_t)gridDim.x * blockDim.x, t0 = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    for (int64_t r = t0; r <= n; r += stride) {
        const uint64_t want = (uint64_t)r << 32;
        int64_t lo = 0, hi = cnt;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if (keys[mid] < want) lo = mid + 1; else hi = mid;
        }
        rowptr[r] = lo;
    }
    for (int64_t i = t0; i < cnt; i += stride) colidx[i] = (int32_t)(keys[i] & 0xffffffffu);
}

size_t align_up(size_t b) { return (b + 255) / 256 * 256; }

size_t cub_temp_bytes(int64_t n_keys)
{
    size_t sort_b = 0, uniq_b = 0;
    cub::DoubleBuffer<uint64_t> db(nullptr, nullptr);
    cub::DeviceRadixSort::SortKeys(nullptr, sort_b, db, (int)n_keys, 0, 64);
    cub::DeviceSelect::Unique(nullptr, uniq_b, (const uint64_t*)nullptr, (uint64_t*)nullptr, (int*)nullptr, (int)n_keys);
    return sort_b > uniq_b ? sort_b : uniq_b;
}

}  // namespace

// two key buffers of 2 m keys each, the primitives' scratch, one counter
size_t edges_scratch_bytes(int64_t m)
{
    if (m <= 0) return 256;
    return 2 * align_up((size_t)(2 * m) * 8) + align_up(cub_temp_bytes(2 * m)) + 256;
}

// Asynchronous on `s`.  colidx needs room for 2 m entries; *n_unique_dev (inside the scratch) and rowptr[n] give the
// number of stored entries afterwards.  `flag` receives bit 2 when a node id is out of range.
cudaError_t launch_adjacency_from_edges(cudaStream_t s, int64_t n, int64_t m, const int32_t* src, const int32_t* dst,
                                        int64_t* rowptr, int32_t* colidx, void* scratch, int* flag, int* launches)
{
    cudaError_t e = cudaMemsetAsync(flag, 0, sizeof(int), s);
    if (e != cudaSuccess) return e;
    if (m == 0) return cudaMemsetAsync(rowptr, 0, (size_t)(n + 1) * sizeof(int64_t), s);
    const int64_t n_keys = 2 * m;
    char* base = static_cast<char*>(scratch);
    uint64_t* keys_a = reinterpret_cast<uint64_t*>(base);
    uint64_t* keys_b = reinterpret_cast<uint64_t*>(base + align_up((size_t)n_keys * 8));
    void* temp = base + 2 * align_up((size_t)n_keys * 8);
    size_t temp_bytes = cub_temp_bytes(n_keys);
    int* n_unique = reinterpret_cast<int*>(base + 2 * align_up((size_t)n_keys * 8) + align_up(temp_bytes));
    const unsigned blocks = (unsigned)std::min<int64_t>(ceil_div(m, 256), (int64_t)sm_count() * 8);
    edge_keys_kernel<<<blocks, 256, 0, s>>>(src, dst, m, n, keys_a, flag);
    ++*launches;
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    cub::DoubleBuffer<uint64_t> db(keys_a, keys_b);
    if ((e = cub::DeviceRadixSort::SortKeys(temp, temp_bytes, db, (int)n_keys, 0, 64, s)) != cudaSuccess) return e;
    uint64_t* sorted = db.Current();
    uint64_t* uniq = db.Alternate();
    temp_bytes = cub_temp_bytes(n_keys);
    if ((e = cub::DeviceSelect::Unique(temp, temp_bytes, (const uint64_t*)sorted, uniq, n_unique, (int)n_keys, s)) != cudaSuccess) return e;
    const unsigned blocks2 = (unsigned)std::min<int64_t>(ceil_div(std::max<int64_t>(n_keys, n + 1), 256), (int64_t)sm_count() * 8);
    csr_from_keys_kernel<<<blocks2, 256, 0, s>>>(uniq, n_unique, n, rowptr, colidx);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace bigcn
