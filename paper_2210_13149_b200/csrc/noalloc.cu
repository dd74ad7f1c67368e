// bigcn_layer_forward_noalloc: one binarized layer with all scratch memory held inside the library.
//
// Who this is for.  bigcn_layer_forward() takes its scratch (the contraction result between the
// bit-GEMM and the aggregation, plus the aggregation's work counter) from a workspace the caller
// allocates, and a context that itself owns a small device allocation.  Some callers cannot allocate
// device memory at all: a service that hands the whole GPU to its own memory pool at start-up, so
// that a later cudaMalloc fails or blocks; or a latency-critical loop in which the device-wide
// synchronisation cudaMalloc implies is not acceptable.  For them this entry point needs neither a
// context nor a workspace: its scratch is a fixed array in the library's device image, which every
// GPU that loads the library holds from load time until the process exits.  The paper has no
// counterpart of this call; it computes exactly what bigcn_layer_forward() computes.
#include <mutex>

#include "bigcn_internal.cuh"

using namespace bigcn;

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime's symbol table, not
// an address a kernel can use: the device address is looked up once per device below.
static __device__ __align__(256) unsigned char g_noalloc_scratch[BIGCN_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
constexpr size_t kCounterBytes = 256;                 // tail of the array: the aggregation's work counter
std::mutex g_setup_mutex;
void* g_scratch_ptr[kMaxDevices] = {};                // device address of g_noalloc_scratch, per device

// Device address of the scratch array on the current device (first call per device resolves it).
cudaError_t scratch_address(void** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ptr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) % 16) == 0; }

}  // namespace

extern "C" bigcn_status bigcn_layer_forward_noalloc(void* cuda_stream, const bigcn_graph* graph,
                                                    const bigcn_layer* layer, const uint32_t* in_bits,
                                                    const float* in_beta, float* h_out, int64_t ldh,
                                                    const bigcn_layer* next, uint32_t* next_bits,
                                                    float* next_beta)
{
    if (!graph || !layer) return BIGCN_ERR_NULL;
    if (graph->n < 0 || graph->n >= (int64_t(1) << 31) || graph->nnz < 0) return BIGCN_ERR_SHAPE;
    if (layer->d_in < 1 || layer->d_out < 1) return BIGCN_ERR_SHAPE;
    if (layer->d_out > BIGCN_MAX_D_OUT || layer->d_in > BIGCN_MAX_D_IN) return BIGCN_ERR_UNSUPPORTED;
    if (!layer->w_bitsT || !layer->alpha) return BIGCN_ERR_NULL;
    if (next && next->d_in != layer->d_out) return BIGCN_ERR_SHAPE;
    if (next && ((next->in_shift == nullptr) != (next->in_scale == nullptr))) return BIGCN_ERR_NULL;
    if (h_out && ldh < layer->d_out) return BIGCN_ERR_SHAPE;
    if (graph->n == 0) return BIGCN_OK;
    if (!graph->rowptr || (graph->nnz > 0 && (!graph->colidx || !graph->val))) return BIGCN_ERR_NULL;
    if (!in_bits || !in_beta) return BIGCN_ERR_NULL;
    if (!h_out && !next) return BIGCN_ERR_NULL;
    if (next && (!next_bits || !next_beta)) return BIGCN_ERR_NULL;
    if (!aligned16(in_bits) || !aligned16(layer->w_bitsT)) return BIGCN_ERR_ALIGN;

    // zeta as integers coded in fp16 (int16 beyond fp16's exact range): 2 bytes per element decide the size limit
    const int fmt = layer->d_in <= 2048 ? kZetaF16 : kZetaI16;
    const int64_t ldz = zeta_ld(layer->d_out, fmt);
    const size_t zeta_bytes = (size_t)graph->n * (size_t)ldz * zeta_elt_bytes(fmt);
    if (zeta_bytes > BIGCN_NOALLOC_SCRATCH_BYTES - kCounterBytes) return BIGCN_ERR_WORKSPACE;   // problem too large for the built-in scratch

    void* scratch = nullptr;
    if (scratch_address(&scratch) != cudaSuccess) return BIGCN_ERR_CUDA;
    unsigned char* base = static_cast<unsigned char*>(scratch);
    void* zeta = base;
    void* counter = base + (BIGCN_NOALLOC_SCRATCH_BYTES - kCounterBytes);

    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    int launches = 0;
    const int64_t stride_in = bigcn_packed_stride_words(layer->d_in);
    // the bit-GEMM overwrites every element of the zeta rows it will read, and the aggregation's
    // launcher zeroes the work counter: nothing of an earlier call's contents is relied on
    if (launch_bitgemm(s, in_bits, stride_in, layer->w_bitsT, stride_in, graph->n, layer->d_in, layer->d_out,
                       in_beta, layer->alpha, fmt, zeta, ldz, nullptr, nullptr, &launches) != cudaSuccess)
        return BIGCN_ERR_CUDA;
    SpmmArgs a;
    a.n = graph->n;
    a.rowptr = graph->rowptr;
    a.colidx = graph->colidx;
    a.val = graph->val;
    a.fmt = fmt;
    a.zeta = zeta;
    a.ldz = ldz;
    a.d_out = layer->d_out;
    a.node_w = in_beta;
    a.col_w = layer->alpha;
    a.h_out = h_out;
    a.ldh = ldh;
    a.next_bits = next ? next_bits : nullptr;
    a.next_stride = next ? bigcn_packed_stride_words(layer->d_out) : 0;
    a.next_beta = next ? next_beta : nullptr;
    a.next_shift = next ? next->in_shift : nullptr;
    a.next_scale = next ? next->in_scale : nullptr;
    a.long_row = 2048;
    a.scratch = counter;
    a.scratch_bytes = kCounterBytes;
    if (launch_spmm(s, a, &launches) != cudaSuccess) return BIGCN_ERR_CUDA;
    return BIGCN_OK;
}
