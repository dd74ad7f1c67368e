// C ABI of libbigcn: contexts, argument validation, workspace carving and the launch sequences.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "bigcn_internal.cuh"
#include "spmm_dev.cuh"

using namespace bigcn;

struct bigcn_ctx {
    int device;
    cudaStream_t stream;
    char err[512];
    void* ws;
    size_t ws_bytes;
    int* d_flag;                 // device status words (owned)
    int launches_i;              // launches of the call in progress
    int64_t launches;
    int zeta_format;             // 0 = auto
    int64_t long_row;            // 0 = default
    int contraction;             // 0 = auto, 1 = bit-count pipe, 2 = tensor cores wherever covered
    int byte_path;               // aggregation of 129..256 byte columns: 0 / 1 = fp32 FMA stream, 2 = integer tensor-core products
    cudaEvent_t ev[2 * BIGCN_MAX_LAYERS + 2];
    bool ev_ready;
};

namespace {

constexpr size_t kAlign = 256;
constexpr int64_t kDefaultLongRow = 2048;

bigcn_status fail(bigcn_ctx* ctx, bigcn_status s, const char* fmt, ...)
{
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return s;
}

bigcn_status cuda_fail(bigcn_ctx* ctx, cudaError_t e, const char* what)
{
    return fail(ctx, BIGCN_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define BIGCN_CUDA(ctx, call)                                        \
    do {                                                             \
        cudaError_t e__ = (call);                                    \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, #call);   \
    } while (0)

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Storage format of zeta for a layer under the context's option.  Automatic choice: integers coded as
// fp16 (exact up to d_in = 2048); for 129..256 output columns the aggregation has a row-aligned stream for
// 256-byte rows of signed bytes that moves half the bytes: plain dots for d_in <= 127, half-dots
// (kZetaI8H, on the tensor-core contraction only: layers of at least 2^20 outputs) for 128 <= d_in <= 256.
// Asked for by option, half-dot bytes also serve narrower rows (up to 128 columns); the automatic choice leaves those
// in fp16: with rows that short the aggregation is bound by instructions per entry, not bytes, and measured level
// (47 columns on 126 M entries: 3.69 + 0.21 ms against 3.72 + 0.16 ms for aggregation + contraction).
// `fp32_only`: the layer's result is only written out as fp32 (a network's last layer); then 33..64 columns also take
// bytes, for which the aggregation has a stream with one stored entry per lane (c4 layer 1: 2.8 -> 1.8 ms).
// narrow_bytes: rows of 33..64 columns may be stored as bytes too (the aggregation then has its one-entry-per-lane
// stream: a last layer written as fp32, or a hidden layer of a graph whose rows are not much shorter than a pass)
int pick_format(const bigcn_ctx* ctx, int d_in, int d_out, int64_t n, bool allow_half = false, bool narrow_bytes = false)
{
    int f = ctx->zeta_format;
    const bool wide = (d_out > 128 && d_out <= 256) || (narrow_bytes && d_out > 32 && d_out <= 64);
    // half-dot bytes keep two side arrays (n node factors, d_out first weight signs) behind the byte rows inside
    // the zeta scratch, which is sized for fp32 rows: they must fit there (they do not for d_out <= 4, where an fp32
    // row is no longer than a byte row)
    const bool side_fits = up((size_t)n * (size_t)zeta_ld(d_out, kZetaI8H)) + up((size_t)n * 4) + (size_t)d_out * 4
                           <= (size_t)n * (size_t)zeta_ld(d_out, kZetaF32) * 4;
    const bool half_ok = allow_half && d_out <= 256 && d_in >= 128 && d_in <= 256 && n >= 64 && ctx->contraction != 1 && side_fits;
    if (f == 0) {
        if (wide && d_in <= 127) f = kZetaI8;
        else if (half_ok && wide && n * (int64_t)d_out >= (int64_t(1) << 20)) f = kZetaI8H;
        else f = kZetaF16;
    }
    if (f == kZetaI8H && !half_ok) f = (wide && d_in <= 127) ? kZetaI8 : kZetaF16;
    if (f == kZetaI8 && d_in > 127) f = kZetaF16;      // |dot| must fit the element type exactly
    if (f == kZetaF16 && d_in > 2048) f = kZetaI16;
    if (f == kZetaI16 && d_in > 32767) f = kZetaF32;
    return f;
}

struct Carver {
    char* base;
    size_t size, off;
    void* take(size_t bytes)
    {
        off = up(off);
        if (off + bytes > size) return nullptr;
        void* p = base + off;
        off += bytes;
        return p;
    }
};

bigcn_status bind_device(bigcn_ctx* ctx)
{
    if (!ctx) return BIGCN_ERR_NULL;
    BIGCN_CUDA(ctx, cudaSetDevice(ctx->device));
    return BIGCN_OK;
}

bigcn_status check_graph(bigcn_ctx* ctx, const bigcn_graph* g)
{
    if (!g) return fail(ctx, BIGCN_ERR_NULL, "graph is null");
    if (g->n < 0 || g->n >= (int64_t(1) << 31) || g->nnz < 0) return fail(ctx, BIGCN_ERR_SHAPE, "graph: n=%lld nnz=%lld out of range", (long long)g->n, (long long)g->nnz);
    if (g->n > 0 && (!g->rowptr || (g->nnz > 0 && (!g->colidx || !g->val))))
        return fail(ctx, BIGCN_ERR_NULL, "graph: rowptr/colidx/val must be given");
    return BIGCN_OK;
}

bigcn_status check_layer(bigcn_ctx* ctx, const bigcn_layer* l, const char* name)
{
    if (!l) return fail(ctx, BIGCN_ERR_NULL, "%s is null", name);
    if (l->d_in < 1 || l->d_out < 1) return fail(ctx, BIGCN_ERR_SHAPE, "%s: d_in=%d d_out=%d must be >= 1", name, l->d_in, l->d_out);
    if (l->d_out > BIGCN_MAX_D_OUT) return fail(ctx, BIGCN_ERR_UNSUPPORTED, "%s: d_out=%d > %d is not supported", name, l->d_out, BIGCN_MAX_D_OUT);
    if (l->d_in > BIGCN_MAX_D_IN) return fail(ctx, BIGCN_ERR_UNSUPPORTED, "%s: d_in=%d > %d is not supported", name, l->d_in, BIGCN_MAX_D_IN);
    if (!l->w_bitsT || !l->alpha) return fail(ctx, BIGCN_ERR_NULL, "%s: w_bitsT/alpha are null", name);
    if ((l->in_shift == nullptr) != (l->in_scale == nullptr)) return fail(ctx, BIGCN_ERR_NULL, "%s: in_shift and in_scale go together", name);
    if (!aligned(l->w_bitsT, 16)) return fail(ctx, BIGCN_ERR_ALIGN, "%s: w_bitsT must be 16-byte aligned", name);
    return BIGCN_OK;
}

// One layer on already validated arguments.  `zeta` is scratch for n * zeta_ld(d_out) elements.
bigcn_status run_layer(bigcn_ctx* ctx, const bigcn_graph* g, const bigcn_layer* layer,
                       const uint32_t* in_bits, const float* in_beta, void* zeta, void* scratch,
                       float* h_out, int64_t ldh, const bigcn_layer* next, uint32_t* next_bits,
                       float* next_beta, int32_t* dbg_dot, float* dbg_zeta,
                       cudaEvent_t ev_mid /*nullable*/)
{
    const bool lane_stream = (next == nullptr && h_out != nullptr) || (next != nullptr && g->nnz >= 8 * g->n);
    const int fmt = pick_format(ctx, layer->d_in, layer->d_out, g->n, /*allow_half=*/true, /*narrow_bytes=*/lane_stream);
    const bool half = fmt == kZetaI8H;
    const int64_t stride_in = bigcn_packed_stride_words(layer->d_in);
    // 33..60 byte columns for the lane-per-entry stream, on the tensor-core contraction: 64-byte rows that carry the node
    // factor in their last four bytes, so that the aggregation needs two lookups per entry, not four or five
    const bool row_tail = (fmt == kZetaI8 || half) && lane_stream && layer->d_out > 32 && layer->d_out <= 60 &&
                          bitgemm_takes_tc(fmt, half ? 2 : ctx->contraction, g->n, layer->d_in, layer->d_out, stride_in, stride_in);
    const int64_t ldz = row_tail ? 64 : zeta_ld(layer->d_out, fmt);
    // half-dot bytes: the node factors carrying the first feature sign and the columns' first weight signs follow
    // the byte rows inside the zeta scratch (which is sized for fp32 rows, four times as much)
    float* nws = nullptr;
    float* col_b0 = nullptr;
    if (half) {
        char* after = static_cast<char*>(zeta) + up((size_t)g->n * ldz);
        nws = reinterpret_cast<float*>(after);
        col_b0 = reinterpret_cast<float*>(after + up((size_t)g->n * 4));
    }
    cudaError_t e = launch_bitgemm(ctx->stream, in_bits, stride_in, layer->w_bitsT, stride_in, g->n,
                                   layer->d_in, layer->d_out, in_beta, layer->alpha, fmt, zeta, ldz,
                                   dbg_dot, dbg_zeta, &ctx->launches_i, half ? 2 : ctx->contraction, nws, col_b0, row_tail ? 1 : 0);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "bit-GEMM launch");
    if (ev_mid) BIGCN_CUDA(ctx, cudaEventRecord(ev_mid, ctx->stream));
    SpmmArgs a;
    a.n = g->n;
    a.nnz = g->nnz;
    a.rowptr = g->rowptr;
    a.colidx = g->colidx;
    a.val = g->val;
    a.fmt = half ? kZetaI8 : fmt;
    a.zeta = zeta;
    a.ldz = ldz;
    a.d_out = layer->d_out;
    a.node_w = half ? nws : in_beta;
    a.col_w = layer->alpha;
    a.half_dots = half;
    a.byte_path = ctx->byte_path;
    a.row_tail = row_tail;
    a.col_b0 = col_b0;
    a.h_out = h_out;
    a.ldh = ldh;
    a.next_bits = next ? next_bits : nullptr;
    a.next_stride = next ? bigcn_packed_stride_words(layer->d_out) : 0;
    a.next_beta = next ? next_beta : nullptr;
    a.next_shift = next ? next->in_shift : nullptr;
    a.next_scale = next ? next->in_scale : nullptr;
    a.long_row = ctx->long_row > 0 ? ctx->long_row : kDefaultLongRow;
    a.scratch = scratch;
    a.scratch_bytes = spmm_scratch_bytes(g->n, g->nnz, layer->d_out);
    e = launch_spmm(ctx->stream, a, &ctx->launches_i);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "SpMM launch");
    return BIGCN_OK;
}

size_t zeta_bytes_max(int64_t n, const int32_t* dims, int n_layers)
{
    size_t m = 0;
    for (int l = 0; l < n_layers; ++l) {
        const size_t b = (size_t)n * (size_t)zeta_ld(dims[l + 1], kZetaF32) * 4;   // fp32 is the widest form
        if (b > m) m = b;
    }
    return m;
}

// Bytes of a slot's input staging buffer: the fp32 features, or -- whichever is larger -- the packed input
// (bits, then beta behind them at the next 256-byte boundary).
size_t staging_in_bytes(int64_t n, int32_t d0)
{
    const size_t dense = (size_t)n * d0 * 4;
    const size_t packed = up((size_t)n * bigcn_packed_stride_words(d0) * 4) + (size_t)n * 4;
    return dense > packed ? dense : packed;
}

void finish_call(bigcn_ctx* ctx)
{
    ctx->launches += ctx->launches_i;
    ctx->launches_i = 0;
}

bigcn_status forward_impl(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layers,
                          int32_t n_layers, const float* X, int64_t ldx, const uint32_t* x_bits,
                          const float* x_beta, float* logits_out, int64_t ldo, bigcn_stats* stats,
                          Carver& ws)
{
    const int64_t n = graph->n;
    int32_t dims[BIGCN_MAX_LAYERS + 1];
    dims[0] = layers[0].d_in;
    for (int l = 0; l < n_layers; ++l) dims[l + 1] = layers[l].d_out;
    int64_t stride_max = 0;
    for (int l = 0; l < n_layers; ++l) stride_max = stride_max > bigcn_packed_stride_words(dims[l]) ? stride_max : bigcn_packed_stride_words(dims[l]);
    void* zeta = ws.take(zeta_bytes_max(n, dims, n_layers));
    void* scratch = ws.take(spmm_scratch_bytes(n, graph->nnz, 0));
    uint32_t* bits[2];
    float* beta[2];
    for (int i = 0; i < 2; ++i) {
        bits[i] = static_cast<uint32_t*>(ws.take((size_t)n * stride_max * 4));
        beta[i] = static_cast<float*>(ws.take((size_t)n * 4));
    }
    if (!zeta || !scratch || !bits[0] || !beta[0] || !bits[1] || !beta[1])
        return fail(ctx, BIGCN_ERR_WORKSPACE, "workspace of %zu bytes is too small (see bigcn_workspace_bytes)", ws.size);

    cudaEvent_t* ev = ctx->ev;
    if (stats) BIGCN_CUDA(ctx, cudaEventRecord(ev[0], ctx->stream));
    const uint32_t* cur_bits = x_bits;
    const float* cur_beta = x_beta;
    if (X) {
        cudaError_t e = launch_pack_rows(ctx->stream, X, n, dims[0], ldx, layers[0].in_shift, layers[0].in_scale,
                                         bits[0], bigcn_packed_stride_words(dims[0]), beta[0], &ctx->launches_i);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "pack launch");
        cur_bits = bits[0];
        cur_beta = beta[0];
    }
    if (stats) BIGCN_CUDA(ctx, cudaEventRecord(ev[1], ctx->stream));
    for (int l = 0; l < n_layers; ++l) {
        const bool last = (l == n_layers - 1);
        const int o = (l + 1) & 1;
        bigcn_status st = run_layer(ctx, graph, &layers[l], cur_bits, cur_beta, zeta, scratch,
                                    last ? logits_out : nullptr, ldo, last ? nullptr : &layers[l + 1],
                                    bits[o], beta[o], nullptr, nullptr, stats ? ev[2 + 2 * l] : nullptr);
        if (st != BIGCN_OK) return st;
        if (stats) BIGCN_CUDA(ctx, cudaEventRecord(ev[3 + 2 * l], ctx->stream));
        cur_bits = bits[o];
        cur_beta = beta[o];
    }
    if (stats) {
        BIGCN_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        memset(stats, 0, sizeof(*stats));
        stats->n_layers = n_layers;
        stats->launches = ctx->launches_i;
        cudaEventElapsedTime(&stats->ms_pack, ev[0], ev[1]);
        for (int l = 0; l < n_layers; ++l) {
            cudaEventElapsedTime(&stats->ms_gemm[l], ev[1 + 2 * l], ev[2 + 2 * l]);
            cudaEventElapsedTime(&stats->ms_spmm[l], ev[2 + 2 * l], ev[3 + 2 * l]);
        }
        cudaEventElapsedTime(&stats->ms_total, ev[0], ev[1 + 2 * n_layers]);
    }
    return BIGCN_OK;
}

bigcn_status check_forward(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layers,
                           int32_t n_layers, const void* logits, int64_t ldo)
{
    bigcn_status st = check_graph(ctx, graph);
    if (st != BIGCN_OK) return st;
    if (!layers) return fail(ctx, BIGCN_ERR_NULL, "layers is null");
    if (n_layers < 1 || n_layers > BIGCN_MAX_LAYERS) return fail(ctx, BIGCN_ERR_SHAPE, "n_layers=%d not in [1, %d]", n_layers, BIGCN_MAX_LAYERS);
    for (int l = 0; l < n_layers; ++l) {
        if ((st = check_layer(ctx, &layers[l], "layer")) != BIGCN_OK) return st;
        if (l > 0 && layers[l].d_in != layers[l - 1].d_out)
            return fail(ctx, BIGCN_ERR_SHAPE, "layer %d: d_in=%d does not match the previous d_out=%d", l, layers[l].d_in, layers[l - 1].d_out);
    }
    if (graph->n > 0 && !logits) return fail(ctx, BIGCN_ERR_NULL, "logits output is null");
    if (ldo < layers[n_layers - 1].d_out) return fail(ctx, BIGCN_ERR_SHAPE, "ldo=%lld < classes=%d", (long long)ldo, layers[n_layers - 1].d_out);
    if (graph->n > 0 && !ctx->ws) return fail(ctx, BIGCN_ERR_WORKSPACE, "no workspace attached");
    return BIGCN_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------------------

extern "C" {

const char* bigcn_status_string(bigcn_status s)
{
    switch (s) {
        case BIGCN_OK: return "ok";
        case BIGCN_ERR_NULL: return "null pointer";
        case BIGCN_ERR_SHAPE: return "bad shape";
        case BIGCN_ERR_ALIGN: return "misaligned pointer";
        case BIGCN_ERR_GRAPH: return "malformed graph";
        case BIGCN_ERR_WORKSPACE: return "workspace missing or too small";
        case BIGCN_ERR_CUDA: return "CUDA error";
        case BIGCN_ERR_UNSUPPORTED: return "unsupported";
        case BIGCN_ERR_INTERNAL: return "device self-check failed";
        case BIGCN_ERR_BUSY: return "pipeline full";
    }
    return "unknown status";
}

bigcn_status bigcn_create(bigcn_ctx** out, int device, void* cuda_stream)
{
    if (!out) return BIGCN_ERR_NULL;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || count == 0 || device < 0 || device >= count) {
        cudaGetLastError();
        return BIGCN_ERR_CUDA;          // no CUDA device: there is no CPU fallback
    }
    if (cudaSetDevice(device) != cudaSuccess) return BIGCN_ERR_CUDA;
    bigcn_ctx* ctx = new (std::nothrow) bigcn_ctx();
    if (!ctx) return BIGCN_ERR_INTERNAL;
    memset(ctx, 0, sizeof(*ctx));
    ctx->device = device;
    ctx->stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMalloc(reinterpret_cast<void**>(&ctx->d_flag), 256) != cudaSuccess ||
        cudaMemset(ctx->d_flag, 0, 256) != cudaSuccess) {
        delete ctx;
        return BIGCN_ERR_CUDA;
    }
    for (auto& e : ctx->ev)
        if (cudaEventCreate(&e) != cudaSuccess) { bigcn_destroy(ctx); return BIGCN_ERR_CUDA; }
    ctx->ev_ready = true;
    *out = ctx;
    return BIGCN_OK;
}

bigcn_status bigcn_destroy(bigcn_ctx* ctx)
{
    if (!ctx) return BIGCN_OK;
    cudaSetDevice(ctx->device);
    for (auto& e : ctx->ev)
        if (e) cudaEventDestroy(e);
    if (ctx->d_flag) cudaFree(ctx->d_flag);
    delete ctx;
    return BIGCN_OK;
}

const char* bigcn_last_error(const bigcn_ctx* ctx) { return ctx ? ctx->err : "context is null"; }

bigcn_status bigcn_set_option(bigcn_ctx* ctx, int32_t option, int64_t value)
{
    if (!ctx) return BIGCN_ERR_NULL;
    switch (option) {
        case BIGCN_OPT_ZETA_FORMAT:
            if (value < 0 || value > 5) return fail(ctx, BIGCN_ERR_SHAPE, "zeta format %lld not in [0, 5]", (long long)value);
            ctx->zeta_format = (int)value;
            return BIGCN_OK;
        case BIGCN_OPT_LONG_ROW:
            if (value < 0) return fail(ctx, BIGCN_ERR_SHAPE, "long-row threshold must be >= 0");
            ctx->long_row = value;
            return BIGCN_OK;
        case BIGCN_OPT_CONTRACTION:
            if (value < 0 || value > 2) return fail(ctx, BIGCN_ERR_SHAPE, "contraction path %lld not in 0..2", (long long)value);
            ctx->contraction = (int)value;
            return BIGCN_OK;
        case BIGCN_OPT_BYTE_AGGREGATION:
            if (value < 0 || value > 3) return fail(ctx, BIGCN_ERR_SHAPE, "byte aggregation path %lld not in 0..3", (long long)value);
            ctx->byte_path = (int)value;
            return BIGCN_OK;
    }
    return fail(ctx, BIGCN_ERR_UNSUPPORTED, "unknown option %d", option);
}

int64_t bigcn_launch_count(const bigcn_ctx* ctx) { return ctx ? ctx->launches : 0; }

bigcn_status bigcn_sync_check(bigcn_ctx* ctx)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    BIGCN_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    BIGCN_CUDA(ctx, cudaGetLastError());
    if (bitgemm_tc_timeouts() != 0) return fail(ctx, BIGCN_ERR_INTERNAL, "a bounded wait on the tensor cores ran out (contraction kernel)");
    if (backward_tc_timeouts() != 0) return fail(ctx, BIGCN_ERR_INTERNAL, "a bounded wait on the tensor cores ran out (backward kernel)");
    if (spmm_tc_timeouts() != 0) return fail(ctx, BIGCN_ERR_INTERNAL, "a bounded wait ran out (tensor-core aggregation kernel)");
    return BIGCN_OK;
}

int64_t bigcn_packed_stride_words(int32_t len)
{
    if (len < 0) return 0;
    return round_up(ceil_div(len, 32), 4);
}

size_t bigcn_workspace_bytes(int64_t n, int64_t nnz, const int32_t* dims, int32_t n_layers, int32_t host_io)
{
    if (n < 0 || !dims || n_layers < 1 || n_layers > BIGCN_MAX_LAYERS) return 0;
    int64_t stride_max = 0;
    int32_t d_max = 0;
    for (int l = 0; l <= n_layers; ++l) {
        if (dims[l] < 1) return 0;
        if (l < n_layers && bigcn_packed_stride_words(dims[l]) > stride_max) stride_max = bigcn_packed_stride_words(dims[l]);
        if (dims[l] > d_max) d_max = dims[l];
    }
    size_t total = up(zeta_bytes_max(n, dims, n_layers)) + up(spmm_scratch_bytes(n, nnz, 0));
    total += 2 * (up((size_t)n * stride_max * 4) + up((size_t)n * 4));
    size_t aux = up(normalize_scratch_bytes(n));
    if (up(col_stats_scratch_bytes(d_max)) > aux) aux = up(col_stats_scratch_bytes(d_max));
    if (host_io > 0) {                                        // staging buffers: one pair per slot
        total += (size_t)host_io * (up(staging_in_bytes(n, dims[0])) + up((size_t)n * dims[n_layers] * 4));
    }
    if (aux > total) total = aux;
    return total + kAlign;
}

bigcn_status bigcn_set_workspace(bigcn_ctx* ctx, void* workspace, size_t bytes)
{
    if (!ctx) return BIGCN_ERR_NULL;
    if (workspace && !aligned(workspace, kAlign)) return fail(ctx, BIGCN_ERR_ALIGN, "workspace must be 256-byte aligned");
    ctx->ws = workspace;
    ctx->ws_bytes = workspace ? bytes : 0;
    return BIGCN_OK;
}

bigcn_status bigcn_normalize_adjacency(bigcn_ctx* ctx, int64_t n, int64_t nnz_in,
                                       const int64_t* rowptr_A, const int32_t* colidx_A,
                                       int64_t* rowptr, int32_t* colidx, float* val, float* dinv,
                                       int64_t* nnz_out)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (n < 0 || n >= (int64_t(1) << 31) || nnz_in < 0) return fail(ctx, BIGCN_ERR_SHAPE, "n=%lld nnz_in=%lld out of range", (long long)n, (long long)nnz_in);
    if (!nnz_out) return fail(ctx, BIGCN_ERR_NULL, "nnz_out is null");
    if (!rowptr) return fail(ctx, BIGCN_ERR_NULL, "rowptr output is null");
    *nnz_out = 0;
    if (n == 0) {
        BIGCN_CUDA(ctx, cudaMemsetAsync(rowptr, 0, sizeof(int64_t), ctx->stream));
        BIGCN_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        return BIGCN_OK;
    }
    if (!rowptr_A || (nnz_in > 0 && !colidx_A) || !colidx || !val || !dinv) return fail(ctx, BIGCN_ERR_NULL, "an input or output array is null");
    if (!ctx->ws || ctx->ws_bytes < normalize_scratch_bytes(n)) return fail(ctx, BIGCN_ERR_WORKSPACE, "needs %zu bytes of workspace", normalize_scratch_bytes(n));
    cudaError_t e = launch_normalize_adjacency(ctx->stream, n, nnz_in, rowptr_A, colidx_A, rowptr, colidx, val, dinv,
                                               ctx->ws, ctx->d_flag, &ctx->launches_i);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "normalize_adjacency launch");
    int flag = 0;
    int64_t total = 0;
    BIGCN_CUDA(ctx, cudaMemcpyAsync(&flag, ctx->d_flag, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    BIGCN_CUDA(ctx, cudaMemcpyAsync(&total, rowptr + n, sizeof(int64_t), cudaMemcpyDeviceToHost, ctx->stream));
    BIGCN_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (flag)
        return fail(ctx, BIGCN_ERR_GRAPH, "adjacency input rejected:%s%s%s%s",
                    (flag & 8) ? " rowptr not monotone from 0 to nnz;" : "",
                    (flag & 2) ? " column index outside [0, n);" : "",
                    (flag & 1) ? " columns not ascending and unique within a row;" : "",
                    (flag & 4) ? " pattern not symmetric;" : "");
    *nnz_out = total;
    return BIGCN_OK;
}

size_t bigcn_edges_workspace_bytes(int64_t n, int64_t m)
{
    if (n < 0 || m < 0 || m >= (int64_t(1) << 30)) return 0;
    return edges_scratch_bytes(m) + kAlign;
}

bigcn_status bigcn_adjacency_from_edges(bigcn_ctx* ctx, int64_t n, int64_t m, const int32_t* src, const int32_t* dst,
                                        int64_t* rowptr_A, int32_t* colidx_A, int64_t* nnz_out)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (n < 0 || n >= (int64_t(1) << 31) || m < 0 || m >= (int64_t(1) << 30)) return fail(ctx, BIGCN_ERR_SHAPE, "n=%lld m=%lld out of range", (long long)n, (long long)m);
    if (!nnz_out || !rowptr_A) return fail(ctx, BIGCN_ERR_NULL, "nnz_out or rowptr_A is null");
    *nnz_out = 0;
    if (m > 0 && (!src || !dst || !colidx_A)) return fail(ctx, BIGCN_ERR_NULL, "src, dst or colidx_A is null");
    if (m > 0 && (!ctx->ws || ctx->ws_bytes < edges_scratch_bytes(m))) return fail(ctx, BIGCN_ERR_WORKSPACE, "needs %zu bytes of workspace (bigcn_edges_workspace_bytes)", edges_scratch_bytes(m));
    cudaError_t e = launch_adjacency_from_edges(ctx->stream, n, m, src, dst, rowptr_A, colidx_A, ctx->ws, ctx->d_flag, &ctx->launches_i);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "adjacency_from_edges");
    int flag = 0;
    int64_t total = 0;
    BIGCN_CUDA(ctx, cudaMemcpyAsync(&flag, ctx->d_flag, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    BIGCN_CUDA(ctx, cudaMemcpyAsync(&total, rowptr_A + n, sizeof(int64_t), cudaMemcpyDeviceToHost, ctx->stream));
    BIGCN_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (flag) return fail(ctx, BIGCN_ERR_GRAPH, "edge list rejected: a node id lies outside [0, n)");
    *nnz_out = total;
    return BIGCN_OK;
}

bigcn_status bigcn_pack_features(bigcn_ctx* ctx, const float* H, int64_t n, int32_t d, int64_t ld,
                                 const float* col_shift, const float* col_scale,
                                 uint32_t* bits_out, int64_t stride_words, float* beta_out)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (n < 0 || d < 1 || ld < d) return fail(ctx, BIGCN_ERR_SHAPE, "n=%lld d=%d ld=%lld", (long long)n, d, (long long)ld);
    if (stride_words < bigcn_packed_stride_words(d) || stride_words % 4 != 0)
        return fail(ctx, BIGCN_ERR_SHAPE, "stride_words=%lld must be a multiple of 4 and >= %lld", (long long)stride_words, (long long)bigcn_packed_stride_words(d));
    if ((col_shift == nullptr) != (col_scale == nullptr)) return fail(ctx, BIGCN_ERR_NULL, "col_shift and col_scale go together");
    if (n == 0) return BIGCN_OK;
    if (!H || !bits_out || !beta_out) return fail(ctx, BIGCN_ERR_NULL, "H, bits_out or beta_out is null");
    if (!aligned(bits_out, 16)) return fail(ctx, BIGCN_ERR_ALIGN, "bits_out must be 16-byte aligned");
    cudaError_t e = launch_pack_rows(ctx->stream, H, n, d, ld, col_shift, col_scale, bits_out, stride_words, beta_out, &ctx->launches_i);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "pack_features launch");
    return BIGCN_OK;
}

bigcn_status bigcn_pack_weights(bigcn_ctx* ctx, const float* W, int32_t d_in, int32_t d_out, int64_t ldw,
                                uint32_t* bitsT_out, int64_t stride_words, float* alpha_out)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (d_in < 1 || d_out < 1 || ldw < d_out) return fail(ctx, BIGCN_ERR_SHAPE, "d_in=%d d_out=%d ldw=%lld", d_in, d_out, (long long)ldw);
    if (stride_words < bigcn_packed_stride_words(d_in) || stride_words % 4 != 0 || stride_words > 65535)
        return fail(ctx, BIGCN_ERR_SHAPE, "stride_words=%lld must be a multiple of 4 in [%lld, 65535]", (long long)stride_words, (long long)bigcn_packed_stride_words(d_in));
    if (!W || !bitsT_out || !alpha_out) return fail(ctx, BIGCN_ERR_NULL, "W, bitsT_out or alpha_out is null");
    if (!aligned(bitsT_out, 16)) return fail(ctx, BIGCN_ERR_ALIGN, "bitsT_out must be 16-byte aligned");
    cudaError_t e = launch_pack_weights(ctx->stream, W, d_in, d_out, ldw, bitsT_out, stride_words, alpha_out, &ctx->launches_i);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "pack_weights launch");
    return BIGCN_OK;
}

bigcn_status bigcn_layer_forward(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layer,
                                 const uint32_t* in_bits, const float* in_beta,
                                 float* h_out, int64_t ldh,
                                 const bigcn_layer* next, uint32_t* next_bits, float* next_beta,
                                 int32_t* dbg_dot, float* dbg_zeta)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if ((st = check_graph(ctx, graph)) != BIGCN_OK) return st;
    if ((st = check_layer(ctx, layer, "layer")) != BIGCN_OK) return st;
    if (next) {
        if (next->d_in != layer->d_out) return fail(ctx, BIGCN_ERR_SHAPE, "next->d_in=%d != layer->d_out=%d", next->d_in, layer->d_out);
        if ((next->in_shift == nullptr) != (next->in_scale == nullptr)) return fail(ctx, BIGCN_ERR_NULL, "next: in_shift and in_scale go together");
    }
    if (h_out && ldh < layer->d_out) return fail(ctx, BIGCN_ERR_SHAPE, "ldh=%lld < d_out=%d", (long long)ldh, layer->d_out);
    if (graph->n == 0) return BIGCN_OK;
    if (!in_bits || !in_beta) return fail(ctx, BIGCN_ERR_NULL, "in_bits or in_beta is null");
    if (!aligned(in_bits, 16)) return fail(ctx, BIGCN_ERR_ALIGN, "in_bits must be 16-byte aligned");
    if (next && (!next_bits || !next_beta)) return fail(ctx, BIGCN_ERR_NULL, "next_bits or next_beta is null");
    if (!h_out && !next) return fail(ctx, BIGCN_ERR_NULL, "neither h_out nor next is given: nothing to compute");
    const int32_t dims[2] = {layer->d_in, layer->d_out};
    const size_t zbytes = up(zeta_bytes_max(graph->n, dims, 1));
    const size_t need = zbytes + up(spmm_scratch_bytes(graph->n, graph->nnz, layer->d_out));
    if (!ctx->ws || ctx->ws_bytes < need) return fail(ctx, BIGCN_ERR_WORKSPACE, "needs %zu bytes of workspace, has %zu", need, ctx->ws_bytes);
    st = run_layer(ctx, graph, layer, in_bits, in_beta, ctx->ws, static_cast<char*>(ctx->ws) + zbytes, h_out, ldh, next, next_bits, next_beta,
                   dbg_dot, dbg_zeta, nullptr);
    finish_call(ctx);
    return st;
}

bigcn_status bigcn_forward(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layers,
                           int32_t n_layers, const float* X, int64_t ldx,
                           float* logits_out, int64_t ldo, bigcn_stats* stats)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if ((st = check_forward(ctx, graph, layers, n_layers, logits_out, ldo)) != BIGCN_OK) return st;
    if (ldx < layers[0].d_in) return fail(ctx, BIGCN_ERR_SHAPE, "ldx=%lld < d_0=%d", (long long)ldx, layers[0].d_in);
    if (graph->n == 0) return BIGCN_OK;
    if (!X) return fail(ctx, BIGCN_ERR_NULL, "X is null");
    Carver ws{static_cast<char*>(ctx->ws), ctx->ws_bytes, 0};
    st = forward_impl(ctx, graph, layers, n_layers, X, ldx, nullptr, nullptr, logits_out, ldo, stats, ws);
    finish_call(ctx);
    return st;
}

bigcn_status bigcn_forward_packed(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layers,
                                  int32_t n_layers, const uint32_t* x_bits, const float* x_beta,
                                  float* logits_out, int64_t ldo, bigcn_stats* stats)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if ((st = check_forward(ctx, graph, layers, n_layers, logits_out, ldo)) != BIGCN_OK) return st;
    if (graph->n == 0) return BIGCN_OK;
    if (!x_bits || !x_beta) return fail(ctx, BIGCN_ERR_NULL, "x_bits or x_beta is null");
    if (!aligned(x_bits, 16)) return fail(ctx, BIGCN_ERR_ALIGN, "x_bits must be 16-byte aligned");
    Carver ws{static_cast<char*>(ctx->ws), ctx->ws_bytes, 0};
    st = forward_impl(ctx, graph, layers, n_layers, nullptr, 0, x_bits, x_beta, logits_out, ldo, stats, ws);
    finish_call(ctx);
    return st;
}

bigcn_status bigcn_forward_host(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layers,
                                int32_t n_layers, const float* X_host, int64_t ldx,
                                float* logits_host, int64_t ldo)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if ((st = check_forward(ctx, graph, layers, n_layers, logits_host, ldo)) != BIGCN_OK) return st;
    const int32_t d0 = layers[0].d_in, classes = layers[n_layers - 1].d_out;
    if (ldx != d0 || ldo != classes) return fail(ctx, BIGCN_ERR_SHAPE, "host buffers must be dense: ldx=%lld (d_0=%d), ldo=%lld (classes=%d)", (long long)ldx, d0, (long long)ldo, classes);
    const int64_t n = graph->n;
    if (n == 0) return BIGCN_OK;
    if (!X_host) return fail(ctx, BIGCN_ERR_NULL, "X_host is null");
    Carver ws{static_cast<char*>(ctx->ws), ctx->ws_bytes, 0};
    float* x_dev = static_cast<float*>(ws.take((size_t)n * d0 * 4));
    float* out_dev = static_cast<float*>(ws.take((size_t)n * classes * 4));
    if (!x_dev || !out_dev) return fail(ctx, BIGCN_ERR_WORKSPACE, "workspace too small for the host staging buffers (size it with host_io = 1)");
    BIGCN_CUDA(ctx, cudaMemcpyAsync(x_dev, X_host, (size_t)n * d0 * 4, cudaMemcpyHostToDevice, ctx->stream));
    st = forward_impl(ctx, graph, layers, n_layers, x_dev, d0, nullptr, nullptr, out_dev, classes, nullptr, ws);
    finish_call(ctx);
    if (st != BIGCN_OK) return st;
    BIGCN_CUDA(ctx, cudaMemcpyAsync(logits_host, out_dev, (size_t)n * classes * 4, cudaMemcpyDeviceToHost, ctx->stream));
    BIGCN_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return BIGCN_OK;
}

struct bigcn_pipeline {
    bigcn_ctx* ctx;
    bigcn_graph graph;
    bigcn_layer layers[BIGCN_MAX_LAYERS];
    int32_t n_layers;
    int32_t slots;
    cudaStream_t up;                                  // host -> device copies
    cudaStream_t down;                                // device -> host copies
    cudaEvent_t x_ready[BIGCN_MAX_PIPELINE_SLOTS];    // the slot's input has arrived
    cudaEvent_t computed[BIGCN_MAX_PIPELINE_SLOTS];   // the slot's forward is done (input consumed, logits written)
    cudaEvent_t delivered[BIGCN_MAX_PIPELINE_SLOTS];  // the slot's logits are in host memory
    bool used[BIGCN_MAX_PIPELINE_SLOTS];
    int64_t submitted;
    int64_t waited;
};

bigcn_status bigcn_pipeline_open(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layers,
                                 int32_t n_layers, int32_t slots, bigcn_pipeline** out)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (!out) return fail(ctx, BIGCN_ERR_NULL, "out is null");
    *out = nullptr;
    if (slots < 1 || slots > BIGCN_MAX_PIPELINE_SLOTS) return fail(ctx, BIGCN_ERR_SHAPE, "slots=%d not in 1..%d", slots, BIGCN_MAX_PIPELINE_SLOTS);
    float dummy = 0.f;                                // check_forward only tests the logits pointer for null
    if ((st = check_forward(ctx, graph, layers, n_layers, &dummy, int64_t(1) << 40)) != BIGCN_OK) return st;
    bigcn_pipeline* p = new (std::nothrow) bigcn_pipeline();
    if (!p) return fail(ctx, BIGCN_ERR_INTERNAL, "out of host memory");
    p->ctx = ctx;
    p->graph = *graph;
    for (int l = 0; l < n_layers; ++l) p->layers[l] = layers[l];
    p->n_layers = n_layers;
    p->slots = slots;
    cudaError_t e = cudaStreamCreateWithFlags(&p->up, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&p->down, cudaStreamNonBlocking);
    for (int s = 0; s < slots && e == cudaSuccess; ++s) {
        e = cudaEventCreateWithFlags(&p->x_ready[s], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->computed[s], cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->delivered[s], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) {
        bigcn_pipeline_close(p);
        return cuda_fail(ctx, e, "pipeline streams and events");
    }
    *out = p;
    return BIGCN_OK;
}

namespace {

// One step of a pipeline from fp32 features (X_host) or from an already binary input (bits_host, beta_host).
bigcn_status pipeline_submit_impl(bigcn_pipeline* p, const float* X_host, const uint32_t* bits_host, const float* beta_host,
                                  float* logits_host)
{
    if (!p) return BIGCN_ERR_NULL;
    bigcn_ctx* ctx = p->ctx;
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (p->submitted - p->waited >= p->slots) return fail(ctx, BIGCN_ERR_BUSY, "all %d slots hold steps that have not been waited for", p->slots);
    const int64_t n = p->graph.n;
    const int32_t d0 = p->layers[0].d_in, classes = p->layers[p->n_layers - 1].d_out;
    const int s = (int)(p->submitted % p->slots);
    if (n == 0) {                                             // nothing to move or compute: the step is complete
        BIGCN_CUDA(ctx, cudaEventRecord(p->delivered[s], p->down));
        ++p->submitted;
        return BIGCN_OK;
    }
    const bool packed = X_host == nullptr;
    if (!logits_host || (packed ? (!bits_host || !beta_host) : false)) return fail(ctx, BIGCN_ERR_NULL, "an input or logits_host is null");
    Carver ws{static_cast<char*>(ctx->ws), ctx->ws_bytes, 0};
    float* x_dev = nullptr;
    float* out_dev = nullptr;
    for (int i = 0; i < p->slots; ++i) {                      // the same carving at every call: slot i keeps its buffers
        float* x = static_cast<float*>(ws.take(staging_in_bytes(n, d0)));
        float* o = static_cast<float*>(ws.take((size_t)n * classes * 4));
        if (!x || !o) return fail(ctx, BIGCN_ERR_WORKSPACE, "workspace too small for %d pairs of staging buffers (size it with host_io = %d)", p->slots, p->slots);
        if (i == s) { x_dev = x; out_dev = o; }
    }
    // copy in: the slot's input buffer is free once the step that used it last has been computed
    if (p->used[s]) BIGCN_CUDA(ctx, cudaStreamWaitEvent(p->up, p->computed[s], 0));
    const size_t bits_bytes = (size_t)n * bigcn_packed_stride_words(d0) * 4;
    uint32_t* bits_dev = reinterpret_cast<uint32_t*>(x_dev);
    float* beta_dev = reinterpret_cast<float*>(reinterpret_cast<char*>(x_dev) + up(bits_bytes));
    if (packed) {                                             // Sec. 5.2: the loaded data is binary -- 1 bit per element and one scalar per node
        BIGCN_CUDA(ctx, cudaMemcpyAsync(bits_dev, bits_host, bits_bytes, cudaMemcpyHostToDevice, p->up));
        BIGCN_CUDA(ctx, cudaMemcpyAsync(beta_dev, beta_host, (size_t)n * 4, cudaMemcpyHostToDevice, p->up));
    } else {
        BIGCN_CUDA(ctx, cudaMemcpyAsync(x_dev, X_host, (size_t)n * d0 * 4, cudaMemcpyHostToDevice, p->up));
    }
    BIGCN_CUDA(ctx, cudaEventRecord(p->x_ready[s], p->up));
    // forward: the slot's logits buffer is free because its last step has been waited for (slots bound above)
    BIGCN_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, p->x_ready[s], 0));
    if (packed) st = forward_impl(ctx, &p->graph, p->layers, p->n_layers, nullptr, 0, bits_dev, beta_dev, out_dev, classes, nullptr, ws);
    else st = forward_impl(ctx, &p->graph, p->layers, p->n_layers, x_dev, d0, nullptr, nullptr, out_dev, classes, nullptr, ws);
    finish_call(ctx);
    if (st != BIGCN_OK) return st;
    BIGCN_CUDA(ctx, cudaEventRecord(p->computed[s], ctx->stream));
    // copy out
    BIGCN_CUDA(ctx, cudaStreamWaitEvent(p->down, p->computed[s], 0));
    BIGCN_CUDA(ctx, cudaMemcpyAsync(logits_host, out_dev, (size_t)n * classes * 4, cudaMemcpyDeviceToHost, p->down));
    BIGCN_CUDA(ctx, cudaEventRecord(p->delivered[s], p->down));
    p->used[s] = true;
    ++p->submitted;
    return BIGCN_OK;
}

}  // namespace

bigcn_status bigcn_pipeline_submit(bigcn_pipeline* p, const float* X_host, float* logits_host)
{
    if (p && p->graph.n > 0 && !X_host) return fail(p->ctx, BIGCN_ERR_NULL, "X_host is null");
    return pipeline_submit_impl(p, X_host, nullptr, nullptr, logits_host);
}

bigcn_status bigcn_pipeline_submit_packed(bigcn_pipeline* p, const uint32_t* bits_host, const float* beta_host, float* logits_host)
{
    return pipeline_submit_impl(p, nullptr, bits_host, beta_host, logits_host);
}

bigcn_status bigcn_pipeline_wait(bigcn_pipeline* p)
{
    if (!p) return BIGCN_ERR_NULL;
    bigcn_ctx* ctx = p->ctx;
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (p->waited == p->submitted) return BIGCN_OK;
    const int s = (int)(p->waited % p->slots);
    ++p->waited;
    BIGCN_CUDA(ctx, cudaEventSynchronize(p->delivered[s]));
    return BIGCN_OK;
}

bigcn_status bigcn_pipeline_close(bigcn_pipeline* p)
{
    if (!p) return BIGCN_ERR_NULL;
    cudaSetDevice(p->ctx->device);
    if (p->up) cudaStreamSynchronize(p->up);
    cudaStreamSynchronize(p->ctx->stream);
    if (p->down) cudaStreamSynchronize(p->down);
    for (int s = 0; s < p->slots; ++s) {
        if (p->x_ready[s]) cudaEventDestroy(p->x_ready[s]);
        if (p->computed[s]) cudaEventDestroy(p->computed[s]);
        if (p->delivered[s]) cudaEventDestroy(p->delivered[s]);
    }
    if (p->up) cudaStreamDestroy(p->up);
    if (p->down) cudaStreamDestroy(p->down);
    delete p;
    return BIGCN_OK;
}

bigcn_status bigcn_col_stats(bigcn_ctx* ctx, const float* H, int64_t n, int32_t d, int64_t ld,
                             float eps, float* shift_out, float* scale_out)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (n < 0 || d < 1 || ld < d || !(eps >= 0.f)) return fail(ctx, BIGCN_ERR_SHAPE, "n=%lld d=%d ld=%lld eps=%g", (long long)n, d, (long long)ld, (double)eps);
    if (!shift_out || !scale_out || (n > 0 && !H)) return fail(ctx, BIGCN_ERR_NULL, "H, shift_out or scale_out is null");
    if (!ctx->ws || ctx->ws_bytes < col_stats_scratch_bytes(d)) return fail(ctx, BIGCN_ERR_WORKSPACE, "needs %zu bytes of workspace", col_stats_scratch_bytes(d));
    cudaError_t e = launch_col_stats(ctx->stream, H, n, d, ld, eps, shift_out, scale_out, ctx->ws, &ctx->launches_i);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "col_stats launch");
    return BIGCN_OK;
}

bigcn_status bigcn_entropy_bins(bigcn_ctx* ctx, const float* H, int64_t n, int32_t d, int64_t ld,
                                int32_t n_bins, float* col_min, float* col_max, uint32_t* counts,
                                double* entropy, double* total)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (n < 0 || n >= (int64_t(1) << 31) || d < 1 || ld < d || n_bins < 1)
        return fail(ctx, BIGCN_ERR_SHAPE, "n=%lld d=%d ld=%lld n_bins=%d", (long long)n, d, (long long)ld, n_bins);
    if (n_bins > entropy_max_bins()) return fail(ctx, BIGCN_ERR_UNSUPPORTED, "n_bins=%d exceeds %d", n_bins, entropy_max_bins());
    if (!col_min || !col_max || !counts || !entropy || !total || (n > 0 && !H))
        return fail(ctx, BIGCN_ERR_NULL, "H or an output is null");
    if (n == 0) {
        BIGCN_CUDA(ctx, cudaMemsetAsync(counts, 0, (size_t)d * n_bins * 4, ctx->stream));
        BIGCN_CUDA(ctx, cudaMemsetAsync(entropy, 0, (size_t)d * 8, ctx->stream));
        BIGCN_CUDA(ctx, cudaMemsetAsync(total, 0, 8, ctx->stream));
        return BIGCN_OK;
    }
    if (!ctx->ws || ctx->ws_bytes < entropy_scratch_bytes(d)) return fail(ctx, BIGCN_ERR_WORKSPACE, "needs %zu bytes of workspace", entropy_scratch_bytes(d));
    cudaError_t e = launch_entropy_bins(ctx->stream, H, n, d, ld, n_bins, col_min, col_max, counts, entropy, total,
                                        ctx->ws, &ctx->launches_i);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "entropy estimate launch");
    return BIGCN_OK;
}

size_t bigcn_backward_workspace_bytes(int64_t n, int32_t d_in, int32_t d_out)
{
    if (n < 0 || d_in < 1 || d_out < 1) return 0;
    return backward_scratch_bytes(n, d_in, d_out) + kAlign;
}

bigcn_status bigcn_layer_backward(bigcn_ctx* ctx, const bigcn_graph* graph, const bigcn_layer* layer,
                                  const float* W, int64_t ldw, const uint32_t* in_bits, const float* in_beta,
                                  const float* g_out, int64_t ldg, float* g_in, int64_t ldgi,
                                  float* g_w, int64_t ldgw)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if ((st = check_graph(ctx, graph)) != BIGCN_OK) return st;
    if ((st = check_layer(ctx, layer, "layer")) != BIGCN_OK) return st;
    const int32_t d_in = layer->d_in, d_out = layer->d_out;
    if (d_out > 512) return fail(ctx, BIGCN_ERR_UNSUPPORTED, "d_out=%d > 512", d_out);
    if (ldw < d_out || ldg < d_out || ldgw < d_out || (g_in && ldgi < d_in))
        return fail(ctx, BIGCN_ERR_SHAPE, "leading dimensions: ldw=%lld ldg=%lld ldgw=%lld ldgi=%lld", (long long)ldw, (long long)ldg, (long long)ldgw, (long long)ldgi);
    if (!W || !g_w) return fail(ctx, BIGCN_ERR_NULL, "W or g_w is null");
    const int64_t n = graph->n;
    if (n > 0 && (!in_bits || !in_beta || !g_out)) return fail(ctx, BIGCN_ERR_NULL, "in_bits, in_beta or g_out is null");
    if (n == 0) {                                             // no nodes: every sum over the nodes is empty
        BIGCN_CUDA(ctx, cudaMemset2DAsync(g_w, (size_t)ldgw * 4, 0, (size_t)d_out * 4, (size_t)d_in, ctx->stream));
        return BIGCN_OK;
    }
    if (!ctx->ws || ctx->ws_bytes < backward_scratch_bytes(n, d_in, d_out))
        return fail(ctx, BIGCN_ERR_WORKSPACE, "needs %zu bytes of workspace (bigcn_backward_workspace_bytes)", backward_scratch_bytes(n, d_in, d_out));
    cudaError_t e = launch_layer_backward(ctx->stream, n, graph->rowptr, graph->colidx, graph->val, d_in, d_out, W, ldw,
                                          layer->alpha, in_bits, bigcn_packed_stride_words(d_in), in_beta, g_out, ldg,
                                          g_in, ldgi, g_w, ldgw, ctx->long_row ? ctx->long_row : kDefaultLongRow, ctx->ws,
                                          &ctx->launches_i);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "backward launch");
    return BIGCN_OK;
}

bigcn_status bigcn_measure_popc_peak(bigcn_ctx* ctx, double* word_steps_per_s)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (!word_steps_per_s) return fail(ctx, BIGCN_ERR_NULL, "word_steps_per_s is null");
    if (!ctx->ws || ctx->ws_bytes < popc_peak_scratch_bytes()) return fail(ctx, BIGCN_ERR_WORKSPACE, "needs %zu bytes of workspace", popc_peak_scratch_bytes());
    cudaError_t e = measure_popc_peak(ctx->stream, ctx->ws, word_steps_per_s, &ctx->launches_i);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "popcount peak measurement");
    return BIGCN_OK;
}

bigcn_status bigcn_measure_gather_peak(bigcn_ctx* ctx, const bigcn_graph* g, int32_t row_bytes, double* ms)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if ((st = check_graph(ctx, g)) != BIGCN_OK) return st;
    if (!ms) return fail(ctx, BIGCN_ERR_NULL, "ms is null");
    if (row_bytes < 16 || row_bytes > 512 || (row_bytes & (row_bytes - 1))) return fail(ctx, BIGCN_ERR_SHAPE, "row_bytes=%d must be a power of two in 16..512", row_bytes);
    const size_t need = up((size_t)g->n * (size_t)row_bytes) + 256;
    if (!ctx->ws || ctx->ws_bytes < need) return fail(ctx, BIGCN_ERR_WORKSPACE, "needs %zu bytes of workspace", need);
    *ms = 0.0;
    if (g->n == 0 || g->nnz == 0) return BIGCN_OK;
    cudaError_t e = measure_gather_peak(ctx->stream, g->colidx, g->nnz, ctx->ws, row_bytes,
                                        static_cast<char*>(ctx->ws) + up((size_t)g->n * (size_t)row_bytes), ms, &ctx->launches_i);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "gather measurement");
    return BIGCN_OK;
}

bigcn_status bigcn_mean_adjacency(bigcn_ctx* ctx, int64_t n, int64_t nnz_in,
                                  const int64_t* rowptr_A, const int32_t* colidx_A,
                                  int64_t* rowptr, int32_t* colidx, float* val, float* inv_deg,
                                  int64_t* nnz_out)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if (n < 0 || n >= (int64_t(1) << 31) || nnz_in < 0) return fail(ctx, BIGCN_ERR_SHAPE, "n=%lld nnz_in=%lld out of range", (long long)n, (long long)nnz_in);
    if (!nnz_out) return fail(ctx, BIGCN_ERR_NULL, "nnz_out is null");
    if (!rowptr) return fail(ctx, BIGCN_ERR_NULL, "rowptr output is null");
    *nnz_out = 0;
    if (n == 0) {
        BIGCN_CUDA(ctx, cudaMemsetAsync(rowptr, 0, sizeof(int64_t), ctx->stream));
        BIGCN_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        return BIGCN_OK;
    }
    if (!rowptr_A || (nnz_in > 0 && (!colidx_A || !colidx || !val)) || !inv_deg) return fail(ctx, BIGCN_ERR_NULL, "an input or output array is null");
    if (!ctx->ws || ctx->ws_bytes < normalize_scratch_bytes(n)) return fail(ctx, BIGCN_ERR_WORKSPACE, "needs %zu bytes of workspace", normalize_scratch_bytes(n));
    cudaError_t e = launch_normalize_adjacency(ctx->stream, n, nnz_in, rowptr_A, colidx_A, rowptr, colidx, val, inv_deg,
                                               ctx->ws, ctx->d_flag, &ctx->launches_i, /*mean=*/true);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "mean_adjacency launch");
    int flag = 0;
    int64_t total = 0;
    BIGCN_CUDA(ctx, cudaMemcpyAsync(&flag, ctx->d_flag, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    BIGCN_CUDA(ctx, cudaMemcpyAsync(&total, rowptr + n, sizeof(int64_t), cudaMemcpyDeviceToHost, ctx->stream));
    BIGCN_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (flag)
        return fail(ctx, BIGCN_ERR_GRAPH, "adjacency input rejected:%s%s%s%s",
                    (flag & 8) ? " rowptr not monotone from 0 to nnz;" : "",
                    (flag & 2) ? " column index outside [0, n);" : "",
                    (flag & 1) ? " columns not ascending and unique within a row;" : "",
                    (flag & 4) ? " pattern not symmetric;" : "");
    *nnz_out = total;
    return BIGCN_OK;
}

bigcn_status bigcn_sage_layer_forward(bigcn_ctx* ctx, const bigcn_graph* mean_graph,
                                      const bigcn_layer* self_layer, const bigcn_layer* nbr_layer,
                                      const uint32_t* in_bits, const float* in_beta,
                                      float* h_out, int64_t ldh,
                                      const bigcn_layer* next, uint32_t* next_bits, float* next_beta)
{
    bigcn_status st = bind_device(ctx);
    if (st != BIGCN_OK) return st;
    if ((st = check_graph(ctx, mean_graph)) != BIGCN_OK) return st;
    if ((st = check_layer(ctx, self_layer, "self_layer")) != BIGCN_OK) return st;
    if ((st = check_layer(ctx, nbr_layer, "nbr_layer")) != BIGCN_OK) return st;
    if (self_layer->d_in != nbr_layer->d_in || self_layer->d_out != nbr_layer->d_out)
        return fail(ctx, BIGCN_ERR_SHAPE, "self and neighbour weights differ in shape (%dx%d vs %dx%d)", self_layer->d_in, self_layer->d_out, nbr_layer->d_in, nbr_layer->d_out);
    const int d_in = self_layer->d_in, d_out = self_layer->d_out;
    if (next) {
        if (next->d_in != d_out) return fail(ctx, BIGCN_ERR_SHAPE, "next->d_in=%d != d_out=%d", next->d_in, d_out);
        if ((next->in_shift == nullptr) != (next->in_scale == nullptr)) return fail(ctx, BIGCN_ERR_NULL, "next: in_shift and in_scale go together");
    }
    if (h_out && ldh < d_out) return fail(ctx, BIGCN_ERR_SHAPE, "ldh=%lld < d_out=%d", (long long)ldh, d_out);
    const int64_t n = mean_graph->n;
    if (n == 0) return BIGCN_OK;
    if (!in_bits || !in_beta) return fail(ctx, BIGCN_ERR_NULL, "in_bits or in_beta is null");
    if (!aligned(in_bits, 16)) return fail(ctx, BIGCN_ERR_ALIGN, "in_bits must be 16-byte aligned");
    if (next && (!next_bits || !next_beta)) return fail(ctx, BIGCN_ERR_NULL, "next_bits or next_beta is null");
    if (!h_out && !next) return fail(ctx, BIGCN_ERR_NULL, "neither h_out nor next is given: nothing to compute");
    const int32_t dims[2] = {d_in, d_out};
    const size_t zbytes = up(zeta_bytes_max(n, dims, 1));                 // fp32 size: room for either form
    const size_t need = 2 * zbytes + up(spmm_scratch_bytes(n, mean_graph->nnz, d_out));
    if (!ctx->ws || ctx->ws_bytes < need) return fail(ctx, BIGCN_ERR_WORKSPACE, "needs %zu bytes of workspace, has %zu", need, ctx->ws_bytes);
    char* base = static_cast<char*>(ctx->ws);
    float* zeta_self = reinterpret_cast<float*>(base);                   // literal fp32 zeta of the node's own term
    void* zeta_nbr = base + zbytes;
    void* counter = base + 2 * zbytes;
    const int64_t stride_in = bigcn_packed_stride_words(d_in);
    const int64_t ld_self = zeta_ld(d_out, kZetaF32);
    cudaError_t e = launch_bitgemm(ctx->stream, in_bits, stride_in, self_layer->w_bitsT, stride_in, n, d_in, d_out,
                                   in_beta, self_layer->alpha, kZetaF32, zeta_self, ld_self, nullptr, nullptr, &ctx->launches_i, ctx->contraction);
    if (e != cudaSuccess) { finish_call(ctx); return cuda_fail(ctx, e, "bit-GEMM (self term) launch"); }
    const int fmt = pick_format(ctx, d_in, d_out, n);
    const int64_t ldz = zeta_ld(d_out, fmt);
    e = launch_bitgemm(ctx->stream, in_bits, stride_in, nbr_layer->w_bitsT, stride_in, n, d_in, d_out,
                       in_beta, nbr_layer->alpha, fmt, zeta_nbr, ldz, nullptr, nullptr, &ctx->launches_i, ctx->contraction);
    if (e != cudaSuccess) { finish_call(ctx); return cuda_fail(ctx, e, "bit-GEMM (neighbour term) launch"); }
    SpmmArgs a;
    a.n = n;
    a.nnz = mean_graph->nnz;
    a.rowptr = mean_graph->rowptr;
    a.colidx = mean_graph->colidx;
    a.val = mean_graph->val;
    a.fmt = fmt;
    a.zeta = zeta_nbr;
    a.ldz = ldz;
    a.d_out = d_out;
    a.node_w = in_beta;
    a.col_w = nbr_layer->alpha;
    a.add = zeta_self;
    a.byte_path = ctx->byte_path;
    a.ld_add = ld_self;
    a.h_out = h_out;
    a.ldh = ldh;
    a.next_bits = next ? next_bits : nullptr;
    a.next_stride = next ? bigcn_packed_stride_words(d_out) : 0;
    a.next_beta = next ? next_beta : nullptr;
    a.next_shift = next ? next->in_shift : nullptr;
    a.next_scale = next ? next->in_scale : nullptr;
    a.long_row = ctx->long_row > 0 ? ctx->long_row : kDefaultLongRow;
    a.scratch = counter;
    a.scratch_bytes = spmm_scratch_bytes(n, mean_graph->nnz, d_out);
    e = launch_spmm(ctx->stream, a, &ctx->launches_i);
    finish_call(ctx);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "SpMM launch");
    return BIGCN_OK;
}

}  // extern "C"
