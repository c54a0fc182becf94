// C ABI of the TAQ library: host-side validation and kernel dispatch.  Nothing here allocates device memory.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>

#include "taq_common.cuh"
#include "taq_ptx.cuh"
#include "taq_sm100.cuh"

namespace taq {

__device__ int g_status_word[2];   // {code, block id}; raised by kernels, read by taq_poll_device_status

static thread_local char tl_error[512] = "";

static taq_status fail(taq_status s, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(tl_error, sizeof(tl_error), fmt, ap);
    va_end(ap);
    return s;
}

static taq_status cuda_fail(cudaError_t e, const char* what) {
    return fail(TAQ_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Address of the status word on the current device (looked up once per device).
static taq_status status_ptr(int** out) {
    static int* cache[64] = {nullptr};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return fail(TAQ_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
    if (!cache[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_status_word);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(status word)");
        cache[dev] = static_cast<int*>(p);
    }
    *out = cache[dev];
    return TAQ_OK;
}

static taq_status check_weight_desc(const taq_weight_desc* d) {
    if (!d) return fail(TAQ_ERR_INVALID_ARG, "weight descriptor is NULL");
    if (d->bits != 4 && d->bits != 8) return fail(TAQ_ERR_INVALID_ARG, "bits must be 4 or 8, got %d", d->bits);
    if (d->n_out < 1 || d->k_in < 8 || d->k_in % 8) return fail(TAQ_ERR_SHAPE, "n_out >= 1 and k_in a positive multiple of 8 required (n_out=%d k_in=%d)", d->n_out, d->k_in);
    if (d->group < 0 || (d->group && d->group % 32)) return fail(TAQ_ERR_SHAPE, "group must be 0 or a multiple of 32, got %d", d->group);
    if (d->bits == 8 && d->group != 0) return fail(TAQ_ERR_UNSUPPORTED, "8-bit weights take one scale per output channel (group = 0)");
    if ((long long)d->n_out * d->k_in > (1LL << 40)) return fail(TAQ_ERR_SHAPE, "matrix too large");
    return TAQ_OK;
}

static taq_status check_layer_desc(const taq_layer_desc* d) {
    if (!d) return fail(TAQ_ERR_INVALID_ARG, "layer descriptor is NULL");
    if (d->batch < 0 || d->n_query < 0) return fail(TAQ_ERR_SHAPE, "negative batch or n_query");
    if (d->heads < 1 || d->channels < 8 || d->channels % d->heads) return fail(TAQ_ERR_SHAPE, "channels (%d) must be a positive multiple of heads (%d)", d->channels, d->heads);
    const int dh = d->channels / d->heads;
    if (dh % 8 || dh > kMaxHeadDim) return fail(TAQ_ERR_SHAPE, "head width %d must be a multiple of 8, at most %d", dh, kMaxHeadDim);
    if (d->n_ctx < 1 || d->n_ctx > kMaxCtx) return fail(TAQ_ERR_SHAPE, "n_ctx must be in [1,%d], got %d", kMaxCtx, d->n_ctx);
    if (d->ctx_dim < 8 || d->ctx_dim % 8) return fail(TAQ_ERR_SHAPE, "ctx_dim must be a positive multiple of 8, got %d", d->ctx_dim);
    if (d->w_bits != 4 && d->w_bits != 8) return fail(TAQ_ERR_INVALID_ARG, "w_bits must be 4 or 8, got %d", d->w_bits);
    if (d->q_bits != 0 && d->q_bits != 8) return fail(TAQ_ERR_INVALID_ARG, "q_bits must be 0 or 8, got %d", d->q_bits);
    if (d->kv_bits != 8 && d->kv_bits != 4) return fail(TAQ_ERR_UNSUPPORTED, "kv_bits must be 8 or 4, got %d", d->kv_bits);
    if (d->p_bits != 8 && d->p_bits != 4) return fail(TAQ_ERR_UNSUPPORTED, "p_bits must be 8 or 4, got %d", d->p_bits);
    if (d->p_log != 0 && d->p_log != 1) return fail(TAQ_ERR_INVALID_ARG, "p_log must be 0 or 1, got %d", d->p_log);
    if (d->max_trigger < 0 || d->max_trigger > d->n_ctx) return fail(TAQ_ERR_SHAPE, "max_trigger must be in [0,n_ctx], got %d", d->max_trigger);
    if ((long long)d->batch * d->n_query > (1LL << 31) - 1) return fail(TAQ_ERR_SHAPE, "batch * n_query too large");
    taq_weight_desc w{d->channels, d->channels, d->w_bits, d->w_group};
    return check_weight_desc(&w);
}

#define TAQ_REQUIRE_PTR(p)                                                              \
    do {                                                                                \
        if (!(p)) return fail(TAQ_ERR_INVALID_ARG, #p " is NULL");                      \
        if (!aligned16(p)) return fail(TAQ_ERR_ALIGNMENT, #p " is not 16-byte aligned"); \
    } while (0)

// Workspace of taq_layer_forward: Q~ (int8 or fp16), its scales, O (fp16); each section 128-byte aligned.
struct Workspace { size_t off_q, off_qs, off_o, total; };
static Workspace workspace_layout(const taq_layer_desc* d, int n_requests) {
    const size_t rows = (size_t)d->batch * d->n_query * n_requests;
    Workspace w;
    w.off_q = 0;
    w.off_qs = align_up(rows * d->channels * (d->q_bits == 8 ? 1 : 2), 128);
    w.off_o = w.off_qs + align_up(rows * d->heads * sizeof(float), 128);
    w.total = w.off_o + align_up(rows * d->channels * sizeof(__half), 128);
    return w;
}

// Launches per kernel family since the last taq_dispatch_reset (host-side counters; see taq_dispatch_counts in taq.h).
static std::atomic<long long> g_dispatch[TAQ_N_KERNEL_FAMILIES];
static void count_launch(int family) { g_dispatch[family].fetch_add(1, std::memory_order_relaxed); }

static taq_status run_linear(const LinearArgs& a, int n_z, cudaStream_t st) {
    cudaError_t e;
    if (sm100_linear_supported(a)) { count_launch(TAQ_KERNEL_LINEAR_TENSOR); e = launch_linear_sm100(a, n_z, st); }
    else { count_launch(TAQ_KERNEL_LINEAR_GENERIC); e = launch_linear_simt(a, n_z, st); }
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "dequant-GEMM launch");
}

static taq_status run_attention(const AttnArgs& a, int n_z, cudaStream_t st) {
    cudaError_t e;
    // C = 320 / 8 heads: up to one wave of CTAs the head-parallel kernel (four heads of a row tile at once) is the shorter
    // chain; beyond that the per-head kernel, which keeps two CTAs on an SM, has the higher throughput.
    const long long c320_ctas = (long long)((a.n_query + 127) / 128) * 2 * n_z;
    if (c320_ctas <= 148 && sm100_attention_c320_supported(a)) { count_launch(TAQ_KERNEL_ATTENTION_TENSOR); e = launch_attention_c320(a, n_z, st); }
    else if (sm100_attention_supported(a)) { count_launch(TAQ_KERNEL_ATTENTION_TENSOR); e = launch_attention_sm100(a, n_z, st); }
    else { count_launch(TAQ_KERNEL_ATTENTION_GENERIC); e = launch_attention_simt(a, n_z, st); }
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "attention launch");
}

// A kernel whose only work is a wait that nothing satisfies: the barrier is initialised and no arrival or copy is ever
// directed at it, so the bounded wait runs out after `limit` cycles, the block records TAQ_ERR_TIMEOUT and returns.
__global__ void wait_expiry_kernel(long long limit, int* status) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        ptx::mbar_init(&bar, 1);
        ptx::mbar_fence_init();
        if (!ptx::mbar_wait(&bar, 0, limit)) raise_status(status, TAQ_ERR_TIMEOUT);
    }
}

}  // namespace taq

using namespace taq;

extern "C" {

const char* taq_status_string(taq_status s) {
    switch (s) {
        case TAQ_OK: return "ok";
        case TAQ_ERR_INVALID_ARG: return "invalid argument";
        case TAQ_ERR_SHAPE: return "unsupported shape";
        case TAQ_ERR_ALIGNMENT: return "misaligned pointer";
        case TAQ_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case TAQ_ERR_UNSUPPORTED: return "unsupported";
        case TAQ_ERR_CUDA: return "CUDA error";
        case TAQ_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

const char* taq_last_error(void) { return tl_error; }
int taq_version(void) { return 1; }

size_t taq_packed_weight_bytes(const taq_weight_desc* d) {
    if (check_weight_desc(d) != TAQ_OK) return 0;
    return weight_layout(d->n_out, d->k_in, d->bits, d->group).total;
}

taq_status taq_pack_weights(const taq_weight_desc* d, const float* W_dev, const float* bias_dev, void* packed_dev,
                            size_t packed_bytes, void* stream) {
    taq_status s = check_weight_desc(d);
    if (s != TAQ_OK) return s;
    TAQ_REQUIRE_PTR(W_dev);
    TAQ_REQUIRE_PTR(packed_dev);
    if (bias_dev && !aligned16(bias_dev)) return fail(TAQ_ERR_ALIGNMENT, "bias_dev is not 16-byte aligned");
    const size_t need = taq_packed_weight_bytes(d);
    if (packed_bytes < need) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "packed buffer has %zu bytes, %zu needed", packed_bytes, need);
    cudaError_t e = launch_pack_weights(*d, W_dev, bias_dev, packed_dev, (cudaStream_t)stream);
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "pack_weights launch");
}

taq_status taq_unpack_weights(const taq_weight_desc* d, const void* packed_dev, int8_t* codes_dev, float* scales_dev, void* stream) {
    taq_status s = check_weight_desc(d);
    if (s != TAQ_OK) return s;
    TAQ_REQUIRE_PTR(packed_dev);
    TAQ_REQUIRE_PTR(codes_dev);
    TAQ_REQUIRE_PTR(scales_dev);
    cudaError_t e = launch_unpack_weights(*d, packed_dev, codes_dev, scales_dev, (cudaStream_t)stream);
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "unpack_weights launch");
}

taq_status taq_quantize_rows(const float* x_dev, int64_t rows, int32_t cols, int32_t qmax, int8_t* codes_dev, float* scales_dev, void* stream) {
    if (rows < 0 || cols < 1) return fail(TAQ_ERR_SHAPE, "rows >= 0 and cols >= 1 required (rows=%lld cols=%d)", (long long)rows, cols);
    if (qmax < 1 || qmax > 127) return fail(TAQ_ERR_INVALID_ARG, "qmax must be in [1,127], got %d", qmax);
    if (rows == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(x_dev);
    TAQ_REQUIRE_PTR(codes_dev);
    TAQ_REQUIRE_PTR(scales_dev);
    cudaError_t e = launch_quantize_rows(x_dev, rows, cols, qmax, codes_dev, scales_dev, (cudaStream_t)stream);
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "quantize_rows launch");
}

taq_status taq_kv_layout_of(const taq_layer_desc* d, taq_kv_layout* out) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (!out) return fail(TAQ_ERR_INVALID_ARG, "out is NULL");
    *out = kv_layout(d->heads, d->n_ctx, d->channels / d->heads, d->max_trigger);
    return TAQ_OK;
}

size_t taq_kv_bytes(const taq_layer_desc* d) {
    if (check_layer_desc(d) != TAQ_OK) return 0;
    return kv_layout(d->heads, d->n_ctx, d->channels / d->heads, d->max_trigger).block_bytes * (size_t)d->batch;
}

static taq_status kv_project_impl(const taq_layer_desc* d, const taq_request* reqs, int n_z, const void* ctx, const void* Wk,
                                  const void* Wv, const uint8_t* mask, void* kv, cudaStream_t st) {
    int* status = nullptr;
    taq_status s = status_ptr(&status);
    if (s != TAQ_OK) return s;
    LinearArgs a{};
    a.x = (const __half*)ctx;
    a.reqs = reqs;
    a.y = kv;
    a.mask = mask;
    a.rows = (long long)d->batch * d->n_ctx;
    a.n_out = d->channels; a.k_in = d->ctx_dim; a.bits = d->w_bits; a.group = d->w_group;
    a.heads = d->heads; a.n_ctx = d->n_ctx; a.max_trigger = d->max_trigger;
    a.epi = EPI_KV; a.kv_qmax = d->kv_bits == 4 ? 7 : 127;
    a.status = status;
    for (int which = 0; which < 2; ++which) {
        a.w = which ? Wv : Wk;
        a.which = which;
        a.kv_which = which;
        s = run_linear(a, n_z, st);
        if (s != TAQ_OK) return s;
    }
    // the same rows once more as MMA-ready operand images for the attention kernel
    cudaError_t e = launch_kv_operands(*d, kv, reqs, reqs ? n_z : d->batch, st);
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "K/V operand image launch");
}

taq_status taq_kv_project(const taq_layer_desc* d, const void* ctx_f16_dev, const void* Wk_packed_dev, const void* Wv_packed_dev,
                          const uint8_t* trig_mask_dev, void* kv_packed_dev, size_t kv_bytes, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch == 0) return TAQ_OK;
    if (d->batch > 65535) return fail(TAQ_ERR_SHAPE, "batch must be at most 65535");
    TAQ_REQUIRE_PTR(ctx_f16_dev);
    TAQ_REQUIRE_PTR(Wk_packed_dev);
    TAQ_REQUIRE_PTR(Wv_packed_dev);
    TAQ_REQUIRE_PTR(kv_packed_dev);
    if (!trig_mask_dev) return fail(TAQ_ERR_INVALID_ARG, "trig_mask_dev is NULL");
    const size_t need = taq_kv_bytes(d);
    if (kv_bytes < need) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "kv buffer has %zu bytes, %zu needed", kv_bytes, need);
    return kv_project_impl(d, nullptr, 1, ctx_f16_dev, Wk_packed_dev, Wv_packed_dev, trig_mask_dev, kv_packed_dev, (cudaStream_t)stream);
}

taq_status taq_kv_finalize(const taq_layer_desc* d, void* kv_packed_dev, size_t kv_bytes, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch == 0) return TAQ_OK;
    if (d->batch > 65535) return fail(TAQ_ERR_SHAPE, "batch must be at most 65535");
    TAQ_REQUIRE_PTR(kv_packed_dev);
    const size_t need = taq_kv_bytes(d);
    if (kv_bytes < need) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "kv buffer has %zu bytes, %zu needed", kv_bytes, need);
    cudaError_t e = launch_kv_operands(*d, kv_packed_dev, nullptr, d->batch, (cudaStream_t)stream);
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "K/V operand image launch");
}

taq_status taq_kv_project_batched(const taq_layer_desc* d, const taq_request* reqs_dev, int32_t n_requests, const void* ctx_f16_dev, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch != 1) return fail(TAQ_ERR_SHAPE, "batched calls take one sequence per request (desc->batch must be 1)");
    if (n_requests < 0 || n_requests > 65535) return fail(TAQ_ERR_SHAPE, "n_requests must be in [0,65535]");
    if (n_requests == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(reqs_dev);
    TAQ_REQUIRE_PTR(ctx_f16_dev);
    return kv_project_impl(d, reqs_dev, n_requests, ctx_f16_dev, nullptr, nullptr, nullptr, nullptr, (cudaStream_t)stream);
}

taq_status taq_quantized_linear(const taq_weight_desc* d, const void* x_f16_dev, int64_t rows, const void* W_packed_dev, void* y_dev,
                                int32_t out_kind, int32_t heads, float* scales_dev, void* stream) {
    taq_status s = check_weight_desc(d);
    if (s != TAQ_OK) return s;
    if (rows < 0 || rows > (1LL << 31) - 1) return fail(TAQ_ERR_SHAPE, "rows out of range");
    if (out_kind != TAQ_OUT_F16 && out_kind != TAQ_OUT_F32 && out_kind != TAQ_OUT_INT8_HEAD_ROWS) return fail(TAQ_ERR_INVALID_ARG, "unknown out_kind %d", out_kind);
    if (d->n_out % 8) return fail(TAQ_ERR_SHAPE, "n_out must be a multiple of 8 for a dequant-GEMM, got %d", d->n_out);
    if (out_kind == TAQ_OUT_INT8_HEAD_ROWS) {
        if (heads < 1 || d->n_out % heads) return fail(TAQ_ERR_SHAPE, "n_out (%d) must be a multiple of heads (%d)", d->n_out, heads);
        const int dh = d->n_out / heads;
        if (dh % 8 || dh > kMaxHeadDim) return fail(TAQ_ERR_SHAPE, "head width %d must be a multiple of 8, at most %d", dh, kMaxHeadDim);
        if (heads > 65535) return fail(TAQ_ERR_SHAPE, "too many heads");
    }
    if (rows == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(x_f16_dev);
    TAQ_REQUIRE_PTR(W_packed_dev);
    TAQ_REQUIRE_PTR(y_dev);
    if (out_kind == TAQ_OUT_INT8_HEAD_ROWS) TAQ_REQUIRE_PTR(scales_dev);
    int* status = nullptr;
    s = status_ptr(&status);
    if (s != TAQ_OK) return s;
    LinearArgs a{};
    a.x = (const __half*)x_f16_dev;
    a.w = W_packed_dev;
    a.y = y_dev;
    a.scales = scales_dev;
    a.rows = rows;
    a.n_out = d->n_out; a.k_in = d->k_in; a.bits = d->bits; a.group = d->group;
    a.heads = out_kind == TAQ_OUT_INT8_HEAD_ROWS ? heads : 1;
    a.epi = out_kind == TAQ_OUT_F16 ? EPI_F16 : out_kind == TAQ_OUT_F32 ? EPI_F32 : EPI_Q8_HEAD;
    a.status = status;
    return run_linear(a, 1, (cudaStream_t)stream);
}

static AttnArgs attn_args(const taq_layer_desc* d, int* status) {
    AttnArgs a{};
    a.batch = d->batch; a.n_query = d->n_query; a.channels = d->channels; a.heads = d->heads; a.n_ctx = d->n_ctx;
    a.max_trigger = d->max_trigger; a.q_bits = d->q_bits; a.p_bits = d->p_bits; a.p_log = d->p_log;
    a.status = status;
    return a;
}

taq_status taq_cross_attention(const taq_layer_desc* d, const void* q_dev, const float* q_scales_dev, const void* kv_packed_dev,
                               const uint8_t* trig_mask_dev, void* o_f16_dev, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch > 65535) return fail(TAQ_ERR_SHAPE, "batch must be at most 65535");
    if (d->batch == 0 || d->n_query == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(q_dev);
    if (d->q_bits == 8) TAQ_REQUIRE_PTR(q_scales_dev);
    TAQ_REQUIRE_PTR(kv_packed_dev);
    TAQ_REQUIRE_PTR(o_f16_dev);
    if (!trig_mask_dev) return fail(TAQ_ERR_INVALID_ARG, "trig_mask_dev is NULL");
    int* status = nullptr;
    s = status_ptr(&status);
    if (s != TAQ_OK) return s;
    AttnArgs a = attn_args(d, status);
    a.q = q_dev; a.q_scales = q_scales_dev; a.kv = kv_packed_dev; a.mask = trig_mask_dev; a.o = (__half*)o_f16_dev;
    return run_attention(a, d->batch, (cudaStream_t)stream);
}

size_t taq_workspace_bytes(const taq_layer_desc* d, int32_t n_requests) {
    if (check_layer_desc(d) != TAQ_OK || n_requests < 1) return 0;
    return workspace_layout(d, n_requests).total;
}

// x -> O: to_q, Q~ = Q_a(Q), attention.  One kernel where the fused kernel covers the shape, otherwise two with Q~
// in the workspace.
static taq_status q_attention_impl(const taq_layer_desc* d, const taq_request* reqs, int n_req, const void* x, const void* Wq, const void* kv,
                                   const uint8_t* mask, void* o_dst, void* ws, int* status, cudaStream_t st) {
    const Workspace W = workspace_layout(d, n_req);
    uint8_t* wsb = (uint8_t*)ws;
    const long long rows_per_z = (long long)d->batch * d->n_query;   // weights are shared by the whole batch
    if (sm100_qattn_supported(*d)) {
        count_launch(TAQ_KERNEL_QUERY_ATTENTION_FUSED);
        cudaError_t e = launch_qattn_sm100(*d, (const __half*)x, Wq, kv, reqs, (__half*)o_dst, reqs ? n_req : d->batch, status, st);
        return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "fused to_q + attention launch");
    }
    LinearArgs q{};                                                     // to_q (+ Q~ = Q_a(Q))
    q.x = (const __half*)x; q.w = Wq; q.reqs = reqs; q.which = 0;
    q.y = wsb + W.off_q; q.scales = (float*)(wsb + W.off_qs);
    q.rows = rows_per_z; q.n_out = d->channels; q.k_in = d->channels; q.bits = d->w_bits; q.group = d->w_group;
    q.heads = d->q_bits == 8 ? d->heads : 1;
    q.epi = d->q_bits == 8 ? EPI_Q8_HEAD : EPI_F16;
    q.status = status;
    taq_status s = run_linear(q, n_req, st);
    if (s != TAQ_OK) return s;

    AttnArgs at = attn_args(d, status);                                 // softmax(Q~K~^T/sqrt(d)), Eq. 3, P.V
    at.q = wsb + W.off_q; at.q_scales = (const float*)(wsb + W.off_qs); at.kv = kv; at.mask = mask; at.reqs = reqs;
    at.o = (__half*)o_dst;
    at.early_kv = 1;            // the kernel before it in the stream is to_q above, which writes the workspace only
    return run_attention(at, reqs ? n_req : d->batch, st);
}

static taq_status layer_forward_impl(const taq_layer_desc* d, const taq_request* reqs, int n_req, const void* x, const void* Wq,
                                     const void* Wout, const void* kv, const uint8_t* mask, void* y, void* ws, cudaStream_t st) {
    int* status = nullptr;
    taq_status s = status_ptr(&status);
    if (s != TAQ_OK) return s;
    if (sm100_layer_supported(*d)) {                                    // the whole pass in one kernel
        count_launch(TAQ_KERNEL_LAYER_FUSED);
        cudaError_t e = launch_layer_sm100(*d, (const __half*)x, Wq, Wout, kv, reqs, (__half*)y, reqs ? n_req : d->batch, status, st);
        return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "fused layer launch");
    }
    const Workspace W = workspace_layout(d, n_req);
    uint8_t* wsb = (uint8_t*)ws;
    s = q_attention_impl(d, reqs, n_req, x, Wq, kv, mask, wsb + W.off_o, ws, status, st);
    if (s != TAQ_OK) return s;

    LinearArgs o{};                                                     // to_out (+ bias)
    o.x = (const __half*)(wsb + W.off_o); o.w = Wout; o.reqs = reqs; o.which = 1;
    o.y = y;
    o.rows = (long long)d->batch * d->n_query; o.n_out = d->channels; o.k_in = d->channels; o.bits = d->w_bits; o.group = d->w_group;
    o.heads = 1; o.epi = EPI_F16; o.status = status;
    o.early_weights = 1;        // the kernel before it in the stream is the attention above, which writes O only
    return run_linear(o, n_req, st);
}

taq_status taq_layer_forward(const taq_layer_desc* d, const void* x_f16_dev, const void* Wq_packed_dev, const void* Wout_packed_dev,
                             const void* kv_packed_dev, const uint8_t* trig_mask_dev, void* y_f16_dev, void* workspace_dev,
                             size_t workspace_bytes, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch > 65535) return fail(TAQ_ERR_SHAPE, "batch must be at most 65535");
    if (d->batch == 0 || d->n_query == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(x_f16_dev);
    TAQ_REQUIRE_PTR(Wq_packed_dev);
    TAQ_REQUIRE_PTR(Wout_packed_dev);
    TAQ_REQUIRE_PTR(kv_packed_dev);
    TAQ_REQUIRE_PTR(y_f16_dev);
    TAQ_REQUIRE_PTR(workspace_dev);
    if (!trig_mask_dev) return fail(TAQ_ERR_INVALID_ARG, "trig_mask_dev is NULL");
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 127u) return fail(TAQ_ERR_ALIGNMENT, "workspace_dev is not 128-byte aligned");
    const size_t need = taq_workspace_bytes(d, 1);
    if (workspace_bytes < need) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    return layer_forward_impl(d, nullptr, 1, x_f16_dev, Wq_packed_dev, Wout_packed_dev, kv_packed_dev, trig_mask_dev, y_f16_dev,
                              workspace_dev, (cudaStream_t)stream);
}

// ---- integer-activation variants (a_bits = 8): per-token int8 inputs of the projections ----------------------------

taq_status taq_quantize_rows_f16(const void* x_f16_dev, int64_t rows, int32_t cols, int8_t* codes_dev, float* scales_dev, void* stream) {
    if (rows < 0 || cols < 8 || cols % 8) return fail(TAQ_ERR_SHAPE, "rows >= 0 and cols a positive multiple of 8 required (rows=%lld cols=%d)", (long long)rows, cols);
    if (rows == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(x_f16_dev);
    TAQ_REQUIRE_PTR(codes_dev);
    TAQ_REQUIRE_PTR(scales_dev);
    cudaError_t e = launch_quantize_rows_f16((const __half*)x_f16_dev, rows, cols, codes_dev, scales_dev, (cudaStream_t)stream);
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "quantize_rows_f16 launch");
}

static taq_status run_linear_i8(const LinearArgs& a, cudaStream_t st) {
    count_launch(TAQ_KERNEL_LINEAR_TENSOR);
    if (!sm100_linear_supported(a))
        return fail(TAQ_ERR_UNSUPPORTED, "integer-activation GEMM: needs k_in a multiple of 16, group 0 or 128, n_out a multiple of 64 or 80 (per-head output: head width 40, 64, 80 or 160)");
    cudaError_t e = launch_linear_sm100(a, 1, st);
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "integer-activation GEMM launch");
}

taq_status taq_quantized_linear_i8(const taq_weight_desc* d, const int8_t* x_codes_dev, const float* x_scales_dev, int64_t rows,
                                   const void* W_packed_dev, void* y_dev, int32_t out_kind, int32_t heads, float* scales_dev, void* stream) {
    taq_status s = check_weight_desc(d);
    if (s != TAQ_OK) return s;
    if (rows < 0 || rows > (1LL << 31) - 1) return fail(TAQ_ERR_SHAPE, "rows out of range");
    if (out_kind != TAQ_OUT_F16 && out_kind != TAQ_OUT_F32 && out_kind != TAQ_OUT_INT8_HEAD_ROWS) return fail(TAQ_ERR_INVALID_ARG, "unknown out_kind %d", out_kind);
    if (out_kind == TAQ_OUT_INT8_HEAD_ROWS) {
        if (heads < 1 || d->n_out % heads) return fail(TAQ_ERR_SHAPE, "n_out (%d) must be a multiple of heads (%d)", d->n_out, heads);
        if (heads > 65535) return fail(TAQ_ERR_SHAPE, "too many heads");
    }
    if (rows == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(x_codes_dev);
    TAQ_REQUIRE_PTR(x_scales_dev);
    TAQ_REQUIRE_PTR(W_packed_dev);
    TAQ_REQUIRE_PTR(y_dev);
    if (out_kind == TAQ_OUT_INT8_HEAD_ROWS) TAQ_REQUIRE_PTR(scales_dev);
    int* status = nullptr;
    s = status_ptr(&status);
    if (s != TAQ_OK) return s;
    LinearArgs a{};
    a.xq = x_codes_dev; a.x_scales = x_scales_dev;
    a.w = W_packed_dev;
    a.y = y_dev;
    a.scales = scales_dev;
    a.rows = rows;
    a.n_out = d->n_out; a.k_in = d->k_in; a.bits = d->bits; a.group = d->group;
    a.heads = out_kind == TAQ_OUT_INT8_HEAD_ROWS ? heads : 1;
    a.epi = out_kind == TAQ_OUT_F16 ? EPI_F16 : out_kind == TAQ_OUT_F32 ? EPI_F32 : EPI_Q8_HEAD;
    a.status = status;
    return run_linear_i8(a, (cudaStream_t)stream);
}

// Workspace of the integer-activation layer pass: activation codes and scales (X, later O), then the sections of the
// ordinary pass.
struct WorkspaceA8 { size_t off_xq, off_xs, base, total; };
static WorkspaceA8 workspace_a8_layout(const taq_layer_desc* d) {
    const size_t rows = (size_t)d->batch * d->n_query;
    WorkspaceA8 w;
    w.off_xq = 0;
    w.off_xs = align_up(rows * d->channels, 128);
    w.base = w.off_xs + align_up(rows * sizeof(float), 128);
    w.total = w.base + workspace_layout(d, 1).total;
    return w;
}

size_t taq_workspace_bytes_a8(const taq_layer_desc* d) {
    if (check_layer_desc(d) != TAQ_OK) return 0;
    return workspace_a8_layout(d).total;
}

taq_status taq_layer_forward_a8(const taq_layer_desc* d, const void* x_f16_dev, const void* Wq_packed_dev, const void* Wout_packed_dev,
                                const void* kv_packed_dev, const uint8_t* trig_mask_dev, void* y_f16_dev, void* workspace_dev,
                                size_t workspace_bytes, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch > 65535) return fail(TAQ_ERR_SHAPE, "batch must be at most 65535");
    if (d->batch == 0 || d->n_query == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(x_f16_dev);
    TAQ_REQUIRE_PTR(Wq_packed_dev);
    TAQ_REQUIRE_PTR(Wout_packed_dev);
    TAQ_REQUIRE_PTR(kv_packed_dev);
    TAQ_REQUIRE_PTR(y_f16_dev);
    TAQ_REQUIRE_PTR(workspace_dev);
    if (!trig_mask_dev) return fail(TAQ_ERR_INVALID_ARG, "trig_mask_dev is NULL");
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 127u) return fail(TAQ_ERR_ALIGNMENT, "workspace_dev is not 128-byte aligned");
    const WorkspaceA8 WA = workspace_a8_layout(d);
    if (workspace_bytes < WA.total) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "workspace has %zu bytes, %zu needed", workspace_bytes, WA.total);
    cudaStream_t st = (cudaStream_t)stream;
    int* status = nullptr;
    s = status_ptr(&status);
    if (s != TAQ_OK) return s;
    if (sm100_layer_a8_supported(*d)) {                                   // the whole integer-activation pass in one kernel
        count_launch(TAQ_KERNEL_LAYER_FUSED_A8);
        cudaError_t e1 = launch_layer_a8_sm100(*d, (const __half*)x_f16_dev, Wq_packed_dev, Wout_packed_dev, kv_packed_dev, (__half*)y_f16_dev,
                                               d->batch, status, st);
        return e1 == cudaSuccess ? TAQ_OK : cuda_fail(e1, "fused integer-activation layer launch");
    }
    uint8_t* wsb = (uint8_t*)workspace_dev;
    int8_t* xq = (int8_t*)(wsb + WA.off_xq);
    float* xs = (float*)(wsb + WA.off_xs);
    uint8_t* base = wsb + WA.base;
    const Workspace W = workspace_layout(d, 1);
    const long long rows = (long long)d->batch * d->n_query;

    cudaError_t e = launch_quantize_rows_f16((const __half*)x_f16_dev, rows, d->channels, xq, xs, st);      // X~ = Q_a(X) per token
    if (e != cudaSuccess) return cuda_fail(e, "quantize_rows_f16 launch");
    LinearArgs q{};                                                                                           // to_q (+ Q~ = Q_a(Q))
    q.xq = xq; q.x_scales = xs; q.w = Wq_packed_dev;
    q.y = base + W.off_q; q.scales = (float*)(base + W.off_qs);
    q.rows = rows; q.n_out = d->channels; q.k_in = d->channels; q.bits = d->w_bits; q.group = d->w_group;
    q.heads = d->q_bits == 8 ? d->heads : 1;
    q.epi = d->q_bits == 8 ? EPI_Q8_HEAD : EPI_F16;
    q.status = status;
    q.early_weights = 1;        // the kernel before it in the stream is the quantizer above, which writes xq / xs only
    s = run_linear_i8(q, st);
    if (s != TAQ_OK) return s;
    AttnArgs at = attn_args(d, status);
    at.q = base + W.off_q; at.q_scales = (const float*)(base + W.off_qs); at.kv = kv_packed_dev; at.mask = trig_mask_dev;
    at.o = (__half*)(base + W.off_o);
    at.early_kv = 1;
    s = run_attention(at, d->batch, st);
    if (s != TAQ_OK) return s;
    e = launch_quantize_rows_f16((const __half*)(base + W.off_o), rows, d->channels, xq, xs, st);            // O~ = Q_a(O) per token
    if (e != cudaSuccess) return cuda_fail(e, "quantize_rows_f16 launch");
    LinearArgs o{};                                                                                           // to_out (+ bias)
    o.xq = xq; o.x_scales = xs; o.w = Wout_packed_dev;
    o.y = y_f16_dev;
    o.rows = rows; o.n_out = d->channels; o.k_in = d->channels; o.bits = d->w_bits; o.group = d->w_group;
    o.heads = 1; o.epi = EPI_F16; o.status = status;
    o.early_weights = 1;
    return run_linear_i8(o, st);
}

size_t taq_kv_project_a8_workspace_bytes(const taq_layer_desc* d) {
    if (check_layer_desc(d) != TAQ_OK) return 0;
    const size_t rows = (size_t)d->batch * d->n_ctx;
    return align_up(rows * d->ctx_dim, 128) + align_up(rows * sizeof(float), 128);
}

taq_status taq_kv_project_a8(const taq_layer_desc* d, const void* ctx_f16_dev, const void* Wk_packed_dev, const void* Wv_packed_dev,
                             const uint8_t* trig_mask_dev, void* kv_packed_dev, size_t kv_bytes, void* workspace_dev, size_t workspace_bytes,
                             void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch == 0) return TAQ_OK;
    if (d->batch > 65535) return fail(TAQ_ERR_SHAPE, "batch must be at most 65535");
    TAQ_REQUIRE_PTR(ctx_f16_dev);
    TAQ_REQUIRE_PTR(Wk_packed_dev);
    TAQ_REQUIRE_PTR(Wv_packed_dev);
    TAQ_REQUIRE_PTR(kv_packed_dev);
    TAQ_REQUIRE_PTR(workspace_dev);
    if (!trig_mask_dev) return fail(TAQ_ERR_INVALID_ARG, "trig_mask_dev is NULL");
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 127u) return fail(TAQ_ERR_ALIGNMENT, "workspace_dev is not 128-byte aligned");
    const size_t need = taq_kv_bytes(d), wneed = taq_kv_project_a8_workspace_bytes(d);
    if (kv_bytes < need) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "kv buffer has %zu bytes, %zu needed", kv_bytes, need);
    if (workspace_bytes < wneed) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "workspace has %zu bytes, %zu needed", workspace_bytes, wneed);
    cudaStream_t st = (cudaStream_t)stream;
    int* status = nullptr;
    s = status_ptr(&status);
    if (s != TAQ_OK) return s;
    const long long rows = (long long)d->batch * d->n_ctx;
    int8_t* cq = (int8_t*)workspace_dev;
    float* cs = (float*)((uint8_t*)workspace_dev + align_up((size_t)rows * d->ctx_dim, 128));
    cudaError_t e = launch_quantize_rows_f16((const __half*)ctx_f16_dev, rows, d->ctx_dim, cq, cs, st);
    if (e != cudaSuccess) return cuda_fail(e, "quantize_rows_f16 launch");
    LinearArgs a{};
    a.xq = cq; a.x_scales = cs;
    a.y = kv_packed_dev;
    a.mask = trig_mask_dev;
    a.rows = rows;
    a.n_out = d->channels; a.k_in = d->ctx_dim; a.bits = d->w_bits; a.group = d->w_group;
    a.heads = d->heads; a.n_ctx = d->n_ctx; a.max_trigger = d->max_trigger;
    a.epi = EPI_KV; a.kv_qmax = d->kv_bits == 4 ? 7 : 127;
    a.status = status;
    for (int which = 0; which < 2; ++which) {
        a.w = which ? Wv_packed_dev : Wk_packed_dev;
        a.which = which;
        a.kv_which = which;
        s = run_linear_i8(a, st);
        if (s != TAQ_OK) return s;
    }
    e = launch_kv_operands(*d, kv_packed_dev, nullptr, d->batch, st);
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "K/V operand image launch");
}

// ---- Eq. 3's M_A chosen independently of Eq. 2's M_KV; the token-sensitivity sweep of Eq. 1 -------------------------

taq_status taq_kv_set_prob_mask(const taq_layer_desc* d, void* kv_packed_dev, size_t kv_bytes, const uint8_t* mask_a_dev, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch == 0) return TAQ_OK;
    if (d->batch > 65535) return fail(TAQ_ERR_SHAPE, "batch must be at most 65535");
    TAQ_REQUIRE_PTR(kv_packed_dev);
    if (!mask_a_dev) return fail(TAQ_ERR_INVALID_ARG, "mask_a_dev is NULL");
    const size_t need = taq_kv_bytes(d);
    if (kv_bytes < need) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "kv buffer has %zu bytes, %zu needed", kv_bytes, need);
    cudaError_t e = launch_kv_operands(*d, kv_packed_dev, nullptr, d->batch, (cudaStream_t)stream, mask_a_dev);
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "K/V operand image launch");
}

struct SensWorkspace { size_t off_masks, off_kv, off_ystar, off_y, off_partials, off_layer, total; };
static SensWorkspace sens_layout(const taq_layer_desc* d) {
    SensWorkspace w;
    const size_t act = align_up((size_t)d->batch * d->n_query * d->channels * sizeof(__half), 128);
    w.off_masks = 0;
    w.off_kv = align_up((size_t)(d->n_ctx + 1) * d->batch * d->n_ctx, 128);
    w.off_ystar = w.off_kv + align_up(taq_kv_bytes(d), 128);
    w.off_y = w.off_ystar + act;
    w.off_partials = w.off_y + act;
    w.off_layer = w.off_partials + align_up(256 * sizeof(double), 128);
    w.total = w.off_layer + workspace_layout(d, 1).total;
    return w;
}

size_t taq_token_sensitivity_workspace_bytes(const taq_layer_desc* d) {
    if (check_layer_desc(d) != TAQ_OK) return 0;
    return sens_layout(d).total;
}

taq_status taq_token_sensitivity(const taq_layer_desc* d, const void* x_f16_dev, const void* ctx_f16_dev, const void* Wq_packed_dev,
                                 const void* Wk_packed_dev, const void* Wv_packed_dev, const void* Wout_packed_dev, double* delta_dev,
                                 void* workspace_dev, size_t workspace_bytes, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch < 1 || d->n_query < 1) return fail(TAQ_ERR_SHAPE, "batch and n_query must be positive");
    if (d->batch > 65535) return fail(TAQ_ERR_SHAPE, "batch must be at most 65535");
    if (d->max_trigger < d->n_ctx) return fail(TAQ_ERR_SHAPE, "the sweep keeps up to n_ctx rows in fp16: max_trigger (%d) must equal n_ctx (%d)", d->max_trigger, d->n_ctx);
    TAQ_REQUIRE_PTR(x_f16_dev);
    TAQ_REQUIRE_PTR(ctx_f16_dev);
    TAQ_REQUIRE_PTR(Wq_packed_dev);
    TAQ_REQUIRE_PTR(Wk_packed_dev);
    TAQ_REQUIRE_PTR(Wv_packed_dev);
    TAQ_REQUIRE_PTR(Wout_packed_dev);
    TAQ_REQUIRE_PTR(delta_dev);
    TAQ_REQUIRE_PTR(workspace_dev);
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 127u) return fail(TAQ_ERR_ALIGNMENT, "workspace_dev is not 128-byte aligned");
    const SensWorkspace W = sens_layout(d);
    if (workspace_bytes < W.total) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "workspace has %zu bytes, %zu needed", workspace_bytes, W.total);
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* wsb = (uint8_t*)workspace_dev;
    uint8_t* masks = wsb + W.off_masks;
    const size_t mask_stride = (size_t)d->batch * d->n_ctx;
    const uint8_t* ones = masks + (size_t)d->n_ctx * mask_stride;
    const long long n = (long long)d->batch * d->n_query * d->channels;
    cudaError_t e = launch_sensitivity_masks(masks, d->batch, d->n_ctx, st);
    if (e != cudaSuccess) return cuda_fail(e, "sensitivity mask launch");
    for (int i = d->n_ctx; i >= 0; --i) {       // i = n_ctx first: the reference y* with no K/V row quantized
        const int which = (i == d->n_ctx) ? d->n_ctx : i;
        void* y = wsb + (which == d->n_ctx ? W.off_ystar : W.off_y);
        s = kv_project_impl(d, nullptr, 1, ctx_f16_dev, Wk_packed_dev, Wv_packed_dev, masks + (size_t)which * mask_stride, wsb + W.off_kv, st);
        if (s != TAQ_OK) return s;
        e = launch_kv_operands(*d, wsb + W.off_kv, nullptr, d->batch, st, ones);      // M_A: every probability column stays fp16
        if (e != cudaSuccess) return cuda_fail(e, "K/V operand image launch");
        s = layer_forward_impl(d, nullptr, 1, x_f16_dev, Wq_packed_dev, Wout_packed_dev, wsb + W.off_kv, ones, y, wsb + W.off_layer, st);
        if (s != TAQ_OK) return s;
        if (which != d->n_ctx) {
            e = launch_mse_f16((const __half*)(wsb + W.off_y), (const __half*)(wsb + W.off_ystar), n, (double*)(wsb + W.off_partials), delta_dev + which, st);
            if (e != cudaSuccess) return cuda_fail(e, "mse launch");
        }
    }
    return TAQ_OK;
}

taq_status taq_query_attention(const taq_layer_desc* d, const void* x_f16_dev, const void* Wq_packed_dev, const void* kv_packed_dev,
                               const uint8_t* trig_mask_dev, void* o_f16_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch > 65535) return fail(TAQ_ERR_SHAPE, "batch must be at most 65535");
    if (d->batch == 0 || d->n_query == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(x_f16_dev);
    TAQ_REQUIRE_PTR(Wq_packed_dev);
    TAQ_REQUIRE_PTR(kv_packed_dev);
    TAQ_REQUIRE_PTR(o_f16_dev);
    TAQ_REQUIRE_PTR(workspace_dev);
    if (!trig_mask_dev) return fail(TAQ_ERR_INVALID_ARG, "trig_mask_dev is NULL");
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 127u) return fail(TAQ_ERR_ALIGNMENT, "workspace_dev is not 128-byte aligned");
    const size_t need = taq_workspace_bytes(d, 1);
    if (workspace_bytes < need) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    int* status = nullptr;
    s = status_ptr(&status);
    if (s != TAQ_OK) return s;
    return q_attention_impl(d, nullptr, 1, x_f16_dev, Wq_packed_dev, kv_packed_dev, trig_mask_dev, o_f16_dev, workspace_dev, status, (cudaStream_t)stream);
}

taq_status taq_layer_forward_batched(const taq_layer_desc* d, const taq_request* reqs_dev, int32_t n_requests, const void* x_f16_dev,
                                     void* y_f16_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch != 1) return fail(TAQ_ERR_SHAPE, "batched calls take one sequence per request (desc->batch must be 1)");
    if (n_requests < 0 || n_requests > 65535) return fail(TAQ_ERR_SHAPE, "n_requests must be in [0,65535]");
    if (n_requests == 0 || d->n_query == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(reqs_dev);
    TAQ_REQUIRE_PTR(x_f16_dev);
    TAQ_REQUIRE_PTR(y_f16_dev);
    TAQ_REQUIRE_PTR(workspace_dev);
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 127u) return fail(TAQ_ERR_ALIGNMENT, "workspace_dev is not 128-byte aligned");
    const size_t need = taq_workspace_bytes(d, n_requests);
    if (workspace_bytes < need) return fail(TAQ_ERR_BUFFER_TOO_SMALL, "workspace has %zu bytes, %zu needed", workspace_bytes, need);
    return layer_forward_impl(d, reqs_dev, n_requests, x_f16_dev, nullptr, nullptr, nullptr, nullptr, y_f16_dev, workspace_dev, (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------------------------
// taq_layer_forward_static: the layer pass for callers that cannot provide a workspace.
// The scratch (Q~, its scales, O) lives in a fixed array inside the library image; each GPU that loads the
// library holds one copy until the process exits.
// ---------------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_workspace[TAQ_STATIC_WORKSPACE_BYTES];

// Device address of the array on the current device.  In host code the array's name is only a handle for the
// runtime, not an address a kernel can use, so the address is asked for once per device and remembered.
static taq_status static_workspace_ptr(unsigned char** out) {
    static unsigned char* cache[64] = {nullptr};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
    if (dev < 0 || dev >= 64) return fail(TAQ_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
    if (!cache[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_workspace);
        if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress(static workspace)");
        cache[dev] = static_cast<unsigned char*>(p);
    }
    *out = cache[dev];
    return TAQ_OK;
}

size_t taq_static_workspace_capacity(void) { return (size_t)TAQ_STATIC_WORKSPACE_BYTES; }

taq_status taq_layer_forward_static(const taq_layer_desc* d, const void* x_f16_dev, const void* Wq_packed_dev, const void* Wout_packed_dev,
                                    const void* kv_packed_dev, const uint8_t* trig_mask_dev, void* y_f16_dev, void* stream) {
    taq_status s = check_layer_desc(d);
    if (s != TAQ_OK) return s;
    if (d->batch > 65535) return fail(TAQ_ERR_SHAPE, "batch must be at most 65535");
    const size_t need = workspace_layout(d, 1).total;
    if (need > (size_t)TAQ_STATIC_WORKSPACE_BYTES)
        return fail(TAQ_ERR_BUFFER_TOO_SMALL, "this layer needs %zu bytes of scratch, the built-in workspace holds %zu; use taq_layer_forward with a caller-owned workspace",
                    need, (size_t)TAQ_STATIC_WORKSPACE_BYTES);
    if (d->batch == 0 || d->n_query == 0) return TAQ_OK;
    TAQ_REQUIRE_PTR(x_f16_dev);
    TAQ_REQUIRE_PTR(Wq_packed_dev);
    TAQ_REQUIRE_PTR(Wout_packed_dev);
    TAQ_REQUIRE_PTR(kv_packed_dev);
    TAQ_REQUIRE_PTR(y_f16_dev);
    if (!trig_mask_dev) return fail(TAQ_ERR_INVALID_ARG, "trig_mask_dev is NULL");
    unsigned char* ws = nullptr;
    s = static_workspace_ptr(&ws);
    if (s != TAQ_OK) return s;
    // Every byte of Q~, its scales and O that a later stage reads is written by the stage before it in this same
    // call, so nothing in the array has to start at zero and what the previous call left there is never read.
    return layer_forward_impl(d, nullptr, 1, x_f16_dev, Wq_packed_dev, Wout_packed_dev, kv_packed_dev, trig_mask_dev, y_f16_dev, ws,
                              (cudaStream_t)stream);
}

taq_status taq_dispatch_counts(int64_t* counts_out, int32_t n) {
    if (!counts_out || n < 0) return fail(TAQ_ERR_INVALID_ARG, "counts_out is NULL or n negative");
    for (int i = 0; i < n; ++i) counts_out[i] = i < TAQ_N_KERNEL_FAMILIES ? (int64_t)g_dispatch[i].load(std::memory_order_relaxed) : 0;
    return TAQ_OK;
}

void taq_dispatch_reset(void) {
    for (int i = 0; i < TAQ_N_KERNEL_FAMILIES; ++i) g_dispatch[i].store(0, std::memory_order_relaxed);
}

taq_status taq_linear_plan(const taq_weight_desc* d, int64_t rows, int32_t out_kind, int32_t heads, int32_t int8_activations,
                           int32_t batched, int32_t* plan_out) {
    taq_status s = check_weight_desc(d);
    if (s != TAQ_OK) return s;
    if (!plan_out) return fail(TAQ_ERR_INVALID_ARG, "plan_out is NULL");
    if (out_kind != TAQ_OUT_F16 && out_kind != TAQ_OUT_F32 && out_kind != TAQ_OUT_INT8_HEAD_ROWS) return fail(TAQ_ERR_INVALID_ARG, "unknown out_kind %d", out_kind);
    if (out_kind == TAQ_OUT_INT8_HEAD_ROWS && (heads < 1 || d->n_out % heads)) return fail(TAQ_ERR_SHAPE, "n_out (%d) must be a multiple of heads (%d)", d->n_out, heads);
    static const taq_request dummy_req = {};
    alignas(16) static const char dummy[16] = {};
    LinearArgs a{};
    if (int8_activations) a.xq = (const int8_t*)dummy; else a.x = (const __half*)dummy;
    a.reqs = batched ? &dummy_req : nullptr;
    a.rows = rows;
    a.n_out = d->n_out; a.k_in = d->k_in; a.bits = d->bits; a.group = d->group;
    a.heads = out_kind == TAQ_OUT_INT8_HEAD_ROWS ? heads : 1;
    a.epi = out_kind == TAQ_OUT_F16 ? EPI_F16 : out_kind == TAQ_OUT_F32 ? EPI_F32 : EPI_Q8_HEAD;
    int out[10];
    linear_plan_of(a, out);
    for (int i = 0; i < 10; ++i) plan_out[i] = out[i];
    return TAQ_OK;
}

taq_status taq_selftest_wait_expiry(int64_t limit_cycles, void* stream) {
    if (limit_cycles < 1 || limit_cycles > (1LL << 31)) return fail(TAQ_ERR_INVALID_ARG, "limit_cycles must be in [1, 2^31]");
    int* status = nullptr;
    taq_status s = status_ptr(&status);
    if (s != TAQ_OK) return s;
    wait_expiry_kernel<<<1, 32, 0, (cudaStream_t)stream>>>((long long)limit_cycles, status);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? TAQ_OK : cuda_fail(e, "wait-expiry self-test launch");
}

taq_status taq_poll_device_status(void* stream, int32_t* block_id_out) {
    int* status = nullptr;
    taq_status s = status_ptr(&status);
    if (s != TAQ_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    int host[2] = {0, 0};
    cudaError_t e = cudaMemcpyAsync(host, status, sizeof(host), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "reading the device status word");
    if (host[0] != 0) {
        e = cudaMemsetAsync(status, 0, sizeof(host), st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return cuda_fail(e, "clearing the device status word");
        if (block_id_out) *block_id_out = host[1];
        return fail((taq_status)host[0], "a kernel raised device status %d (%s) in block %d", host[0], taq_status_string((taq_status)host[0]), host[1]);
    }
    if (block_id_out) *block_id_out = -1;
    return TAQ_OK;
}

}  // extern "C"
