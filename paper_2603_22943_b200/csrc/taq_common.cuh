// Shared device/host definitions of the TAQ library: packed-blob header, K~/V~ block layout, status word.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "taq.h"

namespace taq {

constexpr uint32_t kWeightMagic = 0x57514154u;  // "TAQW" little-endian
constexpr int kMaxCtx = 128;                    // T <= 128
constexpr int kMaxHeadDim = 256;

// First 64 bytes of a packed weight blob (layout documented in taq.h).
struct PackedHeader {
    uint32_t magic, version, n_out, k_in, bits, group, n_groups, has_bias;
    uint64_t off_codes, off_scales, off_bias, total_bytes;
};
static_assert(sizeof(PackedHeader) == 64, "header is 64 bytes");

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct WeightLayout {
    int n_groups;
    int group_len;          // effective group length (k_in when group == 0)
    size_t row_bytes;       // bytes of codes per output channel
    size_t off_codes, off_scales, off_bias, total;
};

__host__ __device__ inline WeightLayout weight_layout(int n_out, int k_in, int bits, int group) {
    WeightLayout L;
    L.group_len = group == 0 ? k_in : group;
    L.n_groups = (k_in + L.group_len - 1) / L.group_len;
    L.row_bytes = bits == 8 ? (size_t)k_in : (size_t)k_in / 2;
    L.off_codes = 128;
    L.off_scales = align_up(L.off_codes + L.row_bytes * n_out, 128);
    L.off_bias = align_up(L.off_scales + sizeof(float) * (size_t)n_out * L.n_groups, 128);
    L.total = align_up(L.off_bias + sizeof(float) * (size_t)n_out, 128);
    return L;
}

// MMA-ready image of one head's K~ and V~ (layout documented in taq.h): present when the tensor-core attention
// kernel covers the shape (head width 40/64/80/160, at most kOperandKeys text tokens).
constexpr int kOperandKeys = 80;                // keys padded to a multiple of the MMA K step
constexpr int kOperandConstBytes = 1024;
struct OperandGeom {
    int dp;                 // head width padded to a multiple of 16
    int kbq;                // 64-wide blocks along the head width
    size_t k_bytes;         // K~ tile: kbq blocks of [kOperandKeys rows][128 bytes]
    size_t vt_bytes;        // V~^T tile: 2 blocks of [dp rows][128 bytes]
    size_t head_bytes;      // k_bytes + vt_bytes + kOperandConstBytes
};
__host__ __device__ inline bool operand_geom(int d, int n_ctx, OperandGeom* g) {
    if ((d != 40 && d != 64 && d != 80 && d != 160) || n_ctx > kOperandKeys) return false;
    g->dp = (d + 15) / 16 * 16;
    g->kbq = (g->dp + 63) / 64;
    g->k_bytes = (size_t)g->kbq * kOperandKeys * 128;
    g->vt_bytes = (size_t)2 * g->dp * 128;
    g->head_bytes = g->k_bytes + g->vt_bytes + kOperandConstBytes;
    return true;
}
// Constants block at the end of a head's image.
struct OperandConsts {
    float logit_factor[kOperandKeys];   // K scale of key j (1 for a trigger row) * log2(e) / sqrt(d); 0 for padding
    uint32_t trig_bits[4];              // bit j set: key j is a trigger token (fp16 probability column, Eq. 3)
};
static_assert(sizeof(OperandConsts) <= kOperandConstBytes, "constants block");

// K~/V~ block of one sequence (layout documented in taq.h).
__host__ __device__ inline taq_kv_layout kv_layout(int heads, int n_ctx, int d, int max_trigger) {
    taq_kv_layout L;
    size_t codes = align_up((size_t)heads * n_ctx * d, 128);
    size_t scales = align_up(sizeof(float) * (size_t)heads * n_ctx, 128);
    size_t trig = align_up(sizeof(__half) * (size_t)max_trigger * heads * d, 128);
    L.off_k_codes = 0;
    L.off_v_codes = codes;
    L.off_k_scales = 2 * codes;
    L.off_v_scales = 2 * codes + scales;
    L.off_k_trigger = 2 * codes + 2 * scales;
    L.off_v_trigger = L.off_k_trigger + trig;
    L.off_trig_slot = L.off_v_trigger + trig;
    L.off_operands = L.off_trig_slot + sizeof(int32_t) * kMaxCtx;
    OperandGeom g;
    L.operand_head_bytes = operand_geom(d, n_ctx, &g) ? g.head_bytes : 0;
    L.block_bytes = L.off_operands + L.operand_head_bytes * heads;
    return L;
}

// Device status word: {code, block id}.  First writer wins.
__device__ inline void raise_status(int* status, int code) {
    if (atomicCAS(&status[0], 0, code) == 0) {
        status[1] = (int)(blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z));
    }
}

// The symmetric quantizer in IEEE binary32: scale = absmax / qmax, code = clamp(rint(x / scale)).
__device__ inline float quant_scale(float absmax, float qmax) { return __fdiv_rn(absmax, qmax); }
__device__ inline int quant_code(float x, float scale, int qmax) {
    if (scale == 0.f) return 0;
    float r = rintf(__fdiv_rn(x, scale));
    r = fminf(fmaxf(r, (float)-qmax), (float)qmax);
    return (int)r;
}

// Position of fan-in element e (0..7) of an aligned group of eight 4-bit codes inside their 32-bit word: even
// elements fill nibbles 0..3, odd elements nibbles 4..7, so that (word >> 4i) & 0x000F000F holds elements 2i and
// 2i+1 in the two halves of a register.
__host__ __device__ inline int w4_nibble_pos(int e) { return (e >> 1) + ((e & 1) << 2); }

__device__ inline int load_code(const uint8_t* codes, size_t row_bytes, int bits, int n, int k) {
    if (bits == 8) return (int)((const int8_t*)codes)[(size_t)n * row_bytes + k];
    const uint32_t word = *reinterpret_cast<const uint32_t*>(codes + (size_t)n * row_bytes + ((k >> 3) << 2));
    return (int)((word >> (4 * w4_nibble_pos(k & 7))) & 0xFu) - 8;
}

// ------------------------------------------------------------------------------------------------------
// Kernel launch arguments shared between translation units.
// ------------------------------------------------------------------------------------------------------
enum Epilogue : int { EPI_F16 = 0, EPI_F32 = 1, EPI_Q8_HEAD = 2, EPI_KV = 3 };

// One dequant-GEMM problem family: y = x W^T.  With `reqs` set, grid.z indexes requests and the weight blob
// (and, for EPI_KV, the output block and mask) come from the request table.
struct LinearArgs {
    const __half* x;            // [z][rows][k_in]
    const int8_t* xq;           // integer-activation variant: int8 codes [z][rows][k_in] instead of x ...
    const float* x_scales;      // ... and one fp32 scale per row [z][rows]
    const void* w;              // packed blob (single problem)
    const taq_request* reqs;    // nullable
    int which;                  // 0: reqs[z].Wq, 1: reqs[z].Wout
    void* y;                    // F16/F32/int8 [z][rows][n_out]; for EPI_KV: kv blocks (single problem)
    float* scales;              // EPI_Q8_HEAD: [z][rows][heads]
    const uint8_t* mask;        // EPI_KV: [batch][T] (single problem)
    long long rows;             // rows per z
    int n_out, k_in, bits, group;
    int heads;                  // EPI_Q8_HEAD / EPI_KV
    int n_ctx, max_trigger;     // EPI_KV: rows = batch * n_ctx
    int kv_which;               // EPI_KV: 0 = K, 1 = V
    int kv_qmax;                // EPI_KV: 127 (int8 rows) or 7 (4-bit rows); 0 is read as 127
    int epi;
    int w_direct;               // (set by the launcher) 1: int8 activations and 8-bit weights: the weight codes are the B
                                // operand as they are and go from the blob into the ring by TMA, no staging or expansion;
                                // 2: fp16 activations and 8-bit weights too large to stage whole: a slice of the codes per
                                // k-block by TMA, expanded by the workers; 0: all codes staged once
    int early_weights;          // the previous kernel in the stream is known not to write the weights: fetch and expand
                                // them before waiting for it
    int head_pair;              // (set by the launcher) EPI_Q8_HEAD with heads twice as wide as the tile: the two CTAs whose
                                // tiles make up a head exchange their rows' absmax through the cluster
    int* status;
};

struct AttnArgs {
    const void* q;              // int8 or fp16 [z][B][N][C]
    const float* q_scales;      // [z][B][N][H] (q_bits = 8)
    const void* kv;             // blocks [B] (single problem)
    const uint8_t* mask;        // [B][T]
    const taq_request* reqs;    // nullable; then B = 1 per request
    __half* o;                  // [z][B][N][C]
    int batch, n_query, channels, heads, n_ctx, max_trigger;
    int q_bits, p_bits;
    int p_log;                  // 1: logarithmic probability codes (p^ = 2^-code) instead of the linear ones
    int early_kv;               // the previous kernel in the stream is known not to write the K~/V~ blocks
    int* status;
};

// Launch with the programmatic-serialization attribute (see ptx::pdl_wait): the kernel's prologue may overlap the
// tail of the previous kernel in the stream.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
// The same with thread-block clusters of `cluster` CTAs.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 cluster, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = cluster.x;
    attr[1].val.clusterDim.y = cluster.y;
    attr[1].val.clusterDim.z = cluster.z;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

cudaError_t launch_linear_simt(const LinearArgs& a, int n_z, cudaStream_t stream);
cudaError_t launch_attention_simt(const AttnArgs& a, int n_z, cudaStream_t stream);
cudaError_t launch_quantize_rows_f16(const __half* x, long long rows, int cols, int8_t* codes, float* scales, cudaStream_t stream);
cudaError_t launch_quantize_rows(const float* x, long long rows, int cols, int qmax, int8_t* codes, float* scales,
                                 cudaStream_t stream);
cudaError_t launch_pack_weights(const taq_weight_desc& d, const float* W, const float* bias, void* packed,
                                cudaStream_t stream);
cudaError_t launch_kv_operands(const taq_layer_desc& d, void* kv, const taq_request* reqs, int n_z, cudaStream_t stream, const uint8_t* mask_a = nullptr);
// Mean squared difference of two fp16 arrays into *out (fp64), deterministic two-stage sum; partials: 256 doubles of scratch.
cudaError_t launch_mse_f16(const __half* a, const __half* b, long long n, double* partials, double* out, cudaStream_t stream);
// masks[i][b][t] = (t != i) for i < T, all ones for i = T  (u8 [T+1][B][T])
cudaError_t launch_sensitivity_masks(uint8_t* masks, int batch, int n_ctx, cudaStream_t stream);
cudaError_t launch_unpack_weights(const taq_weight_desc& d, const void* packed, int8_t* codes, float* scales,
                                  cudaStream_t stream);

}  // namespace taq
