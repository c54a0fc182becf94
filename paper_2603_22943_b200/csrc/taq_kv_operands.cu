// Builds the operand images of K~/V~ blocks: the mixed-precision rows of Eq. 2 once more, as the fp16 tiles the
// tensor-core attention kernel multiplies with (128-byte-swizzled, K-major), plus the per-key constants of the
// softmax.  Done once per prompt, right after the K/V projection, so that the per-step attention kernel stages
// a head with one bulk copy and no arithmetic.
#include "taq_common.cuh"
#include "taq_ptx.cuh"

namespace taq {

namespace {

// One CTA per (head, sequence).
// `mask_a` (nullable, u8 [sequences][T]) overrides which probability columns stay fp16 (Eq. 3's M_A); by default they
// are the columns of the fp16 K/V rows (M_A = M_KV).
__global__ void __launch_bounds__(256) kv_operands_kernel(const taq_layer_desc d, uint8_t* kv, const taq_request* reqs, const uint8_t* mask_a) {
    const int H = d.heads, T = d.n_ctx, D = d.channels / d.heads;
    const int h = blockIdx.x, z = blockIdx.y;
    const taq_kv_layout KL = kv_layout(H, T, D, d.max_trigger);
    OperandGeom g;
    if (!operand_geom(D, T, &g)) return;
    uint8_t* blk = reqs ? (uint8_t*)reqs[z].kv : kv + (size_t)z * KL.block_bytes;
    const int8_t* kc = (const int8_t*)(blk + KL.off_k_codes) + (size_t)h * T * D;
    const int8_t* vc = (const int8_t*)(blk + KL.off_v_codes) + (size_t)h * T * D;
    const float* ks = (const float*)(blk + KL.off_k_scales) + (size_t)h * T;
    const float* vs = (const float*)(blk + KL.off_v_scales) + (size_t)h * T;
    const __half* kt = (const __half*)(blk + KL.off_k_trigger);
    const __half* vt = (const __half*)(blk + KL.off_v_trigger);
    const int32_t* slot = (const int32_t*)(blk + KL.off_trig_slot);
    uint8_t* img = blk + KL.off_operands + (size_t)h * KL.operand_head_bytes;
    uint8_t* k_img = img;
    uint8_t* vt_img = img + g.k_bytes;
    OperandConsts* cst = reinterpret_cast<OperandConsts*>(img + g.k_bytes + g.vt_bytes);
    const size_t k_block = (size_t)kOperandKeys * 128, vt_block = (size_t)g.dp * 128;

    // K~ tile: element (key j, channel c)
    for (int idx = threadIdx.x; idx < kOperandKeys * g.kbq * 64; idx += blockDim.x) {
        const int j = idx / (g.kbq * 64), c = idx % (g.kbq * 64);
        __half v = __float2half_rn(0.f);
        if (j < T && c < D) {
            const int sl = slot[j];
            v = sl >= 0 ? kt[((size_t)sl * H + h) * D + c] : __int2half_rn((int)kc[(size_t)j * D + c]);
        }
        *reinterpret_cast<__half*>(k_img + (c / 64) * k_block + ptx::sw128_offset(j, (c % 64) / 8) + (c % 8) * 2) = v;
    }
    // V~^T tile: element (channel c, key j); ordinary rows are the fp16 operand of code * scale
    for (int idx = threadIdx.x; idx < g.dp * 128; idx += blockDim.x) {
        const int c = idx / 128, j = idx % 128;
        __half v = __float2half_rn(0.f);
        if (j < T && c < D) {
            const int sl = slot[j];
            v = sl >= 0 ? vt[((size_t)sl * H + h) * D + c] : __float2half_rn(__fmul_rn((float)vc[(size_t)j * D + c], vs[j]));
        }
        *reinterpret_cast<__half*>(vt_img + (j / 64) * vt_block + ptx::sw128_offset(c, (j % 64) / 8) + (j % 8) * 2) = v;
    }
    // constants
    const float logit_unit = 1.4426950408889634f / sqrtf((float)D);
    for (int j = threadIdx.x; j < kOperandKeys; j += blockDim.x)
        cst->logit_factor[j] = j < T ? (slot[j] >= 0 ? 1.0f : ks[j]) * logit_unit : 0.f;
    if (threadIdx.x < 4) {
        uint32_t bits = 0;
        for (int i = 0; i < 32; ++i) {
            const int j = threadIdx.x * 32 + i;
            if (j < T && (mask_a ? mask_a[(size_t)z * T + j] != 0 : slot[j] >= 0)) bits |= 1u << i;
        }
        cst->trig_bits[threadIdx.x] = bits;
    }
}

}  // namespace

cudaError_t launch_kv_operands(const taq_layer_desc& d, void* kv, const taq_request* reqs, int n_z, cudaStream_t stream, const uint8_t* mask_a) {
    OperandGeom g;
    if (n_z == 0 || !operand_geom(d.channels / d.heads, d.n_ctx, &g)) return cudaSuccess;
    dim3 grid(d.heads, n_z);
    kv_operands_kernel<<<grid, 256, 0, stream>>>(d, (uint8_t*)kv, reqs, mask_a);
    return cudaGetLastError();
}

}  // namespace taq
