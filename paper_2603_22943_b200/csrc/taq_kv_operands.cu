// Builds the operand images of K~/V~ blocks: the mixed-precision rows of Eq. 2 once more, as the fp16 tiles the
// tensor-core attention kernel multiplies with (128-byte-swizzled, K-major), plus the per-key constants of the
// softmax.  Done once per prompt, right after the K/V projection, so that the per-step attention kernel stages
// a head with one bulk copy and no arithmetic.
#include "taq_common.cuh"
#include "taq_ptx.cuh"

namespace taq {

namespace {

// One CTA per (head, sequence).  The head's codes and scales are staged in shared memory (coalesced 8-byte loads);
// every thread then builds whole 16-byte chunks of the tiles: 8 channels of one key for K~, 8 keys of one channel for
// V~^T (the transposition happens in shared memory).
// `mask_a` (nullable, u8 [sequences][T]) overrides which probability columns stay fp16 (Eq. 3's M_A); by default they
// are the columns of the fp16 K/V rows (M_A = M_KV).
__global__ void __launch_bounds__(256) kv_operands_kernel(const taq_layer_desc d, uint8_t* kv, const taq_request* reqs, const uint8_t* mask_a) {
    const int H = d.heads, T = d.n_ctx, D = d.channels / d.heads;
    const int h = blockIdx.x, z = blockIdx.y;
    const taq_kv_layout KL = kv_layout(H, T, D, d.max_trigger);
    OperandGeom g;
    if (!operand_geom(D, T, &g)) return;
    uint8_t* blk = reqs ? (uint8_t*)reqs[z].kv : kv + (size_t)z * KL.block_bytes;
    const __half* kt = (const __half*)(blk + KL.off_k_trigger);
    const __half* vt = (const __half*)(blk + KL.off_v_trigger);
    uint8_t* img = blk + KL.off_operands + (size_t)h * KL.operand_head_bytes;
    uint8_t* k_img = img;
    uint8_t* vt_img = img + g.k_bytes;
    OperandConsts* cst = reinterpret_cast<OperandConsts*>(img + g.k_bytes + g.vt_bytes);
    const size_t k_block = (size_t)kOperandKeys * 128, vt_block = (size_t)g.dp * 128;

    __shared__ __align__(16) int8_t s_kc[kOperandKeys * kMaxHeadDim];
    __shared__ __align__(16) int8_t s_vc[kOperandKeys * kMaxHeadDim];
    __shared__ float s_ks[kOperandKeys], s_vs[kOperandKeys];
    __shared__ int s_slot[kOperandKeys];
    {
        const uint2* kc8 = reinterpret_cast<const uint2*>(blk + KL.off_k_codes + (size_t)h * T * D);      // T * D is a multiple of 8
        const uint2* vc8 = reinterpret_cast<const uint2*>(blk + KL.off_v_codes + (size_t)h * T * D);
        for (int i = threadIdx.x; i < T * D / 8; i += blockDim.x) {
            reinterpret_cast<uint2*>(s_kc)[i] = kc8[i];
            reinterpret_cast<uint2*>(s_vc)[i] = vc8[i];
        }
        const float* ks = (const float*)(blk + KL.off_k_scales) + (size_t)h * T;
        const float* vs = (const float*)(blk + KL.off_v_scales) + (size_t)h * T;
        const int32_t* slot = (const int32_t*)(blk + KL.off_trig_slot);
        for (int j = threadIdx.x; j < kOperandKeys; j += blockDim.x) {
            s_ks[j] = j < T ? ks[j] : 0.f;
            s_vs[j] = j < T ? vs[j] : 0.f;
            s_slot[j] = j < T ? slot[j] : -1;
        }
    }
    __syncthreads();

    // K~ tile: chunk = 8 channels of key j
    const int kch = g.kbq * 8;
    for (int idx = threadIdx.x; idx < kOperandKeys * kch; idx += blockDim.x) {
        const int j = idx / kch, cc = idx % kch, c0 = cc * 8;
        uint4 out = make_uint4(0, 0, 0, 0);
        if (j < T && c0 < D) {
            const int sl = s_slot[j];
            if (sl >= 0) {
                out = *reinterpret_cast<const uint4*>(kt + ((size_t)sl * H + h) * D + c0);
            } else {
                __half2 hv[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    hv[e] = __halves2half2(__int2half_rn((int)s_kc[j * D + c0 + 2 * e]), __int2half_rn((int)s_kc[j * D + c0 + 2 * e + 1]));
                out = *reinterpret_cast<uint4*>(hv);
            }
        }
        *reinterpret_cast<uint4*>(k_img + (cc / 8) * k_block + ptx::sw128_offset(j, cc % 8)) = out;
    }
    // V~^T tile: chunk = 8 keys of channel c; ordinary rows are the fp16 operand of code * scale
    for (int idx = threadIdx.x; idx < g.dp * 16; idx += blockDim.x) {
        const int c = idx / 16, jc = idx % 16;
        __half hv[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int j = jc * 8 + e;
            __half v = __float2half_rn(0.f);
            if (j < T && c < D) {
                const int sl = s_slot[j];
                v = sl >= 0 ? vt[((size_t)sl * H + h) * D + c] : __float2half_rn(__fmul_rn((float)s_vc[j * D + c], s_vs[j]));
            }
            hv[e] = v;
        }
        *reinterpret_cast<uint4*>(vt_img + (jc / 8) * vt_block + ptx::sw128_offset(c, jc % 8)) = *reinterpret_cast<uint4*>(hv);
    }
    // constants
    const float logit_unit = 1.4426950408889634f / sqrtf((float)D);
    for (int j = threadIdx.x; j < kOperandKeys; j += blockDim.x)
        cst->logit_factor[j] = j < T ? (s_slot[j] >= 0 ? 1.0f : s_ks[j]) * logit_unit : 0.f;
    if (threadIdx.x < 4) {
        uint32_t bits = 0;
        for (int i = 0; i < 32; ++i) {
            const int j = threadIdx.x * 32 + i;
            if (j < T && (mask_a ? mask_a[(size_t)z * T + j] != 0 : s_slot[j] >= 0)) bits |= 1u << i;
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
