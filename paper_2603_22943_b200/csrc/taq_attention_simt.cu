// Generic fused TAQ attention on CUDA cores (any head width up to 256, any T up to 128).
// One CTA = one (sequence, head, block of query rows).  K~ and V~ of that head sit in shared memory as fp16:
// ordinary rows hold their integer codes (exact in fp16) next to a per-row scale, trigger rows hold their fp16
// values with scale 1, so one inner product serves both kinds of row (Eq. 2).  A warp owns a query row: the
// lanes split the T keys for the scores and the softmax (max and sum by warp shuffles), apply Eq. 3 to the
// probabilities, then split the d output channels for P.V.  Scores and probabilities stay on chip.
#include "taq_common.cuh"

namespace taq {

constexpr int ATT_WARPS = 4;
constexpr int ATT_ROWS = 16;   // query rows per CTA

__global__ void __launch_bounds__(ATT_WARPS * 32) attention_simt_kernel(const AttnArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int d = a.channels / a.heads, T = a.n_ctx, C = a.channels;
    const int ldk = d + 2;
    __half* Ks = reinterpret_cast<__half*>(smem_raw);          // [T][ldk]
    __half* Vs = Ks + (size_t)T * ldk;                           // [T][ldk]  (ordinary rows already times scale)
    float* ksc = reinterpret_cast<float*>(Vs + (size_t)T * ldk);  // [T] logit scale of key j (includes 1/sqrt(d))
    float* qs = ksc + kMaxCtx;                                   // [ATT_WARPS][d]
    float* ps = qs + ATT_WARPS * d;                              // [ATT_WARPS][kMaxCtx]
    unsigned char* msk = reinterpret_cast<unsigned char*>(ps + ATT_WARPS * kMaxCtx);   // [T]

    const int h = blockIdx.y;
    const int zb = blockIdx.z;                                   // sequence index (batch entry or request)
    const int b = a.reqs ? 0 : zb;
    const taq_kv_layout KL = kv_layout(a.heads, T, d, a.max_trigger);
    const uint8_t* blk = a.reqs ? (const uint8_t*)a.reqs[zb].kv : (const uint8_t*)a.kv + (size_t)b * KL.block_bytes;
    const uint8_t* mask = a.reqs ? a.reqs[zb].trig_mask : a.mask + (size_t)b * T;
    const int8_t* kc = (const int8_t*)(blk + KL.off_k_codes) + (size_t)h * T * d;
    const int8_t* vc = (const int8_t*)(blk + KL.off_v_codes) + (size_t)h * T * d;
    const float* ks = (const float*)(blk + KL.off_k_scales) + (size_t)h * T;
    const float* vs = (const float*)(blk + KL.off_v_scales) + (size_t)h * T;
    const __half* kt = (const __half*)(blk + KL.off_k_trigger);
    const __half* vt = (const __half*)(blk + KL.off_v_trigger);
    const int32_t* slot = (const int32_t*)(blk + KL.off_trig_slot);
    const float inv_sqrt_d = 1.0f / sqrtf((float)d);

    for (int idx = threadIdx.x; idx < T * d; idx += blockDim.x) {
        const int j = idx / d, c = idx % d;
        const int sl = slot[j];
        __half kv, vv;
        if (sl >= 0) {
            kv = kt[((size_t)sl * a.heads + h) * d + c];
            vv = vt[((size_t)sl * a.heads + h) * d + c];
        } else {
            kv = __int2half_rn((int)kc[idx]);
            vv = __float2half_rn(__fmul_rn((float)vc[idx], vs[j]));   // fp16 operand of the dequantized row
        }
        Ks[j * ldk + c] = kv;
        Vs[j * ldk + c] = vv;
    }
    for (int j = threadIdx.x; j < T; j += blockDim.x) {
        ksc[j] = (slot[j] >= 0 ? 1.0f : ks[j]) * inv_sqrt_d;
        msk[j] = mask[j];
    }
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* q = qs + warp * d;
    float* p = ps + warp * kMaxCtx;
    const size_t seq_off = (size_t)zb * a.n_query;
    for (int r = warp; r < ATT_ROWS; r += ATT_WARPS) {
        const int n = blockIdx.x * ATT_ROWS + r;
        if (n >= a.n_query) break;
        float sq = 1.0f;
        if (a.q_bits == 8) {
            const int8_t* qrow = (const int8_t*)a.q + (seq_off + n) * C + h * d;
            for (int c = lane; c < d; c += 32) q[c] = (float)qrow[c];
            sq = a.q_scales[(seq_off + n) * a.heads + h];
        } else {
            const __half* qrow = (const __half*)a.q + (seq_off + n) * C + h * d;
            for (int c = lane; c < d; c += 32) q[c] = __half2float(qrow[c]);
        }
        __syncwarp();
        // scores: lane owns keys lane, lane+32, ...
        float s[4];
        float mx = -INFINITY;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int j = lane + 32 * u;
            s[u] = -INFINITY;
            if (j < T) {
                float acc = 0.f;
                const __half* kr = Ks + j * ldk;
                for (int c = 0; c < d; c += 2) {
                    const float2 k2 = __half22float2(*reinterpret_cast<const __half2*>(kr + c));
                    acc = fmaf(q[c], k2.x, acc);
                    acc = fmaf(q[c + 1], k2.y, acc);
                }
                s[u] = acc * (sq * ksc[j]);
                mx = fmaxf(mx, s[u]);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        float sum = 0.f;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (lane + 32 * u < T) { s[u] = expf(s[u] - mx); sum += s[u]; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int j = lane + 32 * u;
            if (j < T) {
                const float pj = __fdiv_rn(s[u], sum);
                float ph;
                const float pmax = a.p_log ? 256.0f : a.p_bits == 4 ? 15.0f : 255.0f;             // the unit of the stored probabilities is 1 / pmax
                if (msk[j] || a.p_bits == 0) ph = __fdiv_rn(__half2float(__float2half_rn(__fmul_rn(pj, pmax))), pmax);     // Eq. 3, trigger column: fp16 in units of 1/pmax
                else if (a.p_log) {                                                                  // logarithmic code: p^ = 2^-clamp(rint(-log2 p))
                    const float cmax = a.p_bits == 4 ? 15.0f : 255.0f;
                    const float code = pj > 0.f ? fminf(fmaxf(rintf(-log2f(pj)), 0.f), cmax) : cmax;
                    ph = code <= 32.f ? exp2f(-code) : 0.f;                                          // (an fp16 operand in units of 1/256)
                }
                else ph = __fdiv_rn(rintf(__fmul_rn(pj, pmax)), pmax);                               // Eq. 3, integer code / pmax
                p[j] = ph;
            }
        }
        __syncwarp();
        __half* orow = a.o + (seq_off + n) * C + h * d;
        for (int c = lane; c < d; c += 32) {
            float acc = 0.f;
            for (int j = 0; j < T; ++j) acc = fmaf(p[j], __half2float(Vs[j * ldk + c]), acc);
            orow[c] = __float2half_rn(acc);
        }
        __syncwarp();
    }
}

static size_t attention_simt_smem(int T, int d) {
    return sizeof(__half) * 2 * (size_t)T * (d + 2) + sizeof(float) * (kMaxCtx + ATT_WARPS * d + ATT_WARPS * kMaxCtx) + kMaxCtx;
}

cudaError_t launch_attention_simt(const AttnArgs& a, int n_z, cudaStream_t stream) {
    if (a.n_query == 0 || n_z == 0) return cudaSuccess;
    const int d = a.channels / a.heads;
    const size_t smem = attention_simt_smem(a.n_ctx, d);
    cudaError_t e = cudaFuncSetAttribute(attention_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((a.n_query + ATT_ROWS - 1) / ATT_ROWS, a.heads, n_z);
    attention_simt_kernel<<<grid, ATT_WARPS * 32, smem, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace taq
