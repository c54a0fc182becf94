// Stand-alone quantizers: activation rows (Q_a of Eq. 2) and weight packing (W8 / W4 per output channel).
// Integer codes are compared bit for bit with the CPU definition, so every floating-point step here is an
// explicit IEEE binary32 operation (__fdiv_rn, rintf); nothing may be contracted or approximated.
#include "taq_common.cuh"

namespace taq {

__device__ inline float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// One warp per row.  Memory-bound: the row is read twice (absmax, then codes); the second read hits L1/L2.
__global__ void __launch_bounds__(256) quantize_rows_kernel(const float* __restrict__ x, long long rows, int cols, int qmax,
                                                            int8_t* __restrict__ codes, float* __restrict__ scales) {
    const int lane = threadIdx.x & 31;
    const long long warps_total = (long long)gridDim.x * (blockDim.x >> 5);
    for (long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < rows; r += warps_total) {
        const float* xr = x + r * cols;
        float a = 0.f;
        if ((cols & 3) == 0) {
            const float4* x4 = reinterpret_cast<const float4*>(xr);
            for (int i = lane; i < cols / 4; i += 32) {
                float4 v = x4[i];
                a = fmaxf(a, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
            }
        } else {
            for (int i = lane; i < cols; i += 32) a = fmaxf(a, fabsf(xr[i]));
        }
        a = warp_max(a);
        const float s = quant_scale(a, (float)qmax);
        if (lane == 0) scales[r] = s;
        int8_t* cr = codes + r * cols;
        if ((cols & 3) == 0) {
            const float4* x4 = reinterpret_cast<const float4*>(xr);
            char4* c4 = reinterpret_cast<char4*>(cr);
            for (int i = lane; i < cols / 4; i += 32) {
                float4 v = x4[i];
                c4[i] = make_char4((signed char)quant_code(v.x, s, qmax), (signed char)quant_code(v.y, s, qmax),
                                   (signed char)quant_code(v.z, s, qmax), (signed char)quant_code(v.w, s, qmax));
            }
        } else {
            for (int i = lane; i < cols; i += 32) cr[i] = (int8_t)quant_code(xr[i], s, qmax);
        }
    }
}

cudaError_t launch_quantize_rows(const float* x, long long rows, int cols, int qmax, int8_t* codes, float* scales,
                                 cudaStream_t stream) {
    if (rows == 0) return cudaSuccess;
    long long blocks = (rows + 7) / 8;
    if (blocks > 148LL * 32) blocks = 148LL * 32;   // grid-stride beyond 32 resident waves
    quantize_rows_kernel<<<(unsigned)blocks, 256, 0, stream>>>(x, rows, cols, qmax, codes, scales);
    return cudaGetLastError();
}

// rint(x / s) clamped to +-127, bit-identical to quant_code (one IEEE division, then rintf) at a fraction of its cost.
// fma(x, r, 1.5 * 2^23) leaves rint(x r) in the low bits.  The rounded quotient fl(x / s) and the product with the
// correctly rounded reciprocal both lie between x r_lo and x r_hi (r two ulps down and up), so when both ends round to
// the same integer that integer is the code; only otherwise the division decides.
__device__ __noinline__ int code_127_by_division(float x, float s) { return (int)fminf(fmaxf(rintf(__fdiv_rn(x, s)), -127.f), 127.f); }
__device__ __forceinline__ int quant_code_127(float x, float s, float r_lo, float r_hi) {
    const uint32_t a = __float_as_uint(fmaf(x, r_lo, 12582912.0f)), c = __float_as_uint(fmaf(x, r_hi, 12582912.0f));
    if (a != c) return code_127_by_division(x, s);     // (fp16 data: about 4 values in 10000, e.g. exactly half of the row maximum)
    return (int)(a << 24) >> 24;                       // the low byte, sign-extended
}

// Per-token quantizer of fp16 activations (the inputs of the integer-activation projections): one warp per row of
// `cols` fp16 values (a multiple of 8), which it keeps in registers between the absmax pass and the code pass when the
// row is short enough (KEEP x 256 columns), so that the row is read once.  Same results as quantize_rows_kernel.
template <int KEEP>
__global__ void __launch_bounds__(256) quantize_rows_f16_kernel(const __half* __restrict__ x, long long rows, int cols,
                                                                int8_t* __restrict__ codes, float* __restrict__ scales) {
    // Launched with the programmatic-serialization attribute: the successor (the integer GEMM) may start its prologue
    // now; this kernel's input may come from the predecessor, so it is read only after the wait.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31;
    const long long warps_total = (long long)gridDim.x * (blockDim.x >> 5);
    const int chunks = cols / 8;                                 // 16-byte chunks of a row
    for (long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < rows; r += warps_total) {
        const uint4* xr = reinterpret_cast<const uint4*>(x + r * cols);
        uint4 keep[KEEP];
        float a = 0.f;
        auto absmax8 = [&](const uint4& v) {
            const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
            for (int e = 0; e < 4; ++e) { const float2 f = __half22float2(h[e]); a = fmaxf(a, fmaxf(fabsf(f.x), fabsf(f.y))); }
        };
#pragma unroll
        for (int j = 0; j < KEEP; ++j) {
            const int i = lane + 32 * j;
            keep[j] = make_uint4(0, 0, 0, 0);
            if (i < chunks) keep[j] = xr[i];
        }
#pragma unroll
        for (int j = 0; j < KEEP; ++j) absmax8(keep[j]);
        for (int i = lane + 32 * KEEP; i < chunks; i += 32) absmax8(xr[i]);
        a = warp_max(a);
        const float s = quant_scale(a, 127.f);
        const float rs = s > 0.f ? __frcp_rn(s) : 0.f;
        const float r_lo = __uint_as_float(__float_as_uint(rs) - 2u), r_hi = __uint_as_float(__float_as_uint(rs) + 2u);
        if (lane == 0) scales[r] = s;
        uint2* cr = reinterpret_cast<uint2*>(codes + r * cols);
        auto encode = [&](const uint4& v) {
            const __half2* h = reinterpret_cast<const __half2*>(&v);
            uint32_t w[2] = {0, 0};
            if (s > 0.f) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __half22float2(h[e]);
                    w[e >> 1] |= ((uint32_t)(quant_code_127(f.x, s, r_lo, r_hi) & 0xFF) | ((uint32_t)(quant_code_127(f.y, s, r_lo, r_hi) & 0xFF) << 8)) << (16 * (e & 1));
                }
            }
            return make_uint2(w[0], w[1]);
        };
#pragma unroll
        for (int j = 0; j < KEEP; ++j) {
            const int i = lane + 32 * j;
            if (i < chunks) cr[i] = encode(keep[j]);
        }
        for (int i = lane + 32 * KEEP; i < chunks; i += 32) cr[i] = encode(xr[i]);
    }
}

cudaError_t launch_quantize_rows_f16(const __half* x, long long rows, int cols, int8_t* codes, float* scales, cudaStream_t stream) {
    if (rows == 0) return cudaSuccess;
    long long blocks = (rows + 7) / 8;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    if (cols <= 512) return launch_pdl(quantize_rows_f16_kernel<2>, dim3((unsigned)blocks), dim3(256), 0, stream, x, rows, cols, codes, scales);
    return launch_pdl(quantize_rows_f16_kernel<8>, dim3((unsigned)blocks), dim3(256), 0, stream, x, rows, cols, codes, scales);
}

// ---- helpers of the token-sensitivity sweep (Eq. 1) -------------------------------------------------------------
__global__ void __launch_bounds__(256) mse_partial_kernel(const __half* __restrict__ a, const __half* __restrict__ b, long long n, double* __restrict__ partials) {
    double acc = 0.0;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const float dlt = __half2float(a[i]) - __half2float(b[i]);
        acc += (double)dlt * (double)dlt;
    }
    __shared__ double sh[256];
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {           // fixed tree: the same sum for the same inputs
        if (threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) partials[blockIdx.x] = sh[0];
}
__global__ void __launch_bounds__(256) mse_final_kernel(const double* __restrict__ partials, long long n, double* __restrict__ out) {
    __shared__ double sh[256];
    sh[threadIdx.x] = partials[threadIdx.x];
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if (threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = sh[0] / (double)n;
}
cudaError_t launch_mse_f16(const __half* a, const __half* b, long long n, double* partials, double* out, cudaStream_t stream) {
    mse_partial_kernel<<<256, 256, 0, stream>>>(a, b, n, partials);
    mse_final_kernel<<<1, 256, 0, stream>>>(partials, n, out);
    return cudaGetLastError();
}
__global__ void sensitivity_masks_kernel(uint8_t* masks, int batch, int n_ctx) {
    const long long total = (long long)(n_ctx + 1) * batch * n_ctx;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int t = (int)(i % n_ctx), which = (int)(i / ((long long)batch * n_ctx));
        masks[i] = (which == n_ctx || t != which) ? 1 : 0;
    }
}
cudaError_t launch_sensitivity_masks(uint8_t* masks, int batch, int n_ctx, cudaStream_t stream) {
    sensitivity_masks_kernel<<<64, 256, 0, stream>>>(masks, batch, n_ctx);
    return cudaGetLastError();
}

// One warp per (output channel, group).
__global__ void __launch_bounds__(256) pack_weights_kernel(const float* __restrict__ W, const float* __restrict__ bias, uint8_t* __restrict__ blob,
                                                           int n_out, int k_in, int bits, int group) {
    const WeightLayout L = weight_layout(n_out, k_in, bits, group);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        PackedHeader h;
        h.magic = kWeightMagic; h.version = 1; h.n_out = n_out; h.k_in = k_in; h.bits = bits; h.group = group;
        h.n_groups = L.n_groups; h.has_bias = bias != nullptr;
        h.off_codes = L.off_codes; h.off_scales = L.off_scales; h.off_bias = L.off_bias; h.total_bytes = L.total;
        *reinterpret_cast<PackedHeader*>(blob) = h;
    }
    const int lane = threadIdx.x & 31;
    const int qmax = bits == 8 ? 127 : 7;
    const long long items = (long long)n_out * L.n_groups;
    const long long warps_total = (long long)gridDim.x * (blockDim.x >> 5);
    float* scales = reinterpret_cast<float*>(blob + L.off_scales);
    float* bias_out = reinterpret_cast<float*>(blob + L.off_bias);
    uint8_t* codes = blob + L.off_codes;
    for (long long it = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); it < items; it += warps_total) {
        const int n = (int)(it / L.n_groups), g = (int)(it % L.n_groups);
        const int lo = g * L.group_len, hi = min(k_in, lo + L.group_len);
        const float* wr = W + (size_t)n * k_in;
        float a = 0.f;
        for (int k = lo + lane; k < hi; k += 32) a = fmaxf(a, fabsf(wr[k]));
        a = warp_max(a);
        const float s = quant_scale(a, (float)qmax);
        if (lane == 0) {
            scales[(size_t)n * L.n_groups + g] = s;
            if (g == 0) bias_out[n] = bias ? bias[n] : 0.f;
        }
        if (bits == 8) {
            for (int k = lo + lane; k < hi; k += 32) ((int8_t*)codes)[(size_t)n * L.row_bytes + k] = (int8_t)quant_code(wr[k], s, qmax);
        } else {
            for (int k = lo + 8 * lane; k < hi; k += 256) {   // group bounds are multiples of 8: a word never straddles groups
                uint32_t word = 0;
#pragma unroll
                for (int e = 0; e < 8; ++e) word |= (uint32_t)(quant_code(wr[k + e], s, qmax) + 8) << (4 * w4_nibble_pos(e));
                *reinterpret_cast<uint32_t*>(codes + (size_t)n * L.row_bytes + (k >> 1)) = word;
            }
        }
    }
}

cudaError_t launch_pack_weights(const taq_weight_desc& d, const float* W, const float* bias, void* packed, cudaStream_t stream) {
    const WeightLayout L = weight_layout(d.n_out, d.k_in, d.bits, d.group);
    long long items = (long long)d.n_out * L.n_groups;
    long long blocks = (items + 7) / 8;
    if (blocks > 148LL * 32) blocks = 148LL * 32;
    pack_weights_kernel<<<(unsigned)blocks, 256, 0, stream>>>(W, bias, (uint8_t*)packed, d.n_out, d.k_in, d.bits, d.group);
    return cudaGetLastError();
}

__global__ void __launch_bounds__(256) unpack_weights_kernel(const uint8_t* __restrict__ blob, int8_t* __restrict__ codes_out,
                                                             float* __restrict__ scales_out, int n_out, int k_in, int bits, int group) {
    const WeightLayout L = weight_layout(n_out, k_in, bits, group);
    const long long total = (long long)n_out * k_in;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
        const int n = (int)(i / k_in), k = (int)(i % k_in);
        codes_out[i] = (int8_t)load_code(blob + L.off_codes, L.row_bytes, bits, n, k);
    }
    const float* scales = reinterpret_cast<const float*>(blob + L.off_scales);
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < (long long)n_out * L.n_groups; i += stride) scales_out[i] = scales[i];
}

cudaError_t launch_unpack_weights(const taq_weight_desc& d, const void* packed, int8_t* codes, float* scales, cudaStream_t stream) {
    long long total = (long long)d.n_out * d.k_in;
    long long blocks = (total + 255) / 256;
    if (blocks > 148LL * 16) blocks = 148LL * 16;
    unpack_weights_kernel<<<(unsigned)blocks, 256, 0, stream>>>((const uint8_t*)packed, codes, scales, d.n_out, d.k_in, d.bits, d.group);
    return cudaGetLastError();
}

}  // namespace taq
