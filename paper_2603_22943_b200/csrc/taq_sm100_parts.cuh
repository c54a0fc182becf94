// Device helpers shared by the Blackwell (tcgen05) kernels: code expansion, quantizing stores, and the row-thread
// pieces of the softmax / Eq. 3.
#pragma once
#include "taq_common.cuh"
#include "taq_ptx.cuh"

namespace taq {
namespace parts {

constexpr int TP = kOperandKeys;     // keys padded to a multiple of 16

// Eight 4-bit codes of one word -> eight fp16 integers in fan-in order.  0x6400 | n read as fp16 is 1024 + n.
__device__ __forceinline__ uint4 codes_w4_to_half(uint32_t p) {
    const __half2 off = __floats2half2_rn(1032.f, 1032.f);                     // 1024 + the nibble bias of 8
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t w = ((p >> (4 * i)) & 0x000F000Fu) | 0x64006400u;
        __half2 h = __hsub2(*reinterpret_cast<__half2*>(&w), off);
        o[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}
// Eight int8 codes -> eight fp16 integers: (code + 128) rides in the mantissa of 0x64xx.
__device__ __forceinline__ uint4 codes_w8_to_half(uint2 raw) {
    const __half2 off = __floats2half2_rn(1152.f, 1152.f);
    const uint32_t w[2] = {raw.x ^ 0x80808080u, raw.y ^ 0x80808080u};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        uint32_t lo = __byte_perm(w[i], 0x64646464u, 0x5140);
        uint32_t hi = __byte_perm(w[i], 0x64646464u, 0x5342);
        __half2 a = __hsub2(*reinterpret_cast<__half2*>(&lo), off);
        __half2 b = __hsub2(*reinterpret_cast<__half2*>(&hi), off);
        o[2 * i] = *reinterpret_cast<uint32_t*>(&a);
        o[2 * i + 1] = *reinterpret_cast<uint32_t*>(&b);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// Eight 4-bit codes of one word -> eight int8 codes in fan-in order (the integer-activation GEMM's weight operand).
__device__ __forceinline__ uint2 codes_w4_to_i8(uint32_t p) {
    const uint32_t even = p & 0x0F0F0F0Fu;              // bytes: elements 0, 4, 1, 5 (+8)
    const uint32_t odd = (p >> 4) & 0x0F0F0F0Fu;        // bytes: elements 2, 6, 3, 7 (+8)
    return make_uint2(__vsub4(__byte_perm(even, odd, 0x6420), 0x08080808u), __vsub4(__byte_perm(even, odd, 0x7531), 0x08080808u));
}

__device__ __forceinline__ uint4 pack8(const float (&w)[8]) {
    uint4 out;
    __half2 h;
    h = __floats2half2_rn(w[0], w[1]); out.x = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2half2_rn(w[2], w[3]); out.y = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2half2_rn(w[4], w[5]); out.z = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2half2_rn(w[6], w[7]); out.w = *reinterpret_cast<uint32_t*>(&h);
    return out;
}

// Eight values -> eight int8 codes rint(x * rs): fma(x, rs, 1.5 * 2^23) leaves the two's-complement code in the low byte.
__device__ __forceinline__ uint2 quant8(const float* x, float rs) {
    uint32_t b[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) b[e] = __float_as_uint(fmaf(x[e], rs, 12582912.0f));
    const uint32_t lo = __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
    const uint32_t hi = __byte_perm(__byte_perm(b[4], b[5], 0x0040), __byte_perm(b[6], b[7], 0x0040), 0x5410);
    return make_uint2(lo, hi);
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

constexpr int HK = TP / 2;           // keys per thread: a row's scores are split between two threads

// Softmax pieces of one thread: its HK raw scores u (integer dot products) -> e_j = 2^(s_j sq - m) with the
// thread's own maximum m (log2 units), and their sum.  Keys at or beyond T get weight exactly 0.
template <bool TAIL_ONLY>
__device__ __forceinline__ void softmax_half(const uint32_t (&u)[HK], const float* factor, float sq, int T, int key0, float (&e)[HK], float& m_out, float& l_out) {
#pragma unroll
    for (int j4 = 0; j4 < HK / 4; ++j4) {
        const float4 f = *reinterpret_cast<const float4*>(factor + 4 * j4);
        e[4 * j4 + 0] = __uint_as_float(u[4 * j4 + 0]) * f.x;
        e[4 * j4 + 1] = __uint_as_float(u[4 * j4 + 1]) * f.y;
        e[4 * j4 + 2] = __uint_as_float(u[4 * j4 + 2]) * f.z;
        e[4 * j4 + 3] = __uint_as_float(u[4 * j4 + 3]) * f.w;
    }
#pragma unroll
    for (int j = 0; j < HK; ++j)
        if (j >= 64 - HK || !TAIL_ONLY) { if (key0 + j >= T) e[j] = -INFINITY; }
    float m4[4] = {-1e30f, -1e30f, -1e30f, -1e30f};          // finite floor: a thread whose keys are all padding
#pragma unroll
    for (int j = 0; j < HK; ++j) m4[j & 3] = fmaxf(m4[j & 3], e[j]);
    const float msq = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * sq;
    float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < HK; ++j) {
        float arg = fmaf(e[j], sq, -msq);
        if (j >= 64 - HK || !TAIL_ONLY) { if (key0 + j >= T) arg = -INFINITY; }      // also when sq = 0
        e[j] = ex2_approx(arg);
        sum4[j & 3] += e[j];
    }
    m_out = msq;
    l_out = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
}

// Eq. 3 on the thread's HK probabilities e_j * k255 (units of 1/255): ordinary columns -> rint (exact, ties to even),
// trigger columns -> fp16.  fma(e, k, 1.5 * 2^23 + 0x6400) leaves the integer code in the low byte and 0x64 above it,
// which read as fp16 is 1024 + code.  `trig` holds the thread's HK trigger bits.  Writes chunks chunk0.. of row `r`.
__device__ __forceinline__ void write_p_half(const float (&e)[HK], float k255, unsigned long long trig, unsigned char* p_tile, int a_block, int r, int chunk0) {
    const __half2 h1024 = __floats2half2_rn(1024.f, 1024.f);
#pragma unroll
    for (int g = 0; g < HK / 8; ++g) {
        const uint32_t bits = (uint32_t)(trig >> (8 * g)) & 0xFFu;
        uint32_t pk[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = g * 8 + 2 * i;
            const uint32_t x0 = __float_as_uint(fmaf(e[j], k255, 12608512.0f));
            const uint32_t x1 = __float_as_uint(fmaf(e[j + 1], k255, 12608512.0f));
            uint32_t w = __byte_perm(x0, x1, 0x5410);
            __half2 hv = __hsub2(*reinterpret_cast<__half2*>(&w), h1024);
            pk[i] = *reinterpret_cast<uint32_t*>(&hv);
        }
        if (bits != 0) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int j = g * 8 + 2 * i;
                __half2 raw = __floats2half2_rn(e[j] * k255, e[j + 1] * k255);
                const uint32_t sel = (((bits >> (2 * i)) & 1u) ? 0x0054u : 0x0010u) | (((bits >> (2 * i + 1)) & 1u) ? 0x7600u : 0x3200u);
                pk[i] = __byte_perm(pk[i], *reinterpret_cast<uint32_t*>(&raw), sel);
            }
        }
        const int chunk = chunk0 + g;
        *reinterpret_cast<uint4*>(p_tile + (chunk >> 3) * a_block + ptx::sw128_offset(r, chunk & 7)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
}

// The logarithmic reading of the probability quantizer: t = e_j * k is 256 p; ordinary columns take
// code = clamp(rint(-log2 p), 0, cmax) = clamp(rint(8 - log2 t), 0, cmax) and are stored as the fp16 value 2^(8 - code)
// (units of 1/256; exact down to the smallest fp16 subnormal at code 32, zero beyond); trigger columns are fp16(t).
__device__ __forceinline__ uint32_t log_code_to_half_bits(float t, float cmax) {
    const float x = 8.0f - __log2f(t);                      // t = 0 -> +inf -> the last code
    const int c = (int)fminf(fmaxf(rintf(x), 0.f), cmax);
    return c <= 22 ? (uint32_t)(23 - c) << 10 : (c <= 32 ? 1u << (32 - c) : 0u);
}
__device__ __forceinline__ void write_p_half_log(const float (&e)[HK], float k256, float cmax, unsigned long long trig, unsigned char* p_tile, int a_block, int r, int chunk0) {
#pragma unroll
    for (int g = 0; g < HK / 8; ++g) {
        const uint32_t bits = (uint32_t)(trig >> (8 * g)) & 0xFFu;
        uint32_t pk[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = g * 8 + 2 * i;
            const float t0 = e[j] * k256, t1 = e[j + 1] * k256;
            uint32_t h0 = log_code_to_half_bits(t0, cmax), h1 = log_code_to_half_bits(t1, cmax);
            if ((bits >> (2 * i)) & 1u) h0 = __half_as_ushort(__float2half_rn(t0));
            if ((bits >> (2 * i + 1)) & 1u) h1 = __half_as_ushort(__float2half_rn(t1));
            pk[i] = h0 | (h1 << 16);
        }
        const int chunk = chunk0 + g;
        *reinterpret_cast<uint4*>(p_tile + (chunk >> 3) * a_block + ptx::sw128_offset(r, chunk & 7)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
}

}  // namespace parts
}  // namespace taq
