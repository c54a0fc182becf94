// Fused TAQ attention on the Blackwell tensor cores (tcgen05 + TMEM), one pass, nothing but Q~ in and O out:
//   S = Q~ K~^T          tcgen05.mma, fp16 operands holding the int8 codes exactly (trigger rows: their fp16 values)
//   A = softmax(S * scale)   one thread per query row, the row's 80 scores live in its registers (TMEM lane)
//   A^ (Eq. 3)            ordinary columns -> uint8 code, trigger columns -> fp16, both in units of 1/255
//   O = A^ V~             tcgen05.mma with the probabilities as the A operand, V~^T (fp16) as B; O = acc / 255
// A CTA owns 128 query rows of one sequence and walks over a group of heads.  Per head the four worker warps stage
// the head's mixed-precision K~ and V~^T (Eq. 2) and the row tile of Q~ codes into 128-byte-swizzled K-major
// operand tiles, a fifth warp issues the MMAs, and the workers (thread = row = TMEM lane) run the softmax and the
// epilogue.  Several CTAs share an SM, so one CTA's staging overlaps another's MMA and softmax.
#include "taq_ptx.cuh"
#include "taq_sm100.cuh"

namespace taq {

namespace {

constexpr int TP = 80;           // keys padded to a multiple of 16
constexpr int ROWS = 128;
constexpr int NWORK = 128;
constexpr int ATT_THREADS = 160;

template <int D>
struct Cfg {
    static constexpr int DP = (D + 15) / 16 * 16;            // head width padded to the MMA K / N granule
    static constexpr int KBQ = (DP + 63) / 64;               // 64-wide k-blocks of the Q~ and K~ tiles
    static constexpr int A_BLOCK = ROWS * 128;
    static constexpr int K_BLOCK = TP * 128;
    static constexpr int VT_BLOCK = DP * 128;
    static constexpr int KBP = 2;                            // k-blocks of the probability tile (64 + 16 keys)
    static constexpr int OFF_A = 0;
    static constexpr int OFF_K = OFF_A + KBQ * A_BLOCK;
    static constexpr int OFF_VT = OFF_K + KBQ * K_BLOCK;
    static constexpr int OFF_P = OFF_VT + KBP * VT_BLOCK;
    static constexpr int OFF_MISC = OFF_P + KBP * A_BLOCK;
    static constexpr int TOTAL = OFF_MISC + 2048 + 1024;     // misc block + slack for 1024-byte alignment
    static constexpr uint32_t TMEM_COLS = (TP + DP) <= 128 ? 128 : 256;
    static_assert(VT_BLOCK % 1024 == 0 && K_BLOCK % 1024 == 0, "operand blocks must keep 1024-byte alignment");
};

struct Misc {
    uint64_t bar_ab, bar_s, bar_p, bar_o;
    uint32_t tmem_base;
    volatile int abort_flag;
    int slot[TP];            // fp16 slot of key j, -1 for an ordinary key, -2 for padding
    float2 fm[TP];           // {logit factor of key j (K scale * log2 e / sqrt d), rounding constant of Eq. 3}
    float vs[TP];            // V scale of key j
};
static_assert(sizeof(Misc) <= 2048, "misc block");

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Eight int8 codes -> eight fp16 integers (exact): 0x64xx is 1024 + xx, so (code + 128) rides in the mantissa.
__device__ __forceinline__ uint4 codes8_to_half(uint2 raw) {
    const __half2 bias = __floats2half2_rn(1152.f, 1152.f);
    uint32_t w[2] = {raw.x ^ 0x80808080u, raw.y ^ 0x80808080u};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        uint32_t lo = __byte_perm(w[i], 0x64646464u, 0x5140);
        uint32_t hi = __byte_perm(w[i], 0x64646464u, 0x5342);
        __half2 a = __hsub2(*reinterpret_cast<__half2*>(&lo), bias);
        __half2 b = __hsub2(*reinterpret_cast<__half2*>(&hi), bias);
        o[2 * i] = *reinterpret_cast<uint32_t*>(&a);
        o[2 * i + 1] = *reinterpret_cast<uint32_t*>(&b);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

template <int D>
__global__ void __launch_bounds__(ATT_THREADS, 2) attention_sm100_kernel(const AttnArgs a, const int heads_per_cta) {
    using C = Cfg<D>;
    constexpr int DP = C::DP;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    Misc* misc = reinterpret_cast<Misc*>(smem + C::OFF_MISC);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = a.n_ctx, H = a.heads, Cch = a.channels;
    const int zb = blockIdx.z;
    const int b = a.reqs ? 0 : zb;
    const int row0 = blockIdx.x * ROWS;
    const int h_begin = blockIdx.y * heads_per_cta;

    if (tid == 0) {
        ptx::mbar_init(&misc->bar_ab, NWORK);
        ptx::mbar_init(&misc->bar_s, 1);
        ptx::mbar_init(&misc->bar_p, NWORK);
        ptx::mbar_init(&misc->bar_o, 1);
        misc->abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == 4) ptx::tmem_alloc(&misc->tmem_base, C::TMEM_COLS);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = misc->tmem_base;
    const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + TP;

    if (warp == 4) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t a_addr = ptx::smem_u32(smem + C::OFF_A), k_addr = ptx::smem_u32(smem + C::OFF_K);
            const uint32_t p_addr = ptx::smem_u32(smem + C::OFF_P), vt_addr = ptx::smem_u32(smem + C::OFF_VT);
            for (int hi = 0; hi < heads_per_cta; ++hi) {
                const uint32_t ph = hi & 1;
                if (!ptx::mbar_wait(&misc->bar_ab, ph)) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
                if (misc->abort_flag) break;
                ptx::tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < DP / 16; ++ks)
                    ptx::mma_f16_ss(tmem_s, ptx::desc_k_sw128(a_addr + (ks / 4) * C::A_BLOCK + (ks % 4) * 32),
                                    ptx::desc_k_sw128(k_addr + (ks / 4) * C::K_BLOCK + (ks % 4) * 32), ptx::idesc_f16_m128(TP), ks != 0);
                ptx::mma_commit(&misc->bar_s);
                if (!ptx::mbar_wait(&misc->bar_p, ph)) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
                if (misc->abort_flag) break;
                ptx::tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < TP / 16; ++ks)
                    ptx::mma_f16_ss(tmem_o, ptx::desc_k_sw128(p_addr + (ks / 4) * C::A_BLOCK + (ks % 4) * 32),
                                    ptx::desc_k_sw128(vt_addr + (ks / 4) * C::VT_BLOCK + (ks % 4) * 32), ptx::idesc_f16_m128(DP), ks != 0);
                ptx::mma_commit(&misc->bar_o);
            }
        }
    } else {
        // ---------------- workers: thread = query row = TMEM lane ----------------
        const taq_kv_layout KL = kv_layout(H, T, D, a.max_trigger);
        const uint8_t* blk = a.reqs ? (const uint8_t*)a.reqs[zb].kv : (const uint8_t*)a.kv + (size_t)b * KL.block_bytes;
        const uint8_t* mask = a.reqs ? a.reqs[zb].trig_mask : a.mask + (size_t)b * T;
        const int32_t* gslot = (const int32_t*)(blk + KL.off_trig_slot);
        const __half* kt = (const __half*)(blk + KL.off_k_trigger);
        const __half* vt = (const __half*)(blk + KL.off_v_trigger);
        const int n = row0 + tid;
        const bool valid = n < a.n_query;
        const size_t grow = (size_t)zb * a.n_query + (valid ? n : 0);
        const float logit_unit = 1.4426950408889634f / sqrtf((float)D);
        const uint32_t lane_addr = (uint32_t)(warp * 32) << 16;
        bool alive = true;

        for (int hi = 0; hi < heads_per_cta && alive; ++hi) {
            const int h = h_begin + hi;
            const uint32_t ph = hi & 1;
            const int8_t* kc = (const int8_t*)(blk + KL.off_k_codes) + (size_t)h * T * D;
            const int8_t* vc = (const int8_t*)(blk + KL.off_v_codes) + (size_t)h * T * D;
            const float* ks = (const float*)(blk + KL.off_k_scales) + (size_t)h * T;
            const float* vs = (const float*)(blk + KL.off_v_scales) + (size_t)h * T;

            // per-key constants of this head
            if (tid < TP) {
                const int j = tid;
                int sl = -2;
                float f = 0.f, m = 0.f, v = 0.f;
                if (j < T) {
                    sl = gslot[j];
                    f = (sl >= 0 ? 1.0f : ks[j]) * logit_unit;
                    m = mask[j] ? 0.f : 12582912.f;        // (x + 1.5*2^23) - 1.5*2^23 rounds x to the nearest-even integer
                    v = vs[j];
                }
                misc->slot[j] = sl;
                misc->fm[j] = make_float2(f, m);
                misc->vs[j] = v;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");

            // K~ tile: [TP keys][DP], ordinary rows as exact fp16 integers, trigger rows as their fp16 values (Eq. 2)
            for (int idx = tid; idx < TP * (DP / 8); idx += NWORK) {
                const int j = idx / (DP / 8), cc = idx % (DP / 8);
                uint4 v = make_uint4(0, 0, 0, 0);
                const int sl = misc->slot[j];
                if (cc * 8 < D && sl != -2) {
                    if (sl >= 0) v = *reinterpret_cast<const uint4*>(kt + ((size_t)sl * H + h) * D + cc * 8);
                    else v = codes8_to_half(*reinterpret_cast<const uint2*>(kc + (size_t)j * D + cc * 8));
                }
                *reinterpret_cast<uint4*>(smem + C::OFF_K + (cc / 8) * C::K_BLOCK + ptx::sw128_offset(j, cc % 8)) = v;
            }
            // V~^T tile: [DP channels][TP keys]; ordinary rows are the fp16 operand of code * scale
            for (int idx = tid; idx < DP * (TP / 8); idx += NWORK) {
                const int c = idx % DP, jc = idx / DP;
                uint32_t pk[4];
#pragma unroll
                for (int i2 = 0; i2 < 4; ++i2) {
                    float v2[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int j = jc * 8 + i2 * 2 + e;
                        const int sl = misc->slot[j];
                        float v = 0.f;
                        if (c < D && sl != -2) {
                            if (sl >= 0) v = __half2float(vt[((size_t)sl * H + h) * D + c]);
                            else v = __fmul_rn((float)vc[(size_t)j * D + c], misc->vs[j]);
                        }
                        v2[e] = v;
                    }
                    __half2 hv = __floats2half2_rn(v2[0], v2[1]);
                    pk[i2] = *reinterpret_cast<uint32_t*>(&hv);
                }
                *reinterpret_cast<uint4*>(smem + C::OFF_VT + (jc / 8) * C::VT_BLOCK + ptx::sw128_offset(c, jc % 8)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            // Q~ tile: this thread's row
            float sq = 1.0f;
            {
#pragma unroll
                for (int cc = 0; cc < DP / 8; ++cc) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (cc * 8 < D && valid) {
                        if (a.q_bits == 8) v = codes8_to_half(*reinterpret_cast<const uint2*>((const int8_t*)a.q + grow * Cch + h * D + cc * 8));
                        else v = *reinterpret_cast<const uint4*>((const __half*)a.q + grow * Cch + h * D + cc * 8);
                    }
                    *reinterpret_cast<uint4*>(smem + C::OFF_A + (cc / 8) * C::A_BLOCK + ptx::sw128_offset(tid, cc % 8)) = v;
                }
                if (a.q_bits == 8) sq = valid ? a.q_scales[grow * H + h] : 0.f;
            }
            ptx::fence_proxy_async_smem();
            ptx::mbar_arrive(&misc->bar_ab);

            // ---- scores -> softmax -> Eq. 3 -> probability operand ----
            alive = __all_sync(0xffffffffu, ptx::mbar_wait(&misc->bar_s, ph) && !misc->abort_flag);
            if (!alive) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; break; }
            ptx::tc_fence_after_sync();
            uint32_t u[TP / 16][16];
#pragma unroll
            for (int c = 0; c < TP / 16; ++c) ptx::tmem_ld16(tmem_s + lane_addr + c * 16, u[c]);
            ptx::tmem_ld_wait(u[0]);
#pragma unroll
            for (int c = 1; c < TP / 16; ++c) ptx::reg_fence(u[c]);
            float s[TP];
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < TP; ++j) {
                s[j] = __uint_as_float(u[j / 16][j % 16]) * misc->fm[j].x;
                if (j >= 64 || T <= 64) { if (j >= T) s[j] = -INFINITY; }
                mx = fmaxf(mx, s[j]);
            }
            const float msq = mx * sq;
            float sum = 0.f;
#pragma unroll
            for (int j = 0; j < TP; ++j) {
                float arg = fmaf(s[j], sq, -msq);
                if (j >= 64 || T <= 64) { if (j >= T) arg = -INFINITY; }      // padded keys: weight exactly 0, also when sq = 0
                s[j] = ex2_approx(arg);
                sum += s[j];
            }
            const float k255 = __fdividef(255.0f, sum);
#pragma unroll
            for (int jc = 0; jc < TP / 8; ++jc) {
                uint32_t pk[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int j = jc * 8 + 2 * i;
                    const float m0 = misc->fm[j].y, m1 = misc->fm[j + 1].y;
                    const float x0 = __fadd_rn(__fadd_rn(s[j] * k255, m0), -m0);
                    const float x1 = __fadd_rn(__fadd_rn(s[j + 1] * k255, m1), -m1);
                    __half2 hv = __floats2half2_rn(x0, x1);
                    pk[i] = *reinterpret_cast<uint32_t*>(&hv);
                }
                *reinterpret_cast<uint4*>(smem + C::OFF_P + (jc / 8) * C::A_BLOCK + ptx::sw128_offset(tid, jc % 8)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            ptx::fence_proxy_async_smem();
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&misc->bar_p);

            // ---- O = acc / 255 -> fp16 ----
            alive = __all_sync(0xffffffffu, ptx::mbar_wait(&misc->bar_o, ph) && !misc->abort_flag);
            if (!alive) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; break; }
            ptx::tc_fence_after_sync();
            __half* orow = a.o + grow * Cch + h * D;
#pragma unroll
            for (int c = 0; c < DP; c += 16) {
                uint32_t v[16];
                ptx::tmem_ld16(tmem_o + lane_addr + c, v);
                ptx::tmem_ld_wait(v);
#pragma unroll
                for (int half8 = 0; half8 < 2; ++half8) {
                    if (c + half8 * 8 < D && valid) {
                        uint32_t pk[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            __half2 hv = __floats2half2_rn(__uint_as_float(v[half8 * 8 + 2 * i]) * (1.0f / 255.0f), __uint_as_float(v[half8 * 8 + 2 * i + 1]) * (1.0f / 255.0f));
                            pk[i] = *reinterpret_cast<uint32_t*>(&hv);
                        }
                        *reinterpret_cast<uint4*>(orow + c + half8 * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
            }
            ptx::tc_fence_before_sync();
        }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

int pick_heads_per_cta(const AttnArgs& a, int n_z) {
    const long long tiles = (long long)((a.n_query + ROWS - 1) / ROWS) * n_z;
    int best = 1;
    for (int hg = a.heads; hg >= 1; --hg) {
        if (a.heads % hg) continue;
        if (tiles * (a.heads / hg) >= 2 * 148 || hg == 1) { best = hg; break; }
    }
    return best;
}

template <int D>
cudaError_t launch_d(const AttnArgs& a, int n_z, cudaStream_t stream) {
    using C = Cfg<D>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(attention_sm100_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::TOTAL);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int hg = pick_heads_per_cta(a, n_z);
    dim3 grid((a.n_query + ROWS - 1) / ROWS, a.heads / hg, n_z);
    attention_sm100_kernel<D><<<grid, ATT_THREADS, C::TOTAL, stream>>>(a, hg);
    return cudaGetLastError();
}

}  // namespace

bool sm100_attention_supported(const AttnArgs& a) {
    const int d = a.channels / a.heads;
    if (d != 40 && d != 64 && d != 80 && d != 160) return false;
    if (a.n_ctx > TP) return false;
    if (a.p_bits != 8) return false;
    if (a.heads > 65535) return false;
    return true;
}

cudaError_t launch_attention_sm100(const AttnArgs& a, int n_z, cudaStream_t stream) {
    if (a.n_query == 0 || n_z == 0) return cudaSuccess;
    switch (a.channels / a.heads) {
        case 40: return launch_d<40>(a, n_z, stream);
        case 64: return launch_d<64>(a, n_z, stream);
        case 80: return launch_d<80>(a, n_z, stream);
        case 160: return launch_d<160>(a, n_z, stream);
    }
    return cudaErrorNotSupported;
}

}  // namespace taq
