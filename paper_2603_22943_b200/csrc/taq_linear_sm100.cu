// Dequant-GEMM on the Blackwell tensor cores: y = x W^T with W^ = fp16(code * scale), fp32 accumulation in TMEM.
//
// One CTA computes a 128-row x BN-column tile.  The packed codes of its BN output channels (a contiguous slice of
// the blob), their scales and biases are fetched once with three bulk copies; K is then walked in blocks of 64
// through a ring of shared-memory stages.  Roles:
//   warp 0       one thread issues the bulk copies and the TMA loads of the fp16 activation tile (128 x 64,
//                128-byte swizzle);
//   warp 1       owns the TMEM allocation; one thread issues tcgen05.mma (M=128, N=BN, K=16) and commits;
//   warps 2..5   expand the 4/8-bit codes from shared memory into the fp16 weight tile (BN x 64, same swizzled
//                K-major layout); afterwards they are the epilogue: each thread owns one accumulator row (TMEM
//                lane) and applies bias / fp16 conversion, or the per-(row, head) int8 quantization Q_a of Eq. 2,
//                or the mixed int8 / fp16 K~,V~ store of Eq. 2.
// The packed weights stay packed in HBM and are read once per CTA.
#include "taq_ptx.cuh"
#include "taq_sm100.cuh"

namespace taq {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int MAX_STAGE = 6;
constexpr int NTHREADS = 192;
constexpr int A_TILE_BYTES = BM * BK * 2;   // 16 KB
constexpr int SMEM_LIMIT = 227 * 1024;

template <int BN>
struct Tile {
    static constexpr int B_TILE_BYTES = ((BN * BK * 2 + 1023) / 1024) * 1024;
    static constexpr int STAGE_BYTES = A_TILE_BYTES + B_TILE_BYTES;
    static constexpr uint32_t TMEM_COLS = BN <= 32 ? 32 : BN <= 64 ? 64 : BN <= 128 ? 128 : 256;
};

struct Bars {
    uint64_t full_a[MAX_STAGE];
    uint64_t full_b[MAX_STAGE];
    uint64_t empty[MAX_STAGE];
    uint64_t w_full;
    uint64_t acc_full;
    uint32_t tmem_base;
    volatile int abort_flag;
};

// Shared-memory plan of one launch (host and device agree through these numbers).
struct Plan {
    int nstage;
    int raw_bytes, scale_bytes, bias_bytes;   // BN rows of codes / scales / bias
    int off_raw, off_scales, off_bias, off_bars, total;
};

template <int BN>
__host__ __device__ inline Plan make_plan(int k_in, int bits, int group, int nstage) {
    const WeightLayout L = weight_layout(BN, k_in, bits, group);
    Plan p;
    p.nstage = nstage;
    p.raw_bytes = (int)(L.row_bytes * BN);
    p.scale_bytes = BN * L.n_groups * 4;
    p.bias_bytes = BN * 4;
    p.off_raw = nstage * Tile<BN>::STAGE_BYTES;
    p.off_scales = p.off_raw + (p.raw_bytes + 127) / 128 * 128;
    p.off_bias = p.off_scales + (p.scale_bytes + 127) / 128 * 128;
    p.off_bars = p.off_bias + (p.bias_bytes + 127) / 128 * 128;
    p.total = p.off_bars + 256 + 1024;        // barriers + slack to align the base to 1024
    return p;
}

// Eight consecutive weights of one output channel -> eight fp16 operands fp16(float(code) * s).
// 0x4B000000 | n read as a float is 2^23 + n, so the integer-to-float conversion is a subtraction.
__device__ __forceinline__ uint4 pack8(const float (&w)[8]) {
    uint4 out;
    __half2 h;
    h = __floats2half2_rn(w[0], w[1]); out.x = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2half2_rn(w[2], w[3]); out.y = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2half2_rn(w[4], w[5]); out.z = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2half2_rn(w[6], w[7]); out.w = *reinterpret_cast<uint32_t*>(&h);
    return out;
}
__device__ __forceinline__ uint4 dequant8_w4(uint32_t p, float s) {
    const uint32_t lo = p & 0x0F0F0F0Fu, hi = (p >> 4) & 0x0F0F0F0Fu;    // nibbles 0,2,4,6 and 1,3,5,7
    float w[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t a = __byte_perm(lo, 0x4B000000u, 0x7440 + i);     // bytes {lo.b_i, 0, 0, 0x4B}
        const uint32_t b = __byte_perm(hi, 0x4B000000u, 0x7440 + i);
        w[2 * i] = __fmul_rn(__uint_as_float(a) - 8388616.0f, s);        // (2^23 + n) - (2^23 + 8) = code
        w[2 * i + 1] = __fmul_rn(__uint_as_float(b) - 8388616.0f, s);
    }
    return pack8(w);
}
__device__ __forceinline__ uint4 dequant8_w8(uint2 p, float s) {
    const uint32_t x0 = p.x ^ 0x80808080u, x1 = p.y ^ 0x80808080u;       // code + 128 in every byte
    float w[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t a = __byte_perm(x0, 0x4B000000u, 0x7440 + i);
        const uint32_t b = __byte_perm(x1, 0x4B000000u, 0x7440 + i);
        w[i] = __fmul_rn(__uint_as_float(a) - 8388736.0f, s);            // (2^23 + code + 128) - (2^23 + 128)
        w[4 + i] = __fmul_rn(__uint_as_float(b) - 8388736.0f, s);
    }
    return pack8(w);
}

// Loads `n8` groups of 8 accumulator columns of this thread's row (all loads issued before the one wait).
template <int N8>
__device__ __forceinline__ void tmem_row_load(uint32_t taddr, uint32_t (&v)[N8][8], int n8) {
#pragma unroll
    for (int i = 0; i < N8; ++i)
        if (i < n8) ptx::tmem_ld8(taddr + i * 8, v[i]);
    ptx::tmem_ld_wait(v[0]);
#pragma unroll
    for (int i = 1; i < N8; ++i) ptx::reg_fence8(v[i]);
}

template <int BN>
__global__ void __launch_bounds__(NTHREADS) linear_sm100_kernel(const __grid_constant__ CUtensorMap tmap_x, const LinearArgs a, const int nstage) {
    using TL = Tile<BN>;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    const Plan P = make_plan<BN>(a.k_in, a.bits, a.group, nstage);
    Bars* bars = reinterpret_cast<Bars*>(smem + P.off_bars);
    constexpr uint32_t TMEM_COLS = TL::TMEM_COLS;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int z = blockIdx.z;
    const int row0 = blockIdx.x * BM;
    const int col0 = blockIdx.y * BN;
    const int n_kb = a.k_in / BK;
    const uint8_t* blob = (const uint8_t*)(a.reqs ? (a.which == 0 ? a.reqs[z].Wq : a.reqs[z].Wout) : a.w);
    const WeightLayout L = weight_layout(a.n_out, a.k_in, a.bits, a.group);

    if (tid == 0) {
        for (int s = 0; s < MAX_STAGE; ++s) {
            ptx::mbar_init(&bars->full_a[s], 1);
            ptx::mbar_init(&bars->full_b[s], 128);
            ptx::mbar_init(&bars->empty[s], 1);
        }
        ptx::mbar_init(&bars->w_full, 1);
        ptx::mbar_init(&bars->acc_full, 1);
        bars->abort_flag = 0;
        ptx::mbar_fence_init();
        ptx::tma_prefetch_desc(&tmap_x);
    }
    if (warp == 1) ptx::tmem_alloc(&bars->tmem_base, TMEM_COLS);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        // ---------------- producer: packed weights once, then activation tiles ----------------
        if (lane == 0) {
            ptx::mbar_arrive_expect_tx(&bars->w_full, (uint32_t)(P.raw_bytes + P.scale_bytes + P.bias_bytes));
            ptx::bulk_load(smem + P.off_raw, blob + L.off_codes + (size_t)col0 * L.row_bytes, (uint32_t)P.raw_bytes, &bars->w_full);
            ptx::bulk_load(smem + P.off_scales, blob + L.off_scales + (size_t)col0 * L.n_groups * 4, (uint32_t)P.scale_bytes, &bars->w_full);
            ptx::bulk_load(smem + P.off_bias, blob + L.off_bias + (size_t)col0 * 4, (uint32_t)P.bias_bytes, &bars->w_full);
            int issued = 0;
            for (int kb = 0; kb < n_kb; ++kb) {
                const int s = kb % nstage;
                if (kb >= nstage && !ptx::mbar_wait(&bars->empty[s], ((kb / nstage) & 1) ^ 1)) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
                if (bars->abort_flag) break;
                ptx::mbar_arrive_expect_tx(&bars->full_a[s], A_TILE_BYTES);
                ptx::tma_load_3d(smem + s * TL::STAGE_BYTES, &tmap_x, &bars->full_a[s], kb * BK, row0, z);
                issued = kb + 1;
            }
            if (bars->abort_flag) {   // give copies that are still in flight a bounded chance to land before the CTA exits
                (void)ptx::mbar_wait(&bars->w_full, 0);
                for (int kb = issued > nstage ? issued - nstage : 0; kb < issued; ++kb) (void)ptx::mbar_wait(&bars->full_a[kb % nstage], (kb / nstage) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_f16_m128(BN);
            for (int kb = 0; kb < n_kb; ++kb) {
                const int s = kb % nstage;
                const uint32_t ph = (kb / nstage) & 1;
                if (!ptx::mbar_wait(&bars->full_a[s], ph) || !ptx::mbar_wait(&bars->full_b[s], ph)) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
                if (bars->abort_flag) break;
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = ptx::smem_u32(smem + s * TL::STAGE_BYTES);
                const uint32_t b_addr = a_addr + A_TILE_BYTES;
#pragma unroll
                for (int k = 0; k < BK / 16; ++k) {
                    ptx::mma_f16_ss(tmem_base, ptx::desc_k_sw128(a_addr + k * 32), ptx::desc_k_sw128(b_addr + k * 32), idesc, (kb | k) != 0);
                }
                ptx::mma_commit(&bars->empty[s]);       // frees the stage once these MMAs have read it
            }
            ptx::mma_commit(&bars->acc_full);            // accumulator complete (arrives even after an abort)
        }
    } else {
        // ---------------- weight expansion (warps 2..5) ----------------
        const int wt = tid - 64;                          // 0..127
        const unsigned char* raw = smem + P.off_raw;
        const float* wscales = reinterpret_cast<const float*>(smem + P.off_scales);
        const float* bias = reinterpret_cast<const float*>(smem + P.off_bias);
        const int row_bytes = (int)L.row_bytes, n_groups = L.n_groups;
        bool ok = ptx::mbar_wait(&bars->w_full, 0);
        if (!ok) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
        for (int kb = 0; kb < n_kb && ok; ++kb) {
            const int s = kb % nstage;
            if (kb >= nstage && !ptx::mbar_wait(&bars->empty[s], ((kb / nstage) & 1) ^ 1)) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
            if (bars->abort_flag) { ok = false; break; }
            unsigned char* b_tile = smem + s * TL::STAGE_BYTES + A_TILE_BYTES;
            const int g = (kb * BK) / L.group_len;
#pragma unroll
            for (int i = 0; i < (BN * 8 + 127) / 128; ++i) {   // 16-byte chunks: 8 per weight row
                const int idx = wt + i * 128;
                if ((BN * 8) % 128 == 0 || idx < BN * 8) {
                    const int n = idx >> 3, c = idx & 7;
                    const float sc = wscales[n * n_groups + g];
                    uint4 v;
                    if (a.bits == 4) v = dequant8_w4(*reinterpret_cast<const uint32_t*>(raw + n * row_bytes + ((kb * BK + c * 8) >> 1)), sc);
                    else v = dequant8_w8(*reinterpret_cast<const uint2*>(raw + n * row_bytes + kb * BK + c * 8), sc);
                    *reinterpret_cast<uint4*>(b_tile + ptx::sw128_offset(n, c)) = v;
                }
            }
            ptx::fence_proxy_async_smem();                // make the generic-proxy writes visible to the tensor core
            ptx::mbar_arrive(&bars->full_b[s]);
        }

        // ---------------- epilogue: one accumulator row per thread ----------------
        const bool done = ptx::mbar_wait(&bars->acc_full, 0);
        if (!done) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
        ptx::tc_fence_after_sync();
        if (done && !bars->abort_flag) {
            const int q = warp & 3;                       // TMEM lane quarter this warp may read
            const int r = q * 32 + lane;
            const long long row = (long long)row0 + r;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
            if (a.epi == EPI_F16 || a.epi == EPI_F32) {
#pragma unroll 1
                for (int c0 = 0; c0 < BN; c0 += 32) {
                    uint32_t v[4][8];
                    const int n8 = (BN - c0) >= 32 ? 4 : (BN - c0) / 8;
                    tmem_row_load<4>(taddr + c0, v, n8);
                    if (row < a.rows) {
                        const size_t o = ((size_t)z * a.rows + row) * a.n_out + col0 + c0;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            if (i < n8) {
                                float f[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) f[e] = __uint_as_float(v[i][e]) + bias[c0 + i * 8 + e];
                                if (a.epi == EPI_F16) {
                                    *reinterpret_cast<uint4*>((__half*)a.y + o + i * 8) = pack8(f);
                                } else {
                                    float4* dst = reinterpret_cast<float4*>((float*)a.y + o + i * 8);
                                    dst[0] = make_float4(f[0], f[1], f[2], f[3]);
                                    dst[1] = make_float4(f[4], f[5], f[6], f[7]);
                                }
                            }
                        }
                    }
                }
            } else if (a.epi == EPI_Q8_HEAD) {
                // Q~ = Q_a(Q): per (row, head) absmax, then codes = rint(x * (1/s)) by one fma whose low byte is the
                // two's-complement code (1.5 * 2^23 + code).  Two passes over TMEM, 40 columns at a time.
                const int d = a.n_out / a.heads;
                const int heads_here = BN / d;
#pragma unroll 1
                for (int hh = 0; hh < heads_here; ++hh) {
                    const int h = col0 / d + hh;
                    float amax = 0.f;
#pragma unroll 1
                    for (int c0 = 0; c0 < d; c0 += 40) {
                        uint32_t v[5][8];
                        const int n8 = (d - c0) >= 40 ? 5 : (d - c0) / 8;
                        tmem_row_load<5>(taddr + hh * d + c0, v, n8);
#pragma unroll
                        for (int i = 0; i < 5; ++i)
                            if (i < n8) {
#pragma unroll
                                for (int e = 0; e < 8; ++e) amax = fmaxf(amax, fabsf(__uint_as_float(v[i][e])));
                            }
                    }
                    const float s = quant_scale(amax, 127.f);
                    const float rs = s > 0.f ? __frcp_rn(s) : 0.f;
#pragma unroll 1
                    for (int c0 = 0; c0 < d; c0 += 40) {
                        uint32_t v[5][8];
                        const int n8 = (d - c0) >= 40 ? 5 : (d - c0) / 8;
                        tmem_row_load<5>(taddr + hh * d + c0, v, n8);
                        if (row < a.rows) {
                            int8_t* dst = (int8_t*)a.y + ((size_t)z * a.rows + row) * a.n_out + h * d + c0;
#pragma unroll
                            for (int i = 0; i < 5; ++i)
                                if (i < n8) {
                                    uint32_t x[8];
#pragma unroll
                                    for (int e = 0; e < 8; ++e) x[e] = __float_as_uint(fmaf(__uint_as_float(v[i][e]), rs, 12582912.0f));
                                    const uint32_t lo = __byte_perm(__byte_perm(x[0], x[1], 0x0040), __byte_perm(x[2], x[3], 0x0040), 0x5410);
                                    const uint32_t hi = __byte_perm(__byte_perm(x[4], x[5], 0x0040), __byte_perm(x[6], x[7], 0x0040), 0x5410);
                                    *reinterpret_cast<uint2*>(dst + i * 8) = make_uint2(lo, hi);
                                }
                        }
                    }
                    if (row < a.rows) a.scales[((size_t)z * a.rows + row) * a.heads + h] = s;
                }
            } else {
                // Eq. 2 for K or V: rows of ordinary tokens -> int8 codes + scale, rows of trigger tokens -> fp16
                const int d = a.n_out / a.heads;
                const int heads_here = BN / d;
                int b = 0, t = 0, slot = -1;
                bool trig = false;
                uint8_t* blk = nullptr;
                taq_kv_layout KL;
                if (row < a.rows) {
                    b = a.reqs ? 0 : (int)(row / a.n_ctx);
                    t = (int)(row % a.n_ctx);
                    const uint8_t* mask = a.reqs ? a.reqs[z].trig_mask : a.mask + (size_t)b * a.n_ctx;
                    KL = kv_layout(a.heads, a.n_ctx, d, a.max_trigger);
                    blk = a.reqs ? (uint8_t*)a.reqs[z].kv : (uint8_t*)a.y + (size_t)b * KL.block_bytes;
                    trig = mask[t] != 0;
                    if (trig) {
                        slot = 0;
                        for (int u = 0; u < t; ++u) slot += mask[u] != 0;
                        if (slot >= a.max_trigger) { raise_status(a.status, TAQ_ERR_SHAPE); slot = -2; }
                    }
                }
#pragma unroll 1
                for (int hh = 0; hh < heads_here; ++hh) {
                    const int h = col0 / d + hh;
                    float amax = 0.f;
#pragma unroll 1
                    for (int c = 0; c < d; c += 8) {
                        uint32_t v[8];
                        ptx::tmem_ld8(taddr + hh * d + c, v);
                        ptx::tmem_ld_wait(v);
#pragma unroll
                        for (int i = 0; i < 8; ++i) amax = fmaxf(amax, fabsf(__uint_as_float(v[i])));
                    }
                    const float s = quant_scale(amax, 127.f);
#pragma unroll 1
                    for (int c = 0; c < d; c += 8) {
                        uint32_t v[8];
                        ptx::tmem_ld8(taddr + hh * d + c, v);
                        ptx::tmem_ld_wait(v);
                        if (row < a.rows) {
                            uint32_t lo = 0, hi = 0;
                            if (!trig) {
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    lo |= (uint32_t)(quant_code(__uint_as_float(v[i]), s, 127) & 0xFF) << (8 * i);
                                    hi |= (uint32_t)(quant_code(__uint_as_float(v[4 + i]), s, 127) & 0xFF) << (8 * i);
                                }
                            }
                            int8_t* cq = (int8_t*)(blk + (a.kv_which ? KL.off_v_codes : KL.off_k_codes)) + ((size_t)h * a.n_ctx + t) * d + c;
                            *reinterpret_cast<uint2*>(cq) = make_uint2(lo, hi);
                            if (slot >= 0) {
                                __half* tr = (__half*)(blk + (a.kv_which ? KL.off_v_trigger : KL.off_k_trigger)) + ((size_t)slot * a.heads + h) * d + c;
                                float f[8];
#pragma unroll
                                for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[i]);
                                *reinterpret_cast<uint4*>(tr) = pack8(f);
                            }
                        }
                    }
                    if (row < a.rows) {
                        ((float*)(blk + (a.kv_which ? KL.off_v_scales : KL.off_k_scales)))[(size_t)h * a.n_ctx + t] = trig ? 0.f : s;
                        if (h == 0 && a.kv_which == 0) ((int32_t*)(blk + KL.off_trig_slot))[t] = slot >= 0 ? slot : -1;
                    }
                }
                if (a.kv_which == 0 && blockIdx.x == 0 && blockIdx.y == 0) {   // slot table beyond T
                    const int nb = a.reqs ? 1 : (int)(a.rows / a.n_ctx);
                    const taq_kv_layout K2 = kv_layout(a.heads, a.n_ctx, d, a.max_trigger);
                    for (int i = wt; i < nb * (kMaxCtx - a.n_ctx); i += 128) {
                        const int bb = i / (kMaxCtx - a.n_ctx), tt = a.n_ctx + i % (kMaxCtx - a.n_ctx);
                        uint8_t* bk = a.reqs ? (uint8_t*)a.reqs[z].kv : (uint8_t*)a.y + (size_t)bb * K2.block_bytes;
                        ((int32_t*)(bk + K2.off_trig_slot))[tt] = -1;
                    }
                }
            }
        }
    }

    // ---------------- teardown ----------------
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// ---- host side -------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

int pick_bn(const LinearArgs& a) {
    if (a.epi == EPI_Q8_HEAD || a.epi == EPI_KV) {
        const int d = a.n_out / a.heads;
        if (d == 40 && a.heads % 2 == 0) return 80;
        if (d == 64 || d == 80 || d == 160) return d;
        return 0;
    }
    if (a.n_out % 160 == 0 && a.rows * (a.n_out / 160) >= 148LL * 128) return 160;
    if (a.n_out % 80 == 0) return 80;
    if (a.n_out % 64 == 0) return 64;
    return 0;
}

// Ring depth: as deep as the K loop needs, but no deeper than three stages when that keeps two CTAs on an SM.
template <int BN>
int pick_nstage(const LinearArgs& a) {
    const int n_kb = a.k_in / BK;
    int best = 0;
    for (int ns = 1; ns <= MAX_STAGE && ns <= (n_kb < 2 ? 2 : n_kb); ++ns) {
        const int total = make_plan<BN>(a.k_in, a.bits, a.group, ns).total;
        if (total > SMEM_LIMIT) break;
        if (ns > 3 && total + 1024 > SMEM_LIMIT / 2 && make_plan<BN>(a.k_in, a.bits, a.group, 3).total + 1024 <= SMEM_LIMIT / 2) break;
        best = ns;
    }
    return best;
}

int nstage_for(const LinearArgs& a, int bn) {
    switch (bn) {
        case 64: return pick_nstage<64>(a);
        case 80: return pick_nstage<80>(a);
        case 160: return pick_nstage<160>(a);
    }
    return 0;
}

template <int BN>
cudaError_t launch_bn(const CUtensorMap& tmap, const LinearArgs& a, int n_z, cudaStream_t stream) {
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(linear_sm100_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int ns = pick_nstage<BN>(a);
    const Plan P = make_plan<BN>(a.k_in, a.bits, a.group, ns);
    dim3 grid((unsigned)((a.rows + BM - 1) / BM), a.n_out / BN, n_z);
    linear_sm100_kernel<BN><<<grid, NTHREADS, P.total, stream>>>(tmap, a, ns);
    return cudaGetLastError();
}

}  // namespace

bool sm100_linear_supported(const LinearArgs& a) {
    if (a.k_in % BK) return false;
    if (a.group != 0 && a.group % BK) return false;
    if (a.rows < 1 || a.rows > (1LL << 31) - 1) return false;
    if (reinterpret_cast<uintptr_t>(a.x) & 15u) return false;
    const int bn = pick_bn(a);
    if (bn == 0) return false;
    if (nstage_for(a, bn) < 2) return false;
    return encode_tiled_fn() != nullptr;
}

cudaError_t launch_linear_sm100(const LinearArgs& a, int n_z, cudaStream_t stream) {
    if (a.rows == 0 || n_z == 0) return cudaSuccess;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return cudaErrorNotSupported;
    CUtensorMap tmap;
    const cuuint64_t dims[3] = {(cuuint64_t)a.k_in, (cuuint64_t)a.rows, (cuuint64_t)n_z};
    const cuuint64_t strides[2] = {(cuuint64_t)a.k_in * 2, (cuuint64_t)a.k_in * 2 * (cuuint64_t)a.rows};
    const cuuint32_t box[3] = {BK, BM, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<__half*>(a.x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    switch (pick_bn(a)) {
        case 64: return launch_bn<64>(tmap, a, n_z, stream);
        case 80: return launch_bn<80>(tmap, a, n_z, stream);
        case 160: return launch_bn<160>(tmap, a, n_z, stream);
    }
    return cudaErrorNotSupported;
}

}  // namespace taq
