// Dequant-GEMM on the Blackwell tensor cores: y = x W^T with W^ = fp16(code * scale), fp32 accumulation in TMEM.
//
// One CTA computes a 128-row x BN-column tile.  K is walked in blocks of 64 through a ring of shared-memory
// stages.  Three roles:
//   warp 0       one thread issues TMA loads of the fp16 activation tile (128 x 64, 128-byte swizzle);
//   warp 1       owns the TMEM allocation; one thread issues tcgen05.mma (M=128, N=BN, K=16) and commits;
//   warps 2..5   read the packed 4/8-bit codes with plain loads, dequantize them and write the fp16 weight tile
//                (BN x 64) into the same swizzled K-major layout; afterwards they are the epilogue: each thread
//                owns one accumulator row (TMEM lane) and applies bias / fp16 conversion, or the per-(row, head)
//                int8 quantization Q_a of Eq. 2, or the mixed int8 / fp16 K~,V~ store of Eq. 2.
// The packed weights are read once per CTA from L2; they stay packed in HBM.
#include "taq_ptx.cuh"
#include "taq_sm100.cuh"

namespace taq {

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int NSTAGE = 4;
constexpr int NTHREADS = 192;
constexpr int A_TILE_BYTES = BM * BK * 2;   // 16 KB

template <int BN>
struct SmemLayout {
    static constexpr int B_TILE_BYTES = BN * BK * 2;
    static constexpr int STAGE_BYTES = A_TILE_BYTES + ((B_TILE_BYTES + 1023) / 1024) * 1024;
    static constexpr int BAR_OFFSET = NSTAGE * STAGE_BYTES;
    static constexpr int TOTAL = BAR_OFFSET + 256 + 1024;   // barriers + slack to align the base to 1024
};

constexpr uint32_t tmem_cols_for(int bn) { return bn <= 32 ? 32 : bn <= 64 ? 64 : bn <= 128 ? 128 : 256; }

struct Bars {
    uint64_t full_a[NSTAGE];
    uint64_t full_b[NSTAGE];
    uint64_t empty[NSTAGE];
    uint64_t acc_full;
    uint32_t tmem_base;
    volatile int abort_flag;
};

// Eight consecutive weights of output channel n starting at fan-in index k (a multiple of 8) -> eight fp16
// operands, packed as 4 x half2.
__device__ __forceinline__ uint4 dequant8(const uint8_t* codes, size_t row_bytes, int bits, int n, int k, float s) {
    float w[8];
    if (bits == 4) {
        const uint32_t p = *reinterpret_cast<const uint32_t*>(codes + (size_t)n * row_bytes + (k >> 1));
#pragma unroll
        for (int i = 0; i < 8; ++i) w[i] = __fmul_rn((float)((int)((p >> (4 * i)) & 0xF) - 8), s);
    } else {
        const uint2 p = *reinterpret_cast<const uint2*>(codes + (size_t)n * row_bytes + k);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            w[i] = __fmul_rn((float)(int8_t)((p.x >> (8 * i)) & 0xFF), s);
            w[4 + i] = __fmul_rn((float)(int8_t)((p.y >> (8 * i)) & 0xFF), s);
        }
    }
    uint4 out;
    __half2 h;
    h = __floats2half2_rn(w[0], w[1]); out.x = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2half2_rn(w[2], w[3]); out.y = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2half2_rn(w[4], w[5]); out.z = *reinterpret_cast<uint32_t*>(&h);
    h = __floats2half2_rn(w[6], w[7]); out.w = *reinterpret_cast<uint32_t*>(&h);
    return out;
}

template <int BN>
__global__ void __launch_bounds__(NTHREADS) linear_sm100_kernel(const __grid_constant__ CUtensorMap tmap_x, const LinearArgs a) {
    using SL = SmemLayout<BN>;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    Bars* bars = reinterpret_cast<Bars*>(smem + SL::BAR_OFFSET);
    constexpr uint32_t TMEM_COLS = tmem_cols_for(BN);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int z = blockIdx.z;
    const int row0 = blockIdx.x * BM;
    const int col0 = blockIdx.y * BN;
    const int n_kb = a.k_in / BK;

    if (tid == 0) {
        for (int s = 0; s < NSTAGE; ++s) {
            ptx::mbar_init(&bars->full_a[s], 1);
            ptx::mbar_init(&bars->full_b[s], 128);
            ptx::mbar_init(&bars->empty[s], 1);
        }
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
        // ---------------- TMA producer: activation tiles ----------------
        if (lane == 0) {
            for (int kb = 0; kb < n_kb; ++kb) {
                const int s = kb % NSTAGE;
                if (kb >= NSTAGE && !ptx::mbar_wait(&bars->empty[s], ((kb / NSTAGE) & 1) ^ 1)) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
                if (bars->abort_flag) break;
                ptx::mbar_arrive_expect_tx(&bars->full_a[s], A_TILE_BYTES);
                ptx::tma_load_3d(smem + s * SL::STAGE_BYTES, &tmap_x, &bars->full_a[s], kb * BK, row0, z);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_f16_m128(BN);
            for (int kb = 0; kb < n_kb; ++kb) {
                const int s = kb % NSTAGE;
                const uint32_t ph = (kb / NSTAGE) & 1;
                if (!ptx::mbar_wait(&bars->full_a[s], ph) || !ptx::mbar_wait(&bars->full_b[s], ph)) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
                if (bars->abort_flag) break;
                ptx::tc_fence_after_sync();
                const uint32_t a_addr = ptx::smem_u32(smem + s * SL::STAGE_BYTES);
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
        // ---------------- weight dequantization (warps 2..5) ----------------
        const int wt = tid - 64;                          // 0..127
        const uint8_t* blob = (const uint8_t*)(a.reqs ? (a.which == 0 ? a.reqs[z].Wq : a.reqs[z].Wout) : a.w);
        const WeightLayout L = weight_layout(a.n_out, a.k_in, a.bits, a.group);
        const uint8_t* codes = blob + L.off_codes;
        const float* wscales = reinterpret_cast<const float*>(blob + L.off_scales);
        bool ok = true;
        for (int kb = 0; kb < n_kb && ok; ++kb) {
            const int s = kb % NSTAGE;
            if (kb >= NSTAGE && !ptx::mbar_wait(&bars->empty[s], ((kb / NSTAGE) & 1) ^ 1)) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
            if (bars->abort_flag) { ok = false; break; }
            unsigned char* b_tile = smem + s * SL::STAGE_BYTES + A_TILE_BYTES;
            const int g = (kb * BK) / L.group_len;
            for (int idx = wt; idx < BN * 8; idx += 128) {   // 16-byte chunks: 8 per weight row
                const int n = idx >> 3, c = idx & 7;
                const float sc = wscales[(size_t)(col0 + n) * L.n_groups + g];
                const uint4 v = dequant8(codes, L.row_bytes, a.bits, col0 + n, kb * BK + c * 8, sc);
                *reinterpret_cast<uint4*>(b_tile + ptx::sw128_offset(n, c)) = v;
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
            const float* bias = reinterpret_cast<const float*>(blob + L.off_bias);
            if (a.epi == EPI_F16 || a.epi == EPI_F32) {
#pragma unroll 1
                for (int c = 0; c < BN; c += 16) {
                    uint32_t v[16];
                    ptx::tmem_ld16(taddr + c, v);
                    ptx::tmem_ld_wait(v);
                    if (row < a.rows) {
                        const size_t o = ((size_t)z * a.rows + row) * a.n_out + col0 + c;
                        if (a.epi == EPI_F16) {
                            uint32_t pk[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                __half2 h = __floats2half2_rn(__uint_as_float(v[2 * i]) + bias[col0 + c + 2 * i], __uint_as_float(v[2 * i + 1]) + bias[col0 + c + 2 * i + 1]);
                                pk[i] = *reinterpret_cast<uint32_t*>(&h);
                            }
                            uint4* dst = reinterpret_cast<uint4*>((__half*)a.y + o);
                            dst[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            dst[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                        } else {
                            float4* dst = reinterpret_cast<float4*>((float*)a.y + o);
#pragma unroll
                            for (int i = 0; i < 4; ++i)
                                dst[i] = make_float4(__uint_as_float(v[4 * i]) + bias[col0 + c + 4 * i], __uint_as_float(v[4 * i + 1]) + bias[col0 + c + 4 * i + 1],
                                                     __uint_as_float(v[4 * i + 2]) + bias[col0 + c + 4 * i + 2], __uint_as_float(v[4 * i + 3]) + bias[col0 + c + 4 * i + 3]);
                        }
                    }
                }
            } else {
                // per-(row, head) symmetric int8: pass 1 absmax, pass 2 codes (TMEM is read twice; it is cheap)
                const int d = a.n_out / a.heads;
                const int heads_here = BN / d;
                int b = 0, t = 0, slot = -1;
                bool trig = false;
                uint8_t* blk = nullptr;
                taq_kv_layout KL;
                if (a.epi == EPI_KV && row < a.rows) {
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
                        if (!(a.epi == EPI_KV && trig)) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                lo |= (uint32_t)(quant_code(__uint_as_float(v[i]), s, 127) & 0xFF) << (8 * i);
                                hi |= (uint32_t)(quant_code(__uint_as_float(v[4 + i]), s, 127) & 0xFF) << (8 * i);
                            }
                        }
                        if (a.epi == EPI_Q8_HEAD) {
                            *reinterpret_cast<uint2*>((int8_t*)a.y + ((size_t)z * a.rows + row) * a.n_out + h * d + c) = make_uint2(lo, hi);
                        } else {
                            int8_t* cq = (int8_t*)(blk + (a.kv_which ? KL.off_v_codes : KL.off_k_codes)) + ((size_t)h * a.n_ctx + t) * d + c;
                            *reinterpret_cast<uint2*>(cq) = make_uint2(lo, hi);
                            if (slot >= 0) {
                                __half* tr = (__half*)(blk + (a.kv_which ? KL.off_v_trigger : KL.off_k_trigger)) + ((size_t)slot * a.heads + h) * d + c;
                                uint32_t pk[4];
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    __half2 hv = __floats2half2_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
                                    pk[i] = *reinterpret_cast<uint32_t*>(&hv);
                                }
                                *reinterpret_cast<uint4*>(tr) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            }
                        }
                        }
                    }
                    if (row < a.rows) {
                        if (a.epi == EPI_Q8_HEAD) a.scales[((size_t)z * a.rows + row) * a.heads + h] = s;
                        else {
                            ((float*)(blk + (a.kv_which ? KL.off_v_scales : KL.off_k_scales)))[(size_t)h * a.n_ctx + t] = trig ? 0.f : s;
                            if (h == 0 && a.kv_which == 0) ((int32_t*)(blk + KL.off_trig_slot))[t] = slot >= 0 ? slot : -1;
                        }
                    }
                }
                if (a.epi == EPI_KV && a.kv_which == 0 && blockIdx.x == 0 && blockIdx.y == 0) {   // slot table beyond T
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
    if (warp == 0 && lane == 0 && bars->abort_flag) {
        // after a failed wait: give copies that are still in flight a bounded chance to land before the CTA exits
        for (int s = 0; s < NSTAGE && s < n_kb; ++s) {
            const int last_kb = ((n_kb - 1 - s) / NSTAGE) * NSTAGE + s;
            (void)ptx::mbar_wait(&bars->full_a[s], (last_kb / NSTAGE) & 1);
        }
    }
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

template <int BN>
cudaError_t launch_bn(const CUtensorMap& tmap, const LinearArgs& a, int n_z, cudaStream_t stream) {
    using SL = SmemLayout<BN>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(linear_sm100_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, SL::TOTAL);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid((unsigned)((a.rows + BM - 1) / BM), a.n_out / BN, n_z);
    linear_sm100_kernel<BN><<<grid, NTHREADS, SL::TOTAL, stream>>>(tmap, a);
    return cudaGetLastError();
}

}  // namespace

bool sm100_linear_supported(const LinearArgs& a) {
    if (a.k_in % BK) return false;
    if (a.group != 0 && a.group % BK) return false;
    if (a.rows < 1 || a.rows > (1LL << 31) - 1) return false;
    if (reinterpret_cast<uintptr_t>(a.x) & 15u) return false;
    if (pick_bn(a) == 0) return false;
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
