// Fused TAQ attention on the Blackwell tensor cores (tcgen05 + TMEM): Q~ in, O out, nothing else touches HBM.
//   S = Q~ K~^T             tcgen05.mma; the fp16 operands hold the int8 codes exactly (trigger rows: fp16 values)
//   A = softmax(S * scale)  one thread per query row; the row's 80 scores live in its registers (TMEM lane)
//   A^ (Eq. 3)              ordinary columns -> uint8 code, trigger columns -> fp16, both in units of 1/255
//   O = A^ V~               tcgen05.mma with the probabilities as the A operand and V~^T (fp16) as B; O = acc/255
// A CTA owns 128 query rows of one sequence and walks over a group of heads, software-pipelined:
//   warps 0-7  two threads per query row (TMEM lane), one per half of the keys: stage the row's Q~ codes of the next
//              head as an fp16 operand tile, softmax + Eq. 3 of the current head (the two threads of a row exchange
//              their partial maximum and sum once per head), epilogue of the previous head;
//   warp 8     one thread issues the MMAs: S of head h+1 is in flight while the rows are in the softmax of head h;
//   warp 9     one thread fetches each head's K~/V~ operand image (written once per prompt by the K/V projection)
//              by bulk copies, one head ahead: the whole image into the second buffer (head widths up to 64), or,
//              with a single buffer, K~ as soon as this head's S is complete and V~^T as soon as its PV is.
// Head widths up to 64: two CTAs share an SM, and the row threads read Q~ and write O themselves.  Head widths 80 and
// 160: one CTA per SM; Q~ tiles arrive and O tiles leave by TMA through a staging buffer.
#include "taq_prof.cuh"
#include "taq_ptx.cuh"
#include "taq_sm100.cuh"
#include "taq_sm100_parts.cuh"
#include <cstring>

namespace taq {

TAQ_PROF_DEFINE(attention)

namespace {

using namespace parts;

constexpr int ROWS = 128;
constexpr int ROW_WARPS = 8;         // two threads per query row
constexpr int MMA_WARP = 8, COPY_WARP = 9;
constexpr int ATT_THREADS = 320;

template <int D>
struct Cfg {
    static constexpr int DP = (D + 15) / 16 * 16;            // head width padded to the MMA K / N granule
    static constexpr int KBQ = (DP + 63) / 64;               // 64-wide k-blocks of the Q~ and K~ tiles
    static constexpr int A_BLOCK = ROWS * 128;
    static constexpr int K_BLOCK = TP * 128;
    static constexpr int VT_BLOCK = DP * 128;
    static constexpr int K_BYTES = KBQ * K_BLOCK;
    static constexpr int VT_BYTES = 2 * VT_BLOCK;
    static constexpr int HEAD_BYTES = K_BYTES + VT_BYTES + kOperandConstBytes;
    static constexpr int KVBUF = D <= 64 ? 2 : 1;            // K~/V~ images in flight
    static constexpr int OBUF = D == 40 ? 2 : 1;             // O accumulators in TMEM
    static constexpr int OFF_KV = 0;
    static constexpr int OFF_Q = OFF_KV + KVBUF * HEAD_BYTES;
    static constexpr int OFF_P = OFF_Q + KBQ * A_BLOCK;
    // One image buffer (wide heads): the next head's K~ loads as soon as this head's S is complete and its V~^T as soon
    // as this head's PV is, each with a barrier of its own; the constants of a head then live in a rotating slot of their
    // own (three slots: the softmax of head h - 1 may still read its slot when the constants of head h + 1 arrive).
    static constexpr bool SPLIT_KV = KVBUF == 1;
    static constexpr int CST_SLOT = 384;
    static constexpr int OFF_CST = OFF_P + 2 * A_BLOCK;
    // Wide heads move Q~ and O by TMA through one staging buffer (a row's codes or outputs of one head are 80 to 320
    // bytes at a stride of the whole channel width: per-thread global accesses of that shape keep the load/store
    // unit busy for longer than the arithmetic takes).  The buffer holds the next head's raw Q~ tile until it has been
    // expanded into the operand tile, then the previous head's O tile until the store has read it; int8 codes get a
    // second, smaller buffer, so that their load never waits for the store.
    static constexpr bool TMA_IO = D >= 80;
    static constexpr int OFF_U = OFF_CST + (SPLIT_KV ? 3 * CST_SLOT : 0);
    static constexpr int UO_BYTES = ROWS * D * 2;                  // an O tile, or a raw fp16 Q tile
    static constexpr int U_BYTES = TMA_IO ? UO_BYTES + ROWS * D : 0; // + a raw int8 Q~ tile, which then has a buffer of its own
    static constexpr int OFF_MISC = OFF_U + U_BYTES;
    static constexpr int TOTAL = OFF_MISC + 4096 + 128 + 1024;   // misc block + slack for 1024-byte alignment
    static constexpr uint32_t TMEM_S = 0, TMEM_O = 2 * TP;
    static constexpr uint32_t TMEM_COLS = (2 * TP + OBUF * DP) <= 256 ? 256 : 512;
    static constexpr int CTAS_PER_SM = (2 * (TOTAL + 1024) <= 232448 && TMEM_COLS == 256) ? 2 : 1;
    static_assert(HEAD_BYTES % 1024 == 0 && K_BYTES % 1024 == 0 && VT_BLOCK % 1024 == 0, "operand tiles must keep 1024-byte alignment");
    static_assert(TOTAL <= 232448, "shared memory budget");
};

struct Misc {
    uint64_t kv_full[2], kv_free[2], q_full, s_full[2], p_full, o_full[2], drain, qraw_full;
    uint32_t tmem_base;
    volatile int abort_flag;
    float2 xchg[2][2][ROWS];     // [head parity][half][row]: (max, sum) of a thread's half of the softmax
};
static_assert(sizeof(Misc) <= 4096 + 128, "misc block");
static_assert(sizeof(OperandConsts) % 16 == 0 && sizeof(OperandConsts) <= 384, "constants slot");

// Half of the query codes (or fp16 values) of one row and head, held in registers between the global load and
// the store into the operand tile: the row's two threads take the lower and the upper half of the 16-byte chunks.
template <int D, bool Q8>
struct QRegs {
    static constexpr int CH2 = (Cfg<D>::DP / 8 + 1) / 2;      // chunks (8 channels) per thread
    uint4 v[Q8 ? (CH2 + 1) / 2 : CH2];
    __device__ __forceinline__ void load(const void* q, size_t elem_off, bool valid, int half) {
        const int c0 = half * CH2;
        if (Q8) {
#pragma unroll
            for (int i = 0; i < (CH2 + 1) / 2; ++i) {
                uint2 lo = make_uint2(0, 0), hi = make_uint2(0, 0);
                if (valid && (c0 + 2 * i) * 8 < D) lo = *reinterpret_cast<const uint2*>((const int8_t*)q + elem_off + (c0 + 2 * i) * 8);
                if (valid && 2 * i + 1 < CH2 && (c0 + 2 * i + 1) * 8 < D) hi = *reinterpret_cast<const uint2*>((const int8_t*)q + elem_off + (c0 + 2 * i + 1) * 8);
                v[i] = make_uint4(lo.x, lo.y, hi.x, hi.y);
            }
        } else {
#pragma unroll
            for (int i = 0; i < CH2; ++i) {
                v[i] = make_uint4(0, 0, 0, 0);
                if (valid && (c0 + i) * 8 < D) v[i] = *reinterpret_cast<const uint4*>((const __half*)q + elem_off + (c0 + i) * 8);
            }
        }
    }
    // local chunk i (8 channels) as fp16 operands; channels beyond D are zero (a zero int8 code maps to fp16 zero)
    __device__ __forceinline__ uint4 chunk(int i) const {
        if (Q8) {
            const uint4 w = v[i / 2];
            return codes_w8_to_half((i & 1) ? make_uint2(w.z, w.w) : make_uint2(w.x, w.y));
        }
        return v[i];
    }
};

template <int D, bool Q8, bool TAIL_ONLY>
__global__ void __launch_bounds__(ATT_THREADS, Cfg<D>::CTAS_PER_SM) attention_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_o, const AttnArgs a, const int heads_per_cta) {
    using C = Cfg<D>;
    constexpr int DP = C::DP;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_u32(smem_dyn) & 1023u)) & 1023u);   // 1024-byte aligned, still provably shared
    Misc* misc = reinterpret_cast<Misc*>(smem + C::OFF_MISC);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = a.n_ctx, H = a.heads, Cch = a.channels;
    const int zb = blockIdx.z;
    const int b = a.reqs ? 0 : zb;
    const int row0 = blockIdx.x * ROWS;
    const int h_begin = blockIdx.y * heads_per_cta;
    const int HG = heads_per_cta;

    TAQ_PROF_INIT
    if (tid == 0) { TAQ_PROF(0); TAQ_GPROF(126); }
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(&misc->kv_full[i], 1);
            ptx::mbar_init(&misc->kv_free[i], 1);
            ptx::mbar_init(&misc->s_full[i], 1);
            ptx::mbar_init(&misc->o_full[i], 1);
        }
        ptx::mbar_init(&misc->q_full, ROW_WARPS);      // one arrival per row warp
        ptx::mbar_init(&misc->p_full, ROW_WARPS);
        ptx::mbar_init(&misc->drain, 1);
        ptx::mbar_init(&misc->qraw_full, 1);
        misc->abort_flag = 0;
        ptx::mbar_fence_init();
    }
    if (warp == MMA_WARP) ptx::tmem_alloc(&misc->tmem_base, C::TMEM_COLS);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = misc->tmem_base;
    ptx::pdl_trigger();

    const taq_kv_layout KL = kv_layout(H, T, D, a.max_trigger);

    if (warp == COPY_WARP) {
        // ---------------- K~/V~ operand images, one head ahead ----------------
        if (lane == 0) {
            if (!a.early_kv) ptx::pdl_wait();             // in general the images may come from the previous kernel
            const uint8_t* blk = a.reqs ? (const uint8_t*)a.reqs[zb].kv : (const uint8_t*)a.kv + (size_t)b * KL.block_bytes;
            const uint8_t* img = blk + KL.off_operands + (size_t)h_begin * KL.operand_head_bytes;
            int issued = 0;
            if (C::SPLIT_KV) {
                // kv_full[0]: K~ and the constants of a head; kv_full[1]: its V~^T
                int issued_v = 0;
                for (int hi = 0; hi < HG; ++hi) {
                    if (hi >= 1 && !ptx::mbar_wait(&misc->s_full[(hi - 1) & 1], ((hi - 1) >> 1) & 1)) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
                    if (misc->abort_flag) break;
                    const uint8_t* src = img + (size_t)hi * KL.operand_head_bytes;
                    ptx::mbar_arrive_expect_tx(&misc->kv_full[0], C::K_BYTES + (uint32_t)sizeof(OperandConsts));
                    ptx::bulk_load(smem + C::OFF_KV, src, C::K_BYTES, &misc->kv_full[0]);
                    ptx::bulk_load(smem + C::OFF_CST + (hi % 3) * C::CST_SLOT, src + C::K_BYTES + C::VT_BYTES, (uint32_t)sizeof(OperandConsts), &misc->kv_full[0]);
                    issued = hi + 1;
                    if (hi >= 1 && !ptx::mbar_wait(&misc->kv_free[0], (hi - 1) & 1)) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
                    if (misc->abort_flag) break;
                    ptx::mbar_arrive_expect_tx(&misc->kv_full[1], C::VT_BYTES);
                    ptx::bulk_load(smem + C::OFF_KV + C::K_BYTES, src + C::K_BYTES, C::VT_BYTES, &misc->kv_full[1]);
                    issued_v = hi + 1;
                }
                if (misc->abort_flag) {   // let copies that were issued land before the CTA goes away
                    if (issued) (void)ptx::mbar_wait(&misc->kv_full[0], (issued - 1) & 1);
                    if (issued_v) (void)ptx::mbar_wait(&misc->kv_full[1], (issued_v - 1) & 1);
                }
            } else {
            for (int hi = 0; hi < HG; ++hi) {
                const int buf = hi % C::KVBUF;
                if (hi >= C::KVBUF && !ptx::mbar_wait(&misc->kv_free[buf], ((hi / C::KVBUF) - 1) & 1)) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
                if (misc->abort_flag) break;
                ptx::mbar_arrive_expect_tx(&misc->kv_full[buf], C::HEAD_BYTES);
                ptx::bulk_load(smem + C::OFF_KV + buf * C::HEAD_BYTES, img + (size_t)hi * KL.operand_head_bytes, C::HEAD_BYTES, &misc->kv_full[buf]);
                issued = hi + 1;
            }
            if (misc->abort_flag) {   // let copies that were issued land before the CTA goes away
                for (int hi = issued > C::KVBUF ? issued - C::KVBUF : 0; hi < issued; ++hi) (void)ptx::mbar_wait(&misc->kv_full[hi % C::KVBUF], (hi / C::KVBUF) & 1);
            }
            }
        }
    } else if (warp == MMA_WARP) {
        // ---------------- MMA issuer ----------------
        // All 32 lanes walk the control flow (warp-uniform loop state and descriptor words); one elected lane issues.
        const bool leader = ptx::elect_one();
        auto wait = [&](uint64_t* bar, uint32_t parity) -> bool { return __all_sync(0xffffffffu, ptx::mbar_wait(bar, parity) && !misc->abort_flag) != 0; };
        constexpr uint32_t HI = ptx::kDescHiSw128;
        const uint32_t q_lo0 = ptx::desc_lo(ptx::smem_u32(smem + C::OFF_Q)), p_lo0 = ptx::desc_lo(ptx::smem_u32(smem + C::OFF_P));
        const uint32_t kv_lo0 = ptx::desc_lo(ptx::smem_u32(smem + C::OFF_KV));
        auto issue_s = [&](int hi) -> bool {
            const int buf = hi % C::KVBUF;
            if (!wait(&misc->kv_full[buf], C::SPLIT_KV ? (hi & 1) : (hi / C::KVBUF) & 1) || !wait(&misc->q_full, hi & 1)) return false;
            ptx::tc_fence_after_sync();
            if (leader) {
                if (hi < 8) TAQ_PROF(80 + hi);
                const uint32_t k_lo = kv_lo0 + buf * (C::HEAD_BYTES >> 4);
#pragma unroll
                for (int ks = 0; ks < DP / 16; ++ks)
                    ptx::mma_f16_ss(tmem_base + C::TMEM_S + (hi & 1) * TP, ptx::desc_join(HI, q_lo0 + (ks / 4) * (C::A_BLOCK >> 4) + (ks % 4) * 2),
                                    ptx::desc_join(HI, k_lo + (ks / 4) * (C::K_BLOCK >> 4) + (ks % 4) * 2), ptx::idesc_f16_m128(TP), ks != 0);
                ptx::mma_commit(&misc->s_full[hi & 1]);
            }
            return true;
        };
        auto issue_pv = [&](int hi) -> bool {
            const int buf = hi % C::KVBUF;
            if (C::SPLIT_KV && !wait(&misc->kv_full[1], hi & 1)) return false;
            if (!wait(&misc->p_full, hi & 1)) return false;
            ptx::tc_fence_after_sync();
            if (leader) {
                if (hi < 8) TAQ_PROF(96 + hi);
                const uint32_t vt_lo = kv_lo0 + ((buf * C::HEAD_BYTES + C::K_BYTES) >> 4);
#pragma unroll
                for (int ks = 0; ks < TP / 16; ++ks)
                    ptx::mma_f16_ss(tmem_base + C::TMEM_O + (hi % C::OBUF) * DP, ptx::desc_join(HI, p_lo0 + (ks / 4) * (C::A_BLOCK >> 4) + (ks % 4) * 2),
                                    ptx::desc_join(HI, vt_lo + (ks / 4) * (C::VT_BLOCK >> 4) + (ks % 4) * 2), ptx::idesc_f16_m128(DP), ks != 0);
                ptx::mma_commit(&misc->o_full[hi % C::OBUF]);
                ptx::mma_commit(&misc->kv_free[buf]);
            }
            return true;
        };
        bool ok = issue_s(0);
        for (int hi = 0; hi < HG && ok; ++hi) {
            if (C::KVBUF == 2) {          // S of the next head first: it runs under this head's softmax
                if (hi + 1 < HG) ok = issue_s(hi + 1);
                if (ok) ok = issue_pv(hi);
            } else {
                // one image buffer: the next head's K~ arrives some time after this head's S; its S goes first if K~
                // and Q~ are there already (it then runs under this head's softmax), else after this head's PV
                const bool early = hi + 1 < HG && __all_sync(0xffffffffu, ptx::mbar_try_wait(&misc->kv_full[0], (hi + 1) & 1) && ptx::mbar_try_wait(&misc->q_full, (hi + 1) & 1)) != 0;
                if (early) ok = issue_s(hi + 1);
                if (ok) ok = issue_pv(hi);
                if (ok && !early && hi + 1 < HG) ok = issue_s(hi + 1);
            }
        }
        if (!ok) {                        // wait (bounded) for whatever was issued before TMEM is given back
            if (leader) {
                raise_status(a.status, TAQ_ERR_TIMEOUT);
                misc->abort_flag = 1;
                ptx::mma_commit(&misc->drain);
            }
            (void)ptx::mbar_wait(&misc->drain, 0);
        }
    } else {
        // ---------------- row threads: two per query row (TMEM lane), each with half of the keys ----------------
        const int q4 = warp & 3, half = warp >> 2;
        const int r = q4 * 32 + lane;
        const int n = row0 + r;
        const bool valid = n < a.n_query;
        const size_t grow = (size_t)zb * a.n_query + (valid ? n : 0);
        const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
        const int key0 = half * HK;
        const float cmax = a.p_bits == 4 ? 15.0f : 255.0f;     // last code
        const float pmax = a.p_log ? 256.0f : cmax;            // probabilities are held in units of 1 / pmax (linear codes: 1 / last code)
        const float inv255 = 1.0f / pmax;
        constexpr int CH2 = QRegs<D, Q8>::CH2;
        constexpr int OC = DP / 2;                       // O columns per thread
        bool alive = true;
        ptx::pdl_wait();                                 // Q~ comes from the previous kernel in the stream
        if (tid == 0) TAQ_PROF(1);

        if constexpr (C::TMA_IO) {
            // ---- Q~ in and O out by TMA through the staging buffer U ----
            // Every warp walks every barrier of the loop, whatever happened to its waits: a warp whose wait ran out
            // skips the work, never a barrier.
            unsigned char* U = smem + C::OFF_U;
            constexpr bool SEPQ = Q8;                        // the raw Q~ tile has its own buffer
            unsigned char* UQ = SEPQ ? U + C::UO_BYTES : U;
            constexpr int QESZ = Q8 ? 1 : 2;
            constexpr uint32_t QRAW_BYTES = (uint32_t)(ROWS * D * QESZ);
            auto all256 = [&]() { asm volatile("bar.sync 5, 256;" ::: "memory"); };
            auto load_q = [&](int hi) {          // one thread: raw Q~ tile of head hi (rows beyond n_query read as zero)
                ptx::mbar_arrive_expect_tx(&misc->qraw_full, QRAW_BYTES);
                ptx::tma_load_3d(UQ, &tmap_q, &misc->qraw_full, (h_begin + hi) * D, row0, zb);
            };
            // raw tile of head hi -> fp16 operand tile.  The 16-byte chunks of the tile are dealt out in linear order (thread t
            // takes chunks t, t + 256, ...): consecutive lanes read consecutive words of the raw tile and write the eight
            // chunk slots of a swizzled operand row, both free of bank conflicts.
            auto stage_q_u = [&](int hi) {
                static_assert(D % 8 == 0 && (ROWS * (D / 8)) % 256 == 0, "chunks per thread");
                constexpr int CPR = D / 8;                   // chunks per row
                alive = alive && __all_sync(0xffffffffu, ptx::mbar_wait(&misc->qraw_full, hi & 1) && !misc->abort_flag);
                if (alive) {
                    uint4 t16[ROWS * CPR / 256];
#pragma unroll
                    for (int i = 0; i < ROWS * CPR / 256; ++i) {
                        const int j = tid + 256 * i;
                        if (Q8) t16[i] = codes_w8_to_half(*reinterpret_cast<const uint2*>(UQ + (size_t)j * 8));
                        else t16[i] = *reinterpret_cast<const uint4*>(UQ + (size_t)j * 16);
                    }
#pragma unroll
                    for (int i = 0; i < ROWS * CPR / 256; ++i) {
                        const int j = tid + 256 * i;
                        const int row = j / CPR, cc = j - row * CPR;
                        *reinterpret_cast<uint4*>(smem + C::OFF_Q + (cc >> 3) * C::A_BLOCK + ptx::sw128_offset(row, cc & 7)) = t16[i];
                    }
                    ptx::fence_proxy_async_smem();
                }
                __syncwarp();
                if (alive && lane == 0) ptx::mbar_arrive(&misc->q_full);
            };
            // this thread's half of O of head hi: acc / 255 -> fp16 into U (the dense [128][D] tile)
            auto stage_o_u = [&](int hi) {
                const uint32_t t_o = tmem_base + C::TMEM_O + (hi % C::OBUF) * DP + half * OC + lane_addr;
                uint32_t v[OC / 8][8];
#pragma unroll
                for (int i = 0; i < OC / 8; ++i) ptx::tmem_ld8(t_o + i * 8, v[i]);
                ptx::tmem_ld_wait(v[0]);
#pragma unroll
                for (int i = 1; i < OC / 8; ++i) ptx::reg_fence8(v[i]);
#pragma unroll
                for (int i = 0; i < OC / 8; ++i) {
                    if (half * OC + i * 8 < D) {
                        uint32_t pk[4];
#pragma unroll
                        for (int e2 = 0; e2 < 4; ++e2) {
                            __half2 hv = __floats2half2_rn(__uint_as_float(v[i][2 * e2]) * inv255, __uint_as_float(v[i][2 * e2 + 1]) * inv255);
                            pk[e2] = *reinterpret_cast<uint32_t*>(&hv);
                        }
                        *reinterpret_cast<uint4*>(U + ((size_t)r * D + half * OC + i * 8) * 2) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    }
                }
                ptx::tc_fence_before_sync();
                ptx::fence_proxy_async_smem();
            };
            auto send_o = [&](int hi) {          // one thread, after the barrier that follows stage_o_u
                ptx::tma_store_3d(&tmap_o, U, (h_begin + hi) * D, row0, zb);
                ptx::bulk_store_commit();
            };

            if (tid == 0) load_q(0);
            float sq = 1.0f, sq_next = 1.0f;
            if (Q8) sq = valid ? __ldg(a.q_scales + grow * H + h_begin) : 0.f;
            stage_q_u(0);
            all256();                                        // U has been read by everybody
            if (tid == 0 && HG > 1) load_q(1);

            for (int hi = 0; hi < HG; ++hi) {
                const uint32_t ph = hi & 1;
                const bool more = hi + 1 < HG;
                if (Q8 && more) sq_next = valid ? __ldg(a.q_scales + grow * H + h_begin + hi + 1) : 0.f;
                alive = alive && __all_sync(0xffffffffu, ptx::mbar_wait(&misc->s_full[ph], (hi >> 1) & 1) && !misc->abort_flag);
                if (tid == 0 && hi < 8) TAQ_PROF(16 + hi);
                float e[HK];
                float k255 = 0.f;
                unsigned long long trig = 0;
                if (alive) {
                    ptx::tc_fence_after_sync();
                    uint32_t u[HK];
                    {
                        const uint32_t t_s = tmem_base + C::TMEM_S + ph * TP + key0 + lane_addr;
                        uint32_t (&u8)[HK / 8][8] = *reinterpret_cast<uint32_t (*)[HK / 8][8]>(&u);
#pragma unroll
                        for (int i = 0; i < HK / 8; ++i) ptx::tmem_ld8(t_s + i * 8, u8[i]);
                        ptx::tmem_ld_wait(u8[0]);
#pragma unroll
                        for (int i = 1; i < HK / 8; ++i) ptx::reg_fence8(u8[i]);
                    }
                    ptx::tc_fence_before_sync();
                    const OperandConsts* cst = C::SPLIT_KV ? reinterpret_cast<const OperandConsts*>(smem + C::OFF_CST + (hi % 3) * C::CST_SLOT)
                                                           : reinterpret_cast<const OperandConsts*>(smem + C::OFF_KV + (hi % C::KVBUF) * C::HEAD_BYTES + C::K_BYTES + C::VT_BYTES);
                    float m_loc, l_loc;
                    softmax_half<TAIL_ONLY>(u, cst->logit_factor + key0, sq, T, key0, e, m_loc, l_loc);
                    trig = half == 0 ? ((unsigned long long)cst->trig_bits[0] | ((unsigned long long)(cst->trig_bits[1] & 0xFFu) << 32))
                                     : ((unsigned long long)(cst->trig_bits[1] >> 8) | ((unsigned long long)cst->trig_bits[2] << 24));
                    misc->xchg[ph][half][r] = make_float2(m_loc, l_loc);
                    asm volatile("bar.sync %0, 64;" ::"r"(1 + q4) : "memory");
                    const float2 other = misc->xchg[ph][half ^ 1][r];
                    const float m_all = fmaxf(m_loc, other.x);
                    const float c_self = ex2_approx(m_loc - m_all), c_other = ex2_approx(other.x - m_all);
                    k255 = __fdividef(pmax * c_self, fmaf(l_loc, c_self, other.y * c_other));
                } else {
                    asm volatile("bar.sync %0, 64;" ::"r"(1 + q4) : "memory");
                }
                // S of this head is complete, so the Q~ operand tile is free: expand the next head's codes, which have had
                // the softmax to arrive
                if (tid == 128 && hi < 8) TAQ_PROF(104 + hi);
                if (more) stage_q_u(hi + 1);
                if (tid == 0 && hi < 8) TAQ_PROF(32 + hi);
                if (tid == 128 && hi < 8) TAQ_PROF(112 + hi);
                if (SEPQ && tid == 0) ptx::bulk_store_wait_read();      // (the store of the head before last: long done)
                all256();                                    // the raw tile has been read by everybody, U by the store
                if (SEPQ && tid == 0 && hi + 2 < HG && alive) load_q(hi + 2);
                if (hi > 0) {                                // O of the previous head: TMEM -> U -> global (TMA store)
                    alive = alive && __all_sync(0xffffffffu, ptx::mbar_wait(&misc->o_full[(hi - 1) % C::OBUF], ((hi - 1) / C::OBUF) & 1) && !misc->abort_flag);
                    if (alive) {
                        ptx::tc_fence_after_sync();
                        stage_o_u(hi - 1);
                    }
                    all256();
                    if (tid == 0 && alive) send_o(hi - 1);
                }
                if (tid == 0 && hi < 8) TAQ_PROF(48 + hi);
                if (alive) {
                    if (a.p_log) write_p_half_log(e, k255, cmax, trig, smem + C::OFF_P, C::A_BLOCK, r, half * (HK / 8));
                    else write_p_half(e, k255, trig, smem + C::OFF_P, C::A_BLOCK, r, half * (HK / 8));
                    ptx::fence_proxy_async_smem();
                    ptx::tc_fence_before_sync();
                }
                __syncwarp();
                if (alive && lane == 0) ptx::mbar_arrive(&misc->p_full);
                if (tid == 0 && hi < 8) TAQ_PROF(64 + hi);
                if (!SEPQ && tid == 0) {                     // shared buffer: once the store has read it, the raw tile of the head after next may land
                    ptx::bulk_store_wait_read();
                    if (hi + 2 < HG && alive) load_q(hi + 2);
                }
                sq = sq_next;
            }
            alive = alive && __all_sync(0xffffffffu, ptx::mbar_wait(&misc->o_full[(HG - 1) % C::OBUF], ((HG - 1) / C::OBUF) & 1) && !misc->abort_flag);
            if (SEPQ) {                                      // the store of the head before must have read U
                if (tid == 0) ptx::bulk_store_wait_read();
                all256();
            }
            if (alive) {
                ptx::tc_fence_after_sync();
                stage_o_u(HG - 1);
            }
            all256();
            if (tid == 0) {
                if (alive) send_o(HG - 1);
                ptx::bulk_store_wait_read();
            }
            if (!alive) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
        } else {
        auto store_o = [&](int hi) {        // this thread's half of O of head hi: acc / 255 -> fp16
            __half* orow = a.o + grow * Cch + (h_begin + hi) * D + half * OC;
            const uint32_t t_o = tmem_base + C::TMEM_O + (hi % C::OBUF) * DP + half * OC + lane_addr;
            uint32_t v[OC / 8][8];
#pragma unroll
            for (int i = 0; i < OC / 8; ++i) ptx::tmem_ld8(t_o + i * 8, v[i]);
            ptx::tmem_ld_wait(v[0]);
#pragma unroll
            for (int i = 1; i < OC / 8; ++i) ptx::reg_fence8(v[i]);
#pragma unroll
            for (int i = 0; i < OC / 8; ++i) {
                if (half * OC + i * 8 < D && valid) {
                    uint32_t pk[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        __half2 hv = __floats2half2_rn(__uint_as_float(v[i][2 * e]) * inv255, __uint_as_float(v[i][2 * e + 1]) * inv255);
                        pk[e] = *reinterpret_cast<uint32_t*>(&hv);
                    }
                    *reinterpret_cast<uint4*>(orow + i * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
            ptx::tc_fence_before_sync();
        };
        auto stage_q = [&](const QRegs<D, Q8>& qr) {
#pragma unroll
            for (int i = 0; i < CH2; ++i) {
                const int cc = half * CH2 + i;
                if (cc < DP / 8) *reinterpret_cast<uint4*>(smem + C::OFF_Q + (cc >> 3) * C::A_BLOCK + ptx::sw128_offset(r, cc & 7)) = qr.chunk(i);
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&misc->q_full);
        };

        QRegs<D, Q8> qr;
        qr.load(a.q, grow * Cch + (size_t)h_begin * D, valid, half);
        float sq = 1.0f, sq_next = 1.0f;
        if (Q8) sq = valid ? a.q_scales[grow * H + h_begin] : 0.f;
        stage_q(qr);

        for (int hi = 0; hi < HG; ++hi) {
            const uint32_t ph = hi & 1;
            const bool more = hi + 1 < HG;
            if (more) {                         // next head's query codes: in flight while this head's S is awaited
                qr.load(a.q, grow * Cch + (size_t)(h_begin + hi + 1) * D, valid, half);
                if (Q8) sq_next = valid ? a.q_scales[grow * H + h_begin + hi + 1] : 0.f;
            }
            alive = __all_sync(0xffffffffu, ptx::mbar_wait(&misc->s_full[ph], (hi >> 1) & 1) && !misc->abort_flag);
            if (!alive) break;
            if (tid == 0 && hi < 8) TAQ_PROF(16 + hi);
            ptx::tc_fence_after_sync();
            uint32_t u[HK];
            {
                const uint32_t t_s = tmem_base + C::TMEM_S + ph * TP + key0 + lane_addr;
                uint32_t (&u8)[HK / 8][8] = *reinterpret_cast<uint32_t (*)[HK / 8][8]>(&u);
#pragma unroll
                for (int i = 0; i < HK / 8; ++i) ptx::tmem_ld8(t_s + i * 8, u8[i]);
                ptx::tmem_ld_wait(u8[0]);
#pragma unroll
                for (int i = 1; i < HK / 8; ++i) ptx::reg_fence8(u8[i]);
            }
            ptx::tc_fence_before_sync();

            // ---- this thread's half of the softmax; the row's two threads then exchange (max, sum) ----
            const OperandConsts* cst = C::SPLIT_KV ? reinterpret_cast<const OperandConsts*>(smem + C::OFF_CST + (hi % 3) * C::CST_SLOT)
                                                   : reinterpret_cast<const OperandConsts*>(smem + C::OFF_KV + (hi % C::KVBUF) * C::HEAD_BYTES + C::K_BYTES + C::VT_BYTES);
            float e[HK];
            float m_loc, l_loc;
            softmax_half<TAIL_ONLY>(u, cst->logit_factor + key0, sq, T, key0, e, m_loc, l_loc);
            const unsigned long long trig = half == 0 ? ((unsigned long long)cst->trig_bits[0] | ((unsigned long long)(cst->trig_bits[1] & 0xFFu) << 32))
                                                      : ((unsigned long long)(cst->trig_bits[1] >> 8) | ((unsigned long long)cst->trig_bits[2] << 24));
            misc->xchg[ph][half][r] = make_float2(m_loc, l_loc);
            asm volatile("bar.sync %0, 64;" ::"r"(1 + q4) : "memory");
            const float2 other = misc->xchg[ph][half ^ 1][r];
            const float m_all = fmaxf(m_loc, other.x);
            const float c_self = ex2_approx(m_loc - m_all), c_other = ex2_approx(other.x - m_all);
            const float k255 = __fdividef(pmax * c_self, fmaf(l_loc, c_self, other.y * c_other));

            // S of this head is complete, so the Q~ tile is free again; the next head's codes, asked for at the top of this
            // iteration, have had the softmax to arrive
            if (more) stage_q(qr);
            if (tid == 0 && hi < 8) TAQ_PROF(32 + hi);
            // the P tile is free once the previous head's PV has completed
            if (hi > 0) {
                alive = __all_sync(0xffffffffu, ptx::mbar_wait(&misc->o_full[(hi - 1) % C::OBUF], ((hi - 1) / C::OBUF) & 1) && !misc->abort_flag);
                if (!alive) break;
                ptx::tc_fence_after_sync();
                if (C::OBUF == 1) store_o(hi - 1);   // one O accumulator: empty it before the next PV may start
            }
            if (tid == 0 && hi < 8) TAQ_PROF(48 + hi);
            if (a.p_log) write_p_half_log(e, k255, cmax, trig, smem + C::OFF_P, C::A_BLOCK, r, half * (HK / 8));
            else write_p_half(e, k255, trig, smem + C::OFF_P, C::A_BLOCK, r, half * (HK / 8));
            ptx::fence_proxy_async_smem();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&misc->p_full);
            if (tid == 0 && hi < 8) TAQ_PROF(64 + hi);

            if (hi > 0 && C::OBUF == 2) store_o(hi - 1);    // under this head's PV
            sq = sq_next;
        }
        if (alive) {
            alive = __all_sync(0xffffffffu, ptx::mbar_wait(&misc->o_full[(HG - 1) % C::OBUF], ((HG - 1) / C::OBUF) & 1) && !misc->abort_flag);
            if (alive) {
                ptx::tc_fence_after_sync();
                store_o(HG - 1);
            }
        }
        if (!alive) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
        }
    }

    if (tid == 0) TAQ_PROF(9);
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) TAQ_GPROF(127);
    if (warp == MMA_WARP) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn3() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

template <int D>
int pick_heads_per_cta(const AttnArgs& a, int n_z) {
    // The largest head group that still fills the GPU's CTA slots to about three quarters.
    const long long tiles = (long long)((a.n_query + ROWS - 1) / ROWS) * n_z;
    const long long want = (long long)148 * Cfg<D>::CTAS_PER_SM * 3 / 4;
    for (int hg = a.heads; hg > 1; --hg) {
        if (a.heads % hg) continue;
        if (tiles * (a.heads / hg) >= want) return hg;
    }
    return 1;
}

template <int D, bool Q8, bool TAIL_ONLY>
cudaError_t launch_k(const AttnArgs& a, int n_z, cudaStream_t stream) {
    using C = Cfg<D>;
    {   // (the attribute belongs to the current device's copy of the function: set on every launch, it is cheap)
        cudaError_t e = cudaFuncSetAttribute(attention_sm100_kernel<D, Q8, TAIL_ONLY>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::TOTAL);
        if (e != cudaSuccess) return e;
    }
    const int hg = pick_heads_per_cta<D>(a, n_z);
    dim3 grid((a.n_query + ROWS - 1) / ROWS, a.heads / hg, n_z);
    CUtensorMap tmap_q, tmap_o;
    memset(&tmap_q, 0, sizeof(tmap_q));
    memset(&tmap_o, 0, sizeof(tmap_o));
    if (C::TMA_IO) {      // Q~ and O as [n_z][n_query][channels] in boxes of 128 rows x one head
        EncodeTiledFn enc = encode_tiled_fn3();
        if (!enc) return cudaErrorNotSupported;
        const cuuint64_t qesz = Q8 ? 1 : 2;
        const cuuint64_t dims[3] = {(cuuint64_t)a.channels, (cuuint64_t)a.n_query, (cuuint64_t)n_z};
        const cuuint64_t qstr[2] = {(cuuint64_t)a.channels * qesz, (cuuint64_t)a.channels * qesz * (cuuint64_t)a.n_query};
        const cuuint64_t ostr[2] = {(cuuint64_t)a.channels * 2, (cuuint64_t)a.channels * 2 * (cuuint64_t)a.n_query};
        const cuuint32_t box[3] = {(cuuint32_t)D, ROWS, 1}, estr[3] = {1, 1, 1};
        if (enc(&tmap_q, Q8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(a.q), dims, qstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return cudaErrorInvalidValue;
        if (enc(&tmap_o, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, (void*)a.o, dims, ostr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    return launch_pdl(attention_sm100_kernel<D, Q8, TAIL_ONLY>, grid, dim3(ATT_THREADS), (size_t)C::TOTAL, stream, tmap_q, tmap_o, a, hg);
}

template <int D>
cudaError_t launch_d(const AttnArgs& a, int n_z, cudaStream_t stream) {
    const bool q8 = a.q_bits == 8, tail = a.n_ctx > 64;
    if (q8) return tail ? launch_k<D, true, true>(a, n_z, stream) : launch_k<D, true, false>(a, n_z, stream);
    return tail ? launch_k<D, false, true>(a, n_z, stream) : launch_k<D, false, false>(a, n_z, stream);
}

}  // namespace

bool sm100_attention_supported(const AttnArgs& a) {
    OperandGeom g;
    if (!operand_geom(a.channels / a.heads, a.n_ctx, &g)) return false;
    if (a.p_bits != 8 && a.p_bits != 4) return false;
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
