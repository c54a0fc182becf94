// Dequant-GEMM on the Blackwell tensor cores: y = x W^T with W^ = code * scale.
//
// The tensor cores never see a scale: the B operand holds the integer codes as fp16 (exact), every scale group
// (128 fan-in elements for W4, the whole row for W8) is accumulated in its own pass into one of two TMEM
// accumulators, and the worker threads fold each finished group into fp32 registers, y += scale[n][g] * acc_g,
// while the tensor core is already on the next group.
//
// One CTA computes a 128-row x BN-column tile.  The packed codes of its BN output channels (a contiguous slice of
// the blob), their scales and biases are fetched once with three bulk copies; K is walked in blocks of 64 through
// a ring of shared-memory stages.  Roles:
//   warp 0       one thread issues the bulk copies and the TMA loads of the fp16 activation tile (128 x 64,
//                128-byte swizzle);
//   warp 1       owns the TMEM allocation; one thread issues tcgen05.mma (M=128, N=BN, K=16) and commits;
//   warps 2..9   workers, two threads per accumulator row (TMEM lane), each owning half of the tile's columns:
//                they expand the 4/8-bit codes from shared memory into the fp16 weight tile (BN x 64, swizzled
//                K-major), fold finished groups into registers, and run the epilogue: bias / fp16 conversion, or
//                the per-(row, head) int8 quantization Q_a of Eq. 2, or the mixed int8 / fp16 K~,V~ of Eq. 2.
// The packed weights stay packed in HBM and are read once per CTA.
#include "taq_ptx.cuh"
#include "taq_sm100.cuh"
#include "taq_sm100_parts.cuh"
#include "taq_prof.cuh"
#include <type_traits>

TAQ_PROF_DEFINE(linear)

namespace taq {

namespace {

using namespace parts;

constexpr int BM = 128;
constexpr int BK = 64;                     // fp16 elements per 128-byte operand row; the int8 variant has 2 BK
constexpr int MAX_STAGE = 6;
constexpr int MAX_PREBUILT = 12;           // k-blocks per CTA whose expanded weight tiles may all be resident at once
constexpr int MAX_ACC = 8;                  // TMEM accumulators (scale groups in flight) per CTA
constexpr int NWORK = 256;                  // worker threads: two per accumulator row
constexpr int NTHREADS = 64 + NWORK;
constexpr int A_TILE_BYTES = BM * BK * 2;   // 16 KB
constexpr int SMEM_LIMIT = 227 * 1024;

template <int BN>
struct Tile {
    static constexpr int HC = BN / 2;                                         // columns per worker thread
    static constexpr int B_TILE_BYTES = ((BN * BK * 2 + 1023) / 1024) * 1024;
    static constexpr int STAGE_BYTES = A_TILE_BYTES + B_TILE_BYTES;
    static constexpr uint32_t TMEM_COLS = 2 * BN <= 128 ? 128 : 2 * BN <= 256 ? 256 : 512;
    static constexpr int CTAS_PER_SM = TMEM_COLS <= 256 ? 2 : 1;
    static_assert(HC % 8 == 0, "a worker's columns come in groups of 8");
};

struct Bars {
    uint64_t full_a[MAX_STAGE];
    uint64_t full_b[MAX_PREBUILT];
    uint64_t empty[MAX_STAGE];
    uint64_t w_full;
    uint64_t acc_full[MAX_ACC];
    uint64_t acc_free[MAX_ACC];
    uint64_t part_full[8], part_got[8], peer_ready;   // K loop split over a CTA pair: hand-over of the second CTA's partial sums
    uint64_t pair_full[4], pair_got[4];               // head split over two column tiles: the rows' absmax from / to the other tile's CTA
    uint32_t tmem_base;
    volatile int abort_flag;
};

// Shared-memory plan of one launch (host and device agree through these numbers).
struct Plan {
    int raw_bytes, scale_bytes, bias_bytes;   // BN rows of codes / scales / bias
    int stage_bytes;                          // one ring stage: the activation tile, plus the weight tile unless prebuilt
    int off_ball;                             // prebuilt: the CTA's expanded weight tiles, one per k-block
    int off_raw, off_scales, off_scales_t, off_bias, off_xchg, off_bars, total;
};

// prebuilt = number of k-blocks of the CTA when all of its expanded weight tiles are resident at once (0: the tiles go
// through the ring with the activations).
template <int BN>
__host__ __device__ inline Plan make_plan(int k_in, int bits, int group, int nstage, int mode, int prebuilt = 0) {
    const WeightLayout L = weight_layout(BN, k_in, bits, group);
    Plan p;
    p.stage_bytes = prebuilt ? A_TILE_BYTES : Tile<BN>::STAGE_BYTES;
    p.off_ball = nstage * p.stage_bytes;
    // codes of the BN channels over the whole fan-in; mode 1: none (the codes are the B operand); mode 2: one 64-byte slice
    // per channel and ring stage
    p.raw_bytes = mode == 1 ? 0 : mode == 2 ? nstage * BN * BK : (int)(L.row_bytes * BN);
    p.scale_bytes = BN * L.n_groups * 4;
    p.bias_bytes = BN * 4;
    p.off_raw = p.off_ball + prebuilt * Tile<BN>::B_TILE_BYTES;
    p.off_scales = p.off_raw + (p.raw_bytes + 127) / 128 * 128;
    p.off_scales_t = p.off_scales + (p.scale_bytes + 127) / 128 * 128;        // [n_groups][BN]
    p.off_bias = p.off_scales_t + (p.scale_bytes + 127) / 128 * 128;
    p.off_xchg = p.off_bias + (p.bias_bytes + 127) / 128 * 128;              // float [2][128]
    p.off_bars = p.off_xchg + 2048;           // float [2][128] exchange between a row's two threads, [128] out and [128] in for the head pair
    p.total = p.off_bars + 1024 + 1024;       // barriers + slack to align the base to 1024
    return p;
}

// I8: the integer-activation variant (the literal W/A reading of Table 1).  The A operand is the int8 codes of the
// per-token-quantized activations, the B operand the int8 weight codes, the accumulators are exact int32; a K block is
// 128 elements (one W4 scale group), and the row's activation scale multiplies the folded sum at the end.
// SPLIT: for launches with few tiles and a long K loop, two CTAs (a cluster of two along x) share one output tile: the first
// takes the lower half of the scale groups (of the k-blocks, when there is one group), the second the upper half; then
// they exchange folded fp32 partial sums through bulk copies between the two shared memories, the first CTA adding and
// storing rows 0..63 of the tile, the second rows 64..127.
template <int BN, bool I8, bool SPLIT>
__global__ void __launch_bounds__(NTHREADS, Tile<BN>::CTAS_PER_SM) linear_sm100_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ CUtensorMap tmap_y, const LinearArgs a, const int nstage, const int prebuilt) {
    using TL = Tile<BN>;
    constexpr int BKE = I8 ? 2 * BK : BK;             // elements per K block
    constexpr int HC = TL::HC;
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_u32(smem_dyn) & 1023u)) & 1023u);   // 1024-byte aligned, still provably shared
    const Plan P = make_plan<BN>(a.k_in, a.bits, a.group, nstage, a.w_direct, prebuilt);
    static_assert(sizeof(Bars) <= 1024, "barrier block");
    Bars* bars = reinterpret_cast<Bars*>(smem + P.off_bars);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int z = blockIdx.z;
    const int rank = SPLIT ? (int)(blockIdx.x & 1) : 0;
    const int row0 = (SPLIT ? (int)(blockIdx.x >> 1) : (int)blockIdx.x) * BM;
    const int col0 = blockIdx.y * BN;
    const int n_kb = (a.k_in + BKE - 1) / BKE;          // (int8: the last block may be ragged; TMA and the expansion zero-fill)
    const uint8_t* blob = (const uint8_t*)(a.reqs ? (a.which == 0 ? a.reqs[z].Wq : a.reqs[z].Wout) : a.w);
    const WeightLayout L = weight_layout(a.n_out, a.k_in, a.bits, a.group);
    const int n_groups = L.n_groups;
    const int kb_per_group = n_groups == 1 ? n_kb : L.group_len / BKE;   // k-blocks in a full group (the last group may be shorter)
    // this CTA's share of the K loop: all of it, one half of the scale groups, or (one scale per output channel) one half
    // of the k-blocks of the only group
    const bool split_kb = SPLIT && n_groups == 1;
    const int g_begin = SPLIT && !split_kb && rank ? n_groups / 2 : 0, g_end = SPLIT && !split_kb && !rank ? n_groups / 2 : n_groups;
    const int kb_begin = split_kb ? (rank ? n_kb / 2 : 0) : g_begin * kb_per_group;
    const int kb_stop = split_kb ? (rank ? n_kb : n_kb / 2) : min(n_kb, g_end * kb_per_group);
    // Accumulators: two (the workers fold one while the tensor core fills the other), or, when the weight tiles are all
    // built before the first fold (prebuilt), one per scale group of the CTA as far as TMEM holds them, so that no MMA
    // waits for a fold.
    const int n_acc = prebuilt ? max(1, min(min(g_end - g_begin, 512 / BN), MAX_ACC)) : 2;
    uint32_t tmem_cols = TL::TMEM_COLS;
    if (prebuilt) for (tmem_cols = 32; tmem_cols < (uint32_t)(n_acc * BN); tmem_cols *= 2) {}
    constexpr uint32_t PART_ROW = (uint32_t)BN * 2u + 16u;           // a thread's fp32 partial sums (BN / 2 columns), padded against bank conflicts

    TAQ_PROF_INIT
    if (tid == 0) { TAQ_PROF(0); TAQ_GPROF(30); }
    if (tid == 0) {
        for (int s = 0; s < MAX_STAGE; ++s) {
            ptx::mbar_init(&bars->full_a[s], 1);
            ptx::mbar_init(&bars->empty[s], 1);
        }
        for (int s = 0; s < MAX_PREBUILT; ++s) ptx::mbar_init(&bars->full_b[s], NWORK / 32);    // one arrival per worker warp
        ptx::mbar_init(&bars->w_full, 1);
        for (int i = 0; i < MAX_ACC; ++i) {
            ptx::mbar_init(&bars->acc_full[i], 1);
            ptx::mbar_init(&bars->acc_free[i], NWORK / 32);
        }
        for (int i = 0; i < 8; ++i) { ptx::mbar_init(&bars->part_full[i], 1); ptx::mbar_init(&bars->part_got[i], 1); }
        ptx::mbar_init(&bars->peer_ready, 1);
        for (int i = 0; i < 4; ++i) { ptx::mbar_init(&bars->pair_full[i], 1); ptx::mbar_init(&bars->pair_got[i], 1); }
        bars->abort_flag = 0;
        ptx::mbar_fence_init();
        if (SPLIT)                                          // the worker warps whose rows this CTA finishes receive a piece each
            for (int i = 0; i < 8; ++i)
                if (((i & 3) >> 1) == rank) ptx::mbar_arrive_expect_tx(&bars->part_full[i], 32u * PART_ROW);
        if (SPLIT && a.head_pair)                           // the TMEM lane quarters whose rows this CTA finishes: (q + 2) & 3 of worker warp q
            for (int ww = 0; ww < 4; ++ww)
                if ((ww >> 1) == rank) ptx::mbar_arrive_expect_tx(&bars->pair_full[(ww + 2) & 3], 128u);
        ptx::tma_prefetch_desc(&tmap_x);
    }
    if (warp == 1) ptx::tmem_alloc(&bars->tmem_base, tmem_cols);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    ptx::pdl_trigger();
    if (SPLIT) ptx::cluster_sync_all();                    // the partner's barriers exist before anything arrives on them

    if (warp == 0) {
        // ---------------- producer: packed weights once, then activation tiles ----------------
        if (lane == 0) {
            if (!a.early_weights) ptx::pdl_wait();        // in general the weights may come from the previous kernel
            const int staged = a.w_direct ? 0 : P.raw_bytes;
            ptx::mbar_arrive_expect_tx(&bars->w_full, (uint32_t)(staged + P.scale_bytes + P.bias_bytes));
            if (staged) ptx::bulk_load(smem + P.off_raw, blob + L.off_codes + (size_t)col0 * L.row_bytes, (uint32_t)P.raw_bytes, &bars->w_full);
            ptx::bulk_load(smem + P.off_scales, blob + L.off_scales + (size_t)col0 * n_groups * 4, (uint32_t)P.scale_bytes, &bars->w_full);
            ptx::bulk_load(smem + P.off_bias, blob + L.off_bias + (size_t)col0 * 4, (uint32_t)P.bias_bytes, &bars->w_full);
            if (a.early_weights) ptx::pdl_wait();         // the activations come from the previous kernel
            TAQ_PROF(1); TAQ_GPROF(28);
            int issued = 0, s = 0;
            uint32_t ph = 0;                               // parity of the ring pass
            for (int kb = kb_begin; kb < kb_stop; ++kb) {
                if (kb - kb_begin >= nstage && !ptx::mbar_wait(&bars->empty[s], ph ^ 1)) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
                if (bars->abort_flag) break;
                ptx::mbar_arrive_expect_tx(&bars->full_a[s], A_TILE_BYTES + (a.w_direct == 1 ? BN * 128 : a.w_direct == 2 ? BN * BK : 0));
                ptx::tma_load_3d(smem + s * P.stage_bytes, &tmap_x, &bars->full_a[s], kb * BKE, row0, z);
                if (a.w_direct == 1) ptx::tma_load_3d(smem + s * P.stage_bytes + A_TILE_BYTES, &tmap_w, &bars->full_a[s], kb * BKE, col0, 0);
                if (a.w_direct == 2) ptx::tma_load_3d(smem + P.off_raw + s * (BN * BK), &tmap_w, &bars->full_a[s], kb * BK, col0, 0);
                issued = kb - kb_begin + 1;
                if (++s == nstage) { s = 0; ph ^= 1; }
            }
            if (bars->abort_flag) {   // give copies that are still in flight a bounded chance to land before the CTA exits
                (void)ptx::mbar_wait(&bars->w_full, 0);
                for (int kb = issued > nstage ? issued - nstage : 0; kb < issued; ++kb) (void)ptx::mbar_wait(&bars->full_a[kb % nstage], (kb / nstage) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer: one accumulation pass per scale group ----------------
        // All 32 lanes walk the control flow, so that loop state and descriptor words stay warp-uniform; one elected lane
        // issues.  The path between two MMAs is kept short: this warp shares its scheduler with worker warps.
        const bool leader = ptx::elect_one();
        auto wait = [&](uint64_t* bar, uint32_t parity) -> bool { return __all_sync(0xffffffffu, ptx::mbar_wait(bar, parity) && !bars->abort_flag) != 0; };
        constexpr uint32_t idesc = I8 ? ptx::idesc_i8_m128(BN) : ptx::idesc_f16_m128(BN);
        constexpr uint32_t HI = ptx::kDescHiSw128;
        const uint32_t lo0 = ptx::desc_lo(ptx::smem_u32(smem));
        int s = 0, kb = kb_begin;
        uint32_t ph = 0;
        bool ok = true;
        for (int g = g_begin; g < g_end && ok; ++g) {
            const int gl = g - g_begin;
            const int buf = gl % n_acc;
            if (gl >= n_acc) {                              // the workers have emptied this accumulator
                if (!wait(&bars->acc_free[buf], (gl / n_acc - 1) & 1)) { ok = false; break; }
                ptx::tc_fence_after_sync();
            }
            const int kb_end = min(kb_stop, kb + kb_per_group);
            for (bool first = true; kb < kb_end && ok; ++kb) {
                // (prebuilt: every weight tile has its own barrier, complete long before its activations arrive)
                if ((a.w_direct != 1 && !wait(&bars->full_b[prebuilt ? kb - kb_begin : s], prebuilt ? 0u : ph)) || !wait(&bars->full_a[s], ph)) { ok = false; break; }
                if (leader) {
                    if (kb < 20) TAQ_PROF(40 + kb);
                    const uint32_t a_lo = lo0 + s * (P.stage_bytes >> 4);
                    const uint32_t b_lo = prebuilt ? lo0 + ((P.off_ball + (kb - kb_begin) * TL::B_TILE_BYTES) >> 4) : a_lo + (A_TILE_BYTES >> 4);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {            // four 32-byte K slices per 128-byte operand row
                        if (I8) ptx::mma_i8_ss(tmem_base + buf * BN, ptx::desc_join(HI, a_lo + 2 * k), ptx::desc_join(HI, b_lo + 2 * k), idesc, !(first && k == 0));
                        else ptx::mma_f16_ss(tmem_base + buf * BN, ptx::desc_join(HI, a_lo + 2 * k), ptx::desc_join(HI, b_lo + 2 * k), idesc, !(first && k == 0));
                    }
                    ptx::mma_commit(&bars->empty[s]);       // frees the stage once these MMAs have read it
                    if (kb + 1 == kb_end) ptx::mma_commit(&bars->acc_full[buf]);
                }
                first = false;
                if (++s == nstage) { s = 0; ph ^= 1; }
            }
        }
        if (!ok && leader) {
            raise_status(a.status, TAQ_ERR_TIMEOUT);
            bars->abort_flag = 1;
            for (int i = 0; i < n_acc; ++i) ptx::mma_commit(&bars->acc_full[i]);        // wake the workers; they see the abort flag
        }
    } else {
        // ---------------- workers (warps 2..9) ----------------
        const int wt = tid - 64;                          // 0..255
        const int q = warp & 3;                           // TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;                 // which half of the tile's columns this thread owns
        const int r = q * 32 + lane;
        long long row = (long long)row0 + r;
        const int cb = half * HC;                         // first owned column inside the tile
        const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + cb;
        const unsigned char* raw = smem + P.off_raw;
        const float* wscales = reinterpret_cast<const float*>(smem + P.off_scales);
        float* scales_t = reinterpret_cast<float*>(smem + P.off_scales_t);
        const float* bias = reinterpret_cast<const float*>(smem + P.off_bias);
        float* xchg = reinterpret_cast<float*>(smem + P.off_xchg);
        const int row_bytes = (int)L.row_bytes;
        bool ok = ptx::mbar_wait(&bars->w_full, 0);
        if (wt == 0) TAQ_PROF(2);
        if (!ok) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
        // scales [BN][n_groups] -> [n_groups][BN], so that a group's scales of consecutive columns are contiguous
        for (int i = wt; i < BN * n_groups; i += NWORK) scales_t[(i % n_groups) * BN + i / n_groups] = wscales[i];
        asm volatile("bar.sync 1, 256;" ::: "memory");

        float y[HC];
#pragma unroll
        for (int c = 0; c < HC; ++c) y[c] = 0.f;

        // y += scale[g] * accumulator of group g (this thread's HC columns of its row)
        auto fold_group = [&](int g) -> bool {
            const int buf = (g - g_begin) % n_acc;
            if (!ptx::mbar_wait(&bars->acc_full[buf], ((g - g_begin) / n_acc) & 1) || bars->abort_flag) return false;
            ptx::tc_fence_after_sync();
            const float* sg = scales_t + g * BN + cb;
#pragma unroll
            for (int c0 = 0; c0 < HC; c0 += 40) {
                constexpr int N8MAX = 5;
                uint32_t v[N8MAX][8];
#pragma unroll
                for (int i = 0; i < N8MAX; ++i)
                    if (c0 + i * 8 < HC) ptx::tmem_ld8(taddr + buf * BN + c0 + i * 8, v[i]);
                ptx::tmem_ld_wait(v[0]);
#pragma unroll
                for (int i = 1; i < N8MAX; ++i) ptx::reg_fence8(v[i]);
#pragma unroll
                for (int i = 0; i < N8MAX; ++i)
                    if (c0 + i * 8 < HC) {
                        const float4 s0 = *reinterpret_cast<const float4*>(sg + c0 + i * 8), s1 = *reinterpret_cast<const float4*>(sg + c0 + i * 8 + 4);
                        float* yy = y + c0 + i * 8;
                        float f[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) f[e] = I8 ? __int2float_rn((int)v[i][e]) : __uint_as_float(v[i][e]);
                        yy[0] = fmaf(f[0], s0.x, yy[0]); yy[1] = fmaf(f[1], s0.y, yy[1]);
                        yy[2] = fmaf(f[2], s0.z, yy[2]); yy[3] = fmaf(f[3], s0.w, yy[3]);
                        yy[4] = fmaf(f[4], s1.x, yy[4]); yy[5] = fmaf(f[5], s1.y, yy[5]);
                        yy[6] = fmaf(f[6], s1.z, yy[6]); yy[7] = fmaf(f[7], s1.w, yy[7]);
                    }
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&bars->acc_free[buf]);
            return true;
        };

        // expand the weight tiles of group g's k-blocks
        int s = 0, kb = kb_begin;
        uint32_t ph = 0;
        auto build_group = [&](int g) -> bool {
            const int kb_end = min(kb_stop, kb + kb_per_group);
            for (; kb < kb_end; ++kb) {
                if (!prebuilt && kb - kb_begin >= nstage && !ptx::mbar_wait(&bars->empty[s], ph ^ 1)) return false;
                if (bars->abort_flag) return false;
                if (a.w_direct == 2 && !ptx::mbar_wait(&bars->full_a[s], ph)) return false;    // this k-block's slice of the codes has arrived
                unsigned char* b_tile = prebuilt ? smem + P.off_ball + (kb - kb_begin) * TL::B_TILE_BYTES : smem + s * P.stage_bytes + A_TILE_BYTES;
                // 16-byte chunks of the fp16 tile: 8 per weight row; this thread owns chunk c of rows n0, n0 + 32, ...
                constexpr int NCH = (BN * 8 + NWORK - 1) / NWORK;
                const int n0 = wt >> 3, c = wt & 7;
                if (I8) {
                    // int8 tile: a chunk is 16 fan-in elements; chunks at or beyond k_in (ragged last block) are zero
                    const int k0 = kb * BKE + c * 16;
                    uint4 cw[NCH];
#pragma unroll
                    for (int i = 0; i < NCH; ++i) {
                        const int n = n0 + (NWORK / 8) * i;
                        cw[i] = make_uint4(0, 0, 0, 0);
                        if (((BN * 8) % NWORK == 0 || n < BN) && k0 < a.k_in) {
                            if (a.bits == 4) {
                                const uint2 p = *reinterpret_cast<const uint2*>(raw + n * row_bytes + (k0 >> 1));
                                const uint2 lo = codes_w4_to_i8(p.x), hi = codes_w4_to_i8(p.y);
                                cw[i] = make_uint4(lo.x, lo.y, hi.x, hi.y);
                            } else {
                                cw[i] = *reinterpret_cast<const uint4*>(raw + n * row_bytes + k0);
                            }
                        }
                    }
#pragma unroll
                    for (int i = 0; i < NCH; ++i) {
                        const int n = n0 + (NWORK / 8) * i;
                        if ((BN * 8) % NWORK == 0 || n < BN) *reinterpret_cast<uint4*>(b_tile + ptx::sw128_offset(n, c)) = cw[i];
                    }
                } else {
                uint2 pw[NCH];
#pragma unroll
                for (int i = 0; i < NCH; ++i) {
                    const int n = n0 + (NWORK / 8) * i;
                    pw[i] = make_uint2(0, 0);
                    if ((BN * 8) % NWORK == 0 || n < BN) {
                        if (a.bits == 4) pw[i].x = *reinterpret_cast<const uint32_t*>(raw + n * row_bytes + kb * (BK / 2) + c * 4);
                        else if (a.w_direct == 2) pw[i] = *reinterpret_cast<const uint2*>(raw + s * (BN * BK) + n * BK + c * 8);
                        else pw[i] = *reinterpret_cast<const uint2*>(raw + n * row_bytes + kb * BK + c * 8);
                    }
                }
#pragma unroll
                for (int i = 0; i < NCH; ++i) {
                    const int n = n0 + (NWORK / 8) * i;
                    if ((BN * 8) % NWORK == 0 || n < BN)
                        *reinterpret_cast<uint4*>(b_tile + ptx::sw128_offset(n, c)) = a.bits == 4 ? codes_w4_to_half(pw[i].x) : codes_w8_to_half(pw[i]);
                }
                }
                ptx::fence_proxy_async_smem();            // make the generic-proxy writes visible to the tensor core
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(&bars->full_b[prebuilt ? kb - kb_begin : s]);
                if (wt == 0 && kb < 20) TAQ_PROF(60 + kb);
                if (++s == nstage) { s = 0; ph ^= 1; }
            }
            return true;
        };

        // prebuilt (fp16 activations, codes staged): two tiles per pass, all loads before the conversions and the stores, one
        // proxy fence for both
        auto build_pair = [&](int kb0, int ntile) {
            constexpr int NCH = (BN * 8 + NWORK - 1) / NWORK;
            const int n0 = wt >> 3, c = wt & 7;
            uint2 pw[2][NCH];
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
                for (int i = 0; i < NCH; ++i) {
                    const int n = n0 + (NWORK / 8) * i;
                    pw[t][i] = make_uint2(0, 0);
                    if (t < ntile && ((BN * 8) % NWORK == 0 || n < BN)) {
                        if (a.bits == 4) pw[t][i].x = *reinterpret_cast<const uint32_t*>(raw + n * row_bytes + (kb0 + t) * (BK / 2) + c * 4);
                        else pw[t][i] = *reinterpret_cast<const uint2*>(raw + n * row_bytes + (kb0 + t) * BK + c * 8);
                    }
                }
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                unsigned char* b_tile = smem + P.off_ball + (kb0 + t - kb_begin) * TL::B_TILE_BYTES;
#pragma unroll
                for (int i = 0; i < NCH; ++i) {
                    const int n = n0 + (NWORK / 8) * i;
                    if (t < ntile && ((BN * 8) % NWORK == 0 || n < BN))
                        *reinterpret_cast<uint4*>(b_tile + ptx::sw128_offset(n, c)) = a.bits == 4 ? codes_w4_to_half(pw[t][i].x) : codes_w8_to_half(pw[t][i]);
                }
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane < ntile) ptx::mbar_arrive(&bars->full_b[kb0 + lane - kb_begin]);
            if (wt == 0 && kb0 < 20) TAQ_PROF(60 + kb0);
        };

        if (prebuilt) {            // every weight tile first (nothing to wait for), then the folds as the groups complete
            if (!I8)
                for (int k2 = kb_begin; k2 < kb_stop && !bars->abort_flag; k2 += 2) build_pair(k2, min(2, kb_stop - k2));
            ok = !bars->abort_flag;
            for (int g = g_begin; g < g_end && ok; ++g) ok = fold_group(g);
        } else {
            for (int g = g_begin; g < g_end && ok; ++g) {
                ok = a.w_direct == 1 ? true : build_group(g);
                if (ok && g > g_begin) ok = fold_group(g - 1);
            }
            if (ok) ok = fold_group(g_end - 1);
        }
        if (!ok) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
        asm volatile("bar.sync 1, 256;" ::: "memory");       // every worker gets here; the decision below is uniform
        ok = !bars->abort_flag;
        ptx::pdl_wait();                                     // (already satisfied: the activations have arrived) orders the stores below
        if (wt == 0) TAQ_PROF(7);
        if (SPLIT) {
            // All of this CTA's MMAs are complete (every group was folded), so its ring is free: it holds the partial sums
            // in transit, each thread's piece at the same place in both CTAs.  The first CTA finishes rows 0..63 of the
            // tile, the second rows 64..127: a worker warp either hands its 32 rows over (one bulk copy between the shared
            // memories, one barrier per warp) or receives the partner's piece and adds it, so both directions of the
            // exchange run at once and each CTA stores half of the tile.
            const int ww = wt >> 5, wl = wt & 31;
            const uint32_t peer = ptx::cluster_ctarank() ^ 1u;   // (clusters are two CTAs along x, times two along y for a head pair)
            const bool keep = ((ww & 3) >> 1) == rank;
            unsigned char* warp_part = smem + (size_t)ww * 32 * PART_ROW;
            float* piece = reinterpret_cast<float*>(warp_part + (size_t)wl * PART_ROW);
            if (wt == 0) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(ptx::smem_u32(&bars->peer_ready), peer));
            if (!keep) {
#pragma unroll
                for (int c = 0; c < HC; c += 4) *reinterpret_cast<float4*>(piece + c) = make_float4(y[c], y[c + 1], y[c + 2], y[c + 3]);
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (wl == 0) {
                    if (ww == 2) TAQ_PROF(11);
                    bool go = ptx::mbar_wait(&bars->peer_ready, 0) && !bars->abort_flag;         // the partner's ring is free, too
                    if (ww == 2) TAQ_PROF(12);
                    if (go) {
                        ptx::bulk_copy_to_cta(ptx::map_to_cta(ptx::smem_u32(warp_part), peer), warp_part, 32u * PART_ROW,
                                              ptx::map_to_cta(ptx::smem_u32(&bars->part_full[ww]), peer));
                        go = ptx::mbar_wait(&bars->part_got[ww], 0);     // this CTA's shared memory is the source: stay until it was read
                    }
                    if (!go) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
                }
                row = a.rows;                                // these rows are stored by the partner
            } else {
                if (!ptx::mbar_wait(&bars->part_full[ww], 0)) {
                    raise_status(a.status, TAQ_ERR_TIMEOUT);
                    bars->abort_flag = 1;
                } else {
#pragma unroll
                    for (int c = 0; c < HC; c += 4) {
                        const float4 p4 = *reinterpret_cast<const float4*>(piece + c);
                        y[c] += p4.x; y[c + 1] += p4.y; y[c + 2] += p4.z; y[c + 3] += p4.w;
                    }
                }
                __syncwarp();
                if (wl == 0) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(ptx::smem_u32(&bars->part_got[ww]), peer));
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");   // pieces read, outgoing copies done: the epilogue stages output there
            ok = !bars->abort_flag;
            if (wt == 0) TAQ_PROF(10);
        }
        if (I8 && ok) {                                      // x~ = code * s_x: the row's activation scale
            const float sx = row < a.rows ? a.x_scales[(size_t)z * a.rows + row] : 0.f;
#pragma unroll
            for (int c = 0; c < HC; ++c) y[c] *= sx;
        }

        // ---------------- epilogue on this thread's HC columns ----------------
        // Dense outputs (fp16, fp32, int8 codes) are staged in shared memory as the plain [128][BN] tile (the ring is free
        // now) and leave by one TMA store per 32 rows, issued as soon as the two warps that own those rows have written
        // them; the tensor map clips rows beyond the matrix.
        const bool stores_rows = !SPLIT || (((warp - 2) & 3) >> 1) == rank;
        auto store_quarter = [&](int esz) {
            ptx::fence_proxy_async_smem();
            asm volatile("bar.sync %0, 64;" ::"r"(3 + q) : "memory");
            if (half == 0 && lane == 0 && stores_rows && (long long)row0 + q * 32 < a.rows) {
                ptx::tma_store_3d(&tmap_y, smem + (size_t)q * 32 * BN * esz, col0, row0 + q * 32, z);
                ptx::bulk_store_commit();
                ptx::bulk_store_wait_read();
            }
        };
        if (ok) {
            if (a.epi == EPI_F16 || a.epi == EPI_F32) {
                const int esz = a.epi == EPI_F16 ? 2 : 4;
                unsigned char* seg = smem + ((size_t)r * BN + cb) * esz;
#pragma unroll
                for (int c = 0; c < HC; c += 8) {
                    float f[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) f[e] = y[c + e] + bias[cb + c + e];
                    if (a.epi == EPI_F16) {
                        *reinterpret_cast<uint4*>(seg + c * 2) = pack8(f);
                    } else {
                        *reinterpret_cast<float4*>(seg + c * 4) = make_float4(f[0], f[1], f[2], f[3]);
                        *reinterpret_cast<float4*>(seg + c * 4 + 16) = make_float4(f[4], f[5], f[6], f[7]);
                    }
                }
                store_quarter(esz);
            } else {
                // Per-(row, head) symmetric int8.  A thread's columns are either whole heads (HC a multiple of d) or half
                // of the tile's single head (d = BN); in the second case the row's two threads exchange their absmax.
                const int d = a.n_out / a.heads;
                const bool whole_heads = HC % d == 0;
                const int dd = whole_heads ? d : HC;                  // columns of one head held by this thread
                int slot = -1;
                bool trig = false;
                int t = 0;
                uint8_t* blk = nullptr;
                taq_kv_layout KL;
                if (a.epi == EPI_KV && row < a.rows) {
                    const int b = a.reqs ? 0 : (int)(row / a.n_ctx);
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
#pragma unroll
                for (int hc = 0; hc < HC; hc += 40) {                 // heads are 40, 64, 80 or 160 wide: steps of 40 or the whole of HC
                    if (hc % dd != 0) continue;
                    const int h = (col0 + cb + hc) / d;
                    const int ch = (col0 + cb + hc) - h * d;          // first column of this piece inside the head
                    float amax = 0.f;
#pragma unroll
                    for (int c = 0; c < HC; ++c)
                        if (c >= hc && c < hc + dd) amax = fmaxf(amax, fabsf(y[c]));
                    if (!whole_heads) {
                        xchg[half * 128 + r] = amax;
                        asm volatile("bar.sync 2, 256;" ::: "memory");
                        amax = fmaxf(amax, xchg[(half ^ 1) * 128 + r]);
                        if (SPLIT && a.head_pair && stores_rows) {
                            // The head's other 80 channels belong to the CTA next to this one along y (same rows, same
                            // half of the K loop): each sends its rows' absmax over (one 128-byte copy between the shared
                            // memories per 32 rows), waits for the other's, and confirms, so that the source outlives the copy.
                            float* out = xchg + 256, * in = xchg + 384;
                            const uint32_t other = ptx::cluster_ctarank() ^ 2u;
                            bool got = true;
                            if (half == 0) {
                                out[r] = amax;
                                ptx::fence_proxy_async_smem();
                                __syncwarp();
                                if (lane == 0)
                                    ptx::bulk_copy_to_cta(ptx::map_to_cta(ptx::smem_u32(in + q * 32), other), out + q * 32, 128u,
                                                          ptx::map_to_cta(ptx::smem_u32(&bars->pair_full[q]), other));
                            }
                            got = ptx::mbar_wait(&bars->pair_full[q], 0);
                            if (got) amax = fmaxf(amax, in[r]);
                            asm volatile("bar.sync %0, 64;" ::"r"(7 + q) : "memory");      // both warps of the quarter have read the piece
                            if (half == 0 && lane == 0) {
                                ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(ptx::smem_u32(&bars->pair_got[q]), other));
                                got = ptx::mbar_wait(&bars->pair_got[q], 0) && got;
                            }
                            if (!got) { raise_status(a.status, TAQ_ERR_TIMEOUT); bars->abort_flag = 1; }
                        }
                    }
                    const float s = quant_scale(amax, a.epi == EPI_KV && a.kv_qmax ? (float)a.kv_qmax : 127.f);
                    const float rs = s > 0.f ? __frcp_rn(s) : 0.f;
                    const bool owner = whole_heads || half == 0;      // writes the head's scale
                    if (a.epi == EPI_Q8_HEAD) {
                        // Q~ = Q_a(Q), Eq. 2 third line
                        unsigned char* seg = smem + (size_t)r * BN + cb;
#pragma unroll
                        for (int c = 0; c < HC; c += 8)
                            if (c >= hc && c < hc + dd) *reinterpret_cast<uint2*>(seg + c) = quant8(y + c, rs);
                        if (hc + dd >= HC) store_quarter(1);  // last head of the piece
                        if (row < a.rows && owner) a.scales[((size_t)z * a.rows + row) * a.heads + h] = s;
                    } else if (row < a.rows) {
                        // Eq. 2 for K or V: rows of ordinary tokens -> int8 codes + scale, rows of trigger tokens -> fp16
                        int8_t* cq = (int8_t*)(blk + (a.kv_which ? KL.off_v_codes : KL.off_k_codes)) + ((size_t)h * a.n_ctx + t) * d + ch;
#pragma unroll
                        for (int c = 0; c < HC; c += 8)
                            if (c >= hc && c < hc + dd) *reinterpret_cast<uint2*>(cq + c - hc) = trig ? make_uint2(0, 0) : quant8(y + c, rs);
                        if (slot >= 0) {
                            __half* tr = (__half*)(blk + (a.kv_which ? KL.off_v_trigger : KL.off_k_trigger)) + ((size_t)slot * a.heads + h) * d + ch;
#pragma unroll
                            for (int c = 0; c < HC; c += 8)
                                if (c >= hc && c < hc + dd) {
                                    float f[8];
#pragma unroll
                                    for (int e = 0; e < 8; ++e) f[e] = y[c + e];
                                    *reinterpret_cast<uint4*>(tr + c - hc) = pack8(f);
                                }
                        }
                        if (owner) {
                            ((float*)(blk + (a.kv_which ? KL.off_v_scales : KL.off_k_scales)))[(size_t)h * a.n_ctx + t] = trig ? 0.f : s;
                            if (h == 0 && a.kv_which == 0) ((int32_t*)(blk + KL.off_trig_slot))[t] = slot >= 0 ? slot : -1;
                        }
                    }
                }
                if (a.epi == EPI_KV && a.kv_which == 0 && blockIdx.x == 0 && blockIdx.y == 0) {   // slot table beyond T
                    const int nb = a.reqs ? 1 : (int)(a.rows / a.n_ctx);
                    const taq_kv_layout K2 = kv_layout(a.heads, a.n_ctx, d, a.max_trigger);
                    for (int i = wt; i < nb * (kMaxCtx - a.n_ctx); i += NWORK) {
                        const int bb = i / (kMaxCtx - a.n_ctx), tt = a.n_ctx + i % (kMaxCtx - a.n_ctx);
                        uint8_t* bk = a.reqs ? (uint8_t*)a.reqs[z].kv : (uint8_t*)a.y + (size_t)bb * K2.block_bytes;
                        ((int32_t*)(bk + K2.off_trig_slot))[tt] = -1;
                    }
                }
            }
        }
    }

    // ---------------- teardown ----------------
    if (tid == 64) TAQ_PROF(8);
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) { TAQ_PROF(9); TAQ_GPROF(29); }
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, tmem_cols);
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

// How the kernel gets at the weight codes: 0 = all codes of the tile's channels staged in shared memory once; 1 = int8
// activations and 8-bit weights: the codes are the B operand, by TMA per k-block; 2 = fp16 activations and 8-bit weights whose
// staged codes would not fit beside a two-stage ring (a 160-wide tile at a fan-in of 1280): a 64-byte slice per channel
// arrives by TMA with every k-block's activations and the workers expand from it.
template <int BN>
int weight_mode(const LinearArgs& a) {
    if (a.bits != 8) return 0;
    if (a.xq) return a.reqs ? 0 : 1;      // (per-request blobs have no common tensor map: their codes are staged)
    return make_plan<BN>(a.k_in, a.bits, a.group, 2, 0).total > SMEM_LIMIT ? (a.reqs ? 0 : 2) : 0;
}

// Bytes of the ring that the epilogue reuses to stage a tile's output before the TMA stores: the dense [128][BN] tile.
template <int BN>
int epilogue_staging_bytes(const LinearArgs& a) {
    if (a.epi == EPI_F16) return BM * BN * 2;
    if (a.epi == EPI_F32) return BM * BN * 4;
    if (a.epi == EPI_Q8_HEAD) return BM * BN;
    return 0;
}

// Ring depth: as deep as the K loop needs, but no deeper than three stages when that keeps two CTAs on an SM, and never
// shallower than the epilogue's staging area (which lives in the ring).  0: this tile width does not fit.
template <int BN>
int pick_nstage(const LinearArgs& a) {
    const int bke = a.xq ? 2 * BK : BK;
    const int direct = weight_mode<BN>(a);
    const int n_kb = (a.k_in + bke - 1) / bke;
    const int half_sm = Tile<BN>::CTAS_PER_SM == 2 ? SMEM_LIMIT / 2 : SMEM_LIMIT;
    const int ns_min = (epilogue_staging_bytes<BN>(a) + Tile<BN>::STAGE_BYTES - 1) / Tile<BN>::STAGE_BYTES;
    const int ns_max = n_kb < 2 ? 2 : n_kb;
    int best = 0;
    for (int ns = 1; ns <= MAX_STAGE && ns <= (ns_max > ns_min ? ns_max : ns_min); ++ns) {
        const int total = make_plan<BN>(a.k_in, a.bits, a.group, ns, direct).total;
        if (total > SMEM_LIMIT) break;
        if (ns > 3 && ns > ns_min && total + 1024 > half_sm && make_plan<BN>(a.k_in, a.bits, a.group, 3, direct).total + 1024 <= half_sm) break;
        best = ns;
    }
    return best >= ns_min ? best : 0;
}

int nstage_for(const LinearArgs& a, int bn) {
    switch (bn) {
        case 64: return pick_nstage<64>(a);
        case 80: return pick_nstage<80>(a);
        case 160: return pick_nstage<160>(a);
    }
    return 0;
}

// EPI_Q8_HEAD with heads of 160 channels: instead of one 160-wide tile per head (whose expanded weight tiles do not fit
// resident) two 80-wide tiles whose CTAs exchange the rows' absmax, when that launch is one wave of split tiles with
// resident weight tiles (clusters of 2 x 2: halves of the K loop along x, halves of the head along y).
bool head_pair_mode(const LinearArgs& a, int n_z);

int pick_bn(const LinearArgs& a, int n_z = 1) {
    // Every column tile re-reads the activation rows, so tiles are as wide as the row count allows while the grid
    // still covers most of the SMs; a width whose ring and staging do not fit shared memory is passed over.
    const long long row_tiles = (a.rows + BM - 1) / BM;
    auto fits = [&](int bn) { return nstage_for(a, bn) >= 2; };
    if (a.epi == EPI_Q8_HEAD || a.epi == EPI_KV) {
        const int d = a.n_out / a.heads;
        if (d == 40 && a.heads % 4 == 0 && row_tiles * (a.n_out / 160) >= 96 && fits(160)) return 160;   // two heads per worker thread
        if (d == 40 && a.heads % 2 == 0) return fits(80) ? 80 : 0;     // one head per worker thread
        if (d == 160 && a.epi == EPI_Q8_HEAD && head_pair_mode(a, n_z)) return 80;
        if (d == 64 || d == 80 || d == 160) return fits(d) ? d : 0;   // one head per tile, split between the row's two threads
        return 0;
    }
    if (a.n_out % 160 == 0 && row_tiles * (a.n_out / 160) >= 96 && fits(160)) return 160;
    if (a.n_out % 80 == 0 && fits(80)) return 80;
    if (a.n_out % 64 == 0 && fits(64)) return 64;
    return 0;
}

// How a launch is laid out: ring depth, whether two CTAs share a tile (split of the K loop), and whether every CTA keeps
// all of its expanded weight tiles resident (`prebuilt` = its number of k-blocks, else 0).
struct Choice { int ns, prebuilt; bool split; };

template <int BN>
Choice choose(const LinearArgs& a, int n_z) {
    const bool i8 = a.xq != nullptr;
    const int mode = weight_mode<BN>(a);
    Choice c{pick_nstage<BN>(a), 0, false};
    const WeightLayout Lw = weight_layout(a.n_out, a.k_in, a.bits, a.group);
    const int bke = i8 ? 2 * BK : BK;
    const int n_kb = (a.k_in + bke - 1) / bke;
    const long long tiles = ((a.rows + BM - 1) / BM) * (a.n_out / BN) * (long long)n_z;
    const int staging = epilogue_staging_bytes<BN>(a);
    const int part = NWORK * (BN * 2 + 16);          // fp32 partial sums in transit between the two CTAs of a split tile
    // few tiles and a long K loop: two CTAs per tile, each with half of the scale groups (or of the k-blocks of a single
    // group: not for integer activations, where a group's sum stays one exact int32 accumulation)
    const bool want_split = (Lw.n_groups >= 2 || !i8) && tiles <= 74 * Tile<BN>::CTAS_PER_SM && n_kb >= 6;
    c.split = want_split && (long long)c.ns * Tile<BN>::STAGE_BYTES >= part;
    // One wave at one CTA per SM, codes staged once, fp16 activations: expand every weight tile of the CTA before the
    // activations arrive (under the previous kernel's tail when the weights are known early), so that the K loop waits
    // for the TMA loads only.
    if (mode == 0 && !i8 && tiles <= 148) {
        for (int with_split = (want_split && 2 * tiles <= 148) ? 1 : 0; with_split >= 0; --with_split) {
            int n_cta = n_kb;
            if (with_split) {
                if (Lw.n_groups == 1) n_cta = n_kb - n_kb / 2;
                else { const int kbg = Lw.group_len / bke, lo = (Lw.n_groups / 2) * kbg; n_cta = lo > n_kb - lo ? lo : n_kb - lo; }
            }
            // the activation ring as deep as shared memory allows: with the weight tiles resident the K loop's pace is
            // the latency of the activation loads divided by the loads in flight
            bool found = false;
            for (int ns = n_cta < MAX_STAGE ? (n_cta < 2 ? 2 : n_cta) : MAX_STAGE; ns >= (n_cta < 3 ? 2 : 3) && !found; --ns) {
                const Plan P = make_plan<BN>(a.k_in, a.bits, a.group, ns, 0, n_cta);
                if (n_cta <= MAX_PREBUILT && P.total <= SMEM_LIMIT && P.off_raw >= staging && (!with_split || P.off_raw >= part)) {
                    c.ns = ns; c.prebuilt = n_cta; c.split = with_split != 0;
                    found = true;
                }
            }
            if (found) break;
        }
    }
    return c;
}

bool head_pair_mode(const LinearArgs& a, int n_z) {
    if (a.epi != EPI_Q8_HEAD || a.heads <= 0 || a.n_out != a.heads * 160 || a.xq || a.reqs) return false;
    if (nstage_for(a, 80) < 2) return false;
    const Choice c = choose<80>(a, n_z);
    return c.split && c.prebuilt > 0;
}

template <int BN>
cudaError_t launch_bn(const CUtensorMap& tmap, EncodeTiledFn enc, LinearArgs a, int n_z, cudaStream_t stream) {
    const bool i8 = a.xq != nullptr;
    const Choice ch = choose<BN>(a, n_z);
    const int ns = ch.ns;
    const bool split = ch.split;
    void (*kern)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const LinearArgs, const int, const int) =
        split ? (i8 ? linear_sm100_kernel<BN, true, true> : linear_sm100_kernel<BN, false, true>)
              : (i8 ? linear_sm100_kernel<BN, true, false> : linear_sm100_kernel<BN, false, false>);
    a.w_direct = weight_mode<BN>(a);
    a.head_pair = (BN == 80 && a.epi == EPI_Q8_HEAD && a.n_out == a.heads * 160) ? 1 : 0;
    if (a.head_pair && !(split && ch.prebuilt)) return cudaErrorNotSupported;
    CUtensorMap tmap_w = tmap;                        // (unused unless w_direct)
    if (a.w_direct) {                                 // the codes section of the blob as an int8 matrix [n_out][k_in]
        const WeightLayout L = weight_layout(a.n_out, a.k_in, a.bits, a.group);
        const cuuint64_t dims[3] = {(cuuint64_t)a.k_in, (cuuint64_t)a.n_out, 1};
        const cuuint64_t strides[2] = {(cuuint64_t)L.row_bytes, (cuuint64_t)L.row_bytes * (cuuint64_t)a.n_out};
        const cuuint32_t box[3] = {(cuuint32_t)(a.w_direct == 1 ? 2 * BK : BK), BN, 1}, estr[3] = {1, 1, 1};    // mode 2: plain rows of 64 codes
        CUresult r = enc(&tmap_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, (void*)((const uint8_t*)a.w + L.off_codes), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, a.w_direct == 1 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    CUtensorMap tmap_y = tmap;                        // (unused by the K~/V~ epilogue, which scatters into the cache block)
    if (a.epi == EPI_F16 || a.epi == EPI_F32 || a.epi == EPI_Q8_HEAD) {   // the output matrix [n_z][rows][n_out] in boxes of 32 rows x BN
        const cuuint64_t esz = a.epi == EPI_F16 ? 2 : a.epi == EPI_F32 ? 4 : 1;
        const cuuint64_t dims[3] = {(cuuint64_t)a.n_out, (cuuint64_t)a.rows, (cuuint64_t)n_z};
        const cuuint64_t strides[2] = {(cuuint64_t)a.n_out * esz, (cuuint64_t)a.n_out * esz * (cuuint64_t)a.rows};
        const cuuint32_t box[3] = {BN, 32, 1}, estr[3] = {1, 1, 1};
        CUresult r = enc(&tmap_y, a.epi == EPI_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : a.epi == EPI_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_UINT8,
                         3, a.y, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    {   // (the attribute belongs to the current device's copy of the function: set on every launch, it is cheap)
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_LIMIT);
        if (e != cudaSuccess) return e;
    }
    const Plan P = make_plan<BN>(a.k_in, a.bits, a.group, ns, a.w_direct, ch.prebuilt);
    dim3 grid((unsigned)((a.rows + BM - 1) / BM) * (split ? 2u : 1u), a.n_out / BN, n_z);
    if (split) return launch_pdl_cluster(kern, grid, dim3(2, a.head_pair ? 2 : 1, 1), dim3(NTHREADS), (size_t)P.total, stream, tmap, tmap_w, tmap_y, a, ns, ch.prebuilt);
    return launch_pdl(kern, grid, dim3(NTHREADS), (size_t)P.total, stream, tmap, tmap_w, tmap_y, a, ns, ch.prebuilt);
}

}  // namespace

bool sm100_linear_supported(const LinearArgs& a) {
    if (a.xq) {       // int8 activations: rows of 16-byte granularity, a scale group = one 128-element K block
        if (a.k_in % 16) return false;
        if (a.group != 0 && a.group != 2 * BK && a.group < a.k_in) return false;
        if (reinterpret_cast<uintptr_t>(a.xq) & 15u) return false;
    } else {
        if (a.k_in % BK) return false;
        if (a.group != 0 && a.group % BK) return false;
        if (reinterpret_cast<uintptr_t>(a.x) & 15u) return false;
    }
    if (a.epi != EPI_KV && (reinterpret_cast<uintptr_t>(a.y) & 15u)) return false;   // the output leaves by TMA stores
    if (a.rows < 1 || a.rows > (1LL << 31) - 1) return false;
    const int bn = pick_bn(a);
    if (bn == 0) return false;
    if (nstage_for(a, bn) < 2) return false;
    return encode_tiled_fn() != nullptr;
}

// The launch plan of a dequant-GEMM as the launcher would take it (no GPU needed): tile width, ring depth, how the codes
// reach the CTA, and the byte ranges of shared memory that the ring, the epilogue's staging area and the fixed sections
// occupy.  out: {bn, nstage, mode, ring_bytes, staging_bytes, off_raw, off_bias, off_bars, total, limit}.  bn = 0: the
// tensor-core kernel does not take this problem.
void linear_plan_of(const LinearArgs& a, int out[10]) {
    for (int i = 0; i < 10; ++i) out[i] = 0;
    out[9] = SMEM_LIMIT;
    bool ok = a.rows >= 1;
    if (a.xq) ok = ok && a.k_in % 16 == 0 && (a.group == 0 || a.group == 2 * BK || a.group >= a.k_in);
    else ok = ok && a.k_in % BK == 0 && (a.group == 0 || a.group % BK == 0);
    if (!ok) return;
    const int bn = pick_bn(a);
    if (bn == 0) return;
    if (nstage_for(a, bn) < 2) return;
    Plan P;
    int ring = 0, staging = 0, mode = 0, ns = 0;
    auto fill = [&](auto bn_c) {
        constexpr int B = decltype(bn_c)::value;
        const Choice c = choose<B>(a, 1);
        mode = weight_mode<B>(a); ns = c.ns;
        P = make_plan<B>(a.k_in, a.bits, a.group, c.ns, mode, c.prebuilt);
        ring = P.off_raw;                          // ring stages (and resident weight tiles): what the epilogue may reuse
        staging = epilogue_staging_bytes<B>(a);
        if (c.split && staging < NWORK * (B * 2 + 16)) staging = NWORK * (B * 2 + 16);
    };
    switch (bn) {
        case 64: fill(std::integral_constant<int, 64>{}); break;
        case 80: fill(std::integral_constant<int, 80>{}); break;
        default: fill(std::integral_constant<int, 160>{}); break;
    }
    out[0] = bn; out[1] = ns; out[2] = mode; out[3] = ring; out[4] = staging;
    out[5] = P.off_raw; out[6] = P.off_bias; out[7] = P.off_bars; out[8] = P.total;
}

cudaError_t launch_linear_sm100(const LinearArgs& a, int n_z, cudaStream_t stream) {
    if (a.rows == 0 || n_z == 0) return cudaSuccess;
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return cudaErrorNotSupported;
    CUtensorMap tmap;
    const bool i8 = a.xq != nullptr;
    const cuuint64_t esz = i8 ? 1 : 2;
    const cuuint64_t dims[3] = {(cuuint64_t)a.k_in, (cuuint64_t)a.rows, (cuuint64_t)n_z};
    const cuuint64_t strides[2] = {(cuuint64_t)a.k_in * esz, (cuuint64_t)a.k_in * esz * (cuuint64_t)a.rows};
    const cuuint32_t box[3] = {(cuuint32_t)(i8 ? 2 * BK : BK), BM, 1};       // 128 bytes of K either way; elements beyond k_in read as zero
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(&tmap, i8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3,
                     i8 ? (void*)const_cast<int8_t*>(a.xq) : (void*)const_cast<__half*>(a.x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    switch (pick_bn(a, n_z)) {
        case 64: return launch_bn<64>(tmap, enc, a, n_z, stream);
        case 80: return launch_bn<80>(tmap, enc, a, n_z, stream);
        case 160: return launch_bn<160>(tmap, enc, a, n_z, stream);
    }
    return cudaErrorNotSupported;
}

}  // namespace taq
