// One denoising-step pass of the TAQ cross-attention layer in one kernel for the SD-1.5 64x64 shape (C = 320, 8 heads of
// 40, W4): to_q, Q~ = Q_a(Q) (Eq. 2, third line), S = Q~ K~^T, softmax, Eq. 3, O = A^ V~, to_out.  Neither Q~ nor the
// scores, probabilities or O ever reach global memory.
//
// A CTA owns 128 query rows of one sequence and four heads (160 channels); the two CTAs that share a row tile form a
// cluster and exchange their halves of O through distributed shared memory.  Warps: 0 producer (TMA / bulk copies),
// 1 MMA issuer, 2..17 workers.  A worker thread is (row r, head hi) from start to end:
//   phase 1  Q = X Wq^T for the CTA's 160 channels: workers expand the packed 4-bit codes to fp16-integer operand tiles
//            (all five K blocks, before X has arrived), one TMEM accumulator per scale group, folded into registers with
//            the group's scales;
//   phase 2  the thread quantizes its 40 values (one head of one row) into the head's Q~ operand tile; the row scale
//            stays in a register;
//   phase 3  all four heads at once: four S accumulators (4 x 80 columns) and four O accumulators (4 x 48) fill the 512
//            TMEM columns.  The thread that quantized (r, hi) also owns that row's 80 scores: maximum, exponentials, sum
//            and Eq. 3 need no exchange between threads.  P (fp16 integers in units of 1/255, trigger columns fp16)
//            overwrites the head's Q~ tile (keys 0..63) plus a 32-byte-swizzled tail tile (keys 64..79);
//   phase 4  to_out for the CTA's 160 output channels over all 320 channels of O.  Each head's O goes, as soon as its own
//            PV product is complete, into 32-channel operand tiles placed where only probability tiles of heads already
//            finished lie; every tile is sent to the partner CTA as soon as it is complete.  The K steps over the CTA's
//            own tiles run while the partner's are in flight (each CTA begins with its own channels; every scale group
//            still has its own accumulator).  The Wout tiles are expanded during phase 3 into the dead K~ buffers, later
//            into the dead V~^T buffers.  Y leaves as one TMA tensor store per head group of 40 channels.
// Shared memory is reused: X tile -> Q~ / P tiles -> O tiles -> Y staging; weight tiles -> K~ and V~^T tiles -> weight ring.
#include "taq_ptx.cuh"
#include "taq_sm100.cuh"
#include "taq_sm100_parts.cuh"
#include "taq_prof.cuh"
#include <type_traits>

TAQ_PROF_DEFINE(layer)

namespace taq {

namespace {

using namespace parts;

constexpr int D = 40, DP = 48, HG = 4;          // head width, padded width, heads per CTA
constexpr int NQ = HG * D;                      // 160 channels per CTA
constexpr int KIN = 320, BK = 64, NKB = KIN / BK;
constexpr int ROWS = 128;
constexpr int NWORK = 512, NTHREADS = 64 + NWORK;
constexpr int MAX_GROUPS = 3;

constexpr int A_TILE = ROWS * 128;              // 16 KB: a 64-wide K block of X, a head's Q~ tile, keys 0..63 of P
constexpr int B_TILE = NQ * 128;                // 20 KB: a 64-wide K block of the expanded weights
constexpr int PB_TILE = ROWS * 32;              // 4 KB: keys 64..79 of P (32-byte rows)
constexpr int O_TILE = ROWS * 64;               // 8 KB: 32 channels of O (64-byte rows)
constexpr int N_OTILE = KIN / 32;
constexpr int K_BYTES = TP * 128;               // 10 KB: one head's K~ image
constexpr int VT_BLOCK = DP * 128, VT_BYTES = 2 * VT_BLOCK;     // 12 KB: one head's V~^T image (keys 0..63, 64..79)
constexpr int Y_STAGE = ROWS * D * 2;           // 10 KB: 40 channels of Y, dense rows of 80 bytes
constexpr int RAW_BYTES = NQ * (KIN / 2);       // 25600: packed codes of the CTA's 160 channels
constexpr int SCALE_BYTES = 2048;               // >= NQ * MAX_GROUPS * 4

constexpr int OFF_R0 = 0;                                   // 80 KB: X tile | Q~/P tiles + P tail tiles | O tiles | Y staging
constexpr int OFF_PB = OFF_R0 + HG * A_TILE;
constexpr int OFF_R1 = OFF_R0 + NKB * A_TILE;               // 60 KB: weight ring of phase 1 | V~^T tiles | ring stages 2, 3 of phase 4
constexpr int OFF_RAW = OFF_R1 + 3 * B_TILE;
constexpr int OFF_SC = OFF_RAW + RAW_BYTES;
constexpr int OFF_SCT = OFF_SC + SCALE_BYTES;
constexpr int OFF_BIAS = OFF_SCT + SCALE_BYTES;
constexpr int OFF_K = ((OFF_BIAS + NQ * 4 + 1023) / 1024) * 1024;       // 40 KB: K~ tiles of the four heads | ring stages 0, 1 of phase 4
constexpr int OFF_CST = OFF_K + HG * K_BYTES;
constexpr int OFF_MISC = OFF_CST + HG * kOperandConstBytes;
static_assert(OFF_PB + HG * PB_TILE <= OFF_R1, "P tiles fit into the X tile");
static_assert(N_OTILE * O_TILE <= NKB * A_TILE, "O tiles fit into the X tile");
static_assert(HG * VT_BYTES <= 3 * B_TILE && 2 * B_TILE <= 3 * B_TILE, "V~^T tiles fit into the phase-1 ring");
static_assert(HG * K_BYTES == 2 * B_TILE, "the K~ tiles are exactly two ring stages");
static_assert(HG * Y_STAGE <= NKB * A_TILE, "Y staging fits into the X tile");
static_assert(NQ * MAX_GROUPS * 4 <= SCALE_BYTES, "scale table");

constexpr int NS4 = 4;                          // ring stages of phase 4
constexpr int NEXP = NWORK - NWORK / HG;        // worker threads that expand the Wout tiles: the warps of heads 0..2
// Phase 1 keeps all five expanded Wq tiles: three in region 1, two where the K~ tiles arrive afterwards.
__device__ __forceinline__ int stage1_offset(int kb) { return kb < 3 ? OFF_R1 + kb * B_TILE : OFF_K + (kb - 3) * B_TILE; }
__host__ __device__ constexpr int stage4_offset(int s) { return s < 2 ? OFF_K + s * B_TILE : OFF_R1 + (s - 2) * B_TILE; }
// O tiles of phase 4 inside region 0.  A CTA's own tile lt (0..4, 32 channels each) is written by heads lt - 1 and lt and
// lies in the probability tile of head max(lt - 1, 0), dead by then (PV products complete in head order); the partner's
// five tiles arrive, once every PV product of this CTA is complete, in the second halves of the other probability tiles
// and in the tail tiles.
__host__ __device__ constexpr int own_tile_offset(int lt) { return OFF_R0 + (lt < 2 ? lt * O_TILE : (lt - 1) * A_TILE); }
__host__ __device__ constexpr int peer_tile_offset(int lt) { return OFF_R0 + (lt < 3 ? (lt + 1) * A_TILE + O_TILE : HG * A_TILE + (lt - 3) * O_TILE); }

struct Misc {
    uint64_t a_full[NKB], w_full, w2_full, kc_full, vt_full;
    uint64_t b1_full[NKB], b4_full[NKB], b4_empty[NS4], tile_done[N_OTILE / 2];       // b4_full: one per Wout tile of the walk
    uint64_t acc_full[MAX_GROUPS];
    uint64_t q_all, s_full[HG], p_full[HG], o_full[HG];
    uint64_t o_all, peer_ready, peer_got, drain;
    uint32_t tmem_base;
    volatile int abort_flag;
};
constexpr int TOTAL = OFF_MISC + (int)sizeof(Misc) + 1024;
static_assert(TOTAL <= 232448, "shared memory budget");

constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TMEM_ACC = 0;                 // phases 1 and 4: one accumulator of NQ columns per scale group
constexpr uint32_t TMEM_S = 0, TMEM_O = HG * TP; // phase 3: S of head hi at hi * 80, O of head hi at 320 + hi * 48
static_assert(HG * TP + HG * DP <= 512 && MAX_GROUPS * NQ <= 512, "TMEM budget");

struct LayerArgs {
    const void* wq;             // packed [C][C] (single problem)
    const void* wout;           // packed [C][C] with bias (layer variant, single problem)
    const void* kv;             // blocks [B] (single problem)
    const taq_request* reqs;    // nullable; then one sequence per request
    __half* o;                  // [z][N][C]  (query-attention variant)
    const void* q;              // attention-only variant: Q~ codes (int8) or Q (fp16) [z][N][C] ...
    const float* q_scales;      // ... and the row scales [z][N][H] (q_bits = 8)
    int n_query, heads, n_ctx, max_trigger, group, q_bits, p_bits;
    long long wait_cycles;      // limit of every device-side wait
    int* status;
};

// The same by the first NT worker threads only (phase 4: the warps of the last head, whose probabilities are the last to
// be complete, take no part, so that the tiles do not wait for them).
template <int NT>
__device__ __forceinline__ void expand_block_by(const unsigned char* raw, int kb, unsigned char* b_tile, int t) {
    constexpr int NCH = (NQ * 8 + NT - 1) / NT;
    uint32_t pw[NCH];
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int id = t + NT * i;
        pw[i] = 0;
        if (id < NQ * 8) pw[i] = *reinterpret_cast<const uint32_t*>(raw + (id >> 3) * (KIN / 2) + kb * (BK / 2) + (id & 7) * 4);
    }
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        const int id = t + NT * i;
        if (id < NQ * 8) *reinterpret_cast<uint4*>(b_tile + ptx::sw128_offset(id >> 3, id & 7)) = codes_w4_to_half(pw[i]);
    }
}

// Expands one 64-wide K block of the packed 4-bit codes at OFF_RAW into a tile of fp16 integers (all worker threads).
__device__ __forceinline__ void expand_block(const unsigned char* raw, int kb, unsigned char* b_tile, int wt) {
    constexpr int NCH = (NQ * 8 + NWORK - 1) / NWORK;       // 16-byte chunks (8 weights) per thread
    const int n0 = wt >> 3, c = wt & 7;
    uint32_t pw[NCH];
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
        pw[i] = 0;
        if (n0 + (NWORK / 8) * i < NQ) pw[i] = *reinterpret_cast<const uint32_t*>(raw + (n0 + (NWORK / 8) * i) * (KIN / 2) + kb * (BK / 2) + c * 4);
    }
#pragma unroll
    for (int i = 0; i < NCH; ++i)
        if (n0 + (NWORK / 8) * i < NQ) *reinterpret_cast<uint4*>(b_tile + ptx::sw128_offset(n0 + (NWORK / 8) * i, c)) = codes_w4_to_half(pw[i]);
}

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// The softmax of one thread's row over all TP keys: raw scores u (integer dot products) -> e_j = 2^(u_j f_j sq - m)
// with the row's own maximum m (log2 units); returns their sum.  Keys at or beyond T get weight exactly 0.
// The softmax of one thread's row over all TP keys: raw scores u (integer dot products) -> e_j = 2^(u_j f_j sq - m)
// with the row's own maximum m (log2 units); returns their sum.  Keys at or beyond T get weight exactly 0; only keys from
// TAIL_FROM on can be such keys (the launcher picks TAIL_FROM <= T).
template <int TAIL_FROM>
__device__ __forceinline__ float softmax_row(const uint32_t (&u)[TP], float (&e)[TP], const float* factor, float sq, int T, float& msq_out) {
    float m4[4] = {-1e30f, -1e30f, -1e30f, -1e30f};          // finite floor
#pragma unroll
    for (int j8 = 0; j8 < TP / 8; ++j8) {
        const float4 f0 = *reinterpret_cast<const float4*>(factor + 8 * j8), f1 = *reinterpret_cast<const float4*>(factor + 8 * j8 + 4);
        const float f[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int j = 8 * j8 + i;
            e[j] = __uint_as_float(u[j]) * f[i];
            if (j >= TAIL_FROM) { if (j >= T) e[j] = -INFINITY; }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) m4[i] = max3(m4[i], e[8 * j8 + i], e[8 * j8 + 4 + i]);
    }
    const float msq = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3])) * sq;
    msq_out = msq;
    // all exponentials first, then the sums: the special-function unit's latency is hidden behind the next arguments
#pragma unroll
    for (int j = 0; j < TP; ++j) {
        float arg = fmaf(e[j], sq, -msq);
        if (j >= TAIL_FROM) { if (j >= T) arg = -INFINITY; }      // also when sq = 0
        e[j] = ex2_approx(arg);
    }
    float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int j = 0; j < TP; ++j) sum4[j & 3] += e[j];
    return (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
}

// Eq. 3, ordinary columns, on the row's TP probabilities e_j * k (units of 1 / pmax): rint (ties to even).
// fma(e, k, 1.5 * 2^23 + 0x6400) leaves the integer code in the low byte and 0x64 above it, which read as fp16 is
// 1024 + code.  Keys 0..63 go to the 128-byte-swizzled tile, keys 64..79 to the 32-byte-swizzled one.  (Trigger columns
// are overwritten afterwards, see trigger_columns.)
__device__ __forceinline__ void write_p_row(const float (&e)[TP], float k, unsigned char* p_tile, unsigned char* p_tail, int r) {
    const __half2 h1024 = __floats2half2_rn(1024.f, 1024.f);
#pragma unroll
    for (int g = 0; g < TP / 8; ++g) {
        uint32_t pk[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = g * 8 + 2 * i;
            const uint32_t x0 = __float_as_uint(fmaf(e[j], k, 12608512.0f));
            const uint32_t x1 = __float_as_uint(fmaf(e[j + 1], k, 12608512.0f));
            uint32_t w = __byte_perm(x0, x1, 0x5410);
            __half2 hv = __hsub2(*reinterpret_cast<__half2*>(&w), h1024);
            pk[i] = *reinterpret_cast<uint32_t*>(&hv);
        }
        unsigned char* dst = g < 8 ? p_tile + ptx::sw128_offset(r, g) : p_tail + ptx::sw32_offset(r, g - 8);
        *reinterpret_cast<uint4*>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
}

// Eq. 3, trigger columns: the probability stays fp16, fp16(e_j k).  A row has at most a few of them, at positions only
// known at run time, so they are not carried through the unrolled code above: e_j is computed once more from the score
// in TMEM with the same instructions (hence the same value) and the two bytes of the code are overwritten.  Up to four
// columns are fetched per round trip to TMEM.  The loop is warp-uniform (`trig` is the same for all rows of a head).
__device__ __forceinline__ void trigger_columns(const uint32_t (&trig)[3], uint32_t t_s, const float* factor, float sq, float msq, float k,
                                                unsigned char* p_tile, unsigned char* p_tail, int r) {
#pragma unroll 1
    for (int w = 0; w < 3; ++w) {
        uint32_t bits = trig[w];
        while (bits) {
            int jj[4];
            uint32_t v[4];
            int n = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                jj[i] = 0;
                if (bits) {
                    const int j = w * 32 + __ffs(bits) - 1;
                    bits &= bits - 1;
                    if (j < TP) { jj[i] = j; n = i + 1; }
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (i < n) v[i] = ptx::tmem_ld1(t_s + jj[i]);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (i < n) {
                    const int j = jj[i];
                    asm volatile("" : "+r"(v[i]));
                    const float t = __uint_as_float(v[i]) * factor[j];
                    const float ej = ex2_approx(fmaf(t, sq, -msq));
                    unsigned char* dst = j < 64 ? p_tile + ptx::sw128_offset(r, j >> 3) : p_tail + ptx::sw32_offset(r, (j - 64) >> 3);
                    *reinterpret_cast<__half*>(dst + (j & 7) * 2) = __float2half_rn(ej * k);
                }
        }
    }
}

// The walk of phase 4 over the five 64-wide K blocks of O: each CTA starts with the channels of its own heads.
//   rank 0: blocks 0, 1, first half of 2 | second half of 2, 3, 4        rank 1: second half of 2, 3, 4 | first half of 2, 1, 0
// Step i of six: K block, which 32-channel halves, and (walk_tile) the order in which the Wout tiles are needed.
__host__ __device__ constexpr int walk_block(int rank, int i) { return rank ? (i < 3 ? 2 + i : 5 - i) : (i < 3 ? i : i - 1); }
__host__ __device__ constexpr int walk_halves(int rank, int i) { return i == 2 - 2 * rank ? (rank ? 2 : 1) : i == 3 ? (rank ? 1 : 2) : 3; }     // bit 0: first half, bit 1: second half
__host__ __device__ constexpr int walk_tile(int rank, int n) { return rank ? (n < 3 ? 2 + n : 4 - n) : n; }            // n-th Wout tile to expand
// Ring stage of a K block's Wout tile: the first four tiles of the walk take stages 0..3, the fifth reuses the stage of a
// tile whose last use comes early (rank 0: block 0, stage 0; rank 1: block 3, stage 1).
__host__ __device__ constexpr int walk_stage(int rank, int kb) { return rank ? (kb >= 2 ? kb - 2 : kb == 1 ? 3 : 1) : (kb < 4 ? kb : 0); }
__host__ __device__ constexpr int walk_reuse_stage(int rank) { return rank ? 1 : 0; }
__host__ __device__ constexpr int walk_order(int rank, int kb) { return rank ? (kb >= 2 ? kb - 2 : 4 - kb) : kb; }        // inverse of walk_tile

// Q_IN: the attention-only variant (taq_cross_attention at this shape): Q~ is given, phases 1 and 4 do not exist; the
// thread reads its 40 query codes from global memory instead of quantizing them.
template <int TAIL_FROM, bool FUSE_OUT, bool Q_IN = false>
__global__ void __launch_bounds__(NTHREADS, 1) layer_c320_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_y, const LayerArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_u32(smem_dyn) & 1023u)) & 1023u);   // 1024-byte aligned
    Misc* misc = reinterpret_cast<Misc*>(smem + OFF_MISC);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = a.n_ctx, H = a.heads;
    const int zb = blockIdx.z;                      // sequence (batch entry or request)
    const int row0 = blockIdx.x * ROWS;
    const int rank = blockIdx.y;                    // which half of the heads; also the CTA's rank in its cluster
    const int h_begin = rank * HG;
    const int col0 = h_begin * D;
    const WeightLayout L = weight_layout(KIN, KIN, 4, a.group);
    const int n_groups = L.n_groups;
    const int kb_per_group = L.group_len / BK;
    const long long WL = a.wait_cycles;

    TAQ_PROF_INIT
    if (tid == 0) { TAQ_PROF(0); TAQ_GPROF(30); }
    if (tid == 0) {
        for (int i = 0; i < NKB; ++i) { ptx::mbar_init(&misc->a_full[i], 1); ptx::mbar_init(&misc->b1_full[i], NWORK / 32); }
        ptx::mbar_init(&misc->w_full, 1);
        ptx::mbar_init(&misc->w2_full, 1);
        ptx::mbar_init(&misc->kc_full, 1);
        ptx::mbar_init(&misc->vt_full, 1);
        for (int i = 0; i < NKB; ++i) ptx::mbar_init(&misc->b4_full[i], NEXP / 32);
        for (int i = 0; i < NS4; ++i) ptx::mbar_init(&misc->b4_empty[i], 1);
        for (int i = 0; i < MAX_GROUPS; ++i) ptx::mbar_init(&misc->acc_full[i], 1);
        ptx::mbar_init(&misc->q_all, NWORK / 32);
        for (int i = 0; i < HG; ++i) {
            ptx::mbar_init(&misc->s_full[i], 1);
            ptx::mbar_init(&misc->p_full[i], NWORK / 32 / HG);     // the four warps of the head
            ptx::mbar_init(&misc->o_full[i], 1);
        }
        for (int lt = 0; lt < N_OTILE / 2; ++lt)                   // the warps of the one or two heads that write the tile
            ptx::mbar_init(&misc->tile_done[lt], (lt == 0 || lt == HG ? 1 : 2) * (NWORK / 32 / HG));
        ptx::mbar_init(&misc->o_all, 1);
        ptx::mbar_init(&misc->peer_ready, 1);
        ptx::mbar_init(&misc->peer_got, 1);
        ptx::mbar_init(&misc->drain, 1);
        misc->abort_flag = 0;
        ptx::mbar_fence_init();
        if (FUSE_OUT) ptx::mbar_arrive_expect_tx(&misc->o_all, (N_OTILE / 2) * O_TILE);     // the partner's five tiles
        ptx::tma_prefetch_desc(&tmap_x);
        ptx::tma_prefetch_desc(&tmap_y);
    }
    if (warp == 1) ptx::tmem_alloc(&misc->tmem_base, TMEM_COLS);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = misc->tmem_base;
    ptx::pdl_trigger();
    // The partner's barriers must exist before anything arrives on them.  Every thread arrives at the cluster barrier
    // here and waits on it much later, right before its warp's first operation on the partner's shared memory (or at
    // the end), so that the barrier's latency stays off the start of the kernel.
    if (FUSE_OUT) ptx::cluster_arrive();
    const uint32_t peer = FUSE_OUT ? (ptx::cluster_ctarank() ^ 1u) : 0u;

    const taq_kv_layout KL = kv_layout(H, T, D, a.max_trigger);
    auto give_up = [&]() { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; };

    if (warp == 0) {
        // ---------------- producer ----------------
        if (lane == 0) {
            // Packed weights are written by taq_pack_weights, which never lets its successor start early: they are complete
            // before this kernel can run at all and are fetched (and expanded) under the previous kernel's tail.
            const uint32_t scale_bytes = (uint32_t)(NQ * n_groups * 4);
            if (!Q_IN) {
                const uint8_t* blob = (const uint8_t*)(a.reqs ? a.reqs[zb].Wq : a.wq);
                ptx::mbar_arrive_expect_tx(&misc->w_full, RAW_BYTES + scale_bytes);
                ptx::bulk_load(smem + OFF_RAW, blob + L.off_codes + (size_t)col0 * L.row_bytes, RAW_BYTES, &misc->w_full);
                ptx::bulk_load(smem + OFF_SC, blob + L.off_scales + (size_t)col0 * n_groups * 4, scale_bytes, &misc->w_full);
            }
            ptx::pdl_wait();                              // X and the K~/V~ block may come from the previous kernel
            TAQ_PROF(1); TAQ_GPROF(28);
            for (int kb = 0; kb < NKB && !Q_IN; ++kb) {   // the whole X tile at once: every K block has its own buffer
                ptx::mbar_arrive_expect_tx(&misc->a_full[kb], A_TILE);
                ptx::tma_load_3d(smem + OFF_R0 + kb * A_TILE, &tmap_x, &misc->a_full[kb], kb * BK, row0, zb);
            }
            const uint8_t* blk = a.reqs ? (const uint8_t*)a.reqs[zb].kv : (const uint8_t*)a.kv + (size_t)zb * KL.block_bytes;
            const uint8_t* img = blk + KL.off_operands + (size_t)h_begin * KL.operand_head_bytes;
            // Phase 1 over (every MMA complete, hence every Wq tile read): the weight tiles become the K~ and V~^T tiles and
            // the packed Wout rows of this CTA's output channels replace the packed Wq rows.
            bool ok = Q_IN || (ptx::mbar_wait(&misc->acc_full[n_groups - 1], 0, WL) && !misc->abort_flag);
            if (ok) {
                ptx::mbar_arrive_expect_tx(&misc->kc_full, HG * (K_BYTES + kOperandConstBytes));
                for (int hi = 0; hi < HG; ++hi) {
                    ptx::bulk_load(smem + OFF_K + hi * K_BYTES, img + (size_t)hi * KL.operand_head_bytes, K_BYTES, &misc->kc_full);
                    ptx::bulk_load(smem + OFF_CST + hi * kOperandConstBytes, img + (size_t)hi * KL.operand_head_bytes + K_BYTES + VT_BYTES, kOperandConstBytes, &misc->kc_full);
                }
                ptx::mbar_arrive_expect_tx(&misc->vt_full, HG * VT_BYTES);
                for (int hi = 0; hi < HG; ++hi)
                    ptx::bulk_load(smem + OFF_R1 + hi * VT_BYTES, img + (size_t)hi * KL.operand_head_bytes + K_BYTES, VT_BYTES, &misc->vt_full);
                if (FUSE_OUT) {
                    const uint8_t* blob2 = (const uint8_t*)(a.reqs ? a.reqs[zb].Wout : a.wout);
                    ptx::mbar_arrive_expect_tx(&misc->w2_full, RAW_BYTES + scale_bytes + NQ * 4);
                    ptx::bulk_load(smem + OFF_RAW, blob2 + L.off_codes + (size_t)col0 * L.row_bytes, RAW_BYTES, &misc->w2_full);
                    ptx::bulk_load(smem + OFF_SC, blob2 + L.off_scales + (size_t)col0 * n_groups * 4, scale_bytes, &misc->w2_full);
                    ptx::bulk_load(smem + OFF_BIAS, blob2 + L.off_bias + (size_t)col0 * 4, NQ * 4, &misc->w2_full);
                }
            }
            if (!ok) give_up();
        }
        if (FUSE_OUT) {
            __syncwarp();
            ptx::cluster_wait();                              // the partner's barriers exist
            if (lane == 0 && !misc->abort_flag) {
                // Every PV product of this CTA is complete when the last one is: its probability tiles may receive the
                // partner's O.  Then this CTA's five O tiles go to the partner, each as soon as the heads that write it
                // have stored their parts and the partner has announced the same about its probability tiles; the copies
                // complete on the partner's o_all barrier.
                bool ok = ptx::mbar_wait(&misc->o_full[HG - 1], 0, WL) && !misc->abort_flag;
                if (ok) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(ptx::smem_u32(&misc->peer_ready), peer));
                ok = ok && ptx::mbar_wait(&misc->peer_ready, 0, WL);
                for (int lt = 0; lt < N_OTILE / 2 && ok; ++lt) {
                    ok = ptx::mbar_wait(&misc->tile_done[lt], 0, WL) && !misc->abort_flag;
                    if (!ok) break;
                    unsigned char* mine = smem + own_tile_offset(lt);
                    ptx::bulk_copy_to_cta(ptx::map_to_cta(ptx::smem_u32(smem + peer_tile_offset(lt)), peer), mine, (uint32_t)O_TILE,
                                          ptx::map_to_cta(ptx::smem_u32(&misc->o_all), peer));
                    if (lt == 0) TAQ_PROF(57);
                }
                if (!ok) give_up();
            }
        }
        if (lane == 0 && misc->abort_flag) {   // give copies that are still in flight a bounded chance to land before the CTA exits
            if (!Q_IN) (void)ptx::mbar_wait(&misc->w_full, 0, WL);
            for (int kb = 0; kb < NKB && !Q_IN; ++kb) (void)ptx::mbar_wait(&misc->a_full[kb], 0, WL);
            // (the image and Wout copies are issued only after phase 1 succeeded; when they were, these waits end with them)
            if (Q_IN || ptx::mbar_try_wait(&misc->acc_full[n_groups - 1], 0)) {
                (void)ptx::mbar_wait(&misc->kc_full, 0, WL);
                (void)ptx::mbar_wait(&misc->vt_full, 0, WL);
                if (FUSE_OUT) (void)ptx::mbar_wait(&misc->w2_full, 0, WL);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // All 32 lanes walk the control flow (waits, loop state and descriptor words stay warp-uniform); one elected lane
        // issues the MMAs and commits.  Its waits are bounded but do not poll the abort flag: the path between two MMAs is
        // kept as short as possible.
        const bool leader = ptx::elect_one();
        bool ok = true;
        auto wait = [&](uint64_t* bar, uint32_t parity) -> bool { return __all_sync(0xffffffffu, ptx::mbar_wait(bar, parity, WL)) != 0; };
        constexpr uint32_t idesc = ptx::idesc_f16_m128(NQ);
        constexpr uint32_t HI128 = ptx::kDescHiSw128, HI64 = ptx::kDescHiSw64, HI32 = ptx::kDescHiSw32;
        const uint32_t r0_lo = ptx::desc_lo(ptx::smem_u32(smem + OFF_R0)), r1_lo = ptx::desc_lo(ptx::smem_u32(smem + OFF_R1));
        const uint32_t pb_lo = ptx::desc_lo(ptx::smem_u32(smem + OFF_PB)), k_lo = ptx::desc_lo(ptx::smem_u32(smem + OFF_K));
        if (!Q_IN) {   // phase 1: one accumulation pass per scale group; every weight tile was expanded before X arrived
            int kb = 0;
            for (int g = 0; g < n_groups && ok; ++g) {
                const int kb_end = min(NKB, kb + kb_per_group);
                for (bool first = true; kb < kb_end && ok; ++kb) {
                    if (!wait(&misc->b1_full[kb], 0) || !wait(&misc->a_full[kb], 0)) { ok = false; break; }
                    if (leader) {
                        TAQ_PROF(2 + kb);
                        const uint32_t a_lo = r0_lo + kb * (A_TILE >> 4), b_lo = ptx::desc_lo(ptx::smem_u32(smem + stage1_offset(kb)));
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            ptx::mma_f16_ss(tmem_base + TMEM_ACC + g * NQ, ptx::desc_join(HI128, a_lo + 2 * k), ptx::desc_join(HI128, b_lo + 2 * k), idesc, !(first && k == 0));
                        if (kb + 1 == kb_end) ptx::mma_commit(&misc->acc_full[g]);
                    }
                    first = false;
                }
            }
        }
        // phase 3: the Q~ tiles of all four heads are in place once every worker warp has arrived (their reads of the
        // phase-1 accumulators, whose columns S and O reuse, are ordered before that arrival)
        ok = ok && wait(&misc->kc_full, 0) && wait(&misc->q_all, 0);
        ptx::tc_fence_after_sync();
        if (ok && leader) {
            TAQ_PROF(10);
#pragma unroll
            for (int hi = 0; hi < HG; ++hi) {
                const uint32_t q_lo = r0_lo + hi * (A_TILE >> 4), kh_lo = k_lo + hi * (K_BYTES >> 4);
#pragma unroll
                for (int ks = 0; ks < DP / 16; ++ks)
                    ptx::mma_f16_ss(tmem_base + TMEM_S + hi * TP, ptx::desc_join(HI128, q_lo + 2 * ks), ptx::desc_join(HI128, kh_lo + 2 * ks), ptx::idesc_f16_m128(TP), ks != 0);
                ptx::mma_commit(&misc->s_full[hi]);
            }
        }
        ok = ok && wait(&misc->vt_full, 0);
        for (int hi = 0; hi < HG && ok; ++hi) {
            if (!wait(&misc->p_full[hi], 0)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            if (leader) {
                TAQ_PROF(11 + hi);
                const uint32_t p_lo = r0_lo + hi * (A_TILE >> 4), pt_lo = pb_lo + hi * (PB_TILE >> 4), v_lo = r1_lo + hi * (VT_BYTES >> 4);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    ptx::mma_f16_ss(tmem_base + TMEM_O + hi * DP, ptx::desc_join(HI128, p_lo + 2 * ks), ptx::desc_join(HI128, v_lo + 2 * ks), ptx::idesc_f16_m128(DP), ks != 0);
                ptx::mma_f16_ss(tmem_base + TMEM_O + hi * DP, ptx::desc_join(HI32, pt_lo), ptx::desc_join(HI128, v_lo + (VT_BLOCK >> 4)), ptx::idesc_f16_m128(DP), true);
                ptx::mma_commit(&misc->o_full[hi]);
            }
        }
        if (FUSE_OUT) {
            ptx::cluster_wait();                          // the partner's barriers exist (peer_got below)
            // phase 4: Y = O Wout^T for this CTA's 160 output channels, in six steps (see walk_block): three over this CTA's
            // own O tiles, each as soon as the heads that write its tiles have stored them, then three over the partner's.
            // The accumulators reuse the columns of S (all read long ago) and, for the third scale group, of O: both
            // CTAs reach that group only after waiting for all five of their own tiles, i.e. for every head's reads of O.
            // The walk is unrolled per rank so that tile addresses, stages and parities are constants: between two MMAs
            // this warp, which shares its scheduler with four worker warps, should have as few instructions as possible.
            auto phase4 = [&](auto rank_c) {
                constexpr int R = decltype(rank_c)::value;
                uint32_t first_mask = 0, last_mask = 0, seen = 0;       // bit i: walk step i begins / completes a scale group
#pragma unroll
                for (int i = 0; i < 6; ++i) {
                    const int g = walk_block(R, i) / kb_per_group;
                    if (!((seen >> g) & 1u)) first_mask |= 1u << i;
                    seen |= 1u << g;
                }
                seen = 0;
#pragma unroll
                for (int i = 5; i >= 0; --i) {
                    const int g = walk_block(R, i) / kb_per_group;
                    if (!((seen >> g) & 1u)) last_mask |= 1u << i;
                    seen |= 1u << g;
                }
                // this CTA's own five O tiles: every head has stored its part (and read its O accumulator)
#pragma unroll
                for (int lt = 0; lt < N_OTILE / 2; ++lt) ok = ok && wait(&misc->tile_done[lt], 0);
                ptx::tc_fence_after_sync();
#pragma unroll
                for (int i = 0; i < 6; ++i) {
                    const int kb = walk_block(R, i), halves = walk_halves(R, i), st = walk_stage(R, kb);
                    const int g = kb / kb_per_group;
                    if (i == 3) {
                        ok = ok && wait(&misc->o_all, 0);
                        // the partner's copies have landed: it may leave without waiting for this CTA any longer
                        if (ok && leader) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(ptx::smem_u32(&misc->peer_got), peer));
                        if (leader) TAQ_PROF(38);
                    } else {
                        // (block 2 returns at step 3 with the tile it already has)
                        ok = ok && wait(&misc->b4_full[walk_order(R, kb)], 0);
                    }
                    if (ok && leader) {
                        TAQ_PROF(40 + i);
                        const uint32_t b_lo = ptx::desc_lo(ptx::smem_u32(smem + stage4_offset(st)));
                        bool acc = !((first_mask >> i) & 1u);
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) {
                            if (!((halves >> hf) & 1)) continue;
                            const int t = 2 * kb + hf;                      // O tile (32 channels) of this half
                            const int off = (t / (N_OTILE / 2)) == R ? own_tile_offset(t % (N_OTILE / 2)) : peer_tile_offset(t % (N_OTILE / 2));
                            const uint32_t o_lo = ptx::desc_lo(ptx::smem_u32(smem + off));
#pragma unroll
                            for (int k = 0; k < 2; ++k) {
                                ptx::mma_f16_ss(tmem_base + TMEM_ACC + g * NQ, ptx::desc_join(HI64, o_lo + 2 * k), ptx::desc_join(HI128, b_lo + 4 * hf + 2 * k), idesc, acc);
                                acc = true;
                            }
                        }
                        if (st == walk_reuse_stage(R) && kb != walk_tile(R, NKB - 1)) ptx::mma_commit(&misc->b4_empty[st]);
                        if ((last_mask >> i) & 1u) ptx::mma_commit(&misc->acc_full[g]);
                    }
                }
            };
            if (rank == 0) phase4(std::integral_constant<int, 0>{}); else phase4(std::integral_constant<int, 1>{});
        }
        if (!ok) {
            if (leader) {
                give_up();
                ptx::mma_commit(&misc->drain);               // wait (bounded) for whatever was issued before TMEM is given back
            }
            (void)ptx::mbar_wait(&misc->drain, 0, WL);
        }
    } else {
        // ---------------- workers (warps 2..17): thread = (row r, head hi) ----------------
        const int wt = tid - 64;
        const int q4 = warp & 3, hi = (warp - 2) >> 2;       // TMEM lane quarter; head
        const int r = q4 * 32 + lane;
        const int n = row0 + r;
        const bool valid = n < a.n_query;
        const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
        const float* wscales = reinterpret_cast<const float*>(smem + OFF_SC);
        float* scales_t = reinterpret_cast<float*>(smem + OFF_SCT);
        const unsigned char* raw = smem + OFF_RAW;
        const int cb = hi * D;
        bool ok = true;
        if (!Q_IN) {
            ok = ptx::mbar_wait(&misc->w_full, 0, WL);
            for (int i = wt; i < NQ * n_groups; i += NWORK) scales_t[(i % n_groups) * NQ + i / n_groups] = wscales[i];
            asm volatile("bar.sync 1, 512;" ::: "memory");
        }

        auto tile_built = [&](uint64_t* bar) {
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(bar);
        };
        float y[D];
        // y += scale[g] * accumulator g for this thread's 40 channels, group by group in the given order
        auto fold_groups = [&](uint32_t parity, bool descending) {
#pragma unroll
            for (int c = 0; c < D; ++c) y[c] = 0.f;
            for (int gi = 0; gi < n_groups && ok; ++gi) {
                const int g = descending ? n_groups - 1 - gi : gi;
                ok = ptx::mbar_wait(&misc->acc_full[g], parity, WL) && !misc->abort_flag;
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const float* sg = scales_t + g * NQ + cb;
                const uint32_t taddr = tmem_base + TMEM_ACC + g * NQ + cb + lane_addr;
                uint32_t v[5][8];
#pragma unroll
                for (int i = 0; i < 5; ++i) ptx::tmem_ld8(taddr + i * 8, v[i]);
                ptx::tmem_ld_wait(v[0]);
#pragma unroll
                for (int i = 1; i < 5; ++i) ptx::reg_fence8(v[i]);
#pragma unroll
                for (int i = 0; i < 5; ++i) {
                    const float4 s0 = *reinterpret_cast<const float4*>(sg + i * 8), s1 = *reinterpret_cast<const float4*>(sg + i * 8 + 4);
                    float* yy = y + i * 8;
                    yy[0] = fmaf(__uint_as_float(v[i][0]), s0.x, yy[0]); yy[1] = fmaf(__uint_as_float(v[i][1]), s0.y, yy[1]);
                    yy[2] = fmaf(__uint_as_float(v[i][2]), s0.z, yy[2]); yy[3] = fmaf(__uint_as_float(v[i][3]), s0.w, yy[3]);
                    yy[4] = fmaf(__uint_as_float(v[i][4]), s1.x, yy[4]); yy[5] = fmaf(__uint_as_float(v[i][5]), s1.y, yy[5]);
                    yy[6] = fmaf(__uint_as_float(v[i][6]), s1.z, yy[6]); yy[7] = fmaf(__uint_as_float(v[i][7]), s1.w, yy[7]);
                }
            }
            ptx::tc_fence_before_sync();
        };

        // ---- phase 1: expand all five Wq tiles (before X has arrived), then fold ----
        if (!Q_IN) {
            for (int kb = 0; kb < NKB; ++kb) {
                if (ok) expand_block(raw, kb, smem + stage1_offset(kb), wt);
                tile_built(&misc->b1_full[kb]);
            }
            fold_groups(0, false);
        }
        if (!ok) give_up();
        if (wt == 0) TAQ_PROF(7);
        // The last group's accumulator is complete, hence every MMA of phase 1 has finished reading shared memory: the
        // X tile may be overwritten without a barrier.

        // ---- phase 2: Q~ = Q_a(Q) of (row, head), written as fp16 integers into the head's operand tile ----
        float sq = 0.f;
        if (Q_IN) {
            // attention only: the row's 40 codes (or fp16 values) of this head come from global memory
            ptx::pdl_wait();                                  // Q~ comes from the previous kernel in the stream
            unsigned char* q_tile = smem + OFF_R0 + hi * A_TILE;
            const size_t grow = (size_t)zb * a.n_query + (valid ? n : 0);
            const size_t elem = grow * (size_t)(H * D) + (size_t)(h_begin + hi) * D;
            // all loads first (read-only path), then the conversions and the stores: one round trip to L2, not five
            uint4 t16[D / 8];
            if (a.q_bits == 8) {
                uint2 c8[D / 8];
#pragma unroll
                for (int cc = 0; cc < D / 8; ++cc)
                    c8[cc] = valid ? __ldg(reinterpret_cast<const uint2*>((const int8_t*)a.q + elem + cc * 8)) : make_uint2(0, 0);
#pragma unroll
                for (int cc = 0; cc < D / 8; ++cc) t16[cc] = codes_w8_to_half(c8[cc]);
            } else {
#pragma unroll
                for (int cc = 0; cc < D / 8; ++cc)
                    t16[cc] = valid ? __ldg(reinterpret_cast<const uint4*>((const __half*)a.q + elem + cc * 8)) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int cc = 0; cc < D / 8; ++cc) *reinterpret_cast<uint4*>(q_tile + ptx::sw128_offset(r, cc)) = t16[cc];
            *reinterpret_cast<uint4*>(q_tile + ptx::sw128_offset(r, D / 8)) = make_uint4(0, 0, 0, 0);   // channels 40..47
            sq = a.q_bits == 8 ? (valid ? __ldg(a.q_scales + grow * H + h_begin + hi) : 0.f) : 1.0f;
        } else {
            float amax = 0.f;
#pragma unroll
            for (int c = 0; c < D; c += 2) amax = max3(amax, fabsf(y[c]), fabsf(y[c + 1]));
            unsigned char* q_tile = smem + OFF_R0 + hi * A_TILE;
            if (a.q_bits == 8) {
                const float sc = quant_scale(amax, 127.f);
                const float rs = sc > 0.f ? __frcp_rn(sc) : 0.f;
                // fma(x, 1/s, 1.5 * 2^23 + 0x6480): the low half-word read as fp16 is 1152 + code
                const __half2 h1152 = __floats2half2_rn(1152.f, 1152.f);
#pragma unroll
                for (int cc = 0; cc < D / 8; ++cc) {
                    uint32_t pk[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t x0 = __float_as_uint(fmaf(y[cc * 8 + 2 * i], rs, 12608640.0f));
                        const uint32_t x1 = __float_as_uint(fmaf(y[cc * 8 + 2 * i + 1], rs, 12608640.0f));
                        uint32_t w = __byte_perm(x0, x1, 0x5410);
                        __half2 hv = __hsub2(*reinterpret_cast<__half2*>(&w), h1152);
                        pk[i] = *reinterpret_cast<uint32_t*>(&hv);
                    }
                    *reinterpret_cast<uint4*>(q_tile + ptx::sw128_offset(r, cc)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
                sq = valid ? sc : 0.f;
            } else {                                    // Q stays fp16
#pragma unroll
                for (int cc = 0; cc < D / 8; ++cc) {
                    float f[8];
#pragma unroll
                    for (int e2 = 0; e2 < 8; ++e2) f[e2] = y[cc * 8 + e2];
                    *reinterpret_cast<uint4*>(q_tile + ptx::sw128_offset(r, cc)) = pack8(f);
                }
                sq = 1.0f;
            }
            *reinterpret_cast<uint4*>(q_tile + ptx::sw128_offset(r, D / 8)) = make_uint4(0, 0, 0, 0);   // channels 40..47
        }
        tile_built(&misc->q_all);
        if (wt == 0) TAQ_PROF(8);

        // ---- phase 3: the 80 scores of (row, head): softmax, Eq. 3, P ----
        ok = ok && ptx::mbar_wait(&misc->kc_full, 0, WL) && ptx::mbar_wait(&misc->s_full[hi], 0, WL) && !misc->abort_flag;
        if (lane == 0 && q4 == 0) TAQ_PROF(16 + hi);           // S seen
        const float pmax = a.p_bits == 4 ? 15.0f : 255.0f;     // probabilities are held in units of 1 / pmax (uint8 or 4-bit codes)
        if (ok) {
            ptx::tc_fence_after_sync();
            float e[TP];
            uint32_t u[TP];
            const uint32_t t_s = tmem_base + TMEM_S + hi * TP + lane_addr;
            {
                uint32_t (&u8)[TP / 8][8] = *reinterpret_cast<uint32_t (*)[TP / 8][8]>(&u);
#pragma unroll
                for (int i = 0; i < TP / 8; ++i) ptx::tmem_ld8(t_s + i * 8, u8[i]);
                ptx::tmem_ld_wait(u8[0]);
#pragma unroll
                for (int i = 1; i < TP / 8; ++i) ptx::reg_fence8(u8[i]);
            }
            const OperandConsts* cst = reinterpret_cast<const OperandConsts*>(smem + OFF_CST + hi * kOperandConstBytes);
            float msq;
            const float l = softmax_row<TAIL_FROM>(u, e, cst->logit_factor, sq, T, msq);
            const float k255 = __fdividef(pmax, l);
            const uint32_t trig[3] = {cst->trig_bits[0], cst->trig_bits[1], cst->trig_bits[2]};
            write_p_row(e, k255, smem + OFF_R0 + hi * A_TILE, smem + OFF_PB + hi * PB_TILE, r);
            trigger_columns(trig, t_s, cst->logit_factor, sq, msq, k255, smem + OFF_R0 + hi * A_TILE, smem + OFF_PB + hi * PB_TILE, r);
        }
        ptx::tc_fence_before_sync();
        tile_built(&misc->p_full[hi]);
        if (lane == 0 && q4 == 0) TAQ_PROF(24 + hi);           // P written

        if (FUSE_OUT) {
            // The first Wout tile of the walk goes into a K~ buffer (dead once every S product is complete) while this
            // head's PV product runs; the second follows after the head's O has been stored.  The warps of the last head,
            // whose probabilities are the last to be complete, take no part in the expansion.
            ok = ok && ptx::mbar_wait(&misc->s_full[HG - 1], 0, WL) && ptx::mbar_wait(&misc->w2_full, 0, WL) && !misc->abort_flag;
            for (int i = wt; i < NQ * n_groups; i += NWORK) scales_t[(i % n_groups) * NQ + i / n_groups] = wscales[i];     // (last read in phase 1)
            if (wt < NEXP) {
                if (ok) expand_block_by<NEXP>(raw, walk_tile(rank, 0), smem + stage4_offset(0), wt);
                tile_built(&misc->b4_full[0]);
            }
            if (wt == 0) TAQ_PROF(34);
        }

        // ---- O of (row, head): the accumulator in units of 1 / pmax -> fp16, as soon as this head's PV product is complete ----
        ok = ok && ptx::mbar_wait(&misc->o_full[hi], 0, WL) && !misc->abort_flag;
        if (ok) {
            ptx::tc_fence_after_sync();
            const float inv = 1.0f / pmax;
            const uint32_t t_o = tmem_base + TMEM_O + hi * DP + lane_addr;
            uint32_t v[D / 8][8];
#pragma unroll
            for (int i = 0; i < D / 8; ++i) ptx::tmem_ld8(t_o + i * 8, v[i]);
            ptx::tmem_ld_wait(v[0]);
#pragma unroll
            for (int i = 1; i < D / 8; ++i) ptx::reg_fence8(v[i]);
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                float f[8];
#pragma unroll
                for (int e2 = 0; e2 < 8; ++e2) f[e2] = __uint_as_float(v[i][e2]) * inv;
                const uint4 o8 = pack8(f);
                if (FUSE_OUT) {           // 8 channels of O as one chunk of the to_out operand tiles
                    const int c = hi * D + i * 8;                    // channel among this CTA's 160
                    *reinterpret_cast<uint4*>(smem + own_tile_offset(c >> 5) + ptx::sw64_offset(r, (c & 31) >> 3)) = o8;
                } else {                  // staged where the head's probability tile was (dead: its PV product is complete)
                    *reinterpret_cast<uint4*>(smem + OFF_R0 + hi * A_TILE + r * (D * 2) + i * 16) = o8;
                }
            }
        }
        ptx::tc_fence_before_sync();
        if (!FUSE_OUT) {
            // the head's 128 x 40 block of O leaves as one TMA tensor store (dense rows of 80 bytes; rows beyond n_query clipped)
            ptx::fence_proxy_async_smem();
            asm volatile("bar.sync %0, 128;" ::"r"(2 + hi) : "memory");
            if (q4 == 0 && lane == 0 && !misc->abort_flag) {
                ptx::tma_store_3d(&tmap_y, smem + OFF_R0 + hi * A_TILE, col0 + cb, row0, zb);
                ptx::bulk_store_commit();
                ptx::bulk_store_wait_read();
            }
        }

        if (FUSE_OUT) {
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) { ptx::mbar_arrive(&misc->tile_done[hi]); ptx::mbar_arrive(&misc->tile_done[hi + 1]); }      // head hi writes tiles hi and hi + 1
            if (wt == 0) TAQ_PROF(32);
            // ---- phase 4: the remaining Wout tiles (the V~^T buffers are dead once every PV product is complete), then fold ----
            if (wt < NEXP) {
                if (ok) expand_block_by<NEXP>(raw, walk_tile(rank, 1), smem + stage4_offset(1), wt);
                tile_built(&misc->b4_full[1]);
                ok = ok && ptx::mbar_wait(&misc->o_full[HG - 1], 0, WL) && !misc->abort_flag;
                for (int i = 2; i < NKB; ++i) {
                    const int s = i < NS4 ? i : walk_reuse_stage(rank);
                    if (i >= NS4 && ok) ok = ptx::mbar_wait(&misc->b4_empty[s], 0, WL) && !misc->abort_flag;
                    if (ok) expand_block_by<NEXP>(raw, walk_tile(rank, i), smem + stage4_offset(s), wt);
                    tile_built(&misc->b4_full[i]);
                }
            }
            if (wt == 0) TAQ_PROF(35);
            asm volatile("bar.sync 1, 512;" ::: "memory");       // the transposed scale table is complete
            fold_groups(1, rank != 0);
            if (wt == 0) TAQ_PROF(36);
            // Every MMA of phase 4 is complete, and the partner has received this CTA's O tiles (peer_got): region 0 is
            // free.  The head group's 128 x 40 block of Y is staged there as dense rows of 80 bytes (conflict-free for
            // row-per-lane 16-byte writes) and leaves as one TMA tensor store; rows beyond n_query are clipped.
            ok = ok && ptx::mbar_wait(&misc->peer_got, 0, WL) && !misc->abort_flag;
            if (!ok) give_up();
            unsigned char* stage = smem + OFF_R0 + hi * Y_STAGE;
            if (ok) {
                const float* bias = reinterpret_cast<const float*>(smem + OFF_BIAS) + cb;
#pragma unroll
                for (int c = 0; c < D; c += 8) {
                    float f[8];
#pragma unroll
                    for (int e2 = 0; e2 < 8; ++e2) f[e2] = y[c + e2] + bias[c + e2];
                    *reinterpret_cast<uint4*>(stage + r * (D * 2) + c * 2) = pack8(f);
                }
            }
            ptx::fence_proxy_async_smem();
            asm volatile("bar.sync %0, 128;" ::"r"(2 + hi) : "memory");
            if (q4 == 0 && lane == 0 && !misc->abort_flag) {
                ptx::tma_store_3d(&tmap_y, stage, col0 + cb, row0, zb);
                ptx::bulk_store_commit();
                ptx::bulk_store_wait_read();                     // shared memory is given back only after the store has read it
            }
            if (wt == 0) { TAQ_PROF(37); TAQ_GPROF(27); }
            ptx::cluster_wait();
        } else if (!ok) {
            give_up();
        }
    }

    // Neither CTA's shared memory may go away while the partner still writes to it or reads from it: each CTA has told
    // its partner (peer_got) that everything it expects from it has landed, and leaves only after hearing the same.
    if (FUSE_OUT && tid == 0 && !ptx::mbar_wait(&misc->peer_got, 0, WL)) raise_status(a.status, TAQ_ERR_TIMEOUT);
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) { TAQ_PROF(9); TAQ_GPROF(29); }
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

long long g_wait_cycles = ptx::kWaitCycles;

}  // namespace

void set_layer_wait_cycles(long long cycles) { g_wait_cycles = cycles > 0 ? cycles : ptx::kWaitCycles; }

bool sm100_layer_supported(const taq_layer_desc& d) { return sm100_qattn_supported(d); }

bool sm100_qattn_supported(const taq_layer_desc& d) {
    if (d.channels != KIN || d.heads * D != KIN) return false;
    if (d.w_bits != 4) return false;
    if (d.w_group != 0 && (d.w_group % BK || (KIN + d.w_group - 1) / d.w_group > MAX_GROUPS)) return false;
    if (d.n_ctx > TP || (d.p_bits != 8 && d.p_bits != 4) || d.p_log) return false;   // (logarithmic codes: the stand-alone attention kernel)
    if (d.n_query < 1) return false;
    return encode_tiled() != nullptr;
}

static cudaError_t launch_c320(const taq_layer_desc& d, const __half* x, const void* wq, const void* kv, const taq_request* reqs, __half* o,
                               const void* wout, __half* y, int n_z, int* status, cudaStream_t stream, const void* q = nullptr, const float* q_scales = nullptr) {
    if (n_z == 0 || d.n_query == 0) return cudaSuccess;
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return cudaErrorNotSupported;
    CUtensorMap tmap;
    const cuuint64_t dims[3] = {(cuuint64_t)KIN, (cuuint64_t)d.n_query, (cuuint64_t)n_z};
    const cuuint64_t strides[2] = {(cuuint64_t)KIN * 2, (cuuint64_t)KIN * 2 * (cuuint64_t)d.n_query};
    const cuuint32_t box[3] = {BK, ROWS, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const bool fuse_out = y != nullptr, q_in = q != nullptr;
    __half* out = fuse_out ? y : o;
    // (the attention-only variant loads no X: its map is built on the output so that the argument is a valid map)
    CUresult r = enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, q_in ? (void*)out : (void*)const_cast<__half*>(x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    LayerArgs a{};
    a.wq = wq; a.kv = kv; a.reqs = reqs; a.o = o; a.wout = wout; a.q = q; a.q_scales = q_scales;
    a.n_query = d.n_query; a.heads = d.heads; a.n_ctx = d.n_ctx; a.max_trigger = d.max_trigger; a.group = d.w_group; a.q_bits = d.q_bits; a.p_bits = d.p_bits;
    a.wait_cycles = g_wait_cycles;
    a.status = status;
    dim3 grid((d.n_query + ROWS - 1) / ROWS, d.heads / HG, n_z);
    const int tail = d.n_ctx > 72 ? 72 : d.n_ctx > 64 ? 64 : 0;     // first key that can lie beyond the context (the kernel masks from there on)
    CUtensorMap tmap_y;                               // the output (Y, or O of the variants without to_out), stored per head group
    {
        const cuuint32_t ybox[3] = {D, ROWS, 1};      // one head group: 40 channels = 80 bytes per row, dense in shared memory
        r = enc(&tmap_y, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, out, dims, strides, ybox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    void (*kern)(const CUtensorMap, const CUtensorMap, const LayerArgs) =
        q_in ? (tail == 72 ? layer_c320_kernel<72, false, true> : tail == 64 ? layer_c320_kernel<64, false, true> : layer_c320_kernel<0, false, true>) :
        fuse_out ? (tail == 72 ? layer_c320_kernel<72, true> : tail == 64 ? layer_c320_kernel<64, true> : layer_c320_kernel<0, true>)
                 : (tail == 72 ? layer_c320_kernel<72, false> : tail == 64 ? layer_c320_kernel<64, false> : layer_c320_kernel<0, false>);
    // (the attribute belongs to the current device's copy of the function: set on every launch, it is cheap)
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TOTAL);
    if (e != cudaSuccess) return e;
    if (fuse_out) return launch_pdl_cluster(kern, grid, dim3(1, 2, 1), dim3(NTHREADS), (size_t)TOTAL, stream, tmap, tmap_y, a);
    return launch_pdl(kern, grid, dim3(NTHREADS), (size_t)TOTAL, stream, tmap, tmap_y, a);
}

cudaError_t launch_qattn_sm100(const taq_layer_desc& d, const __half* x, const void* wq, const void* kv, const taq_request* reqs, __half* o,
                               int n_z, int* status, cudaStream_t stream) {
    return launch_c320(d, x, wq, kv, reqs, o, nullptr, nullptr, n_z, status, stream);
}

// The attention core alone at the same shape (taq_cross_attention): Q~ given, all four heads of a CTA at once.
bool sm100_attention_c320_supported(const AttnArgs& a) {
    if (a.channels != KIN || a.heads * D != KIN || a.n_ctx > TP || (a.p_bits != 8 && a.p_bits != 4) || a.p_log || a.n_query < 1) return false;
    if ((reinterpret_cast<uintptr_t>(a.q) & 15u) || (reinterpret_cast<uintptr_t>(a.o) & 15u)) return false;
    return encode_tiled() != nullptr;
}

cudaError_t launch_attention_c320(const AttnArgs& a, int n_z, cudaStream_t stream) {
    taq_layer_desc d{};
    d.batch = a.batch; d.n_query = a.n_query; d.channels = a.channels; d.heads = a.heads; d.n_ctx = a.n_ctx; d.max_trigger = a.max_trigger;
    d.q_bits = a.q_bits; d.p_bits = a.p_bits; d.w_bits = 4; d.w_group = 128;
    return launch_c320(d, nullptr, nullptr, a.kv, a.reqs, a.o, nullptr, nullptr, n_z, a.status, stream, a.q, a.q_scales);
}

cudaError_t launch_layer_sm100(const taq_layer_desc& d, const __half* x, const void* wq, const void* wout, const void* kv, const taq_request* reqs,
                               __half* y, int n_z, int* status, cudaStream_t stream) {
    return launch_c320(d, x, wq, kv, reqs, nullptr, wout, y, n_z, status, stream);
}

}  // namespace taq
