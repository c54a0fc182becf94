// The integer-activation (int8 X and O) layer pass in one kernel for the SD-1.5 64x64 shape (C = 320, 8 heads of 40, W4);
// the fp16-activation pass lives in taq_layer_c320_sm100.cu.  Only the A8 instantiation of the template below is built.
// to_q and the TAQ attention in one kernel: Q never leaves the SM.  A CTA owns 128 query rows of one sequence and four heads (160 output channels of to_q):
//   phase 1  Q = X Wq^T for its 160 channels: the dequant-GEMM of taq_linear_sm100.cu (integer-code operands, one
//            accumulation pass per scale group; here every group - at most three - has its own TMEM accumulator,
//            so the tensor core never waits for the workers, who fold the groups into registers at the end);
//   phase 2  Q~ = Q_a(Q) (Eq. 2, third line) per (row, head) straight from those registers into the fp16-integer
//            operand tiles of the four heads; the row scales stay in shared memory;
//   phase 3  per head: S = Q~ K~^T, softmax, Eq. 3, O = A^ V~ as in taq_attention_sm100.cu.  The sixteen worker warps
//            form two groups of eight (two threads per row each); group g takes heads g and g + 2, so that one
//            group's exponentials overlap the other group's stores, exchanges and waits.  O is stored as fp16.
//   phase 4  (layer variant only) to_out: the two CTAs that share a row tile form a cluster.  Each writes its four
//            heads' O as fp16 operand tiles (32 channels each) into its own shared memory; the producer thread sends
//            them to the partner CTA with bulk copies between the two shared memories as they complete.  Then each
//            CTA computes Y = O Wout^T + b for its own 160 output channels over all 320 channels of O with the
//            machinery of phase 1.  Neither Q~ nor O ever reaches global memory.
// Shared memory is used twice: the X tile and the weight ring of phase 1 become the Q~ tiles and the two P tiles.
// Warps: 0 producer (TMA / bulk copies), 1 MMA issuer, 2..17 workers (four threads per row: one head each in
// phases 1 and 2, (group, key half) in phase 3).
#include "taq_ptx.cuh"
#include "taq_sm100.cuh"
#include "taq_sm100_parts.cuh"
#include "taq_prof.cuh"

TAQ_PROF_DEFINE(qattn)

namespace taq {

namespace {

using namespace parts;

constexpr int D = 40, DP = 48, HG = 4;          // head width, padded width, heads per CTA
constexpr int NQ = HG * D;                      // 160 to_q channels per CTA
constexpr int HC = D;                           // channels per worker thread in phases 1 and 2: one head
constexpr int KIN = 320, BK = 64, NKB = KIN / BK;
constexpr int ROWS = 128;
constexpr int NWORK = 512, NTHREADS = 64 + NWORK;
constexpr int NBSTAGE = 3;                      // ring of expanded weight tiles

constexpr int A_TILE = ROWS * 128;              // 16 KB: one 64-wide K block of X, or one head's Q~ tile, or half of P
constexpr int B_TILE = NQ * 128;                // 20 KB
constexpr int K_BLOCK = TP * 128, VT_BLOCK = DP * 128;
constexpr int K_BYTES = K_BLOCK, VT_BYTES = 2 * VT_BLOCK;
constexpr int MAX_GROUPS = 3;                    // one TMEM accumulator of NQ columns per scale group
constexpr int RAW_BYTES = NQ * (KIN / 2);       // 25600 (W4)
constexpr int SCALE_BYTES = ((NQ * MAX_GROUPS * 4 + 127) / 128) * 128;

constexpr int OFF_A = 0;                                    // phase 1: X tile, 5 K blocks
constexpr int OFF_B = OFF_A + NKB * A_TILE;                 // phase 1: weight ring
constexpr int OFF_Q = 0;                                    // phase 3: Q~ tiles of the four heads
constexpr int OFF_P = OFF_Q + HG * A_TILE;                  // phase 3: one probability tile (two K blocks) per group
constexpr int OFF_XCHG = OFF_P + 4 * A_TILE;                // phase 3: float2 [iteration][group][half][row], 8 KB
constexpr int OFF_RAW = OFF_B + NBSTAGE * B_TILE;            // packed codes of the CTA's 160 channels (Wq, later Wout)
static_assert(OFF_XCHG + 8192 <= OFF_RAW, "exchange buffer must fit behind the P tiles");
constexpr int OFF_SC = OFF_RAW + RAW_BYTES;
constexpr int OFF_SCT = OFF_SC + SCALE_BYTES;
constexpr int OFF_BIAS = OFF_SCT + SCALE_BYTES;                            // phase 4: bias of the CTA's 160 channels
constexpr int OFF_K = ((OFF_BIAS + NQ * 4 + 1023) / 1024) * 1024;          // K~ tiles, one buffer per group
constexpr int OFF_VT = OFF_K + 2 * K_BYTES;                                // V~^T tiles, one buffer per group
constexpr int OFF_CST = OFF_VT + 2 * VT_BYTES;                             // per-key constants of all four heads
constexpr int OFF_MISC = OFF_CST + HG * kOperandConstBytes;
static_assert(OFF_P + 4 * A_TILE <= OFF_RAW, "phase-3 tiles must fit into the phase-1 region");

struct Misc {
    uint64_t a_full[NKB], b_full[NBSTAGE], b_empty[NBSTAGE], w_full, acc_full[MAX_GROUPS];
    uint64_t w2_full, s_done, pv_done, peer_ready, peer_got, o_all, piece_done[3];      // layer variant (phase 4)
    uint64_t q_all, k_full[2], vt_full[2], c_full, s_full[2], s_free[2], p_full[2], o_full[2], drain;
    uint32_t tmem_base;
    volatile int abort_flag;
    float sq[HG][ROWS];              // Q~ row scales
    uint64_t xq_full;                // integer-activation variant: the int8 activation tiles are in place (X, later O)
    float sx[ROWS];                  //   per-token scale of X, later of O
    float xmax[4][ROWS];             //   partial absmax of a row's four threads
};
constexpr int TOTAL = OFF_MISC + (int)sizeof(Misc) + 1024;
static_assert(TOTAL <= 232448, "shared memory budget");

constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TMEM_ACC = 0;                 // phase 1: up to three accumulators of NQ columns
constexpr uint32_t TMEM_S = 0, TMEM_O = 2 * TP;  // phase 3: one S and one O accumulator per group (reuses the columns)

struct QAttnArgs {
    const __half* x;            // [z][B][N][C]
    const void* wq;             // packed [C][C] (single problem)
    const void* kv;             // blocks [B] (single problem)
    const taq_request* reqs;    // nullable; then one sequence per request
    __half* o;                  // [z][B][N][C]  (query-attention variant)
    const void* wout;           // packed [C][C] (layer variant, single problem)
    __half* y;                  // [z][B][N][C]  (layer variant)
    int n_query, heads, n_ctx, max_trigger, group, q_bits, p_bits;
    int* status;
};

// O of phase 4 (the A operand of to_out) lives in ten tiles of 32 channels: 128 rows of 64 bytes with the 64-byte swizzle.
// Tiles 0..7 reuse the Q~ tiles, tiles 8 and 9 the K~ buffers; both are dead once the S products of all four heads have
// been computed.  A CTA produces five of them (heads 0..3: tiles 0..4, heads 4..7: tiles 5..9) and receives the other
// five from its partner, as bulk copies of contiguous runs of tiles ("pieces") that leave as soon as they are complete.
constexpr int O_TILE = ROWS * 64;                // 8 KB
constexpr int N_OTILE = KIN / 32;
__device__ __forceinline__ int o_tile_offset(int t) { return t < 8 ? OFF_Q + t * O_TILE : OFF_K + (t - 8) * O_TILE; }
static_assert(8 * O_TILE == HG * A_TILE && 2 * K_BYTES >= 2 * O_TILE, "the Q~ tiles and K~ buffers must hold the ten O tiles");
static_assert(HG * D == 5 * 32 && KIN == 2 * HG * D, "O tile ownership assumes 160 of 320 channels per CTA");
constexpr int OCH = DP / 2;                      // O columns per thread (two threads per row in phase 3)
// Bit t set: the threads of half `half` of head h (0..7) store chunks of O tile t.
__device__ __forceinline__ uint32_t o_tiles_touched(int h, int half) {
    uint32_t m = 0;
#pragma unroll
    for (int i = 0; i < OCH / 8; ++i)
        if (half * OCH + i * 8 < D) m |= 1u << ((h * D + half * OCH + i * 8) >> 5);
    return m;
}
// Pieces of a CTA's five tiles: the first leaves after the first head of each group (80 channels cover two tiles and a
// half), the next when group 0 has stored its second head, the last when group 1 has; tiles 7 and 8 are not adjacent in
// shared memory.
constexpr int MAX_PIECES = 3;
__device__ __forceinline__ int o_pieces(int h_begin, int (&first)[MAX_PIECES], int (&count)[MAX_PIECES]) {
    if (h_begin == 0) { first[0] = 0; count[0] = 2; first[1] = 2; count[1] = 1; first[2] = 3; count[2] = 2; return 3; }
    first[0] = 5; count[0] = 2; first[1] = 7; count[1] = 1; first[2] = 8; count[2] = 2;
    return 3;
}

// Expands the packed 4-bit codes at OFF_RAW into the ring of fp16 weight tiles, K block by K block (all worker threads).
// One copy of this code serves phase 1 and phase 4.  Takes and returns the ring position: bits 0..1 stage, bit 2 pass
// parity, bit 3 set when a wait ran out.
__device__ __noinline__ uint32_t build_weight_tiles(unsigned char* smem, Misc* misc, int first_pass, int wt, int lane, int s, uint32_t ph) {
    const unsigned char* raw = smem + OFF_RAW;
    bool ok = true;
    for (int kb = 0; kb < NKB; ++kb) {
        if ((!first_pass || kb >= NBSTAGE) && !ptx::mbar_wait(&misc->b_empty[s], ph ^ 1)) ok = false;
        if (!ok || misc->abort_flag) { ok = false; break; }
        unsigned char* b_tile = smem + OFF_B + s * B_TILE;
        constexpr int NCH = (NQ * 8 + NWORK - 1) / NWORK;       // 16-byte chunks (8 weights) per thread and K block
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
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&misc->b_full[s]);
        if (++s == NBSTAGE) { s = 0; ph ^= 1; }
    }
    return (uint32_t)s | (ph << 2) | (ok ? 0u : 8u);
}

// Integer-activation variant: the same codes as int8, one tile per 128-element K block (= one scale group of the W4
// format); the ring of three stages holds all three blocks of a projection at once.  Same calling convention.
constexpr int NKB8 = (KIN + 127) / 128;
static_assert(NKB8 == NBSTAGE, "the three int8 K blocks fill the ring exactly");
__device__ __noinline__ uint32_t build_weight_tiles_i8(unsigned char* smem, Misc* misc, int first_pass, int wt, int lane, int s, uint32_t ph) {
    const unsigned char* raw = smem + OFF_RAW;
    bool ok = true;
    for (int kb = 0; kb < NKB8; ++kb) {
        if (!first_pass && !ptx::mbar_wait(&misc->b_empty[s], ph ^ 1)) ok = false;
        if (!ok || misc->abort_flag) { ok = false; break; }
        unsigned char* b_tile = smem + OFF_B + s * B_TILE;
        constexpr int NCH = (NQ * 8 + NWORK - 1) / NWORK;       // 16-byte chunks (16 weights) per thread and K block
        const int n0 = wt >> 3, c = wt & 7;
        const int k0 = kb * 128 + c * 16;                       // first fan-in element of the chunk; beyond KIN: zeros
        uint2 pw[NCH];
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
            pw[i] = make_uint2(0x88888888u, 0x88888888u);       // nibble 8 = code 0
            if (n0 + (NWORK / 8) * i < NQ && k0 < KIN) pw[i] = *reinterpret_cast<const uint2*>(raw + (n0 + (NWORK / 8) * i) * (KIN / 2) + (k0 >> 1));
        }
#pragma unroll
        for (int i = 0; i < NCH; ++i)
            if (n0 + (NWORK / 8) * i < NQ) {
                const uint2 lo = codes_w4_to_i8(pw[i].x), hi = codes_w4_to_i8(pw[i].y);
                *reinterpret_cast<uint4*>(b_tile + ptx::sw128_offset(n0 + (NWORK / 8) * i, c)) = make_uint4(lo.x, lo.y, hi.x, hi.y);
            }
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&misc->b_full[s]);
        if (++s == NBSTAGE) { s = 0; ph ^= 1; }
    }
    return (uint32_t)s | (ph << 2) | (ok ? 0u : 8u);
}

// One code rint(x / s), clamped to +-127, exactly as the stand-alone quantizer defines it (one IEEE division, then rintf):
// the rare path of quant16 below, one shared copy of the division.
__device__ __noinline__ uint32_t code_by_division(float x, float s) {
    return (uint32_t)(int)fminf(fmaxf(rintf(__fdiv_rn(x, s)), -127.f), 127.f);
}
// Sixteen codes.  fma(x, r, 1.5 * 2^23) leaves rint(x r) in the low byte.  The definition's rounded quotient fl(x / s) and
// the product with the correctly rounded reciprocal both lie between x r_lo and x r_hi (r two ulps down and up: each of
// them is off the exact quotient by at most one relative 2^-24), so when both ends round to the same integer that
// integer is the definition's code.  Otherwise the element is divided.  fp16 data makes that less rare than one would
// think - a value that is exactly half of the row maximum sits exactly on a boundary - about 4 codes in 10000, so the
// fix-up touches single elements, not the chunk.
__device__ __forceinline__ uint4 quant16(uint4 lo8, uint4 hi8, float s, float rs) {
    const float r_lo = __uint_as_float(__float_as_uint(rs) - 2u), r_hi = __uint_as_float(__float_as_uint(rs) + 2u);
    const uint4 v[2] = {lo8, hi8};
    uint32_t b[16];
    uint32_t differ = 0;
#pragma unroll
    for (int u = 0; u < 2; ++u) {
        const __half2* h = reinterpret_cast<const __half2*>(&v[u]);
#pragma unroll
        for (int e2 = 0; e2 < 4; ++e2) {
            const float2 f = __half22float2(h[e2]);
            const uint32_t a0 = __float_as_uint(fmaf(f.x, r_lo, 12582912.0f)), a1 = __float_as_uint(fmaf(f.y, r_lo, 12582912.0f));
            differ |= (a0 ^ __float_as_uint(fmaf(f.x, r_hi, 12582912.0f))) | (a1 ^ __float_as_uint(fmaf(f.y, r_hi, 12582912.0f)));
            b[8 * u + 2 * e2] = a0;
            b[8 * u + 2 * e2 + 1] = a1;
        }
    }
    if (differ) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const __half2* h = reinterpret_cast<const __half2*>(&v[u]);
#pragma unroll
            for (int e2 = 0; e2 < 4; ++e2) {
                const float2 f = __half22float2(h[e2]);
                if (b[8 * u + 2 * e2] != __float_as_uint(fmaf(f.x, r_hi, 12582912.0f))) b[8 * u + 2 * e2] = code_by_division(f.x, s);
                if (b[8 * u + 2 * e2 + 1] != __float_as_uint(fmaf(f.y, r_hi, 12582912.0f))) b[8 * u + 2 * e2 + 1] = code_by_division(f.y, s);
            }
        }
    }
    uint4 out;
    out.x = __byte_perm(__byte_perm(b[0], b[1], 0x0040), __byte_perm(b[2], b[3], 0x0040), 0x5410);
    out.y = __byte_perm(__byte_perm(b[4], b[5], 0x0040), __byte_perm(b[6], b[7], 0x0040), 0x5410);
    out.z = __byte_perm(__byte_perm(b[8], b[9], 0x0040), __byte_perm(b[10], b[11], 0x0040), 0x5410);
    out.w = __byte_perm(__byte_perm(b[12], b[13], 0x0040), __byte_perm(b[14], b[15], 0x0040), 0x5410);
    return out;
}

// Integer-activation variant: Q_a per token inside the CTA (all 512 worker threads; four threads per row, 80 channels
// each).  `from_o` = 0: the row's fp16 values are read from the X tile (five 64-channel blocks, 128-byte swizzle);
// 1: from the ten 32-channel O tiles (64-byte swizzle).  Two streaming passes over the row piece, written as real loops
// (this code runs once per CTA: short code is fetch time saved): absmax, exchanged between the row's four threads
// through shared memory, then the codes, which go into three int8 tiles elsewhere in shared memory (K blocks of 128
// channels, 128-byte rows and swizzle, channels 320..383 zero) at the offsets dst[0..2].
__device__ __noinline__ void quantize_tokens(unsigned char* smem, Misc* misc, int from_o, int r, int part, int lane, int dst0, int dst1, int dst2) {
    auto chunk = [&](int cg) -> uint4 {                  // 8-channel chunk cg (0..39) of row r
        const unsigned char* src = from_o ? smem + o_tile_offset(cg >> 2) + ptx::sw64_offset(r, cg & 3)
                                          : smem + OFF_A + (cg >> 3) * A_TILE + ptx::sw128_offset(r, cg & 7);
        return *reinterpret_cast<const uint4*>(src);
    };
    __half2 m2 = __floats2half2_rn(0.f, 0.f);
#pragma unroll 1
    for (int j = 0; j < 10; ++j) {
        const uint4 v = chunk(10 * part + j);
        const __half2* h = reinterpret_cast<const __half2*>(&v);
        m2 = __hmax2(m2, __hmax2(__hmax2(__habs2(h[0]), __habs2(h[1])), __hmax2(__habs2(h[2]), __habs2(h[3]))));
    }
    misc->xmax[part][r] = fmaxf(__low2float(m2), __high2float(m2));
    asm volatile("bar.sync 1, 512;" ::: "memory");
    const float amax = fmaxf(fmaxf(misc->xmax[0][r], misc->xmax[1][r]), fmaxf(misc->xmax[2][r], misc->xmax[3][r]));
    const float sc = quant_scale(amax, 127.f);
    const float rs = sc > 0.f ? __frcp_rn(sc) : 0.f;
    if (part == 0) misc->sx[r] = sc;
#pragma unroll 1
    for (int j = 0; j < 5; ++j) {                        // 16 channels -> one 16-byte chunk of int8 codes
        const int c16 = 5 * part + j;                    // 16-channel chunk of the row, 0..19
        const uint4 codes = sc > 0.f ? quant16(chunk(2 * c16), chunk(2 * c16 + 1), sc, rs) : make_uint4(0, 0, 0, 0);
        const int tile = c16 >> 3;
        *reinterpret_cast<uint4*>(smem + (tile == 0 ? dst0 : tile == 1 ? dst1 : dst2) + ptx::sw128_offset(r, c16 & 7)) = codes;
    }
    *reinterpret_cast<uint4*>(smem + dst2 + ptx::sw128_offset(r, 4 + part)) = make_uint4(0, 0, 0, 0);
    ptx::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(&misc->xq_full);
}

// A8: the integer-activation layer pass.  X is quantized per token (Q_a over all 320 channels) inside the CTA, to_q and
// to_out run as int8 x int8 -> int32 MMAs with one accumulator per 128-wide scale group, and O is quantized per token
// from its fp16 tiles once both CTAs' halves are there.
template <bool TAIL_ONLY, bool FUSE_OUT, bool A8 = false>
__global__ void __launch_bounds__(NTHREADS, 1) qattn_c320_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_y, const QAttnArgs a) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_u32(smem_dyn) & 1023u)) & 1023u);   // 1024-byte aligned, still provably shared
    Misc* misc = reinterpret_cast<Misc*>(smem + OFF_MISC);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int T = a.n_ctx, H = a.heads;
    const int zb = blockIdx.z;                      // sequence (batch entry or request)
    const int row0 = blockIdx.x * ROWS;
    const int h_begin = blockIdx.y * HG;
    const int col0 = h_begin * D;
    const WeightLayout L = weight_layout(KIN, KIN, 4, a.group);
    const int n_groups = L.n_groups;
    const int kb_per_group = L.group_len / BK;

    TAQ_PROF_INIT
    if (tid == 0) { TAQ_PROF(0); TAQ_GPROF(30); }
    if (tid == 0) {
        for (int i = 0; i < NKB; ++i) ptx::mbar_init(&misc->a_full[i], 1);
        for (int i = 0; i < NBSTAGE; ++i) {
            ptx::mbar_init(&misc->b_full[i], NWORK / 32);
            ptx::mbar_init(&misc->b_empty[i], 1);
        }
        ptx::mbar_init(&misc->w_full, 1);
        for (int i = 0; i < MAX_GROUPS; ++i) ptx::mbar_init(&misc->acc_full[i], 1);
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(&misc->k_full[i], 1);
            ptx::mbar_init(&misc->vt_full[i], 1);
            ptx::mbar_init(&misc->s_full[i], 1);
            ptx::mbar_init(&misc->s_free[i], NWORK / 64);     // one arrival per warp of the group
            ptx::mbar_init(&misc->p_full[i], NWORK / 64);
            ptx::mbar_init(&misc->o_full[i], 1);
        }
        ptx::mbar_init(&misc->c_full, 1);
        ptx::mbar_init(&misc->w2_full, 1);
        ptx::mbar_init(&misc->s_done, 1);
        ptx::mbar_init(&misc->pv_done, 1);
        ptx::mbar_init(&misc->peer_ready, 1);
        ptx::mbar_init(&misc->peer_got, 1);
        // every worker warp of this CTA, and one arrival that announces the bytes of the partner's five tiles
        ptx::mbar_init(&misc->o_all, NWORK / 32 + 1);
        {
            int first[MAX_PIECES], count[MAX_PIECES];
            const int np = o_pieces(h_begin, first, count);
            for (int k = 0; k < MAX_PIECES; ++k) {      // arrivals: one per (warp, head) that stores into the piece
                const uint32_t pm = k < np ? ((1u << count[k]) - 1u) << first[k] : 0u;
                int cnt = 0;
                for (int hi = 0; hi < HG; ++hi)
                    for (int hf = 0; hf < 2; ++hf) cnt += (o_tiles_touched(h_begin + hi, hf) & pm) ? NWORK / 128 : 0;
                ptx::mbar_init(&misc->piece_done[k], cnt > 0 ? cnt : 1);
            }
        }
        ptx::mbar_init(&misc->q_all, NWORK / 32);
        ptx::mbar_init(&misc->xq_full, NWORK / 32);
        ptx::mbar_init(&misc->drain, 1);
        misc->abort_flag = 0;
        ptx::mbar_fence_init();
        if (FUSE_OUT) ptx::mbar_arrive_expect_tx(&misc->o_all, (N_OTILE / 2) * O_TILE);
        ptx::tma_prefetch_desc(&tmap_x);
        if (FUSE_OUT) ptx::tma_prefetch_desc(&tmap_y);
    }
    if (warp == 1) ptx::tmem_alloc(&misc->tmem_base, TMEM_COLS);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem_base = misc->tmem_base;
    ptx::pdl_trigger();
    if (FUSE_OUT) ptx::cluster_sync_all();                   // the partner's barriers exist before anything arrives on them
    const uint32_t peer = FUSE_OUT ? (ptx::cluster_ctarank() ^ 1u) : 0u;

    const taq_kv_layout KL = kv_layout(H, T, D, a.max_trigger);

    if (warp == 0) {
        // ---------------- producer ----------------
        if (lane == 0) {
            // Packed weights are written by taq_pack_weights, which never lets its successor start early: they are complete
            // before this kernel can run at all and are fetched (and expanded) under the previous kernel's tail.
            const uint8_t* blob = (const uint8_t*)(a.reqs ? a.reqs[zb].Wq : a.wq);
            const uint32_t scale_bytes = (uint32_t)(NQ * n_groups * 4);
            ptx::mbar_arrive_expect_tx(&misc->w_full, RAW_BYTES + scale_bytes);
            ptx::bulk_load(smem + OFF_RAW, blob + L.off_codes + (size_t)col0 * L.row_bytes, RAW_BYTES, &misc->w_full);
            ptx::bulk_load(smem + OFF_SC, blob + L.off_scales + (size_t)col0 * n_groups * 4, scale_bytes, &misc->w_full);
            ptx::pdl_wait();                              // X (and in general the K~/V~ block) may come from the previous kernel
            TAQ_PROF(1); TAQ_GPROF(28);
            for (int kb = 0; kb < NKB; ++kb) {            // the whole X tile at once: every K block has its own buffer
                ptx::mbar_arrive_expect_tx(&misc->a_full[kb], A_TILE);
                ptx::tma_load_3d(smem + OFF_A + kb * A_TILE, &tmap_x, &misc->a_full[kb], kb * BK, row0, zb);
            }
            const uint8_t* blk = a.reqs ? (const uint8_t*)a.reqs[zb].kv : (const uint8_t*)a.kv + (size_t)zb * KL.block_bytes;
            const uint8_t* img = blk + KL.off_operands + (size_t)h_begin * KL.operand_head_bytes;
            // K~/V~ operand images: the constants of all four heads at once; K~ and V~^T tiles of head hi go to the
            // buffers of group hi & 1.  A group's K~ buffer is free again as soon as its S has been computed, its V~^T
            // buffer after its PV, so the second head's tiles arrive under the first head's softmax.
            auto load_consts = [&]() {
                ptx::mbar_arrive_expect_tx(&misc->c_full, HG * kOperandConstBytes);
                for (int hi = 0; hi < HG; ++hi)
                    ptx::bulk_load(smem + OFF_CST + hi * kOperandConstBytes, img + (size_t)hi * KL.operand_head_bytes + K_BYTES + VT_BYTES, kOperandConstBytes, &misc->c_full);
            };
            auto load_k = [&](int hi) {
                ptx::mbar_arrive_expect_tx(&misc->k_full[hi & 1], K_BYTES);
                ptx::bulk_load(smem + OFF_K + (hi & 1) * K_BYTES, img + (size_t)hi * KL.operand_head_bytes, K_BYTES, &misc->k_full[hi & 1]);
            };
            auto load_vt = [&](int hi) {
                ptx::mbar_arrive_expect_tx(&misc->vt_full[hi & 1], VT_BYTES);
                ptx::bulk_load(smem + OFF_VT + (hi & 1) * VT_BYTES, img + (size_t)hi * KL.operand_head_bytes + K_BYTES, VT_BYTES, &misc->vt_full[hi & 1]);
            };
            // (integer-activation variant: the int8 X tiles occupy this region during phase 1; the images follow below)
            if (!A8) { load_consts(); load_k(0); load_k(1); load_vt(0); load_vt(1); }
            int k_issued = 2, vt_issued = 2;
            if (FUSE_OUT) {       // phase 1 no longer needs the packed Wq: fetch the packed Wout rows of this CTA's output channels
                if (!ptx::mbar_wait(&misc->acc_full[n_groups - 1], 0)) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
                if (!misc->abort_flag) {
                    const uint8_t* blob2 = (const uint8_t*)(a.reqs ? a.reqs[zb].Wout : a.wout);
                    ptx::mbar_arrive_expect_tx(&misc->w2_full, RAW_BYTES + scale_bytes + NQ * 4);
                    ptx::bulk_load(smem + OFF_RAW, blob2 + L.off_codes + (size_t)col0 * L.row_bytes, RAW_BYTES, &misc->w2_full);
                    ptx::bulk_load(smem + OFF_SC, blob2 + L.off_scales + (size_t)col0 * n_groups * 4, scale_bytes, &misc->w2_full);
                    ptx::bulk_load(smem + OFF_BIAS, blob2 + L.off_bias + (size_t)col0 * 4, NQ * 4, &misc->w2_full);
                }
            }
            if (A8 && !misc->abort_flag) { load_consts(); load_k(0); load_k(1); load_vt(0); load_vt(1); }    // phase 1 is over
            for (int g = 0; g < 2 && !misc->abort_flag; ++g) {
                if (!ptx::mbar_wait(&misc->s_full[g], 0)) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; break; }
                load_k(2 + g);
                ++k_issued;
            }
            for (int g = 0; g < 2 && !misc->abort_flag; ++g) {
                if (!ptx::mbar_wait(&misc->o_full[g], 0)) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; break; }
                load_vt(2 + g);
                ++vt_issued;
            }
            if (FUSE_OUT && !misc->abort_flag) {
                // phase 4: this CTA's O tiles go to the partner, piece by piece, as soon as every warp that stores into a
                // piece has arrived and the partner has announced that its Q~ tiles and K~ buffers are dead; the copies
                // complete on the partner's o_all barrier
                int first[MAX_PIECES], count[MAX_PIECES];
                const int np = o_pieces(h_begin, first, count);
                bool sent = ptx::mbar_wait(&misc->peer_ready, 0);
                for (int k = 0; k < np && sent; ++k) {
                    sent = ptx::mbar_wait(&misc->piece_done[k], 0) && !misc->abort_flag;
                    if (!sent) break;
                    unsigned char* piece = smem + o_tile_offset(first[k]);
                    ptx::bulk_copy_to_cta(ptx::map_to_cta(ptx::smem_u32(piece), peer), piece, (uint32_t)(count[k] * O_TILE),
                                          ptx::map_to_cta(ptx::smem_u32(&misc->o_all), peer));
                    TAQ_PROF(57 + k);
                }
                if (!sent) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
            }
            if (misc->abort_flag) {   // give copies that are still in flight a bounded chance to land before the CTA exits
                (void)ptx::mbar_wait(&misc->w_full, 0);
                (void)ptx::mbar_wait(&misc->c_full, 0);
                if (FUSE_OUT) (void)ptx::mbar_wait(&misc->w2_full, 0);
                for (int kb = 0; kb < NKB; ++kb) (void)ptx::mbar_wait(&misc->a_full[kb], 0);
                for (int hi = k_issued - 2; hi < k_issued; ++hi) (void)ptx::mbar_wait(&misc->k_full[hi & 1], (hi >> 1) & 1);
                for (int hi = vt_issued - 2; hi < vt_issued; ++hi) (void)ptx::mbar_wait(&misc->vt_full[hi & 1], (hi >> 1) & 1);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // All 32 lanes walk the control flow (waits, loop state, descriptor words stay warp-uniform and cheap); one
        // elected lane issues the MMAs and commits.  The issue path is kept short on purpose: this warp shares its
        // scheduler with four worker warps, and every instruction it needs between two MMAs delays the tensor core.
        const bool leader = ptx::elect_one();
        bool ok = true;
        auto wait = [&](uint64_t* bar, uint32_t parity) -> bool { return __all_sync(0xffffffffu, ptx::mbar_wait(bar, parity) && !misc->abort_flag) != 0; };
        constexpr uint32_t idesc = ptx::idesc_f16_m128(NQ);
        constexpr uint32_t HI128 = ptx::kDescHiSw128, HI64 = ptx::kDescHiSw64;
        const uint32_t a_lo0 = ptx::desc_lo(ptx::smem_u32(smem + OFF_A)), b_lo0 = ptx::desc_lo(ptx::smem_u32(smem + OFF_B));
        const uint32_t q_lo0 = ptx::desc_lo(ptx::smem_u32(smem + OFF_Q)), p_lo0 = ptx::desc_lo(ptx::smem_u32(smem + OFF_P));
        const uint32_t k_lo0 = ptx::desc_lo(ptx::smem_u32(smem + OFF_K)), vt_lo0 = ptx::desc_lo(ptx::smem_u32(smem + OFF_VT));
        int s = 0;                                       // weight ring position and pass parity, continued in phase 4
        uint32_t ph = 0;
        if (A8) {   // phase 1, integer: K block g is scale group g, all three weight tiles fit the ring
            ok = wait(&misc->xq_full, 0);
            for (int g = 0; g < NKB8 && ok; ++g) {
                if (!wait(&misc->b_full[g], 0)) { ok = false; break; }
                if (leader) {
                    TAQ_PROF(2 + g);
                    const uint32_t a_lo = k_lo0 + g * (A_TILE >> 4), b_lo = b_lo0 + g * (B_TILE >> 4);      // X~ tiles sit in the K~/V~ region
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        ptx::mma_i8_ss(tmem_base + TMEM_ACC + g * NQ, ptx::desc_join(HI128, a_lo + 2 * k), ptx::desc_join(HI128, b_lo + 2 * k), ptx::idesc_i8_m128(NQ), k != 0);
                    ptx::mma_commit(&misc->b_empty[g]);
                    ptx::mma_commit(&misc->acc_full[g]);
                }
            }
            s = 0; ph = 1;                               // the ring has been passed once
        } else {   // phase 1: one accumulation pass per scale group
            int kb = 0;
            for (int g = 0; g < n_groups && ok; ++g) {
                const int kb_end = min(NKB, kb + kb_per_group);
                for (bool first = true; kb < kb_end && ok; ++kb) {
                    if (!wait(&misc->a_full[kb], 0) || !wait(&misc->b_full[s], ph)) { ok = false; break; }
                    if (leader) {
                        TAQ_PROF(2 + kb);
                        const uint32_t a_lo = a_lo0 + kb * (A_TILE >> 4), b_lo = b_lo0 + s * (B_TILE >> 4);
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            ptx::mma_f16_ss(tmem_base + TMEM_ACC + g * NQ, ptx::desc_join(HI128, a_lo + 2 * k), ptx::desc_join(HI128, b_lo + 2 * k), idesc, !(first && k == 0));
                        ptx::mma_commit(&misc->b_empty[s]);
                        if (kb + 1 == kb_end) ptx::mma_commit(&misc->acc_full[g]);
                    }
                    first = false;
                    if (++s == NBSTAGE) { s = 0; ph ^= 1; }
                }
            }
        }
        // phase 3: the Q~ tiles of all four heads are in place once every worker warp has arrived (their reads of the
        // phase-1 accumulators, whose columns S and O reuse, are ordered before that arrival)
        ok = ok && wait(&misc->q_all, 0);
        ptx::tc_fence_after_sync();
        // group g (heads g, g + 2) owns K~/V~ buffer g, S accumulator g, O accumulator g and P tile g
        auto issue_s = [&](int g, int it) -> bool {
            const int hi = g + 2 * it;
            if (!wait(&misc->k_full[g], it) || (it > 0 && !wait(&misc->s_free[g], it - 1))) return false;
            ptx::tc_fence_after_sync();                  // the group's loads of its previous S
            if (leader) {
                const uint32_t qh_lo = q_lo0 + hi * (A_TILE >> 4), kg_lo = k_lo0 + g * (K_BYTES >> 4);
#pragma unroll
                for (int ks = 0; ks < DP / 16; ++ks)
                    ptx::mma_f16_ss(tmem_base + TMEM_S + g * TP, ptx::desc_join(HI128, qh_lo + 2 * ks), ptx::desc_join(HI128, kg_lo + 2 * ks), ptx::idesc_f16_m128(TP), ks != 0);
                ptx::mma_commit(&misc->s_full[g]);       // (also tells the producer that the group's K~ buffer is free)
            }
            return true;
        };
        auto issue_pv = [&](int g, int it) -> bool {
            if (!wait(&misc->p_full[g], it) || !wait(&misc->vt_full[g], it)) return false;     // (the group has emptied O before it arrives)
            ptx::tc_fence_after_sync();
            if (leader) {
                const uint32_t pg_lo = p_lo0 + g * 2 * (A_TILE >> 4), vg_lo = vt_lo0 + g * (VT_BYTES >> 4);
#pragma unroll
                for (int ks = 0; ks < TP / 16; ++ks)
                    ptx::mma_f16_ss(tmem_base + TMEM_O + g * DP, ptx::desc_join(HI128, pg_lo + (ks / 4) * (A_TILE >> 4) + (ks % 4) * 2),
                                    ptx::desc_join(HI128, vg_lo + (ks / 4) * (VT_BLOCK >> 4) + (ks % 4) * 2), ptx::idesc_f16_m128(DP), ks != 0);
                ptx::mma_commit(&misc->o_full[g]);       // (also tells the producer that the group's V~^T buffer is free)
            }
            return true;
        };
        // S of a group's second head is issued as soon as its K~ tile has arrived and the group holds the first
        // head's scores in registers, i.e. under the first head's softmax
        for (int it = 0; it < 2 && ok; ++it)
            for (int g = 0; g < 2 && ok; ++g) ok = issue_s(g, it);
        if (FUSE_OUT && ok) {     // all S products done: the Q~ tiles and K~ buffers of this CTA may receive O tiles
            if (leader) ptx::mma_commit(&misc->s_done);
            ok = wait(&misc->s_done, 0);
            if (ok && leader) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(ptx::smem_u32(&misc->peer_ready), peer));
        }
        for (int it = 0; it < 2 && ok; ++it)
            for (int g = 0; g < 2 && ok; ++g) ok = issue_pv(g, it);
        if (FUSE_OUT && ok) {
            if (leader) ptx::mma_commit(&misc->pv_done);             // the P tiles become the weight ring of phase 4
            // phase 4: Y = O Wout^T for this CTA's 160 output channels, once both CTAs' O tiles are complete
            ok = wait(&misc->o_all, 0);
            // the partner's copies have landed: it may leave without waiting for this CTA any longer
            if (ok && leader) ptx::mbar_arrive_cluster_relaxed(ptx::map_to_cta(ptx::smem_u32(&misc->peer_got), peer));
            if (leader) TAQ_PROF(38);
            ptx::tc_fence_after_sync();                  // the workers' loads of the last O accumulators
            if (A8) {    // integer to_out: the workers have turned the fp16 O tiles into three int8 tiles (in the Q~ region)
                ok = ok && wait(&misc->xq_full, 1);
                for (int g = 0; g < NKB8 && ok; ++g) {
                    if (!wait(&misc->b_full[g], 1)) { ok = false; break; }
                    if (leader) {
                        TAQ_PROF(40 + g);
                        const uint32_t o_lo = g == 0 ? p_lo0 : g == 1 ? vt_lo0 : ptx::desc_lo(ptx::smem_u32(smem + OFF_RAW));
                        const uint32_t b_lo = b_lo0 + g * (B_TILE >> 4);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            ptx::mma_i8_ss(tmem_base + TMEM_ACC + g * NQ, ptx::desc_join(HI128, o_lo + 2 * k), ptx::desc_join(HI128, b_lo + 2 * k), ptx::idesc_i8_m128(NQ), k != 0);
                        ptx::mma_commit(&misc->b_empty[g]);
                        ptx::mma_commit(&misc->acc_full[g]);
                    }
                }
            }
            int kb = 0;
            for (int g = 0; g < n_groups && ok && !A8; ++g) {
                const int kb_end = min(NKB, kb + kb_per_group);
                for (bool first = true; kb < kb_end && ok; ++kb) {
                    if (!wait(&misc->b_full[s], ph)) { ok = false; break; }
                    if (leader) {
                        TAQ_PROF(40 + kb);
                        // the 64-wide weight block spans O tiles 2 kb and 2 kb + 1 (adjacent, except tiles 7 and 8)
                        const uint32_t o_lo = kb < 4 ? q_lo0 + 2 * kb * (O_TILE >> 4) : k_lo0;
                        const uint32_t b_lo = b_lo0 + s * (B_TILE >> 4);
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            ptx::mma_f16_ss(tmem_base + TMEM_ACC + g * NQ, ptx::desc_join(HI64, o_lo + (k >> 1) * (O_TILE >> 4) + (k & 1) * 2), ptx::desc_join(HI128, b_lo + 2 * k), idesc, !(first && k == 0));
                        ptx::mma_commit(&misc->b_empty[s]);
                        if (kb + 1 == kb_end) ptx::mma_commit(&misc->acc_full[g]);
                    }
                    first = false;
                    if (++s == NBSTAGE) { s = 0; ph ^= 1; }
                }
            }
        }
        if (!ok) {
            if (leader) {
                raise_status(a.status, TAQ_ERR_TIMEOUT);
                misc->abort_flag = 1;
                ptx::mma_commit(&misc->drain);               // wait (bounded) for whatever was issued before TMEM is given back
            }
            (void)ptx::mbar_wait(&misc->drain, 0);
        }
    } else {
        // ---------------- workers (warps 2..17): four threads per row ----------------
        const int wt = tid - 64;
        const int q4 = warp & 3, part = (warp - 2) >> 2;    // TMEM lane quarter; which head (phases 1, 2) / (group, half) (phase 3)
        const int r = q4 * 32 + lane;
        const int n = row0 + r;
        const bool valid = n < a.n_query;
        const size_t grow = (size_t)zb * a.n_query + (valid ? n : 0);
        const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
        const float* wscales = reinterpret_cast<const float*>(smem + OFF_SC);
        float* scales_t = reinterpret_cast<float*>(smem + OFF_SCT);
        bool ok = ptx::mbar_wait(&misc->w_full, 0);
        for (int i = wt; i < NQ * n_groups; i += NWORK) scales_t[(i % n_groups) * NQ + i / n_groups] = wscales[i];
        asm volatile("bar.sync 1, 512;" ::: "memory");

        // ---- phase 1: expand weight tiles; fold each finished group: y = this thread's head (40 channels) of its row ----
        float y[HC];
#pragma unroll
        for (int c = 0; c < HC; ++c) y[c] = 0.f;
        const int cb = part * HC;
        int s = 0;                                           // weight ring position and pass parity, continued in phase 4
        uint32_t ph = 0;
        auto build_tiles = [&](int first_pass) {
            const uint32_t st = A8 ? build_weight_tiles_i8(smem, misc, first_pass, wt, lane, s, ph) : build_weight_tiles(smem, misc, first_pass, wt, lane, s, ph);
            s = (int)(st & 3u); ph = (st >> 2) & 1u;
            if (st >> 3) ok = false;
        };
        auto fold_groups = [&](uint32_t parity) {            // y += scale[g] * accumulator g, as each group completes
        for (int g = 0; g < n_groups && ok; ++g) {             // later groups are still being multiplied while this one is folded
            ok = ptx::mbar_wait(&misc->acc_full[g], parity) && !misc->abort_flag;
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
                float f[8];
#pragma unroll
                for (int e2 = 0; e2 < 8; ++e2) f[e2] = A8 ? __int2float_rn((int)v[i][e2]) : __uint_as_float(v[i][e2]);
                yy[0] = fmaf(f[0], s0.x, yy[0]); yy[1] = fmaf(f[1], s0.y, yy[1]);
                yy[2] = fmaf(f[2], s0.z, yy[2]); yy[3] = fmaf(f[3], s0.w, yy[3]);
                yy[4] = fmaf(f[4], s1.x, yy[4]); yy[5] = fmaf(f[5], s1.y, yy[5]);
                yy[6] = fmaf(f[6], s1.z, yy[6]); yy[7] = fmaf(f[7], s1.w, yy[7]);
            }
        }
        ptx::tc_fence_before_sync();
        };
        build_tiles(1);
        if (A8) {                                            // X~ = Q_a(X) per token, from the fp16 tile that TMA brought
            for (int kb = 0; kb < NKB && ok; ++kb) ok = ptx::mbar_wait(&misc->a_full[kb], 0) && !misc->abort_flag;
            quantize_tokens(smem, misc, 0, r, part, lane, OFF_K, OFF_K + A_TILE, OFF_K + 2 * A_TILE);
        }
        fold_groups(0);
        if (A8) {
            const float sxr = misc->sx[r];
#pragma unroll
            for (int c = 0; c < HC; ++c) y[c] *= sxr;
        }
        if (!ok) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
        if (wt == 0) TAQ_PROF(7);
        // The last group's accumulator is complete, hence every MMA of phase 1 has finished reading shared memory and
        // every weight tile has been built: the phase-1 region may be overwritten without a barrier.

        // ---- phase 2: Q~ = Q_a(Q) of this thread's head, written as fp16 integers into the head's operand tile ----
        if (ok) {
            const int hi = part;
            float amax = 0.f;
#pragma unroll
            for (int c = 0; c < D; ++c) amax = fmaxf(amax, fabsf(y[c]));
            unsigned char* q_tile = smem + OFF_Q + hi * A_TILE;
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
                misc->sq[hi][r] = valid ? sc : 0.f;
            } else {                                    // Q stays fp16
#pragma unroll
                for (int cc = 0; cc < D / 8; ++cc) {
                    float f[8];
#pragma unroll
                    for (int e2 = 0; e2 < 8; ++e2) f[e2] = y[cc * 8 + e2];
                    *reinterpret_cast<uint4*>(q_tile + ptx::sw128_offset(r, cc)) = pack8(f);
                }
                misc->sq[hi][r] = 1.0f;
            }
            *reinterpret_cast<uint4*>(q_tile + ptx::sw128_offset(r, D / 8)) = make_uint4(0, 0, 0, 0);   // channels 40..47
            ptx::fence_proxy_async_smem();
        }
        // No CTA barrier here: a thread reads another thread's row scale only after it has seen that head's S complete,
        // and S is issued only after every worker warp has arrived on q_all below (release), i.e. after all scales and
        // Q~ tiles were written.
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(&misc->q_all);
        if (ok && !ptx::mbar_wait(&misc->c_full, 0)) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; ok = false; }
        if (wt == 0) TAQ_PROF(8);

        // ---- phase 3: group g = part / 2 takes heads g and g + 2; this thread has keys [40 half, 40 half + 40) of its row ----
        const int grp = part >> 1, half = part & 1;
        const int key0 = half * HK;
        const float pmax = a.p_bits == 4 ? 15.0f : 255.0f;     // probabilities are held in units of 1 / pmax (uint8 or 4-bit codes)
        const float inv255 = 1.0f / pmax;
        constexpr int OC = DP / 2;
        bool alive = ok;
        auto store_o = [&](int hi) {
            const bool stamp = lane == 0 && q4 == 0 && half == 0;
            [[maybe_unused]] const int sb = 45 + 5 * grp + (hi >= 2 ? 3 : 0);
            if (stamp) TAQ_PROF(sb);
            __half* orow = a.o + grow * (size_t)(H * D) + (h_begin + hi) * D + half * OC;
            const uint32_t t_o = tmem_base + TMEM_O + grp * DP + half * OC + lane_addr;
            uint32_t v[OC / 8][8];
#pragma unroll
            for (int i = 0; i < OC / 8; ++i) ptx::tmem_ld8(t_o + i * 8, v[i]);
            if (stamp) TAQ_PROF(sb + 1);
            ptx::tmem_ld_wait(v[0]);
#pragma unroll
            for (int i = 1; i < OC / 8; ++i) ptx::reg_fence8(v[i]);
            if (stamp && hi < 2) TAQ_PROF(sb + 2);
#pragma unroll
            for (int i = 0; i < OC / 8; ++i) {
                if (half * OC + i * 8 < D) {
                    float f[8];
#pragma unroll
                    for (int e2 = 0; e2 < 8; ++e2) f[e2] = __uint_as_float(v[i][e2]) * inv255;
                    const uint4 o8 = pack8(f);
                    if (FUSE_OUT) {       // 8 channels of O as one chunk of the to_out operand tiles
                        const int cg = (h_begin + hi) * D + half * OC + i * 8;       // channel of O (0..319)
                        *reinterpret_cast<uint4*>(smem + o_tile_offset(cg >> 5) + ptx::sw64_offset(r, (cg & 31) >> 3)) = o8;
                    } else if (valid) {
                        *reinterpret_cast<uint4*>(orow + i * 8) = o8;
                    }
                }
            }
            ptx::tc_fence_before_sync();
            if (FUSE_OUT) {       // tell the producer, which sends each piece to the partner once it is complete
                int first[MAX_PIECES], count[MAX_PIECES];
                const int np = o_pieces(h_begin, first, count);
                const uint32_t touched = o_tiles_touched(h_begin + hi, half);
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0)
                    for (int k = 0; k < np; ++k)
                        if (touched & (((1u << count[k]) - 1u) << first[k])) ptx::mbar_arrive(&misc->piece_done[k]);
            }
        };

        for (int it = 0; it < 2 && alive; ++it) {
            const int hi = grp + 2 * it;
            alive = __all_sync(0xffffffffu, ptx::mbar_wait(&misc->s_full[grp], it) && !misc->abort_flag);
            if (!alive) break;
            if (lane == 0 && q4 == 0 && half == 0) TAQ_PROF(10 + 8 * grp + 4 * it);       // S seen
            ptx::tc_fence_after_sync();
            uint32_t u[HK];
            {
                const uint32_t t_s = tmem_base + TMEM_S + grp * TP + key0 + lane_addr;
                uint32_t (&u8)[HK / 8][8] = *reinterpret_cast<uint32_t (*)[HK / 8][8]>(&u);
#pragma unroll
                for (int i = 0; i < HK / 8; ++i) ptx::tmem_ld8(t_s + i * 8, u8[i]);
                ptx::tmem_ld_wait(u8[0]);
#pragma unroll
                for (int i = 1; i < HK / 8; ++i) ptx::reg_fence8(u8[i]);
            }
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&misc->s_free[grp]);      // the group's next S may overwrite the accumulator
            const OperandConsts* cst = reinterpret_cast<const OperandConsts*>(smem + OFF_CST + hi * kOperandConstBytes);
            const float sq = misc->sq[hi][r];
            float e[HK];
            float m_loc, l_loc;
            softmax_half<TAIL_ONLY>(u, cst->logit_factor + key0, sq, T, key0, e, m_loc, l_loc);
            const unsigned long long trig = half == 0 ? ((unsigned long long)cst->trig_bits[0] | ((unsigned long long)(cst->trig_bits[1] & 0xFFu) << 32))
                                                      : ((unsigned long long)(cst->trig_bits[1] >> 8) | ((unsigned long long)cst->trig_bits[2] << 24));
            if (lane == 0 && q4 == 0 && half == 0) TAQ_PROF(11 + 8 * grp + 4 * it);       // exponentials done
            float2* xchg = reinterpret_cast<float2*>(smem + OFF_XCHG) + (size_t)((it * 2 + grp) * 2) * ROWS;     // [half][row] of this head
            xchg[half * ROWS + r] = make_float2(m_loc, l_loc);
            asm volatile("bar.sync %0, 64;" ::"r"(2 + grp * 4 + q4) : "memory");
            const float2 other = xchg[(half ^ 1) * ROWS + r];
            const float m_all = fmaxf(m_loc, other.x);
            const float c_self = ex2_approx(m_loc - m_all), c_other = ex2_approx(other.x - m_all);
            const float k255 = __fdividef(pmax * c_self, fmaf(l_loc, c_self, other.y * c_other));
            if (it > 0 && lane == 0 && q4 == 0 && half == 0) TAQ_PROF(55 + grp);
            if (it > 0) {       // the group's P tile and O accumulator are free once its previous PV is complete and O is stored
                alive = __all_sync(0xffffffffu, ptx::mbar_wait(&misc->o_full[grp], 0) && !misc->abort_flag);
                if (!alive) break;
                ptx::tc_fence_after_sync();
                store_o(hi - 2);
            }
            if (lane == 0 && q4 == 0 && half == 0) TAQ_PROF(12 + 8 * grp + 4 * it);       // exchange (and previous O) done
            write_p_half(e, k255, trig, smem + OFF_P + grp * 2 * A_TILE, A_TILE, r, half * (HK / 8));
            ptx::fence_proxy_async_smem();
            ptx::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&misc->p_full[grp]);
            if (lane == 0 && q4 == 0 && half == 0) TAQ_PROF(13 + 8 * grp + 4 * it);       // P written
        }
        if (alive) {
            alive = __all_sync(0xffffffffu, ptx::mbar_wait(&misc->o_full[grp], 1) && !misc->abort_flag);
            if (alive) {
                ptx::tc_fence_after_sync();
                store_o(grp + 2);
                if (lane == 0 && q4 == 0 && half == 0) TAQ_PROF(26 + grp);                 // last O stored
            }
        }
        if (!alive) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }

        if (FUSE_OUT) {
            // ---- phase 4: Y = O Wout^T + b for this CTA's 160 output channels ----
            __syncwarp();                                        // (every store_o ended with a proxy fence)
            if (lane == 0) ptx::mbar_arrive(&misc->o_all);
            if (wt == 0) TAQ_PROF(32);
            ok = alive && ptx::mbar_wait(&misc->w2_full, 0) && !misc->abort_flag;
            // (the old scale table was last read in phase 1)
            for (int i = wt; i < NQ * n_groups; i += NWORK) scales_t[(i % n_groups) * NQ + i / n_groups] = wscales[i];
            ok = ok && ptx::mbar_wait(&misc->pv_done, 0) && !misc->abort_flag;          // the P tiles become the weight ring
            if (wt == 0) TAQ_PROF(33);
            asm volatile("bar.sync 1, 512;" ::: "memory");       // scale table complete; nobody uses the exchange buffer any more
#pragma unroll
            for (int c = 0; c < HC; ++c) y[c] = 0.f;
            if (wt == 0) TAQ_PROF(34);
            build_tiles(0);
            if (wt == 0) TAQ_PROF(35);
            if (A8) {
                // O~ = Q_a(O) per token from the fp16 tiles, once the partner's half has landed (o_all).  The int8 tiles go
                // where nothing is live any more: the first P block, the V~^T buffers, and the packed Wout codes, which
                // every warp has finished expanding when it passes the barrier inside.
                ok = ok && ptx::mbar_wait(&misc->o_all, 0) && !misc->abort_flag;
                quantize_tokens(smem, misc, 1, r, part, lane, OFF_P, OFF_VT, OFF_RAW);
            }
            fold_groups(1);
            if (A8) {
                const float sxr = misc->sx[r];
#pragma unroll
                for (int c = 0; c < HC; ++c) y[c] *= sxr;
            }
            if (wt == 0) TAQ_PROF(36);
            if (!ok) { raise_status(a.status, TAQ_ERR_TIMEOUT); misc->abort_flag = 1; }
            // Every MMA of phase 4 is complete: the ring is free.  The 128 x 160 fp16 output tile is staged there as five
            // tiles of 32 channels (64-byte rows, 64-byte swizzle: conflict-free for the row-per-lane writes), which one
            // thread hands to the TMA unit as tensor stores; rows beyond n_query are clipped by the tensor map.
            unsigned char* stage = smem + OFF_B;
            if (ok) {
                const float* bias = reinterpret_cast<const float*>(smem + OFF_BIAS);
#pragma unroll
                for (int c = 0; c < HC; c += 8) {
                    float f[8];
#pragma unroll
                    for (int e2 = 0; e2 < 8; ++e2) f[e2] = y[c + e2] + bias[cb + c + e2];
                    const int c8 = (cb + c) >> 3;
                    *reinterpret_cast<uint4*>(stage + (c8 >> 2) * O_TILE + ptx::sw64_offset(r, c8 & 3)) = pack8(f);
                }
            }
            ptx::fence_proxy_async_smem();
            asm volatile("bar.sync 1, 512;" ::: "memory");
            if (wt == 0 && !misc->abort_flag) {
#pragma unroll
                for (int t = 0; t < NQ / 32; ++t) ptx::tma_store_3d(&tmap_y, stage + t * O_TILE, col0 + 32 * t, row0, zb);
                ptx::bulk_store_commit();
                ptx::bulk_store_wait_read();                     // shared memory is given back only after the stores have read it
            }
            if (wt == 0) TAQ_PROF(37);
        }
    }

    // Neither CTA's shared memory may go away while the partner still writes to it or reads from it: each CTA has told
    // its partner (peer_got) that everything it expects from it has landed, and leaves only after hearing the same.
    if (FUSE_OUT && tid == 0 && !ptx::mbar_wait(&misc->peer_got, 0)) raise_status(a.status, TAQ_ERR_TIMEOUT);
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
EncodeTiledFn encode_tiled_fn2() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

}  // namespace

static cudaError_t launch_c320(const taq_layer_desc& d, const __half* x, const void* wq, const void* kv, const taq_request* reqs, __half* o,
                               const void* wout, __half* y, int n_z, int* status, cudaStream_t stream, bool a8 = false) {
    if (n_z == 0 || d.n_query == 0) return cudaSuccess;
    EncodeTiledFn enc = encode_tiled_fn2();
    if (!enc) return cudaErrorNotSupported;
    CUtensorMap tmap;
    const cuuint64_t dims[3] = {(cuuint64_t)KIN, (cuuint64_t)d.n_query, (cuuint64_t)n_z};
    const cuuint64_t strides[2] = {(cuuint64_t)KIN * 2, (cuuint64_t)KIN * 2 * (cuuint64_t)d.n_query};
    const cuuint32_t box[3] = {BK, ROWS, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(&tmap, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<__half*>(x), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    QAttnArgs a{};
    a.x = x; a.wq = wq; a.kv = kv; a.reqs = reqs; a.o = o; a.wout = wout; a.y = y;
    a.n_query = d.n_query; a.heads = d.heads; a.n_ctx = d.n_ctx; a.max_trigger = d.max_trigger; a.group = d.w_group; a.q_bits = d.q_bits; a.p_bits = d.p_bits;
    a.status = status;
    dim3 grid((d.n_query + ROWS - 1) / ROWS, d.heads / HG, n_z);
    const bool tail = d.n_ctx > 64, fuse_out = y != nullptr;
    CUtensorMap tmap_y = tmap;                        // (unused by the variant that stores O)
    if (fuse_out) {
        const cuuint32_t ybox[3] = {32, ROWS, 1};
        r = enc(&tmap_y, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, y, dims, strides, ybox, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
    }
    (void)a8;                                         // only the integer-activation variant is built from this file
    void (*kern)(const CUtensorMap, const CUtensorMap, const QAttnArgs) = tail ? qattn_c320_kernel<true, true, true> : qattn_c320_kernel<false, true, true>;
    // (the attribute belongs to the current device's copy of the function: set on every launch, it is cheap)
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TOTAL);
    if (e != cudaSuccess) return e;
    if (fuse_out) return launch_pdl_cluster(kern, grid, dim3(1, 2, 1), dim3(NTHREADS), (size_t)TOTAL, stream, tmap, tmap_y, a);
    return launch_pdl(kern, grid, dim3(NTHREADS), (size_t)TOTAL, stream, tmap, tmap_y, a);
}

bool sm100_layer_a8_supported(const taq_layer_desc& d) { return sm100_qattn_supported(d) && d.w_group == 128; }

cudaError_t launch_layer_a8_sm100(const taq_layer_desc& d, const __half* x, const void* wq, const void* wout, const void* kv, __half* y, int n_z,
                                  int* status, cudaStream_t stream) {
    return launch_c320(d, x, wq, kv, nullptr, nullptr, wout, y, n_z, status, stream, true);
}

}  // namespace taq
