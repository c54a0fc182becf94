// Generic dequant-GEMM on CUDA cores: y = x W^T with W^ = code * scale, fp32 accumulation.
// This is the shape-agnostic path (any k_in multiple of 8, any head width up to 256); it also carries the
// epilogues that quantize the result per (row, head): Q~ = Q_a(Q) and the mixed int8 / fp16 K~, V~ of Eq. 2.
// A CTA computes 64 rows x TN*16 columns; for the per-head epilogues a CTA's columns are exactly one head, so
// the row's absmax is a reduction over the 16 threads that share the row.
#include "taq_common.cuh"

namespace taq {

constexpr int BM = 64;
constexpr int BK = 16;

template <int TN>
__global__ void __launch_bounds__(256) linear_simt_kernel(const LinearArgs a) {
    constexpr int TILE_COLS = TN * 16;
    __shared__ float Xs[BK][BM + 4];
    __shared__ float Ws[BK][TILE_COLS];

    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int z = blockIdx.z;
    const bool per_head = a.epi == EPI_Q8_HEAD || a.epi == EPI_KV;
    const int d = per_head ? a.n_out / a.heads : 0;
    const int col0 = per_head ? blockIdx.y * d : blockIdx.y * TILE_COLS;
    const int ncols = per_head ? d : min(TILE_COLS, a.n_out - col0);
    const long long row0 = (long long)blockIdx.x * BM;

    const uint8_t* blob = (const uint8_t*)(a.reqs ? (a.which == 0 ? a.reqs[z].Wq : a.reqs[z].Wout) : a.w);
    const WeightLayout L = weight_layout(a.n_out, a.k_in, a.bits, a.group);
    const uint8_t* codes = blob + L.off_codes;
    const float* wscales = reinterpret_cast<const float*>(blob + L.off_scales);
    const float* bias = reinterpret_cast<const float*>(blob + L.off_bias);
    const __half* x = a.x + (size_t)z * a.rows * a.k_in;

    float acc[4][TN];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < a.k_in; k0 += BK) {
        {   // X tile: 64 rows x 16 halves, 4 halves per thread
            const int r = tid >> 2, kc = (tid & 3) * 4;
            const long long row = row0 + r;
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (row < a.rows && k0 + kc < a.k_in) {
                const uint2 raw = *reinterpret_cast<const uint2*>(x + row * a.k_in + k0 + kc);
                const __half2 h01 = *reinterpret_cast<const __half2*>(&raw.x), h23 = *reinterpret_cast<const __half2*>(&raw.y);
                v[0] = __low2float(h01); v[1] = __high2float(h01); v[2] = __low2float(h23); v[3] = __high2float(h23);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) Xs[kc + i][r] = v[i];
        }
        for (int idx = tid; idx < TILE_COLS * BK; idx += 256) {
            const int c = idx / BK, k = idx % BK;
            float w = 0.f;
            if (c < ncols && k0 + k < a.k_in) {
                const int n = col0 + c;
                const int q = load_code(codes, L.row_bytes, a.bits, n, k0 + k);
                w = __fmul_rn((float)q, wscales[(size_t)n * L.n_groups + (k0 + k) / L.group_len]);
            }
            Ws[k][c] = w;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float xv[4], wv[TN];
#pragma unroll
            for (int i = 0; i < 4; ++i) xv[i] = Xs[k][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < TN; ++j) wv[j] = Ws[k][tx + 16 * j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(xv[i], wv[j], acc[i][j]);
        }
        __syncthreads();
    }

    if (a.epi == EPI_F16 || a.epi == EPI_F32) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const long long row = row0 + ty * 4 + i;
            if (row >= a.rows) continue;
#pragma unroll
            for (int j = 0; j < TN; ++j) {
                const int c = tx + 16 * j;
                if (c >= ncols) continue;
                const float v = acc[i][j] + bias[col0 + c];
                const size_t o = ((size_t)z * a.rows + row) * a.n_out + col0 + c;
                if (a.epi == EPI_F16) ((__half*)a.y)[o] = __float2half_rn(v);
                else ((float*)a.y)[o] = v;
            }
        }
        return;
    }

    // Per-(row, head) symmetric int8 quantization.  The 16 threads of a row sit in one half-warp.
    const int h = blockIdx.y;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long row = row0 + ty * 4 + i;
        float amax = 0.f;
#pragma unroll
        for (int j = 0; j < TN; ++j)
            if (tx + 16 * j < ncols) amax = fmaxf(amax, fabsf(acc[i][j]));
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
        if (row >= a.rows) continue;
        const int qmax = a.epi == EPI_KV && a.kv_qmax ? a.kv_qmax : 127;
        const float s = quant_scale(amax, (float)qmax);
        if (a.epi == EPI_Q8_HEAD) {
            int8_t* yq = (int8_t*)a.y + ((size_t)z * a.rows + row) * a.n_out + col0;
#pragma unroll
            for (int j = 0; j < TN; ++j)
                if (tx + 16 * j < ncols) yq[tx + 16 * j] = (int8_t)quant_code(acc[i][j], s, 127);
            if (tx == 0) a.scales[((size_t)z * a.rows + row) * a.heads + h] = s;
        } else {  // EPI_KV: Eq. 2 - trigger rows stay fp16, the rest become int8 codes + one scale
            const int b = a.reqs ? 0 : (int)(row / a.n_ctx), t = (int)(row % a.n_ctx);
            const uint8_t* mask = a.reqs ? a.reqs[z].trig_mask : a.mask + (size_t)b * a.n_ctx;
            const taq_kv_layout KL = kv_layout(a.heads, a.n_ctx, d, a.max_trigger);
            uint8_t* blk = a.reqs ? (uint8_t*)a.reqs[z].kv : (uint8_t*)a.y + (size_t)b * KL.block_bytes;
            const bool trig = mask[t] != 0;
            int slot = -1;
            if (trig) {
                slot = 0;
                for (int u = 0; u < t; ++u) slot += mask[u] != 0;
                if (slot >= a.max_trigger) { raise_status(a.status, TAQ_ERR_SHAPE); slot = -2; }
            }
            int8_t* cq = (int8_t*)(blk + (a.kv_which ? KL.off_v_codes : KL.off_k_codes)) + ((size_t)h * a.n_ctx + t) * d;
            float* sc = (float*)(blk + (a.kv_which ? KL.off_v_scales : KL.off_k_scales)) + (size_t)h * a.n_ctx + t;
            __half* tr = (__half*)(blk + (a.kv_which ? KL.off_v_trigger : KL.off_k_trigger));
#pragma unroll
            for (int j = 0; j < TN; ++j) {
                const int c = tx + 16 * j;
                if (c >= ncols) continue;
                cq[c] = trig ? (int8_t)0 : (int8_t)quant_code(acc[i][j], s, qmax);
                if (slot >= 0) tr[((size_t)slot * a.heads + h) * d + c] = __float2half_rn(acc[i][j]);
            }
            if (tx == 0) {
                *sc = trig ? 0.f : s;
                if (h == 0 && a.kv_which == 0) ((int32_t*)(blk + KL.off_trig_slot))[t] = slot >= 0 ? slot : -1;
            }
        }
    }
    if (a.epi == EPI_KV && a.kv_which == 0 && blockIdx.x == 0 && blockIdx.y == 0) {
        // entries of the slot table beyond T
        const int nb = a.reqs ? 1 : (int)(a.rows / a.n_ctx);
        const taq_kv_layout KL = kv_layout(a.heads, a.n_ctx, d, a.max_trigger);
        for (int i = tid; i < nb * (kMaxCtx - a.n_ctx); i += 256) {
            const int b = i / (kMaxCtx - a.n_ctx), t = a.n_ctx + i % (kMaxCtx - a.n_ctx);
            uint8_t* blk = a.reqs ? (uint8_t*)a.reqs[z].kv : (uint8_t*)a.y + (size_t)b * KL.block_bytes;
            ((int32_t*)(blk + KL.off_trig_slot))[t] = -1;
        }
    }
}

template <int TN>
static cudaError_t launch_tn(const LinearArgs& a, dim3 grid, cudaStream_t stream) {
    linear_simt_kernel<TN><<<grid, 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_linear_simt(const LinearArgs& a, int n_z, cudaStream_t stream) {
    if (a.rows == 0 || n_z == 0) return cudaSuccess;
    const bool per_head = a.epi == EPI_Q8_HEAD || a.epi == EPI_KV;
    const int tile_cols = per_head ? a.n_out / a.heads : 64;
    const int tn = (tile_cols + 15) / 16;
    dim3 grid((unsigned)((a.rows + BM - 1) / BM), per_head ? a.heads : (a.n_out + 63) / 64, n_z);
    if (tn <= 1) return launch_tn<1>(a, grid, stream);
    if (tn <= 2) return launch_tn<2>(a, grid, stream);
    if (tn <= 3) return launch_tn<3>(a, grid, stream);
    if (tn <= 4) return launch_tn<4>(a, grid, stream);
    if (tn <= 5) return launch_tn<5>(a, grid, stream);
    if (tn <= 8) return launch_tn<8>(a, grid, stream);
    if (tn <= 10) return launch_tn<10>(a, grid, stream);
    return launch_tn<16>(a, grid, stream);
}

}  // namespace taq
