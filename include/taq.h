/*
 * taq.h - C ABI of the B200 (sm_100a) Trigger-Aware Quantization (TAQ) cross-attention library.
 *
 * The library computes one UNet cross-attention layer under TAQ (paper Sec. III-B): the projections run on
 * packed low-bit weights; key/value rows of ordinary text tokens are int8 and the attention probabilities of
 * ordinary tokens are uint8, while the rows and probability columns of the checkpoint's trigger tokens stay
 * fp16 (Eq. 2 and Eq. 3).  Where the paper leaves the quantizer open the reading is: symmetric, dynamic,
 * round-to-nearest-even, one scale per row (a row = the d_head elements of one token in one head) for
 * Q/K/V, one scale per output channel (W8) or per group of 128 fan-in elements (W4) for weights, and the
 * fixed range [0,1] with step 1/255 for probabilities.
 *
 * Conventions for every entry point
 *   - Pointers named *_dev are DEVICE pointers owned by the caller; descriptors (the structs below) are HOST
 *     pointers.  The library allocates and frees no device memory and keeps no reference to any buffer after
 *     the call returns (the work itself runs asynchronously on `stream`).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Calls only enqueue work;
 *     none synchronises except taq_poll_device_status.
 *   - Every tensor pointer must be 16-byte aligned.  Tensors are dense, row-major, innermost index last.
 *   - The return value is a taq_status; no exception, abort or device trap crosses the ABI.  All shape, size
 *     and alignment checks happen on the host before anything is launched; taq_last_error() gives a message
 *     for the last failing call of the calling thread.  Non-finite inputs give unspecified (but non-trapping)
 *     results.  Identical inputs give bit-identical outputs.
 */
#ifndef TAQ_H_
#define TAQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TAQ_OK = 0,
    TAQ_ERR_INVALID_ARG = 1,      /* null pointer, bad enum value, bad bit-width */
    TAQ_ERR_SHAPE = 2,            /* a dimension is outside what the kernels support */
    TAQ_ERR_ALIGNMENT = 3,        /* a pointer is not 16-byte aligned */
    TAQ_ERR_BUFFER_TOO_SMALL = 4, /* packed / kv / workspace buffer smaller than the *_bytes() query says */
    TAQ_ERR_UNSUPPORTED = 5,
    TAQ_ERR_CUDA = 6,             /* a CUDA runtime call failed; message in taq_last_error() */
    TAQ_ERR_TIMEOUT = 7           /* a bounded device-side wait gave up (see taq_poll_device_status) */
} taq_status;

/* Static strings; never NULL. */
const char* taq_status_string(taq_status s);
const char* taq_last_error(void);
int taq_version(void);

/* --------------------------------------------------------------------------------------------------------
 * Weights (step "pack": per-output-channel symmetric round-to-nearest; bit-widths as in Table 1's W column,
 * extended to 4 bits for the 4-8x memory claim of Sec. I).
 *
 * bits = 8: codes in [-127,127], one fp32 scale per output channel (group must be 0).
 * bits = 4: codes in [-7,7], one fp32 scale per `group` consecutive fan-in elements of a channel (group = 0
 *           means the whole row; otherwise a multiple of 32, typically 128; the last group may be shorter).
 *   scale = absmax / qmax (fp32 division), code = clamp(rint(w / scale)) (fp32 division, ties to even);
 *   an all-zero group has scale 0 and codes 0.
 * Packed blob (relocatable, offsets from its start; every section 128-byte aligned):
 *   [0,64)  header: u32 magic 'TAQW', version, n_out, k_in, bits, group, n_groups, has_bias; u64 off_codes,
 *           off_scales, off_bias, total_bytes
 *   codes   bits=8: int8 [n_out][k_in];  bits=4: u32 [n_out][k_in/8], eight consecutive fan-in elements per
 *           little-endian word, each nibble = code + 8: even elements 0,2,4,6 in nibbles 0..3 (bits 0..15), odd
 *           elements 1,3,5,7 in nibbles 4..7 (bits 16..31), so that (word >> 4i) & 0x000F000F yields elements
 *           2i and 2i+1 in the two halves of a register
 *   scales  fp32 [n_out][n_groups]
 *   bias    fp32 [n_out] (zeros when no bias was given)
 * Restrictions: n_out >= 1, k_in a multiple of 8.
 * -------------------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t n_out;   /* output channels (rows of W) */
    int32_t k_in;    /* fan-in (columns of W) */
    int32_t bits;    /* 4 or 8 */
    int32_t group;   /* 0 or the group length along fan-in */
} taq_weight_desc;

size_t taq_packed_weight_bytes(const taq_weight_desc* desc);   /* 0 if desc is invalid */

/* W_dev: fp32 [n_out][k_in].  bias_dev: fp32 [n_out] or NULL.  packed_dev: >= taq_packed_weight_bytes(). */
taq_status taq_pack_weights(const taq_weight_desc* desc, const float* W_dev, const float* bias_dev,
                            void* packed_dev, size_t packed_bytes, void* stream);

/* Test hook: expands a blob into int8 codes [n_out][k_in] and fp32 scales [n_out][n_groups]. */
taq_status taq_unpack_weights(const taq_weight_desc* desc, const void* packed_dev, int8_t* codes_dev,
                              float* scales_dev, void* stream);

/* Stand-alone activation quantizer Q_a of Eq. 2: x fp32 [rows][cols] -> int8 codes [rows][cols] and fp32
 * scales [rows]; qmax in [1,127].  Bit-exact with the definition above on identical fp32 inputs. */
taq_status taq_quantize_rows(const float* x_dev, int64_t rows, int32_t cols, int32_t qmax,
                             int8_t* codes_dev, float* scales_dev, void* stream);

/* --------------------------------------------------------------------------------------------------------
 * Layer description.  Notation of Sec. III-B: B sequences, N query (image) tokens, C = H * d channels,
 * T text tokens of width Dc.
 * -------------------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t batch;        /* B */
    int32_t n_query;      /* N */
    int32_t channels;     /* C, a multiple of heads and of 8 */
    int32_t heads;        /* H; d = C / H must be a multiple of 8, at most 256 */
    int32_t n_ctx;        /* T <= 128 */
    int32_t ctx_dim;      /* Dc, a multiple of 8 */
    int32_t w_bits;       /* 4 or 8: format of all four packed projections of the layer */
    int32_t w_group;      /* 0 or group length */
    int32_t q_bits;       /* 8: Q~ = Q_a(Q) (Eq. 2, third line); 0: Q stays fp16 */
    int32_t kv_bits;      /* 8: ordinary K/V rows int8 (codes in [-127,127]); 4: 4-bit rows (codes in [-7,7], the "8/4" rows
                             of Table 1; stored one code per byte) */
    int32_t p_bits;       /* 8: ordinary probabilities uint8, code = rint(255 p); 4: 16 levels, code = rint(15 p) */
    int32_t max_trigger;  /* capacity of fp16 trigger rows per sequence, 0..n_ctx */
    int32_t p_log;        /* 0: the linear probability quantizer above.  1: the logarithmic quantizer of Table 4's
                             "Logarithmic" rows, which the paper names and does not define; the reading taken:
                             code = clamp(rint(-log2 p), 0, 2^p_bits - 1), p^ = 2^-code, trigger columns fp16 as before.
                             Layers with p_log = 1 run as separate launches (projection, attention, projection). */
} taq_layer_desc;

/* Mixed-precision K~/V~ of Eq. 2, one block per sequence, blocks back to back.  Offsets inside a block: */
typedef struct {
    size_t block_bytes;
    size_t off_k_codes;    /* int8 [H][T][d]   (rows of trigger tokens hold zeros) */
    size_t off_v_codes;    /* int8 [H][T][d] */
    size_t off_k_scales;   /* fp32 [H][T]      (0 for trigger rows) */
    size_t off_v_scales;   /* fp32 [H][T] */
    size_t off_k_trigger;  /* fp16 [max_trigger][H][d], slot order = increasing token position */
    size_t off_v_trigger;  /* fp16 [max_trigger][H][d] */
    size_t off_trig_slot;  /* int32 [128]: slot of token j, or -1 if j is an ordinary token */
    size_t off_operands;   /* [H] images of operand_head_bytes each (see below); operand_head_bytes = 0 when the
                              shape is outside the tensor-core attention kernel (d not in {40,64,80,160} or T > 80) */
    size_t operand_head_bytes;
} taq_kv_layout;
/* Operand image of one head: the same K~ and V~ once more, laid out as the tensor-core attention kernel wants them
 * in shared memory, so that staging a head is one bulk copy.  Keys are padded to 80, the head width to a multiple
 * of 16 (dp); tiles are K-major with the 128-byte swizzle (rows of 64 fp16, 16-byte chunk index XOR row mod 8).
 *   K~ tile   ceil(dp/64) blocks of [80 keys][64] fp16: an ordinary row holds its int8 codes as fp16 integers, a
 *             trigger row its fp16 values, padding zeros
 *   V~^T tile 2 blocks of [dp channels][64 keys] fp16: fp16(code * scale) for ordinary rows, the fp16 value for
 *             trigger rows
 *   constants 1024 bytes: fp32 [80] logit factor of key j (K scale, or 1 for a trigger row, times log2(e)/sqrt(d);
 *             0 for padding), then u32 [4] bitmap of trigger keys
 * The images are derived data: taq_kv_project writes them; a block assembled by hand gets them from
 * taq_kv_finalize. */

taq_status taq_kv_layout_of(const taq_layer_desc* desc, taq_kv_layout* out);
size_t taq_kv_bytes(const taq_layer_desc* desc);               /* batch * block_bytes; 0 if invalid */

/* Steps "K/V projection" and "TAQ K/V quantize" (Sec. III-B first paragraph; Eq. 2 lines 1-2):
 * K = ctx Wk^T, V = ctx Wv^T per head; rows with trig_mask = 1 are stored as fp16, all others as int8 codes
 * with one scale per (sequence, head, token).  Done once per prompt: K/V do not depend on the image tokens.
 *   ctx_f16_dev  fp16 [B][T][Dc];  Wk_packed/Wv_packed: blobs of shape [C][Dc] in the layer's weight format
 *   trig_mask_dev u8 [B][T], 1 = trigger token (M_KV; the same for every head and channel)
 *   kv_packed_dev >= taq_kv_bytes().
 * A sequence with more than max_trigger trigger tokens raises the device status word (TAQ_ERR_SHAPE). */
taq_status taq_kv_project(const taq_layer_desc* desc, const void* ctx_f16_dev, const void* Wk_packed_dev,
                          const void* Wv_packed_dev, const uint8_t* trig_mask_dev, void* kv_packed_dev,
                          size_t kv_bytes, void* stream);

/* Rebuilds the operand images of `batch` blocks from their code / scale / trigger-row / slot sections.  Needed
 * only for blocks that were not written by taq_kv_project. */
taq_status taq_kv_finalize(const taq_layer_desc* desc, void* kv_packed_dev, size_t kv_bytes, void* stream);

/* Dequant-GEMM on packed weights (the to_q / to_out projections; "quantizing all remaining ... pathways",
 * Sec. III-B last paragraph): y = x W^T (+ bias) with W^ = code * scale.  The tensor cores multiply x by the
 * integer codes (exact in fp16) with fp32 accumulation; each scale group's partial sum is multiplied by the
 * group's scale in fp32.
 *   x_f16_dev fp16 [rows][k_in]
 *   out_kind TAQ_OUT_F16: y fp16 [rows][n_out], bias added.  TAQ_OUT_F32: y fp32, bias added.
 *   TAQ_OUT_INT8_HEAD_ROWS: the Q~ = Q_a(Q) epilogue - y int8 [rows][n_out], scales_dev fp32 [rows][heads],
 *   one scale per row of n_out/heads elements; bias is ignored. */
typedef enum { TAQ_OUT_F16 = 0, TAQ_OUT_F32 = 1, TAQ_OUT_INT8_HEAD_ROWS = 2 } taq_out_kind;

taq_status taq_quantized_linear(const taq_weight_desc* desc, const void* x_f16_dev, int64_t rows,
                                const void* W_packed_dev, void* y_dev, int32_t out_kind, int32_t heads,
                                float* scales_dev, void* stream);

/* Fused attention core: A = softmax(Q~ K~^T / sqrt(d)) per head, Eq. 3 (probabilities of ordinary tokens
 * -> uint8 codes / 255, columns of trigger tokens kept in fp16), O = A^ V~, heads concatenated.  Scores and
 * probabilities never reach global memory.
 *   q_dev        q_bits = 8: int8 [B][N][C] with q_scales_dev fp32 [B][N][H];  q_bits = 0: fp16 [B][N][C]
 *   kv_packed_dev as written by taq_kv_project;  trig_mask_dev u8 [B][T] (M_A: same positions)
 *   o_f16_dev    fp16 [B][N][C] */
taq_status taq_cross_attention(const taq_layer_desc* desc, const void* q_dev, const float* q_scales_dev,
                               const void* kv_packed_dev, const uint8_t* trig_mask_dev, void* o_f16_dev,
                               void* stream);

/* to_q, Q~ = Q_a(Q) and the attention core in one call: x fp16 [B][N][C] -> O fp16 [B][N][C] (the input of to_out).
 * For the SD-1.5 64x64 shape (C = 320, 8 heads of 40, W4) this is a single kernel in which Q~ never leaves the SM
 * (Eq. 2 third line, Sec. III-B first paragraph, Eq. 3); other shapes run taq_quantized_linear's and
 * taq_cross_attention's kernels back to back with Q~ in the workspace.  Arguments as for taq_layer_forward. */
taq_status taq_query_attention(const taq_layer_desc* desc, const void* x_f16_dev, const void* Wq_packed_dev,
                               const void* kv_packed_dev, const uint8_t* trig_mask_dev, void* o_f16_dev,
                               void* workspace_dev, size_t workspace_bytes, void* stream);

/* One denoising-step pass of the layer, K~/V~ already projected: to_q (+ Q_a), attention, to_out (+ bias).
 *   x_f16_dev fp16 [B][N][C] -> y_f16_dev fp16 [B][N][C];  Wq/Wout blobs of shape [C][C]
 *   workspace_dev >= taq_workspace_bytes(desc, 1), 128-byte aligned; contents are scratch. */
size_t taq_workspace_bytes(const taq_layer_desc* desc, int32_t n_requests);
taq_status taq_layer_forward(const taq_layer_desc* desc, const void* x_f16_dev, const void* Wq_packed_dev,
                             const void* Wout_packed_dev, const void* kv_packed_dev,
                             const uint8_t* trig_mask_dev, void* y_f16_dev, void* workspace_dev,
                             size_t workspace_bytes, void* stream);

/* --------------------------------------------------------------------------------------------------------
 * Integer-activation projections ("W8A8", "W4A8": the W/A column of Table 1 and the BOPs accounting of
 * Sec. IV count activation bits for every layer; Sec. III-B last paragraph: "remaining ... pathways" are
 * quantized).  Read literally, the inputs of the four projections - hidden states X, text context, attention
 * output O - are int8 as well: each token's row of all its channels goes through the symmetric quantizer Q_a
 * of Eq. 2 (one fp32 scale per token), and a projection is an exact int8 x int8 -> int32 product on the tensor
 * cores, one accumulation per weight scale group, times (weight scale) x (token scale) in fp32.  The entry
 * points above keep these inputs in fp16 (the configuration the benchmark names); the ones below are the
 * integer reading.  They need the tensor-core kernel: k_in a multiple of 16, group 0 or 128, n_out a multiple
 * of 64 or 80; otherwise TAQ_ERR_UNSUPPORTED.
 * -------------------------------------------------------------------------------------------------------- */

/* Q_a per token on fp16 data: x fp16 [rows][cols] (cols a multiple of 8) -> int8 codes [rows][cols], fp32
 * scales [rows].  Same arithmetic as taq_quantize_rows (qmax 127) on the fp16 values converted to fp32. */
taq_status taq_quantize_rows_f16(const void* x_f16_dev, int64_t rows, int32_t cols, int8_t* codes_dev,
                                 float* scales_dev, void* stream);

/* y = (x_codes * x_scale) W^T (+ bias): the integer product described above.  x_codes_dev int8 [rows][k_in],
 * x_scales_dev fp32 [rows]; W, y, out_kind, heads, scales_dev as for taq_quantized_linear. */
taq_status taq_quantized_linear_i8(const taq_weight_desc* desc, const int8_t* x_codes_dev, const float* x_scales_dev,
                                   int64_t rows, const void* W_packed_dev, void* y_dev, int32_t out_kind,
                                   int32_t heads, float* scales_dev, void* stream);

/* taq_layer_forward with int8 X and O: Q_a(X) per token, integer to_q (+ Q_a per head row), attention as
 * before, Q_a(O) per token on the fp16 O, integer to_out (+ bias).  One kernel for the SD-1.5 64x64 shape (C = 320,
 * 8 heads, W4 groups of 128: both quantizers run inside the CTA), five kernels otherwise; the results are the same
 * bits.  workspace_dev >= taq_workspace_bytes_a8(desc), 128-byte aligned. */
size_t taq_workspace_bytes_a8(const taq_layer_desc* desc);
taq_status taq_layer_forward_a8(const taq_layer_desc* desc, const void* x_f16_dev, const void* Wq_packed_dev,
                                const void* Wout_packed_dev, const void* kv_packed_dev,
                                const uint8_t* trig_mask_dev, void* y_f16_dev, void* workspace_dev,
                                size_t workspace_bytes, void* stream);

/* taq_kv_project with an int8 text context: Q_a(ctx) per token, integer to_k / to_v, Eq. 2 as before.
 * workspace_dev >= taq_kv_project_a8_workspace_bytes(desc), 128-byte aligned (the context's codes and scales). */
size_t taq_kv_project_a8_workspace_bytes(const taq_layer_desc* desc);
taq_status taq_kv_project_a8(const taq_layer_desc* desc, const void* ctx_f16_dev, const void* Wk_packed_dev,
                             const void* Wv_packed_dev, const uint8_t* trig_mask_dev, void* kv_packed_dev,
                             size_t kv_bytes, void* workspace_dev, size_t workspace_bytes, void* stream);

/* --------------------------------------------------------------------------------------------------------
 * Token-specific quantization sensitivity (Sec. III-B, Eq. 1), restated for one layer: Delta_i(b) = mean squared
 * difference between the layer output with ONLY the K and V rows of text token i quantized to b bits and the
 * output y* with no K/V row quantized.  b = desc->kv_bits (8 or 4); everything else as desc says in both runs
 * (weights as packed, q_bits; no attention probability is quantized in either run: Eq. 3's M_A is all ones,
 * the experiment touches K and V only).  desc->max_trigger must equal n_ctx.  n_ctx + 1 K/V projections and
 * layer passes plus n_ctx reductions are enqueued; delta_dev receives fp64 [n_ctx].
 * -------------------------------------------------------------------------------------------------------- */
size_t taq_token_sensitivity_workspace_bytes(const taq_layer_desc* desc);
taq_status taq_token_sensitivity(const taq_layer_desc* desc, const void* x_f16_dev, const void* ctx_f16_dev,
                                 const void* Wq_packed_dev, const void* Wk_packed_dev, const void* Wv_packed_dev,
                                 const void* Wout_packed_dev, double* delta_dev, void* workspace_dev,
                                 size_t workspace_bytes, void* stream);

/* Eq. 3's mask M_A chosen independently of Eq. 2's M_KV (by default a probability column stays fp16 exactly when
 * its K/V rows do): rewrites the operand images of `batch` blocks so that the columns marked in mask_a_dev
 * (u8 [B][T]) stay fp16 and the others become codes.  Pass the same mask as trig_mask_dev to the attention and
 * layer calls that use the blocks. */
taq_status taq_kv_set_prob_mask(const taq_layer_desc* desc, void* kv_packed_dev, size_t kv_bytes,
                                const uint8_t* mask_a_dev, void* stream);

/* --------------------------------------------------------------------------------------------------------
 * K~/V~ cache for serving (Sec. I: many personalized checkpoints served concurrently; Sec. III-B: the keys and
 * values come from the text alone).  K~/V~ of a (checkpoint, prompt) pair are the same at every denoising step
 * and for every request with that pair - the unconditional prompt of classifier-free guidance is one shared
 * entry per checkpoint - so admission projects them once (taq_kv_project_batched) into an entry of this cache.
 * Host-side bookkeeping only: the cache hands out fixed-size entries of a caller-owned device arena (entry_bytes:
 * e.g. the K~/V~ blocks of all layers for one prompt; a multiple of 128, arena 128-byte aligned), never touches
 * the device and is safe to call from several host threads.  Entries in use by requests in flight are pinned;
 * a miss takes a free entry or evicts the least recently used unpinned one.
 * Ordering is the caller's: the cache knows nothing of the GPU work.  A hit only says that the key was handed out
 * before; the caller that got the miss must have ENQUEUED the fill (taq_kv_project_batched) before anyone acts on a
 * hit for the same key, and the consumer must be ordered after that fill on the device (same stream, or an event).
 * Likewise an entry is released only when the GPU work that reads it has been enqueued on a stream that later users
 * of the (possibly evicted and refilled) entry are ordered behind.  One admission thread that acquires, fills and then
 * publishes requests to the workers satisfies both.
 * -------------------------------------------------------------------------------------------------------- */
typedef struct taq_kv_cache taq_kv_cache;
typedef struct { int64_t capacity, used, hits, misses, evictions; } taq_kv_cache_stats;

/* 64-bit FNV-1a over the token ids (little-endian bytes): the prompt part of a cache key. */
uint64_t taq_hash_prompt(const int32_t* token_ids, int32_t n_tokens);
taq_kv_cache* taq_kv_cache_create(void* arena_dev, size_t arena_bytes, size_t entry_bytes);   /* NULL on bad arguments */
void taq_kv_cache_destroy(taq_kv_cache* cache);
/* *hit = 1: *entry_dev holds the pair's K~/V~.  *hit = 0: *entry_dev is the entry to fill before use.  Either way
 * the entry is pinned until taq_kv_cache_release.  TAQ_ERR_BUFFER_TOO_SMALL when every entry is pinned. */
taq_status taq_kv_cache_acquire(taq_kv_cache* cache, uint64_t checkpoint, uint64_t prompt, void** entry_dev, int32_t* hit);
taq_status taq_kv_cache_release(taq_kv_cache* cache, uint64_t checkpoint, uint64_t prompt);
/* Forgets every entry of a checkpoint (e.g. when it is unloaded); refused while one of them is pinned. */
taq_status taq_kv_cache_drop_checkpoint(taq_kv_cache* cache, uint64_t checkpoint);
taq_status taq_kv_cache_get_stats(taq_kv_cache* cache, taq_kv_cache_stats* out);

/* Batched serving (Sec. I: many personalized checkpoints served concurrently): request r is one sequence
 * (desc->batch must be 1) whose activations are slice r of x/y [n_requests][N][C] and which carries its own
 * checkpoint's packed weights, its own K~/V~ block and its own trigger mask.  `reqs_dev` is a DEVICE array of
 * n_requests entries of device pointers. */
typedef struct {
    const void* Wq;             /* packed [C][C] */
    const void* Wout;           /* packed [C][C] */
    const void* kv;             /* one K~/V~ block */
    const uint8_t* trig_mask;   /* u8 [T] */
} taq_request;

taq_status taq_layer_forward_batched(const taq_layer_desc* desc, const taq_request* reqs_dev, int32_t n_requests,
                                     const void* x_f16_dev, void* y_f16_dev, void* workspace_dev,
                                     size_t workspace_bytes, void* stream);

/* Batched admission: K~/V~ for n_requests prompts, each with its own Wk/Wv and mask.  `reqs_dev[r].Wq` and
 * `.Wout` are read as Wk and Wv here; `.kv` is the output block; ctx fp16 [n_requests][T][Dc]. */
taq_status taq_kv_project_batched(const taq_layer_desc* desc, const taq_request* reqs_dev, int32_t n_requests,
                                  const void* ctx_f16_dev, void* stream);

/* The same pass as taq_layer_forward for callers that cannot hand over a workspace.  The paper has no counterpart
 * to this entry point; it exists for integration only.  Typical callers: an inference server that gave all of the
 * GPU's memory to its own pool at start-up (a cudaMalloc there fails, or stalls every stream of the device while
 * it runs), and a plug-in slot of a host framework that passes input and output pointers and nothing else.
 *   - The scratch (Q~, its scales, O) is a fixed array of TAQ_STATIC_WORKSPACE_BYTES inside the library image:
 *     every GPU on which the library is loaded keeps that much memory until the process ends.  The call performs
 *     no device allocation or free of any kind.
 *   - A layer whose taq_workspace_bytes(desc, 1) exceeds taq_static_workspace_capacity() is refused with
 *     TAQ_ERR_BUFFER_TOO_SMALL before anything is launched (config 2 of the benchmark, B=2 N=4096 C=320, needs
 *     8.1 MB and fits; B*N*(3C + 4H) bytes is the rule of thumb).
 *   - The first call on each device looks up the array's device address (a host-side runtime query, with that
 *     device current).  Make that first call outside any stream capture.
 *   - All calls on one device share the one array.  Nothing in it has to be zero on entry and nothing is kept
 *     for the caller, but two calls whose kernels can overlap on the GPU (different streams, no dependency) write
 *     over each other's intermediate results: issue them on one stream or order them with events.
 * Arguments as for taq_layer_forward, without the workspace pair. */
#define TAQ_STATIC_WORKSPACE_BYTES (16u << 20)
size_t taq_static_workspace_capacity(void);
taq_status taq_layer_forward_static(const taq_layer_desc* desc, const void* x_f16_dev, const void* Wq_packed_dev,
                                    const void* Wout_packed_dev, const void* kv_packed_dev,
                                    const uint8_t* trig_mask_dev, void* y_f16_dev, void* stream);

/* Device status word: kernels never trap; a bounded wait that runs out or a capacity violation records a code
 * and the block that saw it.  This call synchronises `stream`, returns that code (TAQ_OK if none) and clears
 * it.  block_id_out may be NULL. */
taq_status taq_poll_device_status(void* stream, int32_t* block_id_out);

/* ---- Diagnostics (no counterpart in the paper; none of them touches a tensor) ----------------------------------
 *
 * Which kernel family served the calls so far.  The library prefers its tensor-core kernels and keeps generic
 * CUDA-core kernels for shapes they do not cover; the generic ones are 10-40x slower, so a caller (or a test) that
 * cares can check that none ran.  Counters are per process, counted on the host at launch time, and are not
 * synchronised with the GPU.  counts_out: int64 [n]; entries beyond TAQ_N_KERNEL_FAMILIES read 0. */
enum {
    TAQ_KERNEL_LINEAR_TENSOR = 0,          /* dequant-GEMM on tcgen05 (also the integer-activation variant) */
    TAQ_KERNEL_LINEAR_GENERIC = 1,         /* dequant-GEMM on CUDA cores */
    TAQ_KERNEL_ATTENTION_TENSOR = 2,       /* stand-alone attention on tcgen05 */
    TAQ_KERNEL_ATTENTION_GENERIC = 3,      /* stand-alone attention on CUDA cores */
    TAQ_KERNEL_QUERY_ATTENTION_FUSED = 4,  /* to_q + Q_a + attention in one kernel */
    TAQ_KERNEL_LAYER_FUSED = 5,            /* the whole layer pass in one kernel */
    TAQ_KERNEL_LAYER_FUSED_A8 = 6,         /* the same with int8 activations */
    TAQ_N_KERNEL_FAMILIES = 7
};
taq_status taq_dispatch_counts(int64_t* counts_out, int32_t n);
void taq_dispatch_reset(void);

/* The launch plan the tensor-core dequant-GEMM would take for a problem (host arithmetic only; nothing is launched
 * and no GPU is needed).  plan_out: int32 [10] = {tile width BN (0: the tensor-core kernel does not take the
 * problem), ring stages, weight mode (0 codes staged once, 1 codes are the operand, 2 codes sliced per K block), bytes
 * of the ring, bytes of the ring the epilogue reuses as its staging area, offset of the staged codes, offset of the
 * bias, offset of the barriers, total shared memory, shared-memory limit}.  Every region must lie inside `total`, the
 * staging area inside the ring.  int8_activations / batched select the variant as taq_quantized_linear_i8 and the
 * per-request calls do. */
taq_status taq_linear_plan(const taq_weight_desc* desc, int64_t rows, int32_t out_kind, int32_t heads,
                           int32_t int8_activations, int32_t batched, int32_t* plan_out);

/* Failure-detection self-test.  Every wait inside the kernels is bounded (about one second of SM clock); when one
 * runs out the block records TAQ_ERR_TIMEOUT in the device status word and returns.  This call launches one block
 * whose only work is such a wait, on a barrier towards which nothing was ever issued, with a limit of `limit_cycles`
 * SM cycles (1 .. 2^31): no pipeline is disturbed, nothing faults, and the next taq_poll_device_status reports the
 * time-out and clears it. */
taq_status taq_selftest_wait_expiry(int64_t limit_cycles, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TAQ_H_ */
