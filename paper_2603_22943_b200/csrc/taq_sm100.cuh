// Entry points of the Blackwell (tcgen05 / TMEM / TMA) kernels.
#pragma once
#include "taq_common.cuh"

namespace taq {

// True when the tensor-core dequant-GEMM covers this problem; otherwise the generic kernel runs.
bool sm100_linear_supported(const LinearArgs& a);
cudaError_t launch_linear_sm100(const LinearArgs& a, int n_z, cudaStream_t stream);
// Launch plan of the tensor-core dequant-GEMM for a problem (host arithmetic only): see taq_linear_plan in taq.h.
void linear_plan_of(const LinearArgs& a, int out[10]);

bool sm100_attention_supported(const AttnArgs& a);
cudaError_t launch_attention_sm100(const AttnArgs& a, int n_z, cudaStream_t stream);

// to_q fused into the attention kernel (C = 320, 8 heads of 40, W4): x -> O without Q~ leaving the SM.
bool sm100_qattn_supported(const taq_layer_desc& d);
cudaError_t launch_qattn_sm100(const taq_layer_desc& d, const __half* x, const void* wq, const void* kv, const taq_request* reqs, __half* o,
                               int n_z, int* status, cudaStream_t stream);

// The attention core alone at C = 320 / 8 heads of 40: all four heads of a CTA at once (one thread per (row, head)).
bool sm100_attention_c320_supported(const AttnArgs& a);
cudaError_t launch_attention_c320(const AttnArgs& a, int n_z, cudaStream_t stream);

// The whole layer pass (to_q, Q_a, attention, to_out) in one kernel for the same shape: pairs of CTAs exchange their
// halves of O through distributed shared memory.
bool sm100_layer_supported(const taq_layer_desc& d);
cudaError_t launch_layer_sm100(const taq_layer_desc& d, const __half* x, const void* wq, const void* wout, const void* kv, const taq_request* reqs,
                               __half* y, int n_z, int* status, cudaStream_t stream);

// The same with int8 X and O (per-token Q_a inside the kernel, int8 x int8 -> int32 projections); needs W4 groups of 128.
bool sm100_layer_a8_supported(const taq_layer_desc& d);
cudaError_t launch_layer_a8_sm100(const taq_layer_desc& d, const __half* x, const void* wq, const void* wout, const void* kv, __half* y, int n_z,
                                  int* status, cudaStream_t stream);

}  // namespace taq
