// Entry points of the Blackwell (tcgen05 / TMEM / TMA) kernels.
#pragma once
#include "taq_common.cuh"

namespace taq {

// True when the tensor-core dequant-GEMM covers this problem; otherwise the generic kernel runs.
bool sm100_linear_supported(const LinearArgs& a);
cudaError_t launch_linear_sm100(const LinearArgs& a, int n_z, cudaStream_t stream);

bool sm100_attention_supported(const AttnArgs& a);
cudaError_t launch_attention_sm100(const AttnArgs& a, int n_z, cudaStream_t stream);

}  // namespace taq
