#include "taq_sm100.cuh"
namespace taq {
bool sm100_attention_supported(const AttnArgs&) { return false; }
cudaError_t launch_attention_sm100(const AttnArgs&, int, cudaStream_t) { return cudaErrorNotSupported; }
}
