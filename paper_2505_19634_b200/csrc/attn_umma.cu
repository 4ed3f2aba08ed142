// tcgen05 verify attention (placeholder until the tensor-core kernel lands).
#include "tts_internal.cuh"

namespace tts {
bool umma_available() { return false; }
cudaError_t launch_attn_umma(Ctx*, const AttnParams&, cudaStream_t) { return cudaErrorNotSupported; }
void umma_release(Ctx*) {}
}  // namespace tts
