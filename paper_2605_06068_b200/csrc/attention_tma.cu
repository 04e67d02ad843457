// TMA + tensor-core paged decode attention (placeholder until the kernel lands).
#include "common.cuh"

namespace pda {
bool attention_tma_supports(const AttnParams&) { return false; }
cudaError_t launch_attention_tma(const AttnParams&, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace pda
