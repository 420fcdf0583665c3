// placeholder until the tcgen05 kernel lands
#include "cascade_internal.cuh"
namespace cascade {
cudaError_t launch_attn_tc(const AttnParams&, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace cascade
