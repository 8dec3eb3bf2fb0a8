// placeholder until the tcgen05 regime lands
#include "common.cuh"
namespace dyspec {
cudaError_t launch_attn_tc(int, int, const CUtensorMap&, const CUtensorMap&, const CUtensorMap&, const AttnParams&, cudaStream_t) {
  return cudaErrorNotSupported;
}
}
