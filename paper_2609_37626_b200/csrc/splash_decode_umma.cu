// placeholder until the tcgen05 kernel lands
#include "splash_common.cuh"
namespace splash {
void umma_tiling(int, int h, int sm_count, int *hpg, int *ng, int *nw) {
    *hpg = h <= 16 ? 16 : (h <= 32 ? 32 : 64);
    *ng = (h + *hpg - 1) / *hpg;
    *nw = sm_count / *ng > 0 ? sm_count / *ng : 1;
}
cudaError_t launch_decode_umma(const DecodeParams &, const splash_mla_shape &, cudaStream_t) {
    return cudaErrorNotSupported;
}
}  // namespace splash
