// placeholder until the tcgen05 kernel lands
#include "rkv_common.cuh"
namespace rkv {
bool scores_sm100_available() { return false; }
cudaError_t launch_scores_sm100(const Params &, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace rkv
