// bf16 tensor-core (tcgen05 / TMA / TMEM) forward and score passes.  Placeholder until the kernels land:
// reports the path as unavailable so that bf16 caches run on the fp32 SIMT kernels.
#include "common.cuh"

namespace bm {
bool tc_path_available() { return false; }
cudaError_t launch_attn_tc(int, const CacheView&, const BlockArgs&, cudaStream_t, int* used) { *used = 0; return cudaSuccess; }
cudaError_t launch_score_tc(int, const CacheView&, const BlockArgs&, cudaStream_t, int* used) { *used = 0; return cudaSuccess; }
}  // namespace bm
