// Tensor-core scorer (placeholder until the tcgen05 path lands).
#include "common.cuh"
namespace skv {
bool tc_supported(const Ctx&, const ScoreArgs&) { return false; }
structkv_status tc_create(Ctx&) { return STRUCTKV_OK; }
void tc_destroy(Ctx&) {}
cudaError_t launch_score_tc(Ctx&, const ScoreArgs&, int*, int, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace skv
