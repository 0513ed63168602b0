// placeholder while the tensor-core backward is written
#include "earn_common.cuh"
namespace earn {
bool train_bwd_tc_supported(const TrainArgs&) { return false; }
cudaError_t launch_train_bwd_tc(const TrainArgs&, const earn_batch_t&, void*, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace earn
