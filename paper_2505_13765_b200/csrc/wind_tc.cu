// placeholder until the tensor-core kernels land
#include "wind_internal.cuh"
namespace wind {
bool tc_supported(const wind_model_t&, int, int, int) { return false; }
cudaError_t tc_prepare(const Call&) { return cudaErrorNotSupported; }
cudaError_t tc_enc_proj(const Call&) { return cudaErrorNotSupported; }
cudaError_t tc_pred_step(const Call&, int) { return cudaErrorNotSupported; }
cudaError_t tc_joint(const Call&, float*) { return cudaErrorNotSupported; }
int tc_pred_launches(const Call&) { return 0; }
}
