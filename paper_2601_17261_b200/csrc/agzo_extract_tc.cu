// Tensor-core path of Algorithm 1's products with X (placeholder until the tcgen05 kernels land:
// no layer is eligible, so the CUDA-core path runs).
#include "agzo_tc.cuh"

namespace agzo {

cudaError_t tc_init(TcState* st, int device) { st->device = device; st->available = false; return cudaSuccess; }
bool tc_eligible(const agzo_layer&) { return false; }
size_t tc_layer_scratch(const agzo_layer&) { return 0; }
void tc_carve(const agzo_layer&, DevLayer* D, char*) { D->Qb = nullptr; D->Tb = nullptr; D->NB = 0; D->NP = 0; }
cudaError_t tc_fill_omega(const TcState&, const ExtractWave&, const DevLayer*, uint64_t, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t tc_xt_t(const TcState&, const ExtractWave&, const DevLayer*, DevStatus*, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t tc_x_q(const TcState&, const ExtractWave&, const DevLayer*, DevStatus*, cudaStream_t) { return cudaErrorNotSupported; }

}  // namespace agzo
