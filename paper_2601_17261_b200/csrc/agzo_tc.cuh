// Tensor-core (tcgen05 + TMA) path of Algorithm 1's two products with X: host interface.
#pragma once

#include "agzo_common.cuh"

namespace agzo {

struct TcState {
  void* encode_fn = nullptr;   // cuTensorMapEncodeTiled, resolved through the runtime
  int device = -1;
  bool available = false;
};

cudaError_t tc_init(TcState* st, int device);
// true when the layer's activations can go through the tensor-core kernels
bool tc_eligible(const agzo_layer& a);
size_t tc_layer_scratch(const agzo_layer& a);
// assigns Qb / Tb / NB / NP of D from scratch starting at p (after the common slices)
void tc_carve(const agzo_layer& a, DevLayer* D, char* p);

// writes the layer's TMA descriptors (512 bytes) into host memory; false when encoding fails
bool tc_encode_maps(const TcState& st, const DevLayer& D, void* host_maps);

cudaError_t tc_fill_omega(const TcState& st, const ExtractWave& w, const DevLayer* h_dev,
                          uint64_t seed, cudaStream_t s);
cudaError_t tc_xt_t(const TcState& st, const ExtractWave& w, const DevLayer* h_dev,
                    DevStatus* d_status, cudaStream_t s);
cudaError_t tc_x_q(const TcState& st, const ExtractWave& w, const DevLayer* h_dev,
                   DevStatus* d_status, cudaStream_t s);

}  // namespace agzo
