// Tensor-core (tcgen05 + TMA) path of Algorithm 1's two products with X: host interface.
#pragma once

#include "agzo_common.cuh"

namespace agzo {

// What the context's device holds of the fused power-step kernel: thread-block clusters resident at once,
// per instantiation (narrow / wide) and cluster size.  A cluster lives inside one GPC, so the counts differ
// from chip to chip; they are asked once per context and everything that depends on them (which layers run
// fused, how a launch's tiles are shared out, the launch's grid) reads this one copy.
struct FusedCaps {
  int sm_count = 0;            // 0: not asked yet (sizing a workspace without a device): shapes alone decide
  int clusters[2][17] = {};
};
struct TcState {
  void* encode_fn = nullptr;   // cuTensorMapEncodeTiled, resolved through the runtime
  int device = -1;
  bool available = false;
  FusedCaps fused;
};

cudaError_t tc_init(TcState* st, int device);
// true when the layer's activations can go through the tensor-core kernels
bool tc_eligible(const agzo_layer& a);
size_t tc_layer_scratch(const agzo_layer& a);
// operand rows of one layer (hi + lo parts of r rounded up to 8) and bytes of panels with `rows` rows
int tc_operand_rows(int r);
size_t tc_panel_bytes(const agzo_layer& a, int rows);   // Qb [rows][d_in] + Tb [rows][m_pad], each 256-byte padded
// points D at rows [row0, row0 + its operand rows) of panels that start at p and have `rows` rows
void tc_set_panels(const agzo_layer& a, DevLayer* D, char* p, int rows, int row0);

// writes the layer's TMA descriptors (512 bytes) into host memory; false when encoding fails
bool tc_encode_maps(const TcState& st, const DevLayer& D, void* host_maps);

// generic bf16 2-D tiled descriptor with the 128-byte swizzle (128 bytes written to `out`)
bool tc_encode_bf16_2d(const TcState& st, void* out, const void* base, uint64_t inner, uint64_t outer,
                       uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_outer);

// ---- tensor-core in-place pass (agzo_rmw_tc.cu)
bool rmw_tc_eligible(const agzo_layer& a);
void rmw_tc_shape(const agzo_layer& a, int panels, bool staged, DevLayer* D);   // fills the rtc_* fields except item0 / wmap
bool rmw_tc_encode_map(const TcState& st, const DevLayer& D, void* host_map);
cudaError_t rmw_tc_init();
// one block that waits on a barrier nothing completes, until the bounded wait gives up (test export)
cudaError_t launch_debug_wait(DevStatus* d_status, cudaStream_t s);
// bytes of the staged R operand images of one layer (every 128-row tile, K atoms of 16 KiB each)
size_t rmw_tc_image_bytes(const agzo_layer& a);
// shared-memory bytes of the B operand area that the layer's items need (after rmw_tc_shape)
int rmw_tc_b_bytes(const DevLayer& D);
// staged: the layers carry R images (DevLayer::rimg); fill: a fill kernel writes them first (not
// needed when an earlier pass with the same seed and layers left them in place)
cudaError_t launch_rmw_tc(const DevLayer* d_layers, const int* d_item_start, int n_layers, int total_items,
                          int max_rp, int max_r, int max_b_bytes, int max_row_tiles, bool staged, bool fill,
                          int slots_wanted, int inflight,
                          uint64_t seed, float coef, const float* d_coef, DevStatus* d_status, int sm_count, cudaStream_t s);

cudaError_t tc_fill_omega(const TcState& st, const ExtractWave& w, const DevLayer* h_dev,
                          uint64_t seed, cudaStream_t s);
// skip_fused: leave out the layers that the fused power-step kernel serves (fz_C > 0)
cudaError_t tc_xt_t(const TcState& st, const ExtractWave& w, const DevLayer* h_dev,
                    DevStatus* d_status, bool skip_fused, cudaStream_t s);
cudaError_t tc_x_q(const TcState& st, const ExtractWave& w, const DevLayer* h_dev,
                   DevStatus* d_status, bool skip_fused, cudaStream_t s);

// ---- fused power step (agzo_extract_fused.cu): Y = X^T (X Q) in one pass over X
// any_size: also cluster sizes that leave more than 30 % of the SMs idle
bool fused_eligible(const FusedCaps* caps, const agzo_layer& a, bool any_size);
int fused_cluster_size(const FusedCaps* caps, const agzo_layer& a, bool any_size);
int fused_slice_cols(const FusedCaps* caps, const agzo_layer& a, bool any_size);   // columns of X per CTA of the cluster, 0 = not eligible
int fused_parts_bound(const agzo_layer& a, int C);              // partial sums of Y a power step can leave, at most
void fused_plan_shares(const FusedCaps& caps, DevLayer* dev, int l0, int l1, int C);   // fills fz_tile0 / fz_first / fz_parts of a wave's layers of size C
int fused_resident_clusters(const FusedCaps& caps, int C);      // clusters of C CTAs the device holds at once
// the split on plain arrays and the first tile of share k (host; the kernel walks the same shares)
int fused_split(const int* tiles, int n, int clusters, int* tile0, int* first, int* parts, int* base, int* rem);
int fused_share_begin(int k, int base, int rem);
cudaError_t fused_init(int sm_count, FusedCaps* caps);   // asks the current device which cluster sizes fit
cudaError_t launch_fused_power_step(const FusedCaps& caps, const ExtractWave& w, const DevLayer* h_dev, int C,
                                    DevStatus* d_status, cudaStream_t s);

}  // namespace agzo
