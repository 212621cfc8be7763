// Allocation-free variant of Algorithm 1 for one layer: the scratch that the extraction
// kernels need lives in a fixed array inside the loaded library image instead of a workspace
// the caller would have to allocate.
//
// Who needs this: code that may not call cudaMalloc at the point where it wants a subspace --
// a forward hook running while another framework owns the allocator (or while a memory pool is
// frozen), a callback invoked from a context where allocation would synchronise the device, a
// process whose memory budget is fixed up front.  Such a caller still owns X and V; it simply
// has nowhere to get a workspace from.
#include <mutex>

#include "agzo_common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 4u << 20;   // 4 MiB, held by every GPU that loads the library
constexpr int kMaxDevices = 64;

// The name below is a host-side handle for the symbol, not a device address: kernels must be
// given the address that cudaGetSymbolAddress returns for the current device.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};

cudaError_t scratch_of_current_device(int* dev_out, unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);   // once per device, with that device current
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = p;
  }
  *dev_out = dev;
  *out = static_cast<unsigned char*>(g_scratch_addr[dev]);
  return cudaSuccess;
}

inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }

// The array is shared by all calls and keeps the previous call's contents: the layer record is
// rewritten and the status word cleared here; every other slice is fully overwritten by the
// kernels before it is read.
__global__ void static_begin_kernel(agzo::DevLayer rec, agzo::DevLayer* dst, agzo::DevStatus* st) {
  *dst = rec;
  st->rank_deficient = 0;
  st->timeout = 0;
  st->where = 0;
  st->pad = 0;
}

__global__ void static_end_kernel(const agzo::DevStatus* st, int32_t* flag) {
  *flag = st->rank_deficient;
}

}  // namespace

extern "C" agzo_status agzo_extract_subspace_static(const void* X, int64_t ldx, int32_t x_dtype,
                                                    int32_t m, int32_t d_in, int32_t r, int32_t K,
                                                    uint64_t seed, uint32_t layer_id, float* V,
                                                    int64_t ldv, int32_t* d_rank_deficient,
                                                    void* stream) {
  using namespace agzo;
  if (!X || !V || m < 1 || d_in < 1 || r < 1 || r > AGZO_MAX_RANK || r > d_in || r > m ||
      ldx < d_in || ldv < d_in || K < 0 || K > 16)
    return AGZO_ERR_INVALID_ARG;
  if (x_dtype != AGZO_BF16 && x_dtype != AGZO_F32) return AGZO_ERR_UNSUPPORTED;
  const size_t es = x_dtype == AGZO_BF16 ? 2 : 4;
  if ((reinterpret_cast<uintptr_t>(X) & (es - 1)) || (reinterpret_cast<uintptr_t>(V) & 3u))
    return AGZO_ERR_INVALID_ARG;

  // token slabs of the X^T T product (same rule as the workspace planner)
  int slab_rows = (m + 31) / 32;
  slab_rows = (slab_rows + 31) / 32 * 32;
  if (slab_rows < 256) slab_rows = 256;
  const int slabs = (m + slab_rows - 1) / slab_rows;
  const size_t gch = ((size_t)d_in + 127) / 128;
  const size_t R = (size_t)r, D = (size_t)d_in, M = (size_t)m;
  const size_t need = 512 + up256(M * R * 4) + up256((size_t)slabs * R * D * 4) + up256(R * D * 4) +
                      up256(gch * R * R * 8) + up256(R * R * 8);
  if (need > kStaticScratchBytes) return AGZO_ERR_WORKSPACE;   // problem too large for the fixed array

  int dev = -1;
  unsigned char* base = nullptr;
  if (scratch_of_current_device(&dev, &base) != cudaSuccess) return AGZO_ERR_CUDA;

  unsigned char* p = base;
  DevLayer* d_rec = reinterpret_cast<DevLayer*>(p);
  DevStatus* d_status = reinterpret_cast<DevStatus*>(p + 384);
  p += 512;
  DevLayer rec{};
  rec.X = X; rec.V = V; rec.ldx = ldx; rec.ldv = ldv;
  rec.x_dtype = x_dtype; rec.d_in = d_in; rec.m = m; rec.r = r; rec.layer_id = layer_id;
  rec.slabs = slabs; rec.slab_rows = slab_rows; rec.gchunks = (int)gch;
  rec.T = reinterpret_cast<float*>(p);      p += up256(M * R * 4);
  rec.Ypart = reinterpret_cast<float*>(p);  p += up256((size_t)slabs * R * D * 4);
  rec.Y = reinterpret_cast<float*>(p);      p += up256(R * D * 4);
  rec.Gpart = reinterpret_cast<double*>(p); p += up256(gch * R * R * 8);
  rec.M = reinterpret_cast<double*>(p);
  static_assert(sizeof(DevLayer) <= 384, "layer record must fit its slot");

  cudaStream_t s = static_cast<cudaStream_t>(stream);
  static_begin_kernel<<<1, 1, 0, s>>>(rec, d_rec, d_status);
  if (cudaGetLastError() != cudaSuccess) return AGZO_ERR_CUDA;

  ExtractWave w{};
  w.d_layers = d_rec;
  w.l0 = 0; w.l1 = 1;
  w.max_m = m; w.max_din = d_in; w.max_r = r; w.max_slabs = slabs; w.max_gchunks = (int)gch;
  if (launch_fill_omega(w, seed, s) != cudaSuccess) return AGZO_ERR_CUDA;     // Omega
  if (launch_xt_t(w, s) != cudaSuccess) return AGZO_ERR_CUDA;                 // Y <- H Omega
  for (int k = 0; k < K; ++k) {
    if (launch_panel_qr(w, d_status, s) != cudaSuccess) return AGZO_ERR_CUDA;  // Q <- qr(Y)
    if (launch_x_q(w, s) != cudaSuccess) return AGZO_ERR_CUDA;
    if (launch_xt_t(w, s) != cudaSuccess) return AGZO_ERR_CUDA;               // Y <- H (H^T Q)
  }
  if (launch_panel_qr(w, d_status, s) != cudaSuccess) return AGZO_ERR_CUDA;    // A <- qr(Y)
  if (d_rank_deficient) {
    static_end_kernel<<<1, 1, 0, s>>>(d_status, d_rank_deficient);
    if (cudaGetLastError() != cudaSuccess) return AGZO_ERR_CUDA;
  }
  return AGZO_OK;
}
