// Shared device/host declarations of the AGZO library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "agzo.h"

namespace agzo {

// ---------------------------------------------------------------- device-side layer record
// Built on the host from an agzo_layer plus the scratch slices the planner assigned.
struct alignas(16) DevLayer {
  void* W;
  void* W16;
  const void* X;
  float* V;
  long long ldw, ldw16, ldx, ldv;
  int w_dtype, x_dtype, d_out, d_in, m, r;
  unsigned layer_id;
  int rmw_mode;          // RmwMode below
  // in-place passes: tiles of this layer are [tile0, tile0 + tiles_r * tiles_c)
  int tile0, tiles_r, tiles_c;
  int vec_ok;            // 16-byte vector path allowed for W (and W16)
  // extraction scratch (device pointers into the workspace)
  float* T;              // [m][r] fp32: Omega, then X Q
  float* Ypart;          // [slabs][r][d_in] fp32 partial sums of X^T T over token slabs
  float* Y;              // [r][d_in] fp32
  double* Gpart;         // [gchunks][r][r] partial Gram matrices
  double* M;             // [r][r] upper-triangular map with Q = Y M
  int slabs, slab_rows;  // token slabs of the X^T T product
  int gchunks;           // column chunks of the Gram reduction
  int x_vec_ok;          // X rows 16-byte aligned
  // tensor-core path panels (bf16 hi/lo splits), null when unused
  __nv_bfloat16* Qb;     // [NB][d_in]   rows 0..r-1 hi parts, rows NP..NP+r-1 lo parts, other rows zero
  __nv_bfloat16* Tb;     // [NB][m_pad]  T transposed, same row split
  const void* tmaps;     // four 128-byte TMA descriptors of this layer: X, Qb, Tb, unused
  long long m_pad;       // row pitch of Tb in elements (m rounded up to 8)
  int NB, NP;
  int xq_order;          // T = X Q: the CTA row of this wave position works on layer (wave start + xq_order), longest rows first
  int fz_C;              // cluster size of the fused power-step kernel for this layer, 0 = unfused kernels
  int fz_slice;          // columns of X per CTA of that cluster
  // The fused kernel's launch for the wave's layers of one cluster size treats their 128-token tiles as one
  // list, cut into equal contiguous shares, one per cluster; a share that ends inside a layer leaves a
  // partial Y for it, so a layer has as many partial sums (in Ypart) as clusters whose shares meet it.
  int fz_tile0;          // index of this layer's first tile in that list
  int fz_first;          // the first share that meets this layer
  int fz_parts;          // partial sums of this layer after a fused power step
  // Consecutive layers that read the same X (q/k/v, gate/up of a transformer block) form a group:
  // their operand panels are adjacent rows of one matrix, the leader's CTAs run both products
  // for all members with N = grp_NB columns, and X is read once per product for the group.
  int grp_role;          // 0 single layer, 1 group leader, 2 member (served by its leader)
  int grp_n;             // leader: number of layers in the group (itself included)
  int grp_NB;            // leader: operand rows of the whole group
  int grp_off;           // first operand row of this layer inside the group's panels
  // tensor-core in-place pass (bf16 W): this layer's work items are
  // [rtc_item0, rtc_item0 + rtc_panels * rtc_chunks); item = (row chunk, group of column panels)
  const void* wmap;      // 128-byte TMA descriptor of W, box = 64 columns x 128 rows; null = CUDA-core pass
  int rtc_item0, rtc_panels, rtc_chunks;   // rtc_panels counts panel GROUPS of rtc_np panels
  int rtc_np;            // column panels per item (they share the R operand of a row tile)
  int rtc_chunk_blocks;  // 128-row blocks per row chunk
  int rtc_cw;            // columns per panel: 256, 128 or 64
  int rtc_rp;            // rank rounded up to a multiple of 16
  // staged R: for r > 16 the split A operand of every 128-row tile is written once per pass to
  // scratch, in the exact shared-memory layout, and the pass copies it in instead of regenerating
  // it for every column panel.  rimg = this layer's first tile image, null = regenerate in the kernel
  unsigned char* rimg;
  int rimg_tile_bytes;   // K atoms * 16 KiB
};

enum RmwMode : int {
  RMW_BF16 = 0,          // W bf16 in place
  RMW_F32 = 1,           // W fp32 in place
  RMW_PAIR_COMPUTE = 2,  // read fp32 master, write W16 = bf16(W + c*Z), W untouched
  RMW_PAIR_UPDATE = 3    // W += c*Z (fp32), W16 = bf16(W)
};

// Device status word (first bytes of the workspace).
struct DevStatus {
  int rank_deficient;
  int timeout;
  int where;
  int pad;
};

constexpr double kRankTol = 1e-4;

// ---------------------------------------------------------------- Philox4x32-10
// Counter-based generator of Salmon et al. (SC'11).  key = step seed, counter =
// (block_lo, block_hi, layer_id, tag).
__host__ __device__ __forceinline__ uint32_t mulhi32(uint32_t a, uint32_t b) {
#ifdef __CUDA_ARCH__
  return __umulhi(a, b);
#else
  return (uint32_t)(((uint64_t)a * (uint64_t)b) >> 32);
#endif
}

__host__ __device__ __forceinline__ uint4 philox4x32_10(uint64_t block, uint32_t layer_id,
                                                        uint32_t tag, uint64_t seed) {
  uint32_t c0 = (uint32_t)block, c1 = (uint32_t)(block >> 32), c2 = layer_id, c3 = tag;
  uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
  for (int i = 0; i < 10; ++i) {
    const uint32_t hi0 = mulhi32(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = mulhi32(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return make_uint4(c0, c1, c2, c3);
}

// Box-Muller on the two word pairs of one block -> four N(0,1) floats.
__device__ __forceinline__ float4 box_muller4(uint4 w) {
  const float k24 = 5.9604644775390625e-8f;  // 2^-24
  const float u1a = (float)((w.x >> 8) + 1u) * k24;
  const float u2a = (float)(w.y >> 8) * k24;
  const float u1b = (float)((w.z >> 8) + 1u) * k24;
  const float u2b = (float)(w.w >> 8) * k24;
  const float sa = sqrtf(-2.0f * logf(u1a));
  const float sb = sqrtf(-2.0f * logf(u1b));
  float sna, csa, snb, csb;
  sincospif(2.0f * u2a, &sna, &csa);
  sincospif(2.0f * u2b, &snb, &csb);
  return make_float4(sa * csa, sa * sna, sb * csb, sb * snb);
}

__device__ __forceinline__ float4 gaussian_block(uint64_t block, uint32_t layer_id, uint32_t tag,
                                                 uint64_t seed) {
  return box_muller4(philox4x32_10(block, layer_id, tag, seed));
}

constexpr uint32_t kTagG = 0, kTagOmega = 1, kTagDense = 2, kTagBasis = 3;

// ---------------------------------------------------------------- launch entry points (host)
// in-place passes; d_coef != nullptr overrides coef
cudaError_t launch_rmw(const DevLayer* d_layers, const int* d_tile_start, int n_layers,
                       int total_tiles, int max_r, int fast_mode_mask, bool any_slow,
                       uint64_t seed, float coef, const float* d_coef, bool pair_update,
                       int sm_count, cudaStream_t s);
cudaError_t launch_dense(void* w, long long n, int dtype, uint64_t seed, uint32_t layer_id,
                         float scale, const float* d_scale, int sm_count, cudaStream_t s);
cudaError_t launch_fill_basis(const DevLayer* d_layers, int n_layers, int max_elems, uint64_t seed, cudaStream_t s);
cudaError_t launch_ghat(const double* fp, const double* fo, float eps, int mode, float* g,
                        cudaStream_t s);
cudaError_t launch_coef(const float* g, float eps, float lr, int kind, float* d_coef,
                        cudaStream_t s);
cudaError_t launch_debug_philox(uint64_t seed, uint32_t layer, uint32_t tag, uint64_t first,
                                uint64_t n, uint32_t* out, int sm_count, cudaStream_t s);
cudaError_t launch_debug_gauss(uint64_t seed, uint32_t layer, uint32_t tag, uint64_t first,
                               uint64_t n, float* out, int sm_count, cudaStream_t s);

// extraction, CUDA-core fp32 path; layers [l0, l1) form one wave
struct ExtractWave {
  const DevLayer* d_layers;   // device array (all layers)
  int l0, l1;
  int max_m, max_din, max_r, max_slabs, max_gchunks;
  long long omega_row0;       // global index of the first local token (token-sharded extraction), else 0
  int y_reduced;              // 1: Y already holds the sum over slabs (and ranks); the panel QR reads it as it is
  int after_fused;            // 1: the last product was a power step, so the layers of the fused kernel have
                              // fz_parts partial sums in Ypart (the others, and everyone after X^T T: slabs)
};
// number of partial sums of Y that the layer's last product left in Ypart
__host__ __device__ inline int y_parts(const DevLayer& L, int after_fused) {
  return (after_fused && L.fz_C) ? L.fz_parts : L.slabs;
}
cudaError_t launch_fill_omega(const ExtractWave& w, uint64_t seed, cudaStream_t s);
cudaError_t launch_xt_t(const ExtractWave& w, cudaStream_t s);      // Ypart = X^T T per slab
cudaError_t launch_x_q(const ExtractWave& w, cudaStream_t s);       // T = X Q (Q read from V)
cudaError_t launch_sum_slabs(const ExtractWave& w, cudaStream_t s);   // Y = sum over slabs of Ypart
cudaError_t launch_panel_qr(const ExtractWave& w, DevStatus* d_status, cudaStream_t s);

}  // namespace agzo
