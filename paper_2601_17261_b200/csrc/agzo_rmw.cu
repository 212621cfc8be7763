// In-place low-rank passes of Algorithm 2: W <- W + c * R A^T with R regenerated from the
// Philox counter inside the kernel (Eq. agzo-perturb).  One grouped launch covers every
// layer of the call; a tile is kTileRows x kTileCols of one layer's W.
//
// HBM-bound for r <= 16: each weight is read once and written once (16-byte accesses, eight
// rows in flight per thread); R for the tile's rows is generated once into shared memory
// and the tile's slice of A^T lives in registers, so neither R nor Delta ever reaches DRAM.
#include "agzo_common.cuh"

namespace agzo {

constexpr int kRmwThreads = 256;
constexpr int kTileCols = 512;   // 64 threads x 8 consecutive columns
constexpr int kTileRows = 256;
constexpr int kRowLanes = 4;     // thread groups that take different rows
constexpr int kRowsInFlight = 8; // rows per thread per sub-block
constexpr int kSubRows = kRowLanes * kRowsInFlight;

__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);   // RNE, a in the low half
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ float round_to_bf16(float a) {
  return __bfloat162float(__float2bfloat16_rn(a));
}

// ------------------------------------------------------------------ tile I/O (16-byte accesses)
// Eight consecutive weights of one row, kept in their storage format until they are used
// (a bf16 row segment is four registers, not eight).
template <int MODE> struct Raw8 { float4 a, b; };
template <> struct Raw8<RMW_BF16> { uint4 q; };

template <int MODE>
__device__ __forceinline__ void load8(const DevLayer& L, long long row, int col, Raw8<MODE>& w) {
  if constexpr (MODE == RMW_BF16) {
    const __nv_bfloat16* p = reinterpret_cast<const __nv_bfloat16*>(L.W) + row * L.ldw + col;
    w.q = __ldcs(reinterpret_cast<const uint4*>(p));
  } else {
    const float* p = reinterpret_cast<const float*>(L.W) + row * L.ldw + col;
    w.a = __ldcs(reinterpret_cast<const float4*>(p));
    w.b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
  }
}

template <int MODE>
__device__ __forceinline__ void unpack8(const Raw8<MODE>& r, float (&w)[8]) {
  if constexpr (MODE == RMW_BF16) {
    w[0] = bf16lo(r.q.x); w[1] = bf16hi(r.q.x); w[2] = bf16lo(r.q.y); w[3] = bf16hi(r.q.y);
    w[4] = bf16lo(r.q.z); w[5] = bf16hi(r.q.z); w[6] = bf16lo(r.q.w); w[7] = bf16hi(r.q.w);
  } else {
    w[0] = r.a.x; w[1] = r.a.y; w[2] = r.a.z; w[3] = r.a.w;
    w[4] = r.b.x; w[5] = r.b.y; w[6] = r.b.z; w[7] = r.b.w;
  }
}

template <int MODE>
__device__ __forceinline__ void store8(const DevLayer& L, long long row, int col, const float (&w)[8]) {
  if (MODE == RMW_BF16 || MODE == RMW_PAIR_COMPUTE || MODE == RMW_PAIR_UPDATE) {
    __nv_bfloat16* p = (MODE == RMW_BF16)
                           ? reinterpret_cast<__nv_bfloat16*>(L.W) + row * L.ldw + col
                           : reinterpret_cast<__nv_bfloat16*>(L.W16) + row * L.ldw16 + col;
    uint4 q;
    q.x = pack_bf16(w[0], w[1]); q.y = pack_bf16(w[2], w[3]);
    q.z = pack_bf16(w[4], w[5]); q.w = pack_bf16(w[6], w[7]);
    __stcs(reinterpret_cast<uint4*>(p), q);
  }
  if (MODE == RMW_F32 || MODE == RMW_PAIR_UPDATE) {
    float* p = reinterpret_cast<float*>(L.W) + row * L.ldw + col;
    __stcs(reinterpret_cast<float4*>(p), make_float4(w[0], w[1], w[2], w[3]));
    __stcs(reinterpret_cast<float4*>(p) + 1, make_float4(w[4], w[5], w[6], w[7]));
  }
}

// ------------------------------------------------------------------ R for the rows of a tile
// sG[row_local * RS + k] = R[row0 + row_local][k]; columns r..RS-1 are zero.
__device__ __forceinline__ void generate_G(float* sG, int RS, int r, long long row0, int nrows,
                                           uint32_t layer_id, uint64_t seed) {
  const long long e_first = row0 * r;
  const long long e_last = e_first + (long long)nrows * r;
  const long long b_first = e_first >> 2;
  const int nb = (int)(((e_last - 1) >> 2) - b_first + 1);
  for (int i = threadIdx.x; i < nb; i += kRmwThreads) {
    const long long b = b_first + i;
    const float4 g = gaussian_block((uint64_t)b, layer_id, kTagG, seed);
    const float gv[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
    for (int lane = 0; lane < 4; ++lane) {
      const long long e = 4 * b + lane;
      if (e >= e_first && e < e_last) {
        const int local = (int)(e - e_first);
        const int rl = local / r;
        sG[rl * RS + (local - rl * r)] = gv[lane];
      }
    }
  }
  if (RS > r) {
    const int pad = RS - r;
    for (int i = threadIdx.x; i < nrows * pad; i += kRmwThreads) {
      const int rl = i / pad;
      sG[rl * RS + r + (i - rl * pad)] = 0.f;
    }
  }
}

// ------------------------------------------------------------------ r <= 16: A^T slice in registers
template <int RC, int MODE>
__device__ __forceinline__ void tile_body_reg(const DevLayer& L, const float* sG, int row0,
                                              int nrows, int col0, float coef) {
  const int cx = threadIdx.x & 63;
  const int ry = threadIdx.x >> 6;
  const int col = col0 + cx * 8;
  if (col >= L.d_in) return;   // d_in is a multiple of 8 on this path

  float v[RC][8];
#pragma unroll
  for (int k = 0; k < RC; ++k) {
    if (k < L.r) {
      const float* p = L.V + (long long)k * L.ldv + col;
      const float4 a = __ldg(reinterpret_cast<const float4*>(p));
      const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
      v[k][0] = a.x; v[k][1] = a.y; v[k][2] = a.z; v[k][3] = a.w;
      v[k][4] = b.x; v[k][5] = b.y; v[k][6] = b.z; v[k][7] = b.w;
    } else {
#pragma unroll
      for (int c = 0; c < 8; ++c) v[k][c] = 0.f;
    }
  }

  for (int sb = 0; sb < nrows; sb += kSubRows) {
    Raw8<MODE> raw[kRowsInFlight];
#pragma unroll
    for (int j = 0; j < kRowsInFlight; ++j) {
      const int rl = sb + ry + j * kRowLanes;
      if (rl < nrows) load8<MODE>(L, (long long)(row0 + rl), col, raw[j]);
    }
#pragma unroll
    for (int j = 0; j < kRowsInFlight; ++j) {
      const int rl = sb + ry + j * kRowLanes;
      if (rl < nrows) {
        float w[8];
        unpack8<MODE>(raw[j], w);
        const float* g = sG + rl * RC;
        float gk[RC];
        if (RC >= 4) {
#pragma unroll
          for (int k4 = 0; k4 < RC / 4; ++k4) {
            const float4 g4 = *reinterpret_cast<const float4*>(g + 4 * k4);
            gk[(4 * k4 + 0) % RC] = g4.x; gk[(4 * k4 + 1) % RC] = g4.y;
            gk[(4 * k4 + 2) % RC] = g4.z; gk[(4 * k4 + 3) % RC] = g4.w;
          }
        } else {
#pragma unroll
          for (int k = 0; k < RC; ++k) gk[k] = g[k];
        }
        float o[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          float z = 0.f;
#pragma unroll
          for (int k = 0; k < RC; ++k) z = fmaf(gk[k], v[k][c], z);   // k ascending, fixed order
          o[c] = fmaf(coef, z, w[c]);
        }
        store8<MODE>(L, (long long)(row0 + rl), col, o);
      }
    }
  }
}

// ------------------------------------------------------------------ 16 < r <= 64: A^T slice in shared memory
template <int MODE>
__device__ __forceinline__ void tile_body_smem(const DevLayer& L, const float* sG, const float* sV,
                                               int RS, int row0, int nrows, int col0, float coef) {
  const int cx = threadIdx.x & 63;
  const int ry = threadIdx.x >> 6;
  const int col = col0 + cx * 8;
  if (col >= L.d_in) return;
  const float* sv = sV + cx * 8;

  for (int sb = 0; sb < nrows; sb += kSubRows) {
    Raw8<MODE> raw[kRowsInFlight];
    float z[kRowsInFlight][8];
#pragma unroll
    for (int j = 0; j < kRowsInFlight; ++j) {
      const int rl = sb + ry + j * kRowLanes;
      if (rl < nrows) load8<MODE>(L, (long long)(row0 + rl), col, raw[j]);
#pragma unroll
      for (int c = 0; c < 8; ++c) z[j][c] = 0.f;
    }
    for (int k4 = 0; k4 < RS; k4 += 4) {
      float4 g4[kRowsInFlight];
#pragma unroll
      for (int j = 0; j < kRowsInFlight; ++j) {
        const int rl = min(sb + ry + j * kRowLanes, nrows - 1);
        g4[j] = *reinterpret_cast<const float4*>(sG + rl * RS + k4);
      }
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const float4 va = *reinterpret_cast<const float4*>(sv + (k4 + kk) * kTileCols);
        const float4 vb = *reinterpret_cast<const float4*>(sv + (k4 + kk) * kTileCols + 4);
        const float vv[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
#pragma unroll
        for (int j = 0; j < kRowsInFlight; ++j) {
          const float gk = kk == 0 ? g4[j].x : kk == 1 ? g4[j].y : kk == 2 ? g4[j].z : g4[j].w;
#pragma unroll
          for (int c = 0; c < 8; ++c) z[j][c] = fmaf(gk, vv[c], z[j][c]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < kRowsInFlight; ++j) {
      const int rl = sb + ry + j * kRowLanes;
      if (rl < nrows) {
        float w[8], o[8];
        unpack8<MODE>(raw[j], w);
#pragma unroll
        for (int c = 0; c < 8; ++c) o[c] = fmaf(coef, z[j][c], w[c]);
        store8<MODE>(L, (long long)(row0 + rl), col, o);
      }
    }
  }
}

__device__ __forceinline__ int find_layer(const int* tile_start, int n_layers, int tile) {
  int lo = 0, hi = n_layers - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (__ldg(tile_start + mid) <= tile) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__device__ __forceinline__ int effective_mode(const DevLayer& L, int pair_update) {
  return (L.rmw_mode == RMW_PAIR_COMPUTE && pair_update) ? RMW_PAIR_UPDATE : L.rmw_mode;
}

// Persistent CTAs stride over the tiles of all layers.  A kernel instance serves the layers
// whose storage mode is MODE and whose pointers allow 16-byte accesses; other tiles are
// skipped (another instance, or the generic kernel, takes them).
template <int RC, int MODE>
__global__ void __launch_bounds__(kRmwThreads, (RC <= 8 ? 2 : 1))
rmw_reg_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ tile_start,
               int n_layers, int total_tiles, uint64_t seed, float coef_imm,
               const float* __restrict__ d_coef, int pair_update) {
  extern __shared__ __align__(16) float smem[];
  __shared__ DevLayer sL;
  float* sG = smem;
  const float coef = d_coef ? __ldg(d_coef) : coef_imm;
  for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
    const int li = find_layer(tile_start, n_layers, tile);
    __syncthreads();   // previous tile is done with sG and sL
    if (threadIdx.x == 0) sL = layers[li];
    __syncthreads();
    const DevLayer& L = sL;
    if (!L.vec_ok || effective_mode(L, pair_update) != MODE) continue;
    const int t = tile - L.tile0;
    const int tr = t / L.tiles_c, tc = t - tr * L.tiles_c;
    const int row0 = tr * kTileRows, col0 = tc * kTileCols;
    const int nrows = min(kTileRows, L.d_out - row0);
    generate_G(sG, RC, L.r, row0, nrows, L.layer_id, seed);
    __syncthreads();
    tile_body_reg<RC, MODE>(L, sG, row0, nrows, col0, coef);
  }
}

template <int MODE>
__global__ void __launch_bounds__(kRmwThreads, 1)
rmw_smem_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ tile_start,
                int n_layers, int total_tiles, int max_rs, uint64_t seed, float coef_imm,
                const float* __restrict__ d_coef, int pair_update) {
  extern __shared__ __align__(16) float smem[];
  __shared__ DevLayer sL;
  float* sG = smem;                              // [kTileRows][RS]
  float* sV = smem + kTileRows * max_rs;         // [RS][kTileCols]
  const float coef = d_coef ? __ldg(d_coef) : coef_imm;
  for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
    const int li = find_layer(tile_start, n_layers, tile);
    __syncthreads();
    if (threadIdx.x == 0) sL = layers[li];
    __syncthreads();
    const DevLayer& L = sL;
    if (!L.vec_ok || effective_mode(L, pair_update) != MODE) continue;
    const int RS = (L.r + 3) & ~3;
    const int t = tile - L.tile0;
    const int tr = t / L.tiles_c, tc = t - tr * L.tiles_c;
    const int row0 = tr * kTileRows, col0 = tc * kTileCols;
    const int nrows = min(kTileRows, L.d_out - row0);
    generate_G(sG, RS, L.r, row0, nrows, L.layer_id, seed);
    for (int i = threadIdx.x; i < RS * kTileCols; i += kRmwThreads) {
      const int k = i / kTileCols, c = i - k * kTileCols;
      sV[i] = (k < L.r && col0 + c < L.d_in) ? __ldg(L.V + (long long)k * L.ldv + col0 + c) : 0.f;
    }
    __syncthreads();
    tile_body_smem<MODE>(L, sG, sV, RS, row0, nrows, col0, coef);
  }
}

// Any pitch, alignment, storage mode and rank; one block per tile, scalar accesses.  Serves
// the layers the vector kernels cannot take.
__global__ void __launch_bounds__(kRmwThreads)
rmw_generic_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ tile_start,
                   int n_layers, int total_tiles, uint64_t seed, float coef_imm,
                   const float* __restrict__ d_coef, int pair_update) {
  __shared__ float sG[32 * AGZO_MAX_RANK];
  __shared__ DevLayer sL;
  const float coef = d_coef ? __ldg(d_coef) : coef_imm;
  for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
    const int li = find_layer(tile_start, n_layers, tile);
    __syncthreads();
    if (threadIdx.x == 0) sL = layers[li];
    __syncthreads();
    const DevLayer& L = sL;
    if (L.vec_ok) continue;
    const int mode = effective_mode(L, pair_update);
    const int r = L.r;
    const int t = tile - L.tile0;
    const int tr = t / L.tiles_c, tc = t - tr * L.tiles_c;
    const int row0 = tr * kTileRows, col0 = tc * kTileCols;
    const int nrows = min(kTileRows, L.d_out - row0);
    for (int sb = 0; sb < nrows; sb += 32) {
      const int nr = min(32, nrows - sb);
      __syncthreads();
      generate_G(sG, r, r, row0 + sb, nr, L.layer_id, seed);
      __syncthreads();
      for (int c = threadIdx.x; c < kTileCols; c += kRmwThreads) {
        const int col = col0 + c;
        if (col >= L.d_in) break;
        for (int rl = 0; rl < nr; ++rl) {
          const long long row = row0 + sb + rl;
          float z = 0.f;
          for (int k = 0; k < r; ++k) z = fmaf(sG[rl * r + k], __ldg(L.V + (long long)k * L.ldv + col), z);
          float w;
          if (mode == RMW_BF16) w = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(L.W)[row * L.ldw + col]);
          else w = reinterpret_cast<const float*>(L.W)[row * L.ldw + col];
          const float o = fmaf(coef, z, w);
          if (mode == RMW_BF16) reinterpret_cast<__nv_bfloat16*>(L.W)[row * L.ldw + col] = __float2bfloat16_rn(o);
          if (mode == RMW_F32 || mode == RMW_PAIR_UPDATE) reinterpret_cast<float*>(L.W)[row * L.ldw + col] = o;
          if (mode == RMW_PAIR_COMPUTE || mode == RMW_PAIR_UPDATE)
            reinterpret_cast<__nv_bfloat16*>(L.W16)[row * L.ldw16 + col] = __float2bfloat16_rn(o);
        }
      }
    }
  }
}

struct RmwArgs {
  const DevLayer* d_layers; const int* d_tile_start; int n_layers, total_tiles;
  uint64_t seed; float coef; const float* d_coef; int pair_update; int sm_count;
};

template <int RC, int MODE>
static cudaError_t launch_reg(const RmwArgs& a, cudaStream_t s) {
  const int per_sm = RC <= 8 ? 2 : 1;
  const int grid = a.total_tiles < a.sm_count * per_sm ? a.total_tiles : a.sm_count * per_sm;
  const size_t smem = (size_t)kTileRows * RC * sizeof(float);
  rmw_reg_kernel<RC, MODE><<<grid, kRmwThreads, smem, s>>>(a.d_layers, a.d_tile_start, a.n_layers,
                                                           a.total_tiles, a.seed, a.coef, a.d_coef,
                                                           a.pair_update);
  return cudaGetLastError();
}

template <int MODE>
static cudaError_t launch_mode(const RmwArgs& a, int max_r, cudaStream_t s) {
  if (max_r <= 1) return launch_reg<1, MODE>(a, s);
  if (max_r <= 2) return launch_reg<2, MODE>(a, s);
  if (max_r <= 4) return launch_reg<4, MODE>(a, s);
  if (max_r <= 8) return launch_reg<8, MODE>(a, s);
  if (max_r <= 16) return launch_reg<16, MODE>(a, s);
  const int max_rs = (max_r + 3) & ~3;
  const size_t smem = ((size_t)kTileRows * max_rs + (size_t)max_rs * kTileCols) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(rmw_smem_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)(((size_t)kTileRows * 64 + (size_t)64 * kTileCols) * sizeof(float)));
  if (e != cudaSuccess) return e;
  const int grid = a.total_tiles < a.sm_count ? a.total_tiles : a.sm_count;
  rmw_smem_kernel<MODE><<<grid, kRmwThreads, smem, s>>>(a.d_layers, a.d_tile_start, a.n_layers,
                                                        a.total_tiles, max_rs, a.seed, a.coef,
                                                        a.d_coef, a.pair_update);
  return cudaGetLastError();
}

cudaError_t launch_rmw(const DevLayer* d_layers, const int* d_tile_start, int n_layers,
                       int total_tiles, int max_r, int fast_mode_mask, bool any_slow,
                       uint64_t seed, float coef, const float* d_coef, bool pair_update,
                       int sm_count, cudaStream_t s) {
  if (total_tiles <= 0) return cudaSuccess;
  RmwArgs a{d_layers, d_tile_start, n_layers, total_tiles, seed, coef, d_coef, pair_update ? 1 : 0, sm_count};
  cudaError_t e = cudaSuccess;
  if (pair_update && (fast_mode_mask & (1 << RMW_PAIR_COMPUTE)))
    fast_mode_mask = (fast_mode_mask & ~(1 << RMW_PAIR_COMPUTE)) | (1 << RMW_PAIR_UPDATE);
  if (e == cudaSuccess && (fast_mode_mask & (1 << RMW_BF16))) e = launch_mode<RMW_BF16>(a, max_r, s);
  if (e == cudaSuccess && (fast_mode_mask & (1 << RMW_F32))) e = launch_mode<RMW_F32>(a, max_r, s);
  if (e == cudaSuccess && (fast_mode_mask & (1 << RMW_PAIR_COMPUTE))) e = launch_mode<RMW_PAIR_COMPUTE>(a, max_r, s);
  if (e == cudaSuccess && (fast_mode_mask & (1 << RMW_PAIR_UPDATE))) e = launch_mode<RMW_PAIR_UPDATE>(a, max_r, s);
  if (e == cudaSuccess && any_slow) {
    const int grid = total_tiles < sm_count * 4 ? total_tiles : sm_count * 4;
    rmw_generic_kernel<<<grid, kRmwThreads, 0, s>>>(d_layers, d_tile_start, n_layers, total_tiles,
                                                    seed, coef, d_coef, pair_update ? 1 : 0);
    e = cudaGetLastError();
  }
  return e;
}

// ------------------------------------------------------------------ dense direction (second case of Eq. agzo-perturb)
// w <- w + c u, u ~ N(0, I) from (seed, layer_id, tag 2), element e = word e & 3 of block e >> 2.
// Scalar form: any pointer, blocks [b_first, b_end).
template <typename T>
__global__ void dense_kernel(T* w, long long n, long long b_first, uint64_t seed, uint32_t layer_id, float scale,
                             const float* d_scale) {
  const float c = d_scale ? scale * __ldg(d_scale) : scale;
  const long long nb = (n + 3) >> 2;
  for (long long b = b_first + blockIdx.x * (long long)blockDim.x + threadIdx.x; b < nb;
       b += (long long)gridDim.x * blockDim.x) {
    const float4 g = gaussian_block((uint64_t)b, layer_id, kTagDense, seed);
    const float gv[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
    for (int lane = 0; lane < 4; ++lane) {
      const long long e = 4 * b + lane;
      if (e < n) w[e] = (T)fmaf(c, gv[lane], (float)w[e]);
    }
  }
}

// Vector form for 16-byte aligned vectors: a thread takes eight consecutive elements (two Philox
// blocks) per step, one 16-byte load and store for bf16, two for fp32.  The pass is bound by the
// arithmetic of one Philox + Box-Muller normal per weight, not by HBM; the wide accesses keep
// the memory side out of the way.
template <typename T>
__global__ void __launch_bounds__(256) dense_vec_kernel(T* w, long long n8, uint64_t seed, uint32_t layer_id, float scale,
                                                        const float* d_scale) {
  const float c = d_scale ? scale * __ldg(d_scale) : scale;
  for (long long g = blockIdx.x * (long long)blockDim.x + threadIdx.x; g < n8; g += (long long)gridDim.x * blockDim.x) {
    const float4 ga = gaussian_block((uint64_t)(2 * g), layer_id, kTagDense, seed);
    const float4 gb = gaussian_block((uint64_t)(2 * g + 1), layer_id, kTagDense, seed);
    const float u[8] = {ga.x, ga.y, ga.z, ga.w, gb.x, gb.y, gb.z, gb.w};
    if constexpr (sizeof(T) == 2) {
      uint4* p = reinterpret_cast<uint4*>(w) + g;
      const uint4 v = *p;
      const uint32_t in[4] = {v.x, v.y, v.z, v.w};
      uint32_t out[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float w0 = __uint_as_float(in[k] << 16), w1 = __uint_as_float(in[k] & 0xFFFF0000u);
        __nv_bfloat162 r = __floats2bfloat162_rn(fmaf(c, u[2 * k], w0), fmaf(c, u[2 * k + 1], w1));
        out[k] = *reinterpret_cast<uint32_t*>(&r);
      }
      *p = make_uint4(out[0], out[1], out[2], out[3]);
    } else {
      float4* p = reinterpret_cast<float4*>(w) + 2 * g;
      float4 a = p[0], b = p[1];
      a.x = fmaf(c, u[0], a.x); a.y = fmaf(c, u[1], a.y); a.z = fmaf(c, u[2], a.z); a.w = fmaf(c, u[3], a.w);
      b.x = fmaf(c, u[4], b.x); b.y = fmaf(c, u[5], b.y); b.z = fmaf(c, u[6], b.z); b.w = fmaf(c, u[7], b.w);
      p[0] = a; p[1] = b;
    }
  }
}

template <typename T>
cudaError_t launch_dense_t(T* w, long long n, uint64_t seed, uint32_t layer_id, float scale, const float* d_scale,
                           int sm_count, cudaStream_t s) {
  const long long cap = (long long)sm_count * 8;      // eight resident blocks of 256 threads per SM
  long long n8 = 0;
  if ((reinterpret_cast<uintptr_t>(w) & 15u) == 0) n8 = n >> 3;
  if (n8 > 0) {
    const int grid = (int)((n8 + 255) / 256 < cap ? (n8 + 255) / 256 : cap);
    dense_vec_kernel<T><<<grid, 256, 0, s>>>(w, n8, seed, layer_id, scale, d_scale);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (8 * n8 < n) {                                    // the rest: blocks from 2 n8 on
    const long long nb = ((n + 3) >> 2) - 2 * n8;
    const int grid = (int)((nb + 255) / 256 < cap ? (nb + 255) / 256 : cap);
    dense_kernel<T><<<grid, 256, 0, s>>>(w, n, 2 * n8, seed, layer_id, scale, d_scale);
    return cudaGetLastError();
  }
  return cudaSuccess;
}

cudaError_t launch_dense(void* w, long long n, int dtype, uint64_t seed, uint32_t layer_id,
                         float scale, const float* d_scale, int sm_count, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  if (dtype == AGZO_BF16)
    return launch_dense_t<__nv_bfloat16>((__nv_bfloat16*)w, n, seed, layer_id, scale, d_scale, sm_count, s);
  return launch_dense_t<float>((float*)w, n, seed, layer_id, scale, d_scale, sm_count, s);
}

// ------------------------------------------------------------------ Gaussian right factor (LOZO comparison)
__global__ void fill_basis_kernel(const DevLayer* __restrict__ layers, uint64_t seed) {
  const DevLayer& L = layers[blockIdx.y];
  const long long n = (long long)L.r * L.d_in;
  const long long nb = (n + 3) >> 2;
  for (long long b = blockIdx.x * (long long)blockDim.x + threadIdx.x; b < nb;
       b += (long long)gridDim.x * blockDim.x) {
    const float4 g = gaussian_block((uint64_t)b, L.layer_id, kTagBasis, seed);
    const float gv[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
    for (int lane = 0; lane < 4; ++lane) {
      const long long e = 4 * b + lane;
      if (e < n) {
        const long long k = e / L.d_in;
        L.V[k * L.ldv + (e - k * L.d_in)] = gv[lane];
      }
    }
  }
}

cudaError_t launch_fill_basis(const DevLayer* d_layers, int n_layers, int max_elems, uint64_t seed, cudaStream_t s) {
  if (n_layers <= 0) return cudaSuccess;
  int gx = (max_elems / 4 + 255) / 256;
  if (gx < 1) gx = 1;
  if (gx > 64) gx = 64;
  fill_basis_kernel<<<dim3((unsigned)gx, (unsigned)n_layers), 256, 0, s>>>(d_layers, seed);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ scalars (Algorithm 2, step 3)
__global__ void ghat_kernel(const double* fp, const double* fo, float eps, int mode, float* g) {
  const double d = *fp - *fo;
  *g = (float)(mode == 0 ? d / (2.0 * (double)eps) : d / (double)eps);
}
cudaError_t launch_ghat(const double* fp, const double* fo, float eps, int mode, float* g, cudaStream_t s) {
  ghat_kernel<<<1, 1, 0, s>>>(fp, fo, eps, mode, g);
  return cudaGetLastError();
}

// kind 0: eps - lr*g   kind 1: -(eps + lr*g)   kind 2: -lr*g
__global__ void coef_kernel(const float* g, float eps, float lr, int kind, float* out) {
  const double lg = (double)lr * (double)*g;
  *out = (float)(kind == 0 ? (double)eps - lg : kind == 1 ? -((double)eps + lg) : -lg);
}
cudaError_t launch_coef(const float* g, float eps, float lr, int kind, float* d_coef, cudaStream_t s) {
  coef_kernel<<<1, 1, 0, s>>>(g, eps, lr, kind, d_coef);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ test exports
__global__ void debug_philox_kernel(uint64_t seed, uint32_t layer, uint32_t tag, uint64_t first,
                                    uint64_t n, uint32_t* out) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n;
       i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t e = first + i;
    const uint4 w = philox4x32_10(e >> 2, layer, tag, seed);
    const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
    out[i] = wv[e & 3];
  }
}
__global__ void debug_gauss_kernel(uint64_t seed, uint32_t layer, uint32_t tag, uint64_t first,
                                   uint64_t n, float* out) {
  for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < n;
       i += (uint64_t)gridDim.x * blockDim.x) {
    const uint64_t e = first + i;
    const float4 g = gaussian_block(e >> 2, layer, tag, seed);
    const float gv[4] = {g.x, g.y, g.z, g.w};
    out[i] = gv[e & 3];
  }
}
cudaError_t launch_debug_philox(uint64_t seed, uint32_t layer, uint32_t tag, uint64_t first,
                                uint64_t n, uint32_t* out, int sm_count, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  const uint64_t cap = (uint64_t)sm_count * 8;
  const int grid = (int)((n + 255) / 256 < cap ? (n + 255) / 256 : cap);
  debug_philox_kernel<<<grid, 256, 0, s>>>(seed, layer, tag, first, n, out);
  return cudaGetLastError();
}
cudaError_t launch_debug_gauss(uint64_t seed, uint32_t layer, uint32_t tag, uint64_t first,
                               uint64_t n, float* out, int sm_count, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  const uint64_t cap = (uint64_t)sm_count * 8;
  const int grid = (int)((n + 255) / 256 < cap ? (n + 255) / 256 : cap);
  debug_gauss_kernel<<<grid, 256, 0, s>>>(seed, layer, tag, first, n, out);
  return cudaGetLastError();
}

}  // namespace agzo
