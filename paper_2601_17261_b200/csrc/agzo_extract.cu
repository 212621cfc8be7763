// Algorithm 1 (SubspaceExtract) on CUDA cores in fp32, plus the panel orthonormalisation
// that both extraction paths share.  This path takes any dtype, pitch and size; the
// tensor-core path (agzo_extract_tc.cu) replaces the two products with X when the layer's
// shape allows it.
//
// Products:  Ypart[s] = X_s^T T_s  per token slab s (summed in slab order later, so the result
//            does not depend on scheduling), and T = X Q.
// qr(Y):     Gram matrix S = Y^T Y accumulated in double, Cholesky S = R^T R with R_kk > 0,
//            Q = Y R^-1.  With the Gram matrix and the factor in double this is as accurate
//            in fp32 as a Householder QR for cond(Y) well below 1e7, and it is the unique
//            positive-diagonal factorisation that the method's definition fixes.
#include "agzo_common.cuh"

namespace agzo {

// ------------------------------------------------------------------ Omega -> T
// Local token t is row row0 + t of the test matrix of the whole batch: element e of the stream is
// (row0 + t) * r + k, so the Philox blocks that cover the local rows are walked, whatever row0 is.
__global__ void fill_omega_kernel(const DevLayer* __restrict__ layers, int l0, uint64_t seed, long long row0) {
  const DevLayer& L = layers[l0 + blockIdx.y];
  const long long n = (long long)L.m * L.r;
  const long long e0 = row0 * L.r;
  const long long b_end = (e0 + n + 3) >> 2;
  for (long long b = (e0 >> 2) + blockIdx.x * (long long)blockDim.x + threadIdx.x; b < b_end;
       b += (long long)gridDim.x * blockDim.x) {
    const float4 g = gaussian_block((uint64_t)b, L.layer_id, kTagOmega, seed);
    const float gv[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
    for (int lane = 0; lane < 4; ++lane) {
      const long long e = 4 * b + lane - e0;
      if (e >= 0 && e < n) L.T[e] = gv[lane];
    }
  }
}

cudaError_t launch_fill_omega(const ExtractWave& w, uint64_t seed, cudaStream_t s) {
  const long long nb = (((long long)w.max_m * w.max_r + 3) >> 2) + 1;
  int gx = (int)((nb + 255) / 256);
  if (gx > 512) gx = 512;
  if (gx < 1) gx = 1;
  fill_omega_kernel<<<dim3(gx, w.l1 - w.l0), 256, 0, s>>>(w.d_layers, w.l0, seed, w.omega_row0);
  return cudaGetLastError();
}

__device__ __forceinline__ float load_x(const DevLayer& L, long long t, int d) {
  return L.x_dtype == AGZO_BF16
             ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(L.X)[t * L.ldx + d])
             : reinterpret_cast<const float*>(L.X)[t * L.ldx + d];
}

// ------------------------------------------------------------------ Ypart[s][k][d] = sum_{t in slab s} X[t][d] T[t][k]
// block: 256 threads = 256 columns d; grid (d chunks, slabs, layers).  Rank handled in chunks of 16.
constexpr int kXtTokens = 32;
__global__ void __launch_bounds__(256) xt_t_kernel(const DevLayer* __restrict__ layers, int l0) {
  const DevLayer& L = layers[l0 + blockIdx.z];
  const int slab = blockIdx.y;
  if (slab >= L.slabs) return;
  const int d0 = blockIdx.x * 256;
  if (d0 >= L.d_in) return;
  const int d = d0 + threadIdx.x;
  const bool d_ok = d < L.d_in;
  const int t_begin = slab * L.slab_rows;
  const int t_end = min(L.m, t_begin + L.slab_rows);
  __shared__ float sT[kXtTokens][16];
  const int r = L.r;
  for (int k0 = 0; k0 < r; k0 += 16) {
    const int kc = min(16, r - k0);
    float acc[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) acc[k] = 0.f;
    for (int tb = t_begin; tb < t_end; tb += kXtTokens) {
      __syncthreads();
      for (int i = threadIdx.x; i < kXtTokens * 16; i += 256) {
        const int tt = i >> 4, k = i & 15;
        sT[tt][k] = (tb + tt < t_end && k < kc) ? L.T[(long long)(tb + tt) * r + k0 + k] : 0.f;
      }
      __syncthreads();
      if (d_ok) {
        const int nt = min(kXtTokens, t_end - tb);
        for (int tt = 0; tt < nt; ++tt) {
          const float x = load_x(L, tb + tt, d);
#pragma unroll
          for (int k = 0; k < 16; ++k) acc[k] = fmaf(x, sT[tt][k], acc[k]);
        }
      }
    }
    if (d_ok) {
      float* out = L.Ypart + ((long long)slab * r + k0) * L.d_in + d;
      for (int k = 0; k < kc; ++k) out[(long long)k * L.d_in] = acc[k];
    }
  }
}

cudaError_t launch_xt_t(const ExtractWave& w, cudaStream_t s) {
  dim3 grid((w.max_din + 255) / 256, w.max_slabs, w.l1 - w.l0);
  xt_t_kernel<<<grid, 256, 0, s>>>(w.d_layers, w.l0);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ T[t][k] = sum_d X[t][d] Q[k][d]   (Q = rows of V)
// one warp per token; Q streamed through shared memory in column chunks.
constexpr int kXqCols = 256;
constexpr int kXqWarps = 8;
__global__ void __launch_bounds__(256) x_q_kernel(const DevLayer* __restrict__ layers, int l0) {
  const DevLayer& L = layers[l0 + blockIdx.y];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tokens_per_block = kXqWarps * 4;
  const int t0 = blockIdx.x * tokens_per_block;
  if (t0 >= L.m) return;
  __shared__ float sQ[16][kXqCols + 1];
  const int r = L.r;
  for (int k0 = 0; k0 < r; k0 += 16) {
    const int kc = min(16, r - k0);
    float acc[4][16];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int k = 0; k < 16; ++k) acc[i][k] = 0.f;
    for (int c0 = 0; c0 < L.d_in; c0 += kXqCols) {
      __syncthreads();
      for (int i = threadIdx.x; i < 16 * kXqCols; i += 256) {
        const int k = i / kXqCols, c = i - k * kXqCols;
        sQ[k][c] = (k < kc && c0 + c < L.d_in) ? L.V[(long long)(k0 + k) * L.ldv + c0 + c] : 0.f;
      }
      __syncthreads();
      const int nc = min(kXqCols, L.d_in - c0);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int t = t0 + warp * 4 + i;
        if (t < L.m) {
          for (int c = lane; c < nc; c += 32) {
            const float x = load_x(L, t, c0 + c);
#pragma unroll
            for (int k = 0; k < 16; ++k) acc[i][k] = fmaf(x, sQ[k][c], acc[i][k]);
          }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int t = t0 + warp * 4 + i;
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        float v = acc[i][k];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0 && t < L.m && k < kc) L.T[(long long)t * r + k0 + k] = v;
      }
    }
  }
}

cudaError_t launch_x_q(const ExtractWave& w, cudaStream_t s) {
  dim3 grid((w.max_m + kXqWarps * 4 - 1) / (kXqWarps * 4), w.l1 - w.l0);
  x_q_kernel<<<grid, 256, 0, s>>>(w.d_layers, w.l0);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ qr(Y), stage 1
// Y[k][d] = sum_s Ypart[s][k][d] (fixed order) and the partial Gram matrix of this block's columns in double.
// A block takes kGramGroup chunks of 128 columns one after another and keeps its sums in registers across
// them.  The panel is fetched four columns per load with a batch of independent loads per thread: the fetch
// latency is what this kernel used to wait for.  The products run on the FP64 tensor cores (mma.sync m8n8k4,
// true double multiply-adds; tcgen05 has no FP64 form): the Gram matrix is cut into 8 x 8 tiles, a warp owns
// whole tiles of the upper triangle and runs through all columns of the block's chunks for them, so no sums
// cross warps and the order of additions is fixed.  Fragments (PTX ISA, m8n8k4 .f64): lane l holds
// A[l / 4][l % 4], B[l % 4][l / 4] and D[l / 4][2 (l % 4) + {0, 1}]; with A = Y[8 bi ..][c ..] and
// B = Y[8 bj ..][c ..]^T both operands are the element (l / 4, l % 4) of a row block of the staged chunk.  Rows
// of the chunk are 132 floats apart, so the 8 x 4 elements a warp reads fall into 32 different banks.
constexpr int kGramCols = 128;
constexpr int kGramGroup = 4;
constexpr int kGramPitch = kGramCols + 4;
constexpr int kApplyMmaMinRank = 16;           // Q = Y M: waves whose largest rank exceeds this take the tensor-core form
constexpr int kGramMmaTilesPerWarp = 5;        // 36 tiles of r = 64 over 8 warps
inline size_t gram_smem_bytes(int max_r) { return (size_t)((max_r + 7) & ~7) * kGramPitch * sizeof(float); }
__device__ __forceinline__ void dmma_m8n8k4(double& c0, double& c1, double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}
__global__ void __launch_bounds__(256) reduce_gram_kernel(const DevLayer* __restrict__ layers, int l0, int y_reduced,
                                                          int after_fused) {
  const DevLayer& L = layers[l0 + blockIdx.y];
  const int nparts = y_parts(L, after_fused);
  const int ngroups = (L.gchunks + kGramGroup - 1) / kGramGroup;
  const int grp = blockIdx.x;
  if (grp >= ngroups) return;
  extern __shared__ __align__(16) unsigned char gram_smem[];
  float* sY = reinterpret_cast<float*>(gram_smem);        // [r8][kGramPitch]
  const int r = L.r, r8 = (r + 7) & ~7, nt = r8 >> 3;
  const int ntiles = nt * (nt + 1) / 2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int fr = lane >> 2, fc = lane & 3;
  // this warp's tiles: t = warp, warp + 8, ... in row-major order of the upper triangle
  int tbi[kGramMmaTilesPerWarp], tbj[kGramMmaTilesPerWarp];
  bool have[kGramMmaTilesPerWarp];
  double acc[kGramMmaTilesPerWarp][2];
#pragma unroll
  for (int q = 0; q < kGramMmaTilesPerWarp; ++q) {
    int t = warp + 8 * q, bi = 0;
    have[q] = t < ntiles;
    while (bi < nt - 1 && t >= nt - bi) { t -= nt - bi; ++bi; }
    tbi[q] = bi;
    tbj[q] = have[q] ? bi + t : bi;
  }
#pragma unroll
  for (int q = 0; q < kGramMmaTilesPerWarp; ++q) acc[q][0] = acc[q][1] = 0.0;
  for (int sub = 0; sub < kGramGroup; ++sub) {
    const int chunk = grp * kGramGroup + sub;
    if (chunk >= L.gchunks) break;
    const int d0 = chunk * kGramCols;
    __syncthreads();                                        // the previous chunk's values have been used
    if ((L.d_in & 3) == 0) {
      // four columns per load and a batch of independent loads per thread before anything waits for one:
      // what this phase costs is the latency of the panel's fetch, paid once per batch instead of per element
      constexpr int kBatch = 4;
      const int nvec = r8 * (kGramCols / 4);
      for (int i0 = threadIdx.x; i0 < nvec; i0 += 256 * kBatch) {
        float4 v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        const int np = y_reduced ? 1 : nparts;
        for (int s = 0; s < np; ++s) {
          float4 t[kBatch];
#pragma unroll
          for (int u = 0; u < kBatch; ++u) {
            const int i = i0 + u * 256;
            const int k = i / (kGramCols / 4), d = d0 + 4 * (i - k * (kGramCols / 4));
            t[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i < nvec && k < r && d < L.d_in) {
              const float* src = y_reduced ? L.Y + (long long)k * L.d_in + d : L.Ypart + ((long long)s * r + k) * L.d_in + d;
              t[u] = *reinterpret_cast<const float4*>(src);
            }
          }
#pragma unroll
          for (int u = 0; u < kBatch; ++u) { v[u].x += t[u].x; v[u].y += t[u].y; v[u].z += t[u].z; v[u].w += t[u].w; }
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const int i = i0 + u * 256;
          if (i >= nvec) continue;
          const int k = i / (kGramCols / 4), c = 4 * (i - k * (kGramCols / 4)), d = d0 + c;
          if (!y_reduced && k < r && d < L.d_in) *reinterpret_cast<float4*>(L.Y + (long long)k * L.d_in + d) = v[u];
          *reinterpret_cast<float4*>(sY + k * kGramPitch + c) = v[u];
        }
      }
    } else
    for (int i = threadIdx.x; i < r8 * kGramCols; i += 256) {
      const int k = i / kGramCols, c = i - k * kGramCols;
      const int d = d0 + c;
      float y = 0.f;
      if (k < r && d < L.d_in) {
        if (y_reduced) {
          y = L.Y[(long long)k * L.d_in + d];
        } else {
          for (int s = 0; s < nparts; ++s) y += L.Ypart[((long long)s * r + k) * L.d_in + d];
          L.Y[(long long)k * L.d_in + d] = y;
        }
      }
      sY[k * kGramPitch + c] = y;
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < kGramMmaTilesPerWarp; ++q) {
      if (have[q]) {
        const float* ya = sY + (8 * tbi[q] + fr) * kGramPitch + fc;
        const float* yb = sY + (8 * tbj[q] + fr) * kGramPitch + fc;
        double c0 = acc[q][0], c1 = acc[q][1];
#pragma unroll 8
        for (int ks = 0; ks < kGramCols / 4; ++ks) dmma_m8n8k4(c0, c1, (double)ya[4 * ks], (double)yb[4 * ks]);
        acc[q][0] = c0; acc[q][1] = c1;
      }
    }
  }
  double* out = L.Gpart + (long long)grp * r * r;
#pragma unroll
  for (int q = 0; q < kGramMmaTilesPerWarp; ++q) {
    if (have[q]) {
      const int i = 8 * tbi[q] + fr;
#pragma unroll
      for (int x = 0; x < 2; ++x) {
        const int j = 8 * tbj[q] + 2 * fc + x;
        if (i < r && j < r && j >= i) out[i * r + j] = acc[q][x];
      }
    }
  }
}

// ------------------------------------------------------------------ qr(Y), stage 2: one block per layer
// S = sum of partial Gram matrices; Cholesky S = R^T R (upper R, positive diagonal); a pivot
// with R_kk <= kRankTol * ||y_k|| (what is left of column k after the columns before it are
// projected out, against the column's own length sqrt(S_kk)) marks a dependent column, which
// becomes zero.  The test is scale-free per column: the columns of Y = H (H^T Q) carry squared
// singular values, so a short column is normal and says nothing about dependence.  M = R^-1 (upper
// triangular, deficient rows and columns zero) is built so that Q = Y M.
//
// What a 64 x 64 factorisation in one block waits for is shared memory, which serves one 64-bit warp access per
// two cycles for the whole SM: with the matrix in shared memory every multiply-add of the trailing update
// costs a load and a store there (measured: 650 of a step's 1800 cycles, the rest latency in the same
// chain).  So the matrix lives in registers: thread (ti, tj) of a 16 x 16 arrangement owns the elements
// (ti + 16 a, tj + 16 c), a, c < 4, of the upper triangle for the whole factorisation, and only row k passes
// through shared memory in step k (published unscaled by its owners, read by everyone after the step's one
// barrier; two buffers in turn, so that the next row can be published while stragglers still read this one).
// Every thread takes the pivot decision itself from the same numbers; one reciprocal square root per pivot
// (R_kk = d rsqrt(d), 1 / d = rsqrt(d)^2).  The finished rows of R go to shared memory for the second half.
//
// M = R^-1 column by column (the columns do not depend on one another), four lanes per column, from the bottom
// up: m_k = 1 / R_kk, then for i = k-1 .. 0  m_i = -(sum_{i<j<=k} R_ij m_j) / R_ii; a deficient index
// contributes nothing and gets zero.  The sums are kept running in registers: lane q owns the rows j = q mod 4
// of its column and, once m_i is known (its owner hands it round), adds R_ji m_i to the rows j < i it owns --
// independent multiply-adds with one shared-memory read each.  The row loop is unrolled over the largest
// rank, so that every register index is a constant.
constexpr int kCholThreads = 256;
constexpr int kCholOwn = AGZO_MAX_RANK / 16;     // rows (and columns) per thread of the 16 x 16 arrangement
static_assert(AGZO_MAX_RANK == 64 && kCholThreads == 4 * AGZO_MAX_RANK, "thread arrangements of chol_kernel");
__global__ void __launch_bounds__(kCholThreads) chol_kernel(const DevLayer* __restrict__ layers, int l0,
                                                            DevStatus* status) {
  const DevLayer& L = layers[l0 + blockIdx.x];
  const int r = L.r, rs = r + 1;        // rows of R are rs doubles apart (bank spread)
  extern __shared__ __align__(16) double chol_smem[];
  double* Sm = chol_smem;               // [r][rs]: R, row by row as the rows become final
  __shared__ double rowbuf[2][AGZO_MAX_RANK];
  __shared__ int bad[AGZO_MAX_RANK];
  __shared__ double own[AGZO_MAX_RANK];   // S_kk before elimination: the squared length of column k
  __shared__ double rinv[AGZO_MAX_RANK];  // 1 / R_kk, 0 for a dependent column
#define S_(i, j) Sm[(i) * rs + (j)]
  const int tid = threadIdx.x;
  const int ti = tid >> 4, tj = tid & 15;
  const int ngroups = (L.gchunks + kGramGroup - 1) / kGramGroup;
  // S = sum of the partial Gram matrices in chunk order, straight into the owners' registers; a thread's
  // elements of one partial matrix are fetched side by side (the lower triangle is never written: not read)
  double sij[kCholOwn][kCholOwn];
#pragma unroll
  for (int a = 0; a < kCholOwn; ++a)
#pragma unroll
    for (int c = 0; c < kCholOwn; ++c) sij[a][c] = 0.0;
  if (r <= 32) {
    // at most 2 x 2 elements per thread: four partial matrices are fetched at a time instead (added in chunk order)
    for (int g0 = 0; g0 < ngroups; g0 += 4) {
      double v[4][2][2];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const double* G = L.Gpart + (long long)min(g0 + u, ngroups - 1) * r * r;
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const int i = ti + 16 * a, j = tj + 16 * c;
            v[u][a][c] = G[(i < r && j < r && j >= i) ? i * r + j : 0];
          }
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            const int i = ti + 16 * a, j = tj + 16 * c;
            sij[a][c] += (g0 + u < ngroups && i < r && j < r && j >= i) ? v[u][a][c] : 0.0;
          }
    }
  } else
  for (int g = 0; g < ngroups; ++g) {
    const double* G = L.Gpart + (long long)g * r * r;
    double v[kCholOwn][kCholOwn];
#pragma unroll
    for (int a = 0; a < kCholOwn; ++a)
#pragma unroll
      for (int c = 0; c < kCholOwn; ++c) {
        const int i = ti + 16 * a, j = tj + 16 * c;
        const bool mine = i < r && j < r && j >= i;
        v[a][c] = G[mine ? i * r + j : 0];                       // unconditional, so that all are in flight at once
      }
#pragma unroll
    for (int a = 0; a < kCholOwn; ++a)
#pragma unroll
      for (int c = 0; c < kCholOwn; ++c) {
        const int i = ti + 16 * a, j = tj + 16 * c;
        sij[a][c] += (i < r && j < r && j >= i) ? v[a][c] : 0.0;
      }
  }
  if (ti == tj) {
#pragma unroll
    for (int a = 0; a < kCholOwn; ++a)
      if (ti + 16 * a < r) own[ti + 16 * a] = sij[a][a];
  }
  double prev_piv = 0.0, prev_rinv = 0.0;
  for (int k = 0; k < r; ++k) {
    double* row = rowbuf[k & 1];
    const int kk = k & 15, ka = k >> 4;
    // a register row is picked with selects (an `if (a == ka)` over the rows would be turned into an indexed,
    // i.e. local-memory, access)
    if (ti == kk) {            // the owners of row k publish it (columns j >= k)
#pragma unroll
      for (int c = 0; c < kCholOwn; ++c) {
        const int j = tj + 16 * c;
        double val = sij[0][c];
        val = ka == 1 ? sij[1][c] : val;
        val = ka == 2 ? sij[2][c] : val;
        val = ka == 3 ? sij[3][c] : val;
        if (j < r && j >= k) row[j] = val;
      }
    }
    if (k > 0 && ti == ((k - 1) & 15)) {   // and the owners of row k - 1, whose pivot everyone knows by now, file it as a row of R
      const int pa = (k - 1) >> 4;
#pragma unroll
      for (int c = 0; c < kCholOwn; ++c) {
        const int j = tj + 16 * c;
        double val = sij[0][c];
        val = pa == 1 ? sij[1][c] : val;
        val = pa == 2 ? sij[2][c] : val;
        val = pa == 3 ? sij[3][c] : val;
        if (j < r && j >= k - 1) S_(k - 1, j) = j == k - 1 ? prev_piv : val * prev_rinv;
      }
    }
    __syncthreads();           // the step's one barrier (own[] and row k are visible)
    const double d = row[k];
    bool b = !(d > 0.0);
    if (!b && d <= kRankTol * kRankTol * own[k]) b = true;
    const double rinv_k = b ? 0.0 : rsqrt(d);
    const double inv = rinv_k * rinv_k;        // 1 / d
    if (tid == 0) {
      bad[k] = b ? 1 : 0;
      rinv[k] = rinv_k;
      if (b) atomicExch(&status->rank_deficient, 1);
    }
    if (!b) {
      double skj[kCholOwn];
#pragma unroll
      for (int c = 0; c < kCholOwn; ++c) skj[c] = tj + 16 * c < r ? row[tj + 16 * c] : 0.0;
#pragma unroll
      for (int a = 0; a < kCholOwn; ++a) {
        const int i = ti + 16 * a;
        if (i > k && i < r) {
          const double t = row[i] * inv;
#pragma unroll
          for (int c = 0; c < kCholOwn; ++c) {
            const int j = tj + 16 * c;
            if (j >= i && j < r) sij[a][c] -= t * skj[c];
          }
        }
      }
    }
    prev_piv = d * rinv_k;                     // sqrt(d), 0 for a dependent column
    prev_rinv = rinv_k;
  }
  if (ti == ((r - 1) & 15) && tj + 16 * ((r - 1) >> 4) == r - 1) S_(r - 1, r - 1) = prev_piv;   // the last row is its pivot alone
  __syncthreads();
  {
    const int k = tid >> 2, q = tid & 3, lane = tid & 31;
    const bool live = k < r && !bad[k < r ? k : 0];
    double mv[AGZO_MAX_RANK / 4];
#pragma unroll
    for (int t = 0; t < AGZO_MAX_RANK / 4; ++t) mv[t] = 0.0;
#pragma unroll
    for (int t4 = AGZO_MAX_RANK / 4 - 1; t4 >= 0; --t4) {
#pragma unroll
      for (int s4 = 3; s4 >= 0; --s4) {
        const int i = 4 * t4 + s4;
        if (i < r) {                                     // the same for every thread of the block
          double mi = 0.0;
          if (s4 == q) {
            if (live && i <= k && !bad[i]) mi = i == k ? rinv[i] : -mv[t4] * rinv[i];
            mv[t4] = mi;                                 // final: 0 above the diagonal and for a deficient row
          }
          mi = __shfl_sync(0xffffffffu, mi, (lane & ~3) | s4);
          if (mi != 0.0) {
#pragma unroll
            for (int t = 0; t < AGZO_MAX_RANK / 4; ++t) {
              const int j = q + 4 * t;
              if (t <= t4 && j < i) mv[t] += S_(j, i) * mi;
            }
          }
        }
      }
    }
    if (k < r) {
#pragma unroll
      for (int t = 0; t < AGZO_MAX_RANK / 4; ++t) {
        const int j = q + 4 * t;
        if (j < r) L.M[j * r + k] = mv[t];
      }
    }
  }
#undef S_
}
size_t chol_smem_bytes(int r) { return (size_t)r * (r + 1) * sizeof(double); }

// ------------------------------------------------------------------ qr(Y), stage 3: Q = Y M
// thread per column d, eight columns of Q at a time (M is upper triangular: column k needs Y's
// columns 0..k); writes Q (fp32) into V and, for the tensor-core path, the bf16 hi/lo panels.
__global__ void __launch_bounds__(128) apply_kernel(const DevLayer* __restrict__ layers, int l0) {
  const DevLayer& L = layers[l0 + blockIdx.y];
  const int d = blockIdx.x * 128 + threadIdx.x;
  extern __shared__ __align__(16) double sM[];   // [r][r8], r8 = r rounded up to 8, padding zero
  const int r = L.r, r8 = (r + 7) & ~7;
  for (int p = threadIdx.x; p < r * r8; p += 128) {
    const int j = p / r8, k = p - j * r8;
    sM[p] = k < r ? L.M[j * r + k] : 0.0;
  }
  __syncthreads();
  if (d >= L.d_in || blockIdx.x * 128 >= L.d_in) return;
  for (int kb = 0; kb < r; kb += 8) {
    double acc[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) acc[u] = 0.0;
    const int jend = min(r, kb + 8);
    for (int j = 0; j < jend; ++j) {
      const double y = (double)L.Y[(long long)j * L.d_in + d];
      const double* m = sM + j * r8 + kb;
#pragma unroll
      for (int u = 0; u < 8; ++u) acc[u] = fma(y, m[u], acc[u]);   // M[j][k] = 0 for j > k
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int k = kb + u;
      if (k >= r) break;
      const float q = (float)acc[u];
      L.V[(long long)k * L.ldv + d] = q;
      if (L.Qb) {
        const __nv_bfloat16 hi = __float2bfloat16_rn(q);
        const __nv_bfloat16 lo = __float2bfloat16_rn(q - __bfloat162float(hi));
        L.Qb[(long long)k * L.d_in + d] = hi;
        L.Qb[(long long)(L.NP + k) * L.d_in + d] = lo;
      }
    }
  }
  if (L.Qb) {   // padding rows of the operand panel stay zero
    for (int k = r; k < L.NP; ++k) {
      L.Qb[(long long)k * L.d_in + d] = __float2bfloat16_rn(0.f);
      L.Qb[(long long)(L.NP + k) * L.d_in + d] = __float2bfloat16_rn(0.f);
    }
  }
}

// The same product for larger ranks on the FP64 tensor cores: Q (r x 128 columns) = M^T (r x r) Y (r x 128) in
// 8 x 8 tiles, A[k][j] = M[j][k], B[j][d] = Y[j][d], K = j in steps of four up to the tile's last k (M is upper
// triangular).  A warp owns two 8-column strips of the block's 128 columns and all k tiles of them, so a B
// fragment serves every k tile at or below it.  Pitches (136 floats for Y, r8 + 4 doubles for M) spread a
// fragment's 32 elements over the banks.
constexpr int kApplyYPitch = kGramCols + 8;
__host__ __device__ inline int apply_m_pitch(int r8) { return ((r8 + 15) & ~15) + 4; }
inline size_t apply_mma_smem_bytes(int max_r) {
  const int r8 = (max_r + 7) & ~7;
  return (size_t)r8 * apply_m_pitch(r8) * sizeof(double) + (size_t)r8 * kApplyYPitch * sizeof(float);
}
__global__ void __launch_bounds__(256) apply_mma_kernel(const DevLayer* __restrict__ layers, int l0) {
  const DevLayer& L = layers[l0 + blockIdx.y];
  const int d0 = blockIdx.x * kGramCols;
  if (d0 >= L.d_in) return;
  extern __shared__ __align__(16) double apply_smem[];
  const int r = L.r, r8 = (r + 7) & ~7, nt = r8 >> 3, mp = apply_m_pitch(r8);
  double* sM = apply_smem;                                   // [r8][mp], rows and columns beyond r zero
  float* sY = reinterpret_cast<float*>(sM + r8 * mp);        // [r8][kApplyYPitch]
  if (r == r8) {               // two doubles per load, a batch of independent loads per thread (M is 256-byte aligned)
    constexpr int kBatchM = 8;
    const int nv2 = r * r / 2, half = r / 2;
    for (int i0 = threadIdx.x; i0 < nv2; i0 += 256 * kBatchM) {
      double2 v[kBatchM];
#pragma unroll
      for (int u = 0; u < kBatchM; ++u) {
        const int i = i0 + u * 256;
        v[u] = i < nv2 ? reinterpret_cast<const double2*>(L.M)[i] : make_double2(0.0, 0.0);
      }
#pragma unroll
      for (int u = 0; u < kBatchM; ++u) {
        const int i = i0 + u * 256;
        if (i >= nv2) continue;
        const int j = i / half, k = 2 * (i - j * half);
        *reinterpret_cast<double2*>(sM + j * mp + k) = v[u];
      }
    }
  } else {
    for (int p = threadIdx.x; p < r8 * r8; p += 256) {
      const int j = p / r8, k = p - j * r8;
      sM[j * mp + k] = (j < r && k < r) ? L.M[j * r + k] : 0.0;
    }
  }
  if ((L.d_in & 3) == 0) {     // four columns per load, a batch of independent loads per thread
    constexpr int kBatch = 4;
    const int nvec = r8 * (kGramCols / 4);
    for (int i0 = threadIdx.x; i0 < nvec; i0 += 256 * kBatch) {
      float4 v[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = i0 + u * 256;
        const int k = i / (kGramCols / 4), d = d0 + 4 * (i - k * (kGramCols / 4));
        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (i < nvec && k < r && d < L.d_in) v[u] = *reinterpret_cast<const float4*>(L.Y + (long long)k * L.d_in + d);
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = i0 + u * 256;
        if (i >= nvec) continue;
        const int k = i / (kGramCols / 4), c = 4 * (i - k * (kGramCols / 4));
        *reinterpret_cast<float4*>(sY + k * kApplyYPitch + c) = v[u];
      }
    }
  } else {
    for (int i = threadIdx.x; i < r8 * kGramCols; i += 256) {
      const int k = i / kGramCols, c = i - k * kGramCols;
      sY[k * kApplyYPitch + c] = (k < r && d0 + c < L.d_in) ? L.Y[(long long)k * L.d_in + d0 + c] : 0.f;
    }
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int fr = lane >> 2, fc = lane & 3;
  double acc[2][AGZO_MAX_RANK / 8][2];
#pragma unroll
  for (int sp = 0; sp < 2; ++sp) {
    const int dc = 8 * (2 * warp + sp);                      // first column of the strip inside the block
#pragma unroll
    for (int kt = 0; kt < AGZO_MAX_RANK / 8; ++kt) acc[sp][kt][0] = acc[sp][kt][1] = 0.0;
    if (d0 + dc >= L.d_in) continue;
    for (int j0 = 0; j0 < r8; j0 += 4) {
      const double b = (double)sY[(j0 + fc) * kApplyYPitch + dc + fr];
      const double* ma = sM + (j0 + fc) * mp + fr;
#pragma unroll
      for (int kt = 0; kt < AGZO_MAX_RANK / 8; ++kt)
        if (kt < nt && 8 * kt + 7 >= j0) dmma_m8n8k4(acc[sp][kt][0], acc[sp][kt][1], ma[8 * kt], b);
    }
  }
  // Q leaves through shared memory (the Y chunk's place), so that the global stores are whole rows of the block:
  // a fragment's own layout would write two columns per thread, i.e. partial sectors of V and of the bf16 panels
  __syncthreads();
#pragma unroll
  for (int sp = 0; sp < 2; ++sp) {
    const int dc = 8 * (2 * warp + sp);
#pragma unroll
    for (int kt = 0; kt < AGZO_MAX_RANK / 8; ++kt)
      if (kt < nt)
        *reinterpret_cast<float2*>(sY + (8 * kt + fr) * kApplyYPitch + dc + 2 * fc) =
            make_float2((float)acc[sp][kt][0], (float)acc[sp][kt][1]);
  }
  __syncthreads();
  const int c = threadIdx.x & (kGramCols - 1), d = d0 + c;
  if (d >= L.d_in) return;
  for (int k = threadIdx.x >> 7; k < r; k += 2) {
    const float q = sY[k * kApplyYPitch + c];
    L.V[(long long)k * L.ldv + d] = q;
    if (L.Qb) {
      const __nv_bfloat16 hi = __float2bfloat16_rn(q);
      const __nv_bfloat16 lo = __float2bfloat16_rn(q - __bfloat162float(hi));
      L.Qb[(long long)k * L.d_in + d] = hi;
      L.Qb[(long long)(L.NP + k) * L.d_in + d] = lo;
    }
  }
  if (L.Qb) {   // padding rows of the operand panel stay zero
    for (int k = r + (threadIdx.x >> 7); k < L.NP; k += 2) {
      L.Qb[(long long)k * L.d_in + d] = __float2bfloat16_rn(0.f);
      L.Qb[(long long)(L.NP + k) * L.d_in + d] = __float2bfloat16_rn(0.f);
    }
  }
}

// Y[k][d] = sum_s Ypart[s][k][d] in slab order, on its own: token-sharded extraction sums Y over
// the ranks before the panel QR reads it
__global__ void __launch_bounds__(256) sum_slabs_kernel(const DevLayer* __restrict__ layers, int l0, int after_fused) {
  const DevLayer& L = layers[l0 + blockIdx.y];
  const int nparts = y_parts(L, after_fused);
  const long long n = (long long)L.r * L.d_in;
  for (long long i = blockIdx.x * 256ll + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
    float y = 0.f;
    for (int s = 0; s < nparts; ++s) y += L.Ypart[(long long)s * n + i];
    L.Y[i] = y;
  }
}

cudaError_t launch_sum_slabs(const ExtractWave& w, cudaStream_t s) {
  long long blocks = ((long long)w.max_r * w.max_din + 255) / 256;
  if (blocks > 256) blocks = 256;
  sum_slabs_kernel<<<dim3((unsigned)blocks, w.l1 - w.l0), 256, 0, s>>>(w.d_layers, w.l0, w.after_fused);
  return cudaGetLastError();
}

cudaError_t launch_panel_qr(const ExtractWave& w, DevStatus* d_status, cudaStream_t s) {
  const int nl = w.l1 - w.l0;
  const dim3 gram_grid((w.max_gchunks + kGramGroup - 1) / kGramGroup, nl);
  reduce_gram_kernel<<<gram_grid, 256, gram_smem_bytes(w.max_r), s>>>(w.d_layers, w.l0, w.y_reduced, w.after_fused);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const size_t chol_bytes = chol_smem_bytes(w.max_r);
  if (chol_bytes > 48 * 1024) {   // above the default limit of dynamic shared memory
    e = cudaFuncSetAttribute(chol_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)chol_smem_bytes(AGZO_MAX_RANK));
    if (e != cudaSuccess) return e;
  }
  chol_kernel<<<nl, kCholThreads, chol_bytes, s>>>(w.d_layers, w.l0, d_status);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (w.max_r > kApplyMmaMinRank) {   // below that the thread-per-column form is faster (5.3 against 3.5 ms per 168 launches at r = 16)
    const size_t bytes = apply_mma_smem_bytes(w.max_r);
    if (bytes > 48 * 1024) {
      e = cudaFuncSetAttribute(apply_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)apply_mma_smem_bytes(AGZO_MAX_RANK));
      if (e != cudaSuccess) return e;
    }
    apply_mma_kernel<<<dim3((w.max_din + kGramCols - 1) / kGramCols, nl), 256, bytes, s>>>(w.d_layers, w.l0);
  } else {
    apply_kernel<<<dim3((w.max_din + 127) / 128, nl), 128, (size_t)w.max_r * ((w.max_r + 7) & ~7) * sizeof(double), s>>>(
        w.d_layers, w.l0);
  }
  return cudaGetLastError();
}

}  // namespace agzo
