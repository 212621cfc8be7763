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
// Y[k][d] = sum_s Ypart[s][k][d] (fixed order) and the partial Gram matrix of this block's
// columns in double.  A block takes kGramGroup chunks of 128 columns one after another and keeps
// its sums in registers across them: thread = (4 x 4 block of the Gram matrix, part of the
// columns), so every pair of loaded values feeds 16 multiply-adds.
constexpr int kGramCols = 128;
constexpr int kGramGroup = 4;
__host__ __device__ inline int gram_csplit(int r4) {   // column parts per chunk: as many as 256 threads allow
  const int nsq = (r4 >> 2) * (r4 >> 2);
  int cs = 16;
  while (cs > 1 && cs * nsq > 256) cs >>= 1;
  return cs;
}
__host__ __device__ inline size_t gram_smem_bytes(int r) {
  const int r4 = (r + 3) & ~3;
  const size_t y = (size_t)r4 * kGramCols * sizeof(float);
  const size_t red = (size_t)gram_csplit(r4) * r4 * r4 * sizeof(double);
  return y > red ? y : red;
}
// the launch serves layers of several ranks, and the need is not monotone in r (fewer column
// parts fit at larger r): take the largest need over all ranks up to the wave's maximum
inline size_t gram_smem_bytes_upto(int max_r) {
  size_t b = 0;
  for (int r = 1; r <= max_r; ++r) b = gram_smem_bytes(r) > b ? gram_smem_bytes(r) : b;
  return b;
}
__global__ void __launch_bounds__(256) reduce_gram_kernel(const DevLayer* __restrict__ layers, int l0, int y_reduced,
                                                          int after_fused) {
  const DevLayer& L = layers[l0 + blockIdx.y];
  const int nparts = y_parts(L, after_fused);
  const int ngroups = (L.gchunks + kGramGroup - 1) / kGramGroup;
  const int grp = blockIdx.x;
  if (grp >= ngroups) return;
  extern __shared__ __align__(16) unsigned char gram_smem[];
  float* sY = reinterpret_cast<float*>(gram_smem);        // [r4][kGramCols]; later reused for the column parts' sums
  const int r = L.r, r4 = (r + 3) & ~3, nb = r4 >> 2;
  const int csplit = gram_csplit(r4), clen = kGramCols / csplit;
  const int unit = threadIdx.x;
  const int sq = unit / csplit, cs = unit - sq * csplit;
  const int bi = sq / nb, bj = sq - bi * nb;
  const bool busy = sq < nb * nb && bj >= bi;               // upper triangle of 4 x 4 blocks
  double acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;
  const int rot = threadIdx.x & 31;
  for (int sub = 0; sub < kGramGroup; ++sub) {
    const int chunk = grp * kGramGroup + sub;
    if (chunk >= L.gchunks) break;
    const int d0 = chunk * kGramCols;
    __syncthreads();                                        // the previous chunk's values have been used
    for (int i = threadIdx.x; i < r4 * kGramCols; i += 256) {
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
      sY[i] = y;
    }
    __syncthreads();
    if (busy) {
      const float* yi = sY + (4 * bi) * kGramCols;
      const float* yj = sY + (4 * bj) * kGramCols;
      // rows are 128 floats apart, so all rows share a bank at equal c: every lane starts at its own
      // column of its part (a fixed rotation, so the sum is the same on every run)
      for (int c = 0; c < clen; ++c) {
        const int cc = cs * clen + ((c + rot) & (clen - 1));
        double a[4], b[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) { a[x] = (double)yi[x * kGramCols + cc]; b[x] = (double)yj[x * kGramCols + cc]; }
#pragma unroll
        for (int x = 0; x < 4; ++x)
#pragma unroll
          for (int y = 0; y < 4; ++y) acc[x][y] = fma(a[x], b[y], acc[x][y]);
      }
    }
  }
  // the column parts of a block are added in a fixed order through shared memory
  __syncthreads();
  double* red = reinterpret_cast<double*>(gram_smem);     // [csplit][r4][r4]
  if (busy) {
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) red[((size_t)cs * r4 + 4 * bi + x) * r4 + 4 * bj + y] = acc[x][y];
  }
  __syncthreads();
  double* out = L.Gpart + (long long)grp * r * r;
  for (int p = threadIdx.x; p < r * r; p += 256) {
    const int i = p / r, j = p - i * r;
    if (j < i) continue;
    double t = 0.0;
    for (int q = 0; q < csplit; ++q) t += red[((size_t)q * r4 + i) * r4 + j];
    out[p] = t;
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
// One barrier per Cholesky step: step k updates the trailing matrix from the still unscaled row
// k (a_ki a_kj / a_kk), and row k is divided by its pivot during step k + 1, which no longer
// reads it.  The columns of M do not depend on one another, so four lanes share a column and all
// columns are solved side by side (back substitution, the lanes splitting each dot product).
constexpr int kCholThreads = 256;
__global__ void __launch_bounds__(kCholThreads) chol_kernel(const DevLayer* __restrict__ layers, int l0,
                                                            DevStatus* status) {
  const DevLayer& L = layers[l0 + blockIdx.x];
  const int r = L.r, rs = r + 1;        // rows of S and M are rs doubles apart (bank spread)
  extern __shared__ __align__(16) double chol_smem[];
  double* Sm = chol_smem;               // [r][rs]
  double* Mm = chol_smem + r * rs;      // [r][rs]; copied to L.M at the end
  __shared__ int bad[AGZO_MAX_RANK];
  __shared__ double own[AGZO_MAX_RANK];   // S_kk before elimination: the squared length of column k
#define S_(i, j) Sm[(i) * rs + (j)]
#define M_(i, j) Mm[(i) * rs + (j)]
  const int tid = threadIdx.x;
  const int ti = tid >> 4, tj = tid & 15;          // 16 x 16 arrangement for the trailing update
  const int ngroups = (L.gchunks + kGramGroup - 1) / kGramGroup;
  for (int p = tid; p < r * r; p += kCholThreads) {
    const int i = p / r, j = p - i * r;
    double acc = 0.0;
    if (j >= i)
      for (int c = 0; c < ngroups; ++c) acc += L.Gpart[(long long)c * r * r + p];   // fixed order
    S_(i, j) = acc;
    M_(i, j) = 0.0;
    if (i == j) own[i] = acc;
  }
  __syncthreads();
  // right-looking Cholesky on the upper triangle; S is overwritten by R.  Every thread takes the
  // pivot decision itself from the same numbers.
  double prev_piv = 0.0;
  for (int k = 0; k < r; ++k) {
    const double d = S_(k, k);
    bool b = !(d > 0.0);
    const double sq = b ? 0.0 : sqrt(d);
    if (!b && d <= kRankTol * kRankTol * own[k]) b = true;
    const double pk = b ? 0.0 : sq;
    if (k > 0) {    // row k - 1 is final now: divide it by its pivot (nobody reads it in this step)
      for (int j = k - 1 + tid; j < r; j += kCholThreads)
        S_(k - 1, j) = j == k - 1 ? prev_piv : (prev_piv > 0.0 ? S_(k - 1, j) / prev_piv : 0.0);
    }
    if (tid == 0) {
      bad[k] = b ? 1 : 0;
      if (b) atomicExch(&status->rank_deficient, 1);
    }
    if (!b) {
      const double inv = 1.0 / d;
      for (int i = k + 1 + ti; i < r; i += 16) {
        const double t = S_(k, i) * inv;
        for (int j = k + 1 + tj; j < r; j += 16)
          if (j >= i) S_(i, j) -= t * S_(k, j);
      }
    }
    prev_piv = pk;
    __syncthreads();
  }
  for (int j = r - 1 + tid; j < r; j += kCholThreads) S_(r - 1, j) = prev_piv;   // the last row is its pivot alone
  __syncthreads();
  // M = R^-1 column by column, four lanes per column: m_k = 1 / R_kk, then for i = k-1 .. 0
  // m_i = -(sum_{i<j<=k} R_ij m_j) / R_ii; a deficient index contributes nothing and gets zero
  for (int c0 = 0; c0 < r; c0 += kCholThreads / 4) {
    const int k = c0 + (tid >> 2), q = tid & 3;
    const bool live = k < r && !bad[k < r ? k : 0];
    if (live && q == 0) M_(k, k) = 1.0 / S_(k, k);
    __syncwarp();
    for (int i = r - 2; i >= 0; --i) {             // the same trip count for every lane of the warp
      double part = 0.0;
      const bool row = live && i < k && !bad[i];
      if (row)
        for (int j = i + 1 + q; j <= k; j += 4) part += S_(i, j) * M_(j, k);
      part += __shfl_xor_sync(0xffffffffu, part, 1);
      part += __shfl_xor_sync(0xffffffffu, part, 2);
      if (row && q == 0) M_(i, k) = -part / S_(i, i);
      __syncwarp();
    }
  }
  __syncthreads();
  for (int p = tid; p < r * r; p += kCholThreads) L.M[p] = M_(p / r, p % r);
#undef S_
#undef M_
}
size_t chol_smem_bytes(int r) { return (size_t)2 * r * (r + 1) * sizeof(double); }

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
  reduce_gram_kernel<<<dim3((w.max_gchunks + kGramGroup - 1) / kGramGroup, nl), 256, gram_smem_bytes_upto(w.max_r), s>>>(
      w.d_layers, w.l0, w.y_reduced, w.after_fused);
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
  apply_kernel<<<dim3((w.max_din + 127) / 128, nl), 128, (size_t)w.max_r * ((w.max_r + 7) & ~7) * sizeof(double), s>>>(
      w.d_layers, w.l0);
  return cudaGetLastError();
}

}  // namespace agzo
