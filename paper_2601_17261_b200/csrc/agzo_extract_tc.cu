// Tensor-core path of Algorithm 1's two products with X on sm_100a: TMA-fed shared-memory
// tiles, tcgen05.mma with fp32 accumulators in TMEM, one elected thread issuing.
//
//   x_q :  T  = H^T Q = X Q        M = 128 tokens, N = NB, K = d_in   (A = X tile, K-major)
//   xt_t:  Y  = H T   = X^T T      M = 128 columns of X, N = NB, K = tokens
//                                  (A = the same kind of X tile read as an MN-major operand)
//
// X is bf16 and exact; Q and T are fp32 quantities, so each is split as hi + lo in bf16 and
// the two parts sit side by side as extra N columns (N = NB = 2*NP, NP = r rounded up to 8):
// the products are exact, the accumulation is fp32, and the column groups are summed in the
// epilogue.  The kernels are HBM-bound (about r flop per byte of X), so the doubled N is free.
//
// Operand panels: Qb [NB][d_in] bf16 (written by the panel-QR apply kernel) and
// Tt [NB][m_pad] bf16 (T transposed; written by x_q's epilogue or by the Omega fill), both
// K-major B operands.  Every wait on an mbarrier is bounded; a wait that runs out sets the
// status word and the CTA leaves through the common exit (TMEM freed).
#include <cuda.h>

#include <cstring>

#include "agzo_ptx.cuh"
#include "agzo_tc.cuh"

namespace agzo {

namespace {

using namespace ptx;

constexpr int kTcThreads = 192;        // warp 0: TMA producer, warp 1: MMA issuer, warps 2..5: epilogue
constexpr int kBoxK = 64;              // elements per 128-byte swizzle row
constexpr int kTileBytes = 64 * kBoxK * 2;   // one [64 rows][64 elems] bf16 box = 8 KiB
constexpr size_t kMinSmem = 80 * 1024;  // keeps at most 2 CTAs per SM: 2 * 128 TMEM columns fit

struct TcShared {
  uint64_t full[8];
  uint64_t empty[8];
  uint64_t accum;
  uint32_t tmem_base;
  int failed;
};

__device__ __forceinline__ uint32_t pow2_cols(int n) {
  uint32_t c = 32;
  while ((int)c < n) c <<= 1;
  return c;
}

__device__ __forceinline__ void split_bf16(float v, __nv_bfloat16* hi, __nv_bfloat16* lo) {
  const __nv_bfloat16 h = __float2bfloat16_rn(v);
  *hi = h;
  *lo = __float2bfloat16_rn(v - __bfloat162float(h));
}

// ---------------------------------------------------------------- T = X Q  (Tt = T^T as bf16 hi/lo)
// One CTA per 128-token tile of one layer.  grid = (max token tiles, layers in the wave).
__global__ void __launch_bounds__(kTcThreads) tc_x_q_kernel(const DevLayer* __restrict__ layers, int l0,
                                                            DevStatus* status, int stages, int skip_fused) {
  // CTA rows are handed out in the order the scheduler starts them: the layers with the longest
  // token rows (largest d_in, longest CTAs) go first so that the wave does not end on them
  const int li = l0 + layers[l0 + blockIdx.y].xq_order;
  const DevLayer& L = layers[li];
  const int t0 = blockIdx.x * 128;
  if (t0 >= L.m || (skip_fused && L.fz_C) || L.grp_role == 2) return;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ TcShared sh;
  const int NB = L.grp_role == 1 ? L.grp_NB : L.NB;   // operand rows: the whole group's for a leader
  const int nmem = L.grp_role == 1 ? L.grp_n : 1;
  const int a_bytes = 2 * kTileBytes;                 // [128 tokens][64 d]
  const int b_bytes = NB * kBoxK * 2;                 // [NB][64 d]
  const int stage_bytes = a_bytes + ((b_bytes + 1023) & ~1023);
  const int nk = (L.d_in + kBoxK - 1) / kBoxK;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint8_t* maps = reinterpret_cast<const uint8_t*>(L.tmaps);
  const void* map_x = maps;            // X  [m][d_in], box 64 x 64
  const void* map_q = maps + 128;      // Qb [NB][d_in], box 64 x NB
  const uint32_t ncols = pow2_cols(NB);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    mbar_init(&sh.accum, 1);
    sh.failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&sh.tmem_base, ncols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      tmap_acquire(map_x);
      tmap_acquire(map_q);
      // With four or more stages, two k-steps are issued together, box by box: the two 128-byte
      // pieces of a token row then reach the memory system back to back (256 contiguous bytes per
      // row instead of 128; 8B shapes, r = 16: T = X Q 20.6 -> 17.6 ms per step).  With three
      // stages waiting for two free ones at a time costs more than it brings.
      bool ok = true;
      int issued = 0;            // k-steps whose loads have been issued
      const int group = stages >= 4 ? 2 : 1;
      for (int k = 0; k < nk && ok; k += group) {
        const int n2 = min(group, nk - k);
        uint8_t* a[2];
        uint64_t* bar[2];
        for (int u = 0; u < n2; ++u) {
          const int kk = k + u, s = kk % stages;
          if (kk >= stages && !mbar_wait(&sh.empty[s], ((kk / stages) - 1) & 1)) { sh.failed = 1; ok = false; break; }
          a[u] = tiles + (size_t)s * stage_bytes;
          bar[u] = &sh.full[s];
          mbar_expect_tx(bar[u], a_bytes + b_bytes);
        }
        if (!ok) break;
        for (int u = 0; u < n2; ++u) tma_load_2d(a[u], map_x, (k + u) * kBoxK, t0, bar[u]);
        for (int u = 0; u < n2; ++u) tma_load_2d(a[u] + kTileBytes, map_x, (k + u) * kBoxK, t0 + 64, bar[u]);
        for (int u = 0; u < n2; ++u) tma_load_2d(a[u] + a_bytes, map_q, (k + u) * kBoxK, 0, bar[u]);
        issued = k + n2;
      }
      if (!ok || sh.failed) {    // leaving early: the copies in flight must land before the CTA goes away
        for (int k = issued > stages ? issued - stages : 0; k < issued; ++k) mbar_wait(&sh.full[k % stages], (k / stages) & 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc(128, NB, 0, 0);
      bool ok = true;
      for (int k = 0; k < nk && ok; ++k) {
        const int s = k % stages;
        if (!mbar_wait(&sh.full[s], (k / stages) & 1)) { sh.failed = 1; ok = false; break; }
        tc_fence_after();
        const uint32_t a = smem_u32(tiles + (size_t)s * stage_bytes);
        const uint32_t b = a + a_bytes;
#pragma unroll
        for (int kk = 0; kk < kBoxK / 16; ++kk) {
          const uint64_t ad = smem_desc(a + kk * 32, 0, 1024);
          const uint64_t bd = smem_desc(b + kk * 32, 0, 1024);
          mma_bf16(tmem, ad, bd, idesc, (k > 0 || kk > 0) ? 1u : 0u);
        }
        mma_commit(&sh.empty[s]);      // the stage is free once these MMAs have read it
      }
      mma_commit(&sh.accum);           // arrives when every MMA issued so far is done
    }
  } else {
    // epilogue: TMEM lane i of this warp's quarter = token t0 + 32*q + lane
    const int q = warp & 3;
    const bool ok = mbar_wait(&sh.accum, 0);
    tc_fence_after();
    if (!ok) sh.failed = 1;
    const int t = t0 + q * 32 + lane;
    if (ok) {
      for (int mi = 0; mi < nmem; ++mi) {               // the layers this CTA serves
        const DevLayer& M = layers[li + mi];
        const int NP = M.NP, off = L.grp_role == 1 ? M.grp_off : 0;
        __nv_bfloat16* Tt = M.Tb;
        const long long mp = M.m_pad;
        for (int k0 = 0; k0 < NP; k0 += 8) {
          float hi[8], lo[8];
          tmem_ld8(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(off + k0), hi);
          tmem_ld8(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(off + NP + k0), lo);
          if (t < L.m) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              __nv_bfloat16 h, l;
              split_bf16(hi[j] + lo[j], &h, &l);
              Tt[(long long)(k0 + j) * mp + t] = h;
              Tt[(long long)(NP + k0 + j) * mp + t] = l;
            }
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (sh.failed && threadIdx.x == 0) { atomicExch(&status->timeout, 1); atomicExch(&status->where, 1); }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, ncols); }
}

// ---------------------------------------------------------------- Ypart[s] = X_s^T T_s
// One CTA per (128 columns of X, token slab) of one layer.  grid = (column chunks, slabs, layers).
__global__ void __launch_bounds__(kTcThreads) tc_xt_t_kernel(const DevLayer* __restrict__ layers, int l0,
                                                             DevStatus* status, int stages, int skip_fused) {
  const DevLayer& L = layers[l0 + blockIdx.z];
  const int d0 = blockIdx.x * 128;
  const int slab = blockIdx.y;
  if (d0 >= L.d_in || slab >= L.slabs || (skip_fused && L.fz_C) || L.grp_role == 2) return;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ TcShared sh;
  const int NB = L.grp_role == 1 ? L.grp_NB : L.NB;
  const int nmem = L.grp_role == 1 ? L.grp_n : 1;
  const int a_bytes = 2 * kTileBytes;                 // two [64 tokens][64 d] boxes: d0.., d0+64..
  const int b_bytes = NB * kBoxK * 2;                 // [NB][64 tokens]
  const int stage_bytes = a_bytes + ((b_bytes + 1023) & ~1023);
  const int t_begin = slab * L.slab_rows;
  const int t_end = min(L.m, t_begin + L.slab_rows);
  const int nk = (t_end - t_begin + kBoxK - 1) / kBoxK;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint8_t* maps = reinterpret_cast<const uint8_t*>(L.tmaps);
  const void* map_x = maps;            // X  [m][d_in], box 64 x 64
  const void* map_t = maps + 256;      // Tt [NB][m],   box 64 x NB
  const uint32_t ncols = pow2_cols(NB);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    mbar_init(&sh.accum, 1);
    sh.failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&sh.tmem_base, ncols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      tmap_acquire(map_x);
      tmap_acquire(map_t);
      int issued = 0;
      for (int k = 0; k < nk; ++k) {
        const int s = k % stages;
        if (k >= stages && !mbar_wait(&sh.empty[s], ((k / stages) - 1) & 1)) { sh.failed = 1; break; }
        uint8_t* a = tiles + (size_t)s * stage_bytes;
        const int tk = t_begin + k * kBoxK;
        mbar_expect_tx(&sh.full[s], a_bytes + b_bytes);
        tma_load_2d(a, map_x, d0, tk, &sh.full[s]);
        tma_load_2d(a + kTileBytes, map_x, d0 + 64, tk, &sh.full[s]);
        tma_load_2d(a + a_bytes, map_t, tk, 0, &sh.full[s]);
        issued = k + 1;
      }
      if (sh.failed) {           // leaving early: the copies in flight must land before the CTA goes away
        for (int k = issued > stages ? issued - stages : 0; k < issued; ++k) mbar_wait(&sh.full[k % stages], (k / stages) & 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc(128, NB, 1, 0);     // A is MN-major: the X tile as X^T
      bool ok = true;
      for (int k = 0; k < nk && ok; ++k) {
        const int s = k % stages;
        if (!mbar_wait(&sh.full[s], (k / stages) & 1)) { sh.failed = 1; ok = false; break; }
        tc_fence_after();
        const uint32_t a = smem_u32(tiles + (size_t)s * stage_bytes);
        const uint32_t b = a + a_bytes;
#pragma unroll
        for (int kk = 0; kk < kBoxK / 16; ++kk) {
          // 16 tokens = two 8-row swizzle atoms = 2048 bytes further down the X boxes
          const uint64_t ad = smem_desc(a + kk * 2048, kTileBytes, 1024);
          const uint64_t bd = smem_desc(b + kk * 32, 0, 1024);
          mma_bf16(tmem, ad, bd, idesc, (k > 0 || kk > 0) ? 1u : 0u);
        }
        mma_commit(&sh.empty[s]);
      }
      mma_commit(&sh.accum);
    }
  } else {
    const int q = warp & 3;
    const bool ok = mbar_wait(&sh.accum, 0);
    tc_fence_after();
    if (!ok) sh.failed = 1;
    const int d = d0 + q * 32 + lane;
    if (ok) {
      for (int mi = 0; mi < nmem; ++mi) {               // the layers this CTA serves (same slabs: same m)
        const DevLayer& M = layers[l0 + blockIdx.z + mi];
        const int r = M.r, NP = M.NP, off = L.grp_role == 1 ? M.grp_off : 0;
        float* out = M.Ypart + (long long)slab * r * L.d_in + d;
        for (int k0 = 0; k0 < NP; k0 += 8) {
          float hi[8], lo[8];
          tmem_ld8(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(off + k0), hi);
          tmem_ld8(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(off + NP + k0), lo);
          if (d < L.d_in) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (k0 + j < r) out[(long long)(k0 + j) * L.d_in] = hi[j] + lo[j];
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (sh.failed && threadIdx.x == 0) { atomicExch(&status->timeout, 1); atomicExch(&status->where, 2); }
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, ncols); }
}

// ---------------------------------------------------------------- Omega -> Tt (hi/lo), pads zero
// Tt is [NB][m_pad] with the tokens contiguous, Omega's stream is row-major over (token, k): a
// thread takes one token and eight consecutive k (at most three Philox blocks), so that for every
// k a warp writes 32 neighbouring tokens.  Local token t is row row0 + t of the whole batch's
// test matrix (see fill_omega_kernel).
__global__ void __launch_bounds__(256) tc_fill_omega_kernel(const DevLayer* __restrict__ layers, int l0, uint64_t seed,
                                                            long long row0) {
  const DevLayer& L = layers[l0 + blockIdx.y];
  const int r = L.r, NP = L.NP, groups = NP >> 3;
  const long long mp = L.m_pad;
  const long long units = (long long)L.m * groups;
  for (long long unit = blockIdx.x * 256ll + threadIdx.x; unit < units; unit += (long long)gridDim.x * 256) {
    const int g = (int)(unit / L.m);
    const long long t = unit - (long long)g * L.m;
    const int nv = min(8, r - 8 * g);                 // live k of this group (the rest is padding)
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = 0.f;
    if (nv > 0) {
      const long long e_first = (row0 + t) * r + 8 * g;
      const long long b0 = e_first >> 2;
      const int off = (int)(e_first & 3);
      const int nblk = (off + nv + 3) >> 2;
      float x[12];
      const float4 ga = gaussian_block((uint64_t)b0, L.layer_id, kTagOmega, seed);
      float4 gb = make_float4(0.f, 0.f, 0.f, 0.f), gc = gb;
      if (nblk > 1) gb = gaussian_block((uint64_t)(b0 + 1), L.layer_id, kTagOmega, seed);
      if (nblk > 2) gc = gaussian_block((uint64_t)(b0 + 2), L.layer_id, kTagOmega, seed);
      x[0] = ga.x; x[1] = ga.y; x[2] = ga.z; x[3] = ga.w;
      x[4] = gb.x; x[5] = gb.y; x[6] = gb.z; x[7] = gb.w;
      x[8] = gc.x; x[9] = gc.y; x[10] = gc.z; x[11] = gc.w;
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float y = off == 0 ? x[u] : off == 1 ? x[u + 1] : off == 2 ? x[u + 2] : x[u + 3];
        v[u] = u < nv ? y : 0.f;
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      __nv_bfloat16 h, l;
      split_bf16(v[u], &h, &l);
      L.Tb[(long long)(8 * g + u) * mp + t] = h;
      L.Tb[(long long)(NP + 8 * g + u) * mp + t] = l;
    }
  }
}

// ---------------------------------------------------------------- the bounded wait, on its own
__global__ void debug_wait_kernel(DevStatus* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0 && !mbar_wait(&bar, 0)) {     // nobody arrives: the wait runs out
    atomicExch(&status->timeout, 1);
    atomicExch(&status->where, 100);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool encode_2d(void* fn, void* out, const void* base, uint64_t inner, uint64_t outer, uint64_t pitch_bytes,
               uint32_t box_inner, uint32_t box_outer) {
  CUtensorMap m;
  const cuuint64_t dims[2] = {inner, outer};
  const cuuint64_t strides[1] = {pitch_bytes};
  const cuuint32_t box[2] = {box_inner, box_outer};
  const cuuint32_t es[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base),
                                                   dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                   // 256-byte promotion: the neighbouring 128 bytes of a row are
                                                   // what the next box of the same rows reads
                                                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  std::memcpy(out, &m, sizeof(m));
  return true;
}

int np_of(int r) { return (r + 7) & ~7; }
long long mpad_of(int m) { return ((long long)m + 7) & ~7ll; }
size_t up256(size_t x) { return (x + 255) / 256 * 256; }

int stages_for(int NB) {
  const int stage = 2 * kTileBytes + ((NB * kBoxK * 2 + 1023) & ~1023);
  int s = (int)((96 * 1024) / stage);
  if (s > 8) s = 8;
  if (s < 2) s = 2;
  return s;
}
size_t smem_for(int NB, int stages) {
  const size_t stage = 2 * kTileBytes + ((NB * kBoxK * 2 + 1023) & ~1023);
  size_t b = stage * stages + 1024;
  return b < kMinSmem ? kMinSmem : b;
}

}  // namespace

bool tc_encode_bf16_2d(const TcState& st, void* out, const void* base, uint64_t inner, uint64_t outer,
                       uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_outer) {
  if (!st.encode_fn) return false;
  return encode_2d(st.encode_fn, out, base, inner, outer, pitch_bytes, box_inner, box_outer);
}

cudaError_t tc_init(TcState* st, int device) {
  st->device = device;
  st->available = false;
  st->encode_fn = nullptr;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
  if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) {
    cudaGetLastError();
    return cudaSuccess;   // the CUDA-core path still works
  }
  int major = 0;
  cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
  st->encode_fn = fn;
  st->available = major == 10;
  if (st->available) {
    e = cudaFuncSetAttribute(tc_x_q_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(tc_xt_t_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e == cudaSuccess) e = rmw_tc_init();
    if (e == cudaSuccess) {
      int sms = 0;
      e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
      if (e == cudaSuccess) e = fused_init(sms, &st->fused);
    }
    if (e != cudaSuccess) { cudaGetLastError(); st->available = false; }
  }
  return cudaSuccess;
}

cudaError_t launch_debug_wait(DevStatus* d_status, cudaStream_t s) {
  debug_wait_kernel<<<1, 32, 0, s>>>(d_status);
  return cudaGetLastError();
}

bool tc_eligible(const agzo_layer& a) {
  return a.X && a.x_dtype == AGZO_BF16 && (reinterpret_cast<uintptr_t>(a.X) & 15u) == 0 && a.ldx % 8 == 0 &&
         a.d_in % 8 == 0 && a.d_in >= 128 && a.m >= 256 && a.r >= 1 && a.r <= AGZO_MAX_RANK;
}

int tc_operand_rows(int r) { return 2 * np_of(r); }

size_t tc_panel_bytes(const agzo_layer& a, int rows) {
  return up256((size_t)rows * (size_t)a.d_in * 2) + up256((size_t)rows * (size_t)mpad_of(a.m) * 2);
}

size_t tc_layer_scratch(const agzo_layer& a) { return tc_panel_bytes(a, tc_operand_rows(a.r)); }

void tc_set_panels(const agzo_layer& a, DevLayer* D, char* p, int rows, int row0) {
  D->NP = np_of(a.r);
  D->NB = 2 * D->NP;
  D->m_pad = mpad_of(a.m);
  __nv_bfloat16* qb = reinterpret_cast<__nv_bfloat16*>(p);
  __nv_bfloat16* tb = reinterpret_cast<__nv_bfloat16*>(p + up256((size_t)rows * (size_t)a.d_in * 2));
  D->Qb = qb + (size_t)row0 * a.d_in;
  D->Tb = tb + (size_t)row0 * D->m_pad;
  D->grp_off = row0;
}

bool tc_encode_maps(const TcState& st, const DevLayer& D, void* host_maps) {
  if (!st.encode_fn) return false;
  uint8_t* out = static_cast<uint8_t*>(host_maps);
  // X [m][ldx]: inner = d_in, outer = m; one box = 64 columns x 64 tokens
  if (!encode_2d(st.encode_fn, out, D.X, (uint64_t)D.d_in, (uint64_t)D.m, (uint64_t)D.ldx * 2, 64, 64)) return false;
  // a group leader's descriptors cover the operand rows of the whole group
  const uint32_t nb = D.grp_role == 1 ? (uint32_t)D.grp_NB : (uint32_t)D.NB;
  // Qb [nb][d_in]: box = 64 columns x nb rows
  if (!encode_2d(st.encode_fn, out + 128, D.Qb, (uint64_t)D.d_in, (uint64_t)nb, (uint64_t)D.d_in * 2, 64, nb))
    return false;
  // Tt [nb][m_pad]: inner extent is the true m so that the padding is read as zero
  if (!encode_2d(st.encode_fn, out + 256, D.Tb, (uint64_t)D.m, (uint64_t)nb, (uint64_t)D.m_pad * 2, 64, nb))
    return false;
  return true;
}

cudaError_t tc_fill_omega(const TcState&, const ExtractWave& w, const DevLayer*, uint64_t seed, cudaStream_t s) {
  const long long units = (long long)w.max_m * ((w.max_r + 7) >> 3);
  int gx = (int)((units + 255) / 256);
  if (gx > 1024) gx = 1024;
  if (gx < 1) gx = 1;
  tc_fill_omega_kernel<<<dim3(gx, w.l1 - w.l0), 256, 0, s>>>(w.d_layers, w.l0, seed, w.omega_row0);
  return cudaGetLastError();
}

cudaError_t tc_xt_t(const TcState&, const ExtractWave& w, const DevLayer* h_dev, DevStatus* d_status,
                    bool skip_fused, cudaStream_t s) {
  int max_nb = 0;
  for (int i = w.l0; i < w.l1; ++i) {
    const int nb = h_dev[i].grp_role == 1 ? h_dev[i].grp_NB : h_dev[i].NB;
    max_nb = nb > max_nb ? nb : max_nb;
  }
  const int stages = stages_for(max_nb);
  dim3 grid((w.max_din + 127) / 128, w.max_slabs, w.l1 - w.l0);
  tc_xt_t_kernel<<<grid, kTcThreads, smem_for(max_nb, stages), s>>>(w.d_layers, w.l0, d_status, stages,
                                                                    skip_fused ? 1 : 0);
  return cudaGetLastError();
}

cudaError_t tc_x_q(const TcState&, const ExtractWave& w, const DevLayer* h_dev, DevStatus* d_status,
                   bool skip_fused, cudaStream_t s) {
  int max_nb = 0;
  for (int i = w.l0; i < w.l1; ++i) {
    const int nb = h_dev[i].grp_role == 1 ? h_dev[i].grp_NB : h_dev[i].NB;
    max_nb = nb > max_nb ? nb : max_nb;
  }
  const int stages = stages_for(max_nb);
  dim3 grid((w.max_m + 127) / 128, w.l1 - w.l0);
  tc_x_q_kernel<<<grid, kTcThreads, smem_for(max_nb, stages), s>>>(w.d_layers, w.l0, d_status, stages,
                                                                   skip_fused ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace agzo
