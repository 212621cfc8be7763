// One power step of Algorithm 1, Y <- H (H^T Q) = X^T (X Q), in a single pass over X.
//
// The two products of a power step meet the same X: T = X Q needs a whole row of X (all of d_in)
// before a single element of Y = X^T T can be formed, so the unfused kernels read X twice.  Here a
// thread-block cluster of C CTAs shares a tile of 64 tokens; CTA c keeps its 512-column slice of
// the tile in shared memory while
//   phase A   its slice's contribution to T (64 x NB, tcgen05.mma M = 64, K = 512) goes to TMEM,
//   exchange  the C partial sums are added up through distributed shared memory in two one-way
//             hops (st.async): each row of the tile is summed in rank order by the CTA that owns
//             it, and the sum is sent to every CTA, so all of them hold the same T,
//   phase C   Y_slice (512 x NB, kept in TMEM across all tiles of the work item) += X_slice^T T
//             (tcgen05.mma M = 128, the resident X boxes read as an MN-major operand).
// X therefore crosses HBM once per power step.  A work item is (layer, token slab); the slab's
// partial Y leaves TMEM once, at the end of the item, and the slabs are summed by the panel QR.
//
// As in the unfused kernels Q and T are fp32 quantities carried as hi + lo bf16 pairs in NB = 2 NP
// operand columns (NP = r rounded up to 8), products exact, accumulation fp32.
//
// Status: correct (same parity tests as the two-sweep kernels) but not faster, so it is an option
// ("extract_fused"), off by default.  Measured on B200 at d_in = 4096, r = 16, clusters of 8
// (timestamps taken inside the kernel): the exchange takes 1.35 us from the last phase-A MMA to
// the T operand being ready (it took 4.4 us with remote loads and cluster-scope release arrives),
// but a tile still takes 3.5 us, because its 32 + 16 tcgen05.mma instructions (M = 64 or 128,
// N = 32, K = 16) cost about 65 to 80 ns each whatever their size -- neither fewer instructions
// in the issuing thread nor independent accumulators changed that.  64 KiB per 3.5 us is 19 GB/s
// per CTA, 2.3 TB/s over the 120 CTAs of 15 resident clusters, against the 6.8 TB/s at which the
// two-sweep kernels read X twice (they need one such instruction per 4 KiB of X and run two CTAs
// per SM).  A fused step needs a product shape with more work per instruction (the 256-wide N
// side on X, tiles of 128 or more tokens) before it can win.
//
// Roles in a CTA: warp 0 TMA producer (Q slice once per item, X slots of [64 tokens][128 columns]
// through a ring), warp 1 MMA issuer (phase A of tile i+1 is issued before phase C of tile i so the
// exchange of one tile overlaps the loads and phase A of the next), two groups of four epilogue warps
// that take alternate tiles (TMEM -> exchange -> T operand; group 0 also writes Y out).  Every wait is bounded; a wait that runs out sets the status
// word and the CTA leaves through the common exit (copies drained, cluster barrier, TMEM freed).
#include <cuda.h>

#include "agzo_ptx.cuh"
#include "agzo_tc.cuh"

namespace agzo {

namespace {

using namespace ptx;

constexpr int kFzThreads = 64 + 2 * 128;   // producer warp, MMA warp, two epilogue groups of four warps
constexpr int kTT = 64;                    // tokens per tile
constexpr int kSliceCols = 512;            // columns of X per CTA
constexpr int kMBlocks = kSliceCols / 128; // M blocks of phase C
constexpr int kSlotBytes = 16 * 1024;      // [64 tokens][128 columns] as two boxes of 64 columns
constexpr int kBoxBytes = 8 * 1024;
constexpr int kMaxRing = 12;
constexpr int kRsFloats = 72 * 16;         // C * ceil(64 / C) <= 72 rows of up to 16 floats
constexpr uint32_t kFzTmemCols = 256;

struct FzShared {
  uint64_t x_full[kMaxRing], x_empty[kMaxRing];
  uint64_t qb_full, qb_empty;
  uint64_t tp_full[2], tp_empty[2];     // T partial in TMEM
  uint64_t tt_full[2], tt_empty[2];     // T operand in shared memory
  uint64_t rs_full[2], ag_full[2];      // exchange: contributions to my rows have landed / the summed T has landed
  uint64_t y_full, y_free;
  uint32_t tmem_base;
  int failed;
};

struct FzItem {
  const DevLayer* L;
  int slab, t_begin, ntiles;
};

// item -> (layer, slab) among the layers of [l0, l1) whose cluster size is C; false past the end
__device__ __forceinline__ bool fz_decode(const DevLayer* layers, int l0, int l1, int C, int item, FzItem* it) {
  for (int l = l0; l < l1; ++l) {
    const DevLayer* L = layers + l;
    if (L->fz_C != C) continue;
    if (item < L->slabs) {
      it->L = L;
      it->slab = item;
      it->t_begin = item * L->slab_rows;
      const int t_end = min(L->m, it->t_begin + L->slab_rows);
      it->ntiles = (t_end - it->t_begin + kTT - 1) / kTT;
      return true;
    }
    item -= L->slabs;
  }
  return false;
}

__device__ __forceinline__ uint32_t swz(int i, int j) {
  return (uint32_t)((i >> 3) * 1024 + (i & 7) * 128 + ((j ^ (i & 7)) << 4));
}

__global__ void __launch_bounds__(kFzThreads, 1)
fused_power_step_kernel(const DevLayer* __restrict__ layers, int l0, int l1, int C, int ring, DevStatus* status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ FzShared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int cluster = (int)cluster_id_x(), nclusters = (int)cluster_count_x();
  const int col0 = rank * kSliceCols;
  // shared-memory carve-up: X ring | Q slice (8 boxes of [NB][64]) | T operand x2 | exchange buffers x2
  uint8_t* sX = base;
  uint8_t* sQ = sX + (size_t)ring * kSlotBytes;
  // NB is a per-layer quantity; the regions are sized for NB = 32
  uint8_t* sTt = sQ + 8 * 32 * 128;
  float* sRs = reinterpret_cast<float*>(sTt + 2 * 32 * 128);    // 2 x [C][rows_per][NP] floats
  float* sAg = sRs + 2 * kRsFloats;                               // 2 x [64][16] floats
  const int rows_per = (kTT + C - 1) / C;                         // token rows of a tile that one CTA sums

  if (threadIdx.x == 0) {
    for (int s = 0; s < ring; ++s) { mbar_init(&sh.x_full[s], 1); mbar_init(&sh.x_empty[s], 1); }
    mbar_init(&sh.qb_full, 1); mbar_init(&sh.qb_empty, 1);
    for (int p = 0; p < 2; ++p) {
      mbar_init(&sh.tp_full[p], 1); mbar_init(&sh.tp_empty[p], 4);
      mbar_init(&sh.tt_full[p], 4); mbar_init(&sh.tt_empty[p], 1);
      mbar_init(&sh.rs_full[p], 1); mbar_init(&sh.ag_full[p], 1);
    }
    mbar_init(&sh.y_full, 1); mbar_init(&sh.y_free, 4);
    sh.failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  if (warp == 1) tmem_alloc(&sh.tmem_base, kFzTmemCols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // every CTA's barriers exist before anyone arrives on them remotely
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------ TMA producer
      int ns = 0, ic = 0;
      bool ok = true;
      FzItem it;
      for (int item = cluster; ok && fz_decode(layers, l0, l1, C, item, &it); item += nclusters, ++ic) {
        const DevLayer& L = *it.L;
        const uint8_t* maps = reinterpret_cast<const uint8_t*>(L.tmaps);
        const void* map_x = maps;
        const void* map_q = maps + 128;
        tmap_acquire(map_x);
        tmap_acquire(map_q);
        const int live = min(kSliceCols, L.d_in - col0);
        const int nq = (live + 63) / 64;                 // live 64-column boxes of this slice
        const int mb = (live + 127) / 128;               // live M blocks
        const int q_box = L.NB * 128;
        if (ic > 0 && !mbar_wait(&sh.qb_empty, (ic - 1) & 1)) { ok = false; break; }
        mbar_expect_tx(&sh.qb_full, (uint32_t)(nq * q_box));
        for (int j = 0; j < nq; ++j) tma_load_2d(sQ + (size_t)j * q_box, map_q, col0 + 64 * j, 0, &sh.qb_full);
        for (int tile = 0; tile < it.ntiles && ok; ++tile) {
          const int t0 = it.t_begin + tile * kTT;
          for (int b = 0; b < mb; ++b, ++ns) {
            const int s = ns % ring, u = ns / ring;
            if (u > 0 && !mbar_wait(&sh.x_empty[s], (u - 1) & 1)) { ok = false; break; }
            uint8_t* slot = sX + (size_t)s * kSlotBytes;
            mbar_expect_tx(&sh.x_full[s], kSlotBytes);
            tma_load_2d(slot, map_x, col0 + 128 * b, t0, &sh.x_full[s]);
            tma_load_2d(slot + kBoxBytes, map_x, col0 + 128 * b + 64, t0, &sh.x_full[s]);
          }
        }
      }
      if (!ok) sh.failed = 1;
      if (!ok || sh.failed) {   // leaving early: the copies in flight must land before the CTA goes away
        for (int k = ns > ring ? ns - ring : 0; k < ns; ++k) mbar_wait(&sh.x_full[k % ring], (k / ring) & 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------ MMA issuer
      int na = 0, nc = 0;      // slots consumed by phase A / phase C
      int ta = 0, tcn = 0;     // tiles issued in phase A / phase C
      int ic = 0;
      bool ok = true;
      FzItem it;
      for (int item = cluster; ok && fz_decode(layers, l0, l1, C, item, &it); item += nclusters, ++ic) {
        const DevLayer& L = *it.L;
        const int NB = L.NB;
        const int live = min(kSliceCols, L.d_in - col0);
        const int mb = (live + 127) / 128;
        const uint32_t q_box = (uint32_t)NB * 128u;
        const uint32_t idesc_a = instr_desc(64, NB, 0, 0);
        const uint32_t idesc_c = instr_desc(128, NB, 1, 0);      // A = resident X boxes read as X^T
        const uint32_t tp_col = (uint32_t)(kMBlocks * NB);       // T partials sit after the Y accumulators
        if (!mbar_wait(&sh.qb_full, ic & 1)) { ok = false; break; }
        if (ic > 0 && !mbar_wait(&sh.y_free, (ic - 1) & 1)) { ok = false; break; }
        for (int step = 0; step <= it.ntiles && ok; ++step) {
          if (step < it.ntiles) {
            // phase A of tile `step`
            const int p = ta & 1, u2 = ta >> 1;
            if (u2 > 0 && !mbar_wait(&sh.tp_empty[p], (u2 - 1) & 1)) { ok = false; break; }
            bool first = true;
            for (int b = 0; b < mb && ok; ++b, ++na) {
              const int s = na % ring, u = na / ring;
              if (!mbar_wait(&sh.x_full[s], u & 1)) { ok = false; break; }
              tc_fence_after();
              const uint32_t slot = smem_u32(sX + (size_t)s * kSlotBytes);
              for (int half = 0; half < 2; ++half) {
                if (128 * b + 64 * half >= live) break;          // box beyond d_in: its Q box was never loaded
                const uint32_t xa = slot + half * kBoxBytes;
                const uint32_t qb = smem_u32(sQ) + (uint32_t)(2 * b + half) * q_box;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                  mma_bf16(tmem + tp_col + (uint32_t)(p * NB), smem_desc(xa + kk * 32, 0, 1024),
                           smem_desc(qb + kk * 32, 0, 1024), idesc_a, first ? 0u : 1u);
                  first = false;
                }
              }
            }
            if (!ok) break;
            mma_commit(&sh.tp_full[p]);
            if (step == it.ntiles - 1) mma_commit(&sh.qb_empty);   // last use of this item's Q slice
            ++ta;
          }
          if (step >= 1) {
            // phase C of tile `step - 1`
            const int p = tcn & 1, u2 = tcn >> 1;
            if (!mbar_wait(&sh.tt_full[p], u2 & 1)) { ok = false; break; }
            tc_fence_after();
            const uint32_t tt = smem_u32(sTt + (size_t)p * 32 * 128);
            for (int b = 0; b < mb; ++b, ++nc) {
              const int s = nc % ring;
              const uint32_t slot = smem_u32(sX + (size_t)s * kSlotBytes);
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {
                // 16 tokens = two 8-row swizzle atoms = 2048 bytes further down both boxes
                mma_bf16(tmem + (uint32_t)(b * NB), smem_desc(slot + kk * 2048, kBoxBytes, 1024),
                         smem_desc(tt + kk * 32, 0, 1024), idesc_c, (step > 1 || kk > 0) ? 1u : 0u);
              }
              mma_commit(&sh.x_empty[s]);
            }
            mma_commit(&sh.tt_empty[p]);
            ++tcn;
          }
        }
        if (ok) mma_commit(&sh.y_full);
      }
      if (!ok) sh.failed = 1;
    }
  } else {
    // ------------------------------------------------ epilogue warps
    // Two groups of four warps take alternate tiles (group = parity of the tile counter), so the
    // latency of one tile's exchange is hidden behind the other group's tile.
    const int q = warp & 3;                 // TMEM lanes 32q .. 32q+31
    const int grp = (warp - 2) >> 2;
    const int et = threadIdx.x - 64 - 128 * grp;   // 0..127 inside the group
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    int te = 0, ic = 0;
    bool ok = true;
    FzItem it;
    for (int item = cluster; ok && fz_decode(layers, l0, l1, C, item, &it); item += nclusters, ++ic) {
      const DevLayer& L = *it.L;
      const int NB = L.NB, NP = L.NP, r = L.r;
      const int live = min(kSliceCols, L.d_in - col0);
      const int mb = (live + 127) / 128;
      const uint32_t tp_col = (uint32_t)(kMBlocks * NB);
      const int hn = NP >> 1;               // values of a T row that one thread sums: NP/2
      for (int tile = 0; tile < it.ntiles && ok; ++tile, ++te) {
        const int p = te & 1, u2 = te >> 1;
        if (p != grp) continue;
        ok = mbar_wait(&sh.tp_full[p], u2 & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        // an M = 64 accumulator keeps row 16q + i in lane 32q + i for i < 16; lanes 16..31 of a warp hold nothing
        float tsum[16];
#pragma unroll
        for (int kq = 0; kq < 2; ++kq) {
          if (kq * 8 < NP) {
            float hi[8], lo[8];
            tmem_ld8(tmem + lane_off + tp_col + (uint32_t)(p * NB + kq * 8), hi);
            tmem_ld8(tmem + lane_off + tp_col + (uint32_t)(p * NB + NP + kq * 8), lo);
#pragma unroll
            for (int j = 0; j < 8; ++j) tsum[kq * 8 + j] = hi[j] + lo[j];
          } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) tsum[kq * 8 + j] = 0.f;
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.tp_empty[p]);
        // Exchange, two one-way hops through st.async (data and its completion travel together):
        //   reduce-scatter  row R of my partial goes to the CTA that owns R (rows_per rows each);
        //   all-gather      the owner adds the C contributions in rank order and sends the sum to everyone.
        // No buffer needs a "free" signal: a peer can only send tile i+2's data after it has received
        // my tile-i sums, which I send after consuming the tile-i contributions.
        float* rs = sRs + p * kRsFloats;          // [C sources][rows_per][NP]
        float* ag = sAg + p * (kTT * 16);         // [64][NP]
        const int my_rows = max(0, min(rows_per, kTT - rank * rows_per));
        if (et == 0) {
          mbar_expect_tx(&sh.rs_full[p], (uint32_t)(C * my_rows * NP * 4));
          mbar_expect_tx(&sh.ag_full[p], (uint32_t)(kTT * NP * 4));
        }
        if (lane < 16) {
          const int R = 16 * q + lane, dest = R / rows_per, lrow = R - dest * rows_per;
          const uint32_t dst = mapa_shared(smem_u32(rs + (rank * rows_per + lrow) * NP), (uint32_t)dest);
          const uint32_t bar = mapa_shared(smem_u32(&sh.rs_full[p]), (uint32_t)dest);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            if (k4 * 4 < NP)
              st_async_f4(dst + k4 * 16, make_float4(tsum[k4 * 4], tsum[k4 * 4 + 1], tsum[k4 * 4 + 2], tsum[k4 * 4 + 3]),
                          bar);
        }
        ok = mbar_wait_cluster(&sh.rs_full[p], u2 & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        {
          const int q4 = NP >> 2;                 // float4 pieces per row
          for (int u = et; u < my_rows * q4; u += 128) {
            const int lrow = u / q4, k4 = u - lrow * q4;
            float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int c = 0; c < C; ++c) {
              const float4 v = *reinterpret_cast<const float4*>(rs + (c * rows_per + lrow) * NP + 4 * k4);
              sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
            }
            const uint32_t off = smem_u32(ag + (rank * rows_per + lrow) * NP + 4 * k4);
            const uint32_t bar = smem_u32(&sh.ag_full[p]);
            for (int c = 0; c < C; ++c) st_async_f4(mapa_shared(off, (uint32_t)c), sum, mapa_shared(bar, (uint32_t)c));
          }
        }
        ok = mbar_wait_cluster(&sh.ag_full[p], u2 & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        // thread = (token row, half of the NP values of T)
        const int row = 16 * q + (lane & 15), kh = (lane >> 4) * hn;
        float acc[8];
        {
          const float4 a = *reinterpret_cast<const float4*>(ag + row * NP + kh);
          acc[0] = a.x; acc[1] = a.y; acc[2] = a.z; acc[3] = a.w;
          float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
          if (hn == 8) b = *reinterpret_cast<const float4*>(ag + row * NP + kh + 4);
          acc[4] = b.x; acc[5] = b.y; acc[6] = b.z; acc[7] = b.w;
        }
        // T operand of phase C: rows = hi parts 0..NP-1 then lo parts, 64 tokens (128 bytes) per row
        if (u2 > 0) {
          ok = mbar_wait(&sh.tt_empty[p], (u2 - 1) & 1);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
        uint8_t* tt = sTt + (size_t)p * 32 * 128;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (j >= hn) break;
          const float v = acc[j];
          const __nv_bfloat16 h = __float2bfloat16_rn(v);
          const __nv_bfloat16 l = __float2bfloat16_rn(v - __bfloat162float(h));
          const int k = kh + j;
          *reinterpret_cast<__nv_bfloat16*>(tt + swz(k, row >> 3) + (row & 7) * 2) = h;
          *reinterpret_cast<__nv_bfloat16*>(tt + swz(NP + k, row >> 3) + (row & 7) * 2) = l;
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.tt_full[p]);
      }
      if (!ok) break;
      if (grp != 0) continue;
      // the item's partial Y: lanes = columns of the slice
      ok = mbar_wait(&sh.y_full, ic & 1);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      for (int b = 0; b < mb; ++b) {
        const int d = col0 + b * 128 + q * 32 + lane;
        float* out = L.Ypart + (long long)it.slab * r * L.d_in + d;
        for (int k0 = 0; k0 < NP; k0 += 8) {
          float hi[8], lo[8];
          tmem_ld8(tmem + lane_off + (uint32_t)(b * NB + k0), hi);
          tmem_ld8(tmem + lane_off + (uint32_t)(b * NB + NP + k0), lo);
          if (d < L.d_in) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
              if (k0 + j < r) out[(long long)(k0 + j) * L.d_in] = hi[j] + lo[j];
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.y_free);
    }
    if (!ok) sh.failed = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (sh.failed && threadIdx.x == 0) { atomicExch(&status->timeout, 1); atomicExch(&status->where, 4); }
  cluster_sync_all();          // no peer reads my exchange buffer or arrives on my barriers after this
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, kFzTmemCols); }
}

int g_max_clusters[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};   // per cluster size, filled on first use

size_t fz_smem_bytes(int ring) {
  return (size_t)ring * kSlotBytes + 8 * 32 * 128 + 2 * 32 * 128 + 2 * kRsFloats * 4 + 2 * kTT * 16 * 4 + 1024;
}
constexpr int kFzRing = 10;

}  // namespace

bool fused_eligible(const agzo_layer& a) {
  return tc_eligible(a) && a.r <= 16 && a.d_in <= 8 * kSliceCols && a.m >= kTT;
}

int fused_cluster_size(const agzo_layer& a) { return (a.d_in + kSliceCols - 1) / kSliceCols; }

cudaError_t fused_init() {
  cudaError_t e = cudaFuncSetAttribute(fused_power_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)fz_smem_bytes(kFzRing));
  return e;
}

// One fused power step for the layers of the wave whose cluster size is C.
cudaError_t launch_fused_power_step(const ExtractWave& w, const DevLayer* h_dev, int C, DevStatus* d_status,
                                    int sm_count, cudaStream_t s) {
  int items = 0;
  for (int i = w.l0; i < w.l1; ++i)
    if (h_dev[i].fz_C == C) items += h_dev[i].slabs;
  if (items == 0) return cudaSuccess;
  const size_t smem = fz_smem_bytes(kFzRing);
  cudaLaunchConfig_t cfg{};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(kFzThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (g_max_clusters[C] == 0) {
    cfg.gridDim = dim3((unsigned)(C * (sm_count / C)));
    int n = 0;
    cudaError_t e = cudaOccupancyMaxActiveClusters(&n, fused_power_step_kernel, &cfg);
    if (e != cudaSuccess) return e;
    g_max_clusters[C] = n > 0 ? n : 1;
  }
  // persistent clusters: never more than can be resident at once (they wait on one another only
  // inside a cluster, but a resident set keeps the schedule static)
  const int nclusters = items < g_max_clusters[C] ? items : g_max_clusters[C];
  cfg.gridDim = dim3((unsigned)(nclusters * C));
  const DevLayer* layers = w.d_layers;
  int l0 = w.l0, l1 = w.l1, ring = kFzRing;
  void* args[] = {(void*)&layers, (void*)&l0, (void*)&l1, (void*)&C, (void*)&ring, (void*)&d_status};
  return cudaLaunchKernelExC(&cfg, (const void*)fused_power_step_kernel, args);
}

}  // namespace agzo
