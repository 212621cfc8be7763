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
constexpr int kRsFloats = 1792;            // C * ceil(8 / C) * 8 * NP floats at most (C = 7, NP = 16)
constexpr uint32_t kFzTmemCols = 256;
constexpr int kLook = 1;                   // phase A runs this many tiles ahead of phase C
constexpr int kBuf = kLook + 1;            // T partial / exchange / T operand buffers in rotation

struct FzShared {
  uint64_t x_full[kMaxRing], x_empty[kMaxRing];
  uint64_t qb_full, qb_empty;
  uint64_t tp_full[kBuf], tp_empty[kBuf];     // T partial in TMEM
  uint64_t tt_full[kBuf];                     // T operand in shared memory: the owners' sums have landed
  uint64_t rs_full[kBuf];                     // exchange: the contributions to the rank indices I own have landed
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
fused_power_step_kernel(const DevLayer* __restrict__ layers, int l0, int l1, int C, int ring, int pf, DevStatus* status) {
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
  float* sRs = reinterpret_cast<float*>(sTt + kBuf * 32 * 128);  // kBuf x [C][cpo][8][NP] floats
  uint8_t* sStage = reinterpret_cast<uint8_t*>(sRs + kBuf * kRsFloats);   // 512 bytes per epilogue warp

  if (threadIdx.x == 0) {
    for (int s = 0; s < ring; ++s) { mbar_init(&sh.x_full[s], 1); mbar_init(&sh.x_empty[s], 1); }
    mbar_init(&sh.qb_full, 1); mbar_init(&sh.qb_empty, 1);
    for (int p = 0; p < kBuf; ++p) {
      mbar_init(&sh.tp_full[p], 1); mbar_init(&sh.tp_empty[p], 4);
      mbar_init(&sh.tt_full[p], 1);
      mbar_init(&sh.rs_full[p], 1);
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
            if (tile + pf < it.ntiles) {     // the tile `pf` steps ahead starts its way from DRAM to L2 now
              tma_prefetch_2d(map_x, col0 + 128 * b, t0 + pf * kTT);
              tma_prefetch_2d(map_x, col0 + 128 * b + 64, t0 + pf * kTT);
            }
          }
        }
      }
      if (!ok) sh.failed = 1;
      if (!ok || sh.failed) {   // leaving early: the copies in flight must land before the CTA goes away
        for (int k = ns > ring ? ns - ring : 0; k < ns; ++k) mbar_wait(&sh.x_full[k % ring], (k / ring) & 1);
      }
    }
  } else if (warp == 1) {
    {
      // ------------------------------------------------ MMA issuer
      // All 32 lanes run this loop and one elected lane issues (mma_bf16_if): the descriptors then
      // stay warp-uniform values, which is what keeps an instruction at its hardware cost.
      const uint32_t go = elect_one();
      int na = 0, nc = 0;      // slots consumed by phase A / phase C
      int ta = 0, tcn = 0;     // tiles issued in phase A / phase C
      int ic = 0;
      bool ok = true;
      FzItem it;
      const uint32_t sq_addr = smem_u32(sQ), sx_addr = smem_u32(sX), stt_addr = smem_u32(sTt);
      for (int item = cluster; ok && fz_decode(layers, l0, l1, C, item, &it); item += nclusters, ++ic) {
        const DevLayer& L = *it.L;
        const int NB = L.NB;
        const int live = min(kSliceCols, L.d_in - col0);
        const int mb = (live + 127) / 128;
        const uint32_t q_box = (uint32_t)NB * 128u;
        const uint32_t idesc_a = instr_desc(64, NB, 0, 0);
        const uint32_t idesc_c = instr_desc(128, NB, 1, 0);      // A = resident X boxes read as X^T
        const uint32_t tp_col = (uint32_t)(kMBlocks * NB);       // T partials sit after the Y accumulators
        if (!mbar_wait_warp(&sh.qb_full, ic & 1)) { ok = false; break; }
        if (ic > 0 && !mbar_wait_warp(&sh.y_free, (ic - 1) & 1)) { ok = false; break; }
        for (int step = 0; step < it.ntiles + kLook && ok; ++step) {
          if (step < it.ntiles) {
            // phase A of tile `step`
            const int p = ta % kBuf, u2 = ta / kBuf;
            if (u2 > 0 && !mbar_wait_warp(&sh.tp_empty[p], (u2 - 1) & 1)) { ok = false; break; }
            const uint32_t d_tp = tmem + tp_col + (uint32_t)(p * NB);
            uint32_t acc = 0u;
            for (int b = 0; b < mb && ok; ++b, ++na) {
              const int s = na % ring, u = na / ring;
              if (!mbar_wait_warp(&sh.x_full[s], u & 1)) { ok = false; break; }
              tc_fence_after();
              const uint32_t slot = sx_addr + (uint32_t)s * kSlotBytes;
              for (int half = 0; half < 2; ++half) {
                if (128 * b + 64 * half >= live) break;          // box beyond d_in: its Q box was never loaded
                const uint64_t xd = smem_desc(slot + half * kBoxBytes, 0, 1024);
                const uint64_t qd = smem_desc(sq_addr + (uint32_t)(2 * b + half) * q_box, 0, 1024);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {                 // 16 columns = 32 bytes = 2 descriptor units further
                  mma_bf16_if(go, d_tp, xd + (uint64_t)(2 * kk), qd + (uint64_t)(2 * kk), idesc_a, acc);
                  acc = 1u;
                }
              }
            }
            if (!ok) break;
            mma_commit_if(go, &sh.tp_full[p]);
            if (step == it.ntiles - 1) mma_commit_if(go, &sh.qb_empty);   // last use of this item's Q slice
            ++ta;
          }
          if (step >= kLook) {
            // phase C of tile `step - kLook`
            const int p = tcn % kBuf, u2 = tcn / kBuf;
            if (!mbar_wait_cluster_warp(&sh.tt_full[p], u2 & 1)) { ok = false; break; }
            fence_proxy_async();      // the operand was written by generic-proxy stores of the owners
            tc_fence_after();
            const uint64_t td = smem_desc(stt_addr + (uint32_t)p * 32u * 128u, 0, 1024);
            for (int b = 0; b < mb; ++b, ++nc) {
              const int s = nc % ring;
              // 16 tokens = two 8-row swizzle atoms = 2048 bytes = 128 descriptor units further down both boxes
              const uint64_t xd = smem_desc(sx_addr + (uint32_t)s * kSlotBytes, kBoxBytes, 1024);
              const uint32_t d_y = tmem + (uint32_t)(b * NB);
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                mma_bf16_if(go, d_y, xd + (uint64_t)(128 * kk), td + (uint64_t)(2 * kk), idesc_c,
                            (step > kLook || kk > 0) ? 1u : 0u);
              mma_commit_if(go, &sh.x_empty[s]);
            }
            ++tcn;
          }
        }
        if (ok) mma_commit_if(go, &sh.y_full);
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
      const int cpo = (kTT / 8 + C - 1) / C;   // token groups of a tile per owner, at most
      for (int tile = 0; tile < it.ntiles && ok; ++tile, ++te) {
        const int p = te % kBuf, u2 = te / kBuf;
        if ((te & 1) != grp) continue;
        ok = mbar_wait(&sh.tp_full[p], u2 & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        // an M = 64 accumulator keeps row 16q + i in lane 32q + i for i < 16; lanes 16..31 of a warp hold nothing.
        // The buffer's NB columns are [hi parts | lo parts]: one load of up to 32 columns brings both.
        float tsum[16];
        {
          uint32_t z[32];
          if (NB == 32) {
            tmem_ld32_issue(tmem + lane_off + tp_col + (uint32_t)(p * NB), z);
          } else {            // NB = 16: the upper 16 registers are not used
            tmem_ld16_issue(tmem + lane_off + tp_col + (uint32_t)(p * NB), z);
          }
          tmem_ld_wait();
#pragma unroll
          for (int k = 0; k < 16; ++k)
            tsum[k] = NB == 32 ? __uint_as_float(z[k]) + __uint_as_float(z[16 + k])
                               : (k < 8 ? __uint_as_float(z[k]) + __uint_as_float(z[8 + k]) : 0.f);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.tp_empty[p]);
        // Exchange, two one-way hops through st.async (data and its completion travel together):
        //   reduce-scatter  the tile's tokens are owned in groups of eight, group j by the CTA of rank j mod C:
        //                   every CTA sends the owner its partial sums of those rows of T;
        //   all-gather      the owner adds the C contributions in rank order, splits the sums into bf16 hi and
        //                   lo parts and writes them straight into the T operand of every CTA of the cluster:
        //                   eight tokens of one operand row are one 16-byte piece.  The bytes are counted on
        //                   the receiver's tt_full barrier, which is what its MMA warp waits for.
        // No buffer needs a "free" signal.  A peer sends tile i + kBuf's data only after its phase A of that
        // tile has completed, hence (its MMAs run in order) after its phase C of tile i, hence after it has
        // received my tile-i sums, which I sent after reading the tile-i contributions.  And the T operand
        // buffer of a receiver is free once its phase A of tile i is complete (phase C of tile i - kBuf was
        // issued before it), which is before it sends the contribution that my sum of tile i waits for.
        float* rs = sRs + p * kRsFloats;          // [C sources][cpo groups][8 tokens][NP]
        const int my_c = (kTT / 8 - rank + C - 1) / C;      // token groups of a tile that this CTA owns
        if (et == 0) {
          mbar_expect_tx(&sh.rs_full[p], (uint32_t)(C * my_c * 8 * NP * 4));
          mbar_expect_tx(&sh.tt_full[p], (uint32_t)(NP * kTT * 4));
        }
        if (lane < 16) {
          const int R = 16 * q + lane, j = R >> 3, dest = j % C, jc = j / C;
          const uint32_t dst = mapa_shared(smem_u32(rs + ((rank * cpo + jc) * 8 + (R & 7)) * NP), (uint32_t)dest);
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
        // Every warp of the group adds the C contributions of an owned token group (lane = (token of the
        // group, four rank indices); the four warps do the same additions, which is cheaper than handing
        // the sums over), passes the bf16 parts through its 512-byte staging block so that a lane then
        // holds one 16-byte piece (eight tokens of one operand row), and sends it to the CTAs d = q mod 4.
        {
          __nv_bfloat16* stage = reinterpret_cast<__nv_bfloat16*>(sStage) + ((grp * 4 + q) * 32 * 8);
          const uint32_t tt_base = smem_u32(sTt) + (uint32_t)p * 32u * 128u;
          const uint32_t tt_bar = smem_u32(&sh.tt_full[p]);
          for (int jc = 0; jc < my_c; ++jc) {
            const int x = lane & 7, kq = lane >> 3;
            if (4 * kq < NP) {
              float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
              for (int c = 0; c < C; ++c) {
                const float4 v = *reinterpret_cast<const float4*>(rs + ((c * cpo + jc) * 8 + x) * NP + 4 * kq);
                sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
              }
              const float sv[4] = {sum.x, sum.y, sum.z, sum.w};
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                const __nv_bfloat16 h = __float2bfloat16_rn(sv[c]);
                stage[(4 * kq + c) * 8 + x] = h;
                stage[(NP + 4 * kq + c) * 8 + x] = __float2bfloat16_rn(sv[c] - __bfloat162float(h));
              }
            }
            __syncwarp();
            if (lane < 2 * NP) {      // operand rows: hi parts 0..NP-1, then lo parts
              const uint4 piece = *reinterpret_cast<const uint4*>(stage + lane * 8);
              const uint32_t pv[4] = {piece.x, piece.y, piece.z, piece.w};
              const uint32_t off = tt_base + swz(lane, rank + C * jc);
              for (int d = q; d < C; d += 4) st_async_u4(mapa_shared(off, (uint32_t)d), pv, mapa_shared(tt_bar, (uint32_t)d));
            }
            __syncwarp();
          }
        }
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
  return (size_t)ring * kSlotBytes + 8 * 32 * 128 + kBuf * 32 * 128 + kBuf * kRsFloats * 4 + 8 * 512 + 1024;
}
constexpr int kFzRing = 10;    // as many slots as fit beside the other regions in 227 KiB

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
  int pf = 2;      // tiles ahead of the loads at which L2 is asked to fetch (no measurable effect between 0 and 4)
  void* args[] = {(void*)&layers, (void*)&l0, (void*)&l1, (void*)&C, (void*)&ring, (void*)&pf, (void*)&d_status};
  return cudaLaunchKernelExC(&cfg, (const void*)fused_power_step_kernel, args);
}

}  // namespace agzo
