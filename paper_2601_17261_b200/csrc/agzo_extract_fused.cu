// One power step of Algorithm 1, Y <- H (H^T Q) = X^T (X Q), with X crossing HBM once.
//
// The two products of a power step meet the same X: T = X Q needs a whole row of X (all of d_in)
// before a single element of Y = X^T T can be formed, so the unfused kernels read X twice from
// HBM.  Here a thread-block cluster of C CTAs shares a tile of 128 tokens; CTA c works on its
// slice of the tile's columns (512 or 768 of them, whichever keeps more of the device busy; C <= 16):
//   phase A   the slice's contribution to T (128 x NB, tcgen05.mma M = 128) goes to TMEM;
//             X streams through a ring of shared-memory slots (first read, from HBM, marked
//             evict-last for L2) and every slot is released as soon as its MMAs have read it,
//   exchange  the C partial sums are added up through distributed shared memory in two one-way
//             hops (st.async): groups of eight token rows are summed in rank order by the CTA that
//             owns them, which writes the bf16 hi/lo parts of the sums straight into the T operand
//             buffer of every CTA of the cluster,
//   phase C   Y_slice (slice x NB, kept in TMEM across a whole run of tiles) += X_slice^T T;
//             the slice is fetched a second time through a second ring with its own producer,
//             two to three tiles behind the first read, so it comes from L2 (measured: a line
//             survives 20 to 50 MB of streaming traffic; this lag is 33 to 50 MB over the grid,
//             and the DRAM counters show X crossing once).
// An earlier version kept the tile resident in shared memory between the phases; the exchange
// takes about 2 us, the ring held 2.5 tiles of 64 KiB, and that residency, not the arithmetic,
// bounded it at 3.6 TB/s.  The tiles of all layers of a launch form one list that is cut into equal
// contiguous shares, one per cluster; where a share ends inside a layer the partial Y leaves TMEM for
// that layer's next partial-sum buffer, and the panel QR adds a layer's partial sums in share order.
//
// As in the unfused kernels Q and T are fp32 quantities carried as hi + lo bf16 pairs in NB = 2 NP
// operand columns (NP = r rounded up to 8), products exact, accumulation fp32.
//
// Roles in a CTA: warp 0 TMA producer of ring A (and of the Q slice, once per piece of the share),
// warp 10 TMA producer of ring C, warp 1 MMA issuer (all lanes run the loop, an elected lane issues;
// it takes whichever phase has its operands, phase A up to two tiles ahead of phase C, so that the
// exchange of a tile overlaps the loads and MMAs of the next two), two groups of four epilogue warps
// that take alternate tiles (TMEM -> exchange; group 0 also writes Y out).  Every wait is bounded; a
// wait that runs out sets the status word and the CTA leaves through the common exit (cluster
// barrier, TMEM freed).
//
// The MMA warp's addresses and descriptors must stay values the compiler can prove warp-uniform (they
// travel in uniform registers); a 64-bit division in this kernel once broke that proof for everything
// after it and cost a third of the kernel's rate, which is why the share arithmetic is the host's.
#include <cuda.h>

#include <vector>

#include "agzo_ptx.cuh"
#include "agzo_tc.cuh"

namespace agzo {

namespace {

using namespace ptx;

constexpr int kFzThreads = 11 * 32;        // producer A, MMA, two epilogue groups of four warps, producer C
constexpr int kWarpProdC = 10;
constexpr int kTT = 128;                   // tokens per tile
constexpr int kGroups = kTT / 8;           // token groups of a tile (the unit of ownership in the exchange)
constexpr int kSliceCols = 512;            // columns of X per CTA ...
constexpr int kWideSliceCols = 768;        // ... and where 16 such slices do not cover d_in
constexpr int kMaxCluster = 16;
constexpr int kSlotBytes = 16 * 1024;      // ring A: [128 tokens][64 columns]; ring C: [64 tokens][128 columns]
constexpr int kBoxBytes = 8 * 1024;        // one TMA box of 64 tokens x 64 columns
constexpr int kMaxRingSlots = 8;
constexpr int kLook = 2;                   // phase A runs up to this many tiles ahead of phase C
constexpr int kBuf = kLook + 1;            // T partial (TMEM) and T operand (shared memory) buffers in rotation
constexpr int kRs = 2;                     // exchange buffers in rotation

// Shared-memory budget of an instantiation.  kWide: 768-column slices (12 boxes of Q instead of 8) or clusters
// of more than 8 CTAs.  kSmall: every layer of the launch has r <= 8, i.e. NB <= 16 operand rows: the Q slice,
// the T operands and the exchange buffers are half as large and the rings get the room (the kernel's rate
// follows the bytes its rings keep in flight).
template <bool kWide, bool kSmall>
struct FzCfg {
  static constexpr int nb_max = kSmall ? 16 : 32;
  static constexpr int q_bytes = (kWide ? 12 : 8) * nb_max * 128;
  static constexpr int tt_bytes = nb_max * 256;                 // T operand: nb_max rows of 128 tokens
  // exchange buffer: C * ceil(16 / C) * 8 * NP floats at most (NP = 16: C = 7; NP = 8: C = 15)
  static constexpr int rs_floats = kSmall ? 1920 : 2688;
  static constexpr int ring_a = kSmall ? (kWide ? 5 : 6) : (kWide ? 4 : 5);
  static constexpr int ring_c = kSmall ? 5 : 4;
  static constexpr size_t smem = (size_t)(ring_a + ring_c) * kSlotBytes + q_bytes + kBuf * tt_bytes +
                                 kRs * rs_floats * 4 + 8 * 512 + 1024;
  static_assert(ring_a <= kMaxRingSlots && ring_c <= kMaxRingSlots, "barrier arrays");
  static_assert(smem + 1024 <= 227 * 1024, "shared memory per CTA");
};

struct FzShared {
  uint64_t xa_full[kMaxRingSlots], xa_empty[kMaxRingSlots];
  uint64_t xc_full[kMaxRingSlots], xc_empty[kMaxRingSlots];
  uint64_t qb_full, qb_empty;
  uint64_t tp_full[kBuf], tp_empty[kBuf];     // T partial in TMEM
  uint64_t tt_full[kBuf];                     // T operand in shared memory: the owners' sums have landed
  uint64_t rs_full[kRs];                      // exchange: the contributions to the token groups I own have landed
  uint64_t y_full, y_free;
  uint32_t tmem_base;
  int failed;
};

// One piece of a cluster's share: tiles of a layer from token t_begin on, whose sum goes to the layer's
// partial Y number `part`.
struct FzItem {
  const DevLayer* L;
  int part, t_begin, ntiles;
};

// `total` tiles cut into G shares: the first `rem` shares have base + 1 tiles, the others base
// (base = total / G, rem = total % G, both worked out on the host: the kernel divides nothing).
__host__ __device__ inline int fz_share_begin(int k, int base, int rem) { return k * base + (k < rem ? k : rem); }
inline int fz_share_of(int off, int base, int rem) {      // the share that holds tile `off`
  const int big = rem * (base + 1);
  return off < big ? off / (base + 1) : rem + (off - big) / base;
}

// Walks the pieces of this cluster's share: the layers of [l0, l1) with cluster size C in order, their tiles
// as one list.  A layer's pieces are numbered from the first share that meets it (fz_first).
struct FzWalk {
  int l, lo, hi;      // next layer to look at; the share's tile range
  __device__ FzWalk(int l0, int cluster, int base, int rem)
      : l(l0), lo(fz_share_begin(cluster, base, rem)), hi(fz_share_begin(cluster + 1, base, rem)) {}
  __device__ bool next(const DevLayer* layers, int l1, int C, int cluster, FzItem* it) {
    for (; l < l1; ++l) {
      const DevLayer* L = layers + l;
      if (L->fz_C != C) continue;
      const int nt = (L->m + kTT - 1) / kTT;
      const int b = max(lo, L->fz_tile0), e = min(hi, L->fz_tile0 + nt);
      if (b >= e) continue;
      it->L = L;
      it->part = cluster - L->fz_first;
      it->t_begin = (b - L->fz_tile0) * kTT;
      it->ntiles = e - b;
      ++l;
      return true;
    }
    return false;
  }
};

__device__ __forceinline__ uint32_t swz(int i, int j) {
  return (uint32_t)((i >> 3) * 1024 + (i & 7) * 128 + ((j ^ (i & 7)) << 4));
}

// kWide: some layer of the launch has 768-column slices (its Q slice takes 12 boxes instead of 8, so ring A
// has one slot less, and its six Y accumulators need more than 256 TMEM columns) or the cluster has more
// than 8 CTAs; only the wide instantiations are marked for cluster sizes beyond the portable 8.
template <bool kWide, bool kSmall>
__global__ void __launch_bounds__(kFzThreads, 1)
fused_power_step_kernel(const DevLayer* __restrict__ layers, int l0, int l1, int C, int share_base, int share_rem,
                        DevStatus* status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  __shared__ FzShared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int cluster = (int)cluster_id_x();
  using Cfg = FzCfg<kWide, kSmall>;
  constexpr int ring_a = Cfg::ring_a, kRingC = Cfg::ring_c;
  constexpr int kTtBytes = Cfg::tt_bytes, kRsFloats = Cfg::rs_floats;
  constexpr uint32_t tmem_cols = kWide ? 512u : 256u;
  // shared-memory carve-up: ring A | ring C | Q slice (boxes of [NB][64]) | T operand x kBuf | exchange buffers x kRs | staging
  uint8_t* sXA = base;
  uint8_t* sXC = sXA + (size_t)ring_a * kSlotBytes;
  uint8_t* sQ = sXC + (size_t)kRingC * kSlotBytes;
  // NB is a per-layer quantity; the regions are sized for the instantiation's largest NB
  uint8_t* sTt = sQ + Cfg::q_bytes;
  float* sRs = reinterpret_cast<float*>(sTt + kBuf * kTtBytes);   // kRs x [C][cpo][8][NP] floats
  uint8_t* sStage = reinterpret_cast<uint8_t*>(sRs + kRs * kRsFloats);   // 512 bytes per epilogue warp

  if (threadIdx.x == 0) {
    for (int s = 0; s < ring_a; ++s) { mbar_init(&sh.xa_full[s], 1); mbar_init(&sh.xa_empty[s], 1); }
    for (int s = 0; s < kRingC; ++s) { mbar_init(&sh.xc_full[s], 1); mbar_init(&sh.xc_empty[s], 1); }
    mbar_init(&sh.qb_full, 1); mbar_init(&sh.qb_empty, 1);
    for (int p = 0; p < kBuf; ++p) {
      mbar_init(&sh.tp_full[p], 1); mbar_init(&sh.tp_empty[p], 4);
      mbar_init(&sh.tt_full[p], 1);
    }
    for (int p = 0; p < kRs; ++p) mbar_init(&sh.rs_full[p], 1);
    mbar_init(&sh.y_full, 1); mbar_init(&sh.y_free, 4);
    sh.failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  if (warp == 1) tmem_alloc(&sh.tmem_base, tmem_cols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // every CTA's barriers exist before anyone arrives on them remotely
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------ TMA producer, ring A: the first read of X (and the Q slice)
      const uint64_t keep = l2_policy_evict_last();
      int ns = 0, ic = 0;
      bool ok = true;
      FzItem it;
      for (FzWalk walk(l0, cluster, share_base, share_rem); ok && walk.next(layers, l1, C, cluster, &it); ++ic) {
        const DevLayer& L = *it.L;
        const uint8_t* maps = reinterpret_cast<const uint8_t*>(L.tmaps);
        const void* map_x = maps;
        const void* map_q = maps + 128;
        tmap_acquire(map_x);
        tmap_acquire(map_q);
        const int col0 = rank * L.fz_slice;
        const int live = min(L.fz_slice, L.d_in - col0);
        const int nq = (live + 63) / 64;                 // live 64-column boxes of this slice
        const int q_box = L.NB * 128;
        if (ic > 0 && !mbar_wait(&sh.qb_empty, (ic - 1) & 1)) { ok = false; break; }
        mbar_expect_tx(&sh.qb_full, (uint32_t)(nq * q_box));
        for (int j = 0; j < nq; ++j) tma_load_2d(sQ + (size_t)j * q_box, map_q, col0 + 64 * j, 0, &sh.qb_full);
        for (int tile = 0; tile < it.ntiles && ok; ++tile) {
          const int t0 = it.t_begin + tile * kTT;
          for (int j = 0; j < nq; ++j, ++ns) {
            const int s = ns % ring_a, u = ns / ring_a;
            if (u > 0 && !mbar_wait(&sh.xa_empty[s], (u - 1) & 1)) { ok = false; break; }
            uint8_t* slot = sXA + (size_t)s * kSlotBytes;
            mbar_expect_tx(&sh.xa_full[s], kSlotBytes);
            tma_load_2d_hint(slot, map_x, col0 + 64 * j, t0, &sh.xa_full[s], keep);
            tma_load_2d_hint(slot + kBoxBytes, map_x, col0 + 64 * j, t0 + 64, &sh.xa_full[s], keep);
          }
        }
      }
      if (!ok) sh.failed = 1;
      if (!ok || sh.failed) {   // leaving early: the copies in flight must land before the CTA goes away
        for (int k = ns > ring_a ? ns - ring_a : 0; k < ns; ++k) mbar_wait(&sh.xa_full[k % ring_a], (k / ring_a) & 1);
      }
    }
  } else if (warp == kWarpProdC) {
    if (lane == 0) {
      // ------------------------------------------------ TMA producer, ring C: the second read, a few boxes behind, from L2
      const uint64_t drop = l2_policy_evict_first();
      int ns = 0;
      bool ok = true;
      FzItem it;
      for (FzWalk walk(l0, cluster, share_base, share_rem); ok && walk.next(layers, l1, C, cluster, &it); ) {
        const DevLayer& L = *it.L;
        const void* map_x = L.tmaps;
        tmap_acquire(map_x);
        const int col0 = rank * L.fz_slice;
        const int live = min(L.fz_slice, L.d_in - col0);
        const int mb = (live + 127) / 128;               // live M blocks
        for (int tile = 0; tile < it.ntiles && ok; ++tile) {
          const int t0 = it.t_begin + tile * kTT;
          for (int b = 0; b < mb && ok; ++b) {
            for (int h = 0; h < 2; ++h, ++ns) {
              const int s = ns % kRingC, u = ns / kRingC;
              if (u > 0 && !mbar_wait(&sh.xc_empty[s], (u - 1) & 1)) { ok = false; break; }
              uint8_t* slot = sXC + (size_t)s * kSlotBytes;
              mbar_expect_tx(&sh.xc_full[s], kSlotBytes);
              tma_load_2d_hint(slot, map_x, col0 + 128 * b, t0 + 64 * h, &sh.xc_full[s], drop);
              tma_load_2d_hint(slot + kBoxBytes, map_x, col0 + 128 * b + 64, t0 + 64 * h, &sh.xc_full[s], drop);
            }
          }
        }
      }
      if (!ok) sh.failed = 1;
      if (!ok || sh.failed) {
        for (int k = ns > kRingC ? ns - kRingC : 0; k < ns; ++k) mbar_wait(&sh.xc_full[k % kRingC], (k / kRingC) & 1);
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
      const uint32_t sq_addr = smem_u32(sQ), sxa_addr = smem_u32(sXA), sxc_addr = smem_u32(sXC), stt_addr = smem_u32(sTt);
      for (FzWalk walk(l0, cluster, share_base, share_rem); ok && walk.next(layers, l1, C, cluster, &it); ++ic) {
        const DevLayer& L = *it.L;
        const int NB = L.NB;
        const int col0 = rank * L.fz_slice;
        const int live = min(L.fz_slice, L.d_in - col0);
        const int nq = (live + 63) / 64, mb = (live + 127) / 128;
        const uint32_t q_box = (uint32_t)NB * 128u;
        const uint32_t idesc_a = instr_desc(128, NB, 0, 0);
        const uint32_t idesc_c = instr_desc(128, NB, 1, 0);      // A = X boxes read as X^T
        const uint32_t tp_col = (uint32_t)((L.fz_slice / 128) * NB);   // T partials sit after the Y accumulators
        if (!mbar_wait_warp(&sh.qb_full, ic & 1)) { ok = false; break; }
        if (ic > 0 && !mbar_wait_warp(&sh.y_free, (ic - 1) & 1)) { ok = false; break; }
        // The two phases are issued as their operands arrive, whichever is ready: phase A of tile a_tile box by
        // box from ring A, phase C of tile c_tile half a block at a time from ring C.  Two rules order them:
        // phase C of a tile needs its T operand (tt_full), and phase A may run at most kLook tiles ahead of
        // phase C -- the T partial and T operand buffers rotate over kBuf = kLook + 1 tiles, and phase A of tile
        // i + kBuf, being issued after phase C of tile i, completes after the last read of the buffers of tile i.
        // The exchange buffers rotate over kRs = 2 tiles only: phase A of tile i + 2 waits until the sums of
        // tile i have landed here (tt_full seen), i.e. until every owner is done with its exchange buffer.
        int a_tile = 0, a_box = 0, c_tile = 0, c_unit = 0;
        bool tt_ready = false;
        uint32_t acc_a = 0u;
        int idle = 0;
        unsigned long long idle_t0 = 0;
        while (c_tile < it.ntiles) {
          bool did = false;
          if (a_tile < it.ntiles && (a_tile <= c_tile + 1 || (a_tile == c_tile + 2 && tt_ready))) {
            const int p = ta % kBuf, u2 = ta / kBuf;
            if (a_box == 0 && u2 > 0 && !mbar_wait_warp(&sh.tp_empty[p], (u2 - 1) & 1)) { ok = false; break; }
            const int s = na % ring_a, u = na / ring_a;
            if (mbar_test_warp(&sh.xa_full[s], u & 1)) {
              tc_fence_after();
              const uint32_t d_tp = tmem + tp_col + (uint32_t)(p * NB);
              const uint64_t xd = smem_desc(sxa_addr + (uint32_t)s * kSlotBytes, 0, 1024);
              const uint64_t qd = smem_desc(sq_addr + (uint32_t)a_box * q_box, 0, 1024);
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {                 // 16 columns = 32 bytes = 2 descriptor units further
                mma_bf16_if(go, d_tp, xd + (uint64_t)(2 * kk), qd + (uint64_t)(2 * kk), idesc_a, acc_a);
                acc_a = 1u;
              }
              mma_commit_if(go, &sh.xa_empty[s]);              // the slot is free once these MMAs have read it
              ++na;
              if (++a_box == nq) {
                mma_commit_if(go, &sh.tp_full[p]);
                if (a_tile == it.ntiles - 1) mma_commit_if(go, &sh.qb_empty);   // last use of this item's Q slice
                a_box = 0; acc_a = 0u; ++a_tile; ++ta;
              }
              did = true;
            }
          }
          if (c_tile < a_tile) {
            const int p = tcn % kBuf, u2 = tcn / kBuf;
            if (!tt_ready && mbar_test_cluster_warp(&sh.tt_full[p], u2 & 1)) {
              fence_proxy_async();      // the operand was written by the owners' stores, not by the async proxy
              tt_ready = true;
            }
            const int s = nc % kRingC, u = nc / kRingC;
            if (tt_ready && mbar_test_warp(&sh.xc_full[s], u & 1)) {
              tc_fence_after();
              const int b = c_unit >> 1, h = c_unit & 1;
              const uint32_t d_y = tmem + (uint32_t)(b * NB);
              // 16 tokens = two 8-row swizzle atoms = 2048 bytes = 128 descriptor units further down both boxes;
              // the T operand holds 64 tokens per 128-byte atom column, NB rows each
              const uint64_t xd = smem_desc(sxc_addr + (uint32_t)s * kSlotBytes, kBoxBytes, 1024);
              const uint64_t th = smem_desc(stt_addr + (uint32_t)p * kTtBytes + (uint32_t)(h * NB * 128), 0, 1024);
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                mma_bf16_if(go, d_y, xd + (uint64_t)(128 * kk), th + (uint64_t)(2 * kk), idesc_c,
                            (c_tile > 0 || h > 0 || kk > 0) ? 1u : 0u);
              mma_commit_if(go, &sh.xc_empty[s]);
              ++nc;
              if (++c_unit == 2 * mb) { c_unit = 0; ++c_tile; ++tcn; tt_ready = false; }
              did = true;
            }
          }
          if (did) {
            idle = 0;
          } else if (++idle >= 1024) {       // nothing was ready a thousand times over: look at the clock
            const unsigned long long now = global_ns();
            if (idle == 1024) idle_t0 = now;
            if (now - idle_t0 > kWaitCapNs) { ok = false; break; }
            idle = 1025;
          }
        }
        if (!ok) break;
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
    for (FzWalk walk(l0, cluster, share_base, share_rem); ok && walk.next(layers, l1, C, cluster, &it); ++ic) {
      const DevLayer& L = *it.L;
      const int NB = L.NB, NP = L.NP, r = L.r;
      const int col0 = rank * L.fz_slice;
      const int live = min(L.fz_slice, L.d_in - col0);
      const int mb = (live + 127) / 128;
      const uint32_t tp_col = (uint32_t)((L.fz_slice / 128) * NB);
      const int cpo = (kGroups + C - 1) / C;   // token groups of a tile per owner, at most
      for (int tile = 0; tile < it.ntiles && ok; ++tile, ++te) {
        const int p = te % kBuf, u2 = te / kBuf;     // T partial and T operand buffers
        const int pr = te % kRs, ur = te / kRs;      // exchange buffer
        if ((te & 1) != grp) continue;
        ok = mbar_wait(&sh.tp_full[p], u2 & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        // an M = 128 accumulator keeps row R in TMEM lane R: this thread holds token row 32q + lane of the tile.
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
        // No buffer needs a "free" signal.  A peer sends the contributions of tile i + 2 only after its phase A
        // of that tile has completed, which it issued after it had received the tile-i sums of every owner, mine
        // among them, and I send those after reading the tile-i contributions.  And the T operand buffer of a
        // receiver is free for tile i + kBuf once its phase A of that tile is complete (its phase C of tile i was
        // issued before it and the MMAs run in order), which is before it sends the contribution that the
        // owners' sums of tile i + kBuf wait for.
        float* rs = sRs + pr * kRsFloats;         // [C sources][cpo groups][8 tokens][NP]
        const int my_c = (kGroups - rank + C - 1) / C;      // token groups of a tile that this CTA owns
        if (et == 0) {
          mbar_expect_tx(&sh.rs_full[pr], (uint32_t)(C * my_c * 8 * NP * 4));
          mbar_expect_tx(&sh.tt_full[p], (uint32_t)(NP * kTT * 4));
        }
        {
          const int R = 32 * q + lane, j = R >> 3, dest = j % C, jc = j / C;
          const uint32_t dst = mapa_shared(smem_u32(rs + ((rank * cpo + jc) * 8 + (R & 7)) * NP), (uint32_t)dest);
          const uint32_t bar = mapa_shared(smem_u32(&sh.rs_full[pr]), (uint32_t)dest);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            if (k4 * 4 < NP)
              st_async_f4(dst + k4 * 16, make_float4(tsum[k4 * 4], tsum[k4 * 4 + 1], tsum[k4 * 4 + 2], tsum[k4 * 4 + 3]),
                          bar);
        }
        ok = mbar_wait_cluster(&sh.rs_full[pr], ur & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        // The group's four warps share the owned token groups and the destinations: with fewer than four
        // owned groups two or four warps take the same group (each adds it up again, which is cheaper than
        // handing the sums over) and send to different CTAs.  Lane = (token of the group, four rank indices)
        // adds the C contributions, the bf16 parts pass through the warp's 512-byte staging block so that a
        // lane then holds one 16-byte piece (eight tokens of one operand row), and sends it.
        {
          __nv_bfloat16* stage = reinterpret_cast<__nv_bfloat16*>(sStage) + ((grp * 4 + q) * 32 * 8);
          const uint32_t tt_base = smem_u32(sTt) + (uint32_t)p * kTtBytes;
          const uint32_t tt_bar = smem_u32(&sh.tt_full[p]);
          const int nsplit = my_c >= 4 ? 1 : (my_c >= 2 ? 2 : 4);   // warps per owned group
          for (int jc = q / nsplit; jc < my_c; jc += 4 / nsplit) {
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
            if (lane < 2 * NP) {      // operand rows: hi parts 0..NP-1, then lo parts; 64 tokens per 128-byte atom
              const uint4 piece = *reinterpret_cast<const uint4*>(stage + lane * 8);
              const uint32_t pv[4] = {piece.x, piece.y, piece.z, piece.w};
              const int j = rank + C * jc;                  // the token group inside the tile
              const uint32_t off = tt_base + (uint32_t)((j >> 3) * (2 * NP * 128)) + swz(lane, j & 7);
              for (int d = q % nsplit; d < C; d += nsplit)
                st_async_u4(mapa_shared(off, (uint32_t)d), pv, mapa_shared(tt_bar, (uint32_t)d));
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
        float* out = L.Ypart + (long long)it.part * r * L.d_in + d;
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
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem, tmem_cols); }
}

using FzKernel = void (*)(const DevLayer*, int, int, int, int, int, DevStatus*);
FzKernel fz_kernel(bool wide, bool small) {
  return wide ? (small ? fused_power_step_kernel<true, true> : fused_power_step_kernel<true, false>)
              : (small ? fused_power_step_kernel<false, true> : fused_power_step_kernel<false, false>);
}
size_t fz_smem_bytes(bool wide, bool small) {
  return wide ? (small ? FzCfg<true, true>::smem : FzCfg<true, false>::smem)
              : (small ? FzCfg<false, true>::smem : FzCfg<false, false>::smem);
}

cudaError_t fz_max_clusters(bool wide, int C, int sm_count, int* n) {
  cudaLaunchConfig_t cfg{};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(kFzThreads);
  cfg.gridDim = dim3((unsigned)(C * (sm_count / C)));
  cfg.dynamicSmemBytes = fz_smem_bytes(wide, false);     // one CTA per SM in every instantiation
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaOccupancyMaxActiveClusters(n, (const void*)fz_kernel(wide, false), &cfg);
}

}  // namespace

// The slice width of a layer: 512 or 768 columns, among those with which the cluster has at most 16 CTAs and
// the exchange buffer of the busiest owner (C sources x its token groups x 8 tokens x NP sums) fits.  A
// cluster has to fit into one GPC, so some sizes leave SMs idle, and the last slice of a layer may be
// partly empty: what counts is the share of the device's SM-time that works on columns of X,
//   (d_in / slice) x resident clusters / SMs.
// The width with the larger share wins (512 on a tie), and below 70 % the layer is left to the two sweeps
// of the unfused kernels, which are faster then; 0 when neither width qualifies.  Before fused_init has
// run (sizing a workspace without a device) the shape alone decides; with any_size the 70 % rule is
// dropped (every cluster size that the device can launch at all).
int fused_slice_cols(const FusedCaps* caps, const agzo_layer& a, bool any_size) {
  const int NP = (a.r + 7) / 8 * 8;
  int best = 0;
  double best_share = -1.0;
  for (int slice : {kSliceCols, kWideSliceCols}) {
    const int C = (a.d_in + slice - 1) / slice;
    if (C > kMaxCluster) continue;
    if (C * ((kGroups + C - 1) / C) * 8 * NP > (NP <= 8 ? FzCfg<false, true>::rs_floats : FzCfg<false, false>::rs_floats))
      continue;
    double share = 0.0;
    if (caps && caps->sm_count) {
      const int resident = caps->clusters[slice > kSliceCols || C > 8][C];
      if (resident <= 0) continue;
      share = (double)a.d_in / slice * resident / caps->sm_count;
      if (!any_size && share < 0.7) continue;
    }
    if (share > best_share) { best = slice; best_share = share; }
  }
  return best;
}

int fused_cluster_size(const FusedCaps* caps, const agzo_layer& a, bool any_size) {
  const int slice = fused_slice_cols(caps, a, any_size);
  return slice ? (a.d_in + slice - 1) / slice : 0;
}

bool fused_eligible(const FusedCaps* caps, const agzo_layer& a, bool any_size) {
  return tc_eligible(a) && a.r <= 16 && a.m >= kTT && fused_slice_cols(caps, a, any_size) != 0;
}

cudaError_t fused_init(int sm_count, FusedCaps* caps) {
  bool big = true;
  for (int wide = 0; wide < 2; ++wide)
    for (int small = 0; small < 2; ++small) {
      cudaError_t e = cudaFuncSetAttribute((const void*)fz_kernel(wide, small), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)fz_smem_bytes(wide, small));
      if (e != cudaSuccess) return e;
      // clusters of more than 8 CTAs are beyond the portable size: ask for them, and use them only if they fit
      if (wide && cudaFuncSetAttribute((const void*)fz_kernel(true, small), cudaFuncAttributeNonPortableClusterSizeAllowed,
                                       1) != cudaSuccess)
        big = false;
    }
  for (int C = 1; C <= kMaxCluster; ++C) {
    int n = 0;
    if (C > 8 || fz_max_clusters(false, C, sm_count, &n) != cudaSuccess) n = 0;
    caps->clusters[0][C] = n;
    n = 0;
    if ((C > 8 && !big) || fz_max_clusters(true, C, sm_count, &n) != cudaSuccess) n = 0;
    caps->clusters[1][C] = n;
  }
  cudaGetLastError();
  caps->sm_count = sm_count;
  return cudaSuccess;
}

int fused_resident_clusters(const FusedCaps& caps, int C) { return C >= 1 && C <= kMaxCluster ? caps.clusters[C > 8][C] : 0; }

// The partial sums of Y that a fused power step can leave for a layer, at most: one per share that meets it.
int fused_parts_bound(const agzo_layer& a, int C) {
  const int nt = (a.m + kTT - 1) / kTT;
  const int shares = 160 / C;      // no device this kernel runs on has more SMs than that
  return nt < shares ? nt : shares;
}

// The arithmetic of the work split on plain arrays (also what the host-side test export runs): layer i has
// tiles[i] tiles; with `clusters` resident clusters there are G = min(total, clusters) shares.  Writes each
// layer's first tile in the list, the first share that meets it and the number of shares that do; returns G
// and the share sizes (base, rem: the first rem shares have base + 1 tiles).
int fused_split(const int* tiles, int n, int clusters, int* tile0, int* first, int* parts, int* base, int* rem) {
  int total = 0;
  for (int i = 0; i < n; ++i) { tile0[i] = total; total += tiles[i]; }
  if (total == 0) { *base = 0; *rem = 0; return 0; }
  const int cap = clusters > 0 ? clusters : 1;
  const int G = total < cap ? total : cap;
  *base = total / G;
  *rem = total % G;
  for (int i = 0; i < n; ++i) {
    first[i] = fz_share_of(tile0[i], *base, *rem);
    parts[i] = tiles[i] > 0 ? fz_share_of(tile0[i] + tiles[i] - 1, *base, *rem) - first[i] + 1 : 0;
  }
  return G;
}
int fused_share_begin(int k, int base, int rem) { return fz_share_begin(k, base, rem); }

// Cuts the tiles of the layers of [l0, l1) with cluster size C into shares: fills fz_tile0, fz_first and fz_parts.
void fused_plan_shares(const FusedCaps& caps, DevLayer* dev, int l0, int l1, int C) {
  std::vector<int> idx, tiles;
  bool wide = C > 8;
  for (int i = l0; i < l1; ++i)
    if (dev[i].fz_C == C) {
      idx.push_back(i);
      tiles.push_back((dev[i].m + kTT - 1) / kTT);
      wide = wide || dev[i].fz_slice > kSliceCols;
    }
  if (idx.empty()) return;
  const int n = (int)idx.size();
  std::vector<int> tile0(n), first(n), parts(n);
  int base = 0, rem = 0;
  fused_split(tiles.data(), n, caps.clusters[wide][C], tile0.data(), first.data(), parts.data(), &base, &rem);
  for (int k = 0; k < n; ++k) {
    dev[idx[k]].fz_tile0 = tile0[k];
    dev[idx[k]].fz_first = first[k];
    dev[idx[k]].fz_parts = parts[k];
  }
}

// One fused power step for the layers of the wave whose cluster size is C.
cudaError_t launch_fused_power_step(const FusedCaps& caps, const ExtractWave& w, const DevLayer* h_dev, int C,
                                    DevStatus* d_status, cudaStream_t s) {
  int total = 0;
  bool wide = C > 8, small = true;
  for (int i = w.l0; i < w.l1; ++i)
    if (h_dev[i].fz_C == C) {
      total += (h_dev[i].m + kTT - 1) / kTT;
      if (h_dev[i].fz_slice > kSliceCols) wide = true;
      if (h_dev[i].NB > 16) small = false;
    }
  if (total == 0) return cudaSuccess;
  if (C < 1 || C > kMaxCluster || caps.clusters[wide][C] <= 0) return cudaErrorInvalidConfiguration;   // the planner picks no such size
  cudaLaunchConfig_t cfg{};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)C;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(kFzThreads);
  cfg.dynamicSmemBytes = fz_smem_bytes(wide, small);
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // persistent clusters, never more than can be resident at once; the same count as fused_plan_shares used
  const int nclusters = total < caps.clusters[wide][C] ? total : caps.clusters[wide][C];
  cfg.gridDim = dim3((unsigned)(nclusters * C));
  const DevLayer* layers = w.d_layers;
  int l0 = w.l0, l1 = w.l1;
  int base = total / nclusters, rem = total % nclusters;
  void* args[] = {(void*)&layers, (void*)&l0, (void*)&l1, (void*)&C, (void*)&base, (void*)&rem, (void*)&d_status};
  return cudaLaunchKernelExC(&cfg, (const void*)fz_kernel(wide, small), args);
}

}  // namespace agzo
