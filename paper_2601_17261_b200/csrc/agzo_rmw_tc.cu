// In-place low-rank pass W <- W + c * R A^T (Eq. agzo-perturb, Algorithm 2) for bf16 weights
// with the rank-r outer product on the tensor cores of sm_100a.
//
// The CUDA-core kernel (agzo_rmw.cu) spends r + 1 fp32 FMAs per weight; from r = 16 on that is
// more arithmetic than the FP32 pipes can do in the time HBM needs to stream the weight once in
// and once out, and measured it falls behind this kernel from r = 3 on.  Here the product Delta = R A^T of a 128-row tile is one small tcgen05.mma chain
// (M = 128, N = the panel's columns, K = 4 * rp), its fp32 result waits in TMEM, and the only
// per-weight work left for the CUDA cores is  w + c * delta  and the rounding to bf16.
//
// Precision: R and A^T are fp32; each is split as hi + lo in bf16.  The operands hold each part
// once (A operand = [Rh | Rl], B operand = [Ah | Al], rp columns each) and the chain runs over
// the four cross products Rh Ah, Rh Al, Rl Ah, Rl Al by pointing the instruction descriptors at
// the parts, so the products are exact and summed in fp32; what is dropped is below 2^-17 of
// each term.
//
// Work item = (layer, chunk of 8 or 32 row tiles, group of up to two adjacent column panels).
// The R operand of a row tile serves every panel of the group, so R is regenerated once per
// 128 x (2 * panel width) weights and the CTA streams up to 1 KiB of every weight row.  For
// ranks above 16 the R operands are not regenerated at all: a fill kernel writes every tile's
// operand image to scratch once per seed and the CTA copies it in (staged R).
//
// Data flow of one CTA (persistent, one per SM):
//   loader thread      TMA-loads 128 x 64 boxes of W into a ring of shared-memory slots
//   R warps (4 or 8)   regenerate the tile's 128 rows of R from the Philox counter and write the
//                      split A operand; at the start of an item they also build the B operand
//                      from the panel's slice of A^T (V)
//   MMA thread         issues the tcgen05.mma chain into one of two TMEM buffers
//   epilogue warps (8) read delta from TMEM and W from the slot, write the new bf16 W back
//                      into the slot
//   storer thread      TMA-stores the slot to the place it was loaded from
// Every wait on an mbarrier is bounded; a wait that runs out sets the status word and the CTA
// leaves through the common exit (copies drained, TMEM freed).
#include <cuda.h>

#include "agzo_ptx.cuh"
#include "agzo_tc.cuh"

namespace agzo {

namespace {

using namespace ptx;

constexpr int kRows = 128;                 // rows of a tile (MMA M)
constexpr int kBoxCols = 64;               // columns of one W box = one 128-byte swizzle row
constexpr int kBoxBytes = kRows * 128;     // 16 KiB
constexpr int kAtomBytesA = kRows * 128;   // one 64-wide K atom of the A operand
constexpr int kBBytes = 32 * 1024;         // B operand of one panel: panel columns x K, always 32 KiB
constexpr int kMaxPanels = 2;              // panels per work item
constexpr int kMaxSlots = 12;
constexpr int kWarpLoader = 0, kWarpMma = 1, kWarpStorer = 2, kWarpEpi0 = 3, kNumEpiWarps = 8,
              kWarpGen0 = kWarpEpi0 + kNumEpiWarps, kMaxGenWarps = 8;
constexpr int kMaxThreads = (kWarpGen0 + kMaxGenWarps) * 32;   // 608
constexpr uint32_t kTmemCols = 512;        // two delta buffers of up to 256 columns

// rp = the rank rounded up to a multiple of 16 (one instruction takes K = 16); an operand row is
// 2 * rp bf16 values, stored as K atoms of 64
__host__ __device__ inline int rtc_rank_padded(int r) { return (r + 15) & ~15; }
__host__ __device__ inline int rtc_katoms(int rp) { return (2 * rp + 63) / 64; }

struct Shared {
  uint64_t full_w[kMaxSlots];    // TMA load of the slot landed
  uint64_t epi_done[kMaxSlots];  // epilogue warps wrote the slot back
  uint64_t empty_w[kMaxSlots];   // TMA store has read the slot
  uint64_t a_full[2], a_empty[2];
  uint64_t b_full, b_empty;
  uint64_t tmem_full[2], tmem_empty[2];
  uint32_t tmem_base;
  int failed;
};

struct Item {
  const DevLayer* L;
  int col0, rb0, rb1, cw, rp, np;   // np = live panels of the group (1 or 2)
  __device__ __forceinline__ int panel_col(int p) const { return col0 + p * cw; }
  __device__ __forceinline__ int nboxes(int p) const {   // boxes of panel p that hold columns of W
    const int left = L_d_in - panel_col(p);
    return min(cw / kBoxCols, (left + kBoxCols - 1) / kBoxCols);
  }
  int L_d_in;
};

__device__ __forceinline__ int find_layer_of_item(const int* start, int n_layers, int item) {
  int lo = 0, hi = n_layers - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (__ldg(start + mid) <= item) lo = mid; else hi = mid - 1;
  }
  return lo;
}

__device__ __forceinline__ Item decode_item(const DevLayer* layers, const int* item_start, int n_layers, int item) {
  Item it;
  const DevLayer* L = layers + find_layer_of_item(item_start, n_layers, item);
  it.L = L;
  it.L_d_in = L->d_in;
  const int local = item - L->rtc_item0;
  const int chunk = local / L->rtc_panels, group = local - chunk * L->rtc_panels;
  it.cw = L->rtc_cw;
  it.rp = L->rtc_rp;
  it.col0 = group * L->rtc_np * it.cw;
  const int nrb = (L->d_out + kRows - 1) / kRows;
  it.rb0 = chunk * L->rtc_chunk_blocks;
  it.rb1 = min(nrb, it.rb0 + L->rtc_chunk_blocks);
  it.np = min(L->rtc_np, (L->d_in - it.col0 + it.cw - 1) / it.cw);
  return it;
}

// byte offset of 16-byte chunk j of row i inside a [rows][128 bytes] block with the 128-byte swizzle
__device__ __forceinline__ uint32_t swz(int i, int j) {
  return (uint32_t)((i >> 3) * 1024 + (i & 7) * 128 + ((j ^ (i & 7)) << 4));
}

__device__ __forceinline__ uint32_t pack2(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);   // a in the low half
  return *reinterpret_cast<uint32_t*>(&p);
}
__device__ __forceinline__ float lo_part(float v) { return v - __bfloat162float(__float2bfloat16_rn(v)); }

// Eight fp32 values -> their bf16 hi parts and bf16 lo parts (v ~ hi + lo)
__device__ __forceinline__ void split8(const float (&v)[8], uint4* hi, uint4* lo) {
  hi->x = pack2(v[0], v[1]); hi->y = pack2(v[2], v[3]); hi->z = pack2(v[4], v[5]); hi->w = pack2(v[6], v[7]);
  lo->x = pack2(lo_part(v[0]), lo_part(v[1])); lo->y = pack2(lo_part(v[2]), lo_part(v[3]));
  lo->z = pack2(lo_part(v[4]), lo_part(v[5])); lo->w = pack2(lo_part(v[6]), lo_part(v[7]));
}

// Writes group g (8 consecutive rank indices) of one operand row: the hi parts at K index 8g,
// the lo parts at rp + 8g (g8 = rp / 8 groups per part).
__device__ __forceinline__ void put_group(uint8_t* base, int atom_bytes, int row, int g, int g8, uint4 hi, uint4 lo) {
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const int cg = q * g8 + g;                     // 16-byte chunk index along K
    uint8_t* p = base + (cg >> 3) * atom_bytes + swz(row, cg & 7);
    *reinterpret_cast<uint4*>(p) = q == 0 ? hi : lo;
  }
}

// Rank indices 8g .. 8g+7 of row `row` of R (d_out x r, i.i.d. N(0,1) from the Philox stream
// (seed, layer_id, tag 0), element e = row * r + k), as bf16 hi parts and bf16 lo parts; zero
// beyond the matrix.
__device__ __forceinline__ void gen_r_group(const DevLayer& L, long long row, int g, uint64_t seed, uint4* hi_out,
                                            uint4* lo_out) {
  const int r = L.r;
  const int nv = row < L.d_out ? min(8, r - 8 * g) : 0;   // live rank indices of this group
  float v[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) v[u] = 0.f;
  if (nv > 0) {
    // elements e_first .. e_first + nv - 1 of the stream: at most three Philox blocks
    const long long e_first = row * r + 8 * g;
    const long long b0 = e_first >> 2;
    const int off = (int)(e_first & 3);
    const int nblk = (off + nv + 3) >> 2;
    float x[12];
    const float4 ga = gaussian_block((uint64_t)b0, L.layer_id, kTagG, seed);
    x[0] = ga.x; x[1] = ga.y; x[2] = ga.z; x[3] = ga.w;
    float4 gb = make_float4(0.f, 0.f, 0.f, 0.f), gc = gb;
    if (nblk > 1) gb = gaussian_block((uint64_t)(b0 + 1), L.layer_id, kTagG, seed);
    if (nblk > 2) gc = gaussian_block((uint64_t)(b0 + 2), L.layer_id, kTagG, seed);
    x[4] = gb.x; x[5] = gb.y; x[6] = gb.z; x[7] = gb.w;
    x[8] = gc.x; x[9] = gc.y; x[10] = gc.z; x[11] = gc.w;
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const float y = off == 0 ? x[u] : off == 1 ? x[u + 1] : off == 2 ? x[u + 2] : x[u + 3];
      v[u] = u < nv ? y : 0.f;
    }
  }
  split8(v, hi_out, lo_out);
}

__global__ void __launch_bounds__(kMaxThreads, 1)
rmw_tc_kernel(const DevLayer* __restrict__ layers, const int* __restrict__ item_start, int n_layers,
              int total_items, int a_bufs, int a_buf_bytes, int b_area_bytes, int slots, int inflight, int staged,
              uint64_t seed,
              float coef_imm,
              const float* __restrict__ d_coef, DevStatus* status) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = base;                                   // a_bufs x a_buf_bytes
  uint8_t* sB = sA + (size_t)a_bufs * a_buf_bytes;      // two panels of kBBytes, or one larger panel
  uint8_t* sW = sB + b_area_bytes;                      // slots x kBoxBytes
  __shared__ Shared sh;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gen_warps = (int)(blockDim.x >> 5) - kWarpGen0;   // 4 for small ranks, 8 otherwise
  const int gen_threads = gen_warps * 32;

  if (threadIdx.x == 0) {
    for (int s = 0; s < slots; ++s) {
      mbar_init(&sh.full_w[s], 1);
      mbar_init(&sh.epi_done[s], kNumEpiWarps);
      mbar_init(&sh.empty_w[s], 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sh.a_full[b], staged ? 1 : gen_warps);   // staged R: one arrive that sets the byte count
      mbar_init(&sh.a_empty[b], 1);
      mbar_init(&sh.tmem_full[b], 1);
      mbar_init(&sh.tmem_empty[b], kNumEpiWarps);
    }
    mbar_init(&sh.b_full, gen_warps);
    mbar_init(&sh.b_empty, 1);
    sh.failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  if (warp == kWarpMma) tmem_alloc(&sh.tmem_base, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh.tmem_base;

  if (warp == kWarpLoader) {
    if (lane == 0) {
      int n = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
        const Item it = decode_item(layers, item_start, n_layers, item);
        const void* map = it.L->wmap;
        tmap_acquire(map);
        for (int rb = it.rb0; rb < it.rb1 && ok; ++rb) {
          for (int p = 0; p < it.np && ok; ++p) {
            const int nb = it.nboxes(p), pc = it.panel_col(p);
            for (int j = 0; j < nb; ++j, ++n) {
              const int s = n % slots, u = n / slots;
              if (u > 0 && !mbar_wait(&sh.empty_w[s], (u - 1) & 1)) { ok = false; break; }
              if (n >= inflight) {              // at most `inflight` loads outstanding: box n - inflight has landed
                const int k = n - inflight;
                if (!mbar_wait(&sh.full_w[k % slots], (k / slots) & 1)) { ok = false; break; }
              }
              mbar_expect_tx(&sh.full_w[s], kBoxBytes);
              tma_load_2d(sW + (size_t)s * kBoxBytes, map, pc + j * kBoxCols, rb * kRows, &sh.full_w[s]);
            }
          }
        }
      }
      if (!ok) sh.failed = 1;
      if (!ok || sh.failed) {   // leaving early: the copies in flight must land before the CTA goes away
        for (int k = n > slots ? n - slots : 0; k < n; ++k) mbar_wait(&sh.full_w[k % slots], (k / slots) & 1);
      }
    }
  } else if (warp == kWarpStorer) {
    if (lane == 0) {
      int n = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
        const Item it = decode_item(layers, item_start, n_layers, item);
        const void* map = it.L->wmap;
        tmap_acquire(map);
        for (int rb = it.rb0; rb < it.rb1 && ok; ++rb) {
          for (int p = 0; p < it.np && ok; ++p) {
            const int nb = it.nboxes(p), pc = it.panel_col(p);
            for (int j = 0; j < nb; ++j, ++n) {
              const int s = n % slots, u = n / slots;
              if (!mbar_wait(&sh.epi_done[s], u & 1)) { ok = false; break; }
              tma_store_2d(map, pc + j * kBoxCols, rb * kRows, sW + (size_t)s * kBoxBytes);
              tma_commit_group();
              if (n > 0) {                      // the previous box's store has read its slot
                tma_wait_group_read<1>();
                mbar_arrive(&sh.empty_w[(n - 1) % slots]);
              }
            }
          }
        }
      }
      tma_wait_group<0>();                    // every store of this CTA is complete
      if (!ok) sh.failed = 1;
    }
  } else if (warp == kWarpMma) {
    if (lane == 0) {
      int t = 0, ta = 0, ic = 0;      // t counts (row tile, panel) pairs, ta row tiles, ic items
      bool ok = true;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++ic) {
        const Item it = decode_item(layers, item_start, n_layers, item);
        if (!mbar_wait(&sh.b_full, ic & 1)) { ok = false; break; }
        const uint32_t idesc = instr_desc(kRows, it.cw, 0, 0);
        const int kpt = it.rp >> 4;                      // instructions (K = 16) per cross product
        const uint32_t b_atom = (uint32_t)it.cw * 128u;
        for (int rb = it.rb0; rb < it.rb1 && ok; ++rb, ++ta) {
          const int ab = ta % a_bufs, au = ta / a_bufs;
          if (!mbar_wait(&sh.a_full[ab], au & 1)) { ok = false; break; }
          const uint32_t a0 = smem_u32(sA + (size_t)ab * a_buf_bytes);
          for (int p = 0; p < it.np; ++p, ++t) {
            const int tb = t & 1, tu = t >> 1;
            if (tu > 0 && !mbar_wait(&sh.tmem_empty[tb], (tu - 1) & 1)) { ok = false; break; }
            tc_fence_after();
            const uint32_t b0 = smem_u32(sB + (size_t)p * kBBytes);
            for (int term = 0; term < 4; ++term) {       // Rh Ah, Rh Al, Rl Ah, Rl Al
              const int ka0 = (term & 2) ? it.rp : 0, kb0 = (term & 1) ? it.rp : 0;   // first K index of the part
              for (int j = 0; j < kpt; ++j) {
                const int ka = ka0 + 16 * j, kb = kb0 + 16 * j;
                const uint64_t ad = smem_desc(a0 + (ka >> 6) * kAtomBytesA + (ka & 63) * 2, 0, 1024);
                const uint64_t bd = smem_desc(b0 + (kb >> 6) * b_atom + (kb & 63) * 2, 0, 1024);
                mma_bf16(tmem + (uint32_t)tb * 256u, ad, bd, idesc, (term | j) ? 1u : 0u);
              }
            }
            mma_commit(&sh.tmem_full[tb]);
          }
          mma_commit(&sh.a_empty[ab]);      // the row tile's R operand has served all its panels
        }
        mma_commit(&sh.b_empty);
      }
      if (!ok) sh.failed = 1;
    }
  } else if (warp >= kWarpGen0) {
    // ------------------------------------------------ operand builders
    // A unit of work is (operand row, group of 8 rank indices): consecutive threads take
    // consecutive rows, so every thread has one or two short independent chains to run.
    const int gt = threadIdx.x - kWarpGen0 * 32;
    int t = 0, ic = 0;
    int last_ab = -1, last_par = 0;      // the bulk copy this thread issued last (staged R)
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x, ++ic) {
      const Item it = decode_item(layers, item_start, n_layers, item);
      const DevLayer& L = *it.L;
      const int r = L.r, g8 = it.rp >> 3;
      // B operand: row n = column col0 + n of the panel, K = [Ah | Al]
      if (ic > 0) {
        ok = mbar_wait(&sh.b_empty, (ic - 1) & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
      }
      const int b_atom = it.cw * 128;
      const int ncols = it.np * it.cw;                   // columns of the whole group
      for (int unit = gt; unit < ncols * g8; unit += gen_threads) {
        const int g = unit / ncols, nn = unit - g * ncols;
        const int p = nn / it.cw, n = nn - p * it.cw;
        const int col = it.col0 + nn;
        float v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int k = 8 * g + u;
          v[u] = (k < r && col < L.d_in) ? __ldg(L.V + (long long)k * L.ldv + col) : 0.f;
        }
        uint4 hi, lo;
        split8(v, &hi, &lo);
        put_group(sB + (size_t)p * kBBytes, b_atom, n, g, g8, hi, lo);
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh.b_full);
      // A operand per tile: row i = R[rb*128 + i][:], K = [Rh | Rl]
      // Staged R needs one thread per tile.  Only its warp walks the tiles: a warp that waited on
      // a_empty without feeding a_full could fall two phases behind and take a later phase for its own.
      if (staged && warp != kWarpGen0) continue;
      for (int rb = it.rb0; rb < it.rb1; ++rb, ++t) {
        const int ab = t % a_bufs, au = t / a_bufs;
        if (au > 0) {
          ok = mbar_wait(&sh.a_empty[ab], (au - 1) & 1);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
        uint8_t* a_base = sA + (size_t)ab * a_buf_bytes;
        if (staged) {          // the tile's operand image was written by the fill kernel: one bulk copy
          if (gt == 0) {
            mbar_expect_tx(&sh.a_full[ab], (uint32_t)L.rimg_tile_bytes);
            bulk_load(a_base, L.rimg + (size_t)rb * L.rimg_tile_bytes, (uint32_t)L.rimg_tile_bytes, &sh.a_full[ab]);
            last_ab = ab; last_par = au & 1;
          }
          continue;
        }
        for (int unit = gt; unit < kRows * g8; unit += gen_threads) {
          const int g = unit >> 7, i = unit & (kRows - 1);
          uint4 hi, lo;
          gen_r_group(L, (long long)rb * kRows + i, g, seed, &hi, &lo);
          put_group(a_base, kAtomBytesA, i, g, g8, hi, lo);
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.a_full[ab]);
      }
    }
    if (!ok) sh.failed = 1;
    // leaving early with a bulk copy in flight: it must land before the CTA goes away
    if (staged && gt == 0 && last_ab >= 0 && (!ok || sh.failed)) mbar_wait(&sh.a_full[last_ab], (uint32_t)last_par);
  } else {
    // ------------------------------------------------ epilogue: thread = row of the tile, 32 columns of each box
    const int e = warp - kWarpEpi0;
    const int q = warp & 3;            // TMEM lanes 32q .. 32q+31 belong to this warp
    const int h = e >> 2;              // which half of a box's 64 columns
    const int i = q * 32 + lane;       // row inside the tile
    const float coef = d_coef ? __ldg(d_coef) : coef_imm;
    uint32_t off[4];                   // this thread's four 16-byte chunks inside any box
#pragma unroll
    for (int c = 0; c < 4; ++c) off[c] = swz(i, h * 4 + c);
    const uint32_t tmem_row = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(h * 32);
    int t = 0, s = 0, u = 0;           // tile counter; ring slot and how often the ring has wrapped
    bool ok = true;
    for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
      const Item it = decode_item(layers, item_start, n_layers, item);
      for (int rbp = it.rb0 * it.np; rbp < it.rb1 * it.np && ok; ++rbp, ++t) {   // (row tile, panel) pairs
        const int tb = t & 1, tu = t >> 1;
        ok = mbar_wait(&sh.tmem_full[tb], tu & 1);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
        const int nb = it.nboxes(rbp % it.np);
        for (int j = 0; j < nb; ++j) {
          ok = mbar_wait(&sh.full_w[s], u & 1);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
          uint32_t z[32];
          tmem_ld32_issue(tmem_row + (uint32_t)(tb * 256 + j * kBoxCols), z);
          uint8_t* slot = sW + (size_t)s * kBoxBytes;
          uint4 w[4];
#pragma unroll
          for (int c = 0; c < 4; ++c) w[c] = *reinterpret_cast<const uint4*>(slot + off[c]);
          tmem_ld_wait();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const uint32_t wi[4] = {w[c].x, w[c].y, w[c].z, w[c].w};
            uint32_t o[4];
#pragma unroll
            for (int p = 0; p < 4; ++p) {
              const float w0 = __uint_as_float(wi[p] << 16), w1 = __uint_as_float(wi[p] & 0xFFFF0000u);
              const float o0 = fmaf(coef, __uint_as_float(z[8 * c + 2 * p]), w0);
              const float o1 = fmaf(coef, __uint_as_float(z[8 * c + 2 * p + 1]), w1);
              o[p] = pack2(o0, o1);
            }
            *reinterpret_cast<uint4*>(slot + off[c]) = make_uint4(o[0], o[1], o[2], o[3]);
          }
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh.epi_done[s]);
          if (++s == slots) { s = 0; u ^= 1; }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0 && ok) mbar_arrive(&sh.tmem_empty[tb]);
      }
    }
    if (!ok) sh.failed = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (sh.failed && threadIdx.x == 0) { atomicExch(&status->timeout, 1); atomicExch(&status->where, 3); }
  if (warp == kWarpMma) { tc_fence_after(); tmem_dealloc(tmem, kTmemCols); }
}

// Staged R: CTA = (row tile, layer); writes the tile's split A operand [Rh | Rl] to
// scratch exactly as rmw_tc_kernel lays it out in shared memory (K atoms of [128 rows][128 bytes],
// 128-byte swizzle), so the pass can bulk-copy it.
__global__ void __launch_bounds__(256) rmw_tc_fill_r_kernel(const DevLayer* __restrict__ layers, uint64_t seed) {
  const DevLayer& L = layers[blockIdx.y];
  if (!L.rimg) return;
  const int rb = blockIdx.x;
  if (rb * kRows >= L.d_out) return;
  const int g8 = L.rtc_rp >> 3;
  uint8_t* img = L.rimg + (size_t)rb * L.rimg_tile_bytes;
  for (int unit = threadIdx.x; unit < kRows * g8; unit += 256) {
    const int g = unit >> 7, i = unit & (kRows - 1);
    uint4 hi, lo;
    gen_r_group(L, (long long)rb * kRows + i, g, seed, &hi, &lo);
    put_group(img, kAtomBytesA, i, g, g8, hi, lo);
  }
}

}  // namespace

// ---------------------------------------------------------------- host side
bool rmw_tc_eligible(const agzo_layer& a) {
  return a.W && !a.W16 && a.w_dtype == AGZO_BF16 && (reinterpret_cast<uintptr_t>(a.W) & 15u) == 0 &&
         (a.ldw * 2) % 16 == 0 && a.d_out >= 1 && a.d_in >= 1 && a.r >= 1 && a.r <= AGZO_MAX_RANK;
}

void rmw_tc_shape(const agzo_layer& a, int panels, bool staged, DevLayer* D) {
  const int rp = rtc_rank_padded(a.r);
  const int katoms = rtc_katoms(rp);                     // 1 (rp <= 32) or 2 K atoms of 64
  // panels == 0: one panel per item while R is cheap to regenerate (rp = 16: the pass is
  // HBM-bound either way and the smaller items balance better), two from there on, where
  // regenerating R is what limits the pass.  With R staged in scratch there is nothing to
  // amortise over a second panel.
  int np = panels == 1 ? 1 : panels == 2 ? kMaxPanels : (rp <= 16 ? 1 : kMaxPanels);
  if (staged && rp > 16) np = 1;
  // Panel width: K atoms x columns x 128 bytes of B operand; a panel of a pair has 32 KiB, a
  // single panel may take 64 KiB
  const int cw = (katoms == 1 || np == 1) ? 256 : 128;
  D->rtc_rp = rp;
  D->rtc_cw = cw;
  D->rtc_np = np;
  D->rtc_panels = (a.d_in + np * cw - 1) / (np * cw);   // panel groups
  // row tiles per item: the B operand is rebuilt once per item, which stalls the MMA pipeline for a
  // few microseconds when the rank is large, so those items are taller
  D->rtc_chunk_blocks = rp >= 32 ? 32 : 8;
  const int nrb = (a.d_out + kRows - 1) / kRows;
  D->rtc_chunks = (nrb + D->rtc_chunk_blocks - 1) / D->rtc_chunk_blocks;
}

bool rmw_tc_encode_map(const TcState& st, const DevLayer& D, void* host_map) {
  // W [d_out][ldw] bf16: inner = d_in, outer = d_out; one box = 64 columns x 128 rows
  return tc_encode_bf16_2d(st, host_map, D.W, (uint64_t)D.d_in, (uint64_t)D.d_out, (uint64_t)D.ldw * 2, kBoxCols,
                           kRows);
}

cudaError_t rmw_tc_init() {
  return cudaFuncSetAttribute(rmw_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);
}

int rmw_tc_b_bytes(const DevLayer& D) {
  return D.rtc_np > 1 ? kMaxPanels * kBBytes : D.rtc_cw * rtc_katoms(D.rtc_rp) * 128;
}

size_t rmw_tc_image_bytes(const agzo_layer& a) {
  const int rp = rtc_rank_padded(a.r);
  const size_t katoms = (size_t)rtc_katoms(rp);
  return (size_t)((a.d_out + kRows - 1) / kRows) * katoms * kAtomBytesA;
}

cudaError_t launch_rmw_tc(const DevLayer* d_layers, const int* d_item_start, int n_layers, int total_items,
                          int max_rp, int max_r, int max_b_bytes, int max_row_tiles, bool staged, bool fill,
                          int slots_wanted, int inflight,
                          uint64_t seed,
                          float coef, const float* d_coef, DevStatus* d_status, int sm_count, cudaStream_t s) {
  if (total_items <= 0) return cudaSuccess;
  if (staged && fill) {
    rmw_tc_fill_r_kernel<<<dim3((unsigned)max_row_tiles, (unsigned)n_layers), 256, 0, s>>>(d_layers, seed);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  const int katoms = rtc_katoms(max_rp);
  const int a_buf_bytes = katoms * kAtomBytesA;
  const int a_bufs = 2;                       // one being refilled while the other feeds the chain
  const int fixed = a_bufs * a_buf_bytes + max_b_bytes;
  int slots = (224 * 1024 - fixed) / kBoxBytes;
  if (slots > kMaxSlots) slots = kMaxSlots;
  if (slots_wanted >= 2 && slots_wanted < slots) slots = slots_wanted;
  const size_t smem = (size_t)fixed + (size_t)slots * kBoxBytes + 1024;
  const int grid = total_items < sm_count ? total_items : sm_count;
  // operand-builder warps: four keep up with the stream for r <= 8, larger ranks get eight
  const int threads = (kWarpGen0 + (max_r <= 8 ? 4 : kMaxGenWarps)) * 32;
  // loads in flight per CTA: enough to cover the HBM latency at this SM's share of the
  // bandwidth (4 to 5 boxes of 16 KiB); more only lengthens the queues in front of the stores
  if (inflight < 1) inflight = max_r <= 8 ? 4 : 5;
  if (inflight > slots) inflight = slots;
  rmw_tc_kernel<<<grid, threads, smem, s>>>(d_layers, d_item_start, n_layers, total_items, a_bufs, a_buf_bytes,
                                             max_b_bytes, slots, inflight, staged ? 1 : 0, seed, coef, d_coef, d_status);
  return cudaGetLastError();
}

}  // namespace agzo
