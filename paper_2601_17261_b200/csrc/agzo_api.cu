// C ABI of the AGZO library: context, host-side validation, workspace planning and the
// sequencing of Algorithm 1 / Algorithm 2 over the grouped kernels.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "agzo_common.cuh"
#include "agzo_tc.cuh"

using namespace agzo;

namespace {

constexpr uint32_t kMagic = 0xA620B200u;
constexpr size_t kAlign = 256;
constexpr size_t kHeaderBytes = 256;          // DevStatus + scalar slots
constexpr size_t kCoefOffset = 64;            // float coefficient slot inside the header
constexpr int64_t kDefaultWaveBytes = 8ll << 30;
constexpr int64_t kL2ResidentWaveBytes = 64ll << 20;   // a wave's X up to this size is still in L2 at its next sweep

inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

struct Plan {
  std::vector<DevLayer> dev;       // one per layer, scratch pointers filled
  std::vector<int> tile_start;     // n + 1
  std::vector<int> wave_end;       // exclusive end index of each extraction wave
  std::vector<int> wave_region;    // scratch region (= helper stream) of each wave, -1 = nothing to do
  std::vector<int64_t> wave_xbytes;   // activation bytes of each wave (a shared X counted once)
  // the Y panels of a wave's layers lie one after another at the end of the wave's scratch, so that a
  // token-sharded run can sum all of them over the ranks in one call
  std::vector<float*> wave_y;
  std::vector<size_t> wave_y_count;   // floats, alignment gaps included
  int regions = 1;
  int total_tiles = 0;
  int max_r = 0;
  int fast_mode_mask = 0;          // storage modes present among layers on the vector path
  bool any_slow = false;           // some layer needs the scalar kernel
  bool has_extract = false;
  // tensor-core in-place pass: work items per layer (prefix, n + 1), zero-length for other layers
  std::vector<int> item_start;
  int total_items = 0;
  int max_rp = 0;
  int max_b_bytes = 0;   // largest B operand area of a tensor-core pass item
  bool staged_r = false;           // the tensor-core pass copies R tiles that a fill kernel wrote to scratch
  int max_row_tiles = 0;
  size_t image_bytes = 0;
};

struct PlanOpts {
  int64_t wave_bytes;
  int extract_path;      // 0 auto, 1 CUDA-core only, 2 tensor-core required
  int rmw_path;          // 0 auto, 1 CUDA-core only, 2 tensor cores wherever a layer allows it
  int rmw_tc_min_rank;   // auto: layers with r >= this use the tensor-core pass
  int rmw_tc_panels;     // column panels per work item of the tensor-core pass (1 or 2)
  int rmw_stage_r;       // 0: stage R in scratch when some rank exceeds 16; 1: never; 2: always
  bool tc_available;
  int extract_fused;     // 1: power steps of eligible layers run in the fused single-pass kernel; 2: also on
                         // cluster sizes that leave much of the device idle
  bool share_inputs;     // consecutive layers with the same X are served by one sweep
  int extract_regions;   // 1: waves run one after another; 2: alternate waves use two scratch regions
                         // and two helper streams, so one wave's small kernels overlap the other's sweeps
  const FusedCaps* fused_caps;   // what the device holds of the fused kernel; null when sizing without a device
};

}  // namespace

struct agzo_ctx {
  uint32_t magic;
  int device;
  int sm_count;
  char* ws;
  size_t ws_bytes;
  int last_cuda;
  int extract_path;        // 0 auto, 1 CUDA-core only, 2 tensor-core required
  int rmw_path;            // 0 auto, 1 CUDA-core only, 2 tensor cores wherever possible
  int rmw_tc_min_rank;
  int rmw_tc_slots;        // ring slots of the tensor-core pass, 0 = as many as fit
  int rmw_tc_inflight;     // loads in flight per CTA, 0 = by rank
  int rmw_tc_panels;       // column panels per work item (1 or 2), 0 = by rank
  int rmw_stage_r;         // 0 auto, 1 never, 2 always
  int64_t wave_bytes;
  int extract_streams;     // 1 or 2 (see PlanOpts::extract_regions)
  int extract_fused;       // 0 off, 1 fused power-step kernel where it pays, 2 wherever a layer's shape allows it
  int share_inputs;        // 1: consecutive layers with the same X share the sweeps over it
  // staged R images in scratch: valid for this seed until the plan changes or extraction uses the scratch
  bool rimg_valid;
  uint64_t rimg_seed;
  cudaStream_t rimg_stream;   // stream the images were written on: another stream refills them
  agzo_allreduce_fn allreduce;   // token-sharded extraction: sums a wave's Y panels over the ranks
  void* allreduce_user;
  int64_t token_offset;    // global index of this rank's first token
  cudaStream_t aux[2];     // helper streams of extraction, forked from and joined to the caller's stream
  cudaEvent_t fork_ev, join_ev[2];
  // descriptors last uploaded
  std::vector<agzo_layer> cached;
  bool cached_valid;
  Plan plan;
  // pinned staging for the upload
  void* h_stage;
  size_t h_stage_bytes;
  cudaEvent_t stage_ev;
  bool stage_pending;
  cudaStream_t stage_stream;  // stream of the last table upload: a call on another stream waits for stage_ev
  TcState tc;
  // measurement aid: event pairs around the launches of one kernel class
  int debug_fail_step_call;   // test option: the n-th internal call of agzo_step fails on the host, 0 = off
  int time_class;
  std::vector<cudaEvent_t> events;   // pairs: start, stop
  size_t events_used;
  int64_t launches;
};

namespace {

#define CU(ctx, expr)                              \
  do {                                             \
    cudaError_t e__ = (expr);                      \
    if (e__ != cudaSuccess) {                      \
      (ctx)->last_cuda = (int)e__;                 \
      return AGZO_ERR_CUDA;                        \
    }                                              \
  } while (0)

// Launch bookkeeping: counts every kernel-launching call and, for the class being timed,
// brackets it with an event pair on the stream.
struct Timed {
  agzo_ctx* c;
  cudaStream_t s;
  bool on;
  Timed(agzo_ctx* ctx, int cls, cudaStream_t st, int n_kernels = 1) : c(ctx), s(st), on(false) {
    c->launches += n_kernels;
    if (c->time_class != cls) return;
    if (c->events_used + 2 > c->events.size()) {
      for (int i = 0; i < 2; ++i) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) return;
        c->events.push_back(e);
      }
    }
    on = cudaEventRecord(c->events[c->events_used], s) == cudaSuccess;
  }
  ~Timed() {
    if (!on) return;
    cudaEventRecord(c->events[c->events_used + 1], s);
    c->events_used += 2;
  }
};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

enum Need { NEED_RMW = 1, NEED_EXTRACT = 2 };

agzo_status validate(const agzo_layer* L, int n, int need) {
  if (n < 0 || n > AGZO_MAX_LAYERS) return AGZO_ERR_INVALID_ARG;
  if (n > 0 && !L) return AGZO_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i) {
    const agzo_layer& a = L[i];
    if (a.reserved != 0) return AGZO_ERR_INVALID_ARG;
    if (a.d_in < 1 || a.d_out < 0) return AGZO_ERR_INVALID_ARG;
    if (a.r < 1 || a.r > AGZO_MAX_RANK || a.r > a.d_in) return AGZO_ERR_INVALID_ARG;
    if (!a.V || a.ldv < a.d_in || (reinterpret_cast<uintptr_t>(a.V) & 3u)) return AGZO_ERR_INVALID_ARG;
    if (need & NEED_RMW) {
      if (a.d_out < 1) return AGZO_ERR_INVALID_ARG;
      if (a.w_dtype != AGZO_BF16 && a.w_dtype != AGZO_F32) return AGZO_ERR_UNSUPPORTED;
      if (!a.W || a.ldw < a.d_in) return AGZO_ERR_INVALID_ARG;
      const size_t es = a.w_dtype == AGZO_BF16 ? 2 : 4;
      if (reinterpret_cast<uintptr_t>(a.W) & (es - 1)) return AGZO_ERR_INVALID_ARG;
      if (a.W16) {
        if (a.w_dtype != AGZO_F32) return AGZO_ERR_UNSUPPORTED;
        if (a.ldw16 < a.d_in || (reinterpret_cast<uintptr_t>(a.W16) & 1u)) return AGZO_ERR_INVALID_ARG;
      }
    }
    if (need & NEED_EXTRACT) {
      if (a.x_dtype != AGZO_BF16 && a.x_dtype != AGZO_F32) return AGZO_ERR_UNSUPPORTED;
      if (!a.X || a.m < 1 || a.ldx < a.d_in || a.r > a.m) return AGZO_ERR_INVALID_ARG;
      const size_t es = a.x_dtype == AGZO_BF16 ? 2 : 4;
      if (reinterpret_cast<uintptr_t>(a.X) & (es - 1)) return AGZO_ERR_INVALID_ARG;
    }
  }
  return AGZO_OK;
}

bool has_x(const agzo_layer& a) { return a.X != nullptr && a.m >= 1; }
bool same_input(const agzo_layer& a, const agzo_layer& b) {
  return a.X == b.X && a.ldx == b.ldx && a.m == b.m && a.d_in == b.d_in && a.x_dtype == b.x_dtype;
}

// Token slabs of the X^T T product.  CUDA-core kernels: 32 slabs at most.  Tensor-core
// kernels: slabs of 2048 tokens (32 pipeline steps per CTA) when the layer has that many.  When
// the call's layers fill the grid by their column blocks alone (long_slabs), a slab is up to
// 16384 tokens: every slab costs a partial Y (r x d_in floats written, and read again by the
// panel QR), and the CTAs' pipelines start and drain less often.
constexpr int kLongSlabColumnBlocks = 1024;   // 128-column blocks over all layers from which slabs are long
void slab_shape(const agzo_layer& a, bool tc, bool long_slabs, int* slabs, int* slab_rows) {
  int rows;
  if (tc) {
    rows = a.m >= 8192 ? (long_slabs ? (a.m < 16384 ? a.m : 16384) : 2048) : (a.m + 3) / 4;
    rows = (rows + 127) / 128 * 128;      // whole tiles of every tensor-core kernel (64 or 128 tokens)
  } else {
    rows = (a.m + 31) / 32;
    rows = (rows + 31) / 32 * 32;
  }
  if (rows < 256) rows = 256;
  *slab_rows = rows;
  *slabs = (a.m + rows - 1) / rows;
}

// scratch bytes one layer needs for extraction (0 when it has no X)
// y_parts_min: room for at least that many partial sums of Y (the fused power step leaves one per share of
// its launch that meets the layer, which can be more than the slabs of X^T T)
size_t layer_scratch(const agzo_layer& a, bool tc, bool long_slabs, bool with_panels = true, int y_parts_min = 0) {
  if (!has_x(a)) return 0;
  int slabs, slab_rows;
  slab_shape(a, tc, long_slabs, &slabs, &slab_rows);
  if (slabs < y_parts_min) slabs = y_parts_min;
  const size_t r = (size_t)a.r, d = (size_t)a.d_in, m = (size_t)a.m;
  const size_t gch = (d + 127) / 128;
  size_t b = 0;
  b += align_up(m * r * 4);                 // T
  b += align_up((size_t)slabs * r * d * 4); // Ypart
  b += align_up(r * d * 4);                 // Y
  b += align_up(gch * r * r * 8);           // Gpart
  b += align_up(r * r * 8);                 // M
  if (tc && with_panels) b += tc_layer_scratch(a);
  return b;
}

constexpr size_t kMapBytes = 512;   // four TMA descriptors per layer
// device tables after the header: layer records | tile prefix and item prefix (n + 1 ints each) | TMA descriptors
size_t prefix_bytes(int n) { return align_up((size_t)2 * (n + 1) * sizeof(int)); }
size_t table_bytes(int n) {
  return align_up((size_t)n * sizeof(DevLayer)) + prefix_bytes(n) + align_up((size_t)n * kMapBytes);
}
size_t maps_offset(int n) { return kHeaderBytes + align_up((size_t)n * sizeof(DevLayer)) + prefix_bytes(n); }

// Builds the device records.  ws == nullptr: only sizes are computed (scratch_needed).
agzo_status build_plan(const agzo_layer* L, int n, char* ws, size_t ws_bytes, const PlanOpts& opts,
                       Plan* plan, size_t* scratch_needed) {
  const int64_t wave_bytes = opts.wave_bytes;
  const int extract_path = opts.extract_path;
  const bool tc_available = opts.tc_available;
  plan->dev.assign(n, DevLayer{});
  plan->tile_start.assign(n + 1, 0);
  plan->wave_end.clear();
  plan->wave_region.clear();
  plan->wave_xbytes.clear();
  plan->wave_y.clear();
  plan->wave_y_count.clear();
  const int regions = opts.extract_regions == 2 ? 2 : 1;
  plan->regions = regions;
  plan->max_r = 0;
  plan->fast_mode_mask = 0;
  plan->any_slow = false;
  plan->has_extract = false;
  plan->item_start.assign(n + 1, 0);
  plan->total_items = 0;
  plan->max_rp = 0;
  plan->max_b_bytes = 0;
  const size_t base = kHeaderBytes + table_bytes(n);
  const size_t scratch_all = ws ? (ws_bytes > base ? ws_bytes - base : 0) : (size_t)-1;
  const size_t scratch_cap = ws ? scratch_all / regions / kAlign * kAlign : (size_t)-1;   // per region
  int real_waves = 0;
  size_t max_wave_scratch = 0;

  // Which layers take the tensor-core pass, and whether their R operands are staged in scratch
  // (ranks above 16): the operand image of every 128-row tile of every such layer, laid out from
  // the start of the scratch area (which extraction uses at other times).
  auto takes_tc_rmw = [&](const agzo_layer& a) {
    return tc_available && opts.rmw_path != 1 && rmw_tc_eligible(a) &&
           (opts.rmw_path == 2 || a.r >= opts.rmw_tc_min_rank);
  };
  {
    size_t img = 0;
    int max_tiles = 0, max_rp_all = 0;
    for (int i = 0; i < n; ++i) {
      if (!takes_tc_rmw(L[i])) continue;
      img += rmw_tc_image_bytes(L[i]);
      max_tiles = std::max(max_tiles, (L[i].d_out + 127) / 128);
      max_rp_all = std::max(max_rp_all, (L[i].r + 7) & ~7);
    }
    const size_t room = ws ? (ws_bytes > base ? ws_bytes - base : 0) : (size_t)-1;
    const bool want = opts.rmw_stage_r == 2 || (opts.rmw_stage_r == 0 && max_rp_all > 16);
    plan->staged_r = want && img > 0 && img <= room;
    plan->max_row_tiles = max_tiles;
    plan->image_bytes = want ? img : 0;
  }
  size_t img_off = 0;
  int tiles = 0;
  long long items = 0;
  for (int i = 0; i < n; ++i) {
    const agzo_layer& a = L[i];
    DevLayer& D = plan->dev[i];
    D.W = a.W; D.W16 = a.W16; D.X = a.X; D.V = a.V;
    D.ldw = a.ldw; D.ldw16 = a.ldw16; D.ldx = a.ldx; D.ldv = a.ldv;
    D.w_dtype = a.w_dtype; D.x_dtype = a.x_dtype;
    D.d_out = a.d_out; D.d_in = a.d_in; D.m = a.m; D.r = a.r;
    D.layer_id = a.layer_id;
    D.rmw_mode = a.W16 ? RMW_PAIR_COMPUTE : (a.w_dtype == AGZO_BF16 ? RMW_BF16 : RMW_F32);
    const size_t es = a.w_dtype == AGZO_BF16 ? 2 : 4;
    bool vec = a.W && aligned16(a.W) && (a.ldw * es) % 16 == 0 && a.d_in % 8 == 0 &&
               aligned16(a.V) && a.ldv % 4 == 0;
    if (a.W16) vec = vec && aligned16(a.W16) && (a.ldw16 * 2) % 16 == 0;
    D.vec_ok = vec ? 1 : 0;
    // bf16 weights of sufficient rank go through the tensor-core pass and get no CUDA-core tiles
    const bool tc_rmw = takes_tc_rmw(a);
    plan->item_start[i] = (int)items;
    if (tc_rmw) {
      rmw_tc_shape(a, opts.rmw_tc_panels, plan->staged_r, &D);
      if (plan->staged_r && ws) {
        D.rimg = reinterpret_cast<unsigned char*>(ws + base + img_off);
        D.rimg_tile_bytes = (int)(rmw_tc_image_bytes(a) / (size_t)((a.d_out + 127) / 128));
      }
      img_off += rmw_tc_image_bytes(a);
      D.rtc_item0 = (int)items;
      items += (long long)D.rtc_panels * D.rtc_chunks;
      if (items > 0x7fffffff) return AGZO_ERR_INVALID_ARG;
      if (D.rtc_rp > plan->max_rp) plan->max_rp = D.rtc_rp;
      plan->max_b_bytes = std::max(plan->max_b_bytes, rmw_tc_b_bytes(D));
      if (ws) D.wmap = ws + maps_offset(n) + (size_t)i * kMapBytes + 384;
    } else if (a.W) {
      if (vec) plan->fast_mode_mask |= 1 << D.rmw_mode; else plan->any_slow = true;
    }
    D.tile0 = tiles;
    D.tiles_c = (a.d_in + 511) / 512;
    D.tiles_r = (a.W && !tc_rmw) ? (a.d_out + 255) / 256 : 0;
    plan->tile_start[i] = tiles;
    const long long nt = (long long)D.tiles_c * D.tiles_r;
    if (tiles + nt > 0x7fffffff) return AGZO_ERR_INVALID_ARG;
    tiles += (int)nt;
    if (a.r > plan->max_r) plan->max_r = a.r;
  }
  plan->tile_start[n] = tiles;
  plan->total_tiles = tiles;
  plan->item_start[n] = (int)items;
  plan->total_items = (int)items;

  // extraction waves: consecutive layers whose activations fit the wave budget and whose
  // scratch fits the workspace
  // A layer that shares its X with a neighbour stays with the two-sweep kernels unless fusing is forced: one
  // sweep serves the whole group there, which moves fewer bytes per layer than one fused pass per layer.
  auto shares_input = [&](int k) {
    if (!opts.share_inputs) return false;
    return (k > 0 && has_x(L[k - 1]) && tc_eligible(L[k - 1]) && same_input(L[k - 1], L[k])) ||
           (k + 1 < n && has_x(L[k + 1]) && tc_eligible(L[k + 1]) && same_input(L[k], L[k + 1]));
  };
  auto runs_fused = [&](const agzo_layer& a) {
    return opts.extract_fused && extract_path != 1 && extract_path != 3 && tc_available && tc_eligible(a) &&
           fused_eligible(opts.fused_caps, a, opts.extract_fused == 2) && (opts.extract_fused == 2 || !shares_input((int)(&a - L)));
  };
  long long column_blocks = 0;
  for (int k = 0; k < n; ++k)
    if (has_x(L[k]) && extract_path != 1 && tc_available && tc_eligible(L[k]))
      column_blocks += (L[k].d_in + 127) / 128;
  const bool long_slabs_any = column_blocks >= kLongSlabColumnBlocks;
  auto long_slabs_for = [&](const agzo_layer&) { return long_slabs_any; };
  auto y_parts_min = [&](const agzo_layer& a) {
    return runs_fused(a) ? fused_parts_bound(a, fused_cluster_size(opts.fused_caps, a, opts.extract_fused == 2)) : 0;
  };
  int i = 0;
  while (i < n) {
    if (!has_x(L[i])) {
      ++i;
      plan->wave_end.push_back(i); plan->wave_region.push_back(-1); plan->wave_xbytes.push_back(0);
      plan->wave_y.push_back(nullptr); plan->wave_y_count.push_back(0);
      continue;
    }
    const int region = real_waves++ % regions;
    plan->has_extract = true;
    size_t used = 0, used_y = 0;    // scratch of the wave so far; the part of it that is Y panels
    int64_t xbytes = 0;
    int j = i;
    const bool wave_tc = extract_path != 1 && tc_available && tc_eligible(L[i]);
    while (j < n && has_x(L[j])) {
      const bool tc = extract_path != 1 && tc_available && tc_eligible(L[j]);
      if (tc != wave_tc) break;      // a wave runs on one kind of kernel
      // a unit is one layer, or a run of consecutive layers that read the same X (one sweep serves all)
      int glen = 1, rows = tc ? tc_operand_rows(L[j].r) : 0;
      if (tc && opts.share_inputs && !runs_fused(L[j])) {
        while (j + glen < n && has_x(L[j + glen]) && same_input(L[j], L[j + glen]) && tc_eligible(L[j + glen]) &&
               !runs_fused(L[j + glen]) &&
               rows + tc_operand_rows(L[j + glen].r) <= 256) {
          rows += tc_operand_rows(L[j + glen].r);
          ++glen;
        }
      }
      auto unit_need = [&](int len, int nrows) {
        size_t b = 0;
        for (int g = 0; g < len; ++g) b += layer_scratch(L[j + g], tc, long_slabs_for(L[j + g]), false, y_parts_min(L[j + g]));
        if (tc) b += tc_panel_bytes(L[j], nrows);
        return b;
      };
      size_t need = unit_need(glen, rows);
      const int64_t xb = (int64_t)L[j].m * L[j].d_in * (L[j].x_dtype == AGZO_BF16 ? 2 : 4);
      if (j > i && (used + need > scratch_cap || xbytes + xb > wave_bytes)) break;
      if (used + need > scratch_cap && glen > 1) {   // the group alone does not fit: fall back to single layers
        glen = 1;
        rows = tc_operand_rows(L[j].r);
        need = unit_need(glen, rows);
      }
      if (used + need > scratch_cap) return AGZO_ERR_WORKSPACE;
      // carve
      size_t need_y = 0;
      for (int g = 0; g < glen; ++g) need_y += align_up((size_t)L[j + g].r * (size_t)L[j + g].d_in * 4);
      if (ws) {
        char* p = ws + base + (size_t)region * scratch_cap + (used - used_y);
        for (int g = 0; g < glen; ++g) {
          DevLayer& D = plan->dev[j + g];
          const agzo_layer& a = L[j + g];
          int slabs, slab_rows;
          slab_shape(a, tc, long_slabs_for(a), &slabs, &slab_rows);
          const size_t r = (size_t)a.r, d = (size_t)a.d_in, m = (size_t)a.m;
          const size_t gch = (d + 127) / 128;
          D.slabs = slabs; D.slab_rows = slab_rows; D.gchunks = (int)gch;
          D.T = reinterpret_cast<float*>(p);      p += align_up(m * r * 4);
          const size_t parts = (size_t)(slabs > y_parts_min(a) ? slabs : y_parts_min(a));
          D.Ypart = reinterpret_cast<float*>(p);  p += align_up(parts * r * d * 4);
          D.Gpart = reinterpret_cast<double*>(p); p += align_up(gch * r * r * 8);
          D.M = reinterpret_cast<double*>(p);     p += align_up(r * r * 8);
        }
        if (tc) {
          int row0 = 0;
          for (int g = 0; g < glen; ++g) {
            DevLayer& D = plan->dev[j + g];
            const agzo_layer& a = L[j + g];
            tc_set_panels(a, &D, p, rows, row0);
            row0 += tc_operand_rows(a.r);
            D.grp_role = glen == 1 ? 0 : (g == 0 ? 1 : 2);
            D.grp_n = g == 0 ? glen : 0;
            D.grp_NB = g == 0 ? rows : 0;
            D.tmaps = ws + maps_offset(n) + (size_t)(j + g) * kMapBytes;
            // the power steps of this layer run fused (X read once per step) where its shape allows
            D.fz_C = runs_fused(a) ? fused_cluster_size(opts.fused_caps, a, opts.extract_fused == 2) : 0;
            D.fz_slice = fused_slice_cols(opts.fused_caps, a, opts.extract_fused == 2);
          }
        }
      }
      used += need;
      used_y += need_y;
      xbytes += xb;
      j += glen;
    }
    if (used > max_wave_scratch) max_wave_scratch = used;
    {   // the Y panels follow everything else of the wave
      char* y0 = ws ? ws + base + (size_t)region * scratch_cap + (used - used_y) : nullptr;
      char* y = y0;
      for (int k = i; k < j && ws; ++k) {
        plan->dev[k].Y = reinterpret_cast<float*>(y);
        y += align_up((size_t)L[k].r * (size_t)L[k].d_in * 4);
      }
      plan->wave_y.push_back(reinterpret_cast<float*>(y0));
      plan->wave_y_count.push_back(used_y / 4);
    }
    {   // order in which T = X Q takes the wave's layers: largest d_in first (stable)
      std::vector<int> ord(j - i);
      for (int k = 0; k < j - i; ++k) ord[k] = k;
      std::stable_sort(ord.begin(), ord.end(), [&](int a, int b) { return L[i + a].d_in > L[i + b].d_in; });
      for (int k = 0; k < j - i; ++k) plan->dev[i + k].xq_order = ord[k];
    }
    if (ws) {
      // A wave whose activations stay in L2 from one sweep to the next gains nothing from the fused kernel
      // (its point is that X crosses HBM once per power step): such a wave takes the two sweeps throughout.
      if (opts.extract_fused != 2 && xbytes <= kL2ResidentWaveBytes)
        for (int k = i; k < j; ++k) plan->dev[k].fz_C = 0;
      // the fused kernel's launches of this wave, one per cluster size: who works on which tiles
      if (opts.fused_caps)
        for (int C = 1; C <= 16; ++C) fused_plan_shares(*opts.fused_caps, plan->dev.data(), i, j, C);
    }
    plan->wave_end.push_back(j);
    plan->wave_region.push_back(region);
    plan->wave_xbytes.push_back(xbytes);
    i = j;
  }
  if (scratch_needed) {
    *scratch_needed = max_wave_scratch * regions + (regions > 1 ? kAlign : 0);
    if (plan->image_bytes > *scratch_needed) *scratch_needed = plan->image_bytes;
  }
  return AGZO_OK;
}

bool same_layers(const agzo_ctx* c, const agzo_layer* L, int n) {
  return c->cached_valid && (int)c->cached.size() == n &&
         (n == 0 || std::memcmp(c->cached.data(), L, (size_t)n * sizeof(agzo_layer)) == 0);
}

DevLayer* dev_layers(agzo_ctx* c) { return reinterpret_cast<DevLayer*>(c->ws + kHeaderBytes); }
int* dev_tiles(agzo_ctx* c, int n) {
  return reinterpret_cast<int*>(c->ws + kHeaderBytes + align_up((size_t)n * sizeof(DevLayer)));
}
int* dev_items(agzo_ctx* c, int n) { return dev_tiles(c, n) + (n + 1); }
DevStatus* dev_status(agzo_ctx* c) { return reinterpret_cast<DevStatus*>(c->ws); }
float* dev_coef(agzo_ctx* c) { return reinterpret_cast<float*>(c->ws + kCoefOffset); }

// Makes the device tables describe `L`; uploads only when the descriptors changed.
agzo_status prepare(agzo_ctx* c, const agzo_layer* L, int n, cudaStream_t s) {
  if (same_layers(c, L, n)) {
    // the tables were uploaded on another stream: this one must not read them before they have landed
    if (c->stage_pending && s != c->stage_stream) CU(c, cudaStreamWaitEvent(s, c->stage_ev, 0));
    return AGZO_OK;
  }
  c->rimg_valid = false;
  if (kHeaderBytes + table_bytes(n) > c->ws_bytes) return AGZO_ERR_WORKSPACE;
  Plan plan;
  PlanOpts opts{c->wave_bytes, c->extract_path, c->rmw_path, c->rmw_tc_min_rank, c->rmw_tc_panels, c->rmw_stage_r,
                c->tc.available, c->extract_fused, c->share_inputs != 0,
                c->allreduce ? 1 : c->extract_streams,    // the ranks' sums run in wave order on the caller's stream
                &c->tc.fused};
  agzo_status st = build_plan(L, n, c->ws, c->ws_bytes, opts, &plan, nullptr);
  if (st == AGZO_ERR_WORKSPACE && opts.extract_regions == 2) {   // a workspace sized for one region
    opts.extract_regions = 1;
    st = build_plan(L, n, c->ws, c->ws_bytes, opts, &plan, nullptr);
  }
  if (st != AGZO_OK) return st;
  const size_t lb = align_up((size_t)n * sizeof(DevLayer));
  const size_t tb = prefix_bytes(n) + (size_t)n * kMapBytes;
  if (c->stage_pending) {
    CU(c, cudaEventSynchronize(c->stage_ev));
    c->stage_pending = false;
  }
  if (lb + tb > c->h_stage_bytes) {
    if (c->h_stage) CU(c, cudaFreeHost(c->h_stage));
    c->h_stage = nullptr;
    c->h_stage_bytes = 0;
    CU(c, cudaMallocHost(&c->h_stage, (lb + tb) * 2));
    c->h_stage_bytes = (lb + tb) * 2;
  }
  if (n > 0) {
    std::memcpy(c->h_stage, plan.dev.data(), (size_t)n * sizeof(DevLayer));
    char* hs = static_cast<char*>(c->h_stage);
    std::memset(hs + lb, 0, tb);
    std::memcpy(hs + lb, plan.tile_start.data(), (size_t)(n + 1) * sizeof(int));
    std::memcpy(hs + lb + (size_t)(n + 1) * sizeof(int), plan.item_start.data(), (size_t)(n + 1) * sizeof(int));
    char* hmaps = hs + lb + prefix_bytes(n);
    for (int i = 0; i < n; ++i) {
      if (plan.dev[i].Qb && plan.dev[i].grp_role != 2 &&
          !tc_encode_maps(c->tc, plan.dev[i], hmaps + (size_t)i * kMapBytes))
        return AGZO_ERR_UNSUPPORTED;
      if (plan.dev[i].wmap && !rmw_tc_encode_map(c->tc, plan.dev[i], hmaps + (size_t)i * kMapBytes + 384))
        return AGZO_ERR_UNSUPPORTED;
    }
    CU(c, cudaMemcpyAsync(c->ws + kHeaderBytes, c->h_stage, lb + tb, cudaMemcpyHostToDevice, s));
    CU(c, cudaEventRecord(c->stage_ev, s));
    c->stage_pending = true;
    c->stage_stream = s;
  }
  c->plan = std::move(plan);
  c->cached.assign(L, L + n);
  c->cached_valid = true;
  return AGZO_OK;
}

agzo_status check_ctx(agzo_ctx* c) {
  if (!c || c->magic != kMagic) return AGZO_ERR_STATE;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != c->device) {
    if (cudaSetDevice(c->device) != cudaSuccess) return AGZO_ERR_CUDA;
  }
  return AGZO_OK;
}

agzo_status rmw_pass(agzo_ctx* c, const agzo_layer* L, int n, uint64_t seed, float coef,
                     const float* d_coef, bool pair_update, cudaStream_t s) {
  agzo_status st = validate(L, n, NEED_RMW);
  if (st != AGZO_OK) return st;
  if (n == 0) return AGZO_OK;
  st = prepare(c, L, n, s);
  if (st != AGZO_OK) return st;
  if (c->plan.total_items > 0) {
    // the passes of one step share the seed, hence R: the images a pass staged serve the next ones
    const bool fill = c->plan.staged_r && !(c->rimg_valid && c->rimg_seed == seed && c->rimg_stream == s);
    c->rimg_valid = false;
    Timed t(c, AGZO_KC_RMW_TC, s, fill ? 2 : 1);
    CU(c, launch_rmw_tc(dev_layers(c), dev_items(c, n), n, c->plan.total_items, c->plan.max_rp, c->plan.max_r,
                        c->plan.max_b_bytes, c->plan.max_row_tiles, c->plan.staged_r, fill, c->rmw_tc_slots,
                        c->rmw_tc_inflight, seed, coef, d_coef, dev_status(c), c->sm_count, s));
    if (c->plan.staged_r) { c->rimg_valid = true; c->rimg_seed = seed; c->rimg_stream = s; }
  }
  if (c->plan.total_tiles > 0) {
    Timed t(c, AGZO_KC_RMW, s);
    CU(c, launch_rmw(dev_layers(c), dev_tiles(c, n), n, c->plan.total_tiles, c->plan.max_r,
                     c->plan.fast_mode_mask, c->plan.any_slow, seed, coef, d_coef, pair_update,
                     c->sm_count, s));
  }
  return AGZO_OK;
}

}  // namespace

// =================================================================== C ABI
extern "C" {

const char* agzo_status_string(agzo_status s) {
  switch (s) {
    case AGZO_OK: return "ok";
    case AGZO_ERR_INVALID_ARG: return "invalid argument";
    case AGZO_ERR_UNSUPPORTED: return "unsupported dtype or mode";
    case AGZO_ERR_CUDA: return "CUDA runtime error";
    case AGZO_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case AGZO_ERR_STATE: return "invalid context";
    case AGZO_ERR_TIMEOUT: return "device-side wait ran out";
    case AGZO_ERR_CALLBACK: return "callback failed (loss or all-reduce)";
    case AGZO_WARN_RANK_DEFICIENT: return "rank-deficient activation panel";
  }
  return "unknown status";
}

int agzo_last_cuda_error(const agzo_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }

agzo_status agzo_workspace_bytes(const agzo_layer* h_layers, int n, size_t* h_bytes) {
  if (!h_bytes) return AGZO_ERR_INVALID_ARG;
  agzo_status st = validate(h_layers, n, 0);
  if (st != AGZO_OK) return st;
  // large enough for either kind of extraction kernel (the "extract_path" option may pick
  // the CUDA-core kernels, whose slabs are shaped differently)
  Plan plan;
  size_t scratch = 0, scratch_cc = 0;
  st = build_plan(h_layers, n, nullptr, 0, PlanOpts{kDefaultWaveBytes, 0, 0, 3, 0, 0, true, 0, false, 2, nullptr}, &plan, &scratch);
  if (st != AGZO_OK) return st;
  st = build_plan(h_layers, n, nullptr, 0, PlanOpts{kDefaultWaveBytes, 1, 1, 0, 1, 1, false, 0, false, 2, nullptr}, &plan, &scratch_cc);
  if (st != AGZO_OK) return st;
  if (scratch_cc > scratch) scratch = scratch_cc;
  // ... and for the fused power step, whose layers keep room for one partial sum of Y per share of a launch
  st = build_plan(h_layers, n, nullptr, 0, PlanOpts{kDefaultWaveBytes, 0, 0, 3, 0, 0, true, 2, false, 2, nullptr}, &plan, &scratch_cc);
  if (st != AGZO_OK) return st;
  if (scratch_cc > scratch) scratch = scratch_cc;
  *h_bytes = kHeaderBytes + table_bytes(n) + scratch + kAlign;
  return AGZO_OK;
}

agzo_status agzo_create(agzo_ctx** out, int device, void* workspace, size_t workspace_bytes) {
  if (!out) return AGZO_ERR_INVALID_ARG;
  *out = nullptr;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) ||
      workspace_bytes < kHeaderBytes)
    return AGZO_ERR_WORKSPACE;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count)
    return AGZO_ERR_CUDA;
  agzo_ctx* c = new (std::nothrow) agzo_ctx();
  if (!c) return AGZO_ERR_INVALID_ARG;
  c->magic = kMagic;
  c->device = device;
  c->ws = static_cast<char*>(workspace);
  c->ws_bytes = workspace_bytes;
  c->last_cuda = 0;
  c->extract_path = 0;
  c->rmw_path = 0;
  c->rmw_tc_min_rank = 3;   // measured: from r = 3 on the tensor-core pass is the faster one
  c->rmw_tc_slots = 0;
  c->rmw_tc_inflight = 0;
  c->rmw_tc_panels = 0;
  c->rmw_stage_r = 0;
  c->wave_bytes = kDefaultWaveBytes;
  c->extract_streams = 2;
  c->extract_fused = 1;
  c->allreduce = nullptr;
  c->rimg_valid = false;
  c->rimg_seed = 0;
  c->rimg_stream = nullptr;
  c->stage_stream = nullptr;
  c->allreduce_user = nullptr;
  c->token_offset = 0;
  c->share_inputs = 1;
  c->aux[0] = c->aux[1] = nullptr;
  c->fork_ev = c->join_ev[0] = c->join_ev[1] = nullptr;
  c->cached_valid = false;
  c->h_stage = nullptr;
  c->h_stage_bytes = 0;
  c->stage_pending = false;
  c->stage_ev = nullptr;
  c->time_class = 0;
  c->debug_fail_step_call = 0;
  c->events_used = 0;
  c->launches = 0;
  cudaError_t e = cudaSetDevice(device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->stage_ev, cudaEventDisableTiming);
  for (int k = 0; k < 2 && e == cudaSuccess; ++k) {
    e = cudaStreamCreateWithFlags(&c->aux[k], cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->join_ev[k], cudaEventDisableTiming);
  }
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->fork_ev, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaMemset(c->ws, 0, kHeaderBytes);
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = tc_init(&c->tc, device);
  if (e != cudaSuccess) {
    if (c->stage_ev) cudaEventDestroy(c->stage_ev);
    if (c->fork_ev) cudaEventDestroy(c->fork_ev);
    for (int k = 0; k < 2; ++k) {
      if (c->join_ev[k]) cudaEventDestroy(c->join_ev[k]);
      if (c->aux[k]) cudaStreamDestroy(c->aux[k]);
    }
    delete c;
    return AGZO_ERR_CUDA;
  }
  *out = c;
  return AGZO_OK;
}

agzo_status agzo_destroy(agzo_ctx* ctx) {
  if (!ctx || ctx->magic != kMagic) return AGZO_ERR_STATE;
  if (ctx->stage_pending) cudaEventSynchronize(ctx->stage_ev);
  if (ctx->h_stage) cudaFreeHost(ctx->h_stage);
  if (ctx->stage_ev) cudaEventDestroy(ctx->stage_ev);
  if (ctx->fork_ev) cudaEventDestroy(ctx->fork_ev);
  for (int k = 0; k < 2; ++k) {
    if (ctx->aux[k]) cudaStreamSynchronize(ctx->aux[k]);
    if (ctx->join_ev[k]) cudaEventDestroy(ctx->join_ev[k]);
    if (ctx->aux[k]) cudaStreamDestroy(ctx->aux[k]);
  }
  for (cudaEvent_t e : ctx->events) cudaEventDestroy(e);
  ctx->magic = 0;
  delete ctx;
  return AGZO_OK;
}

agzo_status agzo_set_option(agzo_ctx* ctx, const char* name, int64_t value) {
  if (!ctx || ctx->magic != kMagic) return AGZO_ERR_STATE;
  if (!name) return AGZO_ERR_INVALID_ARG;
  if (std::strcmp(name, "extract_path") == 0) {
    if (value < 0 || value > 3) return AGZO_ERR_INVALID_ARG;
    ctx->extract_path = (int)value;
  } else if (std::strcmp(name, "rmw_path") == 0) {
    if (value < 0 || value > 2) return AGZO_ERR_INVALID_ARG;
    ctx->rmw_path = (int)value;
  } else if (std::strcmp(name, "rmw_tc_min_rank") == 0) {
    if (value < 1 || value > AGZO_MAX_RANK) return AGZO_ERR_INVALID_ARG;
    ctx->rmw_tc_min_rank = (int)value;
  } else if (std::strcmp(name, "rmw_tc_inflight") == 0) {
    if (value < 0 || value > 64) return AGZO_ERR_INVALID_ARG;
    ctx->rmw_tc_inflight = (int)value;
    return AGZO_OK;
  } else if (std::strcmp(name, "rmw_stage_r") == 0) {
    if (value < 0 || value > 2) return AGZO_ERR_INVALID_ARG;
    ctx->rmw_stage_r = (int)value;
  } else if (std::strcmp(name, "rmw_tc_panels") == 0) {
    if (value < 0 || value > 2) return AGZO_ERR_INVALID_ARG;
    ctx->rmw_tc_panels = (int)value;
  } else if (std::strcmp(name, "rmw_tc_slots") == 0) {
    if (value < 0 || value > 64) return AGZO_ERR_INVALID_ARG;
    ctx->rmw_tc_slots = (int)value;
    return AGZO_OK;
  } else if (std::strcmp(name, "share_inputs") == 0) {
    if (value < 0 || value > 1) return AGZO_ERR_INVALID_ARG;
    ctx->share_inputs = (int)value;
  } else if (std::strcmp(name, "extract_fused") == 0) {
    if (value < 0 || value > 2) return AGZO_ERR_INVALID_ARG;
    ctx->extract_fused = (int)value;
  } else if (std::strcmp(name, "extract_streams") == 0) {
    if (value < 1 || value > 2) return AGZO_ERR_INVALID_ARG;
    ctx->extract_streams = (int)value;
  } else if (std::strcmp(name, "wave_bytes") == 0) {
    if (value < 0) return AGZO_ERR_INVALID_ARG;
    ctx->wave_bytes = value;
  } else if (std::strcmp(name, "debug_fail_step_call") == 0) {
    if (value < 0 || value > 16) return AGZO_ERR_INVALID_ARG;
    ctx->debug_fail_step_call = (int)value;
    return AGZO_OK;
  } else if (std::strcmp(name, "time_kernel_class") == 0) {
    if (value < 0 || value > 9) return AGZO_ERR_INVALID_ARG;
    ctx->time_class = (int)value;
    return AGZO_OK;
  } else {
    return AGZO_ERR_INVALID_ARG;
  }
  ctx->cached_valid = false;   // the plan depends on the options
  return AGZO_OK;
}

agzo_status agzo_set_allreduce(agzo_ctx* ctx, agzo_allreduce_fn fn, void* user, int64_t token_offset) {
  if (!ctx || ctx->magic != kMagic) return AGZO_ERR_STATE;
  if (token_offset < 0 || (!fn && token_offset != 0)) return AGZO_ERR_INVALID_ARG;
  ctx->allreduce = fn;
  ctx->allreduce_user = user;
  ctx->token_offset = token_offset;
  ctx->cached_valid = false;   // the number of scratch regions depends on it
  return AGZO_OK;
}

agzo_status agzo_read_counters(agzo_ctx* ctx, double* h_ms, int64_t* h_timed, int64_t* h_total) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  double ms = 0.0;
  for (size_t i = 0; i + 1 < ctx->events_used; i += 2) {
    CU(ctx, cudaEventSynchronize(ctx->events[i + 1]));
    float t = 0.f;
    CU(ctx, cudaEventElapsedTime(&t, ctx->events[i], ctx->events[i + 1]));
    ms += (double)t;
  }
  if (h_ms) *h_ms = ms;
  if (h_timed) *h_timed = (int64_t)(ctx->events_used / 2);
  if (h_total) *h_total = ctx->launches;
  ctx->events_used = 0;
  ctx->launches = 0;
  return AGZO_OK;
}

agzo_status agzo_query_cluster_capacity(agzo_ctx* ctx, int32_t* h_clusters) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (!h_clusters) return AGZO_ERR_INVALID_ARG;
  for (int C = 0; C <= 16; ++C) h_clusters[C] = ctx->tc.available ? fused_resident_clusters(ctx->tc.fused, C) : 0;
  return AGZO_OK;
}

agzo_status agzo_query_fused(agzo_ctx* ctx, const agzo_layer* h_layers, int n, int32_t* h_cluster, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (!h_cluster || n < 0) return AGZO_ERR_INVALID_ARG;
  st = validate(h_layers, n, 0);
  if (st != AGZO_OK) return st;
  if (n == 0) return AGZO_OK;
  st = prepare(ctx, h_layers, n, static_cast<cudaStream_t>(stream));
  if (st != AGZO_OK) return st;
  for (int i = 0; i < n; ++i) h_cluster[i] = ctx->plan.dev[i].fz_C;
  return AGZO_OK;
}

agzo_status agzo_poll(agzo_ctx* ctx, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  DevStatus h{};
  CU(ctx, cudaMemcpyAsync(&h, dev_status(ctx), sizeof(h), cudaMemcpyDeviceToHost, s));
  CU(ctx, cudaMemsetAsync(dev_status(ctx), 0, sizeof(DevStatus), s));
  CU(ctx, cudaStreamSynchronize(s));
  if (h.timeout) return AGZO_ERR_TIMEOUT;
  if (h.rank_deficient) return AGZO_WARN_RANK_DEFICIENT;
  return AGZO_OK;
}

agzo_status agzo_extract_subspace(agzo_ctx* ctx, const agzo_layer* h_layers, int n, uint64_t seed,
                                  int K, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (K < 0 || K > 16) return AGZO_ERR_INVALID_ARG;
  st = validate(h_layers, n, NEED_EXTRACT);
  if (st != AGZO_OK) return st;
  if (n == 0) return AGZO_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (ctx->extract_path >= 2)
    for (int i = 0; i < n; ++i)
      if (!ctx->tc.available || !tc_eligible(h_layers[i])) return AGZO_ERR_UNSUPPORTED;
  st = prepare(ctx, h_layers, n, s);
  if (st != AGZO_OK) return st;
  ctx->rimg_valid = false;   // extraction takes the scratch area

  const Plan& P = ctx->plan;
  // With two scratch regions, alternate waves run on two helper streams forked from the
  // caller's stream: the short, latency-bound kernels of one wave (panel QR) overlap the
  // other wave's sweeps over X.  Everything is joined back before the call returns.
  int n_real = 0;
  for (int rg : P.wave_region) n_real += rg >= 0;
  const bool forked = P.regions == 2 && n_real >= 2;
  if (forked) {
    CU(ctx, cudaEventRecord(ctx->fork_ev, s));
    for (int k = 0; k < 2; ++k) CU(ctx, cudaStreamWaitEvent(ctx->aux[k], ctx->fork_ev, 0));
  }
  auto run_waves = [&]() -> agzo_status {
    int l0 = 0;
    for (size_t wv = 0; wv < P.wave_end.size(); ++wv) {
      const int l1 = P.wave_end[wv];
      ExtractWave w{};
      w.d_layers = dev_layers(ctx);
      w.l0 = l0; w.l1 = l1;
      w.omega_row0 = ctx->allreduce ? ctx->token_offset : 0;
      w.y_reduced = ctx->allreduce ? 1 : 0;
      bool all_tc = ctx->extract_path != 1;
      for (int i = l0; i < l1; ++i) {
        const DevLayer& D = P.dev[i];
        if (D.m > w.max_m) w.max_m = D.m;
        if (D.d_in > w.max_din) w.max_din = D.d_in;
        if (D.r > w.max_r) w.max_r = D.r;
        if (D.slabs > w.max_slabs) w.max_slabs = D.slabs;
        if (D.gchunks > w.max_gchunks) w.max_gchunks = D.gchunks;
        if (!D.Qb) all_tc = false;
      }
      l0 = l1;
      if (w.max_m == 0 || P.wave_region[wv] < 0) continue;
      cudaStream_t ws = forked ? ctx->aux[P.wave_region[wv]] : s;
      DevStatus* dst = dev_status(ctx);
      auto panel_qr = [&]() -> cudaError_t {
        Timed t(ctx, AGZO_KC_PANEL_QR, ws, 3);
        return launch_panel_qr(w, dst, ws);
      };
      // token-sharded run: Y = sum over ranks of X_p^T T_p, all panels of the wave in one call
      auto sum_over_ranks = [&]() -> agzo_status {
        if (!ctx->allreduce) return AGZO_OK;
        {
          Timed t(ctx, AGZO_KC_PANEL_QR, ws);
          CU(ctx, launch_sum_slabs(w, ws));
        }
        if (ctx->allreduce(ctx->allreduce_user, ws, P.wave_y[wv], P.wave_y_count[wv]) != 0) return AGZO_ERR_CALLBACK;
        return AGZO_OK;
      };
      auto omega = [&]() -> cudaError_t {
        Timed t(ctx, AGZO_KC_OMEGA, ws);
        return all_tc ? tc_fill_omega(ctx->tc, w, P.dev.data(), seed, ws) : launch_fill_omega(w, seed, ws);
      };
      // layers served by the fused power-step kernel, by cluster size; the rest take T = X Q, Y = X^T T
      unsigned fz_classes = 0;
      bool any_unfused = false;
      for (int i = w.l0; i < w.l1; ++i) {
        if (all_tc && P.dev[i].fz_C) fz_classes |= 1u << P.dev[i].fz_C; else any_unfused = true;
      }
      auto xt_t = [&](bool skip_fused) -> cudaError_t {       // Y <- H T
        Timed t(ctx, all_tc ? AGZO_KC_TC_XT_T : AGZO_KC_XT_T, ws);
        return all_tc ? tc_xt_t(ctx->tc, w, P.dev.data(), dst, skip_fused, ws) : launch_xt_t(w, ws);
      };
      auto x_q = [&]() -> cudaError_t {        // T <- H^T Q
        Timed t(ctx, all_tc ? AGZO_KC_TC_X_Q : AGZO_KC_X_Q, ws);
        return all_tc ? tc_x_q(ctx->tc, w, P.dev.data(), dst, true, ws) : launch_x_q(w, ws);
      };
      auto power_fused = [&]() -> cudaError_t {              // Y <- H (H^T Q) in one pass
        for (int C = 1; C <= 16; ++C) {
          if (!(fz_classes & (1u << C))) continue;
          Timed t(ctx, AGZO_KC_FUSED_POWER, ws);
          cudaError_t e = launch_fused_power_step(ctx->tc.fused, w, P.dev.data(), C, dst, ws);
          if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
      };
      agzo_status sr;
      CU(ctx, omega());                        // Omega
      CU(ctx, xt_t(false));                    // Y <- H Omega
      for (int k = 0; k < K; ++k) {
        if ((sr = sum_over_ranks()) != AGZO_OK) return sr;
        CU(ctx, panel_qr());                   // Q <- qr(Y)
        if (fz_classes) {
          CU(ctx, power_fused());
          w.after_fused = 1;                   // their partial sums are now one per share, not one per slab
        }
        if (any_unfused) {
          CU(ctx, x_q());
          CU(ctx, xt_t(true));                 // Y <- H (H^T Q)
        }
      }
      if ((sr = sum_over_ranks()) != AGZO_OK) return sr;
      CU(ctx, panel_qr());                     // A <- qr(Y)
    }
    return AGZO_OK;
  };
  st = run_waves();
  if (forked) {   // join also when a launch failed: the caller's stream must not run ahead of the helpers
    for (int k = 0; k < 2; ++k) {
      cudaError_t e = cudaEventRecord(ctx->join_ev[k], ctx->aux[k]);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(s, ctx->join_ev[k], 0);
      if (e != cudaSuccess && st == AGZO_OK) { ctx->last_cuda = (int)e; st = AGZO_ERR_CUDA; }
    }
  }
  return st;
}

agzo_status agzo_perturb(agzo_ctx* ctx, const agzo_layer* h_layers, int n, uint64_t seed,
                         float scale, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  return rmw_pass(ctx, h_layers, n, seed, scale, nullptr, false, static_cast<cudaStream_t>(stream));
}

agzo_status agzo_restore(agzo_ctx* ctx, const agzo_layer* h_layers, int n, uint64_t seed,
                         float scale, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  // a master/compute pair is restored by rewriting W16 = bf16(W): coefficient 0 on the pair path
  bool any_pair = false, any_plain = false;
  for (int i = 0; h_layers && i < n; ++i) (h_layers[i].W16 ? any_pair : any_plain) = true;
  if (any_pair && any_plain) return AGZO_ERR_UNSUPPORTED;
  const float c = any_pair ? 0.0f : -scale;
  return rmw_pass(ctx, h_layers, n, seed, c, nullptr, false, static_cast<cudaStream_t>(stream));
}

agzo_status agzo_update(agzo_ctx* ctx, const agzo_layer* h_layers, int n, uint64_t seed, float lr,
                        const float* d_ghat, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (!d_ghat) return AGZO_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = validate(h_layers, n, NEED_RMW);
  if (st != AGZO_OK) return st;
  if (n == 0) return AGZO_OK;
  ctx->launches += 1;
  CU(ctx, launch_coef(d_ghat, 0.f, lr, 2, dev_coef(ctx), s));
  return rmw_pass(ctx, h_layers, n, seed, 0.f, dev_coef(ctx), true, s);
}

agzo_status agzo_ghat(agzo_ctx* ctx, const double* d_f_plus, const double* d_f_other, float eps,
                      int mode, float* d_ghat, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (!d_f_plus || !d_f_other || !d_ghat || !(eps > 0.f) || (mode != 0 && mode != 1))
    return AGZO_ERR_INVALID_ARG;
  ctx->launches += 1;
  CU(ctx, launch_ghat(d_f_plus, d_f_other, eps, mode, d_ghat, static_cast<cudaStream_t>(stream)));
  return AGZO_OK;
}

agzo_status agzo_restore_update(agzo_ctx* ctx, const agzo_layer* h_layers, int n, uint64_t seed,
                                float eps, float lr, int mode, const float* d_ghat, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (!d_ghat || (mode != 0 && mode != 1)) return AGZO_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = validate(h_layers, n, NEED_RMW);
  if (st != AGZO_OK) return st;
  if (n == 0) return AGZO_OK;
  bool any_pair = false, any_plain = false;
  for (int i = 0; i < n; ++i) (h_layers[i].W16 ? any_pair : any_plain) = true;
  if (any_pair && any_plain) return AGZO_ERR_UNSUPPORTED;
  // a pair's master was never perturbed: only the update term applies to it
  ctx->launches += 1;
  CU(ctx, launch_coef(d_ghat, eps, lr, any_pair ? 2 : mode, dev_coef(ctx), s));
  return rmw_pass(ctx, h_layers, n, seed, 0.f, dev_coef(ctx), true, s);
}

agzo_status agzo_step(agzo_ctx* ctx, const agzo_layer* h_layers, int n, const agzo_params* p,
                      agzo_loss_fn loss, void* user, double* d_losses2, float* d_ghat,
                      void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (!p || !loss || !d_losses2 || !d_ghat || !(p->eps > 0.f) || (p->mode != 0 && p->mode != 1) || p->K < 0 ||
      p->K > 16)
    return AGZO_ERR_INVALID_ARG;
  st = validate(h_layers, n, NEED_RMW | NEED_EXTRACT);
  if (st != AGZO_OK) return st;
  bool any_pair = false, any_plain = false;
  for (int i = 0; i < n; ++i) (h_layers[i].W16 ? any_pair : any_plain) = true;
  if (any_pair && any_plain) return AGZO_ERR_UNSUPPORTED;
  double* d_fplus = d_losses2;
  double* d_fother = d_losses2 + 1;
  float* d_g = d_ghat;

  // The library knows where the weights sit at every moment: W0 + outstanding * Delta.  Whatever
  // fails after the first pass -- the callback or one of the library's own calls -- the inverse of
  // the outstanding perturbation is applied before the error is returned.
  float outstanding = 0.f;
  int call = 0;     // internal calls of this step, counted for the host-side fault injection of the tests
  auto injected = [&]() { return ++call == ctx->debug_fail_step_call; };
  auto fail = [&](agzo_status why) {
    if (outstanding != 0.f) agzo_restore(ctx, h_layers, n, p->seed, outstanding, stream);
    return why;
  };

  // step 1: unperturbed forward (fills X), then Algorithm 1 per layer
  if (loss(user, stream, 0, d_fother) != 0) return AGZO_ERR_CALLBACK;
  st = injected() ? AGZO_ERR_CUDA : agzo_extract_subspace(ctx, h_layers, n, p->seed, p->K, stream);
  if (st != AGZO_OK) return st;
  // step 2: W + eps*Delta
  st = injected() ? AGZO_ERR_CUDA : agzo_perturb(ctx, h_layers, n, p->seed, p->eps, stream);
  if (st != AGZO_OK) return st;
  outstanding = p->eps;
  if (loss(user, stream, 1, d_fplus) != 0) return fail(AGZO_ERR_CALLBACK);
  if (p->mode == 0) {
    // a pair is always rebuilt from the untouched master, so its flip is -eps, not -2 eps
    st = injected() ? AGZO_ERR_CUDA
                    : agzo_perturb(ctx, h_layers, n, p->seed, any_pair ? -p->eps : -2.0f * p->eps, stream);
    if (st != AGZO_OK) return fail(st);
    outstanding = -p->eps;
    if (loss(user, stream, 2, d_fother) != 0) return fail(AGZO_ERR_CALLBACK);
  }
  st = injected() ? AGZO_ERR_CUDA : agzo_ghat(ctx, d_fplus, d_fother, p->eps, p->mode, d_g, stream);
  if (st != AGZO_OK) return fail(st);
  // step 3: restore and update in one pass
  st = injected() ? AGZO_ERR_CUDA
                  : agzo_restore_update(ctx, h_layers, n, p->seed, p->eps, p->lr, p->mode, d_g, stream);
  if (st != AGZO_OK) return fail(st);
  return AGZO_OK;
}

agzo_status agzo_fill_gaussian_basis(agzo_ctx* ctx, const agzo_layer* h_layers, int n, uint64_t seed,
                                     void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  st = validate(h_layers, n, 0);
  if (st != AGZO_OK) return st;
  if (n == 0) return AGZO_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  st = prepare(ctx, h_layers, n, s);
  if (st != AGZO_OK) return st;
  int max_elems = 0;
  for (int i = 0; i < n; ++i) max_elems = std::max(max_elems, h_layers[i].r * h_layers[i].d_in);
  ctx->launches += 1;
  CU(ctx, launch_fill_basis(dev_layers(ctx), n, max_elems, seed, s));
  return AGZO_OK;
}

agzo_status agzo_perturb_dense(agzo_ctx* ctx, void* w, int64_t n_elems, int dtype, uint64_t seed,
                               uint32_t layer_id, float scale, const float* d_scale, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (n_elems < 0 || (n_elems > 0 && !w)) return AGZO_ERR_INVALID_ARG;
  if (dtype != AGZO_BF16 && dtype != AGZO_F32) return AGZO_ERR_UNSUPPORTED;
  ctx->launches += 1;
  CU(ctx, launch_dense(w, n_elems, dtype, seed, layer_id, scale, d_scale, ctx->sm_count,
                       static_cast<cudaStream_t>(stream)));
  return AGZO_OK;
}

agzo_status agzo_debug_philox(agzo_ctx* ctx, uint64_t seed, uint32_t layer_id, uint32_t tag,
                              uint64_t first, uint64_t n, uint32_t* d_words, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (n > 0 && !d_words) return AGZO_ERR_INVALID_ARG;
  CU(ctx, launch_debug_philox(seed, layer_id, tag, first, n, d_words, ctx->sm_count, static_cast<cudaStream_t>(stream)));
  return AGZO_OK;
}

agzo_status agzo_debug_gaussian(agzo_ctx* ctx, uint64_t seed, uint32_t layer_id, uint32_t tag,
                                uint64_t first, uint64_t n, float* d_vals, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (n > 0 && !d_vals) return AGZO_ERR_INVALID_ARG;
  CU(ctx, launch_debug_gauss(seed, layer_id, tag, first, n, d_vals, ctx->sm_count, static_cast<cudaStream_t>(stream)));
  return AGZO_OK;
}

agzo_status agzo_debug_fused_split(const int32_t* h_tiles, int n, int clusters, int32_t* h_tile0, int32_t* h_first,
                                   int32_t* h_parts, int32_t* h_share_begin, int32_t* h_shares) {
  if (n < 0 || clusters < 1 || (n > 0 && (!h_tiles || !h_tile0 || !h_first || !h_parts)) || !h_share_begin || !h_shares)
    return AGZO_ERR_INVALID_ARG;
  long long total = 0;
  for (int i = 0; i < n; ++i) {
    if (h_tiles[i] < 0) return AGZO_ERR_INVALID_ARG;
    total += h_tiles[i];
  }
  if (total > (1ll << 30)) return AGZO_ERR_INVALID_ARG;
  int base = 0, rem = 0;
  const int G = fused_split(h_tiles, n, clusters, h_tile0, h_first, h_parts, &base, &rem);
  for (int k = 0; k <= G; ++k) h_share_begin[k] = fused_share_begin(k, base, rem);
  *h_shares = G;
  return AGZO_OK;
}

agzo_status agzo_debug_wait_timeout(agzo_ctx* ctx, void* stream) {
  agzo_status st = check_ctx(ctx);
  if (st != AGZO_OK) return st;
  if (!ctx->tc.available) return AGZO_ERR_UNSUPPORTED;
  CU(ctx, launch_debug_wait(dev_status(ctx), static_cast<cudaStream_t>(stream)));
  return AGZO_OK;
}

}  // extern "C"
