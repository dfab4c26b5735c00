// C-ABI of the routing library: context, argument checks, launch planning, dispatch.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "tlr.h"
#include "tlr_common.cuh"
#include "tlr_tc.cuh"

namespace tlr {

constexpr int kMaxChunks = 192;       // upper bound on partials per row (sizes the workspace)
constexpr int kMaxTimedLaunches = 4096;

const Tuning& tuning() {
  static const Tuning t = [] {
    Tuning v = {};
    v.tc8_inline = 1;
    if (const char* e = getenv("TLR_TC_GRANULE")) v.granule = atoi(e);
    if (getenv("TLR_TC_EVEN_TILES") != nullptr) v.even_tiles = 1;
    if (const char* e = getenv("TLR_TC_RINGS")) {
      int a = 0, b = 0;
      if (sscanf(e, "%d,%d", &a, &b) == 2) {
        v.ring_a = a;
        v.ring_b = b;
      }
    }
    if (const char* e = getenv("TLR_TC8_INLINE")) v.tc8_inline = e[0] == '0' ? 0 : 1;
    if (const char* e = getenv("TLR_FINISH_THREADS")) v.finish_threads = atoi(e);
    if (getenv("TLR_TC_ROW_COST") != nullptr) v.row_cost = 1;
    return v;
  }();
  return t;
}

// Chooses the vocabulary decomposition: every unit gets the same number of tiles, and the
// number of chunks minimises the load of the busiest worker -- (waves of units) x (rows of the
// largest chunk + a fixed cost per tile) -- so that workers finish together.  With a learned
// router in the launch (mlp_hidden > 0) one more unit per row unit, over the rows of its first
// layer, follows the vocabulary units in the same round-robin order and is counted in the loads.
void tc_plan(int n, int V, int cta, int workers, int max_chunks, int mlp_hidden, TcPlan* plan) {
  int g = 16 * cta;
  {
    const int e = tuning().granule;   // tuning switch
    if (e >= g && e <= 256 && e % g == 0 && 256 % e == 0) g = e;
  }
  const int row_units = (n + 128 * cta - 1) / (128 * cta);
  const int granules = (V + g - 1) / g;
  const int mlp_rows = mlp_hidden > 0 ? ((mlp_hidden + 16 * cta - 1) / (16 * cta)) * (16 * cta) : 0;
  const long long mlp_tiles = (mlp_rows + 255) / 256;
  const long long mlp_cost = mlp_rows + 24 * mlp_tiles;
  int hi = granules < max_chunks ? granules : max_chunks;
  if (hi < 1) hi = 1;
  long long best_cost = -1, best_passes = 0;
  int best = 1, best_tiles = 1;
  for (int c = 1; c <= hi; ++c) {
    const long long gmax = (granules + c - 1) / c;
    const long long tiles = (gmax * g + 255) / 256;
    const long long units = 1ll * row_units * c;
    const long long unit_cost = gmax * g + 24 * tiles;
    // Pair mode: a tile costs a pass over all of h whatever its width (the pair MMA takes as long with 32
    // columns as with 256), so the busiest worker's TILE count is compared first and the row-based cost only
    // decides between plans with the same count.
    const bool by_passes = cta == 2 && !tuning().even_tiles && !tuning().row_cost;
    long long cost, passes = 0;
    if (mlp_rows == 0) {
      const long long waves = (units + workers - 1) / workers;
      cost = waves * unit_cost;
      passes = waves * tiles;
    } else {
      // worker w takes units w, w + workers, ...: vocabulary units first, then the row_units router units
      const long long full = units / workers, rem = units % workers;
      cost = 0;
      for (int w = 0; w < workers; ++w) {
        const long long nv = full + (w < rem ? 1 : 0);
        const long long j0 = ((w - rem) % workers + workers) % workers;   // first router unit of this worker
        const long long nm = j0 < row_units ? 1 + (row_units - 1 - j0) / workers : 0;
        const long long load = nv * unit_cost + nm * mlp_cost;
        if (load > cost) cost = load;
        if (nv * tiles + nm * mlp_tiles > passes) passes = nv * tiles + nm * mlp_tiles;
      }
    }
    if (!by_passes) passes = 0;
    if (best_cost < 0 || passes < best_passes || (passes == best_passes && cost < best_cost)) {
      best_cost = cost;
      best_passes = passes;
      best = c;
      best_tiles = static_cast<int>(tiles);
    }
  }
  plan->row_units = row_units;
  plan->chunks = best;
  plan->granule_rows = g;
  plan->granules = granules;
  plan->tiles_per_unit = best_tiles;
  plan->mlp_rows = mlp_rows;
  // How a unit's chunk is cut into tiles.  A tile costs a pass over all of h whatever its width,
  // so where the tensor pipe matters (pairs of CTAs, n > 128) the chunk is cut into full 256-row
  // tiles plus one remainder tile.  With one CTA per worker the path is HBM-bound and a narrow
  // remainder tile only lowers the bytes in flight, so the tiles are of equal size there.
  plan->full_tiles_first = 0;
  if (cta == 2 && !tuning().even_tiles) {   // (a tuning switch)
    const long long gmax = (granules + best - 1) / best;
    const long long full = 256 / g;
    plan->full_tiles_first = 1;
    plan->tiles_per_unit = static_cast<int>((gmax + full - 1) / full);
  }
  if (plan->tiles_per_unit < mlp_tiles) plan->tiles_per_unit = static_cast<int>(mlp_tiles);
}

}  // namespace tlr

using tlr::Partial;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct tlr_ctx {
  int device = 0;
  int sm_count = 0;
  int d = 0, V = 0, max_n = 0;
  const void* W = nullptr;
  tlr_path forced = TLR_PATH_AUTO;
  bool tc_ok = false;
  EncodeTiledFn encode = nullptr;
  CUtensorMap map_w128, map_w64, map_w16;

  Partial* partials = nullptr;
  unsigned int* ticket = nullptr;
  uint32_t* status = nullptr;

  // staging for tlr_route_host
  // One device block holds the six outputs of a call back to back, so that one copy brings
  // them all to a pinned host mirror: token[n] conf[n] entropy[n] routed_idx[n] count mask[n].
  // Two slots, so that two host calls can be in flight (tlr_route_host_submit / _collect): slot s is used by
  // every second call.
  void* h_stage[2] = {nullptr, nullptr};
  unsigned char* out_stage[2] = {nullptr, nullptr};    // device, 17 * max_n + 8 bytes
  unsigned char* out_pinned[2] = {nullptr, nullptr};   // pinned host mirror of the same size, + an aligned 4-byte status word
  unsigned char* out_mapped[2] = {nullptr, nullptr};   // the mirror as the device sees it (kernels write the results into it), or null
  cudaEvent_t slot_done[2] = {nullptr, nullptr};       // recorded behind a submitted call's last kernel
  cudaStream_t copy_stream = nullptr;                  // large pinned h: copy-engine transfer beside the previous call's kernels
  cudaEvent_t copy_done[2] = {nullptr, nullptr};       // ... and the event the call's own stream waits for
  int slot_n[2] = {0, 0};
  int slot_next = 0;        // slot of the next submit
  int slots_in_flight = 0;  // submitted and not yet collected (0..2); the oldest is slot (slot_next - in_flight) & 1

  // learned router (tlr_set_router_mlp)
  int mlp_hidden = 0;
  const void* mlp_W1 = nullptr;
  const float* mlp_b1 = nullptr;
  const float* mlp_w2 = nullptr;
  float mlp_b2 = 0.f;
  float* mlp_scores = nullptr;     // [max_n][hidden blocks] partial sums of the output layer
  int mlp_blocks_cap = 0;

  // fp8 copy of W (tlr_create_fp8): e4m3 codes, one scale per row; h is split into two e4m3 parts per call
  bool fp8 = false;
  const float* wscale = nullptr;
  uint8_t* h_parts = nullptr;     // [2][tc8_max_rows()][d]
  float* hscale = nullptr;        // [tc8_max_rows()]

  // test hook (tlr_debug_inject)
  int debug_kind = 0;
  unsigned long long debug_wait_ns = 0;

  bool timing = false;
  std::vector<cudaEvent_t> events;   // pairs, created lazily
  int timed = 0;

  // Everything a call needs that depends only on (n, learned router in the launch or not): planned once
  // and kept, so that a repeated call does no planning, reads no environment variable and -- when h sits
  // at the same address as last time -- encodes no tensor map.
  struct Step {
    int n = -1;
    bool mlp = false;
    tlr_plan plan;
    tlr::TcConfig cfg;
    tlr::TcParams params;     // all but the per-call fields
    tlr::TcMaps maps;
    const void* h_mapped = nullptr;   // the address maps.h was encoded for
    const void* h_other = nullptr;    // ... and the address before that, with its map (two staging buffers alternate)
    CUtensorMap h_other_map;
    int workers = 0;
  };
  static constexpr int kSteps = 8;
  Step steps[kSteps];
  int next_step = 0;
  // vocabulary-sharded step with the fused exchange (tlr_shard_attach): pointer tables on the device, one per
  // parity of the call's epoch -- where this rank's summaries and flag go on every peer -- and this GPU's own block
  int shard_rank = -1, shard_count = 0;
  uint32_t shard_epoch = 0;
  Partial** peer_slot[2] = {nullptr, nullptr};
  uint32_t** peer_flag[2] = {nullptr, nullptr};
  unsigned char* my_block = nullptr;
  // learned router inside the projection launch: tensor maps over W1 (needs d % 8 == 0 and an aligned W1)
  bool mlp_fused = false;
  CUtensorMap map_m128, map_m64, map_m16;
};

namespace {

// Rows of `cols` e4m3 bytes, boxes of 128 bytes x box_rows, 128-byte swizzle.
bool make_map8(tlr_ctx* c, CUtensorMap* map, const void* base, int rows, int cols, int box_rows) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols)};
  const cuuint32_t box[2] = {128u, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem[2] = {1u, 1u};
  const CUresult r = c->encode(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box,
                               elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool make_map(tlr_ctx* c, CUtensorMap* map, const void* base, int rows, int cols, int box_rows) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
  const cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem[2] = {1u, 1u};
  const CUresult r = c->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
                               elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

tlr_path pick_path(const tlr_ctx* c) {
  if (c->forced == TLR_PATH_SIMT) return TLR_PATH_SIMT;
  return c->tc_ok ? TLR_PATH_TC : TLR_PATH_SIMT;
}

void forget_steps(tlr_ctx* c) {
  for (auto& st : c->steps) st.n = -1;
}

// Plans a call of n rows (with or without the learned router inside the projection launch).
void plan_step(const tlr_ctx* c, int n, bool mlp, tlr_ctx::Step* st) {
  const tlr_path path = pick_path(c);
  tlr_plan* out = &st->plan;
  st->n = n;
  st->mlp = mlp;
  st->h_mapped = nullptr;
  st->h_other = nullptr;
  st->workers = 0;
  out->path = path;
  out->launches = n > 0 ? 2 : 1;
  out->reserved = 0;
  tlr::TcParams& p = st->params;
  p = tlr::TcParams{};
  if (c->fp8 || path == TLR_PATH_TC) {
    tlr::TcConfig& cfg = st->cfg;
    tlr::TcPlan tp;
    int workers_max;
    if (c->fp8) {
      tlr::tc8_configure(n <= tlr::tc8_max_rows() ? n : tlr::tc8_max_rows(), c->d, &cfg);
      workers_max = c->sm_count;
      tlr::tc_plan(n <= 128 ? n : 128, c->V, 1, workers_max, tlr::kMaxChunks, 0, &tp);
      out->launches = n > 0 ? (cfg.inline_split ? 2 : 3) : 1;
    } else {
      tlr::tc_configure(n, &cfg);
      workers_max = c->sm_count / cfg.cta;
      tlr::tc_plan(n, c->V, cfg.cta, workers_max, tlr::kMaxChunks, mlp ? c->mlp_hidden : 0, &tp);
    }
    const int units = (tp.chunks + (tp.mlp_rows > 0 ? 1 : 0)) * tp.row_units;
    st->workers = units < workers_max ? units : workers_max;
    out->vocab_chunks = tp.chunks;
    out->row_units = tp.row_units;
    out->grid = st->workers * cfg.cta;
    out->block = tlr::tc_threads();
    out->smem_bytes = cfg.smem_bytes;
    p.n = n;
    p.d = c->d;
    p.V = c->V;
    p.row_units = tp.row_units;
    p.chunks = tp.chunks;
    p.granules = tp.granules;
    p.tiles_per_unit = tp.tiles_per_unit;
    p.full_tiles_first = tp.full_tiles_first;
    p.granule_rows = tp.granule_rows;
    p.a_rows = cfg.a_rows;
    p.part_rows = cfg.part_rows;
    p.a_stages = cfg.a_stages;
    p.b_stages = cfg.b_stages;
    p.wait_limit_ns = c->debug_wait_ns;
    p.debug_drop_w_copies = c->debug_kind == 1 ? 1 : 0;
    p.w_wait = 0;
    p.mlp_hidden = tp.mlp_rows > 0 ? c->mlp_hidden : 0;
    p.mlp_rows = tp.mlp_rows;
    p.mlp_b1 = c->mlp_b1;
    p.mlp_w2 = c->mlp_w2;
    p.mlp_out = c->mlp_scores;
    p.inline_split = cfg.inline_split;
    p.hscale = c->hscale;
    p.wscale = c->wscale;
    p.partials = c->partials;
    p.status = c->status;
    st->maps.w128 = c->map_w128;
    st->maps.w64 = c->map_w64;
    st->maps.w16 = c->map_w16;
    st->maps.m128 = mlp ? c->map_m128 : c->map_w128;
    st->maps.m64 = mlp ? c->map_m64 : c->map_w64;
    st->maps.m16 = mlp ? c->map_m16 : c->map_w16;
  } else {
    int chunks, grid, block, smem;
    tlr::simt_plan(n, c->d, c->V, c->sm_count, &chunks, &grid, &block, &smem);
    out->vocab_chunks = chunks;
    out->row_units = (n + 7) / 8;
    out->grid = grid;
    out->block = block;
    out->smem_bytes = smem;
  }
}

// The kept plan of (n, mlp), planned now if it is not there (the oldest slot is reused).
tlr_ctx::Step* step_for(tlr_ctx* c, int n, bool mlp) {
  for (auto& st : c->steps)
    if (st.n == n && st.mlp == mlp) return &st;
  tlr_ctx::Step* st = &c->steps[c->next_step];
  c->next_step = (c->next_step + 1) % tlr_ctx::kSteps;
  plan_step(c, n, mlp, st);
  return st;
}

void free_all(tlr_ctx* c) {
  cudaFree(c->partials);
  cudaFree(c->ticket);
  cudaFree(c->status);
  for (int q = 0; q < 2; ++q) {
    cudaFree(c->h_stage[q]);
    cudaFree(c->out_stage[q]);
    cudaFreeHost(c->out_pinned[q]);
    if (c->slot_done[q] != nullptr) cudaEventDestroy(c->slot_done[q]);
    if (c->copy_done[q] != nullptr) cudaEventDestroy(c->copy_done[q]);
  }
  if (c->copy_stream != nullptr) cudaStreamDestroy(c->copy_stream);
  cudaFree(c->mlp_scores);
  cudaFree(c->h_parts);
  cudaFree(c->hscale);
  for (int q = 0; q < 2; ++q) {
    cudaFree(c->peer_slot[q]);
    cudaFree(c->peer_flag[q]);
  }
  for (cudaEvent_t e : c->events) cudaEventDestroy(e);
  delete c;
}

// What both kinds of context share: the device check, the workspace, the staging buffers of
// tlr_route_host and the driver's tensor-map encoder (c->encode stays null if it cannot be had).
tlr_status new_context(int d, int V, const void* W_dev, int max_n, tlr_ctx** out) {
  if (static_cast<long long>(V) + 256 > 0x7fffffffll) return TLR_ERR_UNSUPPORTED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TLR_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return TLR_ERR_CUDA;
  if (prop.major != 10) return TLR_ERR_UNSUPPORTED;   // the kernels are built for sm_100a only
  tlr_ctx* c = new (std::nothrow) tlr_ctx();
  if (c == nullptr) return TLR_ERR_NOMEM;
  c->device = dev;
  c->sm_count = prop.multiProcessorCount;
  c->d = d;
  c->V = V;
  c->max_n = max_n;
  c->W = W_dev;
  const size_t np = static_cast<size_t>(max_n);
  bool ok = true;
  ok = ok && cudaMalloc(&c->partials, np * tlr::kMaxChunks * sizeof(Partial)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->ticket, sizeof(unsigned int)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->status, sizeof(uint32_t)) == cudaSuccess;
  for (int q = 0; q < 2; ++q) {
    ok = ok && cudaMalloc(&c->h_stage[q], np * d * 2) == cudaSuccess;
    ok = ok && cudaMalloc(&c->out_stage[q], np * 17 + 8) == cudaSuccess;
    ok = ok && cudaHostAlloc(reinterpret_cast<void**>(&c->out_pinned[q]), np * 17 + 8 + 8, cudaHostAllocMapped) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->slot_done[q], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&c->copy_done[q], cudaEventDisableTiming) == cudaSuccess;
  }
  ok = ok && cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    free_all(c);
    return TLR_ERR_NOMEM;
  }
  for (int q = 0; q < 2; ++q) {
    if (cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->out_mapped[q]), c->out_pinned[q], 0) != cudaSuccess) {
      cudaGetLastError();
      c->out_mapped[q] = nullptr;   // tlr_route_host then stages the outputs in device memory and copies them
    }
  }
  if (cudaMemset(c->ticket, 0, sizeof(unsigned int)) != cudaSuccess ||
      cudaMemset(c->status, 0, sizeof(uint32_t)) != cudaSuccess) {
    free_all(c);
    return TLR_ERR_CUDA;
  }
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
      qres == cudaDriverEntryPointSuccess && fn != nullptr)
    c->encode = reinterpret_cast<EncodeTiledFn>(fn);
  cudaGetLastError();
  *out = c;
  return TLR_OK;
}

// Enqueues the projection kernel of a call with n > 0 rows: chunk partials into ctx->partials.
tlr_status launch_projection(tlr_ctx* ctx, const void* h_bf16_dev, int n, tlr_ctx::Step* st, cudaStream_t stream) {
  cudaEvent_t ev0 = nullptr, ev1 = nullptr;
  if (ctx->timing && ctx->timed < tlr::kMaxTimedLaunches) {
    const size_t need = 2 * static_cast<size_t>(ctx->timed + 1);
    while (ctx->events.size() < need) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return TLR_ERR_CUDA;
      ctx->events.push_back(e);
    }
    ev0 = ctx->events[2 * ctx->timed];
    ev1 = ctx->events[2 * ctx->timed + 1];
    if (cudaEventRecord(ev0, stream) != cudaSuccess) return TLR_ERR_CUDA;
  }
  cudaError_t e;
  if (ctx->fp8) {
    const tlr::TcConfig& cfg = st->cfg;
    if (!cfg.inline_split &&
        tlr::launch_h_split(h_bf16_dev, n, ctx->d, cfg.part_rows, ctx->h_parts, ctx->hscale, stream) != cudaSuccess)
      return TLR_ERR_CUDA;
    if (st->h_mapped != ctx->h_parts) {      // the two parts stacked: one box is the whole operand slab
      if (!make_map8(ctx, &st->maps.h, ctx->h_parts, cfg.a_rows, ctx->d, cfg.a_rows)) return TLR_ERR_CUDA;
      st->h_mapped = ctx->h_parts;
    }
    st->params.h = h_bf16_dev;
    e = tlr::launch_tc8_projection(st->maps, st->params, cfg, st->workers, stream);
  } else if (st->plan.path == TLR_PATH_TC) {
    if (st->h_mapped != h_bf16_dev) {
      // the map in use moves to the second place; if that one was made for this address, it comes back
      const void* was = st->h_mapped;
      const CUtensorMap was_map = st->maps.h;
      if (st->h_other == h_bf16_dev && h_bf16_dev != nullptr) {
        st->maps.h = st->h_other_map;
      } else if (!make_map(ctx, &st->maps.h, h_bf16_dev, n, ctx->d, st->cfg.a_rows)) {
        st->h_mapped = nullptr;
        return TLR_ERR_CUDA;
      }
      st->h_other = was;
      st->h_other_map = was_map;
      st->h_mapped = h_bf16_dev;
    }
    e = tlr::launch_tc_projection(st->maps, st->params, st->cfg, st->workers, stream);
  } else {
    tlr::SimtLaunch a;
    a.W = ctx->W;
    a.h = h_bf16_dev;
    a.n = n;
    a.d = ctx->d;
    a.V = ctx->V;
    a.chunks = st->plan.vocab_chunks;
    a.partials = ctx->partials;
    e = tlr::launch_simt_projection(a, stream);
  }
  if (e != cudaSuccess) return TLR_ERR_CUDA;
  if (ev1 != nullptr) {
    if (cudaEventRecord(ev1, stream) != cudaSuccess) return TLR_ERR_CUDA;
    ctx->timed += 1;
  }
  return TLR_OK;
}

}  // namespace

static tlr_status route_step(tlr_ctx* ctx, const void* h_bf16_dev, int32_t n, float tau, const tlr_route_options* opt,
                             int32_t* token_dev, float* conf_dev, float* entropy_dev, uint8_t* route_mask_dev,
                             int32_t* routed_idx_dev, int32_t* routed_count_dev, void* cuda_stream,
                             uint32_t* status_copy);

extern "C" {

const char* tlr_status_string(tlr_status s) {
  switch (s) {
    case TLR_OK: return "ok";
    case TLR_ERR_ARG: return "invalid argument";
    case TLR_ERR_ALIGN: return "pointer not 16-byte aligned";
    case TLR_ERR_UNSUPPORTED: return "unsupported device or shape";
    case TLR_ERR_CUDA: return "CUDA call failed";
    case TLR_ERR_NOMEM: return "device memory allocation failed";
    case TLR_ERR_TOO_MANY_ROWS: return "n exceeds max_n of the context";
    case TLR_ERR_DEVICE_STATUS: return "a kernel raised a device status flag";
  }
  return "unknown status";
}

tlr_status tlr_create(int32_t d, int32_t V, const void* W_bf16_dev, int32_t max_n, tlr_ctx** out) {
  if (out == nullptr) return TLR_ERR_ARG;
  *out = nullptr;
  if (d <= 0 || V <= 0 || max_n <= 0 || W_bf16_dev == nullptr) return TLR_ERR_ARG;
  if ((reinterpret_cast<uintptr_t>(W_bf16_dev) & 15u) != 0) return TLR_ERR_ALIGN;
  tlr_ctx* c = nullptr;
  const tlr_status st = new_context(d, V, W_bf16_dev, max_n, &c);
  if (st != TLR_OK) return st;

  // Tensor-core path: needs 16-byte row pitch for TMA, and the driver's tensor-map encoder.
  if (d % 8 == 0) {
    if (c->encode != nullptr && make_map(c, &c->map_w128, W_bf16_dev, V, d, 128) &&
        make_map(c, &c->map_w64, W_bf16_dev, V, d, 64) && make_map(c, &c->map_w16, W_bf16_dev, V, d, 16) &&
        tlr::tc_prepare() == cudaSuccess)
      c->tc_ok = true;
    cudaGetLastError();
    if (!c->tc_ok) {   // on an sm_100 device with d % 8 == 0 this must work; do not fall back silently
      free_all(c);
      return TLR_ERR_CUDA;
    }
  }
  *out = c;
  return TLR_OK;
}

tlr_status tlr_create_fp8(int32_t d, int32_t V, const void* W_e4m3_dev, const float* wscale_dev, int32_t max_n,
                          tlr_ctx** out) {
  if (out == nullptr) return TLR_ERR_ARG;
  *out = nullptr;
  if (d <= 0 || V <= 0 || max_n <= 0 || W_e4m3_dev == nullptr || wscale_dev == nullptr) return TLR_ERR_ARG;
  if ((reinterpret_cast<uintptr_t>(W_e4m3_dev) & 15u) != 0 || (reinterpret_cast<uintptr_t>(wscale_dev) & 3u) != 0)
    return TLR_ERR_ALIGN;
  if (d % 16 != 0) return TLR_ERR_UNSUPPORTED;         // rows of 8-bit W must be multiples of 16 bytes for TMA
  tlr_ctx* c = nullptr;
  const tlr_status st = new_context(d, V, W_e4m3_dev, max_n, &c);
  if (st != TLR_OK) return st;
  c->wscale = wscale_dev;
  c->fp8 = true;
  const size_t rows8 = static_cast<size_t>(tlr::tc8_max_rows());
  if (cudaMalloc(&c->h_parts, 2 * rows8 * d) != cudaSuccess || cudaMalloc(&c->hscale, rows8 * sizeof(float)) != cudaSuccess) {
    cudaGetLastError();
    free_all(c);
    return TLR_ERR_NOMEM;
  }
  if (c->encode != nullptr && make_map8(c, &c->map_w128, W_e4m3_dev, V, d, 128) &&
      make_map8(c, &c->map_w64, W_e4m3_dev, V, d, 64) && make_map8(c, &c->map_w16, W_e4m3_dev, V, d, 16) &&
      tlr::tc8_prepare() == cudaSuccess)
    c->tc_ok = true;
  cudaGetLastError();
  if (!c->tc_ok) {
    free_all(c);
    return TLR_ERR_CUDA;
  }
  *out = c;
  return TLR_OK;
}

tlr_status tlr_destroy(tlr_ctx* ctx) {
  if (ctx == nullptr) return TLR_OK;
  free_all(ctx);
  return TLR_OK;
}

tlr_status tlr_set_router_mlp(tlr_ctx* ctx, int32_t d_hidden, const void* W1_bf16_dev, const float* b1_dev,
                              const float* w2_dev, float b2) {
  if (ctx == nullptr || d_hidden <= 0 || W1_bf16_dev == nullptr || b1_dev == nullptr || w2_dev == nullptr)
    return TLR_ERR_ARG;
  const int blocks = tlr::mlp_hidden_blocks(d_hidden);
  if (ctx->mlp_scores == nullptr || blocks > ctx->mlp_blocks_cap) {
    cudaFree(ctx->mlp_scores);
    ctx->mlp_scores = nullptr;
    if (cudaMalloc(&ctx->mlp_scores, static_cast<size_t>(ctx->max_n) * blocks * sizeof(float)) != cudaSuccess) {
      cudaGetLastError();
      ctx->mlp_hidden = 0;
      ctx->mlp_fused = false;
      forget_steps(ctx);
      return TLR_ERR_NOMEM;
    }
    ctx->mlp_blocks_cap = blocks;
  }
  ctx->mlp_hidden = d_hidden;
  ctx->mlp_W1 = W1_bf16_dev;
  ctx->mlp_b1 = b1_dev;
  ctx->mlp_w2 = w2_dev;
  ctx->mlp_b2 = b2;
  // Where the tensor-core kernel runs, W1's rows are walked by that kernel as one more unit per row unit
  // (same staged h, same MMAs); that needs tensor maps over W1, i.e. 16-byte rows at a 16-byte aligned base.
  ctx->mlp_fused = false;
  if (ctx->tc_ok && !ctx->fp8 && ctx->d % 8 == 0 && (reinterpret_cast<uintptr_t>(W1_bf16_dev) & 15u) == 0 &&
      make_map(ctx, &ctx->map_m128, W1_bf16_dev, d_hidden, ctx->d, 128) &&
      make_map(ctx, &ctx->map_m64, W1_bf16_dev, d_hidden, ctx->d, 64) &&
      make_map(ctx, &ctx->map_m16, W1_bf16_dev, d_hidden, ctx->d, 16))
    ctx->mlp_fused = true;
  forget_steps(ctx);
  return TLR_OK;
}

tlr_status tlr_debug_plan_tiles(int32_t n, int32_t V, int32_t sm_count, int32_t mlp_hidden, int32_t* out,
                                int32_t capacity, int32_t* count, tlr_plan* plan_out) {
  if (n <= 0 || V <= 0 || sm_count < 2 || mlp_hidden < 0 || count == nullptr || capacity < 0 ||
      (capacity > 0 && out == nullptr))
    return TLR_ERR_ARG;
  tlr::TcConfig cfg;
  tlr::TcPlan tp;
  tlr::tc_configure(n, &cfg);
  const int workers_max = sm_count / cfg.cta;
  tlr::tc_plan(n, V, cfg.cta, workers_max, tlr::kMaxChunks, mlp_hidden, &tp);
  const int units = (tp.chunks + (tp.mlp_rows > 0 ? 1 : 0)) * tp.row_units;
  const int workers = units < workers_max ? units : workers_max;
  tlr::TcParams p = {};
  p.n = n;
  p.V = V;
  p.row_units = tp.row_units;
  p.chunks = tp.chunks;
  p.granules = tp.granules;
  p.tiles_per_unit = tp.tiles_per_unit;
  p.full_tiles_first = tp.full_tiles_first;
  p.granule_rows = tp.granule_rows;
  p.mlp_hidden = tp.mlp_rows > 0 ? mlp_hidden : 0;
  p.mlp_rows = tp.mlp_rows;
  *count = tlr::tc_enumerate_tiles(p, cfg.cta, workers, out, capacity);
  if (plan_out != nullptr) {
    plan_out->path = TLR_PATH_TC;
    plan_out->grid = workers * cfg.cta;
    plan_out->block = tlr::tc_threads();
    plan_out->row_units = tp.row_units;
    plan_out->vocab_chunks = tp.chunks;
    plan_out->smem_bytes = cfg.smem_bytes;
    plan_out->launches = 2;
    plan_out->reserved = tp.granule_rows;
  }
  return TLR_OK;
}

tlr_status tlr_debug_inject(tlr_ctx* ctx, int32_t kind, uint32_t wait_limit_ms) {
  if (ctx == nullptr || (kind != 0 && kind != 1)) return TLR_ERR_ARG;
  ctx->debug_kind = kind;
  ctx->debug_wait_ns = static_cast<unsigned long long>(wait_limit_ms) * 1000000ull;
  forget_steps(ctx);
  return TLR_OK;
}

tlr_status tlr_set_path(tlr_ctx* ctx, tlr_path path) {
  if (ctx == nullptr) return TLR_ERR_ARG;
  if (path != TLR_PATH_AUTO && path != TLR_PATH_SIMT && path != TLR_PATH_TC) return TLR_ERR_ARG;
  if (path == TLR_PATH_TC && !ctx->tc_ok) return TLR_ERR_UNSUPPORTED;
  if (path == TLR_PATH_SIMT && ctx->fp8) return TLR_ERR_UNSUPPORTED;
  ctx->forced = path;
  forget_steps(ctx);
  return TLR_OK;
}

tlr_status tlr_plan_query(tlr_ctx* ctx, int32_t n, tlr_plan* out) {
  if (ctx == nullptr || out == nullptr || n < 0) return TLR_ERR_ARG;
  if (n > ctx->max_n) return TLR_ERR_TOO_MANY_ROWS;
  *out = step_for(ctx, n, false)->plan;
  return TLR_OK;
}

tlr_status tlr_route(tlr_ctx* ctx, const void* h_bf16_dev, int32_t n, float tau, int32_t* token_dev, float* conf_dev,
                     float* entropy_dev, uint8_t* route_mask_dev, int32_t* routed_idx_dev, int32_t* routed_count_dev,
                     void* cuda_stream) {
  return tlr_route_ex(ctx, h_bf16_dev, n, tau, nullptr, token_dev, conf_dev, entropy_dev, route_mask_dev,
                      routed_idx_dev, routed_count_dev, cuda_stream);
}

tlr_status tlr_route_ex(tlr_ctx* ctx, const void* h_bf16_dev, int32_t n, float tau, const tlr_route_options* opt,
                        int32_t* token_dev, float* conf_dev, float* entropy_dev, uint8_t* route_mask_dev,
                        int32_t* routed_idx_dev, int32_t* routed_count_dev, void* cuda_stream) {
  return route_step(ctx, h_bf16_dev, n, tau, opt, token_dev, conf_dev, entropy_dev, route_mask_dev, routed_idx_dev,
                    routed_count_dev, cuda_stream, nullptr);
}

}  // extern "C"

// One routing step; status_copy (optional, device-visible) receives the status word after the last row.
static tlr_status route_step(tlr_ctx* ctx, const void* h_bf16_dev, int32_t n, float tau, const tlr_route_options* opt,
                             int32_t* token_dev, float* conf_dev, float* entropy_dev, uint8_t* route_mask_dev,
                             int32_t* routed_idx_dev, int32_t* routed_count_dev, void* cuda_stream,
                             uint32_t* status_copy) {
  if (ctx == nullptr || n < 0 || routed_count_dev == nullptr) return TLR_ERR_ARG;
  if (opt != nullptr && opt->seq_len > 0 && (n % opt->seq_len != 0 || opt->first_routed_dev == nullptr))
    return TLR_ERR_ARG;
  if (opt != nullptr && opt->seq_len < 0) return TLR_ERR_ARG;
  const bool want_mlp = opt != nullptr && (opt->score_source == TLR_SCORE_MLP || opt->mlp_score_dev != nullptr);
  if (opt != nullptr && opt->score_source != TLR_SCORE_CONF && opt->score_source != TLR_SCORE_MLP) return TLR_ERR_ARG;
  if (want_mlp && ctx->mlp_hidden == 0) return TLR_ERR_ARG;
  if (n > ctx->max_n) return TLR_ERR_TOO_MANY_ROWS;
  if (ctx->fp8 && n > tlr::tc8_max_rows()) return TLR_ERR_UNSUPPORTED;   // the fp8 copy serves decode batches only
  if (n > 0) {
    if (h_bf16_dev == nullptr || token_dev == nullptr || conf_dev == nullptr || entropy_dev == nullptr ||
        route_mask_dev == nullptr || routed_idx_dev == nullptr)
      return TLR_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(h_bf16_dev) & 15u) != 0) return TLR_ERR_ALIGN;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

  // the learned router runs inside the projection launch wherever the tensor-core kernel of the bf16 head runs
  const bool mlp_inside = want_mlp && ctx->mlp_fused && !ctx->fp8 && pick_path(ctx) == TLR_PATH_TC;
  tlr_ctx::Step* st = step_for(ctx, n, mlp_inside);
  const tlr_plan& plan = st->plan;

  if (n > 0) {
    const tlr_status ps = launch_projection(ctx, h_bf16_dev, n, st, stream);
    if (ps != TLR_OK) return ps;
  }

  if (want_mlp && !mlp_inside && n > 0) {
    tlr::MlpLaunch m;
    m.h = h_bf16_dev;
    m.W1 = ctx->mlp_W1;
    m.b1 = ctx->mlp_b1;
    m.w2 = ctx->mlp_w2;
    m.b2 = ctx->mlp_b2;
    m.n = n;
    m.d = ctx->d;
    m.d_hidden = ctx->mlp_hidden;
    m.partial = ctx->mlp_scores;
    if (tlr::launch_mlp_score(m, stream) != cudaSuccess) return TLR_ERR_CUDA;
  }

  tlr::FinishLaunch f = {};
  f.partials = ctx->partials;
  f.n = n;
  f.chunks = plan.vocab_chunks;
  f.row_stride = plan.vocab_chunks;
  f.chunk_stride = 1;
  f.tau = tau;
  f.mlp_partial = want_mlp ? ctx->mlp_scores : nullptr;
  f.mlp_blocks = want_mlp ? (mlp_inside ? 1 : tlr::mlp_hidden_blocks(ctx->mlp_hidden)) : 0;
  f.mlp_b2 = ctx->mlp_b2;
  f.decide_on_mlp = (opt != nullptr && opt->score_source == TLR_SCORE_MLP) ? 1 : 0;
  f.mlp_score_out = opt != nullptr ? opt->mlp_score_dev : nullptr;
  f.tau_rows = opt != nullptr ? opt->tau_per_row_dev : nullptr;
  f.route_above = (opt != nullptr && opt->route_above != 0) ? 1 : 0;
  f.seq_len = opt != nullptr ? opt->seq_len : 0;
  f.first_routed = opt != nullptr ? opt->first_routed_dev : nullptr;
  f.token = token_dev;
  f.conf = conf_dev;
  f.entropy = entropy_dev;
  f.route_mask = route_mask_dev;
  f.routed_idx = routed_idx_dev;
  f.routed_count = routed_count_dev;
  f.ticket = ctx->ticket;
  f.status = ctx->status;
  f.status_copy = status_copy;
  if (tlr::launch_finish(f, stream) != cudaSuccess) return TLR_ERR_CUDA;
  return TLR_OK;
}

extern "C" {

tlr_status tlr_shard_summary(tlr_ctx* ctx, const void* h_bf16_dev, int32_t n, int32_t v_offset, void* summary_dev,
                             void* cuda_stream) {
  if (ctx == nullptr || n < 0 || v_offset < 0) return TLR_ERR_ARG;
  if (n > ctx->max_n) return TLR_ERR_TOO_MANY_ROWS;
  if (n == 0) return TLR_OK;
  if (h_bf16_dev == nullptr || summary_dev == nullptr) return TLR_ERR_ARG;
  if ((reinterpret_cast<uintptr_t>(h_bf16_dev) & 15u) != 0 || (reinterpret_cast<uintptr_t>(summary_dev) & 15u) != 0)
    return TLR_ERR_ALIGN;
  if (static_cast<long long>(v_offset) + ctx->V + 256 > 0x7fffffffll) return TLR_ERR_UNSUPPORTED;
  if (ctx->fp8 && n > tlr::tc8_max_rows()) return TLR_ERR_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  tlr_ctx::Step* st = step_for(ctx, n, false);
  const tlr_plan& plan = st->plan;
  const tlr_status ps = launch_projection(ctx, h_bf16_dev, n, st, stream);
  if (ps != TLR_OK) return ps;
  if (tlr::launch_shard_summary(ctx->partials, n, plan.vocab_chunks, v_offset, static_cast<Partial*>(summary_dev),
                                stream) != cudaSuccess)
    return TLR_ERR_CUDA;
  return TLR_OK;
}

tlr_status tlr_shard_finish(tlr_ctx* ctx, const void* summaries_dev, int32_t shards, int32_t n, float tau,
                            int32_t* token_dev, float* conf_dev, float* entropy_dev, uint8_t* route_mask_dev,
                            int32_t* routed_idx_dev, int32_t* routed_count_dev, void* cuda_stream) {
  if (ctx == nullptr || n < 0 || routed_count_dev == nullptr || shards < 1 || shards > tlr::kMaxChunks)
    return TLR_ERR_ARG;
  if (n > ctx->max_n) return TLR_ERR_TOO_MANY_ROWS;
  if (n > 0) {
    if (summaries_dev == nullptr || token_dev == nullptr || conf_dev == nullptr || entropy_dev == nullptr ||
        route_mask_dev == nullptr || routed_idx_dev == nullptr)
      return TLR_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(summaries_dev) & 15u) != 0) return TLR_ERR_ALIGN;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  tlr::FinishLaunch f = {};
  f.partials = static_cast<const Partial*>(summaries_dev);   // read in place: summary of shard g, row i at [g * n + i]
  f.n = n;
  f.chunks = shards;
  f.row_stride = 1;
  f.chunk_stride = n;
  f.tau = tau;
  f.token = token_dev;
  f.conf = conf_dev;
  f.entropy = entropy_dev;
  f.route_mask = route_mask_dev;
  f.routed_idx = routed_idx_dev;
  f.routed_count = routed_count_dev;
  f.ticket = ctx->ticket;
  f.status = ctx->status;
  if (tlr::launch_finish(f, stream) != cudaSuccess) return TLR_ERR_CUDA;
  return TLR_OK;
}

// Layout of a GPU's exchange block for `shards` ranks and max_n rows: two sets (one per parity of the epoch) of
// `shards` flags, padded to 256 bytes, then two sets of `shards` slots of max_n summaries.
static size_t shard_header_bytes(int shards) { return (static_cast<size_t>(2) * shards * 4 + 255) & ~static_cast<size_t>(255); }

size_t tlr_shard_block_bytes(int32_t max_n, int32_t shards) {
  if (max_n <= 0 || shards <= 0) return 0;
  return shard_header_bytes(shards) + static_cast<size_t>(2) * shards * max_n * sizeof(Partial);
}

tlr_status tlr_debug_shard_table(int32_t max_n, int32_t rank, int32_t shards, void* const* peer_block_dev,
                                 int32_t parity, void** slot_out, void** flag_out) {
  if (max_n <= 0 || shards < 1 || rank < 0 || rank >= shards || peer_block_dev == nullptr || slot_out == nullptr ||
      flag_out == nullptr || (parity != 0 && parity != 1))
    return TLR_ERR_ARG;
  const size_t hdr = shard_header_bytes(shards);
  const size_t np = static_cast<size_t>(max_n);
  for (int g = 0; g < shards; ++g) {
    unsigned char* base = static_cast<unsigned char*>(peer_block_dev[g]);
    flag_out[g] = reinterpret_cast<uint32_t*>(base) + (static_cast<size_t>(parity) * shards + rank);
    slot_out[g] = reinterpret_cast<Partial*>(base + hdr) + (static_cast<size_t>(parity) * shards + rank) * np;
  }
  return TLR_OK;
}

tlr_status tlr_shard_attach(tlr_ctx* ctx, int32_t rank, int32_t shards, void* const* peer_block_dev) {
  if (ctx == nullptr || peer_block_dev == nullptr || shards < 1 || shards > tlr::kMaxChunks || rank < 0 ||
      rank >= shards)
    return TLR_ERR_ARG;
  for (int g = 0; g < shards; ++g) {
    if (peer_block_dev[g] == nullptr) return TLR_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(peer_block_dev[g]) & 255u) != 0) return TLR_ERR_ALIGN;
  }
  for (int q = 0; q < 2; ++q) {
    cudaFree(ctx->peer_slot[q]);
    cudaFree(ctx->peer_flag[q]);
    ctx->peer_slot[q] = nullptr;
    ctx->peer_flag[q] = nullptr;
    std::vector<Partial*> slots(shards);
    std::vector<uint32_t*> flags(shards);
    if (tlr_debug_shard_table(ctx->max_n, rank, shards, peer_block_dev, q, reinterpret_cast<void**>(slots.data()),
                              reinterpret_cast<void**>(flags.data())) != TLR_OK)
      return TLR_ERR_ARG;
    if (cudaMalloc(&ctx->peer_slot[q], shards * sizeof(Partial*)) != cudaSuccess ||
        cudaMalloc(&ctx->peer_flag[q], shards * sizeof(uint32_t*)) != cudaSuccess) {
      cudaGetLastError();
      ctx->shard_count = 0;
      return TLR_ERR_NOMEM;
    }
    if (cudaMemcpy(ctx->peer_slot[q], slots.data(), shards * sizeof(Partial*), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(ctx->peer_flag[q], flags.data(), shards * sizeof(uint32_t*), cudaMemcpyHostToDevice) != cudaSuccess) {
      ctx->shard_count = 0;
      return TLR_ERR_CUDA;
    }
  }
  ctx->shard_rank = rank;
  ctx->shard_count = shards;
  ctx->shard_epoch = 0;
  ctx->my_block = static_cast<unsigned char*>(peer_block_dev[rank]);
  return TLR_OK;
}

tlr_status tlr_shard_push(tlr_ctx* ctx, const void* h_bf16_dev, int32_t n, int32_t v_offset, void* cuda_stream) {
  if (ctx == nullptr || n < 0 || v_offset < 0 || ctx->shard_count == 0) return TLR_ERR_ARG;
  if (n > ctx->max_n) return TLR_ERR_TOO_MANY_ROWS;
  if (n > 0) {
    if (h_bf16_dev == nullptr) return TLR_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(h_bf16_dev) & 15u) != 0) return TLR_ERR_ALIGN;
  }
  if (static_cast<long long>(v_offset) + ctx->V + 256 > 0x7fffffffll) return TLR_ERR_UNSUPPORTED;
  if (ctx->fp8 && n > tlr::tc8_max_rows()) return TLR_ERR_UNSUPPORTED;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int chunks = 1;
  if (n > 0) {
    tlr_ctx::Step* st = step_for(ctx, n, false);
    chunks = st->plan.vocab_chunks;
    const tlr_status ps = launch_projection(ctx, h_bf16_dev, n, st, stream);
    if (ps != TLR_OK) return ps;
  }
  ctx->shard_epoch += 1;
  if (ctx->shard_epoch == 0) ctx->shard_epoch = 2;    // (wrapped: keep the parity sequence, never publish 0)
  const int q = static_cast<int>(ctx->shard_epoch & 1u);
  tlr::ShardPush a;
  a.partials = ctx->partials;
  a.n = n;
  a.chunks = chunks;
  a.v_offset = v_offset;
  a.shards = ctx->shard_count;
  a.peer_slot = ctx->peer_slot[q];
  a.peer_flag = ctx->peer_flag[q];
  a.epoch = ctx->shard_epoch;
  a.ticket = ctx->ticket;
  if (tlr::launch_shard_push(a, stream) != cudaSuccess) return TLR_ERR_CUDA;
  return TLR_OK;
}

tlr_status tlr_shard_finish_fused(tlr_ctx* ctx, int32_t n, float tau, int32_t* token_dev, float* conf_dev,
                                  float* entropy_dev, uint8_t* route_mask_dev, int32_t* routed_idx_dev,
                                  int32_t* routed_count_dev, void* cuda_stream) {
  if (ctx == nullptr || n < 0 || routed_count_dev == nullptr || ctx->shard_count == 0 || ctx->shard_epoch == 0)
    return TLR_ERR_ARG;
  if (n > ctx->max_n) return TLR_ERR_TOO_MANY_ROWS;
  if (n > 0 && (token_dev == nullptr || conf_dev == nullptr || entropy_dev == nullptr || route_mask_dev == nullptr ||
                routed_idx_dev == nullptr))
    return TLR_ERR_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const int q = static_cast<int>(ctx->shard_epoch & 1u);
  const int G = ctx->shard_count;
  const size_t np = static_cast<size_t>(ctx->max_n);
  tlr::FinishLaunch f = {};
  f.partials = reinterpret_cast<const Partial*>(ctx->my_block + shard_header_bytes(G)) + static_cast<size_t>(q) * G * np;
  f.n = n;
  f.chunks = G;
  f.row_stride = 1;
  f.chunk_stride = ctx->max_n;
  f.wait_flags = reinterpret_cast<const uint32_t*>(ctx->my_block) + static_cast<size_t>(q) * G;
  f.wait_count = G;
  f.wait_value = ctx->shard_epoch;
  f.wait_limit_ns = ctx->debug_wait_ns != 0 ? ctx->debug_wait_ns : 2000000000ull;
  f.tau = tau;
  f.token = token_dev;
  f.conf = conf_dev;
  f.entropy = entropy_dev;
  f.route_mask = route_mask_dev;
  f.routed_idx = routed_idx_dev;
  f.routed_count = routed_count_dev;
  f.ticket = ctx->ticket;
  f.status = ctx->status;
  if (tlr::launch_finish(f, stream) != cudaSuccess) return TLR_ERR_CUDA;
  return TLR_OK;
}

tlr_status tlr_rows_merge(const int32_t* gathered_idx_dev, const int32_t* counts_dev, const int32_t* row_offsets_dev,
                          int32_t ranks, int32_t cap, int32_t* global_idx_dev, int32_t* global_count_dev,
                          void* cuda_stream) {
  if (ranks < 1 || ranks > 65535 || cap < 0 || counts_dev == nullptr || row_offsets_dev == nullptr ||
      global_count_dev == nullptr || (cap > 0 && (gathered_idx_dev == nullptr || global_idx_dev == nullptr)))
    return TLR_ERR_ARG;
  if (tlr::launch_rows_merge(gathered_idx_dev, counts_dev, row_offsets_dev, ranks, cap, global_idx_dev,
                             global_count_dev, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
    return TLR_ERR_CUDA;
  return TLR_OK;
}

tlr_status tlr_route_host_submit(tlr_ctx* ctx, const void* h_bf16_host, int32_t n, float tau, void* cuda_stream) {
  if (ctx == nullptr || n < 0) return TLR_ERR_ARG;
  if (n > ctx->max_n) return TLR_ERR_TOO_MANY_ROWS;
  if (n > 0 && h_bf16_host == nullptr) return TLR_ERR_ARG;
  if (ctx->slots_in_flight >= 2) return TLR_ERR_ARG;     // collect one first
  const int q = ctx->slot_next;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const size_t nn = static_cast<size_t>(n);
  if (n > 0) {
    // h comes in by a copy kernel when the GPU can read the caller's buffer directly (pinned or
    // registered host memory): the projection kernel is then launched while h is still on its way
    // (see tlr_hostio.cu).  Pageable memory goes through the copy engine.
    const size_t bytes = nn * ctx->d * 2;
    cudaPointerAttributes attr;
    const void* mapped = nullptr;
    bool pinned = false;
    if (cudaPointerGetAttributes(&attr, h_bf16_host) == cudaSuccess && attr.type == cudaMemoryTypeHost) {
      pinned = true;
      mapped = attr.devicePointer;
    }
    cudaGetLastError();
    // Above a few MB the copy engine is faster than the copy kernel and there is nothing left to hide.
    const bool by_kernel = mapped != nullptr && bytes <= (4u << 20) && (bytes & 15u) == 0 &&
                           (reinterpret_cast<uintptr_t>(h_bf16_host) & 15u) == 0;
    if (by_kernel) {
      if (tlr::launch_host_copy(mapped, ctx->h_stage[q], bytes, stream) != cudaSuccess) return TLR_ERR_CUDA;
    } else if (pinned) {
      // A large pinned batch: the copy engine brings it in on the context's own stream, beside the kernels of
      // the call before it (this slot's last user has been collected, so its staging buffer is free), and the
      // call's stream waits for the transfer only.
      if (cudaMemcpyAsync(ctx->h_stage[q], h_bf16_host, bytes, cudaMemcpyHostToDevice, ctx->copy_stream) != cudaSuccess ||
          cudaEventRecord(ctx->copy_done[q], ctx->copy_stream) != cudaSuccess ||
          cudaStreamWaitEvent(stream, ctx->copy_done[q], 0) != cudaSuccess)
        return TLR_ERR_CUDA;
    } else if (cudaMemcpyAsync(ctx->h_stage[q], h_bf16_host, bytes, cudaMemcpyHostToDevice, stream) != cudaSuccess) {
      return TLR_ERR_CUDA;
    }
  }
  // layout of the output block for this n (all offsets are multiples of 4)
  const size_t off_conf = 4 * nn, off_ent = 8 * nn, off_idx = 12 * nn, off_count = 16 * nn, off_mask = 16 * nn + 4;
  const size_t out_bytes = 17 * nn + 4;
  unsigned char* pin = ctx->out_pinned[q];
  const size_t off_status = (static_cast<size_t>(ctx->max_n) * 17 + 8 + 3) & ~static_cast<size_t>(3);   // a 4-byte word
  uint32_t* pin_status = reinterpret_cast<uint32_t*>(pin + off_status);
  // The kernels write the six outputs and the status word straight into the pinned host block
  // (4 KB at n = 256); without a device view of it they go to device memory and are copied.
  const bool direct = ctx->out_mapped[q] != nullptr;
  unsigned char* dev = direct ? ctx->out_mapped[q] : ctx->out_stage[q];
  const tlr_status st = route_step(ctx, ctx->h_stage[q], n, tau, nullptr, reinterpret_cast<int32_t*>(dev),
                                   reinterpret_cast<float*>(dev + off_conf), reinterpret_cast<float*>(dev + off_ent),
                                   dev + off_mask, reinterpret_cast<int32_t*>(dev + off_idx),
                                   reinterpret_cast<int32_t*>(dev + off_count), cuda_stream,
                                   direct ? reinterpret_cast<uint32_t*>(dev + off_status) : nullptr);
  if (st != TLR_OK) return st;
  if (!direct && (cudaMemcpyAsync(pin, dev, out_bytes, cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
                  cudaMemcpyAsync(pin_status, ctx->status, 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess))
    return TLR_ERR_CUDA;
  if (cudaEventRecord(ctx->slot_done[q], stream) != cudaSuccess) return TLR_ERR_CUDA;
  ctx->slot_n[q] = n;
  ctx->slot_next = q ^ 1;
  ctx->slots_in_flight += 1;
  return TLR_OK;
}

tlr_status tlr_route_host_collect(tlr_ctx* ctx, int32_t* token_host, float* conf_host, float* entropy_host,
                                  uint8_t* route_mask_host, int32_t* routed_idx_host, int32_t* routed_count_host) {
  if (ctx == nullptr || routed_count_host == nullptr || ctx->slots_in_flight <= 0) return TLR_ERR_ARG;
  const int q = (ctx->slot_next - ctx->slots_in_flight) & 1;     // the oldest call in flight
  if (cudaEventSynchronize(ctx->slot_done[q]) != cudaSuccess) return TLR_ERR_CUDA;
  ctx->slots_in_flight -= 1;
  const size_t nn = static_cast<size_t>(ctx->slot_n[q]);
  const size_t off_conf = 4 * nn, off_ent = 8 * nn, off_idx = 12 * nn, off_count = 16 * nn, off_mask = 16 * nn + 4;
  const unsigned char* pin = ctx->out_pinned[q];
  const size_t off_status = (static_cast<size_t>(ctx->max_n) * 17 + 8 + 3) & ~static_cast<size_t>(3);
  int32_t count = 0;
  memcpy(&count, pin + off_count, 4);
  *routed_count_host = count;
  if (nn > 0) {
    if (token_host) memcpy(token_host, pin, 4 * nn);
    if (conf_host) memcpy(conf_host, pin + off_conf, 4 * nn);
    if (entropy_host) memcpy(entropy_host, pin + off_ent, 4 * nn);
    if (route_mask_host) memcpy(route_mask_host, pin + off_mask, nn);
    if (routed_idx_host && count > 0) memcpy(routed_idx_host, pin + off_idx, 4 * static_cast<size_t>(count));
  }
  uint32_t status = 0;
  memcpy(&status, pin + off_status, 4);
  if (status & TLR_DEV_WAIT_TIMEOUT) return TLR_ERR_DEVICE_STATUS;
  return TLR_OK;
}

tlr_status tlr_route_host(tlr_ctx* ctx, const void* h_bf16_host, int32_t n, float tau, int32_t* token_host,
                          float* conf_host, float* entropy_host, uint8_t* route_mask_host, int32_t* routed_idx_host,
                          int32_t* routed_count_host, void* cuda_stream) {
  if (ctx == nullptr || routed_count_host == nullptr) return TLR_ERR_ARG;
  if (ctx->slots_in_flight != 0) return TLR_ERR_ARG;     // not while submitted calls are waiting to be collected
  const tlr_status st = tlr_route_host_submit(ctx, h_bf16_host, n, tau, cuda_stream);
  if (st != TLR_OK) return st;
  return tlr_route_host_collect(ctx, token_host, conf_host, entropy_host, route_mask_host, routed_idx_host,
                                routed_count_host);
}

tlr_status tlr_last_device_status(tlr_ctx* ctx, uint32_t* out_host) {
  if (ctx == nullptr || out_host == nullptr) return TLR_ERR_ARG;
  if (cudaDeviceSynchronize() != cudaSuccess) return TLR_ERR_CUDA;
  if (cudaMemcpy(out_host, ctx->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return TLR_ERR_CUDA;
  if (cudaMemset(ctx->status, 0, 4) != cudaSuccess) return TLR_ERR_CUDA;
  return TLR_OK;
}

tlr_status tlr_set_kernel_timing(tlr_ctx* ctx, int32_t enabled) {
  if (ctx == nullptr) return TLR_ERR_ARG;
  ctx->timing = enabled != 0;
  return TLR_OK;
}

tlr_status tlr_read_kernel_timing(tlr_ctx* ctx, int32_t* launches_out, float* total_ms_out) {
  if (ctx == nullptr || launches_out == nullptr || total_ms_out == nullptr) return TLR_ERR_ARG;
  float total = 0.f;
  for (int i = 0; i < ctx->timed; ++i) {
    if (cudaEventSynchronize(ctx->events[2 * i + 1]) != cudaSuccess) return TLR_ERR_CUDA;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->events[2 * i], ctx->events[2 * i + 1]) != cudaSuccess) return TLR_ERR_CUDA;
    total += ms;
  }
  *launches_out = ctx->timed;
  *total_ms_out = total;
  ctx->timed = 0;
  return TLR_OK;
}

}  // extern "C"
