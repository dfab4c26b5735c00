// tlr_route_static: the routing step for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc on the hot path, or at all: a
// serving process that has already handed every spare byte of HBM to its KV-cache
// pool (an allocation would fail, or would force the pool to shrink), a latency-bound
// decode loop that cannot absorb the device-wide synchronisation an allocation may
// imply, or a plug-in whose host forbids allocations inside its callbacks.  The
// regular entry points keep their scratch (the per-row partial results that the
// projection kernel writes and the merge kernel reads, plus a ticket counter) in a
// context created by tlr_create, which allocates.  This file offers the same step
// with that scratch in a fixed array that is part of the library image instead.
//
// The array lives in every GPU's memory from the moment the library is loaded on it
// until the process exits (about 3 MiB).  It is shared by every call and keeps the
// previous call's contents; the only part that must start at zero, the ticket
// counter, is cleared on the stream at the start of each call.  Two calls whose
// kernels overlap on the GPU (different streams, different host threads) race on it.
#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>

#include "tlr.h"
#include "tlr_common.cuh"
#include "tlr_tc.cuh"

namespace {

constexpr int kStaticMaxRows = TLR_STATIC_MAX_ROWS;
constexpr int kStaticMaxChunks = 192;
constexpr size_t kPartialBytes = static_cast<size_t>(kStaticMaxRows) * kStaticMaxChunks * sizeof(tlr::Partial);
constexpr size_t kTicketOffset = kPartialBytes;        // unsigned int
constexpr size_t kStatusOffset = kPartialBytes + 64;   // uint32_t, used when the caller passes no status word
constexpr size_t kScratchBytes = kPartialBytes + 256;

// The scratch itself.  In host code this name is only a handle for the runtime's symbol
// lookup, never a device address: the address is obtained per device below.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kMaxDevices = 64;
struct DeviceSetup {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_static_scratch on this device
  int sm_count = 0;
  bool tc_ready = false;
};
DeviceSetup g_setup[kMaxDevices];
EncodeTiledFn g_encode = nullptr;
std::mutex g_mutex;

// Once per device, with that device current.
tlr_status setup_device(int dev, DeviceSetup** out) {
  if (dev < 0 || dev >= kMaxDevices) return TLR_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceSetup& s = g_setup[dev];
  if (!s.ready) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return TLR_ERR_CUDA;
    if (prop.major != 10) return TLR_ERR_UNSUPPORTED;
    unsigned char* addr = nullptr;
    if (cudaGetSymbolAddress((void**)&addr, g_static_scratch) != cudaSuccess || addr == nullptr) {
      cudaGetLastError();
      return TLR_ERR_CUDA;
    }
    s.scratch = addr;
    s.sm_count = prop.multiProcessorCount;
    if (g_encode == nullptr) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult q;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
          q == cudaDriverEntryPointSuccess)
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    // The tensor-core kernel must be usable on such a device; if its set-up failed (a transient
    // error), nothing is recorded and the next call tries again.
    if (g_encode == nullptr || tlr::tc_prepare() != cudaSuccess) {
      cudaGetLastError();
      return TLR_ERR_CUDA;
    }
    s.tc_ready = true;
    s.ready = true;
  }
  *out = &s;
  return TLR_OK;
}

bool encode_map(CUtensorMap* map, const void* base, int rows, int cols, int box_rows) {
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
  const cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t elem[2] = {1u, 1u};
  return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

extern "C" tlr_status tlr_route_static(int32_t d, int32_t V, const void* W_bf16_dev, const void* h_bf16_dev,
                                       int32_t n, float tau, int32_t* token_dev, float* conf_dev, float* entropy_dev,
                                       uint8_t* route_mask_dev, int32_t* routed_idx_dev, int32_t* routed_count_dev,
                                       uint32_t* status_dev, void* cuda_stream) {
  if (d <= 0 || V <= 0 || n < 0 || W_bf16_dev == nullptr || routed_count_dev == nullptr) return TLR_ERR_ARG;
  if (n > kStaticMaxRows) return TLR_ERR_TOO_MANY_ROWS;   // the fixed scratch holds TLR_STATIC_MAX_ROWS rows
  if (static_cast<long long>(V) + 256 > 0x7fffffffll) return TLR_ERR_UNSUPPORTED;
  if (n > 0 && (h_bf16_dev == nullptr || token_dev == nullptr || conf_dev == nullptr || entropy_dev == nullptr ||
                route_mask_dev == nullptr || routed_idx_dev == nullptr))
    return TLR_ERR_ARG;
  if ((reinterpret_cast<uintptr_t>(W_bf16_dev) & 15u) != 0 ||
      (n > 0 && (reinterpret_cast<uintptr_t>(h_bf16_dev) & 15u) != 0))
    return TLR_ERR_ALIGN;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TLR_ERR_CUDA;
  DeviceSetup* s = nullptr;
  const tlr_status st = setup_device(dev, &s);
  if (st != TLR_OK) return st;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  tlr::Partial* partials = reinterpret_cast<tlr::Partial*>(s->scratch);
  unsigned int* ticket = reinterpret_cast<unsigned int*>(s->scratch + kTicketOffset);
  uint32_t* status = status_dev != nullptr ? status_dev : reinterpret_cast<uint32_t*>(s->scratch + kStatusOffset);

  int chunks = 1;
  tlr::TcConfig cfg;
  tlr::TcPlan tp = {};
  tlr::TcMaps maps;
  int workers = 0;
  const bool tc = d % 8 == 0;
  if (n > 0 && tc) {
    if (!s->tc_ready) return TLR_ERR_CUDA;   // no silent change of kernel
    tlr::tc_configure(n, &cfg);
    const int workers_max = s->sm_count / cfg.cta;
    tlr::tc_plan(n, V, cfg.cta, workers_max, kStaticMaxChunks, 0, &tp);
    chunks = tp.chunks;
    const int units = tp.chunks * tp.row_units;
    workers = units < workers_max ? units : workers_max;
    if (!encode_map(&maps.h, h_bf16_dev, n, d, cfg.a_rows) || !encode_map(&maps.w128, W_bf16_dev, V, d, 128) ||
        !encode_map(&maps.w64, W_bf16_dev, V, d, 64) || !encode_map(&maps.w16, W_bf16_dev, V, d, 16))
      return TLR_ERR_CUDA;
    maps.m128 = maps.w128;
    maps.m64 = maps.w64;
    maps.m16 = maps.w16;
  }

  // The ticket must start at zero; the partials are fully rewritten for the rows in use.  These two
  // clears are enqueued only once nothing on the host can fail any more except the launches themselves.
  if (cudaMemsetAsync(ticket, 0, sizeof(unsigned int), stream) != cudaSuccess) return TLR_ERR_CUDA;
  if (cudaMemsetAsync(status, 0, sizeof(uint32_t), stream) != cudaSuccess) return TLR_ERR_CUDA;

  if (n > 0) {
    if (tc) {
      tlr::TcParams p = {};
      p.n = n;
      p.d = d;
      p.V = V;
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
      // W is an argument of this call, so the kernel that precedes it in the stream may have written it:
      // the W producer waits for that kernel like every other warp does.
      p.w_wait = 1;
      p.partials = partials;
      p.status = status;
      if (tlr::launch_tc_projection(maps, p, cfg, workers, stream) != cudaSuccess) return TLR_ERR_CUDA;
    } else {
      int grid, block, smem;
      tlr::simt_plan(n, d, V, s->sm_count, &chunks, &grid, &block, &smem);
      tlr::SimtLaunch a;
      a.W = W_bf16_dev;
      a.h = h_bf16_dev;
      a.n = n;
      a.d = d;
      a.V = V;
      a.chunks = chunks;
      a.partials = partials;
      if (tlr::launch_simt_projection(a, stream) != cudaSuccess) return TLR_ERR_CUDA;
    }
  }

  tlr::FinishLaunch f = {};
  f.partials = partials;
  f.n = n;
  f.chunks = chunks;
  f.row_stride = chunks;
  f.chunk_stride = 1;
  f.tau = tau;
  f.mlp_partial = nullptr;
  f.mlp_blocks = 0;
  f.mlp_b2 = 0.f;
  f.decide_on_mlp = 0;
  f.mlp_score_out = nullptr;
  f.tau_rows = nullptr;
  f.route_above = 0;
  f.seq_len = 0;
  f.first_routed = nullptr;
  f.token = token_dev;
  f.conf = conf_dev;
  f.entropy = entropy_dev;
  f.route_mask = route_mask_dev;
  f.routed_idx = routed_idx_dev;
  f.routed_count = routed_count_dev;
  f.ticket = ticket;
  f.status = status;
  if (tlr::launch_finish(f, stream) != cudaSuccess) return TLR_ERR_CUDA;
  return TLR_OK;
}
