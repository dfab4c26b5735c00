// bf16 head: instantiations of the tensor-core projection kernel (one CTA per worker for
// n <= 128, a pair of CTAs above), their shared-memory configuration and launch, and the host
// view of the schedule the kernel walks.
#include <cuda.h>
#include <cuda_bf16.h>

#include "tlr_common.cuh"
#include "tlr_tc.cuh"
#include "tlr_tc_kernel.cuh"

namespace tlr {

int tc_threads() { return kThreads; }

// Host enumeration of the schedule the kernel walks (the same tile_of the device code uses):
// one record {worker, unit, row0, v0, rows} per non-empty tile of CTA rank 0, in walking order.
// Tiles of learned-router units are reported with v0 counted from V upwards.
int tc_enumerate_tiles(const TcParams& p, int cta, int workers, int* out, int capacity) {
  int count = 0;
  const int units = (p.chunks + (p.mlp_hidden > 0 ? 1 : 0)) * p.row_units;
  for (int w = 0; w < workers; ++w) {
    for (int unit = w; unit < units; unit += workers) {
      const Unit un = cta == 2 ? unit_of<2>(p, unit, 0) : unit_of<1>(p, unit, 0);
      for (int t = 0; t < p.tiles_per_unit; ++t) {
        const Tile tl = tile_of(p, un, t);
        if (tl.rows == 0) continue;
        if (count < capacity) {
          int* r = out + 5 * count;
          r[0] = w;
          r[1] = unit;
          r[2] = un.row0;
          r[3] = un.chunk < 0 ? p.V + tl.v0 : tl.v0;
          r[4] = tl.rows;
        }
        ++count;
      }
    }
  }
  return count;
}

// Ring depths and shared-memory size for a given n.  The h ring is short (L2 latency),
// the W ring takes everything that is left (HBM latency).
void tc_configure(int n, TcConfig* c) {
  const int cta = n > kBlockM ? 2 : 1;
  int a_rows = kBlockM;
  if (cta == 1) {
    a_rows = ((n + 15) / 16) * 16;
    if (a_rows < 16) a_rows = 16;
    if (a_rows > kBlockM) a_rows = kBlockM;
  }
  const int a_stage = a_rows * kRowBytes;
  const int b_stage = (kBlockN / cta) * kRowBytes;
  // h slabs come from L2 (about a microsecond away under load) and one is consumed per W
  // slab, so the h ring needs about half the depth of the W ring to keep up.
  int sa = cta == 2 ? 4 : (a_rows <= 32 ? 6 : 4);
  const int budget = kSmemLimit - 1024 - kBarrierBytes - kScratchBytes;
  int sb = (budget - sa * a_stage) / b_stage;
  if (sb > kMaxBStages) sb = kMaxBStages;
  // Tuning override: TLR_TC_RINGS="<h stages>,<W stages>" (ignored if it does not fit).
  const Tuning& tn = tuning();
  if (tn.ring_a >= 1 && tn.ring_a <= kRelease && tn.ring_b >= 1 && tn.ring_b <= kMaxBStages &&
      tn.ring_a * a_stage + tn.ring_b * b_stage <= budget) {
    sa = tn.ring_a;
    sb = tn.ring_b;
  }
  c->cta = cta;
  c->a_rows = a_rows;
  c->part_rows = a_rows;
  c->a_stages = sa;
  c->b_stages = sb;
  c->inline_split = 0;
  c->smem_bytes = 1024 + sa * a_stage + sb * b_stage + kBarrierBytes + kScratchBytes;
}

cudaError_t tc_prepare() {
  cudaError_t e = cudaFuncSetAttribute(tc_projection_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kSmemLimit);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(tc_projection_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
}

cudaError_t launch_tc_projection(const TcMaps& maps, const TcParams& p, const TcConfig& c, int workers,
                                 cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(workers * c.cta), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = static_cast<size_t>(c.smem_bytes);
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  if (c.cta == 1) {
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tc_projection_kernel<1>, maps, p);
  }
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, tc_projection_kernel<2>, maps, p);
}

}  // namespace tlr
