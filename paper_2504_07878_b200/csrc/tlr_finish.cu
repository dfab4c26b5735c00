// Merge of the per-chunk partial results, the scores, the route decision and the
// ordered stream compaction of routed rows -- one launch.
//
// Phase 1 (all blocks): one warp per row folds that row's `chunks` partials with the
//   associative merge rule (lanes stride the partials, then a shuffle butterfly),
//   and lane 0 writes token, conf = 1/s, entropy = ln s - t/s and the route flag
//   conf < tau (Sec. 3.1 of the paper: routed when the score falls below the threshold).
// Phase 2 (the block that finishes last, found with a fence + ticket counter, no
//   spinning): ballot / popcount / prefix-sum compaction of the flags into the
//   ascending index list, and the count.
#include "tlr_common.cuh"

namespace tlr {

constexpr int kFinishWarps = 8;
constexpr int kFinishThreads = kFinishWarps * 32;

__global__ void __launch_bounds__(kFinishThreads)
finish_kernel(const FinishLaunch a) {
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * kFinishWarps + warp;
  // Programmatic dependent launch: let the next kernel in the stream be scheduled now (it
  // waits for this grid to complete before touching memory), then wait for the projection
  // kernel's partials.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (row < a.n) {
    const Partial* p = a.partials + (size_t)row * a.chunks;
    Partial acc = empty_partial();
    for (int j = lane; j < a.chunks; j += 32) {
      const float4 raw = __ldcg(reinterpret_cast<const float4*>(p + j));
      Partial q;
      q.m = raw.x;
      q.idx = __float_as_int(raw.y);
      q.s = raw.z;
      q.t = raw.w;
      acc = merge(acc, q);
    }
    acc = warp_merge(acc);
    if (lane == 0) {
      float conf = 1.0f / acc.s;
      float ent = logf(acc.s) - acc.t / acc.s;
      const bool finite = (conf == conf) && (ent == ent) && acc.s > 0.f && acc.s < INFINITY;
      if (finite) {
        conf = fminf(conf, 1.0f);
        ent = fmaxf(ent, 0.0f);
      } else {
        conf = __int_as_float(0x7fc00000);   // NaN: fails "conf >= tau", so the row is routed
        ent = conf;
        atomicOr(a.status, TLR_DEV_NONFINITE);
      }
      a.token[row] = acc.idx;
      a.conf[row] = conf;
      a.entropy[row] = ent;
      // "not (conf >= tau)": equals conf < tau for numbers, and routes a NaN row.
      a.route_mask[row] = (conf >= a.tau) ? 0 : 1;
    }
  }

  // ---- which block is last?
  __shared__ int is_last;
  __shared__ int warp_count[kFinishWarps];
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned int t = atomicAdd(a.ticket, 1u);
    is_last = (t == gridDim.x - 1) ? 1 : 0;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();

  // ---- ordered compaction by the last block
  int base_out = 0;
  for (int base = 0; base < a.n; base += kFinishThreads) {
    const int i = base + threadIdx.x;
    const int flag = (i < a.n) ? (int)__ldcg(a.route_mask + i) : 0;
    const unsigned int bal = __ballot_sync(0xffffffffu, flag != 0);
    if (lane == 0) warp_count[warp] = __popc(bal);
    __syncthreads();
    int before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < kFinishWarps; ++w) {
      const int c = warp_count[w];
      before += (w < warp) ? c : 0;
      total += c;
    }
    if (flag) a.routed_idx[base_out + before + __popc(bal & ((1u << lane) - 1u))] = i;
    base_out += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    *a.routed_count = base_out;
    *a.ticket = 0u;  // ready for the next call on this context
  }
}

cudaError_t launch_finish(const FinishLaunch& a, cudaStream_t stream) {
  const int blocks = a.n > 0 ? (a.n + kFinishWarps - 1) / kFinishWarps : 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
  cfg.blockDim = dim3(kFinishThreads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, finish_kernel, a);
}

}  // namespace tlr
