// Sharded forms of the routing step (several GPUs, one process each).
//
// Vocabulary sharding (decode batches): each GPU holds a contiguous range of W's rows.  A shard's
// projection kernel leaves chunk partials as usual; they are folded into ONE 16-byte summary per row whose
// token index is global (shard offset added).  The summaries of all shards then reach every GPU in one of two
// ways, and the ordinary merge kernel scores, decides and compacts them (it reads the block of summaries,
// laid out [shards][rows], in place).  The merge of summaries is the same associative rule as the merge of
// chunk partials, so the sharded result differs from the one-GPU result only by fp32 summation order.
//   shard_summary_kernel  writes the summaries locally; the caller exchanges them (an all-gather of
//                         n x 16 bytes per GPU).
//   shard_push_kernel     the fused exchange: every summary is stored straight into this rank's slot of every
//                         peer's exchange block (plain peer stores; no peer loads, no multicast), and when
//                         the last block is done -- a system-wide fence after the stores -- this rank's flag on
//                         every peer is set to the call's epoch.  The peers' merge kernels wait on their own
//                         flags (bounded).
//
// Row sharding (prefill batches): every GPU routes its own rows; rows_merge_kernel turns the gathered
// per-rank index lists into one ascending list of global row numbers.
#include "tlr_common.cuh"

namespace tlr {

namespace {

constexpr int kWarps = 8;

// One warp folds one row's chunk partials; every lane ends with the result.
__device__ __forceinline__ Partial row_summary(const Partial* __restrict__ partials, int row, int chunks, int v_offset,
                                               int lane) {
  Partial acc = empty_partial();
  for (int j = lane; j < chunks; j += 32) {
    const float4 raw = __ldcg(reinterpret_cast<const float4*>(partials + static_cast<size_t>(row) * chunks + j));
    Partial q;
    q.m = raw.x;
    q.idx = __float_as_int(raw.y);
    q.s = raw.z;
    q.t = raw.w;
    acc = merge(acc, q);
  }
  acc = warp_merge(acc);
  if (acc.idx != kNoToken) acc.idx += v_offset;
  return acc;
}

__global__ void __launch_bounds__(kWarps * 32)
shard_summary_kernel(const Partial* __restrict__ partials, int n, int chunks, int v_offset,
                     Partial* __restrict__ summary) {
  const int row = blockIdx.x * kWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= n) return;
  const Partial acc = row_summary(partials, row, chunks, v_offset, lane);
  if (lane == 0) summary[row] = acc;
}

__global__ void __launch_bounds__(kWarps * 32)
shard_push_kernel(const ShardPush a) {
  const int row = blockIdx.x * kWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  // Programmatic dependent launch: scheduled while the projection kernel finishes, and the merge kernel behind
  // this one may be scheduled now; the partials are read only after the projection has completed.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (row < a.n) {
    const Partial acc = row_summary(a.partials, row, a.chunks, a.v_offset, lane);
    for (int g = lane; g < a.shards; g += 32) a.peer_slot[g][row] = acc;     // lane g stores to peer g
  }
  // every summary of this block is on its way; the last block to get here publishes the flags
  __threadfence_system();
  __shared__ int is_last;
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned int t = atomicAdd(a.ticket, 1u);
    is_last = (t == gridDim.x - 1) ? 1 : 0;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence_system();      // the other blocks' stores (fenced before their tickets) precede the flags
  for (int g = threadIdx.x; g < a.shards; g += blockDim.x) {
    uint32_t* f = a.peer_flag[g];
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(f), "r"(a.epoch) : "memory");
  }
  if (threadIdx.x == 0) *a.ticket = 0u;
}

// One block per rank: the rank's routed rows, shifted to global row numbers, go behind the lists of the
// ranks before it (counts are few, so every block adds them up itself).
__global__ void __launch_bounds__(256)
rows_merge_kernel(const int32_t* __restrict__ gathered_idx, const int32_t* __restrict__ counts,
                  const int32_t* __restrict__ row_offsets, int ranks, int cap, int32_t* __restrict__ global_idx,
                  int32_t* __restrict__ global_count) {
  const int g = blockIdx.x;
  int before = 0, total = 0;
  for (int r = 0; r < ranks; ++r) {
    const int c = counts[r];
    before += r < g ? c : 0;
    total += c;
  }
  const int mine = counts[g], off = row_offsets[g];
  for (int j = threadIdx.x; j < mine; j += blockDim.x)
    global_idx[before + j] = gathered_idx[static_cast<size_t>(g) * cap + j] + off;
  if (g == 0 && threadIdx.x == 0) *global_count = total;
}

}  // namespace

cudaError_t launch_shard_summary(const Partial* partials, int n, int chunks, int v_offset, Partial* summary,
                                 cudaStream_t stream) {
  if (n <= 0) return cudaSuccess;
  shard_summary_kernel<<<(n + kWarps - 1) / kWarps, kWarps * 32, 0, stream>>>(partials, n, chunks, v_offset, summary);
  return cudaGetLastError();
}

cudaError_t launch_shard_push(const ShardPush& a, cudaStream_t stream) {
  const int blocks = a.n > 0 ? (a.n + kWarps - 1) / kWarps : 1;   // n == 0 still publishes the flags
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
  cfg.blockDim = dim3(kWarps * 32, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, shard_push_kernel, a);
}

cudaError_t launch_rows_merge(const int32_t* gathered_idx, const int32_t* counts, const int32_t* row_offsets,
                              int ranks, int cap, int32_t* global_idx, int32_t* global_count, cudaStream_t stream) {
  rows_merge_kernel<<<ranks, 256, 0, stream>>>(gathered_idx, counts, row_offsets, ranks, cap, global_idx, global_count);
  return cudaGetLastError();
}

}  // namespace tlr
