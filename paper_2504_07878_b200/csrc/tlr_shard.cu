// Vocabulary-sharded decode: each GPU holds a contiguous range of W's rows.
//
// A shard's projection kernel leaves chunk partials as usual; shard_summary_kernel folds them
// into ONE 16-byte summary per row whose token index is global (shard offset added).  The
// summaries of all shards are exchanged by the caller (an all-gather of n x 16 bytes per GPU)
// and shard_gather_kernel lays the gathered block [shards][n] out as partials [n][shards],
// which the ordinary merge kernel then scores, decides and compacts.  The merge of summaries
// is the same associative rule as the merge of chunk partials, so the sharded result differs
// from the one-GPU result only by fp32 summation order.
#include "tlr_common.cuh"

namespace tlr {

namespace {

constexpr int kWarps = 8;

// One warp per row: lanes stride the row's partials, then a shuffle butterfly.
__global__ void __launch_bounds__(kWarps * 32)
shard_summary_kernel(const Partial* __restrict__ partials, int n, int chunks, int v_offset,
                     Partial* __restrict__ summary) {
  const int row = blockIdx.x * kWarps + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= n) return;
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
  if (lane == 0) {
    if (acc.idx != kNoToken) acc.idx += v_offset;
    summary[row] = acc;
  }
}

__global__ void shard_gather_kernel(const Partial* __restrict__ gathered, int shards, int n,
                                    Partial* __restrict__ partials) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;   // index into [n][shards]
  if (i >= n * shards) return;
  const int row = i / shards, g = i - row * shards;
  partials[i] = gathered[static_cast<size_t>(g) * n + row];
}

}  // namespace

cudaError_t launch_shard_summary(const Partial* partials, int n, int chunks, int v_offset, Partial* summary,
                                 cudaStream_t stream) {
  if (n <= 0) return cudaSuccess;
  shard_summary_kernel<<<(n + kWarps - 1) / kWarps, kWarps * 32, 0, stream>>>(partials, n, chunks, v_offset, summary);
  return cudaGetLastError();
}

cudaError_t launch_shard_gather(const Partial* gathered, int shards, int n, Partial* partials, cudaStream_t stream) {
  if (n <= 0) return cudaSuccess;
  const int total = n * shards;
  shard_gather_kernel<<<(total + 255) / 256, 256, 0, stream>>>(gathered, shards, n, partials);
  return cudaGetLastError();
}

}  // namespace tlr
