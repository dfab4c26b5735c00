// Shared device-side definitions of the routing kernels: the per-row partial result
// that the projection kernels emit and the rule that merges two of them.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "tlr.h"

namespace tlr {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr int kNoToken = 0x7fffffff;

// Online-softmax summary of one row over a range of the vocabulary:
//   m   = max logit in the range          idx = lowest vocabulary index attaining it
//   s   = sum exp(z - m)                  t   = sum exp(z - m) * (z - m)
// With the whole vocabulary folded in: conf = 1/s, entropy = ln s - t/s.
// An empty range is (m = -inf, idx = kNoToken, s = 0, t = 0).
struct __align__(16) Partial {
  float m;
  int idx;
  float s;
  float t;
};

__device__ __forceinline__ Partial empty_partial() {
  Partial p;
  p.m = -INFINITY;
  p.idx = kNoToken;
  p.s = 0.f;
  p.t = 0.f;
  return p;
}

// Associative and commutative merge; ties on m go to the lower vocabulary index.
__device__ __forceinline__ Partial merge(const Partial& a, const Partial& b) {
  Partial r;
  const bool a_wins = (a.m > b.m) || (a.m == b.m && a.idx <= b.idx);
  r.m = a_wins ? a.m : b.m;
  r.idx = a_wins ? a.idx : b.idx;
  // Rescale each side to the new maximum.  A side with s == 0 (an empty range) contributes
  // nothing: its m is -inf, which must not reach the arithmetic below.  A NaN sum is not
  // "empty": it goes through and poisons the result, which the final step then flags.
  float s = 0.f, t = 0.f;
  if (!(a.s == 0.f)) {
    const float da = a.m - r.m;  // <= 0
    const float ea = exp2f(da * kLog2e);
    s += a.s * ea;
    t += ea * (a.t + da * a.s);
  }
  if (!(b.s == 0.f)) {
    const float db = b.m - r.m;
    const float eb = exp2f(db * kLog2e);
    s += b.s * eb;
    t += eb * (b.t + db * b.s);
  }
  r.s = s;
  r.t = t;
  return r;
}

__device__ __forceinline__ Partial shfl_xor(const Partial& p, int lane_mask) {
  Partial r;
  r.m = __shfl_xor_sync(0xffffffffu, p.m, lane_mask);
  r.idx = __shfl_xor_sync(0xffffffffu, p.idx, lane_mask);
  r.s = __shfl_xor_sync(0xffffffffu, p.s, lane_mask);
  r.t = __shfl_xor_sync(0xffffffffu, p.t, lane_mask);
  return r;
}

__device__ __forceinline__ Partial warp_merge(Partial p) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) p = merge(p, shfl_xor(p, off));
  return p;
}

// Host-side launchers (one per .cu file).  All enqueue on `stream` and return the
// launch error, if any.
struct SimtLaunch {
  const void* W;
  const void* h;
  int n, d, V;
  int chunks;       // vocabulary chunks (partials per row)
  Partial* partials;  // [n][chunks]
};
cudaError_t launch_simt_projection(const SimtLaunch& a, cudaStream_t stream);
void simt_plan(int n, int d, int V, int sm_count, int* chunks, int* grid, int* block, int* smem);

struct FinishLaunch {
  const Partial* partials;  // partial j of row i at partials[i * row_stride + j * chunk_stride]
  int n, chunks;
  int row_stride, chunk_stride;   // [n][chunks]: (chunks, 1); a block gathered shard-major [shards][rows]: (1, rows)
  // optional: before reading the partials, wait until wait_flags[0 .. wait_count) all hold wait_value (flags that
  // other GPUs set after storing their summaries into this GPU's memory); bounded by wait_limit_ns, after which
  // TLR_DEV_WAIT_TIMEOUT is raised and the kernel goes on with what is there
  const uint32_t* wait_flags;
  int wait_count;
  uint32_t wait_value;
  unsigned long long wait_limit_ns;
  float tau;
  const float* mlp_partial;   // optional [n][mlp_blocks]: partial sums of the learned router's output layer
  int mlp_blocks;
  float mlp_b2;
  int decide_on_mlp;          // 1: the learned score is compared with tau instead of conf
  float* mlp_score_out;       // optional [n]: the learned score
  const float* tau_rows;    // optional per-row thresholds [n]
  int route_above;          // 0: route iff conf < tau; 1: route iff conf > tau
  int seq_len;              // > 0: also report the first routed position of every sequence
  int32_t* first_routed;    // [n / seq_len] when seq_len > 0
  int32_t* token;
  float* conf;
  float* entropy;
  uint8_t* route_mask;
  int32_t* routed_idx;
  int32_t* routed_count;
  unsigned int* ticket;     // zero before the launch; the kernel leaves it zero again
  uint32_t* status;
  uint32_t* status_copy;    // optional: receives the status word once every row is scored (host-mapped memory)
};
cudaError_t launch_finish(const FinishLaunch& a, cudaStream_t stream);

// Vocabulary-sharded decode (tlr_shard.cu): one summary per row from a shard's chunk partials,
// and the gathered summaries [shards][n] laid out as partials [n][shards].
cudaError_t launch_shard_summary(const Partial* partials, int n, int chunks, int v_offset, Partial* summary,
                                 cudaStream_t stream);
// Fused exchange: the summaries are stored straight into slot `rank` of every peer's exchange block and, once all
// rows are out, this rank's flag in every peer's flag array is set to `epoch` (peer stores only).
struct ShardPush {
  const Partial* partials;   // this shard's chunk partials [n][chunks]
  int n, chunks, v_offset;
  int shards;                // peers, this rank included
  Partial* const* peer_slot; // device array [shards]: where this rank's n summaries go on peer g
  uint32_t* const* peer_flag;  // device array [shards]: this rank's flag on peer g
  uint32_t epoch;
  unsigned int* ticket;      // zero before the launch; left zero
};
cudaError_t launch_shard_push(const ShardPush& a, cudaStream_t stream);
// Row-sharded batches: the ranks' routed-index lists (slot g = rank g's list, `cap` entries each, the first
// counts[g] valid) become one ascending list of global row numbers, idx + row_offset[g].
cudaError_t launch_rows_merge(const int32_t* gathered_idx, const int32_t* counts, const int32_t* row_offsets,
                              int ranks, int cap, int32_t* global_idx, int32_t* global_count, cudaStream_t stream);

// Copy of `bytes` (a multiple of 16) from host memory the device can read directly to device
// memory, done by a kernel so that the projection kernel behind it can be launched early.
cudaError_t launch_host_copy(const void* src_mapped, void* dst, size_t bytes, cudaStream_t stream);

struct MlpLaunch {
  const void* h;        // bf16 [n][d]
  const void* W1;       // bf16 [d_hidden][d]
  const float* b1;      // [d_hidden]
  const float* w2;      // [d_hidden]
  float b2;
  int n, d, d_hidden;
  float* partial;       // [n][mlp_hidden_blocks(d_hidden)] out
};
int mlp_hidden_blocks(int d_hidden);
cudaError_t launch_mlp_score(const MlpLaunch& a, cudaStream_t stream);

}  // namespace tlr
