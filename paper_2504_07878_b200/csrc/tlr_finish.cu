// Merge of the per-chunk partial results, the scores, the route decision and the
// ordered stream compaction of routed rows -- one launch.
//
// Per row (a group of lanes, a whole warp for large n): lanes stride the row's partials; a shuffle butterfly finds the
// global maximum and its lowest index, each lane rescales its own partials to that
// maximum once, and a second butterfly adds the sums.  Lane 0 writes token,
// conf = 1/s, entropy = ln s - t/s and the route flag conf < tau (Sec. 3.1 of the
// paper: routed when the score falls below the threshold).
//
// Compaction (ballot / popcount / prefix sum, ascending order):
//   n <= 1024  a thread-block cluster of up to 8 blocks folds the rows (a group of L lanes
//              per row, all rows at once) and store the route flags into block 0's shared memory;
//              after a cluster barrier block 0 compacts them.  No ticket, no second launch, one L2
//              round trip for the partials.  The blocks
//              have 512 threads where a lane group still owns at most 6 partials (else 1024):
//              that size fits on an SM beside a CTA of the tensor-core projection kernel, so
//              the blocks are resident and waiting before that kernel ends, and the next
//              call's CTAs do not have to wait for the merge to leave their SMs.
//   larger n   many blocks of 8 warps; the block that finishes last (fence + ticket
//              counter, no spinning) compacts the flags of all rows.
#include "tlr_common.cuh"
#include "tlr_tc.cuh"

namespace tlr {

constexpr int kFinishWarps = 8;
constexpr int kFinishThreads = kFinishWarps * 32;
constexpr int kSmallThreads = 1024;
constexpr int kSmallRows = 1024;
constexpr int kPerLane = 6;            // ceil(192 / 32): the most partials a lane can own

// Folds one row's partials.  Every lane returns the same result.
__device__ __forceinline__ Partial fold_row(const Partial* __restrict__ p, int chunks, int chunk_stride, int lane) {
  Partial q[kPerLane];
  float m = -INFINITY;
  int idx = kNoToken;
#pragma unroll
  for (int k = 0; k < kPerLane; ++k) {
    const int j = lane + 32 * k;
    if (j < chunks) {
      const float4 raw = __ldcg(reinterpret_cast<const float4*>(p + static_cast<size_t>(j) * chunk_stride));
      q[k].m = raw.x;
      q[k].idx = __float_as_int(raw.y);
      q[k].s = raw.z;
      q[k].t = raw.w;
    } else {
      q[k] = empty_partial();
    }
    if (q[k].m > m || (q[k].m == m && q[k].idx < idx)) {
      m = q[k].m;
      idx = q[k].idx;
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, m, off);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, off);
    if (om > m || (om == m && oi < idx)) {
      m = om;
      idx = oi;
    }
  }
  float s = 0.f, t = 0.f;
#pragma unroll
  for (int k = 0; k < kPerLane; ++k) {
    if (!(q[k].s == 0.f)) {           // an empty range contributes nothing; a NaN sum goes through
      const float dm = q[k].m - m;    // <= 0
      const float e = exp2f(dm * kLog2e);
      s += q[k].s * e;
      t += e * (q[k].t + dm * q[k].s);
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, off);
    t += __shfl_xor_sync(0xffffffffu, t, off);
  }
  Partial r;
  r.m = m;
  r.idx = idx;
  r.s = s;
  r.t = t;
  return r;
}

// Scores and decision of one row from its folded summary; returns the route flag.
__device__ __forceinline__ int score_row(const Partial& acc, const FinishLaunch& a, int row) {
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
  // "not (conf >= tau)": equals conf < tau for numbers, and routes a NaN row; likewise
  // "not (conf <= tau)" for the opposite polarity.
  const float tau = a.tau_rows != nullptr ? a.tau_rows[row] : a.tau;
  float score = conf;
  if (a.mlp_partial != nullptr) {
    // learned score: the output layer's partial sums in a fixed order, then the sigmoid
    float v = a.mlp_b2;
    for (int b = 0; b < a.mlp_blocks; ++b) v += __ldcg(a.mlp_partial + static_cast<size_t>(row) * a.mlp_blocks + b);
    const float learned = 1.0f / (1.0f + expf(-v));
    if (a.mlp_score_out != nullptr) a.mlp_score_out[row] = learned;
    if (a.decide_on_mlp) score = learned;
  }
  const int flag = a.route_above ? ((score <= tau) ? 0 : 1) : ((score >= tau) ? 0 : 1);
  a.token[row] = acc.idx;
  a.conf[row] = conf;
  a.entropy[row] = ent;
  a.route_mask[row] = static_cast<uint8_t>(flag);
  return flag;
}

// First routed position of every sequence: an atomic minimum per sequence over the
// routed rows.  Called by the one block that compacts, before (init) and during the pass.
__device__ __forceinline__ void first_routed_init(const FinishLaunch& a) {
  if (a.seq_len > 0) {
    for (int b = threadIdx.x; b < a.n / a.seq_len; b += blockDim.x) a.first_routed[b] = a.seq_len;
    __syncthreads();
  }
}
__device__ __forceinline__ void first_routed_note(const FinishLaunch& a, int row) {
  if (a.seq_len > 0) atomicMin(a.first_routed + row / a.seq_len, row % a.seq_len);
}

// Programmatic dependent launch: let the next kernel in the stream be scheduled now (it
// waits for this grid to complete before touching memory), then wait for the projection
// kernel's partials.
__device__ __forceinline__ void pdl_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Vocabulary-sharded step with the fused exchange: the other GPUs store their summaries into this GPU's
// memory and then set a flag each.  Warp 0 of every block polls the flags (lane g watches flag g, g + 32, ...)
// with acquire loads at system scope until all hold the expected value or the time limit runs out; the
// block then goes on either way (after a time-out the status word says the outputs are not to be trusted).
__device__ __forceinline__ void wait_for_peers(const FinishLaunch& a) {
  if (a.wait_flags == nullptr) return;
  if (threadIdx.x < 32) {
    unsigned long long t0 = 0;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
    for (;;) {
      bool mine = true;
      for (int g = threadIdx.x; g < a.wait_count; g += 32) {
        uint32_t v;
        asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(a.wait_flags + g) : "memory");
        mine = mine && (v == a.wait_value);
      }
      if (__all_sync(0xffffffffu, mine)) break;
      unsigned long long t1;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
      if (__any_sync(0xffffffffu, t1 - t0 > a.wait_limit_ns)) {
        if (threadIdx.x == 0) atomicOr(a.status, TLR_DEV_WAIT_TIMEOUT);
        break;
      }
      __nanosleep(200);
    }
  }
  __syncthreads();
}

// Cluster of gridDim.x blocks, n <= 1024.  A group of L lanes (L a power of two) folds one
// row in two passes over its partials: maximum and index first, then the sums rescaled to
// that maximum.  L is chosen on the host so that every row has its group: n * L <=
// gridDim.x * 1024.
__global__ void __launch_bounds__(kSmallThreads)
finish_small_kernel(const FinishLaunch a, const int L) {
  __shared__ int warp_count[kSmallThreads / 32];
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int group = (blockIdx.x * blockDim.x + threadIdx.x) / L;
  const int gl = threadIdx.x & (L - 1);
  pdl_enter();
  wait_for_peers(a);
  __shared__ unsigned char flags[kSmallRows];
  const bool single_block = gridDim.x == 1;
  {
    const int row = group;
    const bool valid = row < a.n;
    const Partial* p = a.partials + static_cast<size_t>(valid ? row : 0) * a.row_stride;
    const size_t cs = static_cast<size_t>(a.chunk_stride);
    float m = -INFINITY;
    int idx = kNoToken;
    float s = 0.f, t = 0.f;
    if ((a.chunks + L - 1) / L <= kPerLane) {
      // few partials per lane: one pass, the partials stay in registers
      Partial q[kPerLane];
#pragma unroll
      for (int k = 0; k < kPerLane; ++k) {
        const int j = gl + L * k;
        if (valid && j < a.chunks) {
          const float4 raw = __ldcg(reinterpret_cast<const float4*>(p + j * cs));
          q[k].m = raw.x;
          q[k].idx = __float_as_int(raw.y);
          q[k].s = raw.z;
          q[k].t = raw.w;
        } else {
          q[k] = empty_partial();
        }
        if (q[k].m > m || (q[k].m == m && q[k].idx < idx)) {
          m = q[k].m;
          idx = q[k].idx;
        }
      }
      for (int off = L >> 1; off > 0; off >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, off);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, off);
        if (om > m || (om == m && oi < idx)) {
          m = om;
          idx = oi;
        }
      }
#pragma unroll
      for (int k = 0; k < kPerLane; ++k) {
        if (!(q[k].s == 0.f)) {         // an empty range contributes nothing; a NaN sum goes through
          const float dm = q[k].m - m;  // <= 0
          const float e = exp2f(dm * kLog2e);
          s += q[k].s * e;
          t += e * (q[k].t + dm * q[k].s);
        }
      }
    } else {
      // many partials per lane: maximum and index first, then the rescaled sums
      if (valid) {
        for (int j = gl; j < a.chunks; j += L) {
          const float2 mi = __ldcg(reinterpret_cast<const float2*>(p + j * cs));
          const int qi = __float_as_int(mi.y);
          if (mi.x > m || (mi.x == m && qi < idx)) {
            m = mi.x;
            idx = qi;
          }
        }
      }
      for (int off = L >> 1; off > 0; off >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, off);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, off);
        if (om > m || (om == m && oi < idx)) {
          m = om;
          idx = oi;
        }
      }
      if (valid) {
        for (int j = gl; j < a.chunks; j += L) {
          const float4 raw = __ldcg(reinterpret_cast<const float4*>(p + j * cs));
          if (!(raw.z == 0.f)) {
            const float dm = raw.x - m;
            const float e = exp2f(dm * kLog2e);
            s += raw.z * e;
            t += e * (raw.w + dm * raw.z);
          }
        }
      }
    }
    for (int off = L >> 1; off > 0; off >>= 1) {
      s += __shfl_xor_sync(0xffffffffu, s, off);
      t += __shfl_xor_sync(0xffffffffu, t, off);
    }
    if (valid && gl == 0) {
      Partial acc;
      acc.m = m;
      acc.idx = idx;
      acc.s = s;
      acc.t = t;
      const int f = score_row(acc, a, row);
      if (single_block) {
        flags[row] = static_cast<unsigned char>(f);
      } else {
        // into block 0's shared memory (distributed shared memory of the cluster): block 0 then compacts
        // without another trip to L2 for the flags
        const uint32_t mine = static_cast<uint32_t>(__cvta_generic_to_shared(&flags[row]));
        uint32_t remote;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(mine), "r"(0));
        asm volatile("st.shared::cluster.u8 [%0], %1;" ::"r"(remote), "r"(f) : "memory");
      }
    }
  }
  if (single_block) {
    __syncthreads();                    // the flags are in this block's shared memory
  } else {
    // The cluster barrier (release / acquire) makes every block's stores into block 0's shared memory
    // visible to block 0, and keeps block 0 (and its shared memory) there until they have been made.
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  }
  if (blockIdx.x != 0) return;
  first_routed_init(a);
  const int warps = blockDim.x >> 5;
  int base_out = 0;
  for (int base = 0; base < a.n; base += blockDim.x) {       // one pass when the block has a thread per row
    const int i = base + threadIdx.x;
    int flag = 0;
    if (i < a.n) flag = static_cast<int>(flags[i]);
    const unsigned int bal = __ballot_sync(0xffffffffu, flag != 0);
    if (lane == 0) warp_count[warp] = __popc(bal);
    __syncthreads();
    int before = 0, total = 0;
    for (int w = 0; w < warps; ++w) {
      const int c = warp_count[w];
      before += (w < warp) ? c : 0;
      total += c;
    }
    if (flag) {
      a.routed_idx[base_out + before + __popc(bal & ((1u << lane) - 1u))] = i;
      first_routed_note(a, i);
    }
    base_out += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    *a.routed_count = base_out;
    if (a.status_copy != nullptr) *a.status_copy = atomicOr(a.status, 0u);   // every row has been scored by now
  }
}

__global__ void __launch_bounds__(kFinishThreads)
finish_kernel(const FinishLaunch a) {
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * kFinishWarps + warp;
  pdl_enter();
  wait_for_peers(a);

  if (row < a.n) {
    const Partial acc = fold_row(a.partials + static_cast<size_t>(row) * a.row_stride, a.chunks, a.chunk_stride, lane);
    if (lane == 0) score_row(acc, a, row);
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
  first_routed_init(a);
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
    if (flag) {
      a.routed_idx[base_out + before + __popc(bal & ((1u << lane) - 1u))] = i;
      first_routed_note(a, i);
    }
    base_out += total;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    *a.routed_count = base_out;
    if (a.status_copy != nullptr) *a.status_copy = atomicOr(a.status, 0u);
    *a.ticket = 0u;  // ready for the next call on this context
  }
}

cudaError_t launch_finish(const FinishLaunch& a, cudaStream_t stream) {
  if (a.chunks > 32 * kPerLane) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (a.n <= kSmallRows) {
    int blocks = 1;
    while (blocks < 8 && blocks * 32 < a.n) blocks <<= 1;       // 32 rows per block until 8 blocks
    // 512-thread blocks fit on an SM beside a CTA of the tensor-core projection kernel, so they
    // are resident (waiting) before it ends and do not keep the next call's CTAs off their SMs;
    // they are used whenever a lane group still owns few enough partials for the one-pass fold.
    auto lanes_for = [&](int threads) {
      int l = 32;
      while (l > 1 && a.n * l > blocks * threads) l >>= 1;
      return l;
    };
    int threads = kSmallThreads;
    if ((a.chunks + lanes_for(512) - 1) / lanes_for(512) <= kPerLane) threads = 512;
    {
      const int e = tuning().finish_threads;   // tuning switch (TLR_FINISH_THREADS)
      if (e == 256 || e == 512 || e == 1024) threads = e;
    }
    const int L = lanes_for(threads);
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = static_cast<unsigned>(blocks);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
    cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
    cfg.blockDim = dim3(static_cast<unsigned>(threads), 1, 1);
    return cudaLaunchKernelEx(&cfg, finish_small_kernel, a, L);
  }
  const int blocks = (a.n + kFinishWarps - 1) / kFinishWarps;
  cfg.gridDim = dim3(static_cast<unsigned>(blocks), 1, 1);
  cfg.blockDim = dim3(kFinishThreads, 1, 1);
  return cudaLaunchKernelEx(&cfg, finish_kernel, a);
}

}  // namespace tlr
