// Learned routing score on the hidden state: score = sigmoid(w2 . relu(W1 h + b1) + b2).
// The router the paper deploys is a small learned classifier (an MLP) fed with the last-layer
// hidden state (Sec. 3.1; Sec. 2.1); neither its width nor its activation nor weights are given, so
// the shape here (one hidden layer, ReLU, sigmoid output) is this library's assumption and
// the weights are the caller's.  Where the tensor-core projection kernel runs, the first layer is
// part of that launch (tlr_tc_kernel.cuh); this CUDA-core kernel serves the shapes it cannot take
// (d % 8 != 0, an unaligned W1, the 8-bit head): a block stages kMlpRows hidden-state rows in shared
// memory and covers kMlpUnits hidden units, eight threads per unit.
#include "tlr_common.cuh"

namespace tlr {

constexpr int kMlpThreads = 256;
constexpr int kMlpRows = 8;          // token rows per block
constexpr int kMlpUnits = 32;        // hidden units per block
constexpr int kMlpSplitK = kMlpThreads / kMlpUnits;   // 8 threads share one hidden unit's dot product

int mlp_hidden_blocks(int d_hidden) { return (d_hidden + kMlpUnits - 1) / kMlpUnits; }

// Block (x = row group, y = hidden-unit group): writes, for each of its rows, the partial sum
// over its hidden units of w2_j * relu(W1_j . h + b1_j).  The merge kernel adds the partials of
// a row in a fixed order, adds b2 and applies the sigmoid, so the score is deterministic.
__global__ void __launch_bounds__(kMlpThreads)
mlp_partial_kernel(const MlpLaunch a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned short* hs = reinterpret_cast<unsigned short*>(smem_raw);  // [kMlpRows][d] bf16 bits
  __shared__ float red[kMlpThreads / 32][kMlpRows];
  // The hidden states may come from the previous kernel in the stream.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int row0 = blockIdx.x * kMlpRows;
  const int d = a.d;
  const unsigned short* h = reinterpret_cast<const unsigned short*>(a.h);
  const unsigned short* W1 = reinterpret_cast<const unsigned short*>(a.W1);
  if (d % 8 == 0 && (reinterpret_cast<uintptr_t>(a.h) & 15) == 0) {
    // rows of a multiple of 8 elements: the staged block is contiguous in h, copy it 16 bytes at a time
    const int vec_per_row = d / 8;
    const uint4* src = reinterpret_cast<const uint4*>(h + static_cast<size_t>(row0) * d);
    uint4* dst = reinterpret_cast<uint4*>(hs);
    const int valid_rows = min(kMlpRows, a.n - row0);
#pragma unroll 4
    for (int i = threadIdx.x; i < kMlpRows * vec_per_row; i += kMlpThreads)
      dst[i] = (i < valid_rows * vec_per_row) ? __ldg(src + i) : make_uint4(0u, 0u, 0u, 0u);
  } else {
    for (int i = threadIdx.x; i < kMlpRows * d; i += kMlpThreads) {
      const int r = i / d, k = i - r * d;
      hs[i] = (row0 + r < a.n) ? h[static_cast<size_t>(row0 + r) * d + k] : static_cast<unsigned short>(0);
    }
  }
  __syncthreads();

  const int unit = blockIdx.y * kMlpUnits + threadIdx.x / kMlpSplitK;   // hidden unit of this thread
  const int part = threadIdx.x % kMlpSplitK;                            // which slice of k it sums
  float acc[kMlpRows];
#pragma unroll
  for (int r = 0; r < kMlpRows; ++r) acc[r] = 0.f;
  if (unit < a.d_hidden) {
    const unsigned short* wrow = W1 + static_cast<size_t>(unit) * d;
    const bool vec = (d % 8 == 0) && ((reinterpret_cast<uintptr_t>(a.W1) & 15) == 0);
    if (vec) {
#pragma unroll 4
      for (int k = part * 8; k < d; k += 8 * kMlpSplitK) {
        const uint4 w8 = __ldg(reinterpret_cast<const uint4*>(wrow + k));
        const unsigned int wv[4] = {w8.x, w8.y, w8.z, w8.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float w_lo = __uint_as_float(wv[q] << 16);
          const float w_hi = __uint_as_float(wv[q] & 0xffff0000u);
#pragma unroll
          for (int r = 0; r < kMlpRows; ++r) {
            const unsigned int hh = *reinterpret_cast<const unsigned int*>(hs + r * d + k + 2 * q);
            acc[r] = fmaf(__uint_as_float(hh << 16), w_lo, acc[r]);
            acc[r] = fmaf(__uint_as_float(hh & 0xffff0000u), w_hi, acc[r]);
          }
        }
      }
    } else {
      for (int k = part; k < d; k += kMlpSplitK) {
        const float w = __uint_as_float(static_cast<unsigned int>(wrow[k]) << 16);
#pragma unroll
        for (int r = 0; r < kMlpRows; ++r)
          acc[r] = fmaf(__uint_as_float(static_cast<unsigned int>(hs[r * d + k]) << 16), w, acc[r]);
      }
    }
  }
  // the kMlpSplitK threads of a unit are adjacent lanes: finish the dot products
#pragma unroll
  for (int r = 0; r < kMlpRows; ++r) {
#pragma unroll
    for (int off = kMlpSplitK / 2; off > 0; off >>= 1) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], off);
  }
  float contrib[kMlpRows];
  const bool owner = (part == 0) && (unit < a.d_hidden);
  const float b1 = owner ? a.b1[unit] : 0.f, w2 = owner ? a.w2[unit] : 0.f;
#pragma unroll
  for (int r = 0; r < kMlpRows; ++r) contrib[r] = owner ? w2 * fmaxf(acc[r] + b1, 0.f) : 0.f;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
  for (int r = 0; r < kMlpRows; ++r) {
    float v = contrib[r];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    if (lane == 0) red[warp][r] = v;
  }
  __syncthreads();
  if (threadIdx.x < kMlpRows && row0 + threadIdx.x < a.n) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kMlpThreads / 32; ++w) v += red[w][threadIdx.x];
    a.partial[static_cast<size_t>(row0 + threadIdx.x) * gridDim.y + blockIdx.y] = v;
  }
}

cudaError_t launch_mlp_score(const MlpLaunch& a, cudaStream_t stream) {
  if (a.n <= 0) return cudaSuccess;
  const int smem = kMlpRows * a.d * 2;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(mlp_partial_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>((a.n + kMlpRows - 1) / kMlpRows),
                     static_cast<unsigned>(mlp_hidden_blocks(a.d_hidden)), 1);
  cfg.blockDim = dim3(kMlpThreads, 1, 1);
  cfg.dynamicSmemBytes = static_cast<size_t>(smem);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, mlp_partial_kernel, a);
}

}  // namespace tlr
