// CUDA-core projection kernel: logits + online-softmax partials with plain FMAs.
// Serves the shapes the TMA-fed tensor-core kernel cannot address (hidden size not a
// multiple of 8, so rows of W are not 16-byte multiples) and is selectable for
// diagnostics.  One thread owns one vocabulary row of a 128-row tile and kRows token
// rows at a time; the block walks its vocabulary chunk tile by tile, each thread
// keeping the running (m, idx, s, t) of its own rows, and the block folds its 128
// thread-partials per token row at the end.
#include <cuda_bf16.h>

#include "tlr_common.cuh"

namespace tlr {

constexpr int kSimtThreads = 128;
constexpr int kRows = 8;

__device__ __forceinline__ float bf16_bits_to_float(unsigned short b) {
  return __uint_as_float(((unsigned int)b) << 16);
}

// Fold one logit into a running summary (z is visited in ascending vocabulary order
// per thread, so a strict comparison keeps the lowest index on ties).
__device__ __forceinline__ void fold(Partial& p, float z, int v) {
  if (z > p.m) {
    if (p.s > 0.f) {
      const float dlt = p.m - z;
      const float sc = exp2f(dlt * kLog2e);
      p.t = sc * (p.t + dlt * p.s);
      p.s = p.s * sc;
    }
    p.m = z;
    p.idx = v;
    p.s += 1.0f;
  } else {
    const float x = z - p.m;
    const float e = exp2f(x * kLog2e);
    p.s += e;
    p.t += e * x;
  }
}

template <bool kVec>
__global__ void __launch_bounds__(kSimtThreads)
simt_projection_kernel(const SimtLaunch a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned short* hs = reinterpret_cast<unsigned short*>(smem_raw);  // [kRows][d] bf16 bits
  __shared__ Partial red[kSimtThreads / 32][kRows];

  const int chunk = blockIdx.x;
  const int row0 = blockIdx.y * kRows;
  const int d = a.d;
  const unsigned short* W = reinterpret_cast<const unsigned short*>(a.W);
  const unsigned short* h = reinterpret_cast<const unsigned short*>(a.h);

  // stage the kRows hidden-state rows (zeros past n)
  for (int i = threadIdx.x; i < kRows * d; i += kSimtThreads) {
    const int r = i / d, k = i - r * d;
    hs[i] = (row0 + r < a.n) ? h[(size_t)(row0 + r) * d + k] : (unsigned short)0;
  }
  __syncthreads();

  // this block's vocabulary range, in 128-row tiles
  const int tiles = (a.V + kSimtThreads - 1) / kSimtThreads;
  const int t0 = (int)(((long long)tiles * chunk) / a.chunks);
  const int t1 = (int)(((long long)tiles * (chunk + 1)) / a.chunks);

  Partial run[kRows];
#pragma unroll
  for (int r = 0; r < kRows; ++r) run[r] = empty_partial();

  for (int tile = t0; tile < t1; ++tile) {
    const int v = tile * kSimtThreads + threadIdx.x;
    if (v >= a.V) continue;
    float acc[kRows];
#pragma unroll
    for (int r = 0; r < kRows; ++r) acc[r] = 0.f;
    const unsigned short* wrow = W + (size_t)v * d;
    if (kVec) {
      for (int k = 0; k < d; k += 8) {
        const uint4 w8 = __ldg(reinterpret_cast<const uint4*>(wrow + k));
        const unsigned int wv[4] = {w8.x, w8.y, w8.z, w8.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float w_lo = __uint_as_float(wv[q] << 16);
          const float w_hi = __uint_as_float(wv[q] & 0xffff0000u);
#pragma unroll
          for (int r = 0; r < kRows; ++r) {
            const unsigned int hh = *reinterpret_cast<const unsigned int*>(hs + r * d + k + 2 * q);
            acc[r] = fmaf(__uint_as_float(hh << 16), w_lo, acc[r]);
            acc[r] = fmaf(__uint_as_float(hh & 0xffff0000u), w_hi, acc[r]);
          }
        }
      }
    } else {
      for (int k = 0; k < d; ++k) {
        const float w = bf16_bits_to_float(wrow[k]);
#pragma unroll
        for (int r = 0; r < kRows; ++r) acc[r] = fmaf(bf16_bits_to_float(hs[r * d + k]), w, acc[r]);
      }
    }
#pragma unroll
    for (int r = 0; r < kRows; ++r) fold(run[r], acc[r], v);
  }

  // block fold: warp butterfly, then the four warp results
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
  for (int r = 0; r < kRows; ++r) {
    const Partial w = warp_merge(run[r]);
    if (lane == 0) red[warp][r] = w;
  }
  __syncthreads();
  if (threadIdx.x < kRows) {
    const int r = threadIdx.x;
    Partial p = red[0][r];
#pragma unroll
    for (int w = 1; w < kSimtThreads / 32; ++w) p = merge(p, red[w][r]);
    if (row0 + r < a.n) a.partials[(size_t)(row0 + r) * a.chunks + chunk] = p;
  }
}

void simt_plan(int n, int d, int V, int sm_count, int* chunks, int* grid, int* block, int* smem) {
  const int tiles = (V + kSimtThreads - 1) / kSimtThreads;
  const int row_blocks = n > 0 ? (n + kRows - 1) / kRows : 1;
  int c = (8 * sm_count) / row_blocks;
  if (c < 1) c = 1;
  if (c > 128) c = 128;
  if (c > tiles) c = tiles;
  *chunks = c;
  *grid = c * row_blocks;
  *block = kSimtThreads;
  *smem = kRows * d * 2;
}

cudaError_t launch_simt_projection(const SimtLaunch& a, cudaStream_t stream) {
  const int smem = kRows * a.d * 2;
  const dim3 grid(a.chunks, (a.n + kRows - 1) / kRows);
  const bool vec = (a.d % 8 == 0) && ((reinterpret_cast<uintptr_t>(a.W) & 15) == 0);
  cudaError_t e;
  if (vec) {
    if (smem > 48 * 1024) {
      e = cudaFuncSetAttribute(simt_projection_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e != cudaSuccess) return e;
    }
    simt_projection_kernel<true><<<grid, kSimtThreads, smem, stream>>>(a);
  } else {
    if (smem > 48 * 1024) {
      e = cudaFuncSetAttribute(simt_projection_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e != cudaSuccess) return e;
    }
    simt_projection_kernel<false><<<grid, kSimtThreads, smem, stream>>>(a);
  }
  return cudaGetLastError();
}

}  // namespace tlr
