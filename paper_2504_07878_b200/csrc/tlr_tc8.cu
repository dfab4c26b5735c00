// Decode batches on an 8-bit (e4m3, one scale per vocabulary row) copy of W.
//
// At decode sizes the step is the time to stream W from HBM; W stored in 8 bits halves it.  The
// tensor core multiplies fp8 by fp8 only (tcgen05.mma kind::f8f6f4), and h is bf16, so h is not
// rounded to fp8 but SPLIT: every row of h is scaled by a power of two r so that its largest
// magnitude lies in [128, 256), and written as the sum of two e4m3 numbers, h / r = p1 + p2 with
// p1 = round(h / r) and p2 = round(h / r - p1).  A bf16 number has 8 significant bits and e4m3
// has 4: the first rounding leaves a remainder of at most 8 units of the bf16 number's last
// place, which the second part holds exactly.  Only elements below 2^-10 of the row's largest
// fall under e4m3's smallest step (2^-9); their error is at most 2^-17 of that largest.
//
// The two parts are stacked along the MMA's M dimension: the operand slab of a K step holds the
// first parts of all token rows and, below them, the second parts, and ONE MMA per K step computes
// both products (products of e4m3 numbers are exact in fp32).  A token's logit is the sum of its two
// accumulator rows; they sit in different lane quadrants of tensor memory, so the epilogue warp of the
// second parts passes its columns through shared memory to the warp of the first parts, which adds
// them, multiplies by r (per token row) and by the weight row's scale, and folds as the bf16 path does.
// One MMA per K step at twice the bf16 rate leaves the tensor pipe half as busy as the bf16 path; the
// bytes from HBM are half.
//
// This file holds what only the 8-bit head has: the split kernel, the shape of the launch and the
// launch of tc8_projection_kernel (the <1, true> instantiation of the projection kernel's body in
// tlr_tc_kernel.cuh; device helpers in tlr_tc8_dev.cuh).
#include <cuda.h>
#include <cuda_bf16.h>

#include "tlr_common.cuh"
#include "tlr_tc.cuh"
#define TLR_DEFINE_TC8_KERNEL
#include "tlr_tc_kernel.cuh"

namespace tlr {

// One block per row of the padded batch (rows >= n are written as zeros): the row's power-of-two
// scale r (largest |h| / r in [128, 256)), and h / r as the sum of two e4m3 arrays, [2][part_rows][d].
__global__ void __launch_bounds__(128)
h_split_kernel(const __nv_bfloat16* __restrict__ h, int n, int d, int part_rows, uint8_t* __restrict__ parts,
               float* __restrict__ hscale) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int row = blockIdx.x;
  const size_t part_stride = static_cast<size_t>(part_rows) * d;
  uint8_t* out = parts + static_cast<size_t>(row) * d;
  if (row >= n) {
    for (int k = threadIdx.x * 2; k < d; k += 256) {
      *reinterpret_cast<uint16_t*>(out + k) = 0;
      *reinterpret_cast<uint16_t*>(out + part_stride + k) = 0;
    }
    return;
  }
  const __nv_bfloat16* src = h + static_cast<size_t>(row) * d;
  float amax = 0.f;
  for (int k = threadIdx.x; k < d; k += 128) amax = fmaxf(amax, fabsf(__bfloat162float(src[k])));
  __shared__ float red[4];
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = amax;
  __syncthreads();
  amax = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
  const float r = split_scale(amax);
  const float inv = 1.0f / r;         // exact: r is a power of two
  if (threadIdx.x == 0) hscale[row] = r;
  for (int k = threadIdx.x * 2; k < d; k += 256) {      // d is a multiple of 16
    uint16_t p1, p2;
    split_pair(__bfloat162float(src[k]) * inv, __bfloat162float(src[k + 1]) * inv, p1, p2);
    *reinterpret_cast<uint16_t*>(out + k) = p1;
    *reinterpret_cast<uint16_t*>(out + part_stride + k) = p2;
  }
}

int tc8_max_rows() { return 128; }

void tc8_configure(int n, int d, TcConfig* c) {
  // rows per part; the operand slab stacks the two parts.  Up to 64 rows both parts go through one MMA (its M holds
  // 2 x 16, 32 or 64 rows); above, every K step takes two MMAs and a part is n rounded up to 16 rows.
  int part_rows = n <= 16 ? 16 : (n <= 32 ? 32 : (n <= 64 ? 64 : ((n + 15) / 16) * 16));
  const int a_stage = 2 * part_rows * kRowBytes;
  const int b_stage = kBlockN * kRowBytes;
  const int k_slabs = (d + kRowBytes - 1) / kRowBytes;
  const int extra = tc8_extra_bytes(part_rows);
  const int budget = kSmemLimit - 1024 - kBarrierBytes - kScratchBytes - extra;
  // n <= 16 and all of h (two parts) small enough: the kernel splits h itself and keeps it resident, one
  // launch less.  TLR_TC8_INLINE=0 is a tuning switch that keeps the separate split kernel.
  bool inl = n <= 16 && k_slabs * 8 <= kSplitLanes * kSplitChunks && tuning().tc8_inline != 0;
  // ... and only while the resident copy leaves the W ring five stages: with four (d = 2048) what the
  // missing launch gains is lost again to the shallower ring
  if (inl && (budget - k_slabs * a_stage) / b_stage < 5) inl = false;
  int sa = inl ? k_slabs : (part_rows <= 32 ? 6 : (part_rows <= 64 ? 4 : 3));
  if (!inl && tuning().ring_a > 0) sa = tuning().ring_a;
  int sb = (budget - sa * a_stage) / b_stage;
  if (sb > kMaxBStages) sb = kMaxBStages;
  c->cta = 1;
  c->a_rows = 2 * part_rows;
  c->part_rows = part_rows;
  c->a_stages = sa;
  c->b_stages = sb;
  c->inline_split = inl ? 1 : 0;
  c->smem_bytes = 1024 + sa * a_stage + sb * b_stage + kBarrierBytes + kScratchBytes + extra;
}

cudaError_t tc8_prepare() {
  return cudaFuncSetAttribute(tc8_projection_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
}

cudaError_t launch_h_split(const void* h_bf16, int n, int d, int part_rows, uint8_t* parts, float* hscale,
                           cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(part_rows), 1, 1);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, h_split_kernel, static_cast<const __nv_bfloat16*>(h_bf16), n, d, part_rows, parts,
                            hscale);
}

cudaError_t launch_tc8_projection(const TcMaps& maps, const TcParams& p, const TcConfig& c, int workers,
                                  cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(workers), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = static_cast<size_t>(c.smem_bytes);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, tc8_projection_kernel, maps, p);
}

}  // namespace tlr
