// Device-side pieces that only the 8-bit (e4m3) head needs: the kind::f8f6f4 MMA and its
// instruction descriptor, e4m3 conversions, and the split of bf16 hidden states into two e4m3
// parts written straight into swizzled operand slabs.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace tlr {
namespace {

// D[tmem] (+)= A[smem] * B[smem]^T, e4m3 inputs, fp32 accumulate, K = 32 per instruction.
__device__ __forceinline__ void umma_e4m3(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Instruction descriptor: fp32 accumulator, e4m3 A and B (format code 0), both K-major.
__device__ __forceinline__ uint32_t instr_desc_e4m3(int m_rows, int n_cols) {
  return (1u << 4) | (static_cast<uint32_t>(n_cols >> 3) << 17) | (static_cast<uint32_t>(m_rows >> 4) << 24);
}

// Two floats -> two e4m3 (round to nearest even, saturating), and back.
__device__ __forceinline__ uint16_t to_e4m3x2(float hi, float lo) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float2 from_e4m3x2(uint16_t v) {   // .x = low byte, .y = high byte
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(v));
  return __half22float2(*reinterpret_cast<__half2*>(&h2));
}

// The power of two r that puts a row's largest magnitude amax into [128, 256) after division.
__device__ __forceinline__ float split_scale(float amax) {
  float r = 1.0f;
  if (amax > 0.f && amax < INFINITY) {
    int e;
    frexpf(amax, &e);                 // amax = f * 2^e, f in [0.5, 1)
    e = e - 8 < -126 ? -126 : (e - 8 > 126 ? 126 : e - 8);   // keeps r and 1/r finite and normal
    r = ldexpf(1.0f, e);
  }
  return r;
}

// x * inv as the sum of two e4m3 numbers: p1 = round(x), p2 = round(x - p1), two elements at a time.
__device__ __forceinline__ void split_pair(float x0, float x1, uint16_t& p1, uint16_t& p2) {
  p1 = to_e4m3x2(x1, x0);
  const float2 f1 = from_e4m3x2(p1);
  p2 = to_e4m3x2(x1 - f1.y, x0 - f1.x);
}

// Splits the (at most 16) rows of h into resident operand slabs, done by 288 threads numbered t (the caller's
// warps 2..10; they synchronise among themselves with named barrier 1).  Slab ks is 32 rows of 128 bytes
// with the 128-byte swizzle TMA would have produced: rows 0..15 hold the first parts, rows 16..31 the
// second parts; the 16-byte chunk c of row r sits at position c ^ (r & 7).  hs_s[r] receives row r's scale
// (hs_s[32 + r] is scratch).  One pass over h: 18 threads per row, each keeps its (at most kSplitChunks) chunks of
// 16 elements in registers between the maximum and the conversion, so the row is read from memory once and all
// loads are in flight together.
constexpr int kSplitThreads = 288;
constexpr int kSplitLanes = kSplitThreads / 16;       // threads per row
constexpr int kSplitChunks = 6;                       // chunks of 16 elements per thread: d <= 16 * 18 * 6 = 1728
__device__ __forceinline__ void split_h_resident(const __nv_bfloat16* __restrict__ hb, int n, int d, int k_slabs,
                                                 unsigned char* slabs, float* hs_s, int t) {
  const int r = t / kSplitLanes, l = t - r * kSplitLanes;
  const int valid_chunks = d >> 4;                          // d is a multiple of 16
  uint4 va[kSplitChunks], vb[kSplitChunks];
  float amax = 0.f;
#pragma unroll
  for (int i = 0; i < kSplitChunks; ++i) {
    const int c = l + kSplitLanes * i;
    va[i] = make_uint4(0u, 0u, 0u, 0u);
    vb[i] = va[i];
    if (r < n && c < valid_chunks) {
      const uint4* src = reinterpret_cast<const uint4*>(hb + static_cast<size_t>(r) * d + c * 16);
      va[i] = __ldg(src);
      vb[i] = __ldg(src + 1);
    }
  }
#pragma unroll
  for (int i = 0; i < kSplitChunks; ++i) {
    const uint32_t w[8] = {va[i].x, va[i].y, va[i].z, va[i].w, vb[i].x, vb[i].y, vb[i].z, vb[i].w};
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[j]));
      amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
    }
  }
  // the row's largest magnitude: non-negative floats order like their bit patterns
  unsigned int* amax_bits = reinterpret_cast<unsigned int*>(hs_s + 32);
  if (t < 16) amax_bits[t] = 0u;
  asm volatile("bar.sync 1, %0;" ::"n"(kSplitThreads) : "memory");   // only the splitting warps; nothing asynchronous is waited for
  atomicMax(amax_bits + r, __float_as_uint(amax));               // (fmaxf drops NaNs, so amax is a number >= 0)
  asm volatile("bar.sync 1, %0;" ::"n"(kSplitThreads) : "memory");
  const float sc = split_scale(__uint_as_float(amax_bits[r]));
  if (l == 0) hs_s[r] = sc;
  const float inv = 1.0f / sc;                                   // exact: a power of two
#pragma unroll
  for (int i = 0; i < kSplitChunks; ++i) {
    const int cc = l + kSplitLanes * i;
    if (cc >= k_slabs * 8) continue;                             // (chunks between d and the slab's end are zeros)
    const int ks = cc >> 3, c = cc & 7;
    const uint32_t w[8] = {va[i].x, va[i].y, va[i].z, va[i].w, vb[i].x, vb[i].y, vb[i].z, vb[i].w};
    uint32_t q1[4] = {0u, 0u, 0u, 0u}, q2[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int j = 0; j < 8; ++j) {                                // two elements per 32-bit word
      const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[j]));
      uint16_t p1, p2;
      split_pair(f.x * inv, f.y * inv, p1, p2);
      q1[j >> 1] |= static_cast<uint32_t>(p1) << (16 * (j & 1));
      q2[j >> 1] |= static_cast<uint32_t>(p2) << (16 * (j & 1));
    }
    unsigned char* dst = slabs + ks * 4096 + r * 128 + ((c ^ (r & 7)) << 4);
    *reinterpret_cast<uint4*>(dst) = make_uint4(q1[0], q1[1], q1[2], q1[3]);
    *reinterpret_cast<uint4*>(dst + 2048) = make_uint4(q2[0], q2[1], q2[2], q2[3]);
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic stores -> the MMA's (async proxy) reads
}

}  // namespace
}  // namespace tlr
