// Decode-batch projection kernel for an fp8 (e4m3, one scale per vocabulary row) copy of W.
//
// At decode sizes the step is the time to stream W from HBM; W stored in 8 bits halves it.  The
// tensor core multiplies fp8 by fp8 only (tcgen05.mma kind::f8f6f4), and h is bf16, so h is not
// rounded to fp8 but SPLIT: every row of h is scaled by a power of two r so that its largest
// magnitude lies in [128, 256), and written as the sum of two e4m3 numbers, h / r = p1 + p2 with
// p1 = round(h / r) and p2 = round(h / r - p1).  A bf16 number has 8 significant bits and e4m3
// has 4: the first rounding leaves a remainder of at most 8 units of the bf16 number's last
// place, which the second part holds exactly.  Only elements below 2^-10 of the row's largest
// fall under e4m3's smallest step (2^-9); their error is at most 2^-17 of that largest.  The
// kernel runs two MMAs per K step, one per part, into the same fp32 accumulator: products of
// e4m3 numbers are exact in fp32, so the accumulator holds sum_k (h/r)[k] * q[v][k] as the bf16
// path would, and the epilogue multiplies by r (per token row) and by the weight row's scale
// before the online-softmax fold.  Two MMAs at twice the bf16 rate cost the tensor time of the
// bf16 path; the bytes from HBM are half.
//
// Structure: as tc_projection_kernel<1> (one CTA per worker; W producer, h producer, MMA issuer,
// two groups of four epilogue warps; rings, barriers, bounded waits, programmatic dependent
// launch, the same static schedule and partials).  Differences: a K slab is 128 elements (128
// bytes of fp8 per row, one swizzle span); an h stage holds both parts of the slab; the
// epilogue warps stage the tile's weight scales in shared memory before they wait for the
// accumulator.  h_split_kernel, launched just before, writes the two parts and the row scales.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <cstdio>
#include <cstdlib>

#include "tlr_common.cuh"
#include "tlr_tc.cuh"
#include "tlr_tc_ptx.cuh"

namespace tlr {

namespace {

constexpr int kBlockM = 64;                  // the MMA's M: the kernel serves at most 64 token rows, and an M = 64
                                             // instruction takes about two thirds of the time of an M = 128 one.
                                             // Its accumulator row r lives in TMEM lane 32 * (r / 16) + r % 16:
                                             // lanes 0..15 of each 32-lane quadrant (checked on the device).
constexpr int kBlockN = 256;                 // max vocabulary rows per tile == accumulator columns
constexpr int kSlabK = 128;                  // fp8 elements per slab row = 128 B = one swizzle span
constexpr int kUmmaK8 = 32;                  // K of one kind::f8f6f4 MMA
constexpr int kRowBytes = 128;
constexpr int kParts = 2;
constexpr int kTmemCols = 512;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 32 * 11;
constexpr int kMaxAStages = 8;
constexpr int kMaxBStages = 8;
constexpr int kRelease = 16;
constexpr int kBarrierBytes = 512;
constexpr int kScratchBytes = kBlockM * 16;   // one Partial per token row
constexpr int kScaleBytes = kEpiWarps * kBlockN * 4;   // a tile's weight scales, one copy per epilogue warp
constexpr int kSmemLimit = 232448;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;

// D[tmem] (+)= A[smem] * B[smem]^T, e4m3 inputs, fp32 accumulate.
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

struct Tile {
  int chunk;
  int v0;
  int rows;
};

__host__ __device__ __forceinline__ Tile tile_of8(const Tc8Params& p, int unit, int t) {
  Tile r;
  r.chunk = unit;                                  // one row unit: unit == chunk
  const int g0 = static_cast<int>((static_cast<long long>(p.granules) * r.chunk) / p.chunks);
  const int g1 = static_cast<int>((static_cast<long long>(p.granules) * (r.chunk + 1)) / p.chunks);
  const int G = g1 - g0;
  const int ga = (G * t) / p.tiles_per_unit;
  const int gb = (G * (t + 1)) / p.tiles_per_unit;
  r.v0 = (g0 + ga) * p.granule_rows;
  r.rows = (gb - ga) * p.granule_rows;
  return r;
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

}  // namespace

// One block per row of the padded batch (rows >= n are written as zeros): the row's power-of-two
// scale r (largest |h| / r in [128, 256)), and h / r as the sum of two e4m3 arrays.
__global__ void __launch_bounds__(128)
h_split_kernel(const __nv_bfloat16* __restrict__ h, int n, int d, int rows_alloc, uint8_t* __restrict__ parts,
               float* __restrict__ hscale) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int row = blockIdx.x;
  const size_t part_stride = static_cast<size_t>(rows_alloc) * d;
  uint8_t* out = parts + static_cast<size_t>(row) * d;
  if (row >= n) {
    for (int k = threadIdx.x * 2; k < d; k += 256) {
#pragma unroll
      for (int q = 0; q < kParts; ++q) *reinterpret_cast<uint16_t*>(out + q * part_stride + k) = 0;
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
  float r = 1.0f;
  if (amax > 0.f && amax < INFINITY) {
    int e;
    frexpf(amax, &e);                 // amax = f * 2^e, f in [0.5, 1)
    e = e - 8 < -126 ? -126 : (e - 8 > 126 ? 126 : e - 8);   // keeps r and 1/r finite and normal
    r = ldexpf(1.0f, e);
  }
  const float inv = 1.0f / r;         // exact: r is a power of two
  if (threadIdx.x == 0) hscale[row] = r;
  for (int k = threadIdx.x * 2; k < d; k += 256) {      // d is a multiple of 16
    const float x0 = __bfloat162float(src[k]) * inv, x1 = __bfloat162float(src[k + 1]) * inv;
    const uint16_t p1 = to_e4m3x2(x1, x0);
    const float2 f1 = from_e4m3x2(p1);
    const float r0 = x0 - f1.x, r1 = x1 - f1.y;
    const uint16_t p2 = to_e4m3x2(r1, r0);
    *reinterpret_cast<uint16_t*>(out + k) = p1;
    *reinterpret_cast<uint16_t*>(out + part_stride + k) = p2;
  }
}

__global__ void __launch_bounds__(kThreads, 1)
tc8_projection_kernel(const __grid_constant__ CUtensorMap map_h,
                      const __grid_constant__ CUtensorMap map_w128,
                      const __grid_constant__ CUtensorMap map_w64,
                      const __grid_constant__ CUtensorMap map_w16,
                      const Tc8Params p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int SA = p.a_stages, SB = p.b_stages;
  const uint32_t a_part_bytes = static_cast<uint32_t>(p.a_rows) * kRowBytes;   // one part of one slab
  const uint32_t a_stage_bytes = a_part_bytes * kParts;
  constexpr uint32_t b_stage_bytes = kBlockN * kRowBytes;
  const uint32_t a_ring = base;
  const uint32_t b_ring = base + SA * a_stage_bytes;
  const uint32_t bar_base = b_ring + SB * b_stage_bytes;
  auto a_full = [&](int s) { return bar_base + 8u * s; };
  auto b_full = [&](int s) { return bar_base + 8u * (kMaxAStages + s); };
  auto released = [&](int j) { return bar_base + 8u * (kMaxAStages + kMaxBStages + j); };
  auto acc_full = [&](int b) { return bar_base + 8u * (kMaxAStages + kMaxBStages + kRelease + b); };
  auto acc_empty = [&](int b) { return bar_base + 8u * (kMaxAStages + kMaxBStages + kRelease + 2 + b); };
  auto xch_full = [&](int q) { return bar_base + 8u * (kMaxAStages + kMaxBStages + kRelease + 4 + q); };
  auto xch_empty = [&](int q) { return bar_base + 8u * (kMaxAStages + kMaxBStages + kRelease + 8 + q); };
  const uint32_t h_ready = bar_base + 8u * (kMaxAStages + kMaxBStages + kRelease + 12);   // h split in place (inline mode)
  constexpr int kNumBarriers = kMaxAStages + kMaxBStages + kRelease + 13;
  static_assert(kNumBarriers * 8 + 16 <= kBarrierBytes, "barrier block too small");
  unsigned char* gen_base = smem_raw + (base - smem_u32(smem_raw));
  unsigned char* tail = gen_base + (bar_base - base);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 8 * kNumBarriers);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  Partial* scratch = reinterpret_cast<Partial*>(tail + kBarrierBytes);
  float* scale_area = reinterpret_cast<float*>(tail + kBarrierBytes + kScratchBytes);
  float* hs_s = scale_area + kEpiWarps * kBlockN;     // inline mode: the 16 rows' power-of-two scales
  const bool inl = p.inline_split != 0;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int worker = blockIdx.x;
  const int workers = gridDim.x;

  if (threadIdx.x == 0) {
    if (!inl) for (int s = 0; s < SA; ++s) mbar_init(a_full(s), 1);   // (inline mode: SA = K slabs, nothing streams)
    mbar_init(h_ready, 9);
    for (int s = 0; s < SB; ++s) mbar_init(b_full(s), 1);
    for (int j = 0; j < kRelease; ++j) mbar_init(released(j), 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full(b), 1);
      mbar_init(acc_empty(b), kEpiWarps);
    }
    for (int q = 0; q < 4; ++q) {
      mbar_init(xch_full(q), 1);
      mbar_init(xch_empty(q), 1);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc<1>(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish<1>();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // The W producer reads only W and the tensor maps, which no kernel writes: it does not wait
  // for the previous kernel (the split of h), so its ring fills meanwhile.
  if (warp != 0) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const int k_slabs = (p.d + kSlabK - 1) / kSlabK;
  if (inl && warp >= 2) {
    // ---- inline mode (n <= 16): the nine warps that have nothing to do yet split h into its two e4m3
    // parts, straight into the resident, 128-byte-swizzled operand slabs (row r of slab ks at
    // ks * 4 KB + r * 128, its 16-byte chunk c at position c ^ (r & 7); second part 2 KB further).
    const int t9 = threadIdx.x - 64;                          // 0 .. 287
    const __nv_bfloat16* hb = static_cast<const __nv_bfloat16*>(p.h);
    if (t9 < 256) {                                           // 16 threads per row: the row's scale
      const int r = t9 >> 4, l = t9 & 15;
      float amax = 0.f;
      if (r < p.n) {
        for (int k = l * 8; k < p.d; k += 128) {
          const uint4 v = __ldg(reinterpret_cast<const uint4*>(hb + static_cast<size_t>(r) * p.d + k));
          const __nv_bfloat162* b2 = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float2 f = __bfloat1622float2(b2[j]);
            amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
          }
        }
      }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
      if (l == 0) {
        float sc = 1.0f;
        if (amax > 0.f && amax < INFINITY) {
          int e;
          frexpf(amax, &e);
          e = e - 8 < -126 ? -126 : (e - 8 > 126 ? 126 : e - 8);
          sc = ldexpf(1.0f, e);
        }
        hs_s[r] = sc;
      }
    }
    asm volatile("bar.sync 1, 288;" ::: "memory");            // warps 2..10 only; nothing asynchronous is waited for
    const int chunks_per_row = k_slabs * 8;
    for (int item = t9; item < 16 * chunks_per_row; item += 288) {
      const int r = item / chunks_per_row, cc = item - r * chunks_per_row;
      const int ks = cc >> 3, c = cc & 7, k0 = cc * 16;
      uint32_t q1[4] = {0u, 0u, 0u, 0u}, q2[4] = {0u, 0u, 0u, 0u};
      if (r < p.n && k0 < p.d) {                              // d is a multiple of 16
        const float inv = 1.0f / hs_s[r];
        const uint4 va = __ldg(reinterpret_cast<const uint4*>(hb + static_cast<size_t>(r) * p.d + k0));
        const uint4 vb = __ldg(reinterpret_cast<const uint4*>(hb + static_cast<size_t>(r) * p.d + k0 + 8));
        const uint32_t w[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
#pragma unroll
        for (int j = 0; j < 8; ++j) {                          // two elements per 32-bit word
          const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[j]));
          const float x0 = f.x * inv, x1 = f.y * inv;
          const uint16_t p1 = to_e4m3x2(x1, x0);
          const float2 f1 = from_e4m3x2(p1);
          const uint16_t p2 = to_e4m3x2(x1 - f1.y, x0 - f1.x);
          q1[j >> 1] |= static_cast<uint32_t>(p1) << (16 * (j & 1));
          q2[j >> 1] |= static_cast<uint32_t>(p2) << (16 * (j & 1));
        }
      }
      unsigned char* dst = gen_base + ks * a_stage_bytes + r * kRowBytes + ((c ^ (r & 7)) << 4);
      *reinterpret_cast<uint4*>(dst) = make_uint4(q1[0], q1[1], q1[2], q1[3]);
      *reinterpret_cast<uint4*>(dst + a_part_bytes) = make_uint4(q2[0], q2[1], q2[2], q2[3]);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic stores -> the MMA's (async proxy) reads
    __syncwarp();
    if (lane == 0) mbar_arrive(h_ready);
  }
  const int units = p.chunks;
  const int T = p.tiles_per_unit;
  const unsigned long long wait_ns = p.wait_limit_ns != 0 ? p.wait_limit_ns : kWaitLimitNs;

  if (warp == 0) {
    // ------------------------------------------------------------------ W producer
    if (lane == 0) {
      int stage = 0, slab = 0;
      bool ok = true;
      for (int unit = worker; unit < units && ok; unit += workers) {
        for (int t = 0; t < T && ok; ++t) {
          const Tile tl = tile_of8(p, unit, t);
          if (tl.rows == 0) continue;
          for (int ks = 0; ks < k_slabs; ++ks, ++slab) {
            if (slab >= SB) {
              const int j = slab - SB;
              if (!mbar_wait(released(j & (kRelease - 1)), (j / kRelease) & 1, abort_flag, p.status, wait_ns)) { ok = false; break; }
            }
            const uint32_t dst = b_ring + stage * b_stage_bytes;
            if (p.debug_drop_w_copies) continue;   // test hook: the copies are "lost", the consumer's wait runs out
            mbar_expect_tx(b_full(stage), tl.rows * kRowBytes);
            int r = 0;
            for (; tl.rows - r >= 128; r += 128) tma_load_2d<1>(dst + r * kRowBytes, &map_w128, b_full(stage), ks * kSlabK, tl.v0 + r);
            for (; tl.rows - r >= 64; r += 64) tma_load_2d<1>(dst + r * kRowBytes, &map_w64, b_full(stage), ks * kSlabK, tl.v0 + r);
            for (; tl.rows - r >= 16; r += 16) tma_load_2d<1>(dst + r * kRowBytes, &map_w16, b_full(stage), ks * kSlabK, tl.v0 + r);
            if (++stage == SB) stage = 0;
          }
        }
      }
      if (!ok) drain_delay();
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------------ h producer (both parts of a slab)
    if (lane == 0 && !inl) {
      int stage = 0, slab = 0;
      bool ok = true;
      for (int unit = worker; unit < units && ok; unit += workers) {
        for (int t = 0; t < T && ok; ++t) {
          const Tile tl = tile_of8(p, unit, t);
          if (tl.rows == 0) continue;
          for (int ks = 0; ks < k_slabs; ++ks, ++slab) {
            if (slab >= SA) {
              const int j = slab - SA;
              if (!mbar_wait(released(j & (kRelease - 1)), (j / kRelease) & 1, abort_flag, p.status, wait_ns)) { ok = false; break; }
            }
            const uint32_t dst = a_ring + stage * a_stage_bytes;
            mbar_expect_tx(a_full(stage), a_stage_bytes);
#pragma unroll
            for (int q = 0; q < kParts; ++q)
              tma_load_2d<1>(dst + q * a_part_bytes, &map_h, a_full(stage), ks * kSlabK, q * p.a_rows);
            if (++stage == SA) stage = 0;
          }
        }
      }
      if (!ok) drain_delay();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    int sa = 0, sb = 0;
    uint32_t pa = 0, pb = 0;
    int slab = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    const uint64_t desc_hi = smem_desc_sw128(0) & 0xffffffff00000000ull;
    const uint32_t desc_lo_fixed = static_cast<uint32_t>(smem_desc_sw128(0) & 0xffffffffull);
    const uint32_t a_lo0 = desc_lo_fixed | ((a_ring & 0x3ffffu) >> 4);
    const uint32_t b_lo0 = desc_lo_fixed | ((b_ring & 0x3ffffu) >> 4);
    const uint32_t a_step = a_stage_bytes >> 4, a_part_step = a_part_bytes >> 4, b_step = b_stage_bytes >> 4;
    if (inl) {                                  // h is resident once the nine warps have split it
      ok = __all_sync(0xffffffffu, mbar_wait(h_ready, 0, abort_flag, p.status, wait_ns));
      tc_fence_after();
    }
    bool ra = inl || mbar_test_wait(a_full(0), 0), rb = mbar_test_wait(b_full(0), 0);
    for (int unit = worker; unit < units && ok; unit += workers) {
      for (int t = 0; t < T && ok; ++t) {
        const Tile tl = tile_of8(p, unit, t);
        if (tl.rows == 0) continue;
        const uint32_t idesc = instr_desc_e4m3(kBlockM, tl.rows);
        ok = __all_sync(0xffffffffu, mbar_wait(acc_empty(acc), acc_phase ^ 1u, abort_flag, p.status, wait_ns));
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kBlockN;
        for (int ks = 0; ks < k_slabs; ++ks, ++slab) {
          if (!__all_sync(0xffffffffu, ra && rb)) {
            const bool got = (inl || mbar_wait(a_full(sa), pa, abort_flag, p.status, wait_ns)) &&
                             mbar_wait(b_full(sb), pb, abort_flag, p.status, wait_ns);
            ok = __all_sync(0xffffffffu, got);
            if (!ok) break;
          }
          tc_fence_after();
          const uint32_t a_lo = a_lo0 + sa * a_step;
          const uint32_t b_lo = b_lo0 + sb * b_step;
          if (++sa == SA) { sa = 0; pa ^= 1u; }
          if (++sb == SB) { sb = 0; pb ^= 1u; }
          ra = inl || mbar_test_wait(a_full(sa), pa);     // (inline mode: stage sa is slab sa, always there)
          rb = mbar_test_wait(b_full(sb), pb);
          if (elect_one()) {
#pragma unroll
            for (int q = 0; q < kParts; ++q) {
#pragma unroll
              for (int k = 0; k < kSlabK / kUmmaK8; ++k) {
                // 32 elements along K inside the swizzle span = +32 bytes = +2 in the address field
                umma_e4m3(d_tmem, desc_hi | (a_lo + q * a_part_step + 2u * k), desc_hi | (b_lo + 2u * k), idesc,
                          (ks | q | k) != 0 ? 1u : 0u);
              }
            }
            umma_commit<1>(released(slab & (kRelease - 1)));
          }
          __syncwarp();
        }
        if (!ok) break;
        if (elect_one()) umma_commit<1>(acc_full(acc));
        __syncwarp();
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2-5, 7-10)
    const int grp = warp >= 7 ? 1 : 0;
    const int ewarp = grp * 4 + (warp & 3);
    const int quad = warp & 3;
    const int row = quad * 16 + (lane & 15);     // lanes 0..15 of the quadrant hold rows 16 quad .. 16 quad + 15
    const bool has_row = lane < 16 && row < p.n; // lanes 16..31 of a quadrant hold nothing with M = 64
    float* ws = scale_area + ewarp * kBlockN;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    uint32_t ord = 0;
    const bool warp_has_rows = quad * 16 < p.n;
    const float hs = has_row ? (inl ? hs_s[row] : p.hscale[row]) : 1.0f;
    for (int unit = worker; unit < units && ok; unit += workers, ++ord) {
      float m = -INFINITY, S = 0.f, cS = 0.f, Tq = 0.f, cT = 0.f;
      int idx = kNoToken;
      int chunk = unit;
      for (int t = 0; t < T && ok; ++t) {
        const Tile tl = tile_of8(p, unit, t);
        if (tl.rows == 0) continue;
        const int v0 = tl.v0;
        const int cols = min(tl.rows, p.V - v0);
        const int half = min(cols, ((tl.rows / 2 + 31) / 32) * 32);
        const int c_begin = grp ? half : 0, c_end = grp ? cols : half;
        // this tile's weight scales into the warp's own area, before the accumulator is waited for
        __syncwarp();
#pragma unroll
        for (int j = 0; j < kBlockN / 32; ++j) {
          const int c = lane + 32 * j;
          ws[c] = (c < cols) ? __ldg(p.wscale + v0 + c) : 0.f;
        }
        __syncwarp();
        if (!mbar_wait(acc_full(acc), acc_phase, abort_flag, p.status, wait_ns)) { ok = false; break; }
        tc_fence_after();
        if (warp_has_rows) {
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + acc * kBlockN;
          for (int c0 = c_begin; c0 < c_end; c0 += 32) {
            float z[32];
            __syncwarp();
            tmem_ld32(taddr + c0, z);
            tmem_ld_wait();
            const int valid = cols - c0;
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const float4 w4 = *reinterpret_cast<const float4*>(ws + c0 + j);
              z[j] = z[j] * hs * w4.x;
              z[j + 1] = z[j + 1] * hs * w4.y;
              z[j + 2] = z[j + 2] * hs * w4.z;
              z[j + 3] = z[j + 3] * hs * w4.w;
            }
            if (valid < 32) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (j >= valid) z[j] = -1.0e30f;
            }
            float cm = fmaxf(z[0], z[1]);
#pragma unroll
            for (int j = 2; j < 32; j += 2) cm = max3(cm, z[j], z[j + 1]);
            if (cm > m) {
              if (m != -INFINITY) {
                const float dl = (cm - m) * kLog2e;
                const float sc = ex2_approx(-dl);
                Tq = sc * (Tq - dl * S);
                cT *= sc;
                S *= sc;
                cS *= sc;
              }
              m = cm;
              int first_j = 31;
#pragma unroll
              for (int j = 30; j >= 0; --j) first_j = (z[j] == cm) ? j : first_j;
              idx = v0 + c0 + first_j;
            }
            const float neg_ml = -m * kLog2e;
            const uint64_t log2e2 = pack2(kLog2e, kLog2e), neg_ml2 = pack2(neg_ml, neg_ml);
            uint64_t ls2 = pack2(0.f, 0.f), lt2 = pack2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              const uint64_t y2 = fma2(pack2(z[j], z[j + 1]), log2e2, neg_ml2);
              float y0, y1;
              unpack2(y2, y0, y1);
              const uint64_t e2 = pack2(ex2_approx(y0), ex2_approx(y1));
              ls2 = add2(ls2, e2);
              lt2 = fma2(e2, y2, lt2);
            }
            float ls0, ls1, lt0, lt1;
            unpack2(ls2, ls0, ls1);
            unpack2(lt2, lt0, lt1);
            {
              const float a = (ls0 + ls1) - cS;
              const float b = S + a;
              cS = (b - S) - a;
              S = b;
            }
            {
              const float a = (lt0 + lt1) - cT;
              const float b = Tq + a;
              cT = (b - Tq) - a;
              Tq = b;
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      Partial out;
      out.m = m;
      out.idx = idx;
      out.s = S;
      out.t = Tq * kLn2;
      if (grp == 1) {
        if (ok && ord > 0) ok = mbar_wait(xch_empty(quad), (ord - 1) & 1u, abort_flag, p.status, wait_ns);
        if (ok) {
          if (lane < 16) scratch[row] = out;
          __syncwarp();
          if (lane == 0) mbar_arrive(xch_full(quad));
        }
      } else {
        if (ok) ok = mbar_wait(xch_full(quad), ord & 1u, abort_flag, p.status, wait_ns);
        if (ok) {
          const Partial other = scratch[row];
          __syncwarp();
          if (lane == 0) mbar_arrive(xch_empty(quad));
          out = merge(out, other);
          if (has_row) p.partials[static_cast<size_t>(row) * p.chunks + chunk] = out;
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<1>(tmem_base, kTmemCols);
  }
}

int tc8_threads() { return kThreads; }
int tc8_max_rows() { return 64; }

void tc8_configure(int n, int d, Tc8Config* c) {
  int a_rows = ((n + 15) / 16) * 16;
  if (a_rows < 16) a_rows = 16;
  if (a_rows > 64) a_rows = 64;
  const int a_stage = kParts * a_rows * kRowBytes;
  const int b_stage = kBlockN * kRowBytes;
  const int k_slabs = (d + kSlabK - 1) / kSlabK;
  const int budget = kSmemLimit - 1024 - kBarrierBytes - kScratchBytes - kScaleBytes - 64;
  // n <= 16 and all of h (two parts) small enough: the kernel splits h itself and keeps it resident, one
  // launch less (decode16-sized step 36.8 -> 35.0 us).  TLR_TC8_INLINE=0 is a tuning switch that keeps the
  // separate split kernel.
  const char* env = getenv("TLR_TC8_INLINE");
  bool inl = n <= 16 && k_slabs <= 16 && !(env != nullptr && env[0] == '0');
  // ... and only while the resident copy leaves the W ring five stages: with four (d = 2048) what the
  // missing launch gains is lost again to the shallower ring (measured: 56.0 vs 56.8 and 58.6 vs 57.9 us)
  if (inl && (budget - k_slabs * a_stage) / b_stage < 5) inl = false;
  int sa = inl ? k_slabs : (a_rows <= 32 ? 6 : 4);
  int sb = (budget - sa * a_stage) / b_stage;
  if (sb > kMaxBStages) sb = kMaxBStages;
  c->a_rows = a_rows;
  c->a_stages = sa;
  c->b_stages = sb;
  c->inline_split = inl ? 1 : 0;
  c->smem_bytes = 1024 + sa * a_stage + sb * b_stage + kBarrierBytes + kScratchBytes + kScaleBytes + 64;
}

cudaError_t tc8_prepare() {
  return cudaFuncSetAttribute(tc8_projection_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
}

cudaError_t launch_h_split(const void* h_bf16, int n, int d, int rows_alloc, uint8_t* parts, float* hscale,
                           cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(rows_alloc), 1, 1);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, h_split_kernel, static_cast<const __nv_bfloat16*>(h_bf16), n, d, rows_alloc, parts,
                            hscale);
}

cudaError_t launch_tc8_projection(const CUtensorMap& map_h, const CUtensorMap& map_w128, const CUtensorMap& map_w64,
                                  const CUtensorMap& map_w16, const Tc8Params& p, const Tc8Config& c, int workers,
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
  return cudaLaunchKernelEx(&cfg, tc8_projection_kernel, map_h, map_w128, map_w64, map_w16, p);
}

}  // namespace tlr
