// Tensor-core projection kernel for sm_100a: the LM-head contraction z = h W^T on
// tcgen05 with the accumulator in tensor memory, operands staged by TMA, and the
// online-softmax reduction (max / argmax / sum-exp / entropy numerator) fused into
// the epilogue, so the n x V logits never leave the SM.
//
// Decomposition.  The vocabulary is cut into `chunks` contiguous ranges of 16-row
// granules; the token rows into units of 128 (one TMEM lane per row).  A work unit is
// (chunk, row unit); units are numbered chunk-major so that CTAs running at the same
// time share W tiles through L2, and each persistent CTA takes units blockIdx.x,
// blockIdx.x + gridDim.x, ...  Inside a unit the chunk is walked in tiles of at most
// 256 vocabulary rows (the MMA's N), each a K-loop over d in slabs of 64 elements.
//
// Roles (warp-specialised, 192 threads):
//   warp 0   TMA producer: fills a ring of kStages {h slab 128x64, W slab Nx64} buffers
//   warp 1   MMA issuer: one thread issues tcgen05.mma (M=128, N=tile, K=16) x4 per slab
//            into one of two 256-column TMEM accumulators; also owns TMEM alloc/free
//   warps 2-5 epilogue: each owns 32 TMEM lanes (rows); reads the finished accumulator
//            32 columns at a time and folds it into per-row (m, idx, S, T) registers
//            while the next tile's MMAs run into the other accumulator.
// At the end of a unit every row's summary is written as one 16-byte partial.
//
// Every mbarrier wait is bounded (wall-clock limit); on expiry the kernel raises
// TLR_DEV_WAIT_TIMEOUT, drains its outstanding copies, frees TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "tlr_common.cuh"
#include "tlr_tc.cuh"

namespace tlr {

namespace {

constexpr int kBlockM = 128;                 // token rows per unit == TMEM lanes
constexpr int kBlockN = 256;                 // max vocabulary rows per tile == accumulator columns
constexpr int kBlockK = 64;                  // bf16 per slab row = 128 B = one swizzle span
constexpr int kUmmaK = 16;
constexpr int kStages = 4;
constexpr int kABytes = kBlockM * kBlockK * 2;   // 16 KiB
constexpr int kBBytes = kBlockN * kBlockK * 2;   // 32 KiB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kTmemCols = 512;
constexpr int kEpiWarps = 4;
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kBarrierBytes = 256;
constexpr int kSmemBytes = 1024 + kStages * kStageBytes + kBarrierBytes;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Bounded wait.  Returns false when the limit expired or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          uint32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicOr(status, TLR_DEV_WAIT_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Arrive on an mbarrier once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives row (lane base + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, laid out
// by TMA with the 128-byte swizzle: 8-row groups 1024 bytes apart (stride offset 64 in
// 16-byte units), leading offset unused (1), descriptor version 1, layout code 2.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t dsc = 0;
  dsc |= static_cast<uint64_t>((saddr & 0x3ffffu) >> 4);
  dsc |= static_cast<uint64_t>(1) << 16;
  dsc |= static_cast<uint64_t>(1024 >> 4) << 32;
  dsc |= static_cast<uint64_t>(1) << 46;
  dsc |= static_cast<uint64_t>(2) << 61;
  return dsc;
}

// Instruction descriptor: fp32 accumulator, bf16 A and B, both K-major, M = 128, N = n_cols.
__device__ __forceinline__ uint32_t instr_desc(int n_cols) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n_cols >> 3) << 17) |
         (static_cast<uint32_t>(kBlockM >> 4) << 24);
}

struct UnitRange {
  int row0;      // first token row of the unit
  int g0, g1;    // granule range of the chunk
};

__device__ __forceinline__ UnitRange unit_range(const TcParams& p, int unit) {
  UnitRange u;
  const int chunk = unit / p.row_units;
  const int ru = unit - chunk * p.row_units;
  u.row0 = ru * kBlockM;
  u.g0 = static_cast<int>((static_cast<long long>(p.granules) * chunk) / p.chunks);
  u.g1 = static_cast<int>((static_cast<long long>(p.granules) * (chunk + 1)) / p.chunks);
  return u;
}

// Tile t of a chunk of G granules split as evenly as possible into T tiles.
__device__ __forceinline__ void tile_range(int G, int T, int t, int* a, int* b) {
  *a = (G * t) / T;
  *b = (G * (t + 1)) / T;
}

}  // namespace

__global__ void __launch_bounds__(kThreads, 1)
tc_projection_kernel(const __grid_constant__ CUtensorMap map_h,
                     const __grid_constant__ CUtensorMap map_w64,
                     const __grid_constant__ CUtensorMap map_w16,
                     const TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment: the swizzle pattern is a function of the shared-memory address.
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = base + kStages * kStageBytes;
  // barrier block: full[kStages], empty[kStages], acc_full[2], acc_empty[2], then tmem slot + abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto acc_full_bar = [&](int b) { return bar_base + 8u * (2 * kStages + b); };
  auto acc_empty_bar = [&](int b) { return bar_base + 8u * (2 * kStages + 2 + b); };
  unsigned char* gen_base = smem_raw + (base - smem_u32(smem_raw));
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + kStages * kStageBytes + 8 * (2 * kStages + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full_bar(b), 1);
      mbar_init(acc_empty_bar(b), kEpiWarps);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int k_slabs = (p.d + kBlockK - 1) / kBlockK;
  const int units = p.chunks * p.row_units;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;  // slabs issued in total
      bool ok = true;
      for (int unit = blockIdx.x; unit < units && ok; unit += gridDim.x) {
        const UnitRange u = unit_range(p, unit);
        const int G = u.g1 - u.g0;
        const int T = (G * 16 + kBlockN - 1) / kBlockN;
        for (int t = 0; t < T && ok; ++t) {
          int ga, gb;
          tile_range(G, T, t, &ga, &gb);
          const int v0 = (u.g0 + ga) * 16;
          const int rows = (gb - ga) * 16;
          for (int ks = 0; ks < k_slabs; ++ks) {
            if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
            const uint32_t sa = base + stage * kStageBytes;
            const uint32_t sb = sa + kABytes;
            mbar_expect_tx(full_bar(stage), kABytes + rows * (kBlockK * 2));
            tma_load_2d(sa, &map_h, full_bar(stage), ks * kBlockK, u.row0);
            int r = 0;
            for (; rows - r >= 64; r += 64)
              tma_load_2d(sb + r * (kBlockK * 2), &map_w64, full_bar(stage), ks * kBlockK, v0 + r);
            for (; rows - r >= 16; r += 16)
              tma_load_2d(sb + r * (kBlockK * 2), &map_w16, full_bar(stage), ks * kBlockK, v0 + r);
            ++issued;
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
      if (!ok) {
        // Drain: wait (bounded) until every slab already issued has landed, so that no
        // copy is still writing shared memory when the CTA exits.
        const int pending = issued < kStages ? issued : kStages;
        int s = stage;
        uint32_t ph = phase;
        for (int i = 0; i < pending; ++i) {
          if (--s < 0) { s = kStages - 1; ph ^= 1u; }
          const unsigned long long t0 = global_ns();
          while (!mbar_try_wait(full_bar(s), ph) && global_ns() - t0 < kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int unit = blockIdx.x; unit < units && ok; unit += gridDim.x) {
        const UnitRange u = unit_range(p, unit);
        const int G = u.g1 - u.g0;
        const int T = (G * 16 + kBlockN - 1) / kBlockN;
        for (int t = 0; t < T && ok; ++t) {
          int ga, gb;
          tile_range(G, T, t, &ga, &gb);
          const uint32_t idesc = instr_desc((gb - ga) * 16);
          if (!mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + acc * kBlockN;
          for (int ks = 0; ks < k_slabs; ++ks) {
            if (!mbar_wait(full_bar(stage), phase, abort_flag, p.status)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sa = base + stage * kStageBytes;
            const uint64_t a_desc = smem_desc_sw128(sa);
            const uint64_t b_desc = smem_desc_sw128(sa + kABytes);
#pragma unroll
            for (int k = 0; k < kBlockK / kUmmaK; ++k) {
              // advancing 16 elements along K inside the swizzle span = +32 bytes = +2 in the address field
              umma_bf16(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (ks | k) != 0 ? 1u : 0u);
            }
            umma_commit(empty_bar(stage));  // frees the slab once these MMAs have read it
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          umma_commit(acc_full_bar(acc));   // accumulator complete
          if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quad = warp & 3;               // TMEM lane quadrant this warp may read
    const int row_in_unit = quad * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int unit = blockIdx.x; unit < units && ok; unit += gridDim.x) {
      const UnitRange u = unit_range(p, unit);
      const int chunk = unit / p.row_units;
      const int G = u.g1 - u.g0;
      const int T_tiles = (G * 16 + kBlockN - 1) / kBlockN;
      const bool warp_has_rows = (u.row0 + quad * 32) < p.n;   // warp-uniform
      // Running summary of this thread's row over the unit.  S = sum 2^y and T = sum 2^y * y
      // with y = (z - m) * log2(e) <= 0; both are accumulated per 32-column group first and
      // then added with a compensated (Kahan) sum, so that one dominant term -- a confident
      // row has S ~ 1 with thousands of terms ~1e-8 after it -- does not swallow the rest.
      float m = -INFINITY, S = 0.f, cS = 0.f, T = 0.f, cT = 0.f;
      int idx = kNoToken;
      for (int t = 0; t < T_tiles && ok; ++t) {
        int ga, gb;
        tile_range(G, T_tiles, t, &ga, &gb);
        const int v0 = (u.g0 + ga) * 16;
        const int cols = min((gb - ga) * 16, p.V - v0);   // valid columns of this tile
        if (!mbar_wait(acc_full_bar(acc), acc_phase, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        if (warp_has_rows) {
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + acc * kBlockN;
          for (int c0 = 0; c0 < cols; c0 += 32) {
            float z[32];
            __syncwarp();                           // the load below is warp-collective
            tmem_ld32(taddr + c0, z);
            tmem_ld_wait();
            const int valid = cols - c0;
            if (valid < 32) {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (j >= valid) z[j] = -1.0e30f;   // finite, so 0 * y stays 0 below
            }
            float cm = z[0];
#pragma unroll
            for (int j = 1; j < 32; ++j) cm = fmaxf(cm, z[j]);
            if (cm > m) {
              if (m != -INFINITY) {
                const float dl = (cm - m) * kLog2e;       // > 0
                const float sc = ex2_approx(-dl);
                T = sc * (T - dl * S);
                cT *= sc;
                S *= sc;
                cS *= sc;
              }
              m = cm;
              int first = 31;
#pragma unroll
              for (int j = 30; j >= 0; --j) first = (z[j] == cm) ? j : first;
              idx = v0 + c0 + first;
            }
            const float neg_ml = -m * kLog2e;
            float ls0 = 0.f, ls1 = 0.f, lt0 = 0.f, lt1 = 0.f;
#pragma unroll
            for (int j = 0; j < 32; j += 2) {
              const float y0 = fmaf(z[j], kLog2e, neg_ml);
              const float y1 = fmaf(z[j + 1], kLog2e, neg_ml);
              const float e0 = ex2_approx(y0);
              const float e1 = ex2_approx(y1);
              ls0 += e0;
              ls1 += e1;
              lt0 = fmaf(e0, y0, lt0);
              lt1 = fmaf(e1, y1, lt1);
            }
            {
              const float a = (ls0 + ls1) - cS;
              const float b = S + a;
              cS = (b - S) - a;
              S = b;
            }
            {
              const float a = (lt0 + lt1) - cT;
              const float b = T + a;
              cT = (b - T) - a;
              T = b;
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(acc_empty_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (ok && u.row0 + row_in_unit < p.n) {
        Partial out;
        out.m = m;
        out.idx = idx;
        out.s = S;
        out.t = T * kLn2;              // sum e^(z-m) (z-m), back in nats
        p.partials[static_cast<size_t>(u.row0 + row_in_unit) * p.chunks + chunk] = out;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

int tc_smem_bytes() { return kSmemBytes; }
int tc_threads() { return kThreads; }

cudaError_t tc_prepare() {
  return cudaFuncSetAttribute(tc_projection_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
}

cudaError_t launch_tc_projection(const CUtensorMap& map_h, const CUtensorMap& map_w64, const CUtensorMap& map_w16,
                                 const TcParams& p, int grid, cudaStream_t stream) {
  tc_projection_kernel<<<grid, kThreads, kSmemBytes, stream>>>(map_h, map_w64, map_w16, p);
  return cudaGetLastError();
}

}  // namespace tlr
