// Tensor-core projection kernel for sm_100a: the LM-head contraction z = h W^T on
// tcgen05 with the accumulator in tensor memory, operands staged by TMA, and the
// online-softmax reduction (max / argmax / sum-exp / entropy numerator) fused into
// the epilogue, so the n x V logits never leave the SM.
//
// One kernel body, three instantiations (two kernels at the end of this file):
//   <1, false>  bf16 head, one CTA per worker, MMA M = 128 token rows     (n <= 128; M = 64 when n <= 64)
//   <2, false>  bf16 head, a cluster of two CTAs per worker, MMA M = 256 rows (cta_group::2): each
//               CTA stages its own 128 rows of h and HALF of the W tile, and the pair's
//               tensor cores read both halves, so a W byte enters shared memory once
//               per 256 token rows.                                       (n > 128)
//   <1, true>   8-bit (e4m3) head for decode batches of at most 128 rows: h is the sum of two e4m3
//               parts, stacked in one operand slab (rows 0.. = first parts, rows part_rows.. =
//               second parts).  Up to 64 rows ONE kind::f8f6f4 MMA per K step covers both parts
//               along its M, and the epilogue adds the two accumulator rows of a token before it
//               folds them; above, two MMAs per K step (one per part) add into the same rows.
//
// Decomposition.  The vocabulary is cut into `chunks` contiguous ranges of granules
// (a multiple of 16 * kCta rows); the token rows into units of 128 * kCta.  A work unit is
// (chunk, row unit); units are numbered chunk-major so that workers running at the
// same time share W through L2, and worker w takes units w, w + workers, ...  Inside
// a unit the chunk is walked in `tiles_per_unit` tiles of at most 256 vocabulary rows
// (the MMA's N), each a K-loop over d in slabs of 128 bytes per row.  With a learned router
// attached (bf16 head) one more unit per row unit follows the vocabulary units: its "vocabulary"
// is the rows of the router's first layer W1, and its epilogue applies bias, ReLU and the output
// layer's weights and sums over the hidden units instead of folding a softmax.
//
// Roles (warp-specialised, 352 threads per CTA):
//   warp 0   W producer: TMA loads of W slabs into a deep ring (W comes from HBM).  W never
//            depends on the previous kernel in the stream, so this warp does not wait for it:
//            under programmatic dependent launch the ring fills while that kernel finishes.
//   warp 6   h producer: TMA loads of h slabs into a short ring (h comes from L2)
//   warp 1   MMA issuer (leader CTA only): tcgen05.mma x4 per slab into one of two
//            256-column TMEM accumulators; also owns TMEM alloc/free
//   warps 2-5 and 7-10  epilogue, two warps per TMEM lane quadrant (32 rows): the first
//            group folds the lower half of a finished accumulator's columns, the second
//            group the upper half, 32 columns at a time, into per-row (m, idx, S, T)
//            registers while the next tile's MMAs run into the other accumulator.  Two
//            warps per scheduler hide each other's tensor-memory load and exp latency, and
//            the time between a worker's last MMA and its last partial -- which nothing
//            overlaps -- halves.
// At the end of a unit the second group hands its summary to the first through shared memory
// and every row's summary is written as one 16-byte partial.
//
// How much of W a CTA keeps in flight decides its streaming rate (latency-bound
// otherwise), so h slabs get their own small ring and, when n is small, a slab of only
// as many rows as n needs; the MMA then reads its remaining A rows from whatever
// follows in shared memory, which only affects accumulator rows that are never used.
//
// Every mbarrier wait is bounded (wall-clock limit); on expiry the kernel raises
// TLR_DEV_WAIT_TIMEOUT, lets its outstanding copies land, frees TMEM and returns.
// No TMA load uses cluster multicast.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>

#include <type_traits>

#include "tlr_common.cuh"
#include "tlr_tc.cuh"
#include "tlr_tc8_dev.cuh"
#include "tlr_tc_ptx.cuh"

namespace tlr {

namespace {

constexpr int kBlockM = 128;                 // token rows per CTA == TMEM lanes
constexpr int kBlockN = 256;                 // max vocabulary rows per tile == accumulator columns
constexpr int kRowBytes = 128;               // bytes per slab row = one swizzle span (64 bf16 or 128 e4m3)
constexpr int kTmemCols = 512;
constexpr int kEpiWarps = 8;                 // two groups of four (one warp per TMEM lane quadrant each)
constexpr int kThreads = 32 * 11;
constexpr int kMaxAStages = 16;              // (the 8-bit head keeps up to 16 resident slabs of h)
constexpr int kMaxBStages = 12;
constexpr int kRelease = 16;                 // >= every ring depth that streams (see the barrier notes in the kernel)
constexpr int kBarrierBytes = 640;
constexpr int kScratchBytes = kBlockM * 16;  // one Partial per row: hand-over between the epilogue groups
constexpr int kSmemLimit = 232448;           // 227 KiB opt-in maximum per CTA
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s
// 8-bit head: weight scales of a tile for each of the four warps that fold, the rows' power-of-two scales,
// and four hand-over buffers (32 columns x lanes floats) between the warps that hold a token's two parts
// (with more than 64 rows nothing is handed over and the buffers' space holds the scales for all eight warps)
constexpr int kScaleBytes = 4 * kBlockN * 4;
constexpr int kRowScaleBytes = 64 * 4;
__host__ __device__ constexpr int tc8_extra_bytes(int part_rows) {
  return kScaleBytes + kRowScaleBytes + 4 * 32 * 4 * (part_rows > 32 ? 32 : 16);
}

// The static schedule, identical in every role: worker w walks units w, w + workers, ...;
// each unit is `tiles_per_unit` tiles (possibly empty ones when the chunk is short).
struct Unit {
  int row0;    // first token row of this CTA in the unit
  int chunk;   // vocabulary chunk; -1 for a learned-router unit
  int g0;      // first granule of the chunk
  int G;       // granules in the chunk
};
struct Tile {
  int v0;      // first vocabulary row of the tile (first row of W1 in a learned-router unit)
  int rows;    // vocabulary rows in the tile (multiple of 16 * kCta); 0 = empty tile
};

// What is fixed for a whole unit (the divisions happen here, once per unit: the tile walk of the MMA-issuing
// warp is on the tensor pipe's critical path and must stay cheap).
template <int kCta>
__host__ __device__ __forceinline__ Unit unit_of(const TcParams& p, int unit, int cta_rank) {
  Unit u;
  const int vocab_units = p.chunks * p.row_units;
  if (unit >= vocab_units) {          // learned-router unit: all rows of W1 for one row unit
    u.chunk = -1;
    u.row0 = ((unit - vocab_units) * kCta + cta_rank) * kBlockM;
    u.g0 = 0;
    u.G = 0;
    return u;
  }
  u.chunk = unit / p.row_units;
  const int ru = unit - u.chunk * p.row_units;
  u.row0 = (ru * kCta + cta_rank) * kBlockM;
  u.g0 = static_cast<int>((static_cast<long long>(p.granules) * u.chunk) / p.chunks);
  const int g1 = static_cast<int>((static_cast<long long>(p.granules) * (u.chunk + 1)) / p.chunks);
  u.G = g1 - u.g0;
  return u;
}

__host__ __device__ __forceinline__ Tile tile_of(const TcParams& p, const Unit& u, int t) {
  Tile r;
  if (u.chunk < 0) {                  // learned-router unit: full 256-row tiles over the rows of W1
    r.v0 = t * kBlockN;
    const int left = p.mlp_rows - r.v0;
    r.rows = left <= 0 ? 0 : (left < kBlockN ? left : kBlockN);
    return r;
  }
  int ga, gb;
  if (p.full_tiles_first) {
    // as many full 256-row tiles as fit, then one remainder tile: a tile costs a pass over all
    // of h whatever its width, so the fewest, widest tiles are the cheapest
    const int full = kBlockN / p.granule_rows;
    ga = full * t < u.G ? full * t : u.G;
    gb = full * (t + 1) < u.G ? full * (t + 1) : u.G;
  } else {
    ga = (u.G * t) / p.tiles_per_unit;
    gb = (u.G * (t + 1)) / p.tiles_per_unit;
  }
  r.v0 = (u.g0 + ga) * p.granule_rows;
  r.rows = (gb - ga) * p.granule_rows;
  return r;
}

// Running online-softmax summary of one token row over the vocabulary rows a thread has seen.
// S = sum 2^y and T = sum 2^y * y with y = (z - m) * log2(e) <= 0; both are accumulated per
// 32-column group first and then added with a compensated (Kahan) sum, so that one dominant term -- a
// confident row has S ~ 1 with thousands of terms ~1e-8 after it -- does not swallow the rest.
struct RowFold {
  float m, S, cS, Tq, cT;
  int idx;
  __device__ __forceinline__ void reset() {
    m = -INFINITY;
    S = cS = Tq = cT = 0.f;
    idx = kNoToken;
  }
  // Folds 32 consecutive logits z[0..32) whose first has vocabulary index col0; only the first
  // `valid` of them exist (the rest lie beyond V).
  __device__ __forceinline__ void group(float (&z)[32], int valid, int col0) {
    if (valid < 32) {
#pragma unroll
      for (int j = 0; j < 32; ++j)
        if (j >= valid) z[j] = -1.0e30f;   // finite, so 0 * y stays 0 below
    }
    float cm = fmaxf(z[0], z[1]);
#pragma unroll
    for (int j = 2; j < 32; j += 2) cm = max3(cm, z[j], z[j + 1]);
    if (cm > m) {
      if (m != -INFINITY) {
        const float dl = (cm - m) * kLog2e;       // > 0
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
      idx = col0 + first_j;
    }
    const float neg_ml = -m * kLog2e;
    const uint64_t log2e2 = pack2(kLog2e, kLog2e), neg_ml2 = pack2(neg_ml, neg_ml);
    uint64_t ls2 = pack2(0.f, 0.f), lt2 = pack2(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < 32; j += 2) {
      const uint64_t y2 = fma2(pack2(z[j], z[j + 1]), log2e2, neg_ml2);   // (z - m) * log2(e)
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
  __device__ __forceinline__ Partial result() const {
    Partial out;
    out.m = m;
    out.idx = idx;
    out.s = S;
    out.t = Tq * kLn2;             // sum e^(z-m) (z-m), back in nats
    return out;
  }
};

}  // namespace

// The kernel body (maps and p are the kernel's own parameters, maps a __grid_constant__ one: TMA reads the
// tensor maps from parameter space).
template <int kCta, bool kFp8>
__device__ __forceinline__ void tc_projection_body(const TcMaps& maps, const TcParams& p) {
  static_assert(!(kFp8 && kCta != 1), "the 8-bit head runs with one CTA per worker");
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment: the swizzle pattern is a function of the shared-memory address.
  // (The dynamic shared memory of both CTAs of a pair starts at the same offset, so the
  // two CTAs compute identical offsets -- which the pair MMA and the peer signals rely on.)
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int SA = p.a_stages, SB = p.b_stages;
  const uint32_t a_stage_bytes = static_cast<uint32_t>(p.a_rows) * kRowBytes;
  constexpr uint32_t b_stage_bytes = (kBlockN / kCta) * kRowBytes;
  constexpr int kSlabElems = kFp8 ? kRowBytes : kRowBytes / 2;   // K elements per slab
  const uint32_t a_ring = base;
  const uint32_t b_ring = base + SA * a_stage_bytes;
  const uint32_t bar_base = b_ring + SB * b_stage_bytes;
  // Barriers: a_full / b_full per ring stage (data landed); released[j] completes when the
  // MMAs of slab number j (mod kRelease) have finished reading shared memory -- one commit
  // per slab serves both rings: the producer of slab i waits for slab i - depth;
  // acc_full / acc_empty per accumulator.
  auto a_full = [&](int s) { return bar_base + 8u * s; };
  auto b_full = [&](int s) { return bar_base + 8u * (kMaxAStages + s); };
  auto released = [&](int j) { return bar_base + 8u * (kMaxAStages + kMaxBStages + j); };
  constexpr int kFixed = kMaxAStages + kMaxBStages + kRelease;
  auto acc_full = [&](int b) { return bar_base + 8u * (kFixed + b); };
  auto acc_empty = [&](int b) { return bar_base + 8u * (kFixed + 2 + b); };
  // xch_full[q]: the second epilogue group's summary of quadrant q is in the scratch block;
  // xch_empty[q]: the first group has read it.
  auto xch_full = [&](int q) { return bar_base + 8u * (kFixed + 4 + q); };
  auto xch_empty = [&](int q) { return bar_base + 8u * (kFixed + 8 + q); };
  // 8-bit head: hx_full[c] / hx_empty[c]: hand-over buffer c holds / has given up 32 columns of second-part sums;
  // h_ready: h has been split in place (inline mode)
  auto hx_full = [&](int c) { return bar_base + 8u * (kFixed + 12 + c); };
  auto hx_empty = [&](int c) { return bar_base + 8u * (kFixed + 16 + c); };
  const uint32_t h_ready = bar_base + 8u * (kFixed + 20);
  constexpr int kNumBarriers = kFixed + 21;
  static_assert(kNumBarriers * 8 + 16 <= kBarrierBytes, "barrier block too small");
  unsigned char* gen_base = smem_raw + (base - smem_u32(smem_raw));
  unsigned char* tail = gen_base + (bar_base - base);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 8 * kNumBarriers);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  Partial* scratch = reinterpret_cast<Partial*>(tail + kBarrierBytes);
  float* scale_area = reinterpret_cast<float*>(tail + kBarrierBytes + kScratchBytes);   // 8-bit head only
  float* hs_s = scale_area + kScaleBytes / 4;
  float* hx_area = hs_s + kRowScaleBytes / 4;
  const bool inl = kFp8 && p.inline_split != 0;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t cta_rank = (kCta == 2) ? cluster_ctarank() : 0u;
  const bool leader = cta_rank == 0;
  const int worker = blockIdx.x / kCta;
  const int workers = gridDim.x / kCta;

  if (threadIdx.x == 0) {
    if (!inl) for (int s = 0; s < SA; ++s) mbar_init(a_full(s), 1);   // (inline mode: SA = K slabs, nothing streams)
    for (int s = 0; s < SB; ++s) mbar_init(b_full(s), 1);
    for (int j = 0; j < kRelease; ++j) mbar_init(released(j), 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full(b), 1);
      mbar_init(acc_empty(b), kEpiWarps * kCta);
    }
    for (int q = 0; q < 4; ++q) {
      mbar_init(xch_full(q), 1);
      mbar_init(xch_empty(q), 1);
      if (kFp8) {
        mbar_init(hx_full(q), 1);
        mbar_init(hx_empty(q), 1);
      }
    }
    if (kFp8) mbar_init(h_ready, 9);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc<kCta>(smem_u32(tmem_slot), kTmemCols);
    tmem_relinquish<kCta>();
  }
  tc_fence_before();
  __syncthreads();
  if (kCta == 2) cluster_sync_all();   // the peer's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Programmatic dependent launch: everything above overlapped the tail of the previous
  // kernel in the stream; from here on its results (h, and the workspace the previous
  // merge kernel was still reading) are needed, so wait for it, then let the merge kernel
  // that follows this one be scheduled early.  The W producer reads only W and the tensor
  // maps, which no kernel writes when W belongs to a context, so it goes ahead (entry points
  // that take W per call set w_wait).
  if (warp != 0 || p.w_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // With at most 64 operand rows (one CTA per worker) the MMAs run with M = 64: such an instruction takes
  // about two thirds of the time of an M = 128 one, and the padding rows were wasted work anyway.  Its
  // accumulator row r lives in TMEM lane 32 * (r / 16) + r % 16, i.e. in lanes 0..15 of each 32-lane
  // quadrant (checked on the device), so an epilogue warp then holds 16 rows instead of 32.
  const bool m64 = kCta == 1 && p.a_rows <= 64;
  // 8-bit head with more than 64 token rows: the two parts of h no longer fit one MMA's M (128 at most with one
  // CTA), so every K step issues two MMAs -- first parts, then second parts, into the same accumulator rows --
  // and the epilogue reads finished logits as on the bf16 head (no hand-over between warps).
  const bool wide = kFp8 && p.part_rows > 64;
  const int k_slabs = (p.d + kSlabElems - 1) / kSlabElems;
  const int units = (p.chunks + (p.mlp_hidden > 0 ? 1 : 0)) * p.row_units;
  const int T = p.tiles_per_unit;
  const unsigned long long wait_ns = p.wait_limit_ns != 0 ? p.wait_limit_ns : kWaitLimitNs;

  if (inl && warp >= 2) {
    // ---- 8-bit head, n <= 16: the nine warps that have nothing to do yet split h into its two e4m3
    // parts, straight into the resident operand slabs
    static_assert(kThreads - 64 == kSplitThreads, "warps 2..10 split h");
    split_h_resident(static_cast<const __nv_bfloat16*>(p.h), p.n, p.d, k_slabs, gen_base, hs_s, threadIdx.x - 64);
    __syncwarp();
    if (lane == 0) mbar_arrive(h_ready);
  }

  if (warp == 0) {
    // ------------------------------------------------------------------ W producer
    if (lane == 0) {
      int stage = 0;
      int slab = 0;     // running slab number, the same in every role
      bool ok = true;
      for (int unit = worker; unit < units && ok; unit += workers) {
        const Unit un = unit_of<kCta>(p, unit, cta_rank);
        for (int t = 0; t < T && ok; ++t) {
          const Tile tl = tile_of(p, un, t);
          if (tl.rows == 0) continue;
          const int my_rows = tl.rows / kCta;                 // this CTA's share of the tile
          const int my_v0 = tl.v0 + static_cast<int>(cta_rank) * my_rows;
          const bool mlp = !kFp8 && un.chunk < 0;
          const CUtensorMap* m128 = mlp ? &maps.m128 : &maps.w128;
          const CUtensorMap* m64p = mlp ? &maps.m64 : &maps.w64;
          const CUtensorMap* m16 = mlp ? &maps.m16 : &maps.w16;
          for (int ks = 0; ks < k_slabs; ++ks, ++slab) {
            if (slab >= SB) {     // the stage is free once slab - SB has been consumed
              const int j = slab - SB;
              if (!mbar_wait(released(j & (kRelease - 1)), (j / kRelease) & 1, abort_flag, p.status, wait_ns)) { ok = false; break; }
            }
            const uint32_t dst = b_ring + stage * b_stage_bytes;
            const uint32_t bar = (kCta == 2) ? map_to_cta(b_full(stage), 0) : b_full(stage);
            if (p.debug_drop_w_copies) continue;   // test hook: the copies are "lost", the consumer's wait runs out
            if (leader) mbar_expect_tx(b_full(stage), tl.rows * kRowBytes);   // both CTAs' bytes
            int r = 0;
            for (; my_rows - r >= 128; r += 128)
              tma_load_2d<kCta>(dst + r * kRowBytes, m128, bar, ks * kSlabElems, my_v0 + r);
            for (; my_rows - r >= 64; r += 64)
              tma_load_2d<kCta>(dst + r * kRowBytes, m64p, bar, ks * kSlabElems, my_v0 + r);
            for (; my_rows - r >= 16; r += 16)
              tma_load_2d<kCta>(dst + r * kRowBytes, m16, bar, ks * kSlabElems, my_v0 + r);
            if (++stage == SB) stage = 0;
          }
        }
      }
      if (!ok) drain_delay();
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------------ h producer
    // (8-bit head: the map covers the two parts stacked, [2 * part_rows][d], so one box is the whole operand slab)
    if (lane == 0 && !inl) {
      int stage = 0;
      int slab = 0;
      bool ok = true;
      for (int unit = worker; unit < units && ok; unit += workers) {
        const Unit un = unit_of<kCta>(p, unit, cta_rank);
        for (int t = 0; t < T && ok; ++t) {
          const Tile tl = tile_of(p, un, t);
          if (tl.rows == 0) continue;
          for (int ks = 0; ks < k_slabs; ++ks, ++slab) {
            if (slab >= SA) {
              const int j = slab - SA;
              if (!mbar_wait(released(j & (kRelease - 1)), (j / kRelease) & 1, abort_flag, p.status, wait_ns)) { ok = false; break; }
            }
            const uint32_t dst = a_ring + stage * a_stage_bytes;
            const uint32_t bar = (kCta == 2) ? map_to_cta(a_full(stage), 0) : a_full(stage);
            if (leader) mbar_expect_tx(a_full(stage), a_stage_bytes * kCta);
            tma_load_2d<kCta>(dst, &maps.h, bar, ks * kSlabElems, kFp8 ? 0 : un.row0);
            if (++stage == SA) stage = 0;
          }
        }
      }
      if (!ok) drain_delay();
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp walks the schedule and waits on the barriers, so that control flow
    // and operands stay warp-uniform; one elected lane issues the MMAs and commits.
    if (leader) {
      int sa = 0, sb = 0;
      uint32_t pa = 0, pb = 0;
      int slab = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      // Descriptor words: the low word carries the start address (in 16-byte units) and the
      // leading offset; the high word is constant.
      const uint64_t desc_hi = smem_desc_sw128(0) & 0xffffffff00000000ull;
      const uint32_t desc_lo_fixed = static_cast<uint32_t>(smem_desc_sw128(0) & 0xffffffffull);
      const uint32_t a_lo0 = desc_lo_fixed | ((a_ring & 0x3ffffu) >> 4);
      const uint32_t b_lo0 = desc_lo_fixed | ((b_ring & 0x3ffffu) >> 4);
      const uint32_t a_step = a_stage_bytes >> 4, b_step = b_stage_bytes >> 4;
      const int mma_m = m64 ? 64 : kBlockM * kCta;
      const uint32_t part_off = static_cast<uint32_t>(p.part_rows * kRowBytes) >> 4;   // second parts, in descriptor units
      if (inl) {                                  // h is resident once the nine warps have split it
        ok = __all_sync(0xffffffffu, mbar_wait(h_ready, 0, abort_flag, p.status, wait_ns));
        tc_fence_after();
      }
      // The barrier state of the next slab is polled before the current slab's MMAs are
      // issued, so the poll's latency overlaps the issue instead of adding to it.
      bool ra = inl || mbar_test_wait(a_full(0), 0), rb = mbar_test_wait(b_full(0), 0);
      for (int unit = worker; unit < units && ok; unit += workers) {
        const Unit un = unit_of<kCta>(p, unit, 0);
        for (int t = 0; t < T && ok; ++t) {
          const Tile tl = tile_of(p, un, t);
          if (tl.rows == 0) continue;
          const uint32_t idesc = kFp8 ? instr_desc_e4m3(mma_m, tl.rows) : instr_desc(mma_m, tl.rows);
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
              for (int k = 0; k < 4; ++k) {
                // a quarter of the swizzle span along K (16 bf16 or 32 e4m3) = +32 bytes = +2 in the address field
                if (kFp8) {
                  umma_e4m3(d_tmem, desc_hi | (a_lo + 2u * k), desc_hi | (b_lo + 2u * k), idesc, (ks | k) != 0 ? 1u : 0u);
                  if (wide) umma_e4m3(d_tmem, desc_hi | (a_lo + part_off + 2u * k), desc_hi | (b_lo + 2u * k), idesc, 1u);
                } else
                  umma_bf16<kCta>(d_tmem, desc_hi | (a_lo + 2u * k), desc_hi | (b_lo + 2u * k), idesc,
                                  (ks | k) != 0 ? 1u : 0u);
              }
              umma_commit<kCta>(released(slab & (kRelease - 1)));   // both slabs are free once these MMAs are done
            }
            __syncwarp();
          }
          if (!ok) break;
          if (elect_one()) umma_commit<kCta>(acc_full(acc));   // accumulator complete (in both CTAs of a pair)
          __syncwarp();
          if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2-5, 7-10)
    const int grp = warp >= 7 ? 1 : 0;       // 0: lower half of a tile's columns, 1: upper half
    const int quad = warp & 3;               // TMEM lane quadrant this warp may read
    // 8-bit head: a token's first part is accumulator row r and its second part row r + part_rows, which lie in
    // different lane quadrants (quadrant q and q + shift), so different warps read them: the warp of the second
    // part (the donor) passes its 32 columns through shared memory to the warp of the first part, which adds
    // them, applies the scales and folds.
    const int shift = (kFp8 && !wide) ? (p.part_rows == 16 ? 1 : 2) : 4;
    const bool donor = kFp8 && !wide && quad >= shift && quad < 2 * shift;
    const bool idle = kFp8 && !wide && quad >= 2 * shift;              // quadrants that hold no operand rows
    const int cquad = donor ? quad - shift : quad;                     // quadrant of the rows this warp works for
    const int row_in_cta = m64 ? cquad * 16 + (lane & 15) : cquad * 32 + lane;
    const bool lane_has_row = !m64 || lane < 16;   // with M = 64 the upper half of a quadrant holds nothing
    const int hx = grp * 2 + cquad;                // hand-over buffer / scale area of this warp pair
    const int hx_lanes = m64 ? 16 : 32;
    float* hx_buf = hx_area + hx * 32 * hx_lanes;
    // (more than 64 rows: all eight warps fold and each stages the tile's scales for itself, in the area the
    // hand-over buffers do not need then)
    float* ws = wide ? hx_area + (grp * 4 + quad) * kBlockN : scale_area + hx * kBlockN;
    uint32_t hx_n = 0;                       // hand-overs done so far by this warp
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    uint32_t ord = 0;                        // ordinal of the unit among this worker's units
    float hs = 1.0f;
    if (kFp8 && !donor && !idle && lane_has_row && row_in_cta < p.n) {
      if (inl) {
        // the scales are written by the splitting warps before they arrive on h_ready
        ok = mbar_wait(h_ready, 0, abort_flag, p.status, wait_ns);
        hs = hs_s[row_in_cta];
      } else {
        hs = p.hscale[row_in_cta];
      }
    }
    if (kFp8) ok = __all_sync(0xffffffffu, ok);
    for (int unit = worker; unit < units && ok; unit += workers, ++ord) {
      const Unit first = unit_of<kCta>(p, unit, cta_rank);
      const bool warp_has_rows = !idle && (first.row0 + (m64 ? cquad * 16 : cquad * 32)) < p.n;   // warp-uniform
      const bool mlp_unit = !kFp8 && first.chunk < 0;
      RowFold f;
      f.reset();
      float mlp_sum = 0.f;
      // The walk over the unit's tiles, compiled twice: once for vocabulary units (the hot loop, free of any
      // learned-router code) and once for learned-router units.
      auto walk_tiles = [&](auto router_tag) {
      constexpr bool kRouter = decltype(router_tag)::value;
      for (int t = 0; t < T && ok; ++t) {
        const Tile tl = tile_of(p, first, t);
        if (tl.rows == 0) continue;
        const int v0 = tl.v0;
        const int cols = min(tl.rows, (kRouter ? p.mlp_hidden : p.V) - v0);   // valid columns of this tile
        // this group's share of them: [0, half) or [half, cols), half a multiple of 32
        const int half = min(cols, ((tl.rows / 2 + 31) / 32) * 32);
        const int c_begin = grp ? half : 0, c_end = grp ? cols : half;
        if (kFp8 && !donor && !idle) {
          // this tile's weight scales into the warp pair's area, before the accumulator is waited for
          __syncwarp();
#pragma unroll
          for (int j = 0; j < kBlockN / 32; ++j) {
            const int c = lane + 32 * j;
            ws[c] = (c < cols) ? __ldg(p.wscale + v0 + c) : 0.f;
          }
          __syncwarp();
        }
        if (!mbar_wait(acc_full(acc), acc_phase, abort_flag, p.status, wait_ns)) { ok = false; break; }
        tc_fence_after();
        if (warp_has_rows) {
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + acc * kBlockN;
          for (int c0 = c_begin; c0 < c_end; c0 += 32) {
            float z[32];
            __syncwarp();                           // the load below is warp-collective
            tmem_ld32(taddr + c0, z);
            tmem_ld_wait();
            if (kFp8 && wide) {
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                const float4 w4 = *reinterpret_cast<const float4*>(ws + c0 + j);
                z[j] = z[j] * hs * w4.x;
                z[j + 1] = z[j + 1] * hs * w4.y;
                z[j + 2] = z[j + 2] * hs * w4.z;
                z[j + 3] = z[j + 3] * hs * w4.w;
              }
            } else if (kFp8) {
              if (donor) {
                // second parts: wait until the partner has taken the previous 32 columns, then hand these over
                if (hx_n > 0 && !mbar_wait(hx_empty(hx), (hx_n - 1) & 1u, abort_flag, p.status, wait_ns)) { ok = false; break; }
                if (lane_has_row) {
#pragma unroll
                  for (int j = 0; j < 32; ++j) hx_buf[j * hx_lanes + (lane & (hx_lanes - 1))] = z[j];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(hx_full(hx));
                ++hx_n;
                continue;
              }
              if (!mbar_wait(hx_full(hx), hx_n & 1u, abort_flag, p.status, wait_ns)) { ok = false; break; }
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                const float4 w4 = *reinterpret_cast<const float4*>(ws + c0 + j);
                const int l = lane & (hx_lanes - 1);
                z[j] = (z[j] + hx_buf[j * hx_lanes + l]) * hs * w4.x;
                z[j + 1] = (z[j + 1] + hx_buf[(j + 1) * hx_lanes + l]) * hs * w4.y;
                z[j + 2] = (z[j + 2] + hx_buf[(j + 2) * hx_lanes + l]) * hs * w4.z;
                z[j + 3] = (z[j + 3] + hx_buf[(j + 3) * hx_lanes + l]) * hs * w4.w;
              }
              __syncwarp();
              if (lane == 0) mbar_arrive(hx_empty(hx));
              ++hx_n;
            }
            if constexpr (kRouter) {
              // hidden units v0 + c0 .. of the learned router: bias, ReLU, output-layer weight, sum
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const int u = v0 + c0 + j;
                if (u < p.mlp_hidden) mlp_sum += __ldg(p.mlp_w2 + u) * fmaxf(z[j] + __ldg(p.mlp_b1 + u), 0.f);
              }
            } else {
              f.group(z, cols - c0, v0 + c0);
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (kFp8) {                                 // a hand-over wait may have run out in some lanes
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) break;
        }
        if (lane == 0) {
          if (kCta == 1) mbar_arrive(acc_empty(acc));
          else mbar_arrive_cluster(map_to_cta(acc_empty(acc), 0));   // the leader's barrier
        }
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      };
      if (mlp_unit) walk_tiles(std::true_type{});
      else walk_tiles(std::false_type{});
      if (donor || idle) continue;
      Partial out = f.result();
      if (mlp_unit) out.s = mlp_sum;
      // The second group hands its summary to the first through the scratch block (bounded
      // waits on both sides: a warp that gave up never leaves its partner waiting forever).
      if (grp == 1) {
        if (ok && ord > 0) ok = mbar_wait(xch_empty(quad), (ord - 1) & 1u, abort_flag, p.status, wait_ns);
        if (ok) {
          if (lane_has_row) scratch[row_in_cta] = out;
          __syncwarp();
          if (lane == 0) mbar_arrive(xch_full(quad));
        }
      } else {
        if (ok) ok = mbar_wait(xch_full(quad), ord & 1u, abort_flag, p.status, wait_ns);
        if (ok) {
          const Partial other = scratch[row_in_cta];
          __syncwarp();
          if (lane == 0) mbar_arrive(xch_empty(quad));
          const bool mine = lane_has_row && first.row0 + row_in_cta < p.n;
          if (mlp_unit) {
            if (mine) p.mlp_out[first.row0 + row_in_cta] = out.s + other.s;   // lower columns first: a fixed order
          } else {
            out = merge(out, other);
            if (mine) p.partials[static_cast<size_t>(first.row0 + row_in_cta) * p.chunks + first.chunk] = out;
          }
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (kCta == 2) cluster_sync_all();   // neither CTA frees TMEM or exits while the peer still works
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc<kCta>(tmem_base, kTmemCols);
  }
}

// bf16 head: one CTA per worker (kCta = 1) or a pair (kCta = 2).
template <int kCta>
__global__ void __launch_bounds__(kThreads, 1)
tc_projection_kernel(const __grid_constant__ TcMaps maps, const TcParams p) {
  tc_projection_body<kCta, false>(maps, p);
}

// 8-bit head (defined in the one file that launches it).  At most 128 registers per thread, so that a block of
// the merge kernel (512 threads) fits on the SM beside this CTA and is resident, waiting, before this kernel ends.
#ifdef TLR_DEFINE_TC8_KERNEL
__global__ void __maxnreg__(128)
tc8_projection_kernel(const __grid_constant__ TcMaps maps, const TcParams p) {
  tc_projection_body<1, true>(maps, p);
}
#endif

}  // namespace tlr
