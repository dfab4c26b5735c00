// Tensor-core projection kernel for sm_100a: the LM-head contraction z = h W^T on
// tcgen05 with the accumulator in tensor memory, operands staged by TMA, and the
// online-softmax reduction (max / argmax / sum-exp / entropy numerator) fused into
// the epilogue, so the n x V logits never leave the SM.
//
// Two instantiations of one kernel:
//   kCta = 1  one CTA per worker, MMA M = 128 token rows            (n <= 128; M = 64 when n <= 64)
//   kCta = 2  a cluster of two CTAs per worker, MMA M = 256 rows (cta_group::2): each
//             CTA stages its own 128 rows of h and HALF of the W tile, and the pair's
//             tensor cores read both halves, so a W byte enters shared memory once
//             per 256 token rows.                                   (n > 128)
//
// Decomposition.  The vocabulary is cut into `chunks` contiguous ranges of granules
// (a multiple of 16 * kCta rows); the token rows into units of 128 * kCta.  A work unit is
// (chunk, row unit); units are numbered chunk-major so that workers running at the
// same time share W through L2, and worker w takes units w, w + workers, ...  Inside
// a unit the chunk is walked in `tiles_per_unit` tiles of at most 256 vocabulary rows
// (the MMA's N), each a K-loop over d in slabs of 64 elements.
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
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdio>
#include <cstdlib>

#include "tlr_common.cuh"
#include "tlr_tc.cuh"
#include "tlr_tc_ptx.cuh"

namespace tlr {

namespace {

constexpr int kBlockM = 128;                 // token rows per CTA == TMEM lanes
constexpr int kBlockN = 256;                 // max vocabulary rows per tile == accumulator columns
constexpr int kBlockK = 64;                  // bf16 per slab row = 128 B = one swizzle span
constexpr int kUmmaK = 16;
constexpr int kRowBytes = kBlockK * 2;       // 128
constexpr int kTmemCols = 512;
constexpr int kEpiWarps = 8;                 // two groups of four (one warp per TMEM lane quadrant each)
constexpr int kThreads = 32 * 11;
constexpr int kMaxAStages = 8;
constexpr int kMaxBStages = 12;
constexpr int kRelease = 16;                 // >= every ring depth (see the barrier notes in the kernel)
constexpr int kBarrierBytes = 512;
constexpr int kScratchBytes = kBlockM * 16;  // one Partial per row: hand-over between the epilogue groups
constexpr int kSmemLimit = 232448;           // 227 KiB opt-in maximum per CTA
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s


// The static schedule, identical in every role: worker w walks units w, w + workers, ...;
// each unit is `tiles_per_unit` tiles (possibly empty ones when the chunk is short).
struct Tile {
  int row0;    // first token row of this CTA in the unit
  int chunk;
  int v0;      // first vocabulary row of the tile
  int rows;    // vocabulary rows in the tile (multiple of 16 * kCta); 0 = empty tile
};

template <int kCta>
__host__ __device__ __forceinline__ Tile tile_of(const TcParams& p, int unit, int t, int cta_rank) {
  Tile r;
  r.chunk = unit / p.row_units;
  const int ru = unit - r.chunk * p.row_units;
  r.row0 = (ru * kCta + cta_rank) * kBlockM;
  const int g0 = static_cast<int>((static_cast<long long>(p.granules) * r.chunk) / p.chunks);
  const int g1 = static_cast<int>((static_cast<long long>(p.granules) * (r.chunk + 1)) / p.chunks);
  const int G = g1 - g0;
  int ga, gb;
  if (p.full_tiles_first) {
    // as many full 256-row tiles as fit, then one remainder tile: a tile costs a pass over all
    // of h whatever its width, so the fewest, widest tiles are the cheapest
    const int full = kBlockN / p.granule_rows;
    ga = full * t < G ? full * t : G;
    gb = full * (t + 1) < G ? full * (t + 1) : G;
  } else {
    ga = (G * t) / p.tiles_per_unit;
    gb = (G * (t + 1)) / p.tiles_per_unit;
  }
  r.v0 = (g0 + ga) * p.granule_rows;
  r.rows = (gb - ga) * p.granule_rows;
  return r;
}

}  // namespace

template <int kCta>
__global__ void __launch_bounds__(kThreads, 1)
tc_projection_kernel(const __grid_constant__ CUtensorMap map_h,
                     const __grid_constant__ CUtensorMap map_w128,
                     const __grid_constant__ CUtensorMap map_w64,
                     const __grid_constant__ CUtensorMap map_w16,
                     const TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment: the swizzle pattern is a function of the shared-memory address.
  // (The dynamic shared memory of both CTAs of a pair starts at the same offset, so the
  // two CTAs compute identical offsets -- which the pair MMA and the peer signals rely on.)
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int SA = p.a_stages, SB = p.b_stages;
  const uint32_t a_stage_bytes = static_cast<uint32_t>(p.a_rows) * kRowBytes;
  constexpr uint32_t b_stage_bytes = (kBlockN / kCta) * kRowBytes;
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
  auto acc_full = [&](int b) { return bar_base + 8u * (kMaxAStages + kMaxBStages + kRelease + b); };
  auto acc_empty = [&](int b) { return bar_base + 8u * (kMaxAStages + kMaxBStages + kRelease + 2 + b); };
  // xch_full[q]: the second epilogue group's summary of quadrant q is in the scratch block;
  // xch_empty[q]: the first group has read it.
  auto xch_full = [&](int q) { return bar_base + 8u * (kMaxAStages + kMaxBStages + kRelease + 4 + q); };
  auto xch_empty = [&](int q) { return bar_base + 8u * (kMaxAStages + kMaxBStages + kRelease + 8 + q); };
  constexpr int kNumBarriers = kMaxAStages + kMaxBStages + kRelease + 12;
  static_assert(kNumBarriers * 8 + 16 <= kBarrierBytes, "barrier block too small");
  unsigned char* gen_base = smem_raw + (base - smem_u32(smem_raw));
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen_base + (bar_base - base) + 8 * kNumBarriers);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  Partial* scratch = reinterpret_cast<Partial*>(gen_base + (bar_base - base) + kBarrierBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t cta_rank = (kCta == 2) ? cluster_ctarank() : 0u;
  const bool leader = cta_rank == 0;
  const int worker = blockIdx.x / kCta;
  const int workers = gridDim.x / kCta;

  if (threadIdx.x == 0) {
    for (int s = 0; s < SA; ++s) mbar_init(a_full(s), 1);
    for (int s = 0; s < SB; ++s) mbar_init(b_full(s), 1);
    for (int j = 0; j < kRelease; ++j) mbar_init(released(j), 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(acc_full(b), 1);
      mbar_init(acc_empty(b), kEpiWarps * kCta);
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
  // maps, which no kernel writes, so it goes ahead.
  if (warp != 0) asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // With at most 64 token rows (one CTA per worker) the MMAs run with M = 64: such an instruction takes
  // about two thirds of the time of an M = 128 one, and the padding rows were wasted work anyway.  Its
  // accumulator row r lives in TMEM lane 32 * (r / 16) + r % 16, i.e. in lanes 0..15 of each 32-lane
  // quadrant (checked on the device), so an epilogue warp then holds 16 rows instead of 32.
  const bool m64 = kCta == 1 && p.a_rows <= 64;
  const int k_slabs = (p.d + kBlockK - 1) / kBlockK;
  const int units = p.chunks * p.row_units;
  const int T = p.tiles_per_unit;
  const unsigned long long wait_ns = p.wait_limit_ns != 0 ? p.wait_limit_ns : kWaitLimitNs;

  if (warp == 0) {
    // ------------------------------------------------------------------ W producer
    if (lane == 0) {
      int stage = 0;
      int slab = 0;     // running slab number, the same in every role
      bool ok = true;
      for (int unit = worker; unit < units && ok; unit += workers) {
        for (int t = 0; t < T && ok; ++t) {
          const Tile tl = tile_of<kCta>(p, unit, t, cta_rank);
          if (tl.rows == 0) continue;
          const int my_rows = tl.rows / kCta;                 // this CTA's share of the tile
          const int my_v0 = tl.v0 + static_cast<int>(cta_rank) * my_rows;
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
              tma_load_2d<kCta>(dst + r * kRowBytes, &map_w128, bar, ks * kBlockK, my_v0 + r);
            for (; my_rows - r >= 64; r += 64)
              tma_load_2d<kCta>(dst + r * kRowBytes, &map_w64, bar, ks * kBlockK, my_v0 + r);
            for (; my_rows - r >= 16; r += 16)
              tma_load_2d<kCta>(dst + r * kRowBytes, &map_w16, bar, ks * kBlockK, my_v0 + r);
            if (++stage == SB) stage = 0;
          }
        }
      }
      if (!ok) drain_delay();
    }
  } else if (warp == 6) {
    // ------------------------------------------------------------------ h producer
    if (lane == 0) {
      int stage = 0;
      int slab = 0;
      bool ok = true;
      for (int unit = worker; unit < units && ok; unit += workers) {
        for (int t = 0; t < T && ok; ++t) {
          const Tile tl = tile_of<kCta>(p, unit, t, cta_rank);
          if (tl.rows == 0) continue;
          for (int ks = 0; ks < k_slabs; ++ks, ++slab) {
            if (slab >= SA) {
              const int j = slab - SA;
              if (!mbar_wait(released(j & (kRelease - 1)), (j / kRelease) & 1, abort_flag, p.status, wait_ns)) { ok = false; break; }
            }
            const uint32_t dst = a_ring + stage * a_stage_bytes;
            const uint32_t bar = (kCta == 2) ? map_to_cta(a_full(stage), 0) : a_full(stage);
            if (leader) mbar_expect_tx(a_full(stage), a_stage_bytes * kCta);
            tma_load_2d<kCta>(dst, &map_h, bar, ks * kBlockK, tl.row0);
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
      // The barrier state of the next slab is polled before the current slab's MMAs are
      // issued, so the poll's latency overlaps the issue instead of adding to it.
      bool ra = mbar_test_wait(a_full(0), 0), rb = mbar_test_wait(b_full(0), 0);
      for (int unit = worker; unit < units && ok; unit += workers) {
        for (int t = 0; t < T && ok; ++t) {
          const Tile tl = tile_of<kCta>(p, unit, t, 0);
          if (tl.rows == 0) continue;
          const uint32_t idesc = instr_desc(m64 ? 64 : kBlockM * kCta, tl.rows);
          ok = __all_sync(0xffffffffu, mbar_wait(acc_empty(acc), acc_phase ^ 1u, abort_flag, p.status, wait_ns));
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + acc * kBlockN;
          for (int ks = 0; ks < k_slabs; ++ks, ++slab) {
            if (!__all_sync(0xffffffffu, ra && rb)) {
              const bool got = mbar_wait(a_full(sa), pa, abort_flag, p.status, wait_ns) &&
                               mbar_wait(b_full(sb), pb, abort_flag, p.status, wait_ns);
              ok = __all_sync(0xffffffffu, got);
              if (!ok) break;
            }
            tc_fence_after();
            const uint32_t a_lo = a_lo0 + sa * a_step;
            const uint32_t b_lo = b_lo0 + sb * b_step;
            if (++sa == SA) { sa = 0; pa ^= 1u; }
            if (++sb == SB) { sb = 0; pb ^= 1u; }
            ra = mbar_test_wait(a_full(sa), pa);
            rb = mbar_test_wait(b_full(sb), pb);
            if (elect_one()) {
#pragma unroll
              for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                // advancing 16 elements along K inside the swizzle span = +32 bytes = +2 in the address field
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
    const int row_in_cta = m64 ? quad * 16 + (lane & 15) : quad * 32 + lane;
    const bool lane_has_row = !m64 || lane < 16;   // with M = 64 the upper half of a quadrant holds nothing
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    uint32_t ord = 0;                        // ordinal of the unit among this worker's units
    for (int unit = worker; unit < units && ok; unit += workers, ++ord) {
      const Tile first = tile_of<kCta>(p, unit, 0, cta_rank);
      const bool warp_has_rows = (first.row0 + (m64 ? quad * 16 : quad * 32)) < p.n;   // warp-uniform
      // Running summary of this thread's row over the unit.  S = sum 2^y and T = sum 2^y * y
      // with y = (z - m) * log2(e) <= 0; both are accumulated per 32-column group first and
      // then added with a compensated (Kahan) sum, so that one dominant term -- a confident
      // row has S ~ 1 with thousands of terms ~1e-8 after it -- does not swallow the rest.
      float m = -INFINITY, S = 0.f, cS = 0.f, Tq = 0.f, cT = 0.f;
      int idx = kNoToken;
      for (int t = 0; t < T && ok; ++t) {
        const Tile tl = tile_of<kCta>(p, unit, t, cta_rank);
        if (tl.rows == 0) continue;
        const int v0 = tl.v0;
        const int cols = min(tl.rows, p.V - v0);   // valid columns of this tile
        // this group's share of them: [0, half) or [half, cols), half a multiple of 32
        const int half = min(cols, ((tl.rows / 2 + 31) / 32) * 32);
        const int c_begin = grp ? half : 0, c_end = grp ? cols : half;
        if (!mbar_wait(acc_full(acc), acc_phase, abort_flag, p.status, wait_ns)) { ok = false; break; }
        tc_fence_after();
        if (warp_has_rows) {
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quad * 32) << 16) + acc * kBlockN;
          for (int c0 = c_begin; c0 < c_end; c0 += 32) {
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
              idx = v0 + c0 + first_j;
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
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if (kCta == 1) mbar_arrive(acc_empty(acc));
          else mbar_arrive_cluster(map_to_cta(acc_empty(acc), 0));   // the leader's barrier
        }
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      Partial out;
      out.m = m;
      out.idx = idx;
      out.s = S;
      out.t = Tq * kLn2;             // sum e^(z-m) (z-m), back in nats
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
          out = merge(out, other);
          if (lane_has_row && first.row0 + row_in_cta < p.n)
            p.partials[static_cast<size_t>(first.row0 + row_in_cta) * p.chunks + first.chunk] = out;
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

int tc_threads() { return kThreads; }

// Host enumeration of the schedule the kernel walks (the same tile_of the device code uses):
// one record {worker, unit, row0, v0, rows} per non-empty tile of CTA rank 0, in walking order.
int tc_enumerate_tiles(const TcParams& p, int cta, int workers, int* out, int capacity) {
  int count = 0;
  const int units = p.chunks * p.row_units;
  for (int w = 0; w < workers; ++w) {
    for (int unit = w; unit < units; unit += workers) {
      for (int t = 0; t < p.tiles_per_unit; ++t) {
        const Tile tl = cta == 2 ? tile_of<2>(p, unit, t, 0) : tile_of<1>(p, unit, t, 0);
        if (tl.rows == 0) continue;
        if (count < capacity) {
          int* r = out + 5 * count;
          r[0] = w;
          r[1] = unit;
          r[2] = tl.row0;
          r[3] = tl.v0;
          r[4] = tl.rows;
        }
        ++count;
      }
    }
  }
  return count;
}

// Ring depths and shared-memory size for a given n.  The h ring is short (L2 latency),
// the W ring takes everything that is left (HBM latency).
void tc_configure(int n, TcConfig* c) {
  const int cta = n > kBlockM ? 2 : 1;
  int a_rows = kBlockM;
  if (cta == 1) {
    a_rows = ((n + 15) / 16) * 16;
    if (a_rows < 16) a_rows = 16;
    if (a_rows > kBlockM) a_rows = kBlockM;
  }
  const int a_stage = a_rows * kRowBytes;
  const int b_stage = (kBlockN / cta) * kRowBytes;
  // h slabs come from L2 (about a microsecond away under load) and one is consumed per W
  // slab, so the h ring needs about half the depth of the W ring to keep up.
  int sa = cta == 2 ? 4 : (a_rows <= 32 ? 6 : 4);
  const int budget = kSmemLimit - 1024 - kBarrierBytes - kScratchBytes;
  int sb = (budget - sa * a_stage) / b_stage;
  if (sb > kMaxBStages) sb = kMaxBStages;
  // Tuning override: TLR_TC_RINGS="<h stages>,<W stages>" (ignored if it does not fit).
  if (const char* env = getenv("TLR_TC_RINGS")) {
    int ea = 0, eb = 0;
    if (sscanf(env, "%d,%d", &ea, &eb) == 2 && ea >= 1 && ea <= kMaxAStages && eb >= 1 && eb <= kMaxBStages &&
        ea * a_stage + eb * b_stage <= budget) {
      sa = ea;
      sb = eb;
    }
  }
  c->cta = cta;
  c->a_rows = a_rows;
  c->a_stages = sa;
  c->b_stages = sb;
  c->smem_bytes = 1024 + sa * a_stage + sb * b_stage + kBarrierBytes + kScratchBytes;
}

cudaError_t tc_prepare() {
  cudaError_t e = cudaFuncSetAttribute(tc_projection_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kSmemLimit);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(tc_projection_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
  return e;
}

cudaError_t launch_tc_projection(const CUtensorMap& map_h, const CUtensorMap& map_w128, const CUtensorMap& map_w64,
                                 const CUtensorMap& map_w16, const TcParams& p, const TcConfig& c, int workers,
                                 cudaStream_t stream) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(workers * c.cta), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = static_cast<size_t>(c.smem_bytes);
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  if (c.cta == 1) {
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, tc_projection_kernel<1>, map_h, map_w128, map_w64, map_w16, p);
  }
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, tc_projection_kernel<2>, map_h, map_w128, map_w64, map_w16, p);
}

}  // namespace tlr
