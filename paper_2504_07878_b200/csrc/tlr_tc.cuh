// Host/device interface of the tensor-core projection kernel (bf16 head and 8-bit head).
#pragma once

#include <cuda.h>

#include "tlr_common.cuh"

namespace tlr {

// Kernel shape for a given n (see tc_configure / tc8_configure).
struct TcConfig {
  int cta;          // 1: one CTA per worker (n <= 128); 2: a pair of CTAs per worker
  int a_rows;       // rows of an h slab held in shared memory (16..128); on the 8-bit head both parts of h stacked
  int part_rows;    // 8-bit head: rows of one part (a_rows / 2); otherwise a_rows
  int a_stages;     // depth of the h ring
  int b_stages;     // depth of the W ring
  int inline_split; // 8-bit head: 1 = n <= 16 and both parts of all of h fit in shared memory -- the kernel splits h
                    // itself at its start and keeps it resident (a_stages == number of K slabs); no split kernel runs
  int smem_bytes;   // dynamic shared memory per CTA
};

// Work decomposition for a given (n, V) on `workers` workers (see tc_plan).
struct TcPlan {
  int row_units;       // ceil(n / (128 * cta))
  int chunks;          // vocabulary chunks == partials per row
  int granule_rows;    // a multiple of 16 * cta
  int granules;        // ceil(V / granule_rows)
  int tiles_per_unit;  // every unit is walked in this many tiles (<= 256 rows each)
  int full_tiles_first;  // 1: full 256-row tiles, then one remainder tile; 0: tiles of equal size
  int mlp_rows;        // learned-router units: hidden width rounded up to the granule (0 = none); one such unit
                       // per row unit follows the vocabulary units
};

struct TcParams {
  int n, d, V;
  int row_units, chunks, granules, tiles_per_unit, full_tiles_first, granule_rows;
  int a_rows, part_rows, a_stages, b_stages;
  unsigned long long wait_limit_ns;   // 0 = the default limit of every barrier wait
  int debug_drop_w_copies;            // test hook: the W producer issues no copies
  int w_wait;                         // 1: W may have been written by the previous kernel in the stream, so the
                                      // W producer waits for it too (entry points that take W per call)
  // learned router inside the launch (bf16 head): one extra unit per row unit over the rows of W1
  int mlp_hidden;                     // hidden width, 0 = no learned router in this launch
  int mlp_rows;                       // hidden width rounded up to the granule
  const float* mlp_b1;                // [mlp_hidden]
  const float* mlp_w2;                // [mlp_hidden]
  float* mlp_out;                     // [n]: sum_j w2_j relu(W1_j . h + b1_j)
  // 8-bit head
  int inline_split;
  const void* h;         // bf16 [n][d], read when inline_split
  const float* hscale;   // [n] power-of-two scale of every row of h (written by the split kernel)
  const float* wscale;   // [V] scale of every row of W
  Partial* partials;     // [n][chunks]
  uint32_t* status;
};

// The tensor maps one launch needs: h, W (boxes of 128, 64 and 16 rows) and, with a learned router, W1.
struct TcMaps {
  CUtensorMap h, w128, w64, w16, m128, m64, m16;
};

int tc_threads();
int tc_enumerate_tiles(const TcParams& p, int cta, int workers, int* out, int capacity);
void tc_configure(int n, TcConfig* c);
void tc_plan(int n, int V, int cta, int workers, int max_chunks, int mlp_hidden, TcPlan* plan);
cudaError_t tc_prepare();   // opt in to the kernels' dynamic shared memory size (once per device)
cudaError_t launch_tc_projection(const TcMaps& maps, const TcParams& p, const TcConfig& c, int workers,
                                 cudaStream_t stream);

// ---- 8-bit head (tlr_tc8.cu): one CTA per worker, n <= tc8_max_rows()
int tc8_max_rows();
void tc8_configure(int n, int d, TcConfig* c);
cudaError_t tc8_prepare();
// h [n][d] bf16 -> parts [2][part_rows][d] e4m3 (rows n.. zero) and hscale[n]
cudaError_t launch_h_split(const void* h_bf16, int n, int d, int part_rows, uint8_t* parts, float* hscale,
                           cudaStream_t stream);
cudaError_t launch_tc8_projection(const TcMaps& maps, const TcParams& p, const TcConfig& c, int workers,
                                  cudaStream_t stream);

// Tuning switches, read from the environment once per process (defaults are the measured best).
struct Tuning {
  int granule;          // TLR_TC_GRANULE: vocabulary granule in rows (0 = default, 16 * cta)
  int even_tiles;       // TLR_TC_EVEN_TILES: equal-size tiles in pair mode
  int ring_a, ring_b;   // TLR_TC_RINGS="a,b": ring depths (0 = default)
  int tc8_inline;       // TLR_TC8_INLINE=0 keeps the separate split kernel
  int finish_threads;   // TLR_FINISH_THREADS: block size of the merge kernel for n <= 1024 (0 = default)
  int row_cost;         // TLR_TC_ROW_COST: pair mode plans by vocabulary rows per worker only, not by tile passes first
};
const Tuning& tuning();

}  // namespace tlr
