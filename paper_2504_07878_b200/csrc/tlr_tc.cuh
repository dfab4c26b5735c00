// Host/device interface of the tensor-core projection kernel.
#pragma once

#include <cuda.h>

#include "tlr_common.cuh"

namespace tlr {

// Kernel shape for a given n (see tc_configure).
struct TcConfig {
  int cta;          // 1: one CTA per worker (n <= 128); 2: a pair of CTAs per worker
  int a_rows;       // rows of an h slab held in shared memory (16..128)
  int a_stages;     // depth of the h ring
  int b_stages;     // depth of the W ring
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
};

struct TcParams {
  int n, d, V;
  int row_units, chunks, granules, tiles_per_unit, full_tiles_first, granule_rows;
  int a_rows, a_stages, b_stages;
  unsigned long long wait_limit_ns;   // 0 = the default limit of every barrier wait
  int debug_drop_w_copies;            // test hook: the W producer issues no copies
  Partial* partials;  // [n][chunks]
  uint32_t* status;
};

// ---- fp8-W decode kernel (tlr_tc8.cu): one CTA per worker, n <= tc8_max_rows()
struct Tc8Config {
  int a_rows;       // rows of an h slab part held in shared memory (16..64)
  int a_stages;     // depth of the h ring (a stage = both parts of one 128-wide slab)
  int b_stages;     // depth of the W ring (a stage = up to 256 rows x 128 bytes)
  int inline_split; // 1: n <= 16 and the two parts of all of h fit in shared memory -- the kernel splits h itself
                    // at its start and keeps it resident (a_stages == number of K slabs); no split kernel runs
  int smem_bytes;
};

struct Tc8Params {
  int n, d, V;
  int chunks, granules, tiles_per_unit, granule_rows;
  int a_rows, a_stages, b_stages;
  unsigned long long wait_limit_ns;
  int debug_drop_w_copies;
  int inline_split;
  const void* h;         // bf16 [n][d], read when inline_split
  const float* hscale;   // [n] power-of-two scale of every row of h (written by the split kernel)
  const float* wscale;   // [V] scale of every row of W
  Partial* partials;     // [n][chunks]
  uint32_t* status;
};

int tc8_threads();
int tc8_max_rows();
void tc8_configure(int n, int d, Tc8Config* c);
cudaError_t tc8_prepare();
// h [n][d] bf16 -> parts [2][rows_alloc][d] e4m3 (rows n.. zero) and hscale[n]
cudaError_t launch_h_split(const void* h_bf16, int n, int d, int rows_alloc, uint8_t* parts, float* hscale,
                           cudaStream_t stream);
cudaError_t launch_tc8_projection(const CUtensorMap& map_h, const CUtensorMap& map_w128, const CUtensorMap& map_w64,
                                  const CUtensorMap& map_w16, const Tc8Params& p, const Tc8Config& c, int workers,
                                  cudaStream_t stream);

int tc_threads();
int tc_enumerate_tiles(const TcParams& p, int cta, int workers, int* out, int capacity);
void tc_configure(int n, TcConfig* c);
void tc_plan(int n, int V, int cta, int workers, int max_chunks, TcPlan* plan);
cudaError_t tc_prepare();   // opt in to the kernels' dynamic shared memory size (once per device)
cudaError_t launch_tc_projection(const CUtensorMap& map_h, const CUtensorMap& map_w128, const CUtensorMap& map_w64,
                                 const CUtensorMap& map_w16, const TcParams& p, const TcConfig& c, int workers,
                                 cudaStream_t stream);

}  // namespace tlr
