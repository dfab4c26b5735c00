// Host/device interface of the tensor-core projection kernel.
#pragma once

#include <cuda.h>

#include "tlr_common.cuh"

namespace tlr {

struct TcParams {
  int n, d, V;
  int row_units;    // ceil(n / 128)
  int chunks;       // vocabulary chunks == partials per row
  int granules;     // ceil(V / 16): the vocabulary in 16-row granules
  Partial* partials;  // [n][chunks]
  uint32_t* status;
};

int tc_smem_bytes();
int tc_threads();
cudaError_t tc_prepare();   // opt in to the kernel's dynamic shared memory size (once per device)
cudaError_t launch_tc_projection(const CUtensorMap& map_h, const CUtensorMap& map_w64, const CUtensorMap& map_w16,
                                 const TcParams& p, int grid, cudaStream_t stream);

// Chooses the number of vocabulary chunks for n rows on `workers` CTAs: the count that
// minimises (waves of units) x (rows per chunk + a fixed per-unit cost), capped at max_chunks.
int tc_choose_chunks(int n, int V, int workers, int max_chunks);

}  // namespace tlr
