// Host-to-device copy of the hidden states done by a kernel instead of the copy engine.
//
// tlr_route_host brings h in from host memory before every step.  A copy-engine transfer
// cannot be the predecessor of a programmatic dependent launch, so the projection kernel
// behind it started only after the last byte had landed and paid its launch, its prologue and
// the fill of its W ring in full.  With the copy done by this kernel -- plain 16-byte loads
// from pinned host memory, which the GPU reads over PCIe -- the projection kernel is launched
// as soon as these blocks are resident, fills its W ring while h is still on its way, and
// waits (griddepcontrol.wait) for this kernel only where it reads h.
#include "tlr_common.cuh"

namespace tlr {

namespace {

constexpr int kCopyThreads = 256;
constexpr int kCopyBlocks = 32;       // 8192 threads x 4 loads in flight each saturate the link

__global__ void __launch_bounds__(kCopyThreads)
host_copy_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t n16) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  for (; i + 3 * stride < n16; i += 4 * stride) {
    const uint4 a = src[i], b = src[i + stride], c = src[i + 2 * stride], d = src[i + 3 * stride];
    dst[i] = a;
    dst[i + stride] = b;
    dst[i + 2 * stride] = c;
    dst[i + 3 * stride] = d;
  }
  for (; i < n16; i += stride) dst[i] = src[i];
  // Nothing above depends on the previous kernel in the stream (two staging buffers alternate between calls),
  // but this kernel must not be complete before that one is: the projection kernel behind it waits for THIS
  // kernel only, and it reuses the workspace the previous call's merge kernel reads.
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace

cudaError_t launch_host_copy(const void* src_mapped, void* dst, size_t bytes, cudaStream_t stream) {
  if (bytes == 0) return cudaSuccess;
  if ((bytes & 15u) != 0) return cudaErrorInvalidValue;
  // A programmatic dependent launch itself: the blocks may become resident, and copy, while the kernels of the
  // previous call in the stream are still running (the wait at the end of the kernel keeps the order of completion).
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kCopyBlocks, 1, 1);
  cfg.blockDim = dim3(kCopyThreads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, host_copy_kernel, static_cast<const uint4*>(src_mapped), static_cast<uint4*>(dst),
                            static_cast<size_t>(bytes / 16));
}

}  // namespace tlr
