// Host -> device transfer of a step's small input (the hidden rows) by a kernel instead of a DMA
// copy.  A copy engine transfer is an ordinary stream operation: the kernel behind it cannot start
// before it has ended.  The joint-logits kernel of a decode step streams its share of W_U before
// it needs the hidden rows, so when the rows are fetched by a kernel launched with programmatic
// serialization the weight stream starts at once and the transfer hides behind it.
#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_sm100.cuh"

namespace z2z {

__global__ void __launch_bounds__(256) k_upload_rows(const uint4* __restrict__ src, uint4* __restrict__ dst, size_t n) {
  sm100::pdl_trigger();                            // the next kernel may start its independent part
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint4 v = make_uint4(0, 0, 0, 0);
  if (i < n) v = __ldcv(src + i);                  // host memory: never served from a cache
  sm100::pdl_wait();                               // earlier kernels may still read the destination
  if (i < n) dst[i] = v;
}

}  // namespace z2z

extern "C" int32_t z2z_upload_rows(const void* h_mapped_src, void* d_dst, size_t bytes, z2z_stream stream) {
  if (bytes == 0) return Z2Z_OK;
  if (!h_mapped_src || !d_dst) { z2z::set_last_error("h_mapped_src / d_dst is NULL"); return Z2Z_ERR_INVALID_ARG; }
  if ((bytes & 15) || (reinterpret_cast<uintptr_t>(h_mapped_src) & 15) || (reinterpret_cast<uintptr_t>(d_dst) & 15)) {
    z2z::set_last_error("z2z_upload_rows needs 16-byte aligned pointers and a multiple of 16 bytes");
    return Z2Z_ERR_INVALID_ARG;
  }
  const size_t n = bytes / 16;
  if (n > ((size_t)1 << 24)) { z2z::set_last_error("z2z_upload_rows is meant for small inputs (<= 256 MiB)"); return Z2Z_ERR_INVALID_ARG; }
  cudaError_t e = z2z::launch_pdl(z2z::k_upload_rows, dim3((unsigned)((n + 255) / 256)), dim3(256), 0,
                                  reinterpret_cast<cudaStream_t>(stream), reinterpret_cast<const uint4*>(h_mapped_src),
                                  reinterpret_cast<uint4*>(d_dst), n);
  if (e != cudaSuccess) { z2z::set_last_error(cudaGetErrorString(e)); return Z2Z_ERR_CUDA; }
  return Z2Z_OK;
}
