// Input embedding of a mixed base-token / hypertoken stream (Figure 2a; Section 2.3 steps 3-4):
// a base token reads its row of the embedding matrix, a hypertoken reads the hyper-embedding the
// session cached when the entry was created.  A pure gather: each output row is read once and
// written once, so the kernel is bound by HBM bandwidth (2 x N x d x element size).
//
// One warp copies one row with 16-byte accesses, several in flight per lane; warps stride over
// the rows with a grid sized to the machine.
#include "z2z_common.cuh"
#include "z2z_internal.h"

namespace z2z {

namespace {
constexpr int kLookupThreads = 256;
constexpr int kLookupUnroll = 4;
}

__global__ void __launch_bounds__(kLookupThreads) k_embed_lookup(
    CbView cb, const int32_t* __restrict__ codes, int N, const int32_t* __restrict__ row_seq,
    const uint4* __restrict__ WE, const uint4* __restrict__ Eh, uint4* __restrict__ out,
    int row_vecs /* 16-byte vectors per row */) {
  const int lane = threadIdx.x & 31;
  const int warps = (gridDim.x * blockDim.x) >> 5;
  for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < N; r += warps) {
    const int z = codes[r];
    const int b = row_seq ? row_seq[r] : r;
    const uint4* src = nullptr;
    if ((unsigned)b < (unsigned)cb.B) {
      if (z >= 0 && z < cb.V) src = WE + (size_t)z * row_vecs;
      else if (z >= cb.V && z - cb.V < cb.n[b]) src = Eh + ((size_t)b * cb.cap + (z - cb.V)) * row_vecs;
    }
    uint4* dst = out + (size_t)r * row_vecs;
    if (!src) {                                   // no such token: zero row, flag the sequence
      if (lane == 0 && z != Z2Z_CODE_NONE && (unsigned)b < (unsigned)cb.B) atomicOr(&cb.status[b], Z2Z_ST_BAD_TOKEN);
      for (int i = lane; i < row_vecs; i += 32) dst[i] = make_uint4(0, 0, 0, 0);
      continue;
    }
    int i = lane;
    for (; i + 32 * (kLookupUnroll - 1) < row_vecs; i += 32 * kLookupUnroll) {
      uint4 v[kLookupUnroll];
#pragma unroll
      for (int u = 0; u < kLookupUnroll; ++u) v[u] = __ldg(src + i + 32 * u);
#pragma unroll
      for (int u = 0; u < kLookupUnroll; ++u) __stcs(dst + i + 32 * u, v[u]);
    }
    for (; i < row_vecs; i += 32) __stcs(dst + i, __ldg(src + i));
  }
}

cudaError_t launch_embed_lookup(const CbView& cb, const int32_t* codes, int N,
                                const int32_t* row_seq, const void* WE, const void* Eh, void* out,
                                int d, int elem_bytes, cudaStream_t s) {
  const int row_vecs = d * elem_bytes / 16;
  const int warps_per_block = kLookupThreads / 32;
  int blocks = (N + warps_per_block - 1) / warps_per_block;
  const int full = 148 * 8;                       // 8 resident blocks of 256 threads per SM
  if (blocks > full) blocks = full;
  k_embed_lookup<<<blocks, kLookupThreads, 0, s>>>(
      cb, codes, N, row_seq, reinterpret_cast<const uint4*>(WE), reinterpret_cast<const uint4*>(Eh),
      reinterpret_cast<uint4*>(out), row_vecs);
  return cudaGetLastError();
}

}  // namespace z2z
