// CUDA-core 64x64x16 tile product  acc[r][j] += sum_k A[r][k] * W[j][k]  with fp32 accumulation.
// Used by the fp32 configuration and as the exact-fp32-activation path of the hyper-encoder;
// the bf16 decode and prefill paths use the tcgen05 kernels instead.
#pragma once
#include "z2z_common.cuh"

namespace z2z {

constexpr int kTJ = 64, kTR = 64, kTK = 16, kTPad = 4;

struct SimtSmem {
  float As[kTK][kTR + kTPad];
  float Ws[kTK][kTJ + kTPad];
};

template <typename T>
__device__ __forceinline__ void load4(const T* p, float (&v)[4]);
template <>
__device__ __forceinline__ void load4<float>(const float* p, float (&v)[4]) {
  float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <>
__device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[4]) {
  uint2 t = *reinterpret_cast<const uint2*>(p);
  v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
  v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
}

// 256 threads.  A: rows r0.. of [R, K] (leading dimension lda), W: rows 0..nW-1 of the tile's own
// base pointer (leading dimension K).  K % 4 == 0.  Rows beyond the bounds contribute zeros.
template <typename TA, typename TW>
__device__ __forceinline__ void simt_tile_mainloop(SimtSmem& sm, const TA* __restrict__ A, int lda,
                                                   int r0, int R, const TW* __restrict__ W, int nW,
                                                   int K, float (&acc)[4][4]) {
  const int t = threadIdx.x;
  const int lrow = t >> 2, lk = (t & 3) * 4;
  const int tx = t & 15, ty = t >> 4;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  const bool a_ok = (r0 + lrow) < R;
  const bool w_ok = lrow < nW;
  const TA* ap = A + (size_t)(r0 + lrow) * lda + lk;
  const TW* wp = W + (size_t)lrow * K + lk;
  for (int k0 = 0; k0 < K; k0 += kTK) {
    float av[4] = {0.f, 0.f, 0.f, 0.f}, wv[4] = {0.f, 0.f, 0.f, 0.f};
    if (a_ok && k0 + lk < K) load4<TA>(ap + k0, av);
    if (w_ok && k0 + lk < K) load4<TW>(wp + k0, wv);
    __syncthreads();                               // previous chunk fully consumed
#pragma unroll
    for (int q = 0; q < 4; ++q) { sm.As[lk + q][lrow] = av[q]; sm.Ws[lk + q][lrow] = wv[q]; }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kTK; ++k) {
      float4 a = *reinterpret_cast<const float4*>(&sm.As[k][ty * 4]);
      float4 w = *reinterpret_cast<const float4*>(&sm.Ws[k][tx * 4]);
      const float ar[4] = {a.x, a.y, a.z, a.w}, wr[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], wr[j], acc[i][j]);
    }
  }
}

}  // namespace z2z
