// Hyper-encoder (paper Section 2.2; Section 3.1: transformer encoder layers): work-list
// construction and the CUDA-core kernels of one encoder pass.  Activations stay in fp32 here;
// weights are read in their storage type.
//
// Row layout of a pass: entry e of the work list owns rows e*M .. e*M+M-1 ("we pad the input
// sequence to length M"); rows at or beyond the entry's length are padding: they are never
// attended to and never pooled, and are kept at zero so that no NaN can appear in them.
#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_simt_tile.cuh"

namespace z2z {

// ---------------------------------------------------------------------------------------------
// Work list
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void block_exclusive_scan_1024(int v, int* smem, int& excl, int& total) {
  const int t = threadIdx.x;
  smem[t] = v;
  __syncthreads();
  for (int o = 1; o < 1024; o <<= 1) {
    int x = t >= o ? smem[t - o] : 0;
    __syncthreads();
    smem[t] += x;
    __syncthreads();
  }
  excl = smem[t] - v;
  total = smem[1023];
  __syncthreads();
}

// mode 0: ranges from first/count (NULL: n_emb[which] .. n);  mode 1: from new_entry (0/1 each)
__global__ void __launch_bounds__(1024) k_entry_offsets(CbView cb, int which, int mode,
                                                        const int32_t* __restrict__ first,
                                                        const int32_t* __restrict__ count,
                                                        const int32_t* __restrict__ new_entry,
                                                        int32_t* __restrict__ off) {
  __shared__ int sm[1024];
  const int b = threadIdx.x;
  int c = 0;
  if (b < cb.B) {
    const int n = cb.n[b];
    if (mode == 1) {
      c = (new_entry[b] >= 0 && new_entry[b] < n) ? 1 : 0;
    } else {
      int f = first ? first[b] : cb.n_emb[which * cb.B + b];
      f = f < 0 ? 0 : (f > n ? n : f);
      c = count ? count[b] : n - f;
      c = c < 0 ? 0 : (c > n - f ? n - f : c);
    }
  }
  int excl, total;
  block_exclusive_scan_1024(c, sm, excl, total);
  if (b < cb.B) off[b] = excl;
  if (b == 0) off[cb.B] = total;
}

__global__ void k_entry_fill(CbView cb, int which, int mode, const int32_t* __restrict__ first,
                             const int32_t* __restrict__ new_entry, EntryList el, int chunk_index) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  const int total = el.off[cb.B];
  if (e == 0) {
    long long left = (long long)total - (long long)chunk_index * el.chunk;
    el.off[cb.B + 1] = (int)(left < 0 ? 0 : (left > el.chunk ? el.chunk : left));
  }
  if (e >= el.chunk) return;
  const long long g = (long long)chunk_index * el.chunk + e;
  if (g >= total) {
    el.seq[e] = -1; el.idx[e] = 0; el.len[e] = 0;
    for (int i = 0; i < cb.M; ++i) el.tok[(size_t)e * cb.M + i] = -1;
    return;
  }
  int lo = 0, hi = cb.B - 1;                     // last b with off[b] <= g
  while (lo < hi) {
    int mid = (lo + hi + 1) >> 1;
    if (el.off[mid] <= g) lo = mid; else hi = mid - 1;
  }
  const int b = lo;
  int f;
  if (mode == 1) f = new_entry[b];
  else {
    f = first ? first[b] : cb.n_emb[which * cb.B + b];
    const int n = cb.n[b];
    f = f < 0 ? 0 : (f > n ? n : f);
  }
  const int k = f + (int)(g - el.off[b]);
  el.seq[e] = b;
  el.idx[e] = k;
  const bool in_book = k >= 0 && k < cb.cap;
  el.len[e] = in_book ? (int)cb.len[(size_t)b * cb.cap + k] : 0;
  for (int i = 0; i < cb.M; ++i)                       // constituents are -1 padded behind the entry's length
    el.tok[(size_t)e * cb.M + i] = in_book ? cb.cons[((size_t)b * cb.cap + k) * cb.M + i] : -1;
}

__global__ void k_mark_embedded(CbView cb, int which) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < cb.B) cb.n_emb[which * cb.B + b] = cb.n[b];
}

__device__ __forceinline__ int entry_len(const CbView& cb, const EntryList& el, int e) {
  const int s = el.seq[e];
  return s < 0 ? 0 : (int)cb.len[(size_t)s * cb.cap + el.idx[e]];
}

// ---------------------------------------------------------------------------------------------
// Pass kernels
// ---------------------------------------------------------------------------------------------
// X[r] = table[y_i] + pos[i] for valid rows, 0 for padding.  grid = rows, block = 128.
template <typename T>
__global__ void __launch_bounds__(128) k_enc_gather(CbView cb, EntryList el,
                                                    const T* __restrict__ table,
                                                    const T* __restrict__ pos, float* __restrict__ X,
                                                    int d) {
  const int r = blockIdx.x, e = r / cb.M, i = r - e * cb.M;
  if (e >= el.off[cb.B + 1]) return;             // beyond the entries of this pass
  const int L = entry_len(cb, el, e);
  float* x = X + (size_t)r * d;
  if (i >= L) {
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4)
      *reinterpret_cast<float4*>(x + c) = make_float4(0.f, 0.f, 0.f, 0.f);
    return;
  }
  const int y = cb.cons[((size_t)el.seq[e] * cb.cap + el.idx[e]) * cb.M + i];
  const T* row = table + (size_t)y * d;
  const T* p = pos + (size_t)i * d;
  for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
    float a[4], b[4];
    load4<T>(row + c, a);
    load4<T>(p + c, b);
    *reinterpret_cast<float4*>(x + c) = make_float4(a[0] + b[0], a[1] + b[1], a[2] + b[2], a[3] + b[3]);
  }
}

__device__ __forceinline__ float block_sum_256(float v, float* sm) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) sm[w] = v;
  __syncthreads();
  float t = (l < (blockDim.x >> 5)) ? sm[l] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  return t;
}

// A[r] = LayerNorm(X[r]) * g + b  (eps 1e-5, biased variance) for valid rows, 0 for padding.
template <typename T>
__global__ void __launch_bounds__(256) k_enc_layernorm(CbView cb, EntryList el,
                                                       const float* __restrict__ X,
                                                       const T* __restrict__ g,
                                                       const T* __restrict__ bta,
                                                       float* __restrict__ A, int d) {
  __shared__ float sm[32];
  const int r = blockIdx.x, e = r / cb.M, i = r - e * cb.M;
  if (e >= el.off[cb.B + 1]) return;
  const int L = entry_len(cb, el, e);
  const float* x = X + (size_t)r * d;
  float* a = A + (size_t)r * d;
  if (i >= L) {
    for (int c = threadIdx.x; c < d; c += blockDim.x) a[c] = 0.f;
    return;
  }
  float s = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) s += x[c];
  const float mean = block_sum_256(s, sm) / (float)d;
  float q = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) { float t = x[c] - mean; q += t * t; }
  const float var = block_sum_256(q, sm) / (float)d;
  const float rstd = 1.0f / sqrtf(var + kLnEps);
  for (int c = threadIdx.x; c < d; c += blockDim.x)
    a[c] = (x[c] - mean) * rstd * to_f32<T>(g[c]) + to_f32<T>(bta[c]);
}

__device__ __forceinline__ float gelu_erf(float x) {
  return 0.5f * x * (1.0f + erff(x * 0.70710678118654752440f));
}

// Y = epilogue(A W^T + bias).  MODE 0: plain; 1: GELU; 2: Y += (in-place residual).
template <typename TW, int MODE>
__global__ void __launch_bounds__(256) k_enc_linear(const float* __restrict__ A, int K,
                                                    const TW* __restrict__ W, int J,
                                                    const TW* __restrict__ bias,
                                                    float* __restrict__ Y, int R,
                                                    const int32_t* __restrict__ n_entries, int M) {
  __shared__ SimtSmem sm;
  const int j0 = blockIdx.x * kTJ, r0 = blockIdx.y * kTR;
  if (r0 >= n_entries[0] * M) return;             // no live entry in this row tile
  float acc[4][4];
  const int nW = J - j0 < kTJ ? J - j0 : kTJ;
  simt_tile_mainloop<float, TW>(sm, A, K, r0, R, W + (size_t)j0 * K, nW, K, acc);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = r0 + ty * 4 + i;
    if (r >= R) continue;
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      const int j = j0 + tx * 4 + jj;
      if (j >= J) continue;
      float v = acc[i][jj] + to_f32<TW>(bias[j]);
      if (MODE == 1) v = gelu_erf(v);
      float* y = Y + (size_t)r * J + j;
      if (MODE == 2) v += *y;
      *y = v;
    }
  }
}

// Bidirectional attention inside one entry (keys = its valid rows only).
// grid (entries, heads), block (32, M): warp y is query row y.
__global__ void k_enc_attention(CbView cb, EntryList el, const float* __restrict__ QKV,
                                float* __restrict__ O, int d, int heads) {
  const int e = blockIdx.x, h = blockIdx.y, i = threadIdx.y, lane = threadIdx.x;
  if (e >= el.off[cb.B + 1]) return;
  const int L = entry_len(cb, el, e);
  const int dh = d / heads;
  float* o = O + ((size_t)e * cb.M + i) * d + (size_t)h * dh;
  if (i >= L) {
    for (int c = lane; c < dh; c += 32) o[c] = 0.f;
    return;
  }
  const float* q = QKV + ((size_t)e * cb.M + i) * 3 * d + (size_t)h * dh;
  const float scale = 1.0f / sqrtf((float)dh);
  float s[kMaxM];
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < kMaxM; ++j) {
    s[j] = -INFINITY;
    if (j < L) {
      const float* kp = QKV + ((size_t)e * cb.M + j) * 3 * d + d + (size_t)h * dh;
      float p = 0.f;
      for (int c = lane; c < dh; c += 32) p = fmaf(q[c], kp[c], p);
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) p += __shfl_xor_sync(0xffffffffu, p, off);
      s[j] = p * scale;
      mx = fmaxf(mx, s[j]);
    }
  }
  float den = 0.f;
#pragma unroll
  for (int j = 0; j < kMaxM; ++j) { s[j] = j < L ? expf(s[j] - mx) : 0.f; den += s[j]; }
  const float inv = 1.0f / den;
  for (int c = lane; c < dh; c += 32) {
    float v = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxM; ++j)
      if (j < L) v = fmaf(s[j] * inv, QKV[((size_t)e * cb.M + j) * 3 * d + 2 * d + (size_t)h * dh + c], v);
    o[c] = v;
  }
}

// cache[seq][idx] = mean over the entry's valid rows.  grid = entries, block = 256.
template <typename T>
__global__ void __launch_bounds__(256) k_enc_pool(CbView cb, EntryList el,
                                                  const float* __restrict__ X, T* __restrict__ cache,
                                                  float* __restrict__ cache_f32, int d) {
  const int e = blockIdx.x;
  if (e >= el.off[cb.B + 1]) return;
  const int L = entry_len(cb, el, e);
  if (L <= 0) return;
  const size_t dst = ((size_t)el.seq[e] * cb.cap + el.idx[e]) * d;
  const float inv = 1.0f / (float)L;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float v = 0.f;
    for (int i = 0; i < L; ++i) v += X[((size_t)e * cb.M + i) * d + c];
    v *= inv;
    cache[dst + c] = from_f32<T>(v);
    if (cache_f32) cache_f32[dst + c] = v;
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
cudaError_t launch_entry_offsets(const CbView& cb, int which, const int32_t* first,
                                 const int32_t* count, const EntryList& el, cudaStream_t s) {
  k_entry_offsets<<<1, 1024, 0, s>>>(cb, which, 0, first, count, nullptr, el.off);
  return cudaGetLastError();
}
cudaError_t launch_entry_offsets_from_new(const CbView& cb, const int32_t* new_entry,
                                          const EntryList& el, cudaStream_t s) {
  k_entry_offsets<<<1, 1024, 0, s>>>(cb, 0, 1, nullptr, nullptr, new_entry, el.off);
  return cudaGetLastError();
}
cudaError_t launch_entry_fill(const CbView& cb, int which, const int32_t* first,
                              const int32_t* new_entry, const EntryList& el, int chunk_index,
                              cudaStream_t s) {
  k_entry_fill<<<(el.chunk + 255) / 256, 256, 0, s>>>(cb, which, new_entry ? 1 : 0, first,
                                                      new_entry, el, chunk_index);
  return cudaGetLastError();
}
cudaError_t launch_mark_embedded(const CbView& cb, int which, cudaStream_t s) {
  k_mark_embedded<<<(cb.B + 255) / 256, 256, 0, s>>>(cb, which);
  return cudaGetLastError();
}

template <typename T>
static cudaError_t encoder_pass_simt(const CbView& cb, const EncoderArgs& a, const EntryList& el,
                                     Prof* prof, cudaStream_t s) {
  const int d = a.d, dff = a.dff, M = cb.M;
  const int E = el.chunk, R = E * M;
  const int32_t* n_live = el.off + cb.B + 1;
  auto W = [&](int i) { return reinterpret_cast<const T*>(a.w[i]); };
  { ProfScope ps(prof, kProfEncOther, 1, s);
    k_enc_gather<T><<<R, 128, 0, s>>>(cb, el, reinterpret_cast<const T*>(a.table), W(0), a.X, d); }
  const dim3 blk(256);
  const int rt = (R + kTR - 1) / kTR;
  for (int l = 0; l < a.layers; ++l) {
    const int o = 1 + 12 * l;
{ ProfScope ps(prof, kProfEncOther, 1, s);
        k_enc_layernorm<T><<<R, 256, 0, s>>>(cb, el, a.X, W(o + 0), W(o + 1), a.A, d);
      }
{ ProfScope ps(prof, kProfEncGemm, 1, s);
        k_enc_linear<T, 0><<<dim3((3 * d + kTJ - 1) / kTJ, rt), blk, 0, s>>>(a.A, d, W(o + 2), 3 * d,
                                                                          W(o + 3), a.QKV, R, n_live, M);
      }
{ ProfScope ps(prof, kProfEncOther, 1, s);
        k_enc_attention<<<dim3(E, a.heads), dim3(32, M), 0, s>>>(cb, el, a.QKV, a.A, d, a.heads);
      }
{ ProfScope ps(prof, kProfEncGemm, 1, s);
        k_enc_linear<T, 2><<<dim3((d + kTJ - 1) / kTJ, rt), blk, 0, s>>>(a.A, d, W(o + 4), d, W(o + 5),
                                                                      a.X, R, n_live, M);
      }
      if (dff == 0) continue;                          // attention-only layer
{ ProfScope ps(prof, kProfEncOther, 1, s);
        k_enc_layernorm<T><<<R, 256, 0, s>>>(cb, el, a.X, W(o + 6), W(o + 7), a.A, d);
      }
{ ProfScope ps(prof, kProfEncGemm, 1, s);
        k_enc_linear<T, 1><<<dim3((dff + kTJ - 1) / kTJ, rt), blk, 0, s>>>(a.A, d, W(o + 8), dff,
                                                                        W(o + 9), a.H, R, n_live, M);
      }
{ ProfScope ps(prof, kProfEncGemm, 1, s);
        k_enc_linear<T, 2><<<dim3((d + kTJ - 1) / kTJ, rt), blk, 0, s>>>(a.H, dff, W(o + 10), d,
                                                                      W(o + 11), a.X, R, n_live, M);
      }
  }
{ ProfScope ps(prof, kProfEncOther, 1, s);
      k_enc_pool<T><<<E, 256, 0, s>>>(cb, el, a.X, reinterpret_cast<T*>(a.cache), a.cache_f32, d);
      }
  return cudaGetLastError();
}

cudaError_t run_encoder_pass(const CbView& cb, const EncoderArgs& a, const EntryList& el,
                             bool use_tensor_cores, Prof* prof, cudaStream_t s) {
  (void)use_tensor_cores;
  if (a.dtype == Z2Z_DTYPE_FP32) return encoder_pass_simt<float>(cb, a, el, prof, s);
  return encoder_pass_simt<__nv_bfloat16>(cb, a, el, prof, s);
}

}  // namespace z2z
