// Hyper-encoder pass on the tensor cores (bf16 weights): the linear layers run in the stream-K
// tcgen05 kernel of z2z_stream.cu; this file holds the element-wise kernels between them and the
// host-side sequencing.  Both encoders (embedding side and unembedding side, paper Section 2.2)
// go through the same launches as two "groups".
//
// Activations are kept to ~16 mantissa bits on the tensor cores by splitting every fp32
// activation x into bf16 hi = rn(x) and lo = rn(x - hi): with bf16 weights w the products hi*w
// and lo*w are exact in fp32, so A.W^T = hi.W^T + lo.W^T with fp32 accumulation.  Rounding the
// activations to a single bf16 would leave the hyper-embeddings outside the 2e-2 tolerance.
//
// Prompt-sized passes may instead round every activation ONCE to fp16 and multiply by fp16 copies
// of the weights (exact for bf16 values within fp16's range), when the caller has lent memory
// for the copies: one MMA per k-step instead of two.  The rounding error (2^-11 relative per
// operand element) stays inside the tolerance with a margin of about 3 at d = 4096; the two-part
// form keeps a margin of about 200 and remains the default.
//
// Rows are PACKED in both kinds of pass: entry e owns the rows row_off[e] .. row_off[e] + len[e],
// there are no padding rows, and only the device knows how many rows a pass has (the word behind
// the last entry slot of row_off).
// Layout of a hi/lo operand: decode-sized passes (stream-K GEMM) keep the two parts of packed
// row r in operand rows 2r and 2r + 1 of a bf16 [2 * Rt, K] matrix, so that the live rows are one
// contiguous range whatever their number; prompt-sized passes (CTA-pair GEMM) keep hi rows
// [0, Rt) first and lo rows [Rt, 2 Rt) after them.
//
// GEMM output.  Every CTA of the stream-K GEMM adds its partial tiles (hi and lo parts summed
// in registers) into ONE fp32 matrix Y[group][Rt][J] with reductions in global memory; Y is all zero
// whenever no GEMM result is pending.  The element-wise kernel after a GEMM reads each element of
// that GEMM's result exactly once and stores zero back ("consume and clear"), for every live row
// of the pass (the GEMM adds nothing to rows beyond them), which restores the invariant for the
// next GEMM.  The session start clears Y once.
//
// Launches per layer: GEMM(qkv) -> [+ bias, attention] -> GEMM(o) -> [+ bias + residual,
// LayerNorm 2] -> GEMM(1) -> [+ bias, GELU] -> GEMM(2) -> [+ bias + residual, LayerNorm 1 of the
// next layer | mean-pool into the cache].  All are launched with programmatic serialization.
// Between two GEMMs the weight stream stands still, so the small kernels are written for latency:
// what a kernel needs about an entry (its length, the base token of a row) is one load from the
// work list, and every data load is issued before the first value is used - whether a row is valid
// only decides what is stored.
#include <cuda_fp16.h>

#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_sm100.cuh"
#include "z2z_stream.h"

namespace z2z {

namespace {

using bf16 = __nv_bfloat16;
constexpr int kNT = kGemmNT;
constexpr int kRowThreads = 256;
constexpr int kMaxVec4 = 8;            // float4 per thread in the row kernels: d <= 8192
constexpr int kNarrowVec4 = 4;         // ... and for d <= 4096, where half the registers do
constexpr int kPairPassMinRows = 1024; // passes of at least this many rows use the CTA-pair GEMM

struct Ptr2 { const void* p[2]; };
struct MPtr2 { void* p[2]; };

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ float4 load_bf16x4(const bf16* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  return make_float4(bf_lo(u.x), bf_hi(u.x), bf_lo(u.y), bf_hi(u.y));
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(a)) |
         ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(b)) << 16);
}
// hi = rn(x), lo = rn(x - hi) for 4 values; 8-byte stores.
__device__ __forceinline__ void split_store4(bf16* hi, bf16* lo, float4 x) {
  const bf16 h0 = __float2bfloat16_rn(x.x), h1 = __float2bfloat16_rn(x.y);
  const bf16 h2 = __float2bfloat16_rn(x.z), h3 = __float2bfloat16_rn(x.w);
  uint2 H, L;
  H.x = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
  H.y = (uint32_t)__bfloat16_as_ushort(h2) | ((uint32_t)__bfloat16_as_ushort(h3) << 16);
  L.x = pack_bf16(x.x - __bfloat162float(h0), x.y - __bfloat162float(h1));
  L.y = pack_bf16(x.z - __bfloat162float(h2), x.w - __bfloat162float(h3));
  *reinterpret_cast<uint2*>(hi) = H;
  *reinterpret_cast<uint2*>(lo) = L;
}
// 4 values rounded once to fp16; one 8-byte store.  `dst` points into an fp16 matrix that shares
// the bf16 operand buffer (same element size).
__device__ __forceinline__ void half_store4(bf16* dst, float4 x) {
  uint2 H;
  H.x = (uint32_t)__half_as_ushort(__float2half_rn(x.x)) | ((uint32_t)__half_as_ushort(__float2half_rn(x.y)) << 16);
  H.y = (uint32_t)__half_as_ushort(__float2half_rn(x.z)) | ((uint32_t)__half_as_ushort(__float2half_rn(x.w)) << 16);
  *reinterpret_cast<uint2*>(dst) = H;
}
// Base tokens of work-list entry e (0 for an unused slot): one load, so that the kernels below can
// issue it together with their data loads instead of ahead of them.
__device__ __forceinline__ int entry_len_tc(const CbView& cb, const EntryList& el, int e) {
  (void)cb;
  return el.len[e];
}
__device__ __forceinline__ float4 unpack_bf16x4(uint2 u) {
  return make_float4(bf_lo(u.x), bf_hi(u.x), bf_lo(u.y), bf_hi(u.y));
}

__device__ __forceinline__ float block_sum(float v, float* sm) {
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

// LayerNorm of a row held in registers (x[v] = 4 columns starting at (tid + v * 256) * 4),
// written as hi/lo bf16.  eps 1e-5, biased variance, two-pass.
// gw / gb: gamma and beta of the thread's columns, packed 4 bf16 per uint2 and loaded by the caller
// together with the row, so that no load waits behind the reductions.
template <int NV, bool HALF = false>
__device__ __forceinline__ void layernorm_split_regs(const float4 (&x)[NV], int nvec, const uint2 (&gw)[NV],
                                                     const uint2 (&gb)[NV], bf16* hi, bf16* lo, int d, float* sm) {
  float s = 0.f;
#pragma unroll
  for (int v = 0; v < NV; ++v)
    if ((int)threadIdx.x + v * kRowThreads < nvec) s += (x[v].x + x[v].y) + (x[v].z + x[v].w);
  const float mean = block_sum(s, sm) / (float)d;
  float q = 0.f;
#pragma unroll
  for (int v = 0; v < NV; ++v)
    if ((int)threadIdx.x + v * kRowThreads < nvec) {
      const float a = x[v].x - mean, bb = x[v].y - mean, c = x[v].z - mean, e = x[v].w - mean;
      q += (a * a + bb * bb) + (c * c + e * e);
    }
  const float rstd = 1.0f / sqrtf(block_sum(q, sm) / (float)d + kLnEps);
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) {
      const float4 gg = unpack_bf16x4(gw[v]), bb = unpack_bf16x4(gb[v]);
      float4 y;
      y.x = (x[v].x - mean) * rstd * gg.x + bb.x;
      y.y = (x[v].y - mean) * rstd * gg.y + bb.y;
      y.z = (x[v].z - mean) * rstd * gg.z + bb.z;
      y.w = (x[v].w - mean) * rstd * gg.w + bb.w;
      if (HALF) half_store4(hi + idx * 4, y);
      else split_store4(hi + idx * 4, lo + idx * 4, y);
    }
  }
}

// X = table[y] + pos for every live packed row; then LN1 of layer 0 -> hi/lo.  grid (rows, groups).
template <int NV>
__global__ void __launch_bounds__(kRowThreads) k_tc_gather_ln(CbView cb, EntryList el, const int* total, Ptr2 table,
                                                              Ptr2 pos, Ptr2 ln_w, Ptr2 ln_b, MPtr2 X, MPtr2 Ahl,
                                                              int d, int has_ln) {
  __shared__ float sm[32];
  sm100::pdl_trigger();            // the next kernel may start its prologue and weight prefetch
  sm100::pdl_wait();               // everything read or written below depends on earlier kernels
  const int r = blockIdx.x, g = blockIdx.y;
  const int y = el.row_tok[r];                    // the row's base token, its place in the entry and the
  const int src = el.row_src[r];                  // row count: three independent loads
  if (r >= *total) return;
  const int i = src % cb.M;
  float* x = reinterpret_cast<float*>(X.p[g]) + (size_t)r * d;
  bf16* hi = reinterpret_cast<bf16*>(Ahl.p[g]) + (size_t)2 * r * d;
  bf16* lo = hi + d;
  const int nvec = d / 4;
  const bf16* row = reinterpret_cast<const bf16*>(table.p[g]) + (size_t)y * d;
  const bf16* pp = reinterpret_cast<const bf16*>(pos.p[g]) + (size_t)i * d;
  const uint2* lw = reinterpret_cast<const uint2*>(ln_w.p[g]);
  const uint2* lb = reinterpret_cast<const uint2*>(ln_b.p[g]);
  float4 xv[NV];
  uint2 gw[NV], gb[NV];
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) {
      const float4 a = load_bf16x4(row + idx * 4), b = load_bf16x4(pp + idx * 4);
      gw[v] = lw[idx]; gb[v] = lb[idx];
      xv[v] = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
      *reinterpret_cast<float4*>(x + idx * 4) = xv[v];
    }
  }
  if (has_ln) layernorm_split_regs<NV>(xv, nvec, gw, gb, hi, lo, d, sm);
}

// x = X[r] + Y[r] + bias for a live packed row (Y consumed and cleared); then LayerNorm -> hi/lo
// for the next GEMM.  grid (rows, groups).  All loads (row count, Y, X, bias, gamma, beta) are
// issued together; whether the row is live only decides what is stored.
template <int NV>
__global__ void __launch_bounds__(kRowThreads) k_tc_reduce_resid_ln(const int* total, float* Y, Ptr2 bias,
                                                                    MPtr2 X, Ptr2 ln_w, Ptr2 ln_b, MPtr2 Ahl,
                                                                    int d, int Rt) {
  __shared__ float sm[32];
  sm100::pdl_trigger();
  sm100::pdl_wait();
  const int r = blockIdx.x, g = blockIdx.y;
  const int live = *total;
  float* y = Y + ((size_t)g * Rt + r) * d;
  float* x = reinterpret_cast<float*>(X.p[g]) + (size_t)r * d;
  const uint2* bs = reinterpret_cast<const uint2*>(bias.p[g]);
  const uint2* lw = reinterpret_cast<const uint2*>(ln_w.p[g]);
  const uint2* lb = reinterpret_cast<const uint2*>(ln_b.p[g]);
  const int nvec = d / 4;
  float4 xv[NV], yv[NV];
  uint2 bv[NV], gw[NV], gb[NV];
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) {
      yv[v] = *reinterpret_cast<const float4*>(y + idx * 4);
      xv[v] = *reinterpret_cast<const float4*>(x + idx * 4);
      bv[v] = bs[idx]; gw[v] = lw[idx]; gb[v] = lb[idx];
    }
  }
  if (r >= live) return;                          // nothing was added to this row of Y: it is still zero
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) {
      *reinterpret_cast<float4*>(y + idx * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
      const float4 b = unpack_bf16x4(bv[v]);
      xv[v] = make_float4(xv[v].x + yv[v].x + b.x, xv[v].y + yv[v].y + b.y, xv[v].z + yv[v].z + b.z,
                          xv[v].w + yv[v].w + b.w);
      *reinterpret_cast<float4*>(x + idx * 4) = xv[v];
    }
  }
  bf16* hi = reinterpret_cast<bf16*>(Ahl.p[g]) + (size_t)2 * r * d;
  layernorm_split_regs<NV>(xv, nvec, gw, gb, hi, hi + d, d, sm);
}

// Last layer: x_i = X[r_i] + Y[r_i] + bias for the entry's rows, cache row = mean_i x_i.
// grid (entries, groups, ceil(d / (4 * kRowThreads))): a thread owns 4 columns of the entry and
// issues the loads of all its rows before it adds.
__global__ void __launch_bounds__(kRowThreads) k_tc_reduce_resid_pool(CbView cb, EntryList el, float* Y, Ptr2 bias,
                                                                      MPtr2 X, MPtr2 cache, MPtr2 cache_f32, int d,
                                                                      int Rt) {
  sm100::pdl_trigger();
  sm100::pdl_wait();
  const int e = blockIdx.x, g = blockIdx.y;
  const int col = ((int)blockIdx.z * kRowThreads + (int)threadIdx.x) * 4;
  if (col >= d) return;
  const int L = entry_len_tc(cb, el, e);
  const int r0 = el.row_off[e];
  const int seq = el.seq[e], idx = el.idx[e];
  const float4 b = load_bf16x4(reinterpret_cast<const bf16*>(bias.p[g]) + col);
  if (L <= 0) return;
  float4 yv[kMaxM], xv[kMaxM];
#pragma unroll
  for (int i = 0; i < kMaxM; ++i)
    if (i < L) {
      const size_t r = (size_t)r0 + i;
      yv[i] = *reinterpret_cast<const float4*>(Y + ((size_t)g * Rt + r) * d + col);
      xv[i] = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(X.p[g]) + r * d + col);
    }
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int i = 0; i < kMaxM; ++i)
    if (i < L) {
      const size_t r = (size_t)r0 + i;
      *reinterpret_cast<float4*>(Y + ((size_t)g * Rt + r) * d + col) = make_float4(0.f, 0.f, 0.f, 0.f);
      acc.x += xv[i].x + yv[i].x + b.x; acc.y += xv[i].y + yv[i].y + b.y;
      acc.z += xv[i].z + yv[i].z + b.z; acc.w += xv[i].w + yv[i].w + b.w;
    }
  const size_t dst = ((size_t)seq * cb.cap + idx) * d + col;
  const float inv = 1.0f / (float)L;
  const float4 m = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
  uint2 o; o.x = pack_bf16(m.x, m.y); o.y = pack_bf16(m.z, m.w);
  *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(cache.p[g]) + dst) = o;
  float* out32 = reinterpret_cast<float*>(cache_f32.p[g]);
  if (out32) *reinterpret_cast<float4*>(out32 + dst) = m;
}

// Zero-layer encoder (the parameter-free averaging variant): cache row = mean of the entry's X rows.
__global__ void __launch_bounds__(kRowThreads) k_tc_pool(CbView cb, EntryList el, MPtr2 X, MPtr2 cache,
                                                         MPtr2 cache_f32, int d) {
  sm100::pdl_trigger();
  sm100::pdl_wait();
  const int e = blockIdx.x, g = blockIdx.y;
  const int L = entry_len_tc(cb, el, e);
  if (L <= 0) return;
  const float* x = reinterpret_cast<const float*>(X.p[g]) + (size_t)el.row_off[e] * d;
  const size_t dst = ((size_t)el.seq[e] * cb.cap + el.idx[e]) * d;
  const float inv = 1.0f / (float)L;
  bf16* out = reinterpret_cast<bf16*>(cache.p[g]);
  float* out32 = reinterpret_cast<float*>(cache_f32.p[g]);
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float v = 0.f;
    for (int i = 0; i < L; ++i) v += x[(size_t)i * d + c];
    v *= inv;
    out[dst + c] = __float2bfloat16_rn(v);
    if (out32) out32[dst + c] = v;
  }
}

// H = GELU(Y + bias) -> hi/lo (Y consumed and cleared) for the live packed rows.  The
// [groups * R, J] results are one flat range of float4; every thread takes kGeluPerThread of them,
// kGeluThreads apart, and issues all of its loads before it computes.
// grid = ceil(groups * R * J / 4 / (kGeluThreads * kGeluPerThread)), R = row capacity of the pass.
constexpr int kGeluThreads = 256, kGeluPerThread = 4;
__global__ void __launch_bounds__(kGeluThreads) k_tc_reduce_gelu(const int* total_rows, float* Y, Ptr2 bias, MPtr2 Hhl,
                                                                 int J, int R, int Rt, int ng) {
  sm100::pdl_trigger();
  sm100::pdl_wait();
  const int J4 = J / 4;
  const long long total = (long long)ng * R * J4;
  const long long base = (long long)blockIdx.x * (kGeluThreads * kGeluPerThread) + threadIdx.x;
  const int live = *total_rows;
  float4 q[kGeluPerThread], bs[kGeluPerThread];
  int row[kGeluPerThread], jj[kGeluPerThread];
#pragma unroll
  for (int k = 0; k < kGeluPerThread; ++k) {
    const long long f = base + (long long)k * kGeluThreads;
    row[k] = -1;
    if (f < total) {
      row[k] = (int)(f / J4);
      jj[k] = (int)(f - (long long)row[k] * J4) * 4;
      const int g = row[k] / R, r = row[k] - g * R;
      q[k] = *reinterpret_cast<const float4*>(Y + ((size_t)g * Rt + r) * J + jj[k]);
      bs[k] = load_bf16x4(reinterpret_cast<const bf16*>(bias.p[g]) + jj[k]);
    }
  }
#pragma unroll
  for (int k = 0; k < kGeluPerThread; ++k) {
    if (row[k] < 0) continue;
    const int g = row[k] / R, r = row[k] - g * R;
    if (r >= live) continue;                       // no row there: Y is still zero, nothing reads the operand row
    *reinterpret_cast<float4*>(Y + ((size_t)g * Rt + r) * J + jj[k]) = make_float4(0.f, 0.f, 0.f, 0.f);
    float4 v = make_float4(q[k].x + bs[k].x, q[k].y + bs[k].y, q[k].z + bs[k].z, q[k].w + bs[k].w);
    v.x = 0.5f * v.x * (1.0f + erff(v.x * 0.70710678118654752440f));
    v.y = 0.5f * v.y * (1.0f + erff(v.y * 0.70710678118654752440f));
    v.z = 0.5f * v.z * (1.0f + erff(v.z * 0.70710678118654752440f));
    v.w = 0.5f * v.w * (1.0f + erff(v.w * 0.70710678118654752440f));
    bf16* hi = reinterpret_cast<bf16*>(Hhl.p[g]) + (size_t)2 * r * J + jj[k];
    split_store4(hi, hi + J, v);
  }
}

// q, k, v = Y + bias for one head of one entry (consumed, cleared, staged in shared memory), then
// bidirectional attention over the entry's rows; output as hi/lo.
// grid (entries, heads, groups), block (32, M), dynamic smem M * 3 * dh floats; dh % 4 == 0.
__global__ void k_tc_qkv_attention(CbView cb, EntryList el, float* Y, Ptr2 bias, MPtr2 Ohl, int d, int heads,
                                   int Rt) {
  extern __shared__ float s_qkv[];
  sm100::pdl_trigger();
  sm100::pdl_wait();
  const int e = blockIdx.x, h = blockIdx.y, g = blockIdx.z, i = threadIdx.y, lane = threadIdx.x;
  const int L = entry_len_tc(cb, el, e);
  const int r = el.row_off[e] + i;               // packed row of position i (only used while i < L)
  const int dh = d / heads;
  if (i < L) {
    const bf16* bs = reinterpret_cast<const bf16*>(bias.p[g]);
    float* y = Y + ((size_t)g * Rt + r) * 3 * d;
    for (int c = lane * 4; c < dh; c += 128) {
      float4 p[3], b[3];
#pragma unroll
      for (int w = 0; w < 3; ++w) {                // the six loads are independent of one another
        const int col = w * d + h * dh + c;
        p[w] = *reinterpret_cast<const float4*>(y + col);
        b[w] = load_bf16x4(bs + col);
      }
#pragma unroll
      for (int w = 0; w < 3; ++w) {
        *reinterpret_cast<float4*>(y + w * d + h * dh + c) = make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4*>(&s_qkv[(i * 3 + w) * dh + c]) =
            make_float4(p[w].x + b[w].x, p[w].y + b[w].y, p[w].z + b[w].z, p[w].w + b[w].w);
      }
    }
  }
  __syncthreads();
  if (i >= L) return;
  const float* q = s_qkv + (i * 3) * dh;
  const float scale = 1.0f / sqrtf((float)dh);
  float s[kMaxM];
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < kMaxM; ++j) {
    s[j] = -INFINITY;
    if (j < L) {
      const float* kp = s_qkv + (j * 3 + 1) * dh;
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
  bf16* hi = reinterpret_cast<bf16*>(Ohl.p[g]) + (size_t)2 * r * d + (size_t)h * dh;
  bf16* lo = hi + d;
  for (int c = lane; c < dh; c += 32) {
    float v = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxM; ++j)
      if (j < L) v = fmaf(s[j] * inv, s_qkv[(j * 3 + 2) * dh + c], v);
    const bf16 hh = __float2bfloat16_rn(v);
    hi[c] = hh;
    lo[c] = __float2bfloat16_rn(v - __bfloat162float(hh));
  }
}

// Packed rows: entry e owns rows row_off[e] .. row_off[e] + len[e], there are no padding rows
// inside entries, and rows at or beyond the total carry nothing.  (With M = 3 or 4 a quarter to a
// third of padded rows would be zeros that the GEMMs load and multiply anyway.)
//
// One block: first packed row of every entry (exclusive scan of the lengths), the total behind the
// last entry slot, the way back from a packed row to (entry, position) and the row's base token.
// E <= 1024 entries.  (The decode step's update kernel writes the same map itself.)
__global__ void __launch_bounds__(1024) k_tc_row_map(CbView cb, EntryList el, int E) {
  __shared__ int warp_sums[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int len = tid < E ? entry_len_tc(cb, el, tid) : 0;
  int inc = len;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += x;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = warp_sums[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += x;
    }
    warp_sums[lane] = w;
  }
  __syncthreads();
  const int excl = inc - len + (warp > 0 ? warp_sums[warp - 1] : 0);
  if (tid < E) {
    el.row_off[tid] = excl;
    for (int i = 0; i < len; ++i) {
      el.row_src[excl + i] = tid * cb.M + i;
      el.row_tok[excl + i] = el.tok[tid * cb.M + i];
    }
  }
  if (tid == 0) el.row_off[E] = warp_sums[31];
}

// X = table[y] + pos for every packed row, then LN1 of layer 0 -> hi/lo.  grid (row capacity).
template <int NV, bool HALF>
__global__ void __launch_bounds__(kRowThreads) k_tc_gather_ln_packed(CbView cb, EntryList el, const int* total,
                                                                     const bf16* table, const bf16* pos, const bf16* ln_w,
                                                                     const bf16* ln_b, float* X, bf16* Ahl, int d, int Rt,
                                                                     int has_ln) {
  __shared__ float sm[32];
  const int r = blockIdx.x;
  if (r >= *total) return;
  const int src = el.row_src[r];
  const int y = el.tok[src], i = src % cb.M;
  float* x = X + (size_t)r * d;
  bf16* hi = Ahl + (size_t)r * d;
  const bf16* row = table + (size_t)y * d;
  const bf16* pp = pos + (size_t)i * d;
  const int nvec = d / 4;
  float4 xv[NV];
  uint2 gw[NV], gb[NV];
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) {
      const float4 a = load_bf16x4(row + idx * 4), b = load_bf16x4(pp + idx * 4);
      gw[v] = reinterpret_cast<const uint2*>(ln_w)[idx];
      gb[v] = reinterpret_cast<const uint2*>(ln_b)[idx];
      xv[v] = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
      *reinterpret_cast<float4*>(x + idx * 4) = xv[v];
    }
  }
  if (has_ln) layernorm_split_regs<NV, HALF>(xv, nvec, gw, gb, hi, hi + (size_t)Rt * d, d, sm);
}

// Mean-pool on packed rows: cache row = mean of the entry's rows of X.  grid (entries,
// ceil(d / (4 * kRowThreads))): a thread owns 4 columns and loads all rows before it adds.
__global__ void __launch_bounds__(kRowThreads) k_tc_pool_packed(CbView cb, EntryList el, const float* X, void* cache,
                                                                float* cache_f32, int d) {
  const int e = blockIdx.x;
  const int col = ((int)blockIdx.y * kRowThreads + (int)threadIdx.x) * 4;
  if (col >= d) return;
  const int L = entry_len_tc(cb, el, e);
  if (L <= 0) return;
  const float* x = X + (size_t)el.row_off[e] * d + col;
  float4 v[kMaxM];
#pragma unroll
  for (int i = 0; i < kMaxM; ++i)
    if (i < L) v[i] = *reinterpret_cast<const float4*>(x + (size_t)i * d);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int i = 0; i < kMaxM; ++i)
    if (i < L) { acc.x += v[i].x; acc.y += v[i].y; acc.z += v[i].z; acc.w += v[i].w; }
  const size_t dst = ((size_t)el.seq[e] * cb.cap + el.idx[e]) * d + col;
  const float inv = 1.0f / (float)L;
  const float4 m = make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
  uint2 o; o.x = pack_bf16(m.x, m.y); o.y = pack_bf16(m.z, m.w);
  *reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(cache) + dst) = o;
  if (cache_f32) *reinterpret_cast<float4*>(cache_f32 + dst) = m;
}

// LayerNorm of the packed rows of X -> hi/lo (the GEMM epilogue has already added bias and
// residual into X).  grid (row capacity), one encoder.
template <int NV, bool HALF>
__global__ void __launch_bounds__(kRowThreads) k_tc_ln_rows(const int* total, const float* X, const bf16* ln_w,
                                                            const bf16* ln_b, bf16* Ahl, int d, int Rt) {
  __shared__ float sm[32];
  const int r = blockIdx.x;
  if (r >= *total) return;
  const float* x = X + (size_t)r * d;
  const int nvec = d / 4;
  float4 xv[NV];
  uint2 gw[NV], gb[NV];
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) {
      xv[v] = *reinterpret_cast<const float4*>(x + idx * 4);
      gw[v] = reinterpret_cast<const uint2*>(ln_w)[idx];
      gb[v] = reinterpret_cast<const uint2*>(ln_b)[idx];
    }
  }
  bf16* hi = Ahl + (size_t)r * d;
  layernorm_split_regs<NV, HALF>(xv, nvec, gw, gb, hi, hi + (size_t)Rt * d, d, sm);
}

// Bidirectional attention inside one entry from fp32 q, k, v of its packed rows [rows, 3d] (bias
// already added); output as hi/lo.  One WARP per (entry, head): all of the item's q, k, v values
// are loaded into registers at once (a lane holds four columns of every row), the L x L scores are
// warp reductions, no shared memory and no block barrier.  MM = compile-time bound on the merge
// size; dh <= 128 (larger heads take the kernel below).  grid = ceil(entries * heads / 8), block 256.
template <int MM, bool HALF>
__global__ void __launch_bounds__(256) k_tc_attention_rows_warp(CbView cb, EntryList el, const float* QKV, bf16* Ohl,
                                                                int E, int d, int heads, int Rt) {
  const int lane = threadIdx.x & 31;
  const int item = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (item >= E * heads) return;
  const int e = item / heads, h = item - e * heads;
  const int L = entry_len_tc(cb, el, e);
  if (L <= 0) return;
  const int dh = d / heads, c = lane * 4;
  const bool on = c < dh;                      // lanes beyond the head's width hold zeros
  const size_t r0 = el.row_off[e];
  const float* y = QKV + r0 * 3 * d + (size_t)h * dh + c;
  float4 q[MM], k[MM], v[MM];
#pragma unroll
  for (int i = 0; i < MM; ++i) {
    q[i] = k[i] = v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < L && on) {
      const float* yi = y + (size_t)i * 3 * d;
      q[i] = *reinterpret_cast<const float4*>(yi);
      k[i] = *reinterpret_cast<const float4*>(yi + d);
      v[i] = *reinterpret_cast<const float4*>(yi + 2 * d);
    }
  }
  const float scale = 1.0f / sqrtf((float)dh);
  bf16* hi = Ohl + r0 * d + (size_t)h * dh + c;
  bf16* lo = hi + (size_t)Rt * d;
#pragma unroll
  for (int i = 0; i < MM; ++i) {
    if (i >= L) break;
    float s[MM];
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < MM; ++j) {
      float p = q[i].x * k[j].x + q[i].y * k[j].y + q[i].z * k[j].z + q[i].w * k[j].w;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) p += __shfl_xor_sync(0xffffffffu, p, off);
      s[j] = j < L ? p * scale : -INFINITY;
      mx = fmaxf(mx, s[j]);
    }
    float den = 0.f;
#pragma unroll
    for (int j = 0; j < MM; ++j) { s[j] = j < L ? expf(s[j] - mx) : 0.f; den += s[j]; }
    const float inv = 1.0f / den;
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int j = 0; j < MM; ++j) {
      const float wj = s[j] * inv;
      o.x = fmaf(wj, v[j].x, o.x); o.y = fmaf(wj, v[j].y, o.y); o.z = fmaf(wj, v[j].z, o.z); o.w = fmaf(wj, v[j].w, o.w);
    }
    if (on) {
      if (HALF) half_store4(hi + (size_t)i * d, o);
      else split_store4(hi + (size_t)i * d, lo + (size_t)i * d, o);
    }
  }
}

// The same for heads wider than 128 columns or merge sizes above 4: staged in shared memory.
// grid (entries, heads), block (32, M), dynamic smem M * 3 * dh floats.
__global__ void k_tc_attention_rows(CbView cb, EntryList el, const float* QKV, bf16* Ohl, int d, int heads, int Rt,
                                    int half) {
  extern __shared__ float s_qkv[];
  const int e = blockIdx.x, h = blockIdx.y, i = threadIdx.y, lane = threadIdx.x;
  const int L = entry_len_tc(cb, el, e);
  if (L <= 0) return;
  const int dh = d / heads;
  const int r = el.row_off[e] + i;
  if (i < L) {
    const float* y = QKV + (size_t)r * 3 * d;
    for (int w = 0; w < 3; ++w)
      for (int c = lane * 4; c < dh; c += 128)
        *reinterpret_cast<float4*>(&s_qkv[(i * 3 + w) * dh + c]) = *reinterpret_cast<const float4*>(y + w * d + h * dh + c);
  }
  __syncthreads();
  if (i >= L) return;
  const float* q = s_qkv + (i * 3) * dh;
  const float scale = 1.0f / sqrtf((float)dh);
  float s[kMaxM];
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < kMaxM; ++j) {
    s[j] = -INFINITY;
    if (j < L) {
      const float* kp = s_qkv + (j * 3 + 1) * dh;
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
  bf16* hi = Ohl + (size_t)r * d + (size_t)h * dh;
  bf16* lo = hi + (size_t)Rt * d;
  for (int c = lane; c < dh; c += 32) {
    float v = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxM; ++j)
      if (j < L) v = fmaf(s[j] * inv, s_qkv[(j * 3 + 2) * dh + c], v);
    if (half) {
      reinterpret_cast<__half*>(hi)[c] = __float2half_rn(v);
    } else {
      const bf16 hh = __float2bfloat16_rn(v);
      hi[c] = hh;
      lo[c] = __float2bfloat16_rn(v - __bfloat162float(hh));
    }
  }
}

// fp16 copy of a bf16 weight tensor (n a multiple of 8).  A bf16 value inside fp16's range converts
// exactly; a value beyond it cannot be represented and raises bit 1 of the error word.
__global__ void __launch_bounds__(256) k_tc_weights_to_half(const bf16* __restrict__ src, __half* __restrict__ dst,
                                                            size_t n8, int* err) {
  bool over = false;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (size_t)gridDim.x * blockDim.x) {
    const uint4 u = reinterpret_cast<const uint4*>(src)[i];
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
    uint32_t o[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float a = bf_lo(w[k]), b = bf_hi(w[k]);
      over |= fabsf(a) > 65504.f || fabsf(b) > 65504.f;
      o[k] = (uint32_t)__half_as_ushort(__float2half_rn(a)) | ((uint32_t)__half_as_ushort(__float2half_rn(b)) << 16);
    }
    reinterpret_cast<uint4*>(dst)[i] = make_uint4(o[0], o[1], o[2], o[3]);
  }
  if (over) atomicOr(err, 2);
}

int sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 148;
  }
  return n;
}

}  // namespace

bool encoder_tc_supported(int d, int dff, int dtype, int heads, int M) {
  if (heads < 1 || (d / heads) % 4 != 0 || (size_t)M * 3 * (d / heads) * 4 > 48 * 1024) return false;
  return dtype == Z2Z_DTYPE_BF16 && d % kNT == 0 && dff % kNT == 0 && d <= 4 * kRowThreads * kMaxVec4;
}

// Prompt-sized pass of ONE encoder (thousands of rows): the linear layers run as CTA-pair GEMMs
// that own whole output tiles, so bias, residual and GELU are applied in their epilogues; only
// attention, LayerNorm and pooling remain as separate kernels.
static cudaError_t run_encoder_pass_pair(const CbView& cb, const EncoderArgs& a, const EntryList& el, int E,
                                         Prof* prof, cudaStream_t s) {
  const int d = a.d, dff = a.dff, M = cb.M;
  const int R = E * M, Rt = (R + 7) / 8 * 8;
  const bool half = a.w_half != nullptr;               // fp16 copies of the linear-layer weights exist
  auto Wp = [&](int i) { return reinterpret_cast<const bf16*>(a.w[i]); };
  const int* total = el.row_off + E;                   // packed rows of this pass (device word)
  const bool narrow = d <= 4 * kRowThreads * kNarrowVec4;      // a row fits four float4 per thread: fewer registers, more CTAs per SM
  auto lnk = half ? (narrow ? k_tc_ln_rows<kNarrowVec4, true> : k_tc_ln_rows<kMaxVec4, true>)
                  : (narrow ? k_tc_ln_rows<kNarrowVec4, false> : k_tc_ln_rows<kMaxVec4, false>);
  PairGemmParams g{};
  g.cb = cb; g.el = el; g.R = R; g.Rt = Rt; g.live_rows = total; g.err = a.err;
  auto gemm = [&](const bf16* act, int K, int widx, int J, int epi, float* out, bf16* out_hl) -> cudaError_t {
    PairGemmParams p = g;
    p.J = J; p.bias = a.w[widx + 1]; p.out = out; p.out_hl = out_hl;
    ProfScope ps(prof, kProfEncGemm, 1, s);
    return launch_pair_gemm(p, act, half ? a.w_half[widx] : a.w[widx], K, epi, half, s);
  };
  {
    ProfScope ps(prof, kProfEncOther, 2, s);
    k_tc_row_map<<<1, 1024, 0, s>>>(cb, el, E);
    auto gk = half ? (narrow ? k_tc_gather_ln_packed<kNarrowVec4, true> : k_tc_gather_ln_packed<kMaxVec4, true>)
                   : (narrow ? k_tc_gather_ln_packed<kNarrowVec4, false> : k_tc_gather_ln_packed<kMaxVec4, false>);
    gk<<<R, kRowThreads, 0, s>>>(cb, el, total, reinterpret_cast<const bf16*>(a.table), Wp(0), a.layers ? Wp(1) : Wp(0),
                                 a.layers ? Wp(2) : Wp(0), a.X, a.Ahl, d, Rt, a.layers > 0 ? 1 : 0);
  }
  const int dh = d / a.heads;
  cudaError_t e;
  for (int l = 0; l < a.layers; ++l) {
    const int o = 1 + 12 * l;
    if ((e = gemm(a.Ahl, d, o + 2, 3 * d, kEpiStore, a.QKV, nullptr)) != cudaSuccess) return e;
    {
      ProfScope ps(prof, kProfEncOther, 1, s);
      if (dh <= 128 && M <= 4) {
        auto ak = half ? k_tc_attention_rows_warp<4, true> : k_tc_attention_rows_warp<4, false>;
        ak<<<(E * a.heads + 7) / 8, 256, 0, s>>>(cb, el, a.QKV, a.Ahl, E, d, a.heads, Rt);
      } else {
        k_tc_attention_rows<<<dim3(E, a.heads), dim3(32, M), (size_t)M * 3 * dh * 4, s>>>(cb, el, a.QKV, a.Ahl, d,
                                                                                           a.heads, Rt, half ? 1 : 0);
      }
    }
    if ((e = gemm(a.Ahl, d, o + 4, d, kEpiResid, a.X, nullptr)) != cudaSuccess) return e;
    if (dff > 0) {                                     // dff == 0: attention-only layer
      {
        ProfScope ps(prof, kProfEncOther, 1, s);
        lnk<<<R, kRowThreads, 0, s>>>(total, a.X, Wp(o + 6), Wp(o + 7), a.Ahl, d, Rt);
      }
      if ((e = gemm(a.Ahl, d, o + 8, dff, kEpiGelu, nullptr, a.Hhl)) != cudaSuccess) return e;
      if ((e = gemm(a.Hhl, dff, o + 10, d, kEpiResid, a.X, nullptr)) != cudaSuccess) return e;
    }
    if (l + 1 < a.layers) {
      ProfScope ps(prof, kProfEncOther, 1, s);
      lnk<<<R, kRowThreads, 0, s>>>(total, a.X, Wp(o + 12), Wp(o + 13), a.Ahl, d, Rt);
    }
  }
  ProfScope ps(prof, kProfEncOther, 1, s);
  k_tc_pool_packed<<<dim3(E, (d / 4 + kRowThreads - 1) / kRowThreads), kRowThreads, 0, s>>>(cb, el, a.X, a.cache,
                                                                                        a.cache_f32, d);
  return cudaGetLastError();
}

// Bytes of fp16 copies of one encoder's linear-layer weights.
size_t encoder_half_bytes(int d, int dff, int layers) {
  return (size_t)layers * ((size_t)4 * d * d + (size_t)2 * d * dff) * 2;
}

// Whether a pass of `entries` work-list slots is a prompt-sized one (CTA-pair GEMMs).
bool encoder_pass_is_prompt_sized(int entries, int chunk, int M) {
  const int E = entries < chunk ? entries : chunk;
  return E * M >= kPairPassMinRows;
}

// Makes fp16 copies of the linear-layer weights of one encoder in `scratch` and fills
// half_ptrs[i] (host array, ABI tensor order) with their device addresses (nullptr elsewhere).
cudaError_t convert_encoder_weights_to_half(const void* const* w, int d, int dff, int layers, void* scratch,
                                            const void** half_ptrs, int* err_word, Prof* prof, cudaStream_t s) {
  char* dst = reinterpret_cast<char*>(scratch);
  for (int i = 0; i < 1 + 12 * layers; ++i) half_ptrs[i] = nullptr;
  const int n_sm = sm_count();
  for (int l = 0; l < layers; ++l) {
    const int o = 1 + 12 * l;
    const int idx[4] = {o + 2, o + 4, o + 8, o + 10};
    const size_t elems[4] = {(size_t)3 * d * d, (size_t)d * d, (size_t)dff * d, (size_t)d * dff};
    for (int k = 0; k < 4; ++k) {
      if (elems[k] == 0) continue;
      ProfScope ps(prof, kProfEncOther, 1, s);
      k_tc_weights_to_half<<<n_sm * 8, 256, 0, s>>>(reinterpret_cast<const bf16*>(w[idx[k]]),
                                                    reinterpret_cast<__half*>(dst), elems[k] / 8, err_word);
      half_ptrs[idx[k]] = dst;
      dst += elems[k] * 2;
    }
  }
  return cudaGetLastError();
}

cudaError_t run_encoder_pass_tc(const CbView& cb, const EncoderArgs* grp, int ng, const EntryList& el,
                                bool rows_mapped, Prof* prof, cudaStream_t s) {
  const EncoderArgs& a0 = grp[0];
  const int d = a0.d, dff = a0.dff, M = cb.M;
  const int E = a0.entries < el.chunk ? a0.entries : el.chunk;
  const int R = E * M;                                 // row capacity of this pass
  if (ng == 1 && R >= kPairPassMinRows) return run_encoder_pass_pair(cb, a0, el, E, prof, s);
  const int Rt = (R + 7) / 8 * 8;                      // rows of the result matrix per group
  const int row_tiles = (Rt + 127) / 128;
  const int* total = el.row_off + E;                   // packed rows of this pass (device word)
  const int n_sm = sm_count();
  const bool narrow = d <= 4 * kRowThreads * kNarrowVec4;      // a row fits four float4 per thread
  auto rlk = narrow ? k_tc_reduce_resid_ln<kNarrowVec4> : k_tc_reduce_resid_ln<kMaxVec4>;
  float* Y = a0.part;                                  // GEMM results, all zero between GEMMs
  const size_t wide = (size_t)(3 * d > dff ? 3 * d : dff);
  if ((size_t)ng * Rt * wide * sizeof(float) > a0.part_bytes) return cudaErrorMemoryAllocation;
  auto P2 = [&](auto f) { Ptr2 p; p.p[0] = f(grp[0]); p.p[1] = ng > 1 ? f(grp[1]) : f(grp[0]); return p; };
  auto M2 = [&](auto f) { MPtr2 p; p.p[0] = f(grp[0]); p.p[1] = ng > 1 ? f(grp[1]) : f(grp[0]); return p; };
  auto W = [&](int i) { return P2([&](const EncoderArgs& a) { return a.w[i]; }); };
  const MPtr2 X = M2([](const EncoderArgs& a) { return (void*)a.X; });
  const MPtr2 Ahl = M2([](const EncoderArgs& a) { return (void*)a.Ahl; });
  const MPtr2 Hhl = M2([](const EncoderArgs& a) { return (void*)a.Hhl; });
  const MPtr2 cache = M2([](const EncoderArgs& a) { return a.cache; });
  const MPtr2 c32 = M2([](const EncoderArgs& a) { return (void*)a.cache_f32; });
  const Ptr2 table = P2([](const EncoderArgs& a) { return a.table; });

  // one GEMM: activations (hi/lo of packed row r in operand rows 2r, 2r + 1; K columns) x weight
  // [J, K], added into Y[group][Rt][J]
  auto gemm = [&](const MPtr2& act, int K, int widx, int J) -> cudaError_t {
    StreamGemmParams p{};
    p.row_tiles = row_tiles; p.groups = ng; p.tiles_per_group = J / kNT;
    p.a_box_rows = row_tiles == 1 ? 2 * Rt : 256;      // one box per stage: all operand rows of a row tile
    // two k-blocks per stage (fewer TMA operations per byte) while at least four stages still fit
    p.ksb = (K % 128 == 0 && stream_gemm_stages(2, p.a_box_rows) >= 4) ? 2 : 1;
    p.ksteps = (K / 64 + p.ksb - 1) / p.ksb;
    p.out = Y; p.J = J; p.Rt = Rt; p.rows_dev = total;
    p.err = a0.err;
    const long long tiles = (long long)row_tiles * ng * p.tiles_per_group;
    const int G = tiles * p.ksteps < n_sm ? (int)(tiles * p.ksteps) : n_sm;     // every CTA owns >= 1 unit
    CUtensorMap maps[4];
    for (int g = 0; g < 2; ++g) {
      const int gg = g < ng ? g : 0;
      if (!make_tmap_bf16_kblocks(&maps[g], act.p[gg], 2ll * Rt, K, p.a_box_rows, p.ksb)) return cudaErrorInvalidValue;
      if (!make_tmap_bf16_kblocks(&maps[2 + g], grp[gg].w[widx], J, K, kNT, p.ksb)) return cudaErrorInvalidValue;
    }
    ProfScope ps(prof, kProfEncGemm, 1, s);
    return launch_stream_gemm(p, maps, G, s);
  };

  if (!rows_mapped) {
    ProfScope ps(prof, kProfEncOther, 1, s);
    k_tc_row_map<<<1, 1024, 0, s>>>(cb, el, E);
  }
  cudaError_t e;
  {
    ProfScope ps(prof, kProfEncOther, 1, s);
    launch_pdl(narrow ? k_tc_gather_ln<kNarrowVec4> : k_tc_gather_ln<kMaxVec4>, dim3(R, ng), dim3(kRowThreads), 0, s, cb, el, total, table, W(0), a0.layers ? W(1) : W(0),
               a0.layers ? W(2) : W(0), X, Ahl, d, a0.layers > 0 ? 1 : 0);
  }
  if (a0.layers == 0) {
    ProfScope ps(prof, kProfEncOther, 1, s);
    launch_pdl(k_tc_pool, dim3(E, ng), dim3(kRowThreads), 0, s, cb, el, X, cache, c32, d);
  }
  const int dh = d / a0.heads;
  for (int l = 0; l < a0.layers; ++l) {
    const int o = 1 + 12 * l;
    const bool last = l + 1 == a0.layers;
    if ((e = gemm(Ahl, d, o + 2, 3 * d)) != cudaSuccess) return e;
    {
      ProfScope ps(prof, kProfEncOther, 1, s);
      launch_pdl(k_tc_qkv_attention, dim3(E, a0.heads, ng), dim3(32, M), (size_t)M * 3 * dh * 4, s, cb, el, Y,
                 W(o + 3), Ahl, d, a0.heads, Rt);
    }
    if ((e = gemm(Ahl, d, o + 4, d)) != cudaSuccess) return e;
    int last_bias = o + 5;                             // bias of the layer's last linear map
    if (dff > 0) {                                     // dff == 0: attention-only layer
      {
        ProfScope ps(prof, kProfEncOther, 1, s);
        launch_pdl(rlk, dim3(R, ng), dim3(kRowThreads), 0, s, total, Y, W(o + 5), X, W(o + 6),
                   W(o + 7), Ahl, d, Rt);
      }
      if ((e = gemm(Ahl, d, o + 8, dff)) != cudaSuccess) return e;
      {
        ProfScope ps(prof, kProfEncOther, 1, s);
        const long long f4 = (long long)ng * R * (dff / 4);
        const int per_cta = kGeluThreads * kGeluPerThread;
        launch_pdl(k_tc_reduce_gelu, dim3((unsigned)((f4 + per_cta - 1) / per_cta)), dim3(kGeluThreads), 0, s, total, Y,
                   W(o + 9), Hhl, dff, R, Rt, ng);
      }
      if ((e = gemm(Hhl, dff, o + 10, d)) != cudaSuccess) return e;
      last_bias = o + 11;
    }
    {
      ProfScope ps(prof, kProfEncOther, 1, s);
      if (last)
        launch_pdl(k_tc_reduce_resid_pool, dim3(E, ng, (d / 4 + kRowThreads - 1) / kRowThreads), dim3(kRowThreads), 0,
                   s, cb, el, Y, W(last_bias), X, cache, c32, d, Rt);
      else
        launch_pdl(rlk, dim3(R, ng), dim3(kRowThreads), 0, s, total, Y, W(last_bias), X, W(o + 12),
                   W(o + 13), Ahl, d, Rt);
    }
  }
  return cudaGetLastError();
}

}  // namespace z2z
