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
// Layout of a hi/lo operand with Rt rows: bf16 [2 * Rt, K], hi rows first, lo rows after.
//
// Launches per layer: GEMM(qkv) -> [sum partials + bias, attention] -> GEMM(o) ->
// [sum + bias + residual, LayerNorm 2] -> GEMM(1) -> [sum + bias, GELU] -> GEMM(2) ->
// [sum + bias + residual, LayerNorm 1 of the next layer | mean-pool into the cache].
#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_stream.h"

namespace z2z {

namespace {

using bf16 = __nv_bfloat16;
constexpr int kNT = kGemmNT;
constexpr int kRowThreads = 256;
constexpr int kMaxVec4 = 8;            // float4 per thread in the row kernels: d <= 8192

// Where the partial tiles of one GEMM live and how they were cut (mirrors GemmSched).
struct PartView {
  const float* part;
  long long slot_stride;     // floats
  long long U, G;            // units and CTAs of the GEMM launch
  int groups, tpg, ksteps;   // tiles per group, k-steps per tile
  int lo_off;                // >0: lo rows sit lo_off rows below the hi rows inside the slot
};

// Slots holding the partial sums of one tile: slots (tile + c) for c in [c0, c1].
struct TileSlots { long long tile; int c0, c1; };
__device__ __forceinline__ TileSlots tile_slots(const PartView& pv, int rt, int g, int t) {
  TileSlots s;
  s.tile = ((long long)rt * pv.groups + g) * pv.tpg + t;
  s.c0 = (int)owner_of(s.tile * pv.ksteps, pv.U, pv.G);
  s.c1 = (int)owner_of((s.tile + 1) * pv.ksteps - 1, pv.U, pv.G);
  return s;
}
// Sum over the slots, in slot order (deterministic), of 4 consecutive columns of local row lr.
__device__ __forceinline__ float4 part_sum4(const PartView& pv, const TileSlots& ts, int lr, int cj) {
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c = ts.c0; c <= ts.c1; ++c) {
    const float* s = pv.part + (ts.tile + c) * pv.slot_stride + (long long)lr * kNT + cj;
    const float4 a = *reinterpret_cast<const float4*>(s);
    acc.x += a.x; acc.y += a.y; acc.z += a.z; acc.w += a.w;
    if (pv.lo_off) {
      const float4 b = *reinterpret_cast<const float4*>(s + (long long)pv.lo_off * kNT);
      acc.x += b.x; acc.y += b.y; acc.z += b.z; acc.w += b.w;
    }
  }
  return acc;
}
__device__ __forceinline__ float part_sum1(const PartView& pv, const TileSlots& ts, int lr, int cj) {
  float acc = 0.f;
  for (int c = ts.c0; c <= ts.c1; ++c) {
    const float* s = pv.part + (ts.tile + c) * pv.slot_stride + (long long)lr * kNT + cj;
    acc += s[0];
    if (pv.lo_off) acc += s[(long long)pv.lo_off * kNT];
  }
  return acc;
}

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

__device__ __forceinline__ int entry_len_tc(const CbView& cb, const EntryList& el, int e) {
  const int s = el.seq[e];
  return s < 0 ? 0 : (int)cb.len[(size_t)s * cb.cap + el.idx[e]];
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
__device__ __forceinline__ void layernorm_split_regs(const float4 (&x)[kMaxVec4], int nvec, const bf16* g,
                                                     const bf16* b, bf16* hi, bf16* lo, int d, float* sm) {
  float s = 0.f;
#pragma unroll
  for (int v = 0; v < kMaxVec4; ++v)
    if ((int)threadIdx.x + v * kRowThreads < nvec) s += (x[v].x + x[v].y) + (x[v].z + x[v].w);
  const float mean = block_sum(s, sm) / (float)d;
  float q = 0.f;
#pragma unroll
  for (int v = 0; v < kMaxVec4; ++v)
    if ((int)threadIdx.x + v * kRowThreads < nvec) {
      const float a = x[v].x - mean, bb = x[v].y - mean, c = x[v].z - mean, e = x[v].w - mean;
      q += (a * a + bb * bb) + (c * c + e * e);
    }
  const float rstd = 1.0f / sqrtf(block_sum(q, sm) / (float)d + kLnEps);
#pragma unroll
  for (int v = 0; v < kMaxVec4; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) {
      const float4 gg = load_bf16x4(g + idx * 4), bb = load_bf16x4(b + idx * 4);
      float4 y;
      y.x = (x[v].x - mean) * rstd * gg.x + bb.x;
      y.y = (x[v].y - mean) * rstd * gg.y + bb.y;
      y.z = (x[v].z - mean) * rstd * gg.z + bb.z;
      y.w = (x[v].w - mean) * rstd * gg.w + bb.w;
      split_store4(hi + idx * 4, lo + idx * 4, y);
    }
  }
}

// X = table[y] + pos for valid rows; then LN1 of layer 0 -> hi/lo.  grid (rows, groups).
__global__ void __launch_bounds__(kRowThreads) k_tc_gather_ln(CbView cb, EntryList el, Ptr2 table, Ptr2 pos,
                                                              Ptr2 ln_w, Ptr2 ln_b, MPtr2 X, MPtr2 Ahl,
                                                              int d, int Rt, int has_ln) {
  __shared__ float sm[32];
  const int r = blockIdx.x, g = blockIdx.y, e = r / cb.M, i = r - e * cb.M;
  if (e >= el.off[cb.B + 1]) return;
  const int L = entry_len_tc(cb, el, e);
  float* x = reinterpret_cast<float*>(X.p[g]) + (size_t)r * d;
  bf16* hi = reinterpret_cast<bf16*>(Ahl.p[g]) + (size_t)r * d;
  bf16* lo = hi + (size_t)Rt * d;
  const int nvec = d / 4;
  if (i >= L) {                                   // padding row: zero everywhere
    for (int idx = threadIdx.x; idx < nvec; idx += kRowThreads) {
      *reinterpret_cast<float4*>(x + idx * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
      *reinterpret_cast<uint2*>(hi + idx * 4) = make_uint2(0u, 0u);
      *reinterpret_cast<uint2*>(lo + idx * 4) = make_uint2(0u, 0u);
    }
    return;
  }
  const int y = cb.cons[((size_t)el.seq[e] * cb.cap + el.idx[e]) * cb.M + i];
  const bf16* row = reinterpret_cast<const bf16*>(table.p[g]) + (size_t)y * d;
  const bf16* pp = reinterpret_cast<const bf16*>(pos.p[g]) + (size_t)i * d;
  float4 xv[kMaxVec4];
#pragma unroll
  for (int v = 0; v < kMaxVec4; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) {
      const float4 a = load_bf16x4(row + idx * 4), b = load_bf16x4(pp + idx * 4);
      xv[v] = make_float4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w);
      *reinterpret_cast<float4*>(x + idx * 4) = xv[v];
    }
  }
  if (has_ln)
    layernorm_split_regs(xv, nvec, reinterpret_cast<const bf16*>(ln_w.p[g]),
                         reinterpret_cast<const bf16*>(ln_b.p[g]), hi, lo, d, sm);
}

// One row: x = X[r] + sum(partials) + bias, in registers.  Tiles' slot ranges are staged in smem.
__device__ __forceinline__ void row_reduce_resid(const PartView& pv, int r, int g, const float* xrow,
                                                 const bf16* bias, int d, int* s_c0, int* s_c1,
                                                 float4 (&xv)[kMaxVec4]) {
  const int nvec = d / 4, rt = r >> 7, lr = r & 127;
#pragma unroll
  for (int v = 0; v < kMaxVec4; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) {
      const int col = idx * 4, t = col / kNT;
      TileSlots ts;
      ts.tile = ((long long)rt * pv.groups + g) * pv.tpg + t; ts.c0 = s_c0[t]; ts.c1 = s_c1[t];
      const float4 p = part_sum4(pv, ts, lr, col - t * kNT);
      const float4 xo = *reinterpret_cast<const float4*>(xrow + col);
      const float4 bs = load_bf16x4(bias + col);
      xv[v] = make_float4(xo.x + p.x + bs.x, xo.y + p.y + bs.y, xo.z + p.z + bs.z, xo.w + p.w + bs.w);
    }
  }
}

__device__ __forceinline__ void stage_tile_slots(const PartView& pv, int rt, int g, int n_tiles, int* s_c0,
                                                 int* s_c1) {
  for (int t = threadIdx.x; t < n_tiles; t += blockDim.x) {
    const TileSlots ts = tile_slots(pv, rt, g, t);
    s_c0[t] = ts.c0; s_c1[t] = ts.c1;
  }
  __syncthreads();
}

// X[r] += sum(partials) + bias; then LayerNorm -> hi/lo for the next GEMM.  grid (rows, groups).
__global__ void __launch_bounds__(kRowThreads) k_tc_reduce_resid_ln(CbView cb, EntryList el, PartView pv,
                                                                    Ptr2 bias, MPtr2 X, Ptr2 ln_w, Ptr2 ln_b,
                                                                    MPtr2 Ahl, int d, int Rt) {
  __shared__ float sm[32];
  __shared__ int s_c0[64], s_c1[64];
  const int r = blockIdx.x, g = blockIdx.y, e = r / cb.M, i = r - e * cb.M;
  if (e >= el.off[cb.B + 1]) return;
  if (i >= entry_len_tc(cb, el, e)) return;      // padding rows stay zero in X and in hi/lo
  stage_tile_slots(pv, r >> 7, g, d / kNT, s_c0, s_c1);
  float* x = reinterpret_cast<float*>(X.p[g]) + (size_t)r * d;
  float4 xv[kMaxVec4];
  row_reduce_resid(pv, r, g, x, reinterpret_cast<const bf16*>(bias.p[g]), d, s_c0, s_c1, xv);
  const int nvec = d / 4;
#pragma unroll
  for (int v = 0; v < kMaxVec4; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) *reinterpret_cast<float4*>(x + idx * 4) = xv[v];
  }
  bf16* hi = reinterpret_cast<bf16*>(Ahl.p[g]) + (size_t)r * d;
  layernorm_split_regs(xv, nvec, reinterpret_cast<const bf16*>(ln_w.p[g]),
                       reinterpret_cast<const bf16*>(ln_b.p[g]), hi, hi + (size_t)Rt * d, d, sm);
}

// Last layer: x_i = X[r_i] + sum(partials) + bias for the entry's valid rows, cache row = mean_i x_i.
// grid (entries, groups).
__global__ void __launch_bounds__(kRowThreads) k_tc_reduce_resid_pool(CbView cb, EntryList el, PartView pv,
                                                                      Ptr2 bias, MPtr2 X, MPtr2 cache,
                                                                      MPtr2 cache_f32, int d) {
  __shared__ int s_c0[64], s_c1[64];
  const int e = blockIdx.x, g = blockIdx.y;
  if (e >= el.off[cb.B + 1]) return;
  const int L = entry_len_tc(cb, el, e);
  if (L <= 0) return;
  const int nvec = d / 4;
  float4 acc[kMaxVec4];
#pragma unroll
  for (int v = 0; v < kMaxVec4; ++v) acc[v] = make_float4(0.f, 0.f, 0.f, 0.f);
  int staged_rt = -1;
  for (int i = 0; i < L; ++i) {
    const int r = e * cb.M + i;
    if ((r >> 7) != staged_rt) {
      __syncthreads();
      stage_tile_slots(pv, r >> 7, g, d / kNT, s_c0, s_c1);
      staged_rt = r >> 7;
    }
    float4 xv[kMaxVec4];
    row_reduce_resid(pv, r, g, reinterpret_cast<const float*>(X.p[g]) + (size_t)r * d,
                     reinterpret_cast<const bf16*>(bias.p[g]), d, s_c0, s_c1, xv);
#pragma unroll
    for (int v = 0; v < kMaxVec4; ++v)
      if ((int)threadIdx.x + v * kRowThreads < nvec) {
        acc[v].x += xv[v].x; acc[v].y += xv[v].y; acc[v].z += xv[v].z; acc[v].w += xv[v].w;
      }
  }
  const size_t dst = ((size_t)el.seq[e] * cb.cap + el.idx[e]) * d;
  const float inv = 1.0f / (float)L;
  bf16* out = reinterpret_cast<bf16*>(cache.p[g]);
  float* out32 = reinterpret_cast<float*>(cache_f32.p[g]);
#pragma unroll
  for (int v = 0; v < kMaxVec4; ++v) {
    const int idx = (int)threadIdx.x + v * kRowThreads;
    if (idx < nvec) {
      const float4 m = make_float4(acc[v].x * inv, acc[v].y * inv, acc[v].z * inv, acc[v].w * inv);
      uint2 o; o.x = pack_bf16(m.x, m.y); o.y = pack_bf16(m.z, m.w);
      *reinterpret_cast<uint2*>(out + dst + idx * 4) = o;
      if (out32) *reinterpret_cast<float4*>(out32 + dst + idx * 4) = m;
    }
  }
}

// Zero-layer encoder (the parameter-free averaging variant): cache row = mean of X rows.
__global__ void __launch_bounds__(kRowThreads) k_tc_pool(CbView cb, EntryList el, MPtr2 X, MPtr2 cache,
                                                         MPtr2 cache_f32, int d) {
  const int e = blockIdx.x, g = blockIdx.y;
  if (e >= el.off[cb.B + 1]) return;
  const int L = entry_len_tc(cb, el, e);
  if (L <= 0) return;
  const float* x = reinterpret_cast<const float*>(X.p[g]);
  const size_t dst = ((size_t)el.seq[e] * cb.cap + el.idx[e]) * d;
  const float inv = 1.0f / (float)L;
  bf16* out = reinterpret_cast<bf16*>(cache.p[g]);
  float* out32 = reinterpret_cast<float*>(cache_f32.p[g]);
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float v = 0.f;
    for (int i = 0; i < L; ++i) v += x[((size_t)e * cb.M + i) * d + c];
    v *= inv;
    out[dst + c] = __float2bfloat16_rn(v);
    if (out32) out32[dst + c] = v;
  }
}

// H = GELU(sum(partials) + bias) -> hi/lo.  grid (tiles, ceil(rows / 4), groups), block 128:
// warp w handles row 4 * blockIdx.y + w, each lane 4 columns of the tile.
__global__ void __launch_bounds__(128) k_tc_reduce_gelu(CbView cb, EntryList el, PartView pv, Ptr2 bias,
                                                        MPtr2 Hhl, int J, int R, int Rt) {
  const int t = blockIdx.x, g = blockIdx.z;
  const int r = blockIdx.y * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= R || r / cb.M >= el.off[cb.B + 1]) return;
  const TileSlots ts = tile_slots(pv, r >> 7, g, t);
  const float4 p = part_sum4(pv, ts, r & 127, lane * 4);
  const int j = t * kNT + lane * 4;
  const float4 bs = load_bf16x4(reinterpret_cast<const bf16*>(bias.p[g]) + j);
  float4 v = make_float4(p.x + bs.x, p.y + bs.y, p.z + bs.z, p.w + bs.w);
  v.x = 0.5f * v.x * (1.0f + erff(v.x * 0.70710678118654752440f));
  v.y = 0.5f * v.y * (1.0f + erff(v.y * 0.70710678118654752440f));
  v.z = 0.5f * v.z * (1.0f + erff(v.z * 0.70710678118654752440f));
  v.w = 0.5f * v.w * (1.0f + erff(v.w * 0.70710678118654752440f));
  bf16* hi = reinterpret_cast<bf16*>(Hhl.p[g]) + (size_t)r * J + j;
  split_store4(hi, hi + (size_t)Rt * J, v);
}

// q, k, v = sum(partials) + bias for one head of one entry (staged in shared memory), then
// bidirectional attention over the entry's valid rows; output as hi/lo.
// grid (entries, heads, groups), block (32, M), dynamic smem M * 3 * dh floats.
__global__ void k_tc_qkv_attention(CbView cb, EntryList el, PartView pv, Ptr2 bias, MPtr2 Ohl, int d,
                                   int heads, int Rt) {
  extern __shared__ float s_qkv[];
  const int e = blockIdx.x, h = blockIdx.y, g = blockIdx.z, i = threadIdx.y, lane = threadIdx.x;
  if (e >= el.off[cb.B + 1]) return;
  const int L = entry_len_tc(cb, el, e);
  const int dh = d / heads;
  const int r = e * cb.M + i;
  if (i < L) {
    const bf16* bs = reinterpret_cast<const bf16*>(bias.p[g]);
    TileSlots ts; ts.tile = -1; ts.c0 = ts.c1 = 0;
    int cur_t = -1;
    for (int w = 0; w < 3; ++w)
      for (int c = lane; c < dh; c += 32) {
        const int col = w * d + h * dh + c, t = col / kNT;
        if (t != cur_t) { ts = tile_slots(pv, r >> 7, g, t); cur_t = t; }
        s_qkv[(i * 3 + w) * dh + c] = part_sum1(pv, ts, r & 127, col - t * kNT) + __bfloat162float(bs[col]);
      }
  }
  __syncthreads();
  if (i >= L) return;                          // padding rows of the operand stay zero
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
  bf16* hi = reinterpret_cast<bf16*>(Ohl.p[g]) + (size_t)r * d + (size_t)h * dh;
  bf16* lo = hi + (size_t)Rt * d;
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
  if (heads < 1 || (size_t)M * 3 * (d / heads) * 4 > 48 * 1024) return false;
  return dtype == Z2Z_DTYPE_BF16 && d % kNT == 0 && dff % kNT == 0 && d <= 4 * kRowThreads * kMaxVec4;
}

cudaError_t run_encoder_pass_tc(const CbView& cb, const EncoderArgs* grp, int ng, const EntryList& el,
                                Prof* prof, cudaStream_t s) {
  const EncoderArgs& a0 = grp[0];
  const int d = a0.d, dff = a0.dff, M = cb.M;
  const int E = a0.entries < el.chunk ? a0.entries : el.chunk;
  const int R = E * M;                                 // rows of this pass
  const int Rt = (R + 7) / 8 * 8;                      // rows per hi (or lo) block
  const int row_tiles = (Rt + 127) / 128;
  const bool stacked = 2 * Rt <= 128;                  // hi and lo rows share one 128-row MMA
  const int n_sm = sm_count();
  int G = n_sm;
  auto P2 = [&](auto f) { Ptr2 p; p.p[0] = f(grp[0]); p.p[1] = ng > 1 ? f(grp[1]) : f(grp[0]); return p; };
  auto M2 = [&](auto f) { MPtr2 p; p.p[0] = f(grp[0]); p.p[1] = ng > 1 ? f(grp[1]) : f(grp[0]); return p; };
  auto W = [&](int i) { return P2([&](const EncoderArgs& a) { return a.w[i]; }); };
  const MPtr2 X = M2([](const EncoderArgs& a) { return (void*)a.X; });
  const MPtr2 Ahl = M2([](const EncoderArgs& a) { return (void*)a.Ahl; });
  const MPtr2 Hhl = M2([](const EncoderArgs& a) { return (void*)a.Hhl; });
  const MPtr2 cache = M2([](const EncoderArgs& a) { return a.cache; });
  const MPtr2 c32 = M2([](const EncoderArgs& a) { return (void*)a.cache_f32; });
  const Ptr2 table = P2([](const EncoderArgs& a) { return a.table; });

  // one GEMM: activations (hi/lo, K columns) x weight [J, K] -> partial tiles
  auto gemm = [&](const MPtr2& act, int K, int widx, int J, PartView& pv) -> cudaError_t {
    StreamGemmParams p{};
    p.row_tiles = row_tiles; p.groups = ng; p.tiles_per_group = J / kNT;
    p.ksteps = (K / 64 + kGemmKSB - 1) / kGemmKSB;
    p.a_parts = stacked ? 1 : 2;
    p.a_box_rows = stacked ? 2 * Rt : (Rt < 128 ? Rt : 128);
    p.a_part_row = Rt;
    p.out_rows = stacked ? 2 * Rt : (Rt < 128 ? Rt : 128);
    p.part = a0.part;
    p.slot_stride = (long long)p.out_rows * kNT;
    p.err = a0.err;
    const long long tiles = (long long)row_tiles * ng * p.tiles_per_group;
    G = tiles * p.ksteps < n_sm ? (int)(tiles * p.ksteps) : n_sm;     // every CTA owns >= 1 unit
    if ((size_t)(tiles + G) * p.slot_stride * 4 > a0.part_bytes) return cudaErrorMemoryAllocation;
    CUtensorMap maps[4];
    for (int g = 0; g < 2; ++g) {
      const int gg = g < ng ? g : 0;
      if (!make_tmap_bf16(&maps[g], act.p[gg], 2ll * Rt, K, p.a_box_rows)) return cudaErrorInvalidValue;
      if (!make_tmap_bf16(&maps[2 + g], grp[gg].w[widx], J, K, kNT)) return cudaErrorInvalidValue;
    }
    pv.part = p.part; pv.slot_stride = p.slot_stride;
    pv.U = tiles * p.ksteps; pv.G = G; pv.groups = ng; pv.tpg = p.tiles_per_group; pv.ksteps = p.ksteps;
    pv.lo_off = stacked ? Rt : 0;
    ProfScope ps(prof, kProfEncGemm, 1, s);
    return launch_stream_gemm(p, maps, G, s);
  };

  cudaError_t e;
  {
    ProfScope ps(prof, kProfEncOther, 1, s);
    k_tc_gather_ln<<<dim3(R, ng), kRowThreads, 0, s>>>(cb, el, table, W(0), a0.layers ? W(1) : W(0),
                                                       a0.layers ? W(2) : W(0), X, Ahl, d, Rt, a0.layers > 0);
  }
  if (a0.layers == 0) {
    ProfScope ps(prof, kProfEncOther, 1, s);
    k_tc_pool<<<dim3(E, ng), kRowThreads, 0, s>>>(cb, el, X, cache, c32, d);
  }
  const int dh = d / a0.heads;
  for (int l = 0; l < a0.layers; ++l) {
    const int o = 1 + 12 * l;
    const bool last = l + 1 == a0.layers;
    PartView pv{};
    if ((e = gemm(Ahl, d, o + 2, 3 * d, pv)) != cudaSuccess) return e;
    {
      ProfScope ps(prof, kProfEncOther, 1, s);
      k_tc_qkv_attention<<<dim3(E, a0.heads, ng), dim3(32, M), (size_t)M * 3 * dh * 4, s>>>(
          cb, el, pv, W(o + 3), Ahl, d, a0.heads, Rt);
    }
    if ((e = gemm(Ahl, d, o + 4, d, pv)) != cudaSuccess) return e;
    {
      ProfScope ps(prof, kProfEncOther, 1, s);
      k_tc_reduce_resid_ln<<<dim3(R, ng), kRowThreads, 0, s>>>(cb, el, pv, W(o + 5), X, W(o + 6), W(o + 7),
                                                               Ahl, d, Rt);
    }
    if ((e = gemm(Ahl, d, o + 8, dff, pv)) != cudaSuccess) return e;
    {
      ProfScope ps(prof, kProfEncOther, 1, s);
      k_tc_reduce_gelu<<<dim3(dff / kNT, (R + 3) / 4, ng), 128, 0, s>>>(cb, el, pv, W(o + 9), Hhl, dff, R, Rt);
    }
    if ((e = gemm(Hhl, dff, o + 10, d, pv)) != cudaSuccess) return e;
    {
      ProfScope ps(prof, kProfEncOther, 1, s);
      if (last)
        k_tc_reduce_resid_pool<<<dim3(E, ng), kRowThreads, 0, s>>>(cb, el, pv, W(o + 11), X, cache, c32, d);
      else
        k_tc_reduce_resid_ln<<<dim3(R, ng), kRowThreads, 0, s>>>(cb, el, pv, W(o + 11), X, W(o + 12), W(o + 13),
                                                                 Ahl, d, Rt);
    }
  }
  return cudaGetLastError();
}

}  // namespace z2z
