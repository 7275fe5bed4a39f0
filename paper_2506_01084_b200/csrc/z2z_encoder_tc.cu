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
#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_stream.h"

namespace z2z {

namespace {

using bf16 = __nv_bfloat16;
constexpr int kNT = kGemmNT;

// Where the partial tiles of one GEMM live and how they were cut (mirrors GemmSched).
struct PartView {
  const float* part;
  long long slot_stride;     // floats
  long long U, G;            // units and CTAs of the GEMM launch
  int groups, tpg, ksteps;   // tiles per group, k-steps per tile
  int out_rows;              // rows per slot
  int lo_off;                // >0: lo rows sit lo_off rows below the hi rows inside the slot
};

// Sum of all partial tiles at (row tile rt, group g, tile t, local row lr, column cj), fixed order.
__device__ __forceinline__ float part_sum(const PartView& pv, int rt, int g, int t, int lr, int cj) {
  const long long tile = ((long long)rt * pv.groups + g) * pv.tpg + t;
  const long long c0 = owner_of(tile * pv.ksteps, pv.U, pv.G);
  const long long c1 = owner_of((tile + 1) * pv.ksteps - 1, pv.U, pv.G);
  float acc = 0.f;
  for (long long c = c0; c <= c1; ++c) {
    const float* s = pv.part + (tile + c) * pv.slot_stride + (long long)lr * kNT + cj;
    acc += s[0];
    if (pv.lo_off) acc += s[(long long)pv.lo_off * kNT];
  }
  return acc;
}

struct Ptr2 { const void* p[2]; };
struct MPtr2 { void* p[2]; };

__device__ __forceinline__ void split_store(bf16* hi, bf16* lo, float x) {
  const bf16 h = __float2bfloat16_rn(x);
  *hi = h;
  *lo = __float2bfloat16_rn(x - __bfloat162float(h));
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

// LayerNorm of one row held in global fp32, written as hi/lo bf16.  Whole block, 256 threads.
__device__ __forceinline__ void row_layernorm_split(const float* x, const bf16* g, const bf16* b,
                                                    bf16* hi, bf16* lo, int d, float* sm) {
  float s = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) s += x[c];
  const float mean = block_sum(s, sm) / (float)d;
  float q = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) { const float t = x[c] - mean; q += t * t; }
  const float rstd = 1.0f / sqrtf(block_sum(q, sm) / (float)d + kLnEps);
  for (int c = threadIdx.x; c < d; c += blockDim.x)
    split_store(hi + c, lo + c, (x[c] - mean) * rstd * __bfloat162float(g[c]) + __bfloat162float(b[c]));
}

// X = table[y] + pos for valid rows; then LN1 of layer 0 -> hi/lo.  grid (rows, groups).
__global__ void __launch_bounds__(256) k_tc_gather_ln(CbView cb, EntryList el, Ptr2 table, Ptr2 pos,
                                                      Ptr2 ln_w, Ptr2 ln_b, MPtr2 X, MPtr2 Ahl,
                                                      int d, int Rt, int has_ln) {
  __shared__ float sm[32];
  const int r = blockIdx.x, g = blockIdx.y, e = r / cb.M, i = r - e * cb.M;
  if (e >= el.off[cb.B + 1]) return;
  const int L = entry_len_tc(cb, el, e);
  float* x = reinterpret_cast<float*>(X.p[g]) + (size_t)r * d;
  bf16* hi = reinterpret_cast<bf16*>(Ahl.p[g]) + (size_t)r * d;
  bf16* lo = hi + (size_t)Rt * d;
  if (i >= L) {
    for (int c = threadIdx.x; c < d; c += blockDim.x) {
      x[c] = 0.f; hi[c] = __float2bfloat16_rn(0.f); lo[c] = __float2bfloat16_rn(0.f);
    }
    return;
  }
  const int y = cb.cons[((size_t)el.seq[e] * cb.cap + el.idx[e]) * cb.M + i];
  const bf16* row = reinterpret_cast<const bf16*>(table.p[g]) + (size_t)y * d;
  const bf16* pp = reinterpret_cast<const bf16*>(pos.p[g]) + (size_t)i * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x) x[c] = __bfloat162float(row[c]) + __bfloat162float(pp[c]);
  __syncthreads();
  if (has_ln)
    row_layernorm_split(x, reinterpret_cast<const bf16*>(ln_w.p[g]), reinterpret_cast<const bf16*>(ln_b.p[g]),
                        hi, lo, d, sm);
}

// Y[r, j] = sum(partials) + bias[j].  MODE 0: fp32 out; MODE 1: GELU then hi/lo out.
// grid (tiles, rows, groups), block = NT threads (one column each).
template <int MODE>
__global__ void __launch_bounds__(kNT) k_tc_reduce_cols(CbView cb, EntryList el, PartView pv, Ptr2 bias,
                                                        MPtr2 out, int J, int Rt) {
  const int t = blockIdx.x, r = blockIdx.y, g = blockIdx.z;
  const int e = r / cb.M;
  if (e >= el.off[cb.B + 1]) return;
  const int j = t * kNT + threadIdx.x;
  float v = part_sum(pv, r >> 7, g, t, r & 127, threadIdx.x) +
            __bfloat162float(reinterpret_cast<const bf16*>(bias.p[g])[j]);
  if (MODE == 0) {
    reinterpret_cast<float*>(out.p[g])[(size_t)r * J + j] = v;
  } else {
    v = 0.5f * v * (1.0f + erff(v * 0.70710678118654752440f));
    bf16* hi = reinterpret_cast<bf16*>(out.p[g]) + (size_t)r * J + j;
    split_store(hi, hi + (size_t)Rt * J, v);
  }
}

// X[r] += sum(partials) + bias; then (optionally) LayerNorm -> hi/lo for the next GEMM.
// grid (rows, groups), block 256.
__global__ void __launch_bounds__(256) k_tc_reduce_resid_ln(CbView cb, EntryList el, PartView pv, Ptr2 bias,
                                                            MPtr2 X, Ptr2 ln_w, Ptr2 ln_b, MPtr2 Ahl,
                                                            int d, int Rt, int has_ln) {
  __shared__ float sm[32];
  const int r = blockIdx.x, g = blockIdx.y, e = r / cb.M, i = r - e * cb.M;
  if (e >= el.off[cb.B + 1]) return;
  const int L = entry_len_tc(cb, el, e);
  if (i >= L) return;                          // padding rows stay zero in X and in hi/lo
  float* x = reinterpret_cast<float*>(X.p[g]) + (size_t)r * d;
  const bf16* bs = reinterpret_cast<const bf16*>(bias.p[g]);
  for (int c = threadIdx.x; c < d; c += blockDim.x)
    x[c] += part_sum(pv, r >> 7, g, c / kNT, r & 127, c % kNT) + __bfloat162float(bs[c]);
  __syncthreads();
  if (has_ln) {
    bf16* hi = reinterpret_cast<bf16*>(Ahl.p[g]) + (size_t)r * d;
    row_layernorm_split(x, reinterpret_cast<const bf16*>(ln_w.p[g]), reinterpret_cast<const bf16*>(ln_b.p[g]),
                        hi, hi + (size_t)Rt * d, d, sm);
  }
}

// Attention inside one entry; fp32 q, k, v in, hi/lo out.  grid (entries, heads, groups), block (32, M).
__global__ void k_tc_attention(CbView cb, EntryList el, MPtr2 QKV, MPtr2 Ohl, int d, int heads, int Rt) {
  const int e = blockIdx.x, h = blockIdx.y, g = blockIdx.z, i = threadIdx.y, lane = threadIdx.x;
  if (e >= el.off[cb.B + 1]) return;
  const int L = entry_len_tc(cb, el, e);
  if (i >= L) return;                          // padding rows of the operand stay zero
  const int dh = d / heads;
  const float* qkv = reinterpret_cast<const float*>(QKV.p[g]);
  bf16* hi = reinterpret_cast<bf16*>(Ohl.p[g]) + ((size_t)e * cb.M + i) * d + (size_t)h * dh;
  bf16* lo = hi + (size_t)Rt * d;
  const float* q = qkv + ((size_t)e * cb.M + i) * 3 * d + (size_t)h * dh;
  const float scale = 1.0f / sqrtf((float)dh);
  float s[kMaxM];
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < kMaxM; ++j) {
    s[j] = -INFINITY;
    if (j < L) {
      const float* kp = qkv + ((size_t)e * cb.M + j) * 3 * d + d + (size_t)h * dh;
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
      if (j < L) v = fmaf(s[j] * inv, qkv[((size_t)e * cb.M + j) * 3 * d + 2 * d + (size_t)h * dh + c], v);
    split_store(hi + c, lo + c, v);
  }
}

// cache[seq][idx] = mean over valid rows.  grid (entries, groups), block 256.
__global__ void __launch_bounds__(256) k_tc_pool(CbView cb, EntryList el, MPtr2 X, MPtr2 cache, MPtr2 cache_f32,
                                                 int d) {
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

bool encoder_tc_supported(int d, int dff, int dtype) {
  return dtype == Z2Z_DTYPE_BF16 && d % kNT == 0 && dff % kNT == 0 && d % 64 == 0 && dff % 64 == 0;
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
  const MPtr2 QKV = M2([](const EncoderArgs& a) { return (void*)a.QKV; });
  const MPtr2 Ahl = M2([](const EncoderArgs& a) { return (void*)a.Ahl; });
  const MPtr2 Hhl = M2([](const EncoderArgs& a) { return (void*)a.Hhl; });
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
    pv.out_rows = p.out_rows; pv.lo_off = stacked ? Rt : 0;
    ProfScope ps(prof, kProfEncGemm, 1, s);
    return launch_stream_gemm(p, maps, G, s);
  };

  cudaError_t e;
  {
    ProfScope ps(prof, kProfEncOther, 1, s);
    k_tc_gather_ln<<<dim3(R, ng), 256, 0, s>>>(cb, el, table, W(0), a0.layers ? W(1) : W(0),
                                               a0.layers ? W(2) : W(0), X, Ahl, d, Rt, a0.layers > 0);
  }
  for (int l = 0; l < a0.layers; ++l) {
    const int o = 1 + 12 * l;
    const bool last = l + 1 == a0.layers;
    PartView pv{};
    if ((e = gemm(Ahl, d, o + 2, 3 * d, pv)) != cudaSuccess) return e;
    {
      ProfScope ps(prof, kProfEncOther, 2, s);
      k_tc_reduce_cols<0><<<dim3(3 * d / kNT, R, ng), kNT, 0, s>>>(cb, el, pv, W(o + 3), QKV, 3 * d, Rt);
      k_tc_attention<<<dim3(E, a0.heads, ng), dim3(32, M), 0, s>>>(cb, el, QKV, Ahl, d, a0.heads, Rt);
    }
    if ((e = gemm(Ahl, d, o + 4, d, pv)) != cudaSuccess) return e;
    {
      ProfScope ps(prof, kProfEncOther, 1, s);
      k_tc_reduce_resid_ln<<<dim3(R, ng), 256, 0, s>>>(cb, el, pv, W(o + 5), X, W(o + 6), W(o + 7), Ahl, d, Rt, 1);
    }
    if ((e = gemm(Ahl, d, o + 8, dff, pv)) != cudaSuccess) return e;
    {
      ProfScope ps(prof, kProfEncOther, 1, s);
      k_tc_reduce_cols<1><<<dim3(dff / kNT, R, ng), kNT, 0, s>>>(cb, el, pv, W(o + 9), Hhl, dff, Rt);
    }
    if ((e = gemm(Hhl, dff, o + 10, d, pv)) != cudaSuccess) return e;
    {
      ProfScope ps(prof, kProfEncOther, 1, s);
      k_tc_reduce_resid_ln<<<dim3(R, ng), 256, 0, s>>>(cb, el, pv, W(o + 11), X, last ? W(0) : W(o + 12),
                                                      last ? W(0) : W(o + 13), Ahl, d, Rt, last ? 0 : 1);
    }
  }
  {
    ProfScope ps(prof, kProfEncOther, 1, s);
    MPtr2 cache = M2([](const EncoderArgs& a) { return a.cache; });
    MPtr2 c32 = M2([](const EncoderArgs& a) { return (void*)a.cache_f32; });
    k_tc_pool<<<dim3(E, ng), 256, 0, s>>>(cb, el, X, cache, c32, d);
  }
  return cudaGetLastError();
}

}  // namespace z2z
