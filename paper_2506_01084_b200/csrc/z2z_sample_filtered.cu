// Top-k / nucleus (top-p) filtered sampling on stored logits (beyond the paper, which only says
// that a token is sampled from the joint distribution over base tokens and hypertokens:
// Section 2.3 step 9).  For decode batches the joint logits of all rows are a few megabytes, so
// they can be stored once (z2z_dynamic_logits with its full-logit output) and filtered here; the
// fused argmax / Gumbel-max path of the logits kernels needs no stored logits.
//
// A cluster of 1 to 8 CTAs per row (as many as keep all rows within one wave of the SMs); every
// pass reads the row from L2 (16-byte loads, two in flight per thread), each CTA its share of the
// columns, and the CTAs add up their maxima, sums and digit histograms through distributed shared
// memory between two cluster barriers:
//   1. m = max l,  Z = sum exp((l - m) / T), in one pass and only when a nucleus is asked for;
//   2. top-k: radix select (4 passes of 8 bits over order-preserving keys of the logits) of the
//      k-th largest logit; everything >= it is kept (ties stay together);
//   3. top-p: the same descent weighted by probability mass: the largest logit v with
//      mass{l >= v} >= p Z; everything >= v is kept;
//   4. Gumbel-max over the kept columns with the noise the fused sampler uses
//      (Philox4x32-10 keyed by the seed, counter (column / 4, row, step), word column % 4).
// The thresholds are found on the logits themselves, not on l / T: a positive scale preserves the
// order, and equal logits stay exactly equal.
#include <cooperative_groups.h>

#include "z2z_common.cuh"
#include "z2z_internal.h"

namespace z2z {

namespace {

constexpr int kSfThreads = 1024;

__device__ __forceinline__ uint32_t order_key(float x) {          // larger float <-> larger key
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Histograms of a radix pass are kept once per lane (bin * 32 + lane): the digits of a pass are
// far from uniform (the first digit is sign and exponent, which almost all logits share), and
// 1024 threads adding to one shared-memory word serialise; a lane's own copy is only ever touched
// by the same lane of other warps and sits in its own bank.
struct SfShared {
  union {
    float mass[256 * 32];
    unsigned int cnt[256 * 32];
  } lanes;
  float red_f[32];
  int red_i[32];
  unsigned int hist[256];       // per digit, this CTA's columns: count (top-k pass) or "occupied" flag (nucleus pass)
  float mass[256];              // per digit, this CTA's columns: probability mass
  unsigned int tot_hist[256];   // the same over all CTAs that share the row
  float tot_mass[256];
  float xf[3];                  // what a CTA shows the others: max, partition sum, best score
  int xi[2];                    // best column, kept columns
  float m, Z;
  unsigned int prefix;
  unsigned int k_left;
  float p_left;
};

__device__ __forceinline__ float block_max(float v, SfShared* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh->red_f[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = sh->red_f[threadIdx.x & 31];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t = fmaxf(t, __shfl_xor_sync(0xffffffffu, t, o));
  return t;
}
__device__ __forceinline__ float block_sum_f(float v, SfShared* sh) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh->red_f[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = sh->red_f[threadIdx.x & 31];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
  return t;
}

// Calls f(logit, column) for every column of a row, each thread its share.  A row is read from L2
// seven to eleven times by one CTA, so what counts is the bytes a thread keeps in flight: 16-byte
// loads, two per thread at a time, when the row starts on a 16-byte boundary.
// `t` is the thread's index among the `nt` threads that share the row (all CTAs of the cluster).
template <typename F>
__device__ __forceinline__ void for_each_logit(const float* __restrict__ l, int C, int t, int nt, F f) {
  if ((reinterpret_cast<uintptr_t>(l) & 15u) == 0) {
    const float4* l4 = reinterpret_cast<const float4*>(l);
    const int C4 = C >> 2;
    int i = t;
    for (; i + nt < C4; i += 2 * nt) {
      const float4 a = l4[i], b = l4[i + nt];
      const int ca = 4 * i, cb = 4 * (i + nt);
      f(a.x, ca); f(a.y, ca + 1); f(a.z, ca + 2); f(a.w, ca + 3);
      f(b.x, cb); f(b.y, cb + 1); f(b.z, cb + 2); f(b.w, cb + 3);
    }
    for (; i < C4; i += nt) {
      const float4 a = l4[i];
      const int ca = 4 * i;
      f(a.x, ca); f(a.y, ca + 1); f(a.z, ca + 2); f(a.w, ca + 3);
    }
    for (int c = (C4 << 2) + t; c < C; c += nt) f(l[c], c);
  } else {
    for (int c = t; c < C; c += nt) f(l[c], c);
  }
}

}  // namespace

__global__ void __launch_bounds__(kSfThreads) k_sample_filtered(const float* __restrict__ logits, long long ld,
                                                                const int32_t* __restrict__ n_cols, int top_k,
                                                                float top_p, float inv_t, uint32_t k0, uint32_t k1,
                                                                uint32_t c2, uint32_t c3, int row_base,
                                                                int32_t* __restrict__ choice, int32_t* __restrict__ kept) {
  __shared__ SfShared sh;
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int G = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();     // CTAs that share the row
  const int r = blockIdx.x / G, tid = threadIdx.x;
  const int gt = rank * kSfThreads + tid, gnt = G * kSfThreads;
  const int C = n_cols[r];
  const float* l = logits + (size_t)r * ld;
  if (C <= 0) { if (tid == 0 && rank == 0) { choice[r] = -1; if (kept) kept[r] = 0; } return; }   // (the whole cluster returns)
  // ---- 1. max and partition sum in one pass (running maximum, sum rescaled when it moves); only
  //         the nucleus filter needs them
  float mx = 0.f, z = 0.f;
  if (top_p < 1.0f) {
    float m = -INFINITY, sum = 0.f;
    for_each_logit(l, C, gt, gnt, [&](float x, int) {
      if (x > m) { sum = sum * expf((m - x) * inv_t) + 1.f; m = x; }
      else if (m > -INFINITY) sum += expf((x - m) * inv_t);     // (-inf logits before any finite one add nothing)
    });
    const float m_cta = block_max(m, &sh);
    // (a thread, or further down a CTA, without columns has m = -inf and adds nothing)
    const float s_cta = block_sum_f(m > -INFINITY ? sum * expf((m - m_cta) * inv_t) : 0.f, &sh);
    if (tid == 0) { sh.xf[0] = m_cta; sh.xf[1] = s_cta; }
    cluster.sync();
    mx = m_cta;
    for (int g = 0; g < G; ++g) mx = fmaxf(mx, *cluster.map_shared_rank(&sh.xf[0], g));
    for (int g = 0; g < G; ++g) {                                                 // same order in every CTA
      const float m_g = *cluster.map_shared_rank(&sh.xf[0], g);
      if (m_g > -INFINITY) z += *cluster.map_shared_rank(&sh.xf[1], g) * expf((m_g - mx) * inv_t);
    }
  }
  unsigned int key_k = 0u, key_p = 0u;
  // ---- 2. k-th largest logit by radix descent on counts
  if (top_k > 0 && top_k < C) {
    if (tid == 0) { sh.prefix = 0u; sh.k_left = (unsigned)top_k; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = tid; i < 256 * 32; i += kSfThreads) sh.lanes.cnt[i] = 0u;
      __syncthreads();
      const unsigned int prefix = sh.prefix;
      for_each_logit(l, C, gt, gnt, [&](float x, int) {
        const uint32_t k = order_key(x);
        if (pass == 0 || (k >> (shift + 8)) == prefix) atomicAdd(&sh.lanes.cnt[((k >> shift) & 255u) * 32 + (tid & 31)], 1u);
      });
      __syncthreads();
      for (int d = tid >> 5; d < 256; d += kSfThreads / 32) {          // a warp sums the 32 copies of a digit
        const unsigned int v = __reduce_add_sync(0xffffffffu, sh.lanes.cnt[d * 32 + (tid & 31)]);
        if ((tid & 31) == 0) sh.hist[d] = v;
      }
      cluster.sync();                                    // every CTA's digit counts are in place
      if (tid < 256) {
        unsigned int v = 0u;
        for (int g = 0; g < G; ++g) v += *cluster.map_shared_rank(&sh.hist[tid], g);
        sh.tot_hist[tid] = v;
      }
      cluster.sync();                                    // ... and have been read by everyone
      if (tid < 32) {
        // from the largest digit down: lane L holds digits 255 - 8 L .. 248 - 8 L; the digit in which
        // the running count reaches what is left is the next digit of the k-th largest key (every
        // CTA of the cluster takes the same decision from the same sums)
        unsigned int h[8], mine = 0u;
#pragma unroll
        for (int j = 0; j < 8; ++j) { h[j] = sh.tot_hist[255 - 8 * tid - j]; mine += h[j]; }
        unsigned int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned int t = __shfl_up_sync(0xffffffffu, incl, o);
          if (tid >= o) incl += t;
        }
        const unsigned int left = sh.k_left;
        const unsigned int cross = __ballot_sync(0xffffffffu, incl >= left);
        const int owner = cross ? __ffs(cross) - 1 : 31;           // never reached: the smallest digit
        if (tid == owner) {
          unsigned int rem = left - (incl - mine), d = 248u - 8u * (unsigned)tid;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (h[j] >= rem || (owner == 31 && j == 7)) { d = 255u - 8u * (unsigned)tid - (unsigned)j; break; }
            rem -= h[j];
          }
          sh.k_left = rem;
          sh.prefix = (prefix << 8) | d;
        }
      }
      __syncthreads();
    }
    key_k = sh.prefix;
  }
  // ---- 3. nucleus threshold by radix descent on probability mass
  if (top_p < 1.0f) {
    __syncthreads();
    if (tid == 0) { sh.prefix = 0u; sh.p_left = top_p * z; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      for (int i = tid; i < 256 * 32; i += kSfThreads) sh.lanes.mass[i] = 0.f;
      if (tid < 256) sh.hist[tid] = 0u;
      __syncthreads();
      const unsigned int prefix = sh.prefix;
      for_each_logit(l, C, gt, gnt, [&](float x, int) {
        const uint32_t k = order_key(x);
        if (pass == 0 || (k >> (shift + 8)) == prefix) {
          const unsigned int d = (k >> shift) & 255u;
          atomicAdd(&sh.lanes.mass[d * 32 + (tid & 31)], expf((x - mx) * inv_t));
          sh.hist[d] = 1u;                                         // occupied (every writer stores 1)
        }
      });
      __syncthreads();
      for (int d = tid >> 5; d < 256; d += kSfThreads / 32) {          // a warp sums the 32 copies of a digit
        float v = sh.lanes.mass[d * 32 + (tid & 31)];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if ((tid & 31) == 0) sh.mass[d] = v;
      }
      cluster.sync();                                    // every CTA's digit masses are in place
      if (tid < 256) {
        float v = 0.f;
        unsigned int occ = 0u;
        for (int g = 0; g < G; ++g) {
          v += *cluster.map_shared_rank(&sh.mass[tid], g);
          occ |= *cluster.map_shared_rank(&sh.hist[tid], g);
        }
        sh.tot_mass[tid] = v; sh.tot_hist[tid] = occ;
      }
      cluster.sync();                                    // ... and have been read by everyone
      if (tid < 32) {
        // the same descent on probability mass (unoccupied digits hold none)
        float h[8], mine = 0.f;
        int low = 256;                                     // smallest occupied digit of this lane
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int d = 255 - 8 * tid - j;
          h[j] = sh.tot_mass[d]; mine += h[j];
          if (sh.tot_hist[d]) low = d;
        }
        float incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const float t = __shfl_up_sync(0xffffffffu, incl, o);
          if (tid >= o) incl += t;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) low = min(low, __shfl_xor_sync(0xffffffffu, low, o));
        const float left = sh.p_left;
        // the owner is the first lane whose running mass reaches what is left AND that finds the
        // digit inside itself (the sums of a lane and of its digits may round differently)
        float rem = left - (incl - mine);
        int dsel = -1;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (dsel < 0) {
            if (h[j] >= rem && sh.tot_hist[255 - 8 * tid - j]) dsel = 255 - 8 * tid - j;
            else rem -= h[j];
          }
        }
        const unsigned int cross = __ballot_sync(0xffffffffu, dsel >= 0);
        if (cross) {
          if (tid == __ffs(cross) - 1) { sh.p_left = rem; sh.prefix = (prefix << 8) | (unsigned)dsel; }
        } else if (tid == 31) {                            // rounding: the mass ran out; keep everything here
          sh.p_left = rem;
          sh.prefix = (prefix << 8) | (unsigned)(low < 256 ? low : 0);
        }
      }
      __syncthreads();
    }
    key_p = sh.prefix;
  }
  const unsigned int key_t = key_k > key_p ? key_k : key_p;
  // ---- 4. Gumbel-max over the kept columns (lowest index on ties)
  float best = -INFINITY;
  int best_c = 0x7fffffff, n_kept = 0;
  for_each_logit(l, C, gt, gnt, [&](float x, int c) {
    if (order_key(x) < key_t) return;
    ++n_kept;
    const Philox4 px = philox4x32_10((uint32_t)(c >> 2), (uint32_t)(row_base + r), c2, c3, k0, k1);
    const float s = fmaf(x, inv_t, gumbel_from_word(philox_word(px, c & 3)));
    if (s > best || (s == best && c < best_c)) { best = s; best_c = c; }
  });
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ob = __shfl_xor_sync(0xffffffffu, best, o);
    const int oc = __shfl_xor_sync(0xffffffffu, best_c, o);
    n_kept += __shfl_xor_sync(0xffffffffu, n_kept, o);
    if (ob > best || (ob == best && oc < best_c)) { best = ob; best_c = oc; }
  }
  __syncthreads();
  if ((tid & 31) == 0) { sh.red_f[tid >> 5] = best; sh.red_i[tid >> 5] = best_c; sh.hist[tid >> 5] = (unsigned)n_kept; }
  __syncthreads();
  if (tid < 32) {
    best = sh.red_f[tid]; best_c = sh.red_i[tid]; n_kept = (int)sh.hist[tid];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oc = __shfl_xor_sync(0xffffffffu, best_c, o);
      n_kept += __shfl_xor_sync(0xffffffffu, n_kept, o);
      if (ob > best || (ob == best && oc < best_c)) { best = ob; best_c = oc; }
    }
    if (tid == 0) { sh.xf[2] = best; sh.xi[0] = best_c; sh.xi[1] = n_kept; }
  }
  cluster.sync();
  if (rank == 0 && tid == 0) {
    best = -INFINITY; best_c = 0x7fffffff; n_kept = 0;
    for (int g = 0; g < G; ++g) {
      const float ob = *cluster.map_shared_rank(&sh.xf[2], g);
      const int oc = *cluster.map_shared_rank(&sh.xi[0], g);
      n_kept += *cluster.map_shared_rank(&sh.xi[1], g);
      if (ob > best || (ob == best && oc < best_c)) { best = ob; best_c = oc; }
    }
    choice[r] = best_c == 0x7fffffff ? -1 : best_c;
    if (kept) kept[r] = n_kept;
  }
  cluster.sync();                                        // no CTA leaves while its shared memory may be read
}

}  // namespace z2z

extern "C" int32_t z2z_sample_filtered(const float* d_logits, int32_t N, int64_t ld, const int32_t* d_n_cols,
                                       int32_t top_k, float top_p, float temperature, uint64_t seed, uint64_t step,
                                       int32_t row_base, int32_t* d_choice, int32_t* d_kept, z2z_stream stream) {
  auto fail = [](const char* msg) { z2z::set_last_error(msg); return (int32_t)Z2Z_ERR_INVALID_ARG; };
  if (N < 0) return fail("N < 0");
  if (N == 0) return Z2Z_OK;
  if (!d_logits || !d_n_cols || !d_choice) return fail("d_logits / d_n_cols / d_choice is NULL");
  if (!(temperature > 0.f)) return fail("sampling needs temperature > 0");
  if (!(top_p > 0.f)) return fail("top_p must be > 0 (>= 1: no nucleus filter)");
  if (ld < 1) return fail("ld < 1");
  // a decode batch has far fewer rows than the GPU has SMs, and one SM reads a row from L2 at a
  // fraction of what the row's passes need: a cluster of G CTAs shares a row (G x N CTAs stay
  // within one wave of the 148 SMs)
  int G = 1;
  while (G < 8 && (long long)N * (2 * G) <= 148) G *= 2;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)N * (unsigned)G);
  lc.blockDim = dim3(z2z::kSfThreads);
  lc.dynamicSmemBytes = 0;
  lc.stream = reinterpret_cast<cudaStream_t>(stream);
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)G; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  lc.attrs = at; lc.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&lc, z2z::k_sample_filtered, d_logits, (long long)ld, d_n_cols, top_k, top_p,
                                     1.0f / temperature, (uint32_t)seed, (uint32_t)(seed >> 32), (uint32_t)step,
                                     (uint32_t)(step >> 32), row_base, d_choice, d_kept);
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) { z2z::set_last_error(cudaGetErrorString(e)); return Z2Z_ERR_CUDA; }
  return Z2Z_OK;
}
