// Joint logits over V u V_h with fused reductions (paper Section 2.3, steps 7-9): CUDA-core
// version.  The column space of a hidden row r of sequence b is
//     [0, V)            rows of W_U, shared by every sequence
//     [V, V + n_vis)    rows of U_h[b], visible to rows of sequence b only
// Columns are cut into tiles of 64; a CTA walks a strided subset of the tiles for one block of
// 64 hidden rows and keeps (max, sum-exp, argmax, best perturbed score) per row in registers, so
// no logit is ever written unless the debug output is requested.  A second small kernel merges
// the per-CTA partial reductions.
#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_simt_tile.cuh"

namespace z2z {

struct TileDesc { const void* base; int col0; int nvalid; int owner; int k0; };

__device__ __forceinline__ TileDesc logits_tile(const CbView& cb, int t, int n_static,
                                                int tiles_per_seq, const void* WU, const void* Uh,
                                                int d, size_t esz) {
  TileDesc td;
  if (t < n_static) {
    td.col0 = t * kTJ; td.k0 = 0; td.owner = -1;
    td.nvalid = cb.V - td.col0 < kTJ ? cb.V - td.col0 : kTJ;
    td.base = reinterpret_cast<const char*>(WU) + (size_t)td.col0 * d * esz;
  } else {
    const int u = t - n_static;
    td.owner = u / tiles_per_seq;
    td.k0 = (u - td.owner * tiles_per_seq) * kTJ;
    td.col0 = cb.V + td.k0;
    const int n = min(cb.n[td.owner], cb.cap);      // a count beyond the cache's rows reads no further than them
    td.nvalid = n - td.k0 < kTJ ? n - td.k0 : kTJ;
    td.base = reinterpret_cast<const char*>(Uh) + ((size_t)td.owner * cb.cap + td.k0) * d * esz;
  }
  return td;
}

template <typename T>
__global__ void __launch_bounds__(256) k_logits_simt(CbView cb, LogitsArgs a, int n_static,
                                                     int tiles_per_seq, int n_tiles) {
  __shared__ SimtSmem sm;
  __shared__ float Cs[kTR][kTJ + 1];
  __shared__ int s_seq[kTR], s_nvis[kTR], s_tgt[kTR];
  __shared__ int s_any;
  const int r0 = blockIdx.y * kTR;
  const int G = gridDim.x, g = blockIdx.x;
  const int t = threadIdx.x;
  if (t < kTR) {
    const int r = r0 + t;
    int sq = -1, nv = 0, tg = -1;
    if (r < a.N) {
      sq = a.row_seq ? a.row_seq[r] : r;
      if (sq < 0 || sq >= cb.B) sq = -1;
      if (sq >= 0) { nv = min(cb.n[sq], cb.cap); if (a.row_nvis) { int q = a.row_nvis[r]; nv = q < nv ? (q < 0 ? 0 : q) : nv; } }
      if (a.targets) tg = a.targets[r];
    }
    s_seq[t] = sq; s_nvis[t] = nv; s_tgt[t] = tg;
  }
  __syncthreads();
  const int row = t >> 2, part = t & 3;            // epilogue role: 4 threads per hidden row
  const int rg = r0 + row;                          // row of this launch
  RowRed red; red.init();
  const uint32_t k0 = (uint32_t)a.seed, k1 = (uint32_t)(a.seed >> 32);
  const uint32_t c2 = (uint32_t)a.step, c3 = (uint32_t)(a.step >> 32);
  const size_t ldbg = (size_t)cb.V + cb.cap;
  for (int tile = g; tile < n_tiles; tile += G) {
    const TileDesc td = logits_tile(cb, tile, n_static, tiles_per_seq, a.WU, a.Uh, a.d, sizeof(T));
    if (td.nvalid <= 0) continue;
    if (td.owner >= 0) {                            // does any row of this block belong to it?
      if (t == 0) s_any = 0;
      __syncthreads();
      if (t < kTR && s_seq[t] == td.owner && s_nvis[t] > td.k0) s_any = 1;
      __syncthreads();
      const int any = s_any;
      __syncthreads();
      if (!any) continue;
    }
    float acc[4][4];
    simt_tile_mainloop<T, T>(sm, reinterpret_cast<const T*>(a.hidden), a.d, r0, a.N,
                             reinterpret_cast<const T*>(td.base), td.nvalid, a.d, acc);
    const int tx = t & 15, ty = t >> 4;
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) Cs[ty * 4 + i][tx * 4 + j] = acc[i][j];
    __syncthreads();
    if (rg < a.N && s_seq[row] >= 0) {
      const int limit = td.owner < 0 ? td.nvalid
                        : (s_seq[row] == td.owner ? min(td.nvalid, s_nvis[row] - td.k0) : 0);
      Philox4 px{0, 0, 0, 0};
      int px_blk = -1;
      for (int j = part * 16; j < part * 16 + 16 && j < limit; ++j) {
        const float l = Cs[row][j];
        const int col = td.col0 + j;
        red.add(l, col);
        if (a.select == Z2Z_SELECT_GUMBEL) {
          if ((col >> 2) != px_blk) {
            px_blk = col >> 2;
            px = philox4x32_10((uint32_t)px_blk, (uint32_t)(a.row_base + rg), c2, c3, k0, k1);
          }
          red.add_score(fmaf(l, a.inv_temperature, gumbel_from_word(philox_word(px, col & 3))), col);
        }
        if (a.logits_debug) a.logits_debug[(size_t)rg * ldbg + col] = l;
        if (col == s_tgt[row] && a.target_logit) a.target_logit[rg] = l;
      }
    }
  }
  // combine the 4 column parts of each row (adjacent lanes), then store the CTA's partial
#pragma unroll
  for (int o = 1; o < 4; o <<= 1) {
    RowRed other;
    other.m = __shfl_xor_sync(0xffffffffu, red.m, o);
    other.s = __shfl_xor_sync(0xffffffffu, red.s, o);
    other.idx = __shfl_xor_sync(0xffffffffu, red.idx, o);
    other.gm = __shfl_xor_sync(0xffffffffu, red.gm, o);
    other.gidx = __shfl_xor_sync(0xffffffffu, red.gidx, o);
    red.merge(other);
  }
  if (part == 0 && rg < a.N) {
    LogitPartial* lp = reinterpret_cast<LogitPartial*>(a.lpart) + (size_t)rg * G + g;
    lp->m = red.m; lp->s = red.s; lp->idx = red.idx; lp->gm = red.gm; lp->gidx = red.gidx;
  }
}

// One warp per row: merge G partials, write the outputs.
__global__ void __launch_bounds__(128) k_logits_merge(LogitsArgs a, int G) {
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= a.N) return;
  const LogitPartial* lp = reinterpret_cast<const LogitPartial*>(a.lpart) + (size_t)r * G;
  RowRed red; red.init();
  for (int g = lane; g < G; g += 32) {
    RowRed o; o.m = lp[g].m; o.s = lp[g].s; o.idx = lp[g].idx; o.gm = lp[g].gm; o.gidx = lp[g].gidx;
    red.merge(o);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    RowRed o;
    o.m = __shfl_xor_sync(0xffffffffu, red.m, off);
    o.s = __shfl_xor_sync(0xffffffffu, red.s, off);
    o.idx = __shfl_xor_sync(0xffffffffu, red.idx, off);
    o.gm = __shfl_xor_sync(0xffffffffu, red.gm, off);
    o.gidx = __shfl_xor_sync(0xffffffffu, red.gidx, off);
    red.merge(o);
  }
  if (lane == 0) {
    if (a.lse) a.lse[r] = red.m + logf(red.s);
    if (a.argmax) a.argmax[r] = red.idx == 0x7fffffff ? -1 : red.idx;
    if (a.max_logit) a.max_logit[r] = red.m;
    if (a.sample) a.sample[r] = red.gidx == 0x7fffffff ? -1 : red.gidx;
  }
}

__global__ void k_fill_nan(float* p, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = __int_as_float(0x7fc00000);
}

cudaError_t run_logits_simt(const CbView& cb, const LogitsArgs& a, LogitsPartInfo* info, Prof* prof,
                            cudaStream_t s) {
  const int n_static = (cb.V + kTJ - 1) / kTJ;
  const int tiles_per_seq = (cb.cap + kTJ - 1) / kTJ;
  const int n_tiles = n_static + cb.B * tiles_per_seq;
  const int row_tiles = (a.N + kTR - 1) / kTR;
  static int n_sm = 0;
  if (!n_sm) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (n_sm <= 0) n_sm = 148;
  }
  int G = (n_sm * 4 + row_tiles - 1) / row_tiles;
  if (G > n_tiles) G = n_tiles;
  while (G > 1 && (size_t)a.N * G * sizeof(LogitPartial) > a.lpart_bytes) --G;
  if ((size_t)a.N * G * sizeof(LogitPartial) > a.lpart_bytes) return cudaErrorInvalidValue;
  if (a.target_logit) {
    ProfScope ps(prof, kProfLogitsMerge, 1, s);
    k_fill_nan<<<(a.N + 255) / 256, 256, 0, s>>>(a.target_logit, a.N);
  }
  {
    ProfScope ps(prof, kProfLogits, 1, s);
    if (a.dtype == Z2Z_DTYPE_FP32)
      k_logits_simt<float><<<dim3(G, row_tiles), 256, 0, s>>>(cb, a, n_static, tiles_per_seq, n_tiles);
    else
      k_logits_simt<__nv_bfloat16><<<dim3(G, row_tiles), 256, 0, s>>>(cb, a, n_static, tiles_per_seq, n_tiles);
  }
  if (info) { info->stride = G; info->count = G; return cudaGetLastError(); }
  ProfScope ps(prof, kProfLogitsMerge, 1, s);
  k_logits_merge<<<(a.N + 3) / 4, 128, 0, s>>>(a, G);
  return cudaGetLastError();
}

__global__ void k_pick_codes(int B, const int32_t* __restrict__ argmax,
                             const int32_t* __restrict__ sample,
                             const int32_t* __restrict__ forced, int32_t* __restrict__ next_codes,
                             int32_t* __restrict__ selected) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int sel = sample ? sample[b] : argmax[b];
  if (selected) selected[b] = sel;
  int code = forced ? forced[b] : sel;
  if (code == Z2Z_CODE_SELECTED) code = sel;
  next_codes[b] = code;
}

cudaError_t launch_pick_codes(int B, const int32_t* argmax, const int32_t* sample,
                              const int32_t* forced, int32_t* next_codes, int32_t* selected,
                              cudaStream_t s) {
  k_pick_codes<<<(B + 127) / 128, 128, 0, s>>>(B, argmax, sample, forced, next_codes, selected);
  return cudaGetLastError();
}

}  // namespace z2z
