// Weight-streaming skinny GEMM on tcgen05 tensor cores, for the HBM-bound decode regime.
//
//   D[r, j] = sum_k A[r, k] * W[j, k]      A: activation rows (bf16, K-major), few
//                                          W: weight rows streamed once from HBM (bf16, K-major)
//
// One persistent CTA per SM.  Warp 0 issues TMA loads into a ring of shared-memory stages, warp 1
// issues tcgen05.mma (fp32 accumulators in tensor memory, double buffered), warps 2-5 drain
// accumulators.  Two kernels share the ring and its barriers:
//   * hyper-encoder linear layers (k_stream_gemm): a tile of 128 weight rows is the MMA's M
//     operand, the packed activation rows (hi and lo part of a row in adjacent operand rows) its
//     N operand, as wide as the rows that exist; work is cut stream-K style, every CTA gets the
//     same number of (tile, k-step) units and adds its accumulators into one fp32 result matrix
//     with reductions in global memory (sums of two or three partial tiles in arrival order);
//   * joint logits for 33 .. 2047 hidden rows (k_stream_logits; paper Section 2.3 steps 7-9):
//     the hidden rows are the 128-row M operand, tiles run over W_U and then over the visible
//     rows of each sequence's U_h; the epilogue keeps max / sum-exp / argmax / best perturbed
//     score per hidden row in registers, so the logits are never written.  Only the hidden rows
//     that exist are loaded: the MMA also reads the shared memory behind them, which only feeds
//     accumulator rows nobody reads (rows of D depend on the same rows of A only).
#include <mutex>
#include <unordered_map>

#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_sm100.cuh"
#include "z2z_stream.h"

namespace z2z {
using namespace sm100;

namespace {

constexpr int kThreads = 192;
constexpr int kTailPad = 16384;          // readable shared memory behind the last A tile

struct Ctrl {
  unsigned long long full[kMaxStages], empty[kMaxStages], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort;
  int vt;                                // logits: number of virtual column tiles
};

__host__ __device__ constexpr int tmem_cols(int nt) {
  return 2 * nt <= 32 ? 32 : (2 * nt <= 64 ? 64 : (2 * nt <= 128 ? 128 : (2 * nt <= 256 ? 256 : 512)));
}

struct Job {
  int amap, wmap;        // tensor map indices
  int arow, wrow;        // first row in A / W tensors
  int kb0, kb1;          // k-step range
  long long slot;        // GEMM: partial slot
  int col0, nvalid, owner, k0;   // logits: first column id, valid rows, owning sequence, first entry
  int rt;                // hidden-row tile
  int nrows;             // weight rows in this job (the MMA's N), multiple of 16
  int wbox_min;          // smallest TMA box of W in rows; boxes are powers of two times this, up
  int wbox_classes;      // to wbox_min << (wbox_classes - 1); tensor map = wmap * classes + class
};

// ---- logits schedule ----------------------------------------------------------------------------
// Columns are dealt in granules of kLogitGran rows: first the granules of W_U, then those of the
// visible rows of each sequence's U_h.  Every CTA owns the same number of granules (+-1); a job
// is a run of up to NT / kLogitGran granules inside one segment (W_U, or one sequence).
struct LogitSched {
  const StreamLogitsParams& p;
  const int* pref;       // shared: prefix of per-sequence granule counts, [B + 1]
  long long u, u1;
  int n_static, vt, ksteps;
  __device__ LogitSched(const StreamLogitsParams& pp, const int* s_pref, int vt_, int NT) : p(pp), pref(s_pref) {
    n_static = (p.cb.V + kLogitGran - 1) / kLogitGran;
    vt = vt_;
    ksteps = p.ksteps;
    const long long U = (long long)p.row_tiles * vt, G = gridDim.x, c = blockIdx.x;
    u = c * U / G;
    u1 = (c + 1) * U / G;
    (void)NT;
  }
  __device__ bool next(Job& j, int NT) {
    if (u >= u1) return false;
    j.rt = (int)(u / vt);
    const int v = (int)(u - (long long)j.rt * vt);
    j.amap = 0; j.arow = j.rt * 128; j.kb0 = 0; j.kb1 = ksteps; j.slot = 0;
    j.wbox_min = kLogitGran; j.wbox_classes = kLogitBoxClasses;
    int remaining, total_rows, g0;
    if (v < n_static) {
      g0 = v; remaining = n_static - v; total_rows = p.cb.V;
      j.wmap = 0; j.wrow = g0 * kLogitGran; j.col0 = g0 * kLogitGran; j.owner = -1; j.k0 = 0;
    } else {
      const int x = v - n_static;
      int lo = 0, hi = p.cb.B - 1;                 // last b with pref[b] <= x
      while (lo < hi) { int mid = (lo + hi + 1) >> 1; if (pref[mid] <= x) lo = mid; else hi = mid - 1; }
      g0 = x - pref[lo]; remaining = pref[lo + 1] - pref[lo] - g0; total_rows = p.cb.n[lo];
      j.owner = lo; j.k0 = g0 * kLogitGran;
      j.wmap = 1; j.wrow = lo * p.cb.cap + j.k0; j.col0 = p.cb.V + j.k0;
    }
    int ng = NT / kLogitGran;
    if (remaining < ng) ng = remaining;
    if (u1 - u < ng) ng = (int)(u1 - u);
    j.nrows = ng * kLogitGran;
    j.nvalid = total_rows - g0 * kLogitGran < j.nrows ? total_rows - g0 * kLogitGran : j.nrows;
    u += ng;
    return true;
  }
};

// ---- roles shared by both kernels -----------------------------------------------------------------
template <int NT, int KSB, int STAGES, class Sched>
__device__ __forceinline__ void producer_role(Sched& sched, Ctrl* ctrl, uint32_t stage_base,
                                              int a_parts, int a_box_rows, int a_part_row,
                                              const CUtensorMap* const* amaps,
                                              const CUtensorMap* const* wmaps) {
  const uint32_t a_part_bytes = (uint32_t)KSB * a_box_rows * 128;
  const uint32_t stage_bytes = a_parts * a_part_bytes + (uint32_t)KSB * NT * 128;   // smem stride of a stage
  const uint64_t pol_w = policy_evict_first(), pol_a = policy_evict_last();
  int stage = 0; uint32_t phase = 0;
  // The weight tiles depend on no earlier kernel, the activation tiles do.  During the first
  // pass over the ring only the weight boxes are issued and the activation boxes are noted; once
  // the ring is full (or the work ends) the producer waits for the preceding kernel and issues
  // them.  With an ordinary launch the wait returns at once.
  struct Deferred { uint32_t dst, bar; int map, row, kb; };
  Deferred def[kMaxStages * 2];
  int n_def = 0, issued = 0;
  bool deps = false;
  auto need_deps = [&]() {
    if (deps) return;
    pdl_wait();
    for (int i = 0; i < n_def; ++i) tma_load_3d(def[i].dst, amaps[def[i].map], 0, def[i].row, def[i].kb, def[i].bar, pol_a);
    deps = true;
  };
  Job j;
  while (sched.next(j, NT)) {
    for (int ks = j.kb0; ks < j.kb1; ++ks) {
      if (issued == STAGES) need_deps();
      if (!mbar_wait(smem_u32(&ctrl->empty[stage]), phase ^ 1u, &ctrl->abort)) return;
      const uint32_t full = smem_u32(&ctrl->full[stage]);
      mbar_expect_tx(full, a_parts * a_part_bytes + (uint32_t)KSB * j.nrows * 128);
      const uint32_t sb = stage_base + (uint32_t)stage * stage_bytes;
      // one box per operand part: KSB k-blocks of the rows, laid out k-block after k-block
      for (int part = 0; part < a_parts; ++part) {
        const uint32_t dst = sb + part * a_part_bytes;
        const int row = j.arow + part * a_part_row;
        if (deps) tma_load_3d(dst, amaps[j.amap], 0, row, ks * KSB, full, pol_a);
        else { def[n_def].dst = dst; def[n_def].bar = full; def[n_def].map = j.amap; def[n_def].row = row; def[n_def].kb = ks * KSB; ++n_def; }
      }
      // the W rows of the job go out as few boxes as possible: largest power-of-two box first
      // (several boxes only with KSB == 1: a box's k-blocks lie one box height apart)
      for (int r0 = 0; r0 < j.nrows;) {
        int cls = j.wbox_classes - 1;
        while (cls > 0 && (j.wbox_min << cls) > j.nrows - r0) --cls;
        tma_load_3d(sb + a_parts * a_part_bytes + r0 * 128, wmaps[j.wmap * j.wbox_classes + cls], 0, j.wrow + r0,
                    ks * KSB, full, pol_w);
        r0 += j.wbox_min << cls;
      }
      ++issued;
      if (++stage == STAGES) { stage = 0; phase ^= 1u; }
    }
  }
  need_deps();
}

template <int NT, int KSB, int STAGES, class Sched>
__device__ __forceinline__ void mma_role(Sched& sched, Ctrl* ctrl, uint32_t stage_base, int a_parts,
                                         int a_box_rows, uint32_t tmem_base) {
  const uint32_t a_part_bytes = (uint32_t)KSB * a_box_rows * 128;
  const uint32_t stage_bytes = a_parts * a_part_bytes + (uint32_t)KSB * NT * 128;
  int stage = 0; uint32_t phase = 0;
  uint32_t job_i = 0;
  Job j;
  while (sched.next(j, NT)) {
    const uint32_t idesc = idesc_bf16_f32(128, j.nrows);
    const uint32_t buf = job_i & 1u, aph = (job_i >> 1) & 1u;
    if (!mbar_wait(smem_u32(&ctrl->acc_empty[buf]), aph ^ 1u, &ctrl->abort)) return;
    tc_fence_after();
    const uint32_t d = tmem_base + buf * NT;
    uint32_t acc = 0;
    for (int ks = j.kb0; ks < j.kb1; ++ks) {
      if (!mbar_wait(smem_u32(&ctrl->full[stage]), phase, &ctrl->abort)) return;
      tc_fence_after();
      const uint32_t sb = stage_base + (uint32_t)stage * stage_bytes;
#pragma unroll
      for (int i = 0; i < KSB; ++i) {
        const uint32_t wb = sb + a_parts * a_part_bytes + i * NT * 128;
        for (int part = 0; part < a_parts; ++part) {
          const uint32_t ab = sb + part * a_part_bytes + i * a_box_rows * 128;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            umma_bf16(d, smem_desc_sw128(ab + k * 32), smem_desc_sw128(wb + k * 32), idesc, acc);
            acc = 1;
          }
        }
      }
      umma_commit(smem_u32(&ctrl->empty[stage]));          // frees the stage when the MMAs are done
      if (++stage == STAGES) { stage = 0; phase ^= 1u; }
    }
    umma_commit(smem_u32(&ctrl->acc_full[buf]));
    ++job_i;
  }
}

template <int STAGES>
__device__ __forceinline__ void setup_barriers(Ctrl* ctrl) {
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&ctrl->full[s]), 1);
      mbar_init(smem_u32(&ctrl->empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctrl->acc_full[b]), 1);
      mbar_init(smem_u32(&ctrl->acc_empty[b]), 4);
    }
    ctrl->abort = 0;
    mbar_init_fence();
  }
}

// =================================================================================================
// GEMM kernel: weights as the M operand, activation rows (hi | lo) as the N operand
// =================================================================================================
struct GemmJob { int g, arow, wrow, kb0, kb1; };
struct GemmWalk {
  const StreamGemmParams& p;
  long long u, u1;
  __device__ GemmWalk(const StreamGemmParams& pp) : p(pp) {
    const long long U = (long long)p.row_tiles * p.groups * p.tiles_per_group * p.ksteps, G = gridDim.x, c = blockIdx.x;
    u = c * U / G;
    u1 = (c + 1) * U / G;
  }
  __device__ bool next(GemmJob& j) {
    if (u >= u1) return false;
    const long long tile = u / p.ksteps;
    j.kb0 = (int)(u - tile * p.ksteps);
    const long long left = u1 - u;
    j.kb1 = (int)((p.ksteps - j.kb0) < left ? p.ksteps : j.kb0 + left);
    const int per_rt = p.groups * p.tiles_per_group;
    const int rt = (int)(tile / per_rt);
    const int rem = (int)(tile - (long long)rt * per_rt);
    j.g = rem / p.tiles_per_group;
    j.arow = rt * 128;
    j.wrow = (rem - j.g * p.tiles_per_group) * kGemmNT;
    u += j.kb1 - j.kb0;
    return true;
  }
};

__host__ __device__ constexpr uint32_t gemm_tmem_cols(int n_act) {
  return 2 * n_act <= 32 ? 32u : (2 * n_act <= 64 ? 64u : (2 * n_act <= 128 ? 128u : (2 * n_act <= 256 ? 256u : 512u)));
}

// Live packed rows of row tile `arow / 128`, rounded up to 8 (at least 8, at most half a box).
__device__ __forceinline__ int gemm_tile_rows8(const StreamGemmParams& p, int live, int arow) {
  int rows = live - arow;
  rows = rows < 1 ? 1 : rows;
  rows = (rows + 7) & ~7;
  const int cap = p.a_box_rows / 2;
  return rows > cap ? cap : rows;
}

template <int KSB, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
k_stream_gemm(const StreamGemmParams p, const __grid_constant__ CUtensorMap tmA0,
              const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmW0,
              const __grid_constant__ CUtensorMap tmW1) {
  constexpr int NT = kGemmNT;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(sm);
  const uint32_t stage_base = smem_u32(sm + 1024);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t a_bytes = (uint32_t)KSB * p.a_box_rows * 128;
  const uint32_t stage_bytes = a_bytes + (uint32_t)KSB * NT * 128;
  const bool narrow_n = p.row_tiles == 1;          // one row tile: the MMA's N follows the live rows
  pdl_trigger();                                   // the next kernel may get resident behind this one
  setup_barriers<STAGES>(ctrl);
  if (warp == 0 && lane == 0) { prefetch_tmap(&tmA0); prefetch_tmap(&tmW0); if (p.groups > 1) { prefetch_tmap(&tmA1); prefetch_tmap(&tmW1); } }
  __syncthreads();
  if (warp == 2) { tmem_alloc(smem_u32(&ctrl->tmem_base), gemm_tmem_cols(p.a_box_rows)); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctrl->tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      // ---- TMA producer.  The weight tiles depend on no earlier kernel, the activation tiles do:
      // during the first pass over the ring only the weight boxes are issued and the activation
      // boxes are noted; once the ring is full (or the work ends) the producer waits for the
      // preceding kernel and issues them.  With an ordinary launch the wait returns at once.
      const CUtensorMap* amaps[2] = {&tmA0, &tmA1};
      const CUtensorMap* wmaps[2] = {&tmW0, &tmW1};
      const uint64_t pol_w = policy_evict_first(), pol_a = policy_evict_last();
      struct Deferred { uint32_t dst, bar; int map, arow, kb; };
      Deferred def[kMaxStages];
      int n_def = 0, issued = 0;
      bool deps = false, ok = true;
      auto need_deps = [&]() {
        if (deps) return;
        pdl_wait();
        for (int i = 0; i < n_def; ++i)
          tma_load_3d(def[i].dst, amaps[def[i].map], 0, 2 * def[i].arow, def[i].kb, def[i].bar, pol_a);
        deps = true;
      };
      int stage = 0; uint32_t phase = 0;
      GemmWalk walk(p);
      GemmJob j;
      while (ok && walk.next(j)) {
        for (int ks = j.kb0; ks < j.kb1; ++ks) {
          if (issued == STAGES) need_deps();
          if (!mbar_wait(smem_u32(&ctrl->empty[stage]), phase ^ 1u, &ctrl->abort)) { ok = false; break; }
          const uint32_t full = smem_u32(&ctrl->full[stage]);
          mbar_expect_tx(full, stage_bytes);        // rows of a box outside the tensor are zero-filled and counted
          const uint32_t sb = stage_base + (uint32_t)stage * stage_bytes;
          tma_load_3d(sb + a_bytes, wmaps[j.g], 0, j.wrow, ks * KSB, full, pol_w);
          if (deps) tma_load_3d(sb, amaps[j.g], 0, 2 * j.arow, ks * KSB, full, pol_a);
          else { def[n_def].dst = sb; def[n_def].bar = full; def[n_def].map = j.g; def[n_def].arow = j.arow; def[n_def].kb = ks * KSB; ++n_def; }
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      need_deps();
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ---- MMA issue: D[128 weight rows][n] += W tile (M operand) x live activation rows (N operand)
      pdl_wait();                                      // the live-row count comes from an earlier kernel
      const int live = *p.rows_dev;
      int stage = 0; uint32_t phase = 0, job_i = 0;
      bool ok = true;
      GemmWalk walk(p);
      GemmJob j;
      while (ok && walk.next(j)) {
        const uint32_t buf = job_i & 1u, aph = (job_i >> 1) & 1u;
        if (!mbar_wait(smem_u32(&ctrl->acc_empty[buf]), aph ^ 1u, &ctrl->abort)) break;
        tc_fence_after();
        // N covers the live operand rows, which sit at the start of the box (a multiple of 16)
        const int n_rows = narrow_n ? 2 * gemm_tile_rows8(p, live, j.arow) : p.a_box_rows;
        const uint32_t idesc = idesc_bf16_f32(128, n_rows);
        const uint32_t d = tmem_base + buf * (uint32_t)p.a_box_rows;
        uint32_t acc = 0;
        for (int ks = j.kb0; ks < j.kb1; ++ks) {
          if (!mbar_wait(smem_u32(&ctrl->full[stage]), phase, &ctrl->abort)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sb = stage_base + (uint32_t)stage * stage_bytes;
#pragma unroll
          for (int i = 0; i < KSB; ++i) {
            const uint32_t ab = sb + (uint32_t)i * p.a_box_rows * 128;
            const uint32_t wb = sb + a_bytes + (uint32_t)i * NT * 128;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              umma_bf16(d, smem_desc_sw128(wb + k * 32), smem_desc_sw128(ab + k * 32), idesc, acc);
              acc = 1;
            }
          }
          umma_commit(smem_u32(&ctrl->empty[stage]));          // frees the stage when the MMAs are done
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(smem_u32(&ctrl->acc_full[buf]));
        ++job_i;
      }
    }
  } else {
    // ---- epilogue: a thread owns one output feature of the tile (its TMEM lane) and walks the
    // live activation rows (pairs of TMEM columns): hi + lo in registers, one reduction per
    // (row, feature)
    pdl_wait();                                      // the result matrix may still be read by the kernel before
    const int live = *p.rows_dev;
    const int q = warp & 3;                          // TMEM lane quarter this warp may read
    const int feature = q * 32 + lane;
    uint32_t job_i = 0;
    GemmWalk walk(p);
    GemmJob j;
    while (walk.next(j)) {
      const uint32_t buf = job_i & 1u, aph = (job_i >> 1) & 1u;
      if (!mbar_wait(smem_u32(&ctrl->acc_full[buf]), aph, &ctrl->abort)) break;
      tc_fence_after();
      int rows = live - j.arow;                      // live activation rows of this row tile
      rows = rows > 128 ? 128 : rows;
      float* dst = p.out + ((size_t)j.g * p.Rt + j.arow) * p.J + j.wrow + feature;
      const uint32_t t0 = tmem_base + ((uint32_t)(q * 32) << 16) + buf * (uint32_t)p.a_box_rows;
#pragma unroll 1
      for (int r0 = 0; r0 < rows; r0 += 8) {
        uint32_t v[16];
        tmem_ld16(t0 + 2 * r0, v);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 8; ++x)
          if (r0 + x < rows) red_add_f32(dst + (size_t)(r0 + x) * p.J, __uint_as_float(v[2 * x]) + __uint_as_float(v[2 * x + 1]));
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctrl->acc_empty[buf]));
      ++job_i;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && ctrl->abort) atomicOr(p.err, 1);
  if (warp == 2) tmem_dealloc(tmem_base, gemm_tmem_cols(p.a_box_rows));
}

// =================================================================================================
// Logits kernel: fused reductions
// =================================================================================================
template <int NT, int KSB, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
k_stream_logits(const StreamLogitsParams p, const __grid_constant__ LogitMaps tm) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Ctrl* ctrl = reinterpret_cast<Ctrl*>(sm);
  int* s_pref = reinterpret_cast<int*>(sm + 1024);              // [B + 1] <= 4100 bytes
  const uint32_t stage_base = smem_u32(sm + 1024 + 5120);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_wait();                                      // the prologue already reads codebook state
  setup_barriers<STAGES>(ctrl);
  for (int b = threadIdx.x; b < p.cb.B; b += kThreads) s_pref[b + 1] = (p.cb.n[b] + kLogitGran - 1) / kLogitGran;
  if (warp == 0 && lane < 1 + 2 * kLogitBoxClasses) prefetch_tmap(lane == 0 ? &tm.h : &tm.w[lane - 1]);
  __syncthreads();
  if (threadIdx.x == 0) {
    s_pref[0] = 0;
    for (int b = 0; b < p.cb.B; ++b) s_pref[b + 1] += s_pref[b];
    ctrl->vt = (p.cb.V + kLogitGran - 1) / kLogitGran + s_pref[p.cb.B];
    if (blockIdx.x == 0) *p.vt_out = ctrl->vt;
  }
  if (warp == 2) { tmem_alloc(smem_u32(&ctrl->tmem_base), tmem_cols(NT)); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = ctrl->tmem_base;
  const int vt = ctrl->vt;

  if (warp == 0) {
    if (lane == 0) {
      const CUtensorMap* amaps[1] = {&tm.h};
      const CUtensorMap* wmaps[2 * kLogitBoxClasses];
      for (int i = 0; i < 2 * kLogitBoxClasses; ++i) wmaps[i] = &tm.w[i];
      LogitSched sched(p, s_pref, vt, NT);
      producer_role<NT, KSB, STAGES>(sched, ctrl, stage_base, 1, p.a_box_rows, 0, amaps, wmaps);
    }
  } else if (warp == 1) {
    if (lane == 0) {
      LogitSched sched(p, s_pref, vt, NT);
      mma_role<NT, KSB, STAGES>(sched, ctrl, stage_base, 1, p.a_box_rows, tmem_base);
    }
  } else {
    const int q = warp & 3;
    const LogitsArgs& a = p.la;
    LogitSched sched(p, s_pref, vt, NT);
    const long long U = (long long)p.row_tiles * vt, G = gridDim.x;
    const uint32_t k0 = (uint32_t)a.seed, k1 = (uint32_t)(a.seed >> 32);
    const uint32_t c2 = (uint32_t)a.step, c3 = (uint32_t)(a.step >> 32);
    const size_t ldbg = (size_t)p.cb.V + p.cb.cap;
    RowRed red; red.init();
    int cur_rt = -1, r = -1, my_seq = -1, my_nvis = 0, my_tgt = -1;
    uint32_t job_i = 0;
    Job j;
    auto flush = [&]() {
      if (cur_rt >= 0 && r < a.N) {
        const long long first = owner_of((long long)cur_rt * vt, U, G);
        LogitPartial* lp = reinterpret_cast<LogitPartial*>(a.lpart) + (size_t)r * p.part_stride + (blockIdx.x - first);
        lp->m = red.m; lp->s = red.s; lp->idx = red.idx; lp->gm = red.gm; lp->gidx = red.gidx;
      }
    };
    while (sched.next(j, NT)) {
      if (j.rt != cur_rt) {
        flush();
        cur_rt = j.rt; red.init();
        r = cur_rt * 128 + q * 32 + lane;
        my_seq = -1; my_nvis = 0; my_tgt = -1;
        if (r < a.N) {
          my_seq = a.row_seq ? a.row_seq[r] : r;
          if (my_seq < 0 || my_seq >= p.cb.B) my_seq = -1;
          if (my_seq >= 0) {
            my_nvis = p.cb.n[my_seq];
            if (a.row_nvis) { const int x = a.row_nvis[r]; my_nvis = x < my_nvis ? (x < 0 ? 0 : x) : my_nvis; }
          }
          if (a.targets) my_tgt = a.targets[r];
        }
      }
      const uint32_t buf = job_i & 1u, aph = (job_i >> 1) & 1u;
      if (!mbar_wait(smem_u32(&ctrl->acc_full[buf]), aph, &ctrl->abort)) break;
      tc_fence_after();
      int limit = 0;
      if (my_seq >= 0) limit = j.owner < 0 ? j.nvalid : (my_seq == j.owner ? min(j.nvalid, my_nvis - j.k0) : 0);
      const int rows_here = a.N - cur_rt * 128;
      if (q * 32 < rows_here && __any_sync(0xffffffffu, limit > 0)) {
#pragma unroll 1
        for (int c0 = 0; c0 < j.nrows; c0 += 32) {
          if (!__any_sync(0xffffffffu, limit > c0)) break;
          uint32_t v[32];
          tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + buf * NT + c0, v);
          tmem_ld_wait();
          Philox4 px{0, 0, 0, 0};
          int px_blk = -1;
#pragma unroll
          for (int x = 0; x < 32; ++x) {
            if (c0 + x < limit) {
              const float l = __uint_as_float(v[x]);
              const int col = j.col0 + c0 + x;
              red.add(l, col);
              if (a.select == Z2Z_SELECT_GUMBEL) {
                if ((col >> 2) != px_blk) {
                  px_blk = col >> 2;
                  px = philox4x32_10((uint32_t)px_blk, (uint32_t)(a.row_base + r), c2, c3, k0, k1);
                }
                red.add_score(fmaf(l, a.inv_temperature, gumbel_from_word(philox_word(px, col & 3))), col);
              }
              if (a.logits_debug) a.logits_debug[(size_t)r * ldbg + col] = l;
              if (col == my_tgt && a.target_logit) a.target_logit[r] = l;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctrl->acc_empty[buf]));
      ++job_i;
    }
    flush();
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && ctrl->abort) atomicOr(p.err, 1);
  if (warp == 2) tmem_dealloc(tmem_base, tmem_cols(NT));
}

// One warp per row: merge the partial reductions of the CTAs that touched the row's tile.
__global__ void __launch_bounds__(128) k_stream_logits_merge(StreamLogitsParams p, int G) {
  const LogitsArgs& a = p.la;
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= a.N) return;
  const long long vt = *p.vt_out, U = (long long)p.row_tiles * vt;
  const int rt = r >> 7;
  const long long first = owner_of((long long)rt * vt, U, G), last = owner_of((long long)(rt + 1) * vt - 1, U, G);
  const LogitPartial* lp = reinterpret_cast<const LogitPartial*>(a.lpart) + (size_t)r * p.part_stride;
  RowRed red; red.init();
  for (int g = lane; g <= (int)(last - first); g += 32) {
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

__global__ void k_fill_nan_f32(float* p, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = __int_as_float(0x7fc00000);
}

// ---- host helpers ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(f);
  }
  return fn;
}

}  // namespace

// Tensor map over a row-major bf16 matrix [rows, cols]; box = 64 columns x box_rows rows,
// 128-byte swizzle, out-of-range elements read as zero.
bool make_tmap_bf16(CUtensorMap* m, const void* base, long long rows, long long cols, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (cols % 8) || box_rows < 1 || box_rows > 256 || rows < 1) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  cuuint32_t es[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map over the same matrix seen as [cols / 64 k-blocks][rows][64]: one box brings
// `box_kb` k-blocks of `box_rows` rows, laid out k-block after k-block (each k-block is then a
// K-major 128-byte-swizzled operand tile).
//
// A map is a pure function of (base, rows, cols, box): the encoded maps are kept, so that a decode
// step, whose operands sit at the same addresses step after step, encodes none in steady state.
namespace {
struct TmapKey {
  const void* base; long long rows, cols; int box_rows, box_kb;
  bool operator==(const TmapKey& o) const {
    return base == o.base && rows == o.rows && cols == o.cols && box_rows == o.box_rows && box_kb == o.box_kb;
  }
};
struct TmapKeyHash {
  size_t operator()(const TmapKey& k) const {
    size_t h = reinterpret_cast<uintptr_t>(k.base) * 0x9E3779B97F4A7C15ull;
    h ^= (size_t)k.rows * 0xC2B2AE3D27D4EB4Full + (size_t)k.cols * 0x165667B19E3779F9ull;
    h ^= ((size_t)k.box_rows << 20) ^ (size_t)k.box_kb;
    return h;
  }
};
constexpr size_t kTmapCacheMax = 4096;           // entries kept; the cache starts over beyond that
std::unordered_map<TmapKey, CUtensorMap, TmapKeyHash> g_tmap_cache;
std::mutex g_tmap_mu;
}  // namespace

bool make_tmap_bf16_kblocks(CUtensorMap* m, const void* base, long long rows, long long cols, int box_rows,
                            int box_kb) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (cols % 64) || box_rows < 1 || box_rows > 256 || box_kb < 1 ||
      box_kb > 256 || rows < 1)
    return false;
  const TmapKey key{base, rows, cols, box_rows, box_kb};
  {
    std::lock_guard<std::mutex> lock(g_tmap_mu);
    auto it = g_tmap_cache.find(key);
    if (it != g_tmap_cache.end()) { *m = it->second; return true; }
  }
  cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
  cuuint64_t strides[2] = {(cuuint64_t)cols * 2, 128};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_kb};
  cuuint32_t es[3] = {1, 1, 1};
  if (fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return false;
  std::lock_guard<std::mutex> lock(g_tmap_mu);
  if (g_tmap_cache.size() >= kTmapCacheMax) g_tmap_cache.clear();
  g_tmap_cache.emplace(key, *m);
  return true;
}

template <int NT, int KSB>
static int pick_stages(int a_parts, int a_box_rows, int extra) {
  const int stage = a_parts * KSB * a_box_rows * 128 + KSB * NT * 128;
  int s = (227 * 1024 - 2048 - extra - kTailPad) / stage;
  return s > kMaxStages ? kMaxStages : s;
}

// Stages of the GEMM ring that fit beside the control block (every operand row an MMA reads is
// loaded or zero-filled, so no readable padding is needed behind the ring).
int stream_gemm_stages(int ksb, int a_box_rows) {
  const int stage = ksb * a_box_rows * 128 + ksb * kGemmNT * 128;
  const int s = (227 * 1024 - 2048) / stage;
  return s > kMaxStages ? kMaxStages : s;
}

template <int KSB, int STAGES>
static cudaError_t launch_gemm_t(const StreamGemmParams& p, const CUtensorMap* maps, int grid, cudaStream_t s) {
  const size_t stage = (size_t)KSB * p.a_box_rows * 128 + (size_t)KSB * kGemmNT * 128;
  const size_t smem = 1024 + 1024 + STAGES * stage;
  auto kern = k_stream_gemm<KSB, STAGES>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(kern, dim3(grid), dim3(kThreads), smem, s, p, maps[0], maps[1], maps[2], maps[3]);
}

// Launches the stream-K GEMM.  maps = {A group 0, A group 1, W group 0, W group 1}, built for
// p.ksb k-blocks per box.
template <int KSB>
static cudaError_t launch_stream_gemm_k(const StreamGemmParams& p, const CUtensorMap* maps, int grid, cudaStream_t s) {
  const int st = stream_gemm_stages(KSB, p.a_box_rows);
  if (st >= 8) return launch_gemm_t<KSB, 8>(p, maps, grid, s);
  if (st >= 6) return launch_gemm_t<KSB, 6>(p, maps, grid, s);
  if (st >= 5) return launch_gemm_t<KSB, 5>(p, maps, grid, s);
  if (st >= 4) return launch_gemm_t<KSB, 4>(p, maps, grid, s);
  if (st >= 3) return launch_gemm_t<KSB, 3>(p, maps, grid, s);
  return cudaErrorInvalidConfiguration;
}
cudaError_t launch_stream_gemm(const StreamGemmParams& p, const CUtensorMap* maps, int grid, cudaStream_t s) {
  if (!p.out || !p.err || !p.rows_dev || p.a_box_rows % 16 || p.a_box_rows < 16 || p.a_box_rows > 256 ||
      (p.row_tiles > 1 && p.a_box_rows != 256))
    return cudaErrorInvalidValue;
  if (p.ksb == 2) return launch_stream_gemm_k<2>(p, maps, grid, s);
  if (p.ksb == 1) return launch_stream_gemm_k<1>(p, maps, grid, s);
  return cudaErrorInvalidValue;
}

template <int NT, int KSB, int STAGES>
static cudaError_t launch_logits_t(const StreamLogitsParams& p, const LogitMaps* maps, int grid, cudaStream_t s) {
  const size_t stage = (size_t)KSB * p.a_box_rows * 128 + (size_t)KSB * NT * 128;
  const size_t smem = 1024 + 1024 + 5120 + STAGES * stage + kTailPad;
  auto kern = k_stream_logits<NT, KSB, STAGES>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<grid, kThreads, smem, s>>>(p, *maps);
  return cudaGetLastError();
}

bool logits_tc_supported(int d, int dtype) { return dtype == Z2Z_DTYPE_BF16 && d % 64 == 0; }

cudaError_t run_logits_tc(const CbView& cb, const LogitsArgs& a, int* vt_word, int* err_word,
                          LogitsPartInfo* info, Prof* prof, cudaStream_t s) {
  if (decode_logits_applies(a)) return run_logits_decode(cb, a, vt_word + 1, err_word, info, prof, s);
  static int n_sm = 0;
  if (!n_sm) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (n_sm <= 0) n_sm = 148;
  }
  StreamLogitsParams p{};
  p.cb = cb; p.la = a;
  p.ksteps = (a.d / 64 + kLogitKSB - 1) / kLogitKSB;
  p.row_tiles = (a.N + 127) / 128;
  p.a_box_rows = a.N >= 128 ? 128 : (a.N + 7) / 8 * 8;
  p.part_stride = (n_sm + p.row_tiles - 1) / p.row_tiles + 2;
  p.vt_out = vt_word; p.err = err_word;
  if ((size_t)a.N * p.part_stride * sizeof(LogitPartial) > a.lpart_bytes) return cudaErrorMemoryAllocation;
  LogitMaps maps;
  if (!make_tmap_bf16_kblocks(&maps.h, a.hidden, a.N, a.d, p.a_box_rows, kLogitKSB)) return cudaErrorInvalidValue;
  for (int c = 0; c < kLogitBoxClasses; ++c) {
    if (!make_tmap_bf16_kblocks(&maps.w[c], a.WU, cb.V, a.d, kLogitGran << c, kLogitKSB)) return cudaErrorInvalidValue;
    if (cb.cap > 0) {
      if (!make_tmap_bf16_kblocks(&maps.w[kLogitBoxClasses + c], a.Uh, (long long)cb.B * cb.cap, a.d, kLogitGran << c, kLogitKSB))
        return cudaErrorInvalidValue;
    } else {
      maps.w[kLogitBoxClasses + c] = maps.w[c];
    }
  }
  // every CTA must own at least one unit: the static tiles alone give a lower bound on the units
  long long units_lb = (long long)p.row_tiles * ((cb.V + kLogitGran - 1) / kLogitGran);
  const int grid = units_lb < n_sm ? (int)units_lb : n_sm;
  p.part_stride = (grid + p.row_tiles - 1) / p.row_tiles + 2;
  if (info) {
    if (p.row_tiles != 1) return cudaErrorInvalidValue;
    info->stride = p.part_stride; info->count = grid;
  }
  return launch_stream_logits(p, &maps, grid, info == nullptr, prof, s);
}

cudaError_t launch_stream_logits(const StreamLogitsParams& p, const LogitMaps* maps, int grid, bool merge,
                                 Prof* prof, cudaStream_t s) {
  constexpr int NT = kLogitNT, KSB = kLogitKSB;
  const LogitsArgs& a = p.la;
  if (a.target_logit) {
    ProfScope ps(prof, kProfLogitsMerge, 1, s);
    k_fill_nan_f32<<<(a.N + 255) / 256, 256, 0, s>>>(a.target_logit, a.N);
  }
  cudaError_t e;
  {
    ProfScope ps(prof, kProfLogits, 1, s);
    const int st = pick_stages<NT, KSB>(1, p.a_box_rows, 5120);
    if (st >= 8) e = launch_logits_t<NT, KSB, 8>(p, maps, grid, s);
    else if (st >= 6) e = launch_logits_t<NT, KSB, 6>(p, maps, grid, s);
    else if (st >= 4) e = launch_logits_t<NT, KSB, 4>(p, maps, grid, s);
    else e = cudaErrorInvalidConfiguration;
  }
  if (e != cudaSuccess || !merge) return e;
  ProfScope ps(prof, kProfLogitsMerge, 1, s);
  k_stream_logits_merge<<<(a.N + 3) / 4, 128, 0, s>>>(p, grid);
  return cudaGetLastError();
}

}  // namespace z2z
