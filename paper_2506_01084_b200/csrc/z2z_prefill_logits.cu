// Joint logits with fused reductions for MANY hidden rows (prompt scoring; paper Section 2.3
// steps 7-9 applied at every compressed position).  This is a dense contraction
//     [N rows] x [V + n_b columns] x d
// and runs on the tcgen05 tensor cores with CTA pairs:
//
//   * a cluster of two CTAs owns a tile of 256 hidden rows x 256 vocabulary columns;
//     `tcgen05.mma.cta_group::2` (M = 256, N = 256, K = 16) reads 128 rows of the hidden tile
//     and 128 rows of the weight tile from EACH CTA's shared memory, so every CTA loads only its
//     own halves (plain TMA loads, no multicast) and the operand traffic per flop is halved;
//   * fp32 accumulators live in tensor memory, 128 lanes x 256 columns per CTA, double
//     buffered: while the pair's tensor cores work on column tile j + 1, the four epilogue
//     warps of each CTA fold tile j into a running (max, sum-exp, argmax) per hidden row, one
//     thread per row, so no logit is ever written;
//   * work unit = (row tile, column strip): the pair sweeps the strip's column tiles (static
//     vocabulary first, then the visible hypertokens of the sequences present in the row tile)
//     with the running reduction in registers.  Units are dealt round-robin to the clusters, so
//     that neighbouring clusters read the same weight tiles at about the same time (L2 reuse).
//
// Roles per CTA: warp 0 lane 0 TMA producer, warp 1 lane 0 MMA issuer (leader CTA only),
// warps 2-5 epilogue.  Every mbarrier wait is bounded; on a timeout the CTA raises an abort flag,
// all roles leave their loops, tensor memory is released and an error word is set.
#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_sm100.cuh"
#include "z2z_stream.h"

namespace z2z {
using namespace sm100;

namespace {

constexpr int kThreads = 192;
constexpr int kTileRows = 256;           // hidden rows per cluster tile (128 per CTA)
constexpr int kTileCols = 256;           // vocabulary columns per tile (128 weight rows loaded per CTA)
constexpr int kStages = 6;               // 32 KB per stage and CTA: A 128 x 64 bf16, B 128 x 64 bf16
constexpr uint32_t kStageBytes = 32768;
constexpr float kLog2e = 1.4426950408889634f;

struct PCtrl {
  unsigned long long full[kStages], empty[kStages], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort;
};

// ---- schedule --------------------------------------------------------------------------------------
// Column tiles of a row tile: v in [0, n_static) are tiles of W_U; then for each sequence b in
// [lo, hi] (the sequences that own rows of the tile) ceil(n_b / 256) tiles of U_h[b].
struct TileRef { int wmap; int wrow; int col0; int owner; int k0; int nvalid; };

struct UnitWalk {
  const PrefillLogitsParams& p;
  int rt, lo, hi, v, v1;        // row tile, sequence range, current / end virtual tile
  int b, tb, acc;               // hyper walk: sequence, tile inside it, virtual index of its tile 0
  __device__ UnitWalk(const PrefillLogitsParams& pp) : p(pp) {}
  __device__ void begin(long long unit) {
    rt = (int)(unit / p.strips);
    const int strip = (int)(unit - (long long)rt * p.strips);
    lo = p.tile_lo[rt]; hi = p.tile_hi[rt];
    const int vt = p.n_static + p.tile_nh[rt];
    v = (int)((long long)strip * vt / p.strips);
    v1 = (int)((long long)(strip + 1) * vt / p.strips);
    b = lo; tb = 0; acc = p.n_static;
    if (v > p.n_static) {                       // position the hyper walk on v
      while (b <= hi) {
        const int nt = (p.cb.n[b] + kTileCols - 1) / kTileCols;
        if (v < acc + nt) { tb = v - acc; break; }
        acc += nt; ++b;
      }
    }
  }
  __device__ bool next(TileRef& t) {
    if (v >= v1) return false;
    if (v < p.n_static) {
      t.wmap = 0; t.wrow = v * kTileCols; t.col0 = t.wrow; t.owner = -1; t.k0 = 0;
      t.nvalid = p.cb.V - t.col0 < kTileCols ? p.cb.V - t.col0 : kTileCols;
    } else {
      int nb = p.cb.n[b];
      while (tb * kTileCols >= nb && b < hi) { ++b; tb = 0; nb = p.cb.n[b]; }   // stays within [lo, hi]
      t.wmap = 1; t.owner = b; t.k0 = tb * kTileCols;
      t.wrow = b * p.cb.cap + t.k0; t.col0 = p.cb.V + t.k0;
      t.nvalid = nb - t.k0 < kTileCols ? nb - t.k0 : kTileCols;
      ++tb;
    }
    ++v;
    return true;
  }
};

// ---- plan: sequence range and hypertoken tiles of every row tile -----------------------------------
__global__ void __launch_bounds__(256) k_prefill_plan(PrefillLogitsParams p) {
  __shared__ int s_lo, s_hi;
  const int rt = blockIdx.x;
  if (threadIdx.x == 0) { s_lo = 0x7fffffff; s_hi = -1; }
  __syncthreads();
  const int r = rt * kTileRows + threadIdx.x;
  if (r < p.la.N) {
    int sq = p.la.row_seq ? p.la.row_seq[r] : r;
    if (sq >= 0 && sq < p.cb.B) { atomicMin(&s_lo, sq); atomicMax(&s_hi, sq); }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int nh = 0;
    for (int b = s_lo; b <= s_hi; ++b) nh += (p.cb.n[b] + kTileCols - 1) / kTileCols;
    p.tile_lo[rt] = s_lo; p.tile_hi[rt] = s_hi; p.tile_nh[rt] = nh;
  }
}

// ---- epilogue helpers ----------------------------------------------------------------------------------
// 32 consecutive columns, all visible: running max / sum-exp / argmax of one hidden row.
__device__ __forceinline__ void fold32(const uint32_t (&v)[32], int col, float& m, float& s, int& idx) {
  float cm = __uint_as_float(v[0]);
#pragma unroll
  for (int x = 1; x < 32; ++x) cm = fmaxf(cm, __uint_as_float(v[x]));
  if (cm > m) {                                   // a new maximum: its first occurrence wins ties
    int at = 31;
#pragma unroll
    for (int x = 30; x >= 0; --x) at = __uint_as_float(v[x]) == cm ? x : at;
    idx = col + at;
    s *= exp2f((m - cm) * kLog2e);
    m = cm;
  }
  const float ms = m * kLog2e;
  float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
  for (int x = 0; x < 32; x += 4) {
    a0 += exp2f(fmaf(__uint_as_float(v[x]), kLog2e, -ms));
    a1 += exp2f(fmaf(__uint_as_float(v[x + 1]), kLog2e, -ms));
    a2 += exp2f(fmaf(__uint_as_float(v[x + 2]), kLog2e, -ms));
    a3 += exp2f(fmaf(__uint_as_float(v[x + 3]), kLog2e, -ms));
  }
  s += (a0 + a1) + (a2 + a3);
}

// =================================================================================================
template <bool GENERIC>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
k_prefill_logits(const PrefillLogitsParams p, const __grid_constant__ CUtensorMap tmH,
                 const __grid_constant__ CUtensorMap tmWU, const __grid_constant__ CUtensorMap tmUh) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  PCtrl* ctrl = reinterpret_cast<PCtrl*>(sm);
  const uint32_t stage_base = smem_u32(sm + 1024);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0: leader (issues the MMAs), 1: peer
  const long long n_clusters = gridDim.x >> 1, cluster_id = blockIdx.x >> 1;
  const long long n_units = (long long)p.row_tiles * p.strips;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&ctrl->full[s]), 1);        // leader: its producer's arrive + bytes of both CTAs
      mbar_init(smem_u32(&ctrl->empty[s]), 1);       // one multicast commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctrl->acc_full[b]), 1);    // one multicast commit
      mbar_init(smem_u32(&ctrl->acc_empty[b]), 8);   // leader: 4 epilogue warps of each CTA
    }
    ctrl->abort = 0;
    mbar_init_fence();
    prefetch_tmap(&tmH); prefetch_tmap(&tmWU); prefetch_tmap(&tmUh);
  }
  __syncthreads();
  if (warp == 2) { tmem_alloc_pair(smem_u32(&ctrl->tmem_base), 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                               // both CTAs' barriers exist before any remote signal
  tc_fence_after();
  const uint32_t tmem_base = ctrl->tmem_base;

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer (both CTAs): own 128 hidden rows, own 128 weight rows ----------
      const uint64_t pol_w = policy_evict_last(), pol_a = policy_evict_last();
      uint32_t full_leader[kStages];
      for (int s = 0; s < kStages; ++s) full_leader[s] = map_to_cta(smem_u32(&ctrl->full[s]), 0);
      UnitWalk w(p);
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (long long u = cluster_id; u < n_units && ok; u += n_clusters) {
        w.begin(u);
        const int arow = w.rt * kTileRows + (int)rank * 128;
        TileRef t;
        while (ok && w.next(t)) {
          const CUtensorMap* wm = t.wmap ? &tmUh : &tmWU;
          const int wrow = t.wrow + (int)rank * 128;
          for (int ks = 0; ks < p.ksteps; ++ks) {
            if (!mbar_wait(smem_u32(&ctrl->empty[stage]), phase ^ 1u, &ctrl->abort)) { ok = false; break; }
            if (rank == 0) mbar_expect_tx(smem_u32(&ctrl->full[stage]), 2 * kStageBytes);
            const uint32_t sb = stage_base + (uint32_t)stage * kStageBytes;
            tma_load_2d_pair(sb, &tmH, ks * 64, arow, full_leader[stage], pol_a);
            tma_load_2d_pair(sb + 16384, wm, ks * 64, wrow, full_leader[stage], pol_w);
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ---------------- MMA issuer (leader only) ------------------------------------------------------
      const uint32_t idesc = idesc_bf16_f32(kTileRows, kTileCols);
      UnitWalk w(p);
      int stage = 0; uint32_t phase = 0, job_i = 0;
      bool ok = true;
      for (long long u = cluster_id; u < n_units && ok; u += n_clusters) {
        w.begin(u);
        TileRef t;
        while (ok && w.next(t)) {
          const uint32_t buf = job_i & 1u, aph = (job_i >> 1) & 1u;
          if (!mbar_wait(smem_u32(&ctrl->acc_empty[buf]), aph ^ 1u, &ctrl->abort)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d = tmem_base + buf * kTileCols;
          uint32_t acc = 0;
          for (int ks = 0; ks < p.ksteps; ++ks) {
            if (!mbar_wait(smem_u32(&ctrl->full[stage]), phase, &ctrl->abort)) { ok = false; break; }
            tc_fence_after();
            const uint32_t sb = stage_base + (uint32_t)stage * kStageBytes;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              umma_bf16_pair(d, smem_desc_sw128(sb + k * 32), smem_desc_sw128(sb + 16384 + k * 32), idesc, acc);
              acc = 1;
            }
            umma_commit_pair(smem_u32(&ctrl->empty[stage]));      // frees the stage in both CTAs
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          umma_commit_pair(smem_u32(&ctrl->acc_full[buf]));       // wakes the epilogues of both CTAs
          ++job_i;
        }
      }
    }
  } else {
    // ---------------- epilogue (both CTAs): thread = hidden row ------------------------------------------
    const int q = warp & 3;                           // tensor-memory lane quarter this warp may read
    const LogitsArgs& a = p.la;
    const uint32_t k0s = (uint32_t)a.seed, k1s = (uint32_t)(a.seed >> 32);
    const uint32_t c2 = (uint32_t)a.step, c3 = (uint32_t)(a.step >> 32);
    const size_t ldbg = (size_t)p.cb.V + p.cb.cap;
    uint32_t acc_empty_leader[2];
    acc_empty_leader[0] = map_to_cta(smem_u32(&ctrl->acc_empty[0]), 0);
    acc_empty_leader[1] = map_to_cta(smem_u32(&ctrl->acc_empty[1]), 0);
    UnitWalk w(p);
    uint32_t job_i = 0;
    bool ok = true;
    for (long long u = cluster_id; u < n_units && ok; u += n_clusters) {
      w.begin(u);
      const int strip = (int)(u - (long long)w.rt * p.strips);
      const int r = w.rt * kTileRows + (int)rank * 128 + q * 32 + lane;
      int my_seq = -1, my_nvis = 0, my_tgt = -1;
      if (r < a.N) {
        my_seq = a.row_seq ? a.row_seq[r] : r;
        if (my_seq < 0 || my_seq >= p.cb.B) my_seq = -1;
        if (my_seq >= 0) {
          my_nvis = p.cb.n[my_seq];
          if (a.row_nvis) { const int x = a.row_nvis[r]; my_nvis = x < my_nvis ? (x < 0 ? 0 : x) : my_nvis; }
        }
        if (a.targets) my_tgt = a.targets[r];
      }
      RowRed red; red.init();
      TileRef t;
      while (w.next(t)) {
        const uint32_t buf = job_i & 1u, aph = (job_i >> 1) & 1u;
        if (!mbar_wait(smem_u32(&ctrl->acc_full[buf]), aph, &ctrl->abort)) { ok = false; break; }
        tc_fence_after();
        int limit = 0;
        if (my_seq >= 0) limit = t.owner < 0 ? t.nvalid : (my_seq == t.owner ? min(t.nvalid, my_nvis - t.k0) : 0);
        const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kTileCols;
        if (!GENERIC && __all_sync(0xffffffffu, limit == kTileCols)) {
#pragma unroll 1
          for (int c0 = 0; c0 < kTileCols; c0 += 32) {
            uint32_t v[32];
            tmem_ld32(tbase + c0, v);
            tmem_ld_wait();
            fold32(v, t.col0 + c0, red.m, red.s, red.idx);
          }
        } else if (__any_sync(0xffffffffu, limit > 0)) {
#pragma unroll 1
          for (int c0 = 0; c0 < kTileCols; c0 += 32) {
            if (!__any_sync(0xffffffffu, limit > c0)) break;
            uint32_t v[32];
            tmem_ld32(tbase + c0, v);
            tmem_ld_wait();
            Philox4 px{0, 0, 0, 0};
            int px_blk = -1;
#pragma unroll
            for (int x = 0; x < 32; ++x) {
              if (c0 + x < limit) {
                const float l = __uint_as_float(v[x]);
                const int col = t.col0 + c0 + x;
                red.add(l, col);
                if (GENERIC) {
                  if (a.select == Z2Z_SELECT_GUMBEL) {
                    if ((col >> 2) != px_blk) {
                      px_blk = col >> 2;
                      px = philox4x32_10((uint32_t)px_blk, (uint32_t)(a.row_base + r), c2, c3, k0s, k1s);
                    }
                    red.add_score(fmaf(l, a.inv_temperature, gumbel_from_word(philox_word(px, col & 3))), col);
                  }
                  if (a.logits_debug) a.logits_debug[(size_t)r * ldbg + col] = l;
                  if (col == my_tgt && a.target_logit) a.target_logit[r] = l;
                }
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(acc_empty_leader[buf]);
        ++job_i;
      }
      if (ok && r < a.N) {
        LogitPartial* lp = reinterpret_cast<LogitPartial*>(a.lpart) + (size_t)r * p.strips + strip;
        lp->m = red.m; lp->s = red.s; lp->idx = red.idx; lp->gm = red.gm; lp->gidx = red.gidx;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && ctrl->abort) atomicOr(p.err, 1);
  cluster_sync_all();                               // nobody leaves while the pair's MMAs may read its memory
  if (warp == 2) tmem_dealloc_pair(tmem_base, 512);
}

// One thread per row: merge the `strips` partial reductions, write the outputs.
__global__ void __launch_bounds__(256) k_prefill_merge(PrefillLogitsParams p) {
  const LogitsArgs& a = p.la;
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= a.N) return;
  const LogitPartial* lp = reinterpret_cast<const LogitPartial*>(a.lpart) + (size_t)r * p.strips;
  RowRed red; red.init();
  for (int g = 0; g < p.strips; ++g) {
    RowRed o; o.m = lp[g].m; o.s = lp[g].s; o.idx = lp[g].idx; o.gm = lp[g].gm; o.gidx = lp[g].gidx;
    red.merge(o);
  }
  if (a.lse) a.lse[r] = red.m + logf(red.s);
  if (a.argmax) a.argmax[r] = red.idx == 0x7fffffff ? -1 : red.idx;
  if (a.max_logit) a.max_logit[r] = red.m;
  if (a.sample) a.sample[r] = red.gidx == 0x7fffffff ? -1 : red.gidx;
}

__global__ void k_fill_nan_rows(float* p, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = __int_as_float(0x7fc00000);
}

}  // namespace

bool prefill_logits_supported(int d, int dtype) { return dtype == Z2Z_DTYPE_BF16 && d % 64 == 0; }

long long prefill_logits_max_rows(size_t lpart_bytes, size_t plan_bytes, int strips) {
  long long by_part = (long long)(lpart_bytes / sizeof(LogitPartial)) / (strips < 1 ? 1 : strips);
  long long by_plan = (long long)(plan_bytes / (3 * sizeof(int32_t))) * kTileRows;
  long long m = by_part < by_plan ? by_part : by_plan;
  return m / kTileRows * kTileRows;
}

static int sm_count_prefill() {
  static int n_sm = 0;
  if (!n_sm) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (n_sm <= 0) n_sm = 148;
  }
  return n_sm;
}

static size_t l2_bytes_prefill() {
  static size_t l2 = 0;
  if (!l2) {
    int dev = 0, v = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&v, cudaDevAttrL2CacheSize, dev);
    l2 = v > 0 ? (size_t)v : ((size_t)64 << 20);
  }
  return l2;
}

// Number of column strips per row tile.  Two conditions:
//   * the hidden-row tiles that are in work at the same time must stay in the L2 cache, because a
//     pair re-reads its 256 x d tile for every column tile of its strip: n_clusters / strips tiles
//     of 512 d bytes within a third of the cache (with one strip at d = 4096 the 74 pairs keep
//     148 MB of tiles in work, more than the cache holds, and every column tile fetches its
//     hidden rows from HBM again: 0.92 instead of 1.15 PFLOP/s at 1.8e5 rows);
//   * the clusters should be busy in the last round too (at least 90 %).
// The smallest split that meets both, at most kPrefillMaxStrips.
static int pick_strips(int row_tiles, int n_clusters, int d) {
  const size_t tile_bytes = (size_t)kTileRows * d * 2;
  const size_t budget = l2_bytes_prefill() / 3;
  int s_min = (int)(((size_t)n_clusters * tile_bytes + budget - 1) / budget);
  if (row_tiles < n_clusters) s_min = (int)(((size_t)row_tiles * tile_bytes + budget - 1) / budget);
  s_min = s_min < 1 ? 1 : (s_min > kPrefillMaxStrips ? kPrefillMaxStrips : s_min);
  int best = s_min; double best_eff = 0.0;
  for (int s = s_min; s <= kPrefillMaxStrips; ++s) {
    const long long units = (long long)row_tiles * s;
    const long long rounds = (units + n_clusters - 1) / n_clusters;
    const double eff = (double)units / (double)(rounds * n_clusters);
    if (eff >= 0.9) return s;
    if (eff > best_eff + 1e-9) { best_eff = eff; best = s; }
  }
  return best;
}

int prefill_logits_strips(int N, int d) {
  return pick_strips((N + kTileRows - 1) / kTileRows, sm_count_prefill() / 2, d);
}

cudaError_t run_logits_prefill(const CbView& cb, const LogitsArgs& a, int32_t* plan, int* err_word, int strips_override,
                               Prof* prof, cudaStream_t s) {
  const int n_sm = sm_count_prefill();
  PrefillLogitsParams p{};
  p.cb = cb; p.la = a;
  p.ksteps = a.d / 64;
  p.row_tiles = (a.N + kTileRows - 1) / kTileRows;
  p.n_static = (cb.V + kTileCols - 1) / kTileCols;
  const int max_clusters = n_sm / 2;
  p.strips = strips_override > 0 ? strips_override : pick_strips(p.row_tiles, max_clusters, a.d);
  if (p.strips > kPrefillMaxStrips) p.strips = kPrefillMaxStrips;
  if (p.strips > p.n_static) p.strips = p.n_static;          // every strip gets at least one tile
  p.tile_lo = plan; p.tile_hi = plan + p.row_tiles; p.tile_nh = plan + 2 * p.row_tiles;
  p.err = err_word;
  if ((size_t)a.N * p.strips * sizeof(LogitPartial) > a.lpart_bytes) return cudaErrorMemoryAllocation;
  CUtensorMap mH, mW, mU;
  if (!make_tmap_bf16(&mH, a.hidden, a.N, a.d, 128)) return cudaErrorInvalidValue;
  if (!make_tmap_bf16(&mW, a.WU, cb.V, a.d, 128)) return cudaErrorInvalidValue;
  if (cb.cap > 0) {
    if (!make_tmap_bf16(&mU, a.Uh, (long long)cb.B * cb.cap, a.d, 128)) return cudaErrorInvalidValue;
  } else {
    mU = mW;
  }
  const long long units = (long long)p.row_tiles * p.strips;
  const int clusters = units < max_clusters ? (int)units : max_clusters;
  const bool generic = a.select == Z2Z_SELECT_GUMBEL || a.logits_debug || a.target_logit;
  {
    ProfScope ps(prof, kProfLogitsMerge, a.target_logit ? 2 : 1, s);
    if (a.target_logit) k_fill_nan_rows<<<(a.N + 255) / 256, 256, 0, s>>>(a.target_logit, a.N);
    k_prefill_plan<<<p.row_tiles, kTileRows, 0, s>>>(p);
  }
  {
    ProfScope ps(prof, kProfLogits, 1, s);
    const size_t smem = 1024 + 1024 + (size_t)kStages * kStageBytes;
    auto kern = generic ? k_prefill_logits<true> : k_prefill_logits<false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<2 * clusters, kThreads, smem, s>>>(p, mH, mW, mU);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  ProfScope ps(prof, kProfLogitsMerge, 1, s);
  k_prefill_merge<<<(a.N + 255) / 256, 256, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace z2z
