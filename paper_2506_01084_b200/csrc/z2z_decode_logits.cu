// Joint logits with fused reductions for a DECODE batch (at most 32 hidden rows; paper Section
// 2.3 steps 7-9).  The step is bound by streaming W_U and the visible rows of every sequence's
// U_h from HBM exactly once, so the kernel is built around the load ring:
//
//   * operands swapped: the weight rows are the 128-row M operand of tcgen05.mma and the batch
//     is its narrow N operand, so an accumulator lane is one VOCABULARY row.  Each of the 128
//     epilogue threads owns one column of the joint logits per job and keeps a running
//     (max, sum-exp, argmax[, best perturbed score]) per hidden row in registers; the threads'
//     reductions are merged once, when the CTA has streamed its share.
//   * every stage of the ring is ONE TMA box of 16 KB: 128 weight rows x 1 k-block (64 columns)
//     or 64 rows x 2 k-blocks (a 3-D tensor map [k-block][row][64]).  The TMA unit's cost is per
//     box, not per byte, so small boxes would cap the stream far below the HBM rate; and since an
//     MMA always spans 128 rows, jobs of fewer than 64 rows would cost more tensor-pipe time per
//     stage than the stage's bytes take to arrive.
//   * the hidden rows are loaded into shared memory once when they fit (RESIDENT), else one box
//     per stage.
//   * work: every CTA first streams a fixed share of W_U in 128-row jobs (known without reading
//     any codebook state, so the first loads are issued right after barrier set-up); the rest
//     of W_U and all U_h rows form a pool of 64-row units that the CTAs claim with an atomic
//     counter, which evens out the differences in streaming speed between SMs.
//
// Roles: warp 0 lane 0 producer (claims work, publishes each job in a shared-memory ring, issues
// TMA), warp 1 lane 0 MMA issuer, warps 2-5 epilogue.  Every wait is bounded; on a timeout the
// CTA raises an abort flag, all roles leave, tensor memory is freed, an error word is set.
#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_sm100.cuh"
#include "z2z_stream.h"

namespace z2z {
using namespace sm100;

namespace {

// Threads per CTA: producer warp, MMA warp, then the epilogue warps.  Up to 16 hidden rows one
// epilogue thread keeps the reductions of every row of its vocabulary row in registers (4 warps, one
// per tensor-memory lane quarter); 17-32 rows are split between two warps per quarter, 16 rows each.
__host__ __device__ constexpr int decode_epi_warps(int nb) { return nb > 16 ? 8 : 4; }
__host__ __device__ constexpr int decode_threads(int nb) { return 64 + 32 * decode_epi_warps(nb); }
constexpr int kGran = 64;                // pool unit / scheduling granule, in weight rows
constexpr int kJobRing = 32;             // published jobs kept (> stages + accumulators in flight)
constexpr int kDecodeMaxStages = 12;
constexpr int kTailPadBytes = 16384;     // readable shared memory behind the last stage

struct DecodeJob {
  int cls;               // 2: 128 rows x 1 k-block per stage, 1: 64 rows x 2 k-blocks, -1: no more work
  int wmap, wrow;        // tensor (0: W_U, 1: U_h) and first row in it
  int col0, nvalid;      // first column id of the joint logits, rows that exist
  int owner, k0;         // U_h: owning sequence and first entry number; W_U: -1, 0
  int pad;
};

struct DecodeCtrl {
  unsigned long long full[kDecodeMaxStages], empty[kDecodeMaxStages], acc_full[2], acc_empty[2];
  unsigned long long job_ready[kJobRing];
  unsigned long long hid_full, pref_ready;
  uint32_t tmem_base;
  int abort;
};

struct DecodeSmem {
  int seq[32], nvis[32], tgt[32];
  RowRed part[4][32];
  DecodeJob jobs[kJobRing];
};

__host__ __device__ constexpr int decode_tmem_cols(int nbp) { return 2 * nbp <= 32 ? 32 : 64; }

template <int NB> struct TmemRow;
template <> struct TmemRow<8> { static __device__ __forceinline__ void ld(uint32_t a, uint32_t (&v)[8]) { tmem_ld8(a, v); } };
template <> struct TmemRow<16> { static __device__ __forceinline__ void ld(uint32_t a, uint32_t (&v)[16]) { tmem_ld16(a, v); } };
template <> struct TmemRow<32> { static __device__ __forceinline__ void ld(uint32_t a, uint32_t (&v)[32]) { tmem_ld32(a, v); } };

// Order-preserving map float -> int, so that a warp-wide integer max finds the float max.
__device__ __forceinline__ int float_key(float x) {
  const int b = __float_as_int(x);
  return b ^ ((b >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float key_float(int k) { return __int_as_float(k ^ ((k >> 31) & 0x7fffffff)); }

// Pool unit u -> job.  Units [0, pool_static) are the W_U granules behind the fixed shares, the
// following ones the granules of U_h, sequence after sequence (pref = prefix of granule counts).
__device__ __forceinline__ bool pool_job(const DecodeLogitsParams& p, const int* pref, int pool_static,
                                         int pool_total, int u, DecodeJob& j) {
  if (u >= pool_total) return false;
  j.cls = 1; j.pad = 0;
  if (u < pool_static) {
    const int g = p.fixed_granules * (int)gridDim.x + u;
    j.wmap = 0; j.wrow = g * kGran; j.col0 = j.wrow; j.owner = -1; j.k0 = 0;
    j.nvalid = p.cb.V - j.wrow < kGran ? p.cb.V - j.wrow : kGran;
    return true;
  }
  const int h = u - pool_static;
  int lo = 0, hi = p.cb.B - 1;                     // last b with pref[b] <= h
  while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (pref[mid] <= h) lo = mid; else hi = mid - 1; }
  j.owner = lo; j.k0 = (h - pref[lo]) * kGran;
  j.wmap = 1; j.wrow = lo * p.cb.cap + j.k0; j.col0 = p.cb.V + j.k0;
  const int left = p.cb.n[lo] - j.k0;
  j.nvalid = left < kGran ? left : kGran;
  return true;
}

template <int NB, bool GENERIC, bool RESIDENT>
__global__ void __launch_bounds__(decode_threads(NB), 1)
k_decode_logits(const DecodeLogitsParams p, const __grid_constant__ DecodeLogitMaps tm) {
  constexpr int NT = 128;
  constexpr int NBP = NB < 16 ? 16 : NB;            // the MMA's N (a multiple of 16 for M = 128)
  constexpr int EW = decode_epi_warps(NB);          // epilogue warps
  constexpr int RW = NB > 16 ? 16 : NB;             // hidden rows one epilogue thread reduces
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  DecodeCtrl* ctrl = reinterpret_cast<DecodeCtrl*>(sm);
  DecodeSmem* ds = reinterpret_cast<DecodeSmem*>(sm + 1024);       // < 4 KB
  int* s_pref = reinterpret_cast<int*>(sm + 5120);                  // [B + 1] <= 4100 bytes
  const uint32_t hid_base = smem_u32(sm + 10240);                   // resident hidden rows, if any
  const int hid_rows = p.hid_rows;
  const uint32_t hid_bytes = RESIDENT ? (uint32_t)p.ksteps * hid_rows * 128 : 0u;
  const uint32_t stage_base = hid_base + ((hid_bytes + 1023u) & ~1023u);
  const uint32_t stage_hid = RESIDENT ? 0u : (uint32_t)((2 * hid_rows * 128 + 1023) & ~1023);
  const uint32_t stage_bytes = NT * 128 + stage_hid;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const LogitsArgs& a = p.la;
  const int STAGES = p.stages;
  if (threadIdx.x == 0) {
    for (int st = 0; st < STAGES; ++st) {
      mbar_init(smem_u32(&ctrl->full[st]), 1);
      mbar_init(smem_u32(&ctrl->empty[st]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctrl->acc_full[b]), 1);
      mbar_init(smem_u32(&ctrl->acc_empty[b]), EW);
    }
    for (int i = 0; i < kJobRing; ++i) mbar_init(smem_u32(&ctrl->job_ready[i]), 1);
    mbar_init(smem_u32(&ctrl->hid_full), 1);
    mbar_init(smem_u32(&ctrl->pref_ready), 1);
    ctrl->abort = 0;
    mbar_init_fence();
  }
  pdl_trigger();                                    // the next kernel may get resident behind this one
  if (warp == 0 && lane < 8) prefetch_tmap(lane == 0 ? &tm.h : (lane < 4 ? &tm.hk[lane - 1] : &tm.w[lane - 4]));
  __syncthreads();                                  // barriers exist; the producer starts at once

  if (warp == 0) {
    if (lane == 0) {
      // ---------------- producer -------------------------------------------------------------------
      const uint64_t pol_w = policy_evict_first(), pol_a = policy_evict_last();
      int stage = 0; uint32_t phase = 0, job_i = 0;
      int issued = 0;
      bool ok = true, deps = false;
      // W_U depends on no earlier kernel: its first stages are issued at once.  Hidden rows and
      // codebook state do: before the ring's first wrap (and before anything else that needs
      // them) the producer waits for the preceding kernel and loads the resident hidden rows.
      auto need_deps = [&]() {
        if (deps) return;
        pdl_wait();
        if (RESIDENT) {
          const uint32_t bar = smem_u32(&ctrl->hid_full);
          mbar_expect_tx(bar, hid_bytes);
          for (int kb = 0; kb < p.ksteps; kb += p.hid_box_kb)
            tma_load_3d(hid_base + (uint32_t)kb * hid_rows * 128, &tm.h, 0, 0, kb, bar, pol_a);
        }
        deps = true;
      };
      if (!RESIDENT) need_deps();                   // every stage carries a box of hidden rows
      auto publish = [&](const DecodeJob& j) {
        const uint32_t slot = job_i % kJobRing;
        ds->jobs[slot] = j;
        mbar_arrive(smem_u32(&ctrl->job_ready[slot]));          // release: the job is visible to waiters
        ++job_i;
      };
      const int g_first = (int)blockIdx.x * p.fixed_granules;
      auto stream = [&](const DecodeJob& j) {
        const int big = j.cls == 2;
        const int ksb = big ? 1 : 2;
        const CUtensorMap* wm = &tm.w[j.wmap * 2 + big];
        const CUtensorMap* hm = &tm.hk[big ? 0 : 1];
        for (int ks = 0; ks < p.ksteps && ok; ks += ksb) {
          if (issued == STAGES) need_deps();
          ++issued;
          if (!mbar_wait(smem_u32(&ctrl->empty[stage]), phase ^ 1u, &ctrl->abort)) { ok = false; break; }
          const uint32_t full = smem_u32(&ctrl->full[stage]);
          mbar_expect_tx(full, NT * 128 + (RESIDENT ? 0u : (uint32_t)(ksb * hid_rows * 128)));
          const uint32_t sb = stage_base + (uint32_t)stage * stage_bytes;
          tma_load_3d(sb, wm, 0, j.wrow, ks, full, pol_w);
          if (!RESIDENT) tma_load_3d(sb + NT * 128, hm, 0, 0, ks, full, pol_a);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      };
      // fixed share: 128-row jobs of W_U, known without any codebook state
      for (int g = g_first; g < g_first + p.fixed_granules && ok; g += 2) {
        const int big = g + 2 <= g_first + p.fixed_granules;     // an odd share ends with one 64-row job
        const int rows = big ? NT : kGran;
        DecodeJob j;
        j.cls = big ? 2 : 1; j.wmap = 0; j.wrow = g * kGran; j.col0 = j.wrow; j.owner = -1; j.k0 = 0; j.pad = 0;
        j.nvalid = p.cb.V - j.wrow < rows ? p.cb.V - j.wrow : rows;
        publish(j);
        stream(j);
      }
      // pool: the rest of W_U and every visible row of U_h, claimed 64 rows at a time
      need_deps();
      if (ok && !mbar_wait(smem_u32(&ctrl->pref_ready), 0, &ctrl->abort)) ok = false;
      if (ok) {
        const int gs = (p.cb.V + kGran - 1) / kGran;
        const int pool_static = gs - p.fixed_granules * (int)gridDim.x;
        const int pool_total = pool_static + s_pref[p.cb.B];
        // Guided claims: two consecutive granules (one 128-row job when they lie in one segment)
        // while more than four rounds of single units are left, then single 64-row units, so that
        // the CTAs finish within one small unit of each other.
        const int single_from = pool_total - 4 * (int)gridDim.x;
        int chunk = 2 <= single_from ? 2 : 1;
        int u = atomicAdd(p.counters, chunk);
        DecodeJob j, j2;
        while (ok && pool_job(p, s_pref, pool_static, pool_total, u, j)) {
          const bool pair = chunk == 2 && pool_job(p, s_pref, pool_static, pool_total, u + 1, j2);
          const bool fused = pair && j2.wmap == j.wmap && j2.owner == j.owner && j2.wrow == j.wrow + kGran;   // one segment
          if (fused) { j.cls = 2; j.nvalid += j2.nvalid; }
          publish(j);
          stream(j);
          if (pair && !fused && ok) { publish(j2); stream(j2); }
          // the next claim is made only now: the stages still in flight cover its latency, and a
          // CTA never holds a unit that another, idle CTA could already be streaming
          chunk = u + chunk + 2 <= single_from ? 2 : 1;
          u = atomicAdd(p.counters, chunk);
        }
      }
      DecodeJob last;
      last.cls = -1; last.wmap = 0; last.wrow = 0; last.col0 = 0; last.nvalid = 0; last.owner = -1; last.k0 = 0; last.pad = 0;
      publish(last);
    }
  } else {
    // ---------------- warps 1-5: session state, tensor memory, then MMA and epilogue roles --------------
    pdl_wait();                                     // codebook counters, row tables, partial slots: all dependent
    if (warp == 1) {                                // prefix of per-sequence granule counts of U_h
      int carry = 0;
      for (int base = 0; base < p.cb.B; base += 32) {
        const int b = base + lane;
        int v = b < p.cb.B ? (p.cb.n[b] + kGran - 1) / kGran : 0;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int x = __shfl_up_sync(0xffffffffu, v, o); if (lane >= o) v += x; }
        if (b < p.cb.B) s_pref[b + 1] = carry + v;
        carry += __shfl_sync(0xffffffffu, v, 31);
      }
      if (lane == 0) s_pref[0] = 0;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctrl->pref_ready));
    } else if (warp == 2) {
      tmem_alloc(smem_u32(&ctrl->tmem_base), decode_tmem_cols(NBP));
      tmem_relinquish();
    } else if (warp == 3) {
      const int r = lane;
      int sq = -1, nv = 0, tg = -1;
      if (r < a.N) {
        sq = a.row_seq ? a.row_seq[r] : r;
        if (sq < 0 || sq >= p.cb.B) sq = -1;
        if (sq >= 0) {
          nv = p.cb.n[sq];
          if (a.row_nvis) { const int x = a.row_nvis[r]; nv = x < nv ? (x < 0 ? 0 : x) : nv; }
        }
        if (a.targets) tg = a.targets[r];
      }
      ds->seq[r] = sq; ds->nvis[r] = nv; ds->tgt[r] = tg;
    }
    tc_fence_before();
    asm volatile("bar.sync 2, %0;" ::"n"(32 + 32 * EW) : "memory");   // all but the producer warp: tensor memory address and row table are set
    tc_fence_after();
  }
  if (warp == 1) {
    if (lane == 0) {
      // ---------------- MMA issuer --------------------------------------------------------------------
      const uint32_t tmem_base = ctrl->tmem_base;
      const uint32_t idesc = idesc_bf16_f32(NT, NBP);
      int stage = 0; uint32_t phase = 0, job_i = 0;
      bool ok = !RESIDENT || mbar_wait(smem_u32(&ctrl->hid_full), 0, &ctrl->abort);
      while (ok) {
        const uint32_t slot = job_i % kJobRing;
        if (!mbar_wait(smem_u32(&ctrl->job_ready[slot]), (job_i / kJobRing) & 1u, &ctrl->abort)) break;
        const DecodeJob j = ds->jobs[slot];
        if (j.cls < 0) break;
        const uint32_t buf = job_i & 1u, aph = (job_i >> 1) & 1u;
        if (!mbar_wait(smem_u32(&ctrl->acc_empty[buf]), aph ^ 1u, &ctrl->abort)) break;
        tc_fence_after();
        const uint32_t d = tmem_base + buf * NBP;
        const int ksb = j.cls == 2 ? 1 : 2;
        const uint32_t kb_bytes = (uint32_t)(j.cls == 2 ? NT : kGran) * 128;   // one k-block of the job's rows
        uint32_t acc = 0;
        for (int ks = 0; ks < p.ksteps; ks += ksb) {
          if (!mbar_wait(smem_u32(&ctrl->full[stage]), phase, &ctrl->abort)) { ok = false; break; }
          tc_fence_after();
          const uint32_t wb = stage_base + (uint32_t)stage * stage_bytes;
          for (int i = 0; i < ksb; ++i) {
            const uint32_t wi = wb + (uint32_t)i * kb_bytes;
            const uint32_t hb = RESIDENT ? hid_base + (uint32_t)(ks + i) * hid_rows * 128
                                         : wb + NT * 128 + (uint32_t)i * hid_rows * 128;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              umma_bf16(d, smem_desc_sw128(wi + k * 32), smem_desc_sw128(hb + k * 32), idesc, acc);
              acc = 1;
            }
          }
          umma_commit(smem_u32(&ctrl->empty[stage]));            // frees the stage once the MMAs have read it
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(smem_u32(&ctrl->acc_full[buf]));
        ++job_i;
      }
    }
  } else if (warp >= 2) {
    // ---------------- epilogue: thread = vocabulary row of the job ------------------------------------
    const uint32_t tmem_base = ctrl->tmem_base;
    const int q = warp & 3;                           // tensor-memory lane quarter this warp may read
    const int h0 = ((warp - 2) >> 2) * RW;            // first hidden row of this warp's share
    const int row_in_job = q * 32 + lane;
    const uint32_t k0 = (uint32_t)a.seed, k1 = (uint32_t)(a.seed >> 32);
    const uint32_t c2 = (uint32_t)a.step, c3 = (uint32_t)(a.step >> 32);
    const size_t ldbg = (size_t)p.cb.V + p.cb.cap;
    float m[RW], s[RW]; int idx[RW];
    float gm[GENERIC ? RW : 1]; int gidx[GENERIC ? RW : 1];
#pragma unroll
    for (int bb = 0; bb < RW; ++bb) { m[bb] = -INFINITY; s[bb] = 0.f; idx[bb] = 0x7fffffff; }
#pragma unroll
    for (int bb = 0; bb < (GENERIC ? RW : 1); ++bb) { gm[bb] = -INFINITY; gidx[bb] = 0x7fffffff; }
    uint32_t job_i = 0;
    while (true) {
      const uint32_t slot = job_i % kJobRing;
      if (!mbar_wait(smem_u32(&ctrl->job_ready[slot]), (job_i / kJobRing) & 1u, &ctrl->abort)) break;
      const DecodeJob j = ds->jobs[slot];
      if (j.cls < 0) break;
      const uint32_t buf = job_i & 1u, aph = (job_i >> 1) & 1u;
      if (!mbar_wait(smem_u32(&ctrl->acc_full[buf]), aph, &ctrl->abort)) break;
      tc_fence_after();
      if (q * 32 < j.nvalid) {                       // warp-uniform: some weight row of this quarter exists
        uint32_t v[RW];
        TmemRow<RW>::ld(tmem_base + ((uint32_t)(q * 32) << 16) + buf * NBP + h0, v);
        tmem_ld_wait();
        if (row_in_job < j.nvalid) {
          const int col = j.col0 + row_in_job;
          const int krow = j.k0 + row_in_job;        // entry number, for hypertoken rows
#pragma unroll
          for (int bb = 0; bb < RW; ++bb) {
            const int hr = h0 + bb;                    // hidden row of the batch
            const int sq = ds->seq[hr];
            const bool vis = sq >= 0 && (j.owner < 0 || (sq == j.owner && krow < ds->nvis[hr]));
            if (vis) {
              const float l = __uint_as_float(v[bb]);
              if (l > m[bb]) { s[bb] = s[bb] * __expf(m[bb] - l) + 1.f; m[bb] = l; idx[bb] = col; }
              else { s[bb] += __expf(l - m[bb]); if (l == m[bb] && col < idx[bb]) idx[bb] = col; }
              if (GENERIC) {
                if (a.select == Z2Z_SELECT_GUMBEL) {
                  const Philox4 px = philox4x32_10((uint32_t)(col >> 2), (uint32_t)(a.row_base + hr), c2, c3, k0, k1);
                  const float sc = fmaf(l, a.inv_temperature, gumbel_from_word(philox_word(px, col & 3)));
                  if (sc > gm[bb] || (sc == gm[bb] && col < gidx[bb])) { gm[bb] = sc; gidx[bb] = col; }
                }
                if (a.logits_debug) a.logits_debug[(size_t)hr * ldbg + col] = l;
                if (col == ds->tgt[hr] && a.target_logit) a.target_logit[hr] = l;
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&ctrl->acc_empty[buf]));
      ++job_i;
    }
    // merge the 128 threads' reductions of every hidden row: the warp's maximum first, then every
    // lane's sum rescaled to it, then the lowest index among the lanes that hold the maximum
#pragma unroll
    for (int bb = 0; bb < RW; ++bb) {
      const float mm = key_float(__reduce_max_sync(0xffffffffu, float_key(m[bb])));
      float ss = m[bb] == -INFINITY ? 0.f : s[bb] * __expf(m[bb] - mm);
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
      const int ii = __reduce_min_sync(0xffffffffu, m[bb] == mm ? idx[bb] : 0x7fffffff);
      float gg = -INFINITY; int gi = 0x7fffffff;
      if (GENERIC) {
        gg = key_float(__reduce_max_sync(0xffffffffu, float_key(gm[bb])));
        gi = __reduce_min_sync(0xffffffffu, gm[bb] == gg ? gidx[bb] : 0x7fffffff);
      }
      if (lane == 0) { RowRed r; r.m = mm; r.s = ss; r.idx = ii; r.gm = gg; r.gidx = gi; ds->part[q][h0 + bb] = r; }
    }
    asm volatile("bar.sync 1, %0;" ::"n"(32 * EW) : "memory");   // the epilogue warps only
    const int t = (warp - 2) * 32 + lane;
    if (t < NB && t < a.N) {
      RowRed red = ds->part[0][t];
      red.merge(ds->part[1][t]); red.merge(ds->part[2][t]); red.merge(ds->part[3][t]);
      LogitPartial* lp = reinterpret_cast<LogitPartial*>(a.lpart) + (size_t)t * p.part_stride + blockIdx.x;
      lp->m = red.m; lp->s = red.s; lp->idx = red.idx; lp->gm = red.gm; lp->gidx = red.gidx;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    if (ctrl->abort) atomicOr(p.err, 1);
    // the last CTA to finish puts the pool counter back to zero for the next launch
    const unsigned done = atomicInc(reinterpret_cast<unsigned*>(p.counters + 1), gridDim.x - 1);
    if (done == gridDim.x - 1) atomicExch(p.counters, 0);
  }
  if (warp == 2) tmem_dealloc(ctrl->tmem_base, decode_tmem_cols(NBP));
}

// One warp per hidden row: merge the partials of all CTAs, write the outputs.
__global__ void __launch_bounds__(128) k_decode_logits_merge(LogitsArgs a, int stride, int count) {
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= a.N) return;
  const LogitPartial* lp = reinterpret_cast<const LogitPartial*>(a.lpart) + (size_t)r * stride;
  RowRed red; red.init();
  for (int g = lane; g < count; g += 32) {
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

__global__ void k_decode_fill_nan(float* p, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = __int_as_float(0x7fc00000);
}

}  // namespace

// Decode batches: at most 32 hidden rows, with any outputs; d a multiple of 256.
bool decode_logits_applies(const LogitsArgs& a) {
  return a.dtype == Z2Z_DTYPE_BF16 && a.d % 256 == 0 && a.N <= 32;
}

template <int NB, bool GENERIC>
static cudaError_t launch_decode(DecodeLogitsParams p, const DecodeLogitMaps& maps, int grid, bool resident,
                                 cudaStream_t s) {
  const size_t hid = resident ? (((size_t)p.ksteps * p.hid_rows * 128 + 1023) & ~(size_t)1023) : 0;
  const size_t stage = 128 * 128 + (resident ? 0 : (((size_t)2 * p.hid_rows * 128 + 1023) & ~(size_t)1023));
  // Shared memory behind the last stage stays readable (kTailPadBytes): an MMA always reads 128
  // weight rows from a k-block's start and 16 or 32 hidden rows, also when fewer were loaded; what
  // it reads beyond them only feeds accumulator rows and columns that nobody looks at.
  const size_t fixed = 1024 + 10240 + hid + kTailPadBytes;
  int st = (int)((227 * 1024 - fixed) / stage);
  if (st > kDecodeMaxStages) st = kDecodeMaxStages;
  if (st < 3) return cudaErrorInvalidConfiguration;
  p.stages = st;
  const size_t smem = fixed + st * stage;
  auto kern = resident ? k_decode_logits<NB, GENERIC, true> : k_decode_logits<NB, GENERIC, false>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(kern, dim3(grid), dim3(decode_threads(NB)), smem, s, p, maps);
}

cudaError_t run_logits_decode(const CbView& cb, const LogitsArgs& a, int* counters, int* err_word,
                              LogitsPartInfo* info, Prof* prof, cudaStream_t s) {
  static int n_sm = 0;
  if (!n_sm) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (n_sm <= 0) n_sm = 148;
  }
  DecodeLogitsParams p{};
  p.cb = cb; p.la = a;
  p.ksteps = a.d / 64;
  p.hid_rows = (a.N + 7) / 8 * 8;
  p.counters = counters; p.err = err_word;
  // hidden rows stay resident in shared memory when they take at most 64 KB
  const bool resident = (size_t)p.ksteps * p.hid_rows * 128 <= 64 * 1024;
  p.hid_box_kb = 4;
  for (int k = 16; k >= 4; --k) if (p.ksteps % k == 0) { p.hid_box_kb = k; break; }
  const int gs = (cb.V + kGran - 1) / kGran;
  const int grid = gs < n_sm ? gs : n_sm;
  // fixed share: nine tenths of W_U; the rest and all of U_h are pooled
  p.fixed_granules = (int)((long long)gs * 9 / 10 / grid);
  DecodeLogitMaps maps;
  if (!make_tmap_bf16_kblocks(&maps.h, a.hidden, a.N, a.d, p.hid_rows, p.hid_box_kb)) return cudaErrorInvalidValue;
  for (int c = 0; c < 3; ++c)
    if (!make_tmap_bf16_kblocks(&maps.hk[c], a.hidden, a.N, a.d, p.hid_rows, 1 << c)) return cudaErrorInvalidValue;
  for (int t = 0; t < 2; ++t) {
    const void* base = t == 0 ? a.WU : a.Uh;
    const long long rows = t == 0 ? (long long)cb.V : (long long)cb.B * cb.cap;
    if (t == 1 && cb.cap == 0) { maps.w[2] = maps.w[0]; maps.w[3] = maps.w[1]; break; }
    if (!make_tmap_bf16_kblocks(&maps.w[t * 2 + 0], base, rows, a.d, kGran, 2)) return cudaErrorInvalidValue;
    if (!make_tmap_bf16_kblocks(&maps.w[t * 2 + 1], base, rows, a.d, 128, 1)) return cudaErrorInvalidValue;
  }
  p.part_stride = grid + 2;
  if ((size_t)a.N * p.part_stride * sizeof(LogitPartial) > a.lpart_bytes) return cudaErrorMemoryAllocation;
  if (info) { info->stride = p.part_stride; info->count = grid; }
  const bool generic = a.select == Z2Z_SELECT_GUMBEL || a.logits_debug || a.target_logit;
  if (a.target_logit) {
    ProfScope ps(prof, kProfLogitsMerge, 1, s);
    k_decode_fill_nan<<<(a.N + 255) / 256, 256, 0, s>>>(a.target_logit, a.N);
  }
  cudaError_t e;
  {
    ProfScope ps(prof, kProfLogits, 1, s);
    if (a.N <= 8) e = generic ? launch_decode<8, true>(p, maps, grid, resident, s) : launch_decode<8, false>(p, maps, grid, resident, s);
    else if (a.N <= 16) e = generic ? launch_decode<16, true>(p, maps, grid, resident, s) : launch_decode<16, false>(p, maps, grid, resident, s);
    else e = generic ? launch_decode<32, true>(p, maps, grid, resident, s) : launch_decode<32, false>(p, maps, grid, resident, s);
  }
  if (e != cudaSuccess || info) return e;
  ProfScope ps(prof, kProfLogitsMerge, 1, s);
  k_decode_logits_merge<<<(a.N + 3) / 4, 128, 0, s>>>(a, p.part_stride, grid);
  return cudaGetLastError();
}

}  // namespace z2z
