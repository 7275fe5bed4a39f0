// Hyper-encoder linear layers for MANY codebook entries (all entries of the prompts; paper
// Section 2.2 applied after Section 2.3 step 2).  With thousands of rows this is a dense
// contraction and runs on CTA pairs like the prompt-scoring logits kernel:
//
//   D[256 rows x 256 cols] = (A_hi + A_lo)[rows, K] . W[cols, K]^T
//
// tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 16), each CTA loading its own 128 activation
// rows (the bf16 hi part and the bf16 lo part, see z2z_encoder_tc.cu) and its own 128 weight rows
// with plain TMA loads; both parts accumulate into the same fp32 tile in tensor memory, which is
// double buffered so that the epilogue of one tile overlaps the mainloop of the next.  Every
// tile is owned by one cluster for its whole K range, so the epilogue can finish the layer:
//   kEpiStore   out[r, c]  = acc + bias                      (q, k, v for the attention kernel)
//   kEpiResid   X[r, c]   += acc + bias                      (attention output / second MLP layer)
//   kEpiGelu    H[r, c]    = split_hi_lo(gelu(acc + bias))   (first MLP layer)
// Rows that are padding of their entry (or lie beyond the pass) are not written (kEpiGelu writes
// zeros there, because the next GEMM reads them).
//
// HALF variant: the activations are ONE fp16 matrix (rounded once, 2^-11 relative) and the weights
// an fp16 copy of the bf16 tensor (exact within fp16's range), so a k-step is one MMA instead of
// two and a stage holds 32 KB instead of 48: half the tensor-core work of the layer.  kEpiGelu
// then writes one fp16 matrix.
//
// Roles per CTA: warp 0 lane 0 TMA producer, warp 1 lane 0 MMA issuer (leader CTA only), warps
// 2-5 epilogue (thread = row).  Every mbarrier wait is bounded.
#include <cuda_fp16.h>

#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_sm100.cuh"
#include "z2z_stream.h"

namespace z2z {
using namespace sm100;

namespace {

constexpr int kThreads = 192;
constexpr int kPgMaxStages = 6;
// Two-part operands: 4 stages of 48 KB per CTA (A hi, A lo, W, each 128 x 64 bf16); one fp16 operand:
// 6 stages of 32 KB (A, W).
__host__ __device__ constexpr int pg_stages(bool half) { return half ? 6 : 4; }
__host__ __device__ constexpr uint32_t pg_stage_bytes(bool half) { return half ? 32768u : 49152u; }

struct PgCtrl {
  unsigned long long full[kPgMaxStages], empty[kPgMaxStages], acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort;
};

template <int EPI, bool HALF>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
k_pair_gemm(const PairGemmParams p, const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW) {
  constexpr int kPgStages = pg_stages(HALF);
  constexpr uint32_t kPgStageBytes = pg_stage_bytes(HALF);
  constexpr uint32_t kWOff = HALF ? 16384u : 32768u;        // weight tile inside a stage
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  PgCtrl* ctrl = reinterpret_cast<PgCtrl*>(sm);
  const uint32_t stage_base = smem_u32(sm + 1024);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0: leader (issues the MMAs), 1: peer
  const int n_clusters = gridDim.x >> 1, cluster_id = blockIdx.x >> 1;
  // only the row tiles that hold rows of live entries of this pass are computed (the host sizes
  // the launch for its upper bound of entries; the count itself is device state)
  int live_rows = *p.live_rows;                     // rows are packed: no padding rows inside entries
  live_rows = live_rows < p.R ? live_rows : p.R;
  const int row_tiles = (live_rows + 255) / 256;
  const int n_tiles = row_tiles * p.col_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPgStages; ++s) {
      mbar_init(smem_u32(&ctrl->full[s]), 1);        // leader: its producer's arrive + bytes of both CTAs
      mbar_init(smem_u32(&ctrl->empty[s]), 1);       // one multicast commit
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&ctrl->acc_full[b]), 1);    // one multicast commit
      mbar_init(smem_u32(&ctrl->acc_empty[b]), 8);   // leader: 4 epilogue warps of each CTA
    }
    ctrl->abort = 0;
    mbar_init_fence();
    prefetch_tmap(&tmA); prefetch_tmap(&tmW);
  }
  __syncthreads();
  if (warp == 2) { tmem_alloc_pair(smem_u32(&ctrl->tmem_base), 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                               // both CTAs' barriers exist before any remote signal
  tc_fence_after();
  const uint32_t tmem_base = ctrl->tmem_base;

  // tile t -> (row tile, column tile): neighbouring clusters take different row tiles of the same
  // column tile, so that a weight tile is read from HBM once and found in L2 by the others
  if (warp == 0) {
    if (lane == 0) {
      // ---------------- TMA producer (both CTAs) ---------------------------------------------------
      const uint64_t pol = policy_evict_last();
      uint32_t full_leader[kPgStages];
      for (int s = 0; s < kPgStages; ++s) full_leader[s] = map_to_cta(smem_u32(&ctrl->full[s]), 0);
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int t = cluster_id; t < n_tiles && ok; t += n_clusters) {
        const int rt = t % row_tiles, ct = t / row_tiles;
        const int arow = rt * 256 + (int)rank * 128;
        const int wrow = ct * 256 + (int)rank * 128;
        for (int ks = 0; ks < p.ksteps; ++ks) {
          if (!mbar_wait(smem_u32(&ctrl->empty[stage]), phase ^ 1u, &ctrl->abort)) { ok = false; break; }
          if (rank == 0) mbar_expect_tx(smem_u32(&ctrl->full[stage]), 2 * kPgStageBytes);
          const uint32_t sb = stage_base + (uint32_t)stage * kPgStageBytes;
          tma_load_2d_pair(sb, &tmA, ks * 64, arow, full_leader[stage], pol);                 // hi rows (HALF: the rows)
          if (!HALF) tma_load_2d_pair(sb + 16384, &tmA, ks * 64, p.Rt + arow, full_leader[stage], pol);   // lo rows
          tma_load_2d_pair(sb + kWOff, &tmW, ks * 64, wrow, full_leader[stage], pol);
          if (++stage == kPgStages) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      // ---------------- MMA issuer (leader only) ------------------------------------------------------
      const uint32_t idesc = HALF ? idesc_f16_f32(256, 256) : idesc_bf16_f32(256, 256);
      int stage = 0; uint32_t phase = 0, job_i = 0;
      bool ok = true;
      for (int t = cluster_id; t < n_tiles && ok; t += n_clusters) {
        const uint32_t buf = job_i & 1u, aph = (job_i >> 1) & 1u;
        if (!mbar_wait(smem_u32(&ctrl->acc_empty[buf]), aph ^ 1u, &ctrl->abort)) break;
        tc_fence_after();
        const uint32_t d = tmem_base + buf * 256;
        uint32_t acc = 0;
        for (int ks = 0; ks < p.ksteps; ++ks) {
          if (!mbar_wait(smem_u32(&ctrl->full[stage]), phase, &ctrl->abort)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sb = stage_base + (uint32_t)stage * kPgStageBytes;
#pragma unroll
          for (int part = 0; part < (HALF ? 1 : 2); ++part)        // hi part, then lo part, into the same accumulator
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              umma_bf16_pair(d, smem_desc_sw128(sb + part * 16384 + k * 32), smem_desc_sw128(sb + kWOff + k * 32),
                             idesc, acc);
              acc = 1;
            }
          umma_commit_pair(smem_u32(&ctrl->empty[stage]));      // frees the stage in both CTAs
          if (++stage == kPgStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(smem_u32(&ctrl->acc_full[buf]));       // wakes the epilogues of both CTAs
        ++job_i;
      }
    }
  } else {
    // ---------------- epilogue (both CTAs): thread = activation row -----------------------------------
    const int q = warp & 3;                           // tensor-memory lane quarter this warp may read
    uint32_t acc_empty_leader[2];
    acc_empty_leader[0] = map_to_cta(smem_u32(&ctrl->acc_empty[0]), 0);
    acc_empty_leader[1] = map_to_cta(smem_u32(&ctrl->acc_empty[1]), 0);
    const __nv_bfloat16* bias = reinterpret_cast<const __nv_bfloat16*>(p.bias);
    uint32_t job_i = 0;
    for (int t = cluster_id; t < n_tiles; t += n_clusters) {
      const int rt = t % row_tiles, ct = t / row_tiles;
      const int r = rt * 256 + (int)rank * 128 + q * 32 + lane;
      const bool valid = r < live_rows;               // packed rows: every row below the total carries data
      const uint32_t buf = job_i & 1u, aph = (job_i >> 1) & 1u;
      if (!mbar_wait(smem_u32(&ctrl->acc_full[buf]), aph, &ctrl->abort)) break;
      tc_fence_after();
      const bool writes = EPI == kEpiGelu ? r < p.Rt : valid;
      if (__any_sync(0xffffffffu, writes)) {
        const uint32_t tbase = tmem_base + ((uint32_t)(q * 32) << 16) + buf * 256;
#pragma unroll 1
        for (int c0 = 0; c0 < 256; c0 += 32) {
          const int col = ct * 256 + c0;
          if (col >= p.J) break;                       // the last column tile may be half outside
          uint32_t v[32];
          tmem_ld32(tbase + c0, v);
          tmem_ld_wait();
          if (!writes) continue;
          float bs[32];
#pragma unroll
          for (int x = 0; x < 32; x += 8) {
            const uint4 u = *reinterpret_cast<const uint4*>(bias + col + x);
            bs[x + 0] = __uint_as_float(u.x << 16); bs[x + 1] = __uint_as_float(u.x & 0xffff0000u);
            bs[x + 2] = __uint_as_float(u.y << 16); bs[x + 3] = __uint_as_float(u.y & 0xffff0000u);
            bs[x + 4] = __uint_as_float(u.z << 16); bs[x + 5] = __uint_as_float(u.z & 0xffff0000u);
            bs[x + 6] = __uint_as_float(u.w << 16); bs[x + 7] = __uint_as_float(u.w & 0xffff0000u);
          }
          if (EPI == kEpiStore || EPI == kEpiResid) {
            float* dst = p.out + (size_t)r * p.J + col;
#pragma unroll
            for (int x = 0; x < 32; x += 4) {
              float4 o = make_float4(__uint_as_float(v[x]) + bs[x], __uint_as_float(v[x + 1]) + bs[x + 1],
                                     __uint_as_float(v[x + 2]) + bs[x + 2], __uint_as_float(v[x + 3]) + bs[x + 3]);
              if (EPI == kEpiResid) {
                const float4 xo = *reinterpret_cast<const float4*>(dst + x);
                o.x += xo.x; o.y += xo.y; o.z += xo.z; o.w += xo.w;
              }
              *reinterpret_cast<float4*>(dst + x) = o;
            }
          } else if (HALF) {
            __half* ho = reinterpret_cast<__half*>(p.out_hl) + (size_t)r * p.J + col;
#pragma unroll
            for (int x = 0; x < 32; x += 8) {
              uint32_t H[4];
#pragma unroll
              for (int y = 0; y < 8; y += 2) {
                float g0 = 0.f, g1 = 0.f;
                if (valid) {
                  const float a0 = __uint_as_float(v[x + y]) + bs[x + y], a1 = __uint_as_float(v[x + y + 1]) + bs[x + y + 1];
                  g0 = 0.5f * a0 * (1.0f + erff(a0 * 0.70710678118654752440f));
                  g1 = 0.5f * a1 * (1.0f + erff(a1 * 0.70710678118654752440f));
                }
                H[y >> 1] = (uint32_t)__half_as_ushort(__float2half_rn(g0)) | ((uint32_t)__half_as_ushort(__float2half_rn(g1)) << 16);
              }
              *reinterpret_cast<uint4*>(ho + x) = make_uint4(H[0], H[1], H[2], H[3]);
            }
          } else {
            __nv_bfloat16* hi = p.out_hl + (size_t)r * p.J + col;
            __nv_bfloat16* lo = hi + (size_t)p.Rt * p.J;
#pragma unroll
            for (int x = 0; x < 32; x += 8) {
              uint32_t H[4], L[4];
#pragma unroll
              for (int y = 0; y < 8; y += 2) {
                float g0 = 0.f, g1 = 0.f;
                if (valid) {
                  const float a0 = __uint_as_float(v[x + y]) + bs[x + y], a1 = __uint_as_float(v[x + y + 1]) + bs[x + y + 1];
                  g0 = 0.5f * a0 * (1.0f + erff(a0 * 0.70710678118654752440f));
                  g1 = 0.5f * a1 * (1.0f + erff(a1 * 0.70710678118654752440f));
                }
                const __nv_bfloat16 h0 = __float2bfloat16_rn(g0), h1 = __float2bfloat16_rn(g1);
                const __nv_bfloat16 l0 = __float2bfloat16_rn(g0 - __bfloat162float(h0));
                const __nv_bfloat16 l1 = __float2bfloat16_rn(g1 - __bfloat162float(h1));
                H[y >> 1] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
                L[y >> 1] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
              }
              *reinterpret_cast<uint4*>(hi + x) = make_uint4(H[0], H[1], H[2], H[3]);
              *reinterpret_cast<uint4*>(lo + x) = make_uint4(L[0], L[1], L[2], L[3]);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(acc_empty_leader[buf]);
      ++job_i;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && ctrl->abort) atomicOr(p.err, 1);
  cluster_sync_all();                               // nobody leaves while the pair's MMAs may read its memory
  if (warp == 2) tmem_dealloc_pair(tmem_base, 512);
}

}  // namespace

template <int EPI, bool HALF>
static cudaError_t launch_pair_gemm_t(const PairGemmParams& p, const CUtensorMap& mA, const CUtensorMap& mW, int clusters,
                                      cudaStream_t s) {
  const size_t smem = 1024 + 1024 + (size_t)pg_stages(HALF) * pg_stage_bytes(HALF);
  auto kern = k_pair_gemm<EPI, HALF>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<2 * clusters, kThreads, smem, s>>>(p, mA, mW);
  return cudaGetLastError();
}

// D = A W^T with the epilogue `epi`, for a pass of R rows.  half == false: A = A_hi + A_lo, two bf16
// blocks of Rt rows each, W bf16.  half == true: A is one fp16 matrix of Rt rows, W an fp16 copy.
cudaError_t launch_pair_gemm(const PairGemmParams& p0, const void* act, const void* W, int K, int epi, bool half,
                             cudaStream_t s) {
  static int n_sm = 0;
  if (!n_sm) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (n_sm <= 0) n_sm = 148;
  }
  PairGemmParams p = p0;
  p.ksteps = K / 64;
  p.row_tiles = (p.R + 255) / 256;
  p.col_tiles = (p.J + 255) / 256;
  CUtensorMap mA, mW;
  // (the element type of a tensor map only fixes the element size and the fill value: bf16 and fp16 alike)
  if (!make_tmap_bf16(&mA, act, (half ? 1ll : 2ll) * p.Rt, K, 128)) return cudaErrorInvalidValue;
  if (!make_tmap_bf16(&mW, W, p.J, K, 128)) return cudaErrorInvalidValue;
  const int tiles = p.row_tiles * p.col_tiles;
  const int clusters = tiles < n_sm / 2 ? tiles : n_sm / 2;
  if (half) {
    if (epi == kEpiStore) return launch_pair_gemm_t<kEpiStore, true>(p, mA, mW, clusters, s);
    if (epi == kEpiResid) return launch_pair_gemm_t<kEpiResid, true>(p, mA, mW, clusters, s);
    return launch_pair_gemm_t<kEpiGelu, true>(p, mA, mW, clusters, s);
  }
  if (epi == kEpiStore) return launch_pair_gemm_t<kEpiStore, false>(p, mA, mW, clusters, s);
  if (epi == kEpiResid) return launch_pair_gemm_t<kEpiResid, false>(p, mA, mW, clusters, s);
  return launch_pair_gemm_t<kEpiGelu, false>(p, mA, mW, clusters, s);
}

}  // namespace z2z
