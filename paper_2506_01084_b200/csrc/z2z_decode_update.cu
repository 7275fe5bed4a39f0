// Middle of the decode step in ONE launch (paper Section 2.3, steps 8-10): finish the joint
// softmax reductions of every sequence from the per-CTA partials of the logits kernel, select the
// token (argmax or Gumbel-max sample, or the caller's forced code; a sequence may sit out), apply the online LZW update,
// and build the work list of new codebook entries for the hyper-encoder pass that follows.
// One warp per sequence; a single block, so that the list can be compacted without a second
// launch.
#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_lzw_dev.cuh"
#include "z2z_sm100.cuh"

namespace z2z {

__global__ void __launch_bounds__(1024) k_decode_update(CbView cb, DecodeUpdateArgs a, EntryList el) {
  __shared__ int s_cnt[1024];
  __shared__ int s_n[1024];                 // hypertokens of the sequence after this step
  __shared__ signed char s_len[1024];       // base tokens of the entry it created
  __shared__ int s_tok[1024][kMaxM];        // ... and the tokens themselves: the work list needs no reload
  __shared__ int s_warp[32];
  sm100::pdl_trigger();
  sm100::pdl_wait();               // the logits partials and the codebook state come from earlier kernels
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  for (int b = tid; b < 1024; b += blockDim.x) s_cnt[b] = 0;
  __syncthreads();
  for (int b = warp; b < cb.B; b += 32) {
    const LzwPrev state = warp_lzw_load(cb, b);            // independent of the selection: loaded ahead of it
    // ---- merge the partial reductions of hidden row b
    const LogitPartial* lp = a.lpart + (size_t)b * a.part_stride;
    RowRed red; red.init();
    for (int g = lane; g < a.part_count; g += 32) {
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
    const int amax = red.idx == 0x7fffffff ? -1 : red.idx;
    const int smp = red.gidx == 0x7fffffff ? -1 : red.gidx;
    const int sel = a.select == Z2Z_SELECT_GUMBEL ? smp : amax;
    int code = a.forced ? a.forced[b] : sel;
    if (code == Z2Z_CODE_SELECTED) code = sel;
    const bool sits_out = a.forced && code == Z2Z_CODE_NONE;   // a finished sequence of the batch
    if (lane == 0) {
      if (a.lse) a.lse[b] = red.m + logf(red.s);
      if (a.selected) a.selected[b] = sel;
      a.next_codes[b] = code;
    }
    // ---- online LZW update with the applied code
    int new_tok = -1;
    const int created = sits_out ? -1 : warp_lzw_step(cb, b, code, state, &new_tok);
    if (lane < cb.M) s_tok[b][lane] = new_tok;
    if (lane == 0) {
      if (a.new_entry) a.new_entry[b] = created;
      s_cnt[b] = created >= 0 ? created + 1 : 0;         // 0: none, else entry number + 1
      s_len[b] = (signed char)(created >= 0 ? state.plen + 1 : 0);
      s_n[b] = state.n + (created >= 0 ? 1 : 0);
    }
  }
  __syncthreads();
  // ---- compact the new entries into the encoder's work list (exclusive scan over sequences): an
  // entry's slot in the list, and the first of the PACKED rows that its base tokens take (the
  // tensor-core pass keeps no padding rows).  Both sums travel in one word: entries in the low
  // half, rows in the high half (at most 1024 entries of at most 8 rows).
  const int mine = tid < cb.B ? s_cnt[tid] : 0;
  const int flag = mine > 0 ? 1 : 0;
  const int my_len = flag ? (int)s_len[tid] : 0;
  const int val = flag | (my_len << 16);
  int incl = val;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += x;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = s_warp[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, w, o);
      if (lane >= o) w += x;
    }
    s_warp[lane] = w;
  }
  __syncthreads();
  const int excl_both = incl - val + (warp > 0 ? s_warp[warp - 1] : 0);
  const int excl = excl_both & 0xffff, row0 = excl_both >> 16;
  const int total = s_warp[31] & 0xffff, total_rows = s_warp[31] >> 16;
  if (tid < cb.B) el.off[tid] = excl;
  if (tid == 0) {
    el.off[cb.B] = total; el.off[cb.B + 1] = total < el.chunk ? total : el.chunk;
    el.row_off[cb.B] = total_rows;                 // the pass that follows is sized for B entries
  }
  if (flag && excl < el.chunk) {
    el.seq[excl] = tid; el.idx[excl] = mine - 1;
    el.len[excl] = my_len;
    el.row_off[excl] = row0;
    for (int i = 0; i < cb.M; ++i) {
      const int tok = s_tok[tid][i];
      el.tok[(size_t)excl * cb.M + i] = tok;
      if (i < my_len) { el.row_src[row0 + i] = excl * cb.M + i; el.row_tok[row0 + i] = tok; }
    }
  }
  for (int e = total + tid; e < el.chunk && e < cb.B; e += blockDim.x) {
    el.seq[e] = -1; el.idx[e] = 0; el.len[e] = 0; el.row_off[e] = total_rows;
    for (int i = 0; i < cb.M; ++i) el.tok[(size_t)e * cb.M + i] = -1;
  }
  // both caches will hold every entry once the encoder pass that follows has run
  int full = 1;
  if (tid < cb.B) {
    const int n = s_n[tid];
    cb.n_emb[tid] = n; cb.n_emb[cb.B + tid] = n;
    full = n >= cb.cap && mine == 0;             // full already when this step began: it created nothing
  }
  // Once every codebook is full no step creates an entry any more.  The host learns it through a
  // word in its own memory and stops launching the hyper-encoder pass (the session number guards
  // against a late store from before a reset).  The word is only written by a step that found every
  // codebook full on entry: the step that creates the last entry still needs its encoder pass, and
  // the host may read the word at any time after this kernel was enqueued.
  if (a.frozen_flag && cb.B <= (int)blockDim.x) {
    const int all_full = __syncthreads_and(full);
    if (all_full && tid == 0) *reinterpret_cast<volatile int*>(a.frozen_flag) = a.epoch;
  }
}

cudaError_t launch_decode_update(const CbView& cb, const DecodeUpdateArgs& a, const EntryList& el,
                                 cudaStream_t s) {
  return launch_pdl(k_decode_update, dim3(1), dim3(1024), 0, s, cb, a, el);
  return cudaGetLastError();
}

}  // namespace z2z
