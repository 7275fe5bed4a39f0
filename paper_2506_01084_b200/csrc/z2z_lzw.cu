// LZW codebook kernels: session reset, prompt compression, online update.
//
// One warp owns one sequence.  The codebook of a sequence is an open-addressing hash table in
// global memory keyed by (prefix code, next base token); a probe is one coalesced 256-byte load of
// a 32-slot bucket followed by a warp ballot.  Entries are never deleted and an insert always
// takes the first empty slot in probe order, so "an empty slot in the bucket" proves absence.
// The parse itself is a dependent chain (each token's lookup needs the previous match), which is
// why the unit of parallelism is the sequence (paper Section 2.4: compression is per document).
#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_lzw_dev.cuh"

namespace z2z {

__global__ void k_codebook_clear(CbView cb) {
  size_t n_hash = (size_t)cb.B * cb.n_slots;
  size_t n_cons = (size_t)cb.B * cb.cap * cb.M;
  size_t n_len = (size_t)cb.B * cb.cap;
  size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = tid; i < n_hash; i += stride) cb.hash[i] = kEmptySlot;
  for (size_t i = tid; i < n_cons; i += stride) cb.cons[i] = -1;
  for (size_t i = tid; i < n_len; i += stride) cb.len[i] = 0;
  for (size_t i = tid; i < (size_t)cb.B; i += stride) {
    cb.n[i] = 0; cb.prev[i] = -1; cb.status[i] = 0; cb.n_emb[i] = 0; cb.n_emb[cb.B + i] = 0;
  }
}

// Prompt compression (Section 2.1; Section 2.3 step 2).  grid = ceil(B / warps per block).
__global__ void __launch_bounds__(128) k_lzw_encode(CbView cb, const int32_t* __restrict__ tokens,
                                                    const int32_t* __restrict__ lens, int T_max,
                                                    int32_t* __restrict__ codes,
                                                    int32_t* __restrict__ code_lens,
                                                    int32_t* __restrict__ entries_after) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (b >= cb.B) return;
  unsigned long long* table = cb.hash + (size_t)b * cb.n_slots;
  int T = lens ? lens[b] : T_max;
  T = T < 0 ? 0 : (T > T_max ? T_max : T);
  const int32_t* x = tokens + (size_t)b * T_max;
  int32_t* out = codes + (size_t)b * T_max;
  int32_t* aft = entries_after ? entries_after + (size_t)b * T_max : nullptr;
  int n = cb.n[b];
  int st = 0;
  int w = -1, wlen = 0, n_out = 0;
  for (int base = 0; base < T; base += 32) {
    int mine = (base + lane < T) ? x[base + lane] : 0;
    int cnt = T - base < 32 ? T - base : 32;
    for (int i = 0; i < cnt; ++i) {
      int c = __shfl_sync(0xffffffffu, mine, i);
      if ((unsigned)c >= (unsigned)cb.V) { st |= Z2Z_ST_BAD_TOKEN; c = 0; }   // not a base token
      if (wlen == 0) { w = c; wlen = 1; continue; }
      Probe p{-1, -1};
      if (wlen < cb.M) {
        p = warp_probe(table, cb.n_slots, (uint32_t)w, (uint32_t)c);
        if (p.found >= 0) { w = cb.V + p.found; ++wlen; continue; }      // match grows
      }
      // longest match ends: emit it, then remember (w ++ c) if allowed
      if (lane == 0) out[n_out] = w;
      if (wlen < cb.M && n < cb.cap) {
        if (p.slot >= 0) {
          if (lane == 0) table[p.slot] = pack_slot((uint32_t)w, (uint32_t)c, (uint32_t)n);
          warp_write_entry(cb, b, n, w, wlen, c);
          ++n;
          if (n >= cb.cap) st |= Z2Z_ST_CAP_FROZEN;
          __syncwarp();                     // the new slot and entry are visible to later probes
        } else {
          st |= Z2Z_ST_TABLE_FULL;
        }
      }
      if (aft && lane == 0) aft[n_out] = n;
      ++n_out;
      w = c; wlen = 1;
    }
  }
  if (wlen > 0) {                             // final flush creates no entry
    if (lane == 0) { out[n_out] = w; if (aft) aft[n_out] = n; }
    ++n_out;
  }
  if (lane == 0) {
    code_lens[b] = n_out;
    cb.n[b] = n;
    if (n_out > 0) cb.prev[b] = w;
    if (st) atomicOr(&cb.status[b], st);
  }
}

// Online update with one new code per sequence (Figure 1; Section 2.3 step 10).
__global__ void __launch_bounds__(128) k_lzw_step(CbView cb, const int32_t* __restrict__ new_codes,
                                                  const uint8_t* __restrict__ active,
                                                  int32_t* __restrict__ new_entry) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (b >= cb.B) return;
  if (active && !active[b]) { if (lane == 0 && new_entry) new_entry[b] = -1; return; }
  const int created = warp_lzw_step(cb, b, new_codes[b]);
  if (lane == 0 && new_entry) new_entry[b] = created;
}

cudaError_t launch_codebook_clear(const CbView& cb, cudaStream_t s) {
  size_t work = (size_t)cb.B * cb.n_slots;
  int blocks = (int)((work + 255) / 256);
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  k_codebook_clear<<<blocks, 256, 0, s>>>(cb);
  return cudaGetLastError();
}

cudaError_t launch_lzw_encode(const CbView& cb, const int32_t* tokens, const int32_t* lens,
                              int T_max, int32_t* codes, int32_t* code_lens,
                              int32_t* entries_after, cudaStream_t s) {
  // one warp per block: every sequence gets its own SM while B <= 148, which keeps each
  // dependent probe chain at the lowest latency the memory system gives
  k_lzw_encode<<<cb.B, 32, 0, s>>>(cb, tokens, lens, T_max, codes, code_lens, entries_after);
  return cudaGetLastError();
}

cudaError_t launch_lzw_step(const CbView& cb, const int32_t* new_codes, const uint8_t* active,
                            int32_t* new_entry, cudaStream_t s) {
  int wpb = 4;
  k_lzw_step<<<(cb.B + wpb - 1) / wpb, wpb * 32, 0, s>>>(cb, new_codes, active, new_entry);
  return cudaGetLastError();
}

}  // namespace z2z
