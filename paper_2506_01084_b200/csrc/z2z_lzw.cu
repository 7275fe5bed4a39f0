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

// The same parse with the sequence's hash table held in shared memory for the duration of the
// kernel (codebooks of up to 8192 entries: 16384 slots, 128 KB).  The parse is a dependent chain
// of one probe per token; the bucket read comes from shared memory instead of L2, and the
// constituents of a new entry are not copied from the table: the phrase just matched IS the last
// `wlen` tokens of the input, so the new row is written from the token registers (the current
// batch of 32 and the one before it).  What remains per token is the chain of warp primitives of
// the probe itself (broadcast, hash, ballot, shuffle): about 240 ns per token against about 290
// with the table in global memory.  One CTA per sequence: warp 0 parses, all warps move the
// table in and out.
constexpr int kEncodeSmemThreads = 128;
constexpr size_t kEncodeSmemMaxBytes = 200 * 1024;

__device__ __forceinline__ Probe warp_probe_smem(const unsigned long long* table, int n_slots, uint32_t prefix,
                                                 uint32_t token) {
  const int lane = threadIdx.x & 31;
  const unsigned long long key = pack_slot(prefix, token, 0) >> 16;
  int bucket = (int)(hash_pair(prefix, token) & (uint32_t)(n_slots - 1)) & ~(kBucket - 1);
  Probe r{-1, -1};
  for (int it = 0; it < n_slots / kBucket; ++it) {          // bounded: at most the whole table
    const unsigned long long s = table[bucket + lane];
    const unsigned hit = __ballot_sync(0xffffffffu, (s >> 16) == key && s != kEmptySlot);
    if (hit) {
      const unsigned long long v = __shfl_sync(0xffffffffu, s, __ffs(hit) - 1);
      r.found = (int)(v & 0xffffu);
      return r;
    }
    const unsigned empty = __ballot_sync(0xffffffffu, s == kEmptySlot);
    if (empty) { r.slot = bucket + __ffs(empty) - 1; return r; }
    bucket = (bucket + kBucket) & (n_slots - 1);
  }
  return r;
}

__global__ void __launch_bounds__(kEncodeSmemThreads) k_lzw_encode_smem(CbView cb, const int32_t* __restrict__ tokens,
                                                                        const int32_t* __restrict__ lens, int T_max,
                                                                        int32_t* __restrict__ codes,
                                                                        int32_t* __restrict__ code_lens,
                                                                        int32_t* __restrict__ entries_after) {
  extern __shared__ unsigned long long s_table[];
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x;
  unsigned long long* table = cb.hash + (size_t)b * cb.n_slots;
  for (int i = threadIdx.x; i < cb.n_slots; i += blockDim.x) s_table[i] = table[i];
  __syncthreads();
  if (threadIdx.x < 32) {
    int T = lens ? lens[b] : T_max;
    T = T < 0 ? 0 : (T > T_max ? T_max : T);
    const int32_t* x = tokens + (size_t)b * T_max;
    int32_t* out = codes + (size_t)b * T_max;
    int32_t* aft = entries_after ? entries_after + (size_t)b * T_max : nullptr;
    int n = cb.n[b];
    int st = 0;
    int w = -1, wlen = 0, n_out = 0;
    int mine = 0, before = 0;                        // tokens [base, base + 32) and [base - 32, base)
    for (int base = 0; base < T; base += 32) {
      before = mine;
      mine = (base + lane < T) ? x[base + lane] : 0;
      if ((unsigned)mine >= (unsigned)cb.V) { if (base + lane < T) st |= Z2Z_ST_BAD_TOKEN; mine = 0; }   // not a base token
      const int cnt = T - base < 32 ? T - base : 32;
      for (int i = 0; i < cnt; ++i) {
        const int c = __shfl_sync(0xffffffffu, mine, i);
        if (wlen == 0) { w = c; wlen = 1; continue; }
        Probe p{-1, -1};
        if (wlen < cb.M) {
          p = warp_probe_smem(s_table, cb.n_slots, (uint32_t)w, (uint32_t)c);
          if (p.found >= 0) { w = cb.V + p.found; ++wlen; continue; }      // match grows
        }
        // longest match ends: emit it, then remember (w ++ c) if allowed
        if (lane == 0) out[n_out] = w;
        if (wlen < cb.M && n < cb.cap) {
          if (p.slot >= 0) {
            if (lane == 0) s_table[p.slot] = pack_slot((uint32_t)w, (uint32_t)c, (uint32_t)n);
            // entry n = input tokens [i - wlen, i] of this batch (negative positions: the batch before)
            const int pos = i - wlen + lane;                               // lane j holds constituent j
            const int from_now = __shfl_sync(0xffffffffu, mine, pos & 31);
            const int from_before = __shfl_sync(0xffffffffu, before, pos & 31);
            if (lane < cb.M) {
              const int v = lane <= wlen ? (pos >= 0 ? from_now : from_before) : -1;
              cb.cons[((size_t)b * cb.cap + n) * cb.M + lane] = v;
            }
            if (lane == 0) cb.len[(size_t)b * cb.cap + n] = (uint8_t)(wlen + 1);
            ++n;
            if (n >= cb.cap) st |= Z2Z_ST_CAP_FROZEN;
            __syncwarp();                     // the new slot is visible to later probes
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
    st = __reduce_or_sync(0xffffffffu, st);     // BAD_TOKEN is found per lane
    if (lane == 0) {
      code_lens[b] = n_out;
      cb.n[b] = n;
      if (n_out > 0) cb.prev[b] = w;
      if (st) atomicOr(&cb.status[b], st);
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < cb.n_slots; i += blockDim.x) table[i] = s_table[i];
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
  const size_t table_bytes = (size_t)cb.n_slots * sizeof(unsigned long long);
  if (table_bytes <= kEncodeSmemMaxBytes) {
    cudaError_t e = cudaFuncSetAttribute(k_lzw_encode_smem, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)table_bytes);
    if (e != cudaSuccess) return e;
    k_lzw_encode_smem<<<cb.B, kEncodeSmemThreads, table_bytes, s>>>(cb, tokens, lens, T_max, codes, code_lens,
                                                                     entries_after);
    return cudaGetLastError();
  }
  // larger codebooks keep the table in global memory.  One warp per block: every sequence gets
  // its own SM while B <= 148, which keeps each dependent probe chain at the lowest latency the
  // memory system gives
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
