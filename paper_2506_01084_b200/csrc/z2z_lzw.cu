// LZW codebook kernels: session reset, prompt compression, online update.
//
// One warp owns one sequence.  The codebook of a sequence is an open-addressing hash table in
// global memory keyed by (prefix code, next base token), probed linearly from an even slot; a warp
// probe is one coalesced 256-byte load of 32 consecutive slots followed by a ballot.  Entries are
// never deleted and an insert always takes the first empty slot in probe order, so an empty slot
// proves absence.
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
// kernel (codebooks of up to 12800 entries: at most 25600 slots, 200 KB).  The parse is a
// dependent chain of one probe per token, and a chain that a single warp executes is paced by the
// number of instructions it issues per token (about one every four to five cycles), not by memory.
// A warp-wide probe spends most of them on warp primitives (broadcast, ballot, shuffle: about
// 240 ns per token with the table in shared memory, 290 with the table in global memory); here
// ONE thread walks the probe sequence two slots (one 16-byte shared-memory load) at a time, which
// at a load factor of at most one half ends after one or two loads: 165-195 ns per token.  The
// rest of warp 0 stages the tokens (the batch after the one being parsed is already in flight)
// and the other warps move the table in and out.  A new entry is the last wlen + 1 input tokens,
// so the chain only records where the phrase starts and how long it is (one word in the first
// constituent slot, one length byte); all threads expand the records into constituent rows from
// the token array after the parse.
constexpr int kEncodeSmemThreads = 128;
constexpr size_t kEncodeSmemMaxBytes = 200 * 1024;

__global__ void __launch_bounds__(kEncodeSmemThreads) k_lzw_encode_smem(CbView cb, const int32_t* __restrict__ tokens,
                                                                        const int32_t* __restrict__ lens, int T_max,
                                                                        int32_t* __restrict__ codes,
                                                                        int32_t* __restrict__ code_lens,
                                                                        int32_t* __restrict__ entries_after) {
  extern __shared__ __align__(16) unsigned long long s_table[];
  __shared__ int4 s_tok[64];                         // two batches of 32 tokens: {c, hash part, c >> 16, c & 0xffff}
  __shared__ int s_n0, s_n1;                         // entries before / after this call
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x;
  unsigned long long* table = cb.hash + (size_t)b * cb.n_slots;
  for (int i = threadIdx.x; i < cb.n_slots; i += blockDim.x) s_table[i] = table[i];
  int T = lens ? lens[b] : T_max;
  T = T < 0 ? 0 : (T > T_max ? T_max : T);
  const int32_t* x = tokens + (size_t)b * T_max;
  int32_t* const cons = cb.cons + (size_t)b * cb.cap * cb.M;
  uint8_t* const len = cb.len + (size_t)b * cb.cap;
  __syncthreads();
  if (threadIdx.x < 32) {
    int32_t* out = codes + (size_t)b * T_max;
    int32_t* aft = entries_after ? entries_after + (size_t)b * T_max : nullptr;
    const int V = cb.V, M = cb.M, cap = cb.cap;
    const uint32_t pair_mask = (uint32_t)(cb.n_slots - 1) & ~1u;
    // a slot as two words: hi = prefix << 8 | token >> 16, lo = token << 16 | entry (all-ones hi = empty)
    const uint2* const slots = reinterpret_cast<const uint2*>(s_table);
    int n = cb.n[b];
    if (lane == 0) s_n0 = n;
    int st = 0;
    int w = -1, wlen = 0, n_out = 0;
    int ahead = lane < T ? x[lane] : 0;              // tokens of the batch after the current one
    for (int base = 0; base < T; base += 32) {
      int mine = ahead;
      ahead = base + 32 + lane < T ? x[base + 32 + lane] : 0;
      if ((unsigned)mine >= (unsigned)V) { if (base + lane < T) st |= Z2Z_ST_BAD_TOKEN; mine = 0; }   // not a base token
      s_tok[(base & 32) + lane] = make_int4(mine, (int)hash_token_part((uint32_t)mine), mine >> 16, mine & 0xffff);
      __syncwarp();
      if (lane == 0) {
        const int cnt = T - base < 32 ? T - base : 32;
        int4 t_next = s_tok[base & 63];
        for (int i = 0; i < cnt; ++i) {
          const int4 t = t_next;
          t_next = s_tok[(base + i + 1) & 63];         // off the chain: ready before the next probe needs it
          const int c = t.x;
          if (wlen == 0) { w = c; wlen = 1; continue; }
          int slot = -1;
          const uint32_t key_hi = ((uint32_t)w << 8) | (uint32_t)t.z;
          if (wlen < M) {
            uint32_t at = hash_join((uint32_t)w, (uint32_t)t.y) & pair_mask;
            int found = -1;
            for (int it = 0; it < cb.n_slots; it += 2) {   // bounded: at most the whole table
              const uint4 pr = *reinterpret_cast<const uint4*>(&slots[at]);      // slots at, at + 1: {lo, hi, lo, hi}
              if (pr.y == key_hi && (pr.x >> 16) == (uint32_t)t.w) { found = (int)(pr.x & 0xffffu); break; }
              if (pr.y == 0xffffffffu) { slot = (int)at; break; }              // (no prefix is 2^24 - 1)
              if (pr.w == key_hi && (pr.z >> 16) == (uint32_t)t.w) { found = (int)(pr.z & 0xffffu); break; }
              if (pr.w == 0xffffffffu) { slot = (int)at + 1; break; }
              at = (at + 2) & pair_mask;
            }
            if (found >= 0) { w = V + found; ++wlen; continue; }          // match grows
          }
          // longest match ends: emit it, then remember (w ++ c) if allowed
          out[n_out] = w;
          if (wlen < M && n < cap) {
            if (slot >= 0) {
              reinterpret_cast<uint2*>(s_table)[slot] = make_uint2(((uint32_t)t.w << 16) | (uint32_t)n, key_hi);
              cons[(size_t)n * M] = base + i - wlen;                       // where the phrase starts
              len[n] = (uint8_t)(wlen + 1);
              ++n;
              if (n >= cap) st |= Z2Z_ST_CAP_FROZEN;
            } else {
              st |= Z2Z_ST_TABLE_FULL;
            }
          }
          if (aft) aft[n_out] = n;
          ++n_out;
          w = c; wlen = 1;
        }
      }
      __syncwarp();                                  // the other half of s_tok may be rewritten
    }
    if (lane == 0) {
      if (wlen > 0) {                                // final flush creates no entry
        out[n_out] = w;
        if (aft) aft[n_out] = n;
        ++n_out;
      }
      code_lens[b] = n_out;
      cb.n[b] = n;
      if (n_out > 0) cb.prev[b] = w;
      s_n1 = n;
    }
    st = __reduce_or_sync(0xffffffffu, st);           // BAD_TOKEN is found per lane
    if (lane == 0 && st) atomicOr(&cb.status[b], st);
  }
  __syncthreads();
  // constituent rows of the entries created here: tokens [start, start + len), -1 padded
  for (int e = s_n0 + threadIdx.x; e < s_n1; e += blockDim.x) {
    const int start = cons[(size_t)e * cb.M];
    const int L = len[e];
    for (int j = 0; j < cb.M; ++j) {
      int v = -1;
      if (j < L) { v = x[start + j]; if ((unsigned)v >= (unsigned)cb.V) v = 0; }
      cons[(size_t)e * cb.M + j] = v;
    }
  }
  for (int i = threadIdx.x; i < cb.n_slots; i += blockDim.x) table[i] = s_table[i];
}

// Online update with one new code per sequence (Figure 1; Section 2.3 step 10).
// none_sits_out: a code equal to Z2Z_CODE_NONE marks a sequence that takes no part in this step.
__global__ void __launch_bounds__(128) k_lzw_step(CbView cb, const int32_t* __restrict__ new_codes,
                                                  const uint8_t* __restrict__ active, int none_sits_out,
                                                  int32_t* __restrict__ new_entry) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (b >= cb.B) return;
  if ((active && !active[b]) || (none_sits_out && new_codes[b] == Z2Z_CODE_NONE)) {
    if (lane == 0 && new_entry) new_entry[b] = -1;
    return;
  }
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
                            int none_sits_out, int32_t* new_entry, cudaStream_t s) {
  int wpb = 4;
  k_lzw_step<<<(cb.B + wpb - 1) / wpb, wpb * 32, 0, s>>>(cb, new_codes, active, none_sits_out, new_entry);
  return cudaGetLastError();
}

}  // namespace z2z
