// LZW decompression on the device (Section 2.1, property 2: the compressed stream decodes
// without a shipped codebook; Section 2.3 steps 11-12: the generated hypertoken stream is turned
// back into base tokens).
//
// Two kernels:
//   k_lzw_replay  (k_lzw_replay_smem while the table fits shared memory) rebuilds (or continues)
//                 each sequence's codebook from the code stream alone by
//                 replaying the online update once per code.  A dependent chain per sequence, so
//                 one warp owns one sequence, keeps the running state in registers and prefetches
//                 (first token, length) of the next 32 codes in one coalesced pass; an entry that
//                 was created inside the current batch of 32 is re-read when its code comes up.
//   k_lzw_expand  turns codes into base tokens with the codebook that is resident: an exclusive
//                 scan of phrase lengths gives every code its output offset, each thread then
//                 copies one phrase.  Blocks are (sequence, chunk of codes); a block finds its
//                 start offset by summing the lengths of the codes before its chunk.
#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_lzw_dev.cuh"

namespace z2z {

namespace {

constexpr int kExpandThreads = 256;
constexpr int kExpandChunk = 2048;          // codes per block

__device__ __forceinline__ int entry_first(const CbView& cb, int b, int code) {
  return code < cb.V ? code : cb.cons[((size_t)b * cb.cap + (code - cb.V)) * cb.M];
}
__device__ __forceinline__ int entry_len(const CbView& cb, int b, int code) {
  return code < cb.V ? 1 : (int)cb.len[(size_t)b * cb.cap + (code - cb.V)];
}

}  // namespace

// Replays the online update (Figure 1; Section 2.3 step 10) for codes[b][0 .. code_lens[b]).
// n_valid[b] = number of codes accepted; replay of a sequence stops at the first code that names
// no hypertoken (BAD_TOKEN; the state is the one after the last accepted code).
__global__ void __launch_bounds__(32) k_lzw_replay(CbView cb, const int32_t* __restrict__ codes,
                                                   const int32_t* __restrict__ code_lens,
                                                   int Tc_max, int32_t* __restrict__ n_valid) {
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x;
  if (b >= cb.B) return;
  unsigned long long* table = cb.hash + (size_t)b * cb.n_slots;
  int Tc = code_lens ? code_lens[b] : Tc_max;
  Tc = Tc < 0 ? 0 : (Tc > Tc_max ? Tc_max : Tc);
  const int32_t* zs = codes + (size_t)b * Tc_max;
  int n = cb.n[b];
  int prev = cb.prev[b];
  int plen = 0, pfirst = -1;
  if (prev >= 0) { plen = entry_len(cb, b, prev); pfirst = entry_first(cb, b, prev); }
  int st = 0, valid = 0;
  bool bad = false;
  for (int base = 0; base < Tc && !bad; base += 32) {
    const int cnt = Tc - base < 32 ? Tc - base : 32;
    const int n_batch = n;                       // entries below this index exist for the whole batch
    int z_mine = -1, f_mine = -1, l_mine = 0;
    if (lane < cnt) {
      z_mine = zs[base + lane];
      if (z_mine >= 0 && z_mine < cb.V + n_batch) {
        f_mine = entry_first(cb, b, z_mine);
        l_mine = entry_len(cb, b, z_mine);
      }
    }
    for (int i = 0; i < cnt; ++i) {
      const int z = __shfl_sync(0xffffffffu, z_mine, i);
      int f = __shfl_sync(0xffffffffu, f_mine, i);
      int l = __shfl_sync(0xffffffffu, l_mine, i);
      if (z < 0 || z > cb.V + n) { bad = true; break; }
      const bool self_ref = (z == cb.V + n);     // the entry this very code creates
      const bool can = prev >= 0 && plen < cb.M && n < cb.cap;
      if (self_ref) {
        if (!can) { bad = true; break; }
        f = pfirst; l = plen + 1;
      } else if (z >= cb.V + n_batch) {          // created earlier in this batch: read it now
        f = entry_first(cb, b, z);
        l = entry_len(cb, b, z);
      }
      if (can) {
        Probe p = warp_probe(table, cb.n_slots, (uint32_t)prev, (uint32_t)f);
        if (p.found < 0) {
          if (p.slot >= 0) {
            if (lane == 0) table[p.slot] = pack_slot((uint32_t)prev, (uint32_t)f, (uint32_t)n);
            warp_write_entry(cb, b, n, prev, plen, f);
            ++n;
            if (n >= cb.cap) st |= Z2Z_ST_CAP_FROZEN;
            __syncwarp();                        // slot and entry visible to the probes that follow
          } else {
            st |= Z2Z_ST_TABLE_FULL;
          }
        } else if (self_ref) {                   // that phrase already has another id
          bad = true; break;
        }
      }
      prev = z; plen = l; pfirst = f;
      ++valid;
    }
  }
  if (bad) st |= Z2Z_ST_BAD_TOKEN;
  if (lane == 0) {
    cb.n[b] = n;
    if (valid > 0) cb.prev[b] = prev;
    n_valid[b] = valid;
    if (st) atomicOr(&cb.status[b], st);
  }
}

// The same replay with the sequence's hash table in shared memory and ONE thread walking the
// probe sequences (as the prompt parse does: a chain that a single warp executes is paced by the
// instructions it issues, and a warp-wide probe of a table in global memory costs a round trip to
// L2 per code).  Beside the table the CTA keeps (first token, length) of every entry and the slot
// each new entry went to: the slot holds (prefix code, last token), which is all that is needed
// to write the entry's constituent row afterwards, by all threads, walking back through the
// prefixes (at most M - 1 steps).
constexpr int kReplaySmemThreads = 128;
constexpr size_t kReplaySmemMaxBytes = 200 * 1024;
__host__ __device__ inline size_t replay_smem_bytes(int n_slots, int cap) {
  return (size_t)n_slots * 8 + (size_t)cap * 4 + (size_t)cap * 2 + 16;
}

__global__ void __launch_bounds__(kReplaySmemThreads) k_lzw_replay_smem(CbView cb, const int32_t* __restrict__ codes,
                                                                        const int32_t* __restrict__ code_lens,
                                                                        int Tc_max, int32_t* __restrict__ n_valid) {
  extern __shared__ __align__(16) unsigned long long s_table[];
  uint32_t* const s_fl = reinterpret_cast<uint32_t*>(s_table + cb.n_slots);          // first token << 8 | length
  uint16_t* const s_slot = reinterpret_cast<uint16_t*>(s_fl + cb.cap);               // slot of each new entry
  __shared__ int s_code[64];
  __shared__ int s_n0, s_n1;
  const int lane = threadIdx.x & 31;
  const int b = blockIdx.x;
  const int V = cb.V, M = cb.M, cap = cb.cap;
  unsigned long long* table = cb.hash + (size_t)b * cb.n_slots;
  int32_t* const cons = cb.cons + (size_t)b * cap * M;
  uint8_t* const len = cb.len + (size_t)b * cap;
  const int n_start = cb.n[b];
  for (int i = threadIdx.x; i < cb.n_slots; i += blockDim.x) s_table[i] = table[i];
  for (int k = threadIdx.x; k < n_start; k += blockDim.x) s_fl[k] = ((uint32_t)cons[(size_t)k * M] << 8) | len[k];
  int Tc = code_lens ? code_lens[b] : Tc_max;
  Tc = Tc < 0 ? 0 : (Tc > Tc_max ? Tc_max : Tc);
  const int32_t* zs = codes + (size_t)b * Tc_max;
  __syncthreads();
  if (threadIdx.x < 32) {
    const uint32_t pair_mask = (uint32_t)(cb.n_slots - 1) & ~1u;
    const uint2* const slots = reinterpret_cast<const uint2*>(s_table);
    int n = n_start;
    int prev = cb.prev[b];
    int plen = 0, pfirst = -1;
    if (prev >= 0) {
      if (prev < V) { plen = 1; pfirst = prev; }
      else { const uint32_t fl = s_fl[prev - V]; plen = (int)(fl & 255u); pfirst = (int)(fl >> 8); }
    }
    int st = 0, valid = 0;
    bool bad = false;
    int ahead = lane < Tc ? zs[lane] : -1;           // codes of the batch after the current one
    for (int base = 0; base < Tc && !bad; base += 32) {
      s_code[(base & 32) + lane] = ahead;
      ahead = base + 32 + lane < Tc ? zs[base + 32 + lane] : -1;
      __syncwarp();
      if (lane == 0) {
        const int cnt = Tc - base < 32 ? Tc - base : 32;
        for (int i = 0; i < cnt; ++i) {
          const int z = s_code[(base + i) & 63];
          if (z < 0 || z > V + n) { bad = true; break; }
          const bool self_ref = (z == V + n);        // the entry this very code creates
          const bool can = prev >= 0 && plen < M && n < cap;
          int f, l;
          if (self_ref) {
            if (!can) { bad = true; break; }
            f = pfirst; l = plen + 1;
          } else if (z < V) {
            f = z; l = 1;
          } else {
            const uint32_t fl = s_fl[z - V];
            f = (int)(fl >> 8); l = (int)(fl & 255u);
          }
          if (can) {
            const uint32_t key_hi = ((uint32_t)prev << 8) | ((uint32_t)f >> 16), key_lo = (uint32_t)f & 0xffffu;
            uint32_t at = hash_pair((uint32_t)prev, (uint32_t)f) & pair_mask;
            int found = -1, slot = -1;
            for (int it = 0; it < cb.n_slots; it += 2) {   // bounded: at most the whole table
              const uint4 pr = *reinterpret_cast<const uint4*>(&slots[at]);      // slots at, at + 1: {lo, hi, lo, hi}
              if (pr.y == key_hi && (pr.x >> 16) == key_lo) { found = (int)(pr.x & 0xffffu); break; }
              if (pr.y == 0xffffffffu) { slot = (int)at; break; }
              if (pr.w == key_hi && (pr.z >> 16) == key_lo) { found = (int)(pr.z & 0xffffu); break; }
              if (pr.w == 0xffffffffu) { slot = (int)at + 1; break; }
              at = (at + 2) & pair_mask;
            }
            if (found < 0) {
              if (slot >= 0) {
                reinterpret_cast<uint2*>(s_table)[slot] = make_uint2((key_lo << 16) | (uint32_t)n, key_hi);
                s_fl[n] = ((uint32_t)pfirst << 8) | (uint32_t)(plen + 1);
                s_slot[n] = (uint16_t)slot;
                ++n;
                if (n >= cap) st |= Z2Z_ST_CAP_FROZEN;
              } else {
                st |= Z2Z_ST_TABLE_FULL;
              }
            } else if (self_ref) {                   // that phrase already has another id
              bad = true; break;
            }
          }
          prev = z; plen = l; pfirst = f;
          ++valid;
        }
      }
      bad = __shfl_sync(0xffffffffu, bad ? 1 : 0, 0) != 0;
    }
    if (lane == 0) {
      if (bad) st |= Z2Z_ST_BAD_TOKEN;
      cb.n[b] = n;
      if (valid > 0) cb.prev[b] = prev;
      n_valid[b] = valid;
      if (st) atomicOr(&cb.status[b], st);
      s_n0 = n_start; s_n1 = n;
    }
  }
  __syncthreads();
  // constituent rows and lengths of the entries created here
  for (int e = s_n0 + threadIdx.x; e < s_n1; e += blockDim.x) {
    int tok[kMaxM];
#pragma unroll
    for (int j = 0; j < kMaxM; ++j) tok[j] = -1;
    const int L = (int)(s_fl[e] & 255u);
    int pos = L - 1, cur = e;
    for (int hop = 0; hop < kMaxM && pos >= 0; ++hop) {          // bounded: a phrase has at most M tokens
      const unsigned long long slot = s_table[s_slot[cur]];
      const int last = (int)((slot >> 16) & 0xffffffu), p = (int)(slot >> 40);
      tok[pos--] = last;
      if (pos < 0) break;                                        // (cannot happen: a prefix remains)
      if (p < V) { tok[pos--] = p; break; }
      const int k = p - V;
      if (k < s_n0) {                                            // an entry from before this call: its row is final
        for (int j = 0; j <= pos; ++j) tok[j] = cons[(size_t)k * M + j];
        pos = -1;
        break;
      }
      cur = k;
    }
    for (int j = 0; j < M; ++j) cons[(size_t)e * M + j] = tok[j];
    len[e] = (uint8_t)L;
  }
  for (int i = threadIdx.x; i < cb.n_slots; i += blockDim.x) table[i] = s_table[i];
}

// Block-wide exclusive scan of one int per thread (kExpandThreads threads); returns the
// thread's exclusive prefix, *total = sum over the block.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();                               // warp_sums free to overwrite
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  int before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < kExpandThreads / 32; ++w) {
    int s = warp_sums[w];
    if (w < warp) before += s;
    all += s;
  }
  *total = all;
  return before + inc - v;
}

// Codes -> base tokens with the resident codebook.  grid = (chunks, B).  limit[b] (or code_lens,
// or Tc_max) bounds the codes of sequence b; expansion stops at the first code that is not below
// V + n_b (BAD_TOKEN) and at T_out_max tokens (OUTPUT_TRUNCATED; token_lens[b] is then T_out_max).
__global__ void __launch_bounds__(kExpandThreads) k_lzw_expand(
    CbView cb, const int32_t* __restrict__ codes, const int32_t* __restrict__ code_lens,
    const int32_t* __restrict__ limit, int Tc_max, int32_t* __restrict__ tokens,
    int32_t* __restrict__ token_lens, int T_out_max) {
  __shared__ int warp_sums[kExpandThreads / 32];
  __shared__ int s_first_bad;
  const int b = blockIdx.y;
  const int tid = threadIdx.x;
  int Tc = code_lens ? code_lens[b] : Tc_max;
  Tc = Tc < 0 ? 0 : (Tc > Tc_max ? Tc_max : Tc);
  const int lim = limit ? (limit[b] < Tc ? limit[b] : Tc) : Tc;
  const int n = cb.n[b];
  const int32_t* zs = codes + (size_t)b * Tc_max;
  const int lo = blockIdx.x * kExpandChunk;
  if (lo > lim) return;                          // the block that holds position `lim` reports the length
  const int hi = lo + kExpandChunk < lim ? lo + kExpandChunk : lim;
  if (tid == 0) s_first_bad = 0x7fffffff;
  __syncthreads();
  // codes before this chunk: total length and validity
  int before = 0;
  for (int i = tid; i < lo; i += kExpandThreads) {
    const int z = zs[i];
    if (z < 0 || z >= cb.V + n) atomicMin(&s_first_bad, i);
    else before += entry_len(cb, b, z);
  }
  int total = 0;
  block_exclusive_scan(before, warp_sums, &total);
  __syncthreads();
  if (s_first_bad != 0x7fffffff) return;         // an earlier block holds the end of the valid prefix
  int offset = total;
  int32_t* out = tokens + (size_t)b * T_out_max;
  bool truncated = false;
  int end_pos = hi;                              // first position this block does not expand
  for (int c0 = lo; c0 < hi; c0 += kExpandThreads) {
    const int i = c0 + tid;
    int z = -1, l = 0;
    if (i < hi) {
      z = zs[i];
      if (z < 0 || z >= cb.V + n) { atomicMin(&s_first_bad, i); z = -1; }
      else l = entry_len(cb, b, z);
    }
    __syncthreads();
    const int first_bad = s_first_bad;
    if (i >= first_bad) l = 0;                   // nothing at or after the first bad code is written
    int sum = 0;
    const int ex = block_exclusive_scan(l, warp_sums, &sum);
    if (l > 0) {
      const int at = offset + ex;
      if (z < cb.V) {
        if (at < T_out_max) out[at] = z; else truncated = true;
      } else {
        const int32_t* src = cb.cons + ((size_t)b * cb.cap + (z - cb.V)) * cb.M;
        for (int j = 0; j < l; ++j) {
          if (at + j < T_out_max) out[at + j] = src[j]; else truncated = true;
        }
      }
    }
    offset += sum;
    if (first_bad != 0x7fffffff) { end_pos = first_bad; break; }
  }
  const int any_trunc = __syncthreads_or(truncated ? 1 : 0);
  const bool bad = end_pos < hi || (s_first_bad != 0x7fffffff);
  // exactly one block owns the end of the expanded prefix: the one where expansion stopped at a
  // bad code, or the one whose chunk holds position `lim`
  const bool owns_end = bad || (lim < lo + kExpandChunk);
  if (tid == 0) {
    int st = 0;
    if (any_trunc) st |= Z2Z_ST_OUTPUT_TRUNCATED;
    if (bad) st |= Z2Z_ST_BAD_TOKEN;           // (a replay that stopped early has set it already)
    if (st) atomicOr(&cb.status[b], st);
    if (owns_end) token_lens[b] = offset < T_out_max ? offset : T_out_max;
  }
}

cudaError_t launch_lzw_decode(const CbView& cb, const int32_t* codes, const int32_t* code_lens,
                              int Tc_max, int replay, int32_t* n_valid, int32_t* tokens,
                              int32_t* token_lens, int T_out_max, cudaStream_t s) {
  if (replay) {
    const size_t smem = replay_smem_bytes(cb.n_slots, cb.cap);
    cudaError_t e;
    if (smem <= kReplaySmemMaxBytes && cb.n_slots <= 65536) {    // (a slot number fits 16 bits)
      e = cudaFuncSetAttribute(k_lzw_replay_smem, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return e;
      k_lzw_replay_smem<<<cb.B, kReplaySmemThreads, smem, s>>>(cb, codes, code_lens, Tc_max, n_valid);
    } else {
      k_lzw_replay<<<cb.B, 32, 0, s>>>(cb, codes, code_lens, Tc_max, n_valid);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  dim3 grid(Tc_max / kExpandChunk + 1, cb.B);
  k_lzw_expand<<<grid, kExpandThreads, 0, s>>>(cb, codes, code_lens, replay ? n_valid : nullptr,
                                               Tc_max, tokens, token_lens, T_out_max);
  return cudaGetLastError();
}

}  // namespace z2z
