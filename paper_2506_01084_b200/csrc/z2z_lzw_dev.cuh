// Warp-level device functions of the LZW codebook, shared by the LZW kernels and by the fused
// decode-step update kernel.  All 32 lanes of a warp call these together for one sequence.
#pragma once
#include "z2z_common.cuh"

namespace z2z {

// Result of a warp probe.
struct Probe {
  int found;        // entry number, or -1
  int slot;         // if absent: first empty slot in probe order (-1: table full)
};

// First slot of the probe sequence of (prefix, token): linear probing from an even slot, so that
// a single thread can walk the sequence two slots (16 bytes) at a time and a warp can look at a
// window of kWindow consecutive slots at once.  Entries are never deleted and an insert takes the
// first empty slot of the sequence, so an empty slot proves that the key is absent.
__device__ __forceinline__ int probe_start(int n_slots, uint32_t prefix, uint32_t token) {
  return (int)(hash_pair(prefix, token) & (uint32_t)(n_slots - 1)) & ~1;
}

// All 32 lanes must call this together: lane l looks at slot (start + l) of the sequence.
__device__ __forceinline__ Probe warp_probe(const unsigned long long* __restrict__ table,
                                            int n_slots, uint32_t prefix, uint32_t token) {
  const int lane = threadIdx.x & 31;
  const unsigned long long key = pack_slot(prefix, token, 0) >> 16;
  int at = probe_start(n_slots, prefix, token);
  Probe r{-1, -1};
  for (int it = 0; it < n_slots / kWindow; ++it) {          // bounded: at most the whole table
    unsigned long long s = table[(at + lane) & (n_slots - 1)];
    unsigned hit = __ballot_sync(0xffffffffu, (s >> 16) == key && s != kEmptySlot);
    if (hit) {
      int src = __ffs(hit) - 1;
      unsigned long long v = __shfl_sync(0xffffffffu, s, src);
      r.found = (int)(v & 0xffffu);
      return r;
    }
    unsigned empty = __ballot_sync(0xffffffffu, s == kEmptySlot);
    if (empty) { r.slot = (at + __ffs(empty) - 1) & (n_slots - 1); return r; }
    at = (at + kWindow) & (n_slots - 1);
  }
  return r;
}

// Write entry k = phrase(w) ++ c.  Lanes 0..M-1 each write one constituent.
__device__ __forceinline__ void warp_write_entry(const CbView& cb, int b, int k, int w, int wlen,
                                                 int c) {
  const int lane = threadIdx.x & 31;
  int32_t* dst = cb.cons + ((size_t)b * cb.cap + k) * cb.M;
  if (lane < cb.M) {
    int v = -1;
    if (lane < wlen) v = (w < cb.V) ? w : cb.cons[((size_t)b * cb.cap + (w - cb.V)) * cb.M + lane];
    else if (lane == wlen) v = c;
    dst[lane] = v;
  }
  if (lane == 0) cb.len[(size_t)b * cb.cap + k] = (uint8_t)(wlen + 1);
}

// The part of a sequence's state that the update needs and that does not depend on the new code;
// a caller that still has to compute the code can load it ahead.  ptok: base token `lane` of the
// previous phrase (-1 beyond its length), so that writing a new entry needs no further load.
struct LzwPrev { int n, prev, plen, ptok; };
__device__ __forceinline__ LzwPrev warp_lzw_load(const CbView& cb, int b) {
  const int lane = threadIdx.x & 31;
  LzwPrev s;
  s.n = cb.n[b];
  s.prev = cb.prev[b];
  s.plen = 0;
  s.ptok = -1;
  if (s.prev >= 0) {
    if (s.prev < cb.V) {
      s.plen = 1;
      if (lane == 0) s.ptok = s.prev;
    } else {
      const size_t e = (size_t)b * cb.cap + (s.prev - cb.V);
      if (lane < cb.M) s.ptok = cb.cons[e * cb.M + lane];      // -1 padded behind the phrase
      s.plen = (int)cb.len[e];
    }
  }
  return s;
}
// Write entry k = phrase(prev) ++ c from the previous phrase's tokens held by the lanes; returns the
// token this lane wrote (-1: padding, or a lane beyond M).
__device__ __forceinline__ int warp_write_entry_from(const CbView& cb, int b, int k, const LzwPrev& s, int c) {
  const int lane = threadIdx.x & 31;
  int v = -1;
  if (lane < cb.M) {
    if (lane < s.plen) v = s.ptok;
    else if (lane == s.plen) v = c;
    cb.cons[((size_t)b * cb.cap + k) * cb.M + lane] = v;
  }
  if (lane == 0) cb.len[(size_t)b * cb.cap + k] = (uint8_t)(s.plen + 1);
  return v;
}
// Online update of sequence b with the newly selected code z (Figure 1; Section 2.3 step 10).
// Candidate entry = phrase(prev) ++ first(phrase(z)); returns the entry created, or -1.
// A code that names no existing (or about-to-exist) hypertoken raises BAD_TOKEN and leaves the
// sequence untouched.
// new_tok (optional): base token `lane` of the entry created (-1 if none / padding).
__device__ __forceinline__ int warp_lzw_step(const CbView& cb, int b, int z, const LzwPrev& s,
                                             int* new_tok = nullptr) {
  const int lane = threadIdx.x & 31;
  if (new_tok) *new_tok = -1;
  unsigned long long* table = cb.hash + (size_t)b * cb.n_slots;
  const int n = s.n;
  const int prev = s.prev;
  int created = -1;
  int st = 0;
  bool ok = !(z < 0 || z > cb.V + n);
  const int plen = s.plen;
  const bool self_ref = ok && (z == cb.V + n);       // the code this very step would create
  if (self_ref && !(prev >= 0 && plen < cb.M && n < cb.cap)) ok = false;
  if (ok) {
    int first;
    if (self_ref) first = prev < cb.V ? prev : cb.cons[((size_t)b * cb.cap + (prev - cb.V)) * cb.M];
    else first = z < cb.V ? z : cb.cons[((size_t)b * cb.cap + (z - cb.V)) * cb.M];
    if (prev >= 0 && plen < cb.M && n < cb.cap) {
      Probe p = warp_probe(table, cb.n_slots, (uint32_t)prev, (uint32_t)first);
      if (p.found < 0) {
        if (p.slot >= 0) {
          if (lane == 0) table[p.slot] = pack_slot((uint32_t)prev, (uint32_t)first, (uint32_t)n);
          const int wrote = warp_write_entry_from(cb, b, n, s, first);
          if (new_tok) *new_tok = wrote;
          created = n;
          if (n + 1 >= cb.cap) st |= Z2Z_ST_CAP_FROZEN;
        } else {
          st |= Z2Z_ST_TABLE_FULL;
        }
      } else if (self_ref) {
        ok = false;                                    // that phrase already has another id
      }
    }
  }
  if (lane == 0) {
    if (!ok) {
      st |= Z2Z_ST_BAD_TOKEN;                          // state stays as it was
    } else {
      cb.prev[b] = z;
      if (created >= 0) cb.n[b] = n + 1;
    }
    if (st) atomicOr(&cb.status[b], st);
  }
  return ok ? created : -1;
}

__device__ __forceinline__ int warp_lzw_step(const CbView& cb, int b, int z) {
  return warp_lzw_step(cb, b, z, warp_lzw_load(cb, b));
}

}  // namespace z2z
