// Shared declarations of the CUDA library: host handle, workspace plan, device-side views of the
// codebook, small numeric helpers.  Product code only; the CPU oracle shares nothing with this.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/z2z.h"

namespace z2z {

constexpr int kMaxM = 8;                 // maximum merge size supported
constexpr int kWindow = 32;              // consecutive hash slots one warp load looks at
constexpr uint64_t kEmptySlot = ~0ull;
constexpr float kLnEps = 1e-5f;

// ---------------------------------------------------------------------------------------------
// Device view of all per-sequence codebook state (lives in the caller's workspace).
//
// hash  [B, n_slots] u64   open addressing (linear probing from an even slot), key = (prefix
//                          code, next base token) -> entry number
//                          slot = prefix << 40 | token << 16 | entry ; all-ones = empty
// cons  [B, cap, M]  i32   base tokens of entry k, -1 padded  (the paper's codebook, Figure 1)
// len   [B, cap]     u8    number of base tokens of entry k
// n     [B]          i32   hypertokens so far
// prev  [B]          i32   last code seen by the online update (-1: none)
// status[B]          i32   Z2Z_ST_* bits
// n_emb [2, B]       i32   entries already embedded into E_h (row 0) / U_h (row 1)
// ---------------------------------------------------------------------------------------------
struct CbView {
  int V, M, cap, B, n_slots;
  unsigned long long* hash;
  int32_t* cons;
  uint8_t* len;
  int32_t* n;
  int32_t* prev;
  int32_t* status;
  int32_t* n_emb;
};

__host__ __device__ inline unsigned long long pack_slot(uint32_t prefix, uint32_t token,
                                                        uint32_t entry) {
  return ((unsigned long long)prefix << 40) | ((unsigned long long)token << 16) |
         (unsigned long long)entry;
}

// Multiplicative hash of the pair, upper bits (tables have at most 2^17 slots: bits 13..29).  The
// token's part does not depend on the running match, so a parser can compute it ahead.
__host__ __device__ inline uint32_t hash_token_part(uint32_t token) { return token * 0x85EBCA77u + 0x165667B1u; }
__host__ __device__ inline uint32_t hash_join(uint32_t prefix, uint32_t token_part) {
  return (prefix * 0x9E3779B1u ^ token_part) >> 13;
}
__host__ __device__ inline uint32_t hash_pair(uint32_t prefix, uint32_t token) {
  return hash_join(prefix, hash_token_part(token));
}

// CTA that owns unit u when U units are dealt to G CTAs as [floor(c U / G), floor((c+1) U / G)).
__host__ __device__ inline long long owner_of(long long u, long long U, long long G) {
  return ((u + 1) * G - 1) / U;
}

// ---------------------------------------------------------------------------------------------
// Workspace plan: byte offsets of every region inside the caller's workspace.
// ---------------------------------------------------------------------------------------------
struct WsPlan {
  int n_slots;
  int enc_chunk_entries;      // entries the encoder processes per pass
  int enc_rows;               // = enc_chunk_entries * M (rows padded to M per entry)
  size_t off_hash, off_cons, off_len, off_n, off_prev, off_status, off_n_emb, state_end;
  size_t off_entry_seq, off_entry_idx, off_entry_len, off_entry_tok, off_row_off, off_row_src, off_row_tok, off_entry_off, off_new_entry, off_sel;
  size_t off_X, off_A, off_QKV, off_H;            // fp32 encoder activations
  size_t off_Ahl, off_Hhl;                        // bf16 hi/lo activations (tensor-core path)
  size_t off_g1_X, off_g1_QKV, off_g1_Ahl, off_g1_Hhl;   // second encoder of the decode step
  size_t off_words;                               // device words: [0] kernel error, [1] logits tiles
  size_t off_part, part_bytes;                    // fp32 GEMM results of the hyper-encoder passes
  size_t off_lpart, lpart_bytes;                  // logits partial reductions
  size_t off_plan, plan_bytes;                    // per-row-tile plan of the prompt-scoring logits kernel
  size_t off_step_out;                            // small per-step outputs
  size_t total;
};

constexpr int kLogitRowChunk = 8192;              // rows per logits launch (larger N loops)
constexpr int kLogitPartRows = 1 << 20;           // partial-reduction slots (rows x groups), 32 bytes each
constexpr int kPrefillPlanTiles = 1 << 14;        // 256-row tiles one prompt-scoring launch may have

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline WsPlan plan_workspace(const z2z_config& c) {
  WsPlan p{};
  int ns = 64;
  while (ns < 2 * c.cap) ns <<= 1;
  p.n_slots = ns;
  long long all = (long long)c.B * (long long)c.cap;
  int chunk = (int)(all < 1024 ? (all < c.B ? c.B : all) : 1024);
  if (chunk < c.B) chunk = c.B;
  if (chunk < 1) chunk = 1;
  p.enc_chunk_entries = chunk;
  p.enc_rows = chunk * c.M;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes, 256); return r; };
  p.off_hash = take((size_t)c.B * ns * 8);
  p.off_cons = take((size_t)c.B * c.cap * c.M * 4);
  p.off_len = take((size_t)c.B * c.cap);
  p.off_n = take((size_t)c.B * 4);
  p.off_prev = take((size_t)c.B * 4);
  p.off_status = take((size_t)c.B * 4);
  p.off_n_emb = take((size_t)2 * c.B * 4);
  p.state_end = o;
  p.off_entry_seq = take((size_t)chunk * 4);
  p.off_entry_idx = take((size_t)chunk * 4);
  p.off_entry_len = take((size_t)chunk * 4);
  p.off_entry_tok = take((size_t)chunk * c.M * 4);
  p.off_row_off = take((size_t)(chunk + 1) * 4);
  p.off_row_src = take((size_t)chunk * c.M * 4);
  p.off_row_tok = take((size_t)chunk * c.M * 4);
  p.off_entry_off = take((size_t)(c.B + 2) * 4);
  p.off_new_entry = take((size_t)c.B * 4);
  p.off_sel = take((size_t)c.B * 4 * 4);
  size_t R = (size_t)p.enc_rows;
  size_t dff = (size_t)(c.enc_dff > 0 ? c.enc_dff : 0);
  size_t wide = dff > (size_t)3 * c.d ? dff : (size_t)3 * c.d;
  // encoder scratch: one full set for prefill passes (group 0) and a decode-sized set (B entries)
  // for the second encoder of the decode step (group 1)
  size_t Rp = (R + 127) / 128 * 128 + 128;
  size_t R1 = ((size_t)c.B * c.M + 127) / 128 * 128 + 128;
  p.off_X = take(Rp * c.d * 4);
  p.off_A = take(Rp * c.d * 4);
  p.off_QKV = take(Rp * 3 * c.d * 4);
  p.off_H = take(Rp * dff * 4);
  p.off_Ahl = take(2 * Rp * c.d * 2);
  p.off_Hhl = take(2 * Rp * dff * 2);
  p.off_g1_X = take(R1 * c.d * 4);
  p.off_g1_QKV = take(R1 * 3 * c.d * 4);
  p.off_g1_Ahl = take(2 * R1 * c.d * 2);
  p.off_g1_Hhl = take(2 * R1 * dff * 2);
  p.part_bytes = ((Rp / 128) * 2 * ((wide + 127) / 128) + 256) * (size_t)65536;
  p.off_part = take(p.part_bytes);
  p.off_words = take(256);
  p.lpart_bytes = (size_t)kLogitPartRows * 32;
  p.off_lpart = take(p.lpart_bytes);
  p.plan_bytes = (size_t)kPrefillPlanTiles * 3 * 4;
  p.off_plan = take(p.plan_bytes);
  p.off_step_out = take((size_t)c.B * 64);
  p.total = o;
  return p;
}

// ---------------------------------------------------------------------------------------------
// Numeric helpers
// ---------------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) {
  return __bfloat162float(x);
}
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3",
// SC'11), written from the published round function.
struct Philox4 { uint32_t x, y, z, w; };
__device__ __forceinline__ Philox4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2,
                                                 uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return Philox4{c0, c1, c2, c3};
}
// Gumbel noise for logit column `col` of `row` at `step`: g = -log(-log u),
// u = ((x >> 9) + 0.5) * 2^-23 in (0, 1), exact in fp32.
__device__ __forceinline__ float gumbel_from_word(uint32_t x) {
  float u = ((float)(x >> 9) + 0.5f) * 1.1920928955078125e-07f;
  return -logf(-logf(u));
}
__device__ __forceinline__ uint32_t philox_word(const Philox4& p, int i) {
  return i == 0 ? p.x : (i == 1 ? p.y : (i == 2 ? p.z : p.w));
}

// Running reduction over logit columns: max / sum-exp / argmax (lowest index on ties) and the
// same for Gumbel-perturbed scores.
struct RowRed {
  float m, s; int idx; float gm; int gidx;
  __device__ __forceinline__ void init() { m = -INFINITY; s = 0.f; idx = 0x7fffffff; gm = -INFINITY; gidx = 0x7fffffff; }
  __device__ __forceinline__ void add(float l, int col) {
    if (l > m) { s = s * __expf(m - l) + 1.f; m = l; idx = col; }
    else { s += __expf(l - m); if (l == m && col < idx) idx = col; }
  }
  __device__ __forceinline__ void add_score(float sc, int col) {
    if (sc > gm || (sc == gm && col < gidx)) { gm = sc; gidx = col; }
  }
  __device__ __forceinline__ void merge(const RowRed& o) {
    if (o.m > m) { s = s * __expf(m - o.m) + o.s; m = o.m; idx = o.idx; }
    else if (o.m == m) { s += o.s; if (o.idx < idx) idx = o.idx; }
    else if (o.m > -INFINITY) { s += o.s * __expf(o.m - m); }
    if (o.gm > gm || (o.gm == gm && o.gidx < gidx)) { gm = o.gm; gidx = o.gidx; }
  }
};

}  // namespace z2z
