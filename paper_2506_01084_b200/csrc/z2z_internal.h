// Internal launch wrappers shared between the translation units of the library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "z2z_common.cuh"
#include "z2z_prof.h"

namespace z2z {

// Launch with programmatic stream serialization: the kernel may begin (up to its pdl_wait())
// while the previous kernel of the stream is still running.  Every kernel launched this way
// calls pdl_wait() before it reads what earlier kernels wrote and before it writes anything.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                              Args&&... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(static_cast<Args&&>(args))...);
}

// ---- z2z_api.cu ------------------------------------------------------------------------------
void set_last_error(const char* msg);      // text returned by z2z_last_error on this thread

// ---- z2z_lzw.cu ------------------------------------------------------------------------------
cudaError_t launch_codebook_clear(const CbView& cb, cudaStream_t s);
cudaError_t launch_lzw_encode(const CbView& cb, const int32_t* tokens, const int32_t* lens,
                              int T_max, int32_t* codes, int32_t* code_lens,
                              int32_t* entries_after, cudaStream_t s);
cudaError_t launch_lzw_decode(const CbView& cb, const int32_t* codes, const int32_t* code_lens,
                              int Tc_max, int replay, int32_t* n_valid, int32_t* tokens,
                              int32_t* token_lens, int T_out_max, cudaStream_t s);
cudaError_t launch_embed_lookup(const CbView& cb, const int32_t* codes, int N,
                                const int32_t* row_seq, const void* WE, const void* Eh, void* out,
                                int d, int elem_bytes, cudaStream_t s);
cudaError_t launch_lzw_step(const CbView& cb, const int32_t* new_codes, const uint8_t* active,
                            int none_sits_out, int32_t* new_entry, cudaStream_t s);

// ---- z2z_encoder.cu --------------------------------------------------------------------------
// Work list of one encoder pass: up to `chunk` entries, entry e -> (sequence, entry number).
struct EntryList {
  int32_t* seq;       // [chunk]  sequence of entry e, -1 = unused slot
  int32_t* idx;       // [chunk]  entry number within the sequence
  int32_t* len;       // [chunk]  base tokens of the entry, 0 for an unused slot
  int32_t* tok;       // [chunk * M]  base token of each row of the entry, -1 for padding rows
  int32_t* row_off;   // [chunk + 1]  tensor-core passes: first packed row of each entry; the row total sits
                      //              behind the last entry slot of the pass
  int32_t* row_src;   // [chunk * M]  tensor-core passes: packed row -> entry * M + position
  int32_t* row_tok;   // [chunk * M]  tensor-core passes: base token of each packed row
  int32_t* off;       // [B + 2]  exclusive prefix sum of per-sequence counts, then the total
  int chunk;
};
struct EncoderArgs {
  int d, dff, heads, layers, M;
  int dtype;
  const void* table;            // [V, d]
  const void* const* w;         // host array of device pointers, ABI order
  const void* const* w_half;    // or NULL: fp16 copies of the linear-layer weights, same order (prompt-sized passes)
  void* cache;                  // [B, cap, d] dtype
  float* cache_f32;             // optional
  float *X, *A, *QKV, *H;       // fp32 scratch, rows = chunk * M
  __nv_bfloat16 *Ahl, *Hhl;     // bf16 hi/lo scratch for the tensor-core path
  float* part;                  // fp32 GEMM results [groups][rows][J], zero between GEMMs
  size_t part_bytes;
  int entries;                  // host bound on the entries of this pass (<= chunk)
  int* err;                     // device error word of the tensor-core kernels
};
bool encoder_tc_supported(int d, int dff, int dtype, int heads, int M);
size_t encoder_half_bytes(int d, int dff, int layers);
bool encoder_pass_is_prompt_sized(int entries, int chunk, int M);
cudaError_t convert_encoder_weights_to_half(const void* const* w, int d, int dff, int layers, void* scratch,
                                            const void** half_ptrs, int* err_word, Prof* prof, cudaStream_t s);
bool logits_tc_supported(int d, int dtype);
// Two encoders (embedding side, unembedding side) run through the same launches.
// rows_mapped: the packed-row map of the work list (row_off, row_src, row_tok) is already there.
cudaError_t run_encoder_pass_tc(const CbView& cb, const EncoderArgs* groups, int n_groups,
                                const EntryList& el, bool rows_mapped, Prof* prof, cudaStream_t s);
// Per-sequence ranges from (first, count) arrays, or "everything since the last call" when NULL.
cudaError_t launch_entry_offsets(const CbView& cb, int which, const int32_t* first,
                                 const int32_t* count, const EntryList& el, cudaStream_t s);
// Ranges of the decode step: the entry created by this step's LZW update, if any.
cudaError_t launch_entry_offsets_from_new(const CbView& cb, const int32_t* new_entry,
                                          const EntryList& el, cudaStream_t s);
cudaError_t launch_entry_fill(const CbView& cb, int which, const int32_t* first,
                              const int32_t* new_entry, const EntryList& el, int chunk_index,
                              cudaStream_t s);
cudaError_t launch_mark_embedded(const CbView& cb, int which, cudaStream_t s);
cudaError_t run_encoder_pass(const CbView& cb, const EncoderArgs& a, const EntryList& el,
                             bool use_tensor_cores, Prof* prof, cudaStream_t s);

// ---- z2z_logits.cu ---------------------------------------------------------------------------
struct LogitsArgs {
  int d, dtype, N;
  const void* hidden;           // [N, d]
  const int32_t* row_seq;       // [N] or NULL
  const int32_t* row_nvis;      // [N] or NULL
  const void* WU;               // [V, d]
  const void* Uh;               // [B, cap, d]
  int select; float inv_temperature; uint64_t seed, step;
  const int32_t* targets;
  float* lse; int32_t* argmax; float* max_logit; int32_t* sample; float* target_logit;
  float* logits_debug;
  void* lpart; size_t lpart_bytes;
  int row_base;                 // global index of row 0 of this launch (sampling counter)
};
// Partial reduction of one hidden row over a subset of the columns.
struct __align__(32) LogitPartial { float m, s; int idx; float gm; int gidx; int pad[3]; };
// Where a logits kernel left its partials when the caller merges them itself (decode step).
struct LogitsPartInfo { int stride, count; };
// When `info` is given the merge kernel is skipped and the layout of the partials is returned.
cudaError_t run_logits_simt(const CbView& cb, const LogitsArgs& a, LogitsPartInfo* info, Prof* prof,
                            cudaStream_t s);
// Tensor-core (tcgen05) version for bf16 (d % 64 == 0).
cudaError_t run_logits_tc(const CbView& cb, const LogitsArgs& a, int* vt_word, int* err_word,
                          LogitsPartInfo* info, Prof* prof, cudaStream_t s);

// ---- z2z_prefill_logits.cu -------------------------------------------------------------------
// Same outputs as run_logits_tc, for many hidden rows (bf16, d % 64 == 0).  `plan` is scratch for
// 3 int32 per 256-row tile.  strips_override > 0 fixes the number of column strips (tests).
bool prefill_logits_supported(int d, int dtype);
// Rows one launch can take with the given scratch when `strips` partials per row are needed.
long long prefill_logits_max_rows(size_t lpart_bytes, size_t plan_bytes, int strips);
int prefill_logits_strips(int N, int d);
cudaError_t run_logits_prefill(const CbView& cb, const LogitsArgs& a, int32_t* plan, int* err_word,
                               int strips_override, Prof* prof, cudaStream_t s);

// ---- z2z_decode_update.cu --------------------------------------------------------------------
struct DecodeUpdateArgs {
  const LogitPartial* lpart; int part_stride, part_count;
  int select;
  const int32_t* forced;
  int32_t* next_codes; int32_t* selected; float* lse; int32_t* new_entry;
  int* frozen_flag;   // host word mapped into the device's address space, or NULL
  int epoch;          // written there once every codebook of the session is full
};
cudaError_t launch_decode_update(const CbView& cb, const DecodeUpdateArgs& a, const EntryList& el,
                                 cudaStream_t s);

// Selected code of the decode step: sample or argmax, overridden by `forced` when given.
cudaError_t launch_pick_codes(int B, const int32_t* argmax, const int32_t* sample,
                              const int32_t* forced, int32_t* next_codes, int32_t* selected,
                              cudaStream_t s);

}  // namespace z2z
