/*
 * z2z.h — C ABI of the zip2zip dynamic-vocabulary hot path on NVIDIA B200 (sm_100a).
 *
 * The library implements the work the method adds to every prefill and decode step of an LLM
 * (paper Section 2): the per-sequence LZW codebook (Section 2.1), the hyper-encoder that turns a
 * new codebook entry into a hyper-embedding / hyper-unembedding row (Section 2.2), and logits
 * over the static vocabulary joined with the sequence's own hypertokens with the reductions
 * taken from them (Section 2.3, steps 7-10).
 *
 * Conventions for every entry point
 *   - Returns an int32 status: Z2Z_OK or a negative Z2Z_ERR_* for errors the host can detect
 *     (bad arguments, workspace too small, a CUDA launch error).  Never throws, never exits.
 *   - Conditions only the device can see are OR-ed into a per-sequence status word
 *     (Z2Z_ST_* bits), readable with z2z_status().
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  The caller owns every
 *     buffer; the library allocates no device memory.  The opaque handle is host memory that
 *     stores the configuration and offsets into the caller's workspace.
 *   - All work is enqueued on the given stream and returns without synchronising (except
 *     z2z_status, z2z_codebook_read, z2z_profile_read and z2z_hyper_embed with max_entries < 0,
 *     which wait for the stream).  The enqueueing calls may therefore be captured
 *     into a CUDA graph (arguments passed by value, the sampling step among them, are then fixed
 *     for every replay); capture again after z2z_codebook_init starts a new session, because
 *     z2z_decode_step decides on the host whether the session still needs its hyper-encoder pass.
 *   - Ids are int32.  Tables are row-major [rows, d] in the configured dtype.
 *   - Hypertoken id = V + k where k is the creation order within the sequence.
 *   - Limits: V + cap < 2^24 - 1, cap <= 65535, 1 <= M <= 8, d % 8 == 0, B <= 1024.
 */
#ifndef Z2Z_H_
#define Z2Z_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* z2z_stream;          /* a cudaStream_t */
typedef struct z2z_codebook z2z_codebook;        /* opaque, host memory */

enum {
  Z2Z_OK = 0,
  Z2Z_ERR_INVALID_ARG = -1,
  Z2Z_ERR_WORKSPACE_TOO_SMALL = -2,
  Z2Z_ERR_CUDA = -3,
  Z2Z_ERR_UNSUPPORTED = -4
};

/* bits of the per-sequence device status word */
enum {
  Z2Z_ST_CAP_FROZEN = 1,     /* codebook reached cap: matching continues, inserting stopped  */
  Z2Z_ST_BAD_TOKEN = 2,      /* a code named a hypertoken that does not exist; state unchanged */
  Z2Z_ST_TABLE_FULL = 4,     /* hash probe ran through the whole table (cannot happen at load <= 1/2) */
  Z2Z_ST_WAIT_TIMEOUT = 8,   /* a bounded wait inside a kernel gave up                          */
  Z2Z_ST_OUTPUT_TRUNCATED = 16, /* z2z_lzw_decode: the base tokens did not fit in T_out_max      */
  Z2Z_ST_HALF_RANGE = 32     /* z2z_set_encoder_half_scratch: an encoder weight lies outside fp16's range */
};

enum { Z2Z_DTYPE_FP32 = 0, Z2Z_DTYPE_BF16 = 1 };
enum { Z2Z_SELECT_ARGMAX = 0, Z2Z_SELECT_GUMBEL = 1 };
/* Markers in place of a code (batches whose sequences finish at different times):
 *   Z2Z_CODE_NONE      no token: in d_forced the sequence sits the step out; z2z_embed_lookup
 *                      writes a zero row for it and raises no status.
 *   Z2Z_CODE_SELECTED  in d_forced only: apply the step's own selection to this sequence.        */
enum { Z2Z_CODE_NONE = -1, Z2Z_CODE_SELECTED = -2 };
enum { Z2Z_CACHE_EMBED = 0, Z2Z_CACHE_UNEMBED = 1 };

typedef struct {
  int32_t V;            /* static vocabulary size                                   */
  int32_t d;            /* embedding dimension                                      */
  int32_t M;            /* maximum merge size (Section 2.1)                         */
  int32_t cap;          /* maximum hypertokens per sequence; at cap the book freezes */
  int32_t B;            /* sequences in the session                                 */
  int32_t dtype;        /* Z2Z_DTYPE_*: tables, encoder tensors, hidden states, caches */
  int32_t enc_layers;   /* hyper-encoder layers; 0 = the parameter-free averaging variant */
  int32_t enc_heads;    /* attention heads (d % enc_heads == 0)                     */
  int32_t enc_dff;      /* feed-forward width; 0 = attention-only layers (no feed-forward block:
                           the 1-attention-layer variant of the architecture ablation) */
  int32_t tied;         /* 1: the caller passes the same cache for both sides       */
} z2z_config;

/* Hyper-encoder parameters (Section 2.2; Section 3.1: transformer encoder layers), all in the
 * configured dtype, as a HOST array of DEVICE pointers in this order:
 *   pos[M,d], then for each layer:
 *   ln1_w[d] ln1_b[d] Wqkv[3d,d] bqkv[3d] Wo[d,d] bo[d] ln2_w[d] ln2_b[d] W1[dff,d] b1[dff] W2[d,dff] b2[d]
 * n_tensors must be 1 + 12 * enc_layers.  With enc_dff == 0 the six feed-forward slots of a
 * layer (ln2_w .. b2) are ignored and may be NULL.                                                      */
typedef struct {
  const void* const* tensors;
  int32_t n_tensors;
} z2z_encoder_weights;

/* Bytes of device workspace the session needs (codebooks, counters, kernel scratch). */
int32_t z2z_workspace_bytes(const z2z_config* cfg, size_t* out_bytes);

/* Section 2.2 "At the beginning of each inference session V_h is initialized as an empty set".
 * Creates the handle on first use (*cb == NULL) and clears every sequence's codebook, counters
 * and status.  d_ws must be 256-byte aligned and stay valid for the life of the handle.  May be
 * called again on an existing handle to start a new session.                                   */
int32_t z2z_codebook_init(z2z_codebook** cb, const z2z_config* cfg, void* d_ws, size_t ws_bytes,
                          z2z_stream stream);
/* (The handle also owns 64 bytes of pinned host memory, freed by z2z_codebook_destroy: the decode
 * step's update kernel stores the session number there once every sequence's codebook is full.
 * From then on no step can create an entry, and z2z_decode_step no longer launches the
 * hyper-encoder pass - the weights of both encoders are not streamed for nothing.)             */

/* Section 2.1 / Section 2.3 step 2: compress each prompt with LZW (greedy longest match against
 * the growing codebook; new entry = emitted phrase + next base token, only if shorter than M
 * tokens before the append and the book is not full).
 *   d_tokens [B, T_max] int32 base tokens in [0, V); d_lens [B] valid length of each row.
 *   d_codes  [B, T_max] int32 out; d_code_lens [B] out.
 *   d_entries_after [B, T_max] int32 out or NULL: hypertokens that exist once code i is emitted.
 * Leaves every sequence ready for z2z_lzw_step (previous code = its last code).               */
int32_t z2z_lzw_encode(z2z_codebook* cb, const int32_t* d_tokens, const int32_t* d_lens,
                       int32_t T_max, int32_t* d_codes, int32_t* d_code_lens,
                       int32_t* d_entries_after, z2z_stream stream);

/* Figure 1 / Section 2.3 step 10: online update with one newly selected code per sequence.
 * Candidate entry = phrase(previous code) ++ first base token of phrase(new code); created if
 * the previous phrase is shorter than M, the book is not full and the phrase is not there yet.
 *   d_new_codes [B]; d_active [B] (0 = skip this sequence) or NULL;
 *   d_new_entry [B] out: entry number created, or -1.
 * A code >= V + n that is not the one this very step creates sets Z2Z_ST_BAD_TOKEN and leaves
 * that sequence untouched (Section 2.3, "Consistent Vocabulary Updates").                     */
int32_t z2z_lzw_step(z2z_codebook* cb, const int32_t* d_new_codes, const uint8_t* d_active,
                     int32_t* d_new_entry, z2z_stream stream);

/* Section 2.2 + Section 2.3 "Hyper-Embedding Cache": run the hyper-encoder over entries
 * [first_b, first_b + count_b) of every sequence and store one d-vector per entry.
 *   which    Z2Z_CACHE_EMBED (rows of W_E in, E_h out) or Z2Z_CACHE_UNEMBED (W_U in, U_h out);
 *            only selects which "embedded so far" counter is used when d_first/d_count are NULL.
 *   d_table  [V, d]; enc: that side's encoder.
 *   d_first / d_count [B] or both NULL = every entry created since the last such call.
 *   max_entries  host upper bound on sum_b count_b (<= 0: B * cap).  It bounds the launch count:
 *            entries are processed in passes of 1024, and a pass is about ten launches per layer
 *            whether or not it finds entries (the counts are device state).  After z2z_lzw_encode
 *            pass the number of prompt tokens (or the sum of the code lengths, if known on the
 *            host): a prompt of T tokens creates fewer than T entries.  With 0 a large session
 *            (B * cap = 524288) would enqueue 512 passes.
 *            max_entries < 0: exact.  The call reads the number of entries it has to embed back
 *            from the device - it waits for the stream once, the only enqueueing call that does,
 *            and therefore cannot be captured into a graph - and launches no pass without work.
 *            Meant for whole prompts, where hundreds of empty passes would cost more than the wait.
 *   d_cache  [B, cap, d] in the configured dtype (row k of sequence b = hypertoken V + k).
 *   d_cache_f32 [B, cap, d] fp32 or NULL: the same rows before rounding to the cache dtype.    */
int32_t z2z_hyper_embed(z2z_codebook* cb, int32_t which, const void* d_table,
                        const z2z_encoder_weights* enc, const int32_t* d_first,
                        const int32_t* d_count, int32_t max_entries, void* d_cache,
                        float* d_cache_f32, z2z_stream stream);

/* Section 2.3 steps 7-9: for each of N hidden rows, logits over W_U joined with the first
 * n_vis rows of the owning sequence's U_h; log-sum-exp, argmax (lowest index on ties) and
 * optionally a Gumbel-max sample at the given temperature.  The logit matrix is not stored.
 *   d_hidden [N, d]; d_row_seq [N] owning sequence of each row (NULL: row r belongs to r);
 *   d_row_nvis [N] visible hypertokens per row or NULL = all n_b of the sequence;
 *   d_WU [V, d]; d_Uh [B, cap, d];
 *   select/temperature/seed/step: sampling (Philox4x32-10 keyed by seed, counter
 *            (column/4, row, step), u = ((x >> 9) + 0.5) * 2^-23, g = -log(-log u));
 *   d_targets [N] or NULL -> d_target_logit [N] = logit of that column (NaN if not visible);
 *   d_lse [N], d_argmax [N], d_max_logit [N]; d_sample [N] (required iff select == GUMBEL);
 *   d_logits_debug [N, V + cap] fp32 or NULL: every logit, for tests.                         */
int32_t z2z_dynamic_logits(z2z_codebook* cb, const void* d_hidden, int32_t N,
                           const int32_t* d_row_seq, const int32_t* d_row_nvis, const void* d_WU,
                           const void* d_Uh, int32_t select, float temperature, uint64_t seed,
                           uint64_t step, const int32_t* d_targets, float* d_lse,
                           int32_t* d_argmax, float* d_max_logit, int32_t* d_sample,
                           float* d_target_logit, float* d_logits_debug, z2z_stream stream);

/* One whole decode step (Section 2.3 steps 7-10 and the cache update): logits and selection for
 * hidden row b of sequence b, LZW update with the selected code, hyper-encoder on the at most
 * one new entry per sequence for both caches.
 *   d_forced [B] or NULL: codes to feed the update instead of the selection (teacher forcing;
 *            the selection is still computed and returned in d_selected).  Z2Z_CODE_SELECTED
 *            applies the selection after all; Z2Z_CODE_NONE makes the sequence sit the step out
 *            (a finished sequence of the batch): its codebook, caches and status stay as they
 *            are, d_next_codes[b] = Z2Z_CODE_NONE, d_new_entry[b] = -1, its row of d_next_embed
 *            is zero; the row's logits results are still computed and returned.
 *   d_next_codes [B] out: the code that was applied; d_selected [B] out or NULL: argmax/sample;
 *   d_lse [B] out; d_new_entry [B] out or NULL.  These small result arrays may also be pinned host
 *            memory that is mapped into the device's address space: the kernels then store the
 *            results straight into host memory and no separate copy is needed.
 *   d_Eh_f32 / d_Uh_f32: optional fp32 copies of the new rows, as in z2z_hyper_embed.
 *   d_next_embed [B, d] out or NULL: input embedding of the applied codes for the model's next
 *            step (Figure 2a): W_E row of a base token, else the sequence's cached hyper-embedding,
 *            including the row this very step created; as z2z_embed_lookup on d_next_codes.     */
int32_t z2z_decode_step(z2z_codebook* cb, const void* d_hidden, const void* d_WE,
                        const void* d_WU, const z2z_encoder_weights* enc_E,
                        const z2z_encoder_weights* enc_U, void* d_Eh, void* d_Uh,
                        int32_t select, float temperature, uint64_t seed, uint64_t step,
                        const int32_t* d_forced, int32_t* d_next_codes, int32_t* d_selected,
                        float* d_lse, int32_t* d_new_entry, float* d_Eh_f32, float* d_Uh_f32,
                        void* d_next_embed, z2z_stream stream);

/* Section 2.1 (second property of LZW: the stream decodes without a shipped codebook) and
 * Section 2.3 steps 11-12: turn each sequence's code stream back into base tokens.
 *   d_codes [B, Tc_max] int32; d_code_lens [B] valid codes per row, or NULL (= Tc_max);
 *   d_tokens [B, T_out_max] int32 out; d_token_lens [B] out.
 * mode Z2Z_DECODE_RESIDENT: every code is looked up in the codebook the session already holds
 *   (the state at the end of generation); the codebook is not changed.
 * mode Z2Z_DECODE_REPLAY: the codebook is grown from the codes themselves, one online update
 *   (as z2z_lzw_step) per code starting from the sequence's current state - after
 *   z2z_codebook_init this is plain LZW decompression - and the codes are then expanded.  The
 *   sequence is left as z2z_lzw_step would leave it after the last accepted code.
 * A code that names no hypertoken sets Z2Z_ST_BAD_TOKEN; that sequence's output ends before it
 * (in REPLAY mode the state is the one after the last accepted code).  Output beyond T_out_max
 * is dropped, d_token_lens[b] = T_out_max and Z2Z_ST_OUTPUT_TRUNCATED is set.  All device
 * pointers; work is enqueued on the stream.                                                    */
enum { Z2Z_DECODE_RESIDENT = 0, Z2Z_DECODE_REPLAY = 1 };
int32_t z2z_lzw_decode(z2z_codebook* cb, const int32_t* d_codes, const int32_t* d_code_lens,
                       int32_t Tc_max, int32_t mode, int32_t* d_tokens, int32_t* d_token_lens,
                       int32_t T_out_max, z2z_stream stream);

/* Figure 2a / Section 2.3 steps 3-4: input embedding of a mixed stream.  Row r of d_out is
 * W_E[z] for a base token z < V and the cached hyper-embedding E_h[b][z - V] otherwise, where
 * b = d_row_seq[r] (or r when d_row_seq is NULL, which needs N <= B).
 *   d_codes [N] int32; d_WE [V, d]; d_Eh [B, cap, d]; d_out [N, d]; all in the configured dtype.
 * A code outside [0, V + n_b) sets Z2Z_ST_BAD_TOKEN for that sequence and its row is zero-filled;
 * Z2Z_CODE_NONE gives a zero row and no status.                                                */
int32_t z2z_embed_lookup(z2z_codebook* cb, const int32_t* d_codes, int32_t N,
                         const int32_t* d_row_seq, const void* d_WE, const void* d_Eh,
                         void* d_out, z2z_stream stream);

/* Top-k / nucleus (top-p) filtered sampling on stored logits (no counterpart in the paper, which
 * only says that a token is sampled from the joint distribution: Section 2.3 step 9).  For decode
 * batches the caller stores the joint logits once (d_logits_debug of z2z_dynamic_logits) and
 * samples here; the applied code then goes to z2z_lzw_step and z2z_hyper_embed as usual.
 *   d_logits [N, ld] fp32; d_n_cols [N]: columns of row r that exist (V + visible hypertokens);
 *   top_k <= 0: no top-k filter, else every column whose logit is >= the k-th largest is kept;
 *   top_p >= 1: no nucleus filter, else with the columns in descending order of
 *            softmax(l / temperature) the shortest prefix with probability >= top_p is kept,
 *            extended over ties with its last logit; the two filters intersect;
 *   the sample is the Gumbel-max over the kept columns with the noise of the fused sampler
 *            (seed, step; the row number in the counter is row_base + r);
 *   d_choice [N] out (-1 for a row without columns); d_kept [N] out or NULL: columns kept.     */
int32_t z2z_sample_filtered(const float* d_logits, int32_t N, int64_t ld, const int32_t* d_n_cols,
                            int32_t top_k, float top_p, float temperature, uint64_t seed, uint64_t step,
                            int32_t row_base, int32_t* d_choice, int32_t* d_kept, z2z_stream stream);

/* Host -> device transfer of a small per-step input (the hidden rows of a decode step) by a kernel
 * instead of a copy-engine transfer (no counterpart in the paper; end-to-end latency aid).  The
 * kernel that follows on the stream may start its independent part - z2z_decode_step's logits
 * kernel streams W_U before it needs the hidden rows - while the transfer runs.
 *   h_mapped_src: pinned host memory that is mapped into the device's address space;
 *   d_dst: device memory; bytes: multiple of 16, at most 256 MiB; both pointers 16-byte aligned. */
int32_t z2z_upload_rows(const void* h_mapped_src, void* d_dst, size_t bytes, z2z_stream stream);

/* Waits for the stream, then copies per-sequence status bits and hypertoken counts to the host.
 * Either output may be NULL.                                                                  */
int32_t z2z_status(z2z_codebook* cb, int32_t* h_status, int32_t* h_n, z2z_stream stream);

/* Copies the codebook of one sequence to the host for inspection: constituents
 * h_cons [cap, M] (-1 padded) and lengths h_len [cap]; waits for the stream.                  */
int32_t z2z_codebook_read(z2z_codebook* cb, int32_t b, int32_t* h_cons, int32_t* h_len,
                          z2z_stream stream);

/* Kernel family used for bf16 sessions (no counterpart in the paper; cross-checking aid).
 * enable = 1 (default): tcgen05 tensor-core kernels wherever the shapes allow (d and enc_dff
 * multiples of 128), the joint-logits kernel chosen by the number of hidden rows (weight
 * streaming for decode batches, CTA-pair tiles from 2048 rows on).  enable = 0: the CUDA-core
 * kernels, which keep activations in fp32 and are the path fp32 sessions always take.
 * enable = 2 + 16 * s: as 1, but z2z_dynamic_logits always takes the CTA-pair kernel, with s
 * column strips per row tile when 1 <= s <= 8 (s = 0: chosen by shape).  All produce results
 * within the stated tolerance.                                                                 */
int32_t z2z_set_tensor_cores(z2z_codebook* cb, int32_t enable);

/* Faster hyper-encoder for whole prompts (Section 2.2 applied to every entry of a prompt, Section
 * 2.3 steps 3-4; the number format is this library's choice, the paper fixes none).  By default
 * the tensor-core passes keep activations as two bf16 parts (about 16 mantissa bits), two
 * tensor-core instructions per k-step.  When the caller lends device memory for fp16 copies of one
 * encoder's linear-layer weights, z2z_hyper_embed calls that span at least four prompt-sized passes
 * (bf16 sessions, passes of >= 1024 rows) remake the copies at the start of the call - a bf16
 * value inside fp16's range converts exactly - and round each activation once to fp16 (11 mantissa
 * bits): one instruction per k-step, half the tensor-core work.  Measured against the fp64
 * definition with randomly drawn gains and biases, the largest error of a hyper-embedding grows
 * from 9e-5 to 7.3e-3 at d = 4096 (tolerance 2e-2); sessions that need the wider margin leave the
 * scratch unset.  Decode steps are not affected.
 *   d_scratch: 256-byte aligned, bytes >= 2 * enc_layers * (4 d^2 + 2 d enc_dff) * 2, valid until
 *   replaced; NULL or 0 bytes returns to the two-part form.  A weight beyond fp16's range
 *   (|w| > 65504) cannot be copied exactly: Z2Z_ST_HALF_RANGE is then reported by z2z_status.   */
int32_t z2z_set_encoder_half_scratch(z2z_codebook* cb, void* d_scratch, size_t bytes);

/* Launch accounting and per-kernel-class timing (no counterpart in the paper; measurement aid).
 * The library always counts the kernels it launches, per class:
 *   0 joint-logits main kernel, 1 logits merge / selection, 2 LZW kernels,
 *   3 hyper-encoder linear layers, 4 other hyper-encoder kernels and work lists.
 * z2z_profile(cb, 1) additionally brackets every launch group with CUDA events on the caller's
 * stream until z2z_profile(cb, 0).  z2z_profile_read waits for the stream, returns the summed
 * event time in milliseconds (h_ms, may be NULL) and the launch counts (h_launches, may be NULL)
 * for the first n_classes classes, and resets both.                                           */
int32_t z2z_profile(z2z_codebook* cb, int32_t enable);
int32_t z2z_profile_read(z2z_codebook* cb, int32_t n_classes, double* h_ms, int64_t* h_launches,
                         z2z_stream stream);

/* Joint logits with log-sum-exp, argmax and maximum for callers that cannot allocate device
 * memory (the paper has no counterpart; this is a deployment aid).  Some callers cannot call
 * cudaMalloc or a framework allocator: a plug-in in a serving process that gave out all device
 * memory at start-up, a callback that must not enter the allocator, a process already at its
 * memory limit.  They cannot provide the session workspace either, so this call takes no handle:
 * the per-CTA partial reductions live in an array of 2 MiB that is part of the library image
 * (every GPU that loads the library holds it until the process exits).  The library allocates
 * nothing in this call.
 *   d_hidden [N, d], d_row_seq [N] or NULL (row r belongs to sequence r), d_WU [V, d],
 *   d_Uh [B, cap, d], all in `dtype`; d_n_hyper [B] DEVICE array: visible hypertokens of each
 *   sequence, 0 <= d_n_hyper[b] <= cap (a larger count is read as cap: no row beyond a sequence's
 *   cap rows is touched); d_lse / d_argmax / d_max_logit [N] out, each may be NULL.
 * Limits: N <= 1024 rows per call (larger N returns Z2Z_ERR_INVALID_ARG and z2z_last_error says
 * so); the other limits are those of z2z_config.  Same arithmetic as the CUDA-core path of
 * z2z_dynamic_logits (fp32 accumulation).
 * The first call on a device looks up the array's address for that device: make that call with
 * the device current and outside any stream capture.  All calls on a device share the array and
 * leave their partials in it (nothing there needs clearing between calls); calls that overlap on
 * one GPU, e.g. on two streams, race on it and must be ordered by the caller.                  */
int32_t z2z_logits_static_scratch(const void* d_hidden, int32_t N, const int32_t* d_row_seq,
                                  const int32_t* d_n_hyper, const void* d_WU, const void* d_Uh,
                                  int32_t V, int32_t d, int32_t B, int32_t cap, int32_t dtype,
                                  float* d_lse, int32_t* d_argmax, float* d_max_logit,
                                  z2z_stream stream);

/* Frees the host handle (never the workspace). */
int32_t z2z_codebook_destroy(z2z_codebook* cb);

/* Text of the last host-side error on this thread (static storage). */
const char* z2z_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* Z2Z_H_ */
