// extern "C" entry points declared in include/z2z.h: argument checks, workspace views, and the
// order in which the kernels of each call are enqueued.  No arithmetic of the method lives here.
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "z2z_common.cuh"
#include "z2z_internal.h"
#include "z2z_stream.h"

struct z2z_codebook {
  z2z_config cfg;
  z2z::WsPlan plan;
  char* ws;
  size_t ws_bytes;
  z2z::CbView view;
  int dff, heads;
  int use_tensor_cores;      // 0: CUDA cores, 1: tensor cores (kernel by shape), 2: prompt-scoring kernel always
  int prefill_strips;        // > 0: fixed number of column strips in the prompt-scoring kernel
  int* h_frozen;             // pinned host word the decode-update kernel writes once every codebook is full
  int epoch;                 // session number: incremented by every z2z_codebook_init
  void* half_scratch;        // caller's memory for fp16 copies of one encoder's linear-layer weights, or NULL
  size_t half_bytes;
  std::vector<const void*> half_ptrs;   // device addresses of the copies, ABI tensor order
  z2z::Prof prof;
};

namespace {

thread_local char g_err[256] = "";

int fail(int code, const char* msg) {
  snprintf(g_err, sizeof(g_err), "%s", msg);
  return code;
}
int fail_cuda(cudaError_t e, const char* where) {
  snprintf(g_err, sizeof(g_err), "%s: %s", where, cudaGetErrorString(e));
  return Z2Z_ERR_CUDA;
}
#define Z2Z_CUDA(call, where)                                  \
  do {                                                         \
    cudaError_t e__ = (call);                                  \
    if (e__ != cudaSuccess) return fail_cuda(e__, where);      \
  } while (0)

int check_config(const z2z_config* c) {
  if (!c) return fail(Z2Z_ERR_INVALID_ARG, "config is NULL");
  if (c->V < 1 || c->d < 8 || c->d % 8 != 0) return fail(Z2Z_ERR_INVALID_ARG, "need V >= 1, d >= 8, d % 8 == 0");
  if (c->M < 1 || c->M > z2z::kMaxM) return fail(Z2Z_ERR_INVALID_ARG, "need 1 <= M <= 8");
  if (c->cap < 0 || c->cap > 65535) return fail(Z2Z_ERR_INVALID_ARG, "need 0 <= cap <= 65535");
  if ((long long)c->V + c->cap >= (1ll << 24) - 1) return fail(Z2Z_ERR_INVALID_ARG, "need V + cap < 2^24 - 1");
  if (c->B < 1 || c->B > 1024) return fail(Z2Z_ERR_INVALID_ARG, "need 1 <= B <= 1024");
  if (c->dtype != Z2Z_DTYPE_FP32 && c->dtype != Z2Z_DTYPE_BF16) return fail(Z2Z_ERR_INVALID_ARG, "unknown dtype");
  if (c->enc_layers < 0 || c->enc_layers > 16) return fail(Z2Z_ERR_INVALID_ARG, "need 0 <= enc_layers <= 16");
  if (c->enc_layers > 0) {
    if (c->enc_heads < 1 || c->d % c->enc_heads != 0) return fail(Z2Z_ERR_INVALID_ARG, "d must be a multiple of enc_heads");
    if (c->enc_dff != 0 && (c->enc_dff < 8 || c->enc_dff % 8 != 0))
      return fail(Z2Z_ERR_INVALID_ARG, "need enc_dff >= 8 and enc_dff % 8 == 0, or enc_dff == 0 (attention-only layers)");
  }
  return Z2Z_OK;
}

z2z::EntryList entry_list(z2z_codebook* cb) {
  z2z::EntryList el;
  el.seq = reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_entry_seq);
  el.idx = reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_entry_idx);
  el.len = reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_entry_len);
  el.tok = reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_entry_tok);
  el.row_off = reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_row_off);
  el.row_src = reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_row_src);
  el.row_tok = reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_row_tok);
  el.off = reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_entry_off);
  el.chunk = cb->plan.enc_chunk_entries;
  return el;
}

z2z::EncoderArgs encoder_args(z2z_codebook* cb, const void* table, const z2z_encoder_weights* enc,
                              void* cache, float* cache_f32, int entries, int group = 0) {
  z2z::EncoderArgs a{};
  a.d = cb->cfg.d; a.dff = cb->dff; a.heads = cb->heads; a.layers = cb->cfg.enc_layers;
  a.M = cb->cfg.M; a.dtype = cb->cfg.dtype;
  a.table = table; a.w = enc->tensors; a.cache = cache; a.cache_f32 = cache_f32;
  a.X = reinterpret_cast<float*>(cb->ws + cb->plan.off_X);
  a.A = reinterpret_cast<float*>(cb->ws + cb->plan.off_A);
  a.QKV = reinterpret_cast<float*>(cb->ws + cb->plan.off_QKV);
  a.H = reinterpret_cast<float*>(cb->ws + cb->plan.off_H);
  a.Ahl = reinterpret_cast<__nv_bfloat16*>(cb->ws + cb->plan.off_Ahl);
  a.Hhl = reinterpret_cast<__nv_bfloat16*>(cb->ws + cb->plan.off_Hhl);
  if (group == 1) {
    a.X = reinterpret_cast<float*>(cb->ws + cb->plan.off_g1_X);
    a.QKV = reinterpret_cast<float*>(cb->ws + cb->plan.off_g1_QKV);
    a.Ahl = reinterpret_cast<__nv_bfloat16*>(cb->ws + cb->plan.off_g1_Ahl);
    a.Hhl = reinterpret_cast<__nv_bfloat16*>(cb->ws + cb->plan.off_g1_Hhl);
  }
  a.part = reinterpret_cast<float*>(cb->ws + cb->plan.off_part);
  a.part_bytes = cb->plan.part_bytes;
  a.entries = entries;
  a.err = reinterpret_cast<int*>(cb->ws + cb->plan.off_words);
  return a;
}

int check_encoder(z2z_codebook* cb, const z2z_encoder_weights* enc) {
  if (!enc || !enc->tensors) return fail(Z2Z_ERR_INVALID_ARG, "encoder weights are NULL");
  if (enc->n_tensors != 1 + 12 * cb->cfg.enc_layers) return fail(Z2Z_ERR_INVALID_ARG, "n_tensors must be 1 + 12 * enc_layers");
  for (int i = 0; i < enc->n_tensors; ++i) {
    // attention-only layers ignore the six feed-forward slots (ln2_w .. b2), which may be NULL
    const bool unused = cb->dff == 0 && i >= 1 && (i - 1) % 12 >= 6;
    if (!enc->tensors[i] && !unused) return fail(Z2Z_ERR_INVALID_ARG, "an encoder tensor is NULL");
  }
  return Z2Z_OK;
}

// Rows at or above which the prompt-scoring kernel (CTA pairs, 256 x 256 tiles) takes over from
// the weight-streaming kernel: enough row tiles to give every cluster work.
constexpr int kPrefillMinRows = 2048;

int logits_call(z2z_codebook* cb, z2z::LogitsArgs a, cudaStream_t s, z2z::LogitsPartInfo* info = nullptr) {
  // rows are processed in blocks so that the partial-reduction scratch stays bounded
  const int N = a.N;
  const size_t esz = cb->cfg.dtype == Z2Z_DTYPE_FP32 ? 4 : 2;
  const size_t ldbg = (size_t)cb->cfg.V + cb->cfg.cap;
  const bool tc = cb->use_tensor_cores && z2z::logits_tc_supported(cb->cfg.d, cb->cfg.dtype);
  const bool prefill = tc && info == nullptr && z2z::prefill_logits_supported(cb->cfg.d, cb->cfg.dtype) &&
                       (cb->use_tensor_cores == 2 || N >= kPrefillMinRows);
  long long chunk = z2z::kLogitRowChunk;
  int prefill_strips = cb->prefill_strips;
  if (prefill) {
    // the number of column strips is fixed for the whole call; when the partial-reduction scratch
    // cannot take all rows at that split, the rows go out in launches of equal size
    if (prefill_strips <= 0) prefill_strips = z2z::prefill_logits_strips(N, cb->cfg.d);
    const long long cap_rows = z2z::prefill_logits_max_rows(cb->plan.lpart_bytes, cb->plan.plan_bytes, prefill_strips);
    if (cap_rows < 256) return fail(Z2Z_ERR_WORKSPACE_TOO_SMALL, "logits scratch too small for one row tile");
    chunk = cap_rows;
    if (chunk < N) {
      const long long launches = (N + cap_rows - 1) / cap_rows;
      chunk = ((N + launches - 1) / launches + 255) / 256 * 256;
      if (chunk > cap_rows) chunk = cap_rows;
    }
  }
  for (long long r0 = 0; r0 < N; r0 += chunk) {
    z2z::LogitsArgs c = a;
    c.N = (int)(N - r0 < chunk ? N - r0 : chunk);
    c.row_base = a.row_base + (int)r0;
    c.hidden = reinterpret_cast<const char*>(a.hidden) + (size_t)r0 * cb->cfg.d * esz;
    if (a.row_seq) c.row_seq = a.row_seq + r0;
    if (a.row_nvis) c.row_nvis = a.row_nvis + r0;
    if (a.targets) c.targets = a.targets + r0;
    if (a.lse) c.lse = a.lse + r0;
    if (a.argmax) c.argmax = a.argmax + r0;
    if (a.max_logit) c.max_logit = a.max_logit + r0;
    if (a.sample) c.sample = a.sample + r0;
    if (a.target_logit) c.target_logit = a.target_logit + r0;
    if (a.logits_debug) c.logits_debug = a.logits_debug + (size_t)r0 * ldbg;
    if (a.row_seq == nullptr && r0 > 0) return fail(Z2Z_ERR_INVALID_ARG, "d_row_seq is required when N > B");
    int* words = reinterpret_cast<int*>(cb->ws + cb->plan.off_words);
    if (prefill) {
      Z2Z_CUDA(z2z::run_logits_prefill(cb->view, c, reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_plan), words,
                                       prefill_strips, &cb->prof, s), "logits (prompt scoring)");
    } else if (tc) {
      Z2Z_CUDA(z2z::run_logits_tc(cb->view, c, words + 1, words, info, &cb->prof, s), "logits (tensor cores)");
    } else {
      Z2Z_CUDA(z2z::run_logits_simt(cb->view, c, info, &cb->prof, s), "logits");
    }
  }
  return Z2Z_OK;
}

}  // namespace

namespace z2z {
// Lets entry points in other files leave their message where z2z_last_error finds it.
void set_last_error(const char* msg) { snprintf(g_err, sizeof(g_err), "%s", msg); }
}  // namespace z2z

extern "C" {

const char* z2z_last_error(void) { return g_err; }

int32_t z2z_workspace_bytes(const z2z_config* cfg, size_t* out_bytes) {
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!out_bytes) return fail(Z2Z_ERR_INVALID_ARG, "out_bytes is NULL");
  z2z_config c = *cfg;
  if (c.enc_layers == 0) { c.enc_dff = 8; }
  *out_bytes = z2z::plan_workspace(c).total;
  return Z2Z_OK;
}

int32_t z2z_codebook_init(z2z_codebook** cb, const z2z_config* cfg, void* d_ws, size_t ws_bytes,
                          z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  int rc = check_config(cfg);
  if (rc) return rc;
  if (!d_ws || (reinterpret_cast<uintptr_t>(d_ws) & 255) != 0) return fail(Z2Z_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  z2z_config c = *cfg;
  if (c.enc_layers == 0) { c.enc_dff = 8; if (c.enc_heads < 1) c.enc_heads = 1; }
  z2z::WsPlan plan = z2z::plan_workspace(c);
  if (ws_bytes < plan.total) return fail(Z2Z_ERR_WORKSPACE_TOO_SMALL, "workspace smaller than z2z_workspace_bytes");
  z2z_codebook* h = *cb;
  if (!h) {
    h = new (std::nothrow) z2z_codebook();
    if (!h) return fail(Z2Z_ERR_INVALID_ARG, "out of host memory");
  }
  h->cfg = c; h->plan = plan; h->ws = reinterpret_cast<char*>(d_ws); h->ws_bytes = ws_bytes;
  h->dff = c.enc_dff; h->heads = c.enc_heads;
  h->use_tensor_cores = 1;
  h->prefill_strips = 0;
  if (!h->h_frozen) {
    // one word of pinned, device-visible host memory (host memory: the device workspace stays the caller's);
    // without it the session simply never learns that its codebooks are frozen
    void* p = nullptr;
    if (cudaHostAlloc(&p, 64, cudaHostAllocMapped | cudaHostAllocPortable) == cudaSuccess) h->h_frozen = reinterpret_cast<int*>(p);
    else (void)cudaGetLastError();
  }
  ++h->epoch;
  if (h->h_frozen) *reinterpret_cast<volatile int*>(h->h_frozen) = 0;
  z2z::CbView& v = h->view;
  v.V = c.V; v.M = c.M; v.cap = c.cap; v.B = c.B; v.n_slots = plan.n_slots;
  v.hash = reinterpret_cast<unsigned long long*>(h->ws + plan.off_hash);
  v.cons = reinterpret_cast<int32_t*>(h->ws + plan.off_cons);
  v.len = reinterpret_cast<uint8_t*>(h->ws + plan.off_len);
  v.n = reinterpret_cast<int32_t*>(h->ws + plan.off_n);
  v.prev = reinterpret_cast<int32_t*>(h->ws + plan.off_prev);
  v.status = reinterpret_cast<int32_t*>(h->ws + plan.off_status);
  v.n_emb = reinterpret_cast<int32_t*>(h->ws + plan.off_n_emb);
  *cb = h;
  Z2Z_CUDA(cudaMemsetAsync(h->ws + plan.off_words, 0, 256, reinterpret_cast<cudaStream_t>(stream)), "codebook_init");
  // the GEMM result matrix of the hyper-encoder passes is all zero between GEMMs; establish that once
  Z2Z_CUDA(cudaMemsetAsync(h->ws + plan.off_part, 0, plan.part_bytes, reinterpret_cast<cudaStream_t>(stream)), "codebook_init");
  z2z::ProfScope ps(&h->prof, z2z::kProfLzw, 1, reinterpret_cast<cudaStream_t>(stream));
  Z2Z_CUDA(z2z::launch_codebook_clear(v, reinterpret_cast<cudaStream_t>(stream)), "codebook_init");
  return Z2Z_OK;
}

int32_t z2z_lzw_encode(z2z_codebook* cb, const int32_t* d_tokens, const int32_t* d_lens,
                       int32_t T_max, int32_t* d_codes, int32_t* d_code_lens,
                       int32_t* d_entries_after, z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (T_max < 0) return fail(Z2Z_ERR_INVALID_ARG, "T_max < 0");
  if (!d_code_lens) return fail(Z2Z_ERR_INVALID_ARG, "d_code_lens is NULL");
  if (T_max > 0 && (!d_tokens || !d_codes)) return fail(Z2Z_ERR_INVALID_ARG, "d_tokens / d_codes is NULL");
  z2z::ProfScope ps(&cb->prof, z2z::kProfLzw, 1, reinterpret_cast<cudaStream_t>(stream));
  Z2Z_CUDA(z2z::launch_lzw_encode(cb->view, d_tokens, d_lens, T_max, d_codes, d_code_lens,
                                  d_entries_after, reinterpret_cast<cudaStream_t>(stream)),
           "lzw_encode");
  return Z2Z_OK;
}

int32_t z2z_lzw_step(z2z_codebook* cb, const int32_t* d_new_codes, const uint8_t* d_active,
                     int32_t* d_new_entry, z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (!d_new_codes) return fail(Z2Z_ERR_INVALID_ARG, "d_new_codes is NULL");
  z2z::ProfScope ps(&cb->prof, z2z::kProfLzw, 1, reinterpret_cast<cudaStream_t>(stream));
  Z2Z_CUDA(z2z::launch_lzw_step(cb->view, d_new_codes, d_active, 0, d_new_entry,
                                reinterpret_cast<cudaStream_t>(stream)), "lzw_step");
  return Z2Z_OK;
}

int32_t z2z_lzw_decode(z2z_codebook* cb, const int32_t* d_codes, const int32_t* d_code_lens,
                       int32_t Tc_max, int32_t mode, int32_t* d_tokens, int32_t* d_token_lens,
                       int32_t T_out_max, z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (mode != Z2Z_DECODE_RESIDENT && mode != Z2Z_DECODE_REPLAY) return fail(Z2Z_ERR_INVALID_ARG, "mode must be Z2Z_DECODE_RESIDENT or Z2Z_DECODE_REPLAY");
  if (Tc_max < 0 || T_out_max < 0) return fail(Z2Z_ERR_INVALID_ARG, "Tc_max / T_out_max < 0");
  if (!d_token_lens) return fail(Z2Z_ERR_INVALID_ARG, "d_token_lens is NULL");
  if (Tc_max > 0 && !d_codes) return fail(Z2Z_ERR_INVALID_ARG, "d_codes is NULL");
  if (T_out_max > 0 && !d_tokens) return fail(Z2Z_ERR_INVALID_ARG, "d_tokens is NULL");
  z2z::ProfScope ps(&cb->prof, z2z::kProfLzw, 1, reinterpret_cast<cudaStream_t>(stream));
  int32_t* n_valid = reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_new_entry);
  Z2Z_CUDA(z2z::launch_lzw_decode(cb->view, d_codes, d_code_lens, Tc_max, mode == Z2Z_DECODE_REPLAY,
                                  n_valid, d_tokens, d_token_lens, T_out_max,
                                  reinterpret_cast<cudaStream_t>(stream)), "lzw_decode");
  return Z2Z_OK;
}

int32_t z2z_embed_lookup(z2z_codebook* cb, const int32_t* d_codes, int32_t N,
                         const int32_t* d_row_seq, const void* d_WE, const void* d_Eh,
                         void* d_out, z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (N < 0) return fail(Z2Z_ERR_INVALID_ARG, "N < 0");
  if (N == 0) return Z2Z_OK;
  if (!d_codes || !d_WE || !d_out) return fail(Z2Z_ERR_INVALID_ARG, "d_codes / d_WE / d_out is NULL");
  if (!d_Eh && cb->cfg.cap > 0) return fail(Z2Z_ERR_INVALID_ARG, "d_Eh is NULL");
  if (!d_row_seq && N > cb->cfg.B) return fail(Z2Z_ERR_INVALID_ARG, "d_row_seq is required when N > B");
  const int eb = cb->cfg.dtype == Z2Z_DTYPE_BF16 ? 2 : 4;
  Z2Z_CUDA(z2z::launch_embed_lookup(cb->view, d_codes, N, d_row_seq, d_WE, d_Eh, d_out, cb->cfg.d, eb,
                                    reinterpret_cast<cudaStream_t>(stream)), "embed_lookup");
  return Z2Z_OK;
}

int32_t z2z_hyper_embed(z2z_codebook* cb, int32_t which, const void* d_table,
                        const z2z_encoder_weights* enc, const int32_t* d_first,
                        const int32_t* d_count, int32_t max_entries, void* d_cache,
                        float* d_cache_f32, z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (which != Z2Z_CACHE_EMBED && which != Z2Z_CACHE_UNEMBED) return fail(Z2Z_ERR_INVALID_ARG, "which must be 0 or 1");
  if (!d_table || !d_cache) return fail(Z2Z_ERR_INVALID_ARG, "d_table / d_cache is NULL");
  if ((d_first == nullptr) != (d_count == nullptr)) return fail(Z2Z_ERR_INVALID_ARG, "d_first and d_count must both be given or both be NULL");
  int rc = check_encoder(cb, enc);
  if (rc) return rc;
  if (cb->cfg.cap == 0) return Z2Z_OK;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  z2z::EntryList el = entry_list(cb);
  z2z::EncoderArgs a = encoder_args(cb, d_table, enc, d_cache, d_cache_f32, el.chunk);
  const bool tc = cb->use_tensor_cores && cb->cfg.enc_layers >= 0 &&
                  z2z::encoder_tc_supported(cb->cfg.d, cb->dff, cb->cfg.dtype, cb->heads, cb->cfg.M);
  {
    z2z::ProfScope ps(&cb->prof, z2z::kProfEncOther, 1, s);
    Z2Z_CUDA(z2z::launch_entry_offsets(cb->view, which, d_first, d_count, el, s), "hyper_embed");
  }
  long long bound = (long long)cb->cfg.B * cb->cfg.cap;
  if (max_entries > 0 && max_entries < bound) bound = max_entries;
  if (max_entries < 0) {
    // exact: read the number of entries this call has to embed back from the device (the one
    // place where an enqueueing call waits for the stream), so that no pass is launched for nothing
    int32_t total = 0;
    int32_t* land = cb->h_frozen ? cb->h_frozen + 8 : &total;      // pinned host word when there is one
    Z2Z_CUDA(cudaMemcpyAsync(land, el.off + cb->cfg.B, 4, cudaMemcpyDeviceToHost, s), "hyper_embed (entry count)");
    Z2Z_CUDA(cudaStreamSynchronize(s), "hyper_embed (entry count)");
    total = *reinterpret_cast<volatile int32_t*>(land);
    if (total >= 0 && total < bound) bound = total;
  }
  const int n_chunks = (int)((bound + el.chunk - 1) / el.chunk);
  // Single-pass fp16 form of the prompt-sized passes: when the caller has lent memory for the
  // weight copies and the call is long enough (several passes) to repay making them.
  a.w_half = nullptr;
  if (tc && cb->half_scratch && cb->cfg.enc_layers > 0 && n_chunks >= 4 &&
      z2z::encoder_pass_is_prompt_sized(a.entries, el.chunk, cb->cfg.M) &&
      cb->half_bytes >= z2z::encoder_half_bytes(cb->cfg.d, cb->dff, cb->cfg.enc_layers)) {
    cb->half_ptrs.assign((size_t)enc->n_tensors, nullptr);
    Z2Z_CUDA(z2z::convert_encoder_weights_to_half(enc->tensors, cb->cfg.d, cb->dff, cb->cfg.enc_layers, cb->half_scratch,
                                                  cb->half_ptrs.data(), a.err, &cb->prof, s), "hyper_embed (fp16 weight copies)");
    a.w_half = cb->half_ptrs.data();
  }
  for (int c = 0; c < n_chunks; ++c) {
    {
      z2z::ProfScope ps(&cb->prof, z2z::kProfEncOther, 1, s);
      Z2Z_CUDA(z2z::launch_entry_fill(cb->view, which, d_first, nullptr, el, c, s), "hyper_embed");
    }
    if (tc) Z2Z_CUDA(z2z::run_encoder_pass_tc(cb->view, &a, 1, el, false, &cb->prof, s), "hyper_embed (tensor cores)");
    else Z2Z_CUDA(z2z::run_encoder_pass(cb->view, a, el, false, &cb->prof, s), "hyper_embed");
  }
  if (!d_first) {
    z2z::ProfScope ps(&cb->prof, z2z::kProfEncOther, 1, s);
    Z2Z_CUDA(z2z::launch_mark_embedded(cb->view, which, s), "hyper_embed");
  }
  return Z2Z_OK;
}

int32_t z2z_dynamic_logits(z2z_codebook* cb, const void* d_hidden, int32_t N,
                           const int32_t* d_row_seq, const int32_t* d_row_nvis, const void* d_WU,
                           const void* d_Uh, int32_t select, float temperature, uint64_t seed,
                           uint64_t step, const int32_t* d_targets, float* d_lse,
                           int32_t* d_argmax, float* d_max_logit, int32_t* d_sample,
                           float* d_target_logit, float* d_logits_debug, z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (N < 0) return fail(Z2Z_ERR_INVALID_ARG, "N < 0");
  if (N == 0) return Z2Z_OK;
  if (!d_hidden || !d_WU) return fail(Z2Z_ERR_INVALID_ARG, "d_hidden / d_WU is NULL");
  if (!d_Uh && cb->cfg.cap > 0) return fail(Z2Z_ERR_INVALID_ARG, "d_Uh is NULL");
  if (!d_row_seq && N > cb->cfg.B) return fail(Z2Z_ERR_INVALID_ARG, "d_row_seq is required when N > B");
  if (select != Z2Z_SELECT_ARGMAX && select != Z2Z_SELECT_GUMBEL) return fail(Z2Z_ERR_INVALID_ARG, "unknown select mode");
  if (select == Z2Z_SELECT_GUMBEL && (!d_sample || !(temperature > 0.f))) return fail(Z2Z_ERR_INVALID_ARG, "sampling needs d_sample and temperature > 0");
  if (d_targets && !d_target_logit) return fail(Z2Z_ERR_INVALID_ARG, "d_targets given without d_target_logit");
  z2z::LogitsArgs a{};
  a.d = cb->cfg.d; a.dtype = cb->cfg.dtype; a.N = N;
  a.hidden = d_hidden; a.row_seq = d_row_seq; a.row_nvis = d_row_nvis; a.WU = d_WU; a.Uh = d_Uh;
  a.select = select; a.inv_temperature = select == Z2Z_SELECT_GUMBEL ? 1.0f / temperature : 1.0f;
  a.seed = seed; a.step = step; a.targets = d_targets;
  a.lse = d_lse; a.argmax = d_argmax; a.max_logit = d_max_logit;
  a.sample = select == Z2Z_SELECT_GUMBEL ? d_sample : nullptr;
  a.target_logit = d_targets ? d_target_logit : nullptr;
  a.logits_debug = d_logits_debug;
  a.lpart = cb->ws + cb->plan.off_lpart; a.lpart_bytes = cb->plan.lpart_bytes;
  a.row_base = 0;
  return logits_call(cb, a, reinterpret_cast<cudaStream_t>(stream));
}

int32_t z2z_decode_step(z2z_codebook* cb, const void* d_hidden, const void* d_WE,
                        const void* d_WU, const z2z_encoder_weights* enc_E,
                        const z2z_encoder_weights* enc_U, void* d_Eh, void* d_Uh,
                        int32_t select, float temperature, uint64_t seed, uint64_t step,
                        const int32_t* d_forced, int32_t* d_next_codes, int32_t* d_selected,
                        float* d_lse, int32_t* d_new_entry, float* d_Eh_f32, float* d_Uh_f32,
                        void* d_next_embed, z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (!d_hidden || !d_WE || !d_WU || !d_Eh || !d_Uh || !d_next_codes) return fail(Z2Z_ERR_INVALID_ARG, "a required pointer is NULL");
  if (select != Z2Z_SELECT_ARGMAX && select != Z2Z_SELECT_GUMBEL) return fail(Z2Z_ERR_INVALID_ARG, "unknown select mode");
  if (select == Z2Z_SELECT_GUMBEL && !(temperature > 0.f)) return fail(Z2Z_ERR_INVALID_ARG, "sampling needs temperature > 0");
  int rc = check_encoder(cb, enc_E);
  if (rc) return rc;
  const bool tied = cb->cfg.tied != 0 || (d_Eh == d_Uh);
  if (!tied) { rc = check_encoder(cb, enc_U); if (rc) return rc; }
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const int B = cb->cfg.B;
  int32_t* sel = reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_sel);
  int32_t* w_argmax = sel;
  int32_t* w_sample = sel + B;
  float* w_max = reinterpret_cast<float*>(sel + 2 * B);
  float* w_lse = reinterpret_cast<float*>(sel + 3 * B);
  int32_t* w_new = d_new_entry ? d_new_entry : reinterpret_cast<int32_t*>(cb->ws + cb->plan.off_new_entry);

  // steps 7-9: joint logits, reductions, selection
  z2z::LogitsArgs a{};
  a.d = cb->cfg.d; a.dtype = cb->cfg.dtype; a.N = B;
  a.hidden = d_hidden; a.WU = d_WU; a.Uh = d_Uh;
  a.select = select; a.inv_temperature = select == Z2Z_SELECT_GUMBEL ? 1.0f / temperature : 1.0f;
  a.seed = seed; a.step = step;
  a.lse = d_lse ? d_lse : w_lse; a.argmax = w_argmax; a.max_logit = w_max;
  a.sample = select == Z2Z_SELECT_GUMBEL ? w_sample : nullptr;
  a.lpart = cb->ws + cb->plan.off_lpart; a.lpart_bytes = cb->plan.lpart_bytes;
  const bool fused = B <= 128;                 // one launch for merge + select + LZW update + work list
  // The frozen-session word is sampled BEFORE this step's update kernel is enqueued, and that kernel
  // only reports codebooks that were already full when it started: a step whose update can still
  // create an entry therefore always runs its hyper-encoder pass, however fast the device is.
  const bool frozen = cb->h_frozen && *reinterpret_cast<volatile int*>(cb->h_frozen) == cb->epoch;
  z2z::EntryList el = entry_list(cb);
  if (fused) {
    z2z::LogitsPartInfo info{0, 0};
    rc = logits_call(cb, a, s, &info);
    if (rc) return rc;
    z2z::DecodeUpdateArgs u{};
    u.lpart = reinterpret_cast<const z2z::LogitPartial*>(a.lpart);
    u.part_stride = info.stride; u.part_count = info.count; u.select = select; u.forced = d_forced;
    u.next_codes = d_next_codes; u.selected = d_selected; u.lse = a.lse; u.new_entry = w_new;
    u.frozen_flag = cb->h_frozen; u.epoch = cb->epoch;
    z2z::ProfScope ps(&cb->prof, z2z::kProfLzw, 1, s);
    Z2Z_CUDA(z2z::launch_decode_update(cb->view, u, el, s), "decode_step");
  } else {
    rc = logits_call(cb, a, s);
    if (rc) return rc;
    {
      z2z::ProfScope ps(&cb->prof, z2z::kProfLogitsMerge, 1, s);
      Z2Z_CUDA(z2z::launch_pick_codes(B, w_argmax, a.sample, d_forced, d_next_codes, d_selected, s), "decode_step");
    }
    // step 10: online LZW update
    {
      z2z::ProfScope ps(&cb->prof, z2z::kProfLzw, 1, s);
      Z2Z_CUDA(z2z::launch_lzw_step(cb->view, d_next_codes, nullptr, d_forced ? 1 : 0, w_new, s), "decode_step");
    }
    if (cb->cfg.cap > 0) {
      z2z::ProfScope ps(&cb->prof, z2z::kProfEncOther, 4, s);
      Z2Z_CUDA(z2z::launch_entry_offsets_from_new(cb->view, w_new, el, s), "decode_step");
      Z2Z_CUDA(z2z::launch_entry_fill(cb->view, 0, nullptr, w_new, el, 0, s), "decode_step");
      Z2Z_CUDA(z2z::launch_mark_embedded(cb->view, 0, s), "decode_step");
      Z2Z_CUDA(z2z::launch_mark_embedded(cb->view, 1, s), "decode_step");
    }
  }
  // cache update: the at most one new entry per sequence, on both sides.  Once an earlier step has
  // reported that every codebook is full nothing can be created any more and the pass is not launched.
  if (cb->cfg.cap > 0 && !frozen) {
    const bool tc = cb->use_tensor_cores && z2z::encoder_tc_supported(cb->cfg.d, cb->dff, cb->cfg.dtype, cb->heads, cb->cfg.M);
    z2z::EncoderArgs g[2];
    g[0] = encoder_args(cb, d_WE, enc_E, d_Eh, d_Eh_f32, B, 0);
    if (!tied) g[1] = encoder_args(cb, d_WU, enc_U, d_Uh, d_Uh_f32, B, 1);
    if (tc) {
      Z2Z_CUDA(z2z::run_encoder_pass_tc(cb->view, g, tied ? 1 : 2, el, fused, &cb->prof, s), "decode_step (tensor cores)");
    } else {
      Z2Z_CUDA(z2z::run_encoder_pass(cb->view, g[0], el, false, &cb->prof, s), "decode_step");
      if (!tied) {
        g[1] = encoder_args(cb, d_WU, enc_U, d_Uh, d_Uh_f32, B, 0);
        Z2Z_CUDA(z2z::run_encoder_pass(cb->view, g[1], el, false, &cb->prof, s), "decode_step");
      }
    }
  }
  if (d_next_embed) {                              // after the cache update: the new row may be the one looked up
    z2z::ProfScope ps(&cb->prof, z2z::kProfEncOther, 1, s);
    Z2Z_CUDA(z2z::launch_embed_lookup(cb->view, d_next_codes, B, nullptr, d_WE, d_Eh, d_next_embed, cb->cfg.d,
                                      cb->cfg.dtype == Z2Z_DTYPE_BF16 ? 2 : 4, s), "decode_step (next embedding)");
  }
  return Z2Z_OK;
}

int32_t z2z_status(z2z_codebook* cb, int32_t* h_status, int32_t* h_n, z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)cb->cfg.B * 4;
  if (h_status) Z2Z_CUDA(cudaMemcpyAsync(h_status, cb->view.status, bytes, cudaMemcpyDeviceToHost, s), "status");
  if (h_n) Z2Z_CUDA(cudaMemcpyAsync(h_n, cb->view.n, bytes, cudaMemcpyDeviceToHost, s), "status");
  int kernel_err = 0;
  Z2Z_CUDA(cudaMemcpyAsync(&kernel_err, cb->ws + cb->plan.off_words, 4, cudaMemcpyDeviceToHost, s), "status");
  Z2Z_CUDA(cudaStreamSynchronize(s), "status");
  if (kernel_err && h_status)
    for (int b = 0; b < cb->cfg.B; ++b)
      h_status[b] |= ((kernel_err & 1) ? Z2Z_ST_WAIT_TIMEOUT : 0) | ((kernel_err & 2) ? Z2Z_ST_HALF_RANGE : 0);
  return Z2Z_OK;
}

int32_t z2z_codebook_read(z2z_codebook* cb, int32_t b, int32_t* h_cons, int32_t* h_len,
                          z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (b < 0 || b >= cb->cfg.B) return fail(Z2Z_ERR_INVALID_ARG, "sequence index out of range");
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const int cap = cb->cfg.cap, M = cb->cfg.M;
  if (cap == 0) return Z2Z_OK;
  if (h_cons)
    Z2Z_CUDA(cudaMemcpyAsync(h_cons, cb->view.cons + (size_t)b * cap * M, (size_t)cap * M * 4,
                             cudaMemcpyDeviceToHost, s), "codebook_read");
  uint8_t* tmp = nullptr;
  if (h_len) {                                     // lengths are bytes on the device, int32 for the caller
    tmp = new (std::nothrow) uint8_t[cap];
    if (!tmp) return fail(Z2Z_ERR_INVALID_ARG, "out of host memory");
    cudaError_t e = cudaMemcpyAsync(tmp, cb->view.len + (size_t)b * cap, cap, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) { delete[] tmp; return fail_cuda(e, "codebook_read"); }
  }
  cudaError_t e = cudaStreamSynchronize(s);
  if (tmp) {
    if (e == cudaSuccess) for (int i = 0; i < cap; ++i) h_len[i] = tmp[i];
    delete[] tmp;
  }
  if (e != cudaSuccess) return fail_cuda(e, "codebook_read");
  return Z2Z_OK;
}

int32_t z2z_set_tensor_cores(z2z_codebook* cb, int32_t enable) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (enable < 0) return fail(Z2Z_ERR_INVALID_ARG, "enable must be >= 0");
  cb->use_tensor_cores = enable == 0 ? 0 : (enable % 16 == 2 ? 2 : 1);
  cb->prefill_strips = enable / 16;
  if (cb->prefill_strips > z2z::kPrefillMaxStrips) cb->prefill_strips = z2z::kPrefillMaxStrips;
  return Z2Z_OK;
}

int32_t z2z_set_encoder_half_scratch(z2z_codebook* cb, void* d_scratch, size_t bytes) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (d_scratch && (reinterpret_cast<uintptr_t>(d_scratch) & 255) != 0) return fail(Z2Z_ERR_INVALID_ARG, "scratch must be 256-byte aligned");
  cb->half_scratch = bytes > 0 ? d_scratch : nullptr;
  cb->half_bytes = d_scratch ? bytes : 0;
  return Z2Z_OK;
}

int32_t z2z_profile(z2z_codebook* cb, int32_t enable) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  cb->prof.timing = enable != 0;
  return Z2Z_OK;
}

int32_t z2z_profile_read(z2z_codebook* cb, int32_t n_classes, double* h_ms, int64_t* h_launches,
                         z2z_stream stream) {
  if (!cb) return fail(Z2Z_ERR_INVALID_ARG, "cb is NULL");
  if (n_classes < 0 || n_classes > z2z::kProfClasses) n_classes = z2z::kProfClasses;
  Z2Z_CUDA(cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)), "profile_read");
  double ms[z2z::kProfClasses] = {0, 0, 0, 0, 0};
  for (auto& r : cb->prof.recs) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess) ms[r.cls] += t;
  }
  for (int i = 0; i < n_classes; ++i) {
    if (h_ms) h_ms[i] = ms[i];
    if (h_launches) h_launches[i] = cb->prof.launches[i];
  }
  cb->prof.release_all();
  for (int i = 0; i < z2z::kProfClasses; ++i) cb->prof.launches[i] = 0;
  return Z2Z_OK;
}

int32_t z2z_codebook_destroy(z2z_codebook* cb) {
  if (cb && cb->h_frozen) cudaFreeHost(cb->h_frozen);
  delete cb;
  return Z2Z_OK;
}

}  // extern "C"
