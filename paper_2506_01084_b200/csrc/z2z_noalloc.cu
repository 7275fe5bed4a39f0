// z2z_logits_static_scratch: joint logits with the reductions, for callers that cannot allocate
// device memory: a plug-in inside a serving process that handed out all of its device memory at
// start-up, a callback running where the framework's allocator must not be entered, a process
// already at its memory limit.  The ordinary entry point keeps the per-CTA partial reductions in
// a workspace the caller allocates; this one keeps them in a fixed array that is part of the
// library image, so the caller passes inputs and outputs only and needs no session handle.
//
// The array exists once per GPU that loads the library and is held until the process exits.
// Its device address is looked up on the first call made on each device (the device that is
// current at that call); make that first call outside any stream capture.  Every call on a
// device shares the array and leaves its partials behind.  Nothing in it has to start at zero:
// every record the merge kernel reads is written by the main kernel of the same call first.
// Two calls that overlap on one GPU (different streams) would overwrite each other's partials,
// so the caller has to order them.
#include <cstdio>
#include <mutex>

#include "z2z_common.cuh"
#include "z2z_internal.h"

namespace {

constexpr int kNoAllocMaxRows = 1024;                       // hidden rows per call
constexpr size_t kNoAllocScratchBytes = (size_t)2 << 20;    // 65536 partial records of 32 bytes
constexpr int kNoAllocMaxDevices = 64;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

// Device address of the array on each device, looked up once per device.  In host code the
// array's name only stands for the symbol; the address a kernel can use comes from the runtime.
void* g_scratch_addr[kNoAllocMaxDevices] = {nullptr};
std::mutex g_scratch_mu;

cudaError_t scratch_for_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kNoAllocMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_scratch_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);        // for the device that is current
    if (e != cudaSuccess) return e;
    if (!p) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" {

int32_t z2z_logits_static_scratch(const void* d_hidden, int32_t N, const int32_t* d_row_seq,
                                  const int32_t* d_n_hyper, const void* d_WU, const void* d_Uh,
                                  int32_t V, int32_t d, int32_t B, int32_t cap, int32_t dtype,
                                  float* d_lse, int32_t* d_argmax, float* d_max_logit,
                                  z2z_stream stream) {
  auto fail = [](int code, const char* msg) { z2z::set_last_error(msg); return code; };
  if (N < 0) return fail(Z2Z_ERR_INVALID_ARG, "N < 0");
  if (N > kNoAllocMaxRows) return fail(Z2Z_ERR_INVALID_ARG, "N exceeds the 1024 rows the built-in scratch array is sized for");
  if (V < 1 || d < 8 || d % 8 != 0 || B < 1 || B > 1024 || cap < 0 || cap > 65535)
    return fail(Z2Z_ERR_INVALID_ARG, "need V >= 1, d >= 8, d % 8 == 0, 1 <= B <= 1024, 0 <= cap <= 65535");
  if (dtype != Z2Z_DTYPE_FP32 && dtype != Z2Z_DTYPE_BF16) return fail(Z2Z_ERR_INVALID_ARG, "unknown dtype");
  if (N == 0) return Z2Z_OK;
  if (!d_hidden || !d_WU || !d_n_hyper) return fail(Z2Z_ERR_INVALID_ARG, "d_hidden / d_WU / d_n_hyper is NULL");
  if (!d_Uh && cap > 0) return fail(Z2Z_ERR_INVALID_ARG, "d_Uh is NULL");
  if (!d_row_seq && N > B) return fail(Z2Z_ERR_INVALID_ARG, "d_row_seq is required when N > B");
  void* scratch = nullptr;
  cudaError_t e = scratch_for_current_device(&scratch);
  if (e != cudaSuccess) {
    char msg[200];
    snprintf(msg, sizeof(msg), "built-in scratch array lookup: %s", cudaGetErrorString(e));
    return fail(Z2Z_ERR_CUDA, msg);
  }
  z2z::CbView cb{};
  cb.V = V; cb.M = 1; cb.cap = cap; cb.B = B; cb.n_slots = 0;
  cb.n = const_cast<int32_t*>(d_n_hyper);                   // only read by the logits kernels
  z2z::LogitsArgs a{};
  a.d = d; a.dtype = dtype; a.N = N;
  a.hidden = d_hidden; a.row_seq = d_row_seq; a.row_nvis = nullptr; a.WU = d_WU; a.Uh = d_Uh;
  a.select = Z2Z_SELECT_ARGMAX; a.inv_temperature = 1.0f; a.seed = 0; a.step = 0;
  a.lse = d_lse; a.argmax = d_argmax; a.max_logit = d_max_logit;
  a.lpart = scratch; a.lpart_bytes = kNoAllocScratchBytes; a.row_base = 0;
  e = z2z::run_logits_simt(cb, a, nullptr, nullptr, reinterpret_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) {
    char msg[200];
    snprintf(msg, sizeof(msg), "logits (built-in scratch): %s", cudaGetErrorString(e));
    return fail(Z2Z_ERR_CUDA, msg);
  }
  return Z2Z_OK;
}

}  // extern "C"
