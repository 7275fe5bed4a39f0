// Launch accounting and optional per-kernel-class CUDA-event timing (host side only).
// Counting is always on; event recording only between z2z_profile(cb, 1) and z2z_profile(cb, 0).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

namespace z2z {

enum ProfClass {
  kProfLogits = 0,       // joint-logits main kernel
  kProfLogitsMerge = 1,  // merge of partial reductions, code selection
  kProfLzw = 2,          // codebook clear / encode / step
  kProfEncGemm = 3,      // hyper-encoder linear layers
  kProfEncOther = 4,     // gather, LayerNorm, attention, pooling, work lists
  kProfClasses = 5
};

struct Prof {
  bool timing = false;
  int64_t launches[kProfClasses] = {0, 0, 0, 0, 0};
  struct Rec { int cls; cudaEvent_t a, b; };
  std::vector<Rec> recs;
  std::vector<cudaEvent_t> pool;
  size_t max_events = 1 << 17;

  cudaEvent_t get_event() {
    if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    return e;
  }
  void release_all() {
    for (auto& r : recs) { pool.push_back(r.a); pool.push_back(r.b); }
    recs.clear();
  }
  ~Prof() {
    release_all();
    for (auto e : pool) cudaEventDestroy(e);
  }
};

// Brackets a group of launches of one class on a stream.
struct ProfScope {
  Prof* p; cudaStream_t s; cudaEvent_t b = nullptr;
  ProfScope(Prof* prof, int cls, int n_launches, cudaStream_t stream) : p(prof), s(stream) {
    if (!p) return;
    p->launches[cls] += n_launches;
    if (p->timing && p->recs.size() * 2 < p->max_events) {
      cudaEvent_t a = p->get_event();
      b = p->get_event();
      if (a && b) { cudaEventRecord(a, s); p->recs.push_back({cls, a, b}); }
      else b = nullptr;
    }
  }
  ~ProfScope() { if (b) cudaEventRecord(b, s); }
};

}  // namespace z2z
