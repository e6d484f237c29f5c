// Optional per-kernel timing with CUDA events.  A launcher opens a Scope naming the kernel
// and its algorithmic work (FLOPs for contractions, bytes moved once for HBM-bound passes);
// when the calling context has tracing on, the launch is bracketed by two events on its
// stream.  Off by default: a Scope then costs one thread-local pointer test.
#pragma once
#include <cuda_runtime.h>

#include <map>
#include <string>
#include <vector>

namespace mrem {

struct TraceTotals { double ms = 0, work = 0; long long launches = 0; int is_flops = 0; };

class Tracer {
 public:
  ~Tracer() { for (cudaEvent_t e : pool_) cudaEventDestroy(e); }
  void begin(const std::string& name, double work, int is_flops, cudaStream_t st) {
    Rec r{name, work, is_flops, next(), next()};
    cudaEventRecord(r.a, st);
    open_ = r;
  }
  void end(cudaStream_t st) {
    cudaEventRecord(open_.b, st);
    recs_.push_back(open_);
  }
  // Folds finished records into the totals (the caller has synchronised the stream).
  void collect() {
    for (const Rec& r : recs_) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess) continue;
      TraceTotals& t = totals_[r.name];
      t.ms += ms; t.work += r.work; t.launches += 1; t.is_flops = r.is_flops;
    }
    recs_.clear();
    used_ = 0;
  }
  void reset() { collect(); totals_.clear(); }
  const std::map<std::string, TraceTotals>& totals() const { return totals_; }

 private:
  struct Rec { std::string name; double work; int is_flops; cudaEvent_t a, b; };
  cudaEvent_t next() {
    if (used_ == pool_.size()) {
      cudaEvent_t e;
      cudaEventCreate(&e);
      pool_.push_back(e);
    }
    return pool_[used_++];
  }
  std::vector<cudaEvent_t> pool_;
  size_t used_ = 0;
  std::vector<Rec> recs_;
  Rec open_{};
  std::map<std::string, TraceTotals> totals_;
};

extern thread_local Tracer* g_tracer;

struct Scope {
  cudaStream_t st;
  bool on;
  Scope(const char* name, double work, int is_flops, cudaStream_t s) : st(s), on(g_tracer != nullptr) {
    if (on) g_tracer->begin(name, work, is_flops, st);
  }
  // name built only when tracing is on
  template <class F>
  Scope(F&& make_name, double work, int is_flops, cudaStream_t s, int) : st(s), on(g_tracer != nullptr) {
    if (on) g_tracer->begin(make_name(), work, is_flops, st);
  }
  ~Scope() { if (on) g_tracer->end(st); }
};

struct TracerGuard {              // installs a context's tracer for the duration of an API call
  Tracer* prev;
  explicit TracerGuard(Tracer* t) : prev(g_tracer) { g_tracer = t; }
  ~TracerGuard() { g_tracer = prev; }
};

}  // namespace mrem
