// Optional per-kernel timing: when enabled, every launch site records a CUDA event on the
// caller's stream; the interval up to the next mark is attributed to the mark's name.
#include "common.cuh"
#include <cstdio>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

namespace muse {

namespace {
struct Mark { const char* name; cudaEvent_t ev; };
std::mutex g_mu;
bool g_on = false;
std::vector<Mark> g_marks;
std::vector<cudaEvent_t> g_pool;
}  // namespace

void prof_mark(const char* name, cudaStream_t st) {
  if (!g_on) return;
  std::lock_guard<std::mutex> lk(g_mu);
  cudaEvent_t ev;
  if (!g_pool.empty()) { ev = g_pool.back(); g_pool.pop_back(); }
  else if (cudaEventCreate(&ev) != cudaSuccess) return;
  cudaEventRecord(ev, st);
  g_marks.push_back({name, ev});
}

}  // namespace muse

using namespace muse;

extern "C" {

int muse_profile(int enable) {
  std::lock_guard<std::mutex> lk(g_mu);
  for (auto& m : g_marks) g_pool.push_back(m.ev);
  g_marks.clear();
  g_on = enable != 0;
  return MUSE_OK;
}

long muse_profile_report(char* buf, size_t cap) {
  std::lock_guard<std::mutex> lk(g_mu);
  if (buf == nullptr || cap == 0) return MUSE_ERR_INVALID_ARG;
  struct Agg { std::string name; long launches; double ms; };
  std::vector<Agg> agg;
  if (!g_marks.empty() && cudaEventSynchronize(g_marks.back().ev) != cudaSuccess) return MUSE_ERR_CUDA;
  for (size_t k = 0; k + 1 < g_marks.size(); ++k) {
    if (g_marks[k].name == nullptr) continue;        // end-of-call marker
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, g_marks[k].ev, g_marks[k + 1].ev) != cudaSuccess) return MUSE_ERR_CUDA;
    size_t a = 0;
    for (; a < agg.size(); ++a) if (agg[a].name == g_marks[k].name) break;
    if (a == agg.size()) agg.push_back({g_marks[k].name, 0, 0.0});
    agg[a].launches += 1; agg[a].ms += ms;
  }
  size_t used = 0;
  for (auto& a : agg) {
    int n = snprintf(buf + used, cap - used, "%s %ld %.6f\n", a.name.c_str(), a.launches, a.ms);
    if (n < 0 || (size_t)n >= cap - used) break;
    used += (size_t)n;
  }
  buf[used < cap ? used : cap - 1] = 0;
  return (long)used;
}

}  // extern "C"
