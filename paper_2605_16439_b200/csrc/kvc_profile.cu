// Optional per-kernel timing of kvc_decode_attend / kvc_compress with CUDA events recorded on the
// launching stream.  Off by default; the benchmark switches it on for its roofline figures.
#include <vector>

#include "kvc_internal.cuh"

namespace kvc {

struct Profile {
  bool on = false;
  size_t cap = 0;                         // bracketed launches that fit the event pool
  std::vector<cudaEvent_t> ev;            // 2 events per bracketed launch
  std::vector<int> kid;                   // kernel id per bracketed launch
};
static Profile g_prof;

bool prof_begin(int kernel_id, cudaStream_t st) {
  Profile& p = g_prof;
  if (!p.on || p.kid.size() >= p.cap) return false;
  p.kid.push_back(kernel_id);
  cudaEventRecord(p.ev[2 * (p.kid.size() - 1)], st);
  return true;
}
void prof_end(cudaStream_t st) {
  Profile& p = g_prof;
  cudaEventRecord(p.ev[2 * (p.kid.size() - 1) + 1], st);
}

}  // namespace kvc

using namespace kvc;

extern "C" {

int kvc_profile_start(int max_launches) {
  Profile& p = g_prof;
  if (max_launches < 0) return KVC_ERR_ARG;
  for (cudaEvent_t e : p.ev) cudaEventDestroy(e);
  p.ev.clear();
  p.kid.clear();
  p.ev.resize((size_t)2 * max_launches);
  for (auto& e : p.ev)
    if (cudaEventCreate(&e) != cudaSuccess) return KVC_ERR_CUDA;
  p.cap = (size_t)max_launches;
  p.kid.reserve(p.cap);
  p.on = true;
  return KVC_OK;
}

int kvc_profile_stop(void) {
  g_prof.on = false;
  return KVC_OK;
}

int kvc_profile_read(int kernel_id, double* total_ms, long long* launches) {
  Profile& p = g_prof;
  if (!total_ms || !launches || kernel_id < 0 || kernel_id >= KVC_KERNEL_COUNT) return KVC_ERR_ARG;
  double t = 0;
  long long n = 0;
  for (size_t i = 0; i < p.kid.size(); ++i) {
    if (p.kid[i] != kernel_id) continue;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, p.ev[2 * i], p.ev[2 * i + 1]) != cudaSuccess) return KVC_ERR_CUDA;
    t += ms;
    ++n;
  }
  *total_ms = t;
  *launches = n;
  return KVC_OK;
}

const char* kvc_kernel_name(int kernel_id) {
  switch (kernel_id) {
    case KVC_KERNEL_SCORES: return "scores";
    case KVC_KERNEL_EXPAND: return "expand";
    case KVC_KERNEL_OUTPUT: return "output";
    case KVC_KERNEL_GATHER_KEYS: return "gather_keys";
    case KVC_KERNEL_PROJECT_VALUES: return "project_values";
    case KVC_KERNEL_MERGE: return "merge";
    case KVC_KERNEL_COMBINE: return "combine";
    case KVC_KERNEL_FUSED: return "fused";
    case KVC_KERNEL_FUSED_TC: return "fused_tc";
    case KVC_KERNEL_FUSED_PAIR: return "fused_pair";
    case KVC_KERNEL_SPLIT_SCORES: return "split_scores";
    case KVC_KERNEL_SPLIT_EXPAND: return "split_expand";
    case KVC_KERNEL_SPLIT_OUTPUT: return "split_output";
    case KVC_KERNEL_RESIDENT: return "resident";
    default: return "?";
  }
}

}  // extern "C"
