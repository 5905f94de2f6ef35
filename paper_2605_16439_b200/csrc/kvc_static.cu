// kvc_decode_attend_static: the decode call for callers that cannot hand the library a scratch buffer
// because they cannot allocate device memory at the point of the call (a serving loop whose memory
// pool is already fully committed to KV blocks, a plug-in running inside someone else's allocator
// with allocation forbidden, a context where cudaMalloc's implicit synchronisation is not tolerable).
// The scratch of kvc_decode_attend lives here in a fixed array in the library's own device image.
#include <mutex>

#include "kvc_internal.cuh"

// Fixed scratch, resident on every GPU that loads this library until the process exits.
static __device__ __align__(256) unsigned char kvc_static_scratch[KVC_STATIC_SCRATCH_BYTES];

namespace {

constexpr int MAX_DEVICES = 64;
std::mutex g_mu;
void* g_scratch_ptr[MAX_DEVICES];   // device address of kvc_static_scratch, per device ordinal
bool g_ready[MAX_DEVICES];

// In host code the array's name is only a handle: the address kernels can use must be asked for,
// once per device and with that device current.
int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return KVC_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_ready[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, kvc_static_scratch) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return KVC_ERR_CUDA;
    }
    g_scratch_ptr[dev] = p;
    g_ready[dev] = true;
  }
  *out = g_scratch_ptr[dev];
  return KVC_OK;
}

}  // namespace

namespace kvc {
int static_scratch(void** out) { return scratch_for_current_device(out); }
}  // namespace kvc

extern "C" {

size_t kvc_static_scratch_bytes(void) { return (size_t)KVC_STATIC_SCRATCH_BYTES; }

int kvc_decode_attend_static(const kvc_layer* L, const void* q, const void* capsules, int B, int R,
                             const void* K_txt, const void* V_txt, int T, int T_cap, void* out, void* stream) {
  if (!L || B < 0 || R < 0 || T < 0 || T_cap < T) return KVC_ERR_ARG;
  if (kvc::ws_layout(L, B, R, T).total > (size_t)KVC_STATIC_SCRATCH_BYTES) return KVC_ERR_WORKSPACE;
  void* scratch = nullptr;
  const int s = scratch_for_current_device(&scratch);
  if (s != KVC_OK) return s;
  return kvc::decode_common(L, q, capsules, B, R, K_txt, V_txt, T, T_cap, out, scratch,
                            static_cast<cudaStream_t>(stream));
}

}  // extern "C"
