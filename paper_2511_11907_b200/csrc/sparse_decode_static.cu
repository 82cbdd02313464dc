// kvswap_sparse_decode_static: the sparse decode attention for callers that cannot provide
// scratch memory.
//
// Some users of this library are not allowed to allocate device memory at the point where they
// call it: an inference server whose memory manager claimed the whole GPU at start-up (a later
// cudaMalloc fails or eats into someone else's budget), or code that runs inside a host
// framework's "enqueue" callback, where allocation is forbidden because cudaMalloc synchronises
// the device and can fail long after the model was loaded.  Such callers still own their inputs
// and outputs, but have nowhere to put the split-K partials that kvswap_sparse_decode keeps in
// its caller-provided workspace.  This file gives them the same computation with the partials in
// a fixed buffer that is part of the library image.
//
// The buffer is a file-scope __device__ array, so every GPU that loads the library carries its
// KVSWAP_STATIC_SCRATCH_BYTES until the process exits, whether or not this entry point is used.
#include <mutex>

#include "common.cuh"

namespace {

// Split-K partials (m, l, acc[d]) of one call.  Nothing in it has to start at zero: the split-K
// kernel overwrites every (sequence, head, split) slot the combine pass reads, so stale contents
// of an earlier call are never observed.
static __device__ __align__(256) unsigned char g_static_scratch[KVSWAP_STATIC_SCRATCH_BYTES];

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel could
// use.  The device address is looked up once per device, with that device current, and cached
// for the life of the process: a process that resets a device (cudaDeviceReset) must not call
// this entry point on it afterwards, since the cached address would be stale.
constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {};

cudaError_t scratch_address(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (ptr == nullptr) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

using namespace kvswap;

extern "C" int kvswap_sparse_decode_static(const kvswap_shape* shape, const void* q, const void* K,
                                           const void* V, const int32_t* group_idx,
                                           const int32_t* n_selected, float* out, float* lse_opt,
                                           void* cuda_stream) {
  Problem p;
  int st = resolve(shape, &p);
  if (st != KVSWAP_OK) return st;
  // The size check comes first of all: a problem that cannot run here is refused whatever else
  // is wrong with the call, before any pointer is looked at.
  Workspace w;
  plan_workspace(p, &w);
  // The first 256 bytes hold the device status word, the partials follow.
  const size_t need = 256 + sizeof(float) * size_t(p.B) * p.Hq * w.splits * (p.d + 2);
  if (need > size_t(KVSWAP_STATIC_SCRATCH_BYTES)) return KVSWAP_ERR_STATIC_SCRATCH;
  if (q == nullptr || K == nullptr || V == nullptr || group_idx == nullptr || n_selected == nullptr ||
      out == nullptr)
    return KVSWAP_ERR_NULL;
  auto mis = [](const void* ptr, uintptr_t a) { return (reinterpret_cast<uintptr_t>(ptr) & (a - 1)) != 0; };
  if (mis(q, 16) || mis(K, 16) || mis(V, 16) || mis(out, 16) || mis(group_idx, 4) || mis(n_selected, 4) ||
      (lse_opt && mis(lse_opt, 4)))
    return KVSWAP_ERR_ALIGN;
  void* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return KVSWAP_ERR_CUDA;
  cudaError_t e = launch_sparse_decode(p, w, q, K, V, group_idx, n_selected,
                                       reinterpret_cast<float*>(static_cast<char*>(scratch) + 256), out, lse_opt,
                                       static_cast<uint32_t*>(scratch), static_cast<cudaStream_t>(cuda_stream));
  return e == cudaSuccess ? KVSWAP_OK : KVSWAP_ERR_CUDA;
}
