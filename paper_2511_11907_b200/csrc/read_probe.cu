// kvswap_read_probe: a read-only streaming pass over a buffer, the calibration the benchmark
// reports beside its roofline figures (what a kernel that does nothing but read reaches on this
// GPU for a given size, and what an empty launch costs).  Plain 16-byte loads, one grid-stride
// loop, four loads in flight per thread; the XOR of everything read goes to `sink` so that the
// loads cannot be dropped.
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvswap.h"

namespace {

__global__ void __launch_bounds__(256) read_probe_kernel(const uint4* __restrict__ src, size_t n_vec, uint32_t* sink) {
  const size_t stride = size_t(gridDim.x) * blockDim.x;
  size_t i = size_t(blockIdx.x) * blockDim.x + threadIdx.x;
  uint32_t acc = 0u;
  for (; i + 3 * stride < n_vec; i += 4 * stride) {
    uint4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k)
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                   : "=r"(v[k].x), "=r"(v[k].y), "=r"(v[k].z), "=r"(v[k].w) : "l"(src + i + k * stride));
#pragma unroll
    for (int k = 0; k < 4; ++k) acc ^= v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
  }
  for (; i < n_vec; i += stride) {
    const uint4 v = src[i];
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
  if (acc == 0x9e3779b9u && sink != nullptr) *sink = acc;   // practically never: keeps the loads alive
}

}  // namespace

extern "C" int kvswap_read_probe(const void* buf, size_t bytes, void* sink, void* cuda_stream) {
  if (buf == nullptr && bytes > 0) return KVSWAP_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(buf) & 15u) || (bytes & 15u)) return KVSWAP_ERR_ALIGN;
  const size_t n_vec = bytes / 16;
  // two waves of four 256-thread CTAs per SM at most; fewer for short buffers
  const size_t want = (n_vec + 256 * 4 - 1) / (256 * 4);
  const int ctas = int(want < 1 ? 1 : want > 148 * 8 ? 148 * 8 : want);
  read_probe_kernel<<<ctas, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(static_cast<const uint4*>(buf), n_vec,
                                                                              static_cast<uint32_t*>(sink));
  return cudaGetLastError() == cudaSuccess ? KVSWAP_OK : KVSWAP_ERR_CUDA;
}
