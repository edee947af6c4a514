// Read-only streaming probe: the practical HBM read ceiling that the bandwidth figures of the HBM-bound kernels
// (dense attention over I_active rows, sink column sum, key pooling) are put beside.  No counterpart in the paper.
#include "focus_common.cuh"

namespace {
constexpr int PROBE_THREADS = 256;
constexpr int PROBE_UNROLL = 8;            // 128-bit loads in flight per thread

__global__ void __launch_bounds__(PROBE_THREADS) stream_read_kernel(const uint4* __restrict__ src, size_t n_vec,
                                                                    uint32_t* __restrict__ checksum) {
  const size_t stride = (size_t)gridDim.x * PROBE_THREADS;
  size_t i = (size_t)blockIdx.x * PROBE_THREADS + threadIdx.x;
  uint32_t acc = 0;
  for (; i + (PROBE_UNROLL - 1) * stride < n_vec; i += PROBE_UNROLL * stride) {
    uint4 v[PROBE_UNROLL];
#pragma unroll
    for (int u = 0; u < PROBE_UNROLL; ++u) v[u] = __ldcs(src + i + u * stride);     // streamed: read once
#pragma unroll
    for (int u = 0; u < PROBE_UNROLL; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
  }
  for (; i < n_vec; i += stride) {
    const uint4 v = __ldcs(src + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0 && acc != 0) atomicXor(checksum, acc);
}
}  // namespace

extern "C" focus_status focus_stream_read(focus_ctx* ctx, const void* ptr, size_t bytes, uint32_t* checksum,
                                          focus_stream stream) {
  if (!ctx || !checksum || (bytes && !ptr) || (bytes & 15) || ((uintptr_t)ptr & 15)) return FOCUS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  if (cudaMemsetAsync(checksum, 0, sizeof(uint32_t), st) != cudaSuccess) return FOCUS_ERR_CUDA;
  if (bytes == 0) return FOCUS_OK;
  const size_t n_vec = bytes / 16;
  size_t want = (n_vec + PROBE_THREADS - 1) / PROBE_THREADS;
  const size_t cap = (size_t)ctx->sm_count * 8;                    // eight resident CTAs per SM
  const unsigned grid = (unsigned)(want < cap ? want : cap);
  stream_read_kernel<<<grid, PROBE_THREADS, 0, st>>>(reinterpret_cast<const uint4*>(ptr), n_vec, checksum);
  FOCUS_CHECK_LAUNCH();
  return FOCUS_OK;
}
