// Two measurement aids for the benchmark: what this GPU does for a kernel that only reads memory, and what a
// launch costs when the kernel does next to nothing.  The verify step's small configurations live near the second
// number, its key/value streaming near the first; both are printed beside the results so that a roofline
// fraction can be read against what the device really gives.
#include "common.cuh"

namespace seqtree {

// Read-only stream: every thread keeps eight independent 16-byte loads in flight, grid-stride over the buffer,
// and folds what it read into one word so that the loads cannot be dropped.  Nothing is written but one word per
// CTA.
__global__ void __launch_bounds__(512) probe_stream_read_kernel(const uint4* __restrict__ src, size_t n16, unsigned long long* sink) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  uint32_t acc = 0u;
  for (; i + 7 * stride < n16; i += 8 * stride) {
    uint4 v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = __ldcs(src + i + k * stride);  // streaming: no reuse is coming
#pragma unroll
    for (int k = 0; k < 8; ++k) acc ^= v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
  }
  for (; i < n16; i += stride) {
    const uint4 v = __ldcs(src + i);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, o);
  __shared__ uint32_t part[16];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t a = 0u;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) a ^= part[w];
    sink[blockIdx.x] = a;
  }
}

// One warp, one load whose address depends on nothing, one store that depends on the load.
__global__ void probe_dependent_load_kernel(const int32_t* __restrict__ src, int32_t* dst) {
  if (threadIdx.x == 0) *dst = *src + 1;
}

}  // namespace seqtree

extern "C" int seq_tree_probe_stream_read(const void* src, size_t bytes, unsigned long long* sink, size_t sink_words, void* stream) {
  if (src == nullptr || sink == nullptr || bytes < 16 || reinterpret_cast<uintptr_t>(src) % 16 != 0) return SEQ_ERR_INVALID_ARG;
  const int grid = seqtree::device_sm_count() * 4;
  if (sink_words < (size_t)grid) return SEQ_ERR_WORKSPACE;
  seqtree::probe_stream_read_kernel<<<grid, 512, 0, (cudaStream_t)stream>>>(static_cast<const uint4*>(src), bytes / 16, sink);
  SEQ_CUDA_OK(cudaGetLastError());
  return SEQ_OK;
}

extern "C" int seq_tree_probe_dependent_load(const int32_t* src, int32_t* dst, void* stream) {
  if (src == nullptr || dst == nullptr) return SEQ_ERR_INVALID_ARG;
  seqtree::probe_dependent_load_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(src, dst);
  SEQ_CUDA_OK(cudaGetLastError());
  return SEQ_OK;
}
