// Shared host/device helpers of the token-tree verification library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "seq_tree.h"

namespace seqtree {

constexpr int kHeadDim = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

#define SEQ_CUDA_OK(expr)                     \
  do {                                        \
    cudaError_t _e = (expr);                  \
    if (_e != cudaSuccess) return SEQ_ERR_CUDA; \
  } while (0)

__device__ __forceinline__ void dev_flag(int32_t* dev_status, int bit) {
  if (dev_status != nullptr) atomicOr(dev_status, bit);
}

// Maximum over the warp in one redux.sync: floats are mapped to integers in the same order (sign-magnitude to
// two's complement), -inf and +inf included.  (A NaN, which fmaxf would drop, comes out as the maximum.)
__device__ __forceinline__ float warp_max(float v) {
  int b = __float_as_int(v);
  b ^= (b >> 31) & 0x7fffffff;
  b = __reduce_max_sync(0xffffffffu, b);
  b ^= (b >> 31) & 0x7fffffff;
  return __int_as_float(b);
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <typename T>
__device__ __forceinline__ float to_float(T x);
template <>
__device__ __forceinline__ float to_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_float<__half>(__half x) { return __half2float(x); }
template <>
__device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_float(float x);
template <>
__device__ __forceinline__ float from_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ __half from_float<__half>(float x) { return __float2half_rn(x); }
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Split-KV partial results: every attention kernel writes, per (split, query head, node),
// an unnormalised fp32 accumulator row plus (m, l): the running maximum of the scores in the
// log2 domain and the sum of 2^(score - m).  combine_splits() merges them.
struct SplitLayout {
  float* o_part;  // [splits][Hq][n][128]
  float2* ml;     // [splits][Hq][n]
};

inline size_t split_workspace_bytes(int splits, int Hq, int n) {
  size_t rows = (size_t)splits * Hq * n;
  return rows * kHeadDim * sizeof(float) + rows * sizeof(float2);
}
inline SplitLayout split_layout(void* workspace, int splits, int Hq, int n) {
  SplitLayout s;
  size_t rows = (size_t)splits * Hq * n;
  s.o_part = reinterpret_cast<float*>(workspace);
  s.ml = reinterpret_cast<float2*>(s.o_part + rows * kHeadDim);
  return s;
}

// Number of SMs of the current device (asked once per device, then remembered; safe from several host threads).
int device_sm_count();

// One-time set-up of a kernel function on a device (its opt-in shared-memory size and the like): `done` is a
// per-device array of flags owned by the call site; `setup` runs once per device, races resolved by repetition
// (the attribute calls are idempotent).
template <typename F>
inline int once_per_device(int* done, F setup) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SEQ_ERR_CUDA;
  if (dev < 0 || dev >= 64) return setup();
  if (__atomic_load_n(&done[dev], __ATOMIC_ACQUIRE)) return SEQ_OK;
  const int rc = setup();
  if (rc == SEQ_OK) __atomic_store_n(&done[dev], 1, __ATOMIC_RELEASE);
  return rc;
}

// attention: argument checks shared by the entry points, and the kernels' host launchers
int validate_attention_params(const seq_tree_attention_params* p);
int launch_attention_simt(const seq_tree_attention_params& p, int splits, cudaStream_t stream);
int simt_default_splits(const seq_tree_attention_params& p);
int launch_combine_splits(const seq_tree_attention_params& p, int splits, cudaStream_t stream);

}  // namespace seqtree
