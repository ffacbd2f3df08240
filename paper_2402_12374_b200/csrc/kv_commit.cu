// seq_tree_kv_commit: the accepted path's key/value rows move to the front of the tree region, in place.
// Pure data movement, bound by latency at the paper's sizes (a few rows per plane): one thread per 16 bytes of a
// plane's rows, a batch of independent loads in flight before the batch's stores.
#include "common.cuh"

namespace seqtree {

constexpr int kCommitThreads = 256;
constexpr int kCommitBatch = 8;

struct CommitArgs {
  uint8_t* cache[2];
  int64_t plane_stride, row_stride;  // bytes
  int32_t planes, cols;              // cols = 16-byte columns per row
  int32_t L_host, n;
  const int32_t* L_dev;  // nullable: the prefix length in device memory (<= L_host)
  const int32_t* path; const int32_t* path_len;
  int32_t* new_prefix_len; int32_t* dev_status;
};

__global__ void __launch_bounds__(kCommitThreads) kv_commit_kernel(const CommitArgs a) {
  __shared__ int32_t s_path[SEQ_MAX_TREE];
  // path_len and the whole path buffer (n entries, as seq_tree_verify owns it) are fetched together: one memory
  // latency instead of two.  Every CTA checks the path for itself: 0 first, strictly ascending, below n.
  const int len = *a.path_len;
  int L = a.L_host;
  if (a.L_dev != nullptr) {
    const int v = *a.L_dev;
    if ((v < 0 || v > a.L_host) && blockIdx.x == 0 && threadIdx.x == 0) dev_flag(a.dev_status, SEQ_DEV_BAD_LENGTH);
    L = min(max(v, 0), a.L_host);
  }
  for (int i = threadIdx.x; i < a.n; i += kCommitThreads) s_path[i] = a.path[i];
  __syncthreads();
  int bad = len < 0 || len > a.n;
  if (!bad)
    for (int i = threadIdx.x; i < len; i += kCommitThreads) {
      const int v = s_path[i];
      bad |= v < 0 || v >= a.n || (i == 0 ? v != 0 : v <= s_path[i - 1]);
    }
  bad = __syncthreads_or(bad);
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (bad) dev_flag(a.dev_status, SEQ_DEV_BAD_PATH);
    if (a.new_prefix_len != nullptr) *a.new_prefix_len = L + (bad ? 0 : len);
  }
  if (bad) return;
  // rows that already sit in place (always the root, often the first levels) are skipped
  int first = 0;
  while (first < len && s_path[first] == first) ++first;
  if (first == len) return;

  const int64_t per_cache = (int64_t)a.planes * a.cols;
  const int64_t total = per_cache * (a.cache[1] != nullptr ? 2 : 1);
  for (int64_t t = (int64_t)blockIdx.x * kCommitThreads + threadIdx.x; t < total; t += (int64_t)gridDim.x * kCommitThreads) {
    const int which = t >= per_cache;
    const int64_t r = t - which * per_cache;
    const int64_t plane = r / a.cols;
    const int col = (int)(r - plane * a.cols);
    uint8_t* base = (which ? a.cache[1] : a.cache[0]) + plane * a.plane_stride + (int64_t)L * a.row_stride + (int64_t)col * 16;
    for (int i0 = first; i0 < len; i0 += kCommitBatch) {
      uint4 v[kCommitBatch];
#pragma unroll
      for (int j = 0; j < kCommitBatch; ++j)  // (past the end: the last row again, not stored)
        v[j] = *reinterpret_cast<const uint4*>(base + (int64_t)s_path[min(i0 + j, len - 1)] * a.row_stride);
#pragma unroll
      for (int j = 0; j < kCommitBatch; ++j)
        if (i0 + j < len) *reinterpret_cast<uint4*>(base + (int64_t)(i0 + j) * a.row_stride) = v[j];
    }
  }
}

}  // namespace seqtree

using namespace seqtree;

extern "C" int seq_tree_kv_commit(const seq_tree_kv_commit_params* p, void* stream) {
  if (p == nullptr || p->k_cache == nullptr || p->path == nullptr || p->path_len == nullptr) return SEQ_ERR_INVALID_ARG;
  if (p->num_planes < 1 || p->n_tree < 1 || p->n_tree > SEQ_MAX_TREE || p->prefix_len < 0) return SEQ_ERR_INVALID_ARG;
  if (p->prefix_len_dev != nullptr && p->prefix_len_dev == p->new_prefix_len) return SEQ_ERR_INVALID_ARG;  // read by some CTAs while another writes
  if (p->row_bytes < 16 || p->row_bytes % 16 != 0 || p->row_stride_bytes < p->row_bytes || p->row_stride_bytes % 16 != 0 ||
      p->plane_stride_bytes % 16 != 0 ||
      p->plane_stride_bytes < ((int64_t)p->prefix_len + p->n_tree) * p->row_stride_bytes)
    return SEQ_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(p->k_cache) % 16 != 0 || reinterpret_cast<uintptr_t>(p->v_cache) % 16 != 0)
    return SEQ_ERR_INVALID_ARG;
  CommitArgs a;
  a.cache[0] = static_cast<uint8_t*>(p->k_cache);
  a.cache[1] = static_cast<uint8_t*>(p->v_cache);
  a.plane_stride = p->plane_stride_bytes; a.row_stride = p->row_stride_bytes;
  a.planes = p->num_planes; a.cols = p->row_bytes / 16;
  a.L_host = p->prefix_len; a.L_dev = p->prefix_len_dev; a.n = p->n_tree;
  a.path = p->path; a.path_len = p->path_len;
  a.new_prefix_len = p->new_prefix_len; a.dev_status = p->dev_status;
  const int64_t total = (int64_t)a.planes * a.cols * (a.cache[1] != nullptr ? 2 : 1);
  const int64_t want = (total + kCommitThreads - 1) / kCommitThreads;
  const long cap = (long)device_sm_count() * 8;
  const int grid = (int)(want < cap ? want : cap);  // at most one wave of 8 CTAs per SM; larger caches loop
  kv_commit_kernel<<<grid, kCommitThreads, 0, static_cast<cudaStream_t>(stream)>>>(a);
  SEQ_CUDA_OK(cudaGetLastError());
  return SEQ_OK;
}
