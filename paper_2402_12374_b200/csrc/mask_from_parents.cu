// seq_tree_mask_from_parents: ancestor bitmasks of a token tree (integer work, run once per tree).
//
// One thread per node walks parent[] from its node to the root.  Because 0 <= parent[i] < i, the
// walk visits bit positions in strictly descending order, so each row is produced word by word
// from the top down and every word is written exactly once.
#include "common.cuh"

namespace seqtree {

__global__ void mask_from_parents_kernel(const int32_t* __restrict__ parent, int32_t n,
                                         uint32_t* __restrict__ mask_bits, int32_t words_per_row,
                                         int32_t* __restrict__ depth, int32_t* dev_status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint32_t* row = mask_bits + (size_t)i * words_per_row;
  int w = i >> 5;
  for (int ww = words_per_row - 1; ww > w; --ww) row[ww] = 0u;
  uint32_t acc = 0u;
  int j = i, links = 0;
  for (int step = 0; step < n; ++step) {  // a valid walk takes at most n-1 links
    const int jw = j >> 5;
    if (jw != w) {
      row[w] = acc;
      for (int ww = w - 1; ww > jw; --ww) row[ww] = 0u;
      acc = 0u;
      w = jw;
    }
    acc |= 1u << (j & 31);
    const int p = parent[j];
    if (p == -1) break;
    if (p < -1 || p >= j) {  // not an earlier node: flagged, read as "no parent"
      dev_flag(dev_status, SEQ_DEV_BAD_PARENT);
      break;
    }
    j = p;
    ++links;
  }
  row[w] = acc;
  for (int ww = w - 1; ww >= 0; --ww) row[ww] = 0u;
  if (depth != nullptr) depth[i] = links;
}

}  // namespace seqtree

extern "C" int seq_tree_mask_from_parents(const int32_t* parent, int32_t n, uint32_t* mask_bits,
                                          int32_t words_per_row, int32_t* depth,
                                          int32_t* dev_status, void* stream) {
  if (parent == nullptr || mask_bits == nullptr) return SEQ_ERR_INVALID_ARG;
  if (n < 1 || n > SEQ_MAX_TREE || words_per_row < (n + 31) / 32) return SEQ_ERR_INVALID_ARG;
  const int block = 128;
  seqtree::mask_from_parents_kernel<<<(n + block - 1) / block, block, 0, (cudaStream_t)stream>>>(
      parent, n, mask_bits, words_per_row, depth, dev_status);
  SEQ_CUDA_OK(cudaGetLastError());
  return SEQ_OK;
}

extern "C" const char* seq_tree_version(void) { return "seqtree 0.1 sm_100a"; }
