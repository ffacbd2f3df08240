// seq_tree_attention: argument checks, kernel choice and workspace sizing.
#include <math.h>

#include "common.cuh"

namespace seqtree {

// Defined in tree_attention_umma.cu.
bool umma_supported(const seq_tree_attention_params& p);
int umma_default_splits(const seq_tree_attention_params& p);
int launch_attention_umma(const seq_tree_attention_params& p, int splits, cudaStream_t stream);
size_t umma_workspace_bytes(const seq_tree_attention_params& p);

static size_t elem_size(int dtype) { return dtype == SEQ_F32 ? 4 : 2; }

int device_sm_count() {
  static int cached[64];  // 0 = not asked yet
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev >= 0 && dev < 64) {
    const int c = __atomic_load_n(&cached[dev], __ATOMIC_RELAXED);
    if (c > 0) return c;
  }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
    cudaGetLastError();
    return 148;  // no device to ask (a host without a GPU sizing a workspace): B200's count
  }
  if (dev >= 0 && dev < 64) __atomic_store_n(&cached[dev], sms, __ATOMIC_RELAXED);
  return sms;
}

int validate_attention_params(const seq_tree_attention_params* p) {
  if (p == nullptr) return SEQ_ERR_INVALID_ARG;
  if (p->q == nullptr || p->k_cache == nullptr || p->v_cache == nullptr || p->out == nullptr ||
      (p->mask_bits == nullptr && p->parent == nullptr))
    return SEQ_ERR_INVALID_ARG;
  if (p->n_tree < 1 || p->n_tree > SEQ_MAX_TREE || p->prefix_len < 0) return SEQ_ERR_INVALID_ARG;
  if (p->num_q_heads < 1 || p->num_kv_heads < 1 || p->num_q_heads % p->num_kv_heads != 0)
    return SEQ_ERR_INVALID_ARG;
  if (p->num_q_heads > 65535) return SEQ_ERR_INVALID_ARG;
  if (p->dtype != SEQ_F16 && p->dtype != SEQ_BF16 && p->dtype != SEQ_F32) return SEQ_ERR_INVALID_ARG;
  if (p->head_dim != kHeadDim) return SEQ_ERR_UNSUPPORTED;
  if ((int64_t)p->prefix_len + p->n_tree > (int64_t)p->kv_capacity) return SEQ_ERR_INVALID_ARG;
  if (p->mask_bits != nullptr && p->mask_words_per_row < (p->n_tree + 31) / 32) return SEQ_ERR_INVALID_ARG;
  if (isnan(p->softmax_scale) || isinf(p->softmax_scale)) return SEQ_ERR_INVALID_ARG;
  const size_t es = elem_size(p->dtype);
  const int64_t strides[] = {p->q_stride_tok,  p->q_stride_head, p->kv_stride_tok,
                             p->kv_stride_head, p->o_stride_tok,  p->o_stride_head};
  for (int64_t s : strides)
    if (s < kHeadDim || (s * (int64_t)es) % 16 != 0) return SEQ_ERR_INVALID_ARG;
  const void* ptrs[] = {p->q, p->k_cache, p->v_cache, p->out};
  for (const void* q : ptrs)
    if (reinterpret_cast<uintptr_t>(q) % 16 != 0) return SEQ_ERR_INVALID_ARG;
  if (p->kernel < 0 || p->kernel > 4) return SEQ_ERR_INVALID_ARG;
  if (p->prefix_len_dev_count < 0) return SEQ_ERR_INVALID_ARG;
  if (p->prefix_len_dev_count > 1 &&
      (p->prefix_len_dev == nullptr || p->num_kv_heads % p->prefix_len_dev_count != 0 || p->kernel == 3))
    return SEQ_ERR_INVALID_ARG;
  return SEQ_OK;
}

// 1 = CUDA cores, 2 = tensor cores
static int choose_kernel(const seq_tree_attention_params& p) {
  const bool ok = umma_supported(p);
  if (p.mask_bits == nullptr) return ok && p.kernel != 1 ? 2 : 0;  // only the tensor-core kernel derives the mask itself
  if (p.kernel == 1) return 1;
  if (p.kernel >= 2) return ok ? 2 : 0;
  if (!ok) return 1;
  // Measured on B200: even with a single query row per kv head (127 of the tile's 128 rows padding) the
  // tensor-core kernel is faster than the CUDA-core one, because it streams K/V once per kv head with
  // TMA while the CUDA-core kernel re-reads them for every (node, head).  The CUDA-core kernel is kept
  // for fp32 inputs and for group sizes that do not divide 128.
  return 2;
}

}  // namespace seqtree

using namespace seqtree;

extern "C" size_t seq_tree_attention_workspace_bytes(const seq_tree_attention_params* p) {
  if (validate_attention_params(p) != SEQ_OK) return 0;
  const int which = choose_kernel(*p);
  if (which == 0) return 0;
  if (which == 2) return umma_workspace_bytes(*p);  // only its stream mode (more units than SMs) needs one
  const int splits = simt_default_splits(*p);
  size_t bytes = splits > 1 ? split_workspace_bytes(splits, p->num_q_heads, p->n_tree) : 0;
  return (bytes + 255) & ~(size_t)255;
}

extern "C" int seq_tree_attention(const seq_tree_attention_params* p, void* stream) {
  int rc = validate_attention_params(p);
  if (rc != SEQ_OK) return rc;
  const int which = choose_kernel(*p);
  if (which == 0) return SEQ_ERR_UNSUPPORTED;
  if (which == 2) return launch_attention_umma(*p, umma_default_splits(*p), (cudaStream_t)stream);
  const int splits = simt_default_splits(*p);
  if (splits > 1) {
    if (p->workspace == nullptr || p->workspace_bytes < split_workspace_bytes(splits, p->num_q_heads, p->n_tree))
      return SEQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(p->workspace) % 256 != 0) return SEQ_ERR_INVALID_ARG;
  }
  return launch_attention_simt(*p, splits, (cudaStream_t)stream);
}
