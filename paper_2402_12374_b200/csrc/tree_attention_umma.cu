// Tensor-core (tcgen05 + TMEM + TMA) tree attention.  Placeholder until the kernel lands.
#include "common.cuh"

namespace seqtree {
bool umma_supported(const seq_tree_attention_params&) { return false; }
int umma_default_splits(const seq_tree_attention_params&) { return 1; }
int launch_attention_umma(const seq_tree_attention_params&, int, cudaStream_t) { return SEQ_ERR_UNSUPPORTED; }
}  // namespace seqtree
