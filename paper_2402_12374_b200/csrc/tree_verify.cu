// seq_tree_verify: entry points, argument checks and the choice of kernel; and the walk of Algorithm 2 from the root
// with its rows in SHARED memory (sampling from the target at T > 0, the every-node hook, batches of requests, and
// devices that cannot place a cluster of 16 CTAs).  The default walk keeps its rows in registers
// (tree_verify_walk.cu); the node-parallel schedule is tree_verify_nodes.cu.
//
// Schedule.  One cluster of CTAs follows the walk (16 CTAs for a single request where the device can place such a
// cluster, 8 per request in a batched launch).  At each visited node the two logit rows
// are cut into contiguous vocabulary slices, one per CTA, brought from HBM once by bulk
// asynchronous copies and kept in shared memory as unnormalised exponentials.  Everything that is
// vocabulary-wide (max, sums, the residual's normaliser, the inverse CDF) is a block reduction
// followed by one exchange over distributed shared memory.  The walk's scalar state is replicated:
// every CTA derives it from the same exchanged numbers with the same instructions, so all CTAs take
// the same branches.
// Per visited node there is one cluster barrier (softmax statistics), per rejection one more.
//
// Arithmetic.  R and D of Algorithm 2 are never materialised.  With p, q the two softmaxes and S
// the rejected set (their entries zeroed in shared memory when rejected), the state after any
// number of rejections is
//     R[t] = max(p[t] - C q[t] - U, 0) / Z ,     D[t] = q[t] / ZD   (or 1/(V-|S|) once the
//                                                                   uniform fallback has fired)
// for scalars C, U, Z, ZD: the residual update  R <- norm(max(R - D, 0))  becomes  C += Z/ZD  (or
// U += Z/(V-|S|) after the fallback) followed by one vocabulary-wide sum for the new Z, and
// the test sum(D) = 0 is taken on the direct sum ZD of the surviving q, never a subtraction.
//
// Each warp owns a contiguous segment of its CTA's slice and keeps its exponentials relative to
// the segment's own maximum (no block-wide maximum is needed); the per-warp sums of the last pass
// are exactly the coarse levels of the final inverse CDF.
#include <cooperative_groups.h>
#include <float.h>
#include <math.h>

#include "common.cuh"
#include "tree_verify_nodes.cuh"

namespace cg = cooperative_groups;

namespace seqtree {

#ifdef SEQ_TRACE
__device__ unsigned long long g_trace[512];
__device__ int g_trace_n;
__shared__ int s_trace_i;
#define TRACE(tag)                                                        \
  do {                                                                    \
    if (blockIdx.x == 0 && threadIdx.x == 0) {                            \
      if ((tag) == 0) s_trace_i = 0;                                      \
      int _i = s_trace_i++;                                               \
      if (_i < 256) { g_trace[2 * _i] = (tag); g_trace[2 * _i + 1] = clock64(); g_trace_n = _i + 1; } \
    }                                                                     \
  } while (0)
#else
#define TRACE(tag) do { } while (0)
#endif

constexpr int kVThreads = 256;
constexpr int kVWarps = kVThreads / 32;
constexpr uint32_t kVSpinLimit = 1u << 22;


// Two instances of the kernel: clusters of 8 CTAs (portable size; batched launches and the all-nodes test hook, where
// many clusters share the GPU) and of 16 (one request per launch: the vocabulary-wide sweeps are half as long, a
// cluster barrier costs about a sixth of a microsecond more).
#define SEQ_VCL 8
#define SEQ_VNS vcl8
#include "tree_verify_impl.cuh"
#undef SEQ_VCL
#undef SEQ_VNS
#define SEQ_VCL 16
#define SEQ_VNS vcl16
#include "tree_verify_impl.cuh"
#undef SEQ_VCL
#undef SEQ_VNS

}  // namespace seqtree

using namespace seqtree;

static int verify_validate(const seq_tree_verify_params* p) {
  if (p == nullptr) return SEQ_ERR_INVALID_ARG;
  if (p->n_tree < 1 || p->n_tree > SEQ_MAX_TREE || p->vocab < 1) return SEQ_ERR_INVALID_ARG;
  if (p->parent == nullptr || p->tokens == nullptr || p->target_logits == nullptr) return SEQ_ERR_INVALID_ARG;
  if (!(p->temperature >= 0.f) || isinf(p->temperature)) return SEQ_ERR_INVALID_ARG;
  if (p->flags & ~(SEQ_VERIFY_ALL_NODES | SEQ_VERIFY_SPECINFER | SEQ_VERIFY_TARGET_SAMPLE | SEQ_VERIFY_SCHED_WALK | SEQ_VERIFY_SCHED_NODES |
                   SEQ_VERIFY_LOGITS_BF16))
    return SEQ_ERR_INVALID_ARG;
  if ((p->flags & SEQ_VERIFY_SCHED_WALK) && (p->flags & SEQ_VERIFY_SCHED_NODES)) return SEQ_ERR_INVALID_ARG;
  if ((p->flags & SEQ_VERIFY_SPECINFER) && (p->flags & SEQ_VERIFY_TARGET_SAMPLE)) return SEQ_ERR_INVALID_ARG;
  const bool all_nodes = p->flags & SEQ_VERIFY_ALL_NODES;
  if (all_nodes) {
    if (p->next_child_out == nullptr) return SEQ_ERR_INVALID_ARG;
  } else if (p->path == nullptr || p->path_len == nullptr || p->bonus_token == nullptr) {
    return SEQ_ERR_INVALID_ARG;
  }
  if (p->temperature > 0.f && p->uniforms == nullptr) return SEQ_ERR_INVALID_ARG;
  if (p->temperature > 0.f && p->draft_logits == nullptr && !(p->flags & SEQ_VERIFY_TARGET_SAMPLE)) return SEQ_ERR_INVALID_ARG;
  // rows start on 16-byte boundaries (8-byte for 16-bit logits)
  const uintptr_t base_align = (p->flags & SEQ_VERIFY_LOGITS_BF16) ? 8 : 16;
  if (p->target_row_stride < p->vocab || p->target_row_stride % 4 != 0 ||
      reinterpret_cast<uintptr_t>(p->target_logits) % base_align != 0)
    return SEQ_ERR_INVALID_ARG;
  if (p->draft_logits != nullptr &&
      (p->draft_row_stride < p->vocab || p->draft_row_stride % 4 != 0 ||
       reinterpret_cast<uintptr_t>(p->draft_logits) % base_align != 0))
    return SEQ_ERR_INVALID_ARG;
  return SEQ_OK;
}

// Which schedule a single request gets.  Measured on the paper's five shapes (bench.py, L2-cold): the walk with its
// rows in registers beats the node-parallel schedule on every one of them, so the walk is what a request gets unless
// the caller asks for the other.
static bool wants_nodes_schedule(const seq_tree_verify_params* p) {
  if (!(p->flags & SEQ_VERIFY_SCHED_NODES)) return false;
  return verify_nodes_supported(p->n_tree, p->vocab, p->flags);
}

extern "C" size_t seq_tree_verify_workspace_bytes(const seq_tree_verify_params* p) {
  if (verify_validate(p) != SEQ_OK) return 0;
  // the walk keeps all its scratch in (distributed) shared memory; the node-parallel schedule needs a few words per node
  return wants_nodes_schedule(p) ? verify_nodes_workspace_bytes(p->n_tree) : 0;
}

// One instance (cluster size) of the launch.
// Slot: a number of its own for every kernel function (two kernels can share a pointer type, hence a template instance).
template <int CL, typename Shared, int Slot, typename Kernel>
static int verify_launch_with(Kernel kernel, VerifyArgs a, int vocab, int n_clusters, bool check_only, cudaStream_t stream) {
  a.slice_cap = (((vocab + CL - 1) / CL) + 3) & ~3;
  static_assert(sizeof(Shared) % 16 == 0, "the slices behind the shared block must stay 16-byte aligned");
  const size_t dyn = sizeof(Shared) + (size_t)2 * a.slice_cap * sizeof(float);
  if (dyn > 227 * 1024) return SEQ_ERR_UNSUPPORTED;  // vocabulary too large for CL slices
  {
    // function attributes once per (kernel instance, device): the largest shared-memory size any vocabulary can ask for
    static int attr_done[64];  // (one array per instantiation of this template, i.e. per Slot)
    const int rc = once_per_device(attr_done, [&]() -> int {
      cudaFuncAttributes fa;
      SEQ_CUDA_OK(cudaFuncGetAttributes(&fa, kernel));
      SEQ_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - (int)fa.sharedSizeBytes));
      if (CL > 8) SEQ_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
      return SEQ_OK;
    });
    if (rc != SEQ_OK) return rc;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_clusters * CL);
  cfg.blockDim = dim3(kVThreads);
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CL;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // start under the previous kernel's tail (see the kernel)
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  if (check_only) {  // can a cluster of this size be placed on this device at all?
    int clusters = 0;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) != cudaSuccess) { cudaGetLastError(); return SEQ_ERR_UNSUPPORTED; }
    return clusters >= 1 ? SEQ_OK : SEQ_ERR_UNSUPPORTED;
  }
  SEQ_CUDA_OK(cudaLaunchKernelEx(&cfg, kernel, a));
  return SEQ_OK;
}

static int verify_launch(const seq_tree_verify_params* p, int batch, int64_t tree_stride, int64_t logits_stride,
                         int64_t unif_stride, int64_t resid_stride, void* stream) {
  VerifyArgs a;
  a.n = p->n_tree; a.V = p->vocab; a.flags = p->flags;
  a.slice_cap = 0;  // per instance
  a.parent = p->parent; a.tokens = p->tokens;
  a.target = p->target_logits; a.target_stride = p->target_row_stride;
  a.draft = p->draft_logits != nullptr ? p->draft_logits : p->target_logits;
  a.draft_stride = p->draft_logits != nullptr ? p->draft_row_stride : p->target_row_stride;
  a.temperature = p->temperature; a.uniforms = p->uniforms;
  a.path = p->path; a.path_len = p->path_len; a.bonus = p->bonus_token;
  a.residual_out = p->residual_out; a.next_child_out = p->next_child_out; a.dev_status = p->dev_status;
  a.tree_stride = tree_stride; a.logits_stride = logits_stride; a.unif_stride = unif_stride; a.resid_stride = resid_stride;
  cudaStream_t s = (cudaStream_t)stream;
  {  // a vocabulary that fits no instance is refused before anything touches the device
    const size_t cap8 = (((size_t)p->vocab + 7) / 8 + 3) & ~(size_t)3, cap16 = (((size_t)p->vocab + 15) / 16 + 3) & ~(size_t)3;
    const bool fits8 = sizeof(vcl8::VShared) + 8 * cap8 <= 227 * 1024, fits16 = sizeof(vcl16::VShared) + 8 * cap16 <= 227 * 1024;
    if (!fits8 && (!fits16 || batch > 0 || (p->flags & SEQ_VERIFY_ALL_NODES))) return SEQ_ERR_UNSUPPORTED;
  }

  // 16-bit logits: served by the walk with its rows in registers only (default mode and the variant without the draft
  // update, T > 0, one request, a device that places a cluster of 16)
  const bool bf16 = (p->flags & SEQ_VERIFY_LOGITS_BF16) != 0;
  if (bf16 && ((p->flags & SEQ_VERIFY_SCHED_NODES) || !verify_walk_supported(p->vocab, p->flags, p->temperature)))
    return SEQ_ERR_UNSUPPORTED;
  if (p->flags & SEQ_VERIFY_SCHED_NODES) {
    if (batch != 0 || !wants_nodes_schedule(p)) return SEQ_ERR_UNSUPPORTED;
    return launch_verify_nodes(a, p->workspace, p->workspace_bytes, 0, s);  // (checks the workspace)
  }
  // The cluster of 16 where the device can place one (asked once per device), else the cluster of 8.
  static int wide_ok[64];  // per device: 0 = not asked yet, 1 = yes, 2 = no
  int dev = 0;
  SEQ_CUDA_OK(cudaGetDevice(&dev));
  int wide = (dev >= 0 && dev < 64) ? __atomic_load_n(&wide_ok[dev], __ATOMIC_ACQUIRE) : 2;
  if (wide == 0) {  // (two threads asking at once get the same answer)
    VerifyArgs one = a;
    wide = verify_launch_with<16, vcl16::VShared, 2>(vcl16::tree_verify_kernel<false>, one, 32000, 1, true, s) == SEQ_OK ? 1 : 2;
    __atomic_store_n(&wide_ok[dev], wide, __ATOMIC_RELEASE);
  }
  if (batch > 0) {
    // A batch that fits the GPU as clusters of 16 side by side runs the walk with its rows in registers, one cluster
    // per request (one request then costs what it costs alone); a larger one the shared-memory walk on clusters of 8,
    // eighteen requests at a time.
    if (wide == 1 && batch * 16 <= device_sm_count() && verify_walk_supported(p->vocab, p->flags, p->temperature))
      return launch_verify_walk(a, false, s, batch);
    if (bf16) return SEQ_ERR_UNSUPPORTED;
    return verify_launch_with<8, vcl8::VShared, 0>(vcl8::tree_verify_kernel<true>, a, p->vocab, batch, false, s);
  }
  if (p->flags & SEQ_VERIFY_ALL_NODES)  // 18 * 8 = 144 CTAs <= 148 SMs
    return verify_launch_with<8, vcl8::VShared, 1>(vcl8::tree_verify_kernel<false>, a, p->vocab, p->n_tree < 18 ? p->n_tree : 18, false, s);
  // One request.  Vocabularies below 8192 tokens gain nothing from more CTAs.
  // the walk with its rows in registers, where a cluster of 16 can be placed and the mode is one it serves
  if (wide == 1 && verify_walk_supported(p->vocab, p->flags, p->temperature)) return launch_verify_walk(a, false, s);
  if (bf16) return SEQ_ERR_UNSUPPORTED;
  if (wide == 1 && p->vocab >= 8192)
    return verify_launch_with<16, vcl16::VShared, 2>(vcl16::tree_verify_kernel<false>, a, p->vocab, 1, false, s);
  return verify_launch_with<8, vcl8::VShared, 1>(vcl8::tree_verify_kernel<false>, a, p->vocab, 1, false, s);
}

extern "C" int seq_tree_verify(const seq_tree_verify_params* p, void* stream) {
  int rc = verify_validate(p);
  if (rc != SEQ_OK) return rc;
  return verify_launch(p, 0, 0, 0, 0, 0, stream);
}

extern "C" int seq_tree_verify_batch(const seq_tree_verify_batch_params* bp, void* stream) {
  if (bp == nullptr) return SEQ_ERR_INVALID_ARG;
  const seq_tree_verify_params* p = &bp->request0;
  int rc = verify_validate(p);
  if (rc != SEQ_OK) return rc;
  if (bp->batch < 1 || bp->batch > 65535 / 8 || (p->flags & SEQ_VERIFY_ALL_NODES)) return SEQ_ERR_INVALID_ARG;
  if (bp->tree_stride < p->n_tree || bp->uniforms_stride < p->n_tree + 1 || bp->logits_stride % 4 != 0 ||
      bp->logits_stride < (int64_t)(p->n_tree - 1) * p->target_row_stride + p->vocab ||
      (p->draft_logits != nullptr && bp->logits_stride < (int64_t)(p->n_tree - 1) * p->draft_row_stride + p->vocab) ||
      (p->residual_out != nullptr && bp->residual_stride < p->vocab))
    return SEQ_ERR_INVALID_ARG;
  return verify_launch(p, bp->batch, bp->tree_stride, bp->logits_stride, bp->uniforms_stride, bp->residual_stride, stream);
}

#ifdef SEQ_TRACE
// debug builds only: copy out and reset the phase timeline recorded by TRACE()
extern "C" int seq_debug_trace_dump(unsigned long long* host_out) {
  int n = 0;
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(&n, seqtree::g_trace_n, sizeof(int));
  if (n > 256) n = 256;
  cudaMemcpyFromSymbol(host_out, seqtree::g_trace, sizeof(unsigned long long) * 2 * n);
  int zero = 0;
  cudaMemcpyToSymbol(seqtree::g_trace_n, &zero, sizeof(int));
  return n;
}
#endif
