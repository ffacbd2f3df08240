// seq_tree_draft_sample: the draft side's draw of a node's children, k tokens without replacement from
// softmax(logits / T), by exponential sort (Section 5, "Implementation Details": the exponential-sort
// algorithm; Algorithm 2's line 5 for all children of a node at once).
//
// Token t gets the key E_t / q_t with E_t = -log(u_t); ascending keys are the draw order.  The kernel works
// with the logarithm of the inverse key, logit_t / T - log(-log u_t) (the softmax normaliser is the same for
// every token of a row and drops out), and takes the k largest in descending order, ties to the lower
// token.  No pass for a maximum or a sum is needed: the row is read once.
//
// One CTA per row.  Every thread computes the scores of its elements (four consecutive tokens at a time,
// 16-byte loads when the row allows them) and remembers its best; scores are kept in shared memory when the
// row fits (vocab <= 48 K), else they are recomputed from the L2-resident row when needed.  A draw is one
// block-wide arg-max over the threads' bests; only the thread that owned the winner looks through its
// elements again.
#include <float.h>
#include <math.h>

#include "common.cuh"

namespace seqtree {

constexpr int kDsThreads = 256;
constexpr int kDsWarps = kDsThreads / 32;
constexpr int kDsMaxK = 64;
constexpr int kDsSmemVocab = 48 * 1024;  // scores of rows up to this long stay in shared memory (192 KB)

struct DraftSampleArgs {
  int32_t n_rows, V, k, vec_ok;
  const float* logits; int64_t logits_stride;
  const float* uniforms; int64_t uniforms_stride;
  float inv_T;
  int32_t* out;
  int32_t* dev_status;
};

// log of the inverse key, up to the row's constant; -inf = no chance (probability 0, or a uniform outside (0,1))
__device__ __forceinline__ float ds_score(float logit, float u, float inv_T, bool& bad) {
  if (!(logit < INFINITY)) { bad = true; return -INFINITY; }  // NaN or +inf logit: flagged, never drawn
  if (!(u > 0.f && u < 1.f)) return -INFINITY;
  return logit * inv_T - logf(-logf(u));
}

__device__ __forceinline__ void ds_better(float& bs, int& bi, float s, int i) {
  if (s > bs || (s == bs && i < bi)) { bs = s; bi = i; }
}

__global__ void __launch_bounds__(kDsThreads) draft_sample_kernel(const DraftSampleArgs a) {
  extern __shared__ float ds_scores[];  // [V] when the row fits, else unused
  __shared__ float w_s[kDsWarps];
  __shared__ int w_i[kDsWarps];
  __shared__ int taken[kDsMaxK];
  __shared__ int winner_i;
  __shared__ float winner_s;
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* lrow = a.logits + (int64_t)row * a.logits_stride;
  const float* urow = a.uniforms + (int64_t)row * a.uniforms_stride;
  const bool in_smem = a.V <= kDsSmemVocab;
  bool bad = false;

  // this thread's elements: groups of four tokens, group g belongs to thread g % kDsThreads
  const int groups = (a.V + 3) >> 2;
  auto score_at = [&](int t) -> float {  // from memory, skipping tokens already drawn (recompute mode)
    return ds_score(lrow[t], urow[t], a.inv_T, bad);
  };
  float bs = -INFINITY;
  int bi = 0x7fffffff;
  for (int g = tid; g < groups; g += kDsThreads) {
    const int t0 = 4 * g;
    float s[4];
    if (a.vec_ok && t0 + 3 < a.V) {
      const float4 x = *reinterpret_cast<const float4*>(lrow + t0);
      const float4 u = *reinterpret_cast<const float4*>(urow + t0);
      s[0] = ds_score(x.x, u.x, a.inv_T, bad); s[1] = ds_score(x.y, u.y, a.inv_T, bad);
      s[2] = ds_score(x.z, u.z, a.inv_T, bad); s[3] = ds_score(x.w, u.w, a.inv_T, bad);
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) s[e] = t0 + e < a.V ? score_at(t0 + e) : -INFINITY;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (t0 + e < a.V) {
        if (in_smem) ds_scores[t0 + e] = s[e];
        ds_better(bs, bi, s[e], t0 + e);
      }
    }
  }
  if (bad) dev_flag(a.dev_status, SEQ_DEV_NONFINITE);

  int32_t* out = a.out + (int64_t)row * a.k;
  for (int r = 0; r < a.k; ++r) {
    // block-wide arg-max of the threads' bests (larger score, then lower token)
    float s = bs;
    int i = bi;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float os = __shfl_xor_sync(0xffffffffu, s, o);
      const int oi = __shfl_xor_sync(0xffffffffu, i, o);
      ds_better(s, i, os, oi);
    }
    if (lane == 0) { w_s[warp] = s; w_i[warp] = i; }
    __syncthreads();
    if (warp == 0) {
      s = lane < kDsWarps ? w_s[lane] : -INFINITY;
      i = lane < kDsWarps ? w_i[lane] : 0x7fffffff;
#pragma unroll
      for (int o = kDsWarps / 2; o > 0; o >>= 1) {
        const float os = __shfl_xor_sync(0xffffffffu, s, o);
        const int oi = __shfl_xor_sync(0xffffffffu, i, o);
        ds_better(s, i, os, oi);
      }
      if (lane == 0) {
        winner_s = s;
        winner_i = i;
        if (s > -INFINITY) { out[r] = i; taken[r] = i; }
      }
    }
    __syncthreads();
    if (!(winner_s > -INFINITY)) {  // nothing with a chance is left: the remaining draws do not exist
      for (int j = r + tid; j < a.k; j += kDsThreads) out[j] = -1;
      return;
    }
    const int wi = winner_i;
    if (((wi >> 2) % kDsThreads) == tid && r + 1 < a.k) {  // the owner of the winner finds its next best
      if (in_smem) ds_scores[wi] = -INFINITY;
      bs = -INFINITY;
      bi = 0x7fffffff;
      for (int g = tid; g < groups; g += kDsThreads) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int t = 4 * g + e;
          if (t >= a.V) break;
          float sc;
          if (in_smem) {
            sc = ds_scores[t];
          } else {
            bool gone = false;
            for (int j = 0; j <= r; ++j) gone |= taken[j] == t;
            bool ignore = false;
            sc = gone ? -INFINITY : ds_score(lrow[t], urow[t], a.inv_T, ignore);
          }
          ds_better(bs, bi, sc, t);
        }
      }
    }
  }
}

}  // namespace seqtree

using namespace seqtree;

extern "C" int seq_tree_draft_sample(const seq_tree_draft_sample_params* p, void* stream) {
  if (p == nullptr || p->draft_logits == nullptr || p->uniforms == nullptr || p->tokens_out == nullptr)
    return SEQ_ERR_INVALID_ARG;
  if (p->n_rows < 1 || p->vocab < 1 || p->k < 1 || p->k > kDsMaxK) return SEQ_ERR_INVALID_ARG;
  if (p->logits_row_stride < p->vocab || p->uniforms_row_stride < p->vocab) return SEQ_ERR_INVALID_ARG;
  if (!(p->temperature > 0.f) || isinf(p->temperature)) return SEQ_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(p->draft_logits) % 4 != 0 || reinterpret_cast<uintptr_t>(p->uniforms) % 4 != 0)
    return SEQ_ERR_INVALID_ARG;
  DraftSampleArgs a;
  a.n_rows = p->n_rows; a.V = p->vocab; a.k = p->k;
  a.logits = p->draft_logits; a.logits_stride = p->logits_row_stride;
  a.uniforms = p->uniforms; a.uniforms_stride = p->uniforms_row_stride;
  a.inv_T = 1.f / p->temperature;
  a.out = p->tokens_out;
  a.dev_status = p->dev_status;
  a.vec_ok = reinterpret_cast<uintptr_t>(p->draft_logits) % 16 == 0 && reinterpret_cast<uintptr_t>(p->uniforms) % 16 == 0 &&
             p->logits_row_stride % 4 == 0 && p->uniforms_row_stride % 4 == 0;
  const size_t smem = p->vocab <= kDsSmemVocab ? (size_t)p->vocab * sizeof(float) : 0;
  SEQ_CUDA_OK(cudaFuncSetAttribute(draft_sample_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kDsSmemVocab * sizeof(float))));
  draft_sample_kernel<<<p->n_rows, kDsThreads, smem, (cudaStream_t)stream>>>(a);
  SEQ_CUDA_OK(cudaGetLastError());
  return SEQ_OK;
}
