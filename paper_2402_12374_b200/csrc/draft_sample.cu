// seq_tree_draft_sample: the draft side's draw of a node's children, k tokens without replacement from
// softmax(logits / T), by exponential sort (Section 5, "Implementation Details": the exponential-sort
// algorithm; the draw s_i ~ D of Algorithm 2's loop, for all children of a node at once).
//
// Token t gets the key E_t / q_t with E_t = -log(u_t); ascending keys are the draw order.  The kernels work
// with the logarithm of the inverse key, logit_t / T - log(-log u_t) (the softmax normaliser is the same for
// every token of a row and drops out), and take the k largest in descending order, ties to the lower
// token.  No pass for a maximum or a sum is needed: a row is read once.
//
// Two launches.  (1) One CTA per (row, chunk of 4096 tokens): every thread computes the scores of its 16
// tokens (16-byte loads when the rows allow them) into shared memory and remembers its best; a draw is one
// block-wide arg-max over the threads' bests, after which only the thread that owned the winner looks through
// its tokens again; the chunk's k best (score, token) pairs go to the workspace.  The k best of a row are
// among the k best of its chunks.  (2) One CTA per row draws k times from those candidates the same way.
// Many small CTAs per SM keep the special-function and load latencies of step (1) covered.
#include <float.h>
#include <math.h>

#include "common.cuh"

namespace seqtree {

constexpr int kDsThreads = 256;
constexpr int kDsWarps = kDsThreads / 32;
constexpr int kDsMaxK = 64;
constexpr int kDsChunk = 4096;                  // tokens per CTA of the first launch
constexpr int kDsPerThread = kDsChunk / kDsThreads;  // 16: four groups of four consecutive tokens

struct DraftSampleArgs {
  int32_t n_rows, V, k, vec_ok, chunks;
  const float* logits; int64_t logits_stride;
  const float* uniforms; int64_t uniforms_stride;
  float inv_T;
  int32_t* out;
  float2* cand;  // [n_rows][chunks][k] (score, token bits)
  int32_t* dev_status;
};

// -log(u) for u in (0, 1) with a relative error of a few 1e-7 everywhere.  The winners of a draw are the
// tokens with SMALL -log u, where the fast logarithm's absolute error (2^-21 near 1) would be a large relative
// one: there -log u = 2 atanh((1 - u) / (1 + u)) is summed as a series (z <= 1/3, seven terms); below 0.5 the
// fast logarithm is good to 3 ulp.
__device__ __forceinline__ float ds_neg_log(float u) {
  if (u < 0.5f) return -__logf(u);
  const float z = __fdividef(1.f - u, 1.f + u), z2 = z * z;
  float p = fmaf(z2, 1.f / 13.f, 1.f / 11.f);
  p = fmaf(p, z2, 1.f / 9.f);
  p = fmaf(p, z2, 1.f / 7.f);
  p = fmaf(p, z2, 1.f / 5.f);
  p = fmaf(p, z2, 1.f / 3.f);
  p = fmaf(p, z2, 1.f);
  return 2.f * z * p;
}
// log of the inverse key, up to the row's constant; -inf = no chance (probability 0, or a uniform outside (0,1))
__device__ __forceinline__ float ds_score(float logit, float u, float inv_T, bool& bad) {
  if (!(logit < INFINITY)) { bad = true; return -INFINITY; }  // NaN or +inf logit: flagged, never drawn
  if (!(u > 0.f && u < 1.f)) return -INFINITY;
  return logit * inv_T - __logf(ds_neg_log(u));
}

__device__ __forceinline__ void ds_better(float& bs, int& bi, float s, int i) {
  if (s > bs || (s == bs && i < bi)) { bs = s; bi = i; }
}

// Warp-wide arg-max of (s, i): larger score, then lower index, in two redux instructions (scores mapped to
// integers in the same order).  Result in every lane.
__device__ __forceinline__ void ds_warp_argmax(float& s, int& i) {
  int b = __float_as_int(s);
  b ^= (b >> 31) & 0x7fffffff;
  const int m = __reduce_max_sync(0xffffffffu, b);
  i = __reduce_min_sync(0xffffffffu, b == m ? i : 0x7fffffff);
  b = m ^ ((m >> 31) & 0x7fffffff);
  s = __int_as_float(b);
}
// Block-wide arg-max.  Result in every thread.  The per-warp results go through one of two shared buffers,
// alternating from call to call (`round`), so that one barrier per call is enough: a thread can be at most one
// call ahead of the slowest reader, which then still reads the other buffer.
__device__ __forceinline__ void ds_block_argmax(float& s, int& i, float (*w_s)[kDsWarps], int (*w_i)[kDsWarps], int round) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, buf = round & 1;
  ds_warp_argmax(s, i);
  if (lane == 0) { w_s[buf][warp] = s; w_i[buf][warp] = i; }
  __syncthreads();
  s = lane < kDsWarps ? w_s[buf][lane] : -INFINITY;
  i = lane < kDsWarps ? w_i[buf][lane] : 0x7fffffff;
  ds_warp_argmax(s, i);
}

// (1) the k best of one chunk of one row, best first; slots past the last token with a chance: (-inf, -1)
__global__ void __launch_bounds__(kDsThreads) draft_sample_chunk_kernel(const DraftSampleArgs a) {
  __shared__ float sc[kDsChunk];
  __shared__ float w_s[2][kDsWarps];
  __shared__ int w_i[2][kDsWarps];
  const int chunk = blockIdx.x, row = blockIdx.y, tid = threadIdx.x;
  const int base = chunk * kDsChunk, cnt = min(kDsChunk, a.V - base);
  const float* lrow = a.logits + (int64_t)row * a.logits_stride + base;
  const float* urow = a.uniforms + (int64_t)row * a.uniforms_stride + base;
  bool bad = false;
  float bs = -INFINITY;
  int bi = 0x7fffffff;
  // group g of four tokens belongs to thread g % 256
#pragma unroll
  for (int j = 0; j < kDsPerThread / 4; ++j) {
    const int t0 = 4 * (tid + kDsThreads * j);
    float s[4];
    if (a.vec_ok && t0 + 3 < cnt) {
      const float4 x = *reinterpret_cast<const float4*>(lrow + t0);
      const float4 u = *reinterpret_cast<const float4*>(urow + t0);
      s[0] = ds_score(x.x, u.x, a.inv_T, bad); s[1] = ds_score(x.y, u.y, a.inv_T, bad);
      s[2] = ds_score(x.z, u.z, a.inv_T, bad); s[3] = ds_score(x.w, u.w, a.inv_T, bad);
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) s[e] = t0 + e < cnt ? ds_score(lrow[t0 + e], urow[t0 + e], a.inv_T, bad) : -INFINITY;
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      sc[t0 + e] = s[e];
      if (t0 + e < cnt) ds_better(bs, bi, s[e], t0 + e);
    }
  }
  if (bad) dev_flag(a.dev_status, SEQ_DEV_NONFINITE);

  float2* cand = a.cand + ((int64_t)row * a.chunks + chunk) * a.k;
  for (int r = 0; r < a.k; ++r) {
    float s = bs;
    int i = bi;
    ds_block_argmax(s, i, w_s, w_i, r);
    if (!(s > -INFINITY)) {  // nothing with a chance is left in this chunk
      for (int j = r + tid; j < a.k; j += kDsThreads) cand[j] = make_float2(-INFINITY, __int_as_float(-1));
      return;
    }
    if (tid == 0) cand[r] = make_float2(s, __int_as_float(base + i));
    if (((i >> 2) % kDsThreads) == tid) {  // the owner of the winner finds its next best
      sc[i] = -INFINITY;
      bs = -INFINITY;
      bi = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < kDsPerThread / 4; ++j) {
        const int t0 = 4 * (tid + kDsThreads * j);
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (t0 + e < cnt) ds_better(bs, bi, sc[t0 + e], t0 + e);
      }
    }
  }
}

// (2) the k best of a row from its chunks' candidates (chunks * k of them), in draw order
__global__ void __launch_bounds__(kDsThreads) draft_sample_merge_kernel(const DraftSampleArgs a) {
  __shared__ float w_s[2][kDsWarps];
  __shared__ int w_i[2][kDsWarps];
  extern __shared__ float2 cs[];  // the row's candidates
  const int row = blockIdx.x, tid = threadIdx.x;
  const int n = a.chunks * a.k;
  const float2* cand = a.cand + (int64_t)row * n;
  for (int j = tid; j < n; j += kDsThreads) cs[j] = cand[j];
  __syncthreads();
  // candidate j belongs to thread j % 256; a thread's best is (score, token), compared like everywhere else
  auto rescan = [&](float& bs, int& bi, int& bj) {
    bs = -INFINITY; bi = 0x7fffffff; bj = -1;
    for (int j = tid; j < n; j += kDsThreads) {
      const float s = cs[j].x;
      const int t = __float_as_int(cs[j].y);
      if (t >= 0 && (s > bs || (s == bs && t < bi))) { bs = s; bi = t; bj = j; }
    }
  };
  float bs; int bi, bj;
  rescan(bs, bi, bj);
  int32_t* out = a.out + (int64_t)row * a.k;
  for (int r = 0; r < a.k; ++r) {
    float s = bs;
    int i = bi;
    ds_block_argmax(s, i, w_s, w_i, r);
    if (!(s > -INFINITY)) {  // the remaining draws do not exist
      for (int j = r + tid; j < a.k; j += kDsThreads) out[j] = -1;
      return;
    }
    if (tid == 0) out[r] = i;
    if (bi == i && bj >= 0) {  // tokens are unique among the candidates: this thread held the winner
      cs[bj] = make_float2(-INFINITY, __int_as_float(-1));
      rescan(bs, bi, bj);
    }
  }
}

}  // namespace seqtree

using namespace seqtree;

static int ds_validate(const seq_tree_draft_sample_params* p) {
  if (p == nullptr || p->draft_logits == nullptr || p->uniforms == nullptr || p->tokens_out == nullptr)
    return SEQ_ERR_INVALID_ARG;
  if (p->n_rows < 1 || p->n_rows > 65535 || p->vocab < 1 || p->k < 1 || p->k > kDsMaxK) return SEQ_ERR_INVALID_ARG;
  if (p->logits_row_stride < p->vocab || p->uniforms_row_stride < p->vocab) return SEQ_ERR_INVALID_ARG;
  if (!(p->temperature > 0.f) || isinf(p->temperature)) return SEQ_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(p->draft_logits) % 4 != 0 || reinterpret_cast<uintptr_t>(p->uniforms) % 4 != 0)
    return SEQ_ERR_INVALID_ARG;
  return SEQ_OK;
}

extern "C" size_t seq_tree_draft_sample_workspace_bytes(const seq_tree_draft_sample_params* p) {
  if (ds_validate(p) != SEQ_OK) return 0;
  const size_t chunks = (p->vocab + kDsChunk - 1) / kDsChunk;
  return (((size_t)p->n_rows * chunks * p->k * sizeof(float2)) + 255) & ~(size_t)255;
}

extern "C" int seq_tree_draft_sample(const seq_tree_draft_sample_params* p, void* stream) {
  const int rc = ds_validate(p);
  if (rc != SEQ_OK) return rc;
  const int chunks = (p->vocab + kDsChunk - 1) / kDsChunk;
  const size_t need = (size_t)p->n_rows * chunks * p->k * sizeof(float2);
  if (p->workspace == nullptr || p->workspace_bytes < need) return SEQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(p->workspace) % 8 != 0) return SEQ_ERR_INVALID_ARG;
  DraftSampleArgs a;
  a.n_rows = p->n_rows; a.V = p->vocab; a.k = p->k; a.chunks = chunks;
  a.logits = p->draft_logits; a.logits_stride = p->logits_row_stride;
  a.uniforms = p->uniforms; a.uniforms_stride = p->uniforms_row_stride;
  a.inv_T = 1.f / p->temperature;
  a.out = p->tokens_out;
  a.cand = static_cast<float2*>(p->workspace);
  a.dev_status = p->dev_status;
  // a chunk starts at a multiple of 4096 tokens, so 16-byte alignment of the rows carries over to the chunks
  a.vec_ok = reinterpret_cast<uintptr_t>(p->draft_logits) % 16 == 0 && reinterpret_cast<uintptr_t>(p->uniforms) % 16 == 0 &&
             p->logits_row_stride % 4 == 0 && p->uniforms_row_stride % 4 == 0;
  const size_t smem = (size_t)chunks * p->k * sizeof(float2);
  if (smem > 200 * 1024) return SEQ_ERR_UNSUPPORTED;  // vocabularies beyond 1.6 M tokens at k = 64
  draft_sample_chunk_kernel<<<dim3(chunks, p->n_rows), kDsThreads, 0, (cudaStream_t)stream>>>(a);
  SEQ_CUDA_OK(cudaGetLastError());
  if (smem > 48 * 1024)
    SEQ_CUDA_OK(cudaFuncSetAttribute(draft_sample_merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  draft_sample_merge_kernel<<<p->n_rows, kDsThreads, smem, (cudaStream_t)stream>>>(a);
  SEQ_CUDA_OK(cudaGetLastError());
  return SEQ_OK;
}
