// Tree-masked attention on CUDA cores: the path for small trees, for the fp32 mode and for
// shapes the tensor-core kernel does not take; plus the split-KV combine used by both kernels.
//
// One CTA per (node i, query head h, split).  Keys are taken in chunks of 32: in a chunk lane l
// scores key l (a full 128-term dot product, q broadcast from shared memory), the warp agrees on
// the running maximum, then all lanes walk the 32 keys together, each lane accumulating 4 of the
// 128 output dimensions.  A key is read only if the row may see it: j < prefix_len, or bit
// (j - prefix_len) of the row's ancestor mask.  Masked keys get probability exactly 0 and their
// K/V rows are never loaded, so junk or NaN there cannot reach the result.
#include "common.cuh"

namespace seqtree {

constexpr int kSimtWarps = 4;

template <typename T>
struct Vec16;  // 16-byte vector load of T
template <>
struct Vec16<float> {
  static constexpr int kElems = 4;
  __device__ static void load(const float* p, float* out) {
    float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  }
};
template <>
struct Vec16<__half> {
  static constexpr int kElems = 8;
  __device__ static void load(const __half* p, float* out) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const __half2* h = reinterpret_cast<const __half2*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __half22float2(h[i]);
      out[2 * i] = f.x; out[2 * i + 1] = f.y;
    }
  }
};
template <>
struct Vec16<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ static void load(const __nv_bfloat16* p, float* out) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 f = __bfloat1622float2(h[i]);
      out[2 * i] = f.x; out[2 * i + 1] = f.y;
    }
  }
};

template <typename T>
__device__ __forceinline__ void load4(const T* p, float* out);
template <>
__device__ __forceinline__ void load4<float>(const float* p, float* out) {
  float4 v = *reinterpret_cast<const float4*>(p);
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}
template <>
__device__ __forceinline__ void load4<__half>(const __half* p, float* out) {
  uint2 v = *reinterpret_cast<const uint2*>(p);
  const __half2* h = reinterpret_cast<const __half2*>(&v);
  float2 a = __half22float2(h[0]), b = __half22float2(h[1]);
  out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
}
template <>
__device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float* out) {
  uint2 v = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
  float2 a = __bfloat1622float2(h[0]), b = __bfloat1622float2(h[1]);
  out[0] = a.x; out[1] = a.y; out[2] = b.x; out[3] = b.y;
}

template <typename T>
__device__ __forceinline__ void store4(T* p, const float* v);
template <>
__device__ __forceinline__ void store4<float>(float* p, const float* v) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
template <>
__device__ __forceinline__ void store4<__half>(__half* p, const float* v) {
  __half2 a = __floats2half2_rn(v[0], v[1]), b = __floats2half2_rn(v[2], v[3]);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}
template <>
__device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, const float* v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

struct SimtArgs {
  const void* q; const void* k; const void* v; void* out;
  const uint32_t* mask_bits;
  float* lse;
  float* o_part; float2* ml;
  int64_t q_stride_tok, q_stride_head, kv_stride_tok, kv_stride_head, o_stride_tok, o_stride_head;
  int32_t n, L_host, Hq, group, mask_wpr, splits;
  int32_t L_count;       // > 1: one prefix length per request, requests stacked as heads
  const int32_t* L_dev;  // nullable: the prefix length in device memory (<= L_host)
  int32_t* dev_status;
  float scale_log2;  // softmax_scale * log2(e)
};

template <typename T>
__global__ void __launch_bounds__(kSimtWarps * 32)
tree_attention_simt_kernel(const SimtArgs a) {
  const int i = blockIdx.x, h = blockIdx.y, split = blockIdx.z;
  const int g = h / a.group;
  int L = a.L_host;
  if (a.L_dev != nullptr) {
    const int v = a.L_dev[a.L_count > 1 ? (g * a.L_count) / (a.Hq / a.group) : 0];
    if ((v < 0 || v > a.L_host) && threadIdx.x == 0) dev_flag(a.dev_status, SEQ_DEV_BAD_LENGTH);
    L = min(max(v, 0), a.L_host);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  __shared__ __align__(16) float q_s[kHeadDim];
  __shared__ float red_m[kSimtWarps], red_l[kSimtWarps];
  __shared__ __align__(16) float red_acc[kSimtWarps][kHeadDim];

  const T* q = reinterpret_cast<const T*>(a.q) + (int64_t)i * a.q_stride_tok + (int64_t)h * a.q_stride_head;
  for (int c = threadIdx.x; c < kHeadDim; c += blockDim.x) q_s[c] = to_float<T>(q[c]) * a.scale_log2;
  __syncthreads();

  const T* kbase = reinterpret_cast<const T*>(a.k) + (int64_t)g * a.kv_stride_head;
  const T* vbase = reinterpret_cast<const T*>(a.v) + (int64_t)g * a.kv_stride_head;
  const uint32_t* mrow = a.mask_bits + (size_t)i * a.mask_wpr;

  // node i can only see tree nodes <= i, so keys end at L + i + 1
  const int n_keys = L + i + 1;
  const int n_chunks = (n_keys + 31) >> 5;
  const int stride = a.splits * kSimtWarps;

  float m = -INFINITY, l = 0.f;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};

  for (int c = split * kSimtWarps + warp; c < n_chunks; c += stride) {
    const int j = (c << 5) + lane;
    bool valid = j < L;
    if (!valid && j < n_keys) {
      const int t = j - L;
      valid = (mrow[t >> 5] >> (t & 31)) & 1u;
    }
    float s = -INFINITY;
    if (valid) {
      const T* kr = kbase + (int64_t)j * a.kv_stride_tok;
      float d0 = 0.f, d1 = 0.f;
#pragma unroll
      for (int c0 = 0; c0 < kHeadDim; c0 += Vec16<T>::kElems) {
        float kv[Vec16<T>::kElems];
        Vec16<T>::load(kr + c0, kv);
#pragma unroll
        for (int e = 0; e < Vec16<T>::kElems; e += 2) {
          d0 = fmaf(kv[e], q_s[c0 + e], d0);
          d1 = fmaf(kv[e + 1], q_s[c0 + e + 1], d1);
        }
      }
      s = d0 + d1;
    }
    const float m_new = fmaxf(m, warp_max(s));
    if (m_new == -INFINITY) continue;  // nothing visible in this chunk (uniform across the warp)
    const float alpha = exp2f(m - m_new);  // m = -inf -> 0
    const float p = valid ? exp2f(s - m_new) : 0.f;
    l = l * alpha + warp_sum(p);
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] *= alpha;
    m = m_new;
    // all lanes walk the chunk's keys together, eight at a time so that the eight V loads are in flight
    // at once; keys the row cannot see have p = 0 exactly and are skipped as whole groups
    const uint32_t live = __ballot_sync(0xffffffffu, p != 0.f);
#pragma unroll
    for (int j0 = 0; j0 < 32; j0 += 8) {
      if (((live >> j0) & 0xFFu) == 0u) continue;
      float pj[8], vv[8][4];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        pj[e] = __shfl_sync(0xffffffffu, p, j0 + e);
        if (pj[e] != 0.f) load4<T>(vbase + (int64_t)((c << 5) + j0 + e) * a.kv_stride_tok + lane * 4, vv[e]);
        else vv[e][0] = vv[e][1] = vv[e][2] = vv[e][3] = 0.f;
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) {
#pragma unroll
        for (int d = 0; d < 4; ++d) acc[d] = fmaf(pj[e], vv[e][d], acc[d]);
      }
    }
  }

  // merge the warps of this CTA
  if (lane == 0) { red_m[warp] = m; red_l[warp] = l; }
  *reinterpret_cast<float4*>(&red_acc[warp][lane * 4]) = make_float4(acc[0], acc[1], acc[2], acc[3]);
  __syncthreads();
  if (warp != 0) return;
  float M = -INFINITY;
#pragma unroll
  for (int w = 0; w < kSimtWarps; ++w) M = fmaxf(M, red_m[w]);
  float Ls = 0.f, o[4] = {0.f, 0.f, 0.f, 0.f};
  if (M != -INFINITY) {
#pragma unroll
    for (int w = 0; w < kSimtWarps; ++w) {
      const float f = exp2f(red_m[w] - M);
      Ls += red_l[w] * f;
      const float4 r = *reinterpret_cast<const float4*>(&red_acc[w][lane * 4]);
      o[0] = fmaf(r.x, f, o[0]); o[1] = fmaf(r.y, f, o[1]);
      o[2] = fmaf(r.z, f, o[2]); o[3] = fmaf(r.w, f, o[3]);
    }
  }
  if (a.splits == 1) {
    const float inv = 1.f / Ls;  // the row always sees itself, so Ls > 0
#pragma unroll
    for (int e = 0; e < 4; ++e) o[e] *= inv;
    T* out = reinterpret_cast<T*>(a.out) + (int64_t)i * a.o_stride_tok + (int64_t)h * a.o_stride_head;
    store4<T>(out + lane * 4, o);
    if (a.lse != nullptr && lane == 0) a.lse[(size_t)h * a.n + i] = (M + log2f(Ls)) * kLn2;
  } else {
    const size_t row = ((size_t)split * a.Hq + h) * a.n + i;
    *reinterpret_cast<float4*>(a.o_part + row * kHeadDim + lane * 4) = make_float4(o[0], o[1], o[2], o[3]);
    if (lane == 0) a.ml[row] = make_float2(M, Ls);
  }
}

// Merge split-KV partials: one warp per (head, node) row, 4 output dimensions per lane.
template <typename T>
__global__ void __launch_bounds__(128)
combine_splits_kernel(const float* __restrict__ o_part, const float2* __restrict__ ml, int splits,
                      int Hq, int n, T* __restrict__ out, int64_t o_stride_tok, int64_t o_stride_head,
                      float* __restrict__ lse) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= Hq * n) return;
  const int h = row / n, i = row - h * n;
  const size_t rows = (size_t)Hq * n;
  float M = -INFINITY;
  for (int s = 0; s < splits; ++s) M = fmaxf(M, ml[s * rows + row].x);
  float Ls = 0.f, o[4] = {0.f, 0.f, 0.f, 0.f};
  for (int s = 0; s < splits; ++s) {
    const float2 p = ml[s * rows + row];
    if (p.x == -INFINITY) continue;
    const float f = exp2f(p.x - M);
    Ls += p.y * f;
    const float4 r = *reinterpret_cast<const float4*>(o_part + (s * rows + row) * kHeadDim + lane * 4);
    o[0] = fmaf(r.x, f, o[0]); o[1] = fmaf(r.y, f, o[1]);
    o[2] = fmaf(r.z, f, o[2]); o[3] = fmaf(r.w, f, o[3]);
  }
  const float inv = 1.f / Ls;
#pragma unroll
  for (int e = 0; e < 4; ++e) o[e] *= inv;
  store4<T>(out + (int64_t)i * o_stride_tok + (int64_t)h * o_stride_head + lane * 4, o);
  if (lse != nullptr && lane == 0) lse[row] = (M + log2f(Ls)) * kLn2;
}

int simt_default_splits(const seq_tree_attention_params& p) {
  // aim for a few CTAs per SM; each split should still own at least ~4 chunks of 32 keys per warp
  const long rows = (long)p.n_tree * p.num_q_heads;
  const int chunks = (p.prefix_len + p.n_tree + 31) / 32;
  int splits = 1;
  while (rows * splits < device_sm_count() * 4 && chunks / (splits * 2 * kSimtWarps) >= 4 && splits < 16) splits *= 2;
  return splits;
}

template <typename T>
static int launch_simt_t(const seq_tree_attention_params& p, int splits, cudaStream_t stream) {
  SimtArgs a;
  a.q = p.q; a.k = p.k_cache; a.v = p.v_cache; a.out = p.out;
  a.mask_bits = p.mask_bits; a.lse = p.lse;
  SplitLayout sl = split_layout(p.workspace, splits, p.num_q_heads, p.n_tree);
  a.o_part = sl.o_part; a.ml = sl.ml;
  a.q_stride_tok = p.q_stride_tok; a.q_stride_head = p.q_stride_head;
  a.kv_stride_tok = p.kv_stride_tok; a.kv_stride_head = p.kv_stride_head;
  a.o_stride_tok = p.o_stride_tok; a.o_stride_head = p.o_stride_head;
  a.n = p.n_tree; a.L_host = p.prefix_len; a.L_dev = p.prefix_len_dev; a.L_count = p.prefix_len_dev_count; a.dev_status = p.dev_status; a.Hq = p.num_q_heads; a.group = p.num_q_heads / p.num_kv_heads;
  a.mask_wpr = p.mask_words_per_row; a.splits = splits;
  const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 0.08838834764831845f;
  a.scale_log2 = scale * kLog2e;
  dim3 grid(p.n_tree, p.num_q_heads, splits);
  tree_attention_simt_kernel<T><<<grid, kSimtWarps * 32, 0, stream>>>(a);
  SEQ_CUDA_OK(cudaGetLastError());
  if (splits > 1) return launch_combine_splits(p, splits, stream);
  return SEQ_OK;
}

int launch_attention_simt(const seq_tree_attention_params& p, int splits, cudaStream_t stream) {
  switch (p.dtype) {
    case SEQ_F16: return launch_simt_t<__half>(p, splits, stream);
    case SEQ_BF16: return launch_simt_t<__nv_bfloat16>(p, splits, stream);
    case SEQ_F32: return launch_simt_t<float>(p, splits, stream);
  }
  return SEQ_ERR_INVALID_ARG;
}

template <typename T>
static int launch_combine_t(const seq_tree_attention_params& p, int splits, cudaStream_t stream) {
  SplitLayout sl = split_layout(p.workspace, splits, p.num_q_heads, p.n_tree);
  const int rows = p.num_q_heads * p.n_tree;
  combine_splits_kernel<T><<<(rows + 3) / 4, 128, 0, stream>>>(
      sl.o_part, sl.ml, splits, p.num_q_heads, p.n_tree, reinterpret_cast<T*>(p.out), p.o_stride_tok,
      p.o_stride_head, p.lse);
  SEQ_CUDA_OK(cudaGetLastError());
  return SEQ_OK;
}

int launch_combine_splits(const seq_tree_attention_params& p, int splits, cudaStream_t stream) {
  switch (p.dtype) {
    case SEQ_F16: return launch_combine_t<__half>(p, splits, stream);
    case SEQ_BF16: return launch_combine_t<__nv_bfloat16>(p, splits, stream);
    case SEQ_F32: return launch_combine_t<float>(p, splits, stream);
  }
  return SEQ_ERR_INVALID_ARG;
}

}  // namespace seqtree

// ---------------------------------------------------------------------------------------------------
// seq_tree_attention_noalloc: the same CUDA-core kernels, with the split-KV partials in a fixed array
// that is part of the library image instead of a caller-provided workspace.
//
// `g_noalloc_scratch` names the array in device code.  In host code the same identifier is only a
// handle for the runtime: its device address has to be asked for with cudaGetSymbolAddress, once per
// device, with that device current; passing the identifier itself to a kernel would hand it a host
// address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SEQ_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_noalloc_ptr[kMaxDevices];  // device address of g_noalloc_scratch on each device, 0 = not looked up yet
}  // namespace

extern "C" int seq_tree_attention_noalloc(const seq_tree_attention_params* p, void* stream) {
  using namespace seqtree;
  int rc = validate_attention_params(p);
  if (rc != SEQ_OK) return rc;
  if (p->mask_bits == nullptr) return SEQ_ERR_UNSUPPORTED;  // the CUDA-core kernel does not derive the mask itself
  const int splits = simt_default_splits(*p);
  const size_t need = splits > 1 ? split_workspace_bytes(splits, p->num_q_heads, p->n_tree) : 0;
  if (need > SEQ_NOALLOC_SCRATCH_BYTES) return SEQ_ERR_WORKSPACE;  // too large for the built-in array

  int dev = -1;
  SEQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return SEQ_ERR_UNSUPPORTED;
  if (g_noalloc_ptr[dev] == nullptr) {  // set-up: first call on this device
    void* ptr = nullptr;
    SEQ_CUDA_OK(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
    if (ptr == nullptr) return SEQ_ERR_CUDA;
    g_noalloc_ptr[dev] = ptr;
  }
  seq_tree_attention_params q = *p;
  q.workspace = g_noalloc_ptr[dev];
  q.workspace_bytes = SEQ_NOALLOC_SCRATCH_BYTES;
  q.kernel = 1;
  return launch_attention_simt(q, splits, (cudaStream_t)stream);
}
