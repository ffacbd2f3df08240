// seq_tree_top_p_filter: nucleus truncation of softmax(logits / T), row by row (the top-p hyperparameter of the
// robustness study, Section 4.2).  One CTA per row.  A histogram of the probability MASS over 2048 equal steps of the
// exponent argument finds the bin in which the cut falls; the tokens of that bin (a few dozen on the paper's shapes)
// are ordered exactly in shared memory by (logit bits, token id); a flat row or a long run of equal logits, whose bin
// holds more than 1024 tokens, takes a radix select on the logit bits (11 + 11 + 10) instead.  Masses are 2^-40 fixed
// point in 64-bit integers: sums are exact and independent of the order of the atomic adds, so the kept set is
// reproducible bit for bit.  A row is read four times (maximum, histogram, collect, write), once from HBM and then
// from L2.
#include <climits>

#include "common.cuh"

namespace seqtree {

constexpr int kTpThreads = 1024;
constexpr int kTpWarps = kTpThreads / 32;
constexpr float kTpScale = 1099511627776.f;  // 2^40
constexpr int kTpCand = 1024;  // tokens of the cut's bin that are ordered in shared memory (more: radix select)

struct TopPArgs {
  const float* logits; int64_t in_stride;
  float* out; int64_t out_stride;
  int32_t V;
  float c2;       // log2(e) / T
  double top_p;
  int32_t* kept_out; int32_t* dev_status;
};

struct TpShared {
  unsigned long long hist[2048];
  // first-level histogram as three 32-bit limbs per bin (native 32-bit shared-memory adds; a 64-bit add is a
  // compare-and-swap loop): mass = lo + hi * 2^21 + top * 2^53, carries moved up when an add wraps
  uint32_t lo[2048], hi[2048], top[2048];
  uint32_t count[1024];
  unsigned long long warp_tot[kTpWarps];
  float warp_max[kTpWarps];
  // results of a level's search
  uint32_t sel_bin; unsigned long long sel_above; unsigned long long sel_mass; uint32_t sel_count;
  int32_t tie_limit;
  int32_t bad, kept, ncand;
  unsigned long long tau_comp;
  unsigned long long sorted_c[kTpCand], sorted_w[kTpCand];  // the cut's bin in order: (key, ~index) and mass
};

// order-preserving map float -> uint32 (ascending)
__device__ __forceinline__ uint32_t tp_key(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
// NaN and +inf count as -inf (never kept)
__device__ __forceinline__ float tp_clean(float x, int& bad) {
  if (!(x < INFINITY)) { bad = 1; return -INFINITY; }
  return x;
}
__device__ __forceinline__ float tp_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ unsigned long long tp_mass(float x, float M, float c2) {
  return __float2ull_rn(tp_ex2((x - M) * c2) * kTpScale);  // (-inf - M) * c2 = -inf -> 0
}

// calls f(index, value) for every element of the row: float4 body with four independent loads in flight per
// thread (the passes are latency-bound otherwise), scalar tail
template <typename F>
__device__ __forceinline__ void tp_for_each(const float* row, int V, F f) {
  const int V4 = V & ~3;
  constexpr int kStride = kTpThreads * 4;
  int i = threadIdx.x * 4;
  for (; i + 3 * kStride < V4; i += 4 * kStride) {
    float4 x[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) x[k] = *reinterpret_cast<const float4*>(row + i + k * kStride);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int j = i + k * kStride;
      f(j, x[k].x); f(j + 1, x[k].y); f(j + 2, x[k].z); f(j + 3, x[k].w);
    }
  }
  {  // up to three more, again loaded together
    float4 x[3];
#pragma unroll
    for (int k = 0; k < 3; ++k)
      if (i + k * kStride < V4) x[k] = *reinterpret_cast<const float4*>(row + i + k * kStride);
#pragma unroll
    for (int k = 0; k < 3; ++k)
      if (i + k * kStride < V4) {
        const int j = i + k * kStride;
        f(j, x[k].x); f(j + 1, x[k].y); f(j + 2, x[k].z); f(j + 3, x[k].w);
      }
  }
  for (int t = V4 + threadIdx.x; t < V; t += kTpThreads) f(t, row[t]);
}

// Exclusive prefix sum over the block's threads in thread order; every thread also gets the total.
__device__ __forceinline__ unsigned long long tp_block_scan(unsigned long long v, TpShared& sh, unsigned long long& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  unsigned long long inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long up = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += up;
  }
  __syncthreads();  // warp_tot free for reuse
  if (lane == 31) sh.warp_tot[warp] = inc;
  __syncthreads();
  unsigned long long before = 0, all = 0;
#pragma unroll 1
  for (int w = 0; w < kTpWarps; ++w) {
    const unsigned long long t = sh.warp_tot[w];
    if (w < warp) before += t;
    all += t;
  }
  total = all;
  return before + inc - v;
}

// Among `bins` bins of sh.hist taken from the highest index down, finds the one in which the running mass reaches
// `target` (> 0, <= the bins' total); leaves its index, the mass above it, its own mass (and token count when
// `with_count`) in sh.sel_*.  bins is 2048 or 1024: two or one bin per thread.
__device__ __forceinline__ void tp_find_crossing(TpShared& sh, int bins, unsigned long long target, bool with_count) {
  const int per = bins / kTpThreads;  // 2 or 1
  const int hi = bins - 1 - (int)threadIdx.x * per;  // this thread's highest bin
  unsigned long long m0 = sh.hist[hi], m1 = per == 2 ? sh.hist[hi - 1] : 0ull;
  unsigned long long total;
  const unsigned long long above = tp_block_scan(m0 + m1, sh, total);
  if (above < target && target <= above + m0) {
    sh.sel_bin = hi; sh.sel_above = above; sh.sel_mass = m0; sh.sel_count = with_count ? sh.count[hi] : 0u;
  } else if (per == 2 && above + m0 < target && target <= above + m0 + m1) {
    sh.sel_bin = hi - 1; sh.sel_above = above + m0; sh.sel_mass = m1; sh.sel_count = with_count ? sh.count[hi - 1] : 0u;
  }
  __syncthreads();
}

// First-level bin of a (cleaned) logit: 2048 equal steps of the exponent argument d = (M - x) * log2(e) / T over
// [0, 40), most probable tokens in the highest bin; -1 beyond (mass below one unit of the fixed point: never kept).
// Sub, multiply by a positive constant and truncation are monotone, so a higher bin never holds a smaller logit.
__device__ __forceinline__ int tp_lbin(float x, float M, float c2) {
  const float d = (M - x) * c2;
  return d < 40.f ? 2047 - (int)(d * 51.2f) : -1;
}

__global__ void __launch_bounds__(kTpThreads, 1) top_p_filter_kernel(const TopPArgs a) {
  extern __shared__ __align__(16) uint8_t tp_smem[];
  TpShared& sh = *reinterpret_cast<TpShared*>(tp_smem);
  const float* row = a.logits + (int64_t)blockIdx.x * a.in_stride;
  float* orow = a.out + (int64_t)blockIdx.x * a.out_stride;
  const int V = a.V, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

  // ---- the row maximum (NaN / +inf flagged and read as -inf), histogram cleared meanwhile
  for (int i = threadIdx.x; i < 2048; i += kTpThreads) { sh.lo[i] = 0u; sh.hi[i] = 0u; sh.top[i] = 0u; }
  if (threadIdx.x == 0) { sh.bad = 0; sh.kept = 0; sh.tie_limit = INT_MAX; sh.ncand = 0; sh.tau_comp = 0ull; }
  int bad = 0;
  float m = -INFINITY;
  tp_for_each(row, V, [&](int, float x) { m = fmaxf(m, tp_clean(x, bad)); });
  m = warp_max(m);
  if (lane == 0) sh.warp_max[warp] = m;
  __syncthreads();
  float M = -INFINITY;
#pragma unroll 1
  for (int w = 0; w < kTpWarps; ++w) M = fmaxf(M, sh.warp_max[w]);
  if (bad) sh.bad = 1;
  if (M == -INFINITY) {  // no token with any mass: nothing to keep
    tp_for_each(row, V, [&](int i, float) { orow[i] = -INFINITY; });
    bad = __syncthreads_or(bad);
    if (threadIdx.x == 0) {
      dev_flag(a.dev_status, SEQ_DEV_DEGENERATE | (bad ? SEQ_DEV_NONFINITE : 0));
      if (a.kept_out != nullptr) a.kept_out[blockIdx.x] = 0;
    }
    return;
  }

  // ---- first level: every token with mass, equal steps of the exponent argument (tokens spread over many bins:
  // few collisions between the atomic adds, and the bin of the cut holds few tokens)
  tp_for_each(row, V, [&](int, float x) {
    int b2 = 0;
    x = tp_clean(x, b2);
    const int lb = tp_lbin(x, M, a.c2);
    if (lb >= 0) {
      const unsigned long long w = tp_mass(x, M, a.c2);
      const uint32_t l = (uint32_t)w & 0x1fffffu, h = (uint32_t)(w >> 21);
      uint32_t carry = h;
      if (l) {
        const uint32_t old = atomicAdd(&sh.lo[lb], l);
        carry += (old + l < old) ? 2048u : 0u;  // a wrap of lo is 2^32 = 2048 units of hi
      }
      if (carry) {
        const uint32_t old = atomicAdd(&sh.hi[lb], carry);
        if (old + carry < old) atomicAdd(&sh.top[lb], 1u);
      }
    }
  });
  __syncthreads();
  for (int i = threadIdx.x; i < 2048; i += kTpThreads)
    sh.hist[i] = (unsigned long long)sh.lo[i] + ((unsigned long long)sh.hi[i] << 21) + ((unsigned long long)sh.top[i] << 53);
  __syncthreads();
  unsigned long long target;
  {
    // the whole mass, then the mass the nucleus has to reach (rounded up, at least one unit)
    const unsigned long long mine = sh.hist[2 * threadIdx.x] + sh.hist[2 * threadIdx.x + 1];
    unsigned long long S;
    tp_block_scan(mine, sh, S);
    const double want = ceil(a.top_p * (double)S);
    target = want < 1.0 ? 1ull : (want >= (double)S ? S : (unsigned long long)want);
  }
  tp_find_crossing(sh, 2048, target, false);
  const int B0 = (int)sh.sel_bin;                    // the bin in which the cut falls
  const unsigned long long rest0 = target - sh.sel_above;  // mass still to find inside it
  __syncthreads();

  // ---- the tokens of that bin, as (key, ~index) so that a larger value means "earlier in the order"
  unsigned long long* cand = sh.hist;               // [kTpCand]   (the histogram is no longer needed)
  unsigned long long* cand_w = sh.hist + kTpCand;   // [kTpCand]
  tp_for_each(row, V, [&](int i, float x) {
    int b2 = 0;
    x = tp_clean(x, b2);
    if (tp_lbin(x, M, a.c2) == B0) {
      const int pos = atomicAdd(&sh.ncand, 1);
      if (pos < kTpCand) {
        cand[pos] = ((unsigned long long)tp_key(x) << 32) | (uint32_t)~(uint32_t)i;
        cand_w[pos] = tp_mass(x, M, a.c2);
      }
    }
  });
  __syncthreads();
  const int ncand = sh.ncand;
  uint32_t tau = 0;          // fallback only: key of the least probable kept token
  bool exact = ncand <= kTpCand;
  if (exact) {
    // rank every candidate among the others (all distinct), lay them out in order, scan the masses
    unsigned long long my_w = 0, my_c = 0;
    if ((int)threadIdx.x < ncand) {
      my_c = cand[threadIdx.x];
      my_w = cand_w[threadIdx.x];
      int rank = 0;
#pragma unroll 4
      for (int j = 0; j < ncand; ++j) rank += cand[j] > my_c;
      sh.sorted_c[rank] = my_c;
      sh.sorted_w[rank] = my_w;
    }
    __syncthreads();
    const unsigned long long w = (int)threadIdx.x < ncand ? sh.sorted_w[threadIdx.x] : 0ull;
    unsigned long long total;
    const unsigned long long before = tp_block_scan(w, sh, total);
    if ((int)threadIdx.x < ncand && before < rest0 && rest0 <= before + w) sh.tau_comp = sh.sorted_c[threadIdx.x];
    __syncthreads();
  } else {
    // ---- many tokens in one bin (a flat row, runs of equal logits): radix select on the key bits inside the bin
    __syncthreads();
    for (int i = threadIdx.x; i < 2048; i += kTpThreads) sh.hist[i] = 0ull;
    __syncthreads();
    tp_for_each(row, V, [&](int, float x) {
      int b2 = 0;
      x = tp_clean(x, b2);
      if (tp_lbin(x, M, a.c2) == B0) atomicAdd(&sh.hist[tp_key(x) >> 21], tp_mass(x, M, a.c2));
    });
    __syncthreads();
    tp_find_crossing(sh, 2048, rest0, false);
    const uint32_t p0 = sh.sel_bin;
    const unsigned long long above0 = sh.sel_above;
    __syncthreads();
    for (int i = threadIdx.x; i < 2048; i += kTpThreads) sh.hist[i] = 0ull;
    __syncthreads();
    tp_for_each(row, V, [&](int, float x) {
      int b2 = 0;
      x = tp_clean(x, b2);
      const uint32_t k = tp_key(x);
      if ((k >> 21) == p0 && tp_lbin(x, M, a.c2) == B0) atomicAdd(&sh.hist[(k >> 10) & 0x7ffu], tp_mass(x, M, a.c2));
    });
    __syncthreads();
    tp_find_crossing(sh, 2048, rest0 - above0, false);
    const uint32_t p1 = (p0 << 11) | sh.sel_bin;
    const unsigned long long above1 = above0 + sh.sel_above;
    __syncthreads();
    for (int i = threadIdx.x; i < 1024; i += kTpThreads) { sh.hist[i] = 0ull; sh.count[i] = 0u; }
    __syncthreads();
    tp_for_each(row, V, [&](int, float x) {
      int b2 = 0;
      x = tp_clean(x, b2);
      const uint32_t k = tp_key(x);
      if ((k >> 10) == p1 && tp_lbin(x, M, a.c2) == B0) {
        atomicAdd(&sh.hist[k & 0x3ffu], tp_mass(x, M, a.c2));
        atomicAdd(&sh.count[k & 0x3ffu], 1u);
      }
    });
    __syncthreads();
    tp_find_crossing(sh, 1024, rest0 - above1, true);
    tau = (p1 << 10) | sh.sel_bin;
    // tokens with exactly that logit share one mass: the first `need` of them in token order are kept
    const uint32_t ties = sh.sel_count;
    const unsigned long long each = sh.sel_mass / (ties ? ties : 1u);
    const unsigned long long rest = rest0 - above1 - sh.sel_above;
    uint32_t need = each ? (uint32_t)((rest + each - 1) / each) : ties;
    need = need < 1u ? 1u : (need > ties ? ties : need);
    __syncthreads();
    if (need < ties) {
      // the cut falls inside a run of equal logits: contiguous chunks per thread, a scan of the tie counts, and the
      // thread whose chunk holds the need-th tie finds its index
      const int len = (V + kTpThreads - 1) / kTpThreads;
      const int lo = min((int)threadIdx.x * len, V), hi = min(lo + len, V);
      unsigned long long cnt = 0;
      for (int i = lo; i < hi; ++i) {
        int b2 = 0;
        cnt += tp_key(tp_clean(row[i], b2)) == tau;
      }
      unsigned long long total;
      const unsigned long long before = tp_block_scan(cnt, sh, total);
      if (before < need && need <= before + cnt) {
        unsigned long long seen = before;
        for (int i = lo; i < hi; ++i) {
          int b2 = 0;
          if (tp_key(tp_clean(row[i], b2)) == tau && ++seen == need) { sh.tie_limit = i; break; }
        }
      }
      __syncthreads();
    }
  }
  const unsigned long long tau_comp = exact ? sh.tau_comp : (((unsigned long long)tau << 32) | (uint32_t)~(uint32_t)min(sh.tie_limit, V - 1));

  // ---- write: the logit itself inside the nucleus, -inf outside.  Inside: a more probable bin, or the cut's bin
  // and not behind the last kept token in the order (key descending, index ascending).
  int kept = 0;
  tp_for_each(row, V, [&](int i, float x) {
    int b2 = 0;
    const float c = tp_clean(x, b2);
    const int lb = tp_lbin(c, M, a.c2);
    const unsigned long long comp = ((unsigned long long)tp_key(c) << 32) | (uint32_t)~(uint32_t)i;
    const bool keep = lb > B0 || (lb == B0 && comp >= tau_comp);
    orow[i] = keep ? x : -INFINITY;
    kept += keep;
  });
  kept = __reduce_add_sync(0xffffffffu, kept);
  if (lane == 0) atomicAdd(&sh.kept, kept);
  __syncthreads();
  if (threadIdx.x == 0) {
    if (a.kept_out != nullptr) a.kept_out[blockIdx.x] = sh.kept;
    if (sh.bad) dev_flag(a.dev_status, SEQ_DEV_NONFINITE);
  }
}

// top_p >= 1: every token stays (rows copied when the call is not in place)
__global__ void top_p_copy_kernel(const TopPArgs a) {
  const float* row = a.logits + (int64_t)blockIdx.x * a.in_stride;
  float* orow = a.out + (int64_t)blockIdx.x * a.out_stride;
  if (row != orow)
    for (int i = threadIdx.x; i < a.V; i += blockDim.x) orow[i] = row[i];
  if (threadIdx.x == 0 && a.kept_out != nullptr) a.kept_out[blockIdx.x] = a.V;
}

}  // namespace seqtree

using namespace seqtree;

extern "C" int seq_tree_top_p_filter(const seq_tree_top_p_params* p, void* stream) {
  if (p == nullptr || p->logits == nullptr || p->out == nullptr) return SEQ_ERR_INVALID_ARG;
  if (p->n_rows < 1 || p->vocab < 1 || p->vocab > (1 << 22)) return SEQ_ERR_INVALID_ARG;
  if (!(p->temperature > 0.f) || isinf(p->temperature) || !(p->top_p > 0.f)) return SEQ_ERR_INVALID_ARG;
  if (p->logits_row_stride < p->vocab || p->out_row_stride < p->vocab || p->logits_row_stride % 4 != 0 ||
      p->out_row_stride % 4 != 0 || reinterpret_cast<uintptr_t>(p->logits) % 16 != 0 ||
      reinterpret_cast<uintptr_t>(p->out) % 16 != 0)
    return SEQ_ERR_INVALID_ARG;
  TopPArgs a;
  a.logits = p->logits; a.in_stride = p->logits_row_stride;
  a.out = p->out; a.out_stride = p->out_row_stride;
  a.V = p->vocab;
  a.c2 = kLog2e / p->temperature;
  a.top_p = (double)p->top_p;
  a.kept_out = p->kept_out; a.dev_status = p->dev_status;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (p->top_p >= 1.f)
    top_p_copy_kernel<<<p->n_rows, 256, 0, s>>>(a);
  else {
    // above the 48 KB a kernel gets without asking; set on every call (cheap, and correct on every device)
    SEQ_CUDA_OK(cudaFuncSetAttribute(top_p_filter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TpShared)));
    top_p_filter_kernel<<<p->n_rows, kTpThreads, sizeof(TpShared), s>>>(a);
  }
  SEQ_CUDA_OK(cudaGetLastError());
  return SEQ_OK;
}
