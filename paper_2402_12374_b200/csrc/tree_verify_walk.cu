// seq_tree_verify, the walk with rows in registers: Algorithm 2 of the Sequoia paper applied from the root down the
// tree (Section 2.2) by ONE cluster of 16 CTAs, the next node's rows already on their way while the current node's
// children are being tested.
//
// The vocabulary is cut into one contiguous slice per CTA and one contiguous segment per warp; a thread keeps its
// 4 * NCH elements of the target row and of the draft row in registers (8 elements per row at 32000 tokens, 32 at
// 128256), so every vocabulary-wide pass (exponentials, the residual's normaliser after a rejection) is a few
// instructions per thread, followed by one warp reduction, one table of per-warp partials pushed into every CTA's
// shared memory, and one cluster barrier.  What the walk will need next is known one step ahead: while child i of
// the current node is being tested, child i's own rows are loaded into a second set of registers (they are needed
// exactly if child i is accepted); on a rejection the loads for child i + 1 are issued before the residual pass, so
// they land behind that pass and its exchange.  A visited node therefore costs its arithmetic and one exchange, not
// a trip to HBM, unless the accepted child was decided within a microsecond.
//
// Arithmetic: R and D of Algorithm 2 are never materialised.  With p, q the two softmaxes and S the rejected set,
//     R[t] = max(p[t] - C q[t] - U, 0) / Z ,     D[t] = q[t] / ZD   (or 1/(V-|S|) once the uniform fallback has fired)
// for scalars C, U, Z, ZD: the residual update R <- norm(max(R - D, 0)) is C += Z/ZD (or U += Z/(V-|S|)) and one sum
// for the new Z; sum(D) is the direct sum of the surviving q.  A rejected token needs no clearing in R: the rejection
// says R[s] < D[s], which makes max(p[s] - C q[s] - U, 0) zero from the new C (or U) on; the final draw applies the
// marks all the same.  The per-warp partial sums of the last pass are the coarse level of the final inverse CDF,
// which the one warp that holds the crossing finishes on its own.
//
// Serves the default mode and the variant without the draft update at T > 0, and - with a kernel of its own at the
// end of this file - greedy decoding (T = 0, every mode); sampling from the target at T > 0, the every-node hook and
// batches run on the kernels of tree_verify.cu.
#include <cooperative_groups.h>
#include <float.h>
#include <limits.h>
#include <math.h>

#include "common.cuh"
#include "trace.cuh"
#include "tree_verify_nodes.cuh"

namespace cg = cooperative_groups;

namespace seqtree {
namespace vwk {

constexpr int kCl = 16;               // CTAs in the cluster (not a portable size: asked for, and checked, at launch)
constexpr int kTh = 256;              // threads per CTA
constexpr int kWarps = kTh / 32;
constexpr int kParts = kCl * kWarps;  // (rank, warp) segments, in vocabulary order
constexpr int kPPL = kParts / 32;     // table entries per lane

struct Shared {
  int32_t parent[SEQ_MAX_TREE];
  int32_t tokens[SEQ_MAX_TREE];
  float uniforms[SEQ_MAX_TREE + 1];
  uint32_t has_child[SEQ_MAX_TREE / 32];
  // The current node's children, listed by warp 0 while the other warps may still be reading the previous node's:
  // two copies, used in turn.
  int32_t kids[2][SEQ_MAX_TREE];      // in ascending order (the order they were drawn in)
  float2 kid_raw[2][SEQ_MAX_TREE];       // (target logit, draft logit) of the current node at each child's token, by rank;
                                      // after the last test: scratch of the final draw's fine level
  int32_t kid_tok[2][SEQ_MAX_TREE];   // by rank: the children's tokens
  uint8_t dup[2][SEQ_MAX_TREE];       // by rank: a child that carries the token of an earlier sibling
  int32_t chunk_cnt[32];              // children among nodes [32 j, 32 j + 32)
  float4 xbuf[2][kParts];             // cluster exchange: one entry per (rank, warp), double-buffered
  int32_t node_flags;
  int32_t pick[2][4];                 // greedy walk, by hop parity: the matching child, the first child with a bad token, the first child
};

__device__ __forceinline__ float fast_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rel_exp(float m, float M, float c2) { return m == -INFINITY ? 0.f : fast_ex2((m - M) * c2); }
__device__ __forceinline__ float resid(float pn, float qn, float Cf, float Uf) { return fmaxf(fmaf(-Cf, qn, pn) - Uf, 0.f); }
__device__ __forceinline__ double sum_lanes(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// 1 / x for a positive double to nearly full precision without the division routine
__device__ __forceinline__ double fast_rcp(double x) {
  double r = (double)__frcp_rn((float)x);
  r = r * (2.0 - x * r);
  return r * (2.0 - x * r);
}
// A logit as the kernels read it: NaN counts as -inf, +inf as the largest finite value (both are flagged).
__device__ __forceinline__ float clean_logit(float x) { return x == x ? fminf(x, FLT_MAX) : -INFINITY; }

struct Ctx {
  Shared* sh;
  int rank, lo, cnt;     // CTA in cluster, its vocabulary slice
  int tid, warp, lane;
  int xpar;
};

// One row slice into registers: NCH independent 16-byte loads per thread, the ragged end element by element;
// positions past the slice read as -inf (probability 0).  A warp holds 128 * NCH consecutive elements, in chunks of
// 128; within a chunk a lane holds four consecutive ones.
__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }  // exact
template <bool kBf16>
__device__ __forceinline__ float load_logit(const void* row, int64_t i) {
  if (kBf16) return bf16_bits_to_float(__ldg(static_cast<const unsigned short*>(row) + i));
  return __ldg(static_cast<const float*>(row) + i);
}
// One row slice into registers, as it lies in memory: NCH independent loads per thread (16 bytes each for fp32 logits,
// 8 for 16-bit ones), the ragged end element by element; positions past the slice read as -inf (probability 0).  A
// warp holds 128 * NCH consecutive elements, in chunks of 128; within a chunk a lane holds four consecutive ones.
// Nothing here touches the loaded values, so the loads stay in flight until widen() is called on them: that is what
// lets the next node's rows travel while the current node is worked on.
template <int NCH, bool kBf16>
struct RawRow { uint32_t w[kBf16 ? 2 * NCH : 4 * NCH]; };
template <int NCH, bool kBf16>
__device__ __forceinline__ void load_row(const Ctx& c, const void* row_v, RawRow<NCH, kBf16>& r) {
  const int first = c.warp * (128 * NCH) + c.lane * 4;
  const int room = c.cnt - first;
  if (kBf16) {
    const unsigned short* base = static_cast<const unsigned short*>(row_v) + c.lo + first;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      uint2 v;
      if (room - 128 * j >= 4) {
        v = __ldcs(reinterpret_cast<const uint2*>(base + 128 * j));
      } else {
        const uint32_t h0 = room - 128 * j > 0 ? __ldcs(base + 128 * j) : 0xFF80u, h1 = room - 128 * j > 1 ? __ldcs(base + 128 * j + 1) : 0xFF80u;
        const uint32_t h2 = room - 128 * j > 2 ? __ldcs(base + 128 * j + 2) : 0xFF80u;  // (0xFF80: -inf)
        v = make_uint2(h0 | (h1 << 16), h2 | (0xFF80u << 16));
      }
      r.w[2 * j] = v.x; r.w[2 * j + 1] = v.y;
    }
  } else {
    const float* base = static_cast<const float*>(row_v) + c.lo + first;
#pragma unroll
    for (int j = 0; j < NCH; ++j) {
      float4 v;
      if (room - 128 * j >= 4) {
        v = __ldcs(reinterpret_cast<const float4*>(base + 128 * j));
      } else {
        v.x = room - 128 * j > 0 ? __ldcs(base + 128 * j) : -INFINITY;
        v.y = room - 128 * j > 1 ? __ldcs(base + 128 * j + 1) : -INFINITY;
        v.z = room - 128 * j > 2 ? __ldcs(base + 128 * j + 2) : -INFINITY;
        v.w = -INFINITY;
      }
      r.w[4 * j] = __float_as_uint(v.x); r.w[4 * j + 1] = __float_as_uint(v.y);
      r.w[4 * j + 2] = __float_as_uint(v.z); r.w[4 * j + 3] = __float_as_uint(v.w);
    }
  }
}
// ... and widened to fp32 (exact)
template <int NCH, bool kBf16>
__device__ __forceinline__ void widen(const RawRow<NCH, kBf16>& r, float* x) {
#pragma unroll
  for (int j = 0; j < NCH; ++j) {
    if (kBf16) {
      x[4 * j] = __uint_as_float(r.w[2 * j] << 16); x[4 * j + 1] = __uint_as_float(r.w[2 * j] & 0xFFFF0000u);
      x[4 * j + 2] = __uint_as_float(r.w[2 * j + 1] << 16); x[4 * j + 3] = __uint_as_float(r.w[2 * j + 1] & 0xFFFF0000u);
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i) x[4 * j + i] = __uint_as_float(r.w[4 * j + i]);
    }
  }
}

// Maximum of the row's logits as the kernel reads them.  A sum of four is NaN or +inf exactly when one of them is NaN
// or +inf (or they mix -inf with +inf), so one comparison per four finds the rows that need cleaning; only then
// (rare) every element is cleaned in place.  `bad` collects whether anything had to be.
template <int NCH>
__device__ __forceinline__ float clean_and_max(float* x, bool& bad) {
  float a0 = -INFINITY, a1 = -INFINITY;
  bool dirty = false;
#pragma unroll
  for (int e = 0; e < 4 * NCH; e += 4) {
    dirty |= !((x[e] + x[e + 1]) + (x[e + 2] + x[e + 3]) < INFINITY);
    a0 = fmaxf(a0, fmaxf(x[e], x[e + 1])); a1 = fmaxf(a1, fmaxf(x[e + 2], x[e + 3]));
  }
  if (dirty) {
    a0 = -INFINITY; a1 = -INFINITY;
#pragma unroll
    for (int e = 0; e < 4 * NCH; ++e) {
      bad |= !(x[e] < INFINITY);
      x[e] = clean_logit(x[e]);
      a0 = fmaxf(a0, x[e]);
    }
  }
  return fmaxf(a0, a1);
}
// x <- 2^((x - m) c2) in place; returns the sum
template <int NCH>
__device__ __forceinline__ float exponentials(float* x, float m, float c2) {
  const float off = m == -INFINITY ? 0.f : -m * c2;  // an all -inf slice stays 0
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int e = 0; e < 4 * NCH; e += 2) {
    x[e] = fast_ex2(fmaf(x[e], c2, off)); x[e + 1] = fast_ex2(fmaf(x[e + 1], c2, off));
    s0 += x[e]; s1 += x[e + 1];
  }
  return s0 + s1;
}

// Every warp of every CTA publishes one float4 to every CTA of the cluster.  On return lane l of every warp holds
// entries l, l + 32, ... (rank-major, i.e. in vocabulary order).
struct Exch { float4 e[kPPL]; };
// ... in two halves, so that work that does not depend on the exchange can run while the barrier gathers
__device__ __forceinline__ void exchange_push(cg::cluster_group& cluster, Ctx& c, float4 mine) {
  if (c.lane < kCl) *cluster.map_shared_rank(&c.sh->xbuf[c.xpar][c.rank * kWarps + c.warp], c.lane) = mine;
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void exchange_pull(Ctx& c, Exch& x) {
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
#pragma unroll
  for (int m = 0; m < kPPL; ++m) x.e[m] = c.sh->xbuf[c.xpar][c.lane + 32 * m];
  c.xpar ^= 1;
}
__device__ __forceinline__ void cluster_exchange(cg::cluster_group& cluster, Ctx& c, float4 mine, Exch& x) {
  exchange_push(cluster, c, mine);
  exchange_pull(c, x);
}

// A batched launch runs one request per cluster: the same code on that request's arrays.
__device__ __forceinline__ VerifyArgs request_args(const VerifyArgs& in) {
  VerifyArgs a = in;
  const int64_t r = blockIdx.x / kCl;
  if (r > 0) {
    a.parent += r * in.tree_stride; a.tokens += r * in.tree_stride;
    a.target = reinterpret_cast<const float*>(reinterpret_cast<const char*>(in.target) + r * in.logits_stride * ((in.flags & SEQ_VERIFY_LOGITS_BF16) ? 2 : 4));
    a.draft = reinterpret_cast<const float*>(reinterpret_cast<const char*>(in.draft) + r * in.logits_stride * ((in.flags & SEQ_VERIFY_LOGITS_BF16) ? 2 : 4));
    a.uniforms += r * in.unif_stride;
    a.path += r * in.tree_stride; a.path_len += r; a.bonus += r;
    if (in.residual_out != nullptr) a.residual_out += r * in.resid_stride;
    if (in.next_child_out != nullptr) a.next_child_out += r * in.tree_stride;
  }
  return a;
}

template <int NCH, bool kBf16>
__global__ void __launch_bounds__(kTh, 1) tree_verify_walk_kernel(const VerifyArgs a_in) {
  const VerifyArgs a = request_args(a_in);
  constexpr int kEsz = kBf16 ? 2 : 4;  // bytes per logit
  const char* const tbase = reinterpret_cast<const char*>(a.target);
  const char* const dbase = reinterpret_cast<const char*>(a.draft);
  constexpr int kE = 4 * NCH;        // elements per thread and row
  constexpr int kSpan = 32 * kE;     // consecutive elements of the slice that one warp holds
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) uint8_t dyn_smem[];
  Shared* sh = reinterpret_cast<Shared*>(dyn_smem);
  Ctx c;
  c.sh = sh;
  c.rank = (int)cluster.block_rank();
  c.lo = min(c.rank * a.slice_cap, a.V);
  c.cnt = min(a.V - c.lo, a.slice_cap);
  c.tid = threadIdx.x; c.warp = threadIdx.x >> 5; c.lane = threadIdx.x & 31;
  c.xpar = 0;
  const bool specinfer = (a.flags & SEQ_VERIFY_SPECINFER) != 0;  // D is never touched: ZD stays 1, S stays empty
  const float c2 = kLog2e / a.temperature;
  const bool leader = c.rank == 0 && c.tid == 0;
  WTRACE_DECL;
  WTRACE(leader, 0);

  // programmatic dependent launch: the next kernel in the stream may be scheduled onto free SMs from now on; nothing
  // above touches global memory, everything below may read what the previous kernel wrote
  if (c.tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  WTRACE(leader, 1);

  float p[kE], q[kE];                // the current node's rows
  RawRow<NCH, kBf16> pn, qn;         // the rows of the child under test, on their way (as they lie in memory)
  {
    // The tree first - a few words per thread, and everything waits for them - then the root's rows.
    int tp[4], tt[4];
    float tu[5];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = c.tid + kTh * k;
      tp[k] = i < a.n ? a.parent[i] : -1;
      tt[k] = i < a.n ? a.tokens[i] : 0;
    }
#pragma unroll
    for (int k = 0; k < 5; ++k) tu[k] = c.tid + kTh * k <= a.n ? a.uniforms[c.tid + kTh * k] : 0.f;
    load_row<NCH, kBf16>(c, tbase, pn);
    if (a.n > 1) load_row<NCH, kBf16>(c, dbase, qn);  // (a root without children: never read)
    if (c.tid < SEQ_MAX_TREE / 32) sh->has_child[c.tid] = 0u;
    if (c.tid == 0) sh->node_flags = 0;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = c.tid + kTh * k;
      if (i < a.n) {
        int pp = tp[k];
        if (i == 0) pp = -1;
        else if (pp < -1 || pp >= i) { if (c.rank == 0) dev_flag(a.dev_status, SEQ_DEV_BAD_PARENT); pp = -1; }
        sh->parent[i] = pp;
        sh->tokens[i] = tt[k];
        if (pp >= 0) atomicOr(&sh->has_child[pp >> 5], 1u << (pp & 31));
      }
    }
#pragma unroll
    for (int k = 0; k < 5; ++k)
      if (c.tid + kTh * k <= a.n) sh->uniforms[c.tid + kTh * k] = tu[k];
    if (c.rank == 0 && a.next_child_out != nullptr)
      for (int i = c.tid; i < a.n; i += kTh) a.next_child_out[i] = -2;  // nodes the walk does not visit
  }
  cluster.sync();  // the tree is in place; every CTA of the cluster is resident before any remote write
  widen<NCH, kBf16>(pn, p);
  widen<NCH, kBf16>(qn, q);  // (a tree of one node: never loaded, never read)
  WTRACE(leader, 2);

  int cur = 0, plen = 0, bonus_found = -1;
  bool cur_has_kids = (sh->has_child[0] & 1u) != 0;
#pragma unroll 1
  for (int hop = 0; hop < a.n; ++hop) {  // a walk visits at most n nodes
    if (leader) a.path[plen] = cur;
    ++plen;
    WTRACE(leader, 10);
    const int np = hop & 1;
    const char* trow = tbase + (int64_t)cur * a.target_stride * kEsz;
    const char* drow = dbase + (int64_t)cur * a.draft_stride * kEsz;
    // ---- exponentials relative to this thread's own maxima, with their sums; the per-warp partials go to every CTA
    const bool need_draft = cur_has_kids;
    bool bad = false;
    const float mp = clean_and_max<NCH>(p, bad);
    const float sp = exponentials<NCH>(p, mp, c2);
    float mq = -INFINITY, sq = 0.f;
    if (need_draft) {
      mq = clean_and_max<NCH>(q, bad);
      sq = exponentials<NCH>(q, mq, c2);
    }
    if (bad) dev_flag(a.dev_status, SEQ_DEV_NONFINITE);
    WTRACE(leader, 13);
    Exch x;
    {
      const float Mwp = warp_max(mp), Mwq = warp_max(mq);
      const float swp = warp_sum(sp * rel_exp(mp, Mwp, c2)), swq = warp_sum(sq * rel_exp(mq, Mwq, c2));
      exchange_push(cluster, c, make_float4(Mwp, swp, Mwq, swq));
    }
    WTRACE(leader, 40);
    // ---- while the cluster's barrier gathers: the node's children, in order, by rank among them; the two logits at
    // each child's token (left in flight); the first child's own rows start their way (they are needed exactly if it
    // is accepted).  (The children arrays are used in turn: a warp may still be reading the previous node's.)
    int n_kids;
    int krank[4];
    float2 kraw[4];
    {
      bool k[4];
      uint32_t b[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int ch = c.tid + kTh * j;
        k[j] = ch < a.n && sh->parent[ch] == cur;
        b[j] = __ballot_sync(0xffffffffu, k[j]);
        if (c.lane == 0) sh->chunk_cnt[kWarps * j + c.warp] = __popc(b[j]);
      }
      __syncthreads();
      const int cc = sh->chunk_cnt[c.lane];
      int inc = cc;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, inc, o);
        if (c.lane >= o) inc += up;
      }
      n_kids = __shfl_sync(0xffffffffu, inc, 31);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        krank[j] = -1;
        const int r = __shfl_sync(0xffffffffu, inc - cc, kWarps * j + c.warp) + __popc(b[j] & ((1u << c.lane) - 1u));
        if (k[j]) {
          const int ch = c.tid + kTh * j, s = sh->tokens[ch];
          sh->kids[np][r] = ch;
          sh->kid_tok[np][r] = s;
          krank[j] = r;
          if (s >= 0 && s < a.V) kraw[j] = make_float2(load_logit<kBf16>(trow, s), load_logit<kBf16>(drow, s));
        }
      }
      __syncthreads();
    }
    int nxt = n_kids > 0 ? sh->kids[np][0] : -1;
    bool nxt_has_kids = false;
    if (nxt >= 0) {
      nxt_has_kids = (sh->has_child[nxt >> 5] >> (nxt & 31)) & 1u;
      load_row<NCH, kBf16>(c, tbase + (int64_t)nxt * a.target_stride * kEsz, pn);
      if (nxt_has_kids) load_row<NCH, kBf16>(c, dbase + (int64_t)nxt * a.draft_stride * kEsz, qn);
    }
    WTRACE(leader, 44);
    if (!specinfer) {  // does an earlier sibling carry the same token?
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (krank[j] >= 0) {
          int d = 0;
          const int s = sh->kid_tok[np][krank[j]];
          for (int r = 0; r < krank[j]; ++r) d |= sh->kid_tok[np][r] == s;
          sh->dup[np][krank[j]] = (uint8_t)d;
        }
    }
    WTRACE(leader, 12);
    exchange_pull(c, x);
    WTRACE(leader, 14);
    float Mp = -INFINITY, Mq = -INFINITY;
#pragma unroll
    for (int m = 0; m < kPPL; ++m) { Mp = fmaxf(Mp, x.e[m].x); Mq = fmaxf(Mq, x.e[m].z); }
    Mp = warp_max(Mp); Mq = warp_max(Mq);
    // (Single precision from here on: the sums have 128 terms of like size, the scalars C, U, Z, ZD a handful of
    // updates; their rounding stays two orders of magnitude inside the 1e-5 band of the parity rule.)
    float part_sum[kPPL];   // residual mass of the (rank, warp) segments lane, lane + 32, ...: the draw's coarse level
    float asum = 0.f, bsum = 0.f;
#pragma unroll
    for (int m = 0; m < kPPL; ++m) {
      part_sum[m] = x.e[m].y * rel_exp(x.e[m].x, Mp, c2);
      asum += part_sum[m];
      bsum += x.e[m].w * rel_exp(x.e[m].z, Mq, c2);
    }
    const float Sp = warp_sum(asum), Sq = warp_sum(bsum);
    if (!(Sp > 0.f)) dev_flag(a.dev_status, SEQ_DEV_DEGENERATE);
    const float invSp = Sp > 0.f ? __frcp_rn(Sp) : 0.f;
    const float invSq = (need_draft && Sq > 0.f) ? __frcp_rn(Sq) : 0.f;
#pragma unroll
    for (int m = 0; m < kPPL; ++m) part_sum[m] *= invSp;
    int mode = (need_draft && !(Sq > 0.f)) ? 1 : 0;  // a draft row without mass: the uniform fallback from the start
    // probabilities in place; this thread's share of sum(D) over the surviving tokens, a direct sum
    const float fp = rel_exp(mp, Mp, c2) * invSp, fq = rel_exp(mq, Mq, c2) * invSq;
    float zd_mine = 0.f;
    {
      float s0 = 0.f, s1 = 0.f;
#pragma unroll
      for (int e = 0; e < kE; e += 2) {
        p[e] *= fp; p[e + 1] *= fp;
        if (need_draft) { q[e] *= fq; q[e + 1] *= fq; s0 += q[e]; s1 += q[e + 1]; }
      }
      zd_mine = s0 + s1;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (krank[j] >= 0) sh->kid_raw[np][krank[j]] = kraw[j];
    __syncthreads();  // the children's logits and repeat marks are in place
    WTRACE(leader, 15);
    float C = 0.f, U = 0.f, Z = 1.f, ZD = 1.f;
    int nS = 0, accepted = -1;
    uint32_t dead = 0u;  // this thread's elements that were rejected (they are in S)
    // ---- Algorithm 2's loop over the children, in their order
#pragma unroll 1
    for (int i = 0; i < n_kids; ++i) {
      const int ch = sh->kids[np][i], s = sh->kid_tok[np][i];
      const bool valid = s >= 0 && s < a.V;
      if (!valid) dev_flag(a.dev_status, SEQ_DEV_BAD_TOKEN);
      // an earlier (hence rejected) sibling carried the same token: it is in S.  (Without the draft update there is
      // no S: a repeated token is tested like any other, and its R is 0 by then.)
      const bool in_S = !specinfer && sh->dup[np][i] != 0;
      bool accept = false;
      if (valid) {
        float ps = 0.f, qs = 0.f;
        if (!in_S) {
          const float2 raw = sh->kid_raw[np][i];
          ps = fast_ex2((clean_logit(raw.x) - Mp) * c2) * invSp;
          qs = fast_ex2((clean_logit(raw.y) - Mq) * c2) * invSq;
        }
        // the acceptance test u < R[s]/D[s], with R[s] = rs/Z and D[s] = qs/ZD (or 1/(V-|S|)); cross-multiplied,
        // which also covers D[s] = 0 (accept iff R[s] > 0)
        const float rs = in_S ? 0.f : resid(ps, qs, C, U);
        const float u = sh->uniforms[ch];
        accept = mode == 0 ? (u * Z * qs < rs * ZD) : (u * Z < rs * (float)(a.V - nS));
      }
      WTRACE(leader, 16);
      if (accept) { accepted = ch; break; }
      // ---- rejected: the next child's rows must start their way, and the residual is updated.  The loads are issued
      // behind the exchange's barrier arrival (its release fence would otherwise wait for them to land).
      const bool more = i + 1 < n_kids;
      if (more) {
        nxt = sh->kids[np][i + 1];
        nxt_has_kids = (sh->has_child[nxt >> 5] >> (nxt & 31)) & 1u;
      }
      if (!valid) {  // (not a token: R and D untouched)
        if (more) {
          load_row<NCH, kBf16>(c, tbase + (int64_t)nxt * a.target_stride * kEsz, pn);
          if (nxt_has_kids) load_row<NCH, kBf16>(c, dbase + (int64_t)nxt * a.draft_stride * kEsz, qn);
        }
        continue;
      }
      // R <- norm(max(R - D, 0)) with D as it stands
      float Cn = C, Un = U;
      if (mode == 0) Cn += Z * __frcp_rn(ZD);
      else if (a.V - nS > 0) Un += Z * __frcp_rn((float)(a.V - nS));
      // the draft update: s leaves D and joins S.  The thread that holds s marks it and re-sums its share of D
      if (!in_S && !specinfer) {
        const int idx = s - c.lo - c.warp * kSpan;
        if (s - c.lo >= 0 && s - c.lo < c.cnt && idx >= 0 && idx < kSpan && ((idx >> 2) & 31) == c.lane) {
          dead |= 1u << (((idx >> 7) << 2) | (idx & 3));
          float s0 = 0.f, s1 = 0.f;
#pragma unroll
          for (int k = 0; k < kE; k += 2) {
            s0 += ((dead >> k) & 1u) ? 0.f : q[k];
            s1 += ((dead >> (k + 1)) & 1u) ? 0.f : q[k + 1];
          }
          zd_mine = s0 + s1;
        }
        nS += 1;
      }
      const float Cnf = Cn, Unf = Un;
      float z0 = 0.f, z1 = 0.f;
#pragma unroll
      for (int e = 0; e < kE; e += 2) { z0 += resid(p[e], q[e], Cnf, Unf); z1 += resid(p[e + 1], q[e + 1], Cnf, Unf); }
      const float zr = warp_sum(z0 + z1), zd = warp_sum(zd_mine);
      WTRACE(leader, 17);
      exchange_push(cluster, c, make_float4(zr, zd, 0.f, 0.f));
      if (more) {
        load_row<NCH, kBf16>(c, tbase + (int64_t)nxt * a.target_stride * kEsz, pn);
        if (nxt_has_kids) load_row<NCH, kBf16>(c, dbase + (int64_t)nxt * a.draft_stride * kEsz, qn);
      }
      exchange_pull(c, x);
      WTRACE(leader, 18);
      float zsum = 0.f, zdsum = 0.f;
#pragma unroll
      for (int m = 0; m < kPPL; ++m) { zsum += x.e[m].x; zdsum += x.e[m].y; }
      const float Zn = warp_sum(zsum), ZDn = warp_sum(zdsum);
      if (Zn > 0.f) {
        C = Cn; U = Un; Z = Zn;
#pragma unroll
        for (int m = 0; m < kPPL; ++m) part_sum[m] = x.e[m].x;
      } else {
        dev_flag(a.dev_status, SEQ_DEV_DEGENERATE);  // impossible in exact arithmetic: keep R
      }
      if (!specinfer) {
        ZD = ZDn;
        if (mode == 0 && !(ZDn > 0.f)) mode = 1;  // no mass left in D: uniform over the non-rejected set
      }
    }
    if (leader && a.next_child_out != nullptr) a.next_child_out[cur] = accepted;
    if (accepted >= 0) {
      // ---- on to the accepted child: its rows are in the second set of registers (or about to land there)
      widen<NCH, kBf16>(pn, p);
      widen<NCH, kBf16>(qn, q);
      cur = accepted;
      cur_has_kids = nxt_has_kids;
      continue;
    }
    WTRACE(leader, 20);
    // ---- no child accepted (or a leaf): x ~ R by inverse CDF in index order with the last uniform
    {
      const bool use_q = need_draft && C != 0.f;
      const float Cf = C, Uf = U;
#pragma unroll
      for (int e = 0; e < kE; ++e) p[e] = resid(p[e], use_q ? q[e] : 0.f, Cf, Uf);  // the residual replaces p
      if (dead) {  // rejected tokens have left the residual for good
#pragma unroll
        for (int e = 0; e < kE; ++e) p[e] = ((dead >> e) & 1u) ? 0.f : p[e];
      }
      const float u = sh->uniforms[a.n];
      // coarse level, every warp for itself: inclusive scan over the (rank, warp) masses, 32 at a time
      double inc[kPPL], before = 0.0;
#pragma unroll
      for (int m = 0; m < kPPL; ++m) {
        double v = (double)part_sum[m];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const double up = __shfl_up_sync(0xffffffffu, v, o);
          if (c.lane >= o) v += up;
        }
        inc[m] = v + before;
        before = __shfl_sync(0xffffffffu, inc[m], 31);
      }
      const double total_mass = before, tgt = (double)u * total_mass;
      int part = -1;
      bool take_last = false;
#pragma unroll
      for (int m = 0; m < kPPL; ++m) {
        const uint32_t hit = __ballot_sync(0xffffffffu, part_sum[m] > 0.f && inc[m] > tgt);
        if (part < 0 && hit) part = 32 * m + __ffs(hit) - 1;
      }
      if (part < 0) {  // rounding left the total at or below the target: the last segment with mass
        take_last = true;
#pragma unroll
        for (int m = kPPL - 1; m >= 0; --m) {
          const uint32_t pos = __ballot_sync(0xffffffffu, part_sum[m] > 0.f);
          if (part < 0 && pos) part = 32 * m + 31 - __clz(pos);
        }
      }
      if (a.residual_out != nullptr) {
        const float inv = total_mass > 0.0 ? (float)fast_rcp(total_mass) : 0.f;
#pragma unroll
        for (int e = 0; e < kE; ++e) {
          const int li = c.warp * kSpan + (e >> 2) * 128 + c.lane * 4 + (e & 3);
          if (li < c.cnt) a.residual_out[c.lo + li] = p[e] * inv;
        }
      }
      if (part < 0) {
        if (leader) { dev_flag(a.dev_status, SEQ_DEV_DEGENERATE); bonus_found = 0; }  // no mass anywhere: token 0
      } else if (part == c.rank * kWarps + c.warp) {
        // fine level, the one warp whose segment holds the crossing
        double incl_part = 0.0, mass_part = 0.0;
#pragma unroll
        for (int m = 0; m < kPPL; ++m) {
          const double i_m = __shfl_sync(0xffffffffu, inc[m], part & 31), s_m = (double)__shfl_sync(0xffffffffu, part_sum[m], part & 31);
          if ((part >> 5) == m) { incl_part = i_m; mass_part = s_m; }
        }
        const double tl = tgt - (incl_part - mass_part);  // the target inside this segment
        // The segment's residual values go to shared memory in vocabulary order (one padding word per 32, so that
        // the reads below do not collide); lane l then owns elements [NCH*4*l, +NCH*4): the lanes' sums are scanned,
        // and the lane that holds the crossing walks its elements.  Rolled loops: this runs in one warp.
        float* seg = reinterpret_cast<float*>(sh->kid_raw[np ^ 1]);
#pragma unroll
        for (int e = 0; e < kE; ++e) {
          const int idx = (e >> 2) * 128 + c.lane * 4 + (e & 3);
          seg[idx + (idx >> 5)] = p[e];
        }
        __syncwarp();
        const int mine0 = kE * c.lane;  // this lane's first element of the segment
        float ls = 0.f;
#pragma unroll 4
        for (int k = 0; k < kE; ++k) { const int idx = mine0 + k; ls += seg[idx + (idx >> 5)]; }
        double incl = (double)ls;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const double up = __shfl_up_sync(0xffffffffu, incl, o);
          if (c.lane >= o) incl += up;
        }
        const uint32_t cross = take_last ? 0u : __ballot_sync(0xffffffffu, ls > 0.f && incl > tl);
        const uint32_t mass = __ballot_sync(0xffffffffu, ls > 0.f);
        if (mass == 0u) {
          if (c.lane == 0) bonus_found = c.lo + c.warp * kSpan;  // (a segment said to have mass has none: its first token)
        } else if (c.lane == (cross ? __ffs(cross) - 1 : 31 - __clz(mass))) {
          double r = incl - (double)ls;
          int pick = -1, last_k = 0;
#pragma unroll 1
          for (int k = 0; k < kE && pick < 0; ++k) {
            const int idx = mine0 + k;
            const float v = seg[idx + (idx >> 5)];
            r += (double)v;
            if (v > 0.f) { last_k = k; if (cross && r > tl) pick = k; }
          }
          if (pick < 0) pick = last_k;  // nothing crosses (rounding, or by design): the last element with mass
          bonus_found = c.lo + c.warp * kSpan + mine0 + pick;
        }
      }
    }
    break;
  }
  WTRACE(leader, 30);
  if (leader) *a.path_len = plen;
  if (bonus_found >= 0) *a.bonus = bonus_found;
  // No closing cluster barrier: remote shared memory is only written before a cluster barrier that every CTA joins,
  // so nothing can still address a CTA that has left.
}


// ---------------------------------------------------------------- greedy decoding (T = 0) -----------------------
// R is the one-hot at the target arg-max (lowest index on ties), a child is accepted iff its token is that arg-max;
// draft logits and uniforms play no part.  Per visited node: the target row in registers, one arg-max over the
// cluster (one exchange), one look at the children.  While the exchange gathers, the row of the node's first child -
// the draft's most probable token, the likeliest match - is requested; any other match is fetched when it is known.
__device__ __forceinline__ int ordered_key(float x) {  // an integer that orders like the (non-NaN) float
  int b = __float_as_int(x);
  return b ^ ((b >> 31) & 0x7fffffff);
}
// (key, index) of the larger key, then the lower index; index 0x7fffffff = nothing
__device__ __forceinline__ void warp_argmax(int& key, int& idx) {
  const int k = idx == 0x7fffffff ? INT_MIN : key;
  const int m = __reduce_max_sync(0xffffffffu, k);
  idx = __reduce_min_sync(0xffffffffu, (k == m) ? idx : 0x7fffffff);
  key = m;
}

template <int NCH, bool kBf16>
__global__ void __launch_bounds__(kTh, 1) tree_verify_greedy_kernel(const VerifyArgs a_in) {
  const VerifyArgs a = request_args(a_in);
  constexpr int kEsz = kBf16 ? 2 : 4;
  constexpr int kE = 4 * NCH, kSpan = 32 * kE;
  const char* const tbase = reinterpret_cast<const char*>(a.target);
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) uint8_t dyn_smem[];
  Shared* sh = reinterpret_cast<Shared*>(dyn_smem);
  Ctx c;
  c.sh = sh;
  c.rank = (int)cluster.block_rank();
  c.lo = min(c.rank * a.slice_cap, a.V);
  c.cnt = min(a.V - c.lo, a.slice_cap);
  c.tid = threadIdx.x; c.warp = threadIdx.x >> 5; c.lane = threadIdx.x & 31;
  c.xpar = 0;
  const bool leader = c.rank == 0 && c.tid == 0;
  if (c.tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  RawRow<NCH, kBf16> pn;
  {
    int tp[4], tt[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = c.tid + kTh * k;
      tp[k] = i < a.n ? a.parent[i] : -1;
      tt[k] = i < a.n ? a.tokens[i] : 0;
    }
    load_row<NCH, kBf16>(c, tbase, pn);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = c.tid + kTh * k;
      if (i < a.n) {
        int pp = tp[k];
        if (i == 0) pp = -1;
        else if (pp < -1 || pp >= i) { if (c.rank == 0) dev_flag(a.dev_status, SEQ_DEV_BAD_PARENT); pp = -1; }
        sh->parent[i] = pp;
        sh->tokens[i] = tt[k];
      }
    }
    if (c.rank == 0 && a.next_child_out != nullptr)
      for (int i = c.tid; i < a.n; i += kTh) a.next_child_out[i] = -2;  // nodes the walk does not visit
  }
  cluster.sync();  // the tree is in place; every CTA of the cluster is resident before any remote write

  int cur = 0, plen = 0, g = 0;
  bool bad = false;
#pragma unroll 1
  for (int hop = 0; hop < a.n; ++hop) {  // a walk visits at most n nodes
    if (leader) a.path[plen] = cur;
    ++plen;
    int32_t* pick = sh->pick[hop & 1];
    if (c.tid < 3) pick[c.tid] = 0x7fffffff;  // (the other set is the one the previous hop may still be reading)
    float x[kE];
    widen<NCH, kBf16>(pn, x);
    // this thread's arg-max: its elements in ascending index order, the first of equal values stays
    int key = INT_MIN, idx = 0x7fffffff;
#pragma unroll
    for (int e = 0; e < kE; ++e) {
      const int local = c.warp * kSpan + (e >> 2) * 128 + c.lane * 4 + (e & 3);
      if (local < c.cnt) {
        bad |= !(x[e] < INFINITY);
        const int k = ordered_key(clean_logit(x[e]));
        if (idx == 0x7fffffff || k > key) { key = k; idx = c.lo + local; }
      }
    }
    warp_argmax(key, idx);
    exchange_push(cluster, c, make_float4(__int_as_float(key), __int_as_float(idx), 0.f, 0.f));
    // ---- while the barrier gathers: the node's first child, and its row on the way
    __syncthreads();  // pick[] is reset
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = c.tid + kTh * k;
      if (i < a.n && sh->parent[i] == cur) atomicMin(&pick[2], i);
    }
    __syncthreads();
    const int first_kid = pick[2];
    if (first_kid != 0x7fffffff) load_row<NCH, kBf16>(c, tbase + (int64_t)first_kid * a.target_stride * kEsz, pn);
    Exch t;
    exchange_pull(c, t);
    key = INT_MIN; idx = 0x7fffffff;
#pragma unroll
    for (int m = 0; m < kPPL; ++m) {  // entries in vocabulary order: the first of equal keys stays
      const int k = __float_as_int(t.e[m].x), i = __float_as_int(t.e[m].y);
      if (i != 0x7fffffff && (idx == 0x7fffffff || k > key)) { key = k; idx = i; }
    }
    warp_argmax(key, idx);
    g = idx == 0x7fffffff ? 0 : idx;
    // ---- the child that carries the arg-max (the first, should several); a child with a token outside the vocabulary
    // is reported if the loop over the children would have met it before the match
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int i = c.tid + kTh * k;
      if (i < a.n && sh->parent[i] == cur) {
        const int s = sh->tokens[i];
        if (s < 0 || s >= a.V) atomicMin(&pick[1], i);
        else if (s == g) atomicMin(&pick[0], i);
      }
    }
    __syncthreads();
    const int match = pick[0];
    if (leader) {
      if (pick[1] < match) dev_flag(a.dev_status, SEQ_DEV_BAD_TOKEN);
      if (a.next_child_out != nullptr) a.next_child_out[cur] = match == 0x7fffffff ? -1 : match;
    }
    if (match == 0x7fffffff) break;
    if (match != first_kid) load_row<NCH, kBf16>(c, tbase + (int64_t)match * a.target_stride * kEsz, pn);
    cur = match;
  }
  if (bad) dev_flag(a.dev_status, SEQ_DEV_NONFINITE);
  if (a.residual_out != nullptr) {
#pragma unroll
    for (int e = 0; e < kE; ++e) {
      const int local = c.warp * kSpan + (e >> 2) * 128 + c.lane * 4 + (e & 3);
      if (local < c.cnt) a.residual_out[c.lo + local] = (c.lo + local == g) ? 1.f : 0.f;
    }
  }
  if (leader) { *a.path_len = plen; *a.bonus = g; }
}

}  // namespace vwk

// Elements a cluster of this kernel holds per row: 16 CTAs x 256 threads x 4 NCH.
bool verify_walk_supported(int vocab, int flags, float temperature) {
  if (flags & SEQ_VERIFY_ALL_NODES) return false;
  if (temperature == 0.f) return vocab >= 1 && (size_t)vocab <= (size_t)vwk::kCl * vwk::kTh * 4 * 8;  // greedy: its own kernel, whatever the mode flags say
  if (flags & SEQ_VERIFY_TARGET_SAMPLE) return false;
  if (!(temperature > 0.f)) return false;
  return vocab >= 1 && (size_t)vocab <= (size_t)vwk::kCl * vwk::kTh * 4 * 8;
}

int launch_verify_walk(const VerifyArgs& a_in, bool check_only, cudaStream_t stream, int requests) {
  VerifyArgs a = a_in;
  a.slice_cap = (((a.V + vwk::kCl - 1) / vwk::kCl) + 3) & ~3;
  const int nch = a.slice_cap <= vwk::kTh * 4 * 2 ? 2 : a.slice_cap <= vwk::kTh * 4 * 4 ? 4 : 8;
  const bool bf16 = (a.flags & SEQ_VERIFY_LOGITS_BF16) != 0;
  const bool greedy = a.temperature == 0.f;
  void (*kernel)(const VerifyArgs) =
      greedy ? (bf16 ? (nch == 2 ? vwk::tree_verify_greedy_kernel<2, true> : nch == 4 ? vwk::tree_verify_greedy_kernel<4, true> : vwk::tree_verify_greedy_kernel<8, true>)
                     : (nch == 2 ? vwk::tree_verify_greedy_kernel<2, false> : nch == 4 ? vwk::tree_verify_greedy_kernel<4, false> : vwk::tree_verify_greedy_kernel<8, false>))
      : bf16 ? (nch == 2 ? vwk::tree_verify_walk_kernel<2, true> : nch == 4 ? vwk::tree_verify_walk_kernel<4, true> : vwk::tree_verify_walk_kernel<8, true>)
             : (nch == 2 ? vwk::tree_verify_walk_kernel<2, false> : nch == 4 ? vwk::tree_verify_walk_kernel<4, false> : vwk::tree_verify_walk_kernel<8, false>);
  const int slot = (nch == 2 ? 0 : nch == 4 ? 1 : 2) + (bf16 ? 3 : 0) + (greedy ? 6 : 0);
  static int attr_done[12][64];
  const int rc = once_per_device(attr_done[slot], [&]() -> int {
    SEQ_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(vwk::Shared)));
    SEQ_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
    return SEQ_OK;
  });
  if (rc != SEQ_OK) return rc;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(vwk::kCl * (requests > 0 ? requests : 1));
  cfg.blockDim = dim3(vwk::kTh);
  cfg.dynamicSmemBytes = sizeof(vwk::Shared);
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = vwk::kCl;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // start under the previous kernel's tail
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

}  // namespace seqtree

#ifdef SEQ_TRACE
// debug builds only: copy out and reset the timeline recorded by WTRACE()
extern "C" int seq_debug_walk_trace(unsigned long long* host_out) {
  int n = 0;
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(&n, seqtree::g_wtrace_n, sizeof(int));
  if (n > 255) n = 255;
  cudaMemcpyFromSymbol(host_out, seqtree::g_wtrace, sizeof(unsigned long long) * 2 * n);
  int zero = 0;
  cudaMemcpyToSymbol(seqtree::g_wtrace_n, &zero, sizeof(int));
  return n;
}
#endif
