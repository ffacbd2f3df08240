// seq_tree_verify, node-parallel schedule: Algorithm 2 of the Sequoia paper for MANY tree nodes at once.
//
// What Algorithm 2 decides at a node (which child is accepted, or none, and then the token drawn from the residual)
// depends on that node's two logit rows, its children's tokens and their uniforms only (Section 2.2 states the
// verification as a recursion from the root; nothing flows from a node to its descendants but "you are visited").
// So the nodes are independent problems, and the walk is a pointer chase over their results:
//
//   * One thread-block cluster per node.  The node's target row (and draft row, if it has children) is read from
//     HBM once, straight into REGISTERS: 512 threads x 32 elements per row and CTA, the vocabulary cut into one
//     contiguous slice per CTA of the cluster and one contiguous kilo-element segment per warp.  Every
//     vocabulary-wide pass of Algorithm 2 (exponentials, the residual's normaliser after a rejection) then runs at
//     register speed; what is left per pass is one warp reduction, one table of per-warp partials pushed into every
//     CTA's shared memory, and one cluster barrier.  The per-warp partials of the last pass are the coarse level of
//     the final inverse CDF, which the one warp that holds the crossing finishes on its own.
//   * Which nodes.  The first wave is nodes 0 .. clusters-1 (node order is a topological order, and for the trees
//     of the paper close to level order).  A cluster that is done looks at the frontier - the deepest node known to
//     be on the accepted path - and claims, with one atomic, an unclaimed node among the frontier itself, its
//     children and its grandchildren: work whose result can still matter.  Nobody ever waits for anybody.
//   * The walk.  Per node one word W[v] takes three facts by atomic OR: claimed; decided (with the accepted child);
//     on the path.  Whoever brings the second of "decided" and "on the path" to a node moves the path on to the
//     accepted child, and on again while that child has been decided already; at a node without an accepted child
//     it writes path_len and the bonus token, which that node's cluster left beside its decision, and raises DONE.
//     Clusters still working on nodes that turned out not to matter see DONE at their next exchange and leave.
//
// Arithmetic: as in the walking kernel (tree_verify.cu).  R and D are never materialised: with p, q the two
// softmaxes, R[t] = max(p[t] - C q[t] - U, 0) / Z and D[t] = q[t] / ZD (or uniform over the non-rejected tokens
// once the draft has no mass left) for scalars C, U, Z, ZD, so a rejection is one scalar update and one sum.
// Each thread keeps its exponentials relative to its own maximum; sum(D) is the direct sum of the surviving q.
//
// The code is kept small on purpose: every phase runs once per node, so its instructions are fetched cold, and a
// first version with every helper inlined at several call sites spent more time fetching code than executing it.
#include <cooperative_groups.h>
#include <float.h>
#include <math.h>
#include <stdlib.h>

#include "common.cuh"
#include "tree_verify_nodes.cuh"

namespace cg = cooperative_groups;

namespace seqtree {
namespace vnp {

#ifdef SEQ_TRACE
// Debug builds only: per cluster a list of (tag, nanosecond clock) events recorded by its leader thread.
__device__ unsigned long long g_ntrace[160][48];
__device__ __forceinline__ unsigned long long ntimer() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define NTRACE(tag)                                                                                         \
  do {                                                                                                      \
    if (c.rank == 0 && c.tid == 0 && c.cid < 160 && c.ntrace_i < 47)                                        \
      g_ntrace[c.cid][++c.ntrace_i] = ((unsigned long long)(tag) << 56) | (ntimer() & 0xFFFFFFFFFFFFFFull); \
  } while (0)
#else
#define NTRACE(tag) do { } while (0)
#endif
#ifdef SEQ_DEBUG_STATE
// Debug builds only: every thread 0 leaves its latest state where a host can read it while the kernel runs.
#define DSTATE(code) do { if (c.tid == 0) reinterpret_cast<volatile unsigned long long*>(ws->W)[512 + c.cid * 2 + c.rank] = (unsigned long long)(code); } while (0)
#else
#define DSTATE(code) do { } while (0)
#endif

constexpr int kTh = 512;              // threads per CTA
constexpr int kWarps = kTh / 32;
constexpr int kChunks = 8;            // 16-byte chunks per thread and row
constexpr int kE = 4 * kChunks;       // elements per thread and row, in registers
constexpr int kWarpSpan = 32 * kE;    // consecutive elements of the slice that one warp holds
constexpr int kMaxCl = 8;             // CTAs per cluster, at most (the portable limit)
constexpr int kMaxParts = kMaxCl * kWarps;
constexpr int kCandMax = 96;          // nodes looked at per claim: the frontier, its children, its grandchildren
constexpr uint32_t kIdleLimit = 1u << 16;

// bits of W[v]
constexpr int kClaimed = 1, kDecided = 2, kOnPath = 4;
constexpr int kFlagShift = 3;         // bits 3..7: data problems seen at the node (raised only if it is on the path)
constexpr int kChildShift = 8;        // bits 8..19: accepted child + 1 (0: none)
constexpr int kDepthShift = 20;       // bits 20..29: the node's depth, set with kOnPath
constexpr int kTokenShift = 32;       // bits 32..63: the token drawn where no child was accepted, + 1

// Global scratch of one call (cleared by the launch).
struct Workspace {
  int32_t rows_read;   // diagnostic: logit rows this call read
  int32_t frontier;    // deepest node known to be on the path
  int32_t done;        // the path has ended
  int32_t pad;
  unsigned long long W[SEQ_MAX_TREE];  // per node: claimed / decided / on the path, and what was decided
};

struct NodeArgs {
  VerifyArgs v;
  Workspace* ws;
  int n_clusters;
};

struct Shared {
  int32_t parent[SEQ_MAX_TREE];
  int32_t tokens[SEQ_MAX_TREE];
  float uniforms[SEQ_MAX_TREE + 1];
  int32_t kids[SEQ_MAX_TREE];         // the current node's children in ascending order (the order they were drawn in)
  float2 kid_raw[SEQ_MAX_TREE];       // (target logit, draft logit) of the current node at each child's token, by rank
  uint8_t dup[SEQ_MAX_TREE];          // by rank: a child that carries the token of an earlier sibling
  int32_t chunk_cnt[32];              // children among nodes [32 j, 32 j + 32)
  float4 xbuf[2][kMaxParts];          // cluster exchange: one entry per (rank, warp), double-buffered
  int32_t ctl[2];                     // DONE as the cluster's leader saw it, pushed with every exchange
  int32_t drawn[2];                   // sampling from the target: the token drawn at this node, pushed to every CTA
  int32_t cand[kCandMax];
  int32_t next_node;                  // the leader's answer to "what now"
  int32_t first_ok;                   // the cluster's first node was still free when the cluster started
  int32_t verdict_code;               // what the publishing thread found out about the node just done
  int32_t node_flags;                 // data problems some thread of the cluster saw at the current node
};

struct Ctx {
  Shared* sh;
  int rank, cl, cid;     // CTA in cluster, cluster size, cluster in grid
  int lo, cnt;           // this CTA's vocabulary slice
  int tid, warp, lane;
  int xpar, dpar;
  int abort;             // DONE seen: stop working on this node
  const int32_t* done_ptr;  // where the cluster's leader thread reads DONE (null: never look)
  int peek[2];           // (leader thread) DONE as read a while ago: asked for at one exchange, handed round at the next
                         // but one, so that the leader never waits for the answer
#ifdef SEQ_TRACE
  int ntrace_i;
#endif
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
__device__ __forceinline__ int ld_acquire(const int32_t* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int ld_relaxed(const int32_t* p) {
  int v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// 1 / x for a positive double to nearly full precision without the division routine: single-precision reciprocal,
// two Newton steps in double.
__device__ __forceinline__ double fast_rcp(double x) {
  double r = (double)__frcp_rn((float)x);
  r = r * (2.0 - x * r);
  return r * (2.0 - x * r);
}
// A logit as the kernels read it: NaN counts as -inf, +inf as the largest finite value (both are flagged).
__device__ __forceinline__ float clean_logit(float x) { return x == x ? fminf(x, FLT_MAX) : -INFINITY; }

template <int CL>
__device__ __forceinline__ void cta_or_cluster_sync(cg::cluster_group& cluster) {
  if (CL == 1) __syncthreads(); else cluster.sync();
}
// One word into the same place of every CTA's shared memory.
template <int CL>
__device__ __forceinline__ void push_word(cg::cluster_group& cluster, int32_t* where, int32_t value) {
  if (CL == 1) *where = value;
  else {
#pragma unroll
    for (int r = 0; r < CL; ++r) *cluster.map_shared_rank(where, r) = value;
  }
}

// Element e (0..31) of this thread sits at this index of the CTA's slice: a warp holds 1024 consecutive elements,
// in eight chunks of 128; within a chunk a lane holds four consecutive ones.
__device__ __forceinline__ int local_index(const Ctx& c, int e) { return c.warp * kWarpSpan + (e >> 2) * 128 + c.lane * 4 + (e & 3); }

// One row slice into registers: 8 independent 16-byte loads per thread (streaming: each row is read once), the
// ragged end element by element; positions past the slice read as -inf (probability 0).
__device__ __forceinline__ void load_row(const Ctx& c, const float* row, float* x) {
  const float* base = row + c.lo + c.warp * kWarpSpan + c.lane * 4;
  const int room = c.cnt - (c.warp * kWarpSpan + c.lane * 4);  // elements of the slice from this lane's first one on
#pragma unroll
  for (int j = 0; j < kChunks; ++j) {
    float4 v;
    if (room - 128 * j >= 4) {
      v = __ldcs(reinterpret_cast<const float4*>(base + 128 * j));
    } else {
      v.x = room - 128 * j > 0 ? __ldcs(base + 128 * j) : -INFINITY;
      v.y = room - 128 * j > 1 ? __ldcs(base + 128 * j + 1) : -INFINITY;
      v.z = room - 128 * j > 2 ? __ldcs(base + 128 * j + 2) : -INFINITY;
      v.w = -INFINITY;
    }
    x[4 * j] = v.x; x[4 * j + 1] = v.y; x[4 * j + 2] = v.z; x[4 * j + 3] = v.w;
  }
}

// Maximum of the row's logits as the kernel reads them.  A sum of four is NaN or +inf exactly when one of them is NaN
// or +inf (or they mix -inf with +inf), so one comparison per four finds the rows that need cleaning; only then
// (rare) every element is cleaned in place.  `bad` collects whether anything had to be.
__device__ __forceinline__ float clean_and_max(float* x, bool& bad) {
  float a0 = -INFINITY, a1 = -INFINITY;
  bool dirty = false;
#pragma unroll
  for (int e = 0; e < kE; e += 4) {
    dirty |= !((x[e] + x[e + 1]) + (x[e + 2] + x[e + 3]) < INFINITY);
    a0 = fmaxf(a0, fmaxf(x[e], x[e + 1])); a1 = fmaxf(a1, fmaxf(x[e + 2], x[e + 3]));
  }
  if (dirty) {
    a0 = -INFINITY; a1 = -INFINITY;
#pragma unroll
    for (int e = 0; e < kE; ++e) {
      bad |= !(x[e] < INFINITY);
      x[e] = clean_logit(x[e]);
      a0 = fmaxf(a0, x[e]);
    }
  }
  return fmaxf(a0, a1);
}
// x <- 2^((x - m) c2) in place; returns the sum
__device__ __forceinline__ float exponentials(float* x, float m, float c2) {
  const float off = m == -INFINITY ? 0.f : -m * c2;  // an all -inf slice stays 0
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int e = 0; e < kE; e += 2) {
    x[e] = fast_ex2(fmaf(x[e], c2, off)); x[e + 1] = fast_ex2(fmaf(x[e + 1], c2, off));
    s0 += x[e]; s1 += x[e + 1];
  }
  return s0 + s1;
}

// Every warp of every CTA publishes one float4 to every CTA of the cluster; the leader thread's view of DONE rides
// along.  On return lane l of every warp holds entries l, l + 32, ... (rank-major, i.e. in vocabulary order).
template <int CL>
struct Exch { float4 e[CL >= 2 ? CL / 2 : 1]; };
template <int CL>
__device__ __forceinline__ void cluster_exchange(cg::cluster_group& cluster, Ctx& c, float4 mine, Exch<CL>& x, float4 filler) {
  constexpr int kPPL = CL >= 2 ? CL / 2 : 1;  // table entries per lane
  Shared* sh = c.sh;
  if (CL == 1) {
    if (c.lane == 0) sh->xbuf[c.xpar][c.warp] = mine;
    if (c.tid == 0) sh->ctl[c.xpar] = c.xpar ? c.peek[1] : c.peek[0];
    __syncthreads();
  } else {
    if (c.lane < CL) *cluster.map_shared_rank(&sh->xbuf[c.xpar][c.rank * kWarps + c.warp], c.lane) = mine;
    if (c.rank == 0 && c.warp == 0) {  // (one lane's view for every CTA: all of them must take the same decision)
      const int seen = __shfl_sync(0xffffffffu, c.xpar ? c.peek[1] : c.peek[0], 0);
      if (c.lane < CL) *cluster.map_shared_rank(&sh->ctl[c.xpar], c.lane) = seen;
    }
    cluster.sync();
  }
  constexpr int parts = CL * kWarps;
#pragma unroll
  for (int m = 0; m < kPPL; ++m)
    x.e[m] = (c.lane + 32 * m < parts) ? sh->xbuf[c.xpar][c.lane + 32 * m] : filler;  // (one CTA: 16 entries for 32 lanes)
  c.abort |= sh->ctl[c.xpar];
  if (c.done_ptr != nullptr && c.rank == 0 && c.warp == 0) {  // for the next exchange but one (same parity)
    if (c.xpar) c.peek[1] = ld_relaxed(c.done_ptr); else c.peek[0] = ld_relaxed(c.done_ptr);
  }
  c.xpar ^= 1;
}

// The path moves on from node v (on the path, decided: `child` accepted, or -1 and `token` drawn) for as long as the
// next node has been decided already.  One thread runs this at a time for any given node: the one that brought the
// second of "decided" and "on the path" to it.  Everything a node's cluster has to say travels in the node's word
// itself, so no fence is needed between a result and its announcement.  Returns the node at which the path ended,
// or -1 if it goes on later.
__device__ __noinline__ int advance(const VerifyArgs& a, Workspace* ws, int v, int child, int token, int depth, int flags) {
  for (;;) {
    a.path[depth] = v;
    if (a.next_child_out != nullptr) a.next_child_out[v] = child;
    if (flags) dev_flag(a.dev_status, flags);  // data problems count only at nodes the walk visits
    if (child < 0) {
      *a.path_len = depth + 1;
      *a.bonus = token;
      atomicExch(&ws->done, 1);
      return v;
    }
    const unsigned long long old = atomicOr(&ws->W[child], (unsigned long long)(kOnPath | ((depth + 1) << kDepthShift)));
    atomicExch(&ws->frontier, child);
    if (!(old & kDecided)) return -1;  // the child's cluster carries on when it gets there
    v = child;
    child = (int)((old >> kChildShift) & 0xFFF) - 1;
    token = (int)(old >> kTokenShift) - 1;
    flags = (int)(old >> kFlagShift) & 31;
    depth += 1;
  }
}

// A node's result goes on record (one thread of its cluster calls this); if the node is already known to be on the
// path, the path moves on.  Returns the verdict for the cluster: 0 nothing more, 1 the path ended at this very node,
// 2 + node: the path ended at that other node.
__device__ __noinline__ int publish(const VerifyArgs& a, Workspace* ws, int node, int accepted, int token, int flags) {
  const unsigned long long mine = (unsigned long long)(kClaimed | kDecided | ((accepted + 1) << kChildShift) | ((flags & 31) << kFlagShift)) |
                                  ((unsigned long long)(unsigned)(accepted < 0 ? token + 1 : 0) << kTokenShift);
  const unsigned long long old = atomicOr(&ws->W[node], mine);
  if ((node == 0 || (old & kOnPath)) && !(old & kDecided)) {
    const int end = advance(a, ws, node, accepted, token, node == 0 ? 0 : (int)(old >> kDepthShift) & 0x3FF, flags & 31);
    if (end == node) return 1;
    if (end >= 0) return 2 + end;
  }
  return 0;
}

// More work for this cluster (run by warp 0 of the leader CTA): an unclaimed node among the frontier, its children
// and its grandchildren, the frontier first, the rest spread over the clusters.  -1: the path has ended.
__device__ __noinline__ int claim(Ctx& c, const NodeArgs& na) {
  Shared* sh = c.sh;
  Workspace* ws = na.ws;
  const int first_dynamic = 0;  // (every node can be claimed: a cluster that starts late may find its first node taken)
  for (uint32_t it = 0; it < kIdleLimit; ++it) {
    // One lane looks, all lanes act on what it saw: lanes that read a changing word for themselves can disagree
    // (they need not run in step), and the warp-wide votes below would then wait for lanes that have left.
    int d = 0, f = 0;
    if (c.lane == 0) { d = ld_acquire(&ws->done); f = ld_relaxed(&ws->frontier); }
    d = __shfl_sync(0xffffffffu, d, 0);
    f = __shfl_sync(0xffffffffu, f, 0);
    if (d) return -1;
    // candidates in the order of their use to the walk: the frontier, its children, its grandchildren (a scan of the
    // parent array, 32 nodes at a time)
    int cnt = 0;
    if (f >= first_dynamic) { if (c.lane == 0) sh->cand[0] = f; cnt = 1; }
    for (int gen = 0; gen < 2; ++gen)
      for (int base = first_dynamic & ~31; base < na.v.n && cnt < kCandMax - 32; base += 32) {
        const int i = base + c.lane;
        int anc = (i < na.v.n && i >= first_dynamic) ? sh->parent[i] : -1;
        if (gen == 1 && anc >= 0) anc = sh->parent[anc];
        const uint32_t is = __ballot_sync(0xffffffffu, anc == f);
        if (anc == f) sh->cand[cnt + __popc(is & ((1u << c.lane) - 1u))] = i;
        cnt += __popc(is);
      }
    __syncwarp();
    uint32_t open_mask[kCandMax / 32];
    int total_open = 0;
#pragma unroll
    for (int m = 0; m < kCandMax / 32; ++m) {
      const int k = c.lane + 32 * m;
      const bool open = k < cnt && !(ld_relaxed(reinterpret_cast<const int32_t*>(&ws->W[sh->cand[k]])) & kClaimed);
      open_mask[m] = __ballot_sync(0xffffffffu, open);
      total_open += __popc(open_mask[m]);
    }
    if (total_open == 0) {  // nothing open near the frontier for now
      __nanosleep(200);
      continue;
    }
    // the frontier itself goes first; otherwise the (cluster mod open)-th open candidate
    int want = ((open_mask[0] & 1u) && sh->cand[0] == f) ? 0 : c.cid % total_open;
    int pick = -1;
#pragma unroll
    for (int m = 0; m < kCandMax / 32; ++m) {
      const int here = __popc(open_mask[m]);
      if (pick < 0 && want < here) {
        uint32_t mk = open_mask[m];
        for (int k = 0; k < want; ++k) mk &= mk - 1;
        pick = 32 * m + __ffs(mk) - 1;
      }
      if (pick < 0) want -= here;
    }
    int got = -1;
    if (c.lane == 0 && pick >= 0 && !(atomicOr(&ws->W[sh->cand[pick]], (unsigned long long)kClaimed) & kClaimed)) got = sh->cand[pick];
    got = __shfl_sync(0xffffffffu, got, 0);
    if (got >= 0) return got;  // else somebody was faster: look again
  }
  return -1;
}

template <int CL>
__global__ void __launch_bounds__(kTh, 1) tree_verify_nodes_kernel(const NodeArgs na) {
  constexpr int kPPL = CL >= 2 ? CL / 2 : 1;
  const VerifyArgs& a = na.v;
  Workspace* ws = na.ws;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) uint8_t dyn_smem[];
  Shared* sh = reinterpret_cast<Shared*>(dyn_smem);
  Ctx c;
  c.sh = sh;
  c.rank = (int)cluster.block_rank();
  c.cl = CL;
  c.cid = blockIdx.x / c.cl;
  c.lo = min(c.rank * a.slice_cap, a.V);
  c.cnt = min(a.V - c.lo, a.slice_cap);
  c.tid = threadIdx.x; c.warp = threadIdx.x >> 5; c.lane = threadIdx.x & 31;
  c.xpar = 0; c.dpar = 0; c.abort = 0; c.done_ptr = nullptr; c.peek[0] = 0; c.peek[1] = 0;
#ifdef SEQ_TRACE
  c.ntrace_i = 0;
#endif
  NTRACE(1);
  const bool greedy = a.temperature == 0.f;
  const bool specinfer = (a.flags & SEQ_VERIFY_SPECINFER) != 0;  // D is never touched: ZD stays 1, S stays empty
  const bool tsample = !greedy && (a.flags & SEQ_VERIFY_TARGET_SAMPLE) != 0;
  const float c2 = greedy ? 0.f : kLog2e / a.temperature;
  const bool leader = c.rank == 0 && c.tid == 0;
  const bool want_verdict = a.residual_out != nullptr;   // only the residual's writer needs to know where the path ended
  const bool more_nodes = a.n > na.n_clusters;           // else every node is some cluster's first

  NTRACE(2);

  float p[kE], q[kE];
  int node = c.cid;              // the first wave: cluster j takes node j (the grid has at most n clusters)
  bool revisit = false;          // second visit to the node at which the path ended, for residual_out only
  {
    unsigned long long first_claim = 0ull;
    if (leader) first_claim = atomicOr(&ws->W[node], (unsigned long long)kClaimed);
    // The tree first - a few words per thread, and everything waits for them - then the first node's target row.
    int tp[2], tt[2];
    float tu[3];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int i = c.tid + kTh * k;
      tp[k] = i < a.n ? a.parent[i] : -1;
      tt[k] = i < a.n ? a.tokens[i] : 0;
    }
#pragma unroll
    for (int k = 0; k < 3; ++k) tu[k] = (!greedy && c.tid + kTh * k <= a.n) ? a.uniforms[c.tid + kTh * k] : 0.f;
    load_row(c, a.target + (int64_t)node * a.target_stride, p);
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int i = c.tid + kTh * k;
      if (i < a.n) {
        int pp = tp[k];
        if (i == 0) pp = -1;
        else if (pp < -1 || pp >= i) { if (c.cid == 0 && c.rank == 0) dev_flag(a.dev_status, SEQ_DEV_BAD_PARENT); pp = -1; }
        sh->parent[i] = pp;
        sh->tokens[i] = tt[k];
      }
    }
#pragma unroll
    for (int k = 0; k < 3; ++k)
      if (c.tid + kTh * k <= a.n) sh->uniforms[c.tid + kTh * k] = tu[k];
    if (c.cid == 0 && c.rank == 0 && a.next_child_out != nullptr) {
      // nodes the walk does not visit read -2.  Written by the root's cluster before it puts the root's decision on
      // record, which every later write to this array follows.
      for (int i = c.tid; i < a.n; i += kTh) a.next_child_out[i] = -2;
      __threadfence();
    }
    if (c.tid == 0) { sh->node_flags = 0; sh->verdict_code = 0; sh->ctl[0] = 0; sh->ctl[1] = 0; }
    // The cluster's first node is claimed like any other (asked for at the very start, answered by now): a cluster that
    // the GPU could only place late may find that an idle one has taken it over, and then looks for other work.
    if (leader) push_word<CL>(cluster, &sh->first_ok, (first_claim & kClaimed) ? 0 : 1);
  }
  cta_or_cluster_sync<CL>(cluster);  // the tree is in place; every CTA of the cluster is resident before any remote write
  NTRACE(3);
  bool skip = sh->first_ok == 0;  // the first node went to another cluster: straight to the search for work
#pragma unroll 1
  for (;;) {
    if (!skip) {
    NTRACE(10);
    DSTATE(100 + node * 1000);
    // ---- (the node's target row is on its way) its children, in order, by rank among them
    const float* trow = a.target + (int64_t)node * a.target_stride;
    const float* drow = a.draft + (int64_t)node * a.draft_stride;
    c.abort = 0;
    c.done_ptr = revisit ? nullptr : &ws->done;
    c.peek[0] = 0; c.peek[1] = 0;
    const int ch0 = c.tid, ch1 = c.tid + kTh;
    const bool k0 = ch0 < a.n && sh->parent[ch0] == node, k1 = ch1 < a.n && sh->parent[ch1] == node;
    const uint32_t b0 = __ballot_sync(0xffffffffu, k0), b1 = __ballot_sync(0xffffffffu, k1);
    if (c.lane == 0) { sh->chunk_cnt[c.warp] = __popc(b0); sh->chunk_cnt[kWarps + c.warp] = __popc(b1); }
    __syncthreads();
    int n_kids, rank0, rank1;
    {
      const int cc = sh->chunk_cnt[c.lane];
      int inc = cc;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, inc, o);
        if (c.lane >= o) inc += up;
      }
      n_kids = __shfl_sync(0xffffffffu, inc, 31);
      rank0 = __shfl_sync(0xffffffffu, inc - cc, c.warp) + __popc(b0 & ((1u << c.lane) - 1u));
      rank1 = __shfl_sync(0xffffffffu, inc - cc, kWarps + c.warp) + __popc(b1 & ((1u << c.lane) - 1u));
    }
    const bool need_draft = !greedy && !tsample && n_kids > 0;
    if (need_draft) load_row(c, drow, q);
    // the two logits at each child's token, for the acceptance tests (every CTA fetches them for itself)
    if (k0) {
      sh->kids[rank0] = ch0;
      const int s = sh->tokens[ch0];
      if (need_draft && s >= 0 && s < a.V) sh->kid_raw[rank0] = make_float2(__ldg(trow + s), __ldg(drow + s));
    }
    if (k1) {
      sh->kids[rank1] = ch1;
      const int s = sh->tokens[ch1];
      if (need_draft && s >= 0 && s < a.V) sh->kid_raw[rank1] = make_float2(__ldg(trow + s), __ldg(drow + s));
    }
    __syncthreads();
    if (need_draft && !specinfer) {  // does an earlier sibling carry the same token?  (read after the next exchange)
      if (k0) { int d = 0; const int s = sh->tokens[ch0]; for (int r = 0; r < rank0; ++r) d |= sh->tokens[sh->kids[r]] == s; sh->dup[rank0] = (uint8_t)d; }
      if (k1) { int d = 0; const int s = sh->tokens[ch1]; for (int r = 0; r < rank1; ++r) d |= sh->tokens[sh->kids[r]] == s; sh->dup[rank1] = (uint8_t)d; }
    }

    int accepted = -1, node_flags = 0;
    int token = 0;          // greedy / sampling from the target: the token fixed at this node (every thread)
    int pub_token = -1;     // no child accepted: the drawn token, in the one thread that puts the node on record
    bool finished = true;
    double total_mass = 1.0;
    bool bad = false;
    Exch<CL> x;

    if (greedy) {
      // arg-max of the target row, lowest index on ties (a thread meets its elements in ascending order)
      float best = -INFINITY;
      int best_idx = 0x7fffffff;
#pragma unroll
      for (int e = 0; e < kE; ++e) {
        const int li = local_index(c, e);
        bad |= !(p[e] < INFINITY) && li < c.cnt;
        const float v = clean_logit(p[e]);
        if (li < c.cnt && (v > best || best_idx == 0x7fffffff)) { best = v; best_idx = c.lo + li; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, best_idx, o);
        if (oi != 0x7fffffff && (best_idx == 0x7fffffff || ob > best || (ob == best && oi < best_idx))) { best = ob; best_idx = oi; }
      }
      if (bad) push_word<CL>(cluster, &sh->node_flags, SEQ_DEV_NONFINITE);
      cluster_exchange(cluster, c, make_float4(best, __int_as_float(best_idx), 0.f, 0.f), x,
                       make_float4(-INFINITY, __int_as_float(0x7fffffff), 0.f, 0.f));
      finished = !c.abort;
      float gb = -INFINITY;
      int gi = 0x7fffffff;
#pragma unroll
      for (int m = 0; m < kPPL; ++m) {
        const float ob = x.e[m].x;
        const int oi = __float_as_int(x.e[m].y);
        if (oi != 0x7fffffff && (gi == 0x7fffffff || ob > gb || (ob == gb && oi < gi))) { gb = ob; gi = oi; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, gb, o);
        const int oi = __shfl_xor_sync(0xffffffffu, gi, o);
        if (oi != 0x7fffffff && (gi == 0x7fffffff || ob > gb || (ob == gb && oi < gi))) { gb = ob; gi = oi; }
      }
      token = gi == 0x7fffffff ? 0 : gi;
      for (int i = 0; i < n_kids && accepted < 0; ++i) {
        const int ch = sh->kids[i], s = sh->tokens[ch];
        if (s < 0 || s >= a.V) node_flags |= SEQ_DEV_BAD_TOKEN;
        else if (s == token) accepted = ch;
      }
      if (accepted < 0 && leader) pub_token = token;
    } else {
      // ---- exponentials relative to this thread's own maxima, with their sums
      NTRACE(11);
      const float mp = clean_and_max(p, bad);
      const float sp = exponentials(p, mp, c2);
      float mq = -INFINITY, sq = 0.f;
      if (need_draft) {
        mq = clean_and_max(q, bad);
        sq = exponentials(q, mq, c2);
      }
      if (bad) push_word<CL>(cluster, &sh->node_flags, SEQ_DEV_NONFINITE);
      NTRACE(12);
      // warp level: common maximum, sums brought to it; then the table of all warps of all CTAs
      const float Mwp = warp_max(mp), Mwq = warp_max(mq);
      const float swp = warp_sum(sp * rel_exp(mp, Mwp, c2)), swq = warp_sum(sq * rel_exp(mq, Mwq, c2));
      cluster_exchange(cluster, c, make_float4(Mwp, swp, Mwq, swq), x, make_float4(-INFINITY, 0.f, -INFINITY, 0.f));
      finished = !c.abort;
      NTRACE(13);
      DSTATE(200 + node * 1000);
      float Mp = -INFINITY, Mq = -INFINITY;
#pragma unroll
      for (int m = 0; m < kPPL; ++m) { Mp = fmaxf(Mp, x.e[m].x); Mq = fmaxf(Mq, x.e[m].z); }
      Mp = warp_max(Mp); Mq = warp_max(Mq);
      double part_sum[kPPL];   // residual mass of the (rank, warp) segments lane, lane + 32, ...: the draw's coarse level
      double asum = 0.0, bsum = 0.0;
#pragma unroll
      for (int m = 0; m < kPPL; ++m) {
        part_sum[m] = (double)x.e[m].y * (double)rel_exp(x.e[m].x, Mp, c2);
        asum += part_sum[m];
        bsum += (double)x.e[m].w * (double)rel_exp(x.e[m].z, Mq, c2);
      }
      const double Sp = sum_lanes(asum), Sq = sum_lanes(bsum);
      if (!(Sp > 0.0)) node_flags |= SEQ_DEV_DEGENERATE;
      const float invSp = Sp > 0.0 ? (float)fast_rcp(Sp) : 0.f;
      const float invSq = (need_draft && Sq > 0.0) ? (float)fast_rcp(Sq) : 0.f;
#pragma unroll
      for (int m = 0; m < kPPL; ++m) part_sum[m] *= (double)invSp;
      int mode = (need_draft && !(Sq > 0.0)) ? 1 : 0;  // a draft row without mass: the uniform fallback from the start
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
      NTRACE(14);
      double C = 0.0, U = 0.0, Z = 1.0, ZD = 1.0;
      int nS = 0;
      uint32_t dead = 0u;  // this thread's elements that were rejected (they are in S)
      // ---- Algorithm 2's loop over the children, in their order
#pragma unroll 1
      for (int i = 0; i < ((tsample || !finished) ? 0 : n_kids); ++i) {
        const int ch = sh->kids[i], s = sh->tokens[ch];
        if (s < 0 || s >= a.V) { node_flags |= SEQ_DEV_BAD_TOKEN; continue; }
        // an earlier (hence rejected) sibling carried the same token: it is in S.  (Without the draft update there
        // is no S: a repeated token is tested like any other, and its R is 0 by then.)
        const bool in_S = !specinfer && sh->dup[i] != 0;
        float pn = 0.f, qn = 0.f;
        if (!in_S) {
          const float2 raw = sh->kid_raw[i];
          pn = fast_ex2((clean_logit(raw.x) - Mp) * c2) * invSp;
          qn = fast_ex2((clean_logit(raw.y) - Mq) * c2) * invSq;
        }
        // the acceptance test u < R[s]/D[s], with R[s] = rs/Z and D[s] = qn/ZD (or 1/(V-|S|)); cross-multiplied,
        // which also covers D[s] = 0 (accept iff R[s] > 0)
        const double rs = in_S ? 0.0 : (double)resid(pn, qn, (float)C, (float)U);
        const double u = (double)sh->uniforms[ch];
        const bool accept = mode == 0 ? (u * Z * (double)qn < rs * ZD) : (u * Z < rs * (double)(a.V - nS));
        if (accept) { accepted = ch; break; }
        // the residual update R <- norm(max(R - D, 0)) with D as it stands
        double Cn = C, Un = U;
        if (mode == 0) Cn += Z * fast_rcp(ZD);
        else if (a.V - nS > 0) Un += Z * fast_rcp((double)(a.V - nS));
        // the draft update: s leaves D and joins S.  The thread that holds s marks it and re-sums its share of D
        // over its surviving tokens (a direct sum); R[s] needs no clearing: the rejection says R[s] < D[s], which
        // makes max(p[s] - C q[s] - U, 0) zero from the new C (or U) on.  The final draw applies the marks.
        if (!in_S && !specinfer) {
          const int idx = s - c.lo;
          if (idx >= 0 && idx < c.cnt && (idx >> 10) == c.warp && ((idx >> 2) & 31) == c.lane) {
            dead |= 1u << ((((idx >> 7) & 7) << 2) | (idx & 3));
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
        const float Cnf = (float)Cn, Unf = (float)Un;
        float z0 = 0.f, z1 = 0.f;
#pragma unroll
        for (int e = 0; e < kE; e += 2) { z0 += resid(p[e], q[e], Cnf, Unf); z1 += resid(p[e + 1], q[e + 1], Cnf, Unf); }
        const float zr = warp_sum(z0 + z1), zd = warp_sum(zd_mine);
        cluster_exchange(cluster, c, make_float4(zr, zd, 0.f, 0.f), x, make_float4(0.f, 0.f, 0.f, 0.f));
        if (c.abort) { finished = false; break; }
        NTRACE(15);
        DSTATE(300 + node * 1000);
        double zsum = 0.0, zdsum = 0.0;
#pragma unroll
        for (int m = 0; m < kPPL; ++m) { zsum += (double)x.e[m].x; zdsum += (double)x.e[m].y; }
        const double Zn = sum_lanes(zsum), ZDn = sum_lanes(zdsum);
        if (Zn > 0.0) {
          C = Cn; U = Un; Z = Zn;
#pragma unroll
          for (int m = 0; m < kPPL; ++m) part_sum[m] = (double)x.e[m].x;
        } else {
          node_flags |= SEQ_DEV_DEGENERATE;  // impossible in exact arithmetic: keep R
        }
        if (!specinfer) {
          ZD = ZDn;
          if (mode == 0 && !(ZDn > 0.0)) mode = 1;  // no mass left in D: uniform over the non-rejected set
        }
      }
      // ---- no child accepted (or a leaf, or sampling from the target): x ~ R by inverse CDF in index order
      if (finished && accepted < 0) {
        NTRACE(16);
        const bool use_q = need_draft && C != 0.0;
        const float Cf = (float)C, Uf = (float)U;
#pragma unroll
        for (int e = 0; e < kE; ++e) p[e] = resid(p[e], use_q ? q[e] : 0.f, Cf, Uf);  // the residual replaces p
        if (dead) {  // rejected tokens have left the residual for good
#pragma unroll
          for (int e = 0; e < kE; ++e) p[e] = ((dead >> e) & 1u) ? 0.f : p[e];
        }
        const float u = tsample ? sh->uniforms[node] : sh->uniforms[a.n];
        // coarse level, every warp for itself: inclusive scan over the (rank, warp) masses, 32 at a time
        double inc[kPPL], before = 0.0;
#pragma unroll
        for (int m = 0; m < kPPL; ++m) {
          double v = part_sum[m];
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, v, o);
            if (c.lane >= o) v += up;
          }
          inc[m] = v + before;
          before = __shfl_sync(0xffffffffu, inc[m], 31);
        }
        total_mass = before;
        const double tgt = (double)u * total_mass;
        int part = -1;
        bool take_last = false;
#pragma unroll
        for (int m = 0; m < kPPL; ++m) {
          const uint32_t hit = __ballot_sync(0xffffffffu, part_sum[m] > 0.0 && inc[m] > tgt);
          if (part < 0 && hit) part = 32 * m + __ffs(hit) - 1;
        }
        if (part < 0) {  // rounding left the total at or below the target: the last segment with mass
          take_last = true;
#pragma unroll
          for (int m = kPPL - 1; m >= 0; --m) {
            const uint32_t pos = __ballot_sync(0xffffffffu, part_sum[m] > 0.0);
            if (part < 0 && pos) part = 32 * m + 31 - __clz(pos);
          }
        }
        int found = -1;
        if (part < 0) {
          node_flags |= SEQ_DEV_DEGENERATE;  // no mass anywhere: token 0
          found = leader ? 0 : -1;
        } else if (part == c.rank * kWarps + c.warp) {
          // fine level, the one warp whose segment holds the crossing: its eight chunks in turn, then the lanes of
          // one chunk, then one lane's four elements
          double incl_part = 0.0, mass_part = 0.0;
#pragma unroll
          for (int m = 0; m < kPPL; ++m) {
            const double i_m = __shfl_sync(0xffffffffu, inc[m], part & 31), s_m = __shfl_sync(0xffffffffu, part_sum[m], part & 31);
            if ((part >> 5) == m) { incl_part = i_m; mass_part = s_m; }
          }
          const double tl = tgt - (incl_part - mass_part);  // the target inside this segment
          // The segment's 1024 residual values go to shared memory in vocabulary order (one padding word per 32, so
          // that the reads below do not collide); lane l then owns elements [32 l, 32 l + 32): the lanes' sums are
          // scanned, and the lane that holds the crossing walks its elements.  Rolled loops: this runs in one warp.
          float* seg = reinterpret_cast<float*>(sh->kid_raw);
#pragma unroll
          for (int e = 0; e < kE; ++e) {
            const int idx = (e >> 2) * 128 + c.lane * 4 + (e & 3);
            seg[idx + (idx >> 5)] = p[e];
          }
          __syncwarp();
          float ls = 0.f;
#pragma unroll 4
          for (int k = 0; k < 32; ++k) ls += seg[33 * c.lane + k];
          double incl = (double)ls;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, incl, o);
            if (c.lane >= o) incl += up;
          }
          const uint32_t cross = take_last ? 0u : __ballot_sync(0xffffffffu, ls > 0.f && incl > tl);
          const uint32_t mass = __ballot_sync(0xffffffffu, ls > 0.f);
          if (mass == 0u) {
            if (c.lane == 0) found = c.lo + c.warp * kWarpSpan;  // (a segment said to have mass has none: its first token)
          } else if (c.lane == (cross ? __ffs(cross) - 1 : 31 - __clz(mass))) {
            double r = incl - (double)ls;
            int pick = -1, last_k = 0;
#pragma unroll 1
            for (int k = 0; k < 32 && pick < 0; ++k) {
              const float v = seg[33 * c.lane + k];
              r += (double)v;
              if (v > 0.f) { last_k = k; if (cross && r > tl) pick = k; }
            }
            if (pick < 0) pick = last_k;  // nothing crosses (rounding, or by design): the last element with mass
            found = c.lo + c.warp * kWarpSpan + 32 * c.lane + pick;
          }
        }
        if (tsample) {
          // the token goes to every CTA; a child that carries it is taken
          const int dp = c.dpar;
          c.dpar ^= 1;
          if (found >= 0) push_word<CL>(cluster, &sh->drawn[dp], found);
          cta_or_cluster_sync<CL>(cluster);
          token = sh->drawn[dp];
          for (int i = 0; i < n_kids && accepted < 0; ++i) {
            const int ch = sh->kids[i], s = sh->tokens[ch];
            if (s < 0 || s >= a.V) node_flags |= SEQ_DEV_BAD_TOKEN;
            else if (s == token) accepted = ch;
          }
          found = (accepted < 0 && leader) ? token : -1;  // the leader puts the node on record
        }
        pub_token = found;
      }
    }
    NTRACE(finished ? 20 : 21);
    DSTATE((finished ? 400 : 450) + node * 1000);

    // ---- the node's result goes on record: by the leader if a child was accepted, by the finder of the token else
    int verdict = 0;
    if (finished && !revisit) {
      if (leader) atomicAdd(&ws->rows_read, need_draft ? 2 : 1);
      if (accepted >= 0 ? leader : pub_token >= 0) {
        verdict = publish(a, ws, node, accepted, pub_token, node_flags | sh->node_flags);
        if (want_verdict) push_word<CL>(cluster, &sh->verdict_code, verdict);
      }
    }
    NTRACE(22);
    DSTATE(500 + node * 1000);
    if (want_verdict) {
      if (!revisit) {
        cta_or_cluster_sync<CL>(cluster);
        verdict = sh->verdict_code;
        cta_or_cluster_sync<CL>(cluster);
        if (c.tid == 0) sh->verdict_code = 0;  // (the next one is pushed after further barriers)
      } else {
        verdict = 1;
      }
      if (verdict == 1 && finished) {
        // R as the bonus token was drawn from it (greedy: the one-hot at the arg-max)
        const float inv = total_mass > 0.0 ? (float)(1.0 / total_mass) : 0.f;
#pragma unroll
        for (int e = 0; e < kE; ++e) {
          const int li = local_index(c, e);
          if (li < c.cnt) a.residual_out[c.lo + li] = greedy ? ((c.lo + li == token) ? 1.f : 0.f) : p[e] * inv;
        }
      }
      if (revisit) break;
      if (verdict >= 2) {  // the path ended at a node that another cluster has left: see to its residual
        node = verdict - 2;
        revisit = true;
      }
    }
    }  // (!skip)
    skip = false;
    // ---- what next
    if (!revisit) {
      if (!more_nodes) break;
      DSTATE(600 + node * 1000);
      if (c.rank == 0 && c.warp == 0) {
        const int nxt = claim(c, na);
        if (c.lane == 0) push_word<CL>(cluster, &sh->next_node, nxt);
      }
      cta_or_cluster_sync<CL>(cluster);
      node = sh->next_node;
      if (c.tid == 0) sh->node_flags = 0;
      cta_or_cluster_sync<CL>(cluster);  // everyone has read it before the leader writes again
      NTRACE(23);
      DSTATE(700 + node * 1000);
      if (node < 0) break;
    }
    load_row(c, a.target + (int64_t)node * a.target_stride, p);  // the next node's target row starts its way
  }
  NTRACE(30);
  DSTATE(999);
  // no remote shared-memory access happens after the last cluster barrier a CTA has passed, so CTAs may leave alone
}

}  // namespace vnp

size_t verify_nodes_workspace_bytes(int n_tree) {
  (void)n_tree;
  return (sizeof(vnp::Workspace) + 255) & ~(size_t)255;
}

static int nodes_cluster_size(int n_tree, int vocab, int sms) {
  const int cap = vnp::kTh * vnp::kE;
  int cl = 1;
  while (cl < vnp::kMaxCl && (size_t)cl * cap < (size_t)vocab) cl *= 2;
  if ((size_t)cl * cap < (size_t)vocab) return 0;
  // a small tree leaves SMs idle: spread a node over more CTAs (shorter sweeps) while every node still has a cluster
  while (cl < vnp::kMaxCl && (long)n_tree * cl * 2 <= sms && vocab >= 2048 * cl * 2) cl *= 2;
  return cl;
}

bool verify_nodes_supported(int n_tree, int vocab, int flags) {
  if (flags & SEQ_VERIFY_ALL_NODES) return false;
  return nodes_cluster_size(n_tree, vocab, device_sm_count()) >= 1;
}

int launch_verify_nodes(const VerifyArgs& a_in, void* workspace, size_t workspace_bytes, int max_clusters, cudaStream_t stream) {
  if (workspace == nullptr || workspace_bytes < verify_nodes_workspace_bytes(a_in.n)) return SEQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) % 16 != 0) return SEQ_ERR_INVALID_ARG;
  const int sms = device_sm_count();
  int cl = nodes_cluster_size(a_in.n, a_in.V, sms);
  if (cl < 1) return SEQ_ERR_UNSUPPORTED;
#ifdef SEQ_TRACE
  if (const char* e = getenv("SEQ_NODES_CL")) { const int want = atoi(e); if (want >= cl && want <= 8) cl = want; }  // debug builds only
#endif
  vnp::NodeArgs na;
  na.v = a_in;
  // a CTA's slice: a multiple of 4 (16-byte loads stay aligned)
  na.v.slice_cap = (((a_in.V + cl - 1) / cl) + 3) & ~3;
  na.ws = static_cast<vnp::Workspace*>(workspace);
  void (*kernel)(const vnp::NodeArgs) = cl == 1 ? vnp::tree_verify_nodes_kernel<1> : cl == 2 ? vnp::tree_verify_nodes_kernel<2>
                                        : cl == 4 ? vnp::tree_verify_nodes_kernel<4> : vnp::tree_verify_nodes_kernel<8>;
  const int slot = cl == 1 ? 0 : cl == 2 ? 1 : cl == 4 ? 2 : 3;
  static int attr_done[4][64];
  const int rc = once_per_device(attr_done[slot], [&]() -> int {
    SEQ_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(vnp::Shared)));
    return SEQ_OK;
  });
  if (rc != SEQ_OK) return rc;
  // as many clusters as the device can hold at once (asked once per device and cluster size): nobody waits for
  // anybody, but a cluster that cannot start leaves its first node to the idle ones, which costs time
  static int resident[4][64];
  int dev = 0;
  SEQ_CUDA_OK(cudaGetDevice(&dev));
  int clusters = (dev >= 0 && dev < 64) ? __atomic_load_n(&resident[slot][dev], __ATOMIC_ACQUIRE) : 0;
  if (clusters == 0) {
    cudaLaunchConfig_t probe = {};
    probe.gridDim = dim3(sms / cl * cl);
    probe.blockDim = dim3(vnp::kTh);
    probe.dynamicSmemBytes = sizeof(vnp::Shared);
    cudaLaunchAttribute pa[1];
    pa[0].id = cudaLaunchAttributeClusterDimension;
    pa[0].val.clusterDim.x = cl; pa[0].val.clusterDim.y = 1; pa[0].val.clusterDim.z = 1;
    probe.attrs = pa;
    probe.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &probe) != cudaSuccess || clusters < 1) { cudaGetLastError(); clusters = sms / cl / 2; }
    if (clusters > sms / cl) clusters = sms / cl;
    if (clusters < 1) clusters = 1;
    if (dev >= 0 && dev < 64) __atomic_store_n(&resident[slot][dev], clusters, __ATOMIC_RELEASE);
  }
  if (clusters > a_in.n) clusters = a_in.n;
  if (max_clusters > 0 && clusters > max_clusters) clusters = max_clusters;
  if (clusters < 1) clusters = 1;
  na.n_clusters = clusters;
  // the few words that say what has been claimed, decided and found on the path start at zero
  SEQ_CUDA_OK(cudaMemsetAsync(workspace, 0, sizeof(vnp::Workspace), stream));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(clusters * cl);
  cfg.blockDim = dim3(vnp::kTh);
  cfg.dynamicSmemBytes = sizeof(vnp::Shared);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cl;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  // (No programmatic stream serialisation here: this kernel must not start before the clearing of its workspace
  // has finished, and with that attribute set it was seen to.)
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  SEQ_CUDA_OK(cudaLaunchKernelEx(&cfg, kernel, na));
  return SEQ_OK;
}

}  // namespace seqtree

#ifdef SEQ_TRACE
extern "C" int seq_debug_nodes_trace(unsigned long long* host_out) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(host_out, seqtree::vnp::g_ntrace, sizeof(unsigned long long) * 160 * 48);
  static unsigned long long zeros[160 * 48];
  cudaMemcpyToSymbol(seqtree::vnp::g_ntrace, zeros, sizeof(zeros));
  return 0;
}
#endif
