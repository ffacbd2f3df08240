// seq_tree_verify: Algorithm 2 of the Sequoia paper walked from the root, on one thread-block
// cluster, plus the final draw x ~ R.
//
// Schedule.  One cluster of 8 CTAs follows the walk.  At each visited node the two logit rows
// are cut into 8 contiguous vocabulary slices, one per CTA, read from HBM once and kept in shared
// memory as unnormalised exponentials; everything that is vocabulary-wide (max, sums, the
// residual's normaliser, the inverse CDF) is a block reduction followed by one exchange over
// distributed shared memory.  The walk's scalar state is replicated: every CTA derives it from
// the same exchanged numbers with the same instructions, so all CTAs take the same branches.
//
// Arithmetic.  R and D of Algorithm 2 are never materialised.  With p, q the two softmaxes and S
// the rejected set (their entries zeroed in shared memory when rejected), the state after any
// number of rejections is
//     R[t] = max(p[t] - C q[t] - U, 0) / Z ,     D[t] = q[t] / ZD   (or 1/(V-|S|) once the
//                                                                   uniform fallback has fired)
// for scalars C, U, Z, ZD: line 9's  R <- norm(max(R - D, 0))  becomes  C += Z/ZD  (or
// U += Z/(V-|S|) after the fallback) followed by one vocabulary-wide sum for the new Z, and
// line 12's sum(D) is the direct sum ZD of the surviving q, never a subtraction.
#include <cooperative_groups.h>
#include <float.h>
#include <math.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace seqtree {

constexpr int kVThreads = 512;
constexpr int kVWarps = kVThreads / 32;
constexpr int kVCluster = 8;
constexpr int kVStaticSmem = 24 * 1024;  // upper bound of the kernel's static shared memory

struct VerifyArgs {
  int32_t n, V, slice_cap, flags;
  const int32_t* parent; const int32_t* tokens;
  const float* target; int64_t target_stride;
  const float* draft; int64_t draft_stride;
  float temperature;
  const float* uniforms;
  int32_t* path; int32_t* path_len; int32_t* bonus;
  float* residual_out; int32_t* next_child_out; int32_t* dev_status;
};

struct VShared {
  int32_t parent[SEQ_MAX_TREE];
  int32_t tokens[SEQ_MAX_TREE];
  float uniforms[SEQ_MAX_TREE + 1];
  int32_t kids[SEQ_MAX_TREE];
  double xbuf[2][kVCluster][4];   // cluster exchange slots, double-buffered
  double wbuf[2][kVWarps][4];     // block reduction slots, double-buffered
  int32_t wcnt[kVWarps];
  int32_t misc[4];
};

// Per-thread copy of the replicated walk state at the current node.
struct NodeState {
  float ip, iq;       // this CTA's factors turning stored exponentials into probabilities
  float mlp[kVCluster], ipr[kVCluster], mlq[kVCluster], iqr[kVCluster];
  double C, U, Z, ZD;
  int mode;           // 0: D proportional to q; 1: uniform over the non-rejected set
  int nS;             // |S|
  int greedy_token;
};

struct Ctx {
  VShared* sh;
  float* ps; float* qs;
  int rank, lo, cnt;
  int wpar, xpar;
  int tid, warp, lane;
};

__device__ __forceinline__ float sanitize_logit(float x, int32_t* dev_status) {
  if (x != x) { dev_flag(dev_status, SEQ_DEV_NONFINITE); return -INFINITY; }
  if (x == INFINITY) { dev_flag(dev_status, SEQ_DEV_NONFINITE); return FLT_MAX; }
  return x;
}
// exponential of one logit relative to its slice maximum (c2 = log2(e)/T)
__device__ __forceinline__ float slice_exp(float x, float mloc, float c2) {
  return mloc == -INFINITY ? 0.f : exp2f((x - mloc) * c2);
}
// unnormalised residual max(p - C q - U, 0) of one token
__device__ __forceinline__ float resid(float pn, float qn, float Cf, float Uf) {
  return fmaxf(fmaf(-Cf, qn, pn) - Uf, 0.f);
}

template <int K, bool kMax>
__device__ __forceinline__ void block_allreduce(Ctx& c, double (&v)[K]) {
#pragma unroll
  for (int k = 0; k < K; ++k) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double other = __shfl_xor_sync(0xffffffffu, v[k], o);
      v[k] = kMax ? fmax(v[k], other) : v[k] + other;
    }
  }
  double (*w)[4] = c.sh->wbuf[c.wpar];
  if (c.lane == 0) {
#pragma unroll
    for (int k = 0; k < K; ++k) w[c.warp][k] = v[k];
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < K; ++k) {
    double acc = w[0][k];
#pragma unroll
    for (int ww = 1; ww < kVWarps; ++ww) acc = kMax ? fmax(acc, w[ww][k]) : acc + w[ww][k];
    v[k] = acc;
  }
  c.wpar ^= 1;
}

// Every CTA publishes K doubles to every CTA of the cluster; on return out[r][k] holds rank r's.
template <int K>
__device__ __forceinline__ void cluster_exchange(cg::cluster_group& cluster, Ctx& c, const double (&v)[K],
                                                 double (&out)[kVCluster][K]) {
  if (c.tid < kVCluster) {
    double* remote = cluster.map_shared_rank(&c.sh->xbuf[c.xpar][c.rank][0], c.tid);
#pragma unroll
    for (int k = 0; k < K; ++k) remote[k] = v[k];
  }
  cluster.sync();
#pragma unroll
  for (int r = 0; r < kVCluster; ++r)
#pragma unroll
    for (int k = 0; k < K; ++k) out[r][k] = c.sh->xbuf[c.xpar][r][k];
  c.xpar ^= 1;
}

// Children of v in ascending node order -> sh->kids; returns their count.
__device__ int build_kids(Ctx& c, int v, int n) {
  // each thread owns two consecutive candidates so that warps and lanes are in node order
  const int c0 = v + 1 + 2 * c.tid;
  const bool f0 = c0 < n && c.sh->parent[c0] == v;
  const bool f1 = c0 + 1 < n && c.sh->parent[c0 + 1] == v;
  const int mine = (int)f0 + (int)f1;
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (c.lane >= o) incl += t;
  }
  if (c.lane == 31) c.sh->wcnt[c.warp] = incl;
  __syncthreads();
  int base = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kVWarps; ++w) {
    const int x = c.sh->wcnt[w];
    if (w < c.warp) base += x;
    total += x;
  }
  int pos = base + incl - mine;
  if (f0) c.sh->kids[pos++] = c0;
  if (f1) c.sh->kids[pos] = c0 + 1;
  __syncthreads();
  return total;
}

// Read this CTA's slice of one logit row into shared memory (sanitised); returns the slice max.
__device__ float load_slice(const Ctx& c, const float* __restrict__ row, float* dst, int32_t* dev_status) {
  float m = -INFINITY;
  const float* src = row + c.lo;
  const int n4 = c.cnt >> 2;
  for (int i = c.tid; i < n4; i += kVThreads) {
    float4 x = __ldg(reinterpret_cast<const float4*>(src) + i);
    x.x = sanitize_logit(x.x, dev_status); x.y = sanitize_logit(x.y, dev_status);
    x.z = sanitize_logit(x.z, dev_status); x.w = sanitize_logit(x.w, dev_status);
    reinterpret_cast<float4*>(dst)[i] = x;
    m = fmaxf(fmaxf(m, fmaxf(x.x, x.y)), fmaxf(x.z, x.w));
  }
  for (int i = (n4 << 2) + c.tid; i < c.cnt; i += kVThreads) {
    const float x = sanitize_logit(__ldg(src + i), dev_status);
    dst[i] = x;
    m = fmaxf(m, x);
  }
  return m;
}

// Runs Algorithm 2's loop at node v.  Returns the accepted child's node id or -1 and leaves in
// `st` (and in ps/qs) the state the final draw needs.
__device__ int process_node(cg::cluster_group& cluster, Ctx& c, const VerifyArgs& a, int v, NodeState& st,
                            bool skip_leaves) {
  const int k = build_kids(c, v, a.n);
  if (k == 0 && skip_leaves) return -1;
  const bool greedy = a.temperature == 0.f;
  const float* trow = a.target + (int64_t)v * a.target_stride;
  const float* drow = a.draft + (int64_t)v * a.draft_stride;

  if (greedy) {
    // arg-max of the target row, lowest index on ties
    float best = -INFINITY;
    int best_idx = 0x7fffffff;
    for (int i = c.tid; i < c.cnt; i += kVThreads) {
      const float x = sanitize_logit(__ldg(trow + c.lo + i), a.dev_status);
      if (x > best || (x == best && c.lo + i < best_idx)) { best = x; best_idx = c.lo + i; }
    }
    double mv[1] = {(double)best};
    block_allreduce<1, true>(c, mv);
    double iv[1] = {(best == (float)mv[0] && best_idx != 0x7fffffff) ? -(double)best_idx : -2147483647.0};
    block_allreduce<1, true>(c, iv);  // max of negated indices = lowest index
    double mine[2] = {mv[0], iv[0]};
    double all[kVCluster][2];
    cluster_exchange<2>(cluster, c, mine, all);
    double gbest = -INFINITY, gidx = -2147483647.0;
#pragma unroll
    for (int r = 0; r < kVCluster; ++r) {
      if (all[r][1] == -2147483647.0) continue;  // empty slice or nothing comparable
      if (all[r][0] > gbest || (all[r][0] == gbest && all[r][1] > gidx)) { gbest = all[r][0]; gidx = all[r][1]; }
    }
    st.greedy_token = gidx == -2147483647.0 ? 0 : (int)(-gidx);
    for (int i = 0; i < k; ++i) {
      const int ch = c.sh->kids[i];
      const int s = c.sh->tokens[ch];
      if (s < 0 || s >= a.V) { dev_flag(a.dev_status, SEQ_DEV_BAD_TOKEN); continue; }
      if (s == st.greedy_token) return ch;
    }
    return -1;
  }

  const float c2 = kLog2e / a.temperature;
  const bool need_draft = k > 0;

  // slices -> shared memory as exponentials relative to the slice maxima, with their sums
  double mx[2];
  mx[0] = (double)load_slice(c, trow, c.ps, a.dev_status);
  mx[1] = need_draft ? (double)load_slice(c, drow, c.qs, a.dev_status) : -INFINITY;
  block_allreduce<2, true>(c, mx);  // its barrier also publishes the raw logits to the block
  const float mlp = (float)mx[0], mlq = (float)mx[1];
  float sp = 0.f, sq = 0.f;
  for (int i = c.tid; i < c.cnt; i += kVThreads) {
    const float e = slice_exp(c.ps[i], mlp, c2);
    c.ps[i] = e;
    sp += e;
    if (need_draft) {
      const float f = slice_exp(c.qs[i], mlq, c2);
      c.qs[i] = f;
      sq += f;
    }
  }
  double sums[2] = {(double)sp, (double)sq};
  block_allreduce<2, false>(c, sums);
  double mine[4] = {mx[0], sums[0], mx[1], sums[1]};
  double all[kVCluster][4];
  cluster_exchange<4>(cluster, c, mine, all);
  {
    double Mp = -INFINITY, Mq = -INFINITY;
#pragma unroll
    for (int r = 0; r < kVCluster; ++r) { Mp = fmax(Mp, all[r][0]); Mq = fmax(Mq, all[r][2]); }
    double fp[kVCluster], fq[kVCluster], Sp = 0.0, Sq = 0.0;
#pragma unroll
    for (int r = 0; r < kVCluster; ++r) {
      fp[r] = all[r][0] == -INFINITY ? 0.0 : (double)exp2f(((float)all[r][0] - (float)Mp) * c2);
      fq[r] = all[r][2] == -INFINITY ? 0.0 : (double)exp2f(((float)all[r][2] - (float)Mq) * c2);
      Sp += all[r][1] * fp[r];
      Sq += all[r][3] * fq[r];
    }
    if (!(Sp > 0.0)) dev_flag(a.dev_status, SEQ_DEV_DEGENERATE);
#pragma unroll
    for (int r = 0; r < kVCluster; ++r) {
      st.mlp[r] = (float)all[r][0];
      st.mlq[r] = (float)all[r][2];
      st.ipr[r] = Sp > 0.0 ? (float)(fp[r] / Sp) : 0.f;
      st.iqr[r] = (need_draft && Sq > 0.0) ? (float)(fq[r] / Sq) : 0.f;
    }
    st.ip = st.ipr[c.rank];
    st.iq = st.iqr[c.rank];
  }
  st.C = 0.0; st.U = 0.0; st.Z = 1.0; st.ZD = 1.0; st.mode = 0; st.nS = 0;
  if (need_draft && st.iqr[0] == 0.f) {
    // the draft row has no mass at all (every logit -inf): Algorithm 2's fallback from the start
    bool any = false;
#pragma unroll
    for (int r = 0; r < kVCluster; ++r) any |= st.iqr[r] != 0.f;
    if (!any) st.mode = 1;
  }

  for (int i = 0; i < k; ++i) {
    const int ch = c.sh->kids[i];
    const int s = c.sh->tokens[ch];
    if (s < 0 || s >= a.V) { dev_flag(a.dev_status, SEQ_DEV_BAD_TOKEN); continue; }
    // s is in S iff an earlier (hence rejected) sibling carried the same token
    int dup = 0;
    for (int j = c.tid; j < i; j += kVThreads) dup |= c.sh->tokens[c.sh->kids[j]] == s;
    const bool in_S = __syncthreads_or(dup) != 0;
    const int owner = s / a.slice_cap;
    float pn = 0.f, qn = 0.f;
    if (!in_S) {
      const float xp = sanitize_logit(__ldg(trow + s), nullptr);
      const float xq = sanitize_logit(__ldg(drow + s), nullptr);
      pn = slice_exp(xp, st.mlp[owner], c2) * st.ipr[owner];
      qn = slice_exp(xq, st.mlq[owner], c2) * st.iqr[owner];
    }
    const float Cf = (float)st.C, Uf = (float)st.U;
    const double Rs = in_S ? 0.0 : (double)resid(pn, qn, Cf, Uf) / st.Z;
    const double Ds = in_S ? 0.0 : (st.mode == 0 ? (double)qn / st.ZD : 1.0 / (double)(a.V - st.nS));
    const double ratio = Ds > 0.0 ? Rs / Ds : (Rs > 0.0 ? (double)INFINITY : 0.0);
    if ((double)c.sh->uniforms[ch] < ratio) return ch;  // line 6-7: accept

    // line 9: R <- norm(max(R - D, 0)) with D as it stands
    double Cn = st.C, Un = st.U;
    if (st.mode == 0) Cn += st.Z / st.ZD;
    else if (a.V - st.nS > 0) Un += st.Z / (double)(a.V - st.nS);
    // lines 10-11: D[s] <- 0, S.add(s)
    if (!in_S) {
      if (owner == c.rank && c.tid == 0) { c.ps[s - c.lo] = 0.f; c.qs[s - c.lo] = 0.f; }
      st.nS += 1;
    }
    __syncthreads();
    const float Cnf = (float)Cn, Unf = (float)Un;
    float zr = 0.f, zd = 0.f;
    for (int t = c.tid; t < c.cnt; t += kVThreads) {
      const float qt = c.qs[t] * st.iq;
      zr += resid(c.ps[t] * st.ip, qt, Cnf, Unf);
      zd += qt;
    }
    double z2[2] = {(double)zr, (double)zd};
    block_allreduce<2, false>(c, z2);
    double zall[kVCluster][2];
    cluster_exchange<2>(cluster, c, z2, zall);
    double Zn = 0.0, ZDn = 0.0;
#pragma unroll
    for (int r = 0; r < kVCluster; ++r) { Zn += zall[r][0]; ZDn += zall[r][1]; }
    if (Zn > 0.0) { st.C = Cn; st.U = Un; st.Z = Zn; }
    else dev_flag(a.dev_status, SEQ_DEV_DEGENERATE);  // keep R
    st.ZD = ZDn;
    if (st.mode == 0 && !(ZDn > 0.0)) st.mode = 1;  // lines 12-15: uniform over the non-rejected set
  }
  return -1;
}

// Line 18, x ~ R by inverse CDF in index order with uniforms[n]; optionally writes R.
__device__ void draw_bonus(cg::cluster_group& cluster, Ctx& c, const VerifyArgs& a, const NodeState& st) {
  const bool greedy = a.temperature == 0.f;
  if (greedy) {
    if (a.residual_out != nullptr)
      for (int t = c.tid; t < c.cnt; t += kVThreads) a.residual_out[c.lo + t] = (c.lo + t == st.greedy_token) ? 1.f : 0.f;
    if (c.rank == 0 && c.tid == 0) *a.bonus = st.greedy_token;
    return;
  }
  const float Cf = (float)st.C, Uf = (float)st.U;
  const bool has_q = st.C != 0.0;  // qs holds this node's draft only if a rejection happened
  // contiguous segment of the slice per warp, a multiple of 32 long
  const int seg = (((c.cnt + kVWarps - 1) / kVWarps) + 31) & ~31;
  const int s_lo = min(c.warp * seg, c.cnt), s_hi = min(s_lo + seg, c.cnt);
  float part = 0.f;
  for (int t = s_lo + c.lane; t < s_hi; t += 32)
    part += resid(c.ps[t] * st.ip, has_q ? c.qs[t] * st.iq : 0.f, Cf, Uf);
  double wsum = warp_sum((double)part);
  double (*w)[4] = c.sh->wbuf[c.wpar];
  if (c.lane == 0) w[c.warp][0] = wsum;
  __syncthreads();
  double cta_sum[1] = {0.0};
#pragma unroll
  for (int ww = 0; ww < kVWarps; ++ww) cta_sum[0] += w[ww][0];
  double ranks[kVCluster][1];
  cluster_exchange<1>(cluster, c, cta_sum, ranks);
  double total = 0.0;
#pragma unroll
  for (int r = 0; r < kVCluster; ++r) total += ranks[r][0];
  const double inv_total = total > 0.0 ? 1.0 / total : 0.0;

  if (a.residual_out != nullptr) {
    const float it = (float)inv_total;
    for (int t = c.tid; t < c.cnt; t += kVThreads)
      a.residual_out[c.lo + t] = resid(c.ps[t] * st.ip, has_q ? c.qs[t] * st.iq : 0.f, Cf, Uf) * it;
  }

  const double tgt = (double)c.sh->uniforms[a.n] * total;
  // rank holding the crossing: first rank whose inclusive sum exceeds tgt, else the last with mass
  int rstar = -1, rlast = -1;
  double excl = 0.0, run = 0.0;
#pragma unroll
  for (int r = 0; r < kVCluster; ++r) {
    if (ranks[r][0] > 0.0) rlast = r;
    if (rstar < 0 && run + ranks[r][0] > tgt) { rstar = r; excl = run; }
    run += ranks[r][0];
  }
  bool take_last = false;
  if (rstar < 0) { rstar = rlast; take_last = true; }
  if (rstar < 0) {  // no mass anywhere: degenerate input, defined output
    if (c.rank == 0 && c.tid == 0) { *a.bonus = 0; dev_flag(a.dev_status, SEQ_DEV_DEGENERATE); }
    return;
  }
  if (c.rank != rstar) return;
  // warp holding the crossing
  double tl = tgt - excl;
  int wstar = -1, wlast = -1;
  double wexcl = 0.0;
  run = 0.0;
#pragma unroll
  for (int ww = 0; ww < kVWarps; ++ww) {
    const double x = w[ww][0];
    if (x > 0.0) wlast = ww;
    if (!take_last && wstar < 0 && run + x > tl) { wstar = ww; wexcl = run; }
    run += x;
  }
  if (wstar < 0) { wstar = wlast; take_last = true; }
  if (c.warp != wstar) return;
  tl -= wexcl;
  double carry = 0.0;
  int found = -1, last_pos = -1;
  for (int base = s_lo; base < s_hi && found < 0; base += 32) {
    const int t = base + c.lane;
    const float val = t < s_hi ? resid(c.ps[t] * st.ip, has_q ? c.qs[t] * st.iq : 0.f, Cf, Uf) : 0.f;
    double incl = (double)val;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double up = __shfl_up_sync(0xffffffffu, incl, o);
      if (c.lane >= o) incl += up;
    }
    const uint32_t pos = __ballot_sync(0xffffffffu, val > 0.f);
    if (pos) last_pos = base + 31 - __clz(pos);
    if (!take_last) {
      const uint32_t hit = __ballot_sync(0xffffffffu, val > 0.f && carry + incl > tl);
      if (hit) found = base + __ffs(hit) - 1;
    }
    carry += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (found < 0) found = last_pos;
  if (c.lane == 0) *a.bonus = c.lo + (found < 0 ? 0 : found);
}

__global__ void __launch_bounds__(kVThreads, 1) tree_verify_kernel(const VerifyArgs a) {
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) float dyn_smem[];
  __shared__ VShared sh;
  Ctx c;
  c.sh = &sh;
  c.ps = dyn_smem;
  c.qs = dyn_smem + a.slice_cap;
  c.rank = (int)cluster.block_rank();
  c.lo = min(c.rank * a.slice_cap, a.V);
  c.cnt = min(a.V - c.lo, a.slice_cap);
  c.wpar = 0; c.xpar = 0;
  c.tid = threadIdx.x; c.warp = threadIdx.x >> 5; c.lane = threadIdx.x & 31;

  for (int i = c.tid; i < a.n; i += kVThreads) {
    int p = a.parent[i];
    if (i == 0) p = -1;
    else if (p < -1 || p >= i) { dev_flag(a.dev_status, SEQ_DEV_BAD_PARENT); p = -1; }
    sh.parent[i] = p;
    sh.tokens[i] = a.tokens[i];
  }
  if (a.temperature != 0.f)
    for (int i = c.tid; i <= a.n; i += kVThreads) sh.uniforms[i] = a.uniforms[i];
  __syncthreads();
  cluster.sync();  // every CTA of the cluster is resident before any remote shared-memory write

  NodeState st;
  st.greedy_token = 0;
  const int cluster_id = blockIdx.x / kVCluster, n_clusters = gridDim.x / kVCluster;

  if (a.flags & SEQ_VERIFY_ALL_NODES) {
    // test hook: every node gets its own run of Algorithm 2's loop; no walk, no final draw
    for (int v = cluster_id; v < a.n; v += n_clusters) {
      const int acc = process_node(cluster, c, a, v, st, true);
      if (c.rank == 0 && c.tid == 0) a.next_child_out[v] = acc;
      __syncthreads();
    }
    cluster.sync();
    return;
  }

  if (a.next_child_out != nullptr && c.rank == 0)
    for (int i = c.tid; i < a.n; i += kVThreads) a.next_child_out[i] = -2;
  __syncthreads();
  int cur = 0, plen = 0;
  for (int hop = 0; hop < a.n; ++hop) {  // a walk visits at most n nodes
    if (c.rank == 0 && c.tid == 0) a.path[plen] = cur;
    ++plen;
    const int acc = process_node(cluster, c, a, cur, st, false);
    if (c.rank == 0 && c.tid == 0 && a.next_child_out != nullptr) a.next_child_out[cur] = acc;
    if (acc < 0) break;
    cur = acc;
    __syncthreads();
  }
  if (c.rank == 0 && c.tid == 0) *a.path_len = plen;
  draw_bonus(cluster, c, a, st);
  cluster.sync();  // no CTA leaves while a sibling may still address its shared memory
}

}  // namespace seqtree

using namespace seqtree;

static int verify_validate(const seq_tree_verify_params* p) {
  if (p == nullptr) return SEQ_ERR_INVALID_ARG;
  if (p->n_tree < 1 || p->n_tree > SEQ_MAX_TREE || p->vocab < 1) return SEQ_ERR_INVALID_ARG;
  if (p->parent == nullptr || p->tokens == nullptr || p->target_logits == nullptr) return SEQ_ERR_INVALID_ARG;
  if (!(p->temperature >= 0.f) || isinf(p->temperature)) return SEQ_ERR_INVALID_ARG;
  if (p->flags & ~SEQ_VERIFY_ALL_NODES) return SEQ_ERR_INVALID_ARG;
  const bool all_nodes = p->flags & SEQ_VERIFY_ALL_NODES;
  if (all_nodes) {
    if (p->next_child_out == nullptr) return SEQ_ERR_INVALID_ARG;
  } else if (p->path == nullptr || p->path_len == nullptr || p->bonus_token == nullptr) {
    return SEQ_ERR_INVALID_ARG;
  }
  if (p->temperature > 0.f && (p->draft_logits == nullptr || p->uniforms == nullptr)) return SEQ_ERR_INVALID_ARG;
  if (p->target_row_stride < p->vocab || p->target_row_stride % 4 != 0 ||
      reinterpret_cast<uintptr_t>(p->target_logits) % 16 != 0)
    return SEQ_ERR_INVALID_ARG;
  if (p->draft_logits != nullptr &&
      (p->draft_row_stride < p->vocab || p->draft_row_stride % 4 != 0 ||
       reinterpret_cast<uintptr_t>(p->draft_logits) % 16 != 0))
    return SEQ_ERR_INVALID_ARG;
  return SEQ_OK;
}

extern "C" size_t seq_tree_verify_workspace_bytes(const seq_tree_verify_params* p) {
  (void)p;
  return 0;  // all scratch lives in (distributed) shared memory
}

extern "C" int seq_tree_verify(const seq_tree_verify_params* p, void* stream) {
  int rc = verify_validate(p);
  if (rc != SEQ_OK) return rc;
  VerifyArgs a;
  a.n = p->n_tree; a.V = p->vocab; a.flags = p->flags;
  a.slice_cap = (((p->vocab + kVCluster - 1) / kVCluster) + 3) & ~3;
  a.parent = p->parent; a.tokens = p->tokens;
  a.target = p->target_logits; a.target_stride = p->target_row_stride;
  a.draft = p->draft_logits != nullptr ? p->draft_logits : p->target_logits;
  a.draft_stride = p->draft_logits != nullptr ? p->draft_row_stride : p->target_row_stride;
  a.temperature = p->temperature; a.uniforms = p->uniforms;
  a.path = p->path; a.path_len = p->path_len; a.bonus = p->bonus_token;
  a.residual_out = p->residual_out; a.next_child_out = p->next_child_out; a.dev_status = p->dev_status;

  const size_t dyn = (size_t)2 * a.slice_cap * sizeof(float);
  if (dyn + kVStaticSmem > 227 * 1024) return SEQ_ERR_UNSUPPORTED;  // vocabulary too large for 8 slices
  SEQ_CUDA_OK(cudaFuncSetAttribute(tree_verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn));

  int n_clusters = 1;
  if (p->flags & SEQ_VERIFY_ALL_NODES) n_clusters = p->n_tree < 18 ? p->n_tree : 18;  // 18 * 8 = 144 CTAs <= 148 SMs
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_clusters * kVCluster);
  cfg.blockDim = dim3(kVThreads);
  cfg.dynamicSmemBytes = dyn;
  cfg.stream = (cudaStream_t)stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kVCluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  SEQ_CUDA_OK(cudaLaunchKernelEx(&cfg, tree_verify_kernel, a));
  return SEQ_OK;
}
