// The verification kernel and everything it is made of, for ONE cluster size: included once per size by
// tree_verify.cu with SEQ_VCL (CTAs per cluster) and SEQ_VNS (a namespace for this instance) defined.
namespace SEQ_VNS {

constexpr int kVCluster = SEQ_VCL;
constexpr int kVParts = kVCluster * kVWarps;  // (rank, warp) segments cover the vocabulary
constexpr int kVPPL = kVParts / 32;           // segments per lane in an exchange: lane l reads segments l, l + 32, ...
static_assert(kVParts % 32 == 0 && kVCluster <= 32, "an exchange reads whole groups of 32 segments; one lane per CTA writes");

struct VShared {
  int32_t parent[SEQ_MAX_TREE];
  int32_t tokens[SEQ_MAX_TREE];
  float uniforms[SEQ_MAX_TREE + 1];
  int32_t kids[SEQ_MAX_TREE];
  // (target exp, draft exp, target segment max, draft segment max) of each child's token, written by
  // the warp that owns the token into every CTA; double-buffered by node so that a CTA that runs
  // ahead never overwrites what a sibling still reads
  float4 kid_pq[2][SEQ_MAX_TREE];
  uint8_t dup[SEQ_MAX_TREE];            // child i carries the token of an earlier sibling
  uint32_t has_child[SEQ_MAX_TREE / 32];
  float4 xbuf[2][kVParts];              // cluster exchange: one entry per (rank, warp), double-buffered
  int32_t wcnt[kVWarps];
  int32_t drawn[2];                     // the token sampled from the target at this node (SEQ_VERIFY_TARGET_SAMPLE)
  uint64_t bar[2];                      // completion of the target / draft slice copies
};

// Per-thread copy of the replicated walk state at the current node.
struct NodeState {
  float c2;             // log2(e)/T
  float Mp, Mq;         // global maxima of the two rows
  float invSp, invSq;   // 1 / sum of exponentials relative to the global maxima
  float ipw, iqw;       // this warp's factors turning its stored exponentials into probabilities
  double C, U, Z, ZD;
  double part_sum[kVPPL];  // residual mass of segments `lane`, `lane + 32`, ... (probability units)
  int mode;             // 0: D proportional to q; 1: uniform over the non-rejected set
  int nS;               // |S|
  int has_q;            // qs holds this node's draft slice
  int greedy_token;     // the token fixed at this node: the target arg-max (T = 0), or the sample from the target
};

struct Ctx {
  VShared* sh;
  float* ps; float* qs;
  int rank, lo, cnt, seg, s_lo, s_hi;  // slice, and this warp's segment of it
  int xpar, npar;
  uint32_t ph[2];
  int tid, warp, lane;
};

__device__ __forceinline__ uint32_t vsmem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ float sanitize_logit(float x, int32_t* dev_status) {
  if (x < INFINITY) return x;  // finite or -inf
  dev_flag(dev_status, SEQ_DEV_NONFINITE);
  return x != x ? -INFINITY : FLT_MAX;
}
__device__ __forceinline__ float fast_ex2(float x) {  // 2^x, relative error 2^-22; 2^-inf = 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^((m - M) c2), and 0 for an empty (all -inf) part
__device__ __forceinline__ float rel_exp(float m, float M, float c2) {
  return m == -INFINITY ? 0.f : fast_ex2((m - M) * c2);
}
// unnormalised residual max(p - C q - U, 0) of one token
__device__ __forceinline__ float resid(float pn, float qn, float Cf, float Uf) {
  return fmaxf(fmaf(-Cf, qn, pn) - Uf, 0.f);
}

// Visit this warp's segment four elements per lane at a time (conflict-free 16-byte accesses);
// f4(t) handles elements t..t+3, f1(t) a single element of the ragged end.
template <typename F4, typename F1>
__device__ __forceinline__ void sweep(const Ctx& c, F4 f4, F1 f1) {
  int t = c.s_lo + 4 * c.lane;
#pragma unroll 1
  for (; t + 3 < c.s_hi; t += 128) f4(t);
#pragma unroll 1
  for (int e = t; e < c.s_hi && e < t + 4; ++e) f1(e);
}

__device__ __forceinline__ double sum_lanes(double v, int width) {  // butterfly over `width` lanes
  for (int o = width >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Every warp of every CTA publishes one float4 to every CTA of the cluster.  On return x.e[m] holds the entry of
// segment lane + 32 m (segments are numbered rank-major, i.e. in vocabulary order).
struct Exch { float4 e[kVPPL]; };
__device__ __forceinline__ void cluster_exchange(cg::cluster_group& cluster, Ctx& c, float4 mine, Exch& x) {
  if (c.lane < kVCluster) *cluster.map_shared_rank(&c.sh->xbuf[c.xpar][c.rank * kVWarps + c.warp], c.lane) = mine;
  cluster.sync();
#pragma unroll
  for (int m = 0; m < kVPPL; ++m) x.e[m] = c.sh->xbuf[c.xpar][c.lane + 32 * m];
  c.xpar ^= 1;
}

__device__ __forceinline__ double part_total(const double* part_sum) {
  double t = part_sum[0];
#pragma unroll
  for (int m = 1; m < kVPPL; ++m) t += part_sum[m];
  return sum_lanes(t, 32);
}

// Children of v in ascending node order -> sh->kids; returns their count.  Two barriers.
__device__ int build_kids(Ctx& c, int v, int n) {
  // each thread owns four consecutive candidates so that warps and lanes are in node order
  const int c0 = v + 1 + 4 * c.tid;
  int f = 0;
#pragma unroll
  for (int e = 0; e < 4; ++e) f |= (int)(c0 + e < n && c.sh->parent[c0 + e] == v) << e;
  const int mine = __popc(f);
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
#pragma unroll
  for (int e = 0; e < 4; ++e)
    if ((f >> e) & 1) c.sh->kids[pos++] = c0 + e;
  __syncthreads();
  return total;
}

// Start the asynchronous copy of this CTA's slice of one row into shared memory (16-byte body only).
__device__ __forceinline__ void start_slice_copy(const Ctx& c, const float* row, float* dst, int which) {
  const uint32_t bytes = (uint32_t)(c.cnt & ~3) * 4u;
  if (bytes == 0) return;
  const uint32_t bar = vsmem_u32(&c.sh->bar[which]);
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(vsmem_u32(dst)), "l"(row + c.lo), "r"(bytes), "r"(bar) : "memory");
}
// Bounded wait for a slice copy; the ragged tail (at most 3 elements) is fetched by the warp that owns it.
__device__ __forceinline__ void finish_slice_copy(Ctx& c, const float* row, float* dst, int which, int32_t* dev_status) {
  if ((c.cnt & ~3) != 0) {
    const uint32_t bar = vsmem_u32(&c.sh->bar[which]);
    uint32_t ok = 0;
    for (uint32_t it = 0; it < kVSpinLimit && !ok; ++it) {
      asm volatile(
          "{\n\t.reg .pred p;\n\t"
          "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
          "selp.u32 %0, 1, 0, p;\n\t}"
          : "=r"(ok) : "r"(bar), "r"(c.ph[which]) : "memory");
    }
    if (!ok) dev_flag(dev_status, SEQ_DEV_TIMEOUT);
    c.ph[which] ^= 1u;
  }
  const int t = (c.cnt & ~3) + c.lane;
  if (t < c.cnt && t >= c.s_lo && t < c.s_hi) dst[t] = __ldg(row + c.lo + t);
  __syncwarp();
}
__device__ __forceinline__ bool node_has_child(const Ctx& c, int v) { return (c.sh->has_child[v >> 5] >> (v & 31)) & 1u; }

// Rare path of the maximum sweep: this warp's segment holds a NaN or +inf logit (or mixes -inf and a huge
// value in one group of four).  Every element is checked, offenders are flagged and replaced in place, and the
// segment maxima are taken again.
__device__ __noinline__ void sanitize_segment(Ctx& c, bool need_draft, int32_t* dev_status, float& mp, float& mq) {
  mp = -INFINITY; mq = -INFINITY;
  for (int t = c.s_lo + c.lane; t < c.s_hi; t += 32) {
    float x = c.ps[t];
    if (!(x < INFINITY)) { x = sanitize_logit(x, dev_status); c.ps[t] = x; }
    mp = fmaxf(mp, x);
    if (need_draft) {
      float y = c.qs[t];
      if (!(y < INFINITY)) { y = sanitize_logit(y, dev_status); c.qs[t] = y; }
      mq = fmaxf(mq, y);
    }
  }
  __syncwarp();
}

// Runs Algorithm 2's loop at node v.  Returns the accepted child's node id or -1 and leaves in
// `st` (and in ps/qs/wseg) the state the final draw needs.
__device__ int draw_token(Ctx& c, const NodeState& st, float u, float Cf, float Uf, float ipw, float iqw,
                          const float* qsrc, double total);

__device__ int process_node(cg::cluster_group& cluster, Ctx& c, const VerifyArgs& a, int v, NodeState& st,
                            bool skip_leaves, bool copies_started) {
  const bool greedy = a.temperature == 0.f;
  const bool specinfer = (a.flags & SEQ_VERIFY_SPECINFER) != 0;  // D is never touched: ZD stays 1, S stays empty
  const bool has_kids = node_has_child(c, v);
  if (skip_leaves && !has_kids) return -1;
  // verification by sampling from the target (at T = 0 that is the greedy branch): the draft plays no part
  const bool tsample = !greedy && (a.flags & SEQ_VERIFY_TARGET_SAMPLE) != 0;
  const bool need_draft = !greedy && !tsample && (has_kids || (copies_started && a.n > 1));
  const float* trow = a.target + (int64_t)v * a.target_stride;
  const float* drow = a.draft + (int64_t)v * a.draft_stride;
  c.npar ^= 1;
  float4* kid_pq = c.sh->kid_pq[c.npar];
  // two slots by node parity: a thread may still be reading the previous node's slot, and cluster barriers
  // lie between this reset and the remote write below
  if (tsample && c.tid == 0) c.sh->drawn[c.npar] = -3;
  if (c.tid == 0 && !copies_started) {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // earlier plain writes to the slices come first
    start_slice_copy(c, trow, c.ps, 0);
    if (need_draft) start_slice_copy(c, drow, c.qs, 1);
  }
  TRACE(1);
  const int k = build_kids(c, v, a.n);  // overlaps the copies
  TRACE(22);
  // duplicates among siblings
#pragma unroll 1
  for (int i = c.tid; i < k; i += kVThreads) {
    const int s = c.sh->tokens[c.sh->kids[i]];
    int d = 0;
#pragma unroll 1
    for (int j = 0; j < i; ++j) d |= c.sh->tokens[c.sh->kids[j]] == s;
    c.sh->dup[i] = (uint8_t)d;
  }
  // (The children's rows are NOT prefetched into L2 here: a bulk prefetch takes a few hundred cycles to issue and the
  // copy of the accepted child's rows then finds the bulk-copy unit busy; measured 0.4 us per step slower on 32000
  // logits and 3 us slower on 128256 than without, wherever in the node's work the prefetch is issued.)
  TRACE(2);
  finish_slice_copy(c, trow, c.ps, 0, a.dev_status);
  if (need_draft) finish_slice_copy(c, drow, c.qs, 1, a.dev_status);
  TRACE(3);

  if (greedy) {
    // arg-max of the target row, lowest index on ties (each lane meets its elements in ascending order)
    float best = -INFINITY;
    int best_idx = 0x7fffffff;
    auto upd = [&](int t) {
      const float x = sanitize_logit(c.ps[t], a.dev_status);
      if (x > best || best_idx == 0x7fffffff) { best = x; best_idx = c.lo + t; }
    };
    sweep(c, [&](int t) { upd(t); upd(t + 1); upd(t + 2); upd(t + 3); }, upd);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, best_idx, o);
      if (oi != 0x7fffffff && (best_idx == 0x7fffffff || ob > best || (ob == best && oi < best_idx))) { best = ob; best_idx = oi; }
    }
    Exch x;
    cluster_exchange(cluster, c, make_float4(best, __int_as_float(best_idx), 0.f, 0.f), x);
    float gb = x.e[0].x; int gi = __float_as_int(x.e[0].y);
#pragma unroll
    for (int m = 1; m < kVPPL; ++m) {
      const float ob = x.e[m].x; const int oi = __float_as_int(x.e[m].y);
      if (oi != 0x7fffffff && (gi == 0x7fffffff || ob > gb || (ob == gb && oi < gi))) { gb = ob; gi = oi; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, gb, o);
      const int oi = __shfl_xor_sync(0xffffffffu, gi, o);
      if (oi != 0x7fffffff && (gi == 0x7fffffff || ob > gb || (ob == gb && oi < gi))) { gb = ob; gi = oi; }
    }
    st.greedy_token = gi == 0x7fffffff ? 0 : gi;
    for (int i = 0; i < k; ++i) {
      const int ch = c.sh->kids[i];
      const int s = c.sh->tokens[ch];
      if (s < 0 || s >= a.V) { dev_flag(a.dev_status, SEQ_DEV_BAD_TOKEN); continue; }
      if (s == st.greedy_token) return ch;
    }
    return -1;
  }

  const float c2 = st.c2;
  // segment maxima; a NaN or +inf logit is flagged and replaced in place (rare path, out of line).  A sum of
  // four elements is NaN or +inf exactly when one of them is NaN or +inf or they mix -inf with +inf, so one
  // comparison per float4 finds the rows that need the slow path.
  float mp = -INFINITY, mq = -INFINITY;
  {
    bool bad = false;
    auto f1 = [&](int t) {
      const float x = c.ps[t];
      bad |= !(x < INFINITY);
      mp = fmaxf(mp, x);
      if (need_draft) { const float y = c.qs[t]; bad |= !(y < INFINITY); mq = fmaxf(mq, y); }
    };
    auto f4 = [&](int t) {
      const float4 x = *reinterpret_cast<const float4*>(c.ps + t);
      bad |= !((x.x + x.y) + (x.z + x.w) < INFINITY);
      mp = fmaxf(mp, fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w)));
      if (need_draft) {
        const float4 y = *reinterpret_cast<const float4*>(c.qs + t);
        bad |= !((y.x + y.y) + (y.z + y.w) < INFINITY);
        mq = fmaxf(mq, fmaxf(fmaxf(y.x, y.y), fmaxf(y.z, y.w)));
      }
    };
    sweep(c, f4, f1);
    if (__any_sync(0xffffffffu, bad)) sanitize_segment(c, need_draft, a.dev_status, mp, mq);
  }
  mp = warp_max(mp);
  mq = warp_max(mq);
  TRACE(4);
  // exponentials relative to the segment maxima, with their sums
  float sp = 0.f, sq = 0.f;
  {
    const float mpe = mp == -INFINITY ? 0.f : mp, mqe = mq == -INFINITY ? 0.f : mq;  // an all -inf segment stays 0
    auto f1 = [&](int t) {
      const float e = fast_ex2((c.ps[t] - mpe) * c2);
      c.ps[t] = e; sp += e;
      if (need_draft) { const float f = fast_ex2((c.qs[t] - mqe) * c2); c.qs[t] = f; sq += f; }
    };
    auto f4 = [&](int t) {
      float4 x = *reinterpret_cast<const float4*>(c.ps + t);
      x.x = fast_ex2((x.x - mpe) * c2); x.y = fast_ex2((x.y - mpe) * c2);
      x.z = fast_ex2((x.z - mpe) * c2); x.w = fast_ex2((x.w - mpe) * c2);
      *reinterpret_cast<float4*>(c.ps + t) = x;
      sp += (x.x + x.y) + (x.z + x.w);
      if (need_draft) {
        float4 y = *reinterpret_cast<const float4*>(c.qs + t);
        y.x = fast_ex2((y.x - mqe) * c2); y.y = fast_ex2((y.y - mqe) * c2);
        y.z = fast_ex2((y.z - mqe) * c2); y.w = fast_ex2((y.w - mqe) * c2);
        *reinterpret_cast<float4*>(c.qs + t) = y;
        sq += (y.x + y.y) + (y.z + y.w);
      }
    };
    sweep(c, f4, f1);
  }
  sp = warp_sum(sp);
  sq = warp_sum(sq);
  __syncwarp();
  // every child's stored exponentials go from the warp that owns its token to all CTAs
  for (int i = c.lane; i < k; i += 32) {
    const int s = c.sh->tokens[c.sh->kids[i]] - c.lo;
    if (s >= c.s_lo && s < c.s_hi) {
      const float4 pq = make_float4(c.ps[s], need_draft ? c.qs[s] : 0.f, mp, mq);
      for (int r = 0; r < kVCluster; ++r) *cluster.map_shared_rank(&kid_pq[i], r) = pq;
    }
  }
  TRACE(5);
  Exch x;
  cluster_exchange(cluster, c, make_float4(mp, sp, mq, sq), x);
  TRACE(6);
  {
    float Mp = x.e[0].x, Mq = x.e[0].z;
#pragma unroll
    for (int m = 1; m < kVPPL; ++m) { Mp = fmaxf(Mp, x.e[m].x); Mq = fmaxf(Mq, x.e[m].z); }
    Mp = warp_max(Mp); Mq = warp_max(Mq);
    double am[kVPPL], asum = 0.0, bsum = 0.0;
#pragma unroll
    for (int m = 0; m < kVPPL; ++m) {
      am[m] = (double)x.e[m].y * (double)rel_exp(x.e[m].x, Mp, c2);
      asum += am[m];
      bsum += (double)x.e[m].w * (double)rel_exp(x.e[m].z, Mq, c2);
    }
    const double Sp = sum_lanes(asum, 32), Sq = sum_lanes(bsum, 32);
    if (!(Sp > 0.0)) dev_flag(a.dev_status, SEQ_DEV_DEGENERATE);
    st.Mp = Mp; st.Mq = Mq;
    st.invSp = Sp > 0.0 ? (float)(1.0 / Sp) : 0.f;
    st.invSq = (need_draft && Sq > 0.0) ? (float)(1.0 / Sq) : 0.f;
#pragma unroll
    for (int m = 0; m < kVPPL; ++m) st.part_sum[m] = am[m] * (double)st.invSp;
    st.mode = (need_draft && !(Sq > 0.0)) ? 1 : 0;  // a draft row without mass: the fallback from the start
  }
  st.ipw = rel_exp(mp, st.Mp, c2) * st.invSp;
  st.iqw = rel_exp(mq, st.Mq, c2) * st.invSq;
  st.C = 0.0; st.U = 0.0; st.Z = 1.0; st.ZD = 1.0; st.nS = 0; st.has_q = need_draft;
  TRACE(7);

  if (tsample) {
    // x ~ P with this node's uniform; the warp that finds x tells every CTA; a child that carries x is taken
    const double total = part_total(st.part_sum);
    const int found = draw_token(c, st, c.sh->uniforms[v], 0.f, 0.f, st.ipw, 0.f, c.ps, total);
    if (found >= 0)
      for (int r = 0; r < kVCluster; ++r) *cluster.map_shared_rank(&c.sh->drawn[c.npar], r) = found;
    cluster.sync();
    int x = c.sh->drawn[c.npar];
    if (x < 0) { dev_flag(a.dev_status, SEQ_DEV_DEGENERATE); x = 0; }  // a target row without mass
    st.greedy_token = x;
    for (int i = 0; i < k; ++i) {
      const int ch = c.sh->kids[i];
      const int s = c.sh->tokens[ch];
      if (s < 0 || s >= a.V) { dev_flag(a.dev_status, SEQ_DEV_BAD_TOKEN); continue; }
      if (s == x) return ch;
    }
    return -1;
  }

  for (int i = 0; i < k; ++i) {
    const int ch = c.sh->kids[i];
    const int s = c.sh->tokens[ch];
    if (s < 0 || s >= a.V) { dev_flag(a.dev_status, SEQ_DEV_BAD_TOKEN); continue; }
    // an earlier (hence rejected) sibling carried the same token: it is in S.  (Without the draft update there is no
    // S: a repeated token is tested like any other, and its R is 0 by then.)
    const bool in_S = !specinfer && c.sh->dup[i] != 0;
    float pn = 0.f, qn = 0.f;
    if (!in_S) {
      const float4 pq = kid_pq[i];
      pn = pq.x * (rel_exp(pq.z, st.Mp, c2) * st.invSp);
      qn = pq.y * (rel_exp(pq.w, st.Mq, c2) * st.invSq);
    }
    // the acceptance test: accept iff u < R[s]/D[s], with R[s] = rs/Z and D[s] = qn/ZD (or 1/(V-|S|)); cross-multiplied,
    // which also covers D[s] = 0 (accept iff R[s] > 0)
    const double rs = in_S ? 0.0 : (double)resid(pn, qn, (float)st.C, (float)st.U);
    const double u = (double)c.sh->uniforms[ch];
    const bool accept = st.mode == 0 ? (u * st.Z * (double)qn < rs * st.ZD) : (u * st.Z < rs * (double)(a.V - st.nS));
    TRACE(8);
    if (accept) return ch;

    // the residual update: R <- norm(max(R - D, 0)) with D as it stands
    double Cn = st.C, Un = st.U;
    if (st.mode == 0) Cn += st.Z / st.ZD;
    else if (a.V - st.nS > 0) Un += st.Z / (double)(a.V - st.nS);
    // the draft update: D[s] <- 0, s joins S; done by the warp that owns s
    if (!in_S && !specinfer) {
      const int sl = s - c.lo;
      if (sl >= c.s_lo && sl < c.s_hi && c.lane == 0) { c.ps[sl] = 0.f; c.qs[sl] = 0.f; }
      st.nS += 1;
    }
    __syncwarp();
    const float Cnf = (float)Cn, Unf = (float)Un, ipw = st.ipw, iqw = st.iqw;
    float zr = 0.f, zd = 0.f;
    {
      auto f1 = [&](int t) {
        const float qt = c.qs[t] * iqw;
        zr += resid(c.ps[t] * ipw, qt, Cnf, Unf);
        zd += qt;
      };
      auto f4 = [&](int t) {
        const float4 x = *reinterpret_cast<const float4*>(c.ps + t);
        const float4 y = *reinterpret_cast<const float4*>(c.qs + t);
        const float q0 = y.x * iqw, q1 = y.y * iqw, q2 = y.z * iqw, q3 = y.w * iqw;
        zr += (resid(x.x * ipw, q0, Cnf, Unf) + resid(x.y * ipw, q1, Cnf, Unf)) +
              (resid(x.z * ipw, q2, Cnf, Unf) + resid(x.w * ipw, q3, Cnf, Unf));
        zd += (q0 + q1) + (q2 + q3);
      };
      sweep(c, f4, f1);
    }
    zr = warp_sum(zr);
    zd = warp_sum(zd);
    TRACE(9);
    cluster_exchange(cluster, c, make_float4(zr, zd, 0.f, 0.f), x);
    TRACE(10);
    double zsum = 0.0, zdsum = 0.0;
#pragma unroll
    for (int m = 0; m < kVPPL; ++m) { zsum += (double)x.e[m].x; zdsum += (double)x.e[m].y; }
    const double Zn = sum_lanes(zsum, 32), ZDn = sum_lanes(zdsum, 32);
    if (Zn > 0.0) {
      st.C = Cn; st.U = Un; st.Z = Zn;
#pragma unroll
      for (int m = 0; m < kVPPL; ++m) st.part_sum[m] = (double)x.e[m].x;
    } else {
      dev_flag(a.dev_status, SEQ_DEV_DEGENERATE);  // keep R
    }
    if (!specinfer) {
      st.ZD = ZDn;
      if (st.mode == 0 && !(ZDn > 0.0)) st.mode = 1;  // no mass left in D: uniform over the non-rejected set
    }
  }
  return -1;
}

// x ~ R by inverse CDF in index order with the uniform u, R being the residual max(p - C q - U, 0) of the
// current node (the target distribution itself when C = U = 0).  Returns the token in lane 0 of the one warp of
// the cluster whose segment holds the crossing, -1 in every other thread, and -3 in every thread when R has no
// mass at all.
__device__ int draw_token(Ctx& c, const NodeState& st, float u, float Cf, float Uf, float ipw, float iqw,
                          const float* qsrc, double total) {
  // inverse CDF over the 64 (rank, warp) segments: inclusive scan across lanes, segments `lane` first
  const double tgt = (double)u * total;
  // inclusive scan over the segments in vocabulary order: across lanes within a group of 32, groups in turn
  double inc[kVPPL], before = 0.0;
  uint32_t hit[kVPPL], pos[kVPPL];
#pragma unroll
  for (int m = 0; m < kVPPL; ++m) {
    double v = st.part_sum[m];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double up = __shfl_up_sync(0xffffffffu, v, o);
      if (c.lane >= o) v += up;
    }
    inc[m] = v + before;
    before = __shfl_sync(0xffffffffu, inc[m], 31);
    hit[m] = __ballot_sync(0xffffffffu, st.part_sum[m] > 0.0 && inc[m] > tgt);
    pos[m] = __ballot_sync(0xffffffffu, st.part_sum[m] > 0.0);
  }
  int part = -1;     // segment holding the crossing
  bool take_last = false;
#pragma unroll
  for (int m = 0; m < kVPPL; ++m)
    if (part < 0 && hit[m]) part = 32 * m + __ffs(hit[m]) - 1;
  if (part < 0) {    // rounding left the total at or below the target: the last segment with mass
    take_last = true;
#pragma unroll
    for (int m = kVPPL - 1; m >= 0; --m)
      if (part < 0 && pos[m]) part = 32 * m + 31 - __clz(pos[m]);
    if (part < 0) return -3;  // no mass anywhere: degenerate input (every thread of the cluster sees this)
  }
  if (part != c.rank * kVWarps + c.warp) return -1;
  double incl_part = 0.0, mass_part = 0.0;
#pragma unroll
  for (int m = 0; m < kVPPL; ++m) {  // (every lane of the owning warp takes part in the shuffles)
    const double i_m = __shfl_sync(0xffffffffu, inc[m], part & 31), s_m = __shfl_sync(0xffffffffu, st.part_sum[m], part & 31);
    if ((part >> 5) == m) { incl_part = i_m; mass_part = s_m; }
  }
  const double tl = tgt - (incl_part - mass_part);  // target within this warp's segment
  double carry = 0.0;
  int found = -1, last_pos = -1;
  for (int base = c.s_lo; base < c.s_hi && found < 0; base += 32) {
    const int t = base + c.lane;
    const float val = t < c.s_hi ? resid(c.ps[t] * ipw, qsrc[t] * iqw, Cf, Uf) : 0.f;
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
  return c.lane == 0 ? c.lo + (found < 0 ? c.s_lo : found) : -1;
}


// Algorithm 2's final draw, x ~ R with uniforms[n]; optionally writes R.  (Greedy, and verification by sampling from the target:
// the token was fixed at the last node, R is the distribution it came from.)
__device__ void draw_bonus(Ctx& c, const VerifyArgs& a, const NodeState& st) {
  if (a.temperature == 0.f) {
    if (a.residual_out != nullptr)
      for (int t = c.tid; t < c.cnt; t += kVThreads) a.residual_out[c.lo + t] = (c.lo + t == st.greedy_token) ? 1.f : 0.f;
    if (c.rank == 0 && c.tid == 0) *a.bonus = st.greedy_token;
    return;
  }
  if (a.flags & SEQ_VERIFY_TARGET_SAMPLE) {
    if (a.residual_out != nullptr)
      for (int t = c.s_lo + c.lane; t < c.s_hi; t += 32) a.residual_out[c.lo + t] = c.ps[t] * st.ipw;
    if (c.rank == 0 && c.tid == 0) *a.bonus = st.greedy_token;
    return;
  }
  const float Cf = (float)st.C, Uf = (float)st.U;
  const bool has_q = st.has_q && (st.C != 0.0);
  const float ipw = st.ipw, iqw = has_q ? st.iqw : 0.f;
  const float* qsrc = has_q ? c.qs : c.ps;  // never dereference a slice that was not loaded
  const double total = part_total(st.part_sum);

  if (a.residual_out != nullptr) {
    const float it = total > 0.0 ? (float)(1.0 / total) : 0.f;
    for (int t = c.s_lo + c.lane; t < c.s_hi; t += 32)
      a.residual_out[c.lo + t] = resid(c.ps[t] * ipw, qsrc[t] * iqw, Cf, Uf) * it;
  }

  const int x = draw_token(c, st, c.sh->uniforms[a.n], Cf, Uf, ipw, iqw, qsrc, total);
  if (x == -3) {
    if (c.rank == 0 && c.tid == 0) { *a.bonus = 0; dev_flag(a.dev_status, SEQ_DEV_DEGENERATE); }
  } else if (x >= 0) {
    *a.bonus = x;
  }
}

template <bool kBatch>
__global__ void __launch_bounds__(kVThreads, 1) tree_verify_kernel(const VerifyArgs a_in) {
  // One request per cluster in a batched launch: the same code on that request's arrays.
  VerifyArgs a_req;
  if (kBatch) {
    const int64_t r = blockIdx.x / kVCluster;
    a_req = a_in;
    a_req.parent += r * a_in.tree_stride; a_req.tokens += r * a_in.tree_stride;
    a_req.target += r * a_in.logits_stride; a_req.draft += r * a_in.logits_stride;
    a_req.uniforms += r * a_in.unif_stride;
    a_req.path += r * a_in.tree_stride; a_req.path_len += r; a_req.bonus += r;
    if (a_in.residual_out != nullptr) a_req.residual_out += r * a_in.resid_stride;
    if (a_in.next_child_out != nullptr) a_req.next_child_out += r * a_in.tree_stride;
  }
  const VerifyArgs& a = kBatch ? a_req : a_in;
  cg::cluster_group cluster = cg::this_cluster();
  extern __shared__ __align__(16) uint8_t dyn_smem[];  // VShared, then the two slices
  VShared& sh = *reinterpret_cast<VShared*>(dyn_smem);
  TRACE(0);
  Ctx c;
  c.sh = &sh;
  c.ps = reinterpret_cast<float*>(dyn_smem + sizeof(VShared));
  c.qs = c.ps + a.slice_cap;
  c.rank = (int)cluster.block_rank();
  c.lo = min(c.rank * a.slice_cap, a.V);
  c.cnt = min(a.V - c.lo, a.slice_cap);
  c.xpar = 0; c.npar = 0; c.ph[0] = 0; c.ph[1] = 0;
  c.tid = threadIdx.x; c.warp = threadIdx.x >> 5; c.lane = threadIdx.x & 31;
  c.seg = (((a.slice_cap + kVWarps - 1) / kVWarps) + 31) & ~31;  // contiguous, a multiple of 32 long
  c.s_lo = min(c.warp * c.seg, c.cnt);
  c.s_hi = min(c.s_lo + c.seg, c.cnt);
  const bool all_nodes = a.flags & SEQ_VERIFY_ALL_NODES;
  const bool greedy = a.temperature == 0.f;

  if (c.tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(vsmem_u32(&sh.bar[0])) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(vsmem_u32(&sh.bar[1])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // programmatic dependent launch: the next kernel in the stream may be scheduled onto free SMs from now on
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  // nothing above touches global memory; everything below may read what the previous kernel in the stream wrote
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (c.tid == 0) {
    if (!all_nodes) {  // the walk always starts at the root: fetch its rows while the tree is being read
      start_slice_copy(c, a.target, c.ps, 0);
      if (!greedy && a.n > 1 && !(a.flags & SEQ_VERIFY_TARGET_SAMPLE)) start_slice_copy(c, a.draft, c.qs, 1);  // draft row 0 is read whenever the tree has children
    }
  }
  if (c.tid < SEQ_MAX_TREE / 32) sh.has_child[c.tid] = 0u;
  __syncthreads();
  for (int i = c.tid; i < a.n; i += kVThreads) {
    int p = a.parent[i];
    if (i == 0) p = -1;
    else if (p < -1 || p >= i) { dev_flag(a.dev_status, SEQ_DEV_BAD_PARENT); p = -1; }
    sh.parent[i] = p;
    sh.tokens[i] = a.tokens[i];
    if (p >= 0) atomicOr(&sh.has_child[p >> 5], 1u << (p & 31));
  }
  if (!greedy)
    for (int i = c.tid; i <= a.n; i += kVThreads) sh.uniforms[i] = a.uniforms[i];
  TRACE(20);
  __syncthreads();
  cluster.sync();  // every CTA of the cluster is resident before any remote shared-memory write
  TRACE(21);

  NodeState st;
  st.greedy_token = 0;
  st.c2 = greedy ? 0.f : kLog2e / a.temperature;
  const int cluster_id = kBatch ? 0 : blockIdx.x / kVCluster, n_clusters = kBatch ? 1 : gridDim.x / kVCluster;

  if (!all_nodes && a.next_child_out != nullptr && c.rank == 0)
    for (int i = c.tid; i < a.n; i += kVThreads) a.next_child_out[i] = -2;
  __syncthreads();
  // One loop (and one copy of the per-node code) serves both schedules: the walk from the root, and the
  // test hook in which every node gets its own run of Algorithm 2's loop (no walk, no final draw).
  int cur = all_nodes ? cluster_id : 0, plen = 0;
  for (int hop = 0; hop < a.n && cur < a.n; ++hop) {  // a walk visits at most n nodes
    if (!all_nodes) {
      if (c.rank == 0 && c.tid == 0) a.path[plen] = cur;
      ++plen;
    }
    const int acc = process_node(cluster, c, a, cur, st, all_nodes, !all_nodes && hop == 0);
    if (c.rank == 0 && c.tid == 0 && a.next_child_out != nullptr) a.next_child_out[cur] = acc;
    if (all_nodes) cur += n_clusters;
    else if (acc < 0) break;
    else cur = acc;
    __syncthreads();  // all reads of this node's slices are done before the next copies land
  }
  if (all_nodes) return;
  if (c.rank == 0 && c.tid == 0) *a.path_len = plen;
  TRACE(11);
  draw_bonus(c, a, st);
  TRACE(12);
  // No closing cluster barrier: remote shared memory is only written before a cluster barrier that
  // every CTA joins, so nothing can still address a CTA that has left.
}

}  // namespace SEQ_VNS
