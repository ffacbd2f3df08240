/*
 * seq_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of what Sequoia's token-tree verification
 * step computes (Chen et al., "Sequoia: Scalable, Robust, and Hardware-aware
 * Speculative Decoding"):
 *   - the ancestor relation of a token tree given as a parent array
 *     (Section 2.2: verification proceeds from the root along parent links);
 *   - the target model's attention over that tree, where a tree token sees
 *     the committed prefix and its own root-to-node path (Section 1: the
 *     whole tree is verified by one forward pass of the target model);
 *   - Algorithm 2 ("Sequoia Sampling and Verification") applied recursively
 *     from the root (Section 2.2), ending with the draw x ~ R;
 *   - the draft side's draw of a node's children without replacement by
 *     exponential sort (Section 5, "Implementation Details");
 *   - verification by sampling from the target (Section 2.2, naive / top-k
 *     sampling), the commit of an accepted path into the cache, and the nucleus
 *     (top-p) truncation of a distribution (Section 4.2's robustness study).
 *
 * Nothing here is blocked, fused or reordered: every function is the
 * definition, or the algorithm's steps in the paper's order and notation, so
 * it can be checked against the paper by eye.  It shares no code, headers,
 * tables or constants with the CUDA library.  Only tests, the smoke check and
 * the benchmark's cpu_baseline leg may call it.
 *
 * Parity pins (tests marked "not gpu"): exact enumeration of Algorithm 2's
 * output distribution (must equal P, Appendix "Proof of correctness"), the
 * printed P=[1,0], Q=[.5,.5] example of Theorem 3.7's proof, the optimal-
 * transport closed form 1-|P-Q|_1/2 at k=1, the cover property, the lemma
 * P(reject at i) = sum max(0, t_i - d_i), reduction of a chain to Algorithm 3,
 * Monte-Carlo; attention against library causal attention (chain tree),
 * single-query decode (star tree) and explicit-sequence brute force; the
 * exponential sort against the exact without-replacement law of ordered pairs
 * (Monte-Carlo), library sorts in its two degenerate cases, and invariants;
 * the commit against a library gather, hand-written cases where a row is both
 * read and overwritten, and the identity "attention of a path node over the
 * tree == causal attention over the committed cache"; the nucleus against the
 * three properties that characterise it, a library sort + cumsum, closed forms.
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC seq_oracle.c -o liboracle.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* data-problem flags reported by the oracle (its own numbering) */
#define ORC_BAD_PARENT 1
#define ORC_BAD_TOKEN 2
#define ORC_NONFINITE 4
#define ORC_DEGENERATE 8
#define ORC_BAD_PATH 32

#define ORC_VARIANT_SEQUOIA 0   /* Algorithm 2 as printed */
#define ORC_VARIANT_SPECINFER 1 /* Algorithm 2 without its draft update (the steps that are Sequoia's addition) */

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* A parent entry is usable iff it is -1 (no parent) or an earlier node.
 * Anything else is flagged and read as -1, so every walk below terminates. */
static int32_t clean_parent(const int32_t* parent, int32_t i, int* flags) {
  int32_t p = parent[i];
  if (p == -1) return -1;
  if (p < -1 || p >= i) {
    if (flags) *flags |= ORC_BAD_PARENT;
    return -1;
  }
  return p;
}

/*
 * Ancestor relation (Section 2.2: the verification walks the tree from its root):
 * bit j of row i is set iff j lies on the walk i, parent[i], parent[parent[i]], ...
 * depth[i] = number of parent links on that walk.
 */
int orc_mask_from_parents(const int32_t* parent, int32_t n, uint32_t* mask_bits,
                          int32_t words_per_row, int32_t* depth) {
  int flags = 0;
  for (int32_t i = 0; i < n; ++i) {
    uint32_t* row = mask_bits + (size_t)i * words_per_row;
    memset(row, 0, sizeof(uint32_t) * (size_t)words_per_row);
    int32_t j = i, links = 0;
    for (;;) {
      row[j >> 5] |= (uint32_t)1 << (j & 31);
      int32_t p = clean_parent(parent, j, &flags);
      if (p < 0) break;
      j = p;
      ++links;
    }
    if (depth) depth[i] = links;
  }
  return flags;
}

/*
 * Tree attention by its definition (Section 1: one target forward pass over
 * all tree tokens; each tree token conditions on the prefix x_{<n} followed by
 * the tokens on its own path, which is the context Algorithm 2's input
 * P(. | x_{<n}) refers to at that node).
 *
 * For query head h (kv head g = h / (Hq/Hkv)) and node i the key set is
 *   J = {0..L-1}  union  {L + a : a on the walk i -> root},
 * and out[i,h,:] = sum_j softmax_j(scale * q.k_j) v_j over j in J.
 * q,out: [n][Hq][d]; k,v: [Hkv][kv_rows][d]; lse: [Hq][n] (natural log), nullable.
 * No mask array is used: the path is gathered by walking parent[].
 */
int orc_tree_attention(const double* q, const double* k, const double* v,
                       const int32_t* parent, int32_t n, int32_t L, int32_t Hq,
                       int32_t Hkv, int32_t d, int32_t kv_rows, double scale,
                       double* out, double* lse) {
  int flags = 0;
  int32_t G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 4) reduction(| : flags)
  for (int32_t h = 0; h < Hq; ++h) {
    for (int32_t i = 0; i < n; ++i) {
      int32_t g = h / G;
      int32_t nkeys = 0;
      int32_t* J = (int32_t*)malloc(sizeof(int32_t) * (size_t)(L + n));
      double* s = (double*)malloc(sizeof(double) * (size_t)(L + n));
      for (int32_t j = 0; j < L; ++j) J[nkeys++] = j;
      for (int32_t a = i; a >= 0; a = clean_parent(parent, a, &flags)) J[nkeys++] = L + a;
      const double* qi = q + ((size_t)i * Hq + h) * d;
      double m = -INFINITY;
      for (int32_t t = 0; t < nkeys; ++t) {
        const double* kj = k + ((size_t)g * kv_rows + J[t]) * d;
        double acc = 0.0;
        for (int32_t c = 0; c < d; ++c) acc += qi[c] * kj[c];
        s[t] = scale * acc;
        if (s[t] > m) m = s[t];
      }
      double denom = 0.0;
      for (int32_t t = 0; t < nkeys; ++t) {
        s[t] = exp(s[t] - m);
        denom += s[t];
      }
      double* o = out + ((size_t)i * Hq + h) * d;
      for (int32_t c = 0; c < d; ++c) o[c] = 0.0;
      for (int32_t t = 0; t < nkeys; ++t) {
        const double* vj = v + ((size_t)g * kv_rows + J[t]) * d;
        double w = s[t] / denom;
        for (int32_t c = 0; c < d; ++c) o[c] += w * vj[c];
      }
      if (lse) lse[(size_t)h * n + i] = m + log(denom);
      free(J);
      free(s);
    }
  }
  return flags;
}

/* softmax(logits / T) in fp64, max-subtracted (Algorithm 2's inputs P and Q
 * are the models' distributions at temperature T, Table 1 column "T"). */
void orc_softmax_T(const float* logits, int32_t V, double T, double* out) {
  double m = -INFINITY;
  for (int32_t t = 0; t < V; ++t) {
    double x = (double)logits[t] / T;
    if (x > m) m = x;
  }
  double z = 0.0;
  for (int32_t t = 0; t < V; ++t) {
    out[t] = exp((double)logits[t] / T - m);
    z += out[t];
  }
  for (int32_t t = 0; t < V; ++t) out[t] /= z;
}

/*
 * Draft-side sampling without replacement by exponential sort (Section 5,
 * implementation details: the paper names the exponential-sort algorithm for
 * sampling without replacement; this is the draw s_i ~ D inside Algorithm 2's loop
 * for all k children of a node at once).
 *
 * Every token t gets an exponential variate E_t = -log(u_t) (u_t uniform on
 * (0,1), supplied by the caller) and the key E_t / q_t with q = softmax(logits/T).
 * The tokens in ascending key order are a sample without replacement from q in
 * draw order: the smallest key is a draw from q, the next one a draw from q
 * renormalised without the first, and so on.  The first k are returned.
 *
 *   logits [V], u [V] (anything outside (0,1) gives that token no chance).
 *   out [k]: the drawn tokens in draw order; -1 once no token with q_t > 0 is left.
 *   keys_out (nullable, [V]): the keys (INFINITY where q_t = 0 or u_t is unusable).
 *   min_rel_gap (nullable): over the k+1 smallest keys in order, the smallest
 *       relative difference (b - a) / b between neighbours: how much room a
 *       lower-precision computation of the keys has before the order changes.
 * Equal keys are taken in token order.  Returns 0.
 */
int orc_draft_sample(const float* logits, int32_t V, double T, const float* u, int32_t k,
                     int32_t* out, double* keys_out, double* min_rel_gap) {
  double* q = (double*)malloc(sizeof(double) * (size_t)V);
  double* key = (double*)malloc(sizeof(double) * (size_t)V);
  unsigned char* taken = (unsigned char*)calloc((size_t)V, 1);
  orc_softmax_T(logits, V, T, q);
  for (int32_t t = 0; t < V; ++t) {
    double ut = (double)u[t];
    if (q[t] > 0.0 && ut > 0.0 && ut < 1.0)
      key[t] = -log(ut) / q[t];
    else
      key[t] = INFINITY;
    if (keys_out) keys_out[t] = key[t];
  }
  if (min_rel_gap) *min_rel_gap = INFINITY;
  double prev = -1.0;
  for (int32_t i = 0; i <= k; ++i) { /* one more than k, for the gap behind the last draw */
    int32_t best = -1;
    for (int32_t t = 0; t < V; ++t)
      if (!taken[t] && key[t] < INFINITY && (best < 0 || key[t] < key[best])) best = t;
    if (i < k) out[i] = best;
    if (best < 0) {
      for (int32_t j = i + 1; j < k; ++j) out[j] = -1;
      break;
    }
    taken[best] = 1;
    if (min_rel_gap && prev >= 0.0 && key[best] > 0.0) {
      double g = (key[best] - prev) / key[best];
      if (g < *min_rel_gap) *min_rel_gap = g;
    }
    prev = key[best];
  }
  free(q);
  free(key);
  free(taken);
  return 0;
}

/*
 * Algorithm 2's loop for ONE node whose k children were already drawn (the
 * draws s_i ~ D are the caller's: child_tok[i] in draw order) and whose
 * uniforms r_i are supplied.  Per child, in the algorithm's order: the
 * acceptance test r_i < R[s_i]/D[s_i]; on rejection the residual update
 * R <- norm(max(R - D, 0)); then the draft update, which is what Sequoia adds
 * to multi-round rejection sampling: s_i leaves D and joins S, D falls back to
 * the uniform distribution over the tokens outside S once it has no mass left,
 * and D is renormalised.
 *
 *   R, D       in: P and Q (length V); out: the residual and draft after the
 *              last executed step, i.e. R is what the final draw x ~ R samples if
 *              no child was accepted.
 *   accepted   index i (0-based) of the accepted child, or -1.
 *   ratio/rnum/dden (nullable, length k): R[s_i]/D[s_i], R[s_i], D[s_i] as
 *              seen by the acceptance test (NaN where the test never ran).
 *   min_gap    (nullable) min over executed tests of |r_i - ratio_i|.
 * Returns flags.
 */
int orc_alg2_node(double* R, double* D, int32_t V, const int32_t* child_tok,
                  const double* child_u, int32_t k, int32_t variant,
                  int32_t* accepted, double* ratio_out, double* rnum_out,
                  double* dden_out, double* min_gap) {
  int flags = 0;
  *accepted = -1;
  unsigned char* S = (unsigned char*)calloc((size_t)V, 1); /* S = {} */
  double* Rn = (double*)malloc(sizeof(double) * (size_t)V);
  if (min_gap) *min_gap = INFINITY;
  for (int32_t i = 0; i < k; ++i) {
    if (ratio_out) ratio_out[i] = NAN;
    if (rnum_out) rnum_out[i] = NAN;
    if (dden_out) dden_out[i] = NAN;
  }
  int32_t n_rejected = 0;
  for (int32_t i = 0; i < k; ++i) { /* one iteration per speculated child */
    int32_t s = child_tok[i];
    if (s < 0 || s >= V) { /* not a token: cannot be accepted, touches nothing */
      flags |= ORC_BAD_TOKEN;
      continue;
    }
    double ratio; /* acceptance test: R[s]/D[s] */
    if (D[s] > 0.0)
      ratio = R[s] / D[s];
    else
      ratio = (R[s] > 0.0) ? INFINITY : 0.0;
    if (ratio_out) ratio_out[i] = ratio;
    if (rnum_out) rnum_out[i] = R[s];
    if (dden_out) dden_out[i] = D[s];
    if (min_gap) {
      double gap = fabs(child_u[i] - ratio);
      if (gap < *min_gap) *min_gap = gap;
    }
    if (child_u[i] < ratio) { /* strict comparison */
      *accepted = i;
      break;
    }
    /* residual update: R <- norm(max(R - D, 0)), with D as it stands (s not yet removed) */
    double Z = 0.0;
    for (int32_t t = 0; t < V; ++t) {
      double x = R[t] - D[t];
      Rn[t] = x > 0.0 ? x : 0.0;
      Z += Rn[t];
    }
    if (Z > 0.0) {
      for (int32_t t = 0; t < V; ++t) R[t] = Rn[t] / Z;
    } else {
      flags |= ORC_DEGENERATE; /* impossible in exact arithmetic; keep R */
    }
    if (variant == ORC_VARIANT_SEQUOIA) {
      D[s] = 0.0; /* draft update: s leaves D ... */
      if (!S[s]) { /* ... and joins S */
        S[s] = 1;
        ++n_rejected;
      }
      double sumD = 0.0; /* mass left in D */
      for (int32_t t = 0; t < V; ++t) sumD += D[t];
      if (sumD == 0.0) { /* none: uniform over the non-rejected set */
        for (int32_t t = 0; t < V; ++t) D[t] = S[t] ? 0.0 : 1.0;
        sumD = (double)(V - n_rejected);
      }
      if (sumD > 0.0) /* renormalise (nothing left to normalise once S is everything) */
        for (int32_t t = 0; t < V; ++t) D[t] /= sumD;
    }
  }
  free(S);
  free(Rn);
  return flags;
}

/* Algorithm 2's final draw, x ~ R, realised by inverse CDF in index order with one uniform:
 * the first t whose inclusive cumulative sum exceeds u; if rounding leaves the
 * total at or below u, the last t with R[t] > 0. */
int32_t orc_sample_inverse_cdf(const double* R, int32_t V, double u) {
  double c = 0.0;
  int32_t last_pos = -1;
  for (int32_t t = 0; t < V; ++t) {
    c += R[t];
    if (R[t] > 0.0) last_pos = t;
    if (c > u) return t;
  }
  return last_pos;
}

/*
 * The whole verification of one tree (Section 2.2: start at the root, apply
 * the per-node algorithm, recurse into the accepted child), Algorithm 2 at
 * every visited node, then the final draw x ~ R at the node where the walk stops.
 *
 *   parent, tokens        [n]; node 0 is the root (parent[0] = -1), tokens[0] unused.
 *   target_logits         row v = next-token logits after node v.
 *   draft_logits          row v = logits v's children were drawn from
 *                         (rows of leaves are never read).
 *   T                     temperature of both distributions; 0 = greedy.
 *   uniforms              [n+1]: entry c tests child node c, entry n draws the bonus.
 *   path/path_len/bonus   visited nodes (root first), their count, the token of the final draw.
 *   residual_out          nullable [V]: R at the final draw.
 *   next_child            nullable [n]: accepted child of each visited node,
 *                         -1 if none, -2 for nodes the walk never reached.
 *   ratio_out             nullable [n]: ratio tested for child node c (NaN if untested).
 *   min_gap               nullable: min |u - ratio| over executed tests.
 * Children of a node are taken in ascending node index (= draw order).
 */
int orc_tree_verify(int32_t n, int32_t V, const int32_t* parent, const int32_t* tokens,
                    const float* target_logits, int64_t target_row_stride,
                    const float* draft_logits, int64_t draft_row_stride, double T,
                    const float* uniforms, int32_t variant, int32_t* path,
                    int32_t* path_len, int32_t* bonus, double* residual_out,
                    int32_t* next_child, double* ratio_out, double* min_gap) {
  int flags = 0;
  double* R = (double*)malloc(sizeof(double) * (size_t)V);
  double* D = (double*)malloc(sizeof(double) * (size_t)V);
  int32_t* kids = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
  int32_t* ktok = (int32_t*)malloc(sizeof(int32_t) * (size_t)n);
  double* ku = (double*)malloc(sizeof(double) * (size_t)n);
  double* kr = (double*)malloc(sizeof(double) * (size_t)n);
  if (next_child)
    for (int32_t i = 0; i < n; ++i) next_child[i] = -2;
  if (ratio_out)
    for (int32_t i = 0; i < n; ++i) ratio_out[i] = NAN;
  if (min_gap) *min_gap = INFINITY;
  for (int32_t i = 1; i < n; ++i) (void)clean_parent(parent, i, &flags);

  int32_t cur = 0, plen = 0;
  path[plen++] = 0;
  for (;;) {
    const float* trow = target_logits + (size_t)cur * (size_t)target_row_stride;
    int32_t k = 0;
    for (int32_t c = cur + 1; c < n; ++c)
      if (parent[c] == cur) kids[k++] = c;
    for (int32_t t = 0; t < V; ++t)
      if (!isfinite(trow[t]) && !(trow[t] < 0 && isinf(trow[t]))) flags |= ORC_NONFINITE;
    int32_t acc = -1;
    if (T == 0.0) {
      /* greedy: P is the one-hot at the target arg-max (lowest index on ties);
       * a child is accepted iff its token is that arg-max. */
      int32_t a = 0;
      for (int32_t t = 1; t < V; ++t)
        if (trow[t] > trow[a]) a = t;
      for (int32_t t = 0; t < V; ++t) R[t] = 0.0;
      R[a] = 1.0;
      for (int32_t i = 0; i < k && acc < 0; ++i) {
        int32_t s = tokens[kids[i]];
        if (s < 0 || s >= V) {
          flags |= ORC_BAD_TOKEN;
          continue;
        }
        if (s == a) acc = i;
      }
    } else {
      orc_softmax_T(trow, V, T, R); /* R <- P */
      if (k > 0) {
        const float* drow = draft_logits + (size_t)cur * (size_t)draft_row_stride;
        orc_softmax_T(drow, V, T, D); /* D <- Q */
        for (int32_t i = 0; i < k; ++i) {
          ktok[i] = tokens[kids[i]];
          ku[i] = (double)uniforms[kids[i]];
        }
        double gap;
        flags |= orc_alg2_node(R, D, V, ktok, ku, k, variant, &acc, kr, NULL, NULL, &gap);
        if (min_gap && gap < *min_gap) *min_gap = gap;
        if (ratio_out)
          for (int32_t i = 0; i < k; ++i) ratio_out[kids[i]] = kr[i];
      }
    }
    if (next_child) next_child[cur] = acc >= 0 ? kids[acc] : -1;
    if (acc < 0) break;
    cur = kids[acc]; /* recurse into the accepted child with fresh R, D */
    path[plen++] = cur;
  }
  *path_len = plen;
  *bonus = orc_sample_inverse_cdf(R, V, (double)uniforms[n]); /* x ~ R */
  if (residual_out) memcpy(residual_out, R, sizeof(double) * (size_t)V);
  free(R);
  free(D);
  free(kids);
  free(ktok);
  free(ku);
  free(kr);
  return flags;
}

/*
 * Verification by sampling from the target (Section 2.2, the paragraph on
 * naive and top-k sampling: a token is sampled from the target distribution
 * at the node and accepted when one of the node's children carries it),
 * applied recursively from the root like Algorithm 2.
 *
 * At node v: x ~ softmax(target_logits[v] / T) by inverse CDF in index order
 * with uniforms[v]; if a child of v carries token x the walk moves to the
 * first such child (ascending node index), else it stops and x is the token
 * emitted there (bonus).  T = 0: x is the arg-max (lowest index on ties).
 * The draft model plays no part.  residual_out (nullable): the distribution
 * the last x was drawn from.  min_gap (nullable): the smallest distance of a
 * used uniform to the two ends of the CDF interval of its x.
 */
int orc_tree_verify_target_sample(int32_t n, int32_t V, const int32_t* parent, const int32_t* tokens,
                                  const float* target_logits, int64_t target_row_stride, double T,
                                  const float* uniforms, int32_t* path, int32_t* path_len,
                                  int32_t* bonus, double* residual_out, int32_t* next_child,
                                  double* min_gap) {
  int flags = 0;
  double* P = (double*)malloc(sizeof(double) * (size_t)V);
  if (next_child)
    for (int32_t i = 0; i < n; ++i) next_child[i] = -2;
  if (min_gap) *min_gap = INFINITY;
  for (int32_t i = 1; i < n; ++i) (void)clean_parent(parent, i, &flags);
  int32_t cur = 0, plen = 0;
  path[plen++] = 0;
  for (;;) {
    const float* trow = target_logits + (size_t)cur * (size_t)target_row_stride;
    for (int32_t t = 0; t < V; ++t)
      if (!isfinite(trow[t]) && !(trow[t] < 0 && isinf(trow[t]))) flags |= ORC_NONFINITE;
    int32_t x;
    if (T == 0.0) {
      x = 0;
      for (int32_t t = 1; t < V; ++t)
        if (trow[t] > trow[x]) x = t;
      for (int32_t t = 0; t < V; ++t) P[t] = 0.0;
      P[x] = 1.0;
    } else {
      orc_softmax_T(trow, V, T, P);
      double u = (double)uniforms[cur];
      x = orc_sample_inverse_cdf(P, V, u);
      if (min_gap) {
        double lo = 0.0;
        for (int32_t t = 0; t < x; ++t) lo += P[t];
        double g1 = fabs(u - lo), g2 = fabs(lo + P[x] - u);
        if (g1 < *min_gap) *min_gap = g1;
        if (g2 < *min_gap) *min_gap = g2;
      }
    }
    int32_t acc = -1;
    for (int32_t c = cur + 1; c < n && acc < 0; ++c)
      if (parent[c] == cur) {
        int32_t s = tokens[c];
        if (s < 0 || s >= V) {
          flags |= ORC_BAD_TOKEN;
          continue;
        }
        if (s == x) acc = c;
      }
    if (next_child) next_child[cur] = acc;
    if (acc < 0) {
      *bonus = x;
      if (residual_out) memcpy(residual_out, P, sizeof(double) * (size_t)V);
      break;
    }
    cur = acc;
    path[plen++] = cur;
  }
  *path_len = plen;
  free(P);
  return flags;
}

/*
 * Algorithm 3 (sequence-based speculative decoding) for one chain, with the
 * two misprints of the listing read as: the target distributions come from the
 * target model, and the final residual is taken iff fewer than gamma tokens
 * were accepted.  p,q: [gamma+1][V] and [gamma][V] distributions; x: the gamma
 * drafted tokens; r: gamma uniforms; u_final: uniform for the last draw.
 * Returns the number of accepted tokens; *t_out is the final token.
 */
int32_t orc_alg3_chain(const double* p, const double* q, int32_t V, int32_t gamma,
                       const int32_t* x, const double* r, double u_final,
                       int32_t* t_out) {
  int32_t s = 0;
  for (int32_t i = 0; i < gamma; ++i) {
    double pi = p[(size_t)i * V + x[i]], qi = q[(size_t)i * V + x[i]];
    double ratio = qi > 0.0 ? pi / qi : (pi > 0.0 ? INFINITY : 0.0);
    if (r[i] < ratio)
      ++s;
    else
      break;
  }
  double* pp = (double*)malloc(sizeof(double) * (size_t)V);
  memcpy(pp, p + (size_t)s * V, sizeof(double) * (size_t)V);
  if (s < gamma) {
    double Z = 0.0;
    for (int32_t t = 0; t < V; ++t) {
      double dlt = p[(size_t)s * V + t] - q[(size_t)s * V + t];
      pp[t] = dlt > 0.0 ? dlt : 0.0;
      Z += pp[t];
    }
    for (int32_t t = 0; t < V; ++t) pp[t] /= Z;
  }
  *t_out = orc_sample_inverse_cdf(pp, V, u_final);
  free(pp);
  return s;
}

/*
 * Commit of an accepted path into the key/value cache: what has to happen
 * between one verification and the next so that the accepted tokens become
 * part of the prefix (Section 2.1: the accepted tokens are kept and decoding
 * goes on from them; the cache itself is left to the implementation).  The
 * tree's rows sit at [L, L+n) of every plane (one plane = the keys or the
 * values of one head of one layer); afterwards row L+i holds what row
 * L+path[i] held, for i in [0, path_len), so that the new prefix is
 * L + path_len rows long.  Every other row is unchanged.  Written out of place
 * (in -> out, both [planes][rows][row_bytes] bytes) so that the definition has
 * no ordering in it.
 *
 * A path is valid iff 0 <= path_len <= n, path[0] == 0, it is strictly
 * ascending and stays below n (a parent always precedes its child); an invalid
 * path raises ORC_BAD_PATH and nothing moves (out == in).
 */
int32_t orc_kv_commit(const uint8_t* in, uint8_t* out, int64_t planes, int64_t rows,
                      int64_t row_bytes, int32_t L, int32_t n, const int32_t* path,
                      int32_t path_len) {
  memcpy(out, in, (size_t)(planes * rows * row_bytes));
  int ok = path_len >= 0 && path_len <= n;
  for (int32_t i = 0; ok && i < path_len; ++i) {
    if (i == 0 ? path[0] != 0 : path[i] <= path[i - 1]) ok = 0;
    if (path[i] < 0 || path[i] >= n) ok = 0;
  }
  if (!ok) return ORC_BAD_PATH;
  for (int64_t h = 0; h < planes; ++h)
    for (int32_t i = 0; i < path_len; ++i)
      memcpy(out + ((size_t)h * rows + (size_t)(L + i)) * row_bytes,
             in + ((size_t)h * rows + (size_t)(L + path[i])) * row_bytes, (size_t)row_bytes);
  return 0;
}

/*
 * Nucleus ("top-p") truncation of a distribution: the hyperparameter of the
 * robustness study (Section 4.2, table "robustness to the top-p
 * hyperparameter").  The paper names the hyperparameter only; the operation is
 * taken as the usual one: with p = softmax(logits / T), order the tokens by
 * decreasing probability (equal probabilities in token order) and keep the
 * shortest prefix of that order whose probabilities add up to at least top_p;
 * every other token gets probability 0 (logit -inf), and the survivors are
 * renormalised by whoever takes the softmax next.  top_p >= 1 keeps every
 * token.  At least one token is always kept.
 *
 *   keep [V]: 1 for tokens inside the nucleus, else 0.  Returns their number.
 *   margins (nullable, [2]): how close the decision was -- [0] = (cumulative
 *       mass up to and including the last kept token) - top_p, [1] = top_p -
 *       (the same without that token); both >= 0, +inf when top_p >= 1.  The
 *       ORDER of the tokens is that of the fp32 logits themselves and leaves
 *       no room for rounding; a lower-precision computation of the masses can
 *       move the cut by one token only when one of the two margins is small.
 * A NaN or +inf logit counts as -inf (never kept) and raises ORC_NONFINITE in
 * *flags (nullable).
 */
typedef struct {
  double p;
  int32_t t;
} orc_pt;

static int orc_pt_desc(const void* a, const void* b) {
  const orc_pt *x = (const orc_pt*)a, *y = (const orc_pt*)b;
  if (x->p > y->p) return -1;
  if (x->p < y->p) return 1;
  return x->t < y->t ? -1 : (x->t > y->t ? 1 : 0);
}

int32_t orc_top_p(const float* logits, int32_t V, double T, double top_p, uint8_t* keep,
                  double* margins, int32_t* flags) {
  float* clean = (float*)malloc(sizeof(float) * (size_t)V);
  double* p = (double*)malloc(sizeof(double) * (size_t)V);
  orc_pt* order = (orc_pt*)malloc(sizeof(orc_pt) * (size_t)V);
  int32_t fl = 0;
  for (int32_t t = 0; t < V; ++t) {
    clean[t] = logits[t];
    if (isnan(logits[t]) || (isinf(logits[t]) && logits[t] > 0)) {
      clean[t] = -INFINITY;
      fl |= ORC_NONFINITE;
    }
  }
  orc_softmax_T(clean, V, T, p);
  for (int32_t t = 0; t < V; ++t) {
    order[t].p = p[t];
    order[t].t = t;
    keep[t] = 0;
  }
  qsort(order, (size_t)V, sizeof(orc_pt), orc_pt_desc);
  int32_t kept = 0;
  double cum = 0.0, over = INFINITY, under = INFINITY;
  if (top_p >= 1.0) {
    for (int32_t t = 0; t < V; ++t) keep[t] = 1;
    kept = V;
  } else {
    for (int32_t i = 0; i < V; ++i) {
      double before = cum;
      cum += order[i].p;
      keep[order[i].t] = 1;
      ++kept;
      if (cum >= top_p) {
        over = cum - top_p;
        under = top_p - before;
        break;
      }
    }
  }
  if (margins) {
    margins[0] = over;
    margins[1] = under;
  }
  if (flags) *flags = fl;
  free(clean);
  free(p);
  free(order);
  return kept;
}
