/*
 * seq_tree.h -- C ABI of the B200 (sm_100a) token-tree verification library.
 *
 * The library computes the per-step numerics of Sequoia's tree-based
 * speculative decoding (Chen et al., arXiv 2402.12374):
 *   (a) the target model's attention over a speculated token tree, and
 *   (b) Algorithm 2 ("Sequoia Sampling and Verification") applied from the
 *       root down the tree, ending in the bonus token drawn from the residual.
 *
 * Conventions shared by every entry point
 *   - All data pointers are DEVICE pointers owned by the caller, valid on the
 *     device that is current when the call is made.  The library allocates
 *     no device memory and never synchronises the host.  Between calls it keeps
 *     only per-device facts that it looks up once (a driver entry point, the
 *     SM count, whether a 16-CTA cluster can be placed, function attributes
 *     already set, the address of the built-in scratch array) and the last 16
 *     tensor maps it has encoded, keyed by the arguments of the encode (pointer,
 *     extents, strides), so that a repeated launch makes no driver call; those
 *     lookups are guarded, so calls may come from several host threads.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Work is enqueued on it and the call returns at once.
 *   - Problems the host can see (null pointers, sizes out of range, bad
 *     alignment, workspace too small) return a negative seq_status and
 *     enqueue nothing.
 *   - Problems only the device can see (a parent that is not an earlier node,
 *     a token id outside the vocabulary, NaN/+inf logits) OR a bit into
 *     *dev_status (nullable), clamp the offending index, and still produce
 *     defined outputs.  Kernels never trap and never wait without a bound;
 *     a bounded wait that runs out sets SEQ_DEV_TIMEOUT.
 *     *dev_status is only ever OR-ed into: the caller zeroes it.
 *   - Trees: n nodes, node 0 is the root (the last committed token: in Section
 *     2.1 the root stands for the current prefix); parent[0] = -1
 *     and 0 <= parent[i] < i.  Siblings are ordered by node index, which is
 *     the order they were drawn in.  1 <= n <= SEQ_MAX_TREE.
 */
#ifndef SEQ_TREE_H_
#define SEQ_TREE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SEQ_MAX_TREE 1024

typedef enum {
  SEQ_OK = 0,
  SEQ_ERR_INVALID_ARG = -1, /* null pointer, size/stride/alignment out of range */
  SEQ_ERR_UNSUPPORTED = -2, /* valid request this build has no kernel for */
  SEQ_ERR_WORKSPACE = -3,   /* workspace_bytes below seq_*_workspace_bytes() */
  SEQ_ERR_CUDA = -4         /* a CUDA runtime/driver call failed */
} seq_status;

typedef enum { SEQ_F16 = 0, SEQ_BF16 = 1, SEQ_F32 = 2 } seq_dtype;

/* bits OR-ed into *dev_status by kernels; 0 = clean */
enum {
  SEQ_DEV_BAD_PARENT = 1,  /* parent[i] not in {-1} u [0,i): read as -1 */
  SEQ_DEV_BAD_TOKEN = 2,   /* token id outside [0,vocab): the child is rejected, R and D untouched */
  SEQ_DEV_NONFINITE = 4,   /* NaN or +inf logit on a visited row */
  SEQ_DEV_DEGENERATE = 8,  /* sum max(R-D,0) == 0 after a rejection (impossible in exact arithmetic): R kept */
  SEQ_DEV_TIMEOUT = 16,    /* a bounded on-chip wait ran out; outputs of that call are undefined */
  SEQ_DEV_BAD_PATH = 32,   /* seq_tree_kv_commit: path not a root-to-node path (see there); nothing was moved */
  SEQ_DEV_BAD_LENGTH = 64  /* *prefix_len_dev outside [0, prefix_len]: clamped into that range */
};

/*
 * seq_tree_mask_from_parents -- ancestor bitmasks of a token tree.
 *
 * Defines which tree tokens a tree token may attend to: itself and the nodes
 * on its path to the root (Section 2.2: the verification walks the tree from
 * its root; Algorithm 2's input P(.|x_<n) at a node is conditioned on exactly
 * that path).  Bit j of row i is set iff j is i or an ancestor of i.
 *
 *   parent        [n] int32, device.  parent[i] = -1 also allowed for i > 0
 *                 (a node with no ancestors).
 *   mask_bits     [n][words_per_row] uint32, device, written in full (unused
 *                 high bits cleared).  words_per_row >= ceil(n/32).
 *   depth         [n] int32, device, nullable: number of parent links from i
 *                 to its root (callers use prefix_len + depth as position id).
 *   dev_status    nullable.
 * Returns SEQ_OK or SEQ_ERR_INVALID_ARG.  Run once per tree: the tree's shape
 * is chosen ahead of time and kept for all decoding steps (Section 4.1).
 */
int seq_tree_mask_from_parents(const int32_t* parent, int32_t n, uint32_t* mask_bits,
                               int32_t words_per_row, int32_t* depth, int32_t* dev_status,
                               void* stream);

/*
 * seq_tree_attention -- attention of the n tree tokens in one target forward
 * pass (Section 1: the whole speculated tree is verified by a single forward
 * pass of the target model).
 *
 * For query head h (kv head h / (num_q_heads/num_kv_heads)) and node i:
 *     out[i,h,:] = sum_j softmax_j(softmax_scale * q[i,h,:].k[g,j,:]) * v[g,j,:]
 * over j in [0, prefix_len)  and  j = prefix_len + a for every a whose bit is
 * set in row i of mask_bits.  Scores, softmax and accumulation are fp32; with
 * 16-bit inputs the probabilities are rounded to the input type before the
 * P.V product on the tensor-core path.
 *
 * Layouts (strides in ELEMENTS, innermost head_dim contiguous):
 *   q, out        element (i,h,c) at i*stride_tok + h*stride_head + c
 *   k_cache,      element (g,j,c) at g*kv_stride_head + j*kv_stride_tok + c;
 *   v_cache       rows [0,prefix_len) hold the prefix, rows [prefix_len,
 *                 prefix_len+n_tree) the tree tokens in node order; rows
 *                 beyond that (up to kv_capacity) are never read into the
 *                 result and may hold anything, NaN included.  The rows below
 *                 prefix_len + n_tree must be finite: a masked key's
 *                 probability is exactly 0, but on the tensor-core path its V
 *                 row still enters the product, and 0 * inf is NaN for every
 *                 row of that 128-row tile.
 *   lse           nullable, [num_q_heads][n_tree] fp32: natural-log
 *                 sum-exp of the scaled scores of each row.
 * head_dim must be 128.  Base pointers and strides must keep every row
 * 16-byte aligned.  dtype selects f16/bf16/f32 for q, k, v and out alike.
 * Mask from the parent array: with mask_bits == NULL and parent != NULL the
 * tensor-core kernel derives each query tile's ancestor rows from parent[]
 * itself (the walk of seq_tree_mask_from_parents, done in shared memory while
 * the first tiles are in flight), so a decoding step needs no separate mask
 * launch; a parent[i] outside {-1} u [0,i) raises SEQ_DEV_BAD_PARENT and is
 * read as -1, as there.  The results are those of a call with the mask_bits of
 * seq_tree_mask_from_parents(parent).  The CUDA-core kernel has no such mode:
 * a request that needs it (fp32, a group size that does not divide 128,
 * kernel == 1) without mask_bits returns SEQ_ERR_UNSUPPORTED.  When mask_bits
 * is given, parent is ignored.
 * workspace: at least seq_tree_attention_workspace_bytes(p) bytes, 256-byte
 * aligned, device; contents undefined before and after.  The size depends on
 * the shape and on p->kernel and may be 0 (workspace may then be NULL): the
 * CUDA-core kernel keeps the partial results of its key-range splits there,
 * the tensor-core kernel the pieces of the query tiles that its CTAs share
 * when there are more (tile, kv head) units than SMs (about 19 MB then).  A
 * call with a workspace that is too small returns SEQ_ERR_WORKSPACE and
 * launches nothing.  Two calls that run concurrently need a workspace each.
 * The results do not depend on the order in which CTAs finish: a call
 * repeated on the same inputs returns the same bits.
 */
typedef struct {
  int32_t n_tree, prefix_len, num_q_heads, num_kv_heads, head_dim;
  int32_t dtype;       /* seq_dtype */
  float softmax_scale; /* <= 0 selects 1/sqrt(head_dim) */
  const void* q;
  int64_t q_stride_tok, q_stride_head;
  const void* k_cache;
  const void* v_cache;
  int64_t kv_stride_tok, kv_stride_head;
  int32_t kv_capacity; /* rows per kv head; >= prefix_len + n_tree */
  const uint32_t* mask_bits;
  int32_t mask_words_per_row;
  void* out;
  int64_t o_stride_tok, o_stride_head;
  float* lse;
  void* workspace;
  size_t workspace_bytes;
  int32_t* dev_status;
  int32_t kernel; /* 0 = choose; 1 = force the CUDA-core kernel; 2 = force the tensor-core kernel; 3, 4 = the tensor-core
                     kernel with its stream / grid schedule forced (tuning and tests; results do not depend on it) */
  const int32_t* parent; /* nullable, [n_tree] int32, device: see "mask from the parent array" above */
  /* nullable, device: the prefix length as the previous step's seq_tree_kv_commit left it.  When given, the kernels
   * read the length from there and prefix_len is only the LARGEST value it can take (it sizes the launch, the
   * workspace and the checks against kv_capacity); the tree's rows then sit at [*prefix_len_dev, *prefix_len_dev +
   * n_tree).  This is what lets one CUDA graph of a whole step (attention, verification, commit) be replayed while
   * the prefix grows (Section 4.1: the tree is fixed so that CUDA graphs can remove the launch overhead).  On the
   * tensor-core path the rows from *prefix_len_dev + n_tree up to kv_capacity are then fetched (not used): they may
   * hold anything, but must be readable.  A value outside [0, prefix_len] raises SEQ_DEV_BAD_LENGTH and is clamped. */
  const int32_t* prefix_len_dev;
  /* 0 or 1: *prefix_len_dev is the length of every head's prefix.  R > 1: a batch of R requests stacked as heads
   * (request r owns kv heads [r * num_kv_heads / R, (r + 1) * num_kv_heads / R) and their query heads; the tree is
   * common, Section 4.1: it is fixed in advance) with one prefix length each, prefix_len_dev[r]; request r's tree
   * rows sit at [prefix_len_dev[r], prefix_len_dev[r] + n_tree) of ITS heads' caches.  R must divide num_kv_heads
   * and prefix_len_dev must be given; the tensor-core kernel then runs its grid schedule (kernel = 3 is refused). */
  int32_t prefix_len_dev_count;
} seq_tree_attention_params;

size_t seq_tree_attention_workspace_bytes(const seq_tree_attention_params* p);
int seq_tree_attention(const seq_tree_attention_params* p, void* stream);

/*
 * seq_tree_attention_noalloc -- the CUDA-core variant of seq_tree_attention for callers that
 * cannot provide scratch memory.  (The paper has no counterpart: this is a deployment convenience.)
 *
 * Who needs it: a serving process whose device memory is handed out once at start-up and frozen
 * afterwards (no allocator is reachable from the decoding loop, or an allocation there would
 * synchronise the device and stall every other stream), and small embedders that link this library
 * without any tensor framework and so have nothing to size or own a workspace with.
 *
 * Same arguments, semantics and results as seq_tree_attention run with kernel = 1 (the CUDA-core
 * kernel, any dtype); p->workspace, p->workspace_bytes and p->kernel are ignored.  The split-KV
 * partial results go to a fixed array of SEQ_NOALLOC_SCRATCH_BYTES that lives inside the library
 * image on every device that loads it, until the process exits.  The call allocates nothing: no
 * cudaMalloc/cudaFree and no allocating library routine.
 *
 *   - A request whose partials need more than SEQ_NOALLOC_SCRATCH_BYTES returns SEQ_ERR_WORKSPACE
 *     and launches nothing (use seq_tree_attention with your own workspace instead).
 *   - The first call on a device looks up the array's device address (one cheap runtime query with
 *     that device current) and remembers it; make that first call during start-up, before any
 *     stream capture is begun on that device.
 *   - All calls share the one array, and it keeps whatever the previous call left there.  Nothing
 *     in it has to start at zero: every partial a call reads was written by that same call.  Two
 *     calls that overlap on the GPU (different streams) race on it; serialise them.
 */
#define SEQ_NOALLOC_SCRATCH_BYTES (384u << 10)
int seq_tree_attention_noalloc(const seq_tree_attention_params* p, void* stream);

/*
 * seq_tree_verify -- Algorithm 2 applied recursively from the root (Section
 * 2.2), then its last line x ~ R at the node where the walk stops.
 *
 * At the current node v with children c_1 < c_2 < ... (node order):
 *   R <- softmax(target_logits[v]/T), D <- softmax(draft_logits[v]/T), S <- {}
 *   for each child c, s = tokens[c]:
 *     accept c  iff  uniforms[c] < R[s]/D[s]          (strict; D[s]=0: +inf if R[s]>0 else 0)
 *     otherwise R <- norm(max(R-D,0)); D[s] <- 0; S <- S u {s};
 *               if sum(D) = 0: D <- uniform over tokens not in S;  D <- norm(D)
 *   an accepted child becomes the current node with fresh R, D, S; when no
 *   child is accepted (or v is a leaf) the bonus token is the first t with
 *   R[0]+..+R[t] > uniforms[n] (the last t with R[t] > 0 if rounding leaves
 *   none).
 * T = 0 is greedy: R is the one-hot at the target arg-max (lowest index on
 * ties), a child is accepted iff its token is that arg-max, draft logits and
 * uniforms are not read.
 *
 *   parent, tokens      [n] int32; tokens[0] is ignored.  A single root.
 *   target_logits       fp32 (bfloat16 with SEQ_VERIFY_LOGITS_BF16), row v at v*target_row_stride: next-token
 *                       logits after node v.
 *   draft_logits        same type, row v at v*draft_row_stride: the logits whose softmax at T
 *                       v's children were drawn from without replacement; rows of leaves
 *                       are never read.  -inf entries are legal (probability 0).
 *   temperature         >= 0, finite; one value for both models.
 *   uniforms            [n+1] fp32 in [0,1): entry c decides child node c, entry n the bonus.
 *   path                [n] int32 out: visited nodes, root first; path_len out: their count
 *                       (accepted tokens are tokens[path[1..path_len-1]]; the step emits
 *                       path_len tokens counting the bonus).
 *   bonus_token         out.
 *   residual_out        nullable [vocab] fp32: the R the bonus token was drawn from.
 *   next_child_out      nullable [n] int32: accepted child of each visited node, -1 if none,
 *                       -2 for nodes the walk did not visit.  With SEQ_VERIFY_ALL_NODES
 *                       every node is processed and gets its own decision.
 * workspace: seq_tree_verify_workspace_bytes(p) bytes, 16-byte aligned, device, contents undefined before the call
 * (the call clears what it needs); afterwards its first int32 holds the number of logit rows the call read (a
 * diagnostic: the walk's own rows are the algorithmic minimum).  Only the node-parallel schedule uses it.
 */
enum {
  SEQ_VERIFY_ALL_NODES = 1,
  /* Algorithm 2 without its draft update (the steps the paper highlights as Sequoia's addition): the draft distribution D
   * is left as it is after a rejection -- the rejected token is neither removed from it nor is it
   * renormalised -- which is SpecInfer's multi-round rejection sampling, the baseline the paper compares
   * its verification with (Section 3.2.2, Algorithm 2's caption; Theorem 3.7's counter-example).  The
   * children of a node are then draws WITH replacement from the draft row and may repeat. */
  SEQ_VERIFY_SPECINFER = 2,
  /* Verification by sampling from the target (Section 2.2, "Naive sampling and top-k sampling"): at every
   * visited node v a token x ~ softmax(target_logits[v] / T) is drawn by inverse CDF in index order with
   * uniforms[v] (entry 0 serves the root); the walk moves to the first child of v that carries x, else it
   * stops and x is bonus_token.  draft_logits is not read and may be NULL; residual_out receives the
   * distribution the last x was drawn from.  At T = 0 this is the arg-max matching of the default mode.
   * Not to be combined with SEQ_VERIFY_SPECINFER. */
  SEQ_VERIFY_TARGET_SAMPLE = 4,
  /* Schedule of a single request (results are those of Algorithm 2 either way; vocabulary-wide sums are taken in
   * another order, so a decision inside the 1e-5 band of its uniform can differ between the two):
   *   walk (the default) -- one cluster of CTAs follows the path from the root and reads only the visited nodes' rows
   *     (plus the rows of children that were tested and rejected, loaded ahead of their test); no workspace.
   *   node-parallel -- one cluster per tree node, first the nodes 0 .. clusters-1, then whatever is unclaimed at and
   *     below the deepest node known to be on the path; the path is assembled from the nodes' decisions by atomics,
   *     nobody waits.  It reads the rows of nodes the walk never visits (speculative work) and needs
   *     seq_tree_verify_workspace_bytes() of workspace; vocabulary up to 131072, not with SEQ_VERIFY_ALL_NODES.
   *     Data problems are reported for visited nodes only.  Measured slower than the walk on all five shapes of the
   *     paper's models; kept selectable.
   * SCHED_NODES without enough workspace returns SEQ_ERR_WORKSPACE, where it does not apply SEQ_ERR_UNSUPPORTED. */
  SEQ_VERIFY_SCHED_WALK = 16,
  SEQ_VERIFY_SCHED_NODES = 32,
  /* target_logits and draft_logits hold bfloat16 instead of fp32 (what a 16-bit language-model head writes; half the
   * bytes per visited node).  Every value is widened to fp32 exactly and the arithmetic is unchanged.  Row strides
   * stay in elements (multiples of 4), rows 8-byte aligned.  One request at T > 0 in the default mode or with
   * SEQ_VERIFY_SPECINFER, on the walk schedule; anything else returns SEQ_ERR_UNSUPPORTED. */
  SEQ_VERIFY_LOGITS_BF16 = 8
};

typedef struct {
  int32_t n_tree, vocab;
  const int32_t* parent;
  const int32_t* tokens;
  const float* target_logits;
  int64_t target_row_stride;
  const float* draft_logits;
  int64_t draft_row_stride;
  float temperature;
  const float* uniforms;
  int32_t* path;
  int32_t* path_len;
  int32_t* bonus_token;
  float* residual_out;
  int32_t* next_child_out;
  void* workspace;
  size_t workspace_bytes;
  int32_t* dev_status;
  int32_t flags; /* 0 or an OR of the SEQ_VERIFY_* values above */
} seq_tree_verify_params;

size_t seq_tree_verify_workspace_bytes(const seq_tree_verify_params* p);
int seq_tree_verify(const seq_tree_verify_params* p, void* stream);

/* seq_tree_verify_batch -- `batch` independent requests in one launch, one cluster of CTAs per request: clusters of 16
 * with the request's rows in registers while the batch fits the device side by side (9 requests on 148 SMs; the
 * modes that seq_tree_verify serves that way), else clusters of 8 with the rows in shared memory (18 clusters run at a
 * time).  Every request is verified as seq_tree_verify would verify it (the same
 * algorithm; seq_tree_verify may spread one request over a larger cluster, so vocabulary-wide sums can round
 * differently and a decision inside the 1e-5 band can differ): same sizes, temperature and flags for all
 * (SEQ_VERIFY_ALL_NODES is not allowed), each with its own tree, tokens, logits and uniforms.  request0 describes request 0; request r's arrays start r strides further:
 *   tree_stride      elements between the requests' parent / tokens / path / next_child_out arrays (>= n_tree);
 *   logits_stride    elements between their target matrices, and between their draft matrices (a multiple of 4,
 *                    large enough for n_tree rows);
 *   uniforms_stride  >= n_tree + 1;   residual_stride  >= vocab (unused when residual_out is NULL).
 * path_len and bonus_token are arrays of `batch` entries; dev_status is one word for all requests.  Returns what
 * seq_tree_verify returns; SEQ_ERR_INVALID_ARG also for a stride that is too small. */
typedef struct {
  seq_tree_verify_params request0;
  int32_t batch;
  int64_t tree_stride, logits_stride, uniforms_stride, residual_stride;
} seq_tree_verify_batch_params;

int seq_tree_verify_batch(const seq_tree_verify_batch_params* p, void* stream);

/*
 * seq_tree_draft_sample -- the draft side's draw of the children of tree nodes: k tokens without
 * replacement from softmax(draft_logits / temperature), for n_rows nodes at once (the draw s_i ~ D inside
 * Algorithm 2's loop, for all children of a node; Section 5, implementation details: the exponential-sort
 * algorithm is the paper's choice for sampling without replacement).  A step before the verify path: its output is the tokens[]
 * of seq_tree_verify's children, in sibling order.
 *
 * Token t of a row gets the key E_t / q_t with E_t = -log(u_t) an exponential variate and q the row's
 * softmax; the tokens in ascending key order are a sample without replacement in draw order, and the
 * first k are returned.  Equal keys are taken in token order.
 *
 *   draft_logits   fp32, row r at r*logits_row_stride (elements), device.  -inf entries are legal
 *                  (probability 0); a NaN or +inf entry raises SEQ_DEV_NONFINITE and is never drawn.
 *   uniforms       fp32 [n_rows][vocab], row r at r*uniforms_row_stride, device: one uniform per (row,
 *                  token); a value outside (0,1) gives its token no chance.  Caller-supplied, so that a
 *                  draw can be repeated and checked.
 *   temperature    > 0, finite.
 *   k              1..64 draws per row.
 *   tokens_out     int32 [n_rows][k], device: the drawn tokens in draw order, -1 where no token with
 *                  positive probability was left.
 *   dev_status     nullable.
 *   workspace      seq_tree_draft_sample_workspace_bytes(p) bytes, 8-byte aligned, device, contents
 *                  undefined before and after: the k best (score, token) pairs of every 4096-token chunk
 *                  of every row (two launches: per-chunk draws, then the row's draws among them).
 * The decision is taken in fp32 (on the logarithm of the inverse key): two keys closer than fp32 resolves
 * may come out in either order.  Returns SEQ_OK, SEQ_ERR_INVALID_ARG, SEQ_ERR_WORKSPACE, or
 * SEQ_ERR_UNSUPPORTED (vocab/4096 * k above 25600).
 */
typedef struct {
  int32_t n_rows, vocab, k;
  const float* draft_logits;
  int64_t logits_row_stride;
  const float* uniforms;
  int64_t uniforms_row_stride;
  float temperature;
  int32_t* tokens_out;
  int32_t* dev_status;
  void* workspace;
  size_t workspace_bytes;
} seq_tree_draft_sample_params;

size_t seq_tree_draft_sample_workspace_bytes(const seq_tree_draft_sample_params* p);
int seq_tree_draft_sample(const seq_tree_draft_sample_params* p, void* stream);

/* ---------------------------------------------------------------------------
 * seq_tree_kv_commit -- makes the accepted path part of the prefix (Section 2.1: the accepted tokens are kept
 * and decoding goes on after them; the key/value cache that makes this possible is the implementation's).
 *
 * The tree's keys and values sit at rows [prefix_len, prefix_len + n_tree) of every plane (one plane = one
 * head of one layer, for the keys or for the values).  After the call, in every plane, row prefix_len + i holds
 * what row prefix_len + path[i] held before it, for i in [0, *path_len); every other row is unchanged.  The
 * next step's prefix is therefore prefix_len + *path_len rows, which is written to *new_prefix_len.  The move
 * is in place and needs no workspace (each thread owns 16 bytes of a plane's rows, takes the rows in ascending
 * order and reads a batch before it writes it; path[j] > path[i] >= i for j > i, so no row is overwritten
 * before its last reader has it).
 *
 *   k_cache, v_cache   device, [num_planes] planes of rows of row_bytes bytes; plane_stride_bytes and
 *                      row_stride_bytes are multiples of 16, the base pointers 16-byte aligned, row_bytes a
 *                      multiple of 16 (<= row_stride_bytes).  v_cache may be NULL (keys only).  The two
 *                      buffers must not overlap.
 *   path, path_len     device, as seq_tree_verify wrote them (path has room for n_tree entries, all of them
 *                      readable): path[0] = 0, strictly ascending, below n_tree, 0 <= *path_len <= n_tree.
 *                      Anything else raises SEQ_DEV_BAD_PATH, moves nothing and
 *                      leaves *new_prefix_len = prefix_len.
 *   new_prefix_len     device, nullable.
 *
 * The caller keeps ownership of everything.  Asynchronous on `stream`; capturable in a CUDA graph.  Returns
 * SEQ_OK, SEQ_ERR_INVALID_ARG (null pointer, size or alignment out of range) or SEQ_ERR_CUDA. */
typedef struct {
  int32_t num_planes;
  int32_t row_bytes;
  int32_t prefix_len, n_tree;
  void* k_cache;
  void* v_cache;
  int64_t plane_stride_bytes, row_stride_bytes;
  const int32_t* path;
  const int32_t* path_len;
  int32_t* new_prefix_len;
  int32_t* dev_status;
  /* nullable, device: the prefix length is read from here and prefix_len is its upper bound (see
   * seq_tree_attention_params).  Must not be the same word as new_prefix_len: CTAs read the one while another
   * writes the other; copy new_prefix_len over it after the call (a 4-byte device copy, capturable). */
  const int32_t* prefix_len_dev;
} seq_tree_kv_commit_params;

int seq_tree_kv_commit(const seq_tree_kv_commit_params* p, void* stream);

/* ---------------------------------------------------------------------------
 * seq_tree_build -- Sequoia's tree construction (Section 3.1: score function, F(tree) = sum of the nodes' scores,
 * Algorithm 1; appendix "Dynamic programming details": the bound on the depth and one acceptance vector per
 * depth).  HOST function, all pointers are host memory; it launches nothing.  Run once, offline: the tree is
 * then fixed for the whole run.
 *
 * Finds a tree with at most max_size nodes, depth (in edges) <= max_depth and at most max_branch children per
 * node that maximises the expected number of generated tokens F under positional acceptance:
 *   acc_rates   [acc_rows][max_branch] doubles in [0, 1]; entry [r][b-1] = probability that the b-th child of a
 *               node at depth r is accepted, given that the node was reached and its earlier children were
 *               rejected.  acc_rows == 1: the same vector at every depth; else acc_rows >= max_depth.
 *   parent_out  [max_size] int32: the tree in level order (parent[0] = -1, parent[i] < i, siblings contiguous
 *               and in rank order), the numbering every other call of this library expects.
 *   size_out    number of nodes of the tree (max_size unless the bounds admit fewer).
 *   expected_out nullable: F of the returned tree.  Several trees can attain it; only F is unique.
 *   table_out   nullable, [(max_size+1)][(max_depth+1)] doubles: entry [n][d] = G(n, d), the largest F over trees
 *               of exactly n nodes and depth <= d; -inf where no such tree exists (and in row 0).  With
 *               acc_rows > 1 column d < max_depth holds the value of the best subtree hanging at depth
 *               max_depth - d instead (only the last column is a whole tree's value).
 * Cost: O(max_size^2 * max_depth * max_branch) time.  Returns SEQ_OK, SEQ_ERR_INVALID_ARG (null pointer, size
 * out of range, max_size above SEQ_MAX_TREE, a rate outside [0, 1] or NaN) or SEQ_ERR_UNSUPPORTED (tables above
 * 10^8 entries). */
typedef struct {
  int32_t max_size, max_depth, max_branch, acc_rows;
  const double* acc_rates;
  int32_t* parent_out;
  int32_t* size_out;
  double* expected_out;
  double* table_out;
} seq_tree_build_params;

int seq_tree_build(const seq_tree_build_params* p);

/* seq_tree_speedup_search -- the hardware-aware choice of the tree's size and depth (Section 4.1): maximises
 * Speedup(n, d) = G(n, d) / (t(n) + d * c) over 1 <= n <= max_size, 0 <= d <= max_depth.  HOST function.
 *   table    [(max_size+1)][(max_depth+1)] as seq_tree_build writes it (-inf entries are skipped);
 *   t_of_n   [max_size+1]: time for the target model to verify n tokens / time to verify one (entry 0 unused),
 *            all > 0, measured by the caller on its hardware;  c: time to draft one token / time to verify one.
 * Ties go to the smaller n, then the smaller d.  speedup_out is nullable.  Returns SEQ_OK or
 * SEQ_ERR_INVALID_ARG. */
int seq_tree_speedup_search(const double* table, int32_t max_size, int32_t max_depth, const double* t_of_n, double c,
                            int32_t* n_out, int32_t* d_out, double* speedup_out);

/* ---------------------------------------------------------------------------
 * seq_tree_top_p_filter -- nucleus ("top-p") truncation of softmax(logits / T), row by row: the top-p
 * hyperparameter of the robustness study (Section 4.2, table "robustness to the top-p hyperparameter"; the paper
 * names the hyperparameter only, the operation is the usual one).  Per row, with p = softmax(logits / T): order
 * the tokens by decreasing p (equal logits in token order) and keep the shortest prefix whose probabilities add
 * up to at least top_p; out[t] = logits[t] for kept tokens (the same bits), -inf for the others, so that a later
 * softmax renormalises over the nucleus.  Apply it to the target rows before seq_tree_verify (the output law is
 * then the truncated target distribution, whatever the draft) and/or to draft rows before seq_tree_draft_sample.
 *
 *   logits, out   device fp32 [n_rows][vocab], rows 16-byte aligned (strides in elements, multiples of 4, >= vocab);
 *                 out may be the same buffer as logits (in place), else the two must not overlap.
 *   temperature   > 0, finite;  top_p > 0 (top_p >= 1: every token is kept, rows are copied unchanged).
 *   kept_out      device, nullable, [n_rows]: the nucleus size of each row.
 * At least one token is kept.  A NaN or +inf logit raises SEQ_DEV_NONFINITE, counts as -inf and comes out as
 * -inf; a row of -inf only raises SEQ_DEV_DEGENERATE and stays -inf (kept 0).  The decision is taken on exact
 * fixed-point sums of fp32 exponentials: it can differ from an exact computation only where the cumulative mass
 * passes top_p within about 1e-6.  Deterministic.  No workspace.  Asynchronous on `stream`; capturable.  Returns
 * SEQ_OK, SEQ_ERR_INVALID_ARG or SEQ_ERR_CUDA. */
typedef struct {
  int32_t n_rows, vocab;
  const float* logits;
  int64_t logits_row_stride;
  float* out;
  int64_t out_row_stride;
  float temperature, top_p;
  int32_t* kept_out;
  int32_t* dev_status;
} seq_tree_top_p_params;

int seq_tree_top_p_filter(const seq_tree_top_p_params* p, void* stream);

/* ---------------------------------------------------------------------------
 * Measurement aids (the paper has no counterpart; Section 4.1 only says that decoding is bound by memory traffic
 * and by launch overhead, which is what these two numbers quantify on the device at hand).  bench.py prints both
 * beside its results.
 *
 * seq_tree_probe_stream_read -- a kernel that only READS `bytes` bytes (16-byte aligned, device) once, eight
 * 16-byte loads in flight per thread, 4 CTAs of 512 threads per SM; one word per CTA is written to sink
 * (device, sink_words >= 4 * the device's SM count, else SEQ_ERR_WORKSPACE).  bytes / its duration is the read
 * bandwidth a key/value stream can hope for.
 * seq_tree_probe_dependent_load -- one warp that loads *src and stores *src + 1 to *dst: the floor of a launch
 * with one dependent trip to memory.
 * Both are asynchronous on `stream`, allocate nothing, and return SEQ_OK, SEQ_ERR_INVALID_ARG, SEQ_ERR_WORKSPACE
 * or SEQ_ERR_CUDA. */
int seq_tree_probe_stream_read(const void* src, size_t bytes, unsigned long long* sink, size_t sink_words, void* stream);
int seq_tree_probe_dependent_load(const int32_t* src, int32_t* dst, void* stream);

/* Library build string ("seqtree <version> sm_100a"); static storage. */
const char* seq_tree_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SEQ_TREE_H_ */
