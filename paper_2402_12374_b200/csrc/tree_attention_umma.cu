// Tree-masked attention on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor
// memory, K/V/Q tiles staged by TMA), for 16-bit inputs.
//
// Work unit: (kv head g, tile of 128 query rows, range of the tile's keys).  A query row is
// a (node, head-in-group) pair, r = i_local * G + hg, so under GQA the G heads that share a kv head
// share every K/V tile.  Per block of 64 keys:
//     S = Q K^T      128x64x128   tcgen05.mma, Q and K K-major in 128-byte-swizzled shared memory
//     P = 2^(scale*S - m) masked  one thread per row: S read from tensor memory, P written back over
//                                 it as packed 16-bit values
//     O += P V       128x128x64   tcgen05.mma, A = P from tensor memory, V MN-major in shared memory
//
// Two chains per CTA, each double-buffered.  Keys are taken in blocks of 64; even blocks of the CTA's
// key range belong to chain A, odd blocks to chain B.  Each chain has two S/P buffers (64 columns
// each) and its own accumulator O in tensor memory (2 x (2*64 + 128) = 512 columns), two K and two V
// stages in shared memory, its own 128 row threads (one warp group), its own MMA-issuing warp and its
// own running (m, l); the chains share Q and the two TMA warps (one for Q and K, one for V: a K stage
// is free once its S is computed, a V stage only after the block's softmax, and K loads must not queue
// behind that).  S of a chain's next block is computed while its row threads still work on the current
// one, so a chain runs at the speed of its softmax, and while one chain exponentiates the tensor pipe
// also works for the other.  Per block a row thread first takes the block maximum (comparisons only),
// settles the reference maximum - it only moves when the block maximum exceeds it by more than 2^8, the
// accumulator row is then rescaled in tensor memory - and then takes the 64 exponentials, which are
// the bottleneck (16 per clock and SM).  Registers are rebalanced with setmaxnreg: 40 for the TMA/MMA
// warp group, 232 for the rows.
//
// Work distribution.  Grid mode: one CTA per (tile, kv head), in as many waves as that takes, or (up to one wave) a
// cluster of 2 to 8 CTAs that split its key range; the thread that arms the barriers requests the Q tile and the
// first K tiles itself, before the CTA-wide barrier.  Stream mode (many units of long tiles): one CTA per SM; the
// 64-key blocks of all units are laid end to end (each tile preceded by a few positions that stand for
// its fixed cost, tiles of a head taken alternately from both ends) and cut into equal ranges.  A CTA
// works through the segments of its range with barrier phases that run on from segment to segment, so
// the next segment's loads and first S are under way while the rows still merge and store.  A tile cut
// by a range boundary is completed by whichever of its CTAs finishes last: the others leave their
// piece (m, l, unnormalised accumulator) in the workspace and count themselves on the tile's counter;
// the pieces are added in CTA order, so the result does not depend on who finishes last.
//
// Merge.  The CTAs that share (tile, kv head) form a thread-block cluster along the key
// range (cs = 1 .. 8); its 2*cs chains share the 16 slices of 8 output columns round-robin.  Every chain pushes,
// for every row, each 8-column piece of its unnormalised fp32 accumulator into the shared memory of
// the chain that owns that slice (the K/V stages, dead by then) and its (m, l) into every CTA, with
// plain remote stores over distributed shared memory; after one cluster barrier each owner reduces
// its slices from local shared memory and writes the final output.  No workspace, no second kernel.
//
// Masking: key j < prefix_len is visible; key prefix_len + t is visible iff bit t of the row's
// ancestor mask; masked scores become -inf before the maximum, so their probability is exactly 0.
// Rows of K/V past prefix_len + n_tree are never fetched: the tensor maps end there and TMA fills
// the rest of a tile with zeros.
//
// Every mbarrier wait is bounded; a wait that runs out raises SEQ_DEV_TIMEOUT and the CTA drains.
//
// The kernel is launched with programmatic stream serialisation: its set-up runs under the previous kernel's tail,
// griddepcontrol.wait precedes its first access to global memory.
#include <cooperative_groups.h>
#include <cstddef>
#include <cuda.h>
#include <stdlib.h>
#include <string.h>

#include "common.cuh"
#include "trace_attention.cuh"

namespace cg = cooperative_groups;

namespace seqtree {

constexpr int kTileM = 128;         // query rows per CTA
constexpr int kBlockN = 64;         // keys per block
constexpr int kUmmaThreads = 384;   // warp group 0: TMA warp, MMA warp, two spare; warp groups 1, 2: rows of chains A, B
constexpr int kRegsLight = 40, kRegsRows = 232;  // after setmaxnreg: 128*40 + 256*232 = 384*168
constexpr int kMaxClusterSplit = 8;
constexpr int kMaxStreamTiles = 128;  // tiles per kv head the stream mode can index
// Stream mode balances cost, not block counts: every tile is laid out with this many extra positions in
// front of its blocks, standing for what starting and finishing a tile costs (about 4 us, in 64-key blocks).
constexpr int kStreamTileCost = 8;

constexpr uint32_t kTileBytes = 128 * 128 * 2;   // the Q tile: 128 rows x 128 elements of 16 bits
constexpr uint32_t kHalfBytes = kTileBytes / 2;  // one 128-row x 64-element sub-tile of Q (128 B rows)
constexpr uint32_t kKvBytes = kBlockN * 128 * 2; // a K or V tile: 64 keys x 128 elements
constexpr uint32_t kKvHalf = kKvBytes / 2;       // one 64-row x 64-element sub-tile of K or V
constexpr float kRescaleThreshold = 8.f;         // log2 units
constexpr float kRescaleLimit = 256.f;           // 2^kRescaleThreshold: no term of a row sum at or below it came from a score above the threshold
constexpr uint32_t kSpinLimit = 1u << 22;

struct UmmaSmem {
  // all tiles 1024-byte aligned (128-byte swizzle atoms are 8 rows x 128 B)
  uint8_t q[kTileBytes];
  uint8_t k[2][2][kKvBytes];  // [chain][stage]; after the last block these 64 KB receive the cluster merge
  uint8_t v[2][2][kKvBytes];  // [chain][stage]
  float2 ml_chain[2][2][kTileM];             // [segment parity][chain]: (m, l) of every row of the two chains of this CTA
  float2 ml_cta[kMaxClusterSplit][kTileM];   // (m, l) of every row of every CTA of the cluster, after its chains are merged
  uint64_t q_full;
  uint64_t k_full[2][2], k_empty[2][2], v_full[2][2], v_empty[2][2], s_full[2][2], p_full[2][2];  // [chain][stage]
  uint64_t pv_done[2];                       // [chain]: one phase per block of the chain
  uint64_t all_done[2];                      // [chain]: every MMA of the chain in this segment has completed (one phase per segment)
  uint64_t o_free;                           // the row threads have read both accumulators (one phase per segment)
  uint32_t tmem_base;
  volatile int abort_flag;
  int32_t abort_seen[2];                     // [segment parity]: abort_flag as one row thread saw it, so that all 256 leave together
  int32_t last_part;                         // stream mode: this CTA completed the tile (broadcast to the row threads)
  // mask from the parent array: the tree, and the ancestor rows of the current tile's nodes (row stride 33 words)
  int32_t parent[SEQ_MAX_TREE];
  uint32_t tile_mask[kTileM][SEQ_MAX_TREE / 32 + 1];
  int32_t tile_prefix[kMaxStreamTiles + 1];  // stream mode: positions of a kv head's layout before its t-th tile
};

static_assert(offsetof(UmmaSmem, v) == offsetof(UmmaSmem, k) + sizeof(UmmaSmem::k), "the cluster merge receives into k and v as one buffer");

struct UmmaArgs {
  int32_t n, L_host, Hq, Hkv, group, mask_wpr, splits, nodes_per_tile, tiles;
  const int32_t* L_dev;   // nullable: the prefix length in device memory (<= L_host)
  int32_t L_count;        // > 1: one length per request, requests stacked as heads (grid schedule only: a CTA has one kv head)
  int32_t zero_tail;      // the K/V maps cover the whole cache: rows past the tree are cleared in shared memory
  // Stream mode (more (tile, kv head) units than SMs): the 64-key blocks of all units, laid end to end, are
  // cut into gridDim.x equal ranges, one per CTA; a tile cut by a range boundary is completed by whichever
  // of its CTAs finishes last, from partial results in the workspace.
  int32_t stream, blocks_per_head_host;
  int64_t total_blocks_host;
  int32_t* ws_count;   // [Hkv * tiles] arrivals per tile, zero on entry and on exit
  float2* ws_ml;       // [2 * gridDim.x][128] (m, l) of a partial result
  float4* ws_o;        // [2 * gridDim.x][2][16][128] its unnormalised accumulator, thread-major
  float scale_log2;
  uint32_t idesc_qk, idesc_pv;
  const uint32_t* mask_bits;
  const int32_t* parent;  // used when mask_bits is null
  void* out; int64_t o_stride_tok, o_stride_head;
  float* lse;
  int32_t* dev_status;
};

// ---------------------------------------------------------------- PTX wrappers ------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises the CTA-wide abort flag) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(UmmaSmem* sm, uint64_t* bar, uint32_t parity, int32_t* dev_status) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u && sm->abort_flag) return false;
  }
  sm->abort_flag = 1;
  dev_flag(dev_status, SEQ_DEV_TIMEOUT);
  return false;
}

__device__ __forceinline__ void tma_load_5d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4) : "memory");
}
__device__ __forceinline__ void tma_load_4d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// True in exactly one lane of a converged warp.  Code that must be issued once per warp (MMAs, commits)
// goes under this predicate while everything around it stays warp-uniform, which keeps descriptors and
// addresses on the uniform datapath.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tc_mma_tmem_a(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

#define SEQ_R32(a, o) \
  "=r"(a[o + 0]), "=r"(a[o + 1]), "=r"(a[o + 2]), "=r"(a[o + 3]), "=r"(a[o + 4]), "=r"(a[o + 5]), "=r"(a[o + 6]),   \
  "=r"(a[o + 7]), "=r"(a[o + 8]), "=r"(a[o + 9]), "=r"(a[o + 10]), "=r"(a[o + 11]), "=r"(a[o + 12]),               \
  "=r"(a[o + 13]), "=r"(a[o + 14]), "=r"(a[o + 15]), "=r"(a[o + 16]), "=r"(a[o + 17]), "=r"(a[o + 18]),            \
  "=r"(a[o + 19]), "=r"(a[o + 20]), "=r"(a[o + 21]), "=r"(a[o + 22]), "=r"(a[o + 23]), "=r"(a[o + 24]),            \
  "=r"(a[o + 25]), "=r"(a[o + 26]), "=r"(a[o + 27]), "=r"(a[o + 28]), "=r"(a[o + 29]), "=r"(a[o + 30]),            \
  "=r"(a[o + 31])
#define SEQ_W32(a, o) \
  "r"(a[o + 0]), "r"(a[o + 1]), "r"(a[o + 2]), "r"(a[o + 3]), "r"(a[o + 4]), "r"(a[o + 5]), "r"(a[o + 6]),          \
  "r"(a[o + 7]), "r"(a[o + 8]), "r"(a[o + 9]), "r"(a[o + 10]), "r"(a[o + 11]), "r"(a[o + 12]), "r"(a[o + 13]),      \
  "r"(a[o + 14]), "r"(a[o + 15]), "r"(a[o + 16]), "r"(a[o + 17]), "r"(a[o + 18]), "r"(a[o + 19]), "r"(a[o + 20]),   \
  "r"(a[o + 21]), "r"(a[o + 22]), "r"(a[o + 23]), "r"(a[o + 24]), "r"(a[o + 25]), "r"(a[o + 26]), "r"(a[o + 27]),   \
  "r"(a[o + 28]), "r"(a[o + 29]), "r"(a[o + 30]), "r"(a[o + 31])

// 32 consecutive fp32 columns of this thread's tensor-memory lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r, int o) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, "
      "%23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : SEQ_R32(r, o) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r, int o) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, "
      "%23, %24, %25, %26, %27, %28, %29, %30, %31};"
      ::SEQ_W32(r, o), "r"(taddr) : "memory");
}

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
      ::"r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(taddr) : "memory");
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Two single-precision values in one 64-bit register, for the packed fused multiply-add and add: half the issue slots.
__device__ __forceinline__ uint64_t pair_of(float lo, float hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpair(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
// lbo/sbo in bytes.  K-major operands: sbo = 1024 (8 rows of 128 B), lbo unused.
// MN-major operands: lbo = stride between 64-element blocks along MN, sbo = 1024 between groups of 8 along K.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
  const uint32_t lo = ((smem_addr >> 4) & 0x3FFFu) | (((lbo >> 4) & 0x3FFFu) << 16);
  const uint32_t hi = ((sbo >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
  return ((uint64_t)hi << 32) | lo;
}

template <bool kBf16>
__device__ __forceinline__ uint32_t pack2(float a, float b) {
  if (kBf16) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
  } else {
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
  }
}

// 32 validity bits for tree indices [t, t+32) of one mask row; negative indices are prefix keys (visible)
__device__ __forceinline__ uint32_t mask_window(const uint32_t* row, int wpr, int n, int t) {
  const int w = t >> 5;  // floor
  const uint32_t lo = w < 0 ? 0xFFFFFFFFu : (w < wpr ? row[w] : 0u);
  const uint32_t hi = (w + 1) < 0 ? 0xFFFFFFFFu : ((w + 1) < wpr ? row[w + 1] : 0u);
  uint32_t bits = __funnelshift_r(lo, hi, t & 31);
  const int nvis = n - t;  // tree indices >= n do not exist, whatever the mask words hold there
  if (nvis < 32) bits &= nvis <= 0 ? 0u : ((1u << nvis) - 1u);
  return bits;
}

template <bool kBf16, bool kStream>
__global__ void __launch_bounds__(kUmmaThreads, 1)
tree_attention_umma_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                           const __grid_constant__ CUtensorMap v_map, const UmmaArgs a) {
  extern __shared__ uint8_t smem_raw[];
  UmmaSmem* sm = reinterpret_cast<UmmaSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  cg::cluster_group cluster = cg::this_cluster();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#ifdef SEQ_TRACE
  int utrace_i = 0;
#endif
  const int split = blockIdx.z;  // the cluster spans blockIdx.z
  if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 10);
#ifdef SEQ_TRACE
  const unsigned cta_lin = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;
  if (threadIdx.x == 128 && cta_lin < 1024) g_cta_times[cta_lin][0] = gtimer();
#endif

  // A CTA works through segments: (kv head, tile, range of the tile's 64-key blocks).  Grid mode: the one
  // segment (blockIdx.y, blockIdx.x, this CTA's share of the cluster's key range).  Stream mode: the pieces
  // of the units that its range [range_lo, range_hi) of the flattened block space overlaps.
  // The prefix length: the host's, or - for a step replayed from one CUDA graph while the prefix grows - read from
  // device memory below (the host's value is then the largest it can be, which the launch was planned for).
  int L = a.L_host;
  int blocks_per_head = a.blocks_per_head_host;
  int64_t total_blocks = a.total_blocks_host;
  int64_t range_lo = 0, range_hi = 1;
  struct Seg { int g, tile, slot_in_head, i0, i1, blk_lo, nblk, nblk_tile; int64_t next; };
  // Stream mode lays the tiles of a kv head out alternating from both ends (0, T-1, 1, T-2, ...): late tiles
  // have more masked blocks, which cost more, and this way every range gets its share of them.
  auto tile_at = [&](int k) { return (k & 1) ? a.tiles - 1 - (k >> 1) : (k >> 1); };
  auto seg_at = [&](int64_t pos) -> Seg {
    Seg x;
    if (!kStream) {
      x.tile = blockIdx.x; x.g = blockIdx.y; x.slot_in_head = x.tile;
      x.i0 = x.tile * a.nodes_per_tile;
      x.i1 = min(x.i0 + a.nodes_per_tile, a.n);
      // keys this tile can see end at L + i1 (a node sees no later node); blocks of this CTA
      x.nblk_tile = (L + x.i1 + kBlockN - 1) / kBlockN;
      x.blk_lo = (int)(((long)split * x.nblk_tile) / a.splits);
      x.nblk = (int)(((long)(split + 1) * x.nblk_tile) / a.splits) - x.blk_lo;
      x.next = 1;
    } else {
      x.g = (int)(pos / blocks_per_head);
      const int rem = (int)(pos % blocks_per_head);
      int lo = 0, hi = a.tiles - 1;  // the last place in the head's layout whose first block is at or before rem
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (sm->tile_prefix[mid] <= rem) lo = mid; else hi = mid - 1;
      }
      x.slot_in_head = lo;
      x.tile = tile_at(lo);
      x.i0 = x.tile * a.nodes_per_tile;
      x.i1 = min(x.i0 + a.nodes_per_tile, a.n);
      // the tile's positions are [vs, ve): kStreamTileCost positions of overhead, then its blocks
      const int vs = sm->tile_prefix[lo], ve = sm->tile_prefix[lo + 1];
      const int end = (int)min((int64_t)ve, (int64_t)rem + (range_hi - pos));  // where this CTA leaves the tile
      const int from = max(rem, vs + kStreamTileCost);
      x.blk_lo = from - (vs + kStreamTileCost);
      x.nblk_tile = ve - vs - kStreamTileCost;
      x.nblk = max(end - from, 0);  // 0: the range ends in the overhead positions, the tile is the next CTA's
      x.next = pos + (end - rem);
    }
    return x;
  };
  // The barriers are armed once.  Their phases run on from segment to segment: a stage barrier counts the
  // blocks its chain has processed so far, q_full / all_done[] / o_free count segments.  So the loads and
  // the first S of the next segment are under way while the row threads still merge and store this one.
  auto init_barriers = [&]() {  // thread 0
    mbar_init(&sm->q_full, 1);
    for (int c = 0; c < 2; ++c) {
      for (int b = 0; b < 2; ++b) {
        mbar_init(&sm->k_full[c][b], 1); mbar_init(&sm->k_empty[c][b], 1);
        mbar_init(&sm->v_full[c][b], 1); mbar_init(&sm->v_empty[c][b], 1);
        mbar_init(&sm->s_full[c][b], 1); mbar_init(&sm->p_full[c][b], 4);
      }
      mbar_init(&sm->pv_done[c], 1);
    }
    mbar_init(&sm->all_done[0], 1); mbar_init(&sm->all_done[1], 1);  // each has one arriver: its chain's MMA warp
    mbar_init(&sm->o_free, 8);    // one arrival per warp of row threads
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  };
  if (threadIdx.x == 0) {
    init_barriers();
    sm->abort_flag = 0;
    // programmatic dependent launch: the next kernel in the stream may be scheduled onto free SMs from now on (it
    // waits, as this one does below, before it touches memory); without the launch attribute this does nothing
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  // ... and everything above ran while the previous kernel in the stream was still finishing.  Nothing before this
  // line reads or writes global memory.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (a.L_dev != nullptr) {
    const int v = a.L_dev[(!kStream && a.L_count > 1) ? ((int)blockIdx.y * a.L_count) / a.Hkv : 0];
    if (v < 0 || v > a.L_host) { if (threadIdx.x == 0) dev_flag(a.dev_status, SEQ_DEV_BAD_LENGTH); }
    L = min(max(v, 0), a.L_host);
    if (kStream) {  // the flattened block space of this prefix length (every warp for itself)
      int sum = 0;
      for (int t = lane; t < a.tiles; t += 32) sum += kStreamTileCost + (L + min((t + 1) * a.nodes_per_tile, a.n) + kBlockN - 1) / kBlockN;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      blocks_per_head = sum;
      total_blocks = (int64_t)sum * a.Hkv;
    }
  }
  if (kStream) {
    range_lo = (total_blocks * (int64_t)blockIdx.x) / (int64_t)gridDim.x;
    range_hi = (total_blocks * (int64_t)(blockIdx.x + 1)) / (int64_t)gridDim.x;
  }
  // Grid schedule: the one segment of this CTA is known from its block index, so the thread that armed the barriers
  // requests the Q tile and the first K tile of each chain right away, before the CTA-wide barrier below and the
  // hand-over to the producer warps (which skip what has been requested here).
  if (!kStream && threadIdx.x == 0) {
    const Seg s0 = seg_at(range_lo);
    if (s0.nblk > 0) {
      mbar_expect_tx(&sm->q_full, kTileBytes);
      tma_load_5d(sm->q, &q_map, &sm->q_full, 0, 0, s0.i0, 0, s0.g);
      for (int jj = 0; jj < 2 && jj < s0.nblk; ++jj) {
        mbar_expect_tx(&sm->k_full[jj][0], kKvBytes);
        tma_load_4d(sm->k[jj][0], &k_map, &sm->k_full[jj][0], 0, (s0.blk_lo + jj) * kBlockN, 0, s0.g);
      }
    }
  }
  if (a.mask_bits == nullptr)
    for (int t = threadIdx.x; t < a.n; t += kUmmaThreads) sm->parent[t] = a.parent[t];
  if (kStream && warp == 2) {  // blocks of a kv head before each place of its layout: four places per lane, then a warp scan
    const int per = (a.tiles + 31) / 32;
    int local[kMaxStreamTiles / 32], sum = 0;
#pragma unroll
    for (int k = 0; k < kMaxStreamTiles / 32; ++k) {
      const int t = lane * per + k;
      local[k] = (k < per && t < a.tiles) ? kStreamTileCost + (L + min((tile_at(t) + 1) * a.nodes_per_tile, a.n) + kBlockN - 1) / kBlockN : 0;
      sum += local[k];
    }
    int incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += v;
    }
    int run = incl - sum;
#pragma unroll
    for (int k = 0; k < kMaxStreamTiles / 32; ++k) {
      const int t = lane * per + k;
      if (k < per && t < a.tiles) sm->tile_prefix[t] = run;
      run += local[k];
    }
    if (lane == 31) sm->tile_prefix[a.tiles] = incl;
  }
  if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 11);
  if (warp == 1) {  // all 512 tensor-memory columns: per chain two S buffers of 64 (P over them), then O_A, O_B
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&sm->tmem_base)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm->tmem_base;
  if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 0);

  if (warp < 4) {
    // ============================ warp group 0: data movement and MMA issue, few registers =========
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsLight));
    int seg_n = 0, base_an = 0, base_bn = 0;  // segments done; blocks chains A, B have processed in them
    uint32_t issued = 0, issued_parity = 0;   // producers: stages (bit 2*chain + stage; bit 4: Q) this warp has requested a tile for, and the phase of the last request
    for (int64_t pos = range_lo; pos < range_hi;) {
    const Seg sg = seg_at(pos);
    if (kStream && sg.nblk == 0) { pos = sg.next; continue; }
    const int g = sg.g, i0 = sg.i0, blk_lo = sg.blk_lo, nblk = sg.nblk;
    const int seg = kStream ? seg_n : 0, base_a = kStream ? base_an : 0, base_b = kStream ? base_bn : 0;  // grid mode: constants
    if (warp == 0 || warp == 3) {
      // ---------------------------------------------------------- TMA producers -----------------
      // Warp 0 loads Q and the K tiles, warp 3 the V tiles.  A K stage is free as soon as its S has been
      // computed, a V stage only after the block's softmax and P.V; in one queue the K loads would wait
      // behind the V stages and arrive just in time instead of a block ahead.
      // The whole warp runs the loop; one elected lane issues the copies (coordinates stay warp-uniform).
      if (nblk > 0) {
        const bool is_v = warp == 3;
        // the Q tile is free when every MMA of the previous segment has completed: the row threads have
        // seen that before they read O (waiting on o_free rather than all_done keeps every waiter of a
        // barrier within one phase of its arrivers)
        if (!is_v && seg > 0 && !mbar_wait(sm, &sm->o_free, (seg - 1) & 1, a.dev_status)) break;
        if (kStream && !is_v && elect_one()) {  // (grid schedule: requested before the roles split, see above)
          mbar_expect_tx(&sm->q_full, kTileBytes);
          tma_load_5d(sm->q, &q_map, &sm->q_full, 0, 0, i0, 0, g);  // both 64-element halves by one copy
        }
        __syncwarp();
        if (kStream && !is_v) { issued |= 16u; issued_parity = (issued_parity & ~16u) | ((uint32_t)(seg & 1) << 4); }
        const CUtensorMap* map = is_v ? &v_map : &k_map;
        for (int jj = (!kStream && !is_v) ? min(2, nblk) : 0; jj < nblk; ++jj) {
          const int c = jj & 1, u = (c ? base_b : base_a) + (jj >> 1);  // chain, the chain's running block count
          const int b = u & 1, w = u >> 1;                              // stage, use count of the stage
          const int row = (blk_lo + jj) * kBlockN;
          uint64_t* full = is_v ? &sm->v_full[c][b] : &sm->k_full[c][b];
          uint64_t* empty = is_v ? &sm->v_empty[c][b] : &sm->k_empty[c][b];
          uint8_t* dst = is_v ? sm->v[c][b] : sm->k[c][b];
          if (w > 0 && !mbar_wait(sm, empty, (w - 1) & 1, a.dev_status)) break;
          if (elect_one()) {
            mbar_expect_tx(full, kKvBytes);
            tma_load_4d(dst, map, full, 0, row, 0, g);  // both 64-element halves by one copy
          }
          __syncwarp();
          issued |= 1u << (2 * c + b);
          issued_parity = (issued_parity & ~(1u << (2 * c + b))) | ((uint32_t)(w & 1) << (2 * c + b));
          if (lane == 0 && !is_v) UTRACE(0, 1);
        }
      }
      __syncwarp();
    } else if (warp <= 2) {
      // ---------------------------------------------------------- MMA issuers -------------------
      // Warp 1 issues for chain A, warp 2 for chain B.  The whole warp runs this code; only the MMAs and
      // commits are issued by one elected lane, so descriptors and addresses stay warp-uniform.
      const int c = warp - 1;
      const int n_c = nblk > c ? (nblk - c + 1) >> 1 : 0;  // blocks of this chain
      // Both MMA warps see every phase of q_full, also in a segment in which their chain has no block: a
      // parity wait must never be two phases behind its barrier.
      const bool q_here = nblk > 0 && mbar_wait(sm, &sm->q_full, seg & 1, a.dev_status);
      if (n_c > 0) {
        const int base = c ? base_b : base_a;
        bool go = q_here;
        // A step along the contraction only moves a descriptor's 14-bit start-address field (16-byte units).
        const uint64_t qd0 = make_desc(smem_u32(sm->q), 16, 1024);
        const uint32_t tmem_o = tmem + 256u + 128u * c;
        // S of block u of the chain: buffer u & 1
        auto issue_qk = [&](int u) -> bool {
          const int b = (base + u) & 1, w = (base + u) >> 1;
          if (!mbar_wait(sm, &sm->k_full[c][b], w & 1, a.dev_status)) return false;
          tc_fence_after();
          const uint64_t kd0 = make_desc(smem_u32(sm->k[c][b]), 16, 1024);
          const uint32_t d = tmem + 128u * c + 64u * b;
          if (elect_one()) {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {  // 16 elements of head_dim per step: 32 bytes inside a 64-element sub-tile
              tc_mma(d, qd0 + (uint64_t)(((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4),
                     kd0 + (uint64_t)(((ks >> 2) * kKvHalf + (ks & 3) * 32) >> 4), a.idesc_qk, ks > 0);
            }
            tc_commit(&sm->k_empty[c][b]);
            tc_commit(&sm->s_full[c][b]);
          }
          __syncwarp();
          if (lane == 0) UTRACE(c == 0 ? 1 : 3, 2);
          return true;
        };
        // two S in flight before the first P is needed
        if (go) go = issue_qk(0);
        if (go && n_c > 1) go = issue_qk(1);
        for (int u = 0; u < n_c && go; ++u) {
          const int b = (base + u) & 1, w = (base + u) >> 1;
          if (!mbar_wait(sm, &sm->p_full[c][b], w & 1, a.dev_status)) break;
          // the first P.V of a segment overwrites O: the row threads must have read the previous segment's
          if (u == 0 && seg > 0 && !mbar_wait(sm, &sm->o_free, (seg - 1) & 1, a.dev_status)) break;
          if (lane == 0) UTRACE(c == 0 ? 1 : 3, 3);
          if (!mbar_wait(sm, &sm->v_full[c][b], w & 1, a.dev_status)) break;
          if (a.zero_tail) {
            // The tensor maps of this mode cover the whole cache, so a block that reaches past the last tree row has
            // fetched rows that may hold anything; their probabilities are exactly 0, but 0 * NaN is not: the rows are
            // cleared here (whole 128-byte rows of both halves: the swizzle stays inside a row), and the clearing is
            // made visible to the tensor core's reads.
            const int live = L + a.n - (blk_lo + 2 * u + c) * kBlockN;  // rows of this block that exist
            if (live < kBlockN) {
              uint4* vt = reinterpret_cast<uint4*>(sm->v[c][b]);
              for (int i = max(live, 0) * 8 + lane; i < kBlockN * 8; i += 32) {
                vt[i] = make_uint4(0u, 0u, 0u, 0u);
                vt[kKvHalf / 16 + i] = make_uint4(0u, 0u, 0u, 0u);
              }
              fence_async_smem();
              __syncwarp();
            }
          }
          tc_fence_after();
          const uint64_t vd0 = make_desc(smem_u32(sm->v[c][b]), kKvHalf, 1024);
          const uint32_t pa = tmem + 128u * c + 64u * b;
          const uint32_t first = u > 0 ? 1u : 0u;
          if (elect_one()) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)  // A = 8 packed columns of P, B = 16 key rows of V per step
              tc_mma_tmem_a(tmem_o, pa + 8u * ks, vd0 + (uint64_t)(ks * (2048 >> 4)), a.idesc_pv, ks > 0 ? 1u : first);
            tc_commit(&sm->v_empty[c][b]);
            tc_commit(&sm->pv_done[c]);
          }
          __syncwarp();
          if (lane == 0) UTRACE(c == 0 ? 1 : 3, 5);
          // S of block u+2 goes where P of block u lives.  tcgen05.mma operations issued by one thread
          // execute in issue order, so this QK^T cannot overtake the P.V just issued.
          if (u + 2 < n_c && !issue_qk(u + 2)) break;
        }
        if (elect_one()) tc_commit(&sm->all_done[c]);  // arrives when every MMA of this chain has completed
        __syncwarp();
      } else if (nblk > 0) {
        // A chain without blocks in this segment.  Its arrival must not overtake the completion of its own
        // previous segment (an asynchronous commit), nor run a phase ahead of the row threads: it waits
        // until they have taken the previous segment's accumulators.
        const bool go = q_here && (seg == 0 || mbar_wait(sm, &sm->o_free, (seg - 1) & 1, a.dev_status));
        if (go && lane == 0) mbar_arrive(&sm->all_done[c]);
      }
      __syncwarp();
    }
    if (a.splits > 1) {  // the two cluster barriers of the merge (see the row threads)
      cluster.sync();
      cluster.sync();
    }
    if (threadIdx.x == 32) UTRACE(1, 9);
    pos = sg.next;
    ++seg_n; base_an += (nblk + 1) >> 1; base_bn += nblk >> 1;
    if (kStream && sm->abort_flag) break;
    }  // segments
    // A CTA that gives up must not leave while a tile it has requested is still on its way into its shared memory
    // (the next CTA on this SM could get that memory): the producers wait, with a bound of their own, for the last
    // tile requested into each stage.  (Whether its consumer has taken that phase or not, the parity test answers
    // when the bytes have landed.  Tiles requested earlier into the same stage landed before the stage was reused.)
    if (sm->abort_flag && (warp == 0 || warp == 3)) {
      for (int st = 0; st < 5; ++st) {
        if (!((issued >> st) & 1u)) continue;
        uint64_t* full = st == 4 ? &sm->q_full : (warp == 3 ? &sm->v_full[st >> 1][st & 1] : &sm->k_full[st >> 1][st & 1]);
        for (uint32_t it = 0; it < (1u << 16); ++it)
          if (mbar_try_wait(full, (issued_parity >> st) & 1u)) break;
      }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
      tc_fence_after();
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
    }
    return;
  }

  // ============================== warp groups 1, 2: one thread per query row of chain A, B ============
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsRows));
  const int chain = (warp >> 2) - 1;
  const int quad = warp & 3;                  // tensor-memory lane quarter this warp may access
  const int r = quad * 32 + lane;             // row of the tile = tensor-memory lane
  const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
  const uint32_t tmem_o = tmem + 256u + 128u * chain + lane_sel;
  int seg_n = 0, base_n = 0;  // segments done; blocks this chain has processed in them
  for (int64_t pos = range_lo; pos < range_hi;) {
  const Seg sg = seg_at(pos);
  if (kStream && sg.nblk == 0) { pos = sg.next; continue; }
  const int g = sg.g, i0 = sg.i0, blk_lo = sg.blk_lo, nblk = sg.nblk;
  const int seg = kStream ? seg_n : 0, base = kStream ? base_n : 0;  // grid mode: constants
  const int i = i0 + r / a.group;             // node of this row
  const int h = g * a.group + r % a.group;
  const bool row_valid = i < a.n;
  // The row's ancestor bits: the caller's mask, or rows derived from the parent array at the start of the
  // segment by the first thread of each node (0 <= parent[j] < j, so a walk ends; anything else is flagged and
  // read as "no parent").  In grid mode the row threads are idle at this point, waiting for the first tiles.
  // (The previous segment's rows are out of use: every row thread has passed that segment's merge barrier.)
  if (a.mask_bits == nullptr) {
    if (chain == 0 && r % a.group == 0) {
      uint32_t* row = sm->tile_mask[r / a.group];
      const int wpr = (a.n + 31) >> 5;
      for (int w = 0; w < wpr; ++w) row[w] = 0u;  // (nodes past the last one see no tree key)
      int j = i;
      for (int step = 0; step < a.n && row_valid; ++step) {
        row[j >> 5] |= 1u << (j & 31);
        const int pj = sm->parent[j];
        if (pj == -1) break;
        if (pj < -1 || pj >= j) { dev_flag(a.dev_status, SEQ_DEV_BAD_PARENT); break; }
        j = pj;
      }
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
  }
  const uint32_t* mrow = a.mask_bits != nullptr ? a.mask_bits + (size_t)min(i, a.n - 1) * a.mask_wpr : sm->tile_mask[r / a.group];
  const int mask_wpr = a.mask_bits != nullptr ? a.mask_wpr : (a.n + 31) >> 5;
  const float sc = a.scale_log2;

  float m_used = -INFINITY, l = 0.f;
  bool ok = true;
  const int n_mine = nblk > chain ? (nblk - chain + 1) >> 1 : 0;  // blocks of this chain
  // A warp whose 32 rows all lie past the tile's last node (small trees fill only part of a 128-row tile) leaves
  // the special-function unit and the issue slots to the warps with real rows; its P rows stay whatever they are
  // (rows of the product are independent).
  const bool warp_live = i0 + (quad * 32) / a.group < a.n;
  for (int u = 0; u < n_mine && ok; ++u) {
    const int jj = 2 * u + chain, b = (base + u) & 1, w = (base + u) >> 1;
    const uint32_t tmem_s = tmem + 128u * chain + 64u * b + lane_sel;
    if (!mbar_wait(sm, &sm->s_full[chain][b], w & 1, a.dev_status)) { ok = false; break; }
    if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 1);
    if (!warp_live) {  // 32 padding rows: nothing to compute, only keep in step with the barriers
      __syncwarp();
      if (lane == 0) mbar_arrive(&sm->p_full[chain][b]);
      continue;
    }
    tc_fence_after();
    uint32_t sreg[64];
    tmem_ld32(tmem_s, sreg, 0);
    tmem_ld32(tmem_s + 32u, sreg, 32);
    const int kb = (blk_lo + jj) * kBlockN;
    const bool masked = kb + kBlockN > L;  // the block reaches into the tree keys (or past the end)
    uint32_t vis[2] = {0xFFFFFFFFu, 0xFFFFFFFFu};
    if (masked) {
      vis[0] = mask_window(mrow, mask_wpr, a.n, kb - L);
      vis[1] = mask_window(mrow, mask_wpr, a.n, kb - L + 32);
    }
    tc_wait_ld();
    if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 2);
    if (masked) {  // masked scores become -inf: probability exactly 0, and they cannot raise the maximum
#pragma unroll
      for (int e = 0; e < 64; ++e)
        if (!(vis[e >> 5] & (1u << (e & 31)))) sreg[e] = __float_as_uint(-INFINITY);
    }
    // P = 2^(scale*s - m) written over S as packed 16-bit values (32 columns, two stores of 16); returns the row sum.
    // (A row without a reference sees nothing in this block: its scores are all -inf and its P are 0.)
    auto exponentials = [&]() -> float {
      const float neg_m = m_used == -INFINITY ? 0.f : -m_used;
      const uint64_t sc2 = pair_of(sc, sc), neg_m2 = pair_of(neg_m, neg_m);
      uint64_t sm2[2] = {pair_of(0.f, 0.f), pair_of(0.f, 0.f)};
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t packed[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {  // two scores at a time: one packed multiply-add, two exponentials, one packed add
          float x0, x1;
          unpair(fma2(pair_of(__uint_as_float(sreg[32 * c + 2 * e]), __uint_as_float(sreg[32 * c + 2 * e + 1])), sc2, neg_m2), x0, x1);
          const float p0 = ex2(x0), p1 = ex2(x1);
          sm2[e & 1] = add2(sm2[e & 1], pair_of(p0, p1));
          packed[e] = pack2<kBf16>(p0, p1);
        }
        tmem_st16(tmem_s + 16u * c, packed);
      }
      float s0, s1, s2, s3;
      unpair(sm2[0], s0, s1);
      unpair(sm2[1], s2, s3);
      return (s0 + s1) + (s2 + s3);
    };
    // The reference maximum only moves when the block maximum exceeds it by more than the threshold, or when the row
    // has no reference yet: rare after the first blocks.  So the exponentials are taken against the reference as it
    // stands, and their sum tells whether that was right: a score more than the threshold above the reference gives a
    // term, hence a sum, above 2^threshold.  Only then (or without a reference) is the block maximum taken, the
    // reference moved, O rescaled, and the pass repeated (the scores are still in registers).
    float alpha = 1.f, sum = 0.f;
    bool settle = __any_sync(0xffffffffu, m_used == -INFINITY);
    if (!settle) {
      sum = exponentials();
      settle = __any_sync(0xffffffffu, !(sum <= kRescaleLimit));
    }
    if (settle) {
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int e = 0; e < 64; e += 2)  // three-input maximum: two scores per instruction
        mx[(e >> 1) & 3] = max3(mx[(e >> 1) & 3], __uint_as_float(sreg[e]), __uint_as_float(sreg[e + 1]));
      const float m_blk = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * sc;  // scale > 0
      const bool move = m_blk > m_used + kRescaleThreshold || (m_used == -INFINITY && m_blk != -INFINITY);
      if (__any_sync(0xffffffffu, move)) {
        if (move) {
          alpha = m_used == -INFINITY ? 0.f : ex2(m_used - m_blk);
          m_used = m_blk;
        }
        if (u > 0) {
          // O may still be taking the chain's previous block: wait for it, then rescale this warp's rows
          if (!mbar_wait(sm, &sm->pv_done[chain], (base + u - 1) & 1, a.dev_status)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t o[32];
            tmem_ld32(tmem_o + 32u * c, o, 0);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(tmem_o + 32u * c, o, 0);
          }
        }
      }
      sum = exponentials();
    }
    if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 3);
    l = l * alpha + sum;
    if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 4);
    tc_wait_st();
    if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 12);
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm->p_full[chain][b]);  // one arrival per warp
    if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 5);
  }
  // Both chains must be done with the tensor pipe before O is read and the K stages are reused.  (A
  // parity wait on pv_done could be fooled here: the other chain may be several phases behind.)
  if (nblk > 0 && ok) ok = mbar_wait(sm, &sm->all_done[0], seg & 1, a.dev_status) && mbar_wait(sm, &sm->all_done[1], seg & 1, a.dev_status);
  tc_fence_after();

  // ---------------------------------------------------------------- merge ------------------------
  // Step 1, inside the CTA: both accumulators live in this CTA's tensor memory and a warp may read
  // any column of its 32 lanes, so the thread of chain c and row r merges columns [64c, 64c+64) of
  // O_A and O_B itself; only (m, l) goes through shared memory.
  if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 6);
  sm->ml_chain[seg & 1][chain][r] = (ok && n_mine > 0) ? make_float2(m_used, l) : make_float2(-INFINITY, 0.f);
  // Whether to stop after this segment is decided once for all row threads: a flag raised between two threads' own
  // reads would send some to the closing barrier and the rest into the next segment's bar.sync, which has no bound.
  if (kStream && threadIdx.x == 128) sm->abort_seen[seg & 1] = sm->abort_flag;
  asm volatile("bar.sync 1, 256;" ::: "memory");  // the 256 row threads only
  const bool stop_here = kStream && sm->abort_seen[seg & 1] != 0;
  float M, Lc;           // reference maximum and denominator of the CTA's merged partial
  float merged[64];      // its columns [64*chain, 64*chain + 64), unnormalised
  {
    const float2 mlA = sm->ml_chain[seg & 1][0][r], mlB = sm->ml_chain[seg & 1][1][r];
    M = fmaxf(mlA.x, mlB.x);
    const float fA = mlA.x == -INFINITY ? 0.f : ex2(mlA.x - M), fB = mlB.x == -INFINITY ? 0.f : ex2(mlB.x - M);
    Lc = mlA.y * fA + mlB.y * fB;
    const int nA = nblk > 0 ? (nblk + 1) >> 1 : 0, nB = nblk >> 1;  // CTA-uniform: which accumulators were written
    const uint32_t oA = tmem + 256u + lane_sel + 64u * chain, oB = oA + 128u;
#pragma unroll
    for (int e = 0; e < 64; ++e) merged[e] = 0.f;
    if (nA > 0 && ok) {
      uint32_t o[64];
      tmem_ld32(oA, o, 0);
      tmem_ld32(oA + 32u, o, 32);
      tc_wait_ld();
#pragma unroll
      for (int e = 0; e < 64; ++e) merged[e] = __uint_as_float(o[e]) * fA;
    }
    if (nB > 0 && ok) {
      uint32_t o[64];
      tmem_ld32(oB, o, 0);
      tmem_ld32(oB + 32u, o, 32);
      tc_wait_ld();
#pragma unroll
      for (int e = 0; e < 64; ++e) merged[e] = fmaf(__uint_as_float(o[e]), fB, merged[e]);
    }
  }
  // both accumulators are in registers: the next segment's first P.V may overwrite them
  if (kStream) {
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(&sm->o_free);
  }
  uint8_t* out_row = reinterpret_cast<uint8_t*>(a.out) + 2 * ((int64_t)i * a.o_stride_tok + (int64_t)h * a.o_stride_head);
  if (kStream && nblk < sg.nblk_tile) {
    // A piece of a tile (stream mode).  Every piece is written to this CTA's slot of the workspace (slot 0
    // if the piece opens the CTA's range, else 1), then counted; the CTA whose count completes the tile
    // adds the other pieces to its own and writes the output.  Nobody waits for anybody.
    // positions of the tile's blocks in the layout, and the CTAs whose ranges hold some of them
    const int64_t t0 = (int64_t)g * blocks_per_head + sm->tile_prefix[sg.slot_in_head] + kStreamTileCost, t1 = t0 + sg.nblk_tile;
    auto cta_lo = [&](int c) { return (total_blocks * (int64_t)c) / (int64_t)gridDim.x; };
    int c_first = (int)((t0 * (int64_t)gridDim.x) / total_blocks);  // the CTA whose range holds block t0 ...
    while (cta_lo(c_first + 1) <= t0) ++c_first;                      // ... exactly
    while (cta_lo(c_first) > t0) --c_first;
    int c_last = c_first;
    while (cta_lo(c_last + 1) < t1) ++c_last;
    const int my_slot = 2 * (int)blockIdx.x + (max(t0, range_lo) == range_lo ? 0 : 1);
    int* cnt = a.ws_count + (size_t)g * a.tiles + sg.tile;
    const int parts = c_last - c_first + 1;
    // If every other piece has been counted already (the usual case for the piece that closes a range: the
    // others were finished long ago), this CTA completes the tile without writing its own piece.
    if (threadIdx.x == 128) {
      const int done = *reinterpret_cast<volatile int*>(cnt) == parts - 1;
      if (done) *cnt = 0;  // leave the counter as it was found
      sm->last_part = done;
    }
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (!sm->last_part) {
      if (chain == 0) a.ws_ml[(size_t)my_slot * kTileM + r] = make_float2(M, Lc);
      float4* my_o = a.ws_o + ((size_t)(my_slot * 2 + chain) * 16) * kTileM + r;
#pragma unroll
      for (int j = 0; j < 16; ++j) my_o[(size_t)j * kTileM] = make_float4(merged[4 * j], merged[4 * j + 1], merged[4 * j + 2], merged[4 * j + 3]);
      __threadfence();
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (threadIdx.x == 128) {
        const int last = atomicAdd(cnt, 1) == parts - 1;
        if (last) *cnt = 0;  // every piece has been counted
        sm->last_part = last;
      }
      asm volatile("bar.sync 1, 256;" ::: "memory");
    }
    if (sm->last_part) {
      // The pieces are added in the order of their CTAs, this CTA's own (from registers) at its place, with one
      // common reference maximum: the result does not depend on which CTA happened to finish last.
      __threadfence();
      auto slot_of = [&](int c) { return 2 * c + (max(t0, cta_lo(c)) == cta_lo(c) ? 0 : 1); };
      float Mg = M;
      for (int c = c_first; c <= c_last; ++c)
        if (c != (int)blockIdx.x) Mg = fmaxf(Mg, __ldcg(a.ws_ml + (size_t)slot_of(c) * kTileM + r).x);
      float Ls = 0.f;
#pragma unroll
      for (int half = 0; half < 2; ++half) {  // 32 columns at a time: the own piece must stay until its turn
        float acc[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) acc[e] = 0.f;
        for (int c = c_first; c <= c_last; ++c) {
          if (c == (int)blockIdx.x) {
            const float f = M == -INFINITY ? 0.f : ex2(M - Mg);
#pragma unroll
            for (int e = 0; e < 32; ++e) acc[e] = fmaf(merged[32 * half + e], f, acc[e]);
            if (half == 0) Ls = fmaf(Lc, f, Ls);
          } else {
            const int slot = slot_of(c);
            const float2 ml = __ldcg(a.ws_ml + (size_t)slot * kTileM + r);
            const float f = ml.x == -INFINITY ? 0.f : ex2(ml.x - Mg);
            const float4* its = a.ws_o + ((size_t)(slot * 2 + chain) * 16 + 8 * half) * kTileM + r;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float4 x = __ldcg(its + (size_t)j * kTileM);
              acc[4 * j] = fmaf(x.x, f, acc[4 * j]);
              acc[4 * j + 1] = fmaf(x.y, f, acc[4 * j + 1]);
              acc[4 * j + 2] = fmaf(x.z, f, acc[4 * j + 2]);
              acc[4 * j + 3] = fmaf(x.w, f, acc[4 * j + 3]);
            }
            if (half == 0) Ls = fmaf(ml.y, f, Ls);
          }
        }
#pragma unroll
        for (int e = 0; e < 32; ++e) merged[32 * half + e] = acc[e];
      }
      M = Mg;
      Lc = Ls;
    }
  }
  if (kStream && nblk < sg.nblk_tile && !sm->last_part) {
    // not the completing piece: nothing to write
  } else if (a.splits == 1) {
    if (row_valid) {
      const float inv = 1.f / Lc;  // the row saw at least its own key, so Lc > 0
#pragma unroll
      for (int e = 0; e < 64; e += 8) {
        uint4 val;
        val.x = pack2<kBf16>(merged[e] * inv, merged[e + 1] * inv);
        val.y = pack2<kBf16>(merged[e + 2] * inv, merged[e + 3] * inv);
        val.z = pack2<kBf16>(merged[e + 4] * inv, merged[e + 5] * inv);
        val.w = pack2<kBf16>(merged[e + 6] * inv, merged[e + 7] * inv);
        *reinterpret_cast<uint4*>(out_row + 2 * (64 * chain + e)) = val;
      }
      if (chain == 0 && a.lse != nullptr) a.lse[(size_t)h * a.n + i] = (M + log2f(Lc)) * kLn2;
    }
  } else {
    // Step 2, across the cluster (cs = 2 .. 8 CTAs along the key range).  The 16 slices of 8 output
    // columns are owned round-robin: slice s by CTA s % cs, as its slot s / cs.  Every CTA pushes each
    // 8-column piece of its merged partial into the owner's receive buffer (the K and V stages, adjacent in
    // shared memory and dead by then: cs * ceil(16 / cs) * 4 KB <= 84 KB of their 128 KB), laid out as float4
    // planes [contributor][slot][half][row], and its (m, l) into every CTA, with plain remote stores; after a
    // cluster barrier each owner reduces its slots locally.
    const int cs = a.splits, slots = (16 + cs - 1) / cs;  // (any cs from 2 to 8; the last slots of some CTAs may be empty)
    tc_fence_before();
    cluster.sync();  // every CTA of the cluster is done with its K and V stages before anyone writes into them
    if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 7);
    // (rows past the tile's last node are padding: nothing of theirs is pushed, reduced or stored)
    if (chain == 0 && row_valid)
      for (int q = 0; q < cs; ++q) *cluster.map_shared_rank(&sm->ml_cta[split][r], q) = make_float2(M, Lc);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      if (!row_valid) break;
      const int s_idx = 8 * chain + j;
      uint4* dst = cluster.map_shared_rank(reinterpret_cast<uint4*>(&sm->k[0][0][0]), s_idx % cs) +
                   ((size_t)(split * slots + s_idx / cs) * 2) * kTileM + r;
      dst[0] = make_uint4(__float_as_uint(merged[8 * j]), __float_as_uint(merged[8 * j + 1]),
                          __float_as_uint(merged[8 * j + 2]), __float_as_uint(merged[8 * j + 3]));
      dst[kTileM] = make_uint4(__float_as_uint(merged[8 * j + 4]), __float_as_uint(merged[8 * j + 5]),
                               __float_as_uint(merged[8 * j + 6]), __float_as_uint(merged[8 * j + 7]));
    }
    cluster.sync();
    if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 8);
    float Mg = -INFINITY;
    for (int q = 0; q < cs; ++q) Mg = fmaxf(Mg, sm->ml_cta[q][r].x);
    float Ls = 0.f;
    for (int q = 0; q < cs; ++q) {
      const float2 mlq = sm->ml_cta[q][r];
      if (mlq.x != -INFINITY) Ls += mlq.y * ex2(mlq.x - Mg);
    }
    const float inv = 1.f / Ls;  // some CTA saw the row's own key, so Ls > 0
    const float4* mine = reinterpret_cast<const float4*>(&sm->k[0][0][0]);
    for (int slot = chain; slot < slots && row_valid; slot += 2) {  // the two warp groups share this CTA's slots
      if (slot * cs + split >= 16) break;  // (cs does not divide 16: this CTA owns one slice fewer)
      float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      for (int q = 0; q < cs; ++q) {
        const float mq = sm->ml_cta[q][r].x;
        if (mq == -INFINITY) continue;
        const float f = ex2(mq - Mg);
        const float4* src = mine + ((size_t)(q * slots + slot) * 2) * kTileM + r;
        const float4 x = src[0], y = src[kTileM];
        acc[0] = fmaf(x.x, f, acc[0]); acc[1] = fmaf(x.y, f, acc[1]); acc[2] = fmaf(x.z, f, acc[2]); acc[3] = fmaf(x.w, f, acc[3]);
        acc[4] = fmaf(y.x, f, acc[4]); acc[5] = fmaf(y.y, f, acc[5]); acc[6] = fmaf(y.z, f, acc[6]); acc[7] = fmaf(y.w, f, acc[7]);
      }
      if (row_valid) {
        uint4 val;
        val.x = pack2<kBf16>(acc[0] * inv, acc[1] * inv);
        val.y = pack2<kBf16>(acc[2] * inv, acc[3] * inv);
        val.z = pack2<kBf16>(acc[4] * inv, acc[5] * inv);
        val.w = pack2<kBf16>(acc[6] * inv, acc[7] * inv);
        *reinterpret_cast<uint4*>(out_row + 2 * (8 * (slot * cs + split))) = val;
      }
    }
    if (split == 0 && chain == 0 && row_valid && a.lse != nullptr) a.lse[(size_t)h * a.n + i] = (Mg + log2f(Ls)) * kLn2;
  }
  if (threadIdx.x == SEQ_TRACE_ROW) UTRACE(2, 9);
  pos = sg.next;
  ++seg_n; base_n += n_mine;
  if (stop_here) break;
  }  // segments
#ifdef SEQ_TRACE
  if (threadIdx.x == 128 && cta_lin < 1024) g_cta_times[cta_lin][1] = gtimer();
#endif
  // no remote access happens after the second cluster barrier, so CTAs may leave independently
  tc_fence_before();
  __syncthreads();  // pairs with warp group 0, whose MMA warp then frees the tensor memory
}

// ---------------------------------------------------------------- host side ---------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static void* cached = nullptr;  // the driver's entry point, looked up once (the same answer from every thread)
  void* p = __atomic_load_n(&cached, __ATOMIC_ACQUIRE);
  if (p == nullptr) {
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || p == nullptr)
      return nullptr;
    __atomic_store_n(&cached, p, __ATOMIC_RELEASE);
  }
  return reinterpret_cast<EncodeTiledFn>(p);
}

// Encoded tensor maps are kept: a caller that launches directly (no CUDA graph) passes the same pointers and shapes
// step after step, and an encode is a driver call of a microsecond or two.  A map depends on nothing but the
// arguments of the encode (the swizzle, interleave, promotion and fill are the same for every map of this file), so
// the key is those arguments, compared byte for byte; 16 entries, replaced in turn; one lock around the table.
namespace {
struct MapKey {
  const void* base;
  cuuint64_t dims[5], strides[4];
  cuuint32_t box[5];
  int32_t rank, dtype;
};
struct MapEntry { MapKey key; CUtensorMap map; bool used; };
MapEntry g_maps[16];
unsigned g_maps_next = 0;
int g_maps_lock = 0;

CUresult encode_cached(EncodeTiledFn encode, CUtensorMap* out, CUtensorMapDataType dt, cuuint32_t rank, const void* base,
                       const cuuint64_t* dims, const cuuint64_t* strides, const cuuint32_t* box) {
  MapKey key;
  memset(&key, 0, sizeof(key));
  key.base = base; key.rank = (int32_t)rank; key.dtype = (int32_t)dt;
  for (cuuint32_t i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
  for (cuuint32_t i = 0; i + 1 < rank; ++i) key.strides[i] = strides[i];
  while (__atomic_exchange_n(&g_maps_lock, 1, __ATOMIC_ACQUIRE) != 0) { }
  for (MapEntry& e : g_maps)
    if (e.used && memcmp(&e.key, &key, sizeof(key)) == 0) {
      *out = e.map;
      __atomic_store_n(&g_maps_lock, 0, __ATOMIC_RELEASE);
      return CUDA_SUCCESS;
    }
  __atomic_store_n(&g_maps_lock, 0, __ATOMIC_RELEASE);
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  const CUresult r = encode(out, dt, rank, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return r;
  while (__atomic_exchange_n(&g_maps_lock, 1, __ATOMIC_ACQUIRE) != 0) { }
  MapEntry& e = g_maps[g_maps_next++ % 16];
  e.key = key; e.map = *out; e.used = true;
  __atomic_store_n(&g_maps_lock, 0, __ATOMIC_RELEASE);
  return CUDA_SUCCESS;
}
}  // namespace

bool umma_supported(const seq_tree_attention_params& p) {
  if (p.dtype != SEQ_F16 && p.dtype != SEQ_BF16) return false;
  const int G = p.num_q_heads / p.num_kv_heads;
  if (G > kTileM || kTileM % G != 0) return false;
  return true;
}

// How the tiles are spread over the SMs.  Grid schedule: one CTA (or a cluster of `splits` CTAs along the key
// range) per (tile, kv head), in as many waves as that takes.  Stream schedule: one CTA per SM, each with an equal range of the
// flattened block space and share the tiles that a range boundary cuts.  p.kernel = 3 / 4 force one of them.
struct UmmaPlan { int splits; bool stream; };
static UmmaPlan umma_plan(const seq_tree_attention_params& p) {
  const int G = p.num_q_heads / p.num_kv_heads;
  const int nodes_per_tile = kTileM / G;
  const int tiles = (p.n_tree + nodes_per_tile - 1) / nodes_per_tile;
  const long units = (long)tiles * p.num_kv_heads;
  const int nblk = (p.prefix_len + p.n_tree + kBlockN - 1) / kBlockN;
  const bool can_stream = tiles <= kMaxStreamTiles && p.prefix_len_dev_count <= 1;  // (a range of the stream schedule crosses kv heads: one length)
  const int kNumSMs = device_sm_count();
#ifdef SEQ_TRACE
  if (const char* e = getenv("SEQ_DEBUG_SPLITS")) return {atoi(e), false};  // debug builds only
#endif
  if (p.kernel == 3 && can_stream) return {1, true};
  // More units than SMs.  Measured over batches of the paper's shapes (5 to 32 requests stacked as heads): plain
  // waves of one CTA per unit win by 5-50 % when tiles are short (a tile cut by a range boundary costs a trip
  // through the workspace, and every CTA starts and finishes two tiles more), the stream schedule wins by 5-15 %
  // when tiles are long (72 blocks and more) or when the last wave would be at most 60 % full.
  if (p.kernel != 4 && can_stream && units > kNumSMs) {
    const long waves = (units + kNumSMs - 1) / kNumSMs;
    const bool last_wave_thin = units * 10 <= waves * kNumSMs * 6;
    if (nblk >= 32 && (last_wave_thin || nblk >= 72)) return {1, true};
  }
  int best = 1;
  double best_cost = -1.0;
  for (int cs = 1; cs <= kMaxClusterSplit; ++cs) {
    if (cs > 1 && cs > nblk) break;
    const long waves = (units * cs + kNumSMs - 1) / kNumSMs;
    // microseconds per wave, fitted to measured launches of the paper's shapes with every split forced: 0.65 per
    // block of a CTA's key range, 4.7 fixed, and 1.6 + 0.5 per CTA beyond two for the merge across the cluster
    const double merge = cs == 1 ? 0.0 : 1.6 + 0.5 * (cs - 2);
    const double cost = (double)waves * (0.65 * ((nblk + cs - 1) / cs) + 4.7 + merge);
    if (best_cost < 0 || cost < best_cost - 1e-9) { best = cs; best_cost = cost; }
  }
  return {best, false};
}

int umma_default_splits(const seq_tree_attention_params& p) { return umma_plan(p).splits; }

static bool umma_stream_mode(const seq_tree_attention_params& p, int splits) {
  (void)splits;
  return umma_plan(p).stream;
}

// Workspace of the stream mode: one arrival counter per (kv head, tile), then two slots per CTA for the
// pieces of tiles that its range cuts: (m, l) per row and the 128 x 128 fp32 accumulator.
static size_t stream_count_bytes(const seq_tree_attention_params& p) {
  const int G = p.num_q_heads / p.num_kv_heads;
  const int nodes_per_tile = kTileM / G;
  const int tiles = (p.n_tree + nodes_per_tile - 1) / nodes_per_tile;
  return ((size_t)tiles * p.num_kv_heads * sizeof(int32_t) + 255) & ~(size_t)255;
}
static size_t stream_ml_bytes() { return (size_t)2 * device_sm_count() * kTileM * sizeof(float2); }
static size_t stream_o_bytes() { return (size_t)2 * device_sm_count() * 2 * 16 * kTileM * sizeof(float4); }

size_t umma_workspace_bytes(const seq_tree_attention_params& p) {
  if (!umma_stream_mode(p, umma_default_splits(p))) return 0;
  return stream_count_bytes(p) + stream_ml_bytes() + stream_o_bytes();
}

int launch_attention_umma(const seq_tree_attention_params& p, int splits, cudaStream_t stream) {
  EncodeTiledFn encode = encode_fn();
  if (encode == nullptr) return SEQ_ERR_CUDA;
  const int G = p.num_q_heads / p.num_kv_heads;
  const int nodes_per_tile = kTileM / G;
  const int tiles = (p.n_tree + nodes_per_tile - 1) / nodes_per_tile;
  const CUtensorMapDataType dt = p.dtype == SEQ_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16;

  CUtensorMap q_map, k_map, v_map;
  {
    // q viewed as [kv head][node][head in group][head_dim]
    // head_dim is split into its two 64-element halves (a dimension of its own, 128 bytes apart) so that one copy
    // brings the tile as [half][row][64 elements], the layout of two 128-byte-swizzled sub-tiles
    cuuint64_t dims[5] = {64, (cuuint64_t)G, (cuuint64_t)p.n_tree, 2, (cuuint64_t)p.num_kv_heads};
    cuuint64_t strides[4] = {(cuuint64_t)p.q_stride_head * 2, (cuuint64_t)p.q_stride_tok * 2, 128,
                             (cuuint64_t)p.q_stride_head * 2 * G};
    cuuint32_t box[5] = {64, (cuuint32_t)G, (cuuint32_t)nodes_per_tile, 2, 1};
    if (encode_cached(encode, &q_map, dt, 5, p.q, dims, strides, box) != CUDA_SUCCESS) return SEQ_ERR_CUDA;
  }
  for (int which = 0; which < 2; ++which) {
    // only the live rows [0, prefix_len + n_tree) are mapped: anything past them reads as zero.  (With the prefix
    // length in device memory the map cannot end there: it covers the cache, and the kernel clears the tail rows.)
    cuuint64_t dims[4] = {64, (cuuint64_t)(p.prefix_len_dev != nullptr ? p.kv_capacity : p.prefix_len + p.n_tree), 2, (cuuint64_t)p.num_kv_heads};
    cuuint64_t strides[3] = {(cuuint64_t)p.kv_stride_tok * 2, 128, (cuuint64_t)p.kv_stride_head * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)kBlockN, 2, 1};
    if (encode_cached(encode, which == 0 ? &k_map : &v_map, dt, 4, which == 0 ? p.k_cache : p.v_cache, dims, strides, box) != CUDA_SUCCESS)
      return SEQ_ERR_CUDA;
  }

  UmmaArgs a;
  a.n = p.n_tree; a.L_host = p.prefix_len; a.Hq = p.num_q_heads; a.Hkv = p.num_kv_heads; a.group = G;
  a.mask_wpr = p.mask_words_per_row; a.splits = splits; a.nodes_per_tile = nodes_per_tile; a.tiles = tiles;
  const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 0.08838834764831845f;
  a.scale_log2 = scale * kLog2e;
  const uint32_t fmt = p.dtype == SEQ_BF16 ? 1u : 0u;
  // instruction descriptor: D fp32 (bit 4), A/B format (bits 7, 10), B major (bit 16), N>>3 (bit 17), M>>4 (bit 24)
  const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(kTileM >> 4) << 24);
  a.idesc_qk = idesc | ((uint32_t)(kBlockN >> 3) << 17);                 // S: N = 64 keys
  a.idesc_pv = idesc | ((uint32_t)(kHeadDim >> 3) << 17) | (1u << 16);   // O: N = 128, V is MN-major
  a.mask_bits = p.mask_bits;
  a.parent = p.parent;
  a.out = p.out; a.o_stride_tok = p.o_stride_tok; a.o_stride_head = p.o_stride_head;
  a.lse = p.lse;
  a.dev_status = p.dev_status;
  a.stream = umma_stream_mode(p, splits) ? 1 : 0;
  a.blocks_per_head_host = 0; a.total_blocks_host = 0;
  a.L_dev = p.prefix_len_dev; a.L_count = p.prefix_len_dev_count; a.zero_tail = p.prefix_len_dev != nullptr ? 1 : 0;
  a.ws_count = nullptr; a.ws_ml = nullptr; a.ws_o = nullptr;
  if (a.stream) {
    const size_t cnt_bytes = stream_count_bytes(p);
    if (p.workspace == nullptr || p.workspace_bytes < cnt_bytes + stream_ml_bytes() + stream_o_bytes()) return SEQ_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(p.workspace) % 256 != 0) return SEQ_ERR_INVALID_ARG;
    for (int t = 0; t < tiles; ++t) {
      const int i1 = (t + 1) * nodes_per_tile < p.n_tree ? (t + 1) * nodes_per_tile : p.n_tree;
      a.blocks_per_head_host += kStreamTileCost + (p.prefix_len + i1 + kBlockN - 1) / kBlockN;
    }
    a.total_blocks_host = (int64_t)a.blocks_per_head_host * p.num_kv_heads;
    uint8_t* ws = static_cast<uint8_t*>(p.workspace);
    a.ws_count = reinterpret_cast<int32_t*>(ws);
    a.ws_ml = reinterpret_cast<float2*>(ws + cnt_bytes);
    a.ws_o = reinterpret_cast<float4*>(ws + cnt_bytes + stream_ml_bytes());
    SEQ_CUDA_OK(cudaMemsetAsync(a.ws_count, 0, cnt_bytes, stream));  // the counters start at zero (the kernel leaves them at zero)
  }

  const size_t smem = sizeof(UmmaSmem) + 1024;
  cudaLaunchConfig_t cfg = {};
  // Stream schedule: one CTA per SM, but never more CTAs than positions in the layout: a range must not be empty
  // (the CTAs that share a cut tile are counted from the ranges, and each of them has to arrive).
  const int sms = device_sm_count();
  const int stream_ctas = a.total_blocks_host < sms ? (int)a.total_blocks_host : sms;
  cfg.gridDim = a.stream ? dim3(stream_ctas, 1, 1) : dim3(tiles, p.num_kv_heads, splits);
  cfg.blockDim = dim3(kUmmaThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = splits;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // start under the previous kernel's tail (see the kernel)
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  // four instantiations: element type x (grid | stream) mode; the grid-mode code carries none of the stream machinery
  auto launch = [&](auto kernel, int which) -> int {
    static int attr_done[4][64];  // the opt-in shared-memory size is set once per kernel and device
    const int rc = once_per_device(attr_done[which], [&]() -> int {
      SEQ_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      return SEQ_OK;
    });
    if (rc != SEQ_OK) return rc;
    SEQ_CUDA_OK(cudaLaunchKernelEx(&cfg, kernel, q_map, k_map, v_map, a));
    return SEQ_OK;
  };
  if (p.dtype == SEQ_BF16) return a.stream ? launch(tree_attention_umma_kernel<true, true>, 0) : launch(tree_attention_umma_kernel<true, false>, 1);
  return a.stream ? launch(tree_attention_umma_kernel<false, true>, 2) : launch(tree_attention_umma_kernel<false, false>, 3);
}

}  // namespace seqtree
