// Tree-masked attention on the 5th-generation tensor cores (tcgen05.mma, accumulators in tensor
// memory, K/V/Q tiles staged by TMA), for 16-bit inputs.
//
// Work unit: one CTA = (kv head g, tile of 128 query rows, split of the key range).  A query row is
// a (node, head-in-group) pair, r = i_local * G + hg, so under GQA the G heads that share a kv head
// share every K/V tile.  Keys are taken in blocks of 128:
//     S = Q K^T      128x128x128  tcgen05.mma, Q and K K-major in 128-byte-swizzled shared memory
//     P = 2^(scale*S - m) masked  one thread per row, S read from tensor memory
//     O += P V       128x128x128  tcgen05.mma, P (16-bit) in shared memory, V MN-major
// Warp 0 issues TMA loads, warp 1 issues MMAs, warps 2..5 own the 128 rows.  S is double-buffered
// in tensor memory so that S(j+1) is computed while the row threads work on block j.  The running
// maximum is only moved when a row's block maximum exceeds it by more than 2^8 (the accumulator is
// then rescaled in tensor memory), so in steady state O is never touched by the row threads.
//
// Masking: key j < prefix_len is visible; key prefix_len + t is visible iff bit t of the row's
// ancestor mask; masked scores become -inf before the maximum, so their probability is exactly 0.
// Rows of K/V past prefix_len + n_tree are never fetched: the tensor maps end there and TMA fills
// the rest of a tile with zeros.
//
// Every mbarrier wait is bounded; a wait that runs out raises SEQ_DEV_TIMEOUT and the CTA drains.
#include <cuda.h>

#include "common.cuh"

namespace seqtree {

constexpr int kTileM = 128;      // query rows per CTA
constexpr int kBlockN = 128;     // keys per block
constexpr int kStages = 2;       // K and V stages each
constexpr int kUmmaThreads = 192;
constexpr uint32_t kTileBytes = 128 * 128 * 2;  // one 128x128 16-bit tile
constexpr uint32_t kHalfBytes = kTileBytes / 2; // one 128-row x 64-element sub-tile (128 B rows)
constexpr float kRescaleThreshold = 8.f;        // log2 units
constexpr uint32_t kSpinLimit = 1u << 22;

struct UmmaSmem {
  // all tiles 1024-byte aligned (128-byte swizzle atoms are 8 rows x 128 B)
  uint8_t q[kTileBytes];
  uint8_t k[kStages][kTileBytes];
  uint8_t v[kStages][kTileBytes];
  uint8_t p[kTileBytes];
  uint64_t q_full, k_full[kStages], k_empty[kStages], v_full[kStages], v_empty[kStages];
  uint64_t s_full[2], s_empty[2], p_full, pv_done;
  uint32_t tmem_base;
  volatile int abort_flag;
};

struct UmmaArgs {
  int32_t n, L, Hq, Hkv, group, mask_wpr, splits, nodes_per_tile, tiles;
  float scale_log2;
  uint32_t idesc_qk, idesc_pv;
  const uint32_t* mask_bits;
  void* out; int64_t o_stride_tok, o_stride_head;
  float* lse; float* o_part; float2* ml;
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

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2) : "memory");
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

template <bool kBf16>
__global__ void __launch_bounds__(kUmmaThreads, 1)
tree_attention_umma_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                           const __grid_constant__ CUtensorMap v_map, const UmmaArgs a) {
  extern __shared__ uint8_t smem_raw[];
  UmmaSmem* sm = reinterpret_cast<UmmaSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, g = blockIdx.y, split = blockIdx.z;

  const int i0 = tile * a.nodes_per_tile;
  const int i1 = min(i0 + a.nodes_per_tile, a.n);
  // keys this tile can see end at L + i1 (a node sees no later node); blocks of this split
  const int nblk_tile = (a.L + i1 + kBlockN - 1) / kBlockN;
  const int blk_lo = (int)(((long)split * nblk_tile) / a.splits);
  const int blk_hi = (int)(((long)(split + 1) * nblk_tile) / a.splits);
  const int nblk = blk_hi - blk_lo;

  if (threadIdx.x == 0) {
    mbar_init(&sm->q_full, 1);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sm->k_full[s], 1); mbar_init(&sm->k_empty[s], 1);
      mbar_init(&sm->v_full[s], 1); mbar_init(&sm->v_empty[s], 1);
    }
    for (int b = 0; b < 2; ++b) { mbar_init(&sm->s_full[b], 1); mbar_init(&sm->s_empty[b], 128); }
    mbar_init(&sm->p_full, 128);
    mbar_init(&sm->pv_done, 1);
    sm->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {  // 512 tensor-memory columns: S0, S1, O (128 each) + spare
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(&sm->tmem_base)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm->tmem_base;
  const uint32_t tmem_s[2] = {tmem, tmem + 128u};
  const uint32_t tmem_o = tmem + 256u;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer ------------------
    if (lane == 0 && nblk > 0) {
      mbar_expect_tx(&sm->q_full, kTileBytes);
      tma_load_4d(sm->q, &q_map, &sm->q_full, 0, 0, i0, g);
      tma_load_4d(sm->q + kHalfBytes, &q_map, &sm->q_full, 64, 0, i0, g);
      for (int jj = 0; jj < nblk; ++jj) {
        const int s = jj % kStages;
        const int row = (blk_lo + jj) * kBlockN;
        if (jj >= kStages && !mbar_wait(sm, &sm->k_empty[s], ((jj / kStages) - 1) & 1, a.dev_status)) break;
        mbar_expect_tx(&sm->k_full[s], kTileBytes);
        tma_load_3d(sm->k[s], &k_map, &sm->k_full[s], 0, row, g);
        tma_load_3d(sm->k[s] + kHalfBytes, &k_map, &sm->k_full[s], 64, row, g);
        if (jj >= kStages && !mbar_wait(sm, &sm->v_empty[s], ((jj / kStages) - 1) & 1, a.dev_status)) break;
        mbar_expect_tx(&sm->v_full[s], kTileBytes);
        tma_load_3d(sm->v[s], &v_map, &sm->v_full[s], 0, row, g);
        tma_load_3d(sm->v[s] + kHalfBytes, &v_map, &sm->v_full[s], 64, row, g);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer --------------------
    if (lane == 0 && nblk > 0) {
      bool ok = mbar_wait(sm, &sm->q_full, 0, a.dev_status);
      auto issue_qk = [&](int j) -> bool {
        const int s = j % kStages, b = j & 1;
        if (!mbar_wait(sm, &sm->k_full[s], (j / kStages) & 1, a.dev_status)) return false;
        if (j >= 2 && !mbar_wait(sm, &sm->s_empty[b], ((j >> 1) - 1) & 1, a.dev_status)) return false;
        tc_fence_after();
        const uint32_t qa = smem_u32(sm->q), ka = smem_u32(sm->k[s]);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {  // 8 steps of 16 along head_dim; 4 per 64-element sub-tile
          const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
          tc_mma(tmem_s[b], make_desc(qa + off, 16, 1024), make_desc(ka + off, 16, 1024), a.idesc_qk, ks > 0);
        }
        tc_commit(&sm->k_empty[s]);
        tc_commit(&sm->s_full[b]);
        return true;
      };
      if (ok) ok = issue_qk(0);
      for (int jj = 0; jj < nblk && ok; ++jj) {
        if (jj + 1 < nblk && !issue_qk(jj + 1)) break;
        const int s = jj % kStages;
        if (!mbar_wait(sm, &sm->p_full, jj & 1, a.dev_status)) break;
        if (!mbar_wait(sm, &sm->v_full[s], (jj / kStages) & 1, a.dev_status)) break;
        tc_fence_after();
        const uint32_t pa = smem_u32(sm->p), va = smem_u32(sm->v[s]);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {  // 8 steps of 16 keys
          const uint64_t adesc = make_desc(pa + (ks >> 2) * kHalfBytes + (ks & 3) * 32, 16, 1024);
          const uint64_t bdesc = make_desc(va + ks * 2048, kHalfBytes, 1024);
          tc_mma(tmem_o, adesc, bdesc, a.idesc_pv, (jj > 0 || ks > 0) ? 1u : 0u);
        }
        tc_commit(&sm->v_empty[s]);
        tc_commit(&sm->pv_done);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ row threads -------------------
    const int quad = warp & 3;                  // tensor-memory lane quarter this warp may access
    const int r = quad * 32 + lane;             // row of the tile = tensor-memory lane
    const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
    const int i = i0 + r / a.group;             // node of this row
    const int hg = r % a.group;
    const bool row_valid = i < a.n;
    const uint32_t* mrow = a.mask_bits + (size_t)min(i, a.n - 1) * a.mask_wpr;

    float m_used = -INFINITY, l = 0.f;
    bool ok = true;
    uint32_t sreg[128];
    for (int jj = 0; jj < nblk && ok; ++jj) {
      const int b = jj & 1;
      if (!mbar_wait(sm, &sm->s_full[b], (jj >> 1) & 1, a.dev_status)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(tmem_s[b] + lane_sel + 32u * c, sreg, 32 * c);
      tc_wait_ld();
      tc_fence_before();
      mbar_arrive(&sm->s_empty[b]);

      // scale, mask, block maximum
      const int kb = (blk_lo + jj) * kBlockN;
      const bool needs_mask = kb + kBlockN > a.L;
      float m_blk = -INFINITY;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t vis = 0xFFFFFFFFu;
        if (needs_mask) vis = mask_window(mrow, a.mask_wpr, a.n, kb - a.L + 32 * c);
#pragma unroll
        for (int e = 0; e < 32; ++e) {
          float s = __uint_as_float(sreg[32 * c + e]) * a.scale_log2;
          s = (vis >> e) & 1u ? s : -INFINITY;
          sreg[32 * c + e] = __float_as_uint(s);
          m_blk = fmaxf(m_blk, s);
        }
      }
      // move the reference maximum only when it is first set or exceeded by more than the threshold
      float alpha = 1.f;
      if (m_blk > m_used + kRescaleThreshold || (m_used == -INFINITY && m_blk != -INFINITY)) {
        alpha = m_used == -INFINITY ? 0.f : ex2(m_used - m_blk);
        m_used = m_blk;
      }
      const float m_eff = m_used == -INFINITY ? 0.f : m_used;
      float sum = 0.f;
      uint32_t packed[64];
#pragma unroll
      for (int e = 0; e < 128; e += 2) {
        const float p0 = ex2(__uint_as_float(sreg[e]) - m_eff);
        const float p1 = ex2(__uint_as_float(sreg[e + 1]) - m_eff);
        sum += p0 + p1;
        packed[e >> 1] = pack2<kBf16>(p0, p1);
      }
      l = l * alpha + sum;

      if (jj > 0) {
        if (!mbar_wait(sm, &sm->pv_done, (jj - 1) & 1, a.dev_status)) { ok = false; break; }
        tc_fence_after();
        if (__any_sync(0xffffffffu, alpha != 1.f)) {  // rescale the accumulator rows of this warp
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint32_t o[32];
            tmem_ld32(tmem_o + lane_sel + 32u * c, o, 0);
            tc_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(tmem_o + lane_sel + 32u * c, o, 0);
          }
          tc_wait_st();
        }
        tc_fence_before();
      }
      // P tile -> shared memory, K-major with 128-byte swizzle: 16-byte chunk c of row r sits at chunk c ^ (r & 7)
      uint8_t* prow = sm->p + r * 128;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const int src = half * 32 + c * 4;
          uint4 val = make_uint4(packed[src], packed[src + 1], packed[src + 2], packed[src + 3]);
          *reinterpret_cast<uint4*>(prow + half * kHalfBytes + ((c ^ (r & 7)) << 4)) = val;
        }
      }
      fence_async_smem();
      mbar_arrive(&sm->p_full);
    }

    // ------------------------------------------------------------ epilogue ----------------------
    if (nblk > 0 && ok) ok = mbar_wait(sm, &sm->pv_done, (nblk - 1) & 1, a.dev_status);
    tc_fence_after();
    const int h = g * a.group + hg;
    if (a.splits == 1) {
      if (ok && nblk > 0) {
        const float inv = 1.f / l;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t o[32];
          tmem_ld32(tmem_o + lane_sel + 32u * c, o, 0);
          tc_wait_ld();
          if (row_valid) {
            uint8_t* dst = reinterpret_cast<uint8_t*>(a.out) + 2 * ((int64_t)i * a.o_stride_tok + (int64_t)h * a.o_stride_head + 32 * c);
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              uint4 val;
              val.x = pack2<kBf16>(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv);
              val.y = pack2<kBf16>(__uint_as_float(o[e + 2]) * inv, __uint_as_float(o[e + 3]) * inv);
              val.z = pack2<kBf16>(__uint_as_float(o[e + 4]) * inv, __uint_as_float(o[e + 5]) * inv);
              val.w = pack2<kBf16>(__uint_as_float(o[e + 6]) * inv, __uint_as_float(o[e + 7]) * inv);
              *reinterpret_cast<uint4*>(dst + 2 * e) = val;
            }
          }
        }
        if (row_valid && a.lse != nullptr) a.lse[(size_t)h * a.n + i] = (m_used + log2f(l)) * kLn2;
      }
    } else {
      const size_t prow_idx = ((size_t)split * a.Hq + h) * a.n + i;
      if (ok && nblk > 0) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t o[32];
          tmem_ld32(tmem_o + lane_sel + 32u * c, o, 0);
          tc_wait_ld();
          if (row_valid) {
            float* dst = a.o_part + prow_idx * kHeadDim + 32 * c;
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              *reinterpret_cast<uint4*>(dst + e) = make_uint4(o[e], o[e + 1], o[e + 2], o[e + 3]);
          }
        }
      }
      if (row_valid) a.ml[prow_idx] = (ok && nblk > 0) ? make_float2(m_used, l) : make_float2(-INFINITY, 0.f);
    }
    tc_fence_before();
  }

  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// ---------------------------------------------------------------- host side ---------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool umma_supported(const seq_tree_attention_params& p) {
  if (p.dtype != SEQ_F16 && p.dtype != SEQ_BF16) return false;
  const int G = p.num_q_heads / p.num_kv_heads;
  if (G > kTileM || kTileM % G != 0) return false;
  return true;
}

int umma_default_splits(const seq_tree_attention_params& p) {
  const int G = p.num_q_heads / p.num_kv_heads;
  const int nodes_per_tile = kTileM / G;
  const int tiles = (p.n_tree + nodes_per_tile - 1) / nodes_per_tile;
  const int ctas = tiles * p.num_kv_heads;
  const int nblk = (p.prefix_len + p.n_tree + kBlockN - 1) / kBlockN;
  int splits = 148 / ctas;  // one CTA per SM: fill the machine in one wave when the tiles alone cannot
  if (splits < 1) splits = 1;
  if (splits > nblk) splits = nblk;
  if (splits > 32) splits = 32;
  return splits;
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
    cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)G, (cuuint64_t)p.n_tree, (cuuint64_t)p.num_kv_heads};
    cuuint64_t strides[3] = {(cuuint64_t)p.q_stride_head * 2, (cuuint64_t)p.q_stride_tok * 2,
                             (cuuint64_t)p.q_stride_head * 2 * G};
    cuuint32_t box[4] = {64, (cuuint32_t)G, (cuuint32_t)nodes_per_tile, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (encode(&q_map, dt, 4, const_cast<void*>(p.q), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return SEQ_ERR_CUDA;
  }
  for (int which = 0; which < 2; ++which) {
    // only the live rows [0, prefix_len + n_tree) are mapped: anything past them reads as zero
    cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)(p.prefix_len + p.n_tree), (cuuint64_t)p.num_kv_heads};
    cuuint64_t strides[2] = {(cuuint64_t)p.kv_stride_tok * 2, (cuuint64_t)p.kv_stride_head * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)kBlockN, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    if (encode(which == 0 ? &k_map : &v_map, dt, 3, const_cast<void*>(which == 0 ? p.k_cache : p.v_cache), dims,
               strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return SEQ_ERR_CUDA;
  }

  UmmaArgs a;
  a.n = p.n_tree; a.L = p.prefix_len; a.Hq = p.num_q_heads; a.Hkv = p.num_kv_heads; a.group = G;
  a.mask_wpr = p.mask_words_per_row; a.splits = splits; a.nodes_per_tile = nodes_per_tile; a.tiles = tiles;
  const float scale = p.softmax_scale > 0.f ? p.softmax_scale : 0.08838834764831845f;
  a.scale_log2 = scale * kLog2e;
  const uint32_t fmt = p.dtype == SEQ_BF16 ? 1u : 0u;
  // instruction descriptor: D fp32 (bit 4), A/B format (bits 7, 10), B major (bit 16), N>>3 (bit 17), M>>4 (bit 24)
  const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(kBlockN >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
  a.idesc_qk = idesc;
  a.idesc_pv = idesc | (1u << 16);
  a.mask_bits = p.mask_bits;
  a.out = p.out; a.o_stride_tok = p.o_stride_tok; a.o_stride_head = p.o_stride_head;
  a.lse = p.lse;
  SplitLayout sl = split_layout(p.workspace, splits, p.num_q_heads, p.n_tree);
  a.o_part = sl.o_part; a.ml = sl.ml;
  a.dev_status = p.dev_status;

  const size_t smem = sizeof(UmmaSmem) + 1024;
  dim3 grid(tiles, p.num_kv_heads, splits);
  if (p.dtype == SEQ_BF16) {
    SEQ_CUDA_OK(cudaFuncSetAttribute(tree_attention_umma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    tree_attention_umma_kernel<true><<<grid, kUmmaThreads, smem, stream>>>(q_map, k_map, v_map, a);
  } else {
    SEQ_CUDA_OK(cudaFuncSetAttribute(tree_attention_umma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    tree_attention_umma_kernel<false><<<grid, kUmmaThreads, smem, stream>>>(q_map, k_map, v_map, a);
  }
  SEQ_CUDA_OK(cudaGetLastError());
  if (splits > 1) return launch_combine_splits(p, splits, stream);
  return SEQ_OK;
}

}  // namespace seqtree
