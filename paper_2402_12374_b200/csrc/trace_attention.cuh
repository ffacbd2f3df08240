// Debug builds only (-DSEQ_TRACE): per-role timelines of the tensor-core attention kernel, one (tag, clock) event per
// 8-byte store, read back through seq_debug_utrace_dump() and seq_debug_cta_times().  Included by
// tree_attention_umma.cu alone (it defines device globals).  Without SEQ_TRACE the UTRACE calls compile to nothing.
#pragma once
namespace seqtree {

#ifndef SEQ_TRACE_ROW
#define SEQ_TRACE_ROW 128  // the row thread whose steps a trace build records
#endif
#ifdef SEQ_TRACE
// Debug builds only: per role (0 TMA, 1 MMA chain A, 2 rows, 3 MMA chain B) a list of (tag, clock) events of
// CTA (0, 0, 0), one 8-byte store each.  SEQ_TRACE_ROLES (bit per role) limits which roles record.
#ifndef SEQ_TRACE_ROLES
#define SEQ_TRACE_ROLES 15
#endif
#ifndef SEQ_TRACE_CTA
#define SEQ_TRACE_CTA 0
#endif

__device__ unsigned long long g_utrace[4][2048];
__device__ unsigned long long g_cta_times[1024][2];
__device__ __forceinline__ unsigned long long gtimer() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
#define UTRACE(role, tag)                                                       \
  do {                                                                          \
    if (((SEQ_TRACE_ROLES) >> (role)) & 1) {                                    \
      if (blockIdx.x == (SEQ_TRACE_CTA) && blockIdx.y == 0 && blockIdx.z == 0 && utrace_i < 2047) \
        g_utrace[role][++utrace_i] = ((unsigned long long)(tag) << 56) | ((unsigned long long)clock64() & 0xFFFFFFFFFFFFFFull); \
    }                                                                           \
  } while (0)
#else
#define UTRACE(role, tag) do { } while (0)
#endif

}  // namespace seqtree

#ifdef SEQ_TRACE
extern "C" int seq_debug_cta_times(unsigned long long* host_out) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(host_out, seqtree::g_cta_times, sizeof(unsigned long long) * 2048);
  return 0;
}
extern "C" int seq_debug_utrace_dump(unsigned long long* host_out) {
  cudaDeviceSynchronize();
  cudaMemcpyFromSymbol(host_out, seqtree::g_utrace, sizeof(unsigned long long) * 4 * 2048);
  static unsigned long long zeros[4 * 2048];
  cudaMemcpyToSymbol(seqtree::g_utrace, zeros, sizeof(zeros));
  return 0;
}
#endif
