// Debug builds only (-DSEQ_TRACE): a timeline of (tag, nanosecond clock) events recorded by one thread of a kernel,
// read back through seq_debug_walk_trace().  Compiles to nothing otherwise.
#pragma once
#ifdef SEQ_TRACE
namespace seqtree {
__device__ unsigned long long g_wtrace[512];
__device__ int g_wtrace_n;
__device__ __forceinline__ unsigned long long wtimer() { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); return t; }
}  // namespace seqtree
#define WTRACE_DECL int wtrace_i = 0
#define WTRACE(cond, tag)                                                                                  \
  do {                                                                                                     \
    if ((cond) && wtrace_i < 255) {                                                                        \
      seqtree::g_wtrace[2 * wtrace_i] = (tag); seqtree::g_wtrace[2 * wtrace_i + 1] = seqtree::wtimer();    \
      seqtree::g_wtrace_n = ++wtrace_i;                                                                    \
    }                                                                                                      \
  } while (0)
#else
#define WTRACE_DECL do { } while (0)
#define WTRACE(cond, tag) do { } while (0)
#endif
