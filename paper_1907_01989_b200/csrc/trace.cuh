// Optional timeline instrumentation (compiled only with -DGI_TRACE, never in the shipped
// library): the leader of each warp role stores the global nanosecond timer at a few events per
// CTA, and a debug entry point copies the table to the host.
#pragma once

#ifdef GI_TRACE
#define GI_TRACE_CTAS 1024
#define GI_TRACE_EVENTS 12
#define GI_TRACE_TABLE(name) __device__ unsigned long long name[GI_TRACE_CTAS * GI_TRACE_EVENTS]
#define GI_TRACE_EVENT(table, ev)                                                       \
  do {                                                                                  \
    if (blockIdx.x < GI_TRACE_CTAS) {                                                   \
      unsigned long long t_;                                                            \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                            \
      table[blockIdx.x * GI_TRACE_EVENTS + (ev)] = t_;                                  \
    }                                                                                   \
  } while (0)
#else
#define GI_TRACE_TABLE(name)
#define GI_TRACE_EVENT(table, ev) ((void)0)
#endif
