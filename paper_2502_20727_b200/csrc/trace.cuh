// Optional in-kernel timeline (compiled in only with -DSPD_TRACE; the regular library has none
// of it).  One thread per thread block stamps the global nanosecond timer at a few fixed points;
// the records land in a fixed device array that spd_trace_read copies to the host.
#pragma once
#include <stdint.h>

namespace spd {

enum TraceEvent : int { TR_START = 0, TR_DEP_DONE = 1, TR_MAIN_DONE = 2, TR_ARRIVED = 3, TR_END = 4 };
enum TraceKernel : int { TRK_QKV = 0, TRK_OPROJ = 1, TRK_GATEUP = 2, TRK_DOWN = 3, TRK_ATTN = 4, TRK_PROLOGUE = 5, TRK_PREFILL = 8 /* + PreEpilogue */ };

#ifdef SPD_TRACE
constexpr unsigned TRACE_CAP = 1u << 21;
extern __device__ unsigned long long g_trace_rec[2 * TRACE_CAP];
extern __device__ unsigned int g_trace_n;

__device__ __forceinline__ void trace(int kernel, int event)
{
    unsigned long long t;
    unsigned smid;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    const unsigned i = atomicAdd(&g_trace_n, 1u);
    if (i < TRACE_CAP) {
        const unsigned cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
        g_trace_rec[2 * i] = t;
        g_trace_rec[2 * i + 1] = ((unsigned long long)kernel << 56) | ((unsigned long long)event << 48) |
                                 ((unsigned long long)(smid & 0xffff) << 32) | cta;
    }
}
#define SPD_TRACE_EVENT(kernel, event) ::spd::trace((kernel), (event))
#else
#define SPD_TRACE_EVENT(kernel, event) ((void)0)
#endif

} // namespace spd
