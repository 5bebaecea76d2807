// Storage and host access of the optional in-kernel timeline (see trace.cuh).
#include "trace.cuh"

#include <cuda_runtime.h>

#ifdef SPD_TRACE
namespace spd {
__device__ unsigned long long g_trace_rec[2 * TRACE_CAP];
__device__ unsigned int g_trace_n;
} // namespace spd

// Copies up to max_records (time_ns, meta) pairs to `out`, resets the log, returns the count
// (or -1 on a CUDA error).  Only present in a -DSPD_TRACE build; not part of the public header.
extern "C" long spd_trace_read(unsigned long long *out, long max_records)
{
    unsigned int n = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    if (cudaMemcpyFromSymbol(&n, spd::g_trace_n, sizeof(n)) != cudaSuccess) return -1;
    if (n > spd::TRACE_CAP) n = spd::TRACE_CAP;
    if ((long)n > max_records) n = (unsigned)max_records;
    if (out && n && cudaMemcpyFromSymbol(out, spd::g_trace_rec, (size_t)n * 16) != cudaSuccess) return -1;
    unsigned int zero = 0;
    if (cudaMemcpyToSymbol(spd::g_trace_n, &zero, sizeof(zero)) != cudaSuccess) return -1;
    return (long)n;
}
#endif
