// Per-block strategy (Sec. 4.2): the progressive sync-sensitivity scan of Sec. 4.2.1 run on the
// library's own forward pass, with the mean squared difference from the all-TP output standing in
// for perplexity (there is no LM head on this path), and the block selection of Algorithm 1.
#include "../../include/spd.h"
#include "common.cuh"

#include <algorithm>
#include <vector>

namespace spd {

// Fixed-shape, fixed-order reduction: block b adds elements b*chunk .. of (a - r)^2 into part[b].
template <typename T>
__global__ void __launch_bounds__(256) sq_diff_kernel(const T *a, const T *r, long n, long chunk, float *part)
{
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float red[8];
    const long lo = (long)blockIdx.x * chunk, hi = lo + chunk < n ? lo + chunk : n;
    float acc = 0.f;
    for (long i = lo + threadIdx.x; i < hi; i += blockDim.x) {
        const float d = to_f<T>(a[i]) - to_f<T>(r[i]);
        acc = fmaf(d, d, acc);
    }
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += red[w];
        part[blockIdx.x] = t;
    }
}

cudaError_t launch_sq_diff(const void *a, const void *r, long n, int dtype_bf16, float *part, int n_blocks, cudaStream_t st)
{
    const long chunk = (n + n_blocks - 1) / n_blocks;
    if (dtype_bf16) return launch_kernel(sq_diff_kernel<bf16>, dim3(n_blocks), dim3(256), 0, st, 0, (const bf16 *)a, (const bf16 *)r, n, chunk, part);
    return launch_kernel(sq_diff_kernel<float>, dim3(n_blocks), dim3(256), 0, st, 0, (const float *)a, (const float *)r, n, chunk, part);
}

} // namespace spd

extern "C" int spd_alg1_plan(const double *sensitivity, int32_t n_blocks, int32_t n_spd, double tau1, double tau2,
                             uint8_t *sync_mask, uint8_t *tier)
{
    if (!sensitivity || !sync_mask || !tier) return SPD_ENULL;
    if (n_blocks < 1 || n_spd < 0 || n_spd > n_blocks || !(tau1 <= tau2)) return SPD_EINVAL;
    // B: block indices in ascending order of S (ties: lower index first)
    std::vector<int> order(n_blocks);
    for (int i = 0; i < n_blocks; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return sensitivity[a] < sensitivity[b]; });
    for (int i = 0; i < n_blocks; ++i) { sync_mask[i] = 1; tier[i] = SPD_TIER_TP; }
    for (int i = 0; i < n_spd; ++i) {
        const int blk = order[i];
        sync_mask[blk] = 0;
        tier[blk] = sensitivity[blk] <= tau1 ? SPD_TIER_ISB : (sensitivity[blk] <= tau2 ? SPD_TIER_SB : SPD_TIER_ESB);
    }
    return SPD_OK;
}
