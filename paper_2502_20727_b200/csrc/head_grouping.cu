// SPD-aware attention head grouping (Sec. 4.2.4): the device kernels that measure the heads
// (attention scores per head, pairwise Euclidean distances of Eq. 2) and the host searches (head
// scattering, Eq. 2; MLP matching, Eq. 3).  The MLP-output norms of Eq. 3 come from the library's
// own prefill kernels (spd_api.cu).
#include "../../include/spd.h"
#include "common.cuh"

#include <algorithm>
#include <math.h>
#include <numeric>
#include <vector>

namespace spd {

// sigma[h][b][i][j] = softmax_j(q_{b,i,h} . k_{b,j,kv(h)} / sqrt(d)) for j <= i, 0 above the diagonal.
// One warp per (token m = b*S + i, head h); keys in steps of 32, K rows from the paged cache.
template <typename T>
__global__ void __launch_bounds__(128) head_scores_kernel(const T *q, const T *k_pages, PageTable pt, int b0, int S, int n_seq, int n_q_heads,
                                                          int d, float *sigma, int *err)
{
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ float sc[]; // [4 warps][S]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m = blockIdx.x * 4 + warp, h = blockIdx.y;
    if (m >= n_seq * S) return;
    const int bi = m / S, i = m % S, kvh = h / (n_q_heads / pt.n_kv_heads);
    float *row = sc + warp * S;
    const T *qp = q + ((long)m * n_q_heads + h) * d;
    const float scale = rsqrtf((float)d);
    float mx = -INFINITY;
    for (int j = lane; j <= i; j += 32) {
        int page = pt.block_table[(long)(b0 + bi) * pt.max_pages + j / pt.block];
        if (page < 0 || page >= pt.n_pages) { atomicOr(err, ERR_PAGE_RANGE); page = 0; }
        const T *kp = k_pages + (((long)page * pt.n_kv_heads + kvh) * pt.block + j % pt.block) * d;
        float s = 0.f;
        for (int e = 0; e < d; ++e) s = fmaf(to_f<T>(qp[e]), to_f<T>(kp[e]), s);
        s *= scale;
        row[j] = s;
        mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    float den = 0.f;
    for (int j = lane; j <= i; j += 32) { const float p = expf(row[j] - mx); row[j] = p; den += p; }
    den = warp_sum(den);
    float *out = sigma + (((long)h * n_seq + bi) * S + i) * S;
    for (int j = lane; j < S; j += 32) out[j] = j <= i ? row[j] / den : 0.f;
}

template <typename T>
cudaError_t launch_head_scores(const void *q, const void *k_pages, PageTable pt, int b0, int S, int n_seq, int n_q_heads, int d,
                               float *sigma, int *err, cudaStream_t st)
{
    dim3 grid((n_seq * S + 3) / 4, n_q_heads);
    return launch_kernel(head_scores_kernel<T>, grid, dim3(128), (size_t)4 * S * sizeof(float), st, 0, (const T *)q, (const T *)k_pages, pt,
                         b0, S, n_seq, n_q_heads, d, sigma, err);
}
template cudaError_t launch_head_scores<bf16>(const void *, const void *, PageTable, int, int, int, int, int, float *, int *, cudaStream_t);
template cudaError_t launch_head_scores<float>(const void *, const void *, PageTable, int, int, int, int, int, float *, int *, cudaStream_t);

// dist[a][b] = || sigma_a - sigma_b ||_2 over the len elements of a head (Eq. 2's d); fixed-order reduction.
__global__ void __launch_bounds__(256) head_distance_kernel(const float *sigma, long len, int n_heads, float *dist)
{
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float red[8];
    const int a = blockIdx.x, b = blockIdx.y;
    const float *pa = sigma + (long)a * len, *pb = sigma + (long)b * len;
    float acc = 0.f;
    for (long i = threadIdx.x; i < len; i += blockDim.x) { const float dd = pa[i] - pb[i]; acc = fmaf(dd, dd, acc); }
    acc = warp_sum(acc);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += red[w];
        dist[(long)a * n_heads + b] = sqrtf(t);
    }
}

cudaError_t launch_head_distance(const float *sigma, long len, int n_heads, float *dist, cudaStream_t st)
{
    return launch_kernel(head_distance_kernel, dim3(n_heads, n_heads), dim3(256), 0, st, 0, sigma, len, n_heads, dist);
}

} // namespace spd

namespace {

// Sum of pairwise distances inside each set (the objective of Eq. 2 summed over the devices).
double scatter_objective(const std::vector<double> &D, int n, const std::vector<int> &dev)
{
    double tot = 0.0;
    for (int a = 0; a < n; ++a)
        for (int b = a + 1; b < n; ++b)
            if (dev[a] == dev[b]) tot += D[(size_t)a * n + b];
    return tot;
}

// Exhaustive search over the partitions of n units into T sets of n/T: unit u goes to a set that is
// not full; a new (empty) set may only be opened in index order, so every partition is seen once.
void scatter_exact(const std::vector<double> &D, int n, int T, int u, std::vector<int> &dev, std::vector<int> &fill, int opened,
                   double cur, double &best, std::vector<int> &best_dev)
{
    if (u == n) {
        if (cur > best) { best = cur; best_dev = dev; }
        return;
    }
    const int cap = n / T;
    for (int s = 0; s < opened + 1 && s < T; ++s) {
        if (fill[s] == cap) continue;
        double add = 0.0;
        for (int v = 0; v < u; ++v)
            if (dev[v] == s) add += D[(size_t)v * n + u];
        dev[u] = s;
        ++fill[s];
        scatter_exact(D, n, T, u + 1, dev, fill, s == opened ? opened + 1 : opened, cur + add, best, best_dev);
        --fill[s];
    }
    dev[u] = -1;
}

} // namespace

extern "C" int spd_head_scatter(const float *dist, int32_t n_heads, int32_t heads_per_unit, int32_t T, int32_t *device_of_unit,
                                double *objective)
{
    if (!dist || !device_of_unit) return SPD_ENULL;
    if (n_heads < 1 || heads_per_unit < 1 || n_heads % heads_per_unit || T < 1) return SPD_EINVAL;
    const int n = n_heads / heads_per_unit;
    if (n % T) return SPD_EINVAL;
    // a unit = the query heads of one KV head (they cannot be separated); distance of units = sum over their head pairs
    std::vector<double> D((size_t)n * n, 0.0);
    for (int a = 0; a < n; ++a)
        for (int b = 0; b < n; ++b) {
            double s = 0.0;
            for (int x = 0; x < heads_per_unit; ++x)
                for (int y = 0; y < heads_per_unit; ++y)
                    s += 0.5 * ((double)dist[(size_t)(a * heads_per_unit + x) * n_heads + b * heads_per_unit + y] +
                                (double)dist[(size_t)(b * heads_per_unit + y) * n_heads + a * heads_per_unit + x]);
            D[(size_t)a * n + b] = a == b ? 0.0 : s;
        }
    std::vector<int> dev(n, -1);
    double best = -1.0;
    if (n <= 12) {
        std::vector<int> cur(n, -1), fill(T, 0);
        scatter_exact(D, n, T, 0, cur, fill, 0, 0.0, best, dev);
    } else {
        // greedy start (contiguous sets), then pairwise swaps between sets while one improves the objective
        const int cap = n / T;
        for (int u = 0; u < n; ++u) dev[u] = u / cap;
        best = scatter_objective(D, n, dev);
        bool improved = true;
        for (int round = 0; improved && round < 1000; ++round) {
            improved = false;
            for (int a = 0; a < n; ++a)
                for (int b = a + 1; b < n; ++b) {
                    if (dev[a] == dev[b]) continue;
                    // gain of swapping a and b: their links to the other members of both sets
                    double gain = 0.0;
                    for (int v = 0; v < n; ++v) {
                        if (v == a || v == b) continue;
                        if (dev[v] == dev[a]) gain += D[(size_t)b * n + v] - D[(size_t)a * n + v];
                        if (dev[v] == dev[b]) gain += D[(size_t)a * n + v] - D[(size_t)b * n + v];
                    }
                    if (gain > 1e-12 * (1.0 + fabs(best))) {
                        std::swap(dev[a], dev[b]);
                        best += gain;
                        improved = true;
                    }
                }
        }
        best = scatter_objective(D, n, dev);
    }
    for (int u = 0; u < n; ++u) device_of_unit[u] = dev[u];
    if (objective) *objective = best;
    return SPD_OK;
}

extern "C" int spd_mlp_match(const double *norms, int32_t T, int32_t *mlp_of_device, double *objective)
{
    if (!norms || !mlp_of_device) return SPD_ENULL;
    if (T < 1 || T > 8) return SPD_EINVAL;
    // all T! matchings <A_i, MLP_m>, the one with the largest sum of output norms wins (first in lexicographic order on ties)
    std::vector<int> perm(T), best_perm(T);
    std::iota(perm.begin(), perm.end(), 0);
    double best = -1.0;
    do {
        double s = 0.0;
        for (int i = 0; i < T; ++i) s += norms[(size_t)i * T + perm[i]];
        if (s > best) { best = s; best_perm = perm; }
    } while (std::next_permutation(perm.begin(), perm.end()));
    for (int i = 0; i < T; ++i) mlp_of_device[i] = best_perm[i];
    if (objective) *objective = best;
    return SPD_OK;
}
