// CUDA-core GEMM used for float32 storage (tensor-core tf32 cannot hold the 1e-4 parity
// bound) and as the bring-up path.  C[z][m][s*Ns + n] = sum_{k in split z} A_s[m][k] W[s*Ns + n][k].
// Shards (s) select both the rows of W and, when a_shard_stride != 0, the A operand: that is
// the shard-batched gate/up projection of an SPD block, where every emulated device has its
// own MLP input.  Splits (z) cut K; for the row-split o_proj of an SPD block the cuts fall on
// shard boundaries and the planes are the per-device partial outputs Y_i, never summed.
#include "common.cuh"

namespace spd {

constexpr int BM = 64, BN = 64, BK = 16;

template <typename T>
__global__ void __launch_bounds__(256) gemm_simt_kernel(GemmProblem p, int tiles_per_shard)
{
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float As[BK][BM + 4];
    __shared__ float Ws[BK][BN + 4];
    const int shard = blockIdx.x / tiles_per_shard;
    const int n0 = (blockIdx.x % tiles_per_shard) * BN; // within the shard
    const int m0 = blockIdx.y * BM;
    const int z = blockIdx.z;
    const int k_begin = z * p.k_per_split;
    const int k_end = min(p.K, k_begin + p.k_per_split);
    const T *A = (const T *)p.A + (long)shard * p.a_shard_stride;
    const T *W = (const T *)p.W + (long)shard * p.n_per_shard * p.ldw;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    float acc[4][4] = {};

    for (int k0 = k_begin; k0 < k_end; k0 += BK) {
        // each thread loads 4 elements of each tile: row = idx / BK, col = idx % BK
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int idx = threadIdx.x + i * 256;
            int r = idx / BK, c = idx % BK;
            int k = k0 + c;
            float av = 0.f, wv = 0.f;
            if (k < k_end) {
                if (m0 + r < p.M) av = to_f<T>(A[(long)(m0 + r) * p.lda + k]);
                if (n0 + r < p.n_per_shard) wv = to_f<T>(W[(long)(n0 + r) * p.ldw + k]);
            }
            As[c][r] = av;
            Ws[c][r] = wv;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            float a[4], w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; w[i] = Ws[k][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
        }
        __syncthreads();
    }
    float *C = p.C + (long)z * p.c_split_stride;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + ty * 4 + i;
        if (m >= p.M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int n = n0 + tx * 4 + j;
            if (n < p.n_per_shard) C[(long)m * p.ldc + (long)shard * p.n_per_shard + n] = acc[i][j];
        }
    }
}

template <typename T> cudaError_t launch_gemm_simt(const GemmProblem &p, cudaStream_t st)
{
    if (p.M <= 0 || p.n_per_shard <= 0) return cudaSuccess;
    int tiles_per_shard = (p.n_per_shard + BN - 1) / BN;
    dim3 grid(tiles_per_shard * p.n_shards, (p.M + BM - 1) / BM, p.splits);
    return launch_kernel(gemm_simt_kernel<T>, grid, dim3(256), 0, st, 0, p, tiles_per_shard);
}
template cudaError_t launch_gemm_simt<float>(const GemmProblem &, cudaStream_t);
template cudaError_t launch_gemm_simt<bf16>(const GemmProblem &, cudaStream_t);

} // namespace spd
