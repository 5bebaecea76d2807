// spd_gemm_bf16_sum_static: the split-K projection GEMM for callers that cannot allocate device
// memory.  The K-split partial planes, which every other path keeps in caller-provided
// memory, live in one fixed array that is part of the loaded library image.
#include "../../include/spd.h"
#include "common.cuh"
#include "gemm_tc.cuh"

#include <initializer_list>
#include <mutex>

using namespace spd;

namespace {

constexpr size_t SCRATCH_FLOATS = SPD_STATIC_SCRATCH_BYTES / sizeof(float);
constexpr int MAX_DEVICES = 64;

// Partial planes [splits][M][batches*N].  On the host this name is only a handle for
// cudaGetSymbolAddress; kernels receive the address that call returns.
static __device__ __align__(256) float g_static_planes[SCRATCH_FLOATS];

std::mutex g_setup_lock;
float *g_planes_of_device[MAX_DEVICES] = {};

// c[m][col] = sum over the split planes, in split order (deterministic).
__global__ void __launch_bounds__(256) sum_planes_kernel(const float *planes, float *c, long plane_elems, int splits)
{
    pdl_launch_dependents();
    pdl_wait();
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= plane_elems) return;
    float acc = 0.f;
    for (int s = 0; s < splits; ++s) acc += planes[(long)s * plane_elems + i];
    c[i] = acc;
}

} // namespace

extern "C" int spd_gemm_bf16_sum_static(const void *a, const void *w, float *c, int32_t M, int32_t N, int32_t K,
                                        int32_t batches, int32_t a_batched, int32_t splits, int32_t swap,
                                        int32_t *err_flag, void *stream)
{
    if (!a || !w || !c || !err_flag) return SPD_ENULL;
    if (M < 1 || N < 1 || K < 8 || K % 8 || batches < 1 || splits < 1 || splits > (K + 63) / 64) return SPD_EINVAL;
    // factor by factor, so that no product of the four 32-bit sizes can wrap before it is compared
    size_t room = SCRATCH_FLOATS;
    for (const int32_t f : {M, batches, N, splits}) {
        if ((size_t)f > room) return SPD_EWORKSPACE;
        room /= (size_t)f;
    }
    const size_t plane_elems = (size_t)M * (size_t)batches * (size_t)N;

    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { note_cuda_error(e); return SPD_ECUDA; }
    if (dev < 0 || dev >= MAX_DEVICES) { note_cuda_error(cudaErrorInvalidDevice); return SPD_ECUDA; }
    float *planes = nullptr;
    {
        // once per device, with that device current: resolve the array's device address
        std::lock_guard<std::mutex> hold(g_setup_lock);
        if (!g_planes_of_device[dev]) {
            float *p = nullptr;
            e = cudaGetSymbolAddress((void **)&p, g_static_planes);
            if (e != cudaSuccess || !p) { note_cuda_error(e != cudaSuccess ? e : cudaErrorInvalidSymbol); return SPD_ECUDA; }
            g_planes_of_device[dev] = p;
        }
        planes = g_planes_of_device[dev];
    }

    TcMap wm, am;
    const int tbox = tc_token_box(swap != 0, M);
    if (make_operand_map(&wm, w, K, N, batches, K, (long)N * K, 128)) return SPD_EINVAL;
    if (make_operand_map(&am, a, K, M, a_batched ? batches : 1, K, (long)M * K, tbox)) return SPD_EINVAL;
    TcGemmArgs g{};
    g.C = planes; g.ldc = (long)batches * N; g.c_batch_stride = N; g.c_split_stride = (long)plane_elems;
    g.t_rows = M; g.w_rows[0] = N; g.batches = batches; g.w_batched = batches > 1; g.t_batched = a_batched && batches > 1;
    g.num_kb = (K + 63) / 64; g.splits = splits; g.err = err_flag;
    const TcMap *wmaps[1] = {&wm};
    cudaStream_t st = (cudaStream_t)stream;
    if ((e = launch_gemm_tc(wmaps, 1, am, g, swap != 0, st)) != cudaSuccess) { note_cuda_error(e); return SPD_ECUDA; }
    // Every element the sum reads was written by the launch above, so nothing has to be cleared.
    const unsigned blocks = (unsigned)((plane_elems + 255) / 256);
    e = launch_kernel(sum_planes_kernel, dim3(blocks), dim3(256), 0, st, 0, (const float *)planes, c, (long)plane_elems, (int)splits);
    if (e != cudaSuccess) { note_cuda_error(e); return SPD_ECUDA; }
    return SPD_OK;
}
