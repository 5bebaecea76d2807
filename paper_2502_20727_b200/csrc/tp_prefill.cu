// Rank mode (one shard per rank, Sec. 3), prompts: shot two of the two-shot exchange that stands for a shard sum
// the block keeps (a TP block: Y_r after o_proj and Z_r after down; an SPD block: Y_r + Z_r after down, Sec. 4.1.1).
//
// Shot one is the tail of the projection (PRE_SCATTER in gemm_prefill.cu): the 128-token tiles of a launch are dealt
// round-robin to the ranks, and every rank stores its fp32 partial rows of a tile into the OWNER's receive plane.
// Here the owner waits - with a time limit - until the flag words of a tile show this step for every column tile and
// source rank, adds the T planes in rank order (so every rank ends up with the same bits), adds the residual, and
// writes the finished rows - fp32 residual stream, gain-scaled bf16 operand of the next GEMM, row sums of squares -
// into EVERY rank's planes (plain peer stores: an all-gather), then publishes the step in every rank's gather flags.
// A last small kernel on each rank waits for the gather flags of all tiles, so that the next projection (a
// dependent launch) finds its whole operand in place.  Nothing waits without a limit: a wait that runs out sets
// error bit 8, and the rest of the call finds the bit and gives up at once.
#include "tp_prefill.cuh"

namespace spd {

namespace {

__device__ __forceinline__ unsigned ld_acquire_sys_u32(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_sys_u32(unsigned *p, unsigned v)
{
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// One warp polls `n` flag words until each shows `step` (or later).  false: gave up (error bit set).
__device__ __forceinline__ bool wait_flags(const unsigned *flags, int n, unsigned step, unsigned long long limit_ns, int *err)
{
    const int lane = threadIdx.x & 31;
    const unsigned long long t0 = timer_ns();
    for (;;) {
        bool done = true;
        for (int e = lane; e < n; e += 32)
            if ((int)(ld_acquire_sys_u32(flags + e) - step) < 0) done = false;
        if (__all_sync(0xffffffffu, done)) return true;
        if ((*(volatile int *)err & ERR_PEER_TIMEOUT) || timer_ns() - t0 > limit_ns) {
            if (lane == 0) atomicOr(err, ERR_PEER_TIMEOUT);
            return false;
        }
    }
}

constexpr int ROWS_PER_BLOCK = 8; // one warp per token row

// grid: (owned tiles) x (128 / ROWS_PER_BLOCK) blocks of 8 warps.
__global__ void __launch_bounds__(256) tp_finish_kernel(TpFinishArgs a)
{
    pdl_launch_dependents();
    if (threadIdx.x == 0) stamp_entry(a.stamp);
    pdl_wait();
    __shared__ int sm_ok;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int slot = blockIdx.x / (128 / ROWS_PER_BLOCK), sub = blockIdx.x % (128 / ROWS_PER_BLOCK);
    const int tile128 = slot * a.T + a.me;
    const unsigned step = *a.step;
    // every source's rows of this tile, all column tiles
    if (warp == 0) {
        const bool ok = wait_flags(a.sflags + (long)slot * a.n_tiles * a.T, a.n_tiles * a.T, step, a.wait_ns, a.err);
        if (lane == 0) sm_ok = ok ? 1 : 0;
    }
    __syncthreads();
    if (!sm_ok) return;
    const int r = sub * ROWS_PER_BLOCK + warp, m = tile128 * 128 + r;
    if (m < a.M) {
        const long row = (long)m * a.H;
        float ssq = 0.f;
        for (int n = 4 * lane; n < a.H; n += 128) {
            float4 x = *(const float4 *)(a.res_in + row + n);
            for (int s = 0; s < a.T; ++s) { // rank order: the same sum on every rank
                const float4 y = __ldcg((const float4 *)(a.rx + (long)s * a.src_stride + (((long)slot * 128 + r) * a.H + n) * 4));
                x.x += y.x; x.y += y.y; x.z += y.z; x.w += y.w;
            }
            ssq += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
            float4 gn = make_float4(1.f, 1.f, 1.f, 1.f);
            if (a.gain) {
                const uint2 u = *(const uint2 *)((const bf16 *)a.gain + n);
                const float2 g0 = __bfloat1622float2(*(const __nv_bfloat162 *)&u.x), g1 = __bfloat1622float2(*(const __nv_bfloat162 *)&u.y);
                gn = make_float4(g0.x, g0.y, g1.x, g1.y);
            }
            const __nv_bfloat162 h0 = __floats2bfloat162_rn(x.x * gn.x, x.y * gn.y), h1 = __floats2bfloat162_rn(x.z * gn.z, x.w * gn.w);
            uint2 hv;
            hv.x = *(const uint32_t *)&h0;
            hv.y = *(const uint32_t *)&h1;
            for (int i = 0; i < a.T; ++i) { // own planes first, then the peers round the ring
                const int d = a.me + i < a.T ? a.me + i : a.me + i - a.T;
                *(float4 *)(a.region[d] + a.off_res_out + (row + n) * 4) = x;
                *(uint2 *)(a.region[d] + a.off_hg + (row + n) * 2) = hv;
            }
        }
        ssq = warp_sum(ssq);
        if (lane == 0)
            for (int d = 0; d < a.T; ++d) *(float *)(a.region[d] + a.off_ss + (long)m * 4) = ssq;
    }
    // the block's rows are on their way to every rank: publish
    __syncthreads();
    if ((int)threadIdx.x < a.T)
        st_release_sys_u32((unsigned *)(a.region[threadIdx.x] + a.off_gflags) + (long)tile128 * (128 / ROWS_PER_BLOCK) + sub, step);
    if (threadIdx.x == 0) stamp_exit(a.stamp);
}

__global__ void __launch_bounds__(32) tp_gather_wait_kernel(const unsigned *gflags, int n_flags, const unsigned *step, unsigned long long wait_ns,
                                                            int *err)
{
    pdl_launch_dependents();
    pdl_wait();
    wait_flags(gflags, n_flags, *step, wait_ns, err);
}

} // namespace

int tp_finish_blocks_per_tile() { return 128 / ROWS_PER_BLOCK; }

cudaError_t launch_tp_finish(const TpFinishArgs &a, cudaStream_t st)
{
    if (a.M <= 0) return cudaSuccess;
    if (a.H % 4 || a.T < 1 || a.T > TP_MAX_RANKS || !a.step || !a.err) return cudaErrorInvalidValue;
    const int tiles = (a.M + 127) / 128;
    const int owned = a.me < tiles ? (tiles - a.me + a.T - 1) / a.T : 0;
    if (owned == 0) return cudaSuccess;
    return launch_kernel(tp_finish_kernel, dim3(owned * (128 / ROWS_PER_BLOCK)), dim3(256), 0, st, 0, a);
}

cudaError_t launch_tp_gather_wait(const unsigned *gflags, int M, const unsigned *step, unsigned long long wait_ns, int *err, cudaStream_t st)
{
    if (M <= 0) return cudaSuccess;
    const int tiles = (M + 127) / 128;
    return launch_kernel(tp_gather_wait_kernel, dim3(1), dim3(32), 0, st, 0, gflags, tiles * (128 / ROWS_PER_BLOCK), step, wait_ns, err);
}

} // namespace spd
