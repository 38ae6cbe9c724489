// Kernels of the batched fixed-point Pong step for sm_100a.
//
//   k_reset            state planes <- reset(seed, env, 0); optional initial obs
//   k_reset_pixels     reset frame into all four ring slots
//   k_rollout_vector   one thread per env, state in registers across T steps,
//                      streams obs / reward / done to HBM
//   k_rollout_pixels   one thread per env for the physics, one warp per frame
//                      for the rasteriser; frames are staged in shared memory
//                      and leave through bulk async copies (16-byte granules)
//   k_fill_actions     action bytes that reproduce the Philox modes
//
// No kernel waits on another block, on a flag or on an mbarrier; the only
// blocking instructions are __syncthreads and cp.async.bulk.wait_group.
#include "pong_kernels.cuh"

namespace pong {

// ---- helpers --------------------------------------------------------------------

__device__ __forceinline__ void flush_tally(const Tally &t, long long *stats)
{
    const int ep = __reduce_add_sync(0xffffffffu, t.episodes);
    if (ep == 0) return;  // warp-uniform
    const int rs = __reduce_add_sync(0xffffffffu, t.sum_return);
    const int ls = __reduce_add_sync(0xffffffffu, t.sum_length);
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(reinterpret_cast<unsigned long long *>(stats + 0), (unsigned long long)(long long)ep);
        atomicAdd(reinterpret_cast<unsigned long long *>(stats + 1), (unsigned long long)(long long)rs);
        atomicAdd(reinterpret_cast<unsigned long long *>(stats + 2), (unsigned long long)(long long)ls);
    }
}

template <int MODE>
__device__ __forceinline__ int pick_action(uint32_t word, const Env &e, const uint8_t *act,
                                           int const_action)
{
    if (MODE == 0) return uniform_action(word);
    if (MODE == 1) return sticky_repeat(word) ? e.prev : uniform_action(word);
    if (MODE == 2) return decode_action_byte(*act, e.prev);
    return const_action;
}

// ---- reset --------------------------------------------------------------------------

__global__ void __launch_bounds__(128) k_reset(const LaunchArgs a)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= a.n) return;
    Env e;
    reset_env(e, a.env_id_base + (uint32_t)n, 0u, a.rk);
    store_env(e, a.plane0, a.plane1, n);
    if (a.obs != nullptr) {
        float2 *o = reinterpret_cast<float2 *>(a.obs + (size_t)n * 6);
        o[0] = make_float2(scale_obs(e.bx), scale_obs(e.by));
        o[1] = make_float2(scale_obs(e.vx), scale_obs(e.vy));
        o[2] = make_float2(scale_obs(e.apy), scale_obs(e.opy));
    }
}

// ---- vector rollout -----------------------------------------------------------------

constexpr int kVecBlock = 64;

// MODE: action source.  FS: compile-time frameskip (0 = run-time value).
// FULL: t0 and T are multiples of 4, so every Philox block serves 4 steps.
template <int MODE, int FS, bool FULL>
__global__ void __launch_bounds__(kVecBlock) k_rollout_vector(const __grid_constant__ LaunchArgs a)
{
    const int n = blockIdx.x * kVecBlock + threadIdx.x;
    const bool valid = n < a.n;
    Tally tally = {0, 0, 0};
    if (valid) {
        Env e;
        load_env(e, a.plane0, a.plane1, n);
        const uint32_t env_id = a.env_id_base + (uint32_t)n;
        const unsigned long long t_begin = a.t0, t_end = a.t0 + (unsigned long long)a.T;
        const size_t stride = (size_t)a.n;
        float2 *obs = reinterpret_cast<float2 *>(a.obs + (size_t)n * 6);
        float *rew = a.reward + n;
        uint8_t *dn = a.done + n;
        const uint8_t *act = MODE == 2 ? a.actions + n : nullptr;

        for (unsigned long long g = t_begin >> 2; g <= (t_end - 1) >> 2; ++g) {
            uint32_t w[4] = {0u, 0u, 0u, 0u};
            if (MODE <= 1) action_words(g, env_id, a.rk, w);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const unsigned long long tt = g * 4 + j;
                if (FULL || (tt >= t_begin && tt < t_end)) {
                    const int action = pick_action<MODE>(w[j], e, act, a.const_action);
                    bool done;
                    const int r = agent_step<FS>(e, action, a.frameskip, env_id, a.rk, tally, done);
                    obs[0] = make_float2(scale_obs(e.bx), scale_obs(e.by));
                    obs[1] = make_float2(scale_obs(e.vx), scale_obs(e.vy));
                    obs[2] = make_float2(scale_obs(e.apy), scale_obs(e.opy));
                    *rew = (float)r;
                    *dn = done ? 1 : 0;
                    obs += stride * 3;
                    rew += stride;
                    dn += stride;
                    if (MODE == 2) act += stride;
                }
            }
        }
        store_env(e, a.plane0, a.plane1, n);
    }
    flush_tally(tally, a.stats);
}

template <int MODE, int FS>
static void launch_vec_full(const LaunchArgs &a, bool full, cudaStream_t s)
{
    const int grid = (a.n + kVecBlock - 1) / kVecBlock;
    if (full)
        k_rollout_vector<MODE, FS, true><<<grid, kVecBlock, 0, s>>>(a);
    else
        k_rollout_vector<MODE, FS, false><<<grid, kVecBlock, 0, s>>>(a);
}

template <int MODE>
static void launch_vec_mode(const LaunchArgs &a, bool full, cudaStream_t s)
{
    if (a.frameskip == 1)
        launch_vec_full<MODE, 1>(a, full, s);
    else if (a.frameskip == 4)
        launch_vec_full<MODE, 4>(a, full, s);
    else
        launch_vec_full<MODE, 0>(a, full, s);
}

cudaError_t launch_rollout_vector(const LaunchArgs &a, cudaStream_t s)
{
    const bool full = (a.t0 % 4 == 0) && (a.T % 4 == 0);
    switch (a.action_mode) {
    case 0: launch_vec_mode<0>(a, full, s); break;
    case 1: launch_vec_mode<1>(a, full, s); break;
    case 2: launch_vec_mode<2>(a, full, s); break;
    default: launch_vec_mode<3>(a, full, s); break;
    }
    return cudaGetLastError();
}

// ---- pixel rollout --------------------------------------------------------------------

constexpr int kPixThreads = 128;  // 4 warps; also the largest env count of a block
constexpr int kPixWarps = kPixThreads / 32;
constexpr int kPixBufPerWarp = 3;  // staging frames per warp, used round-robin
constexpr int kPixSmemBytes = kPixWarps * kPixBufPerWarp * kFrameBytes + kPixThreads * 4 + kPixThreads;

__device__ __forceinline__ uint32_t smem_addr(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

// Bulk async copy of `bytes` (multiple of 16) from shared to global memory;
// both addresses 16-byte aligned.
__device__ __forceinline__ void bulk_store(void *gdst, const void *ssrc, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 :: "l"(gdst), "r"(smem_addr(ssrc)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit()
{
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int PENDING>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" :: "n"(PENDING) : "memory");
}
__device__ __forceinline__ void fence_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// One warp paints one 84x84 frame into shared memory.  Output pixel (i, j)
// samples source row i*192/84 and source column j*160/84; the agent's paddle
// (source columns 148..151) falls on output columns 78-79, the opponent's
// (8..11) on 5-6; a source column is sampled by at most one output column.
__device__ __forceinline__ void render_frame(uint8_t *buf, uint32_t geom, int lane)
{
    uint4 *q = reinterpret_cast<uint4 *>(buf);
    for (int k = lane; k < kFrameBytes / 16; k += 32) q[k] = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();
    const int ap = geom & 255u, op = (geom >> 8) & 255u;
    const int bxp = (geom >> 16) & 255u, byp = geom >> 24;
    for (int i = lane; i < kFrameH; i += 32) {
        const int sr = (i * 192) / 84;
        uint8_t *row = buf + i * kFrameW;
        if ((unsigned)(sr - ap) < 16u) { row[78] = 255; row[79] = 255; }
        if ((unsigned)(sr - op) < 16u) { row[5] = 255; row[6] = 255; }
        if ((unsigned)(sr - byp) < 2u) {
#pragma unroll
            for (int dc = 0; dc < 2; ++dc) {
                const int c = bxp + dc;
                const int j = (c * 21 + 39) / 40;  // smallest j with j*160/84 >= c
                if (j < kFrameW && (j * 160) / 84 == c) row[j] = 255;
            }
        }
    }
}

// The block owns envs [first, first + count): thread i < count runs env
// first + i.  Per agent step: physics by the env threads, geometry handed over
// in shared memory, then the warps paint and send the frames.
template <int MODE>
__global__ void __launch_bounds__(kPixThreads) k_rollout_pixels(const __grid_constant__ LaunchArgs a,
                                                                const int envs_per_block)
{
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t *frames = smem;
    uint32_t *geom = reinterpret_cast<uint32_t *>(smem + kPixWarps * kPixBufPerWarp * kFrameBytes);
    uint8_t *ended = reinterpret_cast<uint8_t *>(geom + kPixThreads);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int first = blockIdx.x * envs_per_block;
    const int count = min(envs_per_block, a.n - first);
    const bool has_env = tid < count;
    const int n = first + tid;
    const uint32_t env_id = a.env_id_base + (uint32_t)n;

    Env e = {};
    Tally tally = {0, 0, 0};
    if (has_env) load_env(e, a.plane0, a.plane1, n);
    uint32_t w[4] = {0u, 0u, 0u, 0u};
    unsigned round = 0;  // staging buffer rotation of this warp

    for (int t = 0; t < a.T; ++t) {
        const unsigned long long tt = a.t0 + (unsigned long long)t;
        if (has_env) {
            if (MODE <= 1 && (t == 0 || (tt & 3) == 0)) action_words(tt >> 2, env_id, a.rk, w);
            const int sel = (int)(tt & 3);
            const uint32_t word = sel == 0 ? w[0] : sel == 1 ? w[1] : sel == 2 ? w[2] : w[3];
            const size_t o = (size_t)t * (size_t)a.n + (size_t)n;
            const int action = pick_action<MODE>(word, e, MODE == 2 ? a.actions + o : nullptr,
                                                 a.const_action);
            bool done;
            const int r = agent_step<0>(e, action, a.frameskip, env_id, a.rk, tally, done);
            a.reward[o] = (float)r;
            a.done[o] = done ? 1 : 0;
            geom[tid] = pack_geometry(e);
            ended[tid] = done ? 1 : 0;
        }
        __syncthreads();
        for (int le = warp; le < count; le += kPixWarps) {
            uint8_t *buf = frames + (warp * kPixBufPerWarp + (round % kPixBufPerWarp)) * kFrameBytes;
            ++round;
            // the copy that last read this buffer is the third most recent group
            if (lane == 0) bulk_wait_read<kPixBufPerWarp - 1>();
            __syncwarp();
            render_frame(buf, geom[le], lane);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
                uint8_t *env_ring = a.ring + (size_t)(first + le) * (kStack * kFrameBytes);
                if (ended[le]) {
                    for (int s = 0; s < kStack; ++s) bulk_store(env_ring + s * kFrameBytes, buf, kFrameBytes);
                } else {
                    bulk_store(env_ring + (size_t)(tt & 3) * kFrameBytes, buf, kFrameBytes);
                }
                bulk_commit();
            }
        }
        __syncthreads();
    }
    if (lane == 0) bulk_wait_read<0>();
    if (has_env) store_env(e, a.plane0, a.plane1, n);
    flush_tally(tally, a.stats);
}

// Envs per block so that the grid is a whole number of waves over the SMs
// (two resident blocks per SM) while no block gets more envs than threads.
static int pixel_envs_per_block(int n, int sm_count)
{
    for (int k = 2;; k += 2) {
        const int slots = sm_count * k;
        const int per = (n + slots - 1) / slots;
        if (per <= kPixThreads) return per;
    }
}

cudaError_t launch_rollout_pixels(const LaunchArgs &a, int sm_count, cudaStream_t s)
{
    const int per = pixel_envs_per_block(a.n, sm_count);
    const int grid = (a.n + per - 1) / per;
    cudaError_t err = cudaSuccess;
#define PONG_PIX(M)                                                                              \
    do {                                                                                         \
        err = cudaFuncSetAttribute(k_rollout_pixels<M>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                   kPixSmemBytes);                                               \
        if (err != cudaSuccess) return err;                                                      \
        k_rollout_pixels<M><<<grid, kPixThreads, kPixSmemBytes, s>>>(a, per);                    \
    } while (0)
    switch (a.action_mode) {
    case 0: PONG_PIX(0); break;
    case 1: PONG_PIX(1); break;
    case 2: PONG_PIX(2); break;
    default: PONG_PIX(3); break;
    }
#undef PONG_PIX
    return cudaGetLastError();
}

// One warp per env: paint the frame of the stored state and copy it to all
// four ring slots.
__global__ void __launch_bounds__(kPixThreads) k_reset_pixels(const __grid_constant__ LaunchArgs a)
{
    __shared__ __align__(128) uint8_t frames[kPixWarps * kFrameBytes];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n = blockIdx.x * kPixWarps + warp;
    if (n >= a.n) return;  // warp-uniform
    Env e;
    load_env(e, a.plane0, a.plane1, n);
    uint8_t *buf = frames + warp * kFrameBytes;
    render_frame(buf, pack_geometry(e), lane);
    fence_async_smem();
    __syncwarp();
    if (lane == 0) {
        uint8_t *env_ring = a.ring + (size_t)n * (kStack * kFrameBytes);
        for (int s = 0; s < kStack; ++s) bulk_store(env_ring + s * kFrameBytes, buf, kFrameBytes);
        bulk_commit();
        bulk_wait_read<0>();
    }
}

cudaError_t launch_reset(const LaunchArgs &a, cudaStream_t s)
{
    k_reset<<<(a.n + 127) / 128, 128, 0, s>>>(a);
    cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) return err;
    if (a.ring != nullptr) {
        k_reset_pixels<<<(a.n + kPixWarps - 1) / kPixWarps, kPixThreads, 0, s>>>(a);
        err = cudaGetLastError();
    }
    return err;
}

// ---- action fill --------------------------------------------------------------------------

// Thread (x = env, y = Philox block): up to four action bytes.
__global__ void __launch_bounds__(128) k_fill_actions(const __grid_constant__ LaunchArgs a,
                                                      const int sticky, uint8_t *__restrict__ out)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= a.n) return;
    const unsigned long long t_begin = a.t0, t_end = a.t0 + (unsigned long long)a.T;
    const unsigned long long g = (t_begin >> 2) + blockIdx.y;
    uint32_t w[4];
    action_words(g, a.env_id_base + (uint32_t)n, a.rk, w);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const unsigned long long tt = g * 4 + j;
        if (tt >= t_begin && tt < t_end) {
            uint8_t b = (uint8_t)uniform_action(w[j]);
            if (sticky && sticky_repeat(w[j])) b |= 4u;
            out[(size_t)(tt - t_begin) * (size_t)a.n + (size_t)n] = b;
        }
    }
}

cudaError_t launch_fill_actions(const LaunchArgs &a, int sticky, uint8_t *out, cudaStream_t s)
{
    const unsigned long long g0 = a.t0 >> 2, g1 = (a.t0 + (unsigned long long)a.T - 1) >> 2;
    const unsigned long long groups = g1 - g0 + 1;
    // gridDim.y is limited to 65535: fill in slabs of whole Philox blocks
    LaunchArgs b = a;
    unsigned long long done_groups = 0;
    while (done_groups < groups) {
        const unsigned long long slab = groups - done_groups < 32768ull ? groups - done_groups : 32768ull;
        const unsigned long long slab_t0 = done_groups == 0 ? a.t0 : (g0 + done_groups) * 4;
        unsigned long long slab_t1 = (g0 + done_groups + slab) * 4;
        if (slab_t1 > a.t0 + (unsigned long long)a.T) slab_t1 = a.t0 + (unsigned long long)a.T;
        b.t0 = slab_t0;
        b.T = (int)(slab_t1 - slab_t0);
        dim3 grid((a.n + 127) / 128, (unsigned)slab);
        k_fill_actions<<<grid, 128, 0, s>>>(b, sticky, out + (size_t)(slab_t0 - a.t0) * (size_t)a.n);
        cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
        done_groups += slab;
    }
    return cudaSuccess;
}

}  // namespace pong
