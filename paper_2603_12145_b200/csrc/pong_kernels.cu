// Kernels of the batched fixed-point Pong step for sm_100a.
//
//   k_reset            state planes <- reset(seed, env, 0); optional initial obs
//   k_reset_pixels     reset frame into all four ring slots
//   k_rollout_vector   one thread per env, state in registers across T steps,
//                      streams obs / reward / done to HBM with per-thread stores
//                      (any n, T, frameskip and action mode)
//   k_rollout_vector_tma  the same rollout for the common case (frameskip 1,
//                      aligned n / t / T, any action mode): outputs are staged in shared
//                      memory 8 steps at a time and leave through TMA tensor stores,
//                      the Philox block of the next four steps is interleaved with
//                      the physics of the current four, rare paths are warp-uniform
//   k_rollout_pixels   one thread per env for the physics, one warp per frame
//                      for the rasteriser; frames are staged in shared memory
//                      and leave through bulk async copies (16-byte granules)
//   k_rollout_pixels_x4  the same for aligned calls (t % 4 == 0, T % 4 == 0): four
//                      agent steps at a time, so that an env's whole 4-slot ring
//                      (28,224 contiguous bytes) is painted in shared memory and
//                      leaves as one bulk copy
//   k_fill_actions     action bytes that reproduce the Philox modes
//
// No kernel waits on another block, on a flag or on an mbarrier; the only
// blocking instructions are __syncthreads and cp.async.bulk.wait_group.
#include <cuda.h>

#include <cstring>

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

// ---- asynchronous copy helpers ---------------------------------------------------------

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
// Same, but until the groups have completed (their global writes are done), not only read
// their shared-memory source.
template <int PENDING>
__device__ __forceinline__ void bulk_wait_done()
{
    asm volatile("cp.async.bulk.wait_group %0;" :: "n"(PENDING) : "memory");
}
__device__ __forceinline__ void fence_async_smem()
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// TMA tensor store of a 2-D box from shared memory; (x, y) is the box origin in
// elements of the tensor map, x * element size a multiple of 16 bytes.  Parts of
// the box outside the tensor are not written.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, const void *ssrc, int x, int y)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 :: "l"(map), "r"(smem_addr(ssrc)), "r"(x), "r"(y) : "memory");
}
// Programmatic dependent launch: wait for the preceding kernel of the stream to
// complete and flush / let the following kernel start its prologue.
__device__ __forceinline__ void grid_dependency_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
__device__ __forceinline__ void grid_dependency_launch()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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
    // launched with the programmatic-dependent-launch attribute: the block may be resident before
    // the preceding kernel of the stream (the previous step, or whatever produced the actions) has
    // finished; nothing of the caller's or the handle's memory is touched before this wait
    grid_dependency_wait();
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
        grid_dependency_launch();
        store_env(e, a.plane0, a.plane1, n);
    }
    flush_tally(tally, a.stats);
}

template <int MODE, int FS>
static void launch_vec_full(const LaunchArgs &a, bool full, cudaStream_t s)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((a.n + kVecBlock - 1) / kVecBlock);
    cfg.blockDim = dim3(kVecBlock);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (full)
        cudaLaunchKernelEx(&cfg, k_rollout_vector<MODE, FS, true>, a);
    else
        cudaLaunchKernelEx(&cfg, k_rollout_vector<MODE, FS, false>, a);
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

// ---- vector rollout, TMA path ---------------------------------------------------------

constexpr int kTmaBlock = 64;  // envs per block (two warps)
constexpr int kTmaStage = 8;   // agent steps staged in shared memory per TMA store

struct VectorMaps {
    CUtensorMap obs;     // [T][3n] 8-byte elements (pairs of floats), box 3*kTmaBlock x kTmaStage
    CUtensorMap reward;  // [T][n] float32, box kTmaBlock x kTmaStage
    CUtensorMap done;    // [T][n] uint8, box kTmaBlock x kTmaStage
};

// Requirements (checked by the launcher): frameskip 1, t0 % 4 == 0,
// T % kTmaStage == 0, n % 16 == 0 (row pitches are multiples of 16 bytes).
// Threads past n run a copy of env n-1 so that every warp stays whole; their
// outputs fall outside the tensor maps and are dropped by the TMA unit.
// QUEUE: spawns from the per-lane queue of pong_rules.cuh (fewer instructions per step).
template <int MODE, bool QUEUE>
__global__ void __launch_bounds__(kTmaBlock) k_rollout_vector_tma(const __grid_constant__ LaunchArgs a,
                                                                  const __grid_constant__ VectorMaps maps)
{
    __shared__ __align__(128) float s_obs[2][kTmaStage][kTmaBlock * 6];
    __shared__ __align__(128) float s_reward[2][kTmaStage][kTmaBlock];
    __shared__ __align__(128) uint8_t s_done[2][kTmaStage][kTmaBlock];

    const int tid = threadIdx.x;
    const int n0 = blockIdx.x * kTmaBlock;
    const bool valid = n0 + tid < a.n;
    const int n = valid ? n0 + tid : a.n - 1;
    const uint32_t env_id = a.env_id_base + (uint32_t)n;
    Tally tally = {0, 0, 0};

    // Philox block of the first four steps: independent of the state, so it runs
    // before the wait on the previous kernel.
    unsigned long long g = a.t0 >> 2;
    PhiloxPipe pipe = {0u, 0u, 0u, 0u};
    if (MODE <= 1) {
        philox_start(pipe, g, env_id);
        philox_rounds<0, 10>(pipe, a.rk);
    }

    grid_dependency_wait();
    FastEnv e;
    {
        Env q;
        load_env(q, a.plane0, a.plane1, n);
        to_fast(e, q);
    }

    const uint8_t *act = MODE == 2 ? a.actions + n : nullptr;
    const size_t act_stride = (size_t)a.n;
    int buf = 0;
    for (int t = 0; t < a.T; t += kTmaStage) {
        // explicit actions of this stage: eight coalesced byte loads issued together,
        // their latency hidden behind the wait below
        uint32_t abyte[kTmaStage];
        if (MODE == 2) {
#pragma unroll
            for (int s = 0; s < kTmaStage; ++s) abyte[s] = act[(size_t)s * act_stride];
            act += (size_t)kTmaStage * act_stride;
        }
        // the store that last read this buffer is the older of the two in flight
        if (tid == 0) bulk_wait_read<1>();
        __syncthreads();
        // reward and done rows start as zeros; a lane writes its entry only on a point or an
        // episode end (5 x 16-byte stores per thread-pair instead of two stores per step)
        {
            uint4 *zr = reinterpret_cast<uint4 *>(&s_reward[buf][0][0]);   // 8 x 64 floats = 128 uint4
            zr[tid] = make_uint4(0u, 0u, 0u, 0u);
            zr[tid + kTmaBlock] = make_uint4(0u, 0u, 0u, 0u);
            uint4 *zd = reinterpret_cast<uint4 *>(&s_done[buf][0][0]);     // 8 x 64 bytes = 32 uint4
            if (tid < kTmaStage * kTmaBlock / 16) zd[tid] = make_uint4(0u, 0u, 0u, 0u);
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kTmaStage / 4; ++q) {
            const uint32_t w[4] = {pipe.c0, pipe.c1, pipe.c2, pipe.c3};
            if (MODE <= 1) {
                ++g;
                philox_start(pipe, g, env_id);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (MODE <= 1) {
                    if (j == 0) philox_rounds<0, 3>(pipe, a.rk);
                    if (j == 1) philox_rounds<3, 6>(pipe, a.rk);
                    if (j == 2) philox_rounds<6, 8>(pipe, a.rk);
                    if (j == 3) philox_rounds<8, 10>(pipe, a.rk);
                }
                const int s = q * 4 + j;
                int action;
                if (MODE == 0) action = uniform_action(w[j]);
                else if (MODE == 1) action = sticky_repeat(w[j]) ? e.prev : uniform_action(w[j]);
                else if (MODE == 2) action = decode_action_byte(abyte[s], e.prev);
                else action = a.const_action;
                e.prev = action;
                fast_frame<QUEUE>(e, action, env_id, a.rk, tally, &s_reward[buf][s][tid], &s_done[buf][s][tid]);
                float2 *o = reinterpret_cast<float2 *>(&s_obs[buf][s][tid * 6]);
                o[0] = make_float2(scale_obs(e.bx), scale_obs(e.by));
                o[1] = make_float2(scale_obs(e.vx), scale_obs(e.vy));
                o[2] = make_float2(scale_obs(e.apy), scale_obs(e.opy));
            }
        }
        fence_async_smem();
        __syncthreads();
        if (tid == 0) {
            tma_store_2d(&maps.obs, &s_obs[buf][0][0], n0 * 3, t);
            tma_store_2d(&maps.reward, &s_reward[buf][0][0], n0, t);
            tma_store_2d(&maps.done, &s_done[buf][0][0], n0, t);
            bulk_commit();
        }
        buf ^= 1;
    }
    // Let the next launch of the stream start its prologue now.  (Triggering right
    // after the state load instead makes its blocks resident and waiting for the
    // whole rollout; at 4-6 blocks per SM that slowed this launch by up to 40 %.)
    grid_dependency_launch();
    if (valid) {
        Env q;
        from_fast(q, e);
        store_env(q, a.plane0, a.plane1, n);
    } else {
        tally.episodes = 0;
        tally.sum_return = 0;
        tally.sum_length = 0;
    }
    flush_tally(tally, a.stats);
    if (tid == 0) bulk_wait_read<0>();
}

typedef CUresult (*TensorMapEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                      const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                      const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kTmaBlocksPerSm = 7;  // 29.7 KB of staging per block in 227 KB of shared memory

// SM count of the current device, asked once per device.
static int resident_sm_count()
{
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
            cudaGetLastError();
            sms = 148;
        }
        cached[dev] = sms;
    }
    return cached[dev];
}

// The driver's tensor-map encoder, looked up once through the runtime (no link
// against libcuda); nullptr if this driver does not have it.
static TensorMapEncodeFn tensor_map_encoder()
{
    static TensorMapEncodeFn fn = []() -> TensorMapEncodeFn {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        return reinterpret_cast<TensorMapEncodeFn>(p);
    }();
    return fn;
}

static bool encode_rows(TensorMapEncodeFn enc, CUtensorMap *m, CUtensorMapDataType type, void *base,
                        uint64_t row_elems, uint64_t rows, uint64_t row_bytes, uint32_t box_elems,
                        uint32_t box_rows)
{
    const cuuint64_t dims[2] = {row_elems, rows};
    const cuuint64_t strides[1] = {row_bytes};
    const cuuint32_t box[2] = {box_elems, box_rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    return enc(m, type, 2, base, dims, strides, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static_assert(sizeof(VectorMaps) == sizeof(VectorMapCache::maps), "three 128-byte tensor maps");

// The maps of [T][n] outputs with boxes of box_envs envs by kTmaStage steps: from the cache if
// it holds them for exactly these buffers and sizes, else encoded (and cached).
static bool vector_maps(const LaunchArgs &a, int box_envs, VectorMapCache *cache, VectorMaps *maps)
{
    if (cache != nullptr && cache->box_envs == box_envs && cache->obs == a.obs && cache->reward == a.reward &&
        cache->done == a.done && cache->n == a.n && cache->T == a.T) {
        memcpy(maps, cache->maps, sizeof(VectorMaps));
        return true;
    }
    TensorMapEncodeFn enc = tensor_map_encoder();
    if (enc == nullptr) return false;
    const uint64_t n = (uint64_t)a.n, T = (uint64_t)a.T;
    if (!encode_rows(enc, &maps->obs, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, a.obs, n * 3, T, n * 24,
                     (uint32_t)box_envs * 3, kTmaStage) ||
        !encode_rows(enc, &maps->reward, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, a.reward, n, T, n * 4,
                     (uint32_t)box_envs, kTmaStage) ||
        !encode_rows(enc, &maps->done, CU_TENSOR_MAP_DATA_TYPE_UINT8, a.done, n, T, n, (uint32_t)box_envs,
                     kTmaStage))
        return false;
    if (cache != nullptr) {
        memcpy(cache->maps, maps, sizeof(VectorMaps));
        cache->obs = a.obs; cache->reward = a.reward; cache->done = a.done;
        cache->n = a.n; cache->T = a.T; cache->box_envs = box_envs;
    }
    return true;
}

// Launches the TMA path if the call qualifies; returns false (nothing launched)
// if it does not, so that the caller uses the general kernel.
static bool try_launch_vector_tma(const LaunchArgs &a, cudaStream_t s, cudaError_t *err,
                                  VectorMapCache *cache = nullptr)
{
    if (a.frameskip != 1) return false;
    if (a.n % 16 != 0 || a.t0 % 4 != 0 || a.T % kTmaStage != 0) return false;
    if (a.n > (1 << 29)) return false;  // box origins 3 * n0 are 32-bit tensor coordinates
    const uintptr_t bases = reinterpret_cast<uintptr_t>(a.obs) | reinterpret_cast<uintptr_t>(a.reward) |
                            reinterpret_cast<uintptr_t>(a.done);
    if (bases % 16 != 0) return false;  // tensor maps need 16-byte aligned bases
    VectorMaps maps;
    if (!vector_maps(a, kTmaBlock, cache, &maps)) return false;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((a.n + kTmaBlock - 1) / kTmaBlock);
    cfg.blockDim = dim3(kTmaBlock);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // Seven blocks fit an SM (shared memory).  A launch whose blocks are all, or nearly all,
    // resident from the start takes as long as one block's T steps at four warps per
    // scheduler, so the instructions per step count: the spawn queue wins there (by 1-3 % at
    // 65,536 envs, 6-12 % between 8,192 and 114,000).  From two waves of blocks on, the launch
    // is bound by the HBM write stream and the plain event path measured 2-4 % faster.
    const bool queue = (long long)cfg.gridDim.x * 4 <= (long long)resident_sm_count() * kTmaBlocksPerSm * 7;
#define PONG_TMA(M)                                                                      \
    *err = queue ? cudaLaunchKernelEx(&cfg, k_rollout_vector_tma<M, true>, a, maps)      \
                 : cudaLaunchKernelEx(&cfg, k_rollout_vector_tma<M, false>, a, maps)
    switch (a.action_mode) {
    case 0: PONG_TMA(0); break;
    case 1: PONG_TMA(1); break;
    case 2: PONG_TMA(2); break;
    default: PONG_TMA(3); break;
    }
#undef PONG_TMA
    return true;
}

// ---- vector rollout, one block per SM with balanced warp chains ------------------------
//
// A warp-step of the rollout costs a scheduler about as many dispatch cycles whatever else
// runs on it, so a launch whose blocks are all resident from the start takes as long as the
// scheduler that holds the most warps.  65,536 envs are 13.84 warps per SM: with small blocks
// two of an SM's four schedulers get four warps, the others three, and the launch runs at
// the four-warp pace while the store stream would allow more.  Here one 16-warp block per SM
// owns a contiguous range of up to 14 chains (a chain = 32 consecutive envs, one lane each,
// with its own two staging buffers and its own TMA tensor stores, so chains never wait for
// one another).  Warp w sits on scheduler w % 4.  The first 4*floor(c/4) chains stay on
// warps 0..11 for the whole launch.  When one or two chains are left over, each alternates
// between two warps on different schedulers (warps 12 and 14, or 13 and 15) every
// kChainSegment stages, so that over the launch every scheduler carries the same number of
// chain-steps.  A hand-over is one pass of the env registers through shared memory between
// two named hardware barriers, each executed exactly once per hand-over by both warps.
constexpr int kChainMax = 14;                 // chains per block (shared memory)
constexpr int kChainWarps = 16;
constexpr int kChainThreads = kChainWarps * 32;
constexpr int kChainSegment = 4;              // stages a leftover chain runs on one warp (1: 43.8 us, 2: 41.7, 3: 41.4, 4: 40.9, 5: 41.3, 8: 42.9 at 65,536 x 128)
constexpr int kHandWords = 12;                // FastEnv as 32-bit words
// stages between two block-wide rendezvous of the chains (T = 128 / 256 / 512 / 1024 at 65,536 envs:
// none 40.6 / 82.2 / 172.9 / 359.4 us, every 4: 45.1 / 85.7 / 167.0 / 328.4, every 8: 41.3 / 78.3 /
// 151.8 / 299.5, every 16: 40.5 / 76.9 / 150.5 / 305.0, every 32: 40.7 / 80.9 / 163.3 / 327.3)
constexpr int kChainLockstep = 16;

struct ChainStage {
    float obs[kTmaStage][32 * 6];
    float reward[kTmaStage][32];
    uint8_t done[kTmaStage][32];
};
static_assert(sizeof(ChainStage) == 7424 && sizeof(ChainStage) % 128 == 0, "stage layout");
constexpr int kChainSmemBytes = kChainMax * 2 * (int)sizeof(ChainStage) + 2 * kHandWords * 32 * 4;

__device__ __forceinline__ void named_barrier(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" :: "r"(id), "r"(threads) : "memory");
}

template <int MODE, bool QUEUE>
__global__ void __launch_bounds__(kChainThreads, 1)
k_rollout_vector_chains(const __grid_constant__ LaunchArgs a, const __grid_constant__ VectorMaps maps)
{
    // no static shared memory in this kernel: the dynamic part starts at the block's window,
    // aligned as declared (TMA tensor stores read 128-byte aligned tiles)
    extern __shared__ __align__(128) uint8_t chain_smem[];
    ChainStage *stages = reinterpret_cast<ChainStage *>(chain_smem);
    uint32_t(*hand)[kHandWords][32] = reinterpret_cast<uint32_t(*)[kHandWords][32]>(stages + kChainMax * 2);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int groups = (a.n + 31) >> 5;
    const int g_lo = (int)((long long)blockIdx.x * groups / gridDim.x);
    const int g_hi = (int)((long long)(blockIdx.x + 1) * groups / gridDim.x);
    const int c = g_hi - g_lo;          // <= kChainMax (launcher)
    const int fixed = c & ~3, extra = c & 3;
    const int S = a.T / kTmaStage;

    // This warp's role: a chain, and which of its segments (runs of seg_len stages) it takes:
    // first, first + 2, ...  A whole chain is one segment.
    int chain = -1, seg_len = S, first = 0, slot = 0;
    if (warp < fixed) {
        chain = warp;
    } else if (warp >= 12) {
        const int k = warp - 12;
        if ((extra == 1 || extra == 2) && fixed >= 4 && S > kChainSegment) {
            if ((k & 1) < extra) {
                slot = k & 1;
                chain = fixed + slot;
                seg_len = kChainSegment;
                first = k >> 1;
            }
        } else if (k < extra) {
            chain = fixed + k;
        }
    }
    if (chain < 0) return;  // whole warps; no block-wide barrier is used anywhere
    const int segments = (S + seg_len - 1) / seg_len;

    const int n0 = (g_lo + chain) * 32;
    const bool valid = n0 + lane < a.n;
    const int n = valid ? n0 + lane : a.n - 1;
    const uint32_t env_id = a.env_id_base + (uint32_t)n;
    const size_t act_stride = (size_t)a.n;
    ChainStage *mine = stages + chain * 2;
    uint32_t(*h)[32] = hand[slot];
    Tally tally = {0, 0, 0};
    FastEnv e;

    for (int j = first; j < segments; j += 2) {
        const int sa = j * seg_len, sb = min(S, sa + seg_len);
        // Philox block of the segment's first four steps: independent of the state, so it
        // runs before the wait for the state
        unsigned long long g = (a.t0 + (unsigned long long)sa * kTmaStage) >> 2;
        PhiloxPipe pipe = {0u, 0u, 0u, 0u};
        if (MODE <= 1) {
            philox_start(pipe, g, env_id);
            philox_rounds<0, 10>(pipe, a.rk);
        }
        // hand-over j-1 -> j uses barriers in_id (state written) and in_id + 1 (the giver's last
        // stage buffer has been read by its store); ids alternate with the hand-over's parity
        const int in_id = 1 + slot * 4 + ((j - 1) & 1) * 2;
        if (j == 0) {
            grid_dependency_wait();
            Env q;
            load_env(q, a.plane0, a.plane1, n);
            to_fast(e, q);
        } else {
            if (j == 1) grid_dependency_wait();
            named_barrier(in_id, 64);
            e.bx = (int)h[0][lane]; e.by = (int)h[1][lane]; e.vx = (int)h[2][lane]; e.vy = (int)h[3][lane];
            e.apy = (int)h[4][lane]; e.opy = (int)h[5][lane]; e.sa = (int)h[6][lane]; e.so = (int)h[7][lane];
            e.left = (int)h[8][lane]; e.episode = (int)h[9][lane]; e.prev = (int)h[10][lane];
            e.spawns = h[11][lane];
        }
        const uint8_t *act = MODE == 2 ? a.actions + n + (size_t)sa * kTmaStage * act_stride : nullptr;
        bool peer_buffer_pending = j > 0;  // the giver's last store may still read buffer (sa+1)&1
        for (int s = sa; s < sb; ++s) {
            uint32_t abyte[kTmaStage];
            if (MODE == 2) {
#pragma unroll
                for (int k = 0; k < kTmaStage; ++k) abyte[k] = act[(size_t)k * act_stride];
                act += (size_t)kTmaStage * act_stride;
            }
            if (peer_buffer_pending && s == sa + 1) {
                named_barrier(in_id + 1, 64);
                peer_buffer_pending = false;
            }
            ChainStage &st = mine[s & 1];
            // Every kChainLockstep stages the block's chains wait for one another.  Left alone they
            // drift apart (a chain never waits for another), and once neighbouring chains write
            // time rows that are far apart the DRAM pages of a row are no longer filled in one go:
            // a 1024-step launch ran at 5.4 TB/s without this and runs at 6.4 TB/s with it.  Each
            // chain has exactly one owner warp at any stage, so 32 * c threads arrive per phase.
            if ((s & (kChainLockstep - 1)) == 0) named_barrier(9, 32 * c);
            // this warp's own store that last read the buffer is the older of its two in flight
            if (lane == 0) bulk_wait_read<1>();
            __syncwarp();
            // reward and done rows start as zeros; a lane writes its entry only on a point or an
            // episode end
            {
                uint4 *zr = reinterpret_cast<uint4 *>(&st.reward[0][0]);   // 8 x 32 floats = 64 uint4
                zr[lane] = make_uint4(0u, 0u, 0u, 0u);
                zr[lane + 32] = make_uint4(0u, 0u, 0u, 0u);
                if (lane < kTmaStage * 32 / 16) reinterpret_cast<uint4 *>(&st.done[0][0])[lane] = make_uint4(0u, 0u, 0u, 0u);
            }
            __syncwarp();
#pragma unroll
            for (int q = 0; q < kTmaStage / 4; ++q) {
                const uint32_t w[4] = {pipe.c0, pipe.c1, pipe.c2, pipe.c3};
                if (MODE <= 1) {
                    ++g;
                    philox_start(pipe, g, env_id);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (MODE <= 1) {
                        if (i == 0) philox_rounds<0, 3>(pipe, a.rk);
                        if (i == 1) philox_rounds<3, 6>(pipe, a.rk);
                        if (i == 2) philox_rounds<6, 8>(pipe, a.rk);
                        if (i == 3) philox_rounds<8, 10>(pipe, a.rk);
                    }
                    const int k = q * 4 + i;
                    int action;
                    if (MODE == 0) action = uniform_action(w[i]);
                    else if (MODE == 1) action = sticky_repeat(w[i]) ? e.prev : uniform_action(w[i]);
                    else if (MODE == 2) action = decode_action_byte(abyte[k], e.prev);
                    else action = a.const_action;
                    e.prev = action;
                    fast_frame<QUEUE>(e, action, env_id, a.rk, tally, &st.reward[k][lane], &st.done[k][lane]);
                    float2 *o = reinterpret_cast<float2 *>(&st.obs[k][lane * 6]);
                    o[0] = make_float2(scale_obs(e.bx), scale_obs(e.by));
                    o[1] = make_float2(scale_obs(e.vx), scale_obs(e.vy));
                    o[2] = make_float2(scale_obs(e.apy), scale_obs(e.opy));
                }
            }
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
                tma_store_2d(&maps.obs, &st.obs[0][0], n0 * 3, s * kTmaStage);
                tma_store_2d(&maps.reward, &st.reward[0][0], n0, s * kTmaStage);
                tma_store_2d(&maps.done, &st.done[0][0], n0, s * kTmaStage);
                bulk_commit();
            }
        }
        if (peer_buffer_pending) named_barrier(in_id + 1, 64);  // a segment of a single stage

        if (j + 1 < segments) {
            // hand over to the other warp of the pair
            const int out_id = 1 + slot * 4 + (j & 1) * 2;
            if (lane == 0) bulk_wait_read<1>();  // the next stage's buffer is free
            h[0][lane] = (uint32_t)e.bx; h[1][lane] = (uint32_t)e.by; h[2][lane] = (uint32_t)e.vx;
            h[3][lane] = (uint32_t)e.vy; h[4][lane] = (uint32_t)e.apy; h[5][lane] = (uint32_t)e.opy;
            h[6][lane] = (uint32_t)e.sa; h[7][lane] = (uint32_t)e.so; h[8][lane] = (uint32_t)e.left;
            h[9][lane] = (uint32_t)e.episode; h[10][lane] = (uint32_t)e.prev; h[11][lane] = e.spawns;
            __syncwarp();
            named_barrier(out_id, 64);
            if (lane == 0) bulk_wait_read<0>();  // and now the last stage's buffer
            __syncwarp();
            named_barrier(out_id + 1, 64);
        } else if (valid) {
            Env q;
            from_fast(q, e);
            store_env(q, a.plane0, a.plane1, n);
        }
    }
    grid_dependency_launch();
    if (!valid) {
        tally.episodes = 0;
        tally.sum_return = 0;
        tally.sum_length = 0;
    }
    flush_tally(tally, a.stats);
    if (lane == 0) bulk_wait_read<0>();
}

// Launches the balanced-chains kernel if the call qualifies (see try_launch_vector_tma for
// the alignment rules; in addition every block must get at most kChainMax chains).  Unless
// forced, it is taken only where it measured faster than the small-block kernel: 13 or 14
// chains on the fullest SM, i.e. 56,833 to 66,304 envs on 148 SMs (41.7 against 46.4 us at
// 65,536 envs, T = 128).  With 12 chains or fewer per SM no scheduler is over-loaded and the
// small blocks' shared TMA issue (one thread per 64 envs instead of one per 32) wins by 1-3 us.
static bool try_launch_vector_chains(const LaunchArgs &a, cudaStream_t s, cudaError_t *err, bool forced,
                                     VectorMapCache *cache = nullptr)
{
    if (a.frameskip != 1) return false;
    if (a.n % 16 != 0 || a.t0 % 4 != 0 || a.T % kTmaStage != 0) return false;
    const uintptr_t bases = reinterpret_cast<uintptr_t>(a.obs) | reinterpret_cast<uintptr_t>(a.reward) |
                            reinterpret_cast<uintptr_t>(a.done);
    if (bases % 16 != 0) return false;
    const int sms = resident_sm_count();
    const int groups = (a.n + 31) / 32;
    const int grid = groups < sms ? groups : sms;
    const int fullest = (groups + grid - 1) / grid;
    if (fullest > kChainMax) return false;
    if (!forced && fullest < 13) return false;
    VectorMaps maps;
    if (!vector_maps(a, 32, cache, &maps)) return false;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kChainThreads);
    cfg.dynamicSmemBytes = kChainSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    // the kernel's shared-memory limit is raised once per device and action mode (an unlocked
    // cache like resident_sm_count's: a second thread at worst sets the same value again)
    static bool limit_set[4][64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
#define PONG_CHAINS(M)                                                                              \
    do {                                                                                            \
        *err = cudaSuccess;                                                                         \
        if (!limit_set[M][dev]) {                                                                   \
            *err = cudaFuncSetAttribute(k_rollout_vector_chains<M, true>,                           \
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, kChainSmemBytes); \
            limit_set[M][dev] = *err == cudaSuccess;                                                \
        }                                                                                           \
        if (*err == cudaSuccess) *err = cudaLaunchKernelEx(&cfg, k_rollout_vector_chains<M, true>, a, maps); \
    } while (0)
    switch (a.action_mode) {
    case 0: PONG_CHAINS(0); break;
    case 1: PONG_CHAINS(1); break;
    case 2: PONG_CHAINS(2); break;
    default: PONG_CHAINS(3); break;
    }
#undef PONG_CHAINS
    return true;
}

// One kernel for the whole call: a fast kernel if the call qualifies, else the general one.
static cudaError_t launch_vector_one(const LaunchArgs &a, cudaStream_t s, VectorMapCache *cache)
{
    cudaError_t fast_err = cudaSuccess;
    if ((a.vector_path == kPathAuto || a.vector_path == kPathChains) &&
        try_launch_vector_chains(a, s, &fast_err, a.vector_path == kPathChains, cache))
        return fast_err != cudaSuccess ? fast_err : cudaGetLastError();
    if (a.vector_path != kPathGeneral && try_launch_vector_tma(a, s, &fast_err, cache))
        return fast_err != cudaSuccess ? fast_err : cudaGetLastError();
    const bool full = (a.t0 % 4 == 0) && (a.T % 4 == 0);
    switch (a.action_mode) {
    case 0: launch_vec_mode<0>(a, full, s); break;
    case 1: launch_vec_mode<1>(a, full, s); break;
    case 2: launch_vec_mode<2>(a, full, s); break;
    default: launch_vec_mode<3>(a, full, s); break;
    }
    return cudaGetLastError();
}

// The steps [from, from + count) of the call `a` as a call of their own.
static LaunchArgs sub_call(const LaunchArgs &a, int from, int count)
{
    LaunchArgs b = a;
    const size_t rows = (size_t)from * (size_t)a.n;
    b.t0 = a.t0 + (unsigned long long)from;
    b.T = count;
    b.obs = a.obs + rows * 6;
    b.reward = a.reward + rows;
    b.done = a.done + rows;
    if (a.actions != nullptr && a.action_mode == 2) b.actions = a.actions + rows;
    return b;
}

// A call that misses the fast kernels only because its first step is not a multiple of 4 or its
// length is not a multiple of the stage is cut in up to three: a head of 1-3 steps (general
// kernel) up to the next multiple of 4, the aligned middle (fast kernel), a tail of 1-7 steps
// (general kernel).  The pieces run back to back on the stream; each starts from the state the
// one before it stored.  *kernels receives the number of launches.
cudaError_t launch_rollout_vector(const LaunchArgs &a, cudaStream_t s, VectorMapCache *cache, int *kernels)
{
    int launched = 1;
    cudaError_t err;
    const int head = (int)((4 - a.t0 % 4) % 4);
    const int middle = a.T > head ? ((a.T - head) / kTmaStage) * kTmaStage : 0;
    const uintptr_t bases = reinterpret_cast<uintptr_t>(a.obs) | reinterpret_cast<uintptr_t>(a.reward) |
                            reinterpret_cast<uintptr_t>(a.done);
    const bool cut = a.vector_path != kPathGeneral && a.frameskip == 1 && a.n % 16 == 0 && bases % 16 == 0 &&
                     middle >= 2 * kTmaStage && middle != a.T;
    if (!cut) {
        err = launch_vector_one(a, s, cache);
    } else {
        launched = 0;
        err = cudaSuccess;
        const int tail = a.T - head - middle;
        if (head > 0) {
            err = launch_vector_one(sub_call(a, 0, head), s, nullptr);
            ++launched;
        }
        if (err == cudaSuccess) {
            err = launch_vector_one(sub_call(a, head, middle), s, cache);
            ++launched;
        }
        if (err == cudaSuccess && tail > 0) {
            err = launch_vector_one(sub_call(a, head + middle, tail), s, nullptr);
            ++launched;
        }
    }
    if (kernels != nullptr) *kernels = launched;
    return err;
}

// ---- pixel rollout --------------------------------------------------------------------

constexpr int kPixThreads = 128;  // 4 warps; also the largest env count of a block
constexpr int kPixWarps = kPixThreads / 32;
constexpr int kPixBufPerWarp = 3;  // staging frames per warp, used round-robin
constexpr int kPixSmemBytes = kPixWarps * kPixBufPerWarp * kFrameBytes + kPixThreads * 4 + kPixThreads;

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
    // An env's ring is written again on the next step (another slot, or all four after a reset),
    // and bulk copies have no order among themselves: the earlier store of the same bytes must
    // have completed, not only read its source.  A warp commits one group per env and step, so
    // with at least kPixBufPerWarp envs the wait that frees the staging buffer (all but the two
    // newest groups complete) already covers the env's previous store; a warp with fewer envs
    // waits for everything.
    const bool few_envs = (count - warp + kPixWarps - 1) / kPixWarps < kPixBufPerWarp;

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
            if (lane == 0) {
                if (few_envs) bulk_wait_done<0>();
                else bulk_wait_done<kPixBufPerWarp - 1>();
            }
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

// Four agent steps per pass.  Steps 4k .. 4k+3 write ring slots 0 .. 3, and a step
// that ends an episode writes its reset frame to all four slots, so after the four
// steps slot s holds the frame of the last step j >= s with j == s or done(j).
// That is worked out per env on the geometry words; then each env's ring is painted
// once and stored as one contiguous 28,224-byte bulk copy: the same bytes per agent
// step as the frame-at-a-time kernel, but every DRAM page is written in one go.
constexpr int kPix4Warps = 3;
constexpr int kPix4Threads = kPix4Warps * 32;
constexpr int kPix4Bufs = 2;  // staged rings per warp
constexpr int kRingBytes = kStack * kFrameBytes;
constexpr int kPix4SmemBytes = kPix4Warps * kPix4Bufs * kRingBytes + kPix4Threads * 16;

template <int MODE>
__global__ void __launch_bounds__(kPix4Threads) k_rollout_pixels_x4(const __grid_constant__ LaunchArgs a,
                                                                   const int envs_per_block)
{
    extern __shared__ __align__(128) uint8_t smem[];
    uint8_t *rings = smem;
    uint4 *geom = reinterpret_cast<uint4 *>(smem + kPix4Warps * kPix4Bufs * kRingBytes);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int first = blockIdx.x * envs_per_block;
    const int count = min(envs_per_block, a.n - first);
    const bool has_env = tid < count;
    const int n = first + tid;
    const uint32_t env_id = a.env_id_base + (uint32_t)n;

    Env e = {};
    Tally tally = {0, 0, 0};
    if (has_env) load_env(e, a.plane0, a.plane1, n);
    unsigned round = 0;
    // The same ring is stored again four steps later: that earlier store must have completed
    // (see k_rollout_pixels); with at least kPix4Bufs envs per warp the buffer wait covers it.
    const bool few_envs = (count - warp + kPix4Warps - 1) / kPix4Warps < kPix4Bufs;

    for (int t = 0; t < a.T; t += 4) {
        if (has_env) {
            uint32_t w[4] = {0u, 0u, 0u, 0u};
            if (MODE <= 1) action_words((a.t0 + (unsigned long long)t) >> 2, env_id, a.rk, w);
            uint32_t g[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const size_t o = (size_t)(t + j) * (size_t)a.n + (size_t)n;
                const int action = pick_action<MODE>(w[j], e, MODE == 2 ? a.actions + o : nullptr,
                                                     a.const_action);
                bool done;
                const int r = agent_step<0>(e, action, a.frameskip, env_id, a.rk, tally, done);
                a.reward[o] = (float)r;
                a.done[o] = done ? 1 : 0;
                const uint32_t gj = pack_geometry(e);
                g[j] = gj;
                if (done) {
#pragma unroll
                    for (int s = 0; s < 4; ++s) g[s] = gj;
                }
            }
            geom[tid] = make_uint4(g[0], g[1], g[2], g[3]);
        }
        __syncthreads();
        for (int le = warp; le < count; le += kPix4Warps) {
            uint8_t *buf = rings + (warp * kPix4Bufs + (round % kPix4Bufs)) * kRingBytes;
            ++round;
            if (lane == 0) {
                if (few_envs) bulk_wait_done<0>();
                else bulk_wait_done<kPix4Bufs - 1>();
            }
            __syncwarp();
            const uint4 gq = geom[le];
            render_frame(buf, gq.x, lane);
            render_frame(buf + kFrameBytes, gq.y, lane);
            render_frame(buf + 2 * kFrameBytes, gq.z, lane);
            render_frame(buf + 3 * kFrameBytes, gq.w, lane);
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
                bulk_store(a.ring + (size_t)(first + le) * kRingBytes, buf, kRingBytes);
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
static int pixel_envs_per_block(int n, int sm_count, int max_per_block)
{
    for (int k = 2;; k += 2) {
        const int slots = sm_count * k;
        const int per = (n + slots - 1) / slots;
        if (per <= max_per_block) return per;
    }
}

static cudaError_t launch_pixels_one(const LaunchArgs &a, int sm_count, cudaStream_t s)
{
    cudaError_t err = cudaSuccess;
    if (a.t0 % 4 == 0 && a.T % 4 == 0) {
        const int per = pixel_envs_per_block(a.n, sm_count, kPix4Threads);
        const int grid = (a.n + per - 1) / per;
#define PONG_PIX4(M)                                                                                \
    do {                                                                                            \
        err = cudaFuncSetAttribute(k_rollout_pixels_x4<M>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                   kPix4SmemBytes);                                                 \
        if (err != cudaSuccess) return err;                                                         \
        k_rollout_pixels_x4<M><<<grid, kPix4Threads, kPix4SmemBytes, s>>>(a, per);                  \
    } while (0)
        switch (a.action_mode) {
        case 0: PONG_PIX4(0); break;
        case 1: PONG_PIX4(1); break;
        case 2: PONG_PIX4(2); break;
        default: PONG_PIX4(3); break;
        }
#undef PONG_PIX4
        return cudaGetLastError();
    }
    const int per = pixel_envs_per_block(a.n, sm_count, kPixThreads);
    const int grid = (a.n + per - 1) / per;
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

// A call that misses the four-steps-per-pass kernel only because it starts or ends off a
// multiple of 4 is cut like a vector call: frame-at-a-time head (1-3 steps), four-step middle,
// frame-at-a-time tail (16,384 envs x 64 steps from t = 1: 1412 us uncut).
cudaError_t launch_rollout_pixels(const LaunchArgs &a, int sm_count, cudaStream_t s, int *kernels)
{
    int launched = 1;
    cudaError_t err;
    const int head = (int)((4 - a.t0 % 4) % 4);
    const int middle = a.T > head ? ((a.T - head) / 4) * 4 : 0;
    if (middle < 8 || middle == a.T) {
        err = launch_pixels_one(a, sm_count, s);
    } else {
        launched = 0;
        err = cudaSuccess;
        const int tail = a.T - head - middle;
        auto piece = [&](int from, int count) {
            LaunchArgs b = a;
            const size_t rows = (size_t)from * (size_t)a.n;
            b.t0 = a.t0 + (unsigned long long)from;
            b.T = count;
            b.reward = a.reward + rows;
            b.done = a.done + rows;
            if (a.actions != nullptr && a.action_mode == 2) b.actions = a.actions + rows;
            ++launched;
            return launch_pixels_one(b, sm_count, s);
        };
        if (head > 0) err = piece(0, head);
        if (err == cudaSuccess) err = piece(head, middle);
        if (err == cudaSuccess && tail > 0) err = piece(head + middle, tail);
    }
    if (kernels != nullptr) *kernels = launched;
    return err;
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

// ---- policy interface ---------------------------------------------------------------------

// Thread (x = env, y = Philox block): the four action words of steps 4g .. 4g+3.
__global__ void __launch_bounds__(128) k_fill_words(const __grid_constant__ LaunchArgs a,
                                                    uint32_t *__restrict__ out)
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
        if (tt >= t_begin && tt < t_end) out[(size_t)(tt - t_begin) * (size_t)a.n + (size_t)n] = w[j];
    }
}

cudaError_t launch_fill_words(const LaunchArgs &a, uint32_t *out, cudaStream_t s)
{
    const unsigned long long g0 = a.t0 >> 2, g1 = (a.t0 + (unsigned long long)a.T - 1) >> 2;
    const unsigned long long groups = g1 - g0 + 1;
    LaunchArgs b = a;
    unsigned long long done_groups = 0;
    while (done_groups < groups) {  // gridDim.y is limited to 65535: slabs of whole Philox blocks
        const unsigned long long slab = groups - done_groups < 32768ull ? groups - done_groups : 32768ull;
        const unsigned long long slab_t0 = done_groups == 0 ? a.t0 : (g0 + done_groups) * 4;
        unsigned long long slab_t1 = (g0 + done_groups + slab) * 4;
        if (slab_t1 > a.t0 + (unsigned long long)a.T) slab_t1 = a.t0 + (unsigned long long)a.T;
        b.t0 = slab_t0;
        b.T = (int)(slab_t1 - slab_t0);
        dim3 grid((a.n + 127) / 128, (unsigned)slab);
        k_fill_words<<<grid, 128, 0, s>>>(b, out + (size_t)(slab_t0 - a.t0) * (size_t)a.n);
        const cudaError_t err = cudaGetLastError();
        if (err != cudaSuccess) return err;
        done_groups += slab;
    }
    return cudaSuccess;
}

__global__ void __launch_bounds__(128) k_sample_actions(const int n, const float *__restrict__ logits,
                                                        const uint32_t *__restrict__ words,
                                                        uint8_t *__restrict__ out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float *l = logits + (size_t)i * 3;
    out[i] = (uint8_t)sample_action(l[0], l[1], l[2], words[i]);
}

cudaError_t launch_sample_actions(int n, const float *logits, const uint32_t *words, uint8_t *out,
                                  cudaStream_t s)
{
    k_sample_actions<<<(n + 127) / 128, 128, 0, s>>>(n, logits, words, out);
    return cudaGetLastError();
}

// ---- integer-ALU rate probe ----------------------------------------------------------------
//
// The rollout is integer min / max / add / compare / select work; on sm_100a those run on
// the half-rate ALU pipe of each scheduler.  This kernel measures what that pipe sustains:
// every thread runs kAluChains independent chains of max / xor / min / xor on registers,
// long enough and at full occupancy, so that the time is
// the pipe's and not latency.  Used by the benchmark for the secondary (compute) ceiling.
constexpr int kAluChains = 8;
constexpr int kAluOpsPerIter = kAluChains * 4;  // max, xor, min, xor per chain

__device__ int g_alu_sink;

__global__ void __launch_bounds__(256) k_alu_probe(const int iters, const int seed)
{
    int v[kAluChains];
#pragma unroll
    for (int c = 0; c < kAluChains; ++c) v[c] = seed + (int)threadIdx.x * (c + 1);
    int d = (int)(threadIdx.x & 7) - 3;
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int c = 0; c < kAluChains; ++c) {
            // four dependent ALU-pipe operations; a logic operation between the min and the max
            // keeps the assembler from merging neighbours into one three-input instruction
            asm volatile("max.s32 %0, %0, %2;\n\txor.b32 %0, %0, %1;\n\tmin.s32 %0, %0, %3;\n\txor.b32 %0, %0, %1;"
                         : "+r"(v[c]) : "r"(d), "r"(c), "r"(kPadYMax + c));
        }
    }
    int acc = 0;
#pragma unroll
    for (int c = 0; c < kAluChains; ++c) acc ^= v[c];
    if (acc == 0x7fffffff) g_alu_sink = acc;  // keeps the chains alive; never true in practice
}

cudaError_t measure_alu_rate(cudaStream_t s, double *warp_instr_per_s)
{
    int dev = 0, sms = 0;
    cudaError_t err = cudaGetDevice(&dev);
    if (err == cudaSuccess) err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (err != cudaSuccess) return err;
    const int blocks = sms * 8, threads = 256, iters = 1024;  // 64 warps per SM, about 0.45 ms per launch
    cudaEvent_t e0, e1;
    if ((err = cudaEventCreate(&e0)) != cudaSuccess) return err;
    if ((err = cudaEventCreate(&e1)) != cudaSuccess) { cudaEventDestroy(e0); return err; }
    k_alu_probe<<<blocks, threads, 0, s>>>(64, 1);  // warm-up
    float best = 0.f;
    for (int rep = 0; rep < 5 && err == cudaSuccess; ++rep) {
        cudaEventRecord(e0, s);
        k_alu_probe<<<blocks, threads, 0, s>>>(iters, rep);
        cudaEventRecord(e1, s);
        err = cudaEventSynchronize(e1);
        float ms = 0.f;
        if (err == cudaSuccess) err = cudaEventElapsedTime(&ms, e0, e1);
        if (err == cudaSuccess && (best == 0.f || ms < best)) best = ms;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (err != cudaSuccess) return err;
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    const double warp_instr = (double)blocks * (threads / 32) * (double)iters * kAluOpsPerIter;
    *warp_instr_per_s = warp_instr / ((double)best * 1e-3);
    return cudaSuccess;
}

}  // namespace pong
