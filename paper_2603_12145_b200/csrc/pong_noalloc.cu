// pong_rollout_static: a rollout entry point that allocates nothing.
//
// Some host programs may not call cudaMalloc at all once they are running: a
// plug-in living inside another runtime that owns the whole memory pool, a
// control loop with a hard latency bound (cudaMalloc and cudaFree synchronise
// the whole device and can take milliseconds), or a process that was given a
// fixed memory budget at start-up and must not fail later for lack of memory.
// For them the env state and the episode counters, which the handle-based API
// keeps in memory obtained from cudaMalloc, live here in one file-scope device
// array of fixed size that every GPU using the library holds from load to exit.
#include "../../include/pong.h"
#include "pong_kernels.cuh"

namespace {

constexpr size_t kPlaneBytes = (size_t)PONG_STATIC_MAX_ENVS * sizeof(int4);
constexpr size_t kScratchBytes = 2 * kPlaneBytes + 256;  // plane0 | plane1 | counters

// The scratch itself.  In host code this name is only a handle for the runtime,
// never an address a kernel could use: the device address is asked for below.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
unsigned char *g_scratch_ptr[kMaxDevices];  // device address per device, 0 = not set up

// Device address of the scratch on the current device; looked up on the first
// call made with that device current.
int scratch_for_current_device(unsigned char **out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return PONG_ECUDA;
    }
    if (g_scratch_ptr[dev] == nullptr) {
        unsigned char *p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_static_scratch) != cudaSuccess ||
            p == nullptr) {
            cudaGetLastError();
            return PONG_ECUDA;
        }
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return PONG_OK;
}

}  // namespace

extern "C" int pong_rollout_static(int n_envs, uint64_t seed, int env_id_base, int T, int action_mode,
                                   const uint8_t *actions, float *obs_buf, float *reward_buf,
                                   uint8_t *done_buf, int64_t *stats_out, void *cuda_stream)
{
    if (n_envs < 1 || T < 1 || env_id_base < 0) return PONG_EINVAL;
    if (n_envs > PONG_STATIC_MAX_ENVS) return PONG_ELIMIT;
    if ((int64_t)env_id_base + n_envs > 0x7fffffffLL) return PONG_EINVAL;
    // [T][n] element counts must stay addressable by the kernels' size_t math (as pong_rollout)
    if ((uint64_t)T * (uint64_t)n_envs > (1ull << 40)) return PONG_EINVAL;
    if (action_mode < PONG_ACT_PHILOX || action_mode > PONG_ACT_CONSTANT) return PONG_EMODE;
    if (obs_buf == nullptr || reward_buf == nullptr || done_buf == nullptr) return PONG_ENULL;
    if ((action_mode == PONG_ACT_EXPLICIT || action_mode == PONG_ACT_CONSTANT) && actions == nullptr)
        return PONG_ENULL;
    if ((reinterpret_cast<uintptr_t>(obs_buf) | reinterpret_cast<uintptr_t>(reward_buf)) % 16 != 0)
        return PONG_EALIGN;
    int const_action = 0;
    if (action_mode == PONG_ACT_CONSTANT) {
        if (actions[0] > 2) return PONG_EINVAL;  // host byte
        const_action = actions[0];
    }

    unsigned char *scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != PONG_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    pong::LaunchArgs a = {};
    a.plane0 = reinterpret_cast<int4 *>(scratch);
    a.plane1 = reinterpret_cast<int4 *>(scratch + kPlaneBytes);
    a.stats = reinterpret_cast<long long *>(scratch + 2 * kPlaneBytes);
    for (int r = 0; r < 10; ++r) {
        a.rk.k[2 * r] = (uint32_t)seed + (uint32_t)r * pong::kPhiloxW0;
        a.rk.k[2 * r + 1] = (uint32_t)(seed >> 32) + (uint32_t)r * pong::kPhiloxW1;
    }
    a.t0 = 0;
    a.env_id_base = (uint32_t)env_id_base;
    a.n = n_envs;
    a.T = T;
    a.frameskip = 1;

    // The array still holds the previous call's counters and states: the
    // counters must start at zero, the states are rewritten by the reset.
    if (cudaMemsetAsync(a.stats, 0, 3 * sizeof(long long), stream) != cudaSuccess) return PONG_ECUDA;
    if (pong::launch_reset(a, stream) != cudaSuccess) return PONG_ECUDA;
    a.action_mode = action_mode;
    a.actions = actions;
    a.const_action = const_action;
    a.obs = obs_buf;
    a.reward = reward_buf;
    a.done = done_buf;
    if (pong::launch_rollout_vector(a, stream) != cudaSuccess) return PONG_ECUDA;
    if (stats_out != nullptr &&
        cudaMemcpyAsync(stats_out, a.stats, 3 * sizeof(long long), cudaMemcpyDeviceToDevice, stream) !=
            cudaSuccess)
        return PONG_ECUDA;
    return PONG_OK;
}
