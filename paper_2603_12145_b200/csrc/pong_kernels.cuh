// Launch interface between the C ABI (pong_api.cu) and the kernels
// (pong_kernels.cu).  Plain pointers and sizes only.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "pong_rules.cuh"

namespace pong {

struct LaunchArgs {
    int4 *plane0;              // [n] {bx, by, vx, vy}
    int4 *plane1;              // [n] {apy, opy, packed counters, episode}
    long long *stats;          // [3] episodes, sum of returns, sum of lengths
    const uint8_t *actions;    // explicit mode: [T][n] action bytes
    float *obs;                // vector mode: [T][n][6]
    uint8_t *ring;             // pixel mode: [n][4][84][84]
    float *reward;             // [T][n]
    uint8_t *done;             // [T][n]
    RoundKeys rk;              // Philox round keys of the seed
    unsigned long long t0;     // global agent step of the first step
    uint32_t env_id_base;
    int n;
    int T;
    int action_mode;           // 0 Philox, 1 sticky, 2 explicit, 3 constant
    int const_action;          // mode 3
    int frameskip;
    int vector_path;           // kPath*: which vector-rollout kernel to use
};

// Vector-rollout kernels (values of pong_set_vector_path).  A forced path that the call
// does not qualify for falls through: chains -> tma -> general.
constexpr int kPathAuto = 0, kPathGeneral = 1, kPathTma = 2, kPathChains = 3;

// The three tensor maps of a vector rollout (obs, reward, done) as last encoded for a handle,
// with what they were encoded for.  Encoding costs the host about a microsecond per map, which
// shows in launches of 20 us and less; a caller that rolls out into the same buffers again
// reuses them.  Opaque here: the CUtensorMap type stays inside pong_kernels.cu.
struct VectorMapCache {
    alignas(64) unsigned char maps[3 * 128];
    const void *obs, *reward, *done;
    int n, T, box_envs;        // box_envs = 0: nothing cached
};

// Each returns the cudaError_t of the launch (cudaGetLastError).
cudaError_t launch_reset(const LaunchArgs &a, cudaStream_t s);          // state + optional obs / ring
cudaError_t launch_rollout_vector(const LaunchArgs &a, cudaStream_t s, VectorMapCache *cache = nullptr,
                                  int *kernels = nullptr);   // *kernels: how many kernels it launched (1-3)
cudaError_t launch_rollout_pixels(const LaunchArgs &a, int sm_count, cudaStream_t s, int *kernels = nullptr);
cudaError_t launch_fill_actions(const LaunchArgs &a, int sticky, uint8_t *out, cudaStream_t s);
cudaError_t launch_fill_words(const LaunchArgs &a, uint32_t *out, cudaStream_t s);
cudaError_t launch_sample_actions(int n, const float *logits, const uint32_t *words, uint8_t *out,
                                  cudaStream_t s);

// Integer-ALU warp instructions per second the device sustains (synchronises the stream).
cudaError_t measure_alu_rate(cudaStream_t s, double *warp_instr_per_s);

}  // namespace pong
