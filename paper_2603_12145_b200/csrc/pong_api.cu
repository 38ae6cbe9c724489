// C ABI of the batched Pong library (declared in include/pong.h): argument
// validation, handle bookkeeping and kernel launches.  Host code only; the
// environment's arithmetic is all in the kernels.
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/pong.h"
#include "pong_kernels.cuh"

struct pong_env {
    int n = 0;
    uint64_t seed = 0;
    pong_config cfg = {PONG_OBS_VECTOR, 1, 0};
    int device = 0;
    int sm_count = 0;
    cudaStream_t stream = nullptr;
    void *block = nullptr;  // one allocation: plane0 | plane1 | stats
    int4 *plane0 = nullptr;
    int4 *plane1 = nullptr;
    long long *stats = nullptr;
    uint64_t t = 0;  // global agent step
    int64_t launches = 0;
    int vector_path = 0;
    pong::RoundKeys rk;
    pong::VectorMapCache map_cache = {};
    // staging for pong_rollout_host, grown on demand
    void *stage = nullptr;
    size_t stage_bytes = 0;
};

namespace {

bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

pong::LaunchArgs base_args(const pong_env *h)
{
    pong::LaunchArgs a;
    std::memset(&a, 0, sizeof(a));
    a.plane0 = h->plane0;
    a.plane1 = h->plane1;
    a.stats = h->stats;
    a.rk = h->rk;
    a.t0 = h->t;
    a.env_id_base = (uint32_t)h->cfg.env_id_base;
    a.n = h->n;
    a.T = 1;
    a.frameskip = h->cfg.frameskip;
    a.vector_path = h->vector_path;
    return a;
}

int do_reset(pong_env *h, void *obs_out)
{
    if (obs_out != nullptr && !aligned(obs_out, 16)) return PONG_EALIGN;
    if (cudaMemsetAsync(h->stats, 0, 3 * sizeof(long long), h->stream) != cudaSuccess) return PONG_ECUDA;
    h->t = 0;
    pong::LaunchArgs a = base_args(h);
    if (h->cfg.obs_mode == PONG_OBS_VECTOR)
        a.obs = static_cast<float *>(obs_out);
    else
        a.ring = static_cast<uint8_t *>(obs_out);
    const cudaError_t err = pong::launch_reset(a, h->stream);
    h->launches += (a.ring != nullptr) ? 2 : 1;
    return err == cudaSuccess ? PONG_OK : PONG_ECUDA;
}

int do_rollout(pong_env *h, int T, int action_mode, const uint8_t *actions, int const_action,
               void *obs, float *reward, uint8_t *done)
{
    pong::LaunchArgs a = base_args(h);
    a.T = T;
    a.action_mode = action_mode;
    a.actions = actions;
    a.const_action = const_action;
    a.reward = reward;
    a.done = done;
    cudaError_t err;
    int kernels = 1;
    if (h->cfg.obs_mode == PONG_OBS_VECTOR) {
        a.obs = static_cast<float *>(obs);
        err = pong::launch_rollout_vector(a, h->stream, &h->map_cache, &kernels);
    } else {
        a.ring = static_cast<uint8_t *>(obs);
        err = pong::launch_rollout_pixels(a, h->sm_count, h->stream, &kernels);
    }
    if (err != cudaSuccess) return PONG_ECUDA;
    h->launches += kernels;
    h->t += (uint64_t)T;
    return PONG_OK;
}

int check_rollout_args(const pong_env *h, int T, int action_mode, const uint8_t *actions,
                       const void *obs, const float *reward, const uint8_t *done, int *const_action)
{
    if (h == nullptr) return PONG_ENULL;
    if (T < 1) return PONG_EINVAL;
    if (action_mode < PONG_ACT_PHILOX || action_mode > PONG_ACT_CONSTANT) return PONG_EMODE;
    if (obs == nullptr || reward == nullptr || done == nullptr) return PONG_ENULL;
    if ((action_mode == PONG_ACT_EXPLICIT || action_mode == PONG_ACT_CONSTANT) && actions == nullptr)
        return PONG_ENULL;
    *const_action = 0;
    if (action_mode == PONG_ACT_CONSTANT) {
        if (actions[0] > 2) return PONG_EINVAL;  // host byte
        *const_action = actions[0];
    }
    // [T][n] element counts must stay addressable by the kernels' size_t math
    if ((uint64_t)T * (uint64_t)h->n > (1ull << 40)) return PONG_EINVAL;
    return PONG_OK;
}

}  // namespace

extern "C" {

int pong_create_ex(pong_env **out, int n_envs, uint64_t seed, const pong_config *cfg)
{
    if (out == nullptr || cfg == nullptr) return PONG_ENULL;
    *out = nullptr;
    if (n_envs < 1) return PONG_EINVAL;
    if (cfg->obs_mode != PONG_OBS_VECTOR && cfg->obs_mode != PONG_OBS_PIXELS) return PONG_EINVAL;
    if (cfg->frameskip < 1 || cfg->frameskip > PONG_MAX_FRAMESKIP) return PONG_EINVAL;
    if (cfg->env_id_base < 0 || (int64_t)cfg->env_id_base + n_envs > 0x7fffffffLL) return PONG_EINVAL;

    pong_env *h = new (std::nothrow) pong_env();
    if (h == nullptr) return PONG_ENOMEM;
    h->n = n_envs;
    h->seed = seed;
    h->cfg = *cfg;
    for (int r = 0; r < 10; ++r) {
        h->rk.k[2 * r] = (uint32_t)seed + (uint32_t)r * pong::kPhiloxW0;
        h->rk.k[2 * r + 1] = (uint32_t)(seed >> 32) + (uint32_t)r * pong::kPhiloxW1;
    }
    cudaDeviceProp prop;
    if (cudaGetDevice(&h->device) != cudaSuccess ||
        cudaGetDeviceProperties(&prop, h->device) != cudaSuccess) {
        cudaGetLastError();
        delete h;
        return PONG_ECUDA;
    }
    h->sm_count = prop.multiProcessorCount;
    const size_t plane_bytes = (size_t)n_envs * sizeof(int4);
    const cudaError_t err = cudaMalloc(&h->block, 2 * plane_bytes + 64);
    if (err != cudaSuccess) {
        cudaGetLastError();
        delete h;
        return err == cudaErrorMemoryAllocation ? PONG_ENOMEM : PONG_ECUDA;
    }
    h->plane0 = static_cast<int4 *>(h->block);
    h->plane1 = h->plane0 + n_envs;
    h->stats = reinterpret_cast<long long *>(h->plane1 + n_envs);
    const int rc = do_reset(h, nullptr);
    if (rc != PONG_OK) {
        cudaFree(h->block);
        delete h;
        return rc;
    }
    *out = h;
    return PONG_OK;
}

int pong_create(pong_env **out, int n_envs, uint64_t seed)
{
    const pong_config cfg = {PONG_OBS_VECTOR, 1, 0};
    return pong_create_ex(out, n_envs, seed, &cfg);
}

int pong_destroy(pong_env *h)
{
    if (h == nullptr) return PONG_OK;
    int rc = PONG_OK;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) rc = PONG_ECUDA;
    if (h->stage != nullptr && cudaFree(h->stage) != cudaSuccess) rc = PONG_ECUDA;
    if (cudaFree(h->block) != cudaSuccess) rc = PONG_ECUDA;
    delete h;
    return rc;
}

int pong_set_stream(pong_env *h, void *cuda_stream)
{
    if (h == nullptr) return PONG_ENULL;
    h->stream = static_cast<cudaStream_t>(cuda_stream);
    return PONG_OK;
}

int pong_set_vector_path(pong_env *h, int path)
{
    if (h == nullptr) return PONG_ENULL;
    if (path < PONG_PATH_AUTO || path > PONG_PATH_CHAINS) return PONG_EINVAL;
    h->vector_path = path;
    return PONG_OK;
}

int pong_reset(pong_env *h, void *obs_out)
{
    if (h == nullptr) return PONG_ENULL;
    return do_reset(h, obs_out);
}

int pong_step(pong_env *h, const uint8_t *actions, void *obs, float *reward, uint8_t *done)
{
    if (h == nullptr || actions == nullptr || obs == nullptr || reward == nullptr || done == nullptr)
        return PONG_ENULL;
    if (!aligned(obs, 16) || !aligned(reward, 16)) return PONG_EALIGN;
    return do_rollout(h, 1, PONG_ACT_EXPLICIT, actions, 0, obs, reward, done);
}

int pong_rollout(pong_env *h, int T, int action_mode, const uint8_t *actions, void *obs_buf,
                 float *reward_buf, uint8_t *done_buf)
{
    int const_action = 0;
    const int rc = check_rollout_args(h, T, action_mode, actions, obs_buf, reward_buf, done_buf,
                                      &const_action);
    if (rc != PONG_OK) return rc;
    if (!aligned(obs_buf, 16) || !aligned(reward_buf, 16)) return PONG_EALIGN;
    return do_rollout(h, T, action_mode, actions, const_action, obs_buf, reward_buf, done_buf);
}

int pong_rollout_host(pong_env *h, int T, int action_mode, const uint8_t *actions_host,
                      void *obs_host, float *reward_host, uint8_t *done_host)
{
    int const_action = 0;
    const int rc = check_rollout_args(h, T, action_mode, actions_host, obs_host, reward_host,
                                      done_host, &const_action);
    if (rc != PONG_OK) return rc;
    const size_t tn = (size_t)T * (size_t)h->n;
    const bool vec = h->cfg.obs_mode == PONG_OBS_VECTOR;
    const size_t obs_bytes = vec ? tn * 6 * sizeof(float) : (size_t)h->n * 4 * PONG_FRAME_BYTES;
    auto up = [](size_t b) { return (b + 255) & ~(size_t)255; };
    const size_t off_reward = up(obs_bytes);
    const size_t off_done = off_reward + up(tn * sizeof(float));
    const size_t off_act = off_done + up(tn);
    const size_t need = off_act + up(action_mode == PONG_ACT_EXPLICIT ? tn : 0);
    if (need > h->stage_bytes) {
        if (cudaStreamSynchronize(h->stream) != cudaSuccess) return PONG_ECUDA;
        if (h->stage != nullptr) cudaFree(h->stage);
        h->stage = nullptr;
        h->stage_bytes = 0;
        if (cudaMalloc(&h->stage, need) != cudaSuccess) {
            cudaGetLastError();
            return PONG_ENOMEM;
        }
        h->stage_bytes = need;
    }
    char *base = static_cast<char *>(h->stage);
    void *d_obs = base;
    float *d_reward = reinterpret_cast<float *>(base + off_reward);
    uint8_t *d_done = reinterpret_cast<uint8_t *>(base + off_done);
    uint8_t *d_act = reinterpret_cast<uint8_t *>(base + off_act);
    const uint8_t *actions = actions_host;
    if (action_mode == PONG_ACT_EXPLICIT) {
        if (cudaMemcpyAsync(d_act, actions_host, tn, cudaMemcpyHostToDevice, h->stream) != cudaSuccess)
            return PONG_ECUDA;
        actions = d_act;
    }
    if (!vec) {
        // the ring is persistent: bring the caller's copy in first
        if (cudaMemcpyAsync(d_obs, obs_host, obs_bytes, cudaMemcpyHostToDevice, h->stream) != cudaSuccess)
            return PONG_ECUDA;
    }
    const int rr = do_rollout(h, T, action_mode, actions, const_action, d_obs, d_reward, d_done);
    if (rr != PONG_OK) return rr;
    if (cudaMemcpyAsync(obs_host, d_obs, obs_bytes, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
        cudaMemcpyAsync(reward_host, d_reward, tn * sizeof(float), cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
        cudaMemcpyAsync(done_host, d_done, tn, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
        cudaStreamSynchronize(h->stream) != cudaSuccess)
        return PONG_ECUDA;
    return PONG_OK;
}

int pong_fill_actions(pong_env *h, int T, int sticky, uint8_t *actions_out)
{
    if (h == nullptr || actions_out == nullptr) return PONG_ENULL;
    if (T < 1 || (uint64_t)T * (uint64_t)h->n > (1ull << 40)) return PONG_EINVAL;
    pong::LaunchArgs a = base_args(h);
    a.T = T;
    const cudaError_t err = pong::launch_fill_actions(a, sticky != 0, actions_out, h->stream);
    if (err != cudaSuccess) return PONG_ECUDA;
    const uint64_t groups = ((h->t + (uint64_t)T - 1) >> 2) - (h->t >> 2) + 1;
    h->launches += (int64_t)((groups + 32767) / 32768);
    return PONG_OK;
}

int pong_fill_words(pong_env *h, int T, uint32_t *words_out)
{
    if (h == nullptr || words_out == nullptr) return PONG_ENULL;
    if (T < 1 || (uint64_t)T * (uint64_t)h->n > (1ull << 40)) return PONG_EINVAL;
    pong::LaunchArgs a = base_args(h);
    a.T = T;
    if (pong::launch_fill_words(a, words_out, h->stream) != cudaSuccess) return PONG_ECUDA;
    const uint64_t groups = ((h->t + (uint64_t)T - 1) >> 2) - (h->t >> 2) + 1;
    h->launches += (int64_t)((groups + 32767) / 32768);
    return PONG_OK;
}

int pong_sample_actions(pong_env *h, const float *logits, const uint32_t *words, uint8_t *actions_out)
{
    if (h == nullptr || logits == nullptr || words == nullptr || actions_out == nullptr) return PONG_ENULL;
    if (pong::launch_sample_actions(h->n, logits, words, actions_out, h->stream) != cudaSuccess)
        return PONG_ECUDA;
    h->launches += 1;
    return PONG_OK;
}

int pong_get_step_counter(pong_env *h, uint64_t *t)
{
    if (h == nullptr || t == nullptr) return PONG_ENULL;
    *t = h->t;
    return PONG_OK;
}

int pong_set_step_counter(pong_env *h, uint64_t t)
{
    if (h == nullptr) return PONG_ENULL;
    h->t = t;
    return PONG_OK;
}

int pong_episode_stats(pong_env *h, int64_t *episodes, int64_t *sum_return, int64_t *sum_length,
                       int clear)
{
    if (h == nullptr) return PONG_ENULL;
    long long v[3] = {0, 0, 0};
    if (cudaMemcpyAsync(v, h->stats, sizeof(v), cudaMemcpyDeviceToHost, h->stream) != cudaSuccess)
        return PONG_ECUDA;
    if (clear && cudaMemsetAsync(h->stats, 0, sizeof(v), h->stream) != cudaSuccess) return PONG_ECUDA;
    if (cudaStreamSynchronize(h->stream) != cudaSuccess) return PONG_ECUDA;
    if (episodes) *episodes = v[0];
    if (sum_return) *sum_return = v[1];
    if (sum_length) *sum_length = v[2];
    return PONG_OK;
}

int pong_get_state(pong_env *h, int32_t *host_soa, uint64_t *t)
{
    if (h == nullptr || host_soa == nullptr) return PONG_ENULL;
    const size_t n = (size_t)h->n;
    std::vector<int4> planes;
    try {
        planes.resize(2 * n);
    } catch (...) {
        return PONG_ENOMEM;
    }
    if (cudaMemcpyAsync(planes.data(), h->plane0, 2 * n * sizeof(int4), cudaMemcpyDeviceToHost,
                        h->stream) != cudaSuccess ||
        cudaStreamSynchronize(h->stream) != cudaSuccess)
        return PONG_ECUDA;
    for (size_t i = 0; i < n; ++i) {
        const int4 a = planes[i], b = planes[n + i];
        host_soa[0 * n + i] = a.x;
        host_soa[1 * n + i] = a.y;
        host_soa[2 * n + i] = a.z;
        host_soa[3 * n + i] = a.w;
        host_soa[4 * n + i] = b.x;
        host_soa[5 * n + i] = b.y;
        host_soa[6 * n + i] = b.z & 31;
        host_soa[7 * n + i] = (b.z >> 5) & 31;
        host_soa[8 * n + i] = (b.z >> 10) & 0x3FFF;
        host_soa[9 * n + i] = b.w;
        host_soa[10 * n + i] = (b.z >> 24) & 3;
    }
    if (t) *t = h->t;
    return PONG_OK;
}

int pong_set_state(pong_env *h, const int32_t *s, uint64_t t)
{
    if (h == nullptr || s == nullptr) return PONG_ENULL;
    const size_t n = (size_t)h->n;
    std::vector<int4> planes;
    try {
        planes.resize(2 * n);
    } catch (...) {
        return PONG_ENOMEM;
    }
    for (size_t i = 0; i < n; ++i) {
        const int bx = s[0 * n + i], by = s[1 * n + i], vx = s[2 * n + i], vy = s[3 * n + i];
        const int apy = s[4 * n + i], opy = s[5 * n + i], sa = s[6 * n + i], so = s[7 * n + i];
        const int len = s[8 * n + i], ep = s[9 * n + i], prev = s[10 * n + i];
        const int avx = vx < 0 ? -vx : vx;
        if (bx < 0 || bx > pong::kCourtW || by < 0 || by > pong::kBallYMax || avx < pong::kVx0 ||
            avx > pong::kVxCap || vy < -pong::kVyCap || vy > pong::kVyCap || apy < 0 ||
            apy > pong::kPadYMax || opy < 0 || opy > pong::kPadYMax || sa < 0 ||
            sa >= pong::kMaxScore || so < 0 || so >= pong::kMaxScore || len < 0 ||
            len >= pong::kMaxFrames || ep < 0 || prev < 0 || prev > 2)
            return PONG_EINVAL;
        planes[i] = make_int4(bx, by, vx, vy);
        planes[n + i] = make_int4(apy, opy, sa | (so << 5) | (len << 10) | (prev << 24), ep);
    }
    if (cudaMemcpyAsync(h->plane0, planes.data(), 2 * n * sizeof(int4), cudaMemcpyHostToDevice,
                        h->stream) != cudaSuccess ||
        cudaStreamSynchronize(h->stream) != cudaSuccess)
        return PONG_ECUDA;
    h->t = t;
    return PONG_OK;
}

int pong_measure_alu_rate(void *cuda_stream, double *warp_instr_per_s)
{
    if (warp_instr_per_s == nullptr) return PONG_ENULL;
    *warp_instr_per_s = 0.0;
    return pong::measure_alu_rate(static_cast<cudaStream_t>(cuda_stream), warp_instr_per_s) == cudaSuccess
               ? PONG_OK
               : PONG_ECUDA;
}

int pong_num_envs(const pong_env *h) { return h ? h->n : PONG_ENULL; }

int64_t pong_launch_count(const pong_env *h) { return h ? h->launches : (int64_t)PONG_ENULL; }

const char *pong_strerror(int code)
{
    switch (code) {
    case PONG_OK: return "ok";
    case PONG_EINVAL: return "invalid argument (size, T, frameskip, obs_mode, action or state value)";
    case PONG_ENULL: return "required pointer is NULL";
    case PONG_EALIGN: return "pointer is not 16-byte aligned";
    case PONG_ECUDA: return "a CUDA runtime call or kernel launch failed";
    case PONG_EMODE: return "unknown action_mode";
    case PONG_ENOMEM: return "out of host or device memory";
    case PONG_ELIMIT: return "size exceeds the fixed maximum of this entry point";
    default: return "unknown error code";
    }
}

}  // extern "C"
