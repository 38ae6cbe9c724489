/*
 * pong.h -- C ABI of the B200 batched fixed-point Pong environment library.
 *
 * The library simulates n independent Pong environments per call on one GPU.
 * It is the "performance environment" of the paper (Sec. 3.1): every output
 * (obs, reward, done) is bit-identical at every step, for every seed and
 * action sequence, to a plain per-env statement of the rules.  The batched
 * single step corresponds to the paper's jit(vmap(step)) (Appendix "JAX
 * Optimization Checklist", items 3-4), the fused multi-step rollout to its
 * lax.scan fusion (item 5), caller-owned output buffers to items 7 / Rust
 * item 2, observation scaling inside the step to item 8, "render only the
 * last skipped frame" to Rust item 3, and "one call for all envs on raw
 * buffers" to Rust item 8.
 *
 * Rule set (Q8 fixed point, 256 units = 1 px, court 160x192 px, y downward;
 * positions are the top-left corner of the 2x2 ball / top edge of a 4x16
 * paddle).  One physics frame with action a in {0 stay, 1 up, 2 down}:
 *   1. agent paddle y += (a==2 ? 768 : a==1 ? -768 : 0), clamped to [0,45056]
 *   2. opponent paddle moves towards the ball centre (before the ball moves)
 *      by at most 512, clamped to [0,45056]
 *   3. ball += velocity
 *   4. y < 0 or y > 48640 mirrors about that wall and negates vy
 *   5. if the ball box overlaps the paddle box it is moving towards
 *      (agent x in [37888,38912), opponent x in [2048,3072), half-open):
 *      |vx| += 16 capped at 1024, vx changes sign, vy += 16 * (ball centre px
 *      - paddle centre px), clamped to +-768
 *   6. ball x > 40960: reward +1, agent point; x < 0: reward -1, opponent
 *      point; either way the ball respawns at the centre with vx = +-512 and
 *      vy uniform in [-384,384] from Philox4x32-10 keyed by
 *      (seed, env, episode, point number)
 *   7. frame count += 1; done when a side has 21 points or at 10000 frames
 *   8. on done the finished episode is added to the episode statistics and
 *      the env resets (a pure function of seed, env, episode number)
 *   9. obs is taken after the reset when done.
 * An agent step is `frameskip` frames with the action repeated, rewards
 * summed, stopping after a frame that ends the episode.
 *
 * Random actions: Philox4x32-10 with key = seed and counter
 * {t/4, global env id, t>>34, 0}; step t uses output word t%4; the low 16
 * bits u give the action (u*3)>>16, the high 16 bits s < 16384 mean "repeat
 * the previous action" in sticky mode.  t is the handle's global agent-step
 * counter (0 after create / reset, +T per rollout).
 *
 * Observations:
 *   vector (obs_mode 0): float32[6] = {ball x, ball y, vx, vy, agent paddle y,
 *     opponent paddle y}, each float32(int) * float32(1/40960), one rounded
 *     multiply.
 *   pixel (obs_mode 1): uint8[n][4][84][84] ring owned by the caller and
 *     persistent between calls.  Pixel (i,j) is 255 when the source pixel
 *     (row i*192/84, column j*160/84, integer division) is covered by a paddle
 *     or the ball, else 0.  Agent step t writes slot t%4; pong_reset and an
 *     auto-reset write the reset frame to all four slots.
 *
 * Conventions
 *   - Every obs / reward / done / actions pointer is a DEVICE pointer owned by
 *     the caller unless its name says host.  The library reads / writes it on
 *     the handle's stream during the call's kernels and never keeps it.
 *   - The library owns only the env state (32 bytes per env) and three int64
 *     statistics counters, allocated by pong_create* and freed by
 *     pong_destroy.
 *   - step / rollout / fill_actions / reset only enqueue work on the handle's
 *     stream and return; episode_stats / get_state / set_state / the *_host
 *     call synchronise that stream.
 *   - Every function returns 0 or a negative PONG_E* code; nothing throws,
 *     aborts, traps or prints.  There is no CPU fallback: without a usable
 *     CUDA device pong_create* fails with PONG_ECUDA.
 *   - A handle is not thread-safe; use one handle per host thread or lock.
 *     The library also keeps small per-device caches (SM count, the address of
 *     pong_rollout_static's array) that are filled on first use without a lock:
 *     make the first call on each device from one thread.
 */
#ifndef PONG_H_
#define PONG_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PONG_OK       0
#define PONG_EINVAL  (-1)  /* bad size, T, frameskip, obs_mode, action value */
#define PONG_ENULL   (-2)  /* required pointer is NULL */
#define PONG_EALIGN  (-3)  /* pointer not aligned as documented */
#define PONG_ECUDA   (-4)  /* a CUDA runtime call or launch failed */
#define PONG_EMODE   (-5)  /* unknown action_mode, or call not valid in this obs_mode */
#define PONG_ENOMEM  (-6)  /* host or device allocation failed */
#define PONG_ELIMIT  (-7)  /* size beyond a fixed maximum of the entry point */

#define PONG_OBS_VECTOR 0
#define PONG_OBS_PIXELS 1

#define PONG_ACT_PHILOX   0  /* in-kernel uniform random actions */
#define PONG_ACT_STICKY   1  /* same, repeating the previous action with p = 1/4 */
#define PONG_ACT_EXPLICIT 2  /* uint8[T][n] device buffer of action bytes */
#define PONG_ACT_CONSTANT 3  /* one action for every env and step */

#define PONG_STATE_FIELDS 11 /* bx by vx vy apy opy score_a score_o ep_len episode prev_action */
#define PONG_FRAME_BYTES  (84 * 84)
#define PONG_MAX_FRAMESKIP 16
#define PONG_STATIC_MAX_ENVS 65536 /* largest batch of pong_rollout_static */

typedef struct pong_env pong_env; /* opaque */

typedef struct {
    int obs_mode;    /* PONG_OBS_VECTOR or PONG_OBS_PIXELS */
    int frameskip;   /* physics frames per agent step, 1..PONG_MAX_FRAMESKIP */
    int env_id_base; /* global id of env 0 of this handle; random draws are keyed by
                        env_id_base + local index, so disjoint ranges on several
                        handles (or GPUs) reproduce one large batch exactly */
} pong_config;

/* Create n_envs (>= 1) envs on the current CUDA device, in episode 0 at global
 * step 0, on the default stream.  pong_create uses {vector obs, frameskip 1,
 * env_id_base 0}.  Allocates 32 bytes per env of device memory: the state of
 * all envs lives in buffers allocated once, up front (Appendix "JAX Optimization
 * Checklist", item 7; "Rust Optimization Checklist", item 2), as structure-of-
 * arrays planes of 32-bit integers (JAX item 6: the smallest type that holds
 * the values; Rust item 8: one object for all envs on raw buffers). */
int pong_create(pong_env **out, int n_envs, uint64_t seed);
int pong_create_ex(pong_env **out, int n_envs, uint64_t seed, const pong_config *cfg);

/* Synchronise the stream and free everything the handle owns.  NULL is OK.
 * (Counterpart of pong_create: the only two calls that touch the allocator,
 * JAX checklist item 7.) */
int pong_destroy(pong_env *h);

/* Use `cuda_stream` (a cudaStream_t, e.g. torch's current stream) for all
 * later calls; NULL selects the default stream.  The caller orders work
 * across streams.  (The env runs on the learner's device and stream so that
 * observations never leave the GPU: Sec. 1 and JAX checklist item 4.) */
int pong_set_stream(pong_env *h, void *cuda_stream);

/* Choose the kernel pong_rollout / pong_step use for vector observations: a
 * tuning and testing knob, results are bit-identical on every path ("do not
 * change the external behaviour", Appendix "Optimization Agent Prompt").
 * AUTO picks by batch size.  GENERAL: per-thread stores, any size.  TMA: 64-env
 * blocks, shared-memory staging, TMA tensor stores.  CHAINS: one block per SM,
 * warp chains balanced over the SM's schedulers.  A forced path the call does
 * not qualify for (alignment, T % 8, frameskip, more than 14 x 32 envs per SM)
 * falls through chains -> tma -> general.  Unless the path is GENERAL, a call whose first
 * step is no multiple of 4 or whose length is no multiple of 8 is run as up to three kernels
 * (general head, fast middle, general tail) when the middle is at least 16 steps. */
#define PONG_PATH_AUTO    0
#define PONG_PATH_GENERAL 1
#define PONG_PATH_TMA     2
#define PONG_PATH_CHAINS  3
int pong_set_vector_path(pong_env *h, int path);

/* All envs to episode 0, global step 0, statistics cleared (the reset of the
 * fixed external API: "step, reset, observation and reward shapes stay as they
 * are", Appendix "Optimization Agent Prompt"; the reset state is a pure
 * function of (seed, env, episode) so that two backends started from the same
 * seed can be compared step by step, Sec. 3.2).  obs_out may be
 * NULL; otherwise it receives the initial observation: float32[n][6]
 * (16-byte aligned) or the whole ring uint8[n][4][84][84] (16-byte aligned),
 * all four slots holding the reset frame. */
int pong_reset(pong_env *h, void *obs_out);

/* One agent step for every env (the batched step of checklist items 3-4).
 * actions: uint8[n]; bit 2 set = repeat the env's previous action, otherwise
 * bits 0-1 = action, the spare code 3 meaning stay.
 * obs: float32[n][6] (vector mode) or the ring (pixel mode); reward:
 * float32[n]; done: uint8[n].  obs and reward 16-byte aligned. */
int pong_step(pong_env *h, const uint8_t *actions, void *obs, float *reward,
              uint8_t *done);

/* T >= 1 agent steps in one launch with the env state held in registers
 * (checklist item 5).  action_mode selects where actions come from;
 * `actions` is the uint8[T][n] device buffer for PONG_ACT_EXPLICIT, a HOST
 * pointer to one byte for PONG_ACT_CONSTANT, and ignored otherwise.
 * obs_buf: float32[T][n][6] (vector mode) or the ring (pixel mode);
 * reward_buf: float32[T][n]; done_buf: uint8[T][n].  obs_buf and reward_buf
 * 16-byte aligned.  Advances the global step by T. */
int pong_rollout(pong_env *h, int T, int action_mode, const uint8_t *actions,
                 void *obs_buf, float *reward_buf, uint8_t *done_buf);

/* Same as pong_rollout but every buffer is HOST memory (pinned memory makes
 * the copies asynchronous and fast): explicit actions are copied to the
 * device, the rollout runs into device staging buffers that the handle
 * allocates on first use and keeps, the results are copied back, and the
 * stream is synchronised before returning. */
int pong_rollout_host(pong_env *h, int T, int action_mode, const uint8_t *actions_host,
                      void *obs_host, float *reward_host, uint8_t *done_host);

/* The "matched actions" of the step-level comparison (Sec. 3.2: both backends
 * are driven by the same seeds and the same action sequence).
 * Write to actions_out (device, uint8[T][n]) the bytes that make
 * PONG_ACT_EXPLICIT reproduce PONG_ACT_PHILOX (sticky = 0) or
 * PONG_ACT_STICKY (sticky = 1) for global steps t .. t+T-1.  Does not advance
 * the global step. */
int pong_fill_actions(pong_env *h, int T, int sticky, uint8_t *actions_out);

/* ---- policy in the loop (the paper's "GRU rollout" setting: a policy network on
 * the same stream produces the actions) ------------------------------------------
 *
 * pong_fill_words writes the Philox action words of global steps t .. t+T-1 to
 * words_out (device uint32[T][n]); they are the uniform numbers of the draws
 * below.  Does not advance the global step.
 *
 * pong_sample_actions draws one action per env from softmax(logits[i][0..2])
 * (device float32[n][3], finite values) with the uniform number words[i] (device
 * uint32[n]) and writes action bytes for pong_step to actions_out (device
 * uint8[n]).  Everything is binary32 in a fixed order so that the draw is
 * reproducible bit for bit:
 *   m = max(l0,l1,l2); ei = expn(li - m); s = (e0 + e1) + e2;
 *   x = ((float)(word >> 8) * 2^-24) * s;  a = x < e0 ? 0 : (x < e0 + e1 ? 1 : 2)
 *   expn(x) = 2^f * 2^n with y = x * log2(e), n = floor(y + 0.5), f = y - n and
 *   2^f = ((((((P6 f + P5) f + P4) f + P3) f + P2) f + P1) f + 1, Pk = ln(2)^k / k!
 *   (0 when y < -150 or n < -126).
 * It uses no state of the handle but its size and stream, so a captured launch
 * can be replayed.
 *
 * pong_get_step_counter / pong_set_step_counter read and set the global agent
 * step t.  They exist for captured launches: a CUDA graph replay runs the kernels
 * but not the host code that counts steps, and capturing runs the host code but
 * not the kernels, so the caller puts the counter right around both.  Only
 * pong_step with vector observations is meant to be replayed that way: its
 * kernel does not use the step number. */
int pong_fill_words(pong_env *h, int T, uint32_t *words_out);
int pong_sample_actions(pong_env *h, const float *logits, const uint32_t *words,
                        uint8_t *actions_out);
int pong_get_step_counter(pong_env *h, uint64_t *t);
int pong_set_step_counter(pong_env *h, uint64_t t);

/* The episode statistics the paper's Level-4 check compares (Sec. 3.2: episode
 * returns and lengths of the two backends), reduced on the device.
 * Episodes finished since create / reset / the last clear: their number, the
 * sum of their returns (agent points - opponent points) and of their lengths
 * in frames.  Exact integers.  Outputs are HOST pointers (any may be NULL).
 * Synchronises the stream. */
int pong_episode_stats(pong_env *h, int64_t *episodes, int64_t *sum_return,
                       int64_t *sum_length, int clear);

/* Checkpoint / restore (the save-state / load-state pair the paper's module
 * translation keeps for every stateful component, Appendix "Module Translation
 * Prompt"; it is also what lets a divergence be replayed from the step before).
 * host_soa is HOST int32[PONG_STATE_FIELDS][n] in the
 * field order named above; t is the global agent step.  set_state validates
 * field ranges (PONG_EINVAL) and leaves statistics untouched.  In pixel mode
 * the ring is the caller's and is not part of the state. */
int pong_get_state(pong_env *h, int32_t *host_soa, uint64_t *t);
int pong_set_state(pong_env *h, const int32_t *host_soa, uint64_t t);

/* Reset-and-rollout in one call that allocates nothing (the paper has no
 * counterpart; this is an addition for hosts that cannot allocate).
 *
 * Who needs it: programs that may not call cudaMalloc while they run - code
 * loaded into another runtime that owns all device memory, loops with a hard
 * latency bound (cudaMalloc / cudaFree stall the whole device), processes held
 * to a memory budget fixed at start-up.  The handle API takes its env state and
 * episode counters from cudaMalloc; this call keeps them in a fixed array inside
 * the library's device image instead (2 MiB + 256 bytes, present on every GPU
 * that loads the library, until the process exits).  It calls no cudaMalloc,
 * cudaFree or other allocating routine.
 *
 * What it does: n_envs envs (1..PONG_STATIC_MAX_ENVS, else PONG_ELIMIT) with
 * global ids env_id_base.., vector obs, frameskip 1, are reset to episode 0 at
 * global step 0 and run for T agent steps, exactly like pong_create_ex +
 * pong_rollout on a fresh handle: obs_buf float32[T][n][6], reward_buf
 * float32[T][n], done_buf uint8[T][n] (device, obs / reward 16-byte aligned),
 * `actions` as for pong_rollout.  stats_out (device int64[3], may be NULL)
 * receives {episodes, sum of returns, sum of lengths} of the episodes finished
 * within the call.  Everything is enqueued on cuda_stream (NULL = default
 * stream) and the call returns without synchronising.
 *
 * Set-up: the first call made with a given device current looks up the
 * array's device address (once per device); make that first call outside any
 * stream capture.
 * Sharing: every call on a device uses the same array, which still holds the
 * previous call's data; the call clears the counters and rewrites the states
 * before use.  Two calls whose GPU work overlaps (different streams, or
 * different host threads) race on the array: serialise them. */
int pong_rollout_static(int n_envs, uint64_t seed, int env_id_base, int T, int action_mode,
                        const uint8_t *actions, float *obs_buf, float *reward_buf,
                        uint8_t *done_buf, int64_t *stats_out, void *cuda_stream);

/* Measurement aid for the compute-side ceiling of the rollout (the paper's optimisation
 * loop profiles before it optimises, Sec. 3.3; a kernel that is all integer min / max / add
 * has the integer pipe as its second roofline next to HBM): runs a register-only kernel of
 * dependent add / max / min chains at full occupancy on the current device and returns the
 * integer-ALU warp instructions per second it sustained (HOST double).  Synchronises
 * cuda_stream.  Allocates nothing. */
int pong_measure_alu_rate(void *cuda_stream, double *warp_instr_per_s);

/* Number of envs / kernels launched by this handle so far (for accounting). */
int pong_num_envs(const pong_env *h);
int64_t pong_launch_count(const pong_env *h);

/* Static description of a PONG_E* code. */
const char *pong_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* PONG_H_ */
