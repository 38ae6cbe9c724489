/*
 * cartpole.h -- C ABI of the B200 batched CartPole environment library.
 *
 * The second small environment of the paper's throughput tables (Table "A6000
 * Ada throughput", row "CartPole JAX (scan)"; Appendix "JAX Optimization
 * Checklist", item 5 quotes CartPole for the gain of fusing a rollout into one
 * kernel).  Same structure as the Pong library: n independent envs per call,
 * a batched single step and a fused T-step rollout with the state in
 * registers, caller-owned output buffers, counter-based randomness, exact
 * step-level agreement with a plain per-env statement of the rules (Sec. 3.1).
 *
 * Rules.  Textbook cart-pole dynamics (Barto, Sutton, Anderson 1983): gravity
 * 9.8, cart mass 1.0, pole mass 0.1, half-length 0.5, force +-10, time step
 * 0.02, explicit Euler.  All arithmetic is IEEE binary32, one rounding per
 * operation, in this order (z = th*th):
 *   s = th * ((((S9*z + S7)*z + S5)*z + S3)*z + 1),  S3 = -1/6, S5 = 1/120,
 *                                     S7 = -1/5040, S9 = 1/362880
 *   c =       (((C8*z + C6)*z + C4)*z + C2)*z + 1,   C2 = -1/2, C4 = 1/24,
 *                                     C6 = -1/720, C8 = 1/40320
 *   temp     = (force + ((0.05 * (thd*thd)) * s)) / 1.1
 *   thetaacc = (9.8*s - c*temp) / (0.5 * (4/3 - (0.1*(c*c)) / 1.1))
 *   xacc     = temp - ((0.05*thetaacc) * c) / 1.1
 *   (1.1 = total mass; every / is a correctly rounded binary32 division)
 *   x += 0.02*xd; xd += 0.02*xacc; th += 0.02*thd; thd += 0.02*thetaacc
 * (velocities of the step's start move the positions).  Then steps += 1,
 * reward = 1, done = x < -2.4 || x > 2.4 || |th| > 12 degrees || steps >= 500.
 * On done the episode's length goes to the statistics, the env resets and the
 * obs is the state after the reset.  Reset(seed, env, episode): Philox4x32-10
 * with counter {0, episode, global env id, 2}, key = seed; each state variable
 * = ((float)(word >> 8) * 2^-24 - 0.5) * 0.1.  Random action of global step t:
 * Philox counter {t/4, global env id, t>>34, 3}, output word t%4, bit 0
 * (0 = push left, 1 = push right).
 *
 * Conventions: as in pong.h.  Every obs / reward / done / actions pointer is a
 * DEVICE pointer owned by the caller unless its name says host; step / rollout
 * / reset enqueue on the handle's stream and return; episode_stats / get_state
 * / set_state synchronise it.  Return 0 or a negative CARTPOLE_E* code; no
 * exceptions, aborts, traps or printing; no CPU fallback.  A handle is not
 * thread-safe, and the library fills a small per-device cache on first use
 * without a lock: make the first rollout on each device from one thread.
 */
#ifndef CARTPOLE_H_
#define CARTPOLE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CARTPOLE_OK       0
#define CARTPOLE_EINVAL  (-1)  /* bad size, T, action or state value */
#define CARTPOLE_ENULL   (-2)  /* required pointer is NULL */
#define CARTPOLE_EALIGN  (-3)  /* obs pointer not 16-byte aligned */
#define CARTPOLE_ECUDA   (-4)  /* a CUDA runtime call or launch failed */
#define CARTPOLE_EMODE   (-5)  /* unknown action_mode */
#define CARTPOLE_ENOMEM  (-6)  /* allocation failed */

#define CARTPOLE_ACT_PHILOX   0  /* in-kernel uniform random actions */
#define CARTPOLE_ACT_EXPLICIT 2  /* uint8[T][n] device buffer, bit 0 = action */
#define CARTPOLE_ACT_CONSTANT 3  /* one action for every env and step */

typedef struct cartpole_env cartpole_env; /* opaque */

/* n_envs >= 1 envs on the current device, episode 0, global step 0.  Global env
 * ids are env_id_base + local index (disjoint ranges on several handles or GPUs
 * reproduce one large batch exactly).  Allocates 24 bytes per env. */
int cartpole_create(cartpole_env **out, int n_envs, uint64_t seed, int env_id_base);
int cartpole_destroy(cartpole_env *h);
int cartpole_set_stream(cartpole_env *h, void *cuda_stream);

/* All envs to episode 0, step 0, statistics cleared; obs_out (float32[n][4],
 * 16-byte aligned) may be NULL. */
int cartpole_reset(cartpole_env *h, float *obs_out);

/* One step: actions uint8[n] (bit 0), obs float32[n][4], reward float32[n],
 * done uint8[n]. */
int cartpole_step(cartpole_env *h, const uint8_t *actions, float *obs, float *reward, uint8_t *done);

/* T >= 1 steps in one launch, state in registers.  `actions`: device uint8[T][n]
 * for CARTPOLE_ACT_EXPLICIT, HOST pointer to one byte for CARTPOLE_ACT_CONSTANT,
 * ignored for CARTPOLE_ACT_PHILOX.  obs float32[T][n][4] (16-byte aligned),
 * reward float32[T][n], done uint8[T][n].  Advances the global step by T. */
int cartpole_rollout(cartpole_env *h, int T, int action_mode, const uint8_t *actions, float *obs,
                     float *reward, uint8_t *done);

/* Same with every buffer in HOST memory (pinned memory recommended); the handle
 * keeps device staging buffers; synchronises the stream before returning. */
int cartpole_rollout_host(cartpole_env *h, int T, int action_mode, const uint8_t *actions_host,
                          float *obs_host, float *reward_host, uint8_t *done_host);

/* Episodes finished since create / reset / the last clear and the sum of their
 * lengths (= returns).  HOST pointers, may be NULL.  Synchronises the stream. */
int cartpole_episode_stats(cartpole_env *h, int64_t *episodes, int64_t *sum_length, int clear);

/* Checkpoint / restore: HOST float32[4][n] = x, xd, th, thd; HOST int32[2][n] =
 * steps, episode; t = global step.  set_state accepts in-play states only
 * (|x| <= 2.4, |th| <= 12 degrees: an env never rests in a state that ends its
 * episode) with |xd|, |thd| <= 1000, steps in 0..499 and episode >= 0; anything
 * else, NaN included, is CARTPOLE_EINVAL. */
int cartpole_get_state(cartpole_env *h, float *host_f, int32_t *host_i, uint64_t *t);
int cartpole_set_state(cartpole_env *h, const float *host_f, const int32_t *host_i, uint64_t t);

/* Which rollout kernel runs (a tuning / testing knob; every path gives the same bits).
 * AUTO picks by batch size.  PLAIN: 128-env blocks.  CHAINS: one block per SM with its warps'
 * load balanced over the SM's schedulers; needs the global step and T to be multiples of 4 and
 * at most 14 x 32 envs per SM, otherwise the plain kernel runs. */
#define CARTPOLE_PATH_AUTO   0
#define CARTPOLE_PATH_PLAIN  1
#define CARTPOLE_PATH_CHAINS 2
int cartpole_set_path(cartpole_env *h, int path);

int cartpole_num_envs(const cartpole_env *h);
int64_t cartpole_launch_count(const cartpole_env *h);
const char *cartpole_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* CARTPOLE_H_ */
