/*
 * cartpole_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * Plain single-threaded CPU statement of a batched CartPole step, the second
 * small environment of the paper's throughput tables (Table "A6000 Ada
 * throughput": CartPole JAX (scan); Appendix "JAX Optimization Checklist",
 * item 5, quotes it for scan fusion).  The paper prints no CartPole code; the
 * dynamics are the textbook cart-pole equations of Barto, Sutton and Anderson
 * (1983) with the usual constants, integrated with the explicit Euler rule.
 *
 * Precision.  The paper states none.  Termination is decided by floating
 * point compares, so both sides must take that decision in the same precision:
 * everything here is IEEE binary32 with one rounding per operation, in the
 * order written below (compile with -ffp-contract=off, no fast-math), and
 * sine / cosine are fixed polynomials rather than a library call, so that a
 * second implementation can reproduce every bit.  One env at a time, plain
 * ifs, its own Philox; shares no code with the CUDA path.
 *
 * One step with action a in {0 push left, 1 push right}:
 *   force = a ? +10 : -10
 *   z = th*th
 *   s = th * ((((S9*z + S7)*z + S5)*z + S3)*z + 1)          sin(th)
 *   c =       (((C8*z + C6)*z + C4)*z + C2)*z + 1            cos(th)
 *   temp     = (force + ((0.05 * (thd*thd)) * s)) / 1.1
 *   thetaacc = (9.8*s - c*temp) / (0.5 * (4/3 - (0.1*(c*c)) / 1.1))
 *   xacc     = temp - ((0.05*thetaacc) * c) / 1.1
 *   (1.1 = total mass of cart and pole; every / is a correctly rounded binary32
 *   division, as the textbook equations are written)
 *   x += 0.02*xd;  xd += 0.02*xacc;  th += 0.02*thd;  thd += 0.02*thetaacc
 *   steps += 1;  reward = 1
 *   done = x < -2.4 || x > 2.4 || th < -TH || th > TH || steps >= 500
 *   on done: the episode (its length) goes to the statistics, episode += 1,
 *   and the env is reset; obs is the state after the reset.
 * Reset(seed, env, episode): Philox4x32-10, counter {0, episode, env, 2}, key =
 * seed; each of x, xd, th, thd = ((float)(word >> 8) * 2^-24 - 0.5) * 0.1,
 * i.e. uniform in [-0.05, 0.05).
 * Random action of global step t: Philox counter {t/4, env, t>>34, 3}, output
 * word t%4, action = word & 1.
 *
 * Pins (tests without a GPU): first-step closed form from rest, exact mirror
 * symmetry, agreement with a binary64 evaluation of the same equations using
 * the library sin / cos over short horizons, termination exactly at the
 * thresholds and at 500 steps, reset a pure function of the counters, Philox
 * keying against a second implementation, all action sequences on short
 * horizons.
 */
#include <stdint.h>
#include <string.h>

typedef struct {
    float x, xd, th, thd;
    int32_t steps;    /* steps taken in this episode */
    int32_t episode;  /* finished episodes */
} cp_env;

typedef struct {
    int64_t episodes;
    int64_t sum_length;
} cp_stats;

static const float CP_GRAVITY = 9.8f;
static const float CP_MASSPOLE = 0.1f;
static const float CP_TOTAL_MASS = 1.1f;    /* cart 1.0 + pole 0.1 */
static const float CP_LENGTH = 0.5f;        /* half the pole's length */
static const float CP_POLEMASS_LENGTH = 0.05f;
static const float CP_FORCE = 10.0f;
static const float CP_TAU = 0.02f;
static const float CP_FOUR_THIRDS = 4.0f / 3.0f;
static const float CP_X_LIMIT = 2.4f;
static const float CP_TH_LIMIT = 0.20943951023931953f; /* 12 degrees */
enum { CP_MAX_STEPS = 500 };

/* Taylor coefficients, rounded once to binary32 */
static const float S3 = -1.0f / 6.0f, S5 = 1.0f / 120.0f, S7 = -1.0f / 5040.0f,
                   S9 = 1.0f / 362880.0f;
static const float C2 = -0.5f, C4 = 1.0f / 24.0f, C6 = -1.0f / 720.0f, C8 = 1.0f / 40320.0f;

static void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

float cp_oracle_sin(float th)
{
    float z = th * th;
    float p = S9;
    p = p * z; p = p + S7;
    p = p * z; p = p + S5;
    p = p * z; p = p + S3;
    p = p * z; p = p + 1.0f;
    return th * p;
}

float cp_oracle_cos(float th)
{
    float z = th * th;
    float q = C8;
    q = q * z; q = q + C6;
    q = q * z; q = q + C4;
    q = q * z; q = q + C2;
    q = q * z; q = q + 1.0f;
    return q;
}

int cp_oracle_action(uint64_t seed, uint32_t env_id, uint64_t t)
{
    uint32_t ctr[4] = { (uint32_t)(t >> 2), env_id, (uint32_t)(t >> 34), 3u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    return (int)(out[t & 3u] & 1u);
}

static float uniform_start(uint32_t word)
{
    float f = (float)(word >> 8);        /* 24 bits: exact */
    f = f * 5.9604644775390625e-08f;      /* 2^-24: exact */
    f = f - 0.5f;                        /* exact */
    return f * 0.1f;                     /* one rounding */
}

void cp_oracle_reset_env(cp_env *e, uint64_t seed, uint32_t env_id, uint32_t episode)
{
    uint32_t ctr[4] = { 0u, episode, env_id, 2u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    philox4x32_10(ctr, key, out);
    e->x = uniform_start(out[0]);
    e->xd = uniform_start(out[1]);
    e->th = uniform_start(out[2]);
    e->thd = uniform_start(out[3]);
    e->steps = 0;
    e->episode = (int32_t)episode;
}

/* One step; returns done (0 / 1).  On done the env is already reset. */
int cp_oracle_step(cp_env *e, int action, uint64_t seed, uint32_t env_id, cp_stats *stats)
{
    float force = action ? CP_FORCE : -CP_FORCE;
    float s = cp_oracle_sin(e->th);
    float c = cp_oracle_cos(e->th);

    float t1 = e->thd * e->thd;
    float t2 = CP_POLEMASS_LENGTH * t1;
    float t3 = t2 * s;
    float t4 = force + t3;
    float temp = t4 / CP_TOTAL_MASS;

    float n1 = CP_GRAVITY * s;
    float n2 = c * temp;
    float num = n1 - n2;
    float c2 = c * c;
    float d1 = CP_MASSPOLE * c2;
    float d2 = d1 / CP_TOTAL_MASS;
    float d3 = CP_FOUR_THIRDS - d2;
    float den = CP_LENGTH * d3;
    float thetaacc = num / den;

    float m1 = CP_POLEMASS_LENGTH * thetaacc;
    float m2 = m1 * c;
    float m3 = m2 / CP_TOTAL_MASS;
    float xacc = temp - m3;

    float dx = CP_TAU * e->xd;
    float dxd = CP_TAU * xacc;
    float dth = CP_TAU * e->thd;
    float dthd = CP_TAU * thetaacc;
    e->x = e->x + dx;
    e->xd = e->xd + dxd;
    e->th = e->th + dth;
    e->thd = e->thd + dthd;
    e->steps += 1;

    int done = 0;
    if (e->x < -CP_X_LIMIT || e->x > CP_X_LIMIT) done = 1;
    if (e->th < -CP_TH_LIMIT || e->th > CP_TH_LIMIT) done = 1;
    if (e->steps >= CP_MAX_STEPS) done = 1;
    if (done) {
        if (stats) {
            stats->episodes += 1;
            stats->sum_length += e->steps;
        }
        cp_oracle_reset_env(e, seed, env_id, (uint32_t)e->episode + 1u);
    }
    return done;
}

void cp_oracle_reset(cp_env *envs, int n, uint64_t seed, uint32_t env_id_base)
{
    for (int i = 0; i < n; ++i) cp_oracle_reset_env(&envs[i], seed, env_id_base + (uint32_t)i, 0u);
}

void cp_oracle_obs(const cp_env *envs, int n, float *obs)
{
    for (int i = 0; i < n; ++i) {
        obs[4 * i + 0] = envs[i].x;
        obs[4 * i + 1] = envs[i].xd;
        obs[4 * i + 2] = envs[i].th;
        obs[4 * i + 3] = envs[i].thd;
    }
}

/* T steps of n envs from global step t0.  action_mode 0: Philox; 2: explicit
 * bytes actions[T][n] (bit 0); 3: the constant actions[0].  obs[T][n][4],
 * reward[T][n] (always 1), done[T][n].  Returns 0, or -1 on a bad mode. */
int cp_oracle_rollout(cp_env *envs, int n, uint64_t seed, uint32_t env_id_base, uint64_t t0, int T,
                      int action_mode, const uint8_t *actions, float *obs, float *reward,
                      uint8_t *done, cp_stats *stats)
{
    if (action_mode != 0 && action_mode != 2 && action_mode != 3) return -1;
    for (int t = 0; t < T; ++t) {
        for (int i = 0; i < n; ++i) {
            uint32_t env_id = env_id_base + (uint32_t)i;
            size_t o = (size_t)t * (size_t)n + (size_t)i;
            int a;
            if (action_mode == 0) a = cp_oracle_action(seed, env_id, t0 + (uint64_t)t);
            else if (action_mode == 2) a = actions[o] & 1u;
            else a = actions[0] & 1u;
            int d = cp_oracle_step(&envs[i], a, seed, env_id, stats);
            obs[4 * o + 0] = envs[i].x;
            obs[4 * o + 1] = envs[i].xd;
            obs[4 * o + 2] = envs[i].th;
            obs[4 * o + 3] = envs[i].thd;
            reward[o] = 1.0f;
            done[o] = (uint8_t)d;
        }
    }
    return 0;
}

int cp_oracle_sizeof_env(void) { return (int)sizeof(cp_env); }
