/*
 * pong_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, single-threaded CPU statement of the batched fixed-point
 * Pong environment step.  It exists so that the CUDA library can be checked
 * against something that can be verified by eye: one env at a time, an
 * array-of-structs state, ordinary `if` statements, no blocking, no fusion,
 * no tables, and its own Philox.  It shares no code, header, table or helper
 * with the CUDA path and must never be called by it.
 *
 * What it follows
 *   - The paper's equivalence contract (Sec. 3.1, "Problem Formulation"):
 *     two implementations are equivalent when obs, reward and done agree at
 *     every step for every seed and action sequence.  For this all-integer
 *     environment "agree" means bit for bit.
 *   - The paper's description of the performance path (Appendix
 *     "JAX Optimization Checklist"): a single-instance step applied to every
 *     env of a batch (item 3), a multi-step rollout that carries the states
 *     and stacks per-step outputs over T (item 5), observations normalised
 *     at the source with a pre-computed constant (item 8), pre-allocated
 *     output buffers (item 7); and, for pixels, the Rust checklist's item 3
 *     (with frame skip only the last frame is rendered).
 *   - The rule set itself (the paper does not print Pong's rules) is the
 *     Q8 fixed-point Pong restated in full in the comments below.
 *
 * Units: Q8 fixed point, 256 units = 1 pixel.  Court 160 x 192 px, y grows
 * downward.  A stored position is the top-left corner of the 2x2 ball or the
 * top edge of a 4x16 paddle.
 *
 * Parity pins (tests that do not need a GPU): Philox known answers and an
 * inverse-round check, hand-computed bounce / score / tracking values, a
 * closed-form rally, per-step invariants, brute force over all short action
 * sequences, exhaustive obs scaling against double precision, rasteriser
 * against paint-then-sample.  The relation of this rule set to the paper's
 * own Pong (whose rules are not published) is: parity unpinned.
 */
#include <stdint.h>
#include <string.h>

/* ---- constants of the rule set (Q8) ------------------------------------ */
enum {
    COURT_W   = 40960,  /* 160 px */
    BALL_SIZE = 512,    /* 2 px */
    BALL_Y_MAX = 48640, /* 190 px: lowest top edge of the ball */
    PAD_H     = 4096,   /* 16 px */
    PAD_W     = 1024,   /* 4 px */
    AGENT_X   = 37888,  /* 148 px */
    OPP_X     = 2048,   /* 8 px */
    PAD_Y_MAX = 45056,  /* 176 px */
    AGENT_SPEED = 768,  /* 3 px per frame */
    OPP_SPEED = 512,    /* 2 px per frame */
    VX_START  = 512,
    VX_INC    = 16,
    VX_CAP    = 1024,
    VY_SPAWN  = 384,
    VY_CAP    = 768,
    MAX_SCORE = 21,
    MAX_STEPS = 10000,
    SPAWN_BX  = 20224,  /* ball centred on x = 80 px */
    SPAWN_BY  = 24320,  /* ball centred on y = 96 px */
    PAD_Y_START = 22528 /* paddle centred on y = 96 px */
};

enum { FRAME_H = 84, FRAME_W = 84, FRAME_BYTES = 84 * 84, STACK = 4 };

typedef struct {
    int32_t bx, by, vx, vy;   /* ball corner and velocity */
    int32_t apy, opy;         /* agent / opponent paddle top edge */
    int32_t score_a, score_o; /* points of the agent / the opponent */
    int32_t ep_len;           /* physics frames in this episode */
    int32_t episode;          /* episodes finished by this env */
    int32_t prev_action;      /* last executed action (0 after a reset) */
} oracle_env;

typedef struct {
    int64_t episodes;   /* finished episodes */
    int64_t sum_return; /* sum over them of score_a - score_o */
    int64_t sum_length; /* sum over them of ep_len */
} oracle_stats;

/* ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11) ------------------ */
/* One round: two 32x32->64 products, a permutation with xors, then the key
 * is bumped by the Weyl constants.  Ten rounds. */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2],
                          uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* ---- random draws, all pure functions of counters ----------------------- */

/* The 32-bit word that decides the action of global agent step t in env
 * env_id: one Philox block serves four consecutive steps (counter word 0 is
 * t/4, the step uses output word t%4).  Bits of t above 2^34 go to counter
 * word 2 so that the draw stays a function of the whole 64-bit t. */
uint32_t oracle_action_word(uint64_t seed, uint32_t env_id, uint64_t t)
{
    uint32_t ctr[4] = { (uint32_t)(t >> 2), env_id, (uint32_t)(t >> 34), 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    return out[t & 3u];
}

/* Uniform action in {0 stay, 1 up, 2 down}: low 16 bits, multiply-high by 3. */
int oracle_action_uniform(uint32_t word)
{
    uint32_t u = word & 0xFFFFu;
    return (int)((u * 3u) >> 16);
}

/* Sticky decision: the high 16 bits fall below 16384 with probability 1/4. */
int oracle_action_repeat(uint32_t word)
{
    uint32_t s = word >> 16;
    return s < 16384u;
}

/* Ball spawn for (seed, env, episode, point): centre of the court, vx sign
 * from bit 0 of word 0, vy uniform in [-384, 384] from word 1. */
void oracle_spawn(oracle_env *e, uint64_t seed, uint32_t env_id,
                  uint32_t episode, uint32_t point)
{
    uint32_t ctr[4] = { point, episode, env_id, 1u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    e->bx = SPAWN_BX;
    e->by = SPAWN_BY;
    e->vx = (out[0] & 1u) ? VX_START : -VX_START;
    e->vy = (int32_t)(((uint64_t)out[1] * 769u) >> 32) - VY_SPAWN;
}

/* Start-of-episode state: a pure function of (seed, env, episode). */
void oracle_reset_env(oracle_env *e, uint64_t seed, uint32_t env_id,
                      uint32_t episode)
{
    e->score_a = 0;
    e->score_o = 0;
    e->ep_len = 0;
    e->prev_action = 0;
    e->episode = (int32_t)episode;
    e->apy = PAD_Y_START;
    e->opy = PAD_Y_START;
    oracle_spawn(e, seed, env_id, episode, 0u);
}

static int32_t clamp_i32(int32_t v, int32_t lo, int32_t hi)
{
    if (v < lo) return lo;
    if (v > hi) return hi;
    return v;
}

/* ---- one physics frame --------------------------------------------------- */
/* Returns the reward of the frame (-1, 0, +1); *done is set to 1 when the
 * episode ended on this frame, in which case the env has already been
 * auto-reset and the finished episode has been added to *stats. */
int oracle_frame(oracle_env *e, int action, uint64_t seed, uint32_t env_id,
                 oracle_stats *stats, int *done)
{
    /* 1. agent paddle: 1 = up (towards y = 0), 2 = down, 3 px per frame */
    if (action == 1) e->apy -= AGENT_SPEED;
    if (action == 2) e->apy += AGENT_SPEED;
    e->apy = clamp_i32(e->apy, 0, PAD_Y_MAX);

    /* 2. opponent paddle: towards the ball centre as it was before the ball
     *    moves, by at most 2 px */
    int32_t d = (e->by + BALL_SIZE / 2) - (e->opy + PAD_H / 2);
    e->opy += clamp_i32(d, -OPP_SPEED, OPP_SPEED);
    e->opy = clamp_i32(e->opy, 0, PAD_Y_MAX);

    /* 3. ball */
    e->bx += e->vx;
    e->by += e->vy;

    /* 4. top / bottom wall: mirror about the wall */
    if (e->by < 0) {
        e->by = -e->by;
        e->vy = -e->vy;
    } else if (e->by > BALL_Y_MAX) {
        e->by = 2 * BALL_Y_MAX - e->by;
        e->vy = -e->vy;
    }

    /* 5. paddle bounce: half-open boxes overlap and the ball is moving
     *    towards that paddle */
    int hit_agent = e->vx > 0 &&
                    e->bx + BALL_SIZE > AGENT_X && e->bx < AGENT_X + PAD_W &&
                    e->by + BALL_SIZE > e->apy && e->by < e->apy + PAD_H;
    int hit_opp = e->vx < 0 &&
                  e->bx + BALL_SIZE > OPP_X && e->bx < OPP_X + PAD_W &&
                  e->by + BALL_SIZE > e->opy && e->by < e->opy + PAD_H;
    if (hit_agent || hit_opp) {
        int32_t pad_y = hit_agent ? e->apy : e->opy;
        int32_t speed = e->vx > 0 ? e->vx : -e->vx;
        speed += VX_INC;
        if (speed > VX_CAP) speed = VX_CAP;
        e->vx = e->vx > 0 ? -speed : speed;
        /* centre offset in whole pixels; both centres are non-negative */
        int32_t dpx = ((e->by + BALL_SIZE / 2) >> 8) - ((pad_y + PAD_H / 2) >> 8);
        e->vy = clamp_i32(e->vy + 16 * dpx, -VY_CAP, VY_CAP);
    }

    /* 6. score: the ball's left edge is past the right / left court edge */
    int reward = 0;
    if (e->bx > COURT_W) {
        reward = 1;
        e->score_a += 1;
    } else if (e->bx < 0) {
        reward = -1;
        e->score_o += 1;
    }
    if (reward != 0)
        oracle_spawn(e, seed, env_id, (uint32_t)e->episode,
                     (uint32_t)(e->score_a + e->score_o));

    /* 7. count the frame; episode end */
    e->ep_len += 1;
    *done = (e->score_a == MAX_SCORE || e->score_o == MAX_SCORE ||
             e->ep_len == MAX_STEPS) ? 1 : 0;

    /* 8. auto-reset */
    if (*done) {
        if (stats) {
            stats->episodes += 1;
            stats->sum_return += e->score_a - e->score_o;
            stats->sum_length += e->ep_len;
        }
        oracle_reset_env(e, seed, env_id, (uint32_t)e->episode + 1u);
    }
    return reward;
}

/* ---- observations -------------------------------------------------------- */
/* Vector obs: six integers, each converted to float32 (exact, |v| < 2^24) and
 * multiplied once, round-to-nearest-even, by float32(1/40960). */
void oracle_obs_vector(const oracle_env *e, float out[6])
{
    const float scale = 1.0f / 40960.0f; /* 0x37CCCCCD */
    const int32_t v[6] = { e->bx, e->by, e->vx, e->vy, e->apy, e->opy };
    for (int k = 0; k < 6; ++k) {
        float f = (float)v[k];
        out[k] = f * scale; /* one fp32 multiply; never a division */
    }
}

/* Pixel obs: 84x84 nearest-neighbour sample of the 160x192 court.  Output
 * pixel (i, j) looks at source row i*192/84 and source column j*160/84
 * (integer division) and is 255 when a paddle or the ball covers that source
 * pixel, else 0.  Q8 positions become pixels by >> 8. */
void oracle_render(const oracle_env *e, uint8_t out[FRAME_BYTES])
{
    int ap = e->apy >> 8, op = e->opy >> 8, bxp = e->bx >> 8, byp = e->by >> 8;
    for (int i = 0; i < FRAME_H; ++i) {
        int sr = i * 192 / 84;
        for (int j = 0; j < FRAME_W; ++j) {
            int sc = j * 160 / 84;
            int lit = 0;
            if (sc >= 148 && sc < 152 && sr >= ap && sr < ap + 16) lit = 1;
            if (sc >= 8 && sc < 12 && sr >= op && sr < op + 16) lit = 1;
            if (sc >= bxp && sc < bxp + 2 && sr >= byp && sr < byp + 2) lit = 1;
            out[i * FRAME_W + j] = lit ? 255 : 0;
        }
    }
}

/* ---- batch drivers -------------------------------------------------------- */

void oracle_reset(oracle_env *envs, int n, uint64_t seed, uint32_t env_id_base)
{
    for (int i = 0; i < n; ++i)
        oracle_reset_env(&envs[i], seed, env_id_base + (uint32_t)i, 0u);
}

/* Initial observation after oracle_reset: vector obs[n,6], or the reset frame
 * in all four slots of ring[n,4,84,84]. */
void oracle_initial_obs(const oracle_env *envs, int n, int obs_mode,
                        float *obs_vec, uint8_t *ring)
{
    for (int i = 0; i < n; ++i) {
        if (obs_mode == 0) {
            oracle_obs_vector(&envs[i], obs_vec + (size_t)i * 6);
        } else {
            uint8_t *slot0 = ring + (size_t)i * STACK * FRAME_BYTES;
            oracle_render(&envs[i], slot0);
            for (int s = 1; s < STACK; ++s)
                memcpy(slot0 + (size_t)s * FRAME_BYTES, slot0, FRAME_BYTES);
        }
    }
}

/* Decode an explicit action byte: bit 2 set = repeat the previous action;
 * otherwise bits 0-1 are the action, the unused code 3 meaning "stay". */
int oracle_decode_action(uint8_t byte, int prev_action)
{
    if (byte & 4u) return prev_action;
    int a = byte & 3u;
    return a == 3 ? 0 : a;
}

/* T agent steps of n envs starting at global agent step t0.
 *   action_mode 0: Philox uniform; 1: Philox + sticky (repeat with p = 1/4);
 *               2: explicit bytes actions[T,n]; 3: the constant actions[0].
 *   frameskip   : physics frames per agent step; the action is repeated, the
 *                 rewards are summed, frames stop after the one that ends the
 *                 episode; only the last executed frame is observed.
 *   obs_mode 0  : obs_vec[T,n,6] float32.
 *   obs_mode 1  : ring[n,4,84,84] uint8, persistent across calls; agent step t
 *                 writes slot t%4; an auto-reset writes all four slots.
 *   reward[T,n] float32, done[T,n] uint8.  Returns 0, or -1 on a bad mode. */
int oracle_rollout(oracle_env *envs, int n, uint64_t seed, uint32_t env_id_base,
                   uint64_t t0, int T, int action_mode, const uint8_t *actions,
                   int frameskip, int obs_mode, float *obs_vec, uint8_t *ring,
                   float *reward, uint8_t *done, oracle_stats *stats)
{
    if (action_mode < 0 || action_mode > 3 || frameskip < 1) return -1;
    for (int t = 0; t < T; ++t) {
        uint64_t tt = t0 + (uint64_t)t;
        for (int i = 0; i < n; ++i) {
            oracle_env *e = &envs[i];
            uint32_t env_id = env_id_base + (uint32_t)i;
            size_t o = (size_t)t * (size_t)n + (size_t)i;

            int a;
            if (action_mode == 0) {
                a = oracle_action_uniform(oracle_action_word(seed, env_id, tt));
            } else if (action_mode == 1) {
                uint32_t w = oracle_action_word(seed, env_id, tt);
                a = oracle_action_repeat(w) ? e->prev_action
                                            : oracle_action_uniform(w);
            } else if (action_mode == 2) {
                a = oracle_decode_action(actions[o], e->prev_action);
            } else {
                a = oracle_decode_action(actions[0], 0);
            }
            e->prev_action = a;

            int rsum = 0, ended = 0;
            for (int k = 0; k < frameskip && !ended; ++k)
                rsum += oracle_frame(e, a, seed, env_id, stats, &ended);

            reward[o] = (float)rsum;
            done[o] = (uint8_t)ended;
            if (obs_mode == 0) {
                oracle_obs_vector(e, obs_vec + o * 6);
            } else {
                uint8_t *base = ring + (size_t)i * STACK * FRAME_BYTES;
                if (ended) {
                    oracle_render(e, base);
                    for (int s = 1; s < STACK; ++s)
                        memcpy(base + (size_t)s * FRAME_BYTES, base, FRAME_BYTES);
                } else {
                    oracle_render(e, base + (size_t)(tt & 3u) * FRAME_BYTES);
                }
            }
        }
    }
    return 0;
}

/* The action bytes that reproduce Philox modes 0 / 1 through the explicit
 * mode: the uniform action, plus bit 2 where the sticky draw says "repeat". */
void oracle_fill_actions(int n, uint64_t seed, uint32_t env_id_base, uint64_t t0,
                         int T, int sticky, uint8_t *actions)
{
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < n; ++i) {
            uint32_t w = oracle_action_word(seed, env_id_base + (uint32_t)i,
                                            t0 + (uint64_t)t);
            uint8_t b = (uint8_t)oracle_action_uniform(w);
            if (sticky && oracle_action_repeat(w)) b |= 4u;
            actions[(size_t)t * (size_t)n + (size_t)i] = b;
        }
}

int oracle_sizeof_env(void) { return (int)sizeof(oracle_env); }

/* ---- policy interface: sampling an action from three logits ---------------- */
/* Used when a policy network drives the env (the paper's "GRU rollout"
 * benchmark, Table "PufferLib comparisons"): the policy emits logits, an action
 * is drawn from softmax(logits) with one uniform number per env and step, and
 * the env steps on it.  The draw compares floating-point numbers, so it is
 * defined in binary32 with a fixed operation order and a fixed polynomial
 * exponential, and the uniform number is an input (the Philox action word of
 * that env and step), so that two implementations agree on every action.
 *
 *   m  = max(l0, l1, l2)
 *   ei = expn(li - m)                       expn(x) = e^x for x <= 0, below
 *   s  = (e0 + e1) + e2
 *   x  = ((float)(word >> 8) * 2^-24) * s   uniform in [0, s)
 *   a  = x < e0 ? 0 : (x < e0 + e1 ? 1 : 2)
 *
 * expn(x): y = x * log2(e); n = floor(y + 0.5); f = y - n in [-0.5, 0.5];
 * 2^f = ((((((P6 f + P5) f + P4) f + P3) f + P2) f + P1) f + 1 with the Taylor
 * coefficients Pk = ln(2)^k / k!; result = 2^f scaled by 2^n (exact), and 0
 * when n < -126.  Relative error below 3e-7 for |x| <= 1 and below 1e-6 for
 * |x| <= 8; for larger |x| the rounding of y dominates (4e-6 at x = -80), where the value no longer matters
 * to a softmax. */
float oracle_expn(float x)
{
    if (!(x <= 0.0f)) x = 0.0f;                 /* callers pass l - max <= 0; NaN -> 0 */
    float y = x * 1.44269504088896340736f;
    if (y < -150.0f) return 0.0f;               /* far below 2^-126; keeps the int conversion in range */
    float t = y + 0.5f;
    float n = (float)(int)t;                    /* truncation towards zero ... */
    if (n > t) n = n - 1.0f;                    /* ... made a floor: n = round(y) */
    if (n < -126.0f) return 0.0f;
    float f = y - n;
    float p = 1.5403530393381608e-4f;           /* ln2^6/720 */
    p = p * f; p = p + 1.3333558146428443e-3f;  /* ln2^5/120 */
    p = p * f; p = p + 9.6181291076284772e-3f;  /* ln2^4/24 */
    p = p * f; p = p + 5.5504108664821580e-2f;  /* ln2^3/6 */
    p = p * f; p = p + 2.4022650695910072e-1f;  /* ln2^2/2 */
    p = p * f; p = p + 6.9314718055994531e-1f;  /* ln2 */
    p = p * f; p = p + 1.0f;
    union { uint32_t u; float f; } scale;
    scale.u = (uint32_t)((int)n + 127) << 23;   /* 2^n, n in [-126, 0] */
    return p * scale.f;
}

int oracle_sample_action(const float logits[3], uint32_t word)
{
    float m = logits[0];
    if (logits[1] > m) m = logits[1];
    if (logits[2] > m) m = logits[2];
    float e0 = oracle_expn(logits[0] - m);
    float e1 = oracle_expn(logits[1] - m);
    float e2 = oracle_expn(logits[2] - m);
    float e01 = e0 + e1;
    float s = e01 + e2;
    float u = (float)(word >> 8);
    u = u * 5.9604644775390625e-08f;            /* 2^-24 */
    float x = u * s;
    if (x < e0) return 0;
    if (x < e01) return 1;
    return 2;
}

/* actions[n] from logits[n][3] and words[n] */
void oracle_sample_actions(int n, const float *logits, const uint32_t *words, uint8_t *actions)
{
    for (int i = 0; i < n; ++i) actions[i] = (uint8_t)oracle_sample_action(logits + 3 * i, words[i]);
}

/* The Philox action words of global steps t0 .. t0+T-1: words[T][n]. */
void oracle_fill_words(int n, uint64_t seed, uint32_t env_id_base, uint64_t t0, int T,
                       uint32_t *words)
{
    for (int t = 0; t < T; ++t)
        for (int i = 0; i < n; ++i)
            words[(size_t)t * (size_t)n + (size_t)i] =
                oracle_action_word(seed, env_id_base + (uint32_t)i, t0 + (uint64_t)t);
}
