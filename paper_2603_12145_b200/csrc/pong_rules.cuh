// Device-side rules of the fixed-point Pong environment: Philox4x32-10, the
// random draws, one physics frame, state packing and observation scaling.
// Everything is integer except the final obs multiply.  Written for sm_100a.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace pong {

// ---- constants (Q8: 256 units = 1 px) -----------------------------------------
constexpr int kCourtW    = 40960;  // 160 px
constexpr int kBallYMax  = 48640;  // 190 px
constexpr int kPadYMax   = 45056;  // 176 px
constexpr int kAgentStep = 768;    // 3 px
constexpr int kOppStep   = 512;    // 2 px
constexpr int kVx0       = 512;
constexpr int kVxInc     = 16;
constexpr int kVxCap     = 1024;
constexpr int kVySpawn   = 384;
constexpr int kVyCap     = 768;
constexpr int kMaxScore  = 21;
constexpr int kMaxFrames = 10000;
constexpr int kSpawnBx   = 20224;
constexpr int kSpawnBy   = 24320;
constexpr int kPadY0     = 22528;
// Ball box vs paddle box, folded into one unsigned range test per axis:
//   bx + 512 > X and bx < X + 1024   <=>  (unsigned)(bx - (X - 511)) < 1535
//   by + 512 > p and by < p + 4096   <=>  (unsigned)(by - p + 511)   < 4607
constexpr int kAgentXLo  = 37888 - 511;
constexpr int kOppXLo    = 2048 - 511;
constexpr unsigned kHitXSpan = 1535u;
constexpr unsigned kHitYSpan = 4607u;

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

constexpr int kFrameH = 84, kFrameW = 84, kFrameBytes = 84 * 84, kStack = 4;

// The ten round keys of a seed, computed once on the host so that a round is
// two wide multiplies and two three-input xors.
struct RoundKeys {
    uint32_t k[20];
};

// Env state held in registers.
struct Env {
    int bx, by, vx, vy;  // ball corner, velocity
    int apy, opy;        // paddle top edges
    int sa, so;          // points of agent / opponent
    int len;             // frames in this episode
    int episode;         // finished episodes
    int prev;            // last executed action
};

// Per-thread episode statistics of one launch.
struct Tally {
    int episodes, sum_return, sum_length;
};

// HBM layout: two int4 planes.  plane0[n] = {bx, by, vx, vy};
// plane1[n] = {apy, opy, packed, episode}, packed = score_a (5 bits) |
// score_o (5) << 5 | ep_len (14) << 10 | prev_action (2) << 24.
__device__ __forceinline__ int pack_counters(const Env &e)
{
    return e.sa | (e.so << 5) | (e.len << 10) | (e.prev << 24);
}

__device__ __forceinline__ void load_env(Env &e, const int4 *__restrict__ plane0,
                                         const int4 *__restrict__ plane1, int n)
{
    const int4 a = plane0[n];
    const int4 b = plane1[n];
    e.bx = a.x; e.by = a.y; e.vx = a.z; e.vy = a.w;
    e.apy = b.x; e.opy = b.y; e.episode = b.w;
    e.sa = b.z & 31;
    e.so = (b.z >> 5) & 31;
    e.len = (b.z >> 10) & 0x3FFF;
    e.prev = (b.z >> 24) & 3;
}

__device__ __forceinline__ void store_env(const Env &e, int4 *__restrict__ plane0,
                                          int4 *__restrict__ plane1, int n)
{
    plane0[n] = make_int4(e.bx, e.by, e.vx, e.vy);
    plane1[n] = make_int4(e.apy, e.opy, pack_counters(e), e.episode);
}

// ---- Philox4x32-10 -------------------------------------------------------------
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2,
                                              uint32_t c3, const RoundKeys &rk,
                                              uint32_t (&out)[4])
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * c0;
        const uint64_t p1 = (uint64_t)kPhiloxM1 * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk.k[2 * r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk.k[2 * r + 1];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Four action words for global steps 4g .. 4g+3 of env `env_id`.
__device__ __forceinline__ void action_words(uint64_t group, uint32_t env_id,
                                             const RoundKeys &rk, uint32_t (&w)[4])
{
    philox4x32_10((uint32_t)group, env_id, (uint32_t)(group >> 32), 0u, rk, w);
}

// (u * 3) >> 16 for the low half-word u, written as the high word of (u << 16) * 3: a shift
// and a multiply-high (which runs on the multiply pipe, not the integer ALU's).
__device__ __forceinline__ int uniform_action(uint32_t word)
{
    return (int)__umulhi(word << 16, 3u);
}

__device__ __forceinline__ bool sticky_repeat(uint32_t word)
{
    return word < (16384u << 16);  // high half-word below 16384
}

__device__ __forceinline__ int decode_action_byte(uint32_t byte, int prev)
{
    const int a = byte & 3u;
    return (byte & 4u) ? prev : (a == 3 ? 0 : a);
}

// Ball spawn keyed by (seed, env, episode, point).
__device__ __forceinline__ void spawn_ball(Env &e, uint32_t env_id, uint32_t episode,
                                           uint32_t point, const RoundKeys &rk)
{
    uint32_t o[4];
    philox4x32_10(point, episode, env_id, 1u, rk, o);
    e.bx = kSpawnBx;
    e.by = kSpawnBy;
    e.vx = (o[0] & 1u) ? kVx0 : -kVx0;
    e.vy = (int)__umulhi(o[1], 769u) - kVySpawn;
}

__device__ __forceinline__ void reset_env(Env &e, uint32_t env_id, uint32_t episode,
                                          const RoundKeys &rk)
{
    e.sa = 0; e.so = 0; e.len = 0; e.prev = 0;
    e.episode = (int)episode;
    e.apy = kPadY0;
    e.opy = kPadY0;
    spawn_ball(e, env_id, episode, 0u, rk);
}

// ---- one physics frame ------------------------------------------------------------
// Returns the reward (-1, 0, +1); `done` says the episode ended on this frame
// (the env is then already reset and the episode is in `tally`).
__device__ __forceinline__ int physics_frame(Env &e, int action, uint32_t env_id,
                                             const RoundKeys &rk, Tally &tally, bool &done)
{
    // 1. agent paddle
    const int delta = action == 2 ? kAgentStep : (action == 1 ? -kAgentStep : 0);
    e.apy = min(max(e.apy + delta, 0), kPadYMax);
    // 2. opponent paddle follows the ball centre as it is before the ball moves:
    //    (by + 256) - (opy + 2048)
    const int d = e.by - e.opy - 1792;
    e.opy = min(max(e.opy + min(max(d, -kOppStep), kOppStep), 0), kPadYMax);
    // 3. ball, 4. walls: mirroring about y = 0 is |y|, about y = 48640 is
    //    97280 - y; the reflected value is always the smaller of the two.
    e.bx += e.vx;
    const int raw = e.by + e.vy;
    const int a = abs(raw);
    const int by = min(a, 2 * kBallYMax - a);
    e.vy = (by != raw) ? -e.vy : e.vy;
    e.by = by;
    // 5. paddle bounce against the paddle the ball is moving towards
    const bool right = e.vx > 0;
    const int px = right ? kAgentXLo : kOppXLo;
    const int py = right ? e.apy : e.opy;
    const bool hit = (unsigned)(e.bx - px) < kHitXSpan &&
                     (unsigned)(e.by - py + 511) < kHitYSpan;
    if (hit) {
        const int s = min(abs(e.vx) + kVxInc, kVxCap);
        e.vx = right ? -s : s;
        const int dpx = ((e.by + 256) >> 8) - ((py + 2048) >> 8);
        e.vy = min(max(e.vy + 16 * dpx, -kVyCap), kVyCap);
    }
    // 6.-8. score, frame count, episode end.  bx < 0 wraps to a huge unsigned.
    e.len += 1;
    int reward = 0;
    done = false;
    const bool scored = (unsigned)e.bx > (unsigned)kCourtW;
    if (scored || e.len == kMaxFrames) {
        if (scored) {
            reward = e.bx > 0 ? 1 : -1;
            e.sa += e.bx > 0 ? 1 : 0;
            e.so += e.bx > 0 ? 0 : 1;
        }
        done = e.sa == kMaxScore || e.so == kMaxScore || e.len == kMaxFrames;
        if (done) {
            tally.episodes += 1;
            tally.sum_return += e.sa - e.so;
            tally.sum_length += e.len;
            e.sa = 0; e.so = 0; e.len = 0; e.prev = 0;
            e.episode += 1;
            e.apy = kPadY0;
            e.opy = kPadY0;
        }
        // a point respawns the ball with point = total points so far; an
        // episode end spawns the first ball of the next episode (point 0)
        spawn_ball(e, env_id, (uint32_t)e.episode, (uint32_t)(e.sa + e.so), rk);
    }
    return reward;
}

// `frameskip` frames with the action repeated; stops after a frame that ends
// the episode.  Returns the summed reward.
template <int FS>
__device__ __forceinline__ int agent_step(Env &e, int action, int frameskip_rt,
                                          uint32_t env_id, const RoundKeys &rk,
                                          Tally &tally, bool &done)
{
    e.prev = action;
    if (FS == 1) {
        return physics_frame(e, action, env_id, rk, tally, done);
    } else {
        const int fs = FS > 0 ? FS : frameskip_rt;
        int rsum = 0;
        done = false;
        for (int k = 0; k < fs && !done; ++k)
            rsum += physics_frame(e, action, env_id, rk, tally, done);
        return rsum;
    }
}

// ---- warp-uniform variant of the frame ------------------------------------------------
// Same arithmetic as physics_frame, organised for a warp whose 32 lanes are all
// live: the two rare paths (paddle bounce, score / episode end) sit behind
// warp-uniform votes and commit their results per lane with selects, so the common
// path is straight-line code.  The frame counter is kept as frames left in the
// episode (kMaxFrames - len) so that the end test is a compare with zero.
//
// With QUEUE, spawns come from a two-entry queue per lane.  A spawn is a pure function
// of (seed, env, episode, point), and the points of an episode are used in order, so the
// spawns an env will need next are known in advance: entry 0 is the spawn of its next
// point in the current episode, entry 1 the one after.  Some lane of a warp scores in
// about every third step, and a Philox block run for it costs the whole warp as much as
// one run for all 32 lanes; with the queue the warp runs Philox only when a lane that
// needs a spawn has none stored (or starts a new episode), and then restocks every
// lane's queue with the same two blocks.  An entry is 11 bits: vy + 384 (0..768) and,
// in bit 10, the sign of vx; 0x7FF marks an empty slot.  Without QUEUE every event runs
// its own Philox block.  Both give the same values; which is faster depends on the launch
// (see the launcher).
struct FastEnv {
    int bx, by, vx, vy, apy, opy;
    int sa, so, left, episode, prev;
    uint32_t spawns;   // entry 0 in bits 0..10, entry 1 in bits 11..21, ones above
};

constexpr uint32_t kSpawnEmpty = 0x7FFu;

__device__ __forceinline__ void to_fast(FastEnv &f, const Env &e)
{
    f.bx = e.bx; f.by = e.by; f.vx = e.vx; f.vy = e.vy; f.apy = e.apy; f.opy = e.opy;
    f.sa = e.sa; f.so = e.so; f.left = kMaxFrames - e.len; f.episode = e.episode; f.prev = e.prev;
    f.spawns = 0xFFFFFFFFu;   // the queue lives within a launch; it starts empty
}

__device__ __forceinline__ void from_fast(Env &e, const FastEnv &f)
{
    e.bx = f.bx; e.by = f.by; e.vx = f.vx; e.vy = f.vy; e.apy = f.apy; e.opy = f.opy;
    e.sa = f.sa; e.so = f.so; e.len = kMaxFrames - f.left; e.episode = f.episode; e.prev = f.prev;
}

// The queue entry of the ball spawned for (episode, point).
__device__ __forceinline__ uint32_t spawn_entry(uint32_t env_id, uint32_t episode, uint32_t point,
                                                const RoundKeys &rk)
{
    uint32_t o[4];
    philox4x32_10(point, episode, env_id, 1u, rk, o);
    return __umulhi(o[1], 769u) | ((o[0] & 1u) << 10);
}

// Score and / or episode end.  Run by the whole warp when any lane has an event;
// only lanes with `ev` commit.  `out` says the ball left the court on this lane.
// `reward` and `done` point at this lane's entries of the staged output rows, which the caller
// has zeroed: only a lane with an event writes them.
template <bool QUEUE>
__device__ __forceinline__ void fast_event(FastEnv &e, bool ev, bool out, uint32_t env_id,
                                           const RoundKeys &rk, Tally &tally, float *reward,
                                           uint8_t *done)
{
    const bool agent_point = e.bx > 0;
    int sa = e.sa + ((out && agent_point) ? 1 : 0);
    int so = e.so + ((out && !agent_point) ? 1 : 0);
    const float r = out ? (agent_point ? 1.f : -1.f) : 0.f;
    const bool dn = sa == kMaxScore || so == kMaxScore || e.left == 0;
    const bool fin = ev && dn;
    tally.episodes += fin ? 1 : 0;
    tally.sum_return += fin ? (sa - so) : 0;
    tally.sum_length += fin ? (kMaxFrames - e.left) : 0;
    const int episode = e.episode + (dn ? 1 : 0);
    sa = dn ? 0 : sa;
    so = dn ? 0 : so;
    uint32_t ent;   // the spawn of this lane's event, as a queue entry
    if (QUEUE) {
        // A new episode makes the stored spawns stale; an empty queue has none.
        const bool need = ev && (dn || (e.spawns & kSpawnEmpty) == kSpawnEmpty);
        if (__any_sync(0xffffffffu, need)) {
            // Restock every lane: a lane with an event takes the spawn of its new point count
            // now, any other lane will next need the one after its current count.
            const uint32_t ep = (uint32_t)(ev ? episode : e.episode);
            const uint32_t point = (uint32_t)(ev ? sa + so : e.sa + e.so + 1);
            const uint32_t e0 = spawn_entry(env_id, ep, point, rk);
            const uint32_t e1 = spawn_entry(env_id, ep, point + 1u, rk);
            e.spawns = e0 | (e1 << 11) | 0xFFC00000u;
        }
        ent = e.spawns & kSpawnEmpty;
        // bit 31 is set: ones move in, the freed slot reads empty
        if (ev) e.spawns = (uint32_t)((int)e.spawns >> 11);
    } else {
        ent = spawn_entry(env_id, (uint32_t)episode, (uint32_t)(sa + so), rk);
    }
    if (ev) {
        e.sa = sa; e.so = so; e.episode = episode;
        e.bx = kSpawnBx; e.by = kSpawnBy;
        e.vx = (ent & 0x400u) ? kVx0 : -kVx0;
        e.vy = (int)(ent & 0x3FFu) - kVySpawn;
        *reward = r;
        *done = dn ? 1 : 0;
        if (dn) { e.left = kMaxFrames; e.apy = kPadY0; e.opy = kPadY0; e.prev = 0; }
    }
}

// One frame; all 32 lanes of the warp must call it together.  The reward and done entries
// (pre-zeroed by the caller) are written only on a point or an episode end.
template <bool QUEUE>
__device__ __forceinline__ void fast_frame(FastEnv &e, int action, uint32_t env_id,
                                           const RoundKeys &rk, Tally &tally, float *reward,
                                           uint8_t *done)
{
    // 0, -768, +768 for action 0, 1, 2 as the polynomial (1152 a - 1920) a: two multiply-adds
    // on the multiply pipe instead of two compares and two selects on the integer ALU
    const int delta = (action * (3 * kAgentStep / 2) - (5 * kAgentStep / 2)) * action;
    e.apy = min(max(e.apy + delta, 0), kPadYMax);
    const int d = e.by - e.opy - 1792;
    e.opy = min(max(e.opy + min(max(d, -kOppStep), kOppStep), 0), kPadYMax);
    e.bx += e.vx;
    const int raw = e.by + e.vy;
    const int a = abs(raw);
    const int by = min(a, 2 * kBallYMax - a);
    e.vy = (by != raw) ? -e.vy : e.vy;
    e.by = by;
    const bool right = e.vx > 0;
    const int px = right ? kAgentXLo : kOppXLo;
    const int py = right ? e.apy : e.opy;
    const bool hit = (unsigned)(e.bx - px) < kHitXSpan &&
                     (unsigned)(e.by - py + 511) < kHitYSpan;
    if (__any_sync(0xffffffffu, hit)) {
        const int s = min(abs(e.vx) + kVxInc, kVxCap);
        const int nvx = right ? -s : s;
        const int dpx = ((e.by + 256) >> 8) - ((py + 2048) >> 8);
        const int nvy = min(max(e.vy + 16 * dpx, -kVyCap), kVyCap);
        e.vx = hit ? nvx : e.vx;
        e.vy = hit ? nvy : e.vy;
    }
    e.left -= 1;
    const bool out = (unsigned)e.bx > (unsigned)kCourtW;
    const bool ev = out || e.left == 0;
    if (__any_sync(0xffffffffu, ev)) fast_event<QUEUE>(e, ev, out, env_id, rk, tally, reward, done);
}

// Philox4x32-10 advanced a few rounds at a time, so that the block for the next
// four steps can be interleaved with the physics of the current four.
struct PhiloxPipe {
    uint32_t c0, c1, c2, c3;
};

__device__ __forceinline__ void philox_start(PhiloxPipe &p, unsigned long long group, uint32_t env_id)
{
    p.c0 = (uint32_t)group; p.c1 = env_id; p.c2 = (uint32_t)(group >> 32); p.c3 = 0u;
}

template <int R0, int R1>
__device__ __forceinline__ void philox_rounds(PhiloxPipe &p, const RoundKeys &rk)
{
#pragma unroll
    for (int r = R0; r < R1; ++r) {
        const uint64_t p0 = (uint64_t)kPhiloxM0 * p.c0;
        const uint64_t p1 = (uint64_t)kPhiloxM1 * p.c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ p.c1 ^ rk.k[2 * r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ p.c3 ^ rk.k[2 * r + 1];
        p.c1 = (uint32_t)p1;
        p.c3 = (uint32_t)p0;
        p.c0 = n0;
        p.c2 = n2;
    }
}

// ---- policy interface: one action from three logits and one uniform word -------------
// e^x for x <= 0 in binary32, fixed order: y = x*log2(e), n = round(y), f = y - n in
// [-0.5, 0.5], 2^f by a degree-6 polynomial, scaled by 2^n through the exponent bits.
__device__ __forceinline__ float expn(float x)
{
    if (!(x <= 0.0f)) x = 0.0f;
    const float y = __fmul_rn(x, 1.44269504088896340736f);
    if (y < -150.0f) return 0.0f;
    const float n = floorf(__fadd_rn(y, 0.5f));
    if (n < -126.0f) return 0.0f;
    const float f = __fsub_rn(y, n);
    float p = 1.5403530393381608e-4f;
    p = __fadd_rn(__fmul_rn(p, f), 1.3333558146428443e-3f);
    p = __fadd_rn(__fmul_rn(p, f), 9.6181291076284772e-3f);
    p = __fadd_rn(__fmul_rn(p, f), 5.5504108664821580e-2f);
    p = __fadd_rn(__fmul_rn(p, f), 2.4022650695910072e-1f);
    p = __fadd_rn(__fmul_rn(p, f), 6.9314718055994531e-1f);
    p = __fadd_rn(__fmul_rn(p, f), 1.0f);
    return __fmul_rn(p, __int_as_float((__float2int_rn(n) + 127) << 23));
}

__device__ __forceinline__ int sample_action(float l0, float l1, float l2, uint32_t word)
{
    const float m = fmaxf(fmaxf(l0, l1), l2);
    const float e0 = expn(__fsub_rn(l0, m));
    const float e1 = expn(__fsub_rn(l1, m));
    const float e2 = expn(__fsub_rn(l2, m));
    const float e01 = __fadd_rn(e0, e1);
    const float s = __fadd_rn(e01, e2);
    const float u = __fmul_rn(__uint2float_rn(word >> 8), 5.9604644775390625e-08f);
    const float x = __fmul_rn(u, s);
    return x < e0 ? 0 : (x < e01 ? 1 : 2);
}

// ---- observations -----------------------------------------------------------------
// float32(v) is exact (|v| < 2^24); one round-to-nearest multiply by
// float32(1/40960) = 0x37CCCCCD.  Never a division, never fused.
__device__ __forceinline__ float scale_obs(int v)
{
    return __fmul_rn(__int2float_rn(v), __int_as_float(0x37CCCCCD));
}

// Whole-pixel geometry of a frame packed in one word: agent paddle row |
// opponent paddle row << 8 | ball column << 16 | ball row << 24 (all <= 190).
__device__ __forceinline__ uint32_t pack_geometry(const Env &e)
{
    return (uint32_t)(e.apy >> 8) | ((uint32_t)(e.opy >> 8) << 8) |
           ((uint32_t)(e.bx >> 8) << 16) | ((uint32_t)(e.by >> 8) << 24);
}

}  // namespace pong
