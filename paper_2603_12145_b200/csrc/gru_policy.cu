// gru_policy.cu -- the recurrent policy of the policy-in-the-loop rollout (the
// paper's "GRU rollout (~2M parameters)" setting, Table "PufferLib comparisons";
// Sec. 4, time breakdown) as sm_100a kernels behind the C ABI of gru_policy.h.
//
// k_gru_cell is the dense part: per 256-env tile and 64-unit slice of the hidden
// state it forms the four pre-activation blocks
//     nx = x W_in^T        r = x W_ir^T + h W_hr^T
//     nh = h W_hn^T        z = x W_iz^T + h W_hz^T
// on the tensor cores (tcgen05.mma, bfloat16 operands staged in shared memory by
// TMA with the 128-byte swizzle, binary32 accumulators in tensor memory) and
// applies biases, gates and the blend in the epilogue straight out of tensor
// memory.  The weights are packed at create time so that one 192-row box holds
// the three gate blocks a stage needs: [n | r | z] rows for the x half of the
// reduction, [r | z | n] for the h half.  With the accumulator columns laid out
// as [nx | r | z | nh], the x half is one N = 192 instruction into columns 0..191
// and the h half one N = 192 instruction into columns 64..255, so r and z collect
// both halves and the two candidate parts stay separate, as the reset gate needs.
// Every MMA accumulates; the epilogue clears an accumulator buffer after reading it.
//
// The kernel runs as clusters of two blocks on the two SMs of a TPC
// (cta_group::2): each block stages its own 128 rows of x / h and HALF of the
// weight box (96 rows), the leader block issues M = 256 instructions that read
// both blocks' shared memory and write both blocks' tensor memory.  A stage is
// 28 KB per block, so shared memory and L2 see 30 % less traffic per tile than
// with one block per tile, which is what bounds this shape.
//
// Roles in a 320-thread block (one block per SM, persistent over tiles):
//   warp 0    TMA producer (one lane): fills a 7-deep ring of {x|h tile, half weight box};
//             both blocks' copies complete on the LEADER's full barrier
//   warp 1    allocates tensor memory; in the leader one lane issues the MMAs and
//             commits to the empty / accumulator-full barriers of both blocks
//   warps 2-9 epilogue: tcgen05.ld, gates, bfloat16 store, tcgen05.st of zeros (a warp
//             may touch only its own quarter of the 128 lanes, so two warps share a
//             quarter and split the 64 columns); two accumulator buffers (2 x 256
//             columns) let the epilogue overlap the next tile's MMAs; both blocks'
//             epilogue warps arrive on the leader's accumulator-empty barrier
// Every mbarrier wait is bounded by a wall-clock limit; a wait that runs out
// raises the block's abort flag, all roles leave their loops, the error word is
// set and the block still frees its tensor memory.
#include <cstdint>
#include <cstring>
#include <new>
#include <vector>

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/gru_policy.h"

namespace {

constexpr int kBM = 128;                         // envs per tile (MMA M)
constexpr int kBK = 64;                          // reduction elements per stage = one 128-byte row
constexpr int kHT = 64;                          // hidden units per tile
constexpr int kBN = 3 * kHT;                     // weight rows per stage (MMA N)
constexpr int kStages = 7;
constexpr int kABytes = kBM * kBK * 2;           // 16 KB: this block's 128 rows
constexpr int kBRows = kBN / 2;                  // this block's half of the weight box
constexpr int kBBytes = kBRows * kBK * 2;        // 12 KB
constexpr int kStageBytes = kABytes + kBBytes;   // 28 KB per block, 56 KB per pair
constexpr int kAccCols = 4 * kHT;                // one accumulator buffer: nx | r | z | nh
constexpr int kTmemCols = 2 * kAccCols;          // 512: all of tensor memory
constexpr int kEpilogueWarps = 8;
constexpr int kCellThreads = 64 + 32 * kEpilogueWarps;
constexpr int kBarrierBytes = 256;
// dynamic shared memory: the stage ring, the barriers, four binary32 bias vectors, the head's weights
// as [H][4], slack to align to 1024
constexpr int cell_smem_bytes(int H, bool with_head)
{
    return kStages * kStageBytes + kBarrierBytes + (with_head ? 8 : 4) * H * 4 + 1024;
}
constexpr int kMaxSmem = 227 * 1024;   // per block on sm_100
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s: far beyond any legitimate wait
constexpr unsigned long long kDrainNs = 200000ull;          // let copies in flight land after an abort

static_assert(kTmemCols == 512, "two accumulator buffers fill tensor memory");
static_assert(kStageBytes % 1024 == 0 && kABytes % 1024 == 0, "swizzled tiles need 1024-byte alignment");

// ---------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}

// Waits for the phase of the given parity to complete.  Gives up (and raises the
// block's abort flag) after kWaitLimitNs, or as soon as another role has raised it.
__device__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    unsigned long long t0 = 0;
    for (uint32_t spin = 0;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 63u) {
            if (*abort_flag) return false;
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}

__device__ __forceinline__ uint32_t cluster_cta_rank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

// The shared::cluster address of this block's shared address `addr` in block `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}

__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// Tile load of this block of the pair; `bar` is a shared::cluster address and may be the peer's barrier.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before_sync()
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_after_sync()
{
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t slot, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot),
                 "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols)
                 : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T over the pair: 256 rows (128 per block), bfloat16
// operands, binary32 accumulate; each block supplies its rows of A and half of B's rows.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                          uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The mbarrier at this shared-memory offset in BOTH blocks of the pair receives one
// arrival once every MMA issued so far by this thread is done.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
        "h"(static_cast<uint16_t>(3))
        : "memory");
}

// 16 consecutive accumulator columns of this thread's lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, "
        "%12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]),
          "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]),
          "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_wait_ld()
{
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Clears 16 consecutive accumulator columns of this thread's lane.
__device__ __forceinline__ void tmem_zero16(uint32_t taddr)
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, "
        "%1, %1, %1, %1};" ::"r"(taddr),
        "r"(0u)
        : "memory");
}

__device__ __forceinline__ void tmem_wait_st()
{
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Shared-memory operand descriptor of a K-major tile whose rows are 128 bytes
// (64 bfloat16) with the 128-byte swizzle, as TMA writes it: 8-row groups are
// 1024 bytes apart (stride offset), the leading offset is not used by swizzled
// K-major layouts (set to 1), descriptor version 1, layout type 2 = 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr)
{
    return static_cast<uint64_t>((addr >> 4) & 0x3FFFu) | (1ull << 16) | (64ull << 32) | (1ull << 46) |
           (2ull << 61);
}

// Instruction descriptor: binary32 accumulator, bfloat16 A and B, both K-major,
// M = 256 across the pair.
__host__ __device__ constexpr uint32_t instr_desc(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
           (static_cast<uint32_t>((2 * kBM) >> 4) << 24);
}

__device__ __forceinline__ float ex2_approx(float v)
{
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}

__device__ __forceinline__ float rcp_approx(float v)
{
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}

constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}

struct CellArgs {
    const __nv_bfloat16 *h_in;
    __nv_bfloat16 *h_out;
    const float *b_r;   // -log2(e) * (b_ir + b_hr): the sigmoid's exponent is a single fma
    const float *b_z;   // -log2(e) * (b_iz + b_hz)
    const float *b_in;
    const float *b_hn;
    const float *head_w4;   // [H][4]: the head's weights by hidden unit, or nullptr (no partial sums)
    float4 *partial;        // [n][H/32]: the head's partial sums of each block of 32 units of h'
    int n;
    int H;
    int *err;
};

// ---------------------------------------------------------------- the cell

__global__ void __launch_bounds__(kCellThreads, 1)
k_gru_cell(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_h,
           const __grid_constant__ CUtensorMap tm_wx, const __grid_constant__ CUtensorMap tm_wh,
           const CellArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;           // stage ring, 1024-byte aligned
    const uint32_t bars = tiles + kStages * kStageBytes;     // mbarriers, 8 bytes each
    uint8_t *bars_ptr = smem_raw + (bars - raw);
    const uint32_t full0 = bars, empty0 = bars + 8 * kStages;
    const uint32_t acc_full0 = bars + 16 * kStages, acc_empty0 = acc_full0 + 16;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(bars_ptr + 16 * kStages + 32);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars_ptr + 16 * kStages + 40);
    float *bias_s = reinterpret_cast<float *>(bars_ptr + kBarrierBytes);   // [4][H]: r, z, in, hn
    float4 *head_s = reinterpret_cast<float4 *>(bias_s + 4 * a.H);         // [H]: the head's weights of a unit

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();        // 0 = leader of the pair
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int KC = a.H / kBK;                 // reduction chunks per half
    const int JT = a.H / kHT;                 // hidden tiles
    const int m_tiles = (a.n + 2 * kBM - 1) / (2 * kBM);
    const int n_tasks = m_tiles * JT;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full0 + 8 * s, 1);     // the leader's own arrive.expect_tx (used in the leader only)
            mbar_init(empty0 + 8 * s, 1);    // one commit from the leader's MMA thread
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full0 + 8 * b, 1);
            mbar_init(acc_empty0 + 8 * b, 2 * kEpilogueWarps);   // both blocks' epilogue warps (leader only)
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(const_cast<uint32_t *>(tmem_slot)), kTmemCols);
    for (int i = threadIdx.x; i < a.H; i += kCellThreads) {
        bias_s[i] = a.b_r[i];
        bias_s[a.H + i] = a.b_z[i];
        bias_s[2 * a.H + i] = a.b_in[i];
        bias_s[3 * a.H + i] = a.b_hn[i];
        if (a.head_w4 != nullptr) head_s[i] = reinterpret_cast<const float4 *>(a.head_w4)[i];
    }
    tc_fence_before_sync();
    cluster_sync_all();          // both blocks' barriers and tensor memory exist from here on
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t s = 0, ph = 0;
            bool ok = true;
            for (int task = pair; task < n_tasks && ok; task += n_pairs) {
                const int mt = task / JT, j = task - mt * JT;
                const int row0 = (2 * mt + static_cast<int>(rank)) * kBM;
                const int wrow0 = j * kBN + static_cast<int>(rank) * kBRows;
                for (int half = 0; half < 2 && ok; ++half) {
                    const CUtensorMap *ta = half ? &tm_h : &tm_x;
                    const CUtensorMap *tb = half ? &tm_wh : &tm_wx;
                    for (int kc = 0; kc < KC; ++kc) {
                        if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) {
                            ok = false;
                            break;
                        }
                        const uint32_t dst = tiles + s * kStageBytes;
                        const uint32_t leader_full = map_to_rank(full0 + 8 * s, 0);
                        if (rank == 0) mbar_expect_tx(full0 + 8 * s, 2 * kStageBytes);
                        tma_load_2d(dst, ta, kc * kBK, row0, leader_full);
                        tma_load_2d(dst + kABytes, tb, kc * kBK, wrow0, leader_full);
                        if (++s == kStages) {
                            s = 0;
                            ph ^= 1u;
                        }
                    }
                }
            }
            // do not leave while the leader's MMAs may still read this block's stages
            for (int i = 0; i < kStages && ok; ++i) {
                ok = mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag);
                if (++s == kStages) {
                    s = 0;
                    ph ^= 1u;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t kIdesc = instr_desc(kBN);
            uint32_t s = 0, ph = 0;
            bool ok = true;
            int it = 0;
            for (int task = pair; task < n_tasks && ok; task += n_pairs, ++it) {
                const uint32_t buf = it & 1, use = (it >> 1) & 1;
                if (!mbar_wait(acc_empty0 + 8 * buf, use, abort_flag)) break;   // cleared by both epilogues
                tc_fence_after_sync();
                const uint32_t d = tmem_base + buf * kAccCols;
                for (int half = 0; half < 2 && ok; ++half) {
                    const uint32_t dh = d + (half ? kHT : 0);   // x half: nx|r|z, h half: r|z|nh
                    for (int kc = 0; kc < KC; ++kc) {
                        if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) {
                            ok = false;
                            break;
                        }
                        tc_fence_after_sync();
                        const uint32_t a_addr = tiles + s * kStageBytes;
                        const uint64_t ad = smem_desc(a_addr), bd = smem_desc(a_addr + kABytes);
#pragma unroll
                        for (int k = 0; k < kBK / 16; ++k) {
                            // 16 elements = 32 bytes further along the swizzled row: +2 in the address field
                            umma_bf16(dh, ad + 2u * k, bd + 2u * k, kIdesc, 1u);
                        }
                        umma_commit_pair(empty0 + 8 * s);   // both blocks' stages are free once these MMAs are done
                        if (++s == kStages) {
                            s = 0;
                            ph ^= 1u;
                        }
                    }
                }
                if (ok) umma_commit_pair(acc_full0 + 8 * buf);
            }
        }
    } else {
        const int q = warp & 3;                       // the quarter of the lanes this warp may touch
        const int c_begin = ((warp - 2) >> 2) * (kHT / 2);   // and its half of the tile's columns
        const int row_in_tile = q * 32 + lane;
        const uint32_t lane_base = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
        // both accumulator buffers start cleared
        for (int b = 0; b < 2; ++b) {
            for (int g = 0; g < 4; ++g)
                for (int c = c_begin; c < c_begin + kHT / 2; c += 16)
                    tmem_zero16(lane_base + b * kAccCols + g * kHT + c);
        }
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
            mbar_arrive_cluster(map_to_rank(acc_empty0, 0));
            mbar_arrive_cluster(map_to_rank(acc_empty0 + 8, 0));
        }
        int it = 0;
        for (int task = pair; task < n_tasks; task += n_pairs, ++it) {
            const int mt = task / JT, j = task - mt * JT;
            const uint32_t buf = it & 1, use = (it >> 1) & 1;
            const bool ready = mbar_wait(acc_full0 + 8 * buf, use, abort_flag);
            if (!__all_sync(0xFFFFFFFFu, ready)) break;
            tc_fence_after_sync();
            const long long row = static_cast<long long>(2 * mt + static_cast<int>(rank)) * kBM + row_in_tile;
            const bool live = row < a.n;
            const uint32_t t0 = lane_base + buf * kAccCols;
            const size_t off = static_cast<size_t>(live ? row : 0) * a.H + static_cast<size_t>(j) * kHT;
            const uint4 *hrow = reinterpret_cast<const uint4 *>(a.h_in + off);
            uint4 *orow = reinterpret_cast<uint4 *>(a.h_out + off);
            float part[3] = {0.0f, 0.0f, 0.0f};   // the head's partial sums over this warp's 32 units
#pragma unroll 1
            for (int c = c_begin; c < c_begin + kHT / 2; c += 16) {
                uint32_t nx[16], r[16], z[16], nh[16];
                tmem_ld16(t0 + c, nx);
                tmem_ld16(t0 + kHT + c, r);
                tmem_ld16(t0 + 2 * kHT + c, z);
                tmem_ld16(t0 + 3 * kHT + c, nh);
                uint4 hv[2];
                hv[0] = live ? __ldg(hrow + c / 8) : make_uint4(0, 0, 0, 0);
                hv[1] = live ? __ldg(hrow + c / 8 + 1) : make_uint4(0, 0, 0, 0);
                const float *bs = bias_s + j * kHT + c;
                tmem_wait_ld();
                tmem_zero16(t0 + c);
                tmem_zero16(t0 + kHT + c);
                tmem_zero16(t0 + 2 * kHT + c);
                tmem_zero16(t0 + 3 * kHT + c);
                const uint32_t hw[8] = {hv[0].x, hv[0].y, hv[0].z, hv[0].w,
                                        hv[1].x, hv[1].y, hv[1].z, hv[1].w};
                uint32_t ow[8];
#pragma unroll
                for (int i4 = 0; i4 < 16; i4 += 4) {
                    const float4 br = *reinterpret_cast<const float4 *>(bs + i4);
                    const float4 bz = *reinterpret_cast<const float4 *>(bs + a.H + i4);
                    const float4 bi = *reinterpret_cast<const float4 *>(bs + 2 * a.H + i4);
                    const float4 bh = *reinterpret_cast<const float4 *>(bs + 3 * a.H + i4);
                    const float brv[4] = {br.x, br.y, br.z, br.w}, bzv[4] = {bz.x, bz.y, bz.z, bz.w};
                    const float biv[4] = {bi.x, bi.y, bi.z, bi.w}, bhv[4] = {bh.x, bh.y, bh.z, bh.w};
                    float o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int i = i4 + e;
                        // sigmoid(v) = 1 / (1 + 2^(-v log2 e)), tanh(v) = 1 - 2 / (2^(2 v log2 e) + 1)
                        const float rr = rcp_approx(1.0f + ex2_approx(fmaf(__uint_as_float(r[i]), -kLog2e, brv[e])));
                        const float zz = rcp_approx(1.0f + ex2_approx(fmaf(__uint_as_float(z[i]), -kLog2e, bzv[e])));
                        const float pre = fmaf(rr, __uint_as_float(nh[i]) + bhv[e], __uint_as_float(nx[i]) + biv[e]);
                        const float cand = fmaf(-2.0f, rcp_approx(ex2_approx(pre * (2.0f * kLog2e)) + 1.0f), 1.0f);
                        const float hold = (i & 1) ? bf16_hi(hw[i / 2]) : bf16_lo(hw[i / 2]);
                        o[e] = fmaf(zz, hold - cand, cand);
                    }
                    ow[i4 / 2] = pack_bf16(o[0], o[1]);
                    ow[i4 / 2 + 1] = pack_bf16(o[2], o[3]);
                    if (a.head_w4 != nullptr) {
                        // the head sees h' as stored: rounded to bfloat16
                        const float hr[4] = {bf16_lo(ow[i4 / 2]), bf16_hi(ow[i4 / 2]), bf16_lo(ow[i4 / 2 + 1]),
                                             bf16_hi(ow[i4 / 2 + 1])};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float4 wv = head_s[j * kHT + c + i4 + e];
                            part[0] = __fmaf_rn(hr[e], wv.x, part[0]);
                            part[1] = __fmaf_rn(hr[e], wv.y, part[1]);
                            part[2] = __fmaf_rn(hr[e], wv.z, part[2]);
                        }
                    }
                }
                if (live) {
                    orow[c / 8] = make_uint4(ow[0], ow[1], ow[2], ow[3]);
                    orow[c / 8 + 1] = make_uint4(ow[4], ow[5], ow[6], ow[7]);
                }
            }
            if (a.head_w4 != nullptr && live)
                a.partial[static_cast<size_t>(row) * (a.H / 32) + (j * kHT + c_begin) / 32] =
                    make_float4(part[0], part[1], part[2], 0.0f);
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_rank(acc_empty0 + 8 * buf, 0));
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        // a wait ran out: report it, then give copies that may still be in flight time to land
        if (threadIdx.x == 0) atomicExch(a.err, 1);
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < kDrainNs) __nanosleep(1000);
    }
    cluster_sync_all();          // neither block leaves while its peer may still touch it
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---------------------------------------------------------------- encoder and head

// Thread t of a block owns the COLS hidden units of group t % (H/COLS), with their encoder
// weights in registers, and row slot t / (H/COLS) (H/COLS need not be a multiple of 32: the
// block is H/COLS times a slot count that is).  The block takes chunks of consecutive envs:
// it brings the weights (once) and the chunk's rows of obs and done bytes into shared memory
// with coalesced loads, so the loop over the chunk has no global load in it; a slot then
// takes kEncodeRows consecutive envs per pass.  Each output is the fma chain from the bias in
// ascending input order, rounded to bfloat16 in pairs; the relu is taken on the packed pair
// (max with +0: rounding keeps the sign, and -0 and NaN become +0 exactly as with
// "acc > 0 ? acc : 0" before the rounding).  A thread's store covers 2 * COLS bytes, a warp's
// 64 * COLS contiguous bytes of a row of x.  Where the env's episode just ended the same units
// of h are cleared.  OD = obs_dim, known at compile time so that the chain is exactly OD long.
constexpr int kEncodeRows = 4;
constexpr int kEncodeMaxThreads = 288;   // two blocks per SM with up to 112 registers per thread
constexpr int kEncodeMaxChunk = 256;     // envs per chunk, a multiple of kEncodeRows

__device__ __forceinline__ uint32_t pack_bf16_relu(float lo, float hi)
{
    const __nv_bfloat162 v = __hmax2(__floats2bfloat162_rn(lo, hi), __floats2bfloat162_rn(0.0f, 0.0f));
    return *reinterpret_cast<const uint32_t *>(&v);
}

// 2 * COLS bytes (COLS = 4 or 8) to a suitably aligned address.
template <int COLS>
__device__ __forceinline__ void store_units(__nv_bfloat16 *dst, const uint32_t (&v)[COLS / 2])
{
    if constexpr (COLS == 8)
        *reinterpret_cast<uint4 *>(dst) = make_uint4(v[0], v[1], v[2], v[3]);
    else
        *reinterpret_cast<uint2 *>(dst) = make_uint2(v[0], v[1]);
}

template <int OD>
struct EncodeShape {
    static constexpr int kCols = OD <= 8 ? 8 : 4;   // hidden units per thread: its weights stay in registers
};

// Shared memory: weights [H][OD] and biases [H] (float4 aligned), then the chunk's obs
// [chunk][OD] and its done bytes [chunk].
template <int OD>
__global__ void __launch_bounds__(kEncodeMaxThreads, 2)
k_encode(const float *__restrict__ obs, const uint8_t *__restrict__ done, __nv_bfloat16 *__restrict__ h,
         __nv_bfloat16 *__restrict__ x_out, const float *__restrict__ enc_w,
         const float *__restrict__ enc_b, int n, int H, int chunk_rows, int obs_aligned)
{
    constexpr int COLS = EncodeShape<OD>::kCols;
    extern __shared__ float4 enc_smem[];
    float *s_obs = reinterpret_cast<float *>(enc_smem + H * (OD + 1) / 4);
    uint8_t *s_done = reinterpret_cast<uint8_t *>(s_obs + chunk_rows * OD);
    const bool mask = done != nullptr && h != nullptr;

    // the chunk's obs: 16-byte pieces where the source allows (a chunk starts at a multiple of
    // four envs, so its first byte is 16-byte aligned if obs is), single words otherwise
    auto stage_chunk = [&](long long r0, int rows) {
        const float *src = obs + static_cast<size_t>(r0) * OD;
        const int words = rows * OD;
        const int vec = obs_aligned ? words / 4 : 0;
        for (int i = threadIdx.x; i < vec; i += blockDim.x)
            reinterpret_cast<float4 *>(s_obs)[i] = __ldg(reinterpret_cast<const float4 *>(src) + i);
        for (int i = 4 * vec + threadIdx.x; i < words; i += blockDim.x) s_obs[i] = __ldg(src + i);
        for (int i = threadIdx.x; i < chunk_rows; i += blockDim.x)
            s_done[i] = (mask && i < rows) ? __ldg(done + r0 + i) : 0;
    };

    {
        const float4 *gw = reinterpret_cast<const float4 *>(enc_w), *gb = reinterpret_cast<const float4 *>(enc_b);
        const int nw = H * OD / 4, nb = H / 4;
        for (int i = threadIdx.x; i < nw; i += blockDim.x) enc_smem[i] = __ldg(gw + i);
        for (int i = threadIdx.x; i < nb; i += blockDim.x) enc_smem[nw + i] = __ldg(gb + i);
    }
    long long r0 = static_cast<long long>(blockIdx.x) * chunk_rows;   // the grid has no more blocks than chunks
    int rows = static_cast<int>(n - r0 < chunk_rows ? n - r0 : chunk_rows);
    stage_chunk(r0, rows);
    __syncthreads();

    const int groups = H / COLS;
    const int slot = threadIdx.x / groups;
    const int group = threadIdx.x - slot * groups;
    const int c = COLS * group;
    const int slots = blockDim.x / groups;
    float w[COLS * OD], b[COLS];
    {
        const float4 *sw = enc_smem + group * (COLS * OD / 4);
        const float4 *sb = enc_smem + H * OD / 4 + group * (COLS / 4);
#pragma unroll
        for (int i = 0; i < COLS * OD / 4; ++i) {
            const float4 v = sw[i];
            w[4 * i] = v.x;
            w[4 * i + 1] = v.y;
            w[4 * i + 2] = v.z;
            w[4 * i + 3] = v.w;
        }
#pragma unroll
        for (int i = 0; i < COLS / 4; ++i) {
            const float4 v = sb[i];
            b[4 * i] = v.x;
            b[4 * i + 1] = v.y;
            b[4 * i + 2] = v.z;
            b[4 * i + 3] = v.w;
        }
    }

    while (true) {
        for (int m = slot * kEncodeRows; m < rows; m += slots * kEncodeRows) {
            const int left = rows - m;   // envs of this pass: kEncodeRows, fewer at the end of the batch
            float o[kEncodeRows * OD];
            if (left >= kEncodeRows) {
#pragma unroll
                for (int i = 0; i < OD; ++i) {   // m is a multiple of 4: 16-byte aligned in shared memory
                    const float4 v = reinterpret_cast<const float4 *>(s_obs + m * OD)[i];
                    o[4 * i] = v.x;
                    o[4 * i + 1] = v.y;
                    o[4 * i + 2] = v.z;
                    o[4 * i + 3] = v.w;
                }
            } else {
#pragma unroll
                for (int r = 0; r < kEncodeRows; ++r) {
                    const int rr = r < left ? r : 0;
#pragma unroll
                    for (int i = 0; i < OD; ++i) o[r * OD + i] = s_obs[(m + rr) * OD + i];
                }
            }
            const uint32_t ended = *reinterpret_cast<const uint32_t *>(s_done + m);   // byte r: env m + r
            __nv_bfloat16 *xrow = x_out + static_cast<size_t>(r0 + m) * H + c;
#pragma unroll
            for (int r = 0; r < kEncodeRows; ++r) {
                if (r >= left) break;
                // COLS independent chains side by side: no fma waits for the one before it
                float acc[COLS];
#pragma unroll
                for (int e = 0; e < COLS; ++e) acc[e] = b[e];
#pragma unroll
                for (int i = 0; i < OD; ++i) {
#pragma unroll
                    for (int e = 0; e < COLS; ++e) acc[e] = __fmaf_rn(o[r * OD + i], w[e * OD + i], acc[e]);
                }
                uint32_t packed[COLS / 2];
#pragma unroll
                for (int e = 0; e < COLS; e += 2) packed[e / 2] = pack_bf16_relu(acc[e], acc[e + 1]);
                store_units<COLS>(xrow + static_cast<size_t>(r) * H, packed);
            }
            if (ended != 0) {   // rare: the cleared units of h
                uint32_t zero[COLS / 2];
#pragma unroll
                for (int e = 0; e < COLS / 2; ++e) zero[e] = 0u;
                __nv_bfloat16 *hrow = h + static_cast<size_t>(r0 + m) * H + c;
#pragma unroll
                for (int r = 0; r < kEncodeRows; ++r)
                    if ((ended >> (8 * r)) & 0xFFu) store_units<COLS>(hrow + static_cast<size_t>(r) * H, zero);
            }
        }
        r0 += static_cast<long long>(gridDim.x) * chunk_rows;
        if (r0 >= n) break;
        rows = static_cast<int>(n - r0 < chunk_rows ? n - r0 : chunk_rows);
        __syncthreads();   // every slot has read the previous chunk
        stage_chunk(r0, rows);
        __syncthreads();
    }
}

// Threads per block: H/cols unit groups times a slot count: the smallest that fills whole
// warps, doubled while the block stays within 256 threads; where whole warps would need
// more than kEncodeMaxThreads, the most slots that fit (the last warp is then partly idle).
int encode_threads(int H, int cols)
{
    const int groups = H / cols;
    int slots = 1;
    while ((groups * slots) % 32 != 0) slots *= 2;
    if (groups * slots > kEncodeMaxThreads) slots = kEncodeMaxThreads / groups;
    while (groups * slots * 2 <= 256) slots *= 2;
    return groups * slots;
}

// The dynamic shared-memory limit is an attribute of the kernel on a device, not of a handle.
// It is only ever raised, so that handles with different hidden sizes can be alive together
// (lowering it for a small policy would make a larger one's next launch fail).
bool raise_dynamic_smem(const void *func, size_t bytes)
{
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, func) != cudaSuccess) return false;
    if (static_cast<size_t>(fa.maxDynamicSharedSizeBytes) >= bytes) return true;
    return cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)) ==
           cudaSuccess;
}

size_t encode_smem_bytes(int H, int obs_dim, int chunk_rows)
{
    return static_cast<size_t>(H) * (obs_dim + 1) * sizeof(float) +
           static_cast<size_t>(chunk_rows) * (obs_dim * sizeof(float) + 1);
}

typedef void (*EncodeKernel)(const float *, const uint8_t *, __nv_bfloat16 *, __nv_bfloat16 *, const float *,
                             const float *, int, int, int, int);

template <int OD>
struct EncodeTable {
    static EncodeKernel get(int obs_dim) { return obs_dim == OD ? k_encode<OD> : EncodeTable<OD - 1>::get(obs_dim); }
    static int cols(int obs_dim) { return obs_dim == OD ? EncodeShape<OD>::kCols : EncodeTable<OD - 1>::cols(obs_dim); }
};
template <>
struct EncodeTable<0> {
    static EncodeKernel get(int) { return nullptr; }
    static int cols(int) { return 4; }
};

// 64 envs per block, one thread per env.  logits[a] = bias + the partial sums of the blocks of
// 32 hidden units in block order, a partial sum being an fma chain from zero over its units in
// ascending order.  The block brings 64 units of its 64 rows at a time through
// shared memory with coalesced loads (rows padded to 33 words so that a thread walking
// its own row meets no bank conflict), the next chunk's loads in flight while the
// current one is summed; the head's weights sit in shared memory as
// [unit][AP] so that one 16-byte broadcast load feeds up to four chains.
constexpr int kHeadRows = 64;    // small blocks: they fit beside a cell block on an SM
constexpr int kHeadPitch = 33;   // words per staged row: 32 data + 1 pad

template <int AP>   // actions padded to 4 or 8
__global__ void __launch_bounds__(kHeadRows)
k_head(const __nv_bfloat16 *__restrict__ h, float *__restrict__ logits, const float *__restrict__ head_w,
       const float *__restrict__ head_b, int n, int H, int A)
{
    extern __shared__ float4 smem_f4[];
    float *w_s = reinterpret_cast<float *>(smem_f4);   // [H][AP], then the staged tile
    uint32_t *tile = reinterpret_cast<uint32_t *>(w_s + AP * H);
    for (int i = threadIdx.x; i < AP * H; i += kHeadRows) {
        const int k = i / AP, a = i - k * AP;
        w_s[i] = a < A ? head_w[static_cast<size_t>(a) * H + k] : 0.0f;
    }
    const int m0 = blockIdx.x * kHeadRows;
    const int m = m0 + threadIdx.x;
    float total[AP], acc[AP];
#pragma unroll
    for (int a = 0; a < AP; ++a) {
        total[a] = a < A ? __ldg(head_b + a) : 0.0f;
        acc[a] = 0.0f;
    }
    // this thread's eight 16-byte pieces of a 64-unit chunk of the block's rows
    auto fetch = [&](int k0, uint4 (&v)[8]) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int piece = i * kHeadRows + threadIdx.x;   // 8 pieces per row
            const int row = piece >> 3, seg = piece & 7;
            v[i] = make_uint4(0, 0, 0, 0);
            if (m0 + row < n)
                v[i] = __ldg(reinterpret_cast<const uint4 *>(h + static_cast<size_t>(m0 + row) * H + k0) + seg);
        }
    };
    uint4 next[8];
    fetch(0, next);
    for (int k0 = 0; k0 < H; k0 += 64) {
        __syncthreads();   // the previous chunk has been read (and, first time, w_s is complete)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int piece = i * kHeadRows + threadIdx.x;
            uint32_t *dst = tile + (piece >> 3) * kHeadPitch + (piece & 7) * 4;
            dst[0] = next[i].x;
            dst[1] = next[i].y;
            dst[2] = next[i].z;
            dst[3] = next[i].w;
        }
        __syncthreads();
        if (k0 + 64 < H) fetch(k0 + 64, next);   // in flight while this chunk is summed
        const uint32_t *mine = tile + threadIdx.x * kHeadPitch;
        const float4 *wk = reinterpret_cast<const float4 *>(w_s + static_cast<size_t>(k0) * AP);
#pragma unroll 8
        for (int p = 0; p < 32; ++p) {
            const uint32_t word = mine[p];
            const float hv[2] = {bf16_lo(word), bf16_hi(word)};
#pragma unroll
            for (int e = 0; e < 2; ++e) {
#pragma unroll
                for (int a4 = 0; a4 < AP / 4; ++a4) {
                    const float4 wv = wk[(2 * p + e) * (AP / 4) + a4];
                    acc[4 * a4 + 0] = __fmaf_rn(hv[e], wv.x, acc[4 * a4 + 0]);
                    acc[4 * a4 + 1] = __fmaf_rn(hv[e], wv.y, acc[4 * a4 + 1]);
                    acc[4 * a4 + 2] = __fmaf_rn(hv[e], wv.z, acc[4 * a4 + 2]);
                    acc[4 * a4 + 3] = __fmaf_rn(hv[e], wv.w, acc[4 * a4 + 3]);
                }
            }
            if ((p & 15) == 15) {   // a block of 32 units ends
#pragma unroll
                for (int a = 0; a < AP; ++a) {
                    total[a] = __fadd_rn(total[a], acc[a]);
                    acc[a] = 0.0f;
                }
            }
        }
    }
    if (m < n) {
#pragma unroll
        for (int a = 0; a < AP; ++a)
            if (a < A) logits[static_cast<size_t>(m) * A + a] = total[a];
    }
}

// logits[a] = bias + the cell kernel's partial sums in block order (A <= 4).
__global__ void __launch_bounds__(256)
k_head_reduce(const float4 *__restrict__ partial, float *__restrict__ logits, const float *__restrict__ head_b,
              int n, int blocks, int A)
{
    const int m = blockIdx.x * blockDim.x + threadIdx.x;
    if (m >= n) return;
    float total[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) total[a] = a < A ? __ldg(head_b + a) : 0.0f;
    const float4 *row = partial + static_cast<size_t>(m) * blocks;
    for (int b = 0; b < blocks; ++b) {
        const float4 v = __ldg(row + b);
        total[0] = __fadd_rn(total[0], v.x);
        total[1] = __fadd_rn(total[1], v.y);
        total[2] = __fadd_rn(total[2], v.z);
        total[3] = __fadd_rn(total[3], v.w);
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
        if (a < A) logits[static_cast<size_t>(m) * A + a] = total[a];
}

// ---------------------------------------------------------------- host side

typedef CUresult (*TensorMapEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                      const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                      const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up once through the runtime (no link
// against libcuda); nullptr if this driver does not have it.
TensorMapEncodeFn tensor_map_encoder()
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

size_t head_smem_bytes(int A, int H)
{
    const int AP = A <= 4 ? 4 : 8;
    return static_cast<size_t>(AP) * H * sizeof(float) + static_cast<size_t>(kHeadRows) * kHeadPitch * 4;
}

// bfloat16 [rows][H] row-major, boxes of 64 elements x box_rows rows, 128-byte swizzle;
// rows past the end read as zero.
bool encode_operand(TensorMapEncodeFn enc, CUtensorMap *m, const void *base, uint64_t H, uint64_t rows,
                    uint32_t box_rows)
{
    const cuuint64_t dims[2] = {H, rows};
    const cuuint64_t strides[1] = {H * 2};
    const cuuint32_t box[2] = {kBK, box_rows};
    const cuuint32_t elem_strides[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box,
               elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

struct gru_policy {
    int H = 0, obs_dim = 0, A = 0;
    int device = 0, sms = 0;
    int pairs = 0;   // clusters of two blocks that can be resident at once
    int top_priority = 0;   // numerically lowest = most urgent launch priority of the device
    int encode_blocks_per_sm = 0;   // resident encoder blocks per SM, found at the first call
    cudaStream_t stream = nullptr;
    int64_t launches = 0;
    __nv_bfloat16 *wx = nullptr, *wh = nullptr;   // packed [H/64][192][H]
    float *b_r = nullptr, *b_z = nullptr, *b_in = nullptr, *b_hn = nullptr;
    float *enc_w = nullptr, *enc_b = nullptr, *head_w = nullptr, *head_b = nullptr;
    float *head_w4 = nullptr;   // [H][4], for the cell kernel's partial sums (n_actions <= 4)
    int *err = nullptr;
    CUtensorMap tm_wx, tm_wh;
};

namespace {

template <typename T>
bool upload(T **dst, const std::vector<T> &src)
{
    if (cudaMalloc(reinterpret_cast<void **>(dst), src.size() * sizeof(T)) != cudaSuccess) return false;
    return cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice) == cudaSuccess;
}

void release(gru_policy *p)
{
    cudaFree(p->wx);
    cudaFree(p->wh);
    cudaFree(p->b_r);
    cudaFree(p->b_z);
    cudaFree(p->b_in);
    cudaFree(p->b_hn);
    cudaFree(p->enc_w);
    cudaFree(p->enc_b);
    cudaFree(p->head_w);
    cudaFree(p->head_b);
    cudaFree(p->head_w4);
    cudaFree(p->err);
    delete p;
}

}  // namespace

extern "C" {

int gru_policy_create(gru_policy **out, int hidden, int obs_dim, int n_actions, const float *enc_w,
                      const float *enc_b, const float *w_ih, const float *w_hh, const float *b_ih,
                      const float *b_hh, const float *head_w, const float *head_b)
{
    if (out == nullptr) return GRU_POLICY_ENULL;
    *out = nullptr;
    if (!enc_w || !enc_b || !w_ih || !w_hh || !b_ih || !b_hh || !head_w || !head_b) return GRU_POLICY_ENULL;
    if (hidden < 64 || hidden > GRU_POLICY_MAX_HIDDEN || hidden % 64 != 0) return GRU_POLICY_EINVAL;
    if (obs_dim < 1 || obs_dim > GRU_POLICY_MAX_OBS) return GRU_POLICY_EINVAL;
    if (n_actions < 1 || n_actions > GRU_POLICY_MAX_ACTIONS) return GRU_POLICY_EINVAL;
    if (tensor_map_encoder() == nullptr) return GRU_POLICY_ECUDA;
    gru_policy *p = new (std::nothrow) gru_policy;
    if (p == nullptr) return GRU_POLICY_ENOMEM;
    const int H = hidden;
    p->H = H;
    p->obs_dim = obs_dim;
    p->A = n_actions;
    cudaDeviceProp prop;
    if (cudaGetDevice(&p->device) != cudaSuccess ||
        cudaGetDeviceProperties(&prop, p->device) != cudaSuccess) {
        cudaGetLastError();
        delete p;
        return GRU_POLICY_ECUDA;
    }
    p->sms = prop.multiProcessorCount;
    int least = 0;
    if (cudaDeviceGetStreamPriorityRange(&least, &p->top_priority) != cudaSuccess) {
        cudaGetLastError();
        p->top_priority = 0;
    }

    // Pack the weights: tile j holds, for the x half, rows [W_in | W_ir | W_iz] of its 64 units
    // and, for the h half, rows [W_hr | W_hz | W_hn]; gate blocks of the inputs are r, z, n.
    const int JT = H / kHT;
    std::vector<__nv_bfloat16> wx(static_cast<size_t>(3) * H * H), wh(wx.size());
    const int x_gate[3] = {2, 0, 1}, h_gate[3] = {0, 1, 2};
    for (int j = 0; j < JT; ++j)
        for (int g = 0; g < 3; ++g)
            for (int i = 0; i < kHT; ++i) {
                const size_t dst = (static_cast<size_t>(j) * kBN + g * kHT + i) * H;
                const size_t sx = (static_cast<size_t>(x_gate[g]) * H + j * kHT + i) * H;
                const size_t sh = (static_cast<size_t>(h_gate[g]) * H + j * kHT + i) * H;
                for (int k = 0; k < H; ++k) {
                    wx[dst + k] = __float2bfloat16_rn(w_ih[sx + k]);
                    wh[dst + k] = __float2bfloat16_rn(w_hh[sh + k]);
                }
            }
    std::vector<float> b_r(H), b_z(H), b_in(H), b_hn(H);
    for (int c = 0; c < H; ++c) {
        b_r[c] = -kLog2e * (b_ih[c] + b_hh[c]);
        b_z[c] = -kLog2e * (b_ih[H + c] + b_hh[H + c]);
        b_in[c] = b_ih[2 * H + c];
        b_hn[c] = b_hh[2 * H + c];
    }
    std::vector<float> head_w4(static_cast<size_t>(H) * 4, 0.0f);
    for (int c = 0; c < H; ++c)
        for (int act = 0; act < n_actions && act < 4; ++act) head_w4[static_cast<size_t>(c) * 4 + act] = head_w[static_cast<size_t>(act) * H + c];
    bool ok = upload(&p->wx, wx) && upload(&p->wh, wh) && upload(&p->b_r, b_r) && upload(&p->b_z, b_z) &&
              upload(&p->b_in, b_in) && upload(&p->b_hn, b_hn) &&
              upload(&p->enc_w, std::vector<float>(enc_w, enc_w + static_cast<size_t>(H) * obs_dim)) &&
              upload(&p->enc_b, std::vector<float>(enc_b, enc_b + H)) &&
              upload(&p->head_w, std::vector<float>(head_w, head_w + static_cast<size_t>(n_actions) * H)) &&
              upload(&p->head_b, std::vector<float>(head_b, head_b + n_actions)) &&
              upload(&p->head_w4, head_w4) &&
              upload(&p->err, std::vector<int>(1, 0));
    if (ok) {
        TensorMapEncodeFn enc = tensor_map_encoder();
        ok = encode_operand(enc, &p->tm_wx, p->wx, H, static_cast<uint64_t>(3) * H, kBRows) &&
             encode_operand(enc, &p->tm_wh, p->wh, H, static_cast<uint64_t>(3) * H, kBRows);
    }
    if (ok) ok = raise_dynamic_smem(reinterpret_cast<const void *>(k_gru_cell),
                                    cell_smem_bytes(H, cell_smem_bytes(H, true) <= kMaxSmem));
    // Ask for the largest shared-memory partition, not the smallest that holds one block, so that
    // small blocks of other kernels can share an SM with a cell block.
    if (ok) ok = cudaFuncSetAttribute(k_gru_cell, cudaFuncAttributePreferredSharedMemoryCarveout,
                                      cudaSharedmemCarveoutMaxShared) == cudaSuccess;
    if (ok) {
        // how many pairs fit on the device at once: the persistent grid is sized to that
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(p->sms & ~1));
        cfg.blockDim = dim3(kCellThreads);
        cfg.dynamicSmemBytes = cell_smem_bytes(H, cell_smem_bytes(H, true) <= kMaxSmem);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int clusters = 0;
        ok = cudaOccupancyMaxActiveClusters(&clusters, k_gru_cell, &cfg) == cudaSuccess && clusters > 0;
        p->pairs = clusters < p->sms / 2 ? clusters : p->sms / 2;
    }
    if (ok && head_smem_bytes(n_actions, H) > 48 * 1024)
        ok = raise_dynamic_smem(reinterpret_cast<const void *>(n_actions <= 4 ? k_head<4> : k_head<8>),
                                head_smem_bytes(n_actions, H));
    if (!ok) {
        cudaGetLastError();
        release(p);
        return GRU_POLICY_ECUDA;
    }
    *out = p;
    return GRU_POLICY_OK;
}

int gru_policy_destroy(gru_policy *p)
{
    if (p == nullptr) return GRU_POLICY_ENULL;
    cudaStreamSynchronize(p->stream);
    release(p);
    return GRU_POLICY_OK;
}

int gru_policy_set_stream(gru_policy *p, void *cuda_stream)
{
    if (p == nullptr) return GRU_POLICY_ENULL;
    p->stream = static_cast<cudaStream_t>(cuda_stream);
    return GRU_POLICY_OK;
}

int gru_policy_encode(gru_policy *p, const float *obs, const uint8_t *done, void *h, void *x_out, int n)
{
    if (p == nullptr || obs == nullptr || x_out == nullptr) return GRU_POLICY_ENULL;
    if (n < 1) return GRU_POLICY_EINVAL;
    if ((reinterpret_cast<uintptr_t>(x_out) | reinterpret_cast<uintptr_t>(h)) % 16 != 0) return GRU_POLICY_EALIGN;
    if (reinterpret_cast<uintptr_t>(obs) % 8 != 0) return GRU_POLICY_EALIGN;
    const int cols = EncodeTable<GRU_POLICY_MAX_OBS>::cols(p->obs_dim);
    const int threads = encode_threads(p->H, cols);
    EncodeKernel kernel = EncodeTable<GRU_POLICY_MAX_OBS>::get(p->obs_dim);
    if (p->encode_blocks_per_sm == 0) {   // resident blocks per SM with the largest chunk
        const size_t most = encode_smem_bytes(p->H, p->obs_dim, kEncodeMaxChunk);
        int per_sm = 0;
        if (!raise_dynamic_smem(reinterpret_cast<const void *>(kernel), most)) return GRU_POLICY_ECUDA;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, most) != cudaSuccess || per_sm < 1) {
            cudaGetLastError();
            per_sm = 1;
        }
        p->encode_blocks_per_sm = per_sm;
    }
    // Chunks of up to kEncodeMaxChunk envs; a batch that one wave of resident blocks can take
    // in one chunk each is cut into that many chunks (whole passes of the block's slots).
    const long long cap = static_cast<long long>(p->sms) * p->encode_blocks_per_sm;
    const int rows_per_pass = threads / (p->H / cols) * kEncodeRows;
    long long chunk = (n + cap - 1) / cap;
    chunk = (chunk + rows_per_pass - 1) / rows_per_pass * rows_per_pass;
    if (chunk > kEncodeMaxChunk) chunk = kEncodeMaxChunk;
    const long long chunks = (n + chunk - 1) / chunk;
    const unsigned blocks = static_cast<unsigned>(chunks < cap ? chunks : cap);
    const int obs_aligned = reinterpret_cast<uintptr_t>(obs) % 16 == 0;
    kernel<<<blocks, static_cast<unsigned>(threads), encode_smem_bytes(p->H, p->obs_dim, static_cast<int>(chunk)), p->stream>>>(
        obs, done, static_cast<__nv_bfloat16 *>(h), static_cast<__nv_bfloat16 *>(x_out), p->enc_w, p->enc_b, n,
        p->H, static_cast<int>(chunk), obs_aligned);
    if (cudaGetLastError() != cudaSuccess) return GRU_POLICY_ECUDA;
    p->launches += 1;
    return GRU_POLICY_OK;
}

static int launch_cell(gru_policy *p, const void *x, const void *h_in, void *h_out, float4 *partial, int n)
{
    if (p == nullptr || x == nullptr || h_in == nullptr || h_out == nullptr) return GRU_POLICY_ENULL;
    if (n < 1) return GRU_POLICY_EINVAL;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(h_in) |
         reinterpret_cast<uintptr_t>(h_out) | reinterpret_cast<uintptr_t>(partial)) % 16 != 0)
        return GRU_POLICY_EALIGN;
    if (h_out == x || h_out == h_in) return GRU_POLICY_EINVAL;
    TensorMapEncodeFn enc = tensor_map_encoder();
    CUtensorMap tm_x, tm_h;
    if (!encode_operand(enc, &tm_x, x, p->H, n, kBM) || !encode_operand(enc, &tm_h, h_in, p->H, n, kBM))
        return GRU_POLICY_ECUDA;
    CellArgs a;
    a.h_in = static_cast<const __nv_bfloat16 *>(h_in);
    a.h_out = static_cast<__nv_bfloat16 *>(h_out);
    a.b_r = p->b_r;
    a.b_z = p->b_z;
    a.b_in = p->b_in;
    a.b_hn = p->b_hn;
    a.head_w4 = partial != nullptr ? p->head_w4 : nullptr;
    a.partial = partial;
    a.n = n;
    a.H = p->H;
    a.err = p->err;
    const long long tasks = static_cast<long long>((n + 2 * kBM - 1) / (2 * kBM)) * (p->H / kHT);
    const long long pairs = tasks < p->pairs ? tasks : p->pairs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(2 * pairs));
    cfg.blockDim = dim3(kCellThreads);
    cfg.dynamicSmemBytes = cell_smem_bytes(p->H, partial != nullptr);
    cfg.stream = p->stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // The cell wants whole SMs; when it is pending together with small kernels of a parallel
    // chain, its blocks are placed first and the small kernels take what is left.
    attr[1].id = cudaLaunchAttributePriority;
    attr[1].val.priority = p->top_priority;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, k_gru_cell, tm_x, tm_h, p->tm_wx, p->tm_wh, a) != cudaSuccess) {
        cudaGetLastError();
        return GRU_POLICY_ECUDA;
    }
    p->launches += 1;
    return GRU_POLICY_OK;
}

int gru_policy_cell(gru_policy *p, const void *x, const void *h_in, void *h_out, int n)
{
    return launch_cell(p, x, h_in, h_out, nullptr, n);
}

size_t gru_policy_workspace_bytes(const gru_policy *p, int n)
{
    if (p == nullptr || n < 1) return 0;
    return static_cast<size_t>(n) * (p->H / 32) * sizeof(float4);
}

int gru_policy_cell_head(gru_policy *p, const void *x, const void *h_in, void *h_out, float *logits,
                         void *workspace, int n)
{
    if (p == nullptr || logits == nullptr || workspace == nullptr) return GRU_POLICY_ENULL;
    if (p->A > 4 || cell_smem_bytes(p->H, true) > kMaxSmem) return GRU_POLICY_EINVAL;
    const int rc = launch_cell(p, x, h_in, h_out, static_cast<float4 *>(workspace), n);
    if (rc != GRU_POLICY_OK) return rc;
    k_head_reduce<<<(n + 255) / 256, 256, 0, p->stream>>>(static_cast<const float4 *>(workspace), logits,
                                                          p->head_b, n, p->H / 32, p->A);
    if (cudaGetLastError() != cudaSuccess) return GRU_POLICY_ECUDA;
    p->launches += 1;
    return GRU_POLICY_OK;
}

int gru_policy_head(gru_policy *p, const void *h, float *logits, int n)
{
    if (p == nullptr || h == nullptr || logits == nullptr) return GRU_POLICY_ENULL;
    if (n < 1) return GRU_POLICY_EINVAL;
    if (reinterpret_cast<uintptr_t>(h) % 16 != 0) return GRU_POLICY_EALIGN;
    const unsigned blocks = static_cast<unsigned>((n + kHeadRows - 1) / kHeadRows);
    (p->A <= 4 ? k_head<4> : k_head<8>)<<<blocks, kHeadRows, head_smem_bytes(p->A, p->H), p->stream>>>(
        static_cast<const __nv_bfloat16 *>(h), logits, p->head_w, p->head_b, n, p->H, p->A);
    if (cudaGetLastError() != cudaSuccess) return GRU_POLICY_ECUDA;
    p->launches += 1;
    return GRU_POLICY_OK;
}

int gru_policy_status(gru_policy *p)
{
    if (p == nullptr) return GRU_POLICY_ENULL;
    if (cudaStreamSynchronize(p->stream) != cudaSuccess) return GRU_POLICY_ECUDA;
    int flag = 0;
    if (cudaMemcpy(&flag, p->err, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return GRU_POLICY_ECUDA;
    if (flag != 0) {
        cudaMemset(p->err, 0, sizeof(int));
        return GRU_POLICY_ETIMEOUT;
    }
    return GRU_POLICY_OK;
}

int gru_policy_hidden(const gru_policy *p) { return p ? p->H : GRU_POLICY_ENULL; }

int64_t gru_policy_launch_count(const gru_policy *p) { return p ? p->launches : 0; }

const char *gru_policy_strerror(int code)
{
    switch (code) {
    case GRU_POLICY_OK: return "ok";
    case GRU_POLICY_EINVAL: return "invalid size or overlapping buffers";
    case GRU_POLICY_ENULL: return "required pointer is NULL";
    case GRU_POLICY_EALIGN: return "x / h pointer not 16-byte aligned";
    case GRU_POLICY_ECUDA: return "CUDA runtime call or launch failed";
    case GRU_POLICY_ENOMEM: return "allocation failed";
    case GRU_POLICY_ETIMEOUT: return "a kernel gave up a bounded wait; its output is invalid";
    default: return "unknown error";
    }
}

}  // extern "C"
