// conv1 (8x8 / 4, C -> 32) of the policy-value network, fused from raw frames to fp16 output.
//
// An 8x8 stride-4 convolution is a 2x2 stride-1 convolution on the space-to-depth(4) image: grid
// pixel (Y, X) carries the 16 C bytes x[c][4Y+uy][4X+ux], and output pixel (y, x) is the sum over the
// four taps (dy, dx) of  pix(y+dy, x+dx) . w[o][dy][dx].  The kernel never builds im2col rows:
//
//   * The 128 rows of an MMA tile are 128 consecutive grid COLUMNS of the batch (flat index
//     q = env * Ws + X), and the kernel marches down the grid rows Y.  Grid row Y of those columns is
//     converted to fp16 once (a zero-extended byte is the fp16 subnormal b * 2^-24, exact; 2^24 / 255
//     goes into the accumulator scale) and written to a ring of operand rows in tensor memory.
//   * Step y multiplies ring entry Y = y by the dy = 0 filter rows and entry Y = y + 1 by the dy = 1
//     filter rows (tcgen05.mma with A from tensor memory, 128 x 64 x 16), so every entry serves two
//     steps: the vertical taps cost no extra conversion.
//   * The two horizontal taps are stacked along N: accumulator columns [0, 32) hold the dx = 0 part of
//     output (y, X), columns [32, 64) the dx = 1 part, which belongs to output (y, X - 1).  The
//     epilogue adds its neighbour lane's upper half to its own lower half, applies scale, bias and
//     ReLU and stores fp16 in the layout conv2 reads.  Warp quarters overlap by one lane (quarter k
//     starts at column 31 k of the tile), so the neighbour is always in the same warp.
//
// Work unit = (tile of 125 grid columns, range of output rows).  One CTA per SM runs a pipeline of
// four roles.  One thread stages groups of grid rows into a ring in shared memory: one tensor-tiled
// TMA box per environment (all channels, group_rows x 4 input rows; the frames are viewed as 32-bit
// words so that a box row is the 4 W contiguous bytes under one grid row).  Two groups of four
// converter warps take alternate grid rows (thread = grid column), expand them in registers and write
// tensor memory; two threads issue the MMAs of alternate steps, each step into the next of several
// accumulators; two groups of four epilogue warps drain alternate steps.  Every role is bound by
// latency chains (shared -> registers -> tensor memory, tensor memory -> registers -> global), which
// is why each exists twice.  All waits are bounded.
#include "conv1_tc.cuh"
#include "tc_ptx.cuh"
#include "tc_host.cuh"

namespace hts {
using namespace tc;

namespace {

// Pipeline shape per channel-group count: NI issuing threads, CGR / EGR groups of four converter / epilogue
// warps, NACC accumulators, R operand rows in the ring, KR grid rows per staged group.
// The barriers carry one parity bit, so every waiter must stay within one phase of the barrier it waits on:
// NI + 1 <= R (see the issuing threads), EGR divides NACC (an accumulator is drained by one epilogue group, in step
// order), and R <= NACC + 1 where issuing threads share an accumulator (NI does not divide NACC).
template <int CG> struct Shape;
template <> struct Shape<1> {
    static constexpr int NI = 4, CGR = 2, EGR = 2, NACC = 4, R = 8, TMEM = 512, PER_SM = 1, KR = 3;
};
template <> struct Shape<2> {
    static constexpr int NI = 3, CGR = 2, EGR = 2, NACC = 4, R = 4, TMEM = 512, PER_SM = 1, KR = 1;
};
template <> struct Shape<4> {       // 32 MMAs per step: tensor-bound
    static constexpr int NI = 2, CGR = 2, EGR = 2, NACC = 2, R = 3, TMEM = 512, PER_SM = 1, KR = 1;
};
template <int CG> constexpr bool shape_ok()
{
    using S = Shape<CG>;
    return S::NI + 1 <= S::R && S::NACC % S::EGR == 0 && (S::NACC % S::NI == 0 || S::R <= S::NACC + 1) &&
           S::NACC * 64 + S::R * 32 * CG <= S::TMEM;
}
static_assert(shape_ok<1>() && shape_ok<2>() && shape_ok<4>(), "pipeline shape breaks the one-phase rule or the tensor-memory budget");
template <int CG> __host__ __device__ constexpr int conv_warp0() { return 1 + Shape<CG>::NI; }          // warp 0 stages, then the issuers
template <int CG> __host__ __device__ constexpr int epi_warp0() { return conv_warp0<CG>() + 4 * Shape<CG>::CGR; }
template <int CG> __host__ __device__ constexpr int threads_of() { return (epi_warp0<CG>() + 4 * Shape<CG>::EGR) * 32; }
constexpr int kTileCols = 124;                  // new grid columns per tile (4 quarters x 31; one more is shared)
constexpr int kChunkBytes = 64 * 128;           // one filter K chunk: 64 rows (dx, o) x 64 fp16
constexpr int kMaxStages = 8;
constexpr int kMaxRing = 8;
constexpr int kMaxAcc = 4;

struct Conv1Params {
    Conv1Plan pl;
    const uint8_t* obs;
    const int32_t* slots;   // frame of each row in obs, or nullptr: row e is frame e
    int pool;               // frames in obs when slots are given
    int n;
    int tiles;              // ceil(n * Ws / 124)
    int splits;             // equal ranges the H1 output rows of a tile are cut into (a divisor of H1)
    int su;                 // output rows (steps) per unit: H1 / splits; a unit stages su + 1 grid rows
    const float* bias;
    const float* inv_scale;
    __half* out;
    int* status;
};

// Frame index of batch row e: e itself, or its slot in the pool.  A slot outside the pool is
// recorded in the status word and frame 0 is read instead (the heads kernel drops that row).
__device__ __forceinline__ size_t frame_of(const Conv1Params& p, int e)
{
    if (!p.slots) return (size_t)e;
    const int sl = p.slots[e];
    if ((unsigned)sl >= (unsigned)p.pool) { atomicCAS(p.status, 0, kStatusBadSlot); return 0; }
    return (size_t)sl;
}

// Four bytes -> four fp16 values without arithmetic: a byte b zero-extended to 16 bits is the fp16
// subnormal b * 2^-24, which the tensor core multiplies exactly; the 2^24 goes into the accumulator scale.
__device__ __forceinline__ void u8x4_to_h4(uint32_t w, uint32_t& lo, uint32_t& hi)
{
    lo = __byte_perm(w, 0u, 0x4140);                    // {b0, 0, b1, 0}
    hi = __byte_perm(w, 0u, 0x4342);                    // {b2, 0, b3, 0}
}

// Position of a role in the CTA's sequence of units.  The CTA's units are u = blockIdx.x + i * gridDim.x; every
// unit has `su` steps (output rows) and su + 1 grid rows, so a role that takes every k-th step or row of the
// CTA's sequence finds its unit by stepping a counter instead of dividing.
struct Walk {
    int i, pos;                 // unit of this CTA, position inside it (step or row)
    int tile, y_base;           // the unit's tile and first output row
    __device__ __forceinline__ void unit(const Conv1Params& p)
    {
        const int u = blockIdx.x + i * gridDim.x;
        tile = u / p.splits;
        y_base = (u - tile * p.splits) * p.su;
    }
    __device__ __forceinline__ void start(const Conv1Params& p, int first) { i = 0; pos = first; }
    // brings pos back below `len` (items per unit); true if the unit changed
    __device__ __forceinline__ bool settle(int len)
    {
        bool moved = false;
        while (pos >= len) { pos -= len; ++i; moved = true; }
        return moved;
    }
};

// CG: groups of four channels.  WC: the frame width when known at compile time (the converter's loads then
// use immediate offsets), 0 = any.
template <int CG, int WC>
__global__ void __launch_bounds__(threads_of<CG>(), Shape<CG>::PER_SM)
conv1_march_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const Conv1Params p)
{
    const Conv1Plan& pl = p.pl;
    constexpr int ACOLS = 32 * CG;                     // tensor-memory columns of one operand row
    using S = Shape<CG>;
    constexpr int KR = S::KR;                          // grid rows per staged group (= pl.group_rows)
    constexpr int NACC = S::NACC;                      // accumulators (= pl.accs)
    constexpr int R = S::R;                            // operand rows in the ring (= pl.ring)
    constexpr int kIssuers = S::NI, kConvGroups = S::CGR, kEpiGroups = S::EGR;
    constexpr int kConvWarp0 = conv_warp0<CG>(), kEpiWarp0 = epi_warp0<CG>(), kThreads = threads_of<CG>();
    const int W = WC ? WC : pl.W;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t w_bar, u8_full[kMaxStages], u8_empty[kMaxStages], a_full[kMaxRing], a_empty[kMaxRing],
        d_full[kMaxAcc], d_empty[kMaxAcc];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ __align__(16) float s_bias[32];
    volatile int* abortp = &abort_flag;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    constexpr int w_bytes = 2 * CG * kChunkBytes;
    uint8_t* s_u8 = sm + w_bytes;
    const int NS = pl.stages;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int units = p.tiles * p.splits;

    if (threadIdx.x == 0) {
        mbar_init(&w_bar, 1);
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&u8_full[s], 1); mbar_init(&u8_empty[s], 4 * kConvGroups); }
        for (int s = 0; s < kMaxRing; ++s) { mbar_init(&a_full[s], 4); mbar_init(&a_empty[s], 2); }
        for (int s = 0; s < kMaxAcc; ++s) { mbar_init(&d_full[s], 1); mbar_init(&d_empty[s], 4); }
        abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmX);
    }
    if (threadIdx.x >= 32 && threadIdx.x < 64) s_bias[threadIdx.x - 32] = p.bias[threadIdx.x - 32];
    if (warp == 1) tmem_alloc(&tmem_slot, S::TMEM);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_slot, tmem_a = tmem_slot + NACC * 64;   // accumulators of 64 columns, then the ring
    if (threadIdx.x == 0) {                                   // the filter does not depend on the previous kernel
        mbar_arrive_expect_tx(&w_bar, (uint32_t)w_bytes);
        for (int dy = 0; dy < 2; ++dy)
            for (int g = 0; g < CG; ++g) tma_load_2d(sm + (dy * CG + g) * kChunkBytes, &tmW, g * 64, dy * 64, &w_bar);
    }
    pdl_wait();
    pdl_trigger();

    const int my_units = blockIdx.x < units ? (units - blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int su = p.su, ru = p.su + 1;                       // steps and grid rows per unit
    const int total_steps = my_units * su;

    if (warp == 0) {
        // ---- staging: groups of KR grid rows, one box per environment the tile touches
        if (lane == 0) {
            int st = 0;
            uint32_t stph = 0;
            bool alive = true;
            Walk w;
            for (w.i = 0; alive && w.i < my_units; ++w.i) {
                w.unit(p);
                const int e_first = (w.tile * kTileCols) / pl.Ws;
                int e_last = (w.tile * kTileCols + kTileCols) / pl.Ws;
                if (e_last > p.n - 1) e_last = p.n - 1;
                const int envs = e_last - e_first + 1;
                for (int Y = w.y_base; Y <= w.y_base + su; Y += KR) {
                    if (!mbar_wait(&u8_empty[st], stph ^ 1u, abortp, p.status, 31)) { alive = false; break; }
                    uint8_t* dst = s_u8 + st * pl.stage_bytes;
                    mbar_arrive_expect_tx(&u8_full[st], (uint32_t)(envs * pl.env_bytes));
                    for (int i = 0; i < envs; ++i)
                        tma_load_4d(dst + i * pl.env_pitch, &tmX, 0, Y, 0, (int)frame_of(p, e_first + i), &u8_full[st]);
                    if (++st == NS) { st = 0; stph ^= 1u; }
                }
            }
        }
    } else if (warp <= kIssuers) {
        // ---- MMA issue: thread g takes the CTA's steps g, g + kIssuers, ...; step k goes to accumulator k % NACC.
        //      Step k of the CTA reads operand rows k + (its unit's index) and the next one.
        if (lane == 0) {
            const int g = warp - 1;
            constexpr uint32_t idesc = instr_desc_f16(0, 128, 64);
            uint64_t bdesc[2][CG];
#pragma unroll
            for (int dy = 0; dy < 2; ++dy)
#pragma unroll
                for (int cg = 0; cg < CG; ++cg) bdesc[dy][cg] = smem_desc_sw128(base + (dy * CG + cg) * kChunkBytes);
            bool alive = mbar_wait(&w_bar, 0, abortp, p.status, 32);
            Walk w;
            w.start(p, g);
            for (int k = g; alive && k < total_steps; k += kIssuers, w.pos += kIssuers) {
                w.settle(su);
                const int r0 = k + w.i, r1 = r0 + 1;                       // operand rows of this step
                const int s0 = r0 % R, s1 = r1 % R;
                const int acc = k % NACC;
                // Operands first, accumulator second.  A barrier carries one parity bit, so a waiting thread must be
                // within one phase of it.  From one step of this thread to its next the operand rows advance by NI, or by
                // NI + 1 across a unit boundary; with NI + 1 <= R the ring entries of this step last held rows that this
                // thread's previous step or an earlier one has read, so their barriers are exactly one phase on.  Once
                // the operands are there, all steps up to k + 1 - R are complete, so the step that last used this
                // accumulator has been issued and the accumulator's barrier is at most one phase behind.
                if (!mbar_wait(&a_full[s0], ((uint32_t)(r0 / R)) & 1u, abortp, p.status, 34)) break;
                if (!mbar_wait(&a_full[s1], ((uint32_t)(r1 / R)) & 1u, abortp, p.status, 34)) break;
                if (!mbar_wait(&d_empty[acc], (((uint32_t)(k / NACC)) & 1u) ^ 1u, abortp, p.status, 33)) break;
                tc_fence_after();
                const uint32_t d_addr = tmem_d + acc * 64;
#pragma unroll
                for (int dy = 0; dy < 2; ++dy) {
                    const uint32_t a_addr = tmem_a + (dy ? s1 : s0) * ACOLS;
#pragma unroll
                    for (int cg = 0; cg < CG; ++cg)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            mma_f16_ts(d_addr, a_addr + cg * 32 + 8 * kk, bdesc[dy][cg] + 2 * kk, idesc, (dy | cg | kk) != 0);
                }
                // an operand row is read by two steps (as the lower and as the upper grid row) and is free once both are
                // done; the first and the last row of a unit are read by one step only, which then arrives for both
                mma_commit(&a_empty[s0]);
                mma_commit(&a_empty[s1]);
                if (w.pos == 0) mma_commit(&a_empty[s0]);
                if (w.pos == su - 1) mma_commit(&a_empty[s1]);
                mma_commit(&d_full[acc]);
            }
        }
    } else if (warp < kEpiWarp0) {
        // ---- convert: thread = grid column q of the tile; group h takes the CTA's grid rows h, h + 2, ...
        const int h = (warp - kConvWarp0) >> 2;
        const int qq = warp & 3;
        const uint32_t st_addr = tmem_a + ((uint32_t)(qq * 32) << 16);
        int st = 0;                                       // staged group
        uint32_t stph = 0;
        int r = 0;                                        // grid rows of this CTA so far
        int pending = -1;                                 // ring entry whose tensor-memory stores are still in flight
        bool alive = true;
        Walk w;
        for (w.i = 0; alive && w.i < my_units; ++w.i) {
            w.unit(p);
            const int q = w.tile * kTileCols + 31 * qq + lane;
            const int e = q / pl.Ws, X = q - e * pl.Ws;
            const int e_first = (w.tile * kTileCols) / pl.Ws;
            // columns past the end of the batch read the start of the buffer: their results are never stored
            const int off = e < p.n ? (e - e_first) * pl.env_pitch + 4 * X : 0;
            int yr = 0;                                   // row inside the staged group
            for (int j = 0; j < ru; ++j, ++r) {
                if (yr == 0 && !mbar_wait_warp(&u8_full[st], stph, abortp, p.status, 35)) { alive = false; break; }
                if (r % kConvGroups == h) {
                    const int s = r % R;
                    const uint8_t* src = s_u8 + st * pl.stage_bytes + off + yr * 4 * W;
#pragma unroll
                    for (int cg = 0; cg < CG; ++cg) {
                        uint32_t v[32];
#pragma unroll
                        for (int c = 0; c < 4; ++c)
#pragma unroll
                            for (int uy = 0; uy < 4; ++uy)
                                u8x4_to_h4(*reinterpret_cast<const uint32_t*>(src + ((cg * 4 + c) * KR * 4 + uy) * W),
                                           v[c * 8 + uy * 2], v[c * 8 + uy * 2 + 1]);
                        if (cg == 0) {
                            if (pending >= 0) {               // the previous row's stores overlapped these loads
                                tmem_st_wait();
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(&a_full[pending]);
                            }
                            if (!mbar_wait_warp(&a_empty[s], (((uint32_t)(r / R)) & 1u) ^ 1u, abortp, p.status, 36)) { alive = false; break; }
                            tc_fence_after();
                        }
                        tmem_st_32x32(st_addr + s * ACOLS + cg * 32, v);
                    }
                    if (!alive) break;
                    pending = s;
                }
                if (++yr == KR || j == ru - 1) {          // done with this staged group (every converter warp arrives)
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&u8_empty[st]);
                    yr = 0;
                    if (++st == NS) { st = 0; stph ^= 1u; }
                }
            }
        }
        if (pending >= 0) {
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&a_full[pending]);
        }
    } else {
        // ---- epilogue: group g drains the CTA's steps g, g + 2, ...; warp quarter = TMEM lane quarter
        const int g = (warp - kEpiWarp0) >> 2;
        const int qq = warp & 3;
        const float inv = *p.inv_scale;
        Walk w;
        w.start(p, g);
        w.i = -1;                                         // forces the per-unit set-up at the first step
        bool valid = false;
        __half* dst0 = nullptr;
        int unit_now = -1;
        w.i = 0;
        for (int k = g; k < total_steps; k += kEpiGroups, w.pos += kEpiGroups) {
            w.settle(su);
            if (w.i != unit_now) {
                unit_now = w.i;
                w.unit(p);
                const int q = w.tile * kTileCols + 31 * qq + lane;
                const int e = q / pl.Ws, X = q - e * pl.Ws;
                valid = lane < 31 && e < p.n && X < pl.W1;
                dst0 = p.out + ((size_t)e * pl.P1s + (X >> 1)) * 128 + (X & 1) * 32;
            }
            const int y = w.y_base + w.pos;
            const int acc = k % NACC;
            if (!mbar_wait_warp(&d_full[acc], ((uint32_t)(k / NACC)) & 1u, abortp, p.status, 37)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_d + acc * 64 + ((uint32_t)(qq * 32) << 16);
            __half* dst = dst0 + ((size_t)(y >> 1) * pl.W1s) * 128 + (y & 1) * 64;
            if constexpr (kThreads * S::PER_SM <= 768) {
                // registers allow it: the whole accumulator row in one round trip to tensor memory
                uint32_t v0[32], v1[32];
                tmem_ld_32x32(taddr, v0);                   // dx = 0 part of this column's output
                tmem_ld_32x32(taddr + 32, v1);              // dx = 1 part of the output one column to the left
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&d_empty[acc]);
#pragma unroll
                for (int j = 0; j < 32; j += 16) {
                    uint32_t pk[8];
#pragma unroll
                    for (int hh = 0; hh < 8; ++hh) {
                        const int c = j + 2 * hh;
                        float a0 = __uint_as_float(v0[c]), a1 = __uint_as_float(v0[c + 1]);
                        add2(a0, a1, __shfl_down_sync(0xffffffffu, __uint_as_float(v1[c]), 1),
                             __shfl_down_sync(0xffffffffu, __uint_as_float(v1[c + 1]), 1));
                        fma2(a0, a1, inv, s_bias[c], s_bias[c + 1]);
                        pk[hh] = relu_pack_h2(a0, a1);
                    }
                    if (valid)
                        asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                                     ::"l"(dst + j), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]),
                                       "r"(pk[6]), "r"(pk[7]) : "memory");
                }
            } else {
                // 64 registers per thread: sixteen output channels per round trip
#pragma unroll
                for (int j = 0; j < 32; j += 16) {
                    uint32_t v0[16], v1[16];
                    tmem_ld_32x16(taddr + j, v0);
                    tmem_ld_32x16(taddr + 32 + j, v1);
                    tmem_ld_wait();
                    if (j == 16) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&d_empty[acc]);
                    }
                    uint32_t pk[8];
#pragma unroll
                    for (int hh = 0; hh < 8; ++hh) {
                        const int c = 2 * hh;
                        float a0 = __uint_as_float(v0[c]), a1 = __uint_as_float(v0[c + 1]);
                        add2(a0, a1, __shfl_down_sync(0xffffffffu, __uint_as_float(v1[c]), 1),
                             __shfl_down_sync(0xffffffffu, __uint_as_float(v1[c + 1]), 1));
                        fma2(a0, a1, inv, s_bias[j + c], s_bias[j + c + 1]);
                        pk[hh] = relu_pack_h2(a0, a1);
                    }
                    if (valid)
                        asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                                     ::"l"(dst + j), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]),
                                       "r"(pk[6]), "r"(pk[7]) : "memory");
                }
            }
        }
    }
    if (*abortp) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_slot, S::TMEM);
}

__global__ void pack_conv1_kernel(const __nv_bfloat16* __restrict__ w, __half* __restrict__ wp, int C,
                                  const float* __restrict__ scale)
{
    const int K = 16 * C;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 128 * K) return;
    const int row = i / K, k = i - row * K;
    const int dy = row >> 6, dx = (row >> 5) & 1, o = row & 31;
    const int c = k >> 4, uy = (k >> 2) & 3, ux = k & 3;
    wp[i] = __float2half_rn(__bfloat162float(w[((o * C + c) * 8 + (4 * dy + uy)) * 8 + (4 * dx + ux)]) * scale[0]);
}

// output-row ranges per tile: enough units that every CTA of the grid gets several, few enough that the extra
// grid row each unit converts (a unit of k steps stages k + 1 rows) stays cheap
int choose_splits(int tiles, int H1, int grid)
{
    int best = 1;
    long best_cost = -1;
    for (int s = 1; s <= H1; ++s) {
        if (H1 % s) continue;                              // equal ranges only
        const int steps = H1 / s;
        if (s > 1 && steps < 2) break;
        const long rounds = ((long)tiles * s + grid - 1) / grid;
        const long cost = rounds * (steps + 2);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    return best;
}

template <int CG, int WC>
hts_status launch_variant(const CUtensorMap& weight_map, const CUtensorMap& frame_map, const Conv1Params& p, int grid,
                          int smem_bytes, cudaStream_t s)
{
    static int smem_set_by_device[kDeviceSlots] = {};
    int& smem_set = smem_set_by_device[device_slot()];
    if (smem_set < smem_bytes) {
        HTS_CUDA(cudaFuncSetAttribute(conv1_march_kernel<CG, WC>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
        // every kernel of the step asks for the largest shared-memory carve-out, so that the SMs are not
        // re-partitioned between consecutive kernels
        HTS_CUDA(cudaFuncSetAttribute(conv1_march_kernel<CG, WC>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
        smem_set = smem_bytes;
    }
    HTS_CUDA(launch_pdl(conv1_march_kernel<CG, WC>, dim3(grid), dim3(threads_of<CG>()), (size_t)smem_bytes, s, weight_map, frame_map, p));
    note_launch();
    return HTS_OK;
}

}  // namespace

bool conv1_plan(const Geometry& g, Conv1Plan* pl)
{
    // TMA boxes over the frames need 16-byte strides: H and W multiples of 4
    if (g.H % 4 || g.W % 4 || (g.C != 4 && g.C != 8 && g.C != 16) || g.W > 1024) return false;
    pl->C = g.C; pl->H = g.H; pl->W = g.W; pl->CG = g.C / 4;
    pl->Hs = g.H / 4; pl->Ws = g.W / 4;
    pl->H1 = pl->Hs - 1; pl->W1 = pl->Ws - 1;
    if (pl->H1 != g.H1 || pl->W1 != g.W1 || pl->Ws < 2 || pl->H1 < 1) return false;
    pl->H1s = (pl->H1 + 1) / 2; pl->W1s = (pl->W1 + 1) / 2; pl->P1s = pl->H1s * pl->W1s;
    pl->env_max = kTileCols / pl->Ws + 2;
    const bool twin = pl->CG == 1;                             // Shape<1>: two CTAs per SM
    pl->group_rows = pl->CG == 1 ? Shape<1>::KR : pl->CG == 2 ? Shape<2>::KR : Shape<4>::KR;
    pl->env_bytes = g.C * pl->group_rows * 4 * g.W;
    pl->env_pitch = (pl->env_bytes + 127) / 128 * 128;
    pl->stage_bytes = pl->env_max * pl->env_pitch;
    pl->ring = pl->CG == 1 ? Shape<1>::R : pl->CG == 2 ? Shape<2>::R : Shape<4>::R;
    pl->accs = pl->CG == 1 ? Shape<1>::NACC : pl->CG == 2 ? Shape<2>::NACC : Shape<4>::NACC;   // accs x 64 + ring x 32 CG columns
    const int fixed = 1024 + 2 * pl->CG * kChunkBytes;
    int st = ((twin ? 112 : 226) * 1024 - fixed) / pl->stage_bytes;
    if (st > kMaxStages) st = kMaxStages;
    if (st < 2) return false;
    pl->stages = st;
    pl->smem_bytes = fixed + st * pl->stage_bytes;
    return true;
}

hts_status conv1_pack_weights(const Conv1Plan& pl, const __nv_bfloat16* w1, __half* packed, const float* scale,
                              cudaStream_t s)
{
    const int total = 128 * 16 * pl.C;
    pack_conv1_kernel<<<(total + 255) / 256, 256, 0, s>>>(w1, packed, pl.C, scale);
    HTS_LAUNCH_CHECK("pack_conv1");
    return HTS_OK;
}

hts_status conv1_launch(const Conv1Plan& pl, const CUtensorMap& weight_map, Conv1MapCache& maps, const uint8_t* obs,
                        const Indexing& ix, int n, const float* bias, const float* inv_scale, __half* out, int* status,
                        cudaStream_t s)
{
    const int sm_count = device_sm_count(device_slot());
    const long cols = (long)n * pl.Ws;
    if (cols >= (1L << 31) - 256) return HTS_ERR_INVALID_ARG;
    // the tensor map over this frame buffer (dense: n frames; gathered: the whole pool)
    const int frames = ix.slots ? ix.pool : n;
    int slot = -1;
    for (int i = 0; i < Conv1MapCache::kEntries; ++i)
        if (maps.ptr[i] == obs && maps.frames[i] == frames) { slot = i; break; }
    if (slot < 0) {
        slot = maps.next;
        maps.next = (maps.next + 1) % Conv1MapCache::kEntries;
        if (!make_frames_map(&maps.map[slot], obs, pl.W, pl.H, pl.C, (uint64_t)frames, pl.group_rows)) {
            maps.ptr[slot] = nullptr;
            return HTS_ERR_CUDA;
        }
        maps.ptr[slot] = obs; maps.frames[slot] = frames;
    }
    Conv1Params p{};
    p.pl = pl; p.obs = obs; p.slots = ix.slots; p.pool = ix.pool; p.n = n;
    p.tiles = (int)((cols + kTileCols - 1) / kTileCols);
    const int max_grid = (pl.CG == 1 ? Shape<1>::PER_SM : 1) * sm_count;
    p.splits = choose_splits(p.tiles, pl.H1, max_grid);
    p.su = pl.H1 / p.splits;
    p.bias = bias; p.inv_scale = inv_scale; p.out = out; p.status = status;
    const long units = (long)p.tiles * p.splits;
    const int grid = units < max_grid ? (int)units : max_grid;
    const CUtensorMap& fm = maps.map[slot];
    if (pl.CG == 1) {
        if (pl.W == 84) return launch_variant<1, 84>(weight_map, fm, p, grid, pl.smem_bytes, s);
        return launch_variant<1, 0>(weight_map, fm, p, grid, pl.smem_bytes, s);
    }
    if (pl.CG == 2) return launch_variant<2, 0>(weight_map, fm, p, grid, pl.smem_bytes, s);
    if (pl.W == 96) return launch_variant<4, 96>(weight_map, fm, p, grid, pl.smem_bytes, s);
    return launch_variant<4, 0>(weight_map, fm, p, grid, pl.smem_bytes, s);
}

}  // namespace hts
