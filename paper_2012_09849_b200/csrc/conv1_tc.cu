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
// Work unit = (tile of 125 grid columns, range of output rows).  A CTA is a pipeline of four roles:
// warp 0 stages the four input rows under a grid row (one bulk copy per environment and channel)
// into a ring in shared memory; warps 4..7 convert (thread = grid column) and write tensor memory;
// lane 0 of warps 1 and 2 issue the MMAs of alternate steps, each into its own accumulator; warps
// 8..11 run the epilogue.  All waits are bounded.
#include "conv1_tc.cuh"
#include "tc_ptx.cuh"

namespace hts {
using namespace tc;

namespace {

constexpr int kThreads = 384;                   // warp 0 copies, 1 and 2 issue, 3 idle, 4..7 convert, 8..11 epilogue
constexpr int kTileCols = 124;                  // new grid columns per tile (4 quarters x 31; one more is shared)
constexpr int kChunkBytes = 64 * 128;           // one filter K chunk: 64 rows (dx, o) x 64 fp16
constexpr int kMaxStages = 8;
constexpr int kMaxRing = 4;

struct Conv1Params {
    Conv1Plan pl;
    const uint8_t* obs;
    const int32_t* slots;   // frame of each row in obs, or nullptr: row e is frame e
    int pool;               // frames in obs when slots are given
    int n;
    int tiles;              // ceil(n * Ws / 124)
    int splits;             // ranges the H1 output rows of a tile are cut into
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

// fp32 pair -> packed fp16 pair with ReLU, saturating at the largest finite fp16
__device__ __forceinline__ uint32_t relu_pack_h2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.relu.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// the unit's tile and output-row range
struct Unit {
    int tile, y0, y1;
    __device__ __forceinline__ void set(int u, int splits, int H1)
    {
        tile = u / splits;
        const int part = u - tile * splits;
        y0 = part * H1 / splits;
        y1 = (part + 1) * H1 / splits;
    }
};

// CG: groups of four channels.  WC: the frame width when known at compile time (the converter's loads then
// use immediate offsets), 0 = any.  NI: issuing threads.
template <int CG, int WC>
__global__ void __launch_bounds__(kThreads, CG == 1 ? 2 : 1)
conv1_march_kernel(const __grid_constant__ CUtensorMap tmW, const Conv1Params p)
{
    const Conv1Plan& pl = p.pl;
    constexpr int C = 4 * CG;
    constexpr int ACOLS = 32 * CG;                     // tensor-memory columns of one operand row
    const int W = WC ? WC : pl.W;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t w_bar, u8_full[kMaxStages], u8_empty[kMaxStages], a_full[kMaxRing], a_empty[kMaxRing], d_full[2], d_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ __align__(16) float s_bias[32];
    volatile int* abortp = &abort_flag;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    constexpr int w_bytes = 2 * CG * kChunkBytes;
    uint8_t* s_u8 = sm + w_bytes;
    const int NS = pl.stages, R = pl.ring;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int units = p.tiles * p.splits;

    if (threadIdx.x == 0) {
        mbar_init(&w_bar, 1);
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&u8_full[s], 1); mbar_init(&u8_empty[s], 128); }
        for (int s = 0; s < kMaxRing; ++s) { mbar_init(&a_full[s], 128); mbar_init(&a_empty[s], 2); }
        for (int s = 0; s < 2; ++s) { mbar_init(&d_full[s], 1); mbar_init(&d_empty[s], 128); }
        abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmW);
    }
    if (threadIdx.x >= 96 && threadIdx.x < 128) s_bias[threadIdx.x - 96] = p.bias[threadIdx.x - 96];
    if (warp == 1) tmem_alloc(&tmem_slot, (uint32_t)pl.tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_slot, tmem_a = tmem_slot + 128;     // two accumulators of 64 columns, then the ring
    if (threadIdx.x == 0) {                                   // the filter does not depend on the previous kernel
        mbar_arrive_expect_tx(&w_bar, (uint32_t)w_bytes);
        for (int dy = 0; dy < 2; ++dy)
            for (int g = 0; g < CG; ++g) tma_load_2d(sm + (dy * CG + g) * kChunkBytes, &tmW, g * 64, dy * 64, &w_bar);
    }
    pdl_wait();
    pdl_trigger();

    if (warp == 0) {
        // ---- staging: the four input rows under grid row Y, for every environment the tile touches
        const size_t chan = (size_t)pl.H * W, frame = chan * C;
        const uint32_t row_bytes = 4u * (uint32_t)W;
        int st = 0;
        uint32_t stph = 0;
        Unit un;
        for (int u = blockIdx.x; u < units; u += gridDim.x) {
            un.set(u, p.splits, pl.H1);
            const int e_first = (un.tile * kTileCols) / pl.Ws;
            int e_last = (un.tile * kTileCols + kTileCols) / pl.Ws;
            if (e_last > p.n - 1) e_last = p.n - 1;
            const int copies = (e_last - e_first + 1) * C;
            bool alive = true;
            for (int Y = un.y0; Y <= un.y1; ++Y) {
                if (!mbar_wait_warp(&u8_empty[st], stph ^ 1u, abortp, p.status, 31)) { alive = false; break; }
                uint8_t* dst = s_u8 + st * pl.stage_bytes;
                if (lane == 0) mbar_arrive_expect_tx(&u8_full[st], (uint32_t)copies * row_bytes);
                __syncwarp();
                for (int i = lane; i < copies; i += 32) {
                    const int ei = i / C, c = i - ei * C;
                    const uint8_t* src = p.obs + frame_of(p, e_first + ei) * frame + c * chan + (size_t)(4 * Y) * W;
                    bulk_load(dst + i * row_bytes, src, row_bytes, &u8_full[st]);
                }
                if (++st == NS) { st = 0; stph ^= 1u; }
            }
            if (!alive) break;
        }
    } else if (warp == 1 || warp == 2) {
        // ---- MMA issue: thread g takes the CTA's steps g, g + 2, ... into accumulator g
        if (lane == 0) {
            const int g = warp - 1;
            constexpr uint32_t idesc = instr_desc_f16(0, 128, 64);
            bool alive = mbar_wait(&w_bar, 0, abortp, p.status, 32);
            const uint32_t d_addr = tmem_d + g * 64;
            int s = 0;                                    // ring entry of grid row Y = y and the parity of its current use
            uint32_t sph = 0;
            int sc = 0;                                   // steps of this CTA so far
            Unit un;
            for (int u = blockIdx.x; alive && u < units; u += gridDim.x) {
                un.set(u, p.splits, pl.H1);
                for (int y = un.y0; y < un.y1; ++y, ++sc) {
                    const int s1 = s + 1 == R ? 0 : s + 1;
                    const uint32_t ph1 = s + 1 == R ? sph ^ 1u : sph;
                    if ((sc & 1) == g) {
                        if (!mbar_wait(&d_empty[g], (((uint32_t)sc >> 1) & 1u) ^ 1u, abortp, p.status, 33)) { alive = false; break; }
                        if (!mbar_wait(&a_full[s], sph, abortp, p.status, 34)) { alive = false; break; }
                        if (!mbar_wait(&a_full[s1], ph1, abortp, p.status, 34)) { alive = false; break; }
                        tc_fence_after();
#pragma unroll
                        for (int dy = 0; dy < 2; ++dy) {
                            const uint32_t a_addr = tmem_a + (dy ? s1 : s) * ACOLS;
#pragma unroll
                            for (int cg = 0; cg < CG; ++cg) {
                                const uint64_t bdesc = smem_desc_sw128(base + (dy * CG + cg) * kChunkBytes);
#pragma unroll
                                for (int k = 0; k < 4; ++k)
                                    mma_f16_ts(d_addr, a_addr + cg * 32 + 8 * k, bdesc + 2 * k, idesc, (dy | cg | k) != 0);
                            }
                        }
                        // an operand row is read by two steps (as the lower and as the upper grid row); the first
                        // and the last row of a unit by one only, which then arrives for both
                        mma_commit(&a_empty[s]);
                        mma_commit(&a_empty[s1]);
                        if (y == un.y0) mma_commit(&a_empty[s]);
                        if (y == un.y1 - 1) mma_commit(&a_empty[s1]);
                        mma_commit(&d_full[g]);
                    }
                    s = s1; sph = ph1;
                }
                if (++s == R) { s = 0; sph ^= 1u; }       // past the unit's last grid row
            }
        }
    } else if (warp >= 4 && warp < 8) {
        // ---- convert: thread = grid column q of the tile, one operand row per staged grid row
        const int qq = warp & 3;
        const uint32_t st_addr = tmem_a + ((uint32_t)(qq * 32) << 16);
        int s = 0, st = 0;
        uint32_t sph = 0, stph = 0;
        Unit un;
        bool alive = true;
        for (int u = blockIdx.x; alive && u < units; u += gridDim.x) {
            un.set(u, p.splits, pl.H1);
            const int q = un.tile * kTileCols + 31 * qq + lane;
            const int e = q / pl.Ws, X = q - e * pl.Ws;
            const int e_first = (un.tile * kTileCols) / pl.Ws;
            // columns past the end of the batch read the start of the buffer: their results are never stored
            const int off = e < p.n ? (e - e_first) * C * 4 * W + 4 * X : 0;
            for (int Y = un.y0; Y <= un.y1; ++Y) {
                if (!mbar_wait_warp(&u8_full[st], stph, abortp, p.status, 35)) { alive = false; break; }
                const uint8_t* src = s_u8 + st * pl.stage_bytes + off;
#pragma unroll
                for (int cg = 0; cg < CG; ++cg) {
                    uint32_t r[32];
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int uy = 0; uy < 4; ++uy)
                            u8x4_to_h4(*reinterpret_cast<const uint32_t*>(src + ((cg * 4 + c) * 4 + uy) * W),
                                       r[c * 8 + uy * 2], r[c * 8 + uy * 2 + 1]);
                    if (cg == CG - 1) mbar_arrive(&u8_empty[st]);         // the staged rows are in registers
                    if (cg == 0) {
                        if (!mbar_wait_warp(&a_empty[s], sph ^ 1u, abortp, p.status, 36)) { alive = false; break; }
                        tc_fence_after();
                    }
                    tmem_st_32x32(st_addr + s * ACOLS + cg * 32, r);
                }
                if (!alive) break;
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(&a_full[s]);
                if (++s == R) { s = 0; sph ^= 1u; }
                if (++st == NS) { st = 0; stph ^= 1u; }
            }
        }
    } else if (warp >= 8) {
        // ---- epilogue: warps 8..11 read TMEM lane quarters 0..3
        const int qq = warp & 3;
        const float inv = *p.inv_scale;
        int sc = 0;
        Unit un;
        bool alive = true;
        for (int u = blockIdx.x; alive && u < units; u += gridDim.x) {
            un.set(u, p.splits, pl.H1);
            const int q = un.tile * kTileCols + 31 * qq + lane;
            const int e = q / pl.Ws, X = q - e * pl.Ws;
            const bool valid = lane < 31 && e < p.n && X < pl.W1;
            __half* dst0 = p.out + ((size_t)e * pl.P1s + (X >> 1)) * 128 + (X & 1) * 32;
            for (int y = un.y0; y < un.y1; ++y, ++sc) {
                const int acc = sc & 1;
                if (!mbar_wait_warp(&d_full[acc], ((uint32_t)sc >> 1) & 1u, abortp, p.status, 37)) { alive = false; break; }
                tc_fence_after();
                const uint32_t taddr = tmem_d + acc * 64 + ((uint32_t)(qq * 32) << 16);
                __half* dst = dst0 + ((size_t)(y >> 1) * pl.W1s) * 128 + (y & 1) * 64;
#pragma unroll
                for (int j = 0; j < 32; j += 16) {
                    uint32_t v0[16], v1[16];
                    tmem_ld_32x16(taddr + j, v0);               // dx = 0 part of this column's output
                    tmem_ld_32x16(taddr + 32 + j, v1);          // dx = 1 part of the output one column to the left
                    tmem_ld_wait();
                    if (j == 16) {
                        tc_fence_before();
                        mbar_arrive(&d_empty[acc]);
                    }
                    uint32_t pk[8];
#pragma unroll
                    for (int hh = 0; hh < 8; ++hh) {
                        const int c = 2 * hh;
                        const float a0 = __uint_as_float(v0[c]) + __shfl_down_sync(0xffffffffu, __uint_as_float(v1[c]), 1);
                        const float a1 = __uint_as_float(v0[c + 1]) + __shfl_down_sync(0xffffffffu, __uint_as_float(v1[c + 1]), 1);
                        pk[hh] = relu_pack_h2(fmaf(a0, inv, s_bias[j + c]), fmaf(a1, inv, s_bias[j + c + 1]));
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
    if (warp == 1) tmem_dealloc(tmem_slot, (uint32_t)pl.tmem_cols);
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
        const int steps = (H1 + s - 1) / s;
        if (s > 1 && steps < 3) break;
        const long rounds = ((long)tiles * s + grid - 1) / grid;
        const long cost = rounds * (steps + 2);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    return best;
}

template <int CG, int WC>
hts_status launch_variant(const CUtensorMap& weight_map, const Conv1Params& p, int grid, int smem_bytes, cudaStream_t s)
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
    HTS_CUDA(launch_pdl(conv1_march_kernel<CG, WC>, dim3(grid), dim3(kThreads), (size_t)smem_bytes, s, weight_map, p));
    note_launch();
    return HTS_OK;
}

}  // namespace

bool conv1_plan(const Geometry& g, Conv1Plan* pl)
{
    // bulk copies of four input rows start and end on 16-byte boundaries when W is a multiple of 4
    if (g.H % 4 || g.W % 4 || (g.C != 4 && g.C != 8 && g.C != 16)) return false;
    pl->C = g.C; pl->H = g.H; pl->W = g.W; pl->CG = g.C / 4;
    pl->Hs = g.H / 4; pl->Ws = g.W / 4;
    pl->H1 = pl->Hs - 1; pl->W1 = pl->Ws - 1;
    if (pl->H1 != g.H1 || pl->W1 != g.W1 || pl->Ws < 2 || pl->H1 < 1) return false;
    pl->H1s = (pl->H1 + 1) / 2; pl->W1s = (pl->W1 + 1) / 2; pl->P1s = pl->H1s * pl->W1s;
    pl->env_max = kTileCols / pl->Ws + 2;
    pl->stage_bytes = (pl->env_max * g.C * 4 * g.W + 127) / 128 * 128;
    const bool two_per_sm = pl->CG == 1;
    pl->ring = pl->CG == 4 ? 3 : 4;
    pl->tmem_cols = two_per_sm ? 256 : 512;                    // 128 for the accumulators + ring x 32 CG
    const int fixed = 1024 + 2 * pl->CG * kChunkBytes;
    const int budget = (two_per_sm ? 112 : 226) * 1024 - fixed;
    int st = budget / pl->stage_bytes;
    if (st > kMaxStages) st = kMaxStages;
    if (st < 3) return false;
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

hts_status conv1_launch(const Conv1Plan& pl, const CUtensorMap& weight_map, const uint8_t* obs, const Indexing& ix, int n,
                        const float* bias, const float* inv_scale, __half* out, int* status, cudaStream_t s)
{
    const int sm_count = device_sm_count(device_slot());
    const long cols = (long)n * pl.Ws;
    if (cols >= (1L << 31) - 256) return HTS_ERR_INVALID_ARG;
    Conv1Params p{};
    p.pl = pl; p.obs = obs; p.slots = ix.slots; p.pool = ix.pool; p.n = n;
    p.tiles = (int)((cols + kTileCols - 1) / kTileCols);
    const int per_sm = pl.CG == 1 ? 2 : 1;
    const int max_grid = per_sm * sm_count;
    p.splits = choose_splits(p.tiles, pl.H1, max_grid);
    p.bias = bias; p.inv_scale = inv_scale; p.out = out; p.status = status;
    const long units = (long)p.tiles * p.splits;
    const int grid = units < max_grid ? (int)units : max_grid;
    if (pl.CG == 1) {
        if (pl.W == 84) return launch_variant<1, 84>(weight_map, p, grid, pl.smem_bytes, s);
        return launch_variant<1, 0>(weight_map, p, grid, pl.smem_bytes, s);
    }
    if (pl.CG == 2) return launch_variant<2, 0>(weight_map, p, grid, pl.smem_bytes, s);
    if (pl.W == 96) return launch_variant<4, 96>(weight_map, p, grid, pl.smem_bytes, s);
    return launch_variant<4, 0>(weight_map, p, grid, pl.smem_bytes, s);
}

}  // namespace hts
