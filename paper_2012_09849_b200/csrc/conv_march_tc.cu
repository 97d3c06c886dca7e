// conv2 (4x4 / 2, as 2x2 taps on the space-to-depth(2) grid, 128 -> 64) and conv3 (3x3 / 1, 64 -> 64) of the
// policy-value network with the A operand in tensor memory.
//
// Same formulation as conv1_tc.cu, minus the byte conversion: the 128 rows of an MMA tile are consecutive grid
// COLUMNS of the batch (flat index q = env * Win + X) and the kernel marches down the grid rows.  Grid row Y of
// those columns (CIN fp16 channels per pixel) is copied once, shared memory -> registers -> tensor memory, into a
// ring of operand rows.  Step y multiplies ring entries y .. y + TY - 1 by the filter rows dy = 0 .. TY - 1
// (tcgen05.mma, A from tensor memory, 128 x (64 TX) x 16), so every entry serves TY steps and nothing is fetched
// once per tap.  The TX taps across are stacked along N: accumulator columns [64 dx, 64 dx + 64) hold the part of
// output (y, X - dx); the epilogue adds the halves of its TX - 1 right-hand neighbour lanes (warp quarters overlap by
// TX - 1 lanes, so the neighbours are in the same warp), applies scale, bias and ReLU and stores fp16 rows of 64
// channels.  Only grid rows and columns that have an output are ever multiplied, apart from the TX - 1 columns at
// the right edge of each environment: conv3 computes 7 of 9 columns (the flat-grid kernel it replaces: 49 of 81
// pixels), conv2 9 of 10.
//
// One CTA per SM: one thread stages a grid row of every environment the tile touches with ONE tensor-tiled TMA box
// ([CIN] x Win pixels x environments, 128-byte swizzle, so that eight neighbouring lanes read their 16-byte chunks
// from different banks); two groups of four converter warps take alternate grid rows; two threads issue the MMAs of
// alternate steps, each into its own accumulator; two groups of four epilogue warps drain alternate steps.
// All waits are bounded.
#include "conv_march_tc.cuh"
#include "tc_ptx.cuh"

namespace hts {
using namespace tc;

namespace {

constexpr int kIssuers = 2, kConvGroups = 2, kEpiGroups = 2;
constexpr int kAcc = 2;                          // accumulators: one per issuing thread and epilogue group
constexpr int kRing = 4;                         // operand rows in tensor memory
constexpr int kConvWarp0 = 4;                    // warp 0 stages, 1 and 2 issue, 3 idle, 4..11 convert, 12..19 epilogue
constexpr int kEpiWarp0 = kConvWarp0 + 4 * kConvGroups;
constexpr int kThreads = (kEpiWarp0 + 4 * kEpiGroups) * 32;
constexpr int kMaxStages = 4;

struct MarchParams {
    ConvMarchPlan pl;
    int n;
    int tiles;              // ceil(n * Win / tile_cols)
    int splits;             // equal ranges the Hout output rows of a tile are cut into
    int su;                 // steps per unit (Hout / splits); a unit stages su + TY - 1 grid rows
    const float* bias;
    const float* inv_scale;
    __half* out;
    int* status;
};

__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar)
{
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                 ::"r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ uint32_t relu_pack_h2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.relu.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Position of a role in the CTA's sequence of units (u = blockIdx.x + i * gridDim.x; all units have `su` steps).
struct Walk {
    int i, pos, tile, y_base;
    __device__ __forceinline__ void unit(const MarchParams& p)
    {
        const int u = blockIdx.x + i * gridDim.x;
        tile = u / p.splits;
        y_base = (u - tile * p.splits) * p.su;
    }
    __device__ __forceinline__ void settle(int len) { while (pos >= len) { pos -= len; ++i; } }
};

template <int TY, int TX, int CIN>
__global__ void __launch_bounds__(kThreads, 1)
conv_march_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const MarchParams p)
{
    constexpr int N = 64 * TX;                         // accumulator columns
    constexpr int KCH = CIN / 64;                      // 64-channel chunks per pixel = 128-byte rows per pixel
    constexpr int ECOLS = CIN / 2;                     // tensor-memory columns of one operand row
    constexpr int R = kRing, NACC = kAcc;
    constexpr int OVL = TX - 1;                        // lanes a warp quarter shares with the next one
    constexpr int kChunkBytes = N * 128;               // one filter chunk: N rows x 64 fp16
    static_assert(kIssuers + TY - 1 <= R, "an issuing thread must stay within one phase of the ring's barriers");
    static_assert(NACC * N + R * ECOLS <= 512, "tensor memory");
    const ConvMarchPlan& pl = p.pl;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t w_bar, in_full[kMaxStages], in_empty[kMaxStages], a_full[R], a_empty[R], d_full[NACC], d_empty[NACC];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ __align__(16) float s_bias[64];
    volatile int* abortp = &abort_flag;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    constexpr int w_bytes = TY * KCH * kChunkBytes;
    uint8_t* s_in = sm + w_bytes;
    const int NS = pl.stages;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int units = p.tiles * p.splits;
    const int Win = pl.Win;

    if (threadIdx.x == 0) {
        mbar_init(&w_bar, 1);
        for (int s = 0; s < kMaxStages; ++s) { mbar_init(&in_full[s], 1); mbar_init(&in_empty[s], 4 * kConvGroups); }
        for (int s = 0; s < R; ++s) { mbar_init(&a_full[s], 4); mbar_init(&a_empty[s], TY); }
        for (int s = 0; s < NACC; ++s) { mbar_init(&d_full[s], 1); mbar_init(&d_empty[s], 4); }
        abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmW);
        tma_prefetch_desc(&tmX);
    }
    if (threadIdx.x >= 96 && threadIdx.x < 128) {
        s_bias[threadIdx.x - 96] = p.bias[threadIdx.x - 96];
        s_bias[threadIdx.x - 64] = p.bias[threadIdx.x - 64];
    }
    if (warp == 1) tmem_alloc(&tmem_slot, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_slot, tmem_a = tmem_slot + NACC * N;
    if (threadIdx.x == 0) {                                   // the filter does not depend on the previous kernel
        mbar_arrive_expect_tx(&w_bar, (uint32_t)w_bytes);
        for (int dy = 0; dy < TY; ++dy)
            for (int hf = 0; hf < KCH; ++hf) tma_load_2d(sm + (dy * KCH + hf) * kChunkBytes, &tmW, hf * 64, dy * N, &w_bar);
    }
    pdl_wait();
    pdl_trigger();

    const int my_units = blockIdx.x < units ? (units - blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    const int su = p.su, ru = p.su + TY - 1;                  // steps and grid rows per unit
    const int total_steps = my_units * su;

    if (warp == 0) {
        // ---- staging: one box per grid row: Win pixels of every environment the tile touches
        if (lane == 0) {
            int st = 0;
            uint32_t stph = 0;
            bool alive = true;
            Walk w;
            for (w.i = 0; alive && w.i < my_units; ++w.i) {
                w.unit(p);
                const int e_first = (w.tile * pl.tile_cols) / Win;
                for (int Y = w.y_base; Y < w.y_base + ru; ++Y) {
                    if (!mbar_wait(&in_empty[st], stph ^ 1u, abortp, p.status, 41)) { alive = false; break; }
                    mbar_arrive_expect_tx(&in_full[st], (uint32_t)(pl.env_max * Win * CIN * 2));
                    if (KCH == 1) tma_load_3d(s_in + st * pl.stage_bytes, &tmX, 0, Y * Win, e_first, &in_full[st]);
                    else tma_load_4d(s_in + st * pl.stage_bytes, &tmX, 0, 0, Y * Win, e_first, &in_full[st]);
                    if (++st == NS) { st = 0; stph ^= 1u; }
                }
            }
        }
    } else if (warp <= kIssuers) {
        // ---- MMA issue: thread g takes the CTA's steps g, g + 2, ... into accumulator g.
        //      Step k of the CTA (unit i) reads operand rows k + i (TY - 1) .. + TY - 1.
        if (lane == 0) {
            const int g = warp - 1;
            constexpr uint32_t idesc = instr_desc_f16(0, 128, N);
            uint64_t bdesc[TY][KCH];
#pragma unroll
            for (int dy = 0; dy < TY; ++dy)
#pragma unroll
                for (int hf = 0; hf < KCH; ++hf) bdesc[dy][hf] = smem_desc_sw128(base + (dy * KCH + hf) * kChunkBytes);
            bool alive = mbar_wait(&w_bar, 0, abortp, p.status, 42);
            const uint32_t d_addr = tmem_d + g * N;
            Walk w;
            w.i = 0; w.pos = g;
            for (int k = g; alive && k < total_steps; k += kIssuers, w.pos += kIssuers) {
                w.settle(su);
                const int r0 = k + w.i * (TY - 1);
                // operands first, accumulator second (a waiter must stay within one phase of a parity barrier:
                // consecutive steps of this thread are 2, or across a unit boundary 2 + TY - 1 <= R, rows apart)
                bool ok = true;
#pragma unroll
                for (int t = 0; t < TY; ++t) ok = ok && mbar_wait(&a_full[(r0 + t) % R], ((uint32_t)((r0 + t) / R)) & 1u, abortp, p.status, 44);
                if (!ok) break;
                if (!mbar_wait(&d_empty[g], (((uint32_t)(k / NACC)) & 1u) ^ 1u, abortp, p.status, 43)) break;
                tc_fence_after();
#pragma unroll
                for (int dy = 0; dy < TY; ++dy) {
                    const uint32_t a_addr = tmem_a + ((r0 + dy) % R) * ECOLS;
#pragma unroll
                    for (int hf = 0; hf < KCH; ++hf)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            mma_f16_ts(d_addr, a_addr + hf * 32 + 8 * kk, bdesc[dy][hf] + 2 * kk, idesc, (dy | hf | kk) != 0);
                }
                // An operand row is free once the TY steps that read it are done.  Rows at the start (end) of a unit have
                // fewer readers; the unit's first (last) step arrives for the missing ones.
#pragma unroll
                for (int t = 0; t < TY; ++t) {
                    uint64_t* bar = &a_empty[(r0 + t) % R];
                    mma_commit(bar);
                    if (w.pos == 0) for (int x = 0; x < TY - 1 - t; ++x) mma_commit(bar);
                    if (w.pos == su - 1) for (int x = 0; x < t; ++x) mma_commit(bar);
                }
                mma_commit(&d_full[g]);
            }
        }
    } else if (warp >= kConvWarp0 && warp < kEpiWarp0) {
        // ---- copy to tensor memory: thread = grid column q of the tile; group h takes the CTA's grid rows h, h + 2, ...
        const int h = (warp - kConvWarp0) >> 2;
        const int qq = warp & 3;
        const uint32_t st_addr = tmem_a + ((uint32_t)(qq * 32) << 16);
        int st = 0;
        uint32_t stph = 0;
        int r = 0;                                        // grid rows of this CTA so far
        int pending = -1;                                 // ring entry whose tensor-memory stores are still in flight
        bool alive = true;
        Walk w;
        for (w.i = 0; alive && w.i < my_units; ++w.i) {
            w.unit(p);
            const int q = w.tile * pl.tile_cols + (32 - OVL) * qq + lane;
            const int e = q / Win, X = q - e * Win;
            const int e_first = (w.tile * pl.tile_cols) / Win;
            // 128-byte row of this pixel inside the staged grid row (columns past the staged environments read row 0:
            // their results are never stored)
            int rho = ((e - e_first) * Win + X) * KCH;
            if (e - e_first >= pl.env_max) rho = 0;
            for (int j = 0; j < ru; ++j, ++r) {
                if (!mbar_wait_warp(&in_full[st], stph, abortp, p.status, 45)) { alive = false; break; }
                if ((r & 1) == h) {
                    const int s = r % R;
                    const uint8_t* src = s_in + st * pl.stage_bytes;
#pragma unroll
                    for (int hf = 0; hf < KCH; ++hf) {
                        const int row = rho + hf;
                        const uint8_t* rp = src + row * 128;
                        const int sw = row & 7;
                        uint32_t v[32];
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const uint4 x = *reinterpret_cast<const uint4*>(rp + ((c ^ sw) << 4));
                            v[4 * c] = x.x; v[4 * c + 1] = x.y; v[4 * c + 2] = x.z; v[4 * c + 3] = x.w;
                        }
                        if (hf == 0) {
                            if (pending >= 0) {               // the previous row's stores overlapped these loads
                                tmem_st_wait();
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(&a_full[pending]);
                            }
                            if (!mbar_wait_warp(&a_empty[s], (((uint32_t)(r / R)) & 1u) ^ 1u, abortp, p.status, 46)) { alive = false; break; }
                            tc_fence_after();
                        }
                        tmem_st_32x32(st_addr + s * ECOLS + hf * 32, v);
                    }
                    if (!alive) break;
                    pending = s;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&in_empty[st]);   // every converter warp arrives once per staged row
                if (++st == NS) { st = 0; stph ^= 1u; }
            }
        }
        if (pending >= 0) {
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&a_full[pending]);
        }
    } else if (warp >= kEpiWarp0) {
        // ---- epilogue: group g drains the CTA's steps g, g + 2, ... (accumulator g); warp quarter = TMEM lane quarter
        const int g = (warp - kEpiWarp0) >> 2;
        const int qq = warp & 3;
        const float inv = *p.inv_scale;
        const int Pout = pl.Hout * pl.Wout;
        Walk w;
        w.i = 0; w.pos = g;
        bool valid = false;
        __half* dst0 = nullptr;
        int unit_now = -1;
        for (int k = g; k < total_steps; k += kEpiGroups, w.pos += kEpiGroups) {
            w.settle(su);
            if (w.i != unit_now) {
                unit_now = w.i;
                w.unit(p);
                const int q = w.tile * pl.tile_cols + (32 - OVL) * qq + lane;
                const int e = q / Win, X = q - e * Win;
                valid = lane < 32 - OVL && e < p.n && X < pl.Wout;
                dst0 = p.out + ((size_t)e * Pout + X) * 64;
            }
            const int y = w.y_base + w.pos;
            if (!mbar_wait_warp(&d_full[g], ((uint32_t)(k / NACC)) & 1u, abortp, p.status, 47)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_d + g * N + ((uint32_t)(qq * 32) << 16);
            __half* dst = dst0 + (size_t)y * pl.Wout * 64;
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 16) {
                uint32_t v[TX][16];
#pragma unroll
                for (int dx = 0; dx < TX; ++dx) tmem_ld_32x16(taddr + dx * 64 + c0, v[dx]);
                tmem_ld_wait();
                if (c0 == 48) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&d_empty[g]);
                }
                uint32_t pk[8];
#pragma unroll
                for (int hh = 0; hh < 8; ++hh) {
                    float a0 = __uint_as_float(v[0][2 * hh]), a1 = __uint_as_float(v[0][2 * hh + 1]);
#pragma unroll
                    for (int dx = 1; dx < TX; ++dx) {      // the part of this output that lane + dx computed
                        a0 += __shfl_down_sync(0xffffffffu, __uint_as_float(v[dx][2 * hh]), dx);
                        a1 += __shfl_down_sync(0xffffffffu, __uint_as_float(v[dx][2 * hh + 1]), dx);
                    }
                    pk[hh] = relu_pack_h2(fmaf(a0, inv, s_bias[c0 + 2 * hh]), fmaf(a1, inv, s_bias[c0 + 2 * hh + 1]));
                }
                if (valid)
                    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                                 ::"l"(dst + c0), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]),
                                   "r"(pk[6]), "r"(pk[7]) : "memory");
            }
        }
    }
    if (*abortp) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_slot, 512);
}

// output-row ranges per tile (equal ranges): enough units for every CTA, few enough that the TY - 1 extra grid rows
// each unit copies stay cheap
int choose_splits(int tiles, int Hout, int TY, int grid)
{
    int best = 1;
    long best_cost = -1;
    for (int s = 1; s <= Hout; ++s) {
        if (Hout % s) continue;
        const int steps = Hout / s;
        const long rounds = ((long)tiles * s + grid - 1) / grid;
        const long cost = rounds * (4 * steps + TY - 1 + 4);   // a copied row costs about a quarter of a step
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = s; }
    }
    return best;
}

template <int TY, int TX, int CIN>
hts_status launch_variant(const ConvMarchPlan& pl, const CUtensorMap& in_map, const CUtensorMap& weight_map, const MarchParams& p,
                          int grid, cudaStream_t s)
{
    static int smem_set_by_device[kDeviceSlots] = {};
    int& smem_set = smem_set_by_device[device_slot()];
    if (smem_set < pl.smem_bytes) {
        HTS_CUDA(cudaFuncSetAttribute(conv_march_kernel<TY, TX, CIN>, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem_bytes));
        HTS_CUDA(cudaFuncSetAttribute(conv_march_kernel<TY, TX, CIN>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
        smem_set = pl.smem_bytes;
    }
    HTS_CUDA(launch_pdl(conv_march_kernel<TY, TX, CIN>, dim3(grid), dim3(kThreads), (size_t)pl.smem_bytes, s, in_map, weight_map, p));
    note_launch();
    return HTS_OK;
}

}  // namespace

bool conv_march_plan(int TY, int TX, int CIN, int Hin, int Win, ConvMarchPlan* pl)
{
    if (!((TY == 2 && TX == 2 && CIN == 128) || (TY == 3 && TX == 3 && CIN == 64))) return false;
    pl->TY = TY; pl->TX = TX; pl->CIN = CIN; pl->Hin = Hin; pl->Win = Win;
    pl->Hout = Hin - TY + 1; pl->Wout = Win - TX + 1;
    if (pl->Hout < 1 || pl->Wout < 1) return false;
    pl->tile_cols = 4 * (32 - (TX - 1));
    pl->env_max = (Win - 1 + pl->tile_cols + (TX - 1) - 1) / Win + 1;   // a tile spans tile_cols + TX - 1 columns from any offset
    if (Win > 256 || pl->env_max > 256) return false;          // TMA box extents
    pl->stage_bytes = (pl->env_max * Win * CIN * 2 + 1023) / 1024 * 1024;
    const int fixed = 1024 + TY * (CIN / 64) * (64 * TX) * 128;
    int st = (226 * 1024 - fixed) / pl->stage_bytes;
    if (st > kMaxStages) st = kMaxStages;
    if (st < 2) return false;
    pl->stages = st;
    pl->smem_bytes = fixed + st * pl->stage_bytes;
    return true;
}

hts_status conv_march_launch(const ConvMarchPlan& pl, const CUtensorMap& in_map, const CUtensorMap& weight_map,
                             const ConvMarchArgs& a, cudaStream_t s)
{
    const int sm_count = device_sm_count(device_slot());
    const long cols = (long)a.n * pl.Win;
    if (cols >= (1L << 31) - 256) return HTS_ERR_INVALID_ARG;
    MarchParams p{};
    p.pl = pl; p.n = a.n;
    p.tiles = (int)((cols + pl.tile_cols - 1) / pl.tile_cols);
    p.splits = choose_splits(p.tiles, pl.Hout, pl.TY, sm_count);
    p.su = pl.Hout / p.splits;
    p.bias = a.bias; p.inv_scale = a.inv_scale; p.out = a.out; p.status = a.status;
    const long units = (long)p.tiles * p.splits;
    const int grid = units < sm_count ? (int)units : sm_count;
    if (pl.TY == 2) return launch_variant<2, 2, 128>(pl, in_map, weight_map, p, grid, s);
    return launch_variant<3, 3, 64>(pl, in_map, weight_map, p, grid, s);
}

}  // namespace hts
