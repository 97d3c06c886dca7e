// Tensor-core path of the actor step (bf16 weights): the convolution and FC layers of the
// policy-value network (Appendix F.1 / F.2) as tcgen05 GEMMs with TMA-fed shared-memory
// operands and fp32 accumulators in tensor memory.
//
// Formulation.  Activations live in HBM/L2 as row-major [pixel rows, channels] matrices.
// A k x k / s convolution with k = 2s is a 2x2/1 convolution on the space-to-depth(s) image,
// and a stride-1 convolution on a flat pixel grid is a sum over taps of row-shifted GEMMs:
//     D[m, o] = sum_tap sum_c X[m + dy*W_in + dx, c] * W[o, tap, c]
// computed for every row m of the input grid; rows whose (y, x) fall outside the output extent
// are discarded by the epilogue.  Every K chunk (64 channels of one tap) is one dense TMA box.
// The FC layer is the same kernel with one tap and a fixed split of K across CTAs; the split
// partials are summed in index order by the heads kernel, so nothing depends on the batch size.
//
// Operand type.  Both MMA operands are fp16 (kind::f16, fp32 accumulation).  The caller's bf16
// weights are multiplied by a per-layer power of two that brings the largest magnitude just
// below 2^15 and converted to fp16: exact for every weight within 2^-29 of the largest (bf16
// has 8 significant bits, fp16 has 11); the epilogue divides the power of two out again.
// Activations are stored as fp16 (clamped at the largest finite value): 11 significant bits
// instead of bf16's 8, which keeps the logits well inside the 2e-2 parity bound.
#include <new>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include "common.cuh"
#include "tc_ptx.cuh"
#include "tc_host.cuh"
#include "conv1_tc.cuh"
#include "conv_res_tc.cuh"

namespace hts {
using namespace tc;

namespace {

constexpr int BM = 128;                 // rows per tile = TMEM lanes
constexpr int BK = 64;                  // 16-bit elements per K chunk = one 128-byte swizzle row
constexpr int STAGES = 3;                 // 3 x 32 KiB: two CTAs per SM, so the 224 FC tiles run in one wave
constexpr int A_BYTES = BM * BK * 2;    // 16 KiB
enum { EPI_SPLITK = 1 };
enum { L_CONV1 = 0, L_CONV2, L_CONV3, L_FC, L_COUNT };

struct GemmParams {
    int taps, cpt;                      // filter taps, K chunks per tap
    int tap_shift[9];                   // row shift of each tap on the flat input grid
    int nk;                             // K chunks handled by one CTA (all of them, or one split)
    int n_env;                          // valid environments (conv) / valid rows (FC)
    int P_in, W_in, H_out, W_out, P_out;   // conv epilogue geometry (pixels per env, grid widths)
    const float* bias;
    const float* inv_scale;             // device scalar: undoes the weight scaling of this layer
    __half* out_h;                      // conv: rows [env*P_out + y*W_out + x][64]
    float* out_f32;                     // split-K partials [split][rows][ldo]
    size_t split_stride;
    int ldo;
    int* status;
};

__device__ __forceinline__ uint32_t pack_relu_h2(float a, float b)
{
    a = fminf(fmaxf(a, 0.f), 65504.f);
    b = fminf(fmaxf(b, 0.f), 65504.f);
    __half2 t = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&t);
}

template <int BN, int EPI>
__global__ void __launch_bounds__(192)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmParams p)
{
    constexpr int B_BYTES = BN * BK * 2;
    constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    constexpr uint32_t TMEM_COLS = BN < 32 ? 32 : BN;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[STAGES], empty_bar[STAGES], accum_bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* tiles = smem_raw + (base - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    volatile int* abortp = &abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&accum_bar, 1);
        abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) tmem_alloc(&tmem_base_slot, TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_slot;
    // The weight halves of the first stages do not depend on the previous kernel: they are on their way while
    // this one still waits for it.
    if (warp == 0 && lane == 0) {
        for (int kc = 0; kc < p.nk && kc < STAGES; ++kc) {
            mbar_arrive_expect_tx(&full_bar[kc], STAGE_BYTES);
            tma_load_2d(tiles + kc * STAGE_BYTES + A_BYTES, &tmB, (blockIdx.z * p.nk + kc) * BK, n0, &full_bar[kc]);
        }
    }
    pdl_wait();
    pdl_trigger();

    if (warp == 0) {
        if (lane == 0) {
            for (int kc = 0; kc < p.nk; ++kc) {
                const int s = kc % STAGES;
                const uint32_t ph = (uint32_t)(kc / STAGES) & 1u;
                if (!mbar_wait(&empty_bar[s], ph ^ 1u, abortp, p.status, 1)) break;
                const int g = blockIdx.z * p.nk + kc;
                const int tap = g / p.cpt, sub = g - tap * p.cpt;
                uint8_t* a_dst = tiles + s * STAGE_BYTES;
                if (kc >= STAGES) {
                    mbar_arrive_expect_tx(&full_bar[s], STAGE_BYTES);
                    tma_load_2d(a_dst + A_BYTES, &tmB, g * BK, n0, &full_bar[s]);
                }
                tma_load_2d(a_dst, &tmA, sub * BK, m0 + p.tap_shift[tap], &full_bar[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_f16(0, BM, BN);
            for (int kc = 0; kc < p.nk; ++kc) {
                const int s = kc % STAGES;
                const uint32_t ph = (uint32_t)(kc / STAGES) & 1u;
                if (!mbar_wait(&full_bar[s], ph, abortp, p.status, 2)) break;
                tc_fence_after();
                const uint32_t a_addr = base + s * STAGE_BYTES;
                const uint64_t adesc = smem_desc_sw128(a_addr);
                const uint64_t bdesc = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
                for (int k = 0; k < BK / 16; ++k)       // 32 bytes further along the swizzled row per K step
                    mma_f16_ss(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, (kc | k) != 0);
                mma_commit(&empty_bar[s]);
            }
            mma_commit(&accum_bar);
        }
    } else {
        // epilogue warps 2..5: warp w may touch TMEM lanes [32*(w%4), 32*(w%4)+32)
        const int q = warp & 3;
        const int r = q * 32 + lane;                    // row of the tile = TMEM lane
        const bool ok = mbar_wait_warp(&accum_bar, 0, abortp, p.status, 3);
        tc_fence_after();
        if (ok) {
            const long m = (long)m0 + r;
            const float inv = *p.inv_scale;
            {
                // The accumulator arrives one row per thread; a row-per-thread store would touch 32
                // lines per instruction.  Each warp turns its 32x32 block through shared memory (the
                // pipeline stages are free by now) so that eight lanes write one full 128-byte line.
                float* stage = reinterpret_cast<float*>(tiles) + (warp - 2) * (32 * 36);
                float* dst = p.out_f32 + blockIdx.z * p.split_stride + (size_t)(m0 + q * 32) * p.ldo + n0;
                const int rl = lane >> 3, c4 = (lane & 7) * 4;
#pragma unroll
                for (int c = 0; c < BN; c += 32) {
                    uint32_t v[32];
                    tmem_ld_32x32(tmem_d + ((uint32_t)(q * 32) << 16) + c, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<float4*>(stage + lane * 36 + j) =
                            make_float4(__uint_as_float(v[j]) * inv, __uint_as_float(v[j + 1]) * inv,
                                        __uint_as_float(v[j + 2]) * inv, __uint_as_float(v[j + 3]) * inv);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int rr = 4 * i + rl;
                        const float4 val = *reinterpret_cast<const float4*>(stage + rr * 36 + c4);
                        if (m0 + q * 32 + rr < p.n_env) *reinterpret_cast<float4*>(dst + (size_t)rr * p.ldo + c + c4) = val;
                    }
                    __syncwarp();
                }
            }
        }
    }
    if (*abortp) {                                      // give copies still in flight time to land
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_d, TMEM_COLS);
}


// ---- FC for small batches with the weights resident: one CTA per (column tile, K range) and slot of row tiles.
// A CTA asks for its whole weight slice (nk chunks of 128 x 64) before it waits for the previous kernel; a CTA of
// this kernel cannot start before the previous kernel's CTA has left its SM, but the hand-over from the last of
// those to the release of the wait (about 1.4 us) is enough for most of the slice.  After the wait only
// activations cross the SM's L2 port: 112 KB per row tile instead of 224 KB.  Used while every CTA has one row
// tile (n <= 640 for 4 x 84 x 84 frames: 31.0 against 31.5 us per step at n = 256, 51.2 against 52.7 us for 512
// football frames); with two tiles per CTA it only equals the kernel above (one CTA per SM streams less from L2
// than two do).  K ranges, the order inside them and the partial planes are those of the kernel above: the same
// bits.
constexpr int FCB_STAGES = 5;                   // activation chunks in flight (16 KiB each)
constexpr int FCB_MAX_NK = 7;                   // weight chunks a CTA can keep: 7 x 16 KiB
constexpr int FCB_MAX_TILES = 1;                // row tiles of a CTA (accumulators of 128 columns)
constexpr int FCB_STAGE_FLOATS = 4 * 32 * 36;   // the epilogue warps' transposing buffers

struct FcbParams {
    int nk;                             // K chunks of one range
    int n_env;                          // valid rows
    int m_tiles;                        // row tiles of the batch
    const float* inv_scale;
    float* out_f32;                     // partial planes [range][rows][512]
    size_t split_stride;
    int* status;
};

__global__ void __launch_bounds__(192)
fc_resident_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const FcbParams p)
{
    constexpr int BN = 128;
    constexpr int B_BYTES = BN * BK * 2;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t b_full[FCB_MAX_NK], a_full[FCB_STAGES], a_empty[FCB_STAGES], acc_full[FCB_MAX_TILES];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    uint8_t* sm_a = sm + FCB_MAX_NK * B_BYTES;
    const uint32_t a_base = base + FCB_MAX_NK * B_BYTES;
    float* sm_stage = reinterpret_cast<float*>(sm_a + FCB_STAGES * A_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * BN, range = blockIdx.y, slot = blockIdx.z, slots = gridDim.z;
    const int my_tiles = slot < p.m_tiles ? (p.m_tiles - slot + slots - 1) / slots : 0;   // <= FCB_MAX_TILES (launcher)
    volatile int* abortp = &abort_flag;

    if (threadIdx.x == 0) {
        for (int i = 0; i < FCB_MAX_NK; ++i) mbar_init(&b_full[i], 1);
        for (int i = 0; i < FCB_STAGES; ++i) { mbar_init(&a_full[i], 1); mbar_init(&a_empty[i], 1); }
        for (int i = 0; i < FCB_MAX_TILES; ++i) mbar_init(&acc_full[i], 1);
        abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (warp == 1) tmem_alloc(&tmem_base_slot, FCB_MAX_TILES * BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_slot;
    if (warp == 0 && lane == 0) {                        // the weights do not depend on the previous kernel
        for (int kc = 0; kc < p.nk; ++kc) {
            mbar_arrive_expect_tx(&b_full[kc], B_BYTES);
            tma_load_2d(sm + kc * B_BYTES, &tmB, (range * p.nk + kc) * BK, n0, &b_full[kc]);
        }
    }
    pdl_wait();
    pdl_trigger();

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            for (int t = 0; t < my_tiles; ++t) {
                const int m0 = (slot + t * slots) * BM;
                for (int kc = 0; kc < p.nk; ++kc, ++it) {
                    const int s = it % FCB_STAGES;
                    if (!mbar_wait(&a_empty[s], (((uint32_t)(it / FCB_STAGES)) & 1u) ^ 1u, abortp, p.status, 71)) { t = my_tiles; break; }
                    mbar_arrive_expect_tx(&a_full[s], A_BYTES);
                    tma_load_2d(sm_a + s * A_BYTES, &tmA, (range * p.nk + kc) * BK, m0, &a_full[s]);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_f16(0, BM, BN);
            int it = 0;
            bool alive = true;
            for (int t = 0; alive && t < my_tiles; ++t) {
                for (int kc = 0; kc < p.nk; ++kc, ++it) {
                    const int s = it % FCB_STAGES;
                    if (t == 0 && !mbar_wait(&b_full[kc], 0, abortp, p.status, 72)) { alive = false; break; }
                    if (!mbar_wait(&a_full[s], ((uint32_t)(it / FCB_STAGES)) & 1u, abortp, p.status, 73)) { alive = false; break; }
                    tc_fence_after();
                    const uint64_t adesc = smem_desc_sw128(a_base + s * A_BYTES);
                    const uint64_t bdesc = smem_desc_sw128(base + kc * B_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        mma_f16_ss(tmem_d + t * BN, adesc + 2 * k, bdesc + 2 * k, idesc, (kc | k) != 0);
                    mma_commit(&a_empty[s]);
                }
                if (alive) mma_commit(&acc_full[t]);
            }
        }
    } else {
        // epilogue warps 2..5: warp w may touch TMEM lanes [32*(w%4), 32*(w%4)+32)
        const int q = warp & 3;
        const float inv = *p.inv_scale;
        float* stage = sm_stage + (warp - 2) * (32 * 36);
        const int rl = lane >> 3, c4 = (lane & 7) * 4;
        for (int t = 0; t < my_tiles; ++t) {
            if (!mbar_wait_warp(&acc_full[t], 0, abortp, p.status, 74)) break;
            tc_fence_after();
            const int m0 = (slot + t * slots) * BM;
            // one row per thread arrives; each warp turns its 32 x 32 blocks through shared memory so that eight
            // lanes write one full 128-byte line
            float* dst = p.out_f32 + range * p.split_stride + (size_t)(m0 + q * 32) * 512 + n0;
#pragma unroll
            for (int c = 0; c < BN; c += 32) {
                uint32_t v[32];
                tmem_ld_32x32(tmem_d + ((uint32_t)(q * 32) << 16) + t * BN + c, v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    *reinterpret_cast<float4*>(stage + lane * 36 + j) =
                        make_float4(__uint_as_float(v[j]) * inv, __uint_as_float(v[j + 1]) * inv,
                                    __uint_as_float(v[j + 2]) * inv, __uint_as_float(v[j + 3]) * inv);
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + rl;
                    const float4 val = *reinterpret_cast<const float4*>(stage + rr * 36 + c4);
                    if (m0 + q * 32 + rr < p.n_env) *reinterpret_cast<float4*>(dst + (size_t)rr * 512 + c + c4) = val;
                }
                __syncwarp();
            }
        }
    }
    if (*abortp) {                                      // give copies still in flight time to land
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_d, FCB_MAX_TILES * BN);
}

// ---- FC for large batches: all K ranges of a tile in one CTA -----------------------------------------
// The FC result is defined as  h = relu(bias + p_0 + p_1 + ... + p_{S-1}),  p_s = inv * (sum over the K chunks of
// range s, accumulated in tensor memory in chunk order), the p_s added in index order in fp32.  Small batches
// spread the S ranges over S CTAs (gemm_tc_kernel writes the p_s, the heads kernel adds them), which fills the
// SMs.  Once there are enough 128 x 128 tiles to fill them anyway, one CTA runs the S ranges of its tile back to
// back, alternating between two accumulators, and its epilogue warps keep the running sum in registers: the same
// operations in the same order (explicitly rounded multiplies and adds, no fused forms), hence the same bits, but
// the hidden layer leaves the chip once (2 KB per observation instead of S x 2 KB) and the copy pipeline never
// drains between ranges.
constexpr int FCL_STAGES = 6;
constexpr int FCL_THREADS = 320;          // warp 0 copies, warp 1 issues, warps 2..9 epilogue (two per lane quarter, 64 columns each)

struct FclParams {
    int splits, cps;                      // K ranges and chunks per range
    int n;                                // valid rows
    const float* bias;                    // [512]
    const float* inv_scale;
    float* h;                             // [n][512]
    int* status;
};

__global__ void __launch_bounds__(FCL_THREADS)
fc_ranges_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const FclParams p)
{
    constexpr int BN = 128;
    constexpr int B_BYTES = BN * BK * 2;
    constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t full_bar[FCL_STAGES], empty_bar[FCL_STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ float s_bias[BN];

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* tiles = smem_raw + (base - smem_u32(smem_raw));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    volatile int* abortp = &abort_flag;
    const int total_chunks = p.splits * p.cps;

    if (threadIdx.x == 0) {
        for (int s = 0; s < FCL_STAGES; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 8); }
        abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmB);
    }
    if (threadIdx.x >= 64 && threadIdx.x < 64 + BN) s_bias[threadIdx.x - 64] = p.bias[n0 + threadIdx.x - 64];
    if (warp == 1) tmem_alloc(&tmem_base_slot, 2 * BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_base_slot;
    pdl_wait();
    pdl_trigger();

    if (warp == 0) {
        if (lane == 0) {
            for (int kc = 0; kc < total_chunks; ++kc) {
                const int s = kc % FCL_STAGES;
                const uint32_t ph = (uint32_t)(kc / FCL_STAGES) & 1u;
                if (!mbar_wait(&empty_bar[s], ph ^ 1u, abortp, p.status, 51)) break;
                uint8_t* a_dst = tiles + s * STAGE_BYTES;
                mbar_arrive_expect_tx(&full_bar[s], STAGE_BYTES);
                tma_load_2d(a_dst, &tmA, kc * BK, m0, &full_bar[s]);
                tma_load_2d(a_dst + A_BYTES, &tmB, kc * BK, n0, &full_bar[s]);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc_f16(0, BM, BN);
            int kc = 0;
            bool alive = true;
            for (int sp = 0; alive && sp < p.splits; ++sp) {
                const int acc = sp & 1;
                if (!mbar_wait(&acc_empty[acc], (((uint32_t)(sp >> 1)) & 1u) ^ 1u, abortp, p.status, 52)) break;
                tc_fence_after();
                for (int c = 0; c < p.cps; ++c, ++kc) {
                    const int s = kc % FCL_STAGES;
                    if (!mbar_wait(&full_bar[s], (uint32_t)(kc / FCL_STAGES) & 1u, abortp, p.status, 53)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = base + s * STAGE_BYTES;
                    const uint64_t adesc = smem_desc_sw128(a_addr), bdesc = smem_desc_sw128(a_addr + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)
                        mma_f16_ss(tmem_d + acc * BN, adesc + 2 * k, bdesc + 2 * k, idesc, (c | k) != 0);
                    mma_commit(&empty_bar[s]);
                }
                if (alive) mma_commit(&acc_full[acc]);
            }
        }
    } else {
        // epilogue warps 2..9: lane quarter warp % 4, columns [64 half, 64 half + 64) of the tile
        const int q = warp & 3, half = (warp - 2) >> 2;
        const float inv = *p.inv_scale;
        float sum[64];
        bool ok = true;
        for (int sp = 0; ok && sp < p.splits; ++sp) {
            const int acc = sp & 1;
            ok = mbar_wait_warp(&acc_full[acc], ((uint32_t)(sp >> 1)) & 1u, abortp, p.status, 54);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_d + acc * BN + half * 64 + ((uint32_t)(q * 32) << 16);
#pragma unroll
            for (int c = 0; c < 64; c += 32) {
                uint32_t v[32];
                tmem_ld_32x32(taddr + c, v);
                tmem_ld_wait();
                if (c == 32) {                            // the accumulator is in registers: hand it back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&acc_empty[acc]);
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float t = __fmul_rn(__uint_as_float(v[j]), inv);           // p_s, as the split kernel stores it
                    sum[c + j] = sp == 0 ? t : __fadd_rn(sum[c + j], t);              // added in index order, as the heads kernel does
                }
            }
        }
        if (ok) {
            // bias, ReLU, and the block turned through shared memory (the pipeline stages are free by now) so that
            // eight lanes write one full 128-byte line
            float* stage = reinterpret_cast<float*>(tiles) + (warp - 2) * (32 * 36);
            float* dst = p.h + (size_t)(m0 + q * 32) * 512 + n0 + half * 64;
            const int rl = lane >> 3, c4 = (lane & 7) * 4;
#pragma unroll
            for (int c = 0; c < 64; c += 32) {
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    *reinterpret_cast<float4*>(stage + lane * 36 + j) =
                        make_float4(fmaxf(__fadd_rn(sum[c + j], s_bias[half * 64 + c + j]), 0.f),
                                    fmaxf(__fadd_rn(sum[c + j + 1], s_bias[half * 64 + c + j + 1]), 0.f),
                                    fmaxf(__fadd_rn(sum[c + j + 2], s_bias[half * 64 + c + j + 2]), 0.f),
                                    fmaxf(__fadd_rn(sum[c + j + 3], s_bias[half * 64 + c + j + 3]), 0.f));
                __syncwarp();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + rl;
                    const float4 val = *reinterpret_cast<const float4*>(stage + rr * 36 + c4);
                    if (m0 + q * 32 + rr < p.n) *reinterpret_cast<float4*>(dst + (size_t)rr * 512 + c + c4) = val;
                }
                __syncwarp();
            }
        }
    }
    if (*abortp) {                                      // give copies still in flight time to land
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000) { }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_d, 2 * BN);
}

// ---- weight scaling and packing ---------------------------------------------------------------
__global__ void absmax_kernel(const __nv_bfloat16* __restrict__ w, size_t n, unsigned* __restrict__ slot)
{
    unsigned m = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float a = fabsf(__bfloat162float(w[i]));
        if (a == a && a < INFINITY) m = max(m, __float_as_uint(a));     // finite magnitudes order like their bits
    }
    for (int k = 16; k > 0; k >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, k));
    if ((threadIdx.x & 31) == 0 && m) atomicMax(slot, m);
}
// scale = 2^(14 - floor(log2 max)): the largest weight lands in [2^14, 2^15)
__global__ void scales_kernel(const unsigned* __restrict__ slots, float* __restrict__ scale, float* __restrict__ inv,
                              float conv1_extra)
{
    const int l = threadIdx.x;
    if (l >= L_COUNT) return;
    const float mx = __uint_as_float(slots[l]);
    int e = 0;
    float s = 1.f;
    if (mx > 0.f) { frexpf(mx, &e); s = ldexpf(1.f, 15 - e); }        // mx = f * 2^e, f in [0.5, 1)
    scale[l] = s;
    inv[l] = (l == L_CONV1 ? conv1_extra : 1.f) / s;
}
__device__ __forceinline__ __half scaled_h(__nv_bfloat16 w, float s) { return __float2half_rn(__bfloat162float(w) * s); }

// conv2: Wp[o][(tap*2 + half)*64 + j], c' = half*64 + j = (uy*2+ux)*32 + c, tap = dy*2+dx,
//        value w2[o][c][2dy+uy][2dx+ux]
__global__ void pack_conv2_kernel(const __nv_bfloat16* __restrict__ w, __half* __restrict__ wp, const float* __restrict__ scale)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 64 * 512) return;
    const int o = i / 512, k = i % 512;
    const int tap = k / 128, cp = k % 128;
    const int dy = tap >> 1, dx = tap & 1, uy = (cp / 32) >> 1, ux = (cp / 32) & 1, c = cp % 32;
    wp[i] = scaled_h(w[((o * 32 + c) * 4 + (2 * dy + uy)) * 4 + (2 * dx + ux)], scale[L_CONV2]);
}
// conv3: Wp[o][(dy*3+dx)*64 + c] = w3[o][c][dy][dx]
__global__ void pack_conv3_kernel(const __nv_bfloat16* __restrict__ w, __half* __restrict__ wp, const float* __restrict__ scale)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 64 * 576) return;
    const int o = i / 576, k = i % 576;
    const int tap = k / 64, c = k % 64;
    wp[i] = scaled_h(w[(o * 64 + c) * 9 + tap], scale[L_CONV3]);
}
// FC: Wp[o][pix*64 + c] = wfc[o][c*P3 + pix]   (activations are stored pixel-major, channel-minor)
__global__ void pack_fc_kernel(const __nv_bfloat16* __restrict__ w, __half* __restrict__ wp, int P3, const float* __restrict__ scale)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int F = 64 * P3;
    if (i >= (size_t)512 * F) return;
    const int o = (int)(i / F), k = (int)(i % F);
    const int pix = k / 64, c = k % 64;
    wp[i] = scaled_h(w[(size_t)o * F + c * P3 + pix], scale[L_FC]);
}
__global__ void bf16_to_f32_kernel(const __nv_bfloat16* __restrict__ src, float* __restrict__ dst, size_t n)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = __bfloat162float(src[i]);
}

// ---- parity taps: internal layouts -> fp32 NCHW ----------------------------------------------------
__global__ void tap_rows_kernel(const __half* __restrict__ src, float* __restrict__ dst, int n, int Cc,
                                int Ho, int Wo, int s2d, int P_rows, int W_rows)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t total = (size_t)n * Cc * Ho * Wo;
    if (idx >= total) return;
    const int x = (int)(idx % Wo), y = (int)((idx / Wo) % Ho), c = (int)((idx / ((size_t)Wo * Ho)) % Cc);
    const size_t e = idx / ((size_t)Wo * Ho * Cc);
    size_t off;
    if (s2d) off = (e * P_rows + (size_t)(y >> 1) * W_rows + (x >> 1)) * (4 * Cc) + ((y & 1) * 2 + (x & 1)) * Cc + c;
    else off = (e * P_rows + (size_t)y * W_rows + x) * Cc + c;
    dst[idx] = __half2float(src[off]);
}

inline unsigned nblk(size_t total, int th) { return (unsigned)((total + th - 1) / th); }

template <int BN, int EPI>
hts_status launch_gemm(const CUtensorMap& a, const CUtensorMap& b, const GemmParams& p, dim3 grid, cudaStream_t s)
{
    constexpr int smem = STAGES * (A_BYTES + BN * BK * 2) + 1024;
    static bool attr_set_by_device[kDeviceSlots] = {};
    bool& attr_set = attr_set_by_device[device_slot()];
    if (!attr_set) {
        HTS_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        HTS_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
        attr_set = true;
    }
    HTS_CUDA(launch_pdl(gemm_tc_kernel<BN, EPI>, grid, dim3(192), (size_t)smem, s, a, b, p));
    note_launch();
    return HTS_OK;
}

hts_status launch_fc_resident(const CUtensorMap& a, const CUtensorMap& b, const FcbParams& p, int ranges, int slots,
                              cudaStream_t s)
{
    constexpr int smem = FCB_MAX_NK * 128 * BK * 2 + FCB_STAGES * A_BYTES + FCB_STAGE_FLOATS * 4 + 1024;
    static bool attr_set_by_device[kDeviceSlots] = {};
    bool& attr_set = attr_set_by_device[device_slot()];
    if (!attr_set) {
        HTS_CUDA(cudaFuncSetAttribute(fc_resident_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        HTS_CUDA(cudaFuncSetAttribute(fc_resident_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
        attr_set = true;
    }
    HTS_CUDA(launch_pdl(fc_resident_kernel, dim3(4, ranges, slots), dim3(192), (size_t)smem, s, a, b, p));
    note_launch();
    return HTS_OK;
}

}  // namespace

struct TcState {
    Geometry g;
    int max_batch;
    int H1s, W1s, P1s;          // space-to-depth(2) grid of the conv1 output
    int P2, P3;
    int splits, cps;            // FC split-K
    bool h_final = false;       // the last forward pass wrote the finished hidden layer (large-batch FC), not partials
    // packed weights
    Conv1Plan pl1;
    Conv1MapCache maps1;
    __half *w1p, *w2p, *w3p, *wfcp;
    float *b1, *b2, *b3, *bfc, *whead, *bhead;
    unsigned* absmax;           // [L_COUNT]
    float *scale, *inv_scale;   // [L_COUNT] each
    // workspace
    __half *a1s, *a2, *a3;
    float *hpart, *h;
    CUtensorMap mW1, mA2, mB2, mA3, mB3, mAfc, mBfc;
    int rows2, rows3;           // activation tile rows of conv2 / conv3
    int* status;
};

hts_status tc_check_geometry(const Geometry& g)
{
    Conv1Plan pl;
    if (!conv1_plan(g, &pl)) return HTS_ERR_SHAPE;
    const int rows2 = conv_res_tile_rows(pl.W1s + 1), rows3 = conv_res_tile_rows(2 * g.W2 + 2);
    if (rows2 > 256 || rows3 > 256) return HTS_ERR_SHAPE;                    // TMA box height
    if (conv_res_smem_bytes(4, 2, rows2) > 227 * 1024 || conv_res_smem_bytes(9, 1, rows3) > 227 * 1024) return HTS_ERR_SHAPE;
    if (g.F % BK) return HTS_ERR_SHAPE;
    // row arithmetic of the conv2 / conv3 epilogues: grids of at most 2048 pixels, at most 64 wide
    if (pl.P1s > 2048 || pl.W1s > 64 || g.H2 * g.W2 > 2048 || g.W2 > 64) return HTS_ERR_SHAPE;
    return HTS_OK;
}

hts_status tc_create(const Geometry& g, int max_batch, int* status, TcState** out,
                     bool (*alloc)(void* ctx, void** p, size_t bytes), void* alloc_ctx)
{
    TcState* t = new (std::nothrow) TcState();
    if (!t) return HTS_ERR_ALLOC;
    t->g = g; t->max_batch = max_batch; t->status = status;
    if (tc_check_geometry(g) != HTS_OK || !conv1_plan(g, &t->pl1)) { delete t; return HTS_ERR_SHAPE; }
    t->H1s = t->pl1.H1s; t->W1s = t->pl1.W1s; t->P1s = t->pl1.P1s;
    t->P2 = g.H2 * g.W2; t->P3 = g.H3 * g.W3;
    const int chunks = g.F / BK;
    t->splits = 1;
    for (int s = 8; s >= 1; --s) if (chunks % s == 0) { t->splits = s; break; }
    t->cps = chunks / t->splits;
    const size_t nb = (size_t)max_batch;
    auto A = [&](auto** p, size_t count) { return alloc(alloc_ctx, reinterpret_cast<void**>(p), count * sizeof(**p)); };
    bool ok = A(&t->w2p, (size_t)64 * 512) && A(&t->w3p, (size_t)64 * 576) && A(&t->wfcp, (size_t)512 * g.F) &&
              A(&t->w1p, (size_t)128 * 16 * g.C) && A(&t->b1, 32) && A(&t->b2, 64) && A(&t->b3, 64) && A(&t->bfc, 512) &&
              A(&t->whead, (size_t)(g.A + 1) * 512) && A(&t->bhead, (size_t)g.A + 1) &&
              A(&t->absmax, L_COUNT) && A(&t->scale, L_COUNT) && A(&t->inv_scale, L_COUNT) &&
              A(&t->a1s, nb * t->P1s * 128) && A(&t->a2, nb * t->P2 * 64) && A(&t->a3, nb * g.F) &&
              A(&t->hpart, (size_t)t->splits * nb * 512) && A(&t->h, nb * 512);
    if (!ok) { delete t; return HTS_ERR_ALLOC; }
    // cells of an odd-sized s2d border that conv1 never writes must hold finite numbers
    if (cudaMemset(t->a1s, 0, nb * t->P1s * 128 * 2) != cudaSuccess) { delete t; return cuda_fail(cudaGetLastError(), "cudaMemset"); }
    t->rows2 = conv_res_tile_rows(t->W1s + 1);
    t->rows3 = conv_res_tile_rows(2 * g.W2 + 2);
    if (t->rows2 > 256 || t->rows3 > 256) { delete t; return HTS_ERR_SHAPE; }
    ok = make_map(&t->mW1, t->w1p, 128, 16 * g.C, (uint64_t)32 * g.C, 64) &&
         make_map(&t->mA2, t->a1s, nb * t->P1s, 128, 256, t->rows2) && make_map(&t->mB2, t->w2p, 64, 512, 1024, 64) &&
         make_map(&t->mA3, t->a2, nb * t->P2, 64, 128, t->rows3) && make_map(&t->mB3, t->w3p, 64, 576, 1152, 64) &&
         make_map(&t->mAfc, t->a3, nb, g.F, (uint64_t)g.F * 2, BM) && make_map(&t->mBfc, t->wfcp, 512, g.F, (uint64_t)g.F * 2, 128);
    if (!ok) { delete t; return HTS_ERR_CUDA; }
    *out = t;
    return HTS_OK;
}

void tc_destroy(TcState* t) { delete t; }

hts_status tc_load_weights(TcState* t, const hts_weights& w, cudaStream_t s)
{
    const Geometry& g = t->g;
    auto bf = [](const void* p) { return static_cast<const __nv_bfloat16*>(p); };
    HTS_CUDA(cudaMemsetAsync(t->absmax, 0, L_COUNT * sizeof(unsigned), s));
    struct Mx { const void* p; size_t n; int l; };
    const Mx mx[] = {{w.conv1_w, (size_t)32 * g.C * 64, L_CONV1}, {w.conv2_w, (size_t)64 * 512, L_CONV2},
                     {w.conv3_w, (size_t)64 * 576, L_CONV3}, {w.fc_w, (size_t)512 * g.F, L_FC}};
    for (const Mx& m : mx) {
        absmax_kernel<<<64, 256, 0, s>>>(bf(m.p), m.n, t->absmax + m.l);
        HTS_LAUNCH_CHECK("absmax");
    }
    // conv1 feeds raw bytes as fp16 subnormals (b * 2^-24): its accumulator scale undoes that and the /255
    scales_kernel<<<1, 32, 0, s>>>(t->absmax, t->scale, t->inv_scale, 16777216.0f / 255.0f);
    HTS_LAUNCH_CHECK("scales");
    hts_status st1 = conv1_pack_weights(t->pl1, bf(w.conv1_w), t->w1p, t->scale + L_CONV1, s);
    if (st1 != HTS_OK) return st1;
    pack_conv2_kernel<<<nblk(64 * 512, 256), 256, 0, s>>>(bf(w.conv2_w), t->w2p, t->scale); HTS_LAUNCH_CHECK("pack_conv2");
    pack_conv3_kernel<<<nblk(64 * 576, 256), 256, 0, s>>>(bf(w.conv3_w), t->w3p, t->scale); HTS_LAUNCH_CHECK("pack_conv3");
    pack_fc_kernel<<<nblk((size_t)512 * g.F, 256), 256, 0, s>>>(bf(w.fc_w), t->wfcp, t->P3, t->scale); HTS_LAUNCH_CHECK("pack_fc");
    struct It { const void* p; float* q; size_t n; };
    const It items[] = {{w.conv1_b, t->b1, 32}, {w.conv2_b, t->b2, 64},
                        {w.conv3_b, t->b3, 64}, {w.fc_b, t->bfc, 512}, {w.pi_w, t->whead, (size_t)g.A * 512},
                        {w.v_w, t->whead + (size_t)g.A * 512, 512}, {w.pi_b, t->bhead, (size_t)g.A}, {w.v_b, t->bhead + g.A, 1}};
    for (const It& it : items) {
        bf16_to_f32_kernel<<<nblk(it.n, 256), 256, 0, s>>>(bf(it.p), it.q, it.n);
        HTS_LAUNCH_CHECK("bf16_to_f32");
    }
    return HTS_OK;
}

hts_status tc_forward(TcState* t, const uint8_t* obs, const Indexing& ix, int n, Profiler& prof, cudaStream_t s)
{
    const Geometry& g = t->g;
    prof.begin(K_CONV1, s);
    hts_status st = conv1_launch(t->pl1, t->mW1, t->maps1, obs, ix, n, t->b1, t->inv_scale + L_CONV1, t->a1s, t->status, s);
    if (st != HTS_OK) return st;
    prof.end(K_CONV1, s);

    // conv2: 2x2 taps on the s2d grid [H1s, W1s] with 128 channels -> [H2, W2] x 64
    ConvResParams c{};
    c.status = t->status; c.n_env = n;
    c.tap_shift[0] = 0; c.tap_shift[1] = 1; c.tap_shift[2] = t->W1s; c.tap_shift[3] = t->W1s + 1;
    c.tile_rows = t->rows2; c.total_rows = n * t->P1s;
    c.P_in = t->P1s; c.W_in = t->W1s; c.H_out = g.H2; c.W_out = g.W2; c.P_out = t->P2;
    c.bias = t->b2; c.out = t->a2; c.inv_scale = t->inv_scale + L_CONV2;
    prof.begin(K_CONV2, s);
    st = conv_res_launch<4, 2>(t->mA2, t->mB2, c, s);
    if (st != HTS_OK) return st;
    prof.end(K_CONV2, s);
    // conv3: 3x3 taps on [H2, W2] x 64 -> [H3, W3] x 64
    for (int dy = 0; dy < 3; ++dy) for (int dx = 0; dx < 3; ++dx) c.tap_shift[dy * 3 + dx] = dy * g.W2 + dx;
    c.tile_rows = t->rows3; c.total_rows = n * t->P2;
    c.P_in = t->P2; c.W_in = g.W2; c.H_out = g.H3; c.W_out = g.W3; c.P_out = t->P3;
    c.bias = t->b3; c.out = t->a3; c.inv_scale = t->inv_scale + L_CONV3;
    prof.begin(K_CONV3, s);
    st = conv_res_launch<9, 1>(t->mA3, t->mB3, c, s);
    if (st != HTS_OK) return st;
    prof.end(K_CONV3, s);
    GemmParams p{};
    p.status = t->status; p.n_env = n;
    // FC: [n, F] x [512, F]^T, K split across blockIdx.z
    p.taps = 1; p.cpt = g.F / BK; p.nk = t->cps; p.tap_shift[0] = 0;
    p.out_f32 = t->hpart; p.split_stride = (size_t)t->max_batch * 512; p.ldo = 512; p.inv_scale = t->inv_scale + L_FC;
    prof.begin(K_FC, s);
    // From 64 tiles on (n > 1920) one CTA per tile running all K ranges beats spreading the ranges over CTAs
    // (measured: 89 against 91 us per step at n = 2048, 139 against 166 at n = 4096, 254 against 298 at n = 8192;
    // at n = 1024 its 32 CTAs would each pull 1.6 MB through one SM's L2 port)
    t->h_final = (long)nblk(n, BM) * 4 >= 64;
    if (t->h_final) {
        constexpr int smem = FCL_STAGES * (A_BYTES + 128 * BK * 2) + 1024;
        static bool attr_set_by_device[kDeviceSlots] = {};
        bool& attr_set = attr_set_by_device[device_slot()];
        if (!attr_set) {
            HTS_CUDA(cudaFuncSetAttribute(fc_ranges_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            HTS_CUDA(cudaFuncSetAttribute(fc_ranges_kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
            attr_set = true;
        }
        const FclParams fp{t->splits, t->cps, n, t->bfc, t->inv_scale + L_FC, t->h, t->status};
        HTS_CUDA(launch_pdl(fc_ranges_kernel, dim3(nblk(n, BM), 4), dim3(FCL_THREADS), (size_t)smem, s, t->mAfc, t->mBfc, fp));
        note_launch();
    } else {
        // Weights resident per CTA when a K range is at most seven chunks and every CTA gets one row tile
        const int m_tiles = (int)nblk(n, BM);
        int slots = device_sm_count(device_slot()) / (4 * t->splits);
        if (slots > m_tiles) slots = m_tiles;
        if (t->cps <= FCB_MAX_NK && slots >= 1 && (m_tiles + slots - 1) / slots <= FCB_MAX_TILES) {
            const FcbParams fp{t->cps, n, m_tiles, t->inv_scale + L_FC, t->hpart, (size_t)t->max_batch * 512, t->status};
            st = launch_fc_resident(t->mAfc, t->mBfc, fp, t->splits, slots, s);
        } else
            st = launch_gemm<128, EPI_SPLITK>(t->mAfc, t->mBfc, p, dim3(nblk(n, BM), 4, t->splits), s);
        if (st != HTS_OK) return st;
    }
    prof.end(K_FC, s);
    return HTS_OK;
}

hts_status tc_heads(TcState* t, const int32_t* env_ids, const int32_t* t_per_env, int32_t tt, uint64_t seed, int n,
                    const Indexing& ix, int32_t* actions, float* logp, float* values, float* entropy, float* logits,
                    cudaStream_t s, const int32_t* given_actions)
{
    if (t->h_final)        // the FC kernel wrote relu(bias + sum of the K ranges) itself
        return launch_heads(t->h, 1, 0, nullptr, t->whead, t->bhead, t->g.A, env_ids, t_per_env, tt, seed, n, ix, t->status,
                            actions, logp, values, entropy, logits, nullptr, s, given_actions);
    return launch_heads(t->hpart, t->splits, (size_t)t->max_batch * 512, t->bfc, t->whead, t->bhead, t->g.A, env_ids,
                        t_per_env, tt, seed, n, ix, t->status, actions, logp, values, entropy, logits, t->h, s, given_actions);
}

hts_status tc_read_activation(TcState* t, int layer, int n, float* out, cudaStream_t s)
{
    const Geometry& g = t->g;
    if (layer == 4) {
        HTS_CUDA(cudaMemcpyAsync(out, t->h, (size_t)n * 512 * sizeof(float), cudaMemcpyDeviceToDevice, s));
        return HTS_OK;
    }
    if (layer == 1)
        tap_rows_kernel<<<nblk((size_t)n * 32 * g.H1 * g.W1, 256), 256, 0, s>>>(t->a1s, out, n, 32, g.H1, g.W1, 1, t->P1s, t->W1s);
    else if (layer == 2)
        tap_rows_kernel<<<nblk((size_t)n * 64 * g.H2 * g.W2, 256), 256, 0, s>>>(t->a2, out, n, 64, g.H2, g.W2, 0, t->P2, g.W2);
    else
        tap_rows_kernel<<<nblk((size_t)n * 64 * g.H3 * g.W3, 256), 256, 0, s>>>(t->a3, out, n, 64, g.H3, g.W3, 0, t->P3, g.W3);
    HTS_LAUNCH_CHECK("tap_rows_kernel");
    return HTS_OK;
}

}  // namespace hts
