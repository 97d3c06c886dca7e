// conv2 / conv3 of the policy-value network as a persistent tcgen05 kernel.
//
// A stride-1 convolution on the flat pixel grid is a sum over filter taps of row-shifted GEMMs
//     D[m, o] = sum_tap sum_c X[m + dy*W_in + dx, c] * W[o, tap, c].
// Each CTA keeps the whole packed filter in shared memory and walks over 128-row tiles of the
// activation matrix.  For a tile it loads rows [m0, m0 + 128 + largest shift) ONCE (one TMA box
// per 64-channel plane, 128-byte swizzle) and every tap reads the same tile through a shared-
// memory descriptor whose start address is moved by `shift` rows: the swizzle is a function of
// the address bits, so a start that is a multiple of 128 bytes keeps the pattern intact.
// Activation tiles sit in a ring; four accumulators live in tensor memory.  Two warps issue MMAs,
// warp g for the CTA's tiles g, g+2, ... into accumulators g and g+2 in turn, and each accumulator
// has its own four epilogue warps, so copies, MMAs and epilogues of different tiles overlap.
// Measured: a 128x64x16 MMA occupies the tensor core for 48 clocks (128 + 64 operand rows of 32
// bytes from shared memory at 128 bytes per clock), one thread issues one every 70 to 100 clocks,
// and one epilogue takes about 2300 clocks per tile; two issuers keep the tensor core busy and
// four epilogue groups keep the issuers from waiting for an accumulator.  Rows whose pixel lies
// outside the output extent are computed and dropped by the epilogue.
#include "conv_res_tc.cuh"
#include "tc_ptx.cuh"

namespace hts {
using namespace tc;

namespace {

constexpr int kAcc = 4;                         // accumulators in tensor memory (64 columns each)
constexpr int kThreads = 128 + kAcc * 128;      // warp 0 copies, warps 1 and 2 issue MMAs, warp 3 idle, then four epilogue warps per accumulator
constexpr int kChunkBytes = 64 * 128;           // one filter K chunk: 64 output channels x 128 bytes

// 256-bit store of eight packed half2 (one 32-byte sector)
__device__ __forceinline__ void st_global_v8(void* ptr, const uint32_t (&v)[8])
{
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"l"(ptr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}

template <int TAPS, int CPT, int NST>
__global__ void __launch_bounds__(kThreads)
conv_res_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, const ConvResParams p)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t w_bar, a_full[NST], a_empty[NST], d_full[kAcc], d_empty[kAcc];
    __shared__ float s_bias[64];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    volatile int* abortp = &abort_flag;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    constexpr int w_bytes = TAPS * CPT * kChunkBytes;
    const int plane_bytes = p.tile_rows * 128;
    const int a_bytes = CPT * plane_bytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles = (p.total_rows + 127) / 128;

    if (threadIdx.x == 0) {
        mbar_init(&w_bar, 1);
        for (int b = 0; b < NST; ++b) { mbar_init(&a_full[b], 1); mbar_init(&a_empty[b], 1); }
        for (int b = 0; b < kAcc; ++b) { mbar_init(&d_full[b], 1); mbar_init(&d_empty[b], 128); }
        abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmA);
        tma_prefetch_desc(&tmW);
    }
    if (threadIdx.x >= 64 && threadIdx.x < 128) s_bias[threadIdx.x - 64] = p.bias[threadIdx.x - 64];
    if (warp == 1) tmem_alloc(&tmem_slot, kAcc * 64);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_slot;

    if (warp == 0 && lane == 0) {                        // the filter does not depend on the previous kernel
        mbar_arrive_expect_tx(&w_bar, w_bytes);
        for (int g = 0; g < TAPS * CPT; ++g) tma_load_2d(sm + g * kChunkBytes, &tmW, g * 64, 0, &w_bar);
    }
    pdl_wait();
    pdl_trigger();

    if (warp == 0) {
        if (lane == 0) {
            int it = 0;
            for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++it) {
                const int b = it % NST;
                if (!mbar_wait(&a_empty[b], (((uint32_t)(it / NST)) & 1u) ^ 1u, abortp, p.status, 21)) break;
                uint8_t* dst = sm + w_bytes + b * a_bytes;
                mbar_arrive_expect_tx(&a_full[b], (uint32_t)a_bytes);
                for (int pl = 0; pl < CPT; ++pl) tma_load_2d(dst + pl * plane_bytes, &tmA, pl * 64, tile * 128, &a_full[b]);
            }
        }
    } else if (warp <= 2) {
        if (lane == 0) {
            // issuing thread g: tiles g, g+2, ... of this CTA, accumulator it % 4 (g, g+2, g, ...)
            const int g = warp - 1;
            constexpr uint32_t idesc = instr_desc_f16(0, 128, 64);
            bool alive = mbar_wait(&w_bar, 0, abortp, p.status, 22);
            int it = g;
            for (int tile = blockIdx.x + g * gridDim.x; alive && tile < tiles; tile += 2 * gridDim.x, it += 2) {
                const int b = it % NST, db = it % kAcc;
                if (!mbar_wait(&a_full[b], ((uint32_t)(it / NST)) & 1u, abortp, p.status, 23)) break;
                if (!mbar_wait(&d_empty[db], (((uint32_t)(it / kAcc)) & 1u) ^ 1u, abortp, p.status, 24)) break;
                tc_fence_after();
                const uint32_t a_addr = base + w_bytes + b * a_bytes;
                const uint32_t d_addr = tmem_d + db * 64;
#pragma unroll
                for (int tap = 0; tap < TAPS; ++tap) {
#pragma unroll
                    for (int pl = 0; pl < CPT; ++pl) {
                        const uint64_t adesc = smem_desc_sw128(a_addr + pl * plane_bytes + p.tap_shift[tap] * 128);
                        const uint64_t bdesc = smem_desc_sw128(base + (tap * CPT + pl) * kChunkBytes);
#pragma unroll
                        for (int k = 0; k < 4; ++k) mma_f16_ss(d_addr, adesc + 2 * k, bdesc + 2 * k, idesc, (tap | pl | k) != 0);
                    }
                }
                mma_commit(&a_empty[b]);
                mma_commit(&d_full[db]);
            }
        }
    } else if (warp >= 4) {
        // four warps per accumulator: group j drains accumulator j, i.e. tiles j, j+4, ... of the CTA
        const int grp = (warp - 4) >> 2;
        const int q = warp & 3;                         // TMEM lane quarter this warp may read
        const int r = q * 32 + lane;
        const float inv = *p.inv_scale;
        int it = grp;
        // Row m of the flat grid = (env, y, x).  The row of this thread advances by the same amount from one of its
        // tiles to the next, so (env, pix) are carried along with one conditional subtraction per tile instead of
        // two divisions, and y = pix / W_in is a multiply: with pix < 2048 and W_in <= 64,
        // (pix * ceil(2^20 / W_in)) >> 20 is exact and the product fits 32 bits (the launcher checks both bounds).
        const uint32_t first = (uint32_t)(blockIdx.x + grp * gridDim.x) * 128u + (uint32_t)r;
        const uint32_t stride = (uint32_t)kAcc * gridDim.x * 128u;
        const int d_env = (int)(stride / (uint32_t)p.P_in), d_pix = (int)(stride - (uint32_t)d_env * (uint32_t)p.P_in);
        int env = (int)(first / (uint32_t)p.P_in), pix = (int)(first - (uint32_t)env * (uint32_t)p.P_in);
        const uint32_t w_magic = ((1u << 20) + (uint32_t)p.W_in - 1u) / (uint32_t)p.W_in;
        for (int tile = blockIdx.x + grp * gridDim.x; tile < tiles; tile += kAcc * gridDim.x, it += kAcc) {
            if (!mbar_wait_warp(&d_full[grp], ((uint32_t)(it / kAcc)) & 1u, abortp, p.status, 25)) break;
            tc_fence_after();
            const int y = (int)(((uint32_t)pix * w_magic) >> 20), x = pix - y * p.W_in;
            const bool valid = env < p.n_env && y < p.H_out && x < p.W_out;
            __half* dst = p.out + ((size_t)env * p.P_out + (size_t)y * p.W_out + x) * 64;
            env += d_env; pix += d_pix;
            if (pix >= p.P_in) { pix -= p.P_in; ++env; }
            uint32_t v0[32], v1[32];
            const uint32_t taddr = tmem_d + grp * 64 + ((uint32_t)(q * 32) << 16);
            tmem_ld_32x32(taddr, v0);
            tmem_ld_32x32(taddr + 32, v1);
            tmem_ld_wait();
            tc_fence_before();
            mbar_arrive(&d_empty[grp]);                 // accumulator is in registers: hand it back
            if (valid) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
#pragma unroll
                    for (int j = 0; j < 32; j += 16) {
                        uint32_t pk[8];
#pragma unroll
                        for (int h = 0; h < 8; ++h) {
                            const int c = j + 2 * h;
                            float x0 = __uint_as_float(half ? v1[c] : v0[c]);
                            float x1 = __uint_as_float(half ? v1[c + 1] : v0[c + 1]);
                            fma2(x0, x1, inv, s_bias[half * 32 + c], s_bias[half * 32 + c + 1]);
                            pk[h] = relu_pack_h2(x0, x1);     // ReLU, round to fp16, clamp at the largest finite value
                        }
                        st_global_v8(dst + half * 32 + j, pk);
                    }
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
    if (warp == 1) tmem_dealloc(tmem_d, kAcc * 64);
}

}  // namespace

template <int TAPS, int CPT>
hts_status conv_res_launch(const CUtensorMap& act_map, const CUtensorMap& weight_map, const ConvResParams& p,
                           cudaStream_t s)
{
    const int dev = device_slot();
    const int sm_count = device_sm_count(dev);
    static int smem_set_by_device[kDeviceSlots] = {};
    int& smem_set = smem_set_by_device[dev];
    constexpr int NST = CPT == 2 ? 4 : 6;        // activation tiles in the ring: two being multiplied, the rest in flight
    const int smem = conv_res_smem_bytes(TAPS, CPT, p.tile_rows);
    if (smem > 227 * 1024) return HTS_ERR_SHAPE;
    if (p.P_in < 1 || p.P_in > 2048 || p.W_in < 1 || p.W_in > 64) return HTS_ERR_SHAPE;   // the epilogue's row arithmetic
    if (smem > smem_set) {
        HTS_CUDA(cudaFuncSetAttribute(conv_res_kernel<TAPS, CPT, NST>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        HTS_CUDA(cudaFuncSetAttribute(conv_res_kernel<TAPS, CPT, NST>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
        smem_set = smem;
    }
    const int tiles = (p.total_rows + 127) / 128;
    const int grid = tiles < sm_count ? tiles : sm_count;
    HTS_CUDA(launch_pdl(conv_res_kernel<TAPS, CPT, NST>, dim3(grid), dim3(kThreads), (size_t)smem, s, act_map, weight_map, p));
    note_launch();
    return HTS_OK;
}

template hts_status conv_res_launch<4, 2>(const CUtensorMap&, const CUtensorMap&, const ConvResParams&, cudaStream_t);
template hts_status conv_res_launch<9, 1>(const CUtensorMap&, const CUtensorMap&, const ConvResParams&, cudaStream_t);

}  // namespace hts
