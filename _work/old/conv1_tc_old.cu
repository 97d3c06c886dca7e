// conv1 (8x8 / 4, C -> 32) of the policy-value network, fused from raw frames to fp16 output.
//
// An 8x8 stride-4 convolution is a 2x2 stride-1 convolution on the space-to-depth(4) image
// (channels c' = c*16 + uy*4 + ux).  One work unit is a band of R output rows of one
// environment: its (R+1) x Ws space-to-depth pixels become the rows of an fp16 tile in shared
// memory (128-byte swizzled rows of 64 channels, one plane per 64 channels), and each filter tap
// (dy,dx) is the same tile read from a start address shifted by dy*Ws+dx rows.  Output row
// m = y*Ws + x of the 128-row MMA tile is pixel (y, x) of the band; x = Ws-1 and rows past the
// band are computed and thrown away.
//
// A CTA is a pipeline of four roles over its units: one thread issues bulk copies
// (cp.async.bulk, one per channel) of the band's uint8 rows into a ring of staged bands; eight
// warps turn a staged band into fp16 (a zero-extended byte is the fp16 subnormal b * 2^-24, exact;
// 2^24 / 255 is folded into the accumulator scale) and write a ring of 64-channel planes (three or
// four); two threads issue the tcgen05.mma (128 x 32 x 16), thread h the 8 * planes of filter row
// dy = h into its own accumulator in tensor memory; four more warps read the two accumulators
// back, add them, apply scale, bias and ReLU and store fp16 in the layout conv2 reads.
// Wide inputs (many planes) fall back to one tile buffer and two staged bands to fit.
#include "conv1_tc.cuh"
#include "tc_ptx.cuh"

namespace hts {
using namespace tc;

namespace {

constexpr int kThreads = 480;                   // warp 0 copies, warps 1 and 14 MMA issue, warps 2..9 convert, warps 10..13 epilogue
constexpr int kConverters = 256;
constexpr int kMaxPlanes = 4;
constexpr int kMaxU8 = 6;
constexpr int kWorkers = 128;
constexpr int kChunkBytes = 32 * 64 * 2;        // one weight K chunk: 32 rows x 128 bytes

struct Conv1Params {
    Conv1Plan pl;
    const uint8_t* obs;
    const int32_t* slots;   // frame of each row in obs, or nullptr: row e is frame e
    int pool;               // frames in obs when slots are given
    int n;
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

template <int CPT>
__global__ void __launch_bounds__(kThreads)
conv1_tc_kernel(const __grid_constant__ CUtensorMap tmW, const Conv1Params p)
{
    const Conv1Plan& pl = p.pl;
    static_assert(CPT == 1 || CPT == 2 || CPT == 4, "planes per tap");
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t w_bar, u8_full[kMaxU8], u8_empty[kMaxU8], plane_full[kMaxPlanes], plane_empty[kMaxPlanes], d_full[2], d_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ float s_bias[32];
    volatile int* abortp = &abort_flag;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    const int plane_bytes = pl.tile_rows * 128;
    const int w_bytes = 4 * CPT * kChunkBytes;
    const int NP = pl.plane_bufs, NU = pl.u8_stages;
    // layout: [weights][ring of NP fp16 planes (64 channels of a band each)][u8 stages: NU]
    uint8_t* s_w = sm;
    uint8_t* s_tile = sm + w_bytes;
    uint8_t* s_u8 = s_tile + NP * plane_bytes;
    const uint32_t a_w = base, a_tile = base + w_bytes;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int units = p.n * pl.bands;
    const int band_in_rows = 4 * (pl.R + 1);

    if (threadIdx.x == 0) {
        mbar_init(&w_bar, 1);
        for (int s = 0; s < kMaxU8; ++s) { mbar_init(&u8_full[s], 1); mbar_init(&u8_empty[s], kConverters); }
        for (int s = 0; s < kMaxPlanes; ++s) { mbar_init(&plane_full[s], kConverters); mbar_init(&plane_empty[s], 2); }
        for (int s = 0; s < 2; ++s) { mbar_init(&d_full[s], 2); mbar_init(&d_empty[s], kWorkers); }
        abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmW);
    }
    if (threadIdx.x >= 64 && threadIdx.x < 96) s_bias[threadIdx.x - 64] = p.bias[threadIdx.x - 64];
    if (warp == 1) tmem_alloc(&tmem_slot, 128);           // two buffers x two accumulators (dy = 0, 1) x 32 columns
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_d = tmem_slot;
    pdl_wait();                                          // frames and the output buffer belong to earlier kernels until here
    pdl_trigger();

    if (warp == 0) {
        // ---- copies: weights once, then each unit's uint8 rows, NU units ahead
        if (lane == 0) {
            mbar_arrive_expect_tx(&w_bar, (uint32_t)w_bytes);
            for (int g = 0; g < 4 * CPT; ++g) tma_load_2d(s_w + g * kChunkBytes, &tmW, g * 64, 0, &w_bar);
            int s = 0;                                    // staged band and the parity of its current use: a ring
            uint32_t sph = 0;                             // walked with counters (NU is not a compile-time constant)
            for (int u = blockIdx.x; u < units; u += gridDim.x) {
                if (!mbar_wait(&u8_empty[s], sph ^ 1u, abortp, p.status, 11)) break;
                const int env = u / pl.bands, band = u - env * pl.bands;
                const int r0 = 4 * band * pl.R;
                int rows = pl.H - r0; rows = rows > band_in_rows ? band_in_rows : rows;
                const uint32_t bytes = (uint32_t)(rows * pl.W);
                mbar_arrive_expect_tx(&u8_full[s], bytes * pl.C);
                const uint8_t* src = p.obs + (frame_of(p, env) * pl.C * pl.H + r0) * pl.W;
                uint8_t* dst = s_u8 + s * pl.u8_stage_bytes;
                for (int c = 0; c < pl.C; ++c)
                    bulk_load(dst + c * band_in_rows * pl.W, src + (size_t)c * pl.H * pl.W, bytes, &u8_full[s]);
                if (++s == NU) { s = 0; sph ^= 1u; }
            }
        }
    } else if (warp == 1 || warp == 14) {
        // ---- MMA issue: thread h takes the two taps of filter row dy = h of every plane into its own
        //      accumulator (one thread issues an MMA every 60 to 130 clocks, the tensor core needs 40)
        if (lane == 0) {
            const int h = warp == 1 ? 0 : 1;
            constexpr uint32_t idesc = instr_desc_f16(0, 128, 32);
            bool alive = mbar_wait(&w_bar, 0, abortp, p.status, 12);
            int it = 0, pb = 0;
            uint32_t pph = 0;
            for (int u = blockIdx.x; alive && u < units; u += gridDim.x, ++it) {
                const int db = it & 1;
                if (!mbar_wait(&d_empty[db], (((uint32_t)it >> 1) & 1u) ^ 1u, abortp, p.status, 16)) break;
                const uint32_t d_addr = tmem_d + db * 64 + h * 32;
                uint32_t acc = 0;
#pragma unroll
                for (int pln = 0; pln < CPT; ++pln) {     // planes arrive one by one: MMAs of plane k overlap the conversion of k+1
                    if (!mbar_wait(&plane_full[pb], pph, abortp, p.status, 13)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t p_addr = a_tile + pb * plane_bytes;
#pragma unroll
                    for (int dx = 0; dx < 2; ++dx) {
                        const int tap = 2 * h + dx;
                        const int shift = h * pl.Ws + dx;
                        const uint64_t adesc = smem_desc_sw128(p_addr + shift * 128);
                        const uint64_t bdesc = smem_desc_sw128(a_w + (tap * CPT + pln) * kChunkBytes);
#pragma unroll
                        for (int k = 0; k < 4; ++k) { mma_f16_ss(d_addr, adesc + 2 * k, bdesc + 2 * k, idesc, acc); acc = 1; }
                    }
                    mma_commit(&plane_empty[pb]);
                    if (++pb == NP) { pb = 0; pph ^= 1u; }
                }
                if (alive) mma_commit(&d_full[db]);
            }
        }
    } else if (warp < 10) {
        // ---- convert: thread owns 16-byte chunk position qq of every 32nd pixel of a plane
        const int tid = threadIdx.x - 64;                // 0..255
        const int qq = tid & 7, slot = tid >> 3;         // slot 0..31
        const int src_q = ((qq >> 1) * band_in_rows + 2 * (qq & 1)) * pl.W;     // channel (qq>>1) of a plane, row pair (qq&1)
        const int plane_src = 4 * band_in_rows * pl.W;                          // four channels per plane
        // This thread's pixels slot, slot + 32, ... of a plane never change: their source and
        // destination offsets are worked out once (the converter warps are bound by instruction issue).
        constexpr int kIters = 7;                        // tile_rows <= 200 pixels / 32 per pass
        int soff[kIters], doff[kIters];
#pragma unroll
        for (int i = 0; i < kIters; ++i) {
            const int ps = slot + 32 * i;
            const int ys = ps / pl.Ws, xs = ps - ys * pl.Ws;
            soff[i] = (4 * ys) * pl.W + 4 * xs;
            doff[i] = ps * 128 + ((qq ^ (ps & 7)) << 4);  // chunk qq of row ps, 128-byte swizzle: qq ^ (ps % 8)
        }
        int it = 0, pb = 0;
        uint32_t pph = 0;
        bool alive = true;
        int s = 0;
        uint32_t sph = 0;
        for (int u = blockIdx.x; alive && u < units; u += gridDim.x, ++it) {
            const int band = u % pl.bands;
            int in_rows = pl.H - 4 * band * pl.R; in_rows = in_rows > band_in_rows ? band_in_rows : in_rows;
            const int pixels = (in_rows >> 2) * pl.Ws;   // space-to-depth pixels present in this band
            if (!mbar_wait_warp(&u8_full[s], sph, abortp, p.status, 14)) break;
            const uint8_t* src = s_u8 + s * pl.u8_stage_bytes + src_q;
#pragma unroll
            for (int pln = 0; pln < CPT; ++pln) {
                if (!mbar_wait_warp(&plane_empty[pb], pph ^ 1u, abortp, p.status, 17)) { alive = false; break; }
                uint8_t* dplane = s_tile + pb * plane_bytes;
                const uint8_t* splane = src + pln * plane_src;
#pragma unroll
                for (int i = 0; i < kIters; ++i) {
                    if (slot + 32 * i < pixels) {
                        const uint8_t* s0 = splane + soff[i];
                        const uint32_t w0 = *reinterpret_cast<const uint32_t*>(s0);
                        const uint32_t w1 = *reinterpret_cast<const uint32_t*>(s0 + pl.W);
                        uint4 o;
                        u8x4_to_h4(w0, o.x, o.y);
                        u8x4_to_h4(w1, o.z, o.w);
                        *reinterpret_cast<uint4*>(dplane + doff[i]) = o;
                    }
                }
                fence_async_proxy();                     // plane stores -> visible to the tensor core's reads
                mbar_arrive(&plane_full[pb]);
                if (++pb == NP) { pb = 0; pph ^= 1u; }
            }
            if (alive) mbar_arrive(&u8_empty[s]);
            if (++s == NU) { s = 0; sph ^= 1u; }
        }
    } else if (warp < 14) {
        // ---- epilogue: warps 10..13 read TMEM lane quarters 2,3,0,1 and add the two accumulators
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const float inv = *p.inv_scale;
        const int ey = row / pl.Ws, ex = row - ey * pl.Ws;
        int it = 0;
        for (int u = blockIdx.x; u < units; u += gridDim.x, ++it) {
            const int db = it & 1;
            const int env = u / pl.bands, band = u - env * pl.bands;
            const int y0 = band * pl.R;
            if (!mbar_wait_warp(&d_full[db], ((uint32_t)it >> 1) & 1u, abortp, p.status, 15)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_d + db * 64 + ((uint32_t)(q * 32) << 16);
            const int yy = y0 + ey;
            const bool valid = ey < pl.R && yy < pl.H1 && ex < pl.W1;
            __half* dst = p.out + ((size_t)env * pl.P1s + (size_t)(yy >> 1) * pl.W1s + (ex >> 1)) * 128 +
                          ((yy & 1) * 2 + (ex & 1)) * 32;
#pragma unroll
            for (int j = 0; j < 32; j += 16) {
                uint32_t v0[16], v1[16];
                tmem_ld_32x16(taddr + j, v0);               // dy = 0 taps
                tmem_ld_32x16(taddr + 32 + j, v1);          // dy = 1 taps
                tmem_ld_wait();
                if (j == 16) {
                    tc_fence_before();
                    mbar_arrive(&d_empty[db]);
                }
                if (valid) {
                    uint32_t pk[8];
#pragma unroll
                    for (int hh = 0; hh < 8; ++hh) {
                        const int c = 2 * hh;
                        const float a0 = __uint_as_float(v0[c]) + __uint_as_float(v1[c]);
                        const float a1 = __uint_as_float(v0[c + 1]) + __uint_as_float(v1[c + 1]);
                        __half2 t = __floats2half2_rn(fmaf(a0, inv, s_bias[j + c]), fmaf(a1, inv, s_bias[j + c + 1]));
                        t = __hmin2(__hmax2(t, __float2half2_rn(0.f)), __float2half2_rn(65504.f));
                        pk[hh] = *reinterpret_cast<uint32_t*>(&t);
                    }
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
    if (warp == 1) tmem_dealloc(tmem_d, 128);
}

// ---------------------------------------------------------------------------------------------
// Four-channel frames (Cs = 64): the A operand goes to tensor memory instead of shared memory.
//
// The shared-memory kernel above is bound by shared-memory bandwidth: each 128x32x16 MMA fetches
// 4 KB of A and 1 KB of B (40 clocks at 128 bytes per clock) and every space-to-depth pixel is
// fetched once per tap.  With tcgen05.mma taking A from tensor memory only B (1 KB) comes from
// shared memory, and tensor memory has no shifted views, so the converter writes the im2col row
// of each output pixel (4 taps x 64 channels = 256 fp16 = 128 columns) straight from registers
// with tcgen05.st.  Rows of a tile are then free to be ANY 128 output pixels: tile t covers pixels
// [128 t, 128 t + 128) of the batch in (env, y, x) order, no row of the MMA is wasted.
//
// One tile: the copy thread brings the input rows under the tile's output rows (at most two
// environments) into a staged buffer.  A is one buffer of four quarters, one per filter tap
// (dy,dx), 32 columns each.  Converter warps 2..5 write the dy = 0 quarters, warps 6..9 the dy = 1
// quarters, each thread its own row.  Two threads issue MMAs, thread h the four K steps of each
// dy = h quarter as it arrives, into its own accumulator (one thread issues an MMA every 55 to
// 110 clocks, and MMAs of two threads into one accumulator would have no defined order); the
// epilogue adds the two in a fixed order.  A quarter is refilled for the next tile as soon as its
// MMAs are done.  Two CTAs share an SM.
constexpr int kTsThreads = 480;      // warp 0 copies, 1 and 14 issue, 2..9 convert, 10..13 epilogue
constexpr int kTsStagesMax = 6;
// bytes of one channel of a staged tile: four input rows per output row a tile can touch, plus the
// closing rows of two environments
__host__ __device__ constexpr int ts_chan_bytes(int W)
{
    return W * (4 * ((128 + (W / 4 - 1) - 2) / (W / 4 - 1) + 1) + 8);
}

// (environment, output row, column) of a pixel that advances by a fixed number of pixels per step
struct PixelWalk {
    int e, y, x;
    int sq, sr, eq, er;              // step = sq rows + sr columns; sq rows = eq environments + er rows
    __device__ void init(uint32_t px, uint32_t step, int H1, int W1)
    {
        const uint32_t g = px / (uint32_t)W1;
        x = (int)(px - g * (uint32_t)W1);
        e = (int)(g / (uint32_t)H1);
        y = (int)(g - (uint32_t)e * (uint32_t)H1);
        sq = (int)(step / (uint32_t)W1); sr = (int)(step - (uint32_t)sq * (uint32_t)W1);
        eq = sq / H1; er = sq - eq * H1;
    }
    __device__ __forceinline__ void advance(int H1, int W1)
    {
        x += sr; y += er; e += eq;
        if (x >= W1) { x -= W1; ++y; }
        if (y >= H1) { y -= H1; ++e; }
    }
};

// rows of the tile that starts at pixel (e0, y0, x0): nA inside e0, nB inside e0 + 1
__device__ __forceinline__ void ts_rows(const Conv1Plan& pl, int n, int e0, int y0, int x0, int& nA, int& nB)
{
    int rows = (x0 + 127) / pl.W1 + 1;
    const int left_batch = (n - e0) * pl.H1 - y0;            // output rows from here to the end of the batch
    if (rows > left_batch) rows = left_batch;
    const int left = pl.H1 - y0;
    nA = rows < left ? rows : left;
    nB = rows - nA;
}

// WC: the frame width when it is known at compile time (the converter's 32 loads per row then use
// immediate offsets instead of computed pointers; its warps are bound by instruction issue), 0 = any.
template <int WC>
__global__ void __launch_bounds__(kTsThreads, 2)
conv1_ts_kernel(const __grid_constant__ CUtensorMap tmW, const Conv1Params p)
{
    const Conv1Plan& pl = p.pl;
    const int W = WC ? WC : pl.W;
    const int chan_bytes = WC ? ts_chan_bytes(WC) : pl.ts_chan_bytes;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t w_bar, u8_full[kTsStagesMax], u8_empty[kTsStagesMax], q_full[4], q_empty[4], d_full[2], d_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ __align__(16) float s_bias[32];
    volatile int* abortp = &abort_flag;

    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    constexpr int w_bytes = 4 * kChunkBytes;
    uint8_t* s_u8 = sm + w_bytes;
    const int NU = pl.ts_stages;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tiles = (int)(((long)p.n * pl.H1 * pl.W1 + 127) / 128);       // the host keeps n*H1*W1 below 2^31
    const uint32_t step = 128u * gridDim.x;

    if (threadIdx.x == 0) {
        mbar_init(&w_bar, 1);
        for (int s = 0; s < kTsStagesMax; ++s) { mbar_init(&u8_full[s], 1); mbar_init(&u8_empty[s], kConverters); }
        for (int s = 0; s < 4; ++s) { mbar_init(&q_full[s], kConverters / 2); mbar_init(&q_empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&d_full[s], 2); mbar_init(&d_empty[s], kWorkers); }
        abort_flag = 0;
        fence_barrier_init();
        tma_prefetch_desc(&tmW);
    }
    if (threadIdx.x >= 64 && threadIdx.x < 96) s_bias[threadIdx.x - 64] = p.bias[threadIdx.x - 64];
    if (warp == 1) tmem_alloc(&tmem_slot, 256);               // columns 0..127 A; 128 + 64 db + 32 h: accumulator h of buffer db
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_a = tmem_slot, tmem_d = tmem_slot + 128;
    if (threadIdx.x == 0) {                                   // the filter does not depend on the previous kernel
        mbar_arrive_expect_tx(&w_bar, (uint32_t)w_bytes);
        for (int g = 0; g < 4; ++g) tma_load_2d(sm + g * kChunkBytes, &tmW, g * 64, 0, &w_bar);
    }
    pdl_wait();
    pdl_trigger();

    if (warp == 0) {
        if (lane == 0) {
            const size_t chan = (size_t)pl.H * pl.W, frame = chan * pl.C;
            PixelWalk first;
            first.init(128u * blockIdx.x, step, pl.H1, pl.W1);
            int s = 0;                                    // staged tile and the parity of its current use
            uint32_t sph = 0;
            for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x, first.advance(pl.H1, pl.W1)) {
                if (!mbar_wait(&u8_empty[s], sph ^ 1u, abortp, p.status, 31)) break;
                int nA, nB;
                ts_rows(pl, p.n, first.e, first.y, first.x, nA, nB);
                const uint32_t bytesA = (uint32_t)((4 * nA + 4) * W), bytesB = nB ? (uint32_t)((4 * nB + 4) * W) : 0u;
                mbar_arrive_expect_tx(&u8_full[s], (bytesA + bytesB) * pl.C);
                // staged layout: channel c at c * ts_chan_bytes; inside it the rows of e0, then the rows of e0 + 1
                uint8_t* dst = s_u8 + s * pl.ts_stage_bytes;
                const uint8_t* srcA = p.obs + frame_of(p, first.e) * frame + (size_t)(4 * first.y) * W;
                for (int c = 0; c < pl.C; ++c) bulk_load(dst + c * chan_bytes, srcA + c * chan, bytesA, &u8_full[s]);
                if (nB) {
                    const uint8_t* srcB = p.obs + frame_of(p, first.e + 1) * frame;
                    for (int c = 0; c < pl.C; ++c) bulk_load(dst + c * chan_bytes + bytesA, srcB + c * chan, bytesB, &u8_full[s]);
                }
                if (++s == NU) { s = 0; sph ^= 1u; }
            }
        }
    } else if (warp == 1 || warp == 14) {
        if (lane == 0) {
            const int h = warp == 1 ? 0 : 1;
            constexpr uint32_t idesc = instr_desc_f16(0, 128, 32);
            bool alive = mbar_wait(&w_bar, 0, abortp, p.status, 32);
            int it = 0;
            for (int tile = blockIdx.x; alive && tile < tiles; tile += gridDim.x, ++it) {
                const int db = it & 1;
                if (!mbar_wait(&d_empty[db], (((uint32_t)it >> 1) & 1u) ^ 1u, abortp, p.status, 33)) break;
                const uint32_t d_addr = tmem_d + db * 64 + h * 32;
#pragma unroll
                for (int dx = 0; dx < 2; ++dx) {
                    const int qd = 2 * h + dx;                // quarter = filter tap = weight chunk
                    if (!mbar_wait(&q_full[qd], (uint32_t)it & 1u, abortp, p.status, 34)) { alive = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const uint64_t bdesc = smem_desc_sw128(base + qd * kChunkBytes) + 2 * k;
                        mma_f16_ts(d_addr, tmem_a + 32 * qd + 8 * k, bdesc, idesc, (dx | k) != 0);
                    }
                    mma_commit(&q_empty[qd]);
                }
                if (alive) mma_commit(&d_full[db]);
            }
        }
    } else if (warp < 10) {
        // ---- convert: thread = row m of the tile; warps 2..5 the dy = 0 quarters, warps 6..9 dy = 1
        const int h = (warp - 2) >> 2;
        const int q = warp & 3, m = q * 32 + lane;
        const uint32_t st_addr = tmem_a + ((uint32_t)(q * 32) << 16) + 64 * h;
        PixelWalk first, mine;
        first.init(128u * blockIdx.x, step, pl.H1, pl.W1);
        mine.init(128u * blockIdx.x + (uint32_t)m, step, pl.H1, pl.W1);
        int it = 0, s = 0;
        uint32_t sph = 0;
        for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++it, first.advance(pl.H1, pl.W1), mine.advance(pl.H1, pl.W1)) {
            // Staged input row under this pixel's window: four rows per output row since the tile's
            // first one, plus the four extra rows that close the first environment's part.  Rows past
            // the end of the batch read the start of the buffer: their results are never stored.
            const int segB = mine.e != first.e;
            const int row = 4 * ((segB ? pl.H1 : 0) + mine.y - first.y + segB + h);
            const int off = mine.e < p.n ? row * W + 4 * mine.x : 0;
            if (!mbar_wait_warp(&u8_full[s], sph, abortp, p.status, 35)) break;
            const uint8_t* src = s_u8 + s * pl.ts_stage_bytes + off;
            bool alive = true;
#pragma unroll
            for (int dx = 0; dx < 2; ++dx) {
                uint32_t r[32];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
#pragma unroll
                    for (int uy = 0; uy < 4; ++uy)
                        u8x4_to_h4(*reinterpret_cast<const uint32_t*>(src + c * chan_bytes + uy * W + 4 * dx), r[c * 8 + uy * 2], r[c * 8 + uy * 2 + 1]);
                }
                if (dx == 1) mbar_arrive(&u8_empty[s]);       // the staged rows are in registers
                if (!mbar_wait_warp(&q_empty[2 * h + dx], ((uint32_t)it & 1u) ^ 1u, abortp, p.status, 36)) { alive = false; break; }
                tc_fence_after();
                tmem_st_32x32(st_addr + 32 * dx, r);
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(&q_full[2 * h + dx]);
            }
            if (!alive) break;
            if (++s == NU) { s = 0; sph ^= 1u; }
        }
    } else if (warp < 14) {
        // ---- epilogue: warps 10..13 read TMEM lane quarters 2,3,0,1
        const int q = warp & 3, m = q * 32 + lane;
        const float inv = *p.inv_scale;
        PixelWalk mine;
        mine.init(128u * blockIdx.x + (uint32_t)m, step, pl.H1, pl.W1);
        int it = 0;
        for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++it, mine.advance(pl.H1, pl.W1)) {
            const int db = it & 1;
            if (!mbar_wait_warp(&d_full[db], ((uint32_t)it >> 1) & 1u, abortp, p.status, 37)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_d + db * 64 + ((uint32_t)(q * 32) << 16);
            __half* dst = p.out + ((size_t)mine.e * pl.P1s + (size_t)(mine.y >> 1) * pl.W1s + (mine.x >> 1)) * 128 +
                          ((mine.y & 1) * 2 + (mine.x & 1)) * 32;
#pragma unroll
            for (int j = 0; j < 32; j += 16) {
                uint32_t v0[16], v1[16];
                tmem_ld_32x16(taddr + j, v0);               // dy = 0 taps
                tmem_ld_32x16(taddr + 32 + j, v1);          // dy = 1 taps
                tmem_ld_wait();
                if (j == 16) {
                    tc_fence_before();
                    mbar_arrive(&d_empty[db]);
                }
                if (mine.e < p.n) {
                    uint32_t pk[8];
#pragma unroll
                    for (int hh = 0; hh < 8; hh += 2) {
                        const int c = 2 * hh;
                        const float4 b4 = *reinterpret_cast<const float4*>(&s_bias[j + c]);
                        __half2 t0 = __floats2half2_rn(fmaf(__uint_as_float(v0[c]) + __uint_as_float(v1[c]), inv, b4.x),
                                                       fmaf(__uint_as_float(v0[c + 1]) + __uint_as_float(v1[c + 1]), inv, b4.y));
                        __half2 t1 = __floats2half2_rn(fmaf(__uint_as_float(v0[c + 2]) + __uint_as_float(v1[c + 2]), inv, b4.z),
                                                       fmaf(__uint_as_float(v0[c + 3]) + __uint_as_float(v1[c + 3]), inv, b4.w));
                        t0 = __hmin2(__hmax2(t0, __float2half2_rn(0.f)), __float2half2_rn(65504.f));
                        t1 = __hmin2(__hmax2(t1, __float2half2_rn(0.f)), __float2half2_rn(65504.f));
                        pk[hh] = *reinterpret_cast<uint32_t*>(&t0);
                        pk[hh + 1] = *reinterpret_cast<uint32_t*>(&t1);
                    }
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
    if (warp == 1) tmem_dealloc(tmem_slot, 256);
}

__global__ void pack_conv1_kernel(const __nv_bfloat16* __restrict__ w, __half* __restrict__ wp, int C,
                                  const float* __restrict__ scale)
{
    const int Cs = 16 * C;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 32 * 4 * Cs) return;
    const int o = i / (4 * Cs), k = i % (4 * Cs);
    const int tap = k / Cs, cp = k % Cs;
    const int dy = tap >> 1, dx = tap & 1, c = cp >> 4, uy = (cp >> 2) & 3, ux = cp & 3;
    wp[i] = __float2half_rn(__bfloat162float(w[((o * C + c) * 8 + (4 * dy + uy)) * 8 + (4 * dx + ux)]) * scale[0]);
}

}  // namespace

bool conv1_plan(const Geometry& g, Conv1Plan* pl)
{
    if (g.C % 4 || g.H % 4 || g.W % 4 || (g.C != 4 && g.C != 8 && g.C != 16)) return false;    // bulk copies then start and end on 16-byte boundaries
    pl->C = g.C; pl->H = g.H; pl->W = g.W;
    pl->Hs = g.H / 4; pl->Ws = g.W / 4; pl->Cs = 16 * g.C;
    pl->H1 = pl->Hs - 1; pl->W1 = pl->Ws - 1;
    if (pl->H1 != g.H1 || pl->W1 != g.W1 || pl->Ws > 64 || pl->Ws < 3 || pl->H1 < 1) return false;
    pl->cpt = pl->Cs / 64;
    const int rmax = 128 / pl->Ws;
    pl->bands = (pl->H1 + rmax - 1) / rmax;
    pl->R = (pl->H1 + pl->bands - 1) / pl->bands;
    pl->tile_rows = (128 + pl->Ws + 1 + 7) / 8 * 8;
    pl->u8_stage_bytes = (g.C * 4 * (pl->R + 1) * g.W + 127) / 128 * 128;
    const int fixed = 1024 + 4 * pl->cpt * kChunkBytes;
    const int plane = pl->tile_rows * 128;
    // The fp16 planes (64 channels of a band each) form a ring.  Narrow inputs: 3 planes = 3 units in
    // flight and 4 staged bands, small enough for two CTAs per SM.  Wide inputs: 4 planes, one CTA per SM.
    pl->plane_bufs = pl->cpt == 1 ? 3 : 4;
    const int budget = (pl->cpt == 1 ? 110 : 226) * 1024 - fixed - pl->plane_bufs * plane;
    pl->u8_stages = budget / pl->u8_stage_bytes;
    if (pl->u8_stages > 4) pl->u8_stages = 4;
    if (pl->u8_stages < 2) return false;
    pl->smem_bytes = fixed + pl->plane_bufs * plane + pl->u8_stages * pl->u8_stage_bytes;
    pl->H1s = (pl->H1 + 1) / 2; pl->W1s = (pl->W1 + 1) / 2; pl->P1s = pl->H1s * pl->W1s;
    // tensor-memory variant: four-channel frames whose image has at least one tile of output pixels
    // (a tile then touches at most two environments)
    pl->ts = pl->cpt == 1 && pl->H1 * pl->W1 >= 128;
    if (pl->ts) {
        pl->ts_chan_bytes = ts_chan_bytes(g.W);                           // one channel of a staged tile (a multiple of 16)
        pl->ts_stage_bytes = (g.C * pl->ts_chan_bytes + 127) / 128 * 128;
        int st = (100 * 1024 - 4 * kChunkBytes) / pl->ts_stage_bytes;     // two CTAs per SM
        if (st > kTsStagesMax) st = kTsStagesMax;
        if (st < 2) pl->ts = 0;
        pl->ts_stages = st;
        pl->ts_smem_bytes = 1024 + 4 * kChunkBytes + st * pl->ts_stage_bytes;
    }
    return true;
}

hts_status conv1_pack_weights(const Conv1Plan& pl, const __nv_bfloat16* w1, __half* packed, const float* scale,
                              cudaStream_t s)
{
    const int total = 32 * 4 * pl.Cs;
    pack_conv1_kernel<<<(total + 255) / 256, 256, 0, s>>>(w1, packed, pl.C, scale);
    HTS_LAUNCH_CHECK("pack_conv1");
    return HTS_OK;
}

hts_status conv1_launch(const Conv1Plan& pl, const CUtensorMap& weight_map, const uint8_t* obs, const Indexing& ix, int n,
                        const float* bias, const float* inv_scale, __half* out, int* status, cudaStream_t s)
{
    const int dev = device_slot();
    const int sm_count = device_sm_count(dev);
    static int smem_set_by_device[kDeviceSlots] = {}, ts_smem_set_by_device[kDeviceSlots] = {};
    int& max_smem_set = smem_set_by_device[dev];
    int& ts_smem_set = ts_smem_set_by_device[dev];
    if (max_smem_set < pl.smem_bytes) {
        HTS_CUDA(cudaFuncSetAttribute(conv1_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem_bytes));
        HTS_CUDA(cudaFuncSetAttribute(conv1_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem_bytes));
        HTS_CUDA(cudaFuncSetAttribute(conv1_tc_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem_bytes));
        // every kernel of the step asks for the largest shared-memory carve-out, so that the SMs are not
        // re-partitioned between consecutive kernels
        HTS_CUDA(cudaFuncSetAttribute(conv1_tc_kernel<1>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
        HTS_CUDA(cudaFuncSetAttribute(conv1_tc_kernel<2>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
        HTS_CUDA(cudaFuncSetAttribute(conv1_tc_kernel<4>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
        max_smem_set = pl.smem_bytes;
    }
    if (pl.ts && (long)n * pl.H1 * pl.W1 < (1L << 31) - 128 * 2 * sm_count) {
        if (ts_smem_set < pl.ts_smem_bytes) {
            HTS_CUDA(cudaFuncSetAttribute(conv1_ts_kernel<84>, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.ts_smem_bytes));
            HTS_CUDA(cudaFuncSetAttribute(conv1_ts_kernel<84>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
            HTS_CUDA(cudaFuncSetAttribute(conv1_ts_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.ts_smem_bytes));
            HTS_CUDA(cudaFuncSetAttribute(conv1_ts_kernel<0>, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
            ts_smem_set = pl.ts_smem_bytes;
        }
        const long total_px = (long)n * pl.H1 * pl.W1;
        const int tiles = (int)((total_px + 127) / 128);
        int grid = 2 * sm_count;
        if (grid > tiles) grid = tiles;
        Conv1Params p{pl, obs, ix.slots, ix.pool, n, bias, inv_scale, out, status};
        if (pl.W == 84) HTS_CUDA(launch_pdl(conv1_ts_kernel<84>, dim3(grid), dim3(kTsThreads), (size_t)pl.ts_smem_bytes, s, weight_map, p));
        else HTS_CUDA(launch_pdl(conv1_ts_kernel<0>, dim3(grid), dim3(kTsThreads), (size_t)pl.ts_smem_bytes, s, weight_map, p));
        note_launch();
        return HTS_OK;
    }
    const int per_sm = (227 * 1024) / (pl.smem_bytes + 1024) > 2 ? 2 : (227 * 1024) / (pl.smem_bytes + 1024);
    const int units = n * pl.bands;
    int grid = sm_count * (per_sm < 1 ? 1 : per_sm);
    if (grid > units) grid = units;
    Conv1Params p{pl, obs, ix.slots, ix.pool, n, bias, inv_scale, out, status};
    if (pl.cpt == 1) HTS_CUDA(launch_pdl(conv1_tc_kernel<1>, dim3(grid), dim3(kThreads), (size_t)pl.smem_bytes, s, weight_map, p));
    else if (pl.cpt == 2) HTS_CUDA(launch_pdl(conv1_tc_kernel<2>, dim3(grid), dim3(kThreads), (size_t)pl.smem_bytes, s, weight_map, p));
    else HTS_CUDA(launch_pdl(conv1_tc_kernel<4>, dim3(grid), dim3(kThreads), (size_t)pl.smem_bytes, s, weight_map, p));
    note_launch();
    return HTS_OK;
}

}  // namespace hts
