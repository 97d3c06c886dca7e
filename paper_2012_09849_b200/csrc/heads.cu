// Policy / value heads and the sampling epilogue of the actor step.
//
// One warp per observation.  The warp forms the 512 hidden units (summing the FC split-K
// partials in index order when asked), takes the A+1 head dot products, then the policy
// distribution (log-softmax, entropy in nats: the H(pi(.|s)) of Eq. 3) and one action by
// Gumbel-max.  The uniforms come from Philox4x32-10 (Salmon et al., SC'11) with counter
// (env_id, t, a/4, 0) and key (seed_lo, seed_hi): the per-observation pseudo-random number
// of Section 4.1, so the action is a function of (seed, env_id, t) and the logits alone.
#include "common.cuh"

namespace hts {
namespace {

constexpr int kHidden = 512;
constexpr int kMaxActions = 64;
constexpr int kMaxSplits = 8;

__device__ __forceinline__ void philox_round(uint32_t (&c)[4], uint32_t k0, uint32_t k1)
{
    const uint32_t hi0 = __umulhi(0xD2511F53u, c[0]), lo0 = 0xD2511F53u * c[0];
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c[2]), lo1 = 0xCD9E8D57u * c[2];
    const uint32_t n0 = hi1 ^ c[1] ^ k0, n2 = hi0 ^ c[3] ^ k1;
    c[0] = n0; c[1] = lo1; c[2] = n2; c[3] = lo0;
}

__device__ __forceinline__ uint32_t philox_word(uint32_t env, uint32_t t, uint32_t block, uint32_t lane4,
                                                uint32_t k0, uint32_t k1)
{
    uint32_t c[4] = {env, t, block, 0u};
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        philox_round(c, k0, k1);
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    return lane4 == 0 ? c[0] : lane4 == 1 ? c[1] : lane4 == 2 ? c[2] : c[3];
}

// u = ((word >> 9) + 1/2) * 2^-23: 23 bits so that the value is exact in fp32 and inside (0,1)
__device__ __forceinline__ float action_uniform(uint32_t env, uint32_t t, int a, uint32_t k0, uint32_t k1)
{
    const uint32_t word = philox_word(env, t, (uint32_t)a >> 2, (uint32_t)a & 3u, k0, k1);
    return ((float)(word >> 9) + 0.5f) * (1.0f / 8388608.0f);
}

__global__ void uniforms_kernel(const int32_t* __restrict__ env_ids, const int32_t* __restrict__ t_per_env,
                                int32_t t_scalar, uint32_t k0, uint32_t k1, int n, int A, float* __restrict__ out)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)n * A) return;
    const int e = (int)(i / A), a = (int)(i % A);
    out[i] = action_uniform((uint32_t)env_ids[e], (uint32_t)(t_per_env ? t_per_env[e] : t_scalar), a, k0, k1);
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
    return v;
}

// Warp sums of eight per-lane values in 9 shuffles instead of 40: at each of the first three levels a lane keeps
// the half of the values that its lane bit selects and hands the other half to its partner, so that after them it
// holds one value summed over 8 lanes; two plain levels finish.  Every lane returns the warp total of value
// 4 * bit4 + 2 * bit3 + bit2 of its lane number.  The order of the additions depends on lane numbers alone.
__device__ __forceinline__ float warp_sum8(const float (&acc)[8], int lane)
{
    const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
    float a4[4], a2[2];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const float send = b4 ? acc[j] : acc[j + 4], keep = b4 ? acc[j + 4] : acc[j];
        a4[j] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const float send = b3 ? a4[j] : a4[j + 2], keep = b3 ? a4[j + 2] : a4[j];
        a2[j] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
    }
    const float send = b2 ? a2[0] : a2[1], keep = b2 ? a2[1] : a2[0];
    float a1 = keep + __shfl_xor_sync(0xffffffffu, send, 4);
    a1 += __shfl_xor_sync(0xffffffffu, a1, 2);
    a1 += __shfl_xor_sync(0xffffffffu, a1, 1);
    return a1;
}

// MAXS: the most split partials a launch may have to sum (1 = the hidden layer is final: few registers, so four
// blocks fit an SM); MINB: blocks per SM the register allocation must allow.  The arithmetic of a row is the same
// in every instantiation.
template <int MAXS, int MINB>
__global__ void __launch_bounds__(256, MINB)
heads_kernel(const float* __restrict__ h_partials, int num_splits, size_t split_stride,
             const float* __restrict__ fc_bias, const float* __restrict__ whead,
             const float* __restrict__ bhead, int A, const int32_t* __restrict__ env_ids,
             const int32_t* __restrict__ t_per_env, int32_t t_scalar, uint32_t key0, uint32_t key1,
             int n, const int32_t* __restrict__ slots, int pool, int* __restrict__ status,
             const int32_t* __restrict__ given,
             int32_t* __restrict__ actions, float* __restrict__ logp,
             float* __restrict__ values, float* __restrict__ entropy, float* __restrict__ logits_out,
             float* __restrict__ h_out)
{
    extern __shared__ float4 s_w4[];                   // [(A+1)*512] head weights, staged once per block
    __shared__ float s_out[8][kMaxActions + 1];
    __shared__ float s_bhead[kMaxActions + 1];
    __shared__ float4 s_fcb[kHidden / 4];
    const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
    {
        const float4* src = reinterpret_cast<const float4*>(whead);
        const int total4 = (A + 1) * (kHidden / 4);
        for (int i = threadIdx.x; i < total4; i += 256) s_w4[i] = src[i];
        // biases too: a global load inside the per-output loop would stall the warp once per iteration
        if (threadIdx.x <= A) s_bhead[threadIdx.x] = bhead[threadIdx.x];
        if (fc_bias && threadIdx.x < kHidden / 4) s_fcb[threadIdx.x] = reinterpret_cast<const float4*>(fc_bias)[threadIdx.x];
    }
    pdl_wait();                                        // the head weights above are older than the previous kernel
    pdl_trigger();
    __syncthreads();
    const float4* sw4 = s_w4;
    // rows are dealt block-first (row g goes to block g % gridDim.x), so a batch of fewer rows than warps on
    // the device still spreads over every block
    for (int e = wib * gridDim.x + blockIdx.x; e < n; e += gridDim.x * 8) {
    const uint32_t env = given ? 0u : (uint32_t)env_ids[e];            // issued early: needed only by the sampler
    const uint32_t tt = given ? 0u : (uint32_t)(t_per_env ? t_per_env[e] : t_scalar);
    // hidden vector: lane l owns units 128*i + 4*l + {0..3}, i = 0..3 (float4 everywhere); split
    // partials are summed in index order
    float4 h[4];
    {
        const float4* hp = reinterpret_cast<const float4*>(h_partials + (size_t)e * kHidden) + lane;
        const size_t stride4 = split_stride / 4;
        float4 part[MAXS][4];
#pragma unroll
        for (int sp = 0; sp < MAXS; ++sp)
#pragma unroll
            for (int i = 0; i < 4; ++i)
                part[sp][i] = hp[(sp < num_splits ? sp : 0) * stride4 + 32 * i];   // unconditional: all loads in flight at once
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float4 v = part[0][i];
#pragma unroll
            for (int sp = 1; sp < MAXS; ++sp)
                if (sp < num_splits) { v.x += part[sp][i].x; v.y += part[sp][i].y; v.z += part[sp][i].z; v.w += part[sp][i].w; }
            if (fc_bias) {
                const float4 bb = s_fcb[32 * i + lane];
                v.x = fmaxf(v.x + bb.x, 0.f); v.y = fmaxf(v.y + bb.y, 0.f); v.z = fmaxf(v.z + bb.z, 0.f); v.w = fmaxf(v.w + bb.w, 0.f);
            }
            h[i] = v;
            if (h_out) reinterpret_cast<float4*>(h_out + (size_t)e * kHidden)[32 * i + lane] = v;
        }
    }
    // Eight outputs per pass: their dot products are independent chains, and one transposing reduction sums all
    // eight over the lanes.  Each output keeps its own fixed summation order.
    for (int o0 = 0; o0 <= A; o0 += 8) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (o0 + j <= A) {                             // the same for every lane
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float4 w = sw4[(o0 + j) * (kHidden / 4) + 32 * i + lane];
                    acc[j] = fmaf(w.x, h[i].x, acc[j]); acc[j] = fmaf(w.y, h[i].y, acc[j]);
                    acc[j] = fmaf(w.z, h[i].z, acc[j]); acc[j] = fmaf(w.w, h[i].w, acc[j]);
                }
            }
        }
        const float tot = warp_sum8(acc, lane);
        const int o = o0 + (lane >> 2);
        if ((lane & 3) == 0 && o <= A) s_out[wib][o] = tot + s_bhead[o];
    }
    __syncwarp();
    const float* lg = s_out[wib];

    float m = -INFINITY;
    for (int a = lane; a < A; a += 32) m = fmaxf(m, lg[a]);
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, k));
    float z = 0.f;
    for (int a = lane; a < A; a += 32) z += expf(lg[a] - m);
    z = warp_sum(z);
    const float lse = m + logf(z);
    float ent = 0.f;
    for (int a = lane; a < A; a += 32) { const float lp = lg[a] - lse; ent -= expf(lp) * lp; }
    ent = warp_sum(ent);

    float best = -INFINITY; int best_a = 0x7fffffff;
    if (given) best_a = given[e];                       // learner's re-evaluation: the stored action, no sampling
    else {
    for (int a = lane; a < A; a += 32) {
        const float u = action_uniform(env, tt, a, key0, key1);
        const float score = lg[a] - logf(-logf(u));
        if (score > best) { best = score; best_a = a; }                        // ascending a: ties keep the lowest
    }
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, k);
        const int oa = __shfl_xor_sync(0xffffffffu, best_a, k);
        if (ob > best || (ob == best && oa < best_a)) { best = ob; best_a = oa; }
    }
    }
    if (logits_out) for (int a = lane; a < A; a += 32) logits_out[(size_t)e * A + a] = lg[a];
    if (lane == 0) {
        int o = e;                                       // dense, or the row's slot of the storage row
        if (slots) {
            o = slots[e];
            if ((unsigned)o >= (unsigned)pool) { if (status) atomicCAS(status, 0, kStatusBadSlot); o = -1; }
        }
        if ((unsigned)best_a >= (unsigned)A) { if (status) atomicCAS(status, 0, kStatusBadAction); o = -1; }
        if (o >= 0) {
            if (actions) actions[o] = best_a;
            logp[o] = lg[best_a] - lse;
            values[o] = lg[A];
            entropy[o] = ent;
        }
    }
    __syncwarp();                                      // s_out[wib] is reused by the next environment
    }
}

}  // namespace

hts_status launch_heads(const float* h_partials, int num_splits, size_t split_stride,
                        const float* fc_bias, const float* whead, const float* bhead, int A,
                        const int32_t* env_ids, const int32_t* t_per_env, int32_t t,
                        uint64_t seed, int n, const Indexing& ix, int* status, int32_t* actions, float* logp,
                        float* values, float* entropy, float* logits, float* h_out, cudaStream_t s,
                        const int32_t* given_actions)
{
    if (num_splits < 1 || num_splits > kMaxSplits) return HTS_ERR_INVALID_ARG;
    const size_t smem = (size_t)(A + 1) * kHidden * sizeof(float);
    const int dev = device_slot();
    const int sm_count = device_sm_count(dev);
    const uint32_t k0 = (uint32_t)(seed & 0xffffffffu), k1 = (uint32_t)(seed >> 32);
    auto launch = [&](auto kernel, int which, int per_sm) -> hts_status {
        static size_t smem_set_by_device[3][kDeviceSlots] = {};
        static bool carveout_set_by_device[3][kDeviceSlots] = {};
        size_t& smem_set = smem_set_by_device[which][dev];
        bool& carveout_set = carveout_set_by_device[which][dev];
        if (smem_set == 0) smem_set = 48 * 1024;        // what a kernel may use without asking
        if (!carveout_set) {
            HTS_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 100));
            carveout_set = true;
        }
        if (smem > smem_set) {
            HTS_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            smem_set = smem;
        }
        // one block per SM until every warp has a row, then as many as are resident together
        int blocks = sm_count;
        while (blocks < per_sm * sm_count && n > 8 * blocks) blocks += sm_count;
        if (blocks > n) blocks = n;
        HTS_CUDA(launch_pdl(kernel, dim3(blocks), dim3(256), smem, s, h_partials, num_splits, split_stride, fc_bias, whead,
                            bhead, A, env_ids, t_per_env, t, k0, k1, n, ix.slots, ix.pool, status, given_actions, actions,
                            logp, values, entropy, logits, h_out));
        note_launch();
        return HTS_OK;
    };
    if (num_splits == 1) return launch(heads_kernel<1, 4>, 0, 4);
    // split partials: while one block per SM gives every row a warp, let the compiler keep all loads of a row in
    // registers (measured 53.3 against 55.3 us per step at n = 1024 with the two-blocks-per-SM register cap)
    if (n <= 8 * sm_count) return launch(heads_kernel<kMaxSplits, 1>, 1, 1);
    return launch(heads_kernel<kMaxSplits, 2>, 2, 2);
}

hts_status launch_uniforms(const int32_t* env_ids, const int32_t* t_per_env, int32_t t, uint64_t seed, int n,
                           int A, float* out, cudaStream_t s)
{
    const size_t total = (size_t)n * A;
    uniforms_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(env_ids, t_per_env, t,
                                                                  (uint32_t)(seed & 0xffffffffu),
                                                                  (uint32_t)(seed >> 32), n, A, out);
    HTS_LAUNCH_CHECK("uniforms_kernel");
    return HTS_OK;
}

}  // namespace hts
