// Sample means over the stored transitions that the learner's objectives are built from:
//   hts_a2c_terms  Section 3: the policy term of Eq. 4, (1/|D|) sum log pi(a|s) (R - V), the value loss
//                  J_V = (1/|D|) sum (R - V)^2 and the mean entropy;
//   hts_ppo_terms  the clipped surrogate of proximal policy optimisation (Schulman et al. 2017, Eq. 7), the
//                  algorithm the football runs of Section 5 use, with the same value loss and entropy.
//
// HBM-bound (16 to 24 bytes per transition).  Each block sums a contiguous range in double precision in a
// fixed order (thread-strided float4 loads, shuffle tree, warp order), writes its partial and takes a
// ticket; the block that draws the last ticket adds the partials in a fixed order.  The grid is a
// function of the count alone, so the result does not depend on timing or on the device's load.
#include <cmath>
#include "common.cuh"

namespace hts {
namespace {

constexpr int kBlocksMax = 2048;
constexpr int kThreads = 256;
constexpr int kPerThread = 8;             // elements a thread covers before another block is worth its launch
constexpr int kMaxSums = 4;

// Partials, the ticket counter and the advantage statistics live in the library image: calls on one device
// must not overlap.
__device__ double g_partial[kBlocksMax][kMaxSums];
__device__ unsigned int g_ticket;
__device__ double g_adv_stats[2];         // mean and 1 / (std + 1e-8) of the advantages (hts_ppo_terms)

__device__ __forceinline__ double warp_sum_d(double v)
{
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
    return v;
}

// An Op names NS sums, how four consecutive elements (float4 group q) or one element i add to them, whether
// its arrays allow float4 loads, and what the last block does with the totals.
template <class Op>
__global__ void __launch_bounds__(kThreads)
sums_kernel(const Op op, long long count, long long per_block)
{
    constexpr int NS = Op::NS;
    __shared__ double s_part[kThreads / 32][NS];
    __shared__ bool s_last;
    const long long lo = (long long)blockIdx.x * per_block;               // per_block is a multiple of 4
    long long hi = lo + per_block; hi = hi > count ? count : hi;
    double acc[NS];
#pragma unroll
    for (int k = 0; k < NS; ++k) acc[k] = 0.0;
    if (op.aligned16()) {
        const long long q_lo = lo >> 2, q_hi = hi >> 2;                    // whole float4 groups of the range
        long long q = q_lo + threadIdx.x;
        for (; q + 3 * kThreads < q_hi; q += 4 * kThreads) {               // four groups per array in flight per thread
            typename Op::Quad g[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) g[u] = op.load4(q + u * kThreads);
#pragma unroll
            for (int u = 0; u < 4; ++u) op.add4(g[u], acc);
        }
        for (; q < q_hi; q += kThreads) op.add4(op.load4(q), acc);
        for (long long i = (q_hi << 2) + threadIdx.x; i < hi; i += kThreads) op.add1(i, acc);   // the last block's ragged tail
    } else {
        for (long long i = lo + threadIdx.x; i < hi; i += kThreads) op.add1(i, acc);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int k = 0; k < NS; ++k) {
        acc[k] = warp_sum_d(acc[k]);
        if (lane == 0) s_part[warp][k] = acc[k];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
        for (int k = 0; k < NS; ++k) {
            double a = 0.0;
            for (int w = 0; w < kThreads / 32; ++w) a += s_part[w][k];
            g_partial[blockIdx.x][k] = a;
        }
        __threadfence();
        s_last = atomicAdd(&g_ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (s_last && threadIdx.x < 32) {
        // lane l adds partials l, l + 32, ... in that order, then the lanes are folded by a shuffle tree: an order
        // fixed by the grid size, whatever the arrival order of the blocks
        __threadfence();
        double tot[NS];
#pragma unroll
        for (int k = 0; k < NS; ++k) tot[k] = 0.0;
        for (unsigned b = threadIdx.x; b < gridDim.x; b += 32)
#pragma unroll
            for (int k = 0; k < NS; ++k) tot[k] += *(volatile double*)&g_partial[b][k];
#pragma unroll
        for (int k = 0; k < NS; ++k) tot[k] = warp_sum_d(tot[k]);
        if (threadIdx.x == 0) {
            op.finish(tot, count);
            g_ticket = 0;                                                    // ready for the next launch
        }
    }
}

template <class Op>
hts_status launch_sums(const Op& op, long long count, cudaStream_t s, const char* name)
{
    long long blocks = (count + (long long)kThreads * kPerThread - 1) / ((long long)kThreads * kPerThread);
    if (blocks > kBlocksMax) blocks = kBlocksMax;
    long long per_block = (count + blocks - 1) / blocks;
    per_block = (per_block + 3) / 4 * 4;
    blocks = (count + per_block - 1) / per_block;
    sums_kernel<Op><<<(unsigned)blocks, kThreads, 0, s>>>(op, count, per_block);
    HTS_LAUNCH_CHECK(name);
    return HTS_OK;
}

inline bool all_aligned16(std::initializer_list<const void*> ps)
{
    uintptr_t x = 0;
    for (const void* p : ps) x |= (uintptr_t)p;
    return (x & 15u) == 0;
}

struct A2cOp {
    static constexpr int NS = 3;
    const float *logp, *values, *entropy, *returns;
    float* out;
    bool vec;
    struct Quad { float4 l, v, h, r; };
    __device__ bool aligned16() const { return vec; }
    __device__ Quad load4(long long q) const
    {
        return Quad{reinterpret_cast<const float4*>(logp)[q], reinterpret_cast<const float4*>(values)[q],
                    reinterpret_cast<const float4*>(entropy)[q], reinterpret_cast<const float4*>(returns)[q]};
    }
    __device__ static void one(float l, float v, float h, float r, double* acc)
    {
        const double a = (double)r - v;
        acc[0] += (double)l * a; acc[1] += a * a; acc[2] += (double)h;
    }
    __device__ void add4(const Quad& g, double* acc) const
    {
        one(g.l.x, g.v.x, g.h.x, g.r.x, acc); one(g.l.y, g.v.y, g.h.y, g.r.y, acc);
        one(g.l.z, g.v.z, g.h.z, g.r.z, acc); one(g.l.w, g.v.w, g.h.w, g.r.w, acc);
    }
    __device__ void add1(long long i, double* acc) const { one(logp[i], values[i], entropy[i], returns[i], acc); }
    __device__ void finish(const double* tot, long long count) const
    {
        const double inv = 1.0 / (double)count;
        out[0] = (float)(tot[0] * inv); out[1] = (float)(tot[1] * inv); out[2] = (float)(tot[2] * inv);
    }
};

// first and second pass over the advantages: mean, then 1 / (population std + 1e-8)
struct AdvMeanOp {
    static constexpr int NS = 1;
    const float* adv;
    bool vec;
    using Quad = float4;
    __device__ bool aligned16() const { return vec; }
    __device__ Quad load4(long long q) const { return reinterpret_cast<const float4*>(adv)[q]; }
    __device__ void add4(const Quad& g, double* acc) const { acc[0] += (double)g.x; acc[0] += (double)g.y; acc[0] += (double)g.z; acc[0] += (double)g.w; }
    __device__ void add1(long long i, double* acc) const { acc[0] += (double)adv[i]; }
    __device__ void finish(const double* tot, long long count) const { g_adv_stats[0] = tot[0] / (double)count; }
};
struct AdvVarOp {
    static constexpr int NS = 1;
    const float* adv;
    bool vec;
    using Quad = float4;
    __device__ bool aligned16() const { return vec; }
    __device__ Quad load4(long long q) const { return reinterpret_cast<const float4*>(adv)[q]; }
    __device__ static void one(float a, double mean, double* acc) { const double d = (double)a - mean; acc[0] += d * d; }
    __device__ void add4(const Quad& g, double* acc) const
    {
        const double m = g_adv_stats[0];
        one(g.x, m, acc); one(g.y, m, acc); one(g.z, m, acc); one(g.w, m, acc);
    }
    __device__ void add1(long long i, double* acc) const { one(adv[i], g_adv_stats[0], acc); }
    __device__ void finish(const double* tot, long long count) const { g_adv_stats[1] = 1.0 / (sqrt(tot[0] / (double)count) + 1e-8); }
};

struct PpoOp {
    static constexpr int NS = 4;
    const float *logp_new, *logp_old, *values, *entropy, *adv, *returns;
    float* out;
    double clip;
    bool normalize, vec;
    struct Quad { float4 ln, lo, v, h, a, r; };
    __device__ bool aligned16() const { return vec; }
    __device__ Quad load4(long long q) const
    {
        return Quad{reinterpret_cast<const float4*>(logp_new)[q], reinterpret_cast<const float4*>(logp_old)[q],
                    reinterpret_cast<const float4*>(values)[q], reinterpret_cast<const float4*>(entropy)[q],
                    reinterpret_cast<const float4*>(adv)[q], reinterpret_cast<const float4*>(returns)[q]};
    }
    __device__ void one(float ln, float lo, float v, float h, float a, float r, double mean, double inv_std, double* acc) const
    {
        const double rho = (double)expf(ln - lo);           // fp32 exponential (2 ulp): the fp64 one would bound the kernel
        const double adv_n = ((double)a - mean) * inv_std;
        const double clipped = fmin(fmax(rho, 1.0 - clip), 1.0 + clip);
        acc[0] += fmin(rho * adv_n, clipped * adv_n);
        const double d = (double)r - v;
        acc[1] += d * d;
        acc[2] += (double)h;
        acc[3] += fabs(rho - 1.0) > clip ? 1.0 : 0.0;
    }
    __device__ void add4(const Quad& g, double* acc) const
    {
        const double m = normalize ? g_adv_stats[0] : 0.0, is = normalize ? g_adv_stats[1] : 1.0;
        one(g.ln.x, g.lo.x, g.v.x, g.h.x, g.a.x, g.r.x, m, is, acc); one(g.ln.y, g.lo.y, g.v.y, g.h.y, g.a.y, g.r.y, m, is, acc);
        one(g.ln.z, g.lo.z, g.v.z, g.h.z, g.a.z, g.r.z, m, is, acc); one(g.ln.w, g.lo.w, g.v.w, g.h.w, g.a.w, g.r.w, m, is, acc);
    }
    __device__ void add1(long long i, double* acc) const
    {
        const double m = normalize ? g_adv_stats[0] : 0.0, is = normalize ? g_adv_stats[1] : 1.0;
        one(logp_new[i], logp_old[i], values[i], entropy[i], adv[i], returns[i], m, is, acc);
    }
    __device__ void finish(const double* tot, long long count) const
    {
        const double inv = 1.0 / (double)count;
        for (int k = 0; k < 4; ++k) out[k] = (float)(tot[k] * inv);
    }
};

}  // namespace
}  // namespace hts

extern "C" hts_status hts_a2c_terms(const float* logp, const float* values, const float* entropy, const float* returns,
                                    int64_t count, float* out3, void* cuda_stream)
{
    using namespace hts;
    if (!logp || !values || !entropy || !returns || !out3 || count < 1) return HTS_ERR_INVALID_ARG;
    const A2cOp op{logp, values, entropy, returns, out3, all_aligned16({logp, values, entropy, returns})};
    return launch_sums(op, (long long)count, static_cast<cudaStream_t>(cuda_stream), "a2c_terms");
}

extern "C" hts_status hts_ppo_terms(const float* logp_new, const float* logp_old, const float* values, const float* entropy,
                                    const float* advantages, const float* returns, int64_t count, float clip,
                                    int32_t normalize_advantages, float* out4, void* cuda_stream)
{
    using namespace hts;
    if (!logp_new || !logp_old || !values || !entropy || !advantages || !returns || !out4 || count < 1) return HTS_ERR_INVALID_ARG;
    if (!(clip > 0.f) || std::isinf(clip)) return HTS_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (normalize_advantages) {
        const bool av = all_aligned16({advantages});
        hts_status st = launch_sums(AdvMeanOp{advantages, av}, (long long)count, s, "adv_mean");
        if (st != HTS_OK) return st;
        st = launch_sums(AdvVarOp{advantages, av}, (long long)count, s, "adv_var");
        if (st != HTS_OK) return st;
    }
    const PpoOp op{logp_new, logp_old, values, entropy, advantages, returns, out4, (double)clip, normalize_advantages != 0,
                   all_aligned16({logp_new, logp_old, values, entropy, advantages, returns})};
    return launch_sums(op, (long long)count, s, "ppo_terms");
}

// ---- the learner's parameter update (Section 4.1 "Delayed gradient", Eq. 5) ---------------------------------
// theta_{j+1} = theta_j + eta * d with the gradient taken (by the caller) at theta_{j-1}.  With the RMSProp
// scaling of the hyper-parameter tables (momentum 0): v <- alpha v + (1 - alpha) g^2, d = g / (sqrt(v) + eps);
// without it d = g.  Elementwise and HBM-bound: 20 bytes per parameter, 22 with the bf16 copy that the actor's
// hts_policy_load_weights takes, written in the same pass.
namespace hts {
namespace {

template <bool PRECOND>
__device__ __forceinline__ float update_one(float theta, float g, float& v, float lr, float alpha, float eps)
{
    float d = g;
    if (PRECOND) {
        v = fmaf(alpha, v, (1.0f - alpha) * g * g);
        d = g / (sqrtf(v) + eps);
    }
    return fmaf(lr, d, theta);
}

// Four parameters per thread and pass when every array is 16-byte aligned (8 for the bf16 copy).
template <bool PRECOND, bool VEC>
__global__ void __launch_bounds__(256)
delayed_update_kernel(float* __restrict__ theta, const float* __restrict__ grad, float* __restrict__ sq_avg,
                      long long count, float lr, float alpha, float eps, __nv_bfloat16* __restrict__ theta_bf16)
{
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    long long done = 0;
    if (VEC) {
        const long long quads = count >> 2;
        for (long long q = tid; q < quads; q += stride) {
            const float4 g = reinterpret_cast<const float4*>(grad)[q];
            float4 t = reinterpret_cast<float4*>(theta)[q];
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (PRECOND) v = reinterpret_cast<float4*>(sq_avg)[q];
            t.x = update_one<PRECOND>(t.x, g.x, v.x, lr, alpha, eps); t.y = update_one<PRECOND>(t.y, g.y, v.y, lr, alpha, eps);
            t.z = update_one<PRECOND>(t.z, g.z, v.z, lr, alpha, eps); t.w = update_one<PRECOND>(t.w, g.w, v.w, lr, alpha, eps);
            reinterpret_cast<float4*>(theta)[q] = t;
            if (PRECOND) reinterpret_cast<float4*>(sq_avg)[q] = v;
            if (theta_bf16) {
                __nv_bfloat162 lo = __floats2bfloat162_rn(t.x, t.y), hi = __floats2bfloat162_rn(t.z, t.w);
                reinterpret_cast<uint2*>(theta_bf16)[q] = make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
            }
        }
        done = quads << 2;
    }
    for (long long i = done + tid; i < count; i += stride) {
        float v = PRECOND ? sq_avg[i] : 0.f;
        const float t = update_one<PRECOND>(theta[i], grad[i], v, lr, alpha, eps);
        theta[i] = t;
        if (PRECOND) sq_avg[i] = v;
        if (theta_bf16) theta_bf16[i] = __float2bfloat16_rn(t);
    }
}

}  // namespace
}  // namespace hts

extern "C" hts_status hts_delayed_update(float* theta, const float* grad, float* sq_avg_or_null, int64_t count,
                                         float lr, float alpha, float eps, void* theta_bf16_or_null, void* cuda_stream)
{
    using namespace hts;
    if (!theta || !grad || count < 1) return HTS_ERR_INVALID_ARG;
    if (!(lr == lr) || std::isinf(lr)) return HTS_ERR_INVALID_ARG;
    if (sq_avg_or_null && (!(alpha >= 0.f && alpha <= 1.f) || !(eps > 0.f) || std::isinf(eps))) return HTS_ERR_INVALID_ARG;
    long long blocks = (count + 256 * 4 - 1) / (256 * 4);
    const long long cap = 16LL * device_sm_count(device_slot());
    if (blocks > cap) blocks = cap;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    __nv_bfloat16* tb = static_cast<__nv_bfloat16*>(theta_bf16_or_null);
    const bool vec = (((uintptr_t)theta | (uintptr_t)grad | (uintptr_t)sq_avg_or_null) & 15u) == 0 && ((uintptr_t)tb & 7u) == 0;
    const unsigned gb = (unsigned)blocks;
    const long long n = (long long)count;
    if (sq_avg_or_null && vec) delayed_update_kernel<true, true><<<gb, 256, 0, s>>>(theta, grad, sq_avg_or_null, n, lr, alpha, eps, tb);
    else if (sq_avg_or_null) delayed_update_kernel<true, false><<<gb, 256, 0, s>>>(theta, grad, sq_avg_or_null, n, lr, alpha, eps, tb);
    else if (vec) delayed_update_kernel<false, true><<<gb, 256, 0, s>>>(theta, grad, nullptr, n, lr, alpha, eps, tb);
    else delayed_update_kernel<false, false><<<gb, 256, 0, s>>>(theta, grad, nullptr, n, lr, alpha, eps, tb);
    HTS_LAUNCH_CHECK("delayed_update_kernel");
    return HTS_OK;
}
