// The three sample means of the actor-critic update (Section 3): the policy term of Eq. 4,
// (1/|D|) sum log pi(a|s) (R - V), the value loss J_V = (1/|D|) sum (R - V)^2 and the mean entropy.
//
// HBM-bound (16 bytes per transition).  Each block sums a contiguous range in double precision in a
// fixed order (thread-strided float4 loads, shuffle tree, warp order), writes its partial and takes a
// ticket; the block that draws the last ticket adds the partials in block order.  The grid is a
// function of the count alone, so the result does not depend on timing or on the device's load.
#include <cmath>
#include "common.cuh"

namespace hts {
namespace {

constexpr int kBlocksMax = 2048;
constexpr int kThreads = 256;
constexpr int kPerThread = 8;             // elements a thread covers before another block is worth its launch

// Partials and the ticket counter live in the library image: calls on one device must not overlap.
__device__ double g_partial[kBlocksMax][3];
__device__ unsigned int g_ticket;

__device__ __forceinline__ double warp_sum_d(double v)
{
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
    return v;
}

__global__ void __launch_bounds__(kThreads)
a2c_terms_kernel(const float* __restrict__ logp, const float* __restrict__ values, const float* __restrict__ entropy,
                 const float* __restrict__ returns, long long count, long long per_block, float* __restrict__ out)
{
    __shared__ double s_part[kThreads / 32][3];
    __shared__ bool s_last;
    const long long lo = (long long)blockIdx.x * per_block;               // per_block is a multiple of 4
    long long hi = lo + per_block; hi = hi > count ? count : hi;
    double pol = 0.0, vl = 0.0, ent = 0.0;
    const bool vec = (((uintptr_t)logp | (uintptr_t)values | (uintptr_t)entropy | (uintptr_t)returns) & 15u) == 0;
    if (vec) {
        const long long q_lo = lo >> 2, q_hi = hi >> 2;                    // whole float4 groups of the range
        const float4* l4 = reinterpret_cast<const float4*>(logp);
        const float4* v4 = reinterpret_cast<const float4*>(values);
        const float4* h4 = reinterpret_cast<const float4*>(entropy);
        const float4* r4 = reinterpret_cast<const float4*>(returns);
        auto add = [&](const float4& l, const float4& v, const float4& h, const float4& r) {
            const double a0 = (double)r.x - v.x, a1 = (double)r.y - v.y, a2 = (double)r.z - v.z, a3 = (double)r.w - v.w;
            pol += (double)l.x * a0; pol += (double)l.y * a1; pol += (double)l.z * a2; pol += (double)l.w * a3;
            vl += a0 * a0; vl += a1 * a1; vl += a2 * a2; vl += a3 * a3;
            ent += (double)h.x; ent += (double)h.y; ent += (double)h.z; ent += (double)h.w;
        };
        long long q = q_lo + threadIdx.x;
        for (; q + 3 * kThreads < q_hi; q += 4 * kThreads) {               // sixteen loads in flight per thread
            float4 l[4], v[4], h[4], r[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) { l[u] = l4[q + u * kThreads]; v[u] = v4[q + u * kThreads]; h[u] = h4[q + u * kThreads]; r[u] = r4[q + u * kThreads]; }
#pragma unroll
            for (int u = 0; u < 4; ++u) add(l[u], v[u], h[u], r[u]);
        }
        for (; q < q_hi; q += kThreads) add(l4[q], v4[q], h4[q], r4[q]);
        for (long long i = (q_hi << 2) + threadIdx.x; i < hi; i += kThreads) {   // the last block's ragged tail
            const double a = (double)returns[i] - values[i];
            pol += (double)logp[i] * a; vl += a * a; ent += (double)entropy[i];
        }
    } else {
        for (long long i = lo + threadIdx.x; i < hi; i += kThreads) {
            const double a = (double)returns[i] - values[i];
            pol += (double)logp[i] * a; vl += a * a; ent += (double)entropy[i];
        }
    }
    pol = warp_sum_d(pol); vl = warp_sum_d(vl); ent = warp_sum_d(ent);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { s_part[warp][0] = pol; s_part[warp][1] = vl; s_part[warp][2] = ent; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, b = 0.0, c = 0.0;
        for (int w = 0; w < kThreads / 32; ++w) { a += s_part[w][0]; b += s_part[w][1]; c += s_part[w][2]; }
        g_partial[blockIdx.x][0] = a; g_partial[blockIdx.x][1] = b; g_partial[blockIdx.x][2] = c;
        __threadfence();
        s_last = atomicAdd(&g_ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (s_last && threadIdx.x < 32) {
        // lane l adds partials l, l + 32, ... in that order, then the lanes are folded by a shuffle tree: an order
        // fixed by the grid size, whatever the arrival order of the blocks
        __threadfence();
        double a = 0.0, b = 0.0, c = 0.0;
        for (unsigned k = threadIdx.x; k < gridDim.x; k += 32) {
            a += *(volatile double*)&g_partial[k][0]; b += *(volatile double*)&g_partial[k][1]; c += *(volatile double*)&g_partial[k][2];
        }
        a = warp_sum_d(a); b = warp_sum_d(b); c = warp_sum_d(c);
        if (threadIdx.x == 0) {
            const double inv = 1.0 / (double)count;
            out[0] = (float)(a * inv); out[1] = (float)(b * inv); out[2] = (float)(c * inv);
            g_ticket = 0;                                                    // ready for the next call
        }
    }
}

}  // namespace
}  // namespace hts

extern "C" hts_status hts_a2c_terms(const float* logp, const float* values, const float* entropy, const float* returns,
                                    int64_t count, float* out3, void* cuda_stream)
{
    using namespace hts;
    if (!logp || !values || !entropy || !returns || !out3 || count < 1) return HTS_ERR_INVALID_ARG;
    long long blocks = (count + (long long)kThreads * kPerThread - 1) / ((long long)kThreads * kPerThread);
    if (blocks > kBlocksMax) blocks = kBlocksMax;
    long long per_block = (count + blocks - 1) / blocks;
    per_block = (per_block + 3) / 4 * 4;
    blocks = (count + per_block - 1) / per_block;
    a2c_terms_kernel<<<(unsigned)blocks, kThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        logp, values, entropy, returns, (long long)count, per_block, out3);
    HTS_LAUNCH_CHECK("a2c_terms_kernel");
    return HTS_OK;
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
