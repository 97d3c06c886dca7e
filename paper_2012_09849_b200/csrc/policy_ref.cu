// fp32 CUDA-core path of the actor step: the check path (fp32 weights) of the policy-value
// network of Appendix F.1 / F.2.  Direct convolution and dot products with fp32 FMAs and a
// fixed summation order per output, so a row's result does not depend on the batch around it.
#include "common.cuh"

namespace hts {
namespace {

__global__ void to_f32_kernel(const void* __restrict__ src, int dtype, float* __restrict__ dst, size_t count)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= count) return;
    dst[i] = (dtype == HTS_DTYPE_FP32) ? static_cast<const float*>(src)[i]
                                       : __bfloat162float(static_cast<const __nv_bfloat16*>(src)[i]);
}

// y[e,o,i,j] = relu(b[o] + sum_{c,u,v} w[o,c,u,v] * x[e,c,i*s+u,j*s+v]);  x is u8/255 or fp32.
template <typename TIn>
__global__ void conv_direct_kernel(const TIn* __restrict__ x, const float* __restrict__ w,
                                   const float* __restrict__ b, float* __restrict__ y,
                                   int n, int C, int H, int W, int O, int k, int s, int Ho, int Wo,
                                   float in_scale)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t total = (size_t)n * O * Ho * Wo;
    if (idx >= total) return;
    const int j = (int)(idx % Wo);
    const int i = (int)((idx / Wo) % Ho);
    const int o = (int)((idx / ((size_t)Wo * Ho)) % O);
    const size_t e = idx / ((size_t)Wo * Ho * O);
    const TIn* xe = x + e * (size_t)C * H * W;
    const float* wo = w + (size_t)o * C * k * k;
    float acc = 0.f;
    for (int c = 0; c < C; ++c)
        for (int u = 0; u < k; ++u) {
            const TIn* xr = xe + ((size_t)c * H + (i * s + u)) * W + j * s;
            const float* wr = wo + (c * k + u) * k;
            for (int v = 0; v < k; ++v) acc = fmaf(wr[v], (float)xr[v], acc);
        }
    acc = fmaf(acc, in_scale, b[o]);
    y[idx] = acc > 0.f ? acc : 0.f;
}

// One warp per (env, output): h[e,o] = relu(b[o] + w[o,:] . x[e,:]); fixed lane-strided order.
__global__ void fc_warp_kernel(const float* __restrict__ x, const float* __restrict__ w,
                               const float* __restrict__ b, float* __restrict__ h, int n, int F, int O)
{
    const size_t warp = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= (size_t)n * O) return;
    const int o = (int)(warp % O);
    const size_t e = warp / O;
    const float* xe = x + e * F;
    const float* wo = w + (size_t)o * F;
    float acc = 0.f;
    for (int f = lane; f < F; f += 32) acc = fmaf(wo[f], xe[f], acc);
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
    if (lane == 0) { acc += b[o]; h[warp] = acc > 0.f ? acc : 0.f; }
}

inline unsigned blocks_for(size_t total, int threads) { return (unsigned)((total + threads - 1) / threads); }

}  // namespace

hts_status ref_convert_weights(const Geometry& g, int dtype, const hts_weights& src,
                               const RefWeights& dst, cudaStream_t s)
{
    struct Item { const void* p; float* q; size_t n; };
    const Item items[] = {
        {src.conv1_w, dst.w1, (size_t)32 * g.C * 64}, {src.conv1_b, dst.b1, 32},
        {src.conv2_w, dst.w2, (size_t)64 * 32 * 16},  {src.conv2_b, dst.b2, 64},
        {src.conv3_w, dst.w3, (size_t)64 * 64 * 9},   {src.conv3_b, dst.b3, 64},
        {src.fc_w, dst.wfc, (size_t)512 * g.F},       {src.fc_b, dst.bfc, 512},
        {src.pi_w, dst.whead, (size_t)g.A * 512},     {src.pi_b, dst.bhead, (size_t)g.A},
        {src.v_w, dst.whead + (size_t)g.A * 512, 512}, {src.v_b, dst.bhead + g.A, 1},
    };
    for (const Item& it : items) {
        to_f32_kernel<<<blocks_for(it.n, 256), 256, 0, s>>>(it.p, dtype, it.q, it.n);
        HTS_LAUNCH_CHECK("to_f32_kernel");
    }
    return HTS_OK;
}

hts_status ref_forward(const Geometry& g, const RefWeights& w, const RefWorkspace& ws,
                       const uint8_t* obs, int n, Profiler& prof, cudaStream_t s)
{
    const int th = 256;
    prof.begin(K_CONV1, s);
    conv_direct_kernel<uint8_t><<<blocks_for((size_t)n * 32 * g.H1 * g.W1, th), th, 0, s>>>(
        obs, w.w1, w.b1, ws.a1, n, g.C, g.H, g.W, 32, 8, 4, g.H1, g.W1, 1.0f / 255.0f);
    HTS_LAUNCH_CHECK("conv1_direct");
    prof.end(K_CONV1, s);
    prof.begin(K_CONV2, s);
    conv_direct_kernel<float><<<blocks_for((size_t)n * 64 * g.H2 * g.W2, th), th, 0, s>>>(
        ws.a1, w.w2, w.b2, ws.a2, n, 32, g.H1, g.W1, 64, 4, 2, g.H2, g.W2, 1.0f);
    HTS_LAUNCH_CHECK("conv2_direct");
    prof.end(K_CONV2, s);
    prof.begin(K_CONV3, s);
    conv_direct_kernel<float><<<blocks_for((size_t)n * 64 * g.H3 * g.W3, th), th, 0, s>>>(
        ws.a2, w.w3, w.b3, ws.a3, n, 64, g.H2, g.W2, 64, 3, 1, g.H3, g.W3, 1.0f);
    HTS_LAUNCH_CHECK("conv3_direct");
    prof.end(K_CONV3, s);
    prof.begin(K_FC, s);
    fc_warp_kernel<<<blocks_for((size_t)n * 512 * 32, th), th, 0, s>>>(ws.a3, w.wfc, w.bfc, ws.h, n, g.F, 512);
    HTS_LAUNCH_CHECK("fc_warp");
    prof.end(K_FC, s);
    return HTS_OK;
}

}  // namespace hts
