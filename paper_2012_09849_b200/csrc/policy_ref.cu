// fp32 CUDA-core path of the actor step: the check path (fp32 weights) of the policy-value
// network of Appendix F.1 / F.2.  Direct convolution and dot products with fp32 FMAs and a
// fixed summation order per output, so a row's result does not depend on the batch around it.
#include <type_traits>
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
// A thread owns one output position and kConvOB output channels (O is a multiple of it): one input load feeds that
// many accumulators, and the weight loads are one address per warp.  Every output is summed over (c, u, v) in
// ascending order, whatever kConvOB: small batches take one channel per thread (more threads), large ones eight.
template <typename TIn, int kConvOB>
__global__ void conv_direct_kernel(const TIn* __restrict__ x, const float* __restrict__ w,
                                   const float* __restrict__ b, float* __restrict__ y,
                                   int n, int C, int H, int W, int O, int k, int s, int Ho, int Wo,
                                   float in_scale, const int32_t* __restrict__ slots, int pool, int* __restrict__ status)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int OBn = O / kConvOB;
    const size_t total = (size_t)n * OBn * Ho * Wo;
    if (idx >= total) return;
    const int j = (int)(idx % Wo);
    const int i = (int)((idx / Wo) % Ho);
    const int o0 = (int)((idx / ((size_t)Wo * Ho)) % OBn) * kConvOB;
    const size_t e = idx / ((size_t)Wo * Ho * OBn);
    size_t frame = e;                                   // dense, or the row's frame of the state buffer
    if (slots) {
        const int sl = slots[e];
        if ((unsigned)sl >= (unsigned)pool) { atomicCAS(status, 0, kStatusBadSlot); frame = 0; }
        else frame = (size_t)sl;
    }
    const TIn* xe = x + frame * (size_t)C * H * W;
    const size_t per_o = (size_t)C * k * k;
    const float* wo = w + (size_t)o0 * per_o;
    float acc[kConvOB];
#pragma unroll
    for (int q = 0; q < kConvOB; ++q) acc[q] = 0.f;
    for (int c = 0; c < C; ++c)
        for (int u = 0; u < k; ++u) {
            const TIn* xr = xe + ((size_t)c * H + (i * s + u)) * W + j * s;
            const float* wr = wo + (c * k + u) * k;
            for (int v = 0; v < k; ++v) {
                const float xv = (float)xr[v];
#pragma unroll
                for (int q = 0; q < kConvOB; ++q) acc[q] = fmaf(wr[q * per_o + v], xv, acc[q]);
            }
        }
#pragma unroll
    for (int q = 0; q < kConvOB; ++q) {
        const float a = fmaf(acc[q], in_scale, b[o0 + q]);
        y[((e * O + o0 + q) * Ho + i) * Wo + j] = a > 0.f ? a : 0.f;
    }
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
                       const uint8_t* obs, const Indexing& ix, int* status, int n, Profiler& prof, cudaStream_t s)
{
    const int th = 256;
    auto conv = [&](auto* x, const float* wt, const float* b, float* y, int C, int H, int W, int O, int k, int st,
                    int Ho, int Wo, float scale, const int32_t* slots, int pool, int* stat) {
        using TIn = std::remove_cv_t<std::remove_pointer_t<decltype(x)>>;
        const size_t outputs = (size_t)n * O * Ho * Wo;
        if (outputs >= (size_t)8 * 2048 * 148)           // a thread for every eight outputs still fills the device
            conv_direct_kernel<TIn, 8><<<blocks_for(outputs / 8, th), th, 0, s>>>(x, wt, b, y, n, C, H, W, O, k, st, Ho, Wo,
                                                                               scale, slots, pool, stat);
        else
            conv_direct_kernel<TIn, 1><<<blocks_for(outputs, th), th, 0, s>>>(x, wt, b, y, n, C, H, W, O, k, st, Ho, Wo,
                                                                            scale, slots, pool, stat);
    };
    prof.begin(K_CONV1, s);
    conv(obs, w.w1, w.b1, ws.a1, g.C, g.H, g.W, 32, 8, 4, g.H1, g.W1, 1.0f / 255.0f, ix.slots, ix.pool, status);
    HTS_LAUNCH_CHECK("conv1_direct");
    prof.end(K_CONV1, s);
    prof.begin(K_CONV2, s);
    conv(static_cast<const float*>(ws.a1), w.w2, w.b2, ws.a2, 32, g.H1, g.W1, 64, 4, 2, g.H2, g.W2, 1.0f, nullptr, 0, nullptr);
    HTS_LAUNCH_CHECK("conv2_direct");
    prof.end(K_CONV2, s);
    prof.begin(K_CONV3, s);
    conv(static_cast<const float*>(ws.a2), w.w3, w.b3, ws.a3, 64, g.H2, g.W2, 64, 3, 1, g.H3, g.W3, 1.0f, nullptr, 0, nullptr);
    HTS_LAUNCH_CHECK("conv3_direct");
    prof.end(K_CONV3, s);
    prof.begin(K_FC, s);
    fc_warp_kernel<<<blocks_for((size_t)n * 512 * 32, th), th, 0, s>>>(ws.a3, w.wfc, w.bfc, ws.h, n, g.F, 512);
    HTS_LAUNCH_CHECK("fc_warp");
    prof.end(K_FC, s);
    return HTS_OK;
}

}  // namespace hts

// ---- actor step that allocates nothing ----------------------------------------------------------
// Scratch for hts_policy_step_noalloc: hidden activations of the four layers plus the stacked
// head weights, as floats.  It lives in the library image, so every GPU that loads the library
// carries these 4 MiB until the process exits.
namespace {
constexpr size_t kNoAllocFloats = size_t(1) << 20;
static __device__ __align__(256) float g_noalloc_scratch[kNoAllocFloats];
constexpr int kMaxDevices = 64;
float* g_noalloc_ptr[kMaxDevices] = {};       // device address of the array, looked up once per device
}  // namespace

extern "C" hts_status hts_policy_step_noalloc(const hts_net_desc* d, const hts_weights* w, const uint8_t* obs,
                                              const int32_t* env_ids, const int32_t* t_per_env, int32_t t,
                                              uint64_t seed, int32_t n, int32_t* actions, float* logp,
                                              float* values, float* entropy, float* logits_or_null,
                                              void* cuda_stream)
{
    using namespace hts;
    if (!d || !w || !obs || !env_ids || !actions || !logp || !values || !entropy) return HTS_ERR_INVALID_ARG;
    const void* const* wp = reinterpret_cast<const void* const*>(w);
    for (int i = 0; i < 12; ++i) if (!wp[i]) return HTS_ERR_INVALID_ARG;
    if (d->weight_dtype != HTS_DTYPE_FP32) return HTS_ERR_UNSUPPORTED;
    if (n < 1 || d->C < 1 || d->num_actions < 1 || d->num_actions > 64) return HTS_ERR_INVALID_ARG;
    if (d->H % 4 || d->W % 4 || d->H < 8 || d->W < 8) return HTS_ERR_SHAPE;
    Geometry g{};
    g.C = d->C; g.H = d->H; g.W = d->W; g.A = d->num_actions;
    g.H1 = conv_out(g.H, 8, 4); g.W1 = conv_out(g.W, 8, 4);
    if (g.H1 < 4 || g.W1 < 4) return HTS_ERR_SHAPE;
    g.H2 = conv_out(g.H1, 4, 2); g.W2 = conv_out(g.W1, 4, 2);
    if (g.H2 < 3 || g.W2 < 3) return HTS_ERR_SHAPE;
    g.H3 = conv_out(g.H2, 3, 1); g.W3 = conv_out(g.W2, 3, 1);
    g.F = 64 * g.H3 * g.W3;
    const size_t nn = (size_t)n;
    const size_t f_a1 = nn * 32 * g.H1 * g.W1, f_a2 = nn * 64 * g.H2 * g.W2, f_a3 = nn * g.F, f_h = nn * 512;
    const size_t f_wh = (size_t)(g.A + 1) * 512, f_bh = (size_t)g.A + 1;
    if (f_a1 + f_a2 + f_a3 + f_h + f_wh + f_bh > kNoAllocFloats) return HTS_ERR_INVALID_ARG;   // batch too large for the fixed scratch

    int dev = 0;
    HTS_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return HTS_ERR_UNSUPPORTED;
    if (!g_noalloc_ptr[dev]) {
        // In host code the array's name is only a handle: the kernels need its device address.
        float* ptr = nullptr;
        HTS_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch));
        g_noalloc_ptr[dev] = ptr;
    }
    float* base = g_noalloc_ptr[dev];
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    RefWorkspace ws{base, base + f_a1, base + f_a1 + f_a2, base + f_a1 + f_a2 + f_a3};
    float* whead = ws.h + f_h;
    float* bhead = whead + f_wh;
    // every scratch float is written before it is read, so nothing has to start at zero
    HTS_CUDA(cudaMemcpyAsync(whead, w->pi_w, (size_t)g.A * 512 * sizeof(float), cudaMemcpyDeviceToDevice, s));
    HTS_CUDA(cudaMemcpyAsync(whead + (size_t)g.A * 512, w->v_w, 512 * sizeof(float), cudaMemcpyDeviceToDevice, s));
    HTS_CUDA(cudaMemcpyAsync(bhead, w->pi_b, (size_t)g.A * sizeof(float), cudaMemcpyDeviceToDevice, s));
    HTS_CUDA(cudaMemcpyAsync(bhead + g.A, w->v_b, sizeof(float), cudaMemcpyDeviceToDevice, s));
    auto f = [](const void* p) { return const_cast<float*>(static_cast<const float*>(p)); };
    const RefWeights rw{f(w->conv1_w), f(w->conv1_b), f(w->conv2_w), f(w->conv2_b), f(w->conv3_w), f(w->conv3_b),
                        f(w->fc_w), f(w->fc_b), whead, bhead};
    Profiler off;
    hts_status st = ref_forward(g, rw, ws, obs, Indexing{}, nullptr, n, off, s);
    if (st != HTS_OK) return st;
    return launch_heads(ws.h, 1, 0, nullptr, whead, bhead, g.A, env_ids, t_per_env, t, seed, n, Indexing{}, nullptr, actions,
                        logp, values, entropy, logits_or_null, nullptr, s);
}
