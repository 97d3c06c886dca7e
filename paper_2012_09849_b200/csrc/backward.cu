// Gradient of the learner objective with respect to the twelve parameter tensors: the quantity Eq. 4 of
// the paper estimates and Eq. 5 adds to the parameters,
//
//     J-hat = (1/n) sum_i [ S_i - value_coef (R_i - V(s_i))^2 + entropy_coef H(pi(.|s_i)) ],
//
// S_i = log pi(a_i|s_i) A_i (actor-critic; the advantage is data) or the clipped surrogate
// min(rho_i A_i, clip(rho_i, 1-clip, 1+clip) A_i), rho_i = exp(log pi(a_i|s_i) - logp_old_i) (PPO).
//
// fp32 CUDA-core kernels on the activations of the fp32 check path (NCHW), layer by layer through the network
// of Appendix F.1 / F.2.  Every sum runs in a fixed order (no atomics): weight gradients of the convolutions
// are summed per batch chunk and the chunks are then added in index order.  These kernels are written for
// correctness and a reproducible result, not tuned: they are not part of the actor's hot path.
#include "common.cuh"

namespace hts {
namespace {

constexpr int kOTile = 8;       // outputs per thread in the dense weight gradient

// d J / d logits and d J / d value of each sample.  dhead[i][0..A-1] = d/d logit_j, dhead[i][A] = d/d V.
__global__ void head_grad_kernel(const float* __restrict__ logits, const float* __restrict__ values,
                                 const int32_t* __restrict__ actions, const float* __restrict__ adv,
                                 const float* __restrict__ ret, const float* __restrict__ logp_old, float value_coef,
                                 float entropy_coef, float clip, int n, int A, int* __restrict__ status,
                                 float* __restrict__ dhead)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const float* lg = logits + (size_t)i * A;
    float* out = dhead + (size_t)i * (A + 1);
    const int a = actions[i];
    if ((unsigned)a >= (unsigned)A) {                    // not used as an index: the row contributes nothing
        if (status) atomicCAS(status, 0, kStatusBadAction);
        for (int j = 0; j <= A; ++j) out[j] = 0.f;
        return;
    }
    float m = -INFINITY;
    for (int j = 0; j < A; ++j) m = fmaxf(m, lg[j]);
    float z = 0.f;
    for (int j = 0; j < A; ++j) z += expf(lg[j] - m);
    const float lse = m + logf(z);
    float ent = 0.f;
    for (int j = 0; j < A; ++j) { const float lp = lg[j] - lse; ent -= expf(lp) * lp; }
    const float inv_n = 1.0f / (float)n;
    float ds = adv[i];                                   // d S_i / d log pi(a_i)
    if (logp_old && clip > 0.f) {
        const float rho = expf((lg[a] - lse) - logp_old[i]);
        const float clipped = fminf(fmaxf(rho, 1.f - clip), 1.f + clip);
        ds = (rho * adv[i] <= clipped * adv[i]) ? rho * adv[i] : 0.f;       // the min takes its first argument
    }
    for (int j = 0; j < A; ++j) {
        const float lp = lg[j] - lse, p = expf(lp);
        // d log pi(a) / d logit_j = [j == a] - p_j ;   d H / d logit_j = -p_j (log p_j + H)
        out[j] = (ds * ((j == a ? 1.f : 0.f) - p) - entropy_coef * p * (lp + ent)) * inv_n;
    }
    out[A] = 2.f * value_coef * (ret[i] - values[i]) * inv_n;
}

// dW[o][k] = sum_i dout[i][o] * in[i][k]   (dout [n][ldo], in [n][K]);  thread = (k, tile of kOTile outputs)
__global__ void dense_wgrad_kernel(const float* __restrict__ dout, int ldo, int O, const float* __restrict__ in, int K,
                                   int n, float* __restrict__ dW)
{
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    const int o0 = blockIdx.y * kOTile;
    if (k >= K) return;
    float acc[kOTile];
#pragma unroll
    for (int j = 0; j < kOTile; ++j) acc[j] = 0.f;
    for (int i = 0; i < n; ++i) {
        const float x = in[(size_t)i * K + k];
        const float* d = dout + (size_t)i * ldo + o0;
#pragma unroll
        for (int j = 0; j < kOTile; ++j) if (o0 + j < O) acc[j] = fmaf(d[j], x, acc[j]);
    }
#pragma unroll
    for (int j = 0; j < kOTile; ++j) if (o0 + j < O) dW[(size_t)(o0 + j) * K + k] = acc[j];
}

// db[o] = sum_i dout[i][o]
__global__ void dense_bgrad_kernel(const float* __restrict__ dout, int ldo, int O, int n, float* __restrict__ db)
{
    const int o = blockIdx.x * blockDim.x + threadIdx.x;
    if (o >= O) return;
    float acc = 0.f;
    for (int i = 0; i < n; ++i) acc += dout[(size_t)i * ldo + o];
    db[o] = acc;
}

// din[i][k] = (act[i][k] > 0) * sum_o dout[i][o] * W[o][k]     (the ReLU of the layer that produced act)
__global__ void dense_dgrad_kernel(const float* __restrict__ dout, int ldo, int O, const float* __restrict__ W, int K,
                                   const float* __restrict__ act, int n, float* __restrict__ din)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)n * K) return;
    const int k = (int)(idx % K);
    const size_t i = idx / K;
    float acc = 0.f;
    if (act[idx] > 0.f) {
        const float* d = dout + i * ldo;
        for (int o = 0; o < O; ++o) acc = fmaf(d[o], W[(size_t)o * K + k], acc);
    }
    din[idx] = acc;
}

// Partial weight and bias gradients of a convolution over one chunk of the batch:
//   part[chunk][p]  p < O C k k : sum_{i in chunk, y, x} dy[i][o][y][x] * in[i][c][y s + u][x s + v]
//                   p >= O C k k: bias o = p - O C k k : sum dy[i][o][y][x]
// A thread owns one (c, u, v) and kWgradOB output channels: one input load feeds that many independent
// accumulators (the dy loads are the same address across most of a warp).  Each element is still summed over
// (i, y, x) in ascending order.
constexpr int kWgradOB = 8;
template <typename TIn>
__global__ void conv_wgrad_kernel(const float* __restrict__ dy, const TIn* __restrict__ in, int n, int C, int H, int W,
                                  int O, int k, int s, int Ho, int Wo, int per_chunk, float* __restrict__ part)
{
    const int per_o = C * k * k, nW = O * per_o, total = nW + O;
    const int nT = nW / kWgradOB;                      // threads that own weights; O more own one bias each
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= nT + O) return;
    const int i0 = blockIdx.y * per_chunk;
    int i1 = i0 + per_chunk; i1 = i1 > n ? n : i1;
    float* out = part + (size_t)blockIdx.y * total;
    const size_t plane = (size_t)Ho * Wo;
    if (q < nT) {
        const int r = q % per_o, o0 = (q / per_o) * kWgradOB;
        const int v = r % k, u = (r / k) % k, c = r / (k * k);
        float acc[kWgradOB];
#pragma unroll
        for (int j = 0; j < kWgradOB; ++j) acc[j] = 0.f;
        for (int i = i0; i < i1; ++i) {
            const float* d = dy + ((size_t)i * O + o0) * plane;
            const TIn* x = in + ((size_t)i * C + c) * H * W + (size_t)u * W + v;
            for (int y = 0; y < Ho; ++y)
                for (int xx = 0; xx < Wo; ++xx) {
                    const float xv = (float)x[(size_t)(y * s) * W + xx * s];
#pragma unroll
                    for (int j = 0; j < kWgradOB; ++j) acc[j] = fmaf(d[j * plane + y * Wo + xx], xv, acc[j]);
                }
        }
#pragma unroll
        for (int j = 0; j < kWgradOB; ++j) out[(size_t)(o0 + j) * per_o + r] = acc[j];
    } else {
        const int o = q - nT;
        float acc = 0.f;
        for (int i = i0; i < i1; ++i) {
            const float* d = dy + ((size_t)i * O + o) * plane;
            for (int t = 0; t < Ho * Wo; ++t) acc += d[t];
        }
        out[nW + o] = acc;
    }
}

// dW / db = in_scale * (chunk partials added in index order)
__global__ void conv_wgrad_reduce_kernel(const float* __restrict__ part, int chunks, int nW, int O, float in_scale,
                                         float* __restrict__ dW, float* __restrict__ db)
{
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    const int total = nW + O;
    if (p >= total) return;
    float acc = 0.f;
    for (int b = 0; b < chunks; ++b) acc += part[(size_t)b * total + p];
    if (p < nW) dW[p] = acc * in_scale; else db[p - nW] = acc;
}

// dx[i][c][Y][X] = (x[i][c][Y][X] > 0) * sum_{o,u,v : Y = y s + u, X = x s + v} dy[i][o][y][x] * w[o][c][u][v]
// A thread owns one input position and kDgradCB channels: every dy value it loads feeds that many independent
// accumulators, and the block's slice of the filter sits in shared memory as [u][v][o][channel], so the inner loop
// is one global load and two shared 16-byte loads per eight multiply-adds.  Taps are visited in ascending (u, v),
// outputs in ascending o: the order of the sum of one element does not depend on the blocking.
constexpr int kDgradCB = 8;
__global__ void __launch_bounds__(256)
conv_dgrad_kernel(const float* __restrict__ dy, const float* __restrict__ w, const float* __restrict__ x,
                  int n, int C, int H, int W, int O, int k, int s, int Ho, int Wo, float* __restrict__ dx)
{
    extern __shared__ float4 s_w4[];                   // [k*k][O][kDgradCB]
    float* s_w = reinterpret_cast<float*>(s_w4);
    const int c0 = blockIdx.y * kDgradCB;
    for (int idx = threadIdx.x; idx < k * k * O * kDgradCB; idx += blockDim.x) {
        const int cc = idx % kDgradCB, o = (idx / kDgradCB) % O, t = idx / (kDgradCB * O);
        const int c = c0 + cc;
        s_w[idx] = c < C ? w[((size_t)o * C + c) * k * k + t] : 0.f;
    }
    __syncthreads();
    const size_t pos = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (pos >= (size_t)n * H * W) return;
    const int X = (int)(pos % W), Y = (int)((pos / W) % H);
    const size_t i = pos / ((size_t)W * H);
    float acc[kDgradCB];
#pragma unroll
    for (int cc = 0; cc < kDgradCB; ++cc) acc[cc] = 0.f;
    const size_t plane = (size_t)Ho * Wo;
    for (int u = Y % s; u < k && u <= Y; u += s) {
        const int y = (Y - u) / s;
        if (y >= Ho) continue;
        for (int v = X % s; v < k && v <= X; v += s) {
            const int xo = (X - v) / s;
            if (xo >= Wo) continue;
            const float* d = dy + i * O * plane + (size_t)y * Wo + xo;
            const float4* wp = s_w4 + (size_t)(u * k + v) * O * (kDgradCB / 4);
#pragma unroll 4
            for (int o = 0; o < O; ++o) {
                const float dv = d[(size_t)o * plane];
                const float4 w0 = wp[2 * o], w1 = wp[2 * o + 1];
                acc[0] = fmaf(dv, w0.x, acc[0]); acc[1] = fmaf(dv, w0.y, acc[1]);
                acc[2] = fmaf(dv, w0.z, acc[2]); acc[3] = fmaf(dv, w0.w, acc[3]);
                acc[4] = fmaf(dv, w1.x, acc[4]); acc[5] = fmaf(dv, w1.y, acc[5]);
                acc[6] = fmaf(dv, w1.z, acc[6]); acc[7] = fmaf(dv, w1.w, acc[7]);
            }
        }
    }
#pragma unroll
    for (int cc = 0; cc < kDgradCB; ++cc) {
        const int c = c0 + cc;
        if (c < C) {
            const size_t idx = ((i * C + c) * H + Y) * W + X;
            dx[idx] = x[idx] > 0.f ? acc[cc] : 0.f;
        }
    }
}

inline unsigned nblk(size_t total, int th) { return (unsigned)((total + th - 1) / th); }

}  // namespace

size_t backward_workspace_floats(const Geometry& g, int max_batch)
{
    const size_t nb = (size_t)max_batch;
    const size_t part = (size_t)kBackwardChunks * ((size_t)64 * 64 * 9 + 64 > (size_t)32 * g.C * 64 + 32
                                                        ? (size_t)64 * 64 * 9 + 64 : (size_t)32 * g.C * 64 + 32);
    return nb * (g.A + 1) + nb * 512 + nb * g.F + nb * 64 * g.H2 * g.W2 + nb * 32 * g.H1 * g.W1 + part;
}

hts_status ref_backward(const Geometry& g, const RefWeights& w, const RefWorkspace& act, const uint8_t* obs, float* ws,
                        const float* logits, const float* values, const int32_t* actions, const float* adv,
                        const float* ret, const float* logp_old, float value_coef, float entropy_coef, float clip,
                        int n, int max_batch, int* status, const hts_grads& out, cudaStream_t s)
{
    const size_t nb = (size_t)max_batch;
    const int A = g.A, th = 256;
    float* dhead = ws;                                   // [n][A+1]
    float* dh = dhead + nb * (A + 1);                    // [n][512]
    float* da3 = dh + nb * 512;                          // [n][F]    (NCHW, as the FC sees it)
    float* da2 = da3 + nb * g.F;                         // [n][64][H2][W2]
    float* da1 = da2 + nb * 64 * g.H2 * g.W2;            // [n][32][H1][W1]
    float* part = da1 + nb * 32 * g.H1 * g.W1;           // chunk partials of one convolution's weight gradient

    head_grad_kernel<<<nblk(n, 128), 128, 0, s>>>(logits, values, actions, adv, ret, logp_old, value_coef, entropy_coef,
                                                   clip, n, A, status, dhead);
    HTS_LAUNCH_CHECK("head_grad_kernel");
    // heads: rows 0..A-1 of the stacked head are the policy, row A the value
    dense_wgrad_kernel<<<dim3(nblk(512, th), nblk(A, kOTile)), th, 0, s>>>(dhead, A + 1, A, act.h, 512, n, out.pi_w);
    HTS_LAUNCH_CHECK("dense_wgrad(pi)");
    dense_wgrad_kernel<<<dim3(nblk(512, th), 1), th, 0, s>>>(dhead + A, A + 1, 1, act.h, 512, n, out.v_w);
    HTS_LAUNCH_CHECK("dense_wgrad(v)");
    dense_bgrad_kernel<<<nblk(A, 64), 64, 0, s>>>(dhead, A + 1, A, n, out.pi_b);
    HTS_LAUNCH_CHECK("dense_bgrad(pi)");
    dense_bgrad_kernel<<<1, 64, 0, s>>>(dhead + A, A + 1, 1, n, out.v_b);
    HTS_LAUNCH_CHECK("dense_bgrad(v)");
    dense_dgrad_kernel<<<nblk((size_t)n * 512, th), th, 0, s>>>(dhead, A + 1, A + 1, w.whead, 512, act.h, n, dh);
    HTS_LAUNCH_CHECK("dense_dgrad(heads)");
    // FC
    dense_wgrad_kernel<<<dim3(nblk(g.F, th), nblk(512, kOTile)), th, 0, s>>>(dh, 512, 512, act.a3, g.F, n, out.fc_w);
    HTS_LAUNCH_CHECK("dense_wgrad(fc)");
    dense_bgrad_kernel<<<nblk(512, 64), 64, 0, s>>>(dh, 512, 512, n, out.fc_b);
    HTS_LAUNCH_CHECK("dense_bgrad(fc)");
    dense_dgrad_kernel<<<nblk((size_t)n * g.F, th), th, 0, s>>>(dh, 512, 512, w.wfc, g.F, act.a3, n, da3);
    HTS_LAUNCH_CHECK("dense_dgrad(fc)");
    // the three convolutions, last to first
    const int chunks = n < kBackwardChunks ? n : kBackwardChunks;
    const int per_chunk = (n + chunks - 1) / chunks;
    const int used = (n + per_chunk - 1) / per_chunk;
    struct Layer { const float* dy; const void* in; bool u8; int C, H, W, O, k, s, Ho, Wo; const float* wt; float *dW, *db, *dx; const float* x_act; };
    const Layer layers[3] = {
        {da3, act.a2, false, 64, g.H2, g.W2, 64, 3, 1, g.H3, g.W3, w.w3, out.conv3_w, out.conv3_b, da2, act.a2},
        {da2, act.a1, false, 32, g.H1, g.W1, 64, 4, 2, g.H2, g.W2, w.w2, out.conv2_w, out.conv2_b, da1, act.a1},
        {da1, obs, true, g.C, g.H, g.W, 32, 8, 4, g.H1, g.W1, w.w1, out.conv1_w, out.conv1_b, nullptr, nullptr}};
    for (const Layer& L : layers) {
        const int nW = L.O * L.C * L.k * L.k, total = nW + L.O;
        if (L.O % kWgradOB) return HTS_ERR_SHAPE;
        const int wthreads = nW / kWgradOB + L.O;
        if (L.u8)
            conv_wgrad_kernel<uint8_t><<<dim3(nblk(wthreads, 128), used), 128, 0, s>>>(
                L.dy, static_cast<const uint8_t*>(L.in), n, L.C, L.H, L.W, L.O, L.k, L.s, L.Ho, L.Wo, per_chunk, part);
        else
            conv_wgrad_kernel<float><<<dim3(nblk(wthreads, 128), used), 128, 0, s>>>(
                L.dy, static_cast<const float*>(L.in), n, L.C, L.H, L.W, L.O, L.k, L.s, L.Ho, L.Wo, per_chunk, part);
        HTS_LAUNCH_CHECK("conv_wgrad_kernel");
        conv_wgrad_reduce_kernel<<<nblk(total, th), th, 0, s>>>(part, used, nW, L.O, L.u8 ? 1.0f / 255.0f : 1.0f, L.dW, L.db);
        HTS_LAUNCH_CHECK("conv_wgrad_reduce_kernel");
        if (L.dx) {
            const size_t w_smem = (size_t)L.k * L.k * L.O * kDgradCB * sizeof(float);
            if (w_smem > 48 * 1024) return HTS_ERR_SHAPE;
            conv_dgrad_kernel<<<dim3(nblk((size_t)n * L.H * L.W, 256), nblk(L.C, kDgradCB)), 256, w_smem, s>>>(
                L.dy, L.wt, L.x_act, n, L.C, L.H, L.W, L.O, L.k, L.s, L.Ho, L.Wo, L.dx);
            HTS_LAUNCH_CHECK("conv_dgrad_kernel");
        }
    }
    return HTS_OK;
}

}  // namespace hts
