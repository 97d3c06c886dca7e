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
template <typename TIn>
__global__ void conv_wgrad_kernel(const float* __restrict__ dy, const TIn* __restrict__ in, int n, int C, int H, int W,
                                  int O, int k, int s, int Ho, int Wo, int per_chunk, float* __restrict__ part)
{
    const int nW = O * C * k * k, total = nW + O;
    const int p = blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= total) return;
    const int i0 = blockIdx.y * per_chunk;
    int i1 = i0 + per_chunk; i1 = i1 > n ? n : i1;
    float acc = 0.f;
    if (p < nW) {
        const int v = p % k, u = (p / k) % k, c = (p / (k * k)) % C, o = p / (k * k * C);
        for (int i = i0; i < i1; ++i) {
            const float* d = dy + ((size_t)i * O + o) * Ho * Wo;
            const TIn* x = in + ((size_t)i * C + c) * H * W + (size_t)u * W + v;
            for (int y = 0; y < Ho; ++y)
                for (int xx = 0; xx < Wo; ++xx) acc = fmaf(d[y * Wo + xx], (float)x[(size_t)(y * s) * W + xx * s], acc);
        }
    } else {
        const int o = p - nW;
        for (int i = i0; i < i1; ++i) {
            const float* d = dy + ((size_t)i * O + o) * Ho * Wo;
            for (int q = 0; q < Ho * Wo; ++q) acc += d[q];
        }
    }
    part[(size_t)blockIdx.y * total + p] = acc;
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
__global__ void conv_dgrad_kernel(const float* __restrict__ dy, const float* __restrict__ w, const float* __restrict__ x,
                                  int n, int C, int H, int W, int O, int k, int s, int Ho, int Wo, float* __restrict__ dx)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)n * C * H * W) return;
    const int X = (int)(idx % W), Y = (int)((idx / W) % H), c = (int)((idx / ((size_t)W * H)) % C);
    const size_t i = idx / ((size_t)W * H * C);
    float acc = 0.f;
    if (x[idx] > 0.f) {
        for (int u = 0; u < k; ++u) {
            const int yy = Y - u;
            if (yy < 0 || yy % s) continue;
            const int y = yy / s;
            if (y >= Ho) continue;
            for (int v = 0; v < k; ++v) {
                const int xx = X - v;
                if (xx < 0 || xx % s) continue;
                const int xo = xx / s;
                if (xo >= Wo) continue;
                const float* d = dy + (i * O) * Ho * Wo + (size_t)y * Wo + xo;
                const float* ww = w + ((size_t)c * k + u) * k + v;
                for (int o = 0; o < O; ++o) acc = fmaf(d[(size_t)o * Ho * Wo], ww[(size_t)o * C * k * k], acc);
            }
        }
    }
    dx[idx] = acc;
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
        if (L.u8)
            conv_wgrad_kernel<uint8_t><<<dim3(nblk(total, 128), used), 128, 0, s>>>(
                L.dy, static_cast<const uint8_t*>(L.in), n, L.C, L.H, L.W, L.O, L.k, L.s, L.Ho, L.Wo, per_chunk, part);
        else
            conv_wgrad_kernel<float><<<dim3(nblk(total, 128), used), 128, 0, s>>>(
                L.dy, static_cast<const float*>(L.in), n, L.C, L.H, L.W, L.O, L.k, L.s, L.Ho, L.Wo, per_chunk, part);
        HTS_LAUNCH_CHECK("conv_wgrad_kernel");
        conv_wgrad_reduce_kernel<<<nblk(total, th), th, 0, s>>>(part, used, nW, L.O, L.u8 ? 1.0f / 255.0f : 1.0f, L.dW, L.db);
        HTS_LAUNCH_CHECK("conv_wgrad_reduce_kernel");
        if (L.dx) {
            conv_dgrad_kernel<<<nblk((size_t)n * L.C * L.H * L.W, th), th, 0, s>>>(L.dy, L.wt, L.x_act, n, L.C, L.H, L.W, L.O, L.k,
                                                                                  L.s, L.Ho, L.Wo, L.dx);
            HTS_LAUNCH_CHECK("conv_dgrad_kernel");
        }
    }
    return HTS_OK;
}

}  // namespace hts
