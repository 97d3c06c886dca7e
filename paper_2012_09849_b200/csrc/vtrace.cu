// V-trace targets and truncated-importance-sampling advantages over the [T,N] rollout storage: the off-policy
// correction of the systems the paper measures its delayed gradient against (Section 2: IMPALA; Appendix C,
// Table A1: "Truncated I.S."), defined in Espeholt et al. 2018 (Section 4.1, Eq. 1; Section 4.2):
//
//   rho_t = min(rho_bar, pi/mu)     c_t = lambda min(c_bar, pi/mu)     pi/mu = exp(log_rhos_t)
//   delta_t = rho_t (r_t + g_t V_{t+1} - V_t)            g_t = gamma (1 - d_t)
//   D_t = delta_t + g_t c_t D_{t+1}      vs_t = V_t + D_t      pg_t = rho_t (r_t + g_t vs_{t+1} - V_t)
//
// D is the same kind of recurrence as the advantage scan (an affine map per row, with a per-element
// coefficient g_t c_t), so the kernel has the same shape: time is cut into chunks of L rows, a thread owns
// VEC adjacent columns of one chunk, loads its rows once (coalesced across env), reduces the chunk to one
// affine map, the block chains the chunk maps through shared memory, and each thread replays its chunk with
// the true incoming D.  One pass over HBM: 21 bytes per element.
#include "common.cuh"

namespace hts {
namespace {

template <int VEC> struct VecT;
template <> struct VecT<1> { using F = float;  using B = uint8_t; };
template <> struct VecT<4> { using F = float4; using B = uchar4;  };

template <int VEC> __device__ __forceinline__ void unpack(const typename VecT<VEC>::F& v, float* o);
template <> __device__ __forceinline__ void unpack<1>(const float& v, float* o) { o[0] = v; }
template <> __device__ __forceinline__ void unpack<4>(const float4& v, float* o) { o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w; }
template <int VEC> __device__ __forceinline__ void unpackb(const typename VecT<VEC>::B& v, float* live);
template <> __device__ __forceinline__ void unpackb<1>(const uint8_t& v, float* l) { l[0] = v ? 0.f : 1.f; }
template <> __device__ __forceinline__ void unpackb<4>(const uchar4& v, float* l) {
    l[0] = v.x ? 0.f : 1.f; l[1] = v.y ? 0.f : 1.f; l[2] = v.z ? 0.f : 1.f; l[3] = v.w ? 0.f : 1.f;
}
template <int VEC> __device__ __forceinline__ typename VecT<VEC>::F pack(const float* o);
template <> __device__ __forceinline__ float pack<1>(const float* o) { return o[0]; }
template <> __device__ __forceinline__ float4 pack<4>(const float* o) { return make_float4(o[0], o[1], o[2], o[3]); }

struct VtraceParams {
    const float *log_rhos, *rewards, *values, *bootstrap;
    const uint8_t* dones;
    float gamma, lambda, rho_bar, c_bar;
    int T, N;
    float *vs, *pg;
};

// blockDim = (32, W).  Block b owns columns [b*32*VEC, (b+1)*32*VEC).  Time is walked from the end in
// super-chunks of W*L rows; warp w owns rows [t0 + w*L, t0 + (w+1)*L) of the super-chunk.
template <int VEC, int L>
__global__ void __launch_bounds__(VEC == 4 ? 512 : 1024)
vtrace_scan_kernel(const VtraceParams p)
{
    using F = typename VecT<VEC>::F;
    using B = typename VecT<VEC>::B;
    extern __shared__ float smem[];                  // [W][32*VEC] S, then P, then V and vs of each chunk's first row
    const int W = blockDim.y;
    const int w = threadIdx.y;
    const int lane = threadIdx.x;
    const int cols = 32 * VEC;
    const int T = p.T, N = p.N;
    const long col = (long)blockIdx.x * cols + lane * VEC;
    const bool col_ok = col < N;                     // N % VEC == 0 is guaranteed by the launcher
    float* sS = smem;
    float* sP = smem + W * cols;

    float carry_in[VEC];                             // D at the first row after this super-chunk
#pragma unroll
    for (int k = 0; k < VEC; ++k) carry_in[k] = 0.f;

    const int span = W * L;
    const int nsuper = (T + span - 1) / span;
    for (int sc = nsuper - 1; sc >= 0; --sc) {
        const int t_begin = sc * span + w * L;       // first row of my chunk
        int rows = T - t_begin; rows = rows > L ? L : rows;   // may be <= 0 in the last super-chunk
        float delta[L][VEC], val[L][VEC], coef[L][VEC], rhog[L][VEC];    // rhog = rho_t g_t
        float S[VEC], P[VEC];
#pragma unroll
        for (int k = 0; k < VEC; ++k) { S[k] = 0.f; P[k] = 1.f; }
        if (col_ok && rows > 0) {
            F r_raw[L], v_raw[L], l_raw[L], vnext_raw; B d_raw[L];
#pragma unroll
            for (int i = 0; i < L; ++i) {
                if (i < rows) {
                    const size_t off = (size_t)(t_begin + i) * N + col;
                    r_raw[i] = *reinterpret_cast<const F*>(p.rewards + off);
                    v_raw[i] = *reinterpret_cast<const F*>(p.values + off);
                    l_raw[i] = *reinterpret_cast<const F*>(p.log_rhos + off);
                    d_raw[i] = *reinterpret_cast<const B*>(p.dones + off);
                }
            }
            const int t_after = t_begin + rows;      // row that supplies V_{t+1} of my last row
            vnext_raw = (t_after < T) ? *reinterpret_cast<const F*>(p.values + (size_t)t_after * N + col)
                                      : *reinterpret_cast<const F*>(p.bootstrap + col);
            float vnext[VEC];
            unpack<VEC>(vnext_raw, vnext);
#pragma unroll
            for (int i = L - 1; i >= 0; --i) {
                if (i < rows) {
                    float live[VEC], lr[VEC], rew[VEC];
                    unpack<VEC>(r_raw[i], rew);
                    unpack<VEC>(v_raw[i], val[i]);
                    unpack<VEC>(l_raw[i], lr);
                    unpackb<VEC>(d_raw[i], live);
#pragma unroll
                    for (int k = 0; k < VEC; ++k) {
                        const float ratio = expf(lr[k]);
                        const float rho = fminf(p.rho_bar, ratio);
                        const float g = p.gamma * live[k];
                        coef[i][k] = g * (p.lambda * fminf(p.c_bar, ratio));
                        rhog[i][k] = rho * g;
                        delta[i][k] = rho * (rew[k] + g * vnext[k] - val[i][k]);
                        S[k] = delta[i][k] + coef[i][k] * S[k];
                        P[k] = coef[i][k] * P[k];
                        vnext[k] = val[i][k];
                    }
                }
            }
        }
        __syncthreads();                             // previous super-chunk's readers are done
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            sS[w * cols + lane * VEC + k] = S[k];
            sP[w * cols + lane * VEC + k] = P[k];
        }
        __syncthreads();
        // chain the chunk maps from the last chunk down; pick up my own incoming D
        float c[VEC], mine[VEC];
#pragma unroll
        for (int k = 0; k < VEC; ++k) { c[k] = carry_in[k]; mine[k] = 0.f; }
        for (int ww = W - 1; ww >= 0; --ww) {
#pragma unroll
            for (int k = 0; k < VEC; ++k) {
                if (ww == w) mine[k] = c[k];
                c[k] = sS[ww * cols + lane * VEC + k] + sP[ww * cols + lane * VEC + k] * c[k];
            }
        }
#pragma unroll
        for (int k = 0; k < VEC; ++k) carry_in[k] = c[k];
        if (col_ok && rows > 0) {
            float a[VEC];                            // D of the row after the current one
#pragma unroll
            for (int k = 0; k < VEC; ++k) a[k] = mine[k];
#pragma unroll
            for (int i = L - 1; i >= 0; --i) {
                if (i < rows) {
                    float vs[VEC], pg[VEC];
#pragma unroll
                    for (int k = 0; k < VEC; ++k) {
                        // pg_t = rho_t (r_t + g_t vs_{t+1} - V_t) = delta_t + rho_t g_t D_{t+1}   (vs' = V' + D')
                        pg[k] = delta[i][k] + rhog[i][k] * a[k];
                        a[k] = delta[i][k] + coef[i][k] * a[k];
                        vs[k] = a[k] + val[i][k];
                    }
                    const size_t off = (size_t)(t_begin + i) * N + col;
                    *reinterpret_cast<F*>(p.vs + off) = pack<VEC>(vs);
                    *reinterpret_cast<F*>(p.pg + off) = pack<VEC>(pg);
                }
            }
        }
    }
}

template <int VEC, int L>
hts_status launch_t(const VtraceParams& p, cudaStream_t s)
{
    int W = (p.T + L - 1) / L;
    const int maxW = (VEC == 4) ? 2 : 32;
    if (W > maxW) W = maxW;
    const int cols = 32 * VEC;
    const unsigned blocks = (unsigned)((p.N + cols - 1) / cols);
    const size_t smem = (size_t)2 * W * cols * sizeof(float);
    vtrace_scan_kernel<VEC, L><<<blocks, dim3(32, W), smem, s>>>(p);
    HTS_LAUNCH_CHECK("vtrace_scan_kernel");
    return HTS_OK;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

hts_status launch_vtrace(const float* log_rhos, const float* rewards, const float* values, const uint8_t* dones,
                         const float* bootstrap, float gamma, float lambda, float rho_bar, float c_bar, int T, int N,
                         float* vs, float* pg, cudaStream_t s)
{
    VtraceParams p{log_rhos, rewards, values, bootstrap, dones, gamma, lambda, rho_bar, c_bar, T, N, vs, pg};
    const bool vec4 = (N % 4 == 0) && aligned(rewards, 16) && aligned(values, 16) && aligned(log_rhos, 16) &&
                      aligned(dones, 4) && aligned(bootstrap, 16) && aligned(vs, 16) && aligned(pg, 16) &&
                      ((long)N * T >= (1L << 22));
    if (vec4) return launch_t<4, 2>(p, s);
    return launch_t<1, 8>(p, s);
}

}  // namespace hts
