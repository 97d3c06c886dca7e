// Advantage / return scan over the [T,N] rollout storage (Section 3 of the paper: n-step
// truncated return; the GAE recurrence generalises it with lambda).
//
//   delta_t = r_t + gamma (1-d_t) V_{t+1} - V_t        A_t = delta_t + gamma lambda (1-d_t) A_{t+1}
//
// The recurrence is a composition of affine maps A_{t+1} -> A_t, so time is cut into chunks of
// L rows that are scanned in parallel: each thread owns VEC adjacent env columns of one chunk,
// loads its rows once (all loads issued before the first use, coalesced across env), reduces
// the chunk to one affine map (S,P), the block chains the W chunk maps through shared memory,
// and every thread replays its chunk with the true incoming advantage.  One pass over HBM:
// 17 bytes per element.  The replay uses the same operation order as the sequential
// recurrence, so only the incoming carry differs from it, by rounding.
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

// blockDim = (32, W).  A warp is CY rows of 32/CY threads: thread (cx, cy) of warp w owns columns
// [b*cols + cx*VEC, +VEC) (cols = 32/CY*VEC columns per block b) and chunk w*CY + cy of the super-chunk.  Time
// is walked from the end in super-chunks of W*CY*L rows.  CY = 1 is a warp across 32*VEC columns; CY = 4 makes
// blocks four times narrower (8 columns: still whole 32-byte sectors per row) so that a problem with few
// columns spreads over four times as many SMs.  Chunk boundaries, and with them every rounding, do not depend
// on CY or W.
template <int VEC, int L, int CY>
__global__ void __launch_bounds__(VEC == 4 ? 512 : 1024)
gae_scan_kernel(const float* __restrict__ rewards, const float* __restrict__ values,
                const uint8_t* __restrict__ dones, const float* __restrict__ bootstrap,
                float gamma, float lambda, int T, int N,
                float* __restrict__ adv, float* __restrict__ ret)
{
    using F = typename VecT<VEC>::F;
    using B = typename VecT<VEC>::B;
    extern __shared__ float smem[];                  // [NC][cols] S, then [NC][cols] P
    constexpr int CXW = 32 / CY;                     // threads of a warp along env
    const int NC = blockDim.y * CY;                  // chunks of a super-chunk
    const int cx = threadIdx.x % CXW;
    const int w = threadIdx.y * CY + threadIdx.x / CXW;      // my chunk of the super-chunk
    const int cols = CXW * VEC;
    const long col = (long)blockIdx.x * cols + cx * VEC;
    const bool col_ok = col < N;                     // N % VEC == 0 is guaranteed by the launcher
    float* sS = smem;
    float* sP = smem + NC * cols;
    const float gl = gamma * lambda;

    float carry_in[VEC];                             // advantage at the first row after this super-chunk
#pragma unroll
    for (int k = 0; k < VEC; ++k) carry_in[k] = 0.f;

    const int span = NC * L;
    const int nsuper = (T + span - 1) / span;
    for (int sc = nsuper - 1; sc >= 0; --sc) {
        const int t_begin = sc * span + w * L;       // first row of my chunk
        int rows = T - t_begin; rows = rows > L ? L : rows;   // may be <= 0 in the last super-chunk
        float delta[L][VEC], val[L][VEC];
        uint32_t live_mask = 0;                      // bit i*VEC+k: row i, column k not done
        float S[VEC], P[VEC];
#pragma unroll
        for (int k = 0; k < VEC; ++k) { S[k] = 0.f; P[k] = 1.f; }
        if (col_ok && rows > 0) {
            F r_raw[L], v_raw[L], vnext_raw; B d_raw[L];
#pragma unroll
            for (int i = 0; i < L; ++i) {
                if (i < rows) {
                    const size_t off = (size_t)(t_begin + i) * N + col;
                    r_raw[i] = *reinterpret_cast<const F*>(rewards + off);
                    v_raw[i] = *reinterpret_cast<const F*>(values + off);
                    d_raw[i] = *reinterpret_cast<const B*>(dones + off);
                }
            }
            const int t_after = t_begin + rows;      // row that supplies V_{t+1} of my last row
            vnext_raw = (t_after < T) ? *reinterpret_cast<const F*>(values + (size_t)t_after * N + col)
                                      : *reinterpret_cast<const F*>(bootstrap + col);
            float vnext[VEC];
            unpack<VEC>(vnext_raw, vnext);
#pragma unroll
            for (int i = L - 1; i >= 0; --i) {
                if (i < rows) {
                    float r[VEC], live[VEC];
                    unpack<VEC>(r_raw[i], r);
                    unpack<VEC>(v_raw[i], val[i]);
                    unpackb<VEC>(d_raw[i], live);
#pragma unroll
                    for (int k = 0; k < VEC; ++k) {
                        delta[i][k] = r[k] + gamma * live[k] * vnext[k] - val[i][k];
                        const float cc = gl * live[k];
                        live_mask |= (live[k] != 0.f ? 1u : 0u) << (i * VEC + k);
                        S[k] = delta[i][k] + cc * S[k];
                        P[k] = cc * P[k];
                        vnext[k] = val[i][k];
                    }
                }
            }
        }
        __syncthreads();                             // previous super-chunk's readers are done
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            sS[w * cols + cx * VEC + k] = S[k];
            sP[w * cols + cx * VEC + k] = P[k];
        }
        __syncthreads();
        // chain the chunk maps from the last chunk down; pick up my own incoming advantage
        float c[VEC], mine[VEC];
#pragma unroll
        for (int k = 0; k < VEC; ++k) { c[k] = carry_in[k]; mine[k] = 0.f; }
        for (int ww = NC - 1; ww >= 0; --ww) {
#pragma unroll
            for (int k = 0; k < VEC; ++k) {
                if (ww == w) mine[k] = c[k];
                c[k] = sS[ww * cols + cx * VEC + k] + sP[ww * cols + cx * VEC + k] * c[k];
            }
        }
#pragma unroll
        for (int k = 0; k < VEC; ++k) carry_in[k] = c[k];
        if (col_ok && rows > 0) {
            float a[VEC];
#pragma unroll
            for (int k = 0; k < VEC; ++k) a[k] = mine[k];
#pragma unroll
            for (int i = L - 1; i >= 0; --i) {
                if (i < rows) {
                    float rt[VEC];
#pragma unroll
                    for (int k = 0; k < VEC; ++k) {
                        const float cc = ((live_mask >> (i * VEC + k)) & 1u) ? gl : 0.f;
                        a[k] = delta[i][k] + cc * a[k];
                        rt[k] = a[k] + val[i][k];
                    }
                    const size_t off = (size_t)(t_begin + i) * N + col;
                    *reinterpret_cast<F*>(adv + off) = pack<VEC>(a);
                    *reinterpret_cast<F*>(ret + off) = pack<VEC>(rt);
                }
            }
        }
    }
}

template <int VEC, int L, int CY>
hts_status launch_t(const float* r, const float* v, const uint8_t* d, const float* b, float gamma,
                    float lambda, int T, int N, float* adv, float* ret, cudaStream_t s)
{
    // Wide problems (VEC == 4) have all the parallelism they need across env: two chunks per block
    // measured best (86 % of the copy bandwidth at T=128, N=2^20).  Narrow ones cut time as finely
    // as a block allows.
    const int chunks = (T + L - 1) / L;
    int W = (chunks + CY - 1) / CY;
    const int maxW = (VEC == 4) ? 2 : 32;
    if (W > maxW) W = maxW;
    const int cols = 32 / CY * VEC;
    const unsigned blocks = (unsigned)((N + cols - 1) / cols);
    const size_t smem = (size_t)2 * W * CY * cols * sizeof(float);
    gae_scan_kernel<VEC, L, CY><<<blocks, dim3(32, W), smem, s>>>(r, v, d, b, gamma, lambda, T, N, adv, ret);
    HTS_LAUNCH_CHECK("gae_scan_kernel");
    return HTS_OK;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

hts_status launch_gae(const float* rewards, const float* values, const uint8_t* dones,
                      const float* bootstrap, float gamma, float lambda, int T, int N,
                      float* adv, float* ret, cudaStream_t s)
{
    // 4 columns per thread needs 16-byte rows; wide problems only (narrow ones want more blocks).
    const bool vec4 = (N % 4 == 0) && aligned(rewards, 16) && aligned(values, 16) && aligned(dones, 4) &&
                      aligned(bootstrap, 16) && aligned(adv, 16) && aligned(ret, 16) &&
                      ((long)N * T >= (1L << 22));
    if (vec4) return launch_t<4, 2, 1>(rewards, values, dones, bootstrap, gamma, lambda, T, N, adv, ret, s);
    // few columns and many rows: 8-column blocks, four chunks per warp (same chunks, same bits, four times the SMs)
    if ((N + 31) / 32 < device_sm_count(device_slot()) / 2 && T >= 4 * 8)
        return launch_t<1, 8, 4>(rewards, values, dones, bootstrap, gamma, lambda, T, N, adv, ret, s);
    return launch_t<1, 8, 1>(rewards, values, dones, bootstrap, gamma, lambda, T, N, adv, ret, s);
}

}  // namespace hts
