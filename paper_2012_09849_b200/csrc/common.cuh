// Shared declarations of the library's translation units (host side + small device helpers).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "hts.h"

namespace hts {

// ---- launch accounting and error capture --------------------------------------------------
void note_launch(int count = 1);
hts_status cuda_fail(cudaError_t e, const char* where);   // records text, returns HTS_ERR_CUDA
#define HTS_CUDA(call)                                                        \
    do {                                                                      \
        cudaError_t e__ = (call);                                             \
        if (e__ != cudaSuccess) return ::hts::cuda_fail(e__, #call);          \
    } while (0)
#define HTS_LAUNCH_CHECK(name)                                                \
    do {                                                                      \
        ::hts::note_launch();                                                 \
        cudaError_t e__ = cudaGetLastError();                                 \
        if (e__ != cudaSuccess) return ::hts::cuda_fail(e__, name);           \
    } while (0)

// Programmatic dependent launch: the kernel may begin (prologue, weight loads) while its
// predecessor on the stream drains; it must execute pdl_wait() before touching anything the
// predecessor wrote or still reads, and calls pdl_trigger() only after that wait, so that "my
// wait has passed" implies "everything two kernels back is complete" along the whole chain.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

inline int conv_out(int extent, int k, int s) { return (extent - k) / s + 1; }

// Kernel attributes (dynamic shared memory, carve-out) belong to a device, and so does the SM count:
// the launchers keep their "already set" marks per device, indexed by this slot.
constexpr int kDeviceSlots = 64;
inline int device_slot()
{
    int d = 0;
    if (cudaGetDevice(&d) != cudaSuccess) { cudaGetLastError(); d = 0; }
    return (d >= 0 && d < kDeviceSlots) ? d : 0;
}
inline int device_sm_count(int slot)
{
    static int count[kDeviceSlots] = {};
    if (!count[slot]) {
        int d = 0, c = 0;
        if (cudaGetDevice(&d) == cudaSuccess && cudaDeviceGetAttribute(&c, cudaDevAttrMultiProcessorCount, d) == cudaSuccess) count[slot] = c;
        else cudaGetLastError();
    }
    return count[slot] > 0 ? count[slot] : 1;
}

// Executor-facing addressing of a step (state buffer -> actors -> storage row, Section 4.1): row e of the
// batch reads frame slots[e] of a pool of `pool` frames and writes its outputs at index slots[e].
// slots == nullptr: frames and outputs are dense, row e at index e.  A slot outside [0, pool) is
// reported through the device status word (kStatusBadSlot); that row reads frame 0 and writes nothing.
struct Indexing {
    const int32_t* slots = nullptr;
    int pool = 0;
};
constexpr int kStatusBadSlot = 100;
constexpr int kStatusBadAction = 101;     // a stored action outside [0, A) met by the re-evaluation of given actions

// Geometry of the fixed four-layer network for one observation shape.
struct Geometry {
    int C, H, W, A;
    int H1, W1, H2, W2, H3, W3, F;
};

// ---- optional per-kernel event timing of the actor step (benchmark support) ------------------
enum KernelId { K_CONV1 = 0, K_CONV2, K_CONV3, K_FC, K_HEADS, K_COUNT };
struct Profiler {
    static constexpr int kCap = 4096;            // event pairs per kernel between two reads
    bool on = false;
    int used[K_COUNT] = {0, 0, 0, 0, 0};
    cudaEvent_t* start[K_COUNT] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t* stop[K_COUNT] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    void begin(int k, cudaStream_t s) { if (on && used[k] < kCap) cudaEventRecord(start[k][used[k]], s); }
    void end(int k, cudaStream_t s) { if (on && used[k] < kCap) { cudaEventRecord(stop[k][used[k]], s); ++used[k]; } }
};

// ---- the fp32 CUDA-core path (the check path for fp32 weights; bf16 contexts never use it) ---
struct RefWeights {            // fp32 device copies in PyTorch layouts
    float *w1, *b1, *w2, *b2, *w3, *b3, *wfc, *bfc;
    float *whead, *bhead;      // [A+1,512], [A+1]: policy rows then the value row
};
struct RefWorkspace { float *a1, *a2, *a3, *h; };   // NCHW fp32 activations, [n,512]

hts_status ref_convert_weights(const Geometry& g, int dtype, const hts_weights& src,
                               const RefWeights& dst, cudaStream_t s);
hts_status ref_forward(const Geometry& g, const RefWeights& w, const RefWorkspace& ws,
                       const uint8_t* obs, const Indexing& ix, int* status, int n, Profiler& prof, cudaStream_t s);

// ---- gradient of the learner objective on the fp32 path (backward.cu) ---------------------------
constexpr int kBackwardChunks = 64;      // batch chunks whose partial weight gradients are added in index order
size_t backward_workspace_floats(const Geometry& g, int max_batch);
hts_status ref_backward(const Geometry& g, const RefWeights& w, const RefWorkspace& act, const uint8_t* obs, float* ws,
                        const float* logits, const float* values, const int32_t* actions, const float* adv,
                        const float* ret, const float* logp_old, float value_coef, float entropy_coef, float clip,
                        int n, int max_batch, int* status, const hts_grads& out, cudaStream_t s);

// ---- the tensor-core path (bf16 weights) -------------------------------------------------------
struct TcState;
hts_status tc_check_geometry(const Geometry& g);          // HTS_ERR_SHAPE if the tensor-core kernels cannot take it (no CUDA call)
hts_status tc_create(const Geometry& g, int max_batch, int* status, TcState** out,
                     bool (*alloc)(void* ctx, void** p, size_t bytes), void* alloc_ctx);
void tc_destroy(TcState* t);
hts_status tc_load_weights(TcState* t, const hts_weights& w, cudaStream_t s);
hts_status tc_forward(TcState* t, const uint8_t* obs, const Indexing& ix, int n, Profiler& prof, cudaStream_t s);
hts_status tc_heads(TcState* t, const int32_t* env_ids, const int32_t* t_per_env, int32_t tt, uint64_t seed, int n,
                    const Indexing& ix, int32_t* actions, float* logp, float* values, float* entropy, float* logits,
                    cudaStream_t s, const int32_t* given_actions = nullptr);
hts_status tc_read_activation(TcState* t, int layer, int n, float* out, cudaStream_t s);

// ---- heads + distribution + sampling epilogue (both paths) --------------------------------
// h_partials: [num_splits][n][512] fp32.  If fc_bias != nullptr the hidden vector is
// relu(fc_bias + sum over splits in index order), else it is h_partials[0] as is.
hts_status launch_heads(const float* h_partials, int num_splits, size_t split_stride,
                        const float* fc_bias, const float* whead, const float* bhead, int A,
                        const int32_t* env_ids, const int32_t* t_per_env, int32_t t,
                        uint64_t seed, int n, const Indexing& ix, int* status, int32_t* actions, float* logp,
                        float* values, float* entropy, float* logits, float* h_out, cudaStream_t s,
                        const int32_t* given_actions = nullptr);
// given_actions != nullptr: no sampling; row e reports log pi(given_actions[e] | s_e) (env_ids, t and seed are
// not read, actions may be nullptr).  An action outside [0, A) sets kStatusBadAction and the row writes nothing.

hts_status launch_uniforms(const int32_t* env_ids, const int32_t* t_per_env, int32_t t, uint64_t seed, int n,
                           int A, float* out, cudaStream_t s);

// ---- self-test of the bounded wait (reports through the status word like any expired wait) ---
hts_status launch_wait_selftest(long long limit_ticks, int* status, cudaStream_t s);

// ---- advantage scan -------------------------------------------------------------------------
hts_status launch_gae(const float* rewards, const float* values, const uint8_t* dones,
                      const float* bootstrap, float gamma, float lambda, int T, int N,
                      float* adv, float* ret, cudaStream_t s);

// ---- V-trace / truncated importance sampling scan ---------------------------------------------
hts_status launch_vtrace(const float* log_rhos, const float* rewards, const float* values, const uint8_t* dones,
                         const float* bootstrap, float gamma, float lambda, float rho_bar, float c_bar, int T, int N,
                         float* vs, float* pg, cudaStream_t s);

}  // namespace hts
