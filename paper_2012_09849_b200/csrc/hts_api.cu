// C ABI of the library: argument validation, context management, launch orchestration.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include "common.cuh"

namespace hts {

static std::atomic<uint64_t> g_launches{0};
static thread_local char g_cuda_error[256] = "";

void note_launch(int count) { g_launches.fetch_add((uint64_t)count, std::memory_order_relaxed); }

hts_status cuda_fail(cudaError_t e, const char* where)
{
    std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", where, cudaGetErrorString(e));
    return HTS_ERR_CUDA;
}

}  // namespace hts

using namespace hts;

struct hts_ctx {
    hts_net_desc desc;
    Geometry g;
    bool loaded = false;
    int last_n = 0;
    RefWeights rw{};              // fp32 check path (weight_dtype fp32)
    RefWorkspace rws{};
    TcState* tc = nullptr;        // tensor-core path (weight_dtype bf16)
    // staging for the host-buffer entry point
    uint8_t* s_obs = nullptr;
    int32_t *s_ids = nullptr, *s_t = nullptr, *s_act = nullptr;
    float *s_logp = nullptr, *s_val = nullptr, *s_ent = nullptr, *s_logits = nullptr;
    float* bw_ws = nullptr;       // backward workspace (allocated by the first hts_policy_gradient)
    float *bw_logits = nullptr, *bw_logp = nullptr, *bw_val = nullptr, *bw_ent = nullptr;
    int* status = nullptr;        // device status word
    Profiler prof;
    void* allocs[112];
    int nalloc = 0;
};

namespace {

template <typename T>
bool dev_alloc(hts_ctx* c, T** p, size_t count)
{
    void* q = nullptr;
    if (c->nalloc >= 112) return false;
    if (cudaMalloc(&q, count * sizeof(T) + 256) != cudaSuccess) { cudaGetLastError(); return false; }
    c->allocs[c->nalloc++] = q;
    *p = static_cast<T*>(q);
    return true;
}

bool raw_alloc(void* c, void** p, size_t bytes)
{
    uint8_t* q = nullptr;
    if (!dev_alloc(static_cast<hts_ctx*>(c), &q, bytes)) return false;
    *p = q;
    return true;
}

struct Range { const void* p; size_t bytes; };
bool overlaps(const Range& a, const Range& b)
{
    if (!a.p || !b.p || !a.bytes || !b.bytes) return false;
    const uintptr_t a0 = (uintptr_t)a.p, a1 = a0 + a.bytes, b0 = (uintptr_t)b.p, b1 = b0 + b.bytes;
    return a0 < b1 && b0 < a1;
}
// outputs must not overlap inputs or each other
bool any_overlap(const Range* in, int nin, const Range* out, int nout)
{
    for (int i = 0; i < nout; ++i) {
        for (int j = 0; j < nin; ++j) if (overlaps(out[i], in[j])) return true;
        for (int j = i + 1; j < nout; ++j) if (overlaps(out[i], out[j])) return true;
    }
    return false;
}

hts_status check_step_args(hts_ctx* ctx, const void* obs, const void* env_ids, int n,
                           const void* actions, const void* logp, const void* values, const void* entropy,
                           bool on_host = false)
{
    if (!ctx || !obs || !env_ids || !actions || !logp || !values || !entropy) return HTS_ERR_INVALID_ARG;
    if (n < 1 || n > ctx->desc.max_batch) return HTS_ERR_INVALID_ARG;
    // the tensor-core path stages frames with bulk copies, which need 16-byte-aligned global addresses
    // (frame, channel and row-group offsets are multiples of 16 because H and W are multiples of 4)
    if (ctx->tc && !on_host && ((uintptr_t)obs & 15u) != 0) return HTS_ERR_INVALID_ARG;
    if (!ctx->loaded) return HTS_ERR_UNSUPPORTED;
    return HTS_OK;
}

hts_status run_step(hts_ctx* ctx, const uint8_t* obs, const Indexing& ix, const int32_t* env_ids, const int32_t* t_per_env,
                    int32_t t, uint64_t seed, int32_t n, int32_t* actions, float* logp, float* values,
                    float* entropy, float* logits, cudaStream_t s, const int32_t* given_actions = nullptr)
{
    const Geometry& g = ctx->g;
    hts_status st;
    if (ctx->tc) {
        st = tc_forward(ctx->tc, obs, ix, n, ctx->prof, s);
        if (st != HTS_OK) return st;
        ctx->prof.begin(K_HEADS, s);
        st = tc_heads(ctx->tc, env_ids, t_per_env, t, seed, n, ix, actions, logp, values, entropy, logits, s, given_actions);
    } else {
        st = ref_forward(g, ctx->rw, ctx->rws, obs, ix, ctx->status, n, ctx->prof, s);
        if (st != HTS_OK) return st;
        ctx->prof.begin(K_HEADS, s);
        st = launch_heads(ctx->rws.h, 1, 0, nullptr, ctx->rw.whead, ctx->rw.bhead, g.A, env_ids, t_per_env, t,
                          seed, n, ix, ctx->status, actions, logp, values, entropy, logits, nullptr, s, given_actions);
    }
    if (st != HTS_OK) return st;
    ctx->prof.end(K_HEADS, s);
    ctx->last_n = n;
    return HTS_OK;
}

}  // namespace

// staging buffer of hts_gae_host, one per device; grows on demand, freed by hts_gae_host_release
static char* g_gae_stage[kDeviceSlots] = {};
static size_t g_gae_stage_bytes[kDeviceSlots] = {};

extern "C" {

hts_status hts_policy_create(const hts_net_desc* d, hts_ctx** out)
{
    if (!d || !out) return HTS_ERR_INVALID_ARG;
    *out = nullptr;
    if (d->C < 1 || d->H < 1 || d->W < 1 || d->max_batch < 1) return HTS_ERR_INVALID_ARG;
    if (d->num_actions < 1 || d->num_actions > 64) return HTS_ERR_INVALID_ARG;
    if (d->weight_dtype != HTS_DTYPE_FP32 && d->weight_dtype != HTS_DTYPE_BF16) return HTS_ERR_INVALID_ARG;
    if (d->H % 4 || d->W % 4 || d->C > 64) return HTS_ERR_SHAPE;
    Geometry g{};
    g.C = d->C; g.H = d->H; g.W = d->W; g.A = d->num_actions;
    if (g.H < 8 || g.W < 8) return HTS_ERR_SHAPE;
    g.H1 = conv_out(g.H, 8, 4); g.W1 = conv_out(g.W, 8, 4);
    if (g.H1 < 4 || g.W1 < 4) return HTS_ERR_SHAPE;
    g.H2 = conv_out(g.H1, 4, 2); g.W2 = conv_out(g.W1, 4, 2);
    if (g.H2 < 3 || g.W2 < 3) return HTS_ERR_SHAPE;
    g.H3 = conv_out(g.H2, 3, 1); g.W3 = conv_out(g.W2, 3, 1);
    g.F = 64 * g.H3 * g.W3;
    if (d->weight_dtype == HTS_DTYPE_BF16) {                 // shape limits of the tensor-core kernels, before any CUDA call
        const hts_status gs = tc_check_geometry(g);
        if (gs != HTS_OK) return gs;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cuda_fail(cudaGetLastError(), "cudaGetDevice");

    hts_ctx* c = new (std::nothrow) hts_ctx();
    if (!c) return HTS_ERR_ALLOC;
    c->desc = *d; c->g = g;
    const size_t nb = (size_t)d->max_batch;
    const int A = g.A;
    bool ok = dev_alloc(c, &c->status, 1);
    if (ok && d->weight_dtype == HTS_DTYPE_BF16) {
        hts_status st = tc_create(g, d->max_batch, c->status, &c->tc, raw_alloc, c);
        if (st != HTS_OK) { hts_policy_destroy(c); return st; }
    } else if (ok) {
        ok = ok && dev_alloc(c, &c->rw.w1, (size_t)32 * g.C * 64) && dev_alloc(c, &c->rw.b1, 32);
        ok = ok && dev_alloc(c, &c->rw.w2, (size_t)64 * 32 * 16) && dev_alloc(c, &c->rw.b2, 64);
        ok = ok && dev_alloc(c, &c->rw.w3, (size_t)64 * 64 * 9) && dev_alloc(c, &c->rw.b3, 64);
        ok = ok && dev_alloc(c, &c->rw.wfc, (size_t)512 * g.F) && dev_alloc(c, &c->rw.bfc, 512);
        ok = ok && dev_alloc(c, &c->rw.whead, (size_t)(A + 1) * 512) && dev_alloc(c, &c->rw.bhead, (size_t)A + 1);
        ok = ok && dev_alloc(c, &c->rws.a1, nb * 32 * g.H1 * g.W1) && dev_alloc(c, &c->rws.a2, nb * 64 * g.H2 * g.W2);
        ok = ok && dev_alloc(c, &c->rws.a3, nb * g.F) && dev_alloc(c, &c->rws.h, nb * 512);
    }
    ok = ok && dev_alloc(c, &c->s_obs, nb * g.C * g.H * g.W);
    ok = ok && dev_alloc(c, &c->s_ids, nb) && dev_alloc(c, &c->s_t, nb) && dev_alloc(c, &c->s_act, nb);
    ok = ok && dev_alloc(c, &c->s_logp, nb) && dev_alloc(c, &c->s_val, nb) && dev_alloc(c, &c->s_ent, nb);
    ok = ok && dev_alloc(c, &c->s_logits, nb * A);
    if (!ok) { hts_policy_destroy(c); return HTS_ERR_ALLOC; }
    if (cudaMemset(c->status, 0, sizeof(int)) != cudaSuccess) {
        hts_status st = cuda_fail(cudaGetLastError(), "cudaMemset");
        hts_policy_destroy(c);
        return st;
    }
    *out = c;
    return HTS_OK;
}

hts_status hts_policy_load_weights(hts_ctx* ctx, const hts_weights* w, void* cuda_stream)
{
    if (!ctx || !w) return HTS_ERR_INVALID_ARG;
    const void* const* p = reinterpret_cast<const void* const*>(w);
    for (int i = 0; i < 12; ++i) if (!p[i]) return HTS_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    hts_status st = ctx->tc ? tc_load_weights(ctx->tc, *w, s)
                            : ref_convert_weights(ctx->g, ctx->desc.weight_dtype, *w, ctx->rw, s);
    if (st != HTS_OK) return st;
    ctx->loaded = true;
    return HTS_OK;
}

hts_status hts_policy_step(hts_ctx* ctx, const uint8_t* obs, const int32_t* env_ids,
                           const int32_t* t_per_env, int32_t t, uint64_t seed, int32_t n,
                           int32_t* actions, float* logp, float* values, float* entropy,
                           float* logits_or_null, void* cuda_stream)
{
    hts_status st = check_step_args(ctx, obs, env_ids, n, actions, logp, values, entropy);
    if (st != HTS_OK) return st;
    const size_t nn = (size_t)n;
    const Range in[] = {{obs, nn * ctx->g.C * ctx->g.H * ctx->g.W}, {env_ids, nn * 4}, {t_per_env, nn * 4}};
    const Range outr[] = {{actions, nn * 4}, {logp, nn * 4}, {values, nn * 4}, {entropy, nn * 4},
                          {logits_or_null, nn * ctx->g.A * 4}};
    if (any_overlap(in, 3, outr, 5)) return HTS_ERR_INVALID_ARG;
    return run_step(ctx, obs, Indexing{}, env_ids, t_per_env, t, seed, n, actions, logp, values, entropy, logits_or_null,
                    static_cast<cudaStream_t>(cuda_stream));
}

hts_status hts_policy_step_indexed(hts_ctx* ctx, const uint8_t* state_buffer, int32_t pool, const int32_t* slots,
                                   const int32_t* env_ids, const int32_t* t_per_env, int32_t t, uint64_t seed,
                                   int32_t n, int32_t* actions_row, float* logp_row, float* values_row,
                                   float* entropy_row, void* cuda_stream)
{
    hts_status st = check_step_args(ctx, state_buffer, env_ids, n, actions_row, logp_row, values_row, entropy_row);
    if (st != HTS_OK) return st;
    if (!slots || pool < 1) return HTS_ERR_INVALID_ARG;
    const size_t nn = (size_t)n, pp = (size_t)pool;
    const Range in[] = {{state_buffer, pp * ctx->g.C * ctx->g.H * ctx->g.W}, {slots, nn * 4}, {env_ids, nn * 4},
                        {t_per_env, nn * 4}};
    const Range outr[] = {{actions_row, pp * 4}, {logp_row, pp * 4}, {values_row, pp * 4}, {entropy_row, pp * 4}};
    if (any_overlap(in, 4, outr, 4)) return HTS_ERR_INVALID_ARG;
    Indexing ix;
    ix.slots = slots; ix.pool = pool;
    return run_step(ctx, state_buffer, ix, env_ids, t_per_env, t, seed, n, actions_row, logp_row, values_row, entropy_row,
                    nullptr, static_cast<cudaStream_t>(cuda_stream));
}

hts_status hts_policy_evaluate(hts_ctx* ctx, const uint8_t* obs, const int32_t* actions, int32_t n, float* logp,
                               float* values, float* entropy, float* logits_or_null, void* cuda_stream)
{
    if (!ctx || !obs || !actions || !logp || !values || !entropy) return HTS_ERR_INVALID_ARG;
    if (n < 1 || n > ctx->desc.max_batch) return HTS_ERR_INVALID_ARG;
    if (ctx->tc && ((uintptr_t)obs & 15u) != 0) return HTS_ERR_INVALID_ARG;
    if (!ctx->loaded) return HTS_ERR_UNSUPPORTED;
    const size_t nn = (size_t)n;
    const Range in[] = {{obs, nn * ctx->g.C * ctx->g.H * ctx->g.W}, {actions, nn * 4}};
    const Range outr[] = {{logp, nn * 4}, {values, nn * 4}, {entropy, nn * 4}, {logits_or_null, nn * ctx->g.A * 4}};
    if (any_overlap(in, 2, outr, 4)) return HTS_ERR_INVALID_ARG;
    return run_step(ctx, obs, Indexing{}, nullptr, nullptr, 0, 0, n, nullptr, logp, values, entropy, logits_or_null,
                    static_cast<cudaStream_t>(cuda_stream), actions);
}

hts_status hts_policy_gradient(hts_ctx* ctx, const uint8_t* obs, const int32_t* actions, const float* advantages,
                               const float* returns, const float* logp_old_or_null, float value_coef, float entropy_coef,
                               float clip, int32_t n, const hts_grads* grads, void* cuda_stream)
{
    if (!ctx || !obs || !actions || !advantages || !returns || !grads) return HTS_ERR_INVALID_ARG;
    float* const* gp = reinterpret_cast<float* const*>(grads);
    for (int i = 0; i < 12; ++i) if (!gp[i]) return HTS_ERR_INVALID_ARG;
    if (n < 1 || n > ctx->desc.max_batch) return HTS_ERR_INVALID_ARG;
    if (!(clip >= 0.f) || !std::isfinite(clip) || !std::isfinite(value_coef) || !std::isfinite(entropy_coef)) return HTS_ERR_INVALID_ARG;
    if (ctx->tc) return HTS_ERR_UNSUPPORTED;
    if (!ctx->loaded) return HTS_ERR_UNSUPPORTED;
    const size_t nb = (size_t)ctx->desc.max_batch;
    if (!ctx->bw_ws) {
        bool ok = dev_alloc(ctx, &ctx->bw_ws, backward_workspace_floats(ctx->g, ctx->desc.max_batch));
        ok = ok && dev_alloc(ctx, &ctx->bw_logits, nb * ctx->g.A) && dev_alloc(ctx, &ctx->bw_logp, nb);
        ok = ok && dev_alloc(ctx, &ctx->bw_val, nb) && dev_alloc(ctx, &ctx->bw_ent, nb);
        if (!ok) { ctx->bw_ws = nullptr; return HTS_ERR_ALLOC; }
    }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    hts_status st = run_step(ctx, obs, Indexing{}, nullptr, nullptr, 0, 0, n, nullptr, ctx->bw_logp, ctx->bw_val, ctx->bw_ent,
                             ctx->bw_logits, s, actions);
    if (st != HTS_OK) return st;
    return ref_backward(ctx->g, ctx->rw, ctx->rws, obs, ctx->bw_ws, ctx->bw_logits, ctx->bw_val, actions, advantages, returns,
                        logp_old_or_null, value_coef, entropy_coef, clip, n, ctx->desc.max_batch, ctx->status, *grads, s);
}

hts_status hts_policy_step_host(hts_ctx* ctx, const uint8_t* obs, const int32_t* env_ids,
                                const int32_t* t_per_env, int32_t t, uint64_t seed, int32_t n,
                                int32_t* actions, float* logp, float* values, float* entropy,
                                float* logits_or_null, void* cuda_stream)
{
    hts_status st = check_step_args(ctx, obs, env_ids, n, actions, logp, values, entropy, true);
    if (st != HTS_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t nn = (size_t)n;
    HTS_CUDA(cudaMemcpyAsync(ctx->s_obs, obs, nn * ctx->g.C * ctx->g.H * ctx->g.W, cudaMemcpyHostToDevice, s));
    HTS_CUDA(cudaMemcpyAsync(ctx->s_ids, env_ids, nn * 4, cudaMemcpyHostToDevice, s));
    if (t_per_env) HTS_CUDA(cudaMemcpyAsync(ctx->s_t, t_per_env, nn * 4, cudaMemcpyHostToDevice, s));
    st = run_step(ctx, ctx->s_obs, Indexing{}, ctx->s_ids, t_per_env ? ctx->s_t : nullptr, t, seed, n, ctx->s_act,
                  ctx->s_logp, ctx->s_val, ctx->s_ent, logits_or_null ? ctx->s_logits : nullptr, s);
    if (st != HTS_OK) return st;
    HTS_CUDA(cudaMemcpyAsync(actions, ctx->s_act, nn * 4, cudaMemcpyDeviceToHost, s));
    HTS_CUDA(cudaMemcpyAsync(logp, ctx->s_logp, nn * 4, cudaMemcpyDeviceToHost, s));
    HTS_CUDA(cudaMemcpyAsync(values, ctx->s_val, nn * 4, cudaMemcpyDeviceToHost, s));
    HTS_CUDA(cudaMemcpyAsync(entropy, ctx->s_ent, nn * 4, cudaMemcpyDeviceToHost, s));
    if (logits_or_null)
        HTS_CUDA(cudaMemcpyAsync(logits_or_null, ctx->s_logits, nn * ctx->g.A * 4, cudaMemcpyDeviceToHost, s));
    HTS_CUDA(cudaStreamSynchronize(s));
    return HTS_OK;
}

hts_status hts_policy_read_activation(hts_ctx* ctx, int32_t layer, int32_t n, float* out, void* cuda_stream)
{
    if (!ctx || !out || layer < 1 || layer > 4) return HTS_ERR_INVALID_ARG;
    if (n < 1 || n > ctx->last_n) return HTS_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    if (ctx->tc) return tc_read_activation(ctx->tc, layer, n, out, s);
    const Geometry& g = ctx->g;
    const float* src = layer == 1 ? ctx->rws.a1 : layer == 2 ? ctx->rws.a2 : layer == 3 ? ctx->rws.a3 : ctx->rws.h;
    const size_t per = layer == 1 ? (size_t)32 * g.H1 * g.W1 : layer == 2 ? (size_t)64 * g.H2 * g.W2
                     : layer == 3 ? (size_t)g.F : 512;
    HTS_CUDA(cudaMemcpyAsync(out, src, per * n * sizeof(float), cudaMemcpyDeviceToDevice, s));
    return HTS_OK;
}

hts_status hts_action_uniforms(const int32_t* env_ids, const int32_t* t_per_env, int32_t t, uint64_t seed,
                               int32_t n, int32_t num_actions, float* out, void* cuda_stream)
{
    if (!env_ids || !out || n < 1 || num_actions < 1 || num_actions > 64) return HTS_ERR_INVALID_ARG;
    return launch_uniforms(env_ids, t_per_env, t, seed, n, num_actions, out, static_cast<cudaStream_t>(cuda_stream));
}

hts_status hts_last_async_error(hts_ctx* ctx)
{
    if (!ctx) return HTS_ERR_INVALID_ARG;
    int word = 0;
    HTS_CUDA(cudaMemcpy(&word, ctx->status, sizeof(int), cudaMemcpyDeviceToHost));
    if (word != 0) {
        HTS_CUDA(cudaMemset(ctx->status, 0, sizeof(int)));
        return (word == kStatusBadSlot || word == kStatusBadAction) ? HTS_ERR_INVALID_ARG : HTS_ERR_TIMEOUT;
    }
    return HTS_OK;
}

hts_status hts_wait_selftest(hts_ctx* ctx, int64_t limit_ticks, void* cuda_stream)
{
    if (!ctx || limit_ticks < 1000 || limit_ticks > 100000000LL) return HTS_ERR_INVALID_ARG;
    return launch_wait_selftest((long long)limit_ticks, ctx->status, static_cast<cudaStream_t>(cuda_stream));
}

hts_status hts_policy_profile(hts_ctx* ctx, int32_t enable)
{
    if (!ctx) return HTS_ERR_INVALID_ARG;
    Profiler& p = ctx->prof;
    if (enable && !p.start[0]) {
        for (int k = 0; k < K_COUNT; ++k) {
            p.start[k] = new (std::nothrow) cudaEvent_t[Profiler::kCap]();
            p.stop[k] = new (std::nothrow) cudaEvent_t[Profiler::kCap]();
            if (!p.start[k] || !p.stop[k]) return HTS_ERR_ALLOC;
            for (int i = 0; i < Profiler::kCap; ++i) {
                HTS_CUDA(cudaEventCreate(&p.start[k][i]));
                HTS_CUDA(cudaEventCreate(&p.stop[k][i]));
            }
        }
    }
    if (enable) for (int k = 0; k < K_COUNT; ++k) p.used[k] = 0;
    p.on = enable != 0;
    return HTS_OK;
}

hts_status hts_policy_profile_read(hts_ctx* ctx, int32_t kernel, float* total_ms, int32_t* launches)
{
    if (!ctx || !total_ms || !launches || kernel < 0 || kernel >= K_COUNT) return HTS_ERR_INVALID_ARG;
    Profiler& p = ctx->prof;
    float sum = 0.f;
    for (int i = 0; i < p.used[kernel]; ++i) {
        float ms = 0.f;
        HTS_CUDA(cudaEventSynchronize(p.stop[kernel][i]));
        HTS_CUDA(cudaEventElapsedTime(&ms, p.start[kernel][i], p.stop[kernel][i]));
        sum += ms;
    }
    *total_ms = sum;
    *launches = p.used[kernel];
    return HTS_OK;
}

const char* hts_policy_kernel_name(int32_t kernel)
{
    static const char* names[K_COUNT] = {"conv1", "conv2", "conv3", "fc", "heads"};
    return (kernel >= 0 && kernel < K_COUNT) ? names[kernel] : "";
}

void hts_policy_destroy(hts_ctx* ctx)
{
    if (!ctx) return;
    for (int k = 0; k < K_COUNT; ++k) {
        if (ctx->prof.start[k]) { for (int i = 0; i < Profiler::kCap; ++i) cudaEventDestroy(ctx->prof.start[k][i]); delete[] ctx->prof.start[k]; }
        if (ctx->prof.stop[k]) { for (int i = 0; i < Profiler::kCap; ++i) cudaEventDestroy(ctx->prof.stop[k][i]); delete[] ctx->prof.stop[k]; }
    }
    if (ctx->tc) tc_destroy(ctx->tc);
    for (int i = 0; i < ctx->nalloc; ++i) cudaFree(ctx->allocs[i]);
    delete ctx;
}

static hts_status check_gae_args(const void* r, const void* v, const void* d, const void* b, float gamma,
                                 float lambda, int T, int N, const void* adv, const void* ret)
{
    if (!r || !v || !d || !b || !adv || !ret) return HTS_ERR_INVALID_ARG;
    if (T < 1 || N < 1) return HTS_ERR_INVALID_ARG;
    if (!(gamma >= 0.f && gamma <= 1.f) || !(lambda >= 0.f && lambda <= 1.f)) return HTS_ERR_INVALID_ARG;   // NaN fails both
    return HTS_OK;
}

hts_status hts_gae(const float* rewards, const float* values, const uint8_t* dones, const float* bootstrap,
                   float gamma, float lambda, int32_t T, int32_t N, float* advantages, float* returns,
                   void* cuda_stream)
{
    hts_status st = check_gae_args(rewards, values, dones, bootstrap, gamma, lambda, T, N, advantages, returns);
    if (st != HTS_OK) return st;
    const size_t tn = (size_t)T * N;
    const Range in[] = {{rewards, tn * 4}, {values, tn * 4}, {dones, tn}, {bootstrap, (size_t)N * 4}};
    const Range outr[] = {{advantages, tn * 4}, {returns, tn * 4}};
    if (any_overlap(in, 4, outr, 2)) return HTS_ERR_INVALID_ARG;
    return launch_gae(rewards, values, dones, bootstrap, gamma, lambda, T, N, advantages, returns,
                      static_cast<cudaStream_t>(cuda_stream));
}

hts_status hts_vtrace(const float* log_rhos, const float* rewards, const float* values, const uint8_t* dones,
                      const float* bootstrap, float gamma, float lambda, float rho_bar, float c_bar, int32_t T, int32_t N,
                      float* vs, float* pg_advantages, void* cuda_stream)
{
    hts_status st = check_gae_args(rewards, values, dones, bootstrap, gamma, lambda, T, N, vs, pg_advantages);
    if (st != HTS_OK) return st;
    if (!log_rhos || !(rho_bar >= 0.f) || !(c_bar >= 0.f)) return HTS_ERR_INVALID_ARG;      // NaN fails both
    const size_t tn = (size_t)T * N;
    const Range in[] = {{log_rhos, tn * 4}, {rewards, tn * 4}, {values, tn * 4}, {dones, tn}, {bootstrap, (size_t)N * 4}};
    const Range outr[] = {{vs, tn * 4}, {pg_advantages, tn * 4}};
    if (any_overlap(in, 5, outr, 2)) return HTS_ERR_INVALID_ARG;
    return launch_vtrace(log_rhos, rewards, values, dones, bootstrap, gamma, lambda, rho_bar, c_bar, T, N, vs, pg_advantages,
                         static_cast<cudaStream_t>(cuda_stream));
}

hts_status hts_gae_host(const float* rewards, const float* values, const uint8_t* dones, const float* bootstrap,
                        float gamma, float lambda, int32_t T, int32_t N, float* advantages, float* returns,
                        void* cuda_stream)
{
    hts_status st = check_gae_args(rewards, values, dones, bootstrap, gamma, lambda, T, N, advantages, returns);
    if (st != HTS_OK) return st;
    const int dev = device_slot();
    char*& stage = g_gae_stage[dev];
    size_t& stage_bytes = g_gae_stage_bytes[dev];
    const size_t tn = (size_t)T * N;
    const size_t tn4 = (tn * 4 + 255) / 256 * 256, tn1 = (tn + 255) / 256 * 256, n4 = ((size_t)N * 4 + 255) / 256 * 256;
    const size_t need = 4 * tn4 + tn1 + n4;
    if (need > stage_bytes) {
        if (stage) cudaFree(stage);
        stage = nullptr; stage_bytes = 0;
        if (cudaMalloc(&stage, need) != cudaSuccess) { cudaGetLastError(); return HTS_ERR_ALLOC; }
        stage_bytes = need;
    }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    float* d_r = reinterpret_cast<float*>(stage);
    float* d_v = reinterpret_cast<float*>(stage + tn4);
    float* d_a = reinterpret_cast<float*>(stage + 2 * tn4);
    float* d_q = reinterpret_cast<float*>(stage + 3 * tn4);
    uint8_t* d_d = reinterpret_cast<uint8_t*>(stage + 4 * tn4);
    float* d_b = reinterpret_cast<float*>(stage + 4 * tn4 + tn1);
    HTS_CUDA(cudaMemcpyAsync(d_r, rewards, tn * 4, cudaMemcpyHostToDevice, s));
    HTS_CUDA(cudaMemcpyAsync(d_v, values, tn * 4, cudaMemcpyHostToDevice, s));
    HTS_CUDA(cudaMemcpyAsync(d_d, dones, tn, cudaMemcpyHostToDevice, s));
    HTS_CUDA(cudaMemcpyAsync(d_b, bootstrap, (size_t)N * 4, cudaMemcpyHostToDevice, s));
    st = launch_gae(d_r, d_v, d_d, d_b, gamma, lambda, T, N, d_a, d_q, s);
    if (st != HTS_OK) return st;
    HTS_CUDA(cudaMemcpyAsync(advantages, d_a, tn * 4, cudaMemcpyDeviceToHost, s));
    HTS_CUDA(cudaMemcpyAsync(returns, d_q, tn * 4, cudaMemcpyDeviceToHost, s));
    HTS_CUDA(cudaStreamSynchronize(s));
    return HTS_OK;
}

hts_status hts_gae_host_release(void)
{
    const int dev = device_slot();
    if (g_gae_stage[dev]) {
        HTS_CUDA(cudaDeviceSynchronize());
        HTS_CUDA(cudaFree(g_gae_stage[dev]));
        g_gae_stage[dev] = nullptr; g_gae_stage_bytes[dev] = 0;
    }
    return HTS_OK;
}

uint64_t hts_launch_count(void) { return hts::g_launches.load(std::memory_order_relaxed); }

const char* hts_last_cuda_error(void) { return hts::g_cuda_error; }

const char* hts_status_string(hts_status s)
{
    switch (s) {
        case HTS_OK: return "HTS_OK";
        case HTS_ERR_INVALID_ARG: return "HTS_ERR_INVALID_ARG";
        case HTS_ERR_SHAPE: return "HTS_ERR_SHAPE";
        case HTS_ERR_ALLOC: return "HTS_ERR_ALLOC";
        case HTS_ERR_CUDA: return "HTS_ERR_CUDA";
        case HTS_ERR_TIMEOUT: return "HTS_ERR_TIMEOUT";
        case HTS_ERR_UNSUPPORTED: return "HTS_ERR_UNSUPPORTED";
    }
    return "HTS_ERR_?";
}

}  // extern "C"
