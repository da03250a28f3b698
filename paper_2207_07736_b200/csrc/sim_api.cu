// Host side of the C ABI declared in include/sim.h: handle, argument checks, launch planning.
// Every step of the hot path runs in the kernels of rollout_s4.cu / rollout_synth.cu; this file
// only validates, slices the T steps into ceil(T/K) launches and advances output pointers.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "../../include/sim.h"
#include "sim_internal.h"

using namespace simk;

struct sim : SimCore {           // the population (kind, sizes, buffers, keys, t) is the part the launch planner sees
    uint64_t seed;
    int device;               // ordinal of the device the handle was created on; every call must find it current
    cudaStream_t stream;
    int last_cuda;
    int64_t launches;
    // staging for sim_rollout_host (allocated on first use)
    cudaStream_t copy_stream;
    cudaEvent_t ev_done[2], ev_copied[2];
    void *stage[2];
    size_t stage_bytes;
    float *d_params;
};

#define SIM_API extern "C" __attribute__((visibility("default")))

static int cuda_fail(sim *s, cudaError_t e)
{
    if (s) s->last_cuda = (int)e;
    return e == cudaErrorMemoryAllocation ? SIM_ENOMEM : SIM_ECUDA;
}
#define CU(s, call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return cuda_fail((s), e_); } while (0)

void simk::expand_round_keys(uint64_t seed, RoundKeys &rk)
{
    uint32_t k0 = (uint32_t)(seed & 0xFFFFFFFFu), k1 = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) {
        rk.k[r][0] = k0; rk.k[r][1] = k1;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
}

// A handle's buffers live on the device it was created on: a call made with another device current would
// launch there on pointers that device cannot use.  Host check only.
static int check_device(sim *s)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cuda_fail(s, e);
    return dev == s->device ? SIM_OK : SIM_ESTATE;
}
#define DEV(s) do { int rc_ = check_device(s); if (rc_ != SIM_OK) return rc_; } while (0)

static bool valid_state_dim(int env_kind, int S)
{
    if (env_kind == SIM_SYNTH) return S >= 4 && S <= 4096 && (S & (S - 1)) == 0;
    return S == 4;
}

SIM_API const char *sim_strerror(int code)
{
    switch (code) {
    case SIM_OK: return "ok";
    case SIM_EINVAL: return "invalid argument";
    case SIM_ENOMEM: return "out of device memory";
    case SIM_ECUDA: return "CUDA error (see sim_last_cuda_error)";
    case SIM_ESTATE: return "call not valid in the handle's current state (e.g. another CUDA device is current than the one it was created on)";
    case SIM_ECAPACITY: return "problem does not fit the fixed scratch array of the no-allocation entry point";
    default: return "unknown error code";
    }
}

SIM_API int sim_last_cuda_error(sim_t *s) { return s ? s->last_cuda : 0; }
SIM_API int64_t sim_launch_count(sim_t *s) { return s ? s->launches : -1; }

static void free_handle(sim *s)
{
    if (!s) return;
    if (s->state) cudaFree(s->state);
    if (s->ep_len) cudaFree(s->ep_len);
    if (s->reset_count) cudaFree(s->reset_count);
    for (int i = 0; i < 2; ++i) {
        if (s->stage[i]) cudaFree(s->stage[i]);
        if (s->ev_done[i]) cudaEventDestroy(s->ev_done[i]);
        if (s->ev_copied[i]) cudaEventDestroy(s->ev_copied[i]);
    }
    if (s->d_params) cudaFree(s->d_params);
    if (s->d_status) cudaFree(s->d_status);
    if (s->copy_stream) cudaStreamDestroy(s->copy_stream);
    delete s;
}

SIM_API int sim_create(sim_t **out, int env_kind, int64_t n_envs, int state_dim, uint64_t seed)
{
    if (!out) return SIM_EINVAL;
    *out = nullptr;
    if (env_kind != SIM_CARTPOLE && env_kind != SIM_ACROBOT && env_kind != SIM_SYNTH) return SIM_EINVAL;
    if (n_envs < 1 || n_envs > 0xFFFFFFFFll) return SIM_EINVAL;
    if (!valid_state_dim(env_kind, state_dim)) return SIM_EINVAL;

    sim *s = new (std::nothrow) sim();          // value-initialised: every field starts at zero
    if (!s) return SIM_ENOMEM;
    s->env_kind = env_kind; s->S = state_dim; s->n = (uint32_t)n_envs; s->seed = seed;
    s->compute_factor = 1;
    expand_round_keys(seed, s->rk);
    cudaError_t e = cudaGetDevice(&s->device);
    if (e == cudaSuccess) e = cudaMalloc(&s->state, (size_t)n_envs * (size_t)state_dim * sizeof(float));
    if (e == cudaSuccess) e = cudaMalloc(&s->ep_len, (size_t)n_envs * sizeof(uint32_t));
    if (e == cudaSuccess) e = cudaMalloc(&s->reset_count, (size_t)n_envs * sizeof(uint32_t));
    if (e != cudaSuccess) { int rc = cuda_fail(nullptr, e); cudaGetLastError(); free_handle(s); return rc; }
    int rc = sim_reset(s);
    if (rc == SIM_OK) {
        e = cudaStreamSynchronize(s->stream);
        if (e != cudaSuccess) rc = cuda_fail(nullptr, e);
    }
    if (rc != SIM_OK) { free_handle(s); return rc; }
    *out = s;
    return SIM_OK;
}

SIM_API int sim_destroy(sim_t *s)
{
    if (!s) return SIM_EINVAL;
    cudaStreamSynchronize(s->stream);
    if (s->copy_stream) cudaStreamSynchronize(s->copy_stream);
    free_handle(s);
    return SIM_OK;
}

SIM_API int sim_set_stream(sim_t *s, void *cuda_stream)
{
    if (!s) return SIM_EINVAL;
    s->stream = (cudaStream_t)cuda_stream;
    return SIM_OK;
}

SIM_API int sim_set_env_offset(sim_t *s, uint64_t env_offset)
{
    if (!s) return SIM_EINVAL;
    if (env_offset + (uint64_t)s->n > (1ull << 32)) return SIM_EINVAL;
    s->env_offset = env_offset;
    return SIM_OK;
}

SIM_API int sim_set_compute_factor(sim_t *s, int compute_factor)
{
    if (!s || compute_factor < 1 || compute_factor > 65536) return SIM_EINVAL;
    s->compute_factor = compute_factor;
    return SIM_OK;
}

SIM_API int sim_set_action_stream(sim_t *s, int mode)
{
    if (!s || (mode != SIM_ACTIONS_WORD && mode != SIM_ACTIONS_BITS)) return SIM_EINVAL;
    if (mode == SIM_ACTIONS_BITS && s->env_kind != SIM_CARTPOLE) return SIM_EINVAL;
    s->action_stream = mode;
    return SIM_OK;
}

SIM_API int sim_set_policy_mode(sim_t *s, int mode)
{
    if (!s || (mode != SIM_POLICY_EXACT && mode != SIM_POLICY_TENSOR && mode != SIM_POLICY_TENSOR_PRECISE)) return SIM_EINVAL;
    if (mode != SIM_POLICY_EXACT && s->env_kind != SIM_CARTPOLE) return SIM_EINVAL;
    if (mode != SIM_POLICY_EXACT && !s->d_status) {
        DEV(s);
        CU(s, cudaMalloc(&s->d_status, sizeof(uint32_t)));
        CU(s, cudaMemsetAsync(s->d_status, 0, sizeof(uint32_t), s->stream));
    }
    s->policy_mode = mode;
    return SIM_OK;
}

SIM_API int sim_get_device_status(sim_t *s, uint32_t *h_flags)
{
    if (!s || !h_flags) return SIM_EINVAL;
    *h_flags = 0u;
    if (!s->d_status) return SIM_OK;
    DEV(s);
    CU(s, cudaMemcpyAsync(h_flags, s->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s->stream));
    CU(s, cudaStreamSynchronize(s->stream));
    return SIM_OK;
}

SIM_API int sim_reset(sim_t *s)
{
    if (!s) return SIM_EINVAL;
    DEV(s);
    CU(s, launch_reset(s->env_kind, s->S, s->state, s->ep_len, s->reset_count, s->n, (uint32_t)s->env_offset, s->rk, s->stream));
    s->launches += 1;
    s->t = 0;
    return SIM_OK;
}

// One launch of K steps of the population `c`, starting at c.t: picks the kernel for the env kind, the policy and
// the launch length.  Output pointers address row 0 of this launch.  Shared by every entry point that rolls out.
cudaError_t simk::launch_planned(const SimCore &c, int K, int policy, const float *d_params, const int8_t *d_actions, float *next_obs,
                                 float *obs, int8_t *act, float *rew, uint8_t *done, cudaStream_t st)
{
    const uint32_t tb0 = (uint32_t)(c.t >> 2);
    const int phase = (int)(c.t & 3);
    if (c.env_kind == SIM_SYNTH) {
        SynthArgs a;
        a.state = c.state; a.ep_len = c.ep_len; a.reset_count = c.reset_count;
        a.n = c.n; a.env_offset = (uint32_t)c.env_offset; a.tb0 = tb0; a.phase = phase; a.K = K; a.C = c.compute_factor;
        a.out_obs = obs; a.out_act = act; a.out_rew = rew; a.out_done = done;
        a.actions = d_actions; a.next_obs = next_obs; a.rk = c.rk;
        return launch_synth(c.S, a, st);
    }
    S4Args a;
    a.state = reinterpret_cast<float4 *>(c.state); a.ep_len = c.ep_len; a.reset_count = c.reset_count;
    a.n = c.n; a.env_offset = (uint32_t)c.env_offset; a.tb0 = tb0; a.phase = phase; a.K = K; a.C = c.compute_factor;
    a.out_obs = reinterpret_cast<float4 *>(obs); a.out_act = act; a.out_rew = rew; a.out_done = done;
    a.actions = d_actions; a.next_obs = reinterpret_cast<float4 *>(next_obs); a.params = d_params; a.status = c.d_status; a.rk = c.rk;
    a.action_bits = (c.action_stream == SIM_ACTIONS_BITS && policy == POLICY_RANDOM) ? 1 : 0;
    if (c.env_kind == SIM_CARTPOLE && policy == POLICY_RANDOM && c.compute_factor == 1)
        return launch_cartpole_random(a, st);
    if (c.env_kind == SIM_ACROBOT && policy == POLICY_RANDOM && K > 4)      // short launches: the scalar kernel has the shorter step latency
        return launch_acrobot_random(a, st);
    if (c.env_kind == SIM_CARTPOLE && policy == POLICY_MLP && c.policy_mode == SIM_POLICY_TENSOR)
        return launch_cartpole_mlp_tc(a, st);
    if (c.env_kind == SIM_CARTPOLE && policy == POLICY_MLP && c.policy_mode == SIM_POLICY_TENSOR_PRECISE)
        return launch_cartpole_mlp_tcp(a, st);
    if (c.env_kind == SIM_CARTPOLE && policy == POLICY_MLP)
        return launch_cartpole_mlp(a, st);
    return launch_s4(c.env_kind, policy, a, st);
}

static int launch_chunk(sim *s, int K, int policy, const float *d_params, const int8_t *d_actions, float *next_obs,
                        float *obs, int8_t *act, float *rew, uint8_t *done)
{
    CU(s, launch_planned(*s, K, policy, d_params, d_actions, next_obs, obs, act, rew, done, s->stream));
    s->launches += 1;
    s->t += (uint64_t)K;
    return SIM_OK;
}

SIM_API int sim_step(sim_t *s, const int8_t *d_actions, float *d_next_obs, float *d_rew, uint8_t *d_done)
{
    if (!s || !d_actions) return SIM_EINVAL;
    DEV(s);
    return launch_chunk(s, 1, POLICY_GIVEN, nullptr, d_actions, d_next_obs, nullptr, nullptr, d_rew, d_done);
}

static int check_rollout_args(sim *s, int T, int K, const void *params)
{
    if (!s || T < 1 || K < 1) return SIM_EINVAL;
    if (params && s->env_kind != SIM_CARTPOLE) return SIM_EINVAL;
    return SIM_OK;
}

SIM_API int sim_rollout(sim_t *s, int T, int K_fused, const float *d_policy_params,
                        float *out_obs, int8_t *out_act, float *out_rew, uint8_t *out_done)
{
    int rc = check_rollout_args(s, T, K_fused, d_policy_params);
    if (rc != SIM_OK) return rc;
    DEV(s);
    const int K = K_fused > T ? T : K_fused;
    const int policy = d_policy_params ? POLICY_MLP : POLICY_RANDOM;
    const size_t n = s->n, S = (size_t)s->S;
    for (int done_steps = 0; done_steps < T; done_steps += K) {
        const int k = (T - done_steps) < K ? (T - done_steps) : K;
        const size_t r0 = (size_t)done_steps * n;
        rc = launch_chunk(s, k, policy, d_policy_params, nullptr, nullptr,
                          out_obs ? out_obs + r0 * S : nullptr, out_act ? out_act + r0 : nullptr,
                          out_rew ? out_rew + r0 : nullptr, out_done ? out_done + r0 : nullptr);
        if (rc != SIM_OK) return rc;
    }
    return SIM_OK;
}

// ---------------------------------------------------------------------------------------------
// Host-buffer rollout: chunks of K steps are computed into one of two device staging buffers
// and copied to the caller's host arrays on a second stream while the next chunk is computed.
// ---------------------------------------------------------------------------------------------
static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

SIM_API int sim_rollout_host(sim_t *s, int T, int K_fused, const float *h_policy_params,
                             float *h_obs, int8_t *h_act, float *h_rew, uint8_t *h_done)
{
    int rc = check_rollout_args(s, T, K_fused, h_policy_params);
    if (rc != SIM_OK) return rc;
    DEV(s);
    const int K = K_fused > T ? T : K_fused;
    const size_t n = s->n, S = (size_t)s->S;
    const size_t rows = (size_t)K * n;
    const size_t off_obs = 0;
    const size_t off_act = off_obs + (h_obs ? align256(rows * S * sizeof(float)) : 0);
    const size_t off_rew = off_act + (h_act ? align256(rows) : 0);
    const size_t off_done = off_rew + (h_rew ? align256(rows * sizeof(float)) : 0);
    const size_t need = off_done + (h_done ? align256(rows) : 0);

    if (!s->copy_stream) {
        CU(s, cudaStreamCreateWithFlags(&s->copy_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            CU(s, cudaEventCreateWithFlags(&s->ev_done[i], cudaEventDisableTiming));
            CU(s, cudaEventCreateWithFlags(&s->ev_copied[i], cudaEventDisableTiming));
        }
    }
    if (need > s->stage_bytes) {
        CU(s, cudaStreamSynchronize(s->stream));
        CU(s, cudaStreamSynchronize(s->copy_stream));
        for (int i = 0; i < 2; ++i) { if (s->stage[i]) cudaFree(s->stage[i]); s->stage[i] = nullptr; }
        s->stage_bytes = 0;
        for (int i = 0; i < 2; ++i) CU(s, cudaMalloc(&s->stage[i], need));
        s->stage_bytes = need;
    }
    const float *d_params = nullptr;
    if (h_policy_params) {
        if (!s->d_params) CU(s, cudaMalloc(&s->d_params, SIM_POLICY_PARAM_COUNT * sizeof(float)));
        CU(s, cudaMemcpyAsync(s->d_params, h_policy_params, SIM_POLICY_PARAM_COUNT * sizeof(float), cudaMemcpyHostToDevice, s->stream));
        d_params = s->d_params;
    }
    const int policy = d_params ? POLICY_MLP : POLICY_RANDOM;

    int chunk = 0;
    for (int done_steps = 0; done_steps < T; done_steps += K, ++chunk) {
        const int b = chunk & 1;
        const int k = (T - done_steps) < K ? (T - done_steps) : K;
        char *base = static_cast<char *>(s->stage[b]);
        if (chunk >= 2) CU(s, cudaStreamWaitEvent(s->stream, s->ev_copied[b], 0));     // buffer b is free again
        rc = launch_chunk(s, k, policy, d_params, nullptr, nullptr,
                          h_obs ? reinterpret_cast<float *>(base + off_obs) : nullptr,
                          h_act ? reinterpret_cast<int8_t *>(base + off_act) : nullptr,
                          h_rew ? reinterpret_cast<float *>(base + off_rew) : nullptr,
                          h_done ? reinterpret_cast<uint8_t *>(base + off_done) : nullptr);
        if (rc != SIM_OK) return rc;
        CU(s, cudaEventRecord(s->ev_done[b], s->stream));
        CU(s, cudaStreamWaitEvent(s->copy_stream, s->ev_done[b], 0));
        const size_t r0 = (size_t)done_steps * n, kr = (size_t)k * n;
        if (h_obs) CU(s, cudaMemcpyAsync(h_obs + r0 * S, base + off_obs, kr * S * sizeof(float), cudaMemcpyDeviceToHost, s->copy_stream));
        if (h_act) CU(s, cudaMemcpyAsync(h_act + r0, base + off_act, kr, cudaMemcpyDeviceToHost, s->copy_stream));
        if (h_rew) CU(s, cudaMemcpyAsync(h_rew + r0, base + off_rew, kr * sizeof(float), cudaMemcpyDeviceToHost, s->copy_stream));
        if (h_done) CU(s, cudaMemcpyAsync(h_done + r0, base + off_done, kr, cudaMemcpyDeviceToHost, s->copy_stream));
        CU(s, cudaEventRecord(s->ev_copied[b], s->copy_stream));
    }
    CU(s, cudaStreamSynchronize(s->copy_stream));
    CU(s, cudaStreamSynchronize(s->stream));
    return SIM_OK;
}

SIM_API int sim_get_state(sim_t *s, float *d_state)
{
    if (!s || !d_state) return SIM_EINVAL;
    DEV(s);
    CU(s, cudaMemcpyAsync(d_state, s->state, (size_t)s->n * s->S * sizeof(float), cudaMemcpyDeviceToDevice, s->stream));
    return SIM_OK;
}

SIM_API int sim_set_state(sim_t *s, const float *d_state)
{
    if (!s || !d_state) return SIM_EINVAL;
    DEV(s);
    CU(s, cudaMemcpyAsync(s->state, d_state, (size_t)s->n * s->S * sizeof(float), cudaMemcpyDeviceToDevice, s->stream));
    return SIM_OK;
}

SIM_API int sim_get_counters(sim_t *s, uint32_t *d_ep_len, uint32_t *d_reset_count, uint64_t *h_t)
{
    if (!s) return SIM_EINVAL;
    DEV(s);
    if (d_ep_len) CU(s, cudaMemcpyAsync(d_ep_len, s->ep_len, (size_t)s->n * 4, cudaMemcpyDeviceToDevice, s->stream));
    if (d_reset_count) CU(s, cudaMemcpyAsync(d_reset_count, s->reset_count, (size_t)s->n * 4, cudaMemcpyDeviceToDevice, s->stream));
    if (h_t) *h_t = s->t;
    return SIM_OK;
}

SIM_API int sim_set_counters(sim_t *s, const uint32_t *d_ep_len, const uint32_t *d_reset_count, uint64_t t)
{
    if (!s) return SIM_EINVAL;
    DEV(s);
    if (d_ep_len) CU(s, cudaMemcpyAsync(s->ep_len, d_ep_len, (size_t)s->n * 4, cudaMemcpyDeviceToDevice, s->stream));
    if (d_reset_count) CU(s, cudaMemcpyAsync(s->reset_count, d_reset_count, (size_t)s->n * 4, cudaMemcpyDeviceToDevice, s->stream));
    s->t = t;
    return SIM_OK;
}

SIM_API int sim_policy_logits(sim_t *s, const float *d_obs, int64_t M, const float *d_params, float *d_logits)
{
    if (!s || !d_obs || !d_params || !d_logits || M < 0) return SIM_EINVAL;
    DEV(s);
    if (s->policy_mode == SIM_POLICY_TENSOR)
        CU(s, launch_policy_logits_tc(d_obs, M, d_params, d_logits, s->d_status, s->stream));
    else if (s->policy_mode == SIM_POLICY_TENSOR_PRECISE)
        CU(s, launch_policy_logits_tcp(d_obs, M, d_params, d_logits, s->d_status, s->stream));
    else
        CU(s, launch_policy_logits(d_obs, M, d_params, d_logits, s->stream));
    if (M > 0) s->launches += 1;
    return SIM_OK;
}

SIM_API int sim_selfcheck_division(sim_t *s, int nums_per_den, uint64_t *h_mismatches)
{
    if (!s || !h_mismatches || nums_per_den < 0) return SIM_EINVAL;
    DEV(s);
    unsigned long long *d_bad = nullptr;
    CU(s, cudaMalloc(&d_bad, sizeof(unsigned long long)));
    cudaError_t e = cudaMemsetAsync(d_bad, 0, sizeof(unsigned long long), s->stream);
    if (e == cudaSuccess) e = launch_division_selfcheck(nums_per_den, d_bad, s->stream);
    unsigned long long h = 0;
    if (e == cudaSuccess) e = cudaMemcpyAsync(&h, d_bad, sizeof(h), cudaMemcpyDeviceToHost, s->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s->stream);
    cudaFree(d_bad);
    if (e != cudaSuccess) return cuda_fail(s, e);
    s->launches += 1;
    *h_mismatches = (uint64_t)h;
    return SIM_OK;
}

// One CTA of the tensor-mode policy with its contractions left out: every wait must give up after about a
// millisecond.  Scratch: 4610 zero parameters, a status word and one word per thread.
SIM_API int sim_selfcheck_tensor_wait(sim_t *s, uint32_t *h_status, uint32_t *h_threads_completed)
{
    if (!s || !h_status || !h_threads_completed) return SIM_EINVAL;
    DEV(s);
    const size_t words = SIM_POLICY_PARAM_COUNT + 1 + 256;
    uint32_t *d = nullptr;
    CU(s, cudaMalloc(&d, words * sizeof(uint32_t)));
    uint32_t h[257] = {0};
    cudaError_t e = cudaMemsetAsync(d, 0, words * sizeof(uint32_t), s->stream);
    if (e == cudaSuccess) e = launch_tensor_wait_selfcheck(reinterpret_cast<const float *>(d), 2000000ll, d + SIM_POLICY_PARAM_COUNT, d + SIM_POLICY_PARAM_COUNT + 1, s->stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h, d + SIM_POLICY_PARAM_COUNT, sizeof(h), cudaMemcpyDeviceToHost, s->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s->stream);
    cudaFree(d);
    if (e != cudaSuccess) return cuda_fail(s, e);
    s->launches += 1;
    *h_status = h[0];
    uint32_t done = 0;
    for (int i = 0; i < 256; ++i) done += h[1 + i];
    *h_threads_completed = done;
    return SIM_OK;
}

SIM_API int sim_acrobot_observation(sim_t *s, const float *d_state, int64_t M, float *d_obs6)
{
    if (!s || !d_state || !d_obs6 || M < 0) return SIM_EINVAL;
    DEV(s);
    CU(s, launch_acrobot_observation(d_state, M, d_obs6, s->stream));
    if (M > 0) s->launches += 1;
    return SIM_OK;
}

SIM_API int sim_episode_returns(sim_t *s, const float *d_rew, const uint8_t *d_done, int T, int64_t n, float *d_carry, float *d_ret)
{
    if (!s || !d_rew || !d_done || !d_ret || T < 0 || n < 0) return SIM_EINVAL;
    DEV(s);
    CU(s, launch_episode_returns(d_rew, d_done, T, n, d_carry, d_ret, s->stream));
    if (T > 0 && n > 0) s->launches += 1;
    return SIM_OK;
}
