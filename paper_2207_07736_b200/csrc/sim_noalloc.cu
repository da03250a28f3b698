// sim_rollout_noalloc: a whole reset + rollout that never allocates.
//
// Some callers cannot call cudaMalloc at the moment they need a rollout: a control or serving
// loop that must not stall (cudaMalloc and cudaFree synchronise the whole device, so every other
// stream waits), a process whose device memory is already handed out in full to a framework's
// caching allocator, or a plug-in that is only allowed to touch the buffers it is given.  For
// them the per-env working memory that sim_create would allocate (state matrix, episode-length
// and reset counters) lives in a fixed array inside the library's device image instead.
//
// The array is a file-scope __device__ symbol.  In host code its name is only a stand-in for the
// symbol, not an address a kernel may use; the device address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and it is that address the kernels receive.
#include <mutex>

#include "../../include/sim.h"
#include "sim_internal.h"

using namespace simk;

static_assert(SIM_NOALLOC_SCRATCH_BYTES % 256 == 0, "scratch capacity must keep the 256-byte alignment of its parts");
static __device__ __align__(256) unsigned char g_noalloc_scratch[SIM_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_setup_lock;
unsigned char *g_scratch_addr[kMaxDevices];     // device address of the array, per device ordinal (nullptr = not looked up yet)

// Device address of the scratch array on the current device; looks it up on the first call per device.
cudaError_t scratch_address(unsigned char **out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> guard(g_setup_lock);
    if (!g_scratch_addr[dev]) {
        unsigned char *ptr = nullptr;
        e = cudaGetSymbolAddress((void **)&ptr, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        if (!ptr) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

size_t round256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

extern "C" __attribute__((visibility("default")))
int sim_rollout_noalloc(int env_kind, int64_t n_envs, int state_dim, uint64_t seed, int T, int K_fused,
                        const float *d_policy_params, float *out_obs, int8_t *out_act, float *out_rew, uint8_t *out_done,
                        void *cuda_stream)
{
    if (env_kind != SIM_CARTPOLE && env_kind != SIM_ACROBOT && env_kind != SIM_SYNTH) return SIM_EINVAL;
    if (n_envs < 1 || n_envs > 0xFFFFFFFFll || T < 1 || K_fused < 1) return SIM_EINVAL;
    if (env_kind == SIM_SYNTH) {
        if (state_dim < 4 || state_dim > 4096 || (state_dim & (state_dim - 1))) return SIM_EINVAL;
    } else if (state_dim != 4) {
        return SIM_EINVAL;
    }
    if (d_policy_params && env_kind != SIM_CARTPOLE) return SIM_EINVAL;

    // layout inside the array: state [n,S] fp32 | ep_len [n] u32 | reset_count [n] u32, each part 256-byte aligned
    const size_t n = (size_t)n_envs, S = (size_t)state_dim;
    const size_t off_len = round256(n * S * sizeof(float));
    const size_t off_rc = off_len + round256(n * sizeof(uint32_t));
    const size_t need = off_rc + round256(n * sizeof(uint32_t));
    if (need > (size_t)SIM_NOALLOC_SCRATCH_BYTES) return SIM_ECAPACITY;

    unsigned char *base = nullptr;
    if (scratch_address(&base) != cudaSuccess) { cudaGetLastError(); return SIM_ECUDA; }
    float *state = reinterpret_cast<float *>(base);
    uint32_t *ep_len = reinterpret_cast<uint32_t *>(base + off_len);
    uint32_t *reset_count = reinterpret_cast<uint32_t *>(base + off_rc);
    cudaStream_t st = (cudaStream_t)cuda_stream;

    // The population lives in the fixed array; everything else is what a fresh handle would hold.
    SimCore c = {};
    c.env_kind = env_kind; c.S = state_dim; c.n = (uint32_t)n; c.env_offset = 0; c.t = 0;
    c.compute_factor = 1; c.action_stream = SIM_ACTIONS_WORD; c.policy_mode = SIM_POLICY_EXACT; c.d_status = nullptr;
    c.state = state; c.ep_len = ep_len; c.reset_count = reset_count;
    expand_round_keys(seed, c.rk);
    // the array keeps whatever the previous call left: the reset kernel rewrites every word this call reads
    if (launch_reset(env_kind, state_dim, state, ep_len, reset_count, c.n, 0u, c.rk, st) != cudaSuccess) { cudaGetLastError(); return SIM_ECUDA; }

    // the same launch planner as sim_rollout: the same kernels for the same (env kind, policy, launch length)
    const int K = K_fused > T ? T : K_fused;
    const int policy = d_policy_params ? POLICY_MLP : POLICY_RANDOM;
    for (int t = 0; t < T; t += K) {
        const int k = (T - t) < K ? (T - t) : K;
        const size_t r0 = (size_t)t * n;
        const cudaError_t e = launch_planned(c, k, policy, d_policy_params, nullptr, nullptr,
                                             out_obs ? out_obs + r0 * S : nullptr, out_act ? out_act + r0 : nullptr,
                                             out_rew ? out_rew + r0 : nullptr, out_done ? out_done + r0 : nullptr, st);
        if (e != cudaSuccess) { cudaGetLastError(); return SIM_ECUDA; }
        c.t += (uint64_t)k;
    }
    return SIM_OK;
}
