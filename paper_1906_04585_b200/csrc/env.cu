// Synthetic environment for the closed actor loop (Algorithm 1, "take N actions ... and store transitions"):
// a stand-in for the simulators, which in the paper run on CPUs and are no part of this library.  It is a
// pure function of (seed, agent, environment, step) built on the SplitMix64 output function
//     sm64(z): z += 0x9E3779B97F4A7C15; z = (z ^ z >> 30) * 0xBF58476D1CE4E5B9;
//              z = (z ^ z >> 27) * 0x94D049BB133111EB; return z ^ z >> 31
//     h(tag, idx) = sm64(sm64(sm64(sm64(seed + agent) + env) + step) + (tag << 56) + idx)
//   observation (tag 0): frames: byte j = byte j % 8 of h(0, j / 8); vectors: element j =
//                        ((h(0, j) >> 40) * 2^-23 - 1) * sqrt(3)   (uniform, unit variance)
//   reward of the transition taken at `step` (tag 1): 1 if h(1, 0) % A == action, else 0
//   done (tag 2): (h(2, 0) >> 40) < 167772   (probability 0.01)
//   uniform for the action draw at `step` (tag 3): (h(3, 0) >> 40) * 2^-24
// The observation does not depend on earlier actions; the reward does.
#include "internal.h"

namespace gala {

__device__ __forceinline__ uint64_t sm64(uint64_t z) {
    z += 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__device__ __forceinline__ uint64_t env_base(uint64_t seed, int agent, int env, long long step) {
    return sm64(sm64(sm64(seed + (uint64_t)agent) + (uint64_t)env) + (uint64_t)step);
}

// One launch per environment step.  If `actions` is given: rewards / dones of the transition taken at `step`.
// If `obs_out` is given: the observation and the action-draw uniform of step `obs_step`.
__global__ void __launch_bounds__(256) env_kernel(EnvArgs a) {
    pdl_wait();
    pdl_launch();
    const int e = blockIdx.y;
    if (a.step_base) {   // steps counted from a counter in device memory (the same launch replayed for every rollout)
        const long long base = *a.step_base;
        a.step += base;
        a.obs_step += base;
    }
    if (a.actions && blockIdx.x == 0 && threadIdx.x == 0) {
        const uint64_t b = env_base(a.seed, a.agent, e, a.step);
        const uint64_t hr = sm64(b + (1ull << 56)), hd = sm64(b + (2ull << 56));
        a.rewards[e] = (int)(hr % (uint64_t)a.n_actions) == a.actions[e] ? 1.0f : 0.0f;
        a.dones[e] = (hd >> 40) < 167772ull ? 1 : 0;
    }
    if (!a.obs_out) return;
    const uint64_t b = env_base(a.seed, a.agent, e, a.obs_step);
    if (blockIdx.x == 0 && threadIdx.x == 0) a.uniforms[e] = (float)(sm64(b + (3ull << 56)) >> 40) * 5.9604644775390625e-8f;
    if (a.frames) {
        uint64_t* out = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(a.obs_out) + (long)e * a.obs_elems);
        const long n8 = a.obs_elems / 8;   // 28224 bytes = 3528 words
        for (long j = blockIdx.x * (long)blockDim.x + threadIdx.x; j < n8; j += (long)gridDim.x * blockDim.x) out[j] = sm64(b + (uint64_t)j);
    } else {
        float* out = reinterpret_cast<float*>(a.obs_out) + (long)e * a.obs_elems;
        for (long j = blockIdx.x * (long)blockDim.x + threadIdx.x; j < a.obs_elems; j += (long)gridDim.x * blockDim.x)
            out[j] = ((float)(sm64(b + (uint64_t)j) >> 40) * 1.1920928955078125e-7f - 1.0f) * 1.7320508f;
    }
}

// *counter += by, after the last environment step of a rollout
__global__ void env_advance_kernel(long long* counter, long long by) {
    pdl_wait();
    pdl_launch();
    if (threadIdx.x == 0 && blockIdx.x == 0) *counter += by;
}
cudaError_t launch_env_advance(long long* counter, long long by, cudaStream_t st) {
    (void)launch_pdl(env_advance_kernel, dim3(1), dim3(32), 0, st, counter, by);
    return cudaGetLastError();
}

cudaError_t launch_env(const EnvArgs& a, int n_envs, cudaStream_t st) {
    if (n_envs < 1 || (a.frames && (a.obs_elems & 7))) return cudaErrorInvalidValue;
    const int bx = a.obs_out ? (a.frames ? 4 : 1) : 1;
    (void)launch_pdl(env_kernel, dim3(bx, n_envs), dim3(256), 0, st, a);
    return cudaGetLastError();
}

}  // namespace gala
