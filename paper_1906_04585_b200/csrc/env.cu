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

// The same for all agents of a lockstep loop in one launch (grid.z = agent), with the action draw folded in: block
// (0, e, i) first draws agent i's action for environment e at `step` from its logits (the inverse-CDF rule of the
// sampling kernel, operation for operation, with the uniform of tag 3 computed in place) and writes the reward and
// the done flag of that transition; all blocks then write the observation of step + 1.  With draw == 0 only the
// observation of `step` itself is written (the one a rollout starts from).
__global__ void __launch_bounds__(256) env_act_all_kernel(EnvActArgs a) {
    pdl_wait();
    pdl_launch();
    const int e = blockIdx.y, i = a.agent0 + blockIdx.z;
    const long long step = a.step + a.step_base[i];
    __shared__ float head_part[8][32];
    __shared__ float head_z[32];
    if (a.draw && blockIdx.x == 0 && a.H > 0) {
        // policy head of this environment: 256 threads over the hidden units, A dot products reduced over the block
        const float* par = a.params + (long)i * a.p_stride;
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        float acc[32];
#pragma unroll
        for (int k = 0; k < 32; k++) acc[k] = 0.0f;
        for (int u = threadIdx.x; u < a.H; u += blockDim.x) {
            float h;
            if (a.split > 0) {
                const float* ps = a.partials + (long)blockIdx.z * a.partial_group_stride + (long)e * a.H + u;
                float sum = 0.0f;
                for (int s = 0; s < a.split; s++) sum += ps[(long)s * a.split_stride];
                h = __bfloat162float(__float2bfloat16(fmaxf(sum + par[a.fcb + u], 0.0f)));
            } else {
                h = __bfloat162float(a.hid[(long)i * a.h_stride + (long)e * a.H + u]);
            }
#pragma unroll
            for (int k = 0; k < 32; k++)
                if (k < a.n_actions) acc[k] = fmaf(h, par[a.piw + (long)k * a.H + u], acc[k]);
        }
#pragma unroll
        for (int k = 0; k < 32; k++) {
            if (k < a.n_actions) {
                float v = acc[k];
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lane == 0) head_part[warp][k] = v;
            }
        }
        __syncthreads();
        if (threadIdx.x < a.n_actions) {
            float v = par[a.pib + threadIdx.x];
            for (int w8 = 0; w8 < 8; w8++) v += head_part[w8][threadIdx.x];
            head_z[threadIdx.x] = v;
        }
        __syncthreads();
    }
    if (a.draw && blockIdx.x == 0 && threadIdx.x == 0) {
        const uint64_t b = env_base(a.seed, i, e, step);
        const float ue = (float)(sm64(b + (3ull << 56)) >> 40) * 5.9604644775390625e-8f;
        const float* z = a.H > 0 ? head_z : a.logits + (long)i * a.logits_stride + (long)e * a.n_actions;
        const int A = a.n_actions;
        float mx = z[0];
        for (int k = 1; k < A; k++) mx = fmaxf(mx, z[k]);
        float sum = 0.0f;
        for (int k = 0; k < A; k++) sum += expf(z[k] - mx);
        float cdf = 0.0f;
        int act = A - 1;
        for (int k = 0; k < A; k++) {
            cdf += expf(z[k] - mx) / sum;
            if (cdf > ue) { act = k; break; }
        }
        const long o = (long)i * a.te_stride + a.te_off + e;
        a.actions[o] = act;
        const uint64_t hr = sm64(b + (1ull << 56)), hd = sm64(b + (2ull << 56));
        a.rewards[o] = (int)(hr % (uint64_t)A) == act ? 1.0f : 0.0f;
        a.dones[o] = (hd >> 40) < 167772ull ? 1 : 0;
    }
    const uint64_t b = env_base(a.seed, i, e, step + (a.draw ? 1 : 0));
    uint8_t* base = reinterpret_cast<uint8_t*>(a.obs_out) + (long)i * a.obs_agent_stride + a.obs_off;
    if (a.frames) {
        uint64_t* out = reinterpret_cast<uint64_t*>(base + (long)e * a.obs_elems);
        const long n8 = a.obs_elems / 8;
        for (long j = blockIdx.x * (long)blockDim.x + threadIdx.x; j < n8; j += (long)gridDim.x * blockDim.x) out[j] = sm64(b + (uint64_t)j);
    } else {
        float* out = reinterpret_cast<float*>(base) + (long)e * a.obs_elems;
        for (long j = blockIdx.x * (long)blockDim.x + threadIdx.x; j < a.obs_elems; j += (long)gridDim.x * blockDim.x)
            out[j] = ((float)(sm64(b + (uint64_t)j) >> 40) * 1.1920928955078125e-7f - 1.0f) * 1.7320508f;
    }
}
cudaError_t launch_env_act_all(const EnvActArgs& a, int n_envs, int n_agents, cudaStream_t st) {
    if (n_envs < 1 || n_agents < 1 || n_agents > 65535 || (a.frames && (a.obs_elems & 7)) || !a.step_base || !a.obs_out ||
        a.n_actions < 1 || a.n_actions > 32)
        return cudaErrorInvalidValue;
    (void)launch_pdl(env_act_all_kernel, dim3(a.frames ? 4 : 1, n_envs, n_agents), dim3(256), 0, st, a);
    return cudaGetLastError();
}
// counter[i] += by for the agents of a lockstep loop
__global__ void env_advance_all_kernel(long long* counters, int n, long long by) {
    pdl_wait();
    pdl_launch();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) counters[i] += by;
}
cudaError_t launch_env_advance_all(long long* counters, int n, long long by, cudaStream_t st) {
    (void)launch_pdl(env_advance_all_kernel, dim3((n + 63) / 64), dim3(64), 0, st, counters, n, by);
    return cudaGetLastError();
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
