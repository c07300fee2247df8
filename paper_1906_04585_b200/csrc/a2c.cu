// Returns, advantages and the A2C objective (Sec. 2, Eqs. 1-4; Algorithm 1 "compute returns
// and advantages"), action sampling (Algorithm 1 acting step), and the small dense layers
// (policy/value heads, MLP trunk) that run on the CUDA cores in fp32.
#include "internal.h"

namespace gala {

__device__ __forceinline__ float ld_in(const void* p, long i, int is_bf16) {
    return is_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[i])
                   : reinterpret_cast<const float*>(p)[i];
}
__device__ __forceinline__ void st_out(void* p, long i, float v, int is_bf16) {
    if (is_bf16) reinterpret_cast<__nv_bfloat16*>(p)[i] = __float2bfloat16_rn(v);
    else reinterpret_cast<float*>(p)[i] = v;
}
__device__ __forceinline__ float act_apply(int act, float z) {
    return act == 1 ? fmaxf(z, 0.0f) : (act == 2 ? tanhf(z) : z);
}
// derivative through the OUTPUT a = act(z)
__device__ __forceinline__ float act_deriv(int act, float a) {
    return act == 1 ? (a > 0.0f ? 1.0f : 0.0f) : (act == 2 ? 1.0f - a * a : 1.0f);
}

// ------------------------------------------------------------------------------------------
// One block per agent.
// Phase 1 - n-step returns truncated at the rollout end: G_T = V(s_T),
//   G_t = r_t + gamma (1 - done_t) G_{t+1}.  Each step is the affine map G -> b + a G with
//   a = gamma (1 - done_t), b = r_t; a warp holds up to 32 consecutive steps of one environment
//   in its lanes and composes the maps with a reverse (suffix) scan of shuffles, so the time
//   axis costs log2(32) steps instead of T.
// Phase 2 - per sample: softmax, log pi(a), entropy, and the derivative of
//   L = mean[-log pi(a) Adv - eta H] + c_v mean[(G - V)^2] w.r.t. logits and value,
//   Adv and G held constant.
__global__ void __launch_bounds__(256) a2c_loss_kernel(LossArgs p) {
    pdl_wait();
    pdl_launch();
    const int agent = blockIdx.x;
    const int T = p.T, E = p.E, A = p.A, S = T * E;
    const float* logits = p.logits + (long)agent * p.B * A;
    const float* values = p.values + (long)agent * p.B;
    const int* actions = reinterpret_cast<const int*>(p.actions.p[agent]);
    const float* rewards = reinterpret_cast<const float*>(p.rewards.p[agent]);
    const unsigned char* dones = reinterpret_cast<const unsigned char*>(p.dones.p[agent]);
    float* G = p.returns + (long)agent * S;
    float* Adv = p.adv + (long)agent * S;
    float* dz = p.dlogits + (long)agent * S * A;
    float* dv = p.dvalues + (long)agent * S;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    for (int e = warp; e < E; e += nwarps) {
        float carry = values[(long)T * E + e];  // bootstrap V(s_T)
        for (int t_hi = T; t_hi > 0; t_hi -= 32) {
            const int t_lo = t_hi > 32 ? t_hi - 32 : 0;
            const int n = t_hi - t_lo;
            const int t = t_lo + lane;
            float a = 1.0f, b = 0.0f;  // identity map for idle lanes
            if (lane < n) {
                a = p.gamma * (dones[(long)t * E + e] ? 0.0f : 1.0f);
                b = rewards[(long)t * E + e];
            }
            // suffix scan: after it lane l holds f_l o f_{l+1} o ... o f_{n-1}
            for (int off = 1; off < 32; off <<= 1) {
                float a2 = __shfl_down_sync(0xffffffffu, a, off);
                float b2 = __shfl_down_sync(0xffffffffu, b, off);
                if (lane + off < 32) { b = a * b2 + b; a = a * a2; }
            }
            float g = a * carry + b;
            if (lane < n) {
                G[(long)t * E + e] = g;
                Adv[(long)t * E + e] = g - values[(long)t * E + e];
            }
            carry = __shfl_sync(0xffffffffu, g, 0);
        }
    }
    __syncthreads();

    float lp = 0.0f, lv = 0.0f, le = 0.0f;
    const float invS = 1.0f / (float)S;
    for (int s = threadIdx.x; s < S; s += blockDim.x) {
        const float* z = logits + (long)s * A;
        float mx = z[0];
        for (int k = 1; k < A; k++) mx = fmaxf(mx, z[k]);
        float sum = 0.0f;
        for (int k = 0; k < A; k++) sum += expf(z[k] - mx);
        const float lse = mx + logf(sum);
        float H = 0.0f;
        for (int k = 0; k < A; k++) { float lg = z[k] - lse; H -= expf(lg) * lg; }
        const int act = actions[s];
        const float adv = Adv[s], g = G[s], v = values[s];
        for (int k = 0; k < A; k++) {
            float lg = z[k] - lse, pi = expf(lg);
            float d = adv * (pi - (k == act ? 1.0f : 0.0f)) + p.ent_coef * pi * (lg + H);
            dz[(long)s * A + k] = d * invS;
        }
        dv[s] = 2.0f * p.vf_coef * (v - g) * invS;
        lp += -(z[act] - lse) * adv;
        lv += (g - v) * (g - v);
        le += H;
    }
    __shared__ float red[3][256];
    red[0][threadIdx.x] = lp; red[1][threadIdx.x] = lv; red[2][threadIdx.x] = le;
    __syncthreads();
    for (int st = 128; st > 0; st >>= 1) {
        if (threadIdx.x < st)
            for (int q = 0; q < 3; q++) red[q][threadIdx.x] += red[q][threadIdx.x + st];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        p.losses[agent * 4 + 0] = red[0][0] * invS;
        p.losses[agent * 4 + 1] = red[1][0] * invS;
        p.losses[agent * 4 + 2] = red[2][0] * invS;
    }
}

cudaError_t launch_a2c_loss(const LossArgs& a, int n_agents, cudaStream_t st) {
    (void)launch_pdl(a2c_loss_kernel, dim3(n_agents), dim3(256), 0, st, a);
    return cudaGetLastError();
}

// Inverse-CDF draw: smallest k with sum_{j<=k} pi_j > u, clamped to A-1.
__global__ void sample_kernel(const float* __restrict__ logits, const float* __restrict__ u,
                              int* __restrict__ actions, int E, int A) {
    pdl_wait();
    pdl_launch();
    int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= E) return;
    const float* z = logits + (long)e * A;
    float mx = z[0];
    for (int k = 1; k < A; k++) mx = fmaxf(mx, z[k]);
    float sum = 0.0f;
    for (int k = 0; k < A; k++) sum += expf(z[k] - mx);
    float cdf = 0.0f;
    int a = A - 1;
    const float ue = u[e];
    for (int k = 0; k < A; k++) {
        cdf += expf(z[k] - mx) / sum;
        if (cdf > ue) { a = k; break; }
    }
    actions[e] = a;
}
cudaError_t launch_sample(const float* logits, const float* uniforms, int* actions, int E, int A,
                          cudaStream_t st) {
    (void)launch_pdl(sample_kernel, dim3((E + 127) / 128), dim3(128), 0, st, logits, uniforms, actions, E, A);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// out[r][o] = act(sum_i in[r][i] W[o][i] + b[o]); one warp per output row r, lanes over o with
// the input row staged in shared memory.
__global__ void __launch_bounds__(256) dense_fwd_kernel(DenseArgs a) {
    pdl_wait();
    pdl_launch();
    extern __shared__ float xin[];  // [warps][in_dim]
    const int g = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const float* W = a.W + (long)g * a.w_stride;
    const float* b = a.b + (long)g * a.w_stride;
    const void* in = a.in.p[g];
    float* xs = xin + warp * a.in_dim;
    for (int r = blockIdx.x * nwarps + warp; r < a.rows; r += gridDim.x * nwarps) {
        for (int i = lane; i < a.in_dim; i += 32) xs[i] = ld_in(in, (long)r * a.in_dim + i, a.in_bf16);
        __syncwarp();
        for (int o = lane; o < a.out_dim; o += 32) {
            float acc = b[o];
            const float* w = W + (long)o * a.in_dim;
            for (int i = 0; i < a.in_dim; i++) acc = fmaf(w[i], xs[i], acc);
            st_out(a.out, (long)g * a.out_stride + (long)r * a.out_dim + o, act_apply(a.act, acc), a.out_bf16);
        }
        __syncwarp();
    }
}
cudaError_t launch_dense_fwd(const DenseArgs& a, int groups, cudaStream_t st) {
    int bx = (a.rows + 7) / 8;
    if (bx > 64) bx = 64;
    dim3 grid(bx, groups);
    (void)launch_pdl(dense_fwd_kernel, dim3(grid), dim3(256), 8 * a.in_dim * sizeof(float), st, a);
    return cudaGetLastError();
}

// Heads: logits[r][k] = h[r] . pi.W[k] + pi.b[k], value[r] = h[r] . v.W + v.b.
// The (A+1) x H head weights are staged in shared memory once per block (they would otherwise be
// re-read from L2 with the full latency for every output); one warp per row, the dot products
// are split over lanes and combined by a butterfly.
__global__ void __launch_bounds__(256) heads_fwd_kernel(HeadsArgs a) {
    pdl_wait();
    pdl_launch();
    extern __shared__ float hsm[];  // [A+1][H] weights, then [warps][H] rows
    const int g = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const float* P = a.params + (long)g * a.p_stride;
    const char* hbase = reinterpret_cast<const char*>(a.h) + (long)g * a.h_stride * (a.h_bf16 ? 2 : 4);
    float* wsm = hsm;
    float* hrow = hsm + (a.A + 1) * a.H + warp * a.H;
    for (int i = threadIdx.x; i < a.A * a.H; i += blockDim.x) wsm[i] = P[a.piw + i];
    for (int i = threadIdx.x; i < a.H; i += blockDim.x) wsm[a.A * a.H + i] = P[a.vw + i];
    __syncthreads();
    for (int r = blockIdx.x * nwarps + warp; r < a.rows; r += gridDim.x * nwarps) {
        for (int i = lane; i < a.H; i += 32) hrow[i] = ld_in(hbase, (long)r * a.H + i, a.h_bf16);
        __syncwarp();
        for (int k = 0; k <= a.A; k++) {
            const float* w = wsm + k * a.H;
            float acc = 0.0f;
            for (int i = lane; i < a.H; i += 32) acc = fmaf(w[i], hrow[i], acc);
            for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (lane == 0) {
                if (k < a.A) a.logits[(long)g * a.logits_stride + (long)r * a.A + k] = acc + P[a.pib + k];
                else a.values[(long)g * a.values_stride + r] = acc + P[a.vb];
            }
        }
        __syncwarp();
    }
}
cudaError_t launch_heads_fwd(const HeadsArgs& a, int groups, cudaStream_t st) {
    int bx = (a.rows + 7) / 8;     // one row per warp while that still gives few enough blocks
    if (bx * groups > 592) bx = (592 + groups - 1) / groups;
    if (bx < 1) bx = 1;
    const size_t smem = (size_t)((a.A + 1) + 8) * a.H * sizeof(float);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(heads_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    (void)launch_pdl(heads_fwd_kernel, dim3(dim3(bx, groups)), dim3(256), smem, st, a);
    return cudaGetLastError();
}

// Heads backward, data part: dpre[s][j] = (sum_k dz[s][k] pi.W[k][j] + dv[s] v.W[j]) * act'(h[s][j]).
__global__ void __launch_bounds__(256) heads_dgrad_kernel(HeadsBwdArgs a) {
    pdl_wait();
    pdl_launch();
    const int g = blockIdx.y;
    const float* P = a.params + (long)g * a.p_stride;
    const char* hbase = reinterpret_cast<const char*>(a.h) + (long)g * a.h_stride * (a.h_bf16 ? 2 : 4);
    const float* dz = a.dlogits + (long)g * a.dlogits_stride;
    const float* dv = a.dvalues + (long)g * a.dvalues_stride;
    const long total = (long)a.rows * a.H;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int s = (int)(idx / a.H), j = (int)(idx % a.H);
        float acc = dv[s] * P[a.vw + j];
        for (int k = 0; k < a.A; k++) acc = fmaf(dz[(long)s * a.A + k], P[a.piw + (long)k * a.H + j], acc);
        const float h = ld_in(hbase, idx, a.h_bf16);
        st_out(a.dpre, (long)g * a.dpre_stride + idx, acc * act_deriv(a.act, h), a.dpre_bf16);
    }
}
// Heads backward, parameter part: d pi.W[k][j] = sum_s dz[s][k] h[s][j] (k = A: value head),
// biases are the plain sums over s.  Serial over s: fixed summation order.
__global__ void __launch_bounds__(256) heads_wgrad_kernel(HeadsBwdArgs a) {
    pdl_wait();
    pdl_launch();
    const int g = blockIdx.y;
    const char* hbase = reinterpret_cast<const char*>(a.h) + (long)g * a.h_stride * (a.h_bf16 ? 2 : 4);
    const float* dz = a.dlogits + (long)g * a.dlogits_stride;
    const float* dv = a.dvalues + (long)g * a.dvalues_stride;
    float* G = a.grad + (long)g * a.g_stride;
    const long nW = (long)(a.A + 1) * a.H;
    const long total = nW + a.A + 1;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        if (idx < nW) {
            const int k = (int)(idx / a.H), j = (int)(idx % a.H);
            float acc = 0.0f;
            if (k < a.A)
                for (int s = 0; s < a.rows; s++) acc = fmaf(dz[(long)s * a.A + k], ld_in(hbase, (long)s * a.H + j, a.h_bf16), acc);
            else
                for (int s = 0; s < a.rows; s++) acc = fmaf(dv[s], ld_in(hbase, (long)s * a.H + j, a.h_bf16), acc);
            if (k < a.A) G[a.piw + (long)k * a.H + j] = acc; else G[a.vw + j] = acc;
        } else {
            const int k = (int)(idx - nW);
            float acc = 0.0f;
            if (k < a.A) { for (int s = 0; s < a.rows; s++) acc += dz[(long)s * a.A + k]; G[a.pib + k] = acc; }
            else { for (int s = 0; s < a.rows; s++) acc += dv[s]; G[a.vb] = acc; }
        }
    }
}
cudaError_t launch_heads_dgrad(const HeadsBwdArgs& a, int groups, cudaStream_t st) {
    long total = (long)a.rows * a.H;
    int bx = (int)((total + 255) / 256);
    if (bx > 256) bx = 256;
    (void)launch_pdl(heads_dgrad_kernel, dim3(dim3(bx, groups)), dim3(256), 0, st, a);
    return cudaGetLastError();
}
cudaError_t launch_heads_wgrad(const HeadsBwdArgs& a, int groups, cudaStream_t st) {
    long tw = (long)(a.A + 1) * (a.H + 1);
    int bw = (int)((tw + 255) / 256);
    (void)launch_pdl(heads_wgrad_kernel, dim3(dim3(bw, groups)), dim3(256), 0, st, a);
    return cudaGetLastError();
}

// Dense layer backward (MLP trunk): gW[o][i] = sum_r dpre[r][o] in[r][i], gb[o] = sum_r dpre[r][o],
// and (if din) din[r][i] = (sum_o dpre[r][o] W[o][i]) * act'(in[r][i]).
__global__ void __launch_bounds__(256) dense_wgrad_kernel(DenseBwdArgs a) {
    pdl_wait();
    pdl_launch();
    const int g = blockIdx.y;
    const float* in = reinterpret_cast<const float*>(a.in.p[g]);
    const float* dp = a.dpre + (long)g * a.dpre_stride;
    float* gW = a.gW + (long)g * a.g_stride;
    float* gb = a.gb + (long)g * a.g_stride;
    const long nW = (long)a.out_dim * a.in_dim, total = nW + a.out_dim;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        float acc = 0.0f;
        if (idx < nW) {
            const int o = (int)(idx / a.in_dim), i = (int)(idx % a.in_dim);
            for (int r = 0; r < a.rows; r++) acc = fmaf(dp[(long)r * a.out_dim + o], in[(long)r * a.in_dim + i], acc);
            gW[idx] = acc;
        } else {
            const int o = (int)(idx - nW);
            for (int r = 0; r < a.rows; r++) acc += dp[(long)r * a.out_dim + o];
            gb[o] = acc;
        }
    }
}
__global__ void __launch_bounds__(256) dense_dgrad_kernel(DenseBwdArgs a) {
    pdl_wait();
    pdl_launch();
    const int g = blockIdx.y;
    const float* in = reinterpret_cast<const float*>(a.in.p[g]);
    const float* dp = a.dpre + (long)g * a.dpre_stride;
    const float* W = a.W + (long)g * a.w_stride;
    float* din = a.din + (long)g * a.din_stride;
    const long total = (long)a.rows * a.in_dim;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int r = (int)(idx / a.in_dim), i = (int)(idx % a.in_dim);
        float acc = 0.0f;
        for (int o = 0; o < a.out_dim; o++) acc = fmaf(dp[(long)r * a.out_dim + o], W[(long)o * a.in_dim + i], acc);
        din[idx] = acc * act_deriv(a.act_in, in[idx]);
    }
}
cudaError_t launch_dense_bwd(const DenseBwdArgs& a, int groups, cudaStream_t st) {
    long tw = (long)a.out_dim * (a.in_dim + 1);
    int bw = (int)((tw + 255) / 256);
    if (bw > 1024) bw = 1024;
    (void)launch_pdl(dense_wgrad_kernel, dim3(dim3(bw, groups)), dim3(256), 0, st, a);
    if (a.din) {
        long td = (long)a.rows * a.in_dim;
        int bd = (int)((td + 255) / 256);
        if (bd > 1024) bd = 1024;
        (void)launch_pdl(dense_dgrad_kernel, dim3(dim3(bd, groups)), dim3(256), 0, st, a);
    }
    return cudaGetLastError();
}

}  // namespace gala
