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
    static size_t opted = 0;   // raised only when a launch needs more (never lowered), so replays of a captured launch need no call
    if (smem > 40 * 1024 && smem > opted) {   // 40 KiB: well below the 48 KiB that need no opt-in
        cudaError_t e = cudaFuncSetAttribute(heads_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        opted = smem;
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

// ------------------------------------------------------------------------------------------
// Heads of the conv net in one kernel (hidden width 512, bf16-stored ReLU activations): policy and
// value outputs, the returns / advantages / objective of a2c_loss_kernel, and the gradient with
// respect to the hidden layer's pre-activation.  The only coupling between samples is the return
// recursion along the time axis of ONE environment, so a block takes a few environments of one
// agent with all their T+1 time steps (rows t*E + e of the agent's batch) and needs no other
// block; the three objective sums go through per-block partials and a fixed-order final sum by the
// agent's last block.  When the hidden layer's product arrives as split-K partial sums, the block
// also finishes that product for its rows (sum in split order, bias, ReLU, rounding to bf16) and
// stores the activations.
constexpr int kHeadsH = 512;
constexpr int kHeadsMaxA1 = 19;   // 18 actions + value

__global__ void __launch_bounds__(256) heads_fused_kernel(HeadsFusedArgs p) {
    extern __shared__ __align__(16) unsigned char hf_smem[];
    const int gz = blockIdx.y, bi = blockIdx.x;
    const int g = agent_slot(p.am, gz);   // the agent's tensors; the rollout pointers come with the launch (gz)
    const int T = p.T, E = p.E, A = p.A, A1 = A + 1, T1 = T + 1;
    const int e0 = bi * p.ne;
    const int ne = min(p.ne, E - e0);
    const int R = ne * T1;              // local row el * (T+1) + t  <->  row t * E + e0 + el of the agent's batch
    const int rcap = p.ne * T1;
    float* Wsm = reinterpret_cast<float*>(hf_smem);                                  // [A1][512]: pi.W rows, then v.W
    __nv_bfloat162* hsm = reinterpret_cast<__nv_bfloat162*>(Wsm + A1 * kHeadsH);     // [rcap][256]
    float* zsm = reinterpret_cast<float*>(hsm + rcap * (kHeadsH / 2));               // [rcap][A1] logits, value
    float* dsm = zsm + rcap * A1;                                                    // [rcap][A1] dL/dlogits, dL/dvalue
    float* gsm = dsm + rcap * A1;                                                    // [rcap] returns
    float* asm_ = gsm + rcap;                                                        // [rcap] advantages
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* P = p.params + (long)g * p.p_stride;
    const long B = p.B;

    // The head weights were last written by the optimiser pass, which lies at least two kernels back, so
    // they are fetched before the wait for the previous kernel.
    if (((p.piw | p.p_stride) & 3) == 0) {   // 16-byte loads when the policy weights are aligned
        const float4* src = reinterpret_cast<const float4*>(P + p.piw);
        for (int i = tid; i < A * (kHeadsH / 4); i += 256) reinterpret_cast<float4*>(Wsm)[i] = src[i];
    } else {
        for (int i = tid; i < A * kHeadsH; i += 256) Wsm[i] = P[p.piw + i];
    }
    for (int i = tid; i < kHeadsH; i += 256) Wsm[A * kHeadsH + i] = P[p.vw + i];
    pdl_wait();
    pdl_launch();
    if (p.partials) {
        const float* pg = p.partials + (long)g * p.partial_group_stride;
        __nv_bfloat16* hout = p.hid_out + (long)g * p.h_stride;
        for (int i = tid; i < R * (kHeadsH / 4); i += 256) {
            const int r = i / (kHeadsH / 4), c4 = i - r * (kHeadsH / 4);
            const int el = r / T1, t = r - el * T1;
            const long row = (long)t * E + e0 + el;
            const float4* src = reinterpret_cast<const float4*>(pg + row * kHeadsH) + c4;
            float4 acc = *src;
            for (int s0 = 1; s0 < p.split; s0 += 4) {   // fixed order; four loads in flight
                float4 v[4];
#pragma unroll
                for (int u = 0; u < 4; u++)
                    v[u] = s0 + u < p.split
                               ? *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(src) + (long)(s0 + u) * p.split_stride)
                               : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int u = 0; u < 4; u++)
                    if (s0 + u < p.split) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
            }
            const float* bg = P + p.fcb + c4 * 4;
            const __nv_bfloat162 h0 = __floats2bfloat162_rn(fmaxf(acc.x + bg[0], 0.f), fmaxf(acc.y + bg[1], 0.f));
            const __nv_bfloat162 h1 = __floats2bfloat162_rn(fmaxf(acc.z + bg[2], 0.f), fmaxf(acc.w + bg[3], 0.f));
            hsm[r * (kHeadsH / 2) + c4 * 2] = h0;
            hsm[r * (kHeadsH / 2) + c4 * 2 + 1] = h1;
            uint2 u;
            u.x = *reinterpret_cast<const unsigned*>(&h0); u.y = *reinterpret_cast<const unsigned*>(&h1);
            *reinterpret_cast<uint2*>(hout + row * kHeadsH + c4 * 4) = u;
        }
    } else {
        const __nv_bfloat16* hin = p.hid + (long)g * p.h_stride;
        for (int i = tid; i < R * (kHeadsH / 8); i += 256) {
            const int r = i / (kHeadsH / 8), c8 = i - r * (kHeadsH / 8);
            const int el = r / T1, t = r - el * T1;
            const long row = (long)t * E + e0 + el;
            reinterpret_cast<uint4*>(hsm + r * (kHeadsH / 2))[c8] = *(reinterpret_cast<const uint4*>(hin + row * kHeadsH) + c8);
        }
    }
    __syncthreads();

    // outputs: a warp takes three rows at a time, their 512 activations spread over the lanes (16 each) and
    // kept in registers, so that every weight fetched from shared memory serves three rows
    for (int r0 = warp * 3; r0 < R; r0 += 24) {
        float hx[3][16];
#pragma unroll
        for (int u = 0; u < 3; u++) {
            const int r = min(r0 + u, R - 1);
#pragma unroll
            for (int i = 0; i < 8; i++) {
                const float2 f = __bfloat1622float2(hsm[r * (kHeadsH / 2) + lane + 32 * i]);
                hx[u][2 * i] = f.x; hx[u][2 * i + 1] = f.y;
            }
        }
        for (int k = 0; k < A1; k++) {
            const float2* w2 = reinterpret_cast<const float2*>(Wsm + k * kHeadsH);
            float acc[3] = {0.0f, 0.0f, 0.0f};
#pragma unroll
            for (int i = 0; i < 8; i++) {
                const float2 w = w2[lane + 32 * i];
#pragma unroll
                for (int u = 0; u < 3; u++) {
                    acc[u] = fmaf(w.x, hx[u][2 * i], acc[u]);
                    acc[u] = fmaf(w.y, hx[u][2 * i + 1], acc[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < 3; u++)
                for (int off = 16; off > 0; off >>= 1) acc[u] += __shfl_xor_sync(0xffffffffu, acc[u], off);
            const float bk = k < A ? P[p.pib + k] : P[p.vb];
            if (lane < 3 && r0 + lane < R) zsm[(r0 + lane) * A1 + k] = (lane == 0 ? acc[0] : lane == 1 ? acc[1] : acc[2]) + bk;
        }
    }
    __syncthreads();
    {
        float* logits = p.logits + (long)g * B * A;
        float* values = p.values + (long)g * B;
        for (int i = tid; i < R * A1; i += 256) {
            const int r = i / A1, k = i - r * A1;
            const int el = r / T1, t = r - el * T1;
            const long row = (long)t * E + e0 + el;
            if (k < A) logits[row * A + k] = zsm[i]; else values[row] = zsm[i];
        }
    }
    const int* actions = reinterpret_cast<const int*>(p.actions.p[gz]);
    const float* rewards = reinterpret_cast<const float*>(p.rewards.p[gz]);
    const unsigned char* dones = reinterpret_cast<const unsigned char*>(p.dones.p[gz]);
    const long S = (long)T * E;
    // returns: a warp per environment, time steps in the lanes, reverse scan of the maps G -> r + gamma (1 - done) G
    for (int el = warp; el < ne; el += 8) {
        const int e = e0 + el;
        float carry = zsm[(el * T1 + T) * A1 + A];   // bootstrap V(s_T)
        for (int t_hi = T; t_hi > 0; t_hi -= 32) {
            const int t_lo = t_hi > 32 ? t_hi - 32 : 0;
            const int n = t_hi - t_lo;
            const int t = t_lo + lane;
            float a = 1.0f, b = 0.0f;
            if (lane < n) {
                a = p.gamma * (dones[(long)t * E + e] ? 0.0f : 1.0f);
                b = rewards[(long)t * E + e];
            }
            for (int off = 1; off < 32; off <<= 1) {
                const float a2 = __shfl_down_sync(0xffffffffu, a, off);
                const float b2 = __shfl_down_sync(0xffffffffu, b, off);
                if (lane + off < 32) { b = a * b2 + b; a = a * a2; }
            }
            const float gt = a * carry + b;
            if (lane < n) {
                gsm[el * T1 + t] = gt;
                asm_[el * T1 + t] = gt - zsm[(el * T1 + t) * A1 + A];
            }
            carry = __shfl_sync(0xffffffffu, gt, 0);
        }
    }
    __syncthreads();

    float lp = 0.0f, lv = 0.0f, le = 0.0f;
    const float invS = 1.0f / (float)S;
    for (int i = tid; i < ne * T; i += 256) {
        const int el = i / T, t = i - el * T;
        const int r = el * T1 + t;
        const long srow = (long)t * E + e0 + el;
        const float* z = zsm + r * A1;
        float mx = z[0];
        for (int k = 1; k < A; k++) mx = fmaxf(mx, z[k]);
        float sum = 0.0f;
        for (int k = 0; k < A; k++) sum += expf(z[k] - mx);
        const float lse = mx + logf(sum);
        float H = 0.0f;
        for (int k = 0; k < A; k++) { const float lg = z[k] - lse; H -= expf(lg) * lg; }
        const int act = actions[srow];
        const float adv = asm_[r], gt = gsm[r], v = z[A];
        float* dz = p.dlogits + ((long)g * S + srow) * A;
        for (int k = 0; k < A; k++) {
            const float lg = z[k] - lse, pi = expf(lg);
            const float d = (adv * (pi - (k == act ? 1.0f : 0.0f)) + p.ent_coef * pi * (lg + H)) * invS;
            dsm[r * A1 + k] = d;
            dz[k] = d;
        }
        const float dvv = 2.0f * p.vf_coef * (v - gt) * invS;
        dsm[r * A1 + A] = dvv;
        {   // the same numbers as one padded row (dlogits, dvalue, zeros) for the weight-gradient kernel
            float* row = p.dzv + ((long)g * S + srow) * (kHeadsMaxA1 + 1);
            for (int k = 0; k < A1; k++) row[k] = dsm[r * A1 + k];
            for (int k = A1; k < kHeadsMaxA1 + 1; k++) row[k] = 0.0f;
        }
        p.dvalues[(long)g * S + srow] = dvv;
        p.returns[(long)g * S + srow] = gt;
        p.adv[(long)g * S + srow] = adv;
        lp += -(z[act] - lse) * adv;
        lv += (gt - v) * (gt - v);
        le += H;
    }
    __shared__ float red[3][256];
    __shared__ bool last;
    red[0][tid] = lp; red[1][tid] = lv; red[2][tid] = le;
    __syncthreads();   // also publishes dsm
    for (int st = 128; st > 0; st >>= 1) {
        if (tid < st)
            for (int q = 0; q < 3; q++) red[q][tid] += red[q][tid + st];
        __syncthreads();
    }
    if (tid == 0) {
        float* lpart = p.loss_partial + ((long)g * E + bi) * 4;
        lpart[0] = red[0][0]; lpart[1] = red[1][0]; lpart[2] = red[2][0];
        __threadfence();
        last = atomicAdd(p.ticket + g, 1u) == gridDim.x - 1;
    }

    // gradient of the hidden pre-activation: thread owns columns 2 tid, 2 tid + 1; its slice of the head
    // weights sits in registers, the samples' dL/dlogits, dL/dvalue are broadcast from shared memory
    float2 wr[kHeadsMaxA1];
#pragma unroll
    for (int k = 0; k < kHeadsMaxA1; k++)
        wr[k] = k < A1 ? reinterpret_cast<const float2*>(Wsm + k * kHeadsH)[tid] : make_float2(0.f, 0.f);
    __nv_bfloat16* dh = p.dh + (long)g * p.dh_stride;
    for (int i = 0; i < ne * T; i++) {
        const int el = i / T, t = i - el * T;
        const int r = el * T1 + t;
        const long srow = (long)t * E + e0 + el;
        float a0 = 0.0f, a1 = 0.0f;
#pragma unroll
        for (int k = 0; k < kHeadsMaxA1; k++)
            if (k < A1) {
                const float d = dsm[r * A1 + k];
                a0 = fmaf(d, wr[k].x, a0);
                a1 = fmaf(d, wr[k].y, a1);
            }
        const float2 h = __bfloat1622float2(hsm[r * (kHeadsH / 2) + tid]);
        const __nv_bfloat162 o = __floats2bfloat162_rn(h.x > 0.0f ? a0 : 0.0f, h.y > 0.0f ? a1 : 0.0f);
        reinterpret_cast<__nv_bfloat162*>(dh + srow * kHeadsH)[tid] = o;
    }
    __syncthreads();
    if (last) {   // the agent's last block adds the blocks' sums in block order
        __threadfence();
        const volatile float* lp0 = p.loss_partial + (long)g * E * 4;
        float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f;
        for (unsigned k0 = 0; k0 < gridDim.x; k0 += 256) {
            const unsigned k = k0 + tid;
            __syncthreads();
            if (k < gridDim.x) { red[0][tid] = lp0[k * 4]; red[1][tid] = lp0[k * 4 + 1]; red[2][tid] = lp0[k * 4 + 2]; }
            __syncthreads();
            if (tid == 0)
                for (unsigned q = 0; q < min(256u, gridDim.x - k0); q++) { s0 += red[0][q]; s1 += red[1][q]; s2 += red[2][q]; }
        }
        if (tid == 0) {
            p.losses[g * 4 + 0] = s0 * invS;
            p.losses[g * 4 + 1] = s1 * invS;
            p.losses[g * 4 + 2] = s2 * invS;
            p.ticket[g] = 0;   // ready for the next launch
        }
    }
}

int heads_fused_envs_per_block(int T, int E, int groups) {
    int ne = 32 / (T + 1);
    if (ne > E) ne = E;
    if (ne < 1) ne = 1;
    while (ne > 1 && (long)groups * ((E + ne - 1) / ne) < 296) ne--;
    return ne;
}
static size_t heads_fused_smem(int A, int rcap) {
    const int A1 = A + 1;
    return (size_t)A1 * kHeadsH * 4 + (size_t)rcap * kHeadsH * 2 + (size_t)rcap * A1 * 8 + (size_t)rcap * 8;
}
bool heads_fused_supported(int T, int E, int A, int H) {
    return H == kHeadsH && A + 1 <= kHeadsMaxA1 && A >= 1 && T >= 1 && E >= 1 &&
           heads_fused_smem(A, T + 1) <= 160 * 1024;
}
int heads_fused_blocks(int T, int E, int groups) {
    const int ne = heads_fused_envs_per_block(T, E, groups);
    return (E + ne - 1) / ne;
}
cudaError_t launch_heads_fused(const HeadsFusedArgs& a0, int groups, cudaStream_t st) {
    HeadsFusedArgs a = a0;
    if (!heads_fused_supported(a.T, a.E, a.A, kHeadsH)) return cudaErrorNotSupported;
    a.ne = heads_fused_envs_per_block(a.T, a.E, groups);
    const size_t smem = heads_fused_smem(a.A, a.ne * (a.T + 1));
    // always opt in: the 48 KiB that need no opt-in include the kernel's static shared memory, so a dynamic size
    // just below 48 KiB would already be refused
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(heads_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(160 * 1024));
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    (void)launch_pdl(heads_fused_kernel, dim3((a.E + a.ne - 1) / a.ne, groups), dim3(256), smem, st, a);
    return cudaGetLastError();
}

// Parameter gradients of the heads, d pi.W[k][j] = sum_s dz[s][k] h[s][j] (k = A: value head) and the
// biases as one more column tile whose "activation" is 1.  A block owns 32 columns of one agent; its
// eight warps take contiguous slices of the samples (lane = column, one accumulator per output row),
// and the slices are added in warp order, so the sum has a fixed order.
__global__ void __launch_bounds__(256) heads_wgrad_tiled_kernel(HeadsBwdArgs a) {
    pdl_wait();
    pdl_launch();
    constexpr int kChunk = 256;
    __shared__ __align__(16) float dzs[kChunk][kHeadsMaxA1 + 1];   // rows of 20 floats; entries from A + 1 on are zero
    __shared__ float part[8][kHeadsMaxA1][32];
    const int g = agent_slot(a.am, blockIdx.y), tile = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int A = a.A, A1 = A + 1, H = a.H;
    const bool bias_tile = tile * 32 >= H;
    const char* hbase = reinterpret_cast<const char*>(a.h) + (long)g * a.h_stride * (a.h_bf16 ? 2 : 4);
    const float* dz = a.dlogits + (long)g * a.dlogits_stride;
    const float* dv = a.dvalues + (long)g * a.dvalues_stride;
    const int j = tile * 32 + lane;
    float acc[kHeadsMaxA1];
#pragma unroll
    for (int k = 0; k < kHeadsMaxA1; k++) acc[k] = 0.0f;
    for (int s0 = 0; s0 < a.rows; s0 += kChunk) {
        const int n = min(kChunk, a.rows - s0);
        __syncthreads();
        if (a.dzv) {   // padded rows written by the fused heads kernel: a straight copy
            const float4* src = reinterpret_cast<const float4*>(a.dzv + ((long)g * a.rows + s0) * (kHeadsMaxA1 + 1));
            for (int i = tid; i < n * ((kHeadsMaxA1 + 1) / 4); i += 256) reinterpret_cast<float4*>(&dzs[0][0])[i] = src[i];
        } else {
            for (int i = tid; i < n * (kHeadsMaxA1 + 1); i += 256) {
                const int s = i / (kHeadsMaxA1 + 1), k = i - s * (kHeadsMaxA1 + 1);
                dzs[s][k] = k < A ? dz[(long)(s0 + s) * A + k] : (k == A ? dv[s0 + s] : 0.0f);
            }
        }
        __syncthreads();
        const int per = (n + 7) / 8;
        const int lo = warp * per, hi = min(n, lo + per);
        for (int sb = lo; sb < hi; sb += 8) {   // eight activations in flight, then their products
            float hv[8];
#pragma unroll
            for (int u = 0; u < 8; u++)
                hv[u] = sb + u < hi ? (bias_tile ? 1.0f : ld_in(hbase, (long)(s0 + sb + u) * H + j, a.h_bf16)) : 0.0f;
#pragma unroll
            for (int u = 0; u < 8; u++) {
                if (sb + u < hi) {
                    const float4* d4 = reinterpret_cast<const float4*>(&dzs[sb + u][0]);
#pragma unroll
                    for (int k4 = 0; k4 < (kHeadsMaxA1 + 1) / 4; k4++) {
                        if (k4 * 4 < A1) {
                            const float4 d = d4[k4];
                            acc[k4 * 4] = fmaf(d.x, hv[u], acc[k4 * 4]);
                            if (k4 * 4 + 1 < kHeadsMaxA1) acc[k4 * 4 + 1] = fmaf(d.y, hv[u], acc[k4 * 4 + 1]);
                            if (k4 * 4 + 2 < kHeadsMaxA1) acc[k4 * 4 + 2] = fmaf(d.z, hv[u], acc[k4 * 4 + 2]);
                            if (k4 * 4 + 3 < kHeadsMaxA1) acc[k4 * 4 + 3] = fmaf(d.w, hv[u], acc[k4 * 4 + 3]);
                        }
                    }
                }
            }
        }
    }
#pragma unroll
    for (int k = 0; k < kHeadsMaxA1; k++)
        if (k < A1) part[warp][k][lane] = acc[k];
    __syncthreads();
    float* G = a.grad + (long)g * a.g_stride;
    for (int i = tid; i < A1 * 32; i += 256) {
        const int k = i >> 5, l = i & 31;
        float s = part[0][k][l];
        for (int w = 1; w < 8; w++) s += part[w][k][l];
        if (!bias_tile) {
            if (k < A) G[a.piw + (long)k * H + tile * 32 + l] = s; else G[a.vw + tile * 32 + l] = s;
        } else if (l == 0) {
            if (k < A) G[a.pib + k] = s; else G[a.vb] = s;
        }
    }
}
cudaError_t launch_heads_wgrad_tiled(const HeadsBwdArgs& a, int groups, cudaStream_t st) {
    if (a.A + 1 > kHeadsMaxA1 || (a.H & 31)) return cudaErrorNotSupported;
    (void)launch_pdl(heads_wgrad_tiled_kernel, dim3(a.H / 32 + 1, groups), dim3(256), 0, st, a);
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
