// Learner step of the small MLP policy / value network (two tanh layers, linear policy and value heads) in one
// kernel: a block takes a few environments of one agent with all their time steps (samples are coupled only
// along the time axis of one environment); the agent's whole parameter vector, the block's part of the rollout
// and every activation live in shared memory.  The blocks of an agent leave partial gradients, and the last of
// them to finish adds these up in block order.  Forward on the (T+1) E observations, n-step returns truncated at the rollout end (Sec. 2),
// advantages, the A2C objective of Eqs. 1-4 and its gradient, backward through the net in fp32, the flat
// gradient, its global norm and the clip coefficient (Table 2).  All sums run in a fixed order.
//
// Shared-memory rows are padded by one float so that "thread = row" loops read distinct banks while the
// weights they share are broadcast.
#include "internal.h"

namespace gala {

constexpr int kMlpThreads = 512;

__device__ __forceinline__ float block_sum_fixed(float v, float* red) {   // fixed-shape tree over the block
    red[threadIdx.x] = v;
    __syncthreads();
    for (int st = kMlpThreads / 2; st > 0; st >>= 1) {
        if ((int)threadIdx.x < st) red[threadIdx.x] += red[threadIdx.x + st];
        __syncthreads();
    }
    const float r = red[0];
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(kMlpThreads) mlp_fused_kernel(MlpFusedArgs a) {
    extern __shared__ __align__(16) float ms[];
    __shared__ float red[kMlpThreads];
    __shared__ bool last;
    const int g = blockIdx.y, bi = blockIdx.x, nb = gridDim.x, tid = threadIdx.x;
    const int D = a.D, H = a.H, A = a.A, A1 = A + 1, T = a.T, EG = a.E;
    const int e0 = bi * a.ne;
    const int E = min(a.ne, EG - e0);          // environments of this block; local row t * E + el <-> row t * EG + e0 + el
    const int B = (T + 1) * E, S = T * E;
    const int BG = (T + 1) * EG, SG = T * EG;  // the agent's whole batch
    const int DP = D + 1, HP = H + 1;
    const long d = a.d;
    float* P = ms;                       // parameters [d] (padded to a multiple of 4)
    float* Gs = P + ((d + 3) & ~3L);     // gradient [d]
    const long bcap = (long)(T + 1) * a.ne, scap = (long)T * a.ne;   // sizes for a full block
    float* xs = Gs + ((d + 3) & ~3L);    // observations [B][D+1]
    float* h1 = xs + bcap * DP;          // [B][H+1]
    float* h2 = h1 + bcap * HP;          // [B][H+1]
    float* z = h2 + bcap * HP;           // [B][A+1] logits, value
    float* dz = z + bcap * A1;           // [S][A+1] dL/dlogits, dL/dvalue
    float* d2 = dz + scap * A1;          // [S][H+1] dL/d(pre-activation 2)
    float* d1 = d2 + scap * HP;          // [S][H+1] dL/d(pre-activation 1)
    float* gt = d1 + scap * HP;          // [S] returns
    float* lt = gt + scap;               // [S][3] objective terms per sample

    pdl_wait();     // the previous kernel in the stream may be the optimiser pass that wrote these parameters
    pdl_launch();
    const float* Pg = a.params + (long)g * a.p_stride;
    for (long i = tid; i < d; i += kMlpThreads) { P[i] = Pg[i]; Gs[i] = 0.0f; }
    const float* obs = reinterpret_cast<const float*>(a.obs.p[g]);
    for (int i = tid; i < B * D; i += kMlpThreads) {
        const int r = i / D, k = i - r * D;
        xs[r * DP + k] = obs[(long)((r / E) * EG + e0 + r % E) * D + k];
    }
    __syncthreads();

    const float *W1 = P + a.l.w1, *b1 = P + a.l.b1, *W2 = P + a.l.w2, *b2 = P + a.l.b2;
    const float *Wpi = P + a.l.piw, *bpi = P + a.l.pib, *Wv = P + a.l.vw, *bv = P + a.l.vb;
    // ---- forward (row index fastest across threads)
    for (int i = tid; i < B * H; i += kMlpThreads) {
        const int r = i % B, o = i / B;
        float acc = b1[o];
        for (int k = 0; k < D; k++) acc = fmaf(W1[o * D + k], xs[r * DP + k], acc);
        h1[r * HP + o] = tanhf(acc);
    }
    __syncthreads();
    for (int i = tid; i < B * H; i += kMlpThreads) {
        const int r = i % B, o = i / B;
        float acc = b2[o];
        for (int k = 0; k < H; k++) acc = fmaf(W2[o * H + k], h1[r * HP + k], acc);
        h2[r * HP + o] = tanhf(acc);
    }
    __syncthreads();
    for (int i = tid; i < B * A1; i += kMlpThreads) {
        const int r = i % B, k = i / B;
        const float* w = k < A ? Wpi + k * H : Wv;
        float acc = k < A ? bpi[k] : bv[0];
        for (int j = 0; j < H; j++) acc = fmaf(w[j], h2[r * HP + j], acc);
        z[r * A1 + k] = acc;
    }
    __syncthreads();
    {   // outputs for the caller (and for inspection): logits, values, hidden activations
        float* lo = a.logits + (long)g * BG * A;
        float* vo = a.values + (long)g * BG;
        for (int i = tid; i < B * A1; i += kMlpThreads) {
            const int r = i / A1, k = i - r * A1;
            const long gr = (long)(r / E) * EG + e0 + r % E;
            if (k < A) lo[gr * A + k] = z[i]; else vo[gr] = z[i];
        }
        float* o1 = a.h1_out + (long)g * BG * H;
        float* o2 = a.h2_out + (long)g * BG * H;
        for (int i = tid; i < B * H; i += kMlpThreads) {
            const int r = i / H, j = i - r * H;
            const long gr = (long)(r / E) * EG + e0 + r % E;
            o1[gr * H + j] = h1[r * HP + j]; o2[gr * H + j] = h2[r * HP + j];
        }
    }
    // ---- returns G_t = r_t + gamma (1 - done_t) G_{t+1}, G_T = V(s_T): one thread per environment
    const int* actions = reinterpret_cast<const int*>(a.actions.p[g]);
    const float* rewards = reinterpret_cast<const float*>(a.rewards.p[g]);
    const unsigned char* dones = reinterpret_cast<const unsigned char*>(a.dones.p[g]);
    for (int e = tid; e < E; e += kMlpThreads) {
        float G = z[(T * E + e) * A1 + A];
        for (int t = T - 1; t >= 0; t--) {
            G = rewards[t * EG + e0 + e] + a.gamma * (dones[t * EG + e0 + e] ? 0.0f : 1.0f) * G;
            gt[t * E + e] = G;
        }
    }
    __syncthreads();
    // ---- objective and its gradient with respect to logits and value (returns and advantages held constant)
    const float invS = 1.0f / (float)SG;
    for (int s = tid; s < S; s += kMlpThreads) {
        const long gs = (long)(s / E) * EG + e0 + s % E;   // the sample's row in the agent's batch
        const float* zz = z + s * A1;
        float mx = zz[0];
        for (int k = 1; k < A; k++) mx = fmaxf(mx, zz[k]);
        float sum = 0.0f;
        for (int k = 0; k < A; k++) sum += expf(zz[k] - mx);
        const float lse = mx + logf(sum);
        float Hn = 0.0f;
        for (int k = 0; k < A; k++) { const float lg = zz[k] - lse; Hn -= expf(lg) * lg; }
        const int act = actions[gs];
        const float G = gt[s], v = zz[A], adv = G - v;
        for (int k = 0; k < A; k++) {
            const float lg = zz[k] - lse, pi = expf(lg);
            dz[s * A1 + k] = (adv * (pi - (k == act ? 1.0f : 0.0f)) + a.ent_coef * pi * (lg + Hn)) * invS;
        }
        dz[s * A1 + A] = 2.0f * a.vf_coef * (v - G) * invS;
        lt[s * 3 + 0] = -(zz[act] - lse) * adv; lt[s * 3 + 1] = (G - v) * (G - v); lt[s * 3 + 2] = Hn;
        a.returns[(long)g * SG + gs] = G;
        a.adv[(long)g * SG + gs] = adv;
    }
    __syncthreads();
    {
        float* dzo = a.dlogits + (long)g * SG * A;
        float* dvo = a.dvalues + (long)g * SG;
        for (int i = tid; i < S * A1; i += kMlpThreads) {
            const int s = i / A1, k = i - s * A1;
            const long gs = (long)(s / E) * EG + e0 + s % E;
            if (k < A) dzo[gs * A + k] = dz[i]; else dvo[gs] = dz[i];
        }
        float l0 = 0.0f, l1 = 0.0f, l2 = 0.0f;
        for (int s = tid; s < S; s += kMlpThreads) { l0 += lt[s * 3]; l1 += lt[s * 3 + 1]; l2 += lt[s * 3 + 2]; }
        l0 = block_sum_fixed(l0, red); l1 = block_sum_fixed(l1, red); l2 = block_sum_fixed(l2, red);
        if (tid == 0) {   // this block's objective sums ride behind its partial gradient
            float* lp = a.partial + ((long)g * a.nb_max + bi) * a.partial_stride + ((d + 3) & ~3L);
            lp[0] = l0; lp[1] = l1; lp[2] = l2;
        }
    }
    // ---- backward
    for (int i = tid; i < S * H; i += kMlpThreads) {       // through the heads and tanh 2
        const int s = i % S, j = i / S;
        float acc = dz[s * A1 + A] * Wv[j];
        for (int k = 0; k < A; k++) acc = fmaf(dz[s * A1 + k], Wpi[k * H + j], acc);
        const float h = h2[s * HP + j];
        d2[s * HP + j] = acc * (1.0f - h * h);
    }
    for (int i = tid; i < A1 * H + A1; i += kMlpThreads) {  // head weights and biases
        float acc = 0.0f;
        if (i < A1 * H) {
            const int k = i / H, j = i - k * H;
            for (int s = 0; s < S; s++) acc = fmaf(dz[s * A1 + k], h2[s * HP + j], acc);
            Gs[(k < A ? a.l.piw + (long)k * H : a.l.vw) + j] = acc;
        } else {
            const int k = i - A1 * H;
            for (int s = 0; s < S; s++) acc += dz[s * A1 + k];
            Gs[k < A ? a.l.pib + k : a.l.vb] = acc;
        }
    }
    __syncthreads();
    for (int i = tid; i < S * H; i += kMlpThreads) {       // through layer 2 and tanh 1
        const int s = i % S, j = i / S;
        float acc = 0.0f;
        for (int o = 0; o < H; o++) acc = fmaf(d2[s * HP + o], W2[o * H + j], acc);
        const float h = h1[s * HP + j];
        d1[s * HP + j] = acc * (1.0f - h * h);
    }
    for (int i = tid; i < H * H + H; i += kMlpThreads) {    // layer 2 weights and biases
        float acc = 0.0f;
        if (i < H * H) {
            const int o = i / H, j = i - o * H;
            for (int s = 0; s < S; s++) acc = fmaf(d2[s * HP + o], h1[s * HP + j], acc);
            Gs[a.l.w2 + i] = acc;
        } else {
            const int o = i - H * H;
            for (int s = 0; s < S; s++) acc += d2[s * HP + o];
            Gs[a.l.b2 + o] = acc;
        }
    }
    __syncthreads();
    for (int i = tid; i < H * D + H; i += kMlpThreads) {    // layer 1 weights and biases
        float acc = 0.0f;
        if (i < H * D) {
            const int o = i / D, k = i - o * D;
            for (int s = 0; s < S; s++) acc = fmaf(d1[s * HP + o], xs[s * DP + k], acc);
            Gs[a.l.w1 + i] = acc;
        } else {
            const int o = i - H * D;
            for (int s = 0; s < S; s++) acc += d1[s * HP + o];
            Gs[a.l.b1 + o] = acc;
        }
    }
    __syncthreads();
    // ---- partial gradient out; the agent's last block adds the partials in block order, then norm and clip
    float* part = a.partial + ((long)g * a.nb_max + bi) * a.partial_stride;
    for (long i = tid; i < d; i += kMlpThreads) part[i] = Gs[i];
    __threadfence();
    __syncthreads();
    if (tid == 0) last = atomicAdd(a.ticket + g, 1u) == (unsigned)nb - 1;
    __syncthreads();
    if (!last) return;
    __threadfence();
    const float* pa = a.partial + (long)g * a.nb_max * a.partial_stride;   // read past L1 (__ldcg): written by other blocks
    float* Gg = a.grad + (long)g * a.g_stride;
    float sq = 0.0f;
    for (long i = tid; i < d; i += kMlpThreads) {
        float v = 0.0f;
        for (int b0 = 0; b0 < nb; b0 += 8) {   // block order; eight loads in flight
            float t[8];
#pragma unroll
            for (int u = 0; u < 8; u++) t[u] = b0 + u < nb ? __ldcg(pa + (long)(b0 + u) * a.partial_stride + i) : 0.0f;
#pragma unroll
            for (int u = 0; u < 8; u++) if (b0 + u < nb) v += t[u];
        }
        Gg[i] = v;
        sq = fmaf(v, v, sq);
    }
    sq = block_sum_fixed(sq, red);
    if (tid == 0) {
        const float nrm = sqrtf(sq);
        a.norm[g] = nrm;
        a.clip[g] = a.max_norm > 0.0f ? fminf(1.0f, a.max_norm / (nrm + 1e-6f)) : 1.0f;
        float l0 = 0.0f, l1 = 0.0f, l2 = 0.0f;
        const long lo = (d + 3) & ~3L;
        for (int b = 0; b < nb; b++) {
            l0 += __ldcg(pa + (long)b * a.partial_stride + lo); l1 += __ldcg(pa + (long)b * a.partial_stride + lo + 1);
            l2 += __ldcg(pa + (long)b * a.partial_stride + lo + 2);
        }
        a.losses[g * 4 + 0] = l0 * invS; a.losses[g * 4 + 1] = l1 * invS; a.losses[g * 4 + 2] = l2 * invS;
        a.ticket[g] = 0;   // ready for the next launch
    }
}

int mlp_fused_envs_per_block(int E) {   // at most kMlpMaxBlocks blocks per agent
    return (E + kMlpMaxBlocks - 1) / kMlpMaxBlocks;
}
size_t mlp_fused_smem(int D, int H, int A, int T, int E, long d) {
    const long ne = mlp_fused_envs_per_block(E);
    const long B = (long)(T + 1) * ne, S = (long)T * ne, A1 = A + 1;
    const long f = 2 * ((d + 3) & ~3L) + B * (D + 1) + 2 * B * (H + 1) + B * A1 + S * A1 + 2 * S * (H + 1) + S + 3 * S;
    return (size_t)f * sizeof(float);
}
bool mlp_fused_supported(int D, int H, int A, int T, int E, long d) {
    return D >= 1 && H >= 1 && A >= 1 && T >= 1 && E >= 1 && mlp_fused_smem(D, H, A, T, E, d) <= 200 * 1024;
}
long mlp_fused_partial_stride(long d) { return ((d + 3) & ~3L) + 4; }
cudaError_t launch_mlp_fused(const MlpFusedArgs& a0, int groups, cudaStream_t st) {
    MlpFusedArgs a = a0;
    if (!mlp_fused_supported(a.D, a.H, a.A, a.T, a.E, a.d) || !a.partial || !a.ticket) return cudaErrorNotSupported;
    a.ne = mlp_fused_envs_per_block(a.E);
    a.nb_max = kMlpMaxBlocks;
    a.partial_stride = mlp_fused_partial_stride(a.d);
    const int nb = (a.E + a.ne - 1) / a.ne;
    const size_t smem = mlp_fused_smem(a.D, a.H, a.A, a.T, a.E, a.d);
    static bool attr = false;
    if (!attr) {
        cudaError_t e = cudaFuncSetAttribute(mlp_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        attr = true;
    }
    (void)launch_pdl(mlp_fused_kernel, dim3(nb, groups), dim3(kMlpThreads), smem, st, a);
    return cudaGetLastError();
}

}  // namespace gala
