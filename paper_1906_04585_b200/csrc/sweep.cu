// Fused RMSProp + gossip pass over the flat parameter vectors (Algorithm 1,
// optimiser step, broadcast and conditional averaging; Eqs. 5-7; Table 2
// RMSProp rows; mixing weights 1/(1+|N_in|) from the footnote of Algorithm 1).
//
// Both forms are pure streaming kernels: every array element is read once and
// written once with 16-byte accesses.
#include <cstdlib>

#include "internal.h"
#include "tcgen05.cuh"

namespace gala {

__device__ __forceinline__ float4 ld_stream(const float* p) {
    // read-once data: bypass L1 allocation
    return __ldcs(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ void st_stream(float* p, float4 v) { __stcs(reinterpret_cast<float4*>(p), v); }

__device__ __forceinline__ void rms1(float& x, float g, float& v, float c, SweepHp hp) {
    float gi = c * g;
    v = hp.alpha * v + (1.0f - hp.alpha) * gi * gi;
    x = x - hp.lr * gi / (sqrtf(v) + hp.eps);
}
__device__ __forceinline__ void rms4(float4& x, float4 g, float4& v, float c, SweepHp hp) {
    rms1(x.x, g.x, v.x, c, hp);
    rms1(x.y, g.y, v.y, c, hp);
    rms1(x.z, g.z, v.z, c, hp);
    rms1(x.w, g.w, v.w, c, hp);
}
__device__ __forceinline__ void st_bf16x4(__nv_bfloat16* p, float4 v) {
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<unsigned*>(&a);
    u.y = *reinterpret_cast<unsigned*>(&b);
    *reinterpret_cast<uint2*>(p) = u;
}

// ------------------------------------------------------------------------------------------
// Per-agent form: y = RMSProp(x, c*g, v); snapshot <- y; x <- y or (y + sum peers)/(1+p).
// g == nullptr: no pending gradient (y = x, v untouched).
template <int P>
__global__ void __launch_bounds__(256) sweep_agent_kernel(float* __restrict__ x, const float* __restrict__ g,
                                                          float* __restrict__ v, float* __restrict__ snap,
                                                          const float* __restrict__ peer0,
                                                          const float* __restrict__ peer1,
                                                          const float* __restrict__ clip,
                                                          __nv_bfloat16* __restrict__ shadow, long n4,
                                                          SweepHp hp) {
    pdl_wait();
    pdl_launch();
    const float c = clip ? *clip : 1.0f;
    const float w = 1.0f / (1.0f + P);
    for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n4; i += (long)gridDim.x * blockDim.x) {
        const long o = i * 4;
        float4 xi = ld_stream(x + o);
        if (g) {
            float4 gi = ld_stream(g + o);
            float4 vi = ld_stream(v + o);
            rms4(xi, gi, vi, c, hp);
            st_stream(v + o, vi);
        }
        st_stream(snap + o, xi);
        if (P >= 1) {
            float4 m = ld_stream(peer0 + o);
            xi.x += m.x; xi.y += m.y; xi.z += m.z; xi.w += m.w;
        }
        if (P >= 2) {
            float4 m = ld_stream(peer1 + o);
            xi.x += m.x; xi.y += m.y; xi.z += m.z; xi.w += m.w;
        }
        if (P >= 1) { xi.x *= w; xi.y *= w; xi.z *= w; xi.w *= w; }
        st_stream(x + o, xi);
        if (shadow) st_bf16x4(shadow + o, xi);
    }
}

cudaError_t launch_sweep_agent(float* x, const float* g, float* v, float* snap_out, const float* peer0,
                               const float* peer1, int n_peers, const float* clip, __nv_bfloat16* shadow,
                               long d_pad, SweepHp hp, cudaStream_t st) {
    long n4 = d_pad / 4;
    int grid = (int)((n4 + 255) / 256);
    if (grid > sm_count() * 8) grid = sm_count() * 8;
    if (grid < 1) grid = 1;
    if (n_peers == 0)
        (void)launch_pdl(sweep_agent_kernel<0>, dim3(grid), dim3(256), 0, st, x, g, v, snap_out, nullptr, nullptr, clip, shadow, n4, hp);
    else if (n_peers == 1)
        (void)launch_pdl(sweep_agent_kernel<1>, dim3(grid), dim3(256), 0, st, x, g, v, snap_out, peer0, nullptr, clip, shadow, n4, hp);
    else
        (void)launch_pdl(sweep_agent_kernel<2>, dim3(grid), dim3(256), 0, st, x, g, v, snap_out, peer0, peer1, clip, shadow, n4, hp);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Synchronous all-agent form: each thread owns one 16-byte column across all agents.  It
// applies RMSProp to every agent's element, parks the results y_i in shared memory (its own
// private column, so no barrier is needed), then forms x_i = (y_i + sum_j y_{i-off_j}) / (1+p)
// from those parked values.  x, g, v are read once and x, v written once: 20 B per parameter,
// independent of the number of in-peers.
constexpr int kSyncUnroll = 4;

template <int P>
__global__ void sweep_sync_kernel(float* __restrict__ x, const float* __restrict__ g, float* __restrict__ v,
                                  const float* __restrict__ clip, __nv_bfloat16* __restrict__ shadow,
                                  int n_agents, long d_pad, long n4, int off0, int off1, SweepHp hp) {
    pdl_wait();
    pdl_launch();
    extern __shared__ float4 ysm[];  // [n_agents][blockDim.x]
    const float w = 1.0f / (1.0f + P);
    for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n4; i += (long)gridDim.x * blockDim.x) {
        const long o = i * 4;
        int a = 0;
        for (; a + kSyncUnroll <= n_agents; a += kSyncUnroll) {
            float4 xi[kSyncUnroll], gi[kSyncUnroll], vi[kSyncUnroll];
#pragma unroll
            for (int u = 0; u < kSyncUnroll; u++) {
                const long off = (long)(a + u) * d_pad + o;
                xi[u] = ld_stream(x + off);
                gi[u] = ld_stream(g + off);
                vi[u] = ld_stream(v + off);
            }
#pragma unroll
            for (int u = 0; u < kSyncUnroll; u++) {
                const float c = clip ? __ldg(clip + a + u) : 1.0f;
                rms4(xi[u], gi[u], vi[u], c, hp);
                st_stream(v + (long)(a + u) * d_pad + o, vi[u]);
                ysm[(a + u) * blockDim.x + threadIdx.x] = xi[u];
            }
        }
        for (; a < n_agents; a++) {
            const long off = (long)a * d_pad + o;
            float4 xi = ld_stream(x + off), gi = ld_stream(g + off), vi = ld_stream(v + off);
            const float c = clip ? __ldg(clip + a) : 1.0f;
            rms4(xi, gi, vi, c, hp);
            st_stream(v + off, vi);
            ysm[a * blockDim.x + threadIdx.x] = xi;
        }
        for (a = 0; a < n_agents; a++) {
            float4 y = ysm[a * blockDim.x + threadIdx.x];
            if (P >= 1) {
                int j = a - off0; if (j < 0) j += n_agents;
                float4 m = ysm[j * blockDim.x + threadIdx.x];
                y.x += m.x; y.y += m.y; y.z += m.z; y.w += m.w;
            }
            if (P >= 2) {
                int j = a - off1; if (j < 0) j += n_agents;
                float4 m = ysm[j * blockDim.x + threadIdx.x];
                y.x += m.x; y.y += m.y; y.z += m.z; y.w += m.w;
            }
            if (P >= 1) { y.x *= w; y.y *= w; y.z *= w; y.w *= w; }
            const long off = (long)a * d_pad + o;
            st_stream(x + off, y);
            if (shadow) st_bf16x4(shadow + off, y);
        }
    }
}

cudaError_t launch_sweep_sync(float* x, const float* g, float* v, const float* clip,
                              __nv_bfloat16* shadow, int n_agents, long d_pad, int n_peers,
                              const int* peer_off, SweepHp hp, int* error_word, cudaStream_t st) {
    long n4 = d_pad / 4;
    {
        int b0 = 0, b1 = 0;
        if (n_peers >= 1) b0 = ((peer_off[0] % n_agents) + n_agents) % n_agents;
        if (n_peers >= 2) b1 = ((peer_off[1] % n_agents) + n_agents) % n_agents;
        // staged tensor-copy kernel first; the register-staged kernel below serves the shapes it declines
        cudaError_t eb = launch_sweep_sync_bulk(x, g, v, clip, shadow, n_agents, d_pad, n_peers, b0, b1, hp,
                                                error_word, st);
        if (eb != cudaErrorNotSupported) return eb;
    }
    // shared memory: n_agents * threads * 16 B, kept under 128 KB so that one block always fits
    int threads = 256;
    while (threads > 32 && (long)n_agents * threads * 16 > 128 * 1024) threads /= 2;
    size_t smem = (size_t)n_agents * threads * 16;
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    long blocks = (n4 + threads - 1) / threads;
    int per_sm = (int)((200 * 1024) / (smem ? smem : 1));
    if (per_sm < 1) per_sm = 1;
    if (per_sm > 8) per_sm = 8;
    long cap = (long)sm_count() * per_sm;
    int grid = (int)(blocks < cap ? blocks : cap);
    if (grid < 1) grid = 1;
    int o0 = 0, o1 = 0;
    if (n_peers >= 1) o0 = ((peer_off[0] % n_agents) + n_agents) % n_agents;
    if (n_peers >= 2) o1 = ((peer_off[1] % n_agents) + n_agents) % n_agents;
    cudaError_t e;
#define GALA_SYNC_LAUNCH(P)                                                                          \
    e = cudaFuncSetAttribute(sweep_sync_kernel<P>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e != cudaSuccess) return e;                                                                  \
    (void)launch_pdl(sweep_sync_kernel<P>, dim3(grid), dim3(threads), smem, st, x, g, v, clip, shadow, n_agents, d_pad, n4, o0, o1, hp);
    if (n_peers == 0) { GALA_SYNC_LAUNCH(0) }
    else if (n_peers == 1) { GALA_SYNC_LAUNCH(1) }
    else if (n_peers == 2) { GALA_SYNC_LAUNCH(2) }
    else return cudaErrorInvalidValue;
#undef GALA_SYNC_LAUNCH
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// Global gradient norm and clip coefficient ("Clip global gradient norm", Table 2):
// c = min(1, max_norm / (||g||_2 + 1e-6)).  Fixed chunking and a fixed-order final sum in
// double precision make the result independent of scheduling.
__global__ void __launch_bounds__(256) grad_norm_kernel(const float* __restrict__ g, long d, long d_pad,
                                                        int agent0, float max_norm, double* partial,
                                                        unsigned* ticket, float* norm, float* clip, NormKnown kn, AgentMap am) {
    pdl_wait();
    pdl_launch();
    const int slot = agent_slot(am, blockIdx.y);
    const int agent = agent0 + slot;
    const float* ga = g + (long)agent * d_pad;
    // The elements to read, [0, d_pad) without the range whose sum of squares is already known, are numbered
    // consecutively and cut into chunks of multiples of 4 floats (the padding [d, d_pad) is zero): 16-byte loads
    const long total = d_pad - kn.count;
    const int chunks = gridDim.x;          // <= kNormChunks: fewer when there is little to read
    const long per = ((total / 4 + chunks - 1) / chunks) * 4;
    const long lo = (long)blockIdx.x * per;
    long hi = lo + per; if (hi > total) hi = total;
    float a0 = 0.0f, a1 = 0.0f, a2 = 0.0f, a3 = 0.0f;
    for (long i = lo + 4L * threadIdx.x; i < hi; i += 4L * blockDim.x) {
        const float4 t = __ldcs(reinterpret_cast<const float4*>(ga + (i < kn.off ? i : i + kn.count)));
        a0 = fmaf(t.x, t.x, a0); a1 = fmaf(t.y, t.y, a1); a2 = fmaf(t.z, t.z, a2); a3 = fmaf(t.w, t.w, a3);
    }
    double acc = ((double)a0 + (double)a1) + ((double)a2 + (double)a3);
    if (kn.partial) {   // the known range: its partial sums, shared out over the agent's threads in slot order
        const float* kp = kn.partial + (long)slot * kn.partial_group_stride;
        for (long k = (long)blockIdx.x * blockDim.x + threadIdx.x; k < kn.n_partials; k += (long)chunks * blockDim.x)
            acc += (double)kp[k];
    }
    __shared__ double red[256];
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s];
        __syncthreads();
    }
    __shared__ bool last;
    if (threadIdx.x == 0) {
        partial[(long)agent * kNormChunks + blockIdx.x] = red[0];
        __threadfence();
        unsigned t = atomicAdd(&ticket[agent], 1u);
        last = (t == (unsigned)chunks - 1);
    }
    __syncthreads();
    if (last && threadIdx.x == 0) {
        __threadfence();
        double s = 0.0;
        for (int k = 0; k < chunks; k++) s += ((volatile double*)partial)[(long)agent * kNormChunks + k];
        float nrm = (float)sqrt(s);
        norm[agent] = nrm;
        float c = 1.0f;
        if (max_norm > 0.0f) c = fminf(1.0f, max_norm / (nrm + 1e-6f));
        clip[agent] = c;
        ticket[agent] = 0;  // ready for the next launch
    }
}

cudaError_t launch_grad_norm(const float* g, long d, long d_pad, int agent0, int n_agents, float max_norm,
                             double* partial, unsigned* ticket, float* norm, float* clip, cudaStream_t st,
                             const NormKnown* known, const AgentMap* am) {
    NormKnown kn{};
    if (known) kn = *known;
    if (!kn.partial) { kn.off = 0; kn.count = 0; kn.n_partials = 0; }
    if ((kn.off | kn.count) & 3 || kn.off + kn.count > d_pad) return cudaErrorInvalidValue;
    // a chunk is at least 8192 floats (32 bytes per thread of a block, twice): with most of the gradient known
    // from partial sums a dozen blocks per agent remain, and the last block's sum over chunks is as short
    long chunks = (d_pad - kn.count + 8191) / 8192;
    if (chunks < 1) chunks = 1;
    if (chunks > kNormChunks) chunks = kNormChunks;
    dim3 grid((unsigned)chunks, n_agents);
    (void)launch_pdl(grad_norm_kernel, dim3(grid), dim3(256), 0, st, g, d, d_pad, agent0, max_norm, partial, ticket, norm, clip, kn, am ? *am : AgentMap{});
    return cudaGetLastError();
}

// Gradient all-reduce of the synchronous A2C baseline (Sec. 5: the agents average their gradients
// before each update): every agent's gradient row is replaced by the mean over agents, summed in
// agent order.  One thread per 16-byte column; reads N*d, writes N*d.
__global__ void __launch_bounds__(256) allreduce_grads_kernel(float* __restrict__ g, int n_agents, long d_pad, long n4) {
    pdl_wait();
    pdl_launch();
    const float inv = 1.0f / (float)n_agents;
    for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n4; i += (long)gridDim.x * blockDim.x) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int a = 0; a < n_agents; a++) {
            const float4 t = *reinterpret_cast<const float4*>(g + (long)a * d_pad + 4 * i);
            acc.x += t.x; acc.y += t.y; acc.z += t.z; acc.w += t.w;
        }
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        for (int a = 0; a < n_agents; a++) *reinterpret_cast<float4*>(g + (long)a * d_pad + 4 * i) = acc;
    }
}
cudaError_t launch_allreduce_grads(float* g, int n_agents, long d_pad, cudaStream_t st) {
    const long n4 = d_pad / 4;
    int grid = (int)((n4 + 255) / 256);
    if (grid > sm_count() * 8) grid = sm_count() * 8;
    (void)launch_pdl(allreduce_grads_kernel, dim3(grid), dim3(256), 0, st, g, n_agents, d_pad, n4);
    return cudaGetLastError();
}

// Distance from consensus ||X - mean over agents||_F (left side of Proposition 1) in one pass:
// per column the sum and the sum of squares over agents in double precision,
// sum_i (x_i - m)^2 = sum_i x_i^2 - (sum_i x_i)^2 / n.  Block partials, fixed-order final sum by
// the last block; writes the squared distance.
constexpr int kConsensusBlocks = 592;
__global__ void __launch_bounds__(256) consensus_kernel(const float* __restrict__ x, int n_agents, long d, long d_pad,
                                                        double* partial, unsigned* ticket, double* out) {
    pdl_wait();
    pdl_launch();
    double acc = 0.0;
    for (long c = blockIdx.x * (long)blockDim.x + threadIdx.x; c < d; c += (long)gridDim.x * blockDim.x) {
        double s = 0.0, ss = 0.0;
        for (int a = 0; a < n_agents; a++) {
            const double t = (double)__ldcs(x + (long)a * d_pad + c);
            s += t; ss += t * t;
        }
        const double dev = ss - s * s / (double)n_agents;
        acc += dev > 0.0 ? dev : 0.0;
    }
    __shared__ double red[256];
    __shared__ bool last;
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int st = 128; st > 0; st >>= 1) {
        if (threadIdx.x < st) red[threadIdx.x] += red[threadIdx.x + st];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        partial[blockIdx.x] = red[0];
        __threadfence();
        last = atomicAdd(ticket, 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (last && threadIdx.x == 0) {
        __threadfence();
        double s = 0.0;
        for (unsigned k = 0; k < gridDim.x; k++) s += ((volatile double*)partial)[k];
        *out = s;
        *ticket = 0;
    }
}
cudaError_t launch_consensus(const float* x, int n_agents, long d, long d_pad, double* partial, unsigned* ticket,
                             double* out, cudaStream_t st) {
    (void)launch_pdl(consensus_kernel, dim3(kConsensusBlocks), dim3(256), 0, st, x, n_agents, d, d_pad, partial, ticket, out);
    return cudaGetLastError();
}

// Frobenius norm of the update matrix alpha * G of a synchronous round, the quantity Proposition 1 sums: row i is
// what the RMSProp step of the next optimiser pass subtracts from agent i's parameters,
//     u = lr * c g / (sqrt(a v + (1 - a) (c g)^2) + eps),
// read from the pending gradient, its clip factor and the second-moment estimate BEFORE that pass.  Block partials
// in double precision, fixed-order final sum by the last block; writes the squared norm over all agents.
__global__ void __launch_bounds__(256) update_norm_kernel(const float* __restrict__ g, const float* __restrict__ v,
                                                          const float* __restrict__ clip, long d_pad, SweepHp hp,
                                                          double* partial, unsigned* ticket, double* out) {
    pdl_wait();
    pdl_launch();
    const int a = blockIdx.y;
    const float c = clip ? clip[a] : 1.0f;
    const long n4 = d_pad / 4;
    const long per = (n4 + gridDim.x - 1) / gridDim.x;
    const long lo = (long)blockIdx.x * per;
    long hi = lo + per; if (hi > n4) hi = n4;
    const float4* g4 = reinterpret_cast<const float4*>(g + (long)a * d_pad);
    const float4* v4 = reinterpret_cast<const float4*>(v + (long)a * d_pad);
    double acc = 0.0;
    for (long i = lo + threadIdx.x; i < hi; i += blockDim.x) {
        const float4 gg = __ldcs(g4 + i), vv = __ldcs(v4 + i);
        const float ge[4] = {gg.x, gg.y, gg.z, gg.w}, ve[4] = {vv.x, vv.y, vv.z, vv.w};
        float s = 0.0f;
#pragma unroll
        for (int e = 0; e < 4; e++) {
            const float gi = c * ge[e];
            const float vn = hp.alpha * ve[e] + (1.0f - hp.alpha) * gi * gi;
            const float u = hp.lr * gi / (sqrtf(vn) + hp.eps);
            s = fmaf(u, u, s);
        }
        acc += (double)s;
    }
    __shared__ double red[256];
    __shared__ bool last;
    red[threadIdx.x] = acc;
    __syncthreads();
    for (int st = 128; st > 0; st >>= 1) {
        if (threadIdx.x < st) red[threadIdx.x] += red[threadIdx.x + st];
        __syncthreads();
    }
    const unsigned blocks = gridDim.x * gridDim.y;
    if (threadIdx.x == 0) {
        partial[blockIdx.y * gridDim.x + blockIdx.x] = red[0];
        __threadfence();
        last = atomicAdd(ticket, 1u) == blocks - 1;
    }
    __syncthreads();
    if (last) {
        __threadfence();
        double s = 0.0;
        for (unsigned k = threadIdx.x; k < blocks; k += blockDim.x) s += ((volatile double*)partial)[k];
        red[threadIdx.x] = s;
        __syncthreads();
        for (int st = 128; st > 0; st >>= 1) {
            if (threadIdx.x < st) red[threadIdx.x] += red[threadIdx.x + st];
            __syncthreads();
        }
        if (threadIdx.x == 0) { *out = red[0]; *ticket = 0; }
    }
}
cudaError_t launch_update_norm(const float* g, const float* v, const float* clip, int n_agents, long d_pad, SweepHp hp,
                               double* partial, unsigned* ticket, double* out, cudaStream_t st) {
    if (n_agents < 1 || (d_pad & 3)) return cudaErrorInvalidValue;
    (void)launch_pdl(update_norm_kernel, dim3(kUpdateNormChunks, n_agents), dim3(256), 0, st, g, v, clip, d_pad, hp, partial,
                     ticket, out);
    return cudaGetLastError();
}

// Straggler injection: occupies the stream for about `usec` microseconds (one sleeping thread).
// Bounded twice: by the requested time (capped by the caller) and by an iteration limit.
__global__ void delay_kernel(unsigned long long usec) {
    pdl_wait();
    pdl_launch();
    unsigned long long t0, t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    for (int i = 0; i < 2000000; i++) {
        __nanosleep(1000);
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        if (t - t0 >= usec * 1000ull) break;
    }
}
// The give-up path of the tensor-core kernels on its own: one thread waits, with the kernels' bounded wait and a
// small limit, on an mbarrier that nothing ever arrives at, and reports as they do - abort flag, then the
// caller's error word - before it returns.  Nothing is left behind: no copy in flight, no tensor memory.
__global__ void wait_runs_out_kernel(unsigned polls, int* error_word) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (!mbar_wait_polls(&bar, 0u, &abort_flag, polls) && abort_flag && error_word) atomicExch(error_word, 1);
}
cudaError_t launch_wait_runs_out(unsigned polls, int* error_word, cudaStream_t st) {
    wait_runs_out_kernel<<<1, 1, 0, st>>>(polls, error_word);
    return cudaGetLastError();
}

cudaError_t launch_delay(unsigned long long usec, cudaStream_t st) {
    (void)launch_pdl(delay_kernel, dim3(1), dim3(1), 0, st, usec);
    return cudaGetLastError();
}

__global__ void cast_bf16_kernel(const float* __restrict__ x, __nv_bfloat16* __restrict__ out, long n4) {
    pdl_wait();
    pdl_launch();
    for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n4; i += (long)gridDim.x * blockDim.x)
        st_bf16x4(out + i * 4, *reinterpret_cast<const float4*>(x + i * 4));
}
cudaError_t launch_cast_bf16(const float* x, __nv_bfloat16* out, long count, cudaStream_t st) {
    long n4 = count / 4;
    int grid = (int)((n4 + 255) / 256);
    if (grid > sm_count() * 8) grid = sm_count() * 8;
    if (grid < 1) grid = 1;
    (void)launch_pdl(cast_bf16_kernel, dim3(grid), dim3(256), 0, st, x, out, n4);
    return cudaGetLastError();
}

}  // namespace gala
