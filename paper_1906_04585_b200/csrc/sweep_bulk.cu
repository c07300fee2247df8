// Synchronous all-agent RMSProp + gossip pass (Algorithm 1 optimiser and gossip steps; Eq. 7 with
// zero delay), staged through shared memory with bulk asynchronous copies.
//
// A CTA walks over tiles of `cols` consecutive parameters.  For one tile it brings the x, g and v
// rows of ALL agents into shared memory with three tensor copies (cp.async.bulk.tensor, one
// [agents x cols] box per array, completion counted on an mbarrier), so the number of bytes in flight per SM is
// set by the stage size (96 KiB) and not by how many registers the threads can spare for loads.
// Four stages of 48 KiB keep loads in flight while other tiles are computed and stored.  The threads then
//   1. apply RMSProp in place (x row -> y, v row -> new v),
//   2. form (y_i + sum_j y_{i-off_j}) / (1+p) into the g rows (no longer needed),
// and a dedicated warp sends the g rows (new x) and v rows back with bulk stores.  x, g, v are read
// once and x, v written once: 20 B per parameter (+2 B for the optional bf16 copy of x, which the
// threads store directly).
#include <cstdlib>

#include "internal.h"

namespace gala {

namespace {

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void bar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s_u32(bar)), "r"(count));
}
__device__ __forceinline__ void bar_expect(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(s_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// bounded: gives up after ~1 s and reports through *error_word (results are then undefined)
__device__ __forceinline__ bool bar_wait(uint64_t* bar, uint32_t parity, int* error_word) {
    for (uint32_t i = 0; i < (1u << 22); i++) {
        if (bar_try(bar, parity)) return true;
        if (i > 64) __nanosleep(i < 4096 ? 32 : 256);
    }
    if (error_word) atomicExch(error_word, 2);
    return false;
}
// One instruction moves a [all agents] x [cols] box of a row-major [n_agents][d_pad] fp32 array
// (column coordinate c0 is a multiple of 4 floats = 16 bytes; columns past d_pad read as zero and
// are not written).
// With few agents a 256-column box is small and the copy engine, which is bound by instructions, cannot keep
// up; the arrays are then seen as [agents][d_pad / 256][256] and a box takes several 256-column blocks
// (wide = 1: c0 is a multiple of 256 and the coordinates are (0, c0 / 256, 0)).
__device__ __forceinline__ void tile_load(void* dst, const CUtensorMap* map, int c0, uint64_t* bar, int wide) {
    if (wide)
        asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                     ::"r"(s_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(c0 >> 8), "r"(0), "r"(s_u32(bar)) : "memory");
    else
        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                     ::"r"(s_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(0), "r"(s_u32(bar)) : "memory");
}
__device__ __forceinline__ void tile_store(const CUtensorMap* map, int c0, const void* src, int wide) {
    if (wide)
        asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                     ::"l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(c0 >> 8), "r"(0), "r"(s_u32(src)) : "memory");
    else
        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                     ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(0), "r"(s_u32(src)) : "memory");
}

// sqrt and the quotient use the hardware approximations (about 1e-7 relative each), far inside the
// 1e-5 this pass is held to; the exact versions cost several times the instructions
__device__ __forceinline__ void rms1(float& x, float g, float& v, float c, SweepHp hp) {
    float gi = c * g;
    v = hp.alpha * v + (1.0f - hp.alpha) * gi * gi;
    float r;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(v));
    x = x - __fdividef(hp.lr * gi, r + hp.eps);
}

}  // namespace

constexpr int kMaxBulkStages = 8;
constexpr int kConsumers = 256;

__device__ __forceinline__ void bar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s_u32(bar)) : "memory");
}

// 288 threads: warps 0-7 compute, warp 8 moves data.
//   full[s]: bytes of a tile have landed in stage s (transaction count)
//   done[s]: all 256 compute threads are finished with stage s
// The mover warp sends a finished stage back with bulk stores and refills the stage it sent back one
// step earlier (whose stores have had a whole step to drain), so neither the compute threads nor the
// loads of the other stages ever wait for a store to leave shared memory.
template <int P>
__global__ void __launch_bounds__(kConsumers + 32, 1)
sweep_sync_bulk_kernel(const __grid_constant__ CUtensorMap mx, const __grid_constant__ CUtensorMap mg,
                       const __grid_constant__ CUtensorMap mv, const float* __restrict__ clip, __nv_bfloat16* __restrict__ shadow, int n_agents, long d_pad,
                       int cols, int kBulkStages, long n_tiles, int off0, int off1, SweepHp hp, int* error_word, int wide) {
    extern __shared__ __align__(128) float smem[];
    __shared__ __align__(8) uint64_t full[kMaxBulkStages];
    __shared__ __align__(8) uint64_t done[kMaxBulkStages];
    __shared__ float clip_s[256];
    const int stage_floats = 3 * n_agents * cols;
    const int row4 = cols / 4;
    const float w = 1.0f / (1.0f + P);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kBulkStages; s++) { bar_init(&full[s], 1); bar_init(&done[s], kConsumers); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();     // the gradients and clip factors come from the kernels before
    pdl_launch();
    for (int a = threadIdx.x; a < n_agents; a += blockDim.x) clip_s[a] = clip ? clip[a] : 1.0f;
    __syncthreads();

    const long first = blockIdx.x, step = gridDim.x;
    const long my_tiles = first < n_tiles ? (n_tiles - first + step - 1) / step : 0;

    if (warp == kConsumers / 32) {
        // ---------------- mover warp (one elected lane issues the tensor copies; issuing the three loads from
        // three lanes side by side was measured and is no faster)
        if (lane == 0) {
            const uint32_t stage_bytes = (uint32_t)stage_floats * 4u;
            auto issue_loads = [&](long k, int stage) {
                const int c0 = (int)((first + k * step) * cols);
                float* sx = smem + (long)stage * stage_floats;
                bar_expect(&full[stage], stage_bytes);
                tile_load(sx, &mx, c0, &full[stage], wide);
                tile_load(sx + n_agents * cols, &mg, c0, &full[stage], wide);
                tile_load(sx + 2 * n_agents * cols, &mv, c0, &full[stage], wide);
            };
            for (int s = 0; s < kBulkStages && s < my_tiles; s++) issue_loads(s, s);
            for (long k = 0; k < my_tiles; k++) {
                const int stage = (int)(k % kBulkStages);
                if (!bar_wait(&done[stage], (uint32_t)(k / kBulkStages) & 1u, error_word)) break;
                const int c0 = (int)((first + k * step) * cols);
                const float* sg = smem + (long)stage * stage_floats + n_agents * cols;
                tile_store(&mx, c0, sg, wide);
                tile_store(&mv, c0, sg + n_agents * cols, wide);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                if (k >= 1 && k - 1 + kBulkStages < my_tiles) {
                    // stage of step k-1: all but the newest group of stores must have left shared memory
                    asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    issue_loads(k - 1 + kBulkStages, (int)((k - 1) % kBulkStages));
                }
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        }
        return;
    }

    // ---------------- compute warps
    for (long k = 0; k < my_tiles; k++) {
        const int stage = (int)(k % kBulkStages);
        const long c0 = (first + k * step) * cols;
        const int nc = (int)min((long)cols, d_pad - c0);
        const int nc4 = nc / 4;
        float4* sx = reinterpret_cast<float4*>(smem + (long)stage * stage_floats);
        float4* sg = sx + n_agents * row4;
        float4* sv = sg + n_agents * row4;
        if (!bar_wait(&full[stage], (uint32_t)(k / kBulkStages) & 1u, error_word)) break;

        // 1. RMSProp in place
        const int total = n_agents * nc4;
        for (int idx = threadIdx.x; idx < total; idx += kConsumers) {
            const int a = idx / nc4, c = idx - a * nc4;
            float4 xi = sx[a * row4 + c], vi = sv[a * row4 + c];
            const float4 gi = sg[a * row4 + c];
            const float cl = clip_s[a];
            rms1(xi.x, gi.x, vi.x, cl, hp); rms1(xi.y, gi.y, vi.y, cl, hp);
            rms1(xi.z, gi.z, vi.z, cl, hp); rms1(xi.w, gi.w, vi.w, cl, hp);
            sx[a * row4 + c] = xi;
            sv[a * row4 + c] = vi;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory");
        // 2. equal-weight average with the in-peers' y (same tile, on chip) into the g rows
        for (int idx = threadIdx.x; idx < total; idx += kConsumers) {
            const int a = idx / nc4, c = idx - a * nc4;
            float4 y = sx[a * row4 + c];
            if (P >= 1) {
                int j = a - off0; if (j < 0) j += n_agents;
                const float4 m = sx[j * row4 + c];
                y.x += m.x; y.y += m.y; y.z += m.z; y.w += m.w;
            }
            if (P >= 2) {
                int j = a - off1; if (j < 0) j += n_agents;
                const float4 m = sx[j * row4 + c];
                y.x += m.x; y.y += m.y; y.z += m.z; y.w += m.w;
            }
            if (P >= 1) { y.x *= w; y.y *= w; y.z *= w; y.w *= w; }
            sg[a * row4 + c] = y;
            if (shadow) {
                __nv_bfloat162 lo = __floats2bfloat162_rn(y.x, y.y), hi = __floats2bfloat162_rn(y.z, y.w);
                uint2 u;
                u.x = *reinterpret_cast<unsigned*>(&lo);
                u.y = *reinterpret_cast<unsigned*>(&hi);
                *reinterpret_cast<uint2*>(shadow + (long)a * d_pad + c0 + 4 * c) = u;
            }
        }
        // make these writes visible to the bulk-copy engine, then hand the stage to the mover warp
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        bar_arrive(&done[stage]);
    }
}

// Returns cudaErrorNotSupported when the shape does not suit this kernel (caller falls back).
cudaError_t launch_sweep_sync_bulk(float* x, const float* g, float* v, const float* clip, __nv_bfloat16* shadow,
                                   int n_agents, long d_pad, int n_peers, int o0, int o1, SweepHp hp,
                                   int* error_word, cudaStream_t st) {
    if (n_agents > 256 || (d_pad % 4) || d_pad > 0x7fffffffL) return cudaErrorNotSupported;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(g) | reinterpret_cast<uintptr_t>(v)) & 15)
        return cudaErrorNotSupported;
    // Three or more stages inside ~200 KiB of shared memory; measured best on 32 agents x 1.7M
    // parameters: 160 columns x 3 stages (6.0 TB/s) against 128 x 4 (5.5) and 256 x 2 (4.3).
    const long budget = 200L * 1024;
    int cols = (int)(budget / (3L * 12 * n_agents));
    cols = cols / 32 * 32;
    // a box edge holds at most 256 elements; wider tiles (few agents) take several 256-column blocks per copy
    const int wide = cols >= 512 && (d_pad & 255) == 0;
    if (wide) { cols = cols / 256 * 256; if (cols > 1024) cols = 1024; }
    else if (cols > 256) cols = 256;
    if (cols < 32) return cudaErrorNotSupported;
    int stages = (int)(budget / ((long)12 * n_agents * cols));
    if (stages > kMaxBulkStages) stages = kMaxBulkStages;
    if (stages < 2) return cudaErrorNotSupported;
    if (gemm_init() != cudaSuccess) return cudaErrorNotSupported;
    CUtensorMap mx, mg, mv;
    bool ok;
    if (wide)
        ok = make_tensor_map_f32_wide(&mx, x, (uint64_t)d_pad, (uint64_t)n_agents, (uint64_t)d_pad * 4, cols / 256, n_agents) &&
             make_tensor_map_f32_wide(&mg, g, (uint64_t)d_pad, (uint64_t)n_agents, (uint64_t)d_pad * 4, cols / 256, n_agents) &&
             make_tensor_map_f32_wide(&mv, v, (uint64_t)d_pad, (uint64_t)n_agents, (uint64_t)d_pad * 4, cols / 256, n_agents);
    else
        ok = make_tensor_map_f32(&mx, x, (uint64_t)d_pad, (uint64_t)n_agents, (uint64_t)d_pad * 4, cols, n_agents) &&
             make_tensor_map_f32(&mg, g, (uint64_t)d_pad, (uint64_t)n_agents, (uint64_t)d_pad * 4, cols, n_agents) &&
             make_tensor_map_f32(&mv, v, (uint64_t)d_pad, (uint64_t)n_agents, (uint64_t)d_pad * 4, cols, n_agents);
    if (!ok) return cudaErrorNotSupported;
    const long n_tiles = (d_pad + cols - 1) / cols;
    const size_t smem = (size_t)stages * 3 * n_agents * cols * 4;
    int grid = (int)(n_tiles < sm_count() ? n_tiles : sm_count());
    cudaError_t e;
#define GALA_BULK_LAUNCH(P)                                                                                  \
    e = cudaFuncSetAttribute(sweep_sync_bulk_kernel<P>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e != cudaSuccess) return e;                                                                          \
    (void)launch_pdl(sweep_sync_bulk_kernel<P>, dim3(grid), dim3(kConsumers + 32), smem, st, mx, mg, mv, clip, shadow, n_agents, d_pad, cols, \
                                                                   stages, n_tiles, o0, o1, hp, error_word, wide);
    if (n_peers == 0) { GALA_BULK_LAUNCH(0) }
    else if (n_peers == 1) { GALA_BULK_LAUNCH(1) }
    else if (n_peers == 2) { GALA_BULK_LAUNCH(2) }
    else return cudaErrorInvalidValue;
#undef GALA_BULK_LAUNCH
    return cudaGetLastError();
}

}  // namespace gala
