// Per-agent form of the fused RMSProp + gossip pass for SEVERAL agents in one launch (Algorithm 1, the
// optimiser step, the non-blocking broadcast and the conditional average of every listed agent; Eqs. 5-6;
// weights 1/(1+|N_in|) from the footnote of Algorithm 1).
//
// Each listed agent i has its own decision, taken on the host when the launch is enqueued: which completed
// snapshot of which in-peer it averages with (or none), where its own new snapshot goes, and whether a
// gradient is pending.  The rows that a work item touches are therefore scattered: x_i, g_i, v_i, up to two
// snapshot rows of other agents, and the agent's own snapshot row.  One item = one agent x one tile of `cols`
// consecutive parameters.  A CTA walks over items; a mover warp brings the item's rows into a ring of
// shared-memory stages with one bulk copy per row (cp.async.bulk, completion counted on an mbarrier), 256
// compute threads apply RMSProp in place and form the average, and the mover warp sends y (the snapshot),
// the new x and the new v back with bulk stores.  Every byte crosses DRAM once:
//   read x, g, v and p snapshots, write x, v and the own snapshot = 24 + 4 p bytes per parameter
//   (+2 for the bf16 copy of x that the compute threads store directly).
#include "internal.h"

namespace gala {

namespace {

__device__ __forceinline__ uint32_t sm_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mb_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(sm_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mb_expect(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(sm_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mb_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(sm_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mb_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(sm_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// bounded: gives up after about a second and reports through *error_word (results are then undefined)
__device__ __forceinline__ bool mb_wait(uint64_t* bar, uint32_t parity, int* error_word) {
    for (uint32_t i = 0; i < (1u << 22); i++) {
        if (mb_try(bar, parity)) return true;
        if (i > 64) __nanosleep(i < 4096 ? 32 : 256);
    }
    if (error_word) atomicExch(error_word, 3);
    return false;
}
// untiled bulk copies; addresses 16-byte aligned, sizes multiples of 16 bytes
__device__ __forceinline__ void row_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(sm_u32(dst)),
                 "l"(src), "r"(bytes), "r"(sm_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void row_store(void* dst, const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(sm_u32(src)), "r"(bytes) : "memory");
}

// sqrt and the quotient use the hardware approximations (about 1e-7 relative each), far inside the
// 1e-5 this pass is held to
__device__ __forceinline__ void rms1(float& x, float g, float& v, float c, SweepHp hp) {
    const float gi = c * g;
    v = hp.alpha * v + (1.0f - hp.alpha) * gi * gi;
    float r;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(v));
    x = x - __fdividef(hp.lr * gi, r + hp.eps);
}

constexpr int kManyStages = 4;
constexpr int kManyConsumers = 256;

}  // namespace

// 288 threads: warps 0-7 compute, warp 8 moves data.  Stage rows: [x][g][v][peer 0][peer 1], `cols` floats each
// (only the rows an item uses are filled).
__global__ void __launch_bounds__(kManyConsumers + 32, 1) sweep_many_kernel(const SweepManyArgs p) {
    extern __shared__ __align__(128) float smem[];
    __shared__ __align__(8) uint64_t full[kManyStages];
    __shared__ __align__(8) uint64_t done[kManyStages];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int cols = p.cols, nst = p.stages;
    const int stage_floats = p.rows * cols;
    const long tiles = (p.d_pad + cols - 1) / cols;
    const long total = tiles * p.n_items;

    if (threadIdx.x == 0) {
        for (int s = 0; s < nst; s++) { mb_init(&full[s], 1); mb_init(&done[s], kManyConsumers); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();     // gradients and clip factors come from the kernels before
    pdl_launch();
    __syncthreads();

    const long first = blockIdx.x, step = gridDim.x;
    const long mine = first < total ? (total - first + step - 1) / step : 0;
    // item k -> (entry of the list, first column, number of columns)
    auto decode = [&](long k, int& e, long& c0, int& nc) {
        const long w = first + k * step;
        e = (int)(w / tiles);
        c0 = (w - (long)e * tiles) * cols;
        nc = (int)min((long)cols, p.d_pad - c0);
    };

    if (warp == kManyConsumers / 32) {
        // ---------------- mover warp: one elected lane issues every bulk copy
        if (lane == 0) {
            auto issue_loads = [&](long k, int stage) {
                int e, nc; long c0;
                decode(k, e, c0, nc);
                const SweepItem it = p.it[e];
                const bool grad = (p.has_grad[e >> 5] >> (e & 31)) & 1u;
                const uint32_t bytes = (uint32_t)nc * 4u;
                const int np = (it.p_row[0] >= 0) + (it.p_row[1] >= 0);
                float* st = smem + (long)stage * stage_floats;
                mb_expect(&full[stage], bytes * (uint32_t)(1 + (grad ? 2 : 0) + np));
                row_load(st, p.x + (long)it.x_row * p.d_pad + c0, bytes, &full[stage]);
                if (grad) {
                    row_load(st + cols, p.g + (long)it.x_row * p.d_pad + c0, bytes, &full[stage]);
                    row_load(st + 2 * cols, p.v + (long)it.x_row * p.d_pad + c0, bytes, &full[stage]);
                }
                if (np >= 1) row_load(st + 3 * cols, p.snap + (long)it.p_row[0] * p.d_pad + c0, bytes, &full[stage]);
                if (np >= 2) row_load(st + 4 * cols, p.snap + (long)it.p_row[1] * p.d_pad + c0, bytes, &full[stage]);
            };
            for (int s = 0; s < nst && s < mine; s++) issue_loads(s, s);
            for (long k = 0; k < mine; k++) {
                const int stage = (int)(k % nst);
                if (!mb_wait(&done[stage], (uint32_t)(k / nst) & 1u, p.error_word)) break;
                int e, nc; long c0;
                decode(k, e, c0, nc);
                const SweepItem it = p.it[e];
                const bool grad = (p.has_grad[e >> 5] >> (e & 31)) & 1u;
                const uint32_t bytes = (uint32_t)nc * 4u;
                const int np = (it.p_row[0] >= 0) + (it.p_row[1] >= 0);
                const float* st = smem + (long)stage * stage_floats;
                row_store(p.snap + (long)it.out_row * p.d_pad + c0, st, bytes);                 // y: the broadcast
                row_store(p.x + (long)it.x_row * p.d_pad + c0, np ? st + cols : st, bytes);     // the average, or y
                if (grad) row_store(p.v + (long)it.x_row * p.d_pad + c0, st + 2 * cols, bytes);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                if (k >= 1 && k - 1 + nst < mine) {
                    // stage of step k-1: all but the newest group of stores must have left shared memory
                    asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    issue_loads(k - 1 + nst, (int)((k - 1) % nst));
                }
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
        }
        return;
    }

    // ---------------- compute warps
    for (long k = 0; k < mine; k++) {
        const int stage = (int)(k % nst);
        int e, nc; long c0;
        decode(k, e, c0, nc);
        const SweepItem it = p.it[e];
        const bool grad = (p.has_grad[e >> 5] >> (e & 31)) & 1u;
        const int np = (it.p_row[0] >= 0) + (it.p_row[1] >= 0);
        const float cl = grad && p.clip ? __ldg(p.clip + it.x_row) : 1.0f;
        const float w = 1.0f / (1.0f + np);
        float4* sx = reinterpret_cast<float4*>(smem + (long)stage * stage_floats);
        float4* sg = sx + cols / 4;
        float4* sv = sg + cols / 4;
        const float4* s0 = sv + cols / 4;
        const float4* s1 = s0 + cols / 4;
        __nv_bfloat16* sh = p.shadow ? p.shadow + (long)it.x_row * p.d_pad + c0 : nullptr;
        if (!mb_wait(&full[stage], (uint32_t)(k / nst) & 1u, p.error_word)) break;
        for (int i = threadIdx.x; i < nc / 4; i += kManyConsumers) {
            float4 y = sx[i];
            if (grad) {
                float4 vi = sv[i];
                const float4 gi = sg[i];
                rms1(y.x, gi.x, vi.x, cl, p.hp); rms1(y.y, gi.y, vi.y, cl, p.hp);
                rms1(y.z, gi.z, vi.z, cl, p.hp); rms1(y.w, gi.w, vi.w, cl, p.hp);
                sx[i] = y;
                sv[i] = vi;
            }
            if (np) {
                const float4 m = s0[i];
                y.x += m.x; y.y += m.y; y.z += m.z; y.w += m.w;
                if (np > 1) {
                    const float4 m1 = s1[i];
                    y.x += m1.x; y.y += m1.y; y.z += m1.z; y.w += m1.w;
                }
                y.x *= w; y.y *= w; y.z *= w; y.w *= w;
                sg[i] = y;
            }
            if (sh) {
                const __nv_bfloat162 lo = __floats2bfloat162_rn(y.x, y.y), hi = __floats2bfloat162_rn(y.z, y.w);
                uint2 u;
                u.x = *reinterpret_cast<const unsigned*>(&lo);
                u.y = *reinterpret_cast<const unsigned*>(&hi);
                *reinterpret_cast<uint2*>(sh + 4 * i) = u;
            }
        }
        // make these writes visible to the bulk-copy engine, then hand the stage to the mover warp
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        mb_arrive(&done[stage]);
    }
}

cudaError_t launch_sweep_many(const SweepManyArgs& args, cudaStream_t st) {
    SweepManyArgs a = args;
    if (a.n_items < 1) return cudaSuccess;
    if (a.n_items > kBatch || (a.d_pad % 4) || a.d_pad < 4) return cudaErrorInvalidValue;
    if ((reinterpret_cast<uintptr_t>(a.x) | reinterpret_cast<uintptr_t>(a.g) | reinterpret_cast<uintptr_t>(a.v) |
         reinterpret_cast<uintptr_t>(a.snap)) & 15)
        return cudaErrorInvalidValue;
    if (a.shadow && (reinterpret_cast<uintptr_t>(a.shadow) & 7)) return cudaErrorInvalidValue;
    int max_np = 0;
    bool any_grad = false;
    for (int e = 0; e < a.n_items; e++) {
        const int np = (a.it[e].p_row[0] >= 0) + (a.it[e].p_row[1] >= 0);
        if (a.it[e].p_row[0] < 0 && a.it[e].p_row[1] >= 0) return cudaErrorInvalidValue;
        if (np > max_np) max_np = np;
        any_grad |= ((a.has_grad[e >> 5] >> (e & 31)) & 1u) != 0;
    }
    if (any_grad && (!a.g || !a.v)) return cudaErrorInvalidValue;
    // rows of a stage: x, g, v and the peers' rows (g doubles as the row the average is formed in); three or
    // four stages inside ~200 KiB, copies of 12-20 KiB each (the copy engine is bound by instructions: large rows)
    a.rows = 3 + max_np;
    const long budget = 200L * 1024;
    a.stages = 3;
    long cols = budget / ((long)a.stages * a.rows * 4);
    cols = cols / 256 * 256;
    if (cols > a.d_pad) { cols = (a.d_pad + 3) / 4 * 4; }
    if (cols < 4) return cudaErrorInvalidValue;
    a.cols = (int)cols;
    while (a.stages < kManyStages && (long)(a.stages + 1) * a.rows * a.cols * 4 <= budget) a.stages++;
    const long tiles = (a.d_pad + a.cols - 1) / a.cols;
    const long total = tiles * a.n_items;
    const size_t smem = (size_t)a.stages * a.rows * a.cols * 4;
    int sms = a.max_ctas > 0 ? a.max_ctas : sm_count();
    const int grid = (int)(total < sms ? total : sms);
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(sweep_many_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 208 * 1024);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    (void)launch_pdl(sweep_many_kernel, dim3(grid), dim3(kManyConsumers + 32), smem, st, a);
    return cudaGetLastError();
}

}  // namespace gala
