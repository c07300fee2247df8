// Weight gradients of conv2 and conv3 (Appendix C.2 network) on the tcgen05 tensor cores, with the
// layer input and the output gradient of a sample resident in shared memory.
//
//     dW[co][tap][ci] = sum over samples and output pixels r of  X[r + shift(tap)][ci] * dY[r][co]
//
// Output pixels are laid out with the pitch of the input image (9 for conv3, 10 for the parity planes
// of conv2), so that "+ shift(tap)" is a constant row offset into one shared-memory image of the
// input, and dY is fetched in the same pitch with the columns beyond the output width filled with
// zeros by TMA.  One MMA is  D[128][64] += A[128 x 16] * B[16 x 64]  with the pixel index as K:
//   A (MN-major): the input image; its 128 rows of D are several taps at once, each an "atom" of
//      channels whose start lies a constant number of bytes after the previous one (the leading byte
//      offset of the descriptor): two conv3 taps of 64 channels, or the four parity planes of conv2
//      (32 channels each, one plane apart) for one (ky / 2, kx / 2)
//   B (MN-major): dY[pixel][co]
// A CTA owns one agent and a slice of its samples; the accumulators of all tap groups (5 x 64 or
// 4 x 64 columns of tensor memory) stay in place over the whole slice, so every sample is read once
// and there is one epilogue per CTA.  With more than one slice per agent the CTAs write partial sums
// that a fixed-order reduction adds up afterwards.
//
//   warp 0    TMA producer (ring of stages: input planes + dY tile of one sample)
//   warp 1    MMA issuer (one thread)
//   warps 2-5 epilogue: D[(tap, ci)][co] -> out[co * KK + tap * CIN + ci], fp32
// Every wait is bounded (see conv.cu).
#include "internal.h"
#include "tcgen05.cuh"

namespace gala {

template <int W> struct WgradTraits;
template <> struct WgradTraits<WG_CONV2> {
    static constexpr int X_LAYOUT = 4, X_ROWB = 64, X_SBO = 512, PLANES = 4, PLANE_ROWS = 100, PLANE_STRIDE = 6656;
    static constexpr int X_BYTES = PLANES * PLANE_STRIDE;
    static constexpr int DY_ROWS = 100, DY_BYTES = 13312, KSTEPS = 6, GROUPS = 4, KK = 512;
};
template <> struct WgradTraits<WG_CONV3> {
    static constexpr int X_LAYOUT = 2, X_ROWB = 128, X_SBO = 1024, PLANES = 1, PLANE_ROWS = 81, PLANE_STRIDE = 11264;
    static constexpr int X_BYTES = PLANES * PLANE_STRIDE;
    static constexpr int DY_ROWS = 81, DY_BYTES = 11264, KSTEPS = 4, GROUPS = 5, KK = 576;
};
constexpr int kWgradMaxStages = 8;
constexpr int kWgradSmemMax = 216 * 1024;

// byte offset of the first atom of tap group g inside the input image, and the distance between atoms
template <int W> __host__ __device__ constexpr void group_view(int g, int& start, int& lbo) {
    if constexpr (W == WG_CONV2) { start = ((g >> 1) * 10 + (g & 1)) * 64; lbo = WgradTraits<W>::PLANE_STRIDE; }
    else {
        // tap pairs (0,1) (2,3) (4,5) (6,7) (8,-) at row shifts ky * 9 + kx
        constexpr int s0[5] = {0, 2, 10, 18, 20}, d[5] = {1, 7, 1, 1, 1};
        start = s0[g] * 128; lbo = d[g] * 128;
    }
}

template <int W>
__global__ void __launch_bounds__(192, 1)
wgrad_resident_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY, const WgradArgs p,
                      const int nst) {
    using T = WgradTraits<W>;
    constexpr int STAGE = T::X_BYTES + T::DY_BYTES;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kWgradMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kWgradMaxStages];
    __shared__ __align__(8) uint64_t acc_full;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int issued_iters;
    __shared__ float bias_part[4][64];

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t tmem_cols = T::GROUPS * 64 > 256 ? 512u : 256u;

    const int gz = blockIdx.x / p.splits, ss = blockIdx.x - gz * p.splits;
    const int slot = agent_slot(p.am, gz);
    const int s_begin = (int)((long)p.samples * ss / p.splits), s_end = (int)((long)p.samples * (ss + 1) / p.splits);
    const int n_it = s_end - s_begin;

    if (threadIdx.x == 0) {
        // a stage is released by the MMA issuer's commit and, when bias sums are wanted, by the four summing warps
        for (int s = 0; s < nst; s++) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], p.bias_out ? 5 : 1); }
        mbar_init(&acc_full, 1);
        abort_flag = 0;
        issued_iters = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    {   // Rows that no copy ever writes (the tail of a plane, the gap up to a multiple of 16 pixels) are read
        // by MMAs whose other operand is zero there; they must hold finite values, so the ring starts zeroed.
        uint4* z = reinterpret_cast<uint4*>(smem);
        const int n16 = nst * STAGE / 16;
        for (int i = threadIdx.x; i < n16; i += blockDim.x) z[i] = make_uint4(0, 0, 0, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = tmem_slot;
    pdl_wait();     // set-up above overlaps the previous kernel; its results are read from here on
    pdl_launch();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        for (int it = 0; it < n_it; it++) {
            const int s = it % nst;
            int go = 1;
            if (lane == 0) go = mbar_wait(&empty_bar[s], ((uint32_t)(it / nst) & 1u) ^ 1u, &abort_flag) ? 1 : 0;
            go = __shfl_sync(0xffffffffu, go, 0);
            if (!go) break;
            if (lane == 0) mbar_expect_tx(&full_bar[s], (uint32_t)(T::PLANES * T::PLANE_ROWS * T::X_ROWB + T::DY_ROWS * 128));
            __syncwarp();
            const int sx = (p.group0 + slot) * p.x_samples + s_begin + it;
            const int sy = (p.group0 + slot) * p.y_samples + s_begin + it;
            uint8_t* dst = smem + s * STAGE;
            if (lane < T::PLANES) {
                if constexpr (W == WG_CONV2) tma_load_5d(dst + lane * T::PLANE_STRIDE, &tmX, &full_bar[s], 32 * (lane & 1), 0, lane >> 1, 0, sx);
                else tma_load_3d(dst, &tmX, &full_bar[s], 0, 0, sx);
            } else if (lane == T::PLANES) {
                tma_load_4d(dst + T::X_BYTES, &tmY, &full_bar[s], 0, 0, 0, sy);
            }
            __syncwarp();
            if (lane == 0) issued_iters = it + 1;
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            // a: MN-major (bit 15), b: MN-major (bit 16), N = 64, M = 128
            const uint32_t idesc = make_instr_desc(64, 1, 1);
            bool ok = true;
            for (int it = 0; ok && it < n_it; it++) {
                const int s = it % nst;
                if (!mbar_wait(&full_bar[s], (uint32_t)(it / nst) & 1u, &abort_flag)) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t x_addr = smem_u32(smem + s * STAGE);
                const uint64_t bd_base = make_smem_desc_raw(x_addr + T::X_BYTES, 2, 1024, 8192);
#pragma unroll
                for (int g = 0; g < T::GROUPS; g++) {
                    int start, lbo;
                    group_view<W>(g, start, lbo);
                    const uint64_t ad_base = make_smem_desc_raw(x_addr + start, T::X_LAYOUT, T::X_SBO, lbo);
#pragma unroll
                    for (int kk = 0; kk < T::KSTEPS; kk++)   // 16 pixels further: 16 rows of either image
                        umma_bf16(tmem_base + (uint32_t)(g * 64), ad_base + (uint64_t)((kk * 16 * T::X_ROWB) >> 4),
                                  bd_base + (uint64_t)((kk * 2048) >> 4), idesc, (it | kk) != 0 ? 1u : 0u);
                }
                umma_commit(&empty_bar[s]);
            }
            if (ok) {
                if (n_it > 0) umma_commit(&acc_full);
                else mbar_arrive(&acc_full);
            }
        }
    } else {
        if (p.bias_out) {
            // ------------------------------------------------ bias gradient: column sums of the dY tiles while they
            // are in shared memory (rows of 64 channels, 128-byte swizzle; rows beyond the output width are zero).
            // The four warps take every fourth row, lane l owns channels 2l, 2l + 1, four independent partial
            // sums per lane keep loads in flight; fixed order: rows, samples, partial sums, warps.
            const int wq = warp - 2;
            float b0[4] = {0.f, 0.f, 0.f, 0.f}, b1[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t lane_off = (uint32_t)((lane & 3) << 2);
            for (int it = 0; it < n_it; it++) {
                const int s = it % nst;
                if (!mbar_wait(&full_bar[s], (uint32_t)(it / nst) & 1u, &abort_flag)) break;
                const uint8_t* dy = smem + s * STAGE + T::X_BYTES;
                for (int r0 = wq; r0 < T::DY_ROWS; r0 += 16) {
                    uint32_t w[4];
#pragma unroll
                    for (int u = 0; u < 4; u++) {
                        const int r = r0 + 4 * u;
                        w[u] = r < T::DY_ROWS ? *reinterpret_cast<const uint32_t*>(dy + r * 128 + (((lane >> 2) ^ (r & 7)) << 4) + lane_off) : 0u;
                    }
#pragma unroll
                    for (int u = 0; u < 4; u++) { b0[u] += __uint_as_float(w[u] << 16); b1[u] += __uint_as_float(w[u] & 0xffff0000u); }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[s]);
            }
            bias_part[wq][2 * lane] = (b0[0] + b0[1]) + (b0[2] + b0[3]);
            bias_part[wq][2 * lane + 1] = (b1[0] + b1[1]) + (b1[2] + b1[3]);
            asm volatile("bar.sync 1, 128;" ::: "memory");   // the four epilogue warps
            if (wq == 0) {
                float* bo = p.bias_out + (long)slot * p.bias_group_stride + (long)ss * p.bias_split_stride;
                for (int c0 = lane; c0 < 64; c0 += 32)
                    bo[c0] = ((bias_part[0][c0] + bias_part[1][c0]) + bias_part[2][c0]) + bias_part[3][c0];
            }
        }
        // ------------------------------------------------ epilogue (once): thread = row (tap, ci) of D
        const int q = warp & 3;
        if (mbar_wait(&acc_full, 0u, &abort_flag)) {
            tcgen05_fence_after();
            const int m = q * 32 + lane;
            float* out = p.out + (long)slot * p.out_group_stride + (long)ss * p.out_split_stride;
#pragma unroll 1
            for (int g = 0; g < T::GROUPS; g++) {
                int col;   // column (tap, ci) of W[co][KK] that row m of group g holds, -1: none
                if constexpr (W == WG_CONV2) {
                    const int pl = m >> 5, ci = m & 31;
                    const int ky = 2 * (g >> 1) + (pl >> 1), kx = 2 * (g & 1) + (pl & 1);
                    col = (ky * 4 + kx) * 32 + ci;
                } else {
                    const int t = 2 * g + (m >> 6);
                    col = t < 9 ? t * 64 + (m & 63) : -1;
                }
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t r[32];
                    if (n_it > 0) tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(g * 64 + c0), r);
                    else {
#pragma unroll
                        for (int j = 0; j < 32; j++) r[j] = 0u;
                    }
                    if (col >= 0) {
                        // for one co the 32 lanes hold 32 consecutive ci: 128 contiguous bytes per store
#pragma unroll
                        for (int j = 0; j < 32; j++) out[(long)(c0 + j) * T::KK + col] = __uint_as_float(r[j]);
                    }
                }
            }
        }
    }

    // teardown
    tcgen05_fence_before();
    __syncthreads();
    if (abort_flag) {
        if (threadIdx.x == 0) {
            if (p.error_word) atomicExch(p.error_word, 20 + W);
            const int issued = issued_iters;
            for (int it = max(0, issued - nst); it < issued; it++) {
                const int s = it % nst;
                const uint32_t ph = (uint32_t)(it / nst) & 1u;
                for (uint32_t i = 0; i < (1u << 16); i++) {
                    if (mbar_try_wait(&full_bar[s], ph)) break;
                    __nanosleep(64);
                }
            }
        }
        __syncthreads();
    }
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------ host side
cudaError_t wgrad_init() {
    static bool done = false;
    if (done) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(wgrad_resident_kernel<WG_CONV2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kWgradSmemMax);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(wgrad_resident_kernel<WG_CONV3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kWgradSmemMax);
    if (e != cudaSuccess) return e;
    done = true;
    return cudaSuccess;
}

bool make_wgrad_maps(int variant, CUtensorMap* x_map, CUtensorMap* y_map, const void* x_base, uint64_t x_samples,
                     const void* y_base, uint64_t y_samples) {
    bool ok = true;
    if (variant == WG_CONV2) {
        // act1 [sample][20][20][32] as [sample][y/2][y%2][x/2][2 px x 32 ch]; dY2 [sample][9][9][64] in pitch 10
        const uint64_t dims[5] = {64, 10, 2, 10, x_samples}, str[4] = {128, 1280, 2560, 25600};
        const uint32_t box[5] = {32, 10, 1, 10, 1};
        ok &= make_tensor_map_nd(x_map, x_base, 5, dims, str, box, 1);
        const uint64_t yd[4] = {64, 9, 9, y_samples}, ys[3] = {128, 1152, 10368};
        const uint32_t yb[4] = {64, 10, 10, 1};
        ok &= make_tensor_map_nd(y_map, y_base, 4, yd, ys, yb, 0);
    } else if (variant == WG_CONV3) {
        // act2 [sample][81][64]; dY3 [sample][7][7][64] in pitch 9
        const uint64_t dims[3] = {64, 81, x_samples}, str[2] = {128, 10368};
        const uint32_t box[3] = {64, 81, 1};
        ok &= make_tensor_map_nd(x_map, x_base, 3, dims, str, box, 0);
        const uint64_t yd[4] = {64, 7, 7, y_samples}, ys[3] = {128, 896, 6272};
        const uint32_t yb[4] = {64, 9, 9, 1};
        ok &= make_tensor_map_nd(y_map, y_base, 4, yd, ys, yb, 0);
    } else return false;
    return ok;
}

template <int W>
static cudaError_t launch_wgrad_v(const CUtensorMap& x, const CUtensorMap& y, const WgradArgs& a, cudaStream_t st) {
    using T = WgradTraits<W>;
    constexpr int STAGE = T::X_BYTES + T::DY_BYTES;
    int nst = (kWgradSmemMax - 1024) / STAGE;
    if (nst > kWgradMaxStages) nst = kWgradMaxStages;
    const size_t smem = (size_t)nst * STAGE + 1024;
    (void)launch_pdl(wgrad_resident_kernel<W>, dim3(a.groups * a.splits), dim3(192), smem, st, x, y, a, nst);
    return cudaGetLastError();
}

cudaError_t launch_wgrad(const CUtensorMap& x, const CUtensorMap& y, const WgradArgs& a, cudaStream_t st) {
    if (a.groups < 1 || a.splits < 1 || a.samples < 1 || a.splits > a.samples || !a.out) return cudaErrorInvalidValue;
    if (a.variant == WG_CONV2) return launch_wgrad_v<WG_CONV2>(x, y, a, st);
    if (a.variant == WG_CONV3) return launch_wgrad_v<WG_CONV3>(x, y, a, st);
    return cudaErrorInvalidValue;
}

}  // namespace gala
