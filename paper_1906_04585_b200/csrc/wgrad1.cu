// Weight gradient of conv1 (8x8, stride 4, 4 -> 32 channels; Appendix C.2 network) on the tcgen05 tensor
// cores, read from the uint8 frames themselves.
//
//     dW[co][ky][kx][ci] = 1/255 * sum over samples and output pixels (oy, ox) of
//                          frame[4 oy + ky][4 ox + kx][ci] * dY[oy][ox][co]
//
// Work unit: five output lines of one sample (a quarter), i.e. 24 input lines = one contiguous piece
// of 8064 bytes, fetched by one bulk copy and widened to bf16 by eight converter warps (0..255 are exact
// in bf16).  The converters lay the lines out as phase planes: plane py holds lines y = 4u + py, a
// line as 21 rows of 16 elements (4 pixels x 4 channels, 32 bytes), row index u * 21 + xq.  With the
// output pixels in the same pitch (r = oy * 21 + ox; dY is fetched in pitch 21, column 20 filled with
// zeros by TMA) the 16 elements (kx % 4, ci) of tap (ky, kx / 4) are row r + (ky / 4) * 21 + kx / 4 of
// plane ky % 4.  Each plane is stored twice, the second copy one row up, so that the eight taps
// (ky % 4, kx / 4) of one ky / 4 start at the same row of eight planes a constant distance apart: they
// are the eight 16-element atoms of one MN-major A operand.  The remaining shift, 21 rows for ky / 4 = 1, is
// moved to the other operand: sum_r X[r + 21][m] dY[r][co] = sum_r' X[r'][m] dY[r' - 21][co], so the B operand
// is two views of the same dY tile, 21 rows apart (rows before and after the tile are zero), as the two
// 32-channel atoms of one MN-major N = 64 operand.  One MMA is
//     D[(ky % 4, kx / 4, kx % 4, ci)][(ky / 4, co)] += A[128 x 16 pixels] * B[16 pixels x 64]
// with the pixel index as K: 8 MMAs per unit instead of 14 with N = 32.  The accumulator (64 columns) stays in
// tensor memory over the CTA's whole slice of samples; there is one epilogue per CTA, and with more than one
// slice per agent the partial sums go through the fixed-order reduction.
//
//   warp 0     producer: bulk copy of the frame lines, TMA copy of the dY tile
//   warp 1     MMA issuer (one thread)
//   warps 2-9  converters; warps 2-5 are also the epilogue
// Every wait is bounded (see conv.cu).
#include "internal.h"
#include "tcgen05.cuh"

namespace gala {

constexpr int kW1Planes = 8, kW1PlaneStride = 4096, kW1XBytes = kW1Planes * kW1PlaneStride;
// dY region of a stage: 24 zero rows, the 105 rows of the tile (five lines in pitch 21), zero rows up to 160
constexpr int kW1DyRows = 105, kW1DyPad = 24, kW1DyBytes = 160 * 64;
constexpr int kW1Stage = kW1XBytes + kW1DyBytes;            // 43008
constexpr int kW1Stages = 4;
constexpr int kW1U8Stages = 4, kW1U8Bytes = 24 * 336, kW1U8Stride = 8192;
constexpr int kW1Smem = kW1Stages * kW1Stage + kW1U8Stages * kW1U8Stride + 1024;
constexpr int kW1ConvWarps = 8, kW1Threads = 64 + 32 * kW1ConvWarps;
constexpr int kW1KSteps = 8;                                // 128 pixel rows of 16 (105 of the tile + the 21-row shift)

__global__ void __launch_bounds__(kW1Threads, 1)
wgrad_conv1_kernel(const __grid_constant__ CUtensorMap tmY, const Wgrad1Args p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kW1Stages];
    __shared__ __align__(8) uint64_t empty_bar[kW1Stages];
    __shared__ __align__(8) uint64_t u8_full[kW1U8Stages];
    __shared__ __align__(8) uint64_t u8_empty[kW1U8Stages];
    __shared__ __align__(8) uint64_t acc_full;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int issued_u8, issued_dy;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* smU = smem + kW1Stages * kW1Stage;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t tmem_cols = 64;

    const int gz = blockIdx.x / p.splits, ss = blockIdx.x - gz * p.splits;
    const int slot = agent_slot(p.am, gz);
    const int s_begin = (int)((long)p.samples * ss / p.splits), s_end = (int)((long)p.samples * (ss + 1) / p.splits);
    const int n_it = (s_end - s_begin) * 4;

    if (threadIdx.x == 0) {
        // a stage is full after the eight converter warps and the dY copy (one arrival with a byte count)
        for (int s = 0; s < kW1Stages; s++) { mbar_init(&full_bar[s], kW1ConvWarps + 1); mbar_init(&empty_bar[s], 1); }
        for (int s = 0; s < kW1U8Stages; s++) { mbar_init(&u8_full[s], 1); mbar_init(&u8_empty[s], kW1ConvWarps); }
        mbar_init(&acc_full, 1);
        abort_flag = 0;
        issued_u8 = 0;
        issued_dy = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    {   // Rows that nothing ever writes (the tail of a plane, the rows around the dY tile) are read by MMAs; the
        // dY rows must be zero and the others finite, so the ring starts zeroed.
        uint4* z = reinterpret_cast<uint4*>(smem);
        const int n16 = kW1Stages * kW1Stage / 16;
        for (int i = threadIdx.x; i < n16; i += blockDim.x) z[i] = make_uint4(0, 0, 0, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = tmem_slot;
    pdl_wait();
    pdl_launch();

    if (warp == 0) {
        // ------------------------------------------------ producer
        const uint8_t* frames = reinterpret_cast<const uint8_t*>(p.obs.p[gz]);
        for (int it = 0; it < n_it; it++) {
            const int sample = s_begin + (it >> 2), q = it & 3;
            const int su = it % kW1U8Stages, s = it % kW1Stages;
            int go = 1;
            if (lane == 0) go = mbar_wait(&u8_empty[su], ((uint32_t)(it / kW1U8Stages) & 1u) ^ 1u, &abort_flag) ? 1 : 0;
            go = __shfl_sync(0xffffffffu, go, 0);
            if (!go) break;
            if (lane == 0) {
                mbar_expect_tx(&u8_full[su], (uint32_t)kW1U8Bytes);
                bulk_load_1d(smU + su * kW1U8Stride, frames + (long)sample * (84 * 336) + q * (20 * 336), (uint32_t)kW1U8Bytes,
                             &u8_full[su]);
                issued_u8 = it + 1;
            }
            if (lane == 0) go = mbar_wait(&empty_bar[s], ((uint32_t)(it / kW1Stages) & 1u) ^ 1u, &abort_flag) ? 1 : 0;
            go = __shfl_sync(0xffffffffu, go, 0);
            if (!go) break;
            if (lane == 0) {
                mbar_expect_tx(&full_bar[s], (uint32_t)(kW1DyRows * 64));
                tma_load_4d(smem + s * kW1Stage + kW1XBytes + kW1DyPad * 64, &tmY, &full_bar[s], 0, 0, 5 * q,
                            (p.group0 + slot) * p.y_samples + sample);
                issued_dy = it + 1;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_instr_desc(64, 1, 1);   // A and B MN-major, N = 64, M = 128
            bool ok = true;
            for (int it = 0; ok && it < n_it; it++) {
                const int s = it % kW1Stages;
                if (!mbar_wait(&full_bar[s], (uint32_t)(it / kW1Stages) & 1u, &abort_flag)) { ok = false; break; }
                tcgen05_fence_after();
                const uint32_t x_addr = smem_u32(smem + s * kW1Stage);
                // B: atom 0 = the tile moved down by 21 rows (ky / 4 = 1), atom 1 = the tile itself (ky / 4 = 0)
                const uint64_t bd_base = make_smem_desc_raw(x_addr + kW1XBytes + (kW1DyPad - 21) * 64, 4, 512, 21 * 64);
                // A: 32-byte rows, groups of 8 rows 256 bytes apart, the eight atoms one plane apart
                const uint64_t ad_base = make_smem_desc_raw(x_addr, 6, 256, kW1PlaneStride);
#pragma unroll
                for (int kk = 0; kk < kW1KSteps; kk++)   // 16 pixels further: 16 rows of either image
                    umma_bf16(tmem_base, ad_base + (uint64_t)((kk * 16 * 32) >> 4), bd_base + (uint64_t)((kk * 16 * 64) >> 4),
                              idesc, (it | kk) != 0 ? 1u : 0u);
                umma_commit(&empty_bar[s]);
            }
            if (ok) {
                if (n_it > 0) umma_commit(&acc_full);
                else mbar_arrive(&acc_full);
            }
        }
    } else {
        // ------------------------------------------------ converters: uint8 lines -> bf16 phase planes, two copies
        const int ct = threadIdx.x - 64;   // 0 .. 32 * kW1ConvWarps - 1
        constexpr int kCT = 32 * kW1ConvWarps, kChunks = 24 * 21;
        bool ok = true;
        for (int it = 0; it < n_it; it++) {
            const int su = it % kW1U8Stages, s = it % kW1Stages;
            if (!mbar_wait(&u8_full[su], (uint32_t)(it / kW1U8Stages) & 1u, &abort_flag)) { ok = false; break; }
            if (!mbar_wait(&empty_bar[s], ((uint32_t)(it / kW1Stages) & 1u) ^ 1u, &abort_flag)) { ok = false; break; }
            const uint8_t* src = smU + su * kW1U8Stride;
            uint8_t* dstage = smem + s * kW1Stage;
#pragma unroll
            for (int k = 0; k < (kChunks + kCT - 1) / kCT; k++) {
                const int ch = ct + k * kCT;          // 16-byte group of the block, 504 in all
                if (ch < kChunks) {
                    const int yl = ch / 21, xq = ch - yl * 21;
                    const uint4 v = *reinterpret_cast<const uint4*>(src + ch * 16);
                    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
                    uint32_t o[8];
#pragma unroll
                    for (int e = 0; e < 4; e++) {
                        o[2 * e] = u8x2_to_bf16x2(w[e], 0);
                        o[2 * e + 1] = u8x2_to_bf16x2(w[e], 2);
                    }
                    // copy 0 at row r, copy 1 (the kx / 4 = 1 taps) at row r - 1; a 32-byte row's halves swap
                    // when bit 7 of its address is set (32-byte swizzle)
                    const int r = (yl >> 2) * 21 + xq;
                    uint8_t* plane = dstage + (yl & 3) * (2 * kW1PlaneStride);
                    {
                        uint8_t* row = plane + r * 32;
                        const int sw = ((r >> 2) & 1) * 16;
                        *reinterpret_cast<uint4*>(row + sw) = make_uint4(o[0], o[1], o[2], o[3]);
                        *reinterpret_cast<uint4*>(row + (sw ^ 16)) = make_uint4(o[4], o[5], o[6], o[7]);
                    }
                    if (r > 0) {
                        const int r1 = r - 1;
                        uint8_t* row = plane + kW1PlaneStride + r1 * 32;
                        const int sw = ((r1 >> 2) & 1) * 16;
                        *reinterpret_cast<uint4*>(row + sw) = make_uint4(o[0], o[1], o[2], o[3]);
                        *reinterpret_cast<uint4*>(row + (sw ^ 16)) = make_uint4(o[4], o[5], o[6], o[7]);
                    }
                }
            }
            // make the generic-proxy writes visible to the tensor core's reads, then hand the stage over
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) { mbar_arrive(&full_bar[s]); mbar_arrive(&u8_empty[su]); }
        }
        // ------------------------------------------------ epilogue (once): thread = row (ky % 4, kx / 4, kx % 4, ci) of D
        if (warp < 6 && ok && mbar_wait(&acc_full, 0u, &abort_flag)) {
            tcgen05_fence_after();
            const int q = warp & 3;
            const int m = q * 32 + lane;
            const int py = m >> 5, b = (m >> 4) & 1, el = m & 15;
            float* out = p.out + (long)slot * p.out_group_stride + (long)ss * p.out_split_stride;
#pragma unroll
            for (int h = 0; h < 2; h++) {
                const int col = ((4 * h + py) * 8 + 4 * b) * 4 + el;   // (ky, kx, ci) inside W[co][256]
                uint32_t r[32];
                if (n_it > 0) tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)((1 - h) * 32), r);
                else {
#pragma unroll
                    for (int j = 0; j < 32; j++) r[j] = 0u;
                }
#pragma unroll
                for (int j = 0; j < 32; j++) out[(long)j * 256 + col] = __uint_as_float(r[j]) * p.scale;
            }
        }
    }

    // teardown
    tcgen05_fence_before();
    __syncthreads();
    if (abort_flag) {
        if (threadIdx.x == 0) {
            if (p.error_word) atomicExch(p.error_word, 30);
            // let copies that were already issued land before the shared memory goes away
            for (int it = max(0, issued_u8 - kW1U8Stages); it < issued_u8; it++) {
                const uint32_t ph = (uint32_t)(it / kW1U8Stages) & 1u;
                for (uint32_t i = 0; i < (1u << 16); i++) {
                    if (mbar_try_wait(&u8_full[it % kW1U8Stages], ph)) break;
                    __nanosleep(64);
                }
            }
            for (uint32_t i = 0; issued_dy > 0 && i < (1u << 14); i++) __nanosleep(64);   // dY copies: no phase to wait on
        }
        __syncthreads();
    }
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// ------------------------------------------------------------------ host side
cudaError_t wgrad1_init() {
    static bool done = false;
    if (done) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(wgrad_conv1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kW1Smem);
    if (e != cudaSuccess) return e;
    done = true;
    return cudaSuccess;
}

// dY1 [sample][20][20][32] fetched as five lines in pitch 21 (the 21st pixel of a line reads as zero)
bool make_wgrad1_map(CUtensorMap* y_map, const void* y_base, uint64_t y_samples) {
    const uint64_t yd[4] = {32, 20, 20, y_samples}, ys[3] = {64, 1280, 25600};
    const uint32_t yb[4] = {32, 21, 5, 1};
    return make_tensor_map_nd(y_map, y_base, 4, yd, ys, yb, 1);
}

cudaError_t launch_wgrad1(const CUtensorMap& y, const Wgrad1Args& a, cudaStream_t st) {
    if (a.groups < 1 || a.groups > kBatch || a.splits < 1 || a.samples < 1 || a.splits > a.samples || !a.out)
        return cudaErrorInvalidValue;
    for (int i = 0; i < a.groups; i++)
        if (!a.obs.p[i] || (reinterpret_cast<uintptr_t>(a.obs.p[i]) & 15)) return cudaErrorInvalidValue;
    (void)launch_pdl(wgrad_conv1_kernel, dim3(a.groups * a.splits), dim3(kW1Threads), (size_t)kW1Smem, st, y, a);
    return cudaGetLastError();
}

}  // namespace gala
