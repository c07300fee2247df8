// Convolutions of the 84x84x4 -> 20x20x32 -> 9x9x64 -> 7x7x64 trunk (Appendix C.2 network), forward
// and data gradient, on the tcgen05 tensor cores with the layer input resident in shared memory.
//
// A convolution is a sum over kernel offsets ("taps") of small products
//     D[pixel][n] += X[pixel + offset(tap)][k] * Wtap[k][n] .
// When the pixels of an image are laid out row after row with a fixed pitch, "pixel + offset" is a
// constant row shift, so every tap reads the SAME shared-memory image of the input, only from a
// start address moved by shift * row_bytes.  The input of one work unit (a sample, or six output
// lines of conv1) is therefore fetched once by TMA - not once per tap - and all weights of the layer
// stay in shared memory while a CTA works on one agent.  Rows whose pixel falls outside the valid
// output range (the pitch minus the output width, the tail of the 128-row MMA tile) are computed
// and dropped by the epilogue.
//
// Strided layers are turned into shifts by splitting the input into phase planes:
//   conv1 (8x8, stride 4): a row of the shared-memory image = one group of 4 pixels x 4 channels of the four
//          input lines y = 4u + py side by side (4 x 16 elements = 128 bytes, 128-byte swizzle; rows whose
//          16 elements ARE the row, 32 bytes wide, make the tensor core fetch its operands at a fraction of
//          the rate: 224 cycles per 128 x 64 x 16 MMA measured against ~70 with 128-byte rows); tap (ky, b):
//          K slice ky % 4 of the row, shift (ky / 4) * 21 + b: 16 MMAs of N = 32 per unit.  (Folding b into
//          N = 64 columns halves the MMAs, but the epilogue must then add column block 1 of the NEXT row to
//          block 0 of a row, across lanes and warps, and that cost more than the MMAs saved: a thread issues
//          an MMA of M = 128, K = 16 every ~80 cycles whatever N <= 128 is, two issuing threads reach one per
//          ~42 cycles at N = 32 and ~50 at N = 64, measured.)  Operands are fp16, not
//          bf16: a byte widens to fp16 with one byte permutation and one packed subtraction for two pixels
//          (0x6400 | b is 1024 + b), and the layer's weights, bf16 values, are exact in fp16 after a scaling
//          by 2^12 that the epilogue takes back (|w| < 16; weights below 2^-26 lose low bits).
//   conv2 (4x4, stride 2): plane (py, px) = pixels (2u + py, 2v + px), 32 channels a row; tap (ky, kx):
//          plane (ky % 2, kx % 2), shift (ky / 2) * 10 + kx / 2
//   conv3 (3x3, stride 1): one plane, shift ky * 9 + kx
// Data gradients use the zero-padded gradient image of the layer output (TMA fills out-of-range
// coordinates with zeros), pitch 11:
//   conv3: dX[y][x] = sum_taps dY[y - ky][x - kx] W[.][ky][kx][.], shift (2 - ky) * 11 + (2 - kx)
//   conv2: the four parity classes (py, px) of input pixels (2u + py, 2v + px) share the shifted dY
//          view of tap (a, b) = (ky / 2, kx / 2) and differ only in the weight block, so they become
//          the N = 4 x 32 columns of one product: shift (1 - a) * 11 + (1 - b)
//
// One CTA (352 threads, persistent over a contiguous range of work units):
//   warp 0    TMA producer: input planes of the next units into a ring of stages; the agent's weights
//             whenever the agent changes
//   warps 1, 10  two MMA issuers (one thread each) that take the units alternately, each with its own
//             tensor-memory accumulator: taps x K-chunks tcgen05.mma per unit.  While one waits for the
//             barriers of its next unit, the tensor pipe works on the other's MMAs.
//   warps 2-9 two epilogue groups of four warps, one per issuer (two accumulator buffers each): tcgen05.ld (a thread owns a
//             pixel), scale / bias / ReLU (+ gate bits) or the ReLU gate, 64 contiguous bytes of bf16 per 32 columns
// Every wait is bounded; when one runs out the CTA raises the caller's error word, lets the copies it
// issued land, frees its tensor memory and returns.
#include "internal.h"
#include "tcgen05.cuh"

namespace gala {

template <int V> struct ConvTraits;
template <> struct ConvTraits<CV_CONV1_FWD> {
    static constexpr int ROWB = 128, LAYOUT = 2, PLANES = 1, PLANE_ROWS = 147, PLANE_STRIDE = 19456;
    static constexpr int TAPS = 4, KKN = 4, BN = 32, PITCH = 21, OH = 6, OW = 20;   // tap 2 dy + b = kernel lines 4 dy .. 4 dy + 3, pixel group b
    // the weights arrive as 16 unswizzled boxes [32 co x 16 k] (box 2 ky + b) and are laid out for the products by
    // the converter warps: tile 2 dy + b = rows co x 128 bytes (K slice ky % 4 at 32 (ky % 4)), 128-byte swizzle
    static constexpr int W_BOXES = 16, W_BOX_BYTES = 1024, B_MN = 0, B_LAYOUT = 2, B_SBO = 1024, B_LBO = 16;
};
template <> struct ConvTraits<CV_CONV2_FWD> {
    static constexpr int ROWB = 64, LAYOUT = 4, PLANES = 4, PLANE_ROWS = 100, PLANE_STRIDE = 6656;
    static constexpr int TAPS = 16, KKN = 2, BN = 64, PITCH = 10, OH = 9, OW = 9;
    static constexpr int W_BOXES = 16, W_BOX_BYTES = 4096, B_MN = 0, B_LAYOUT = 4, B_SBO = 512, B_LBO = 16;
};
template <> struct ConvTraits<CV_CONV3_FWD> {
    static constexpr int ROWB = 128, LAYOUT = 2, PLANES = 1, PLANE_ROWS = 81, PLANE_STRIDE = 11264;
    static constexpr int TAPS = 9, KKN = 4, BN = 64, PITCH = 9, OH = 7, OW = 7;
    static constexpr int W_BOXES = 9, W_BOX_BYTES = 8192, B_MN = 0, B_LAYOUT = 2, B_SBO = 1024, B_LBO = 16;
};
template <> struct ConvTraits<CV_CONV2_DGRAD> {
    static constexpr int ROWB = 128, LAYOUT = 2, PLANES = 1, PLANE_ROWS = 121, PLANE_STRIDE = 16384;
    static constexpr int TAPS = 4, KKN = 4, BN = 128, PITCH = 11, OH = 10, OW = 10;
    static constexpr int W_BOXES = 16, W_BOX_BYTES = 4096, B_MN = 1, B_LAYOUT = 4, B_SBO = 512, B_LBO = 4096;
};
template <> struct ConvTraits<CV_CONV3_DGRAD> {
    static constexpr int ROWB = 128, LAYOUT = 2, PLANES = 1, PLANE_ROWS = 121, PLANE_STRIDE = 16384;
    static constexpr int TAPS = 9, KKN = 4, BN = 64, PITCH = 11, OH = 9, OW = 9;
    static constexpr int W_BOXES = 9, W_BOX_BYTES = 8192, B_MN = 1, B_LAYOUT = 2, B_SBO = 1024, B_LBO = 8192;
};

constexpr int kConvMaxStages = 8;
constexpr int kConvSlack = 8 * 1024;             // rows an MMA reads past the last plane of the ring
constexpr int kConvEpiWarpBytes = 512;           // an epilogue warp's copy of the layer's bias
constexpr int kConvSmemMax = 224 * 1024;
constexpr int kConv1SmemMax = 226 * 1024;           // conv1 forward: all a block may have but 1 KB for the static part
// conv1 reads the uint8 frames themselves.  An agent's frames are one long run of groups of four lines
// (1344 bytes each, 21 per frame), and output line L of that run (frame L / 21, line L % 21; line 20 of a
// frame does not exist and is dropped) needs groups L and L + 1.  A unit is six consecutive output lines
// wherever frames begin and end: 126 of the 128 rows of an MMA are pixel slots.  The seven groups behind
// them are one contiguous piece, staged as it is and widened to an fp16 plane by four more warps.
constexpr int kC1Lines = 6;                          // output lines of a unit
constexpr int kC1Group = 4 * 336;                    // bytes of four input lines
constexpr int kU8Stages = 8;                        // two line blocks in flight per converter warp
constexpr int kU8Bytes = (kC1Lines + 1) * kC1Group;  // 9408
constexpr int kU8Stride = 9472;
constexpr int kC1ConvWarps = 4;                     // conv1: warps that widen the uint8 lines, a whole unit each in turn
// (15 warps in all, so that 128 registers a thread fit).  A ring slot must always be handled by
// the same converter warp, in order: a wait for a slot's later phase passes at once while an earlier one is pending.
static_assert(kU8Stages % kC1ConvWarps == 0, "a byte ring slot belongs to one converter warp");
static_assert(kC1ConvWarps % 2 == 0, "a stage belongs to one converter warp and to one of the two issuers");
constexpr float kC1WeightScale = 4096.0f;           // conv1's weights enter the products as fp16(w * 2^12)
constexpr int kConvThreads = 352, kConv1Threads = 352 + 32 * kC1ConvWarps;

// plane and row shift of a tap
template <int V> __host__ __device__ constexpr void tap_view(int t, int& plane, int& shift) {
    if constexpr (V == CV_CONV1_FWD) { plane = 0; shift = (t >> 1) * 21 + (t & 1); }
    else if constexpr (V == CV_CONV2_FWD) { const int ky = t >> 2, kx = t & 3; plane = (ky & 1) * 2 + (kx & 1); shift = (ky >> 1) * 10 + (kx >> 1); }
    else if constexpr (V == CV_CONV3_FWD) { const int ky = t / 3; plane = 0; shift = ky * 9 + (t - ky * 3); }
    else if constexpr (V == CV_CONV2_DGRAD) { plane = 0; shift = (1 - (t >> 1)) * 11 + (1 - (t & 1)); }
    else { const int ky = t / 3; plane = 0; shift = (2 - ky) * 11 + (2 - (t - ky * 3)); }
}
// first column (inside W[co][(ky, kx, ci)]) of the weight box that goes to shared-memory slot j
template <int V> __device__ __forceinline__ int weight_col(int j) {
    if constexpr (V == CV_CONV1_FWD) return j * 16;
    else if constexpr (V == CV_CONV2_FWD) return j * 32;
    else if constexpr (V == CV_CONV2_DGRAD) {
        // slot = tap * 4 + class: the four classes of a tap side by side form its N = 128 operand
        const int t = j >> 2, cls = j & 3;
        return (((cls >> 1) + 2 * (t >> 1)) * 4 + (cls & 1) + 2 * (t & 1)) * 32;
    } else return j * 64;
}

// units of one agent: a sample each, except conv1 (six output lines of the agent's run of frames)
template <int V> __host__ __device__ __forceinline__ int units_per_group(int rows) {
    if constexpr (V == CV_CONV1_FWD) return (21 * rows + kC1Lines - 1) / kC1Lines;
    else return rows;
}
// gz: agent within the launch; s: sample (conv1: unit within the agent)
struct UnitCoord { int gz, s; };
template <int V> __device__ __forceinline__ UnitCoord decode_unit(int u, int rows) {
    const int upg = units_per_group<V>(rows);
    UnitCoord c;
    c.gz = u / upg;
    c.s = u - c.gz * upg;
    return c;
}

// Lane j leaves with the sum over the warp's lanes of their v[j] (v is used up): five exchange steps, each
// halving the values a lane still holds; the order of the additions is fixed.
__device__ __forceinline__ float warp_reduce_scatter32(float (&v)[32], int lane) {
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const bool hi = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < s; i++) {
            const float send = hi ? v[i] : v[i + s];
            const float keep = hi ? v[i + s] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
        }
    }
    return v[0];
}

// BIAS (conv2 data gradient only): also leave the per-channel sums of the result behind, see ConvArgs::bias_partial.
template <int V, bool BIAS = false>
__global__ void __launch_bounds__(V == CV_CONV1_FWD ? kConv1Threads : kConvThreads, 1)
conv_resident_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const ConvArgs p,
                     const int nst, const long total_units) {
    using T = ConvTraits<V>;
    constexpr int STAGE = T::PLANES * T::PLANE_STRIDE;
    constexpr int W_BYTES = T::W_BOXES * T::W_BOX_BYTES;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kConvMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kConvMaxStages];
    __shared__ __align__(8) uint64_t acc_full[4];
    __shared__ __align__(8) uint64_t acc_empty[4];
    __shared__ __align__(8) uint64_t w_full, w_empty;
    __shared__ __align__(8) uint64_t w_conv;        // conv1: the weights in shared memory have been turned into fp16
    __shared__ __align__(8) uint64_t u8_full[kU8Stages];
    __shared__ __align__(8) uint64_t u8_empty[kU8Stages];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int issued_iters, issued_w;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* smW = smem;
    uint8_t* smX = smem + W_BYTES;
    uint8_t* smE = smX + nst * STAGE + (V == CV_CONV1_FWD ? 1024 : kConvSlack);
    uint8_t* smU = smE + 8 * kConvEpiWarpBytes;   // conv1 only: ring of uint8 line blocks
    uint8_t* smWraw = smU + kU8Stages * kU8Stride;   // conv1 only: the agent's weights as the tensor copies deliver them
    constexpr bool kU8 = V == CV_CONV1_FWD;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr uint32_t tmem_cols = 4u * T::BN;   // 128, 256 or 512: two accumulators per issuer

    // contiguous range of units of this CTA: at most a few agents, so few weight reloads
    const int u_begin = (int)(total_units * blockIdx.x / gridDim.x);
    const int u_end = (int)(total_units * (blockIdx.x + 1) / gridDim.x);

    if (threadIdx.x == 0) {
        // conv1: a stage is filled by one converting warp, otherwise by TMA (one arrival with a byte count)
        for (int s = 0; s < nst; s++) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int s = 0; s < kU8Stages; s++) { mbar_init(&u8_full[s], 1); mbar_init(&u8_empty[s], 1); }
        for (int b = 0; b < 4; b++) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
        mbar_init(&w_full, 1);
        mbar_init(&w_empty, 2);             // one commit per issuer
        mbar_init(&w_conv, 1);
        abort_flag = 0;
        issued_iters = 0;
        issued_w = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // The weights of the first agent are fetched before the wait for the previous kernel where they were written
    // at least two kernels back (by the optimiser pass or a state upload, with conv1's forward pass in between).
    // conv1's forward pass itself may be the very next kernel after a per-agent optimiser pass: it fetches them
    // after the wait.
    auto first_weights = [&]() {
        if (warp == 0 && u_begin < u_end) {
            __syncwarp();
            if (lane == 0) { mbar_expect_tx(&w_full, (uint32_t)W_BYTES); issued_w = 1; }
            __syncwarp();
            const int group = p.group0 + agent_slot(p.am, decode_unit<V>(u_begin, p.rows).gz);
            if (lane < T::W_BOXES) tma_load_3d((kU8 ? smWraw : smW) + lane * T::W_BOX_BYTES, &tmW, &w_full, weight_col<V>(lane), 0, group);
        }
    };
    if constexpr (V != CV_CONV1_FWD) first_weights();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                     "r"(tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = tmem_slot;
    pdl_wait();     // set-up above overlaps the previous kernel; its results are read from here on
    pdl_launch();
    if constexpr (V == CV_CONV1_FWD) first_weights();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        int it = 0, wl = 1;
        int cur_g = u_begin < u_end ? decode_unit<V>(u_begin, p.rows).gz : -1;   // already on its way
        for (int u = u_begin; u < u_end; u++, it++) {
            const UnitCoord c = decode_unit<V>(u, p.rows);
            const int group = p.group0 + agent_slot(p.am, c.gz);
            if (c.gz != cur_g) {
                // new agent: its weights replace the previous agent's once both issuers have signalled that
                // every MMA that read those is done
                int go = 1;
                if (lane == 0) go = mbar_wait(&w_empty, (uint32_t)(wl - 1) & 1u, &abort_flag) ? 1 : 0;
                go = __shfl_sync(0xffffffffu, go, 0);
                if (!go) break;
                if (lane == 0) mbar_expect_tx(&w_full, (uint32_t)W_BYTES);
                __syncwarp();
                if (lane < T::W_BOXES) tma_load_3d((kU8 ? smWraw : smW) + lane * T::W_BOX_BYTES, &tmW, &w_full, weight_col<V>(lane), 0, group);
                __syncwarp();
                cur_g = c.gz;
                wl++;
                if (lane == 0) issued_w = wl;
            }
            if constexpr (kU8) {
                // groups 6v .. 6v+6 of the agent's frames, as stored: one bulk copy (shorter at the very end)
                const int su = it % kU8Stages;
                int go = 1;
                if (lane == 0) go = mbar_wait(&u8_empty[su], ((uint32_t)(it / kU8Stages) & 1u) ^ 1u, &abort_flag) ? 1 : 0;
                go = __shfl_sync(0xffffffffu, go, 0);
                if (!go) break;
                if (lane == 0) {
                    const int left = 21 * p.rows - kC1Lines * c.s;   // groups from this unit's first to the last
                    const uint32_t bytes = left < kC1Lines + 1 ? (uint32_t)(left * kC1Group) : (uint32_t)kU8Bytes;
                    mbar_expect_tx(&u8_full[su], bytes);
                    const uint8_t* src = reinterpret_cast<const uint8_t*>(p.obs.p[c.gz]) + (long)c.s * (kC1Lines * kC1Group);
                    bulk_load_1d(smU + su * kU8Stride, src, bytes, &u8_full[su]);
                    issued_iters = it + 1;
                }
                continue;
            }
            const int s = it % nst;
            int go = 1;
            if (lane == 0) go = mbar_wait(&empty_bar[s], ((uint32_t)(it / nst) & 1u) ^ 1u, &abort_flag) ? 1 : 0;
            go = __shfl_sync(0xffffffffu, go, 0);
            if (!go) break;
            if (lane == 0) mbar_expect_tx(&full_bar[s], (uint32_t)(T::PLANES * T::PLANE_ROWS * T::ROWB));
            __syncwarp();
            const int sample = group * p.a_samples + c.s;
            if (lane < T::PLANES) {
                uint8_t* dst = smX + s * STAGE + lane * T::PLANE_STRIDE;
                if constexpr (V == CV_CONV2_FWD) tma_load_5d(dst, &tmX, &full_bar[s], 32 * (lane & 1), 0, lane >> 1, 0, sample);
                else if constexpr (V == CV_CONV3_FWD) tma_load_3d(dst, &tmX, &full_bar[s], 0, 0, sample);
                else if constexpr (V == CV_CONV2_DGRAD) tma_load_4d(dst, &tmX, &full_bar[s], 0, -1, -1, sample);
                else tma_load_4d(dst, &tmX, &full_bar[s], 0, -2, -2, sample);
            }
            __syncwarp();
            if (lane == 0) issued_iters = it + 1;
        }
    } else if (warp == 1 || warp == 10) {
        // ------------------------------------------------ MMA issuers: warp 1 takes the even units, warp 10 the odd
        // A barrier tells its phases apart by one bit, so whoever waits on it must see every phase, in order: a wait
        // for a phase that is two ahead of the barrier passes at once, one for a phase two behind never ends.  With
        // two issuers a stage must therefore always come back to the same issuer: the ring has an even number of
        // stages (conv1's has one per converting warp, and an even number of those).
        if (lane == 0) {
            const int ii = warp == 1 ? 0 : 1;
            const uint32_t idesc = make_instr_desc(T::BN, 0, T::B_MN, kU8);   // conv1: fp16 operands
            const uint64_t bd_base = make_smem_desc_raw(smem_u32(smW), T::B_LAYOUT, T::B_SBO, T::B_LBO);
            int it = 0, cur_g = -1, wl = 0;
            const int upg = units_per_group<V>(p.rows);
            int gz = u_begin / upg, g_end = (gz + 1) * upg;     // the agent of unit u and where its units end
            int s = -1;                                         // stage of unit u and the parity of its use
            uint32_t s_par = 0u;
            for (int u = u_begin; u < u_end; u++, it++) {
                if (++s == nst) { s = 0; s_par ^= 1u; }
                // Both issuers follow every change of agent: each reports (through a commit, so only once its
                // MMAs are complete) that it is done with the old weights, then waits for the new ones.
                if (u >= g_end) { gz++; g_end += upg; }
                if (gz != cur_g) {
                    if (cur_g >= 0) umma_commit(&w_empty);
                    if (!mbar_wait(kU8 ? &w_conv : &w_full, (uint32_t)wl & 1u, &abort_flag)) break;
                    wl++;
                    cur_g = gz;
                }
                if ((it & 1) != ii) continue;
                const int k = it >> 1;                  // this issuer's k-th unit goes to its buffer k % 2
                const int ab = ii * 2 + (k & 1);
                if (!mbar_wait(&acc_empty[ab], (((uint32_t)k >> 1) & 1u) ^ 1u, &abort_flag)) break;
                if (!mbar_wait(&full_bar[s], s_par, &abort_flag)) break;
                tcgen05_fence_after();
                const uint32_t tmem_acc = tmem_base + (uint32_t)ab * T::BN;
                const uint32_t x_addr = smem_u32(smX + s * STAGE);
                // One thread issues every MMA, so the loop is unrolled completely: the tap's plane, row shift
                // and weight slot fold into constants that are added to the address field of two base
                // descriptors (16-byte units; the ring and the weights lie below 256 KiB, so no carry leaves it).
                const uint64_t ad_base = make_smem_desc_raw(x_addr, T::LAYOUT, 8 * T::ROWB, 16);
#pragma unroll
                for (int t = 0; t < T::TAPS; t++) {
                    int plane, shift;
                    tap_view<V>(t, plane, shift);
                    const uint32_t a_off = plane * T::PLANE_STRIDE + shift * T::ROWB;
                    const uint32_t b_off = (V == CV_CONV2_DGRAD ? t * 4 : V == CV_CONV1_FWD ? t * 4 : t) * T::W_BOX_BYTES;
#pragma unroll
                    for (int kk = 0; kk < T::KKN; kk++) {
                        // K = 16 further on: 32 B along a K-major row, 16 rows of an MN-major tile
                        const uint32_t bk = T::B_MN ? kk * 16 * (T::B_LAYOUT == 4 ? 64 : 128) : kk * 32;
                        umma_bf16(tmem_acc, ad_base + (uint64_t)((a_off + kk * 32) >> 4), bd_base + (uint64_t)((b_off + bk) >> 4),
                                  idesc, (t | kk) != 0 ? 1u : 0u);
                    }
                }
                umma_commit(&empty_bar[s]);     // the stage may be refilled ...
                umma_commit(&acc_full[ab]);     // ... and the accumulator read, once the MMAs above are done
            }
        }
    } else if (warp >= 11) {
        // ------------------------------------------------ conv1: uint8 lines -> fp16 phase planes
        // Line yl of the block (28 lines = 7 groups of 4) is K slice yl % 4 of row (yl / 4) * 21 + xq for its 16-byte
        // group xq (4 pixels x 4 channels): 32 bytes of fp16 as two 16-byte pieces, piece c of a row at
        // 16 (c ^ (row & 7)) (128-byte swizzle).  0..255 are exact in fp16; 1/255 is applied after the MMAs.
        // The same warps turn an agent's weights, which arrive as bf16, into fp16(w * 2^12) where they lie.
        // Converter warp cw takes the units cw, cw + 4, ... of the CTA's range, a whole unit each: the fixed cost of a
        // hand-over (two waits, the proxy fence, two arrivals: some 500 cycles) is then paid by one warp per unit
        // while the others are busy with other units.  A warp owns one stage and two slots of the byte ring, so every
        // barrier it waits on is its own and it sees each of their phases in turn.  Converter warp 0 also lays out every agent's weights when it
        // comes to the agent's first unit (always the same warp, so that it waits for the weight copies in their
        // order: a wait for a later copy's phase would pass at once while an earlier one is still pending).
        if constexpr (kU8) {
            const int cw = warp - 11;
            constexpr int kChunks = 4 * (kC1Lines + 1) * 21;   // 16-byte groups of a block, 588
            // where a lane's k-th group goes inside a stage (the same for every unit): row, K slice, swizzle
            int dst_off[(kChunks + 31) / 32];
#pragma unroll
            for (int k = 0; k < (kChunks + 31) / 32; k++) {
                const int ch = lane + 32 * k;
                const int yl = ch / 21, xq = ch - yl * 21;
                const int r = (yl >> 2) * 21 + xq;
                dst_off[k] = r * 128 + ((((yl & 3) * 2) ^ (r & 7)) << 4);
            }
            const int upg = units_per_group<V>(p.rows);
            int prev_g = -1, wl = 0, it = 0;
            bool ok = true;
            int gz = u_begin / upg, g_end = (gz + 1) * upg;
            for (int u = u_begin; ok && u < u_end; u++, it++) {
                if (u >= g_end) { gz++; g_end += upg; }
                const bool mine = it % kC1ConvWarps == cw;
                if (gz != prev_g) {
                    if (cw == 0) {
                        // (the MMAs that read the previous agent's laid-out weights are complete: the producer waited
                        // for both issuers' commits before it asked for these)
                        if (!mbar_wait(&w_full, (uint32_t)wl & 1u, &abort_flag)) break;
                        for (int ch = lane; ch < W_BYTES / 16; ch += 32) {
                            // 16-byte piece hh of row co of box j = 2 ky + b  ->  tile 2 (ky / 4) + b, row co, K slice ky % 4
                            const int j = ch >> 6, co = (ch >> 1) & 31, hh = ch & 1;
                            const int ky = j >> 1, nrow = (j & 1) * 32 + co;
                            uint4 v = *reinterpret_cast<const uint4*>(smWraw + ch * 16);
                            uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                            for (int e = 0; e < 4; e++) {
                                float lo = __uint_as_float(w4[e] << 16) * kC1WeightScale;
                                float hi = __uint_as_float(w4[e] & 0xffff0000u) * kC1WeightScale;
                                lo = fminf(fmaxf(lo, -65504.0f), 65504.0f);
                                hi = fminf(fmaxf(hi, -65504.0f), 65504.0f);
                                const __half2 h = __floats2half2_rn(lo, hi);
                                w4[e] = *reinterpret_cast<const uint32_t*>(&h);
                            }
                            *reinterpret_cast<uint4*>(smW + (ky >> 2) * 8192 + nrow * 128 + ((((ky & 3) * 2 + hh) ^ (nrow & 7)) << 4)) =
                                make_uint4(w4[0], w4[1], w4[2], w4[3]);
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&w_conv);
                    }
                    wl++;
                    prev_g = gz;
                }
                if (!mine) continue;
                const int su = it % kU8Stages, s = it % nst;
                if (!mbar_wait(&u8_full[su], (uint32_t)(it / kU8Stages) & 1u, &abort_flag)) break;
                if (!mbar_wait(&empty_bar[s], ((uint32_t)(it / nst) & 1u) ^ 1u, &abort_flag)) break;
                const uint8_t* src = smU + su * kU8Stride;
                uint8_t* dstage = smX + s * STAGE;
                // Line yl of the block (28 lines = 7 groups of 4) is K slice yl % 4 of row (yl / 4) * 21 + xq for its
                // 16-byte group xq (4 pixels x 4 channels): 32 bytes of fp16 as two 16-byte pieces, piece c of a row at
                // 16 (c ^ (row & 7)) (128-byte swizzle).  0..255 are exact in fp16; 1/255 is applied after the MMAs.
                // Five 16-byte groups a lane are fetched before any of them is widened and stored: the compiler cannot
                // know that the byte ring and the stage do not overlap, so loads written after a store wait for it.
                constexpr int kPer = (kChunks + 31) / 32;   // groups a lane, 19
#pragma unroll
                for (int k0 = 0; k0 < kPer; k0 += 5) {
                    uint4 v[5];
#pragma unroll
                    for (int k = 0; k < 5; k++) {
                        const int ch = lane + 32 * (k0 + k);
                        if (k0 + k < kPer && ch < kChunks) v[k] = *reinterpret_cast<const uint4*>(src + ch * 16);
                    }
#pragma unroll
                    for (int k = 0; k < 5; k++) {
                        const int ch = lane + 32 * (k0 + k);
                        if (k0 + k < kPer && ch < kChunks) {
                            const uint32_t w[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
                            uint32_t o[8];
#pragma unroll
                            for (int e = 0; e < 4; e++) {
                                o[2 * e] = u8x2_to_f16x2(w[e], 0);
                                o[2 * e + 1] = u8x2_to_f16x2(w[e], 2);
                            }
                            uint8_t* d0 = dstage + dst_off[k0 + k];
                            *reinterpret_cast<uint4*>(d0) = make_uint4(o[0], o[1], o[2], o[3]);
                            *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(reinterpret_cast<uintptr_t>(d0) ^ 16)) =
                                make_uint4(o[4], o[5], o[6], o[7]);
                        }
                    }
                }
                // make the generic-proxy writes visible to the tensor core's reads, then hand the stage over
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) { mbar_arrive(&full_bar[s]); mbar_arrive(&u8_empty[su]); }
            }
        }
    } else {
        // ------------------------------------------------ epilogue: group eg drains the accumulators of issuer eg
        // A thread owns one row of the tile (one pixel): per 32-column block it reads its 32 accumulators
        // from tensor memory, applies scale / bias / ReLU or the ReLU gate, and stores 64 contiguous bytes.
        // The gate values depend only on the unit, so they are fetched before the wait for the MMAs.
        const int eg = (warp - 2) >> 2;
        const int q = warp & 3;                    // lane quarter of tensor memory this warp may read
        constexpr int kLastRow = (T::OH - 1) * T::PITCH + T::OW - 1;   // last row of a tile that is a real pixel
        constexpr bool kFwd = V == CV_CONV1_FWD || V == CV_CONV2_FWD || V == CV_CONV3_FWD;
        constexpr int NCH = T::BN / 32;
        float* sbias = reinterpret_cast<float*>(smE + (warp - 2) * kConvEpiWarpBytes);   // this warp's copy of the bias
        const int m = q * 32 + lane;
        const int pa = m / T::PITCH, pb = m - pa * T::PITCH;
        const bool in_tile = pa < T::OH && pb < T::OW;
        // element offset of this thread's pixel inside the agent's tensor (pixel (2a, 2b) for the conv2 gradient)
        auto pixel_off = [&](const UnitCoord& c) -> long {
            if constexpr (V == CV_CONV1_FWD) {   // line L of the run = line L % 21 of frame L / 21
                const int L = kC1Lines * c.s + pa, f = L / 21;
                return ((long)f * 400 + (L - f * 21) * 20 + pb) * 32;
            }
            else if constexpr (V == CV_CONV2_FWD) return ((long)c.s * 81 + pa * 9 + pb) * 64;
            else if constexpr (V == CV_CONV3_FWD) return ((long)c.s * 49 + pa * 7 + pb) * 64;
            else if constexpr (V == CV_CONV2_DGRAD) return ((long)c.s * 400 + (2 * pa) * 20 + 2 * pb) * 32;
            else return ((long)c.s * 81 + pa * 9 + pb) * 64;
        };
        // ReLU gates of the layer input, one bit per channel (bit set: the activation was positive), written
        // by the forward pass of the layer below.  They depend only on the unit, so the words of the NEXT
        // tile of this group are fetched before the current one is processed.
        uint32_t gate[kFwd ? 1 : NCH];
        auto load_gates = [&](int u, uint32_t* g) {
            if constexpr (!kFwd) {
#pragma unroll
                for (int ch = 0; ch < NCH; ch++) g[ch] = 0u;
                if (u < u_end && in_tile) {
                    const UnitCoord c = decode_unit<V>(u, p.rows);
                    const uint32_t* gp = p.gate_in + (long)agent_slot(p.am, c.gz) * p.gate_group_stride + pixel_off(c) / 32;
                    if constexpr (V == CV_CONV2_DGRAD) {   // words of pixels (2a, 2b), (2a, 2b+1), (2a+1, 2b), (2a+1, 2b+1)
                        const uint2 g0 = __ldg(reinterpret_cast<const uint2*>(gp));
                        const uint2 g1 = __ldg(reinterpret_cast<const uint2*>(gp + 20));
                        g[0] = g0.x; g[1] = g0.y; g[2] = g1.x; g[3] = g1.y;
                    } else {                               // the two words (64 channels) of pixel (a, b)
                        const uint2 g0 = __ldg(reinterpret_cast<const uint2*>(gp));
                        g[0] = g0.x; g[1] = g0.y;
                    }
                }
            }
        };
        load_gates(u_begin + eg, gate);
        int cur_g = -1;
        int it = eg;
        // conv2 data gradient: the sum over pixels of what is stored (= the bias gradient of conv1) is kept per
        // thread while the CTA stays with an agent and leaves as one slice per agent, CTA and epilogue warp.  A
        // warp writes a slice for EVERY agent in the CTA's range of units, also where its group had no unit.
        static_assert(!BIAS || V == CV_CONV2_DGRAD, "bias slices come from conv2's data gradient only");
        constexpr bool kBias = BIAS;
        float bacc[kBias ? 32 : 1];
#pragma unroll
        for (int j = 0; j < (kBias ? 32 : 1); j++) bacc[j] = 0.0f;
        const bool bias_on = kBias && u_begin < u_end;
        int bg = bias_on ? decode_unit<V>(u_begin, p.rows).gz : 0;     // agent that bacc belongs to
        auto bias_flush = [&](int upto) {      // slices of agents bg .. upto - 1; bacc restarts at zero
            if constexpr (kBias) {
                for (; bg < upto; bg++) {
                    const float sum = warp_reduce_scatter32(bacc, lane);
                    p.bias_partial[(((long)agent_slot(p.am, bg) * kConvMaxGrid + blockIdx.x) * 8 + (warp - 2)) * 32 + lane] = sum;
#pragma unroll
                    for (int j = 0; j < 32; j++) bacc[j] = 0.0f;
                }
            }
        };
        for (int u = u_begin + eg; u < u_end; u += 2, it += 2) {
            const UnitCoord c = decode_unit<V>(u, p.rows);
            const long off = pixel_off(c);
            bool valid = in_tile;
            if constexpr (V == CV_CONV1_FWD) {   // not the line between two frames, not past the last frame
                const int L = kC1Lines * c.s + pa;
                valid = in_tile && L % 21 < 20 && L < 21 * p.rows;
            }
            const int slot_ag = agent_slot(p.am, c.gz);
            __nv_bfloat16* out = p.out + (long)slot_ag * p.out_group_stride + off;
            // column block c0 -> where it goes: forward, conv3 gradient: channels c0.. of the pixel; conv2
            // gradient: block = parity class (py, px) -> pixel (2a + py, 2b + px), all 32 channels
            auto block_add = [](int c0) -> int {
                if constexpr (V == CV_CONV2_DGRAD) return ((c0 >> 6) * 20 + ((c0 >> 5) & 1)) * 32;
                else return c0;
            };
            uint32_t gate_next[kFwd ? 1 : NCH];
            if (bias_on && c.gz != bg) bias_flush(c.gz);
            if constexpr (kFwd) {
                if (c.gz != cur_g) {
                    const float* bias = p.bias + (long)(p.group0 + slot_ag) * p.bias_group_stride;
                    __syncwarp();
                    for (int j = lane; j < T::BN; j += 32) sbias[j] = __ldg(bias + j);
                    __syncwarp();
                    cur_g = c.gz;
                }
            } else {
                load_gates(u + 2, gate_next);
            }
            const int ab = eg * 2 + ((it >> 1) & 1);
            if (!mbar_wait(&acc_full[ab], ((uint32_t)it >> 2) & 1u, &abort_flag)) break;
            tcgen05_fence_after();
            if (q * 32 <= kLastRow) {
                const uint32_t tmem_acc = tmem_base + (uint32_t)ab * T::BN + ((uint32_t)(q * 32) << 16);
                // 16 columns (one 32-byte store) at a time, the load of the next 16 in flight meanwhile
                constexpr int NSUB = 2 * NCH;
                uint32_t rr[2][16];
                tmem_ld16_issue(tmem_acc, rr[0]);
                uint32_t bits = 0u;
#pragma unroll
                for (int sb = 0; sb < NSUB; sb++) {
                    const int ch = sb >> 1, h = sb & 1;        // 32-column block, half of it
                    uint32_t (&r)[16] = rr[sb & 1];
                    tmem_ld16_wait(r);
                    if (sb + 1 < NSUB) tmem_ld16_issue(tmem_acc + (uint32_t)((sb + 1) * 16), rr[(sb + 1) & 1]);
                    uint32_t o[8];
#pragma unroll
                    for (int j = 0; j < 8; j++) {
                        float v0 = __uint_as_float(r[2 * j]), v1 = __uint_as_float(r[2 * j + 1]);
                        if constexpr (kFwd) {
                            const float2 bv = *reinterpret_cast<const float2*>(sbias + sb * 16 + 2 * j);
                            v0 = fmaxf(fmaf(v0, p.scale, bv.x), 0.0f);
                            v1 = fmaxf(fmaf(v1, p.scale, bv.y), 0.0f);
                        } else {
                            if (!((gate[ch] >> (16 * h + 2 * j)) & 1u)) v0 = 0.0f;
                            if (!((gate[ch] >> (16 * h + 2 * j + 1)) & 1u)) v1 = 0.0f;
                        }
                        o[j] = pack2(v0, v1);
                        if constexpr (kBias) {
                            if (valid) { bacc[16 * h + 2 * j] += v0; bacc[16 * h + 2 * j + 1] += v1; }
                        }
                        if constexpr (kFwd) {   // gate of the stored (rounded) activation
                            if (o[j] & 0x00007fffu) bits |= 1u << (16 * h + 2 * j);
                            if (o[j] & 0x7fff0000u) bits |= 1u << (16 * h + 2 * j + 1);
                        }
                    }
                    if (valid) {   // a 32-byte store fills a whole sector
                        st_global_v8(out + block_add(ch * 32) + 16 * h, o);
                        if constexpr (kFwd) {
                            if (h == 1 && p.gate_out) p.gate_out[(long)slot_ag * p.gate_group_stride + off / 32 + ch] = bits;
                        }
                    }
                    if (h == 1) bits = 0u;
                }
            }
            if constexpr (!kFwd) {
#pragma unroll
                for (int ch = 0; ch < NCH; ch++) gate[ch] = gate_next[ch];
            }
            // this warp no longer reads the accumulator buffer
            tcgen05_fence_before();
            if (lane == 0) mbar_arrive(&acc_empty[ab]);
        }
        if (bias_on) bias_flush(decode_unit<V>(u_end - 1, p.rows).gz + 1);
    }

    // teardown
    tcgen05_fence_before();
    __syncthreads();
    if (abort_flag) {
        if (threadIdx.x == 0) {
            if (p.error_word) atomicExch(p.error_word, 10 + V);   // which kernel gave up
            // let copies that were already issued land before the shared memory goes away
            const int issued = issued_iters;
            const int ring = kU8 ? kU8Stages : nst;
            for (int it = max(0, issued - ring); it < issued; it++) {
                const int s = it % ring;
                const uint32_t ph = (uint32_t)(it / ring) & 1u;
                for (uint32_t i = 0; i < (1u << 16); i++) {
                    if (mbar_try_wait(kU8 ? &u8_full[s] : &full_bar[s], ph)) break;
                    __nanosleep(64);
                }
            }
            if (issued_w > 0)
                for (uint32_t i = 0; i < (1u << 16); i++) {
                    if (mbar_try_wait(&w_full, (uint32_t)(issued_w - 1) & 1u)) break;
                    __nanosleep(64);
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
template <int V> static cudaError_t conv_attr() {
    return cudaFuncSetAttribute(conv_resident_kernel<V>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                V == CV_CONV1_FWD ? kConv1SmemMax : kConvSmemMax);
}
cudaError_t conv_init() {
    static bool done = false;
    if (done) return cudaSuccess;
    cudaError_t e;
    if ((e = conv_attr<CV_CONV1_FWD>()) != cudaSuccess) return e;
    if ((e = conv_attr<CV_CONV2_FWD>()) != cudaSuccess) return e;
    if ((e = conv_attr<CV_CONV3_FWD>()) != cudaSuccess) return e;
    if ((e = conv_attr<CV_CONV2_DGRAD>()) != cudaSuccess) return e;
    if ((e = conv_attr<CV_CONV3_DGRAD>()) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(conv_resident_kernel<CV_CONV2_DGRAD, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  kConvSmemMax)) != cudaSuccess) return e;
    done = true;
    return cudaSuccess;
}

bool make_conv_maps(int variant, CUtensorMap* x_map, CUtensorMap* w_map, const void* x_base, uint64_t samples,
                    const void* w_base, uint64_t groups, uint64_t w_group_stride_elems) {
    bool ok = true;
    switch (variant) {
    case CV_CONV1_FWD: {   // bf16 frames [sample][84][84][4] as [sample][y/4][y%4][x/4][4 px x 4 ch]
        const uint64_t dims[5] = {16, 21, 4, 21, samples}, str[4] = {32, 672, 2688, 56448};
        const uint32_t box[5] = {16, 21, 1, 6, 1};
        ok &= make_tensor_map_nd(x_map, x_base, 5, dims, str, box, 2);
        const uint64_t wd[3] = {256, 32, groups}, ws[2] = {512, w_group_stride_elems * 2};
        const uint32_t wb[3] = {16, 32, 1};
        ok &= make_tensor_map_nd(w_map, w_base, 3, wd, ws, wb, 3);   // unswizzled: the kernel lays them out itself
        break;
    }
    case CV_CONV2_FWD: {   // act1 [sample][20][20][32] as [sample][y/2][y%2][x/2][2 px x 32 ch]
        const uint64_t dims[5] = {64, 10, 2, 10, samples}, str[4] = {128, 1280, 2560, 25600};
        const uint32_t box[5] = {32, 10, 1, 10, 1};
        ok &= make_tensor_map_nd(x_map, x_base, 5, dims, str, box, 1);
        break;
    }
    case CV_CONV3_FWD: {   // act2 [sample][81 pixels][64]
        const uint64_t dims[3] = {64, 81, samples}, str[2] = {128, 10368};
        const uint32_t box[3] = {64, 81, 1};
        ok &= make_tensor_map_nd(x_map, x_base, 3, dims, str, box, 0);
        break;
    }
    case CV_CONV2_DGRAD: { // dY2 [sample][9][9][64], boxes reach one pixel past every edge
        const uint64_t dims[4] = {64, 9, 9, samples}, str[3] = {128, 1152, 10368};
        const uint32_t box[4] = {64, 11, 11, 1};
        ok &= make_tensor_map_nd(x_map, x_base, 4, dims, str, box, 0);
        break;
    }
    case CV_CONV3_DGRAD: { // dY3 [sample][7][7][64], boxes reach two pixels past every edge
        const uint64_t dims[4] = {64, 7, 7, samples}, str[3] = {128, 896, 6272};
        const uint32_t box[4] = {64, 11, 11, 1};
        ok &= make_tensor_map_nd(x_map, x_base, 4, dims, str, box, 0);
        break;
    }
    default: return false;
    }
    if (variant == CV_CONV2_FWD || variant == CV_CONV2_DGRAD) {   // W2[64][512]: 32-column blocks
        const uint64_t wd[3] = {512, 64, groups}, ws[2] = {1024, w_group_stride_elems * 2};
        const uint32_t wb[3] = {32, 64, 1};
        ok &= make_tensor_map_nd(w_map, w_base, 3, wd, ws, wb, 1);
    } else if (variant == CV_CONV3_FWD || variant == CV_CONV3_DGRAD) {   // W3[64][576]: 64-column blocks
        const uint64_t wd[3] = {576, 64, groups}, ws[2] = {1152, w_group_stride_elems * 2};
        const uint32_t wb[3] = {64, 64, 1};
        ok &= make_tensor_map_nd(w_map, w_base, 3, wd, ws, wb, 0);
    }
    return ok;
}

int conv_grid(long units, int max_ctas) {
    const int most = sm_count() < kConvMaxGrid ? sm_count() : kConvMaxGrid;
    int grid = (int)(units < most ? units : most);
    if (max_ctas > 0 && grid > max_ctas) grid = max_ctas;
    return grid;
}

template <int V>
static cudaError_t launch_conv_v(const CUtensorMap& x, const CUtensorMap& w, const ConvArgs& a, cudaStream_t st) {
    using T = ConvTraits<V>;
    constexpr int STAGE = T::PLANES * T::PLANE_STRIDE;
    // conv1's MMAs read at most two rows past a stage (shift 21 + 128 rows against 147): 1 KB of slack is plenty
    constexpr int slack = V == CV_CONV1_FWD ? 1024 : kConvSlack;
    constexpr int smem_max = V == CV_CONV1_FWD ? kConv1SmemMax : kConvSmemMax;
    constexpr int fixed = T::W_BOXES * T::W_BOX_BYTES + slack + 8 * kConvEpiWarpBytes + 1024 +
                          (V == CV_CONV1_FWD ? kU8Stages * kU8Stride + T::W_BOXES * T::W_BOX_BYTES : 0);
    int nst = (smem_max - fixed) / STAGE;
    if (nst > kConvMaxStages) nst = kConvMaxStages;
    if constexpr (V == CV_CONV1_FWD) {   // one stage per converter warp (see kC1ConvWarps)
        if (nst < kC1ConvWarps) return cudaErrorInvalidValue;
        nst = kC1ConvWarps;
    }
    else if (nst > 2) nst &= ~1;   // two issuers: a stage always returns to the same one (see the kernel)
    if (nst < 2) return cudaErrorInvalidValue;
    const long units = (long)a.groups * units_per_group<V>(a.rows);
    if (units <= 0) return cudaSuccess;
    if (units > 0x7fffffffL) return cudaErrorInvalidValue;
    const size_t smem = (size_t)fixed + (size_t)nst * STAGE;
    const int grid = conv_grid(units, a.max_ctas);
    const dim3 block(V == CV_CONV1_FWD ? kConv1Threads : kConvThreads);
    if constexpr (V == CV_CONV2_DGRAD) {
        if (a.bias_partial) {
            (void)launch_pdl(conv_resident_kernel<V, true>, dim3(grid), block, smem, st, x, w, a, nst, units);
            return cudaGetLastError();
        }
    }
    (void)launch_pdl(conv_resident_kernel<V>, dim3(grid), block, smem, st, x, w, a, nst, units);
    return cudaGetLastError();
}

cudaError_t launch_conv(const CUtensorMap& x, const CUtensorMap& w, const ConvArgs& a, cudaStream_t st) {
    if (a.groups < 1 || a.rows < 0 || !a.out) return cudaErrorInvalidValue;
    const bool fwd = a.variant == CV_CONV1_FWD || a.variant == CV_CONV2_FWD || a.variant == CV_CONV3_FWD;
    if (fwd ? !a.bias : !a.gate_in) return cudaErrorInvalidValue;
    switch (a.variant) {
    case CV_CONV1_FWD: return launch_conv_v<CV_CONV1_FWD>(x, w, a, st);
    case CV_CONV2_FWD: return launch_conv_v<CV_CONV2_FWD>(x, w, a, st);
    case CV_CONV3_FWD: return launch_conv_v<CV_CONV3_FWD>(x, w, a, st);
    case CV_CONV2_DGRAD: return launch_conv_v<CV_CONV2_DGRAD>(x, w, a, st);
    case CV_CONV3_DGRAD: return launch_conv_v<CV_CONV3_DGRAD>(x, w, a, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace gala
