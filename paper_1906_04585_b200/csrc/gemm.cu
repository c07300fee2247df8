// Grouped bf16 GEMM on the 5th-generation tensor cores (tcgen05) for sm_100a.
//
//   D[g] (M x N, fp32 accumulate) = A[g] (M x K) * B[g] (N x K)^T       g = group (agent)
//
// Either operand may be stored K-contiguous ("K-major": [rows][K]) or M/N-contiguous
// ("MN-major": [K][rows]); the four combinations cover forward (both K-major), data-gradient
// (B MN-major) and weight-gradient (both MN-major) products of the conv / dense layers without
// any transposed copy in global memory.
//
// Structure of one CTA (192 threads, persistent: it loops over 128 x block_n output tiles):
//   warp 0   : TMA producer - cp.async.bulk.tensor (3-D maps: inner, rows, group) into a ring of
//              128-byte-swizzled shared-memory stages that runs on across tiles
//   warp 1   : allocates tensor memory (two accumulator buffers), issues tcgen05.mma (one elected
//              thread), releases stages and publishes finished accumulators with tcgen05.commit
//   warps 2-5: epilogue - tcgen05.ld the fp32 accumulator of the previous tile out of tensor memory
//              (each warp its own 32-lane quarter) while the next tile is being multiplied, re-tile
//              it through shared memory so that global stores coalesce, apply scale / bias / ReLU /
//              mask, store
// Every mbarrier wait is bounded: when a wait runs out the CTA raises an abort flag, sets the
// caller's error word, drains what it has in flight, frees its tensor memory and returns.
#include "internal.h"
#include "tcgen05.cuh"

namespace gala {

constexpr int BM = 128;          // tile rows (UMMA M)
constexpr int BK = 64;           // K per stage = one 128-byte swizzle atom of bf16
constexpr int kStages = 4;
constexpr int kStageA = BM * BK * 2;    // 16 KiB
constexpr int kStageB = 128 * BK * 2;   // room for block_n = 128
constexpr int kSmemBytes = 216 * 1024;   // most dynamic shared memory a launch may ask for (four stages of a 128 x 256 tile)

// ------------------------------------------------------------------ kernel
// Work decomposition shared by the three roles: tile index -> (group, split, m-tile, n-tile), n fastest
// so that CTAs running side by side share an A tile in L2.
struct TileCoord { int gz, split, m0, n0, kt_begin, num_k; };
__device__ __forceinline__ TileCoord decode_tile(const GemmArgs& p, long tile, int mt, int nt) {
    TileCoord t;
    const int n_t = (int)(tile % nt);
    const long r = tile / nt;
    const int m_t = (int)(r % mt);
    const int z = (int)(r / mt);
    t.gz = z / p.split_k; t.split = z % p.split_k;
    t.m0 = m_t * p.tile_rows; t.n0 = n_t * p.block_n;
    const int k_tiles = p.k_steps;
    const int per_split = (k_tiles + p.split_k - 1) / p.split_k;
    t.kt_begin = t.split * per_split;
    const int kt_end = min(k_tiles, t.kt_begin + per_split);
    t.num_k = max(0, kt_end - t.kt_begin);
    return t;
}

constexpr int kEpiRowBytes = 32 * 4 + 16;          // 32 fp32 columns of one row + 16 B against bank conflicts
constexpr int kEpiWarpBytes = 32 * kEpiRowBytes;   // staging area of one epilogue warp

// Persistent CTA: loops over output tiles.  The shared-memory ring runs on across tiles, and the
// accumulator is double-buffered in tensor memory, so the loads and MMAs of tile i+1 overlap the
// epilogue of tile i.
__global__ void __launch_bounds__(192, 2)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const GemmArgs p, const int a_mn, const int b_mn, const long total_tiles, const int mt,
                    const int nt) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t full_bar[kStages];
    __shared__ __align__(8) uint64_t empty_bar[kStages];
    __shared__ __align__(8) uint64_t acc_full[2];
    __shared__ __align__(8) uint64_t acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_flag;
    __shared__ int issued_iters;

    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int nst = p.stages;
    const int BN = p.block_n;
    const int stage_a = p.stage_a_bytes, stage_b = p.stage_b_bytes;
    uint8_t* smA = smem;
    uint8_t* smB = smem + nst * stage_a;
    uint8_t* smE = smB + nst * stage_b;   // epilogue staging, 4 x kEpiWarpBytes
    const int conv = p.conv_mode;
    // geometry of the implicit convolutions: patches per sample and 64-element blocks per patch
    const int cQ = p.conv_layer == 1 ? 8 : 9;
    const int sw64 = conv && p.conv_layer == 0;   // conv1: 64-byte rows

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t acc_cols = BN < 32 ? 32u : (uint32_t)BN;
    const uint32_t tmem_cols = 2u * acc_cols;   // 64, 128 or 256: a power of two

    if (threadIdx.x == 0) {
        for (int s = 0; s < nst; s++) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; b++) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
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
    if (conv) {
        // The boxes of the convolution modes fill only part of a stage (98 of 128 rows, 81 of 96, ...).
        // The rest must read as zero wherever it takes part in a reduction, so the ring starts zeroed;
        // TMA never writes those rows afterwards.
        uint4* z = reinterpret_cast<uint4*>(smem);
        const int n16 = nst * (stage_a + stage_b) / 16;
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
        // The whole warp walks the K steps.  Lane 0 waits for the stage and posts the byte count; the
        // (up to four) tensor copies of a K step are then issued by lanes 0..3 side by side, because one
        // thread needs some 200 ns per copy instruction.
        const uint32_t bytes = (uint32_t)kStageA + (uint32_t)(BN * BK * 2);
        const uint32_t box_bytes = (uint32_t)(p.box_rows * (sw64 ? 64 : 128));   // one [patches or pixels][channels] box
        int it = 0;
        bool ok = true;
        for (long tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
            const TileCoord t = decode_tile(p, tile, mt, nt);
            const int group = p.group0 + agent_slot(p.am, t.gz);
            for (int k = 0; k < t.num_k; k++, it++) {
                const int s = it % nst;
                const uint32_t ph = (uint32_t)(it / nst) & 1u;
                int go = 1;
                if (lane == 0) go = mbar_wait(&empty_bar[s], ph ^ 1u, &abort_flag) ? 1 : 0;
                go = __shfl_sync(0xffffffffu, go, 0);
                if (!go) { ok = false; break; }
                const int k0 = (t.kt_begin + k) * BK;
                uint8_t* a = smA + s * stage_a;
                uint8_t* b = smB + s * stage_b;
                if (conv) {
                    // kernel offset of 64-element block q of a patch, and the TMA coordinates of the
                    // [patch][channel] box that holds it for samples s0, s0+1, ...
                    auto load_block = [&](uint8_t* dst, int q, int s0) {
                        if (p.conv_layer == 0) {
                            // conv1: frames seen as [sample][y/4][y%4][ox][8 px x 4 ch] with windows that overlap
                            // by half (ox advances 4 px); q = kernel row ky, s0 = sample*4 + quarter of the sample
                            // (5 of the 20 output rows, 100 patches)
                            tma_load_5d(dst, &tmA, &full_bar[s], 0, 0, q & 3, (q >> 2) + 5 * (s0 & 3),
                                        group * p.a_samples + (s0 >> 2));
                        } else if (p.conv_layer == 1) {   // conv2: input seen as [sample][y/2][y%2][x/2][64]
                            const int ky = q >> 1, h = q & 1;
                            tma_load_5d(dst, &tmA, &full_bar[s], 0, h, ky & 1, ky >> 1, group * p.a_samples + s0);
                        } else {                   // conv3: input [sample][y][x][64]
                            const int ky = q / 3, kx = q - ky * 3;
                            tma_load_4d(dst, &tmA, &full_bar[s], 0, kx, ky, group * p.a_samples + s0);
                        }
                    };
                    if (conv == CONV_DGRAD || conv == CONV_FWD) {
                        // A K step covers up to kpack kernel offsets ("blocks").  Block j of the step gets an A
                        // box at a + j * a_sub and a B box at b + j * b_sub; lanes 0..nq-1 fetch the A boxes,
                        // lanes nq..2nq-1 the B boxes.  a_sub is the box size rounded up to 1 KiB, not a full
                        // 128-row image: the rows an MMA reads past the box only feed output rows that the
                        // epilogue drops.
                        const int kelems = sw64 ? 32 : BK;   // K elements per block
                        const int kp = p.kpack;
                        const uint32_t a_sub = (uint32_t)p.a_sub_bytes, b_sub = (uint32_t)(BN * kelems * 2);
                        const int q0 = (t.kt_begin + k) * kp;
                        const int nq = min(kp, p.conv_q - q0);
                        if (lane == 0) mbar_expect_tx(&full_bar[s], (uint32_t)nq * (box_bytes + b_sub));
                        __syncwarp();
                        const int j = lane < nq ? lane : lane - nq;
                        const int q = q0 + j;
                        if (lane < 2 * nq) {
                            if (conv == CONV_FWD) {
                                if (lane < nq) load_block(a + j * a_sub, q, (t.m0 / p.tile_rows) * p.conv_nb);
                                else tma_load_3d(b + j * b_sub, &tmB, &full_bar[s], q * kelems, t.n0, group);
                            } else {
                                // data gradient: block = kernel offset; the dY box is shifted by it, the weights'
                                // [co][ci] block of that offset is a 64-wide column block of W[co][(ky, kx, ci)]
                                int sample, oy_shift, ox_shift, wcol;
                                if (p.conv_layer == 2) {      // conv3, stride 1: pixel (y, x) <- dY[y - ky][x - kx]
                                    sample = t.m0 / 81;
                                    oy_shift = q / 3; ox_shift = q - oy_shift * 3;
                                    wcol = q * 64;
                                } else {                      // conv2, stride 2: class (py, px), pixel (2a+py, 2c+px)
                                    sample = t.m0 / 400;      //   <- dY[a - dy][c - dx] with ky = py + 2dy, kx = px + 2dx
                                    const int cls = (t.m0 / 100) & 3;
                                    oy_shift = q >> 1; ox_shift = q & 1;
                                    wcol = (((cls >> 1) + 2 * oy_shift) * 4 + (cls & 1) + 2 * ox_shift) * 32;
                                }
                                if (lane < nq) tma_load_4d(a + j * a_sub, &tmA, &full_bar[s], 0, -ox_shift, -oy_shift,
                                                           group * p.a_samples + sample);
                                else tma_load_3d(b + j * b_sub, &tmB, &full_bar[s], wcol, 0, group);
                            }
                        }
                    } else if (sw64) {
                        // conv1 weight gradient: M tile = 4 kernel rows x 32 elements (4 boxes), K step = the
                        // 100 patches of one quarter sample; dY1 rows of the same patches from a [sample][400][32] map
                        const int ks = t.kt_begin + k;
                        if (lane == 0) mbar_expect_tx(&full_bar[s], box_bytes * 5u);
                        __syncwarp();
                        if (lane < 4) load_block(a + lane * p.kstep_rows * 64, (t.m0 / 128) * 4 + lane, ks);
                        else if (lane == 4) tma_load_3d(b, &tmB, &full_bar[s], t.n0, (ks & 3) * 100, group * p.b_samples + (ks >> 2));
                    } else {
                        const int q0 = t.m0 / 64, s0 = (t.kt_begin + k) * p.conv_nb;
                        const int nq = (q0 + 1 < cQ) ? 2 : 1;
                        if (lane == 0) mbar_expect_tx(&full_bar[s], box_bytes * (uint32_t)(nq + 1));
                        __syncwarp();
                        if (lane < nq) load_block(a + lane * p.kstep_rows * 128, q0 + lane, s0);
                        else if (lane == 2) tma_load_4d(b, &tmB, &full_bar[s], t.n0, 0, s0, group);
                    }
                } else {
                    if (lane == 0) mbar_expect_tx(&full_bar[s], bytes);
                    __syncwarp();
                    if (lane < 2) {          // A: one box (K-major) or two 64-wide boxes (MN-major)
                        if (!a_mn) { if (lane == 0) tma_load_3d(a, &tmA, &full_bar[s], k0, t.m0, group); }
                        else tma_load_3d(a + lane * 8192, &tmA, &full_bar[s], t.m0 + 64 * lane, k0, group);
                    } else if (lane < 6) {   // B likewise (up to four boxes for 256 columns)
                        const int j = lane - 2;
                        if (!b_mn) { if (j == 0) tma_load_3d(b, &tmB, &full_bar[s], k0, t.n0, group); }
                        else if (j < BN / 64) tma_load_3d(b + j * 8192, &tmB, &full_bar[s], t.n0 + 64 * j, k0, group);
                    }
                }
                __syncwarp();
                if (lane == 0) issued_iters = it + 1;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = make_instr_desc(BN, a_mn, b_mn);
            int it = 0, local = 0;
            bool ok = true;
            for (long tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x, local++) {
                const TileCoord t = decode_tile(p, tile, mt, nt);
                const int ab = local & 1;
                // the epilogue must have drained this accumulator buffer (two tiles ago)
                if (!mbar_wait(&acc_empty[ab], (((uint32_t)local >> 1) & 1u) ^ 1u, &abort_flag)) break;
                tcgen05_fence_after();
                const uint32_t tmem_acc = tmem_base + (uint32_t)ab * acc_cols;
                for (int k = 0; k < t.num_k; k++, it++) {
                    const int s = it % nst;
                    const uint32_t ph = (uint32_t)(it / nst) & 1u;
                    if (!mbar_wait(&full_bar[s], ph, &abort_flag)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t a_addr = smem_u32(smA + s * stage_a);
                    const uint32_t b_addr = smem_u32(smB + s * stage_b);
                    if (conv == CONV_WGRAD) {
                        // a K step is kstep_rows patches (the padding rows are zero on both sides)
                        const uint32_t row_bytes = sw64 ? 64u : 128u;
                        const uint32_t atom = (uint32_t)p.kstep_rows * row_bytes;
                        for (int kk = 0; kk < p.kstep_rows / 16; kk++) {
                            const uint64_t ad = make_smem_desc(a_addr + kk * 16 * row_bytes, 1, atom, sw64);
                            const uint64_t bd = make_smem_desc(b_addr + kk * 16 * row_bytes, 1, atom, sw64);
                            umma_bf16(tmem_acc, ad, bd, idesc, (k | kk) != 0 ? 1u : 0u);
                        }
                    } else if (conv == CONV_FWD || conv == CONV_DGRAD) {
                        // up to kpack blocks per step (see the producer); B is K-major (forward: weights as
                        // stored) or MN-major (data gradient: the offset's [co][ci] block)
                        const int kelems = sw64 ? 32 : BK;
                        const uint32_t a_sub = (uint32_t)p.a_sub_bytes, b_sub = (uint32_t)(BN * kelems * 2);
                        const int nq = min(p.kpack, p.conv_q - (t.kt_begin + k) * p.kpack);
                        for (int j = 0; j < nq; j++)
                            for (int kk = 0; kk < kelems / 16; kk++) {
                                const uint64_t ad = make_smem_desc(a_addr + j * a_sub + kk * 32, 0, 8192u, sw64);
                                const uint64_t bd = make_smem_desc(b_addr + j * b_sub + (b_mn ? kk * 2048 : kk * 32), b_mn, 8192u, sw64);
                                umma_bf16(tmem_acc, ad, bd, idesc, (k | j | kk) != 0 ? 1u : 0u);
                            }
                    } else {
#pragma unroll
                        for (int kk = 0; kk < BK / 16; kk++) {
                            // one UMMA consumes K = 16: 32 B along a K-major row, 16 rows (2048 B) of an MN-major tile
                            const uint64_t ad = make_smem_desc(a_addr + (a_mn ? kk * 2048 : kk * 32), a_mn);
                            const uint64_t bd = make_smem_desc(b_addr + (b_mn ? kk * 2048 : kk * 32), b_mn);
                            umma_bf16(tmem_acc, ad, bd, idesc, (k | kk) != 0 ? 1u : 0u);
                        }
                    }
                    umma_commit(&empty_bar[s]);
                }
                if (!ok) break;
                if (t.num_k > 0) umma_commit(&acc_full[ab]);   // arrives when the MMAs above have completed
                else mbar_arrive(&acc_full[ab]);               // empty K range: nothing to wait for
            }
        }
    } else {
        // ------------------------------------------------ epilogue warps 2..5 -> lane quarters 2,3,0,1
        const int q = warp & 3;
        uint8_t* stage = smE + (warp - 2) * kEpiWarpBytes;
        const bool out_bf16 = p.flags & EPI_OUT_BF16, relu = p.flags & EPI_RELU;
        const bool transpose = p.flags & EPI_TRANSPOSE, use_mask = p.flags & EPI_MASK;
        const bool vec_ok = out_bf16 ? ((p.ldc & 7) == 0 && (reinterpret_cast<uintptr_t>(p.out) & 15) == 0 &&
                                        (p.out_group_stride & 7) == 0 && (p.out_split_stride & 7) == 0)
                                     : ((p.ldc & 3) == 0 && (reinterpret_cast<uintptr_t>(p.out) & 15) == 0 &&
                                        (p.out_group_stride & 3) == 0 && (p.out_split_stride & 3) == 0);
        // 32-byte stores need every row start on a 32-byte boundary
        const bool direct_ok = !transpose &&
                               (out_bf16 ? ((p.ldc & 15) == 0 && (reinterpret_cast<uintptr_t>(p.out) & 31) == 0 &&
                                            (p.out_group_stride & 15) == 0 && (p.out_split_stride & 15) == 0)
                                         : ((p.ldc & 7) == 0 && (reinterpret_cast<uintptr_t>(p.out) & 31) == 0 &&
                                            (p.out_group_stride & 7) == 0 && (p.out_split_stride & 7) == 0));
        const bool direct_bias_vec = p.bias && (reinterpret_cast<uintptr_t>(p.bias) & 15) == 0 && (p.bias_group_stride & 3) == 0;
        const bool mask_vec = use_mask && (reinterpret_cast<uintptr_t>(p.mask) & 7) == 0 && (p.mask_group_stride & 3) == 0;
        int local = 0;
        for (long tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, local++) {
            const TileCoord t = decode_tile(p, tile, mt, nt);
            const int ab = local & 1;
            // gate words of this thread's row (one per 32 columns): they depend only on the tile, so they are
            // fetched before the wait for the MMAs
            uint32_t gws[8];
#pragma unroll
            for (int j = 0; j < 8; j++) gws[j] = 0xffffffffu;
            if (p.flags & EPI_GATE) {
                const int m = t.m0 + q * 32 + lane;
                if (m < p.M) {
                    const uint32_t* gp = p.gate + (long)agent_slot(p.am, t.gz) * p.gate_group_stride + (long)m * (p.N >> 5) + (t.n0 >> 5);
                    const int nw = (p.N - t.n0) >> 5;
#pragma unroll
                    for (int j = 0; j < 8; j++)
                        if (j < nw && 32 * j < BN) gws[j] = __ldg(gp + j);
                }
            }
            if (!mbar_wait(&acc_full[ab], ((uint32_t)local >> 1) & 1u, &abort_flag)) break;
            tcgen05_fence_after();
            const uint32_t tmem_acc = tmem_base + (uint32_t)ab * acc_cols;
            const int slot = agent_slot(p.am, t.gz);
            const int group = p.group0 + slot;
            const long obase = (long)slot * p.out_group_stride + (long)t.split * p.out_split_stride;
            // block sums of squares are kept per agent: the tile index as it would be in a launch over all agents
            const long sq_tile = tile + (long)(slot - t.gz) * mt * nt;
            const float* bias = p.bias ? p.bias + (long)group * p.bias_group_stride : nullptr;
            const __nv_bfloat16* mask = use_mask ? p.mask + (long)slot * p.mask_group_stride : nullptr;
            const int mw = t.m0 + q * 32;   // first row of this warp
            const bool rowmap = p.flags & EPI_ROWMAP_S2;
            // element offset (inside the group) of output row r of this tile
            auto row_off = [&](int r) -> long {
                if (!rowmap) return (long)(t.m0 + r) * p.ldc;
                const int sample = t.m0 / 400, cls = (t.m0 / 100) & 3;
                const int ra = r / 10, rc = r - ra * 10;
                return ((long)(sample * 20 + 2 * ra + (cls >> 1)) * 20 + 2 * rc + (cls & 1)) * p.ldc;
            };
            for (int c0 = 0; c0 < BN; c0 += 32) {
                uint32_t r[32];
                if (t.num_k > 0) {
                    tmem_ld32(tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
                } else {
#pragma unroll
                    for (int j = 0; j < 32; j++) r[j] = 0u;
                }
                if (p.flags & EPI_GATE) {
                    uint32_t gw = gws[0];
#pragma unroll
                    for (int j = 1; j < 8; j++)
                        if (c0 == 32 * j) gw = gws[j];
#pragma unroll
                    for (int j = 0; j < 32; j++)
                        if (!((gw >> j) & 1u)) r[j] = 0u;
                }
                const int nb = t.n0 + c0;
                if (mw >= p.M || q * 32 >= p.tile_rows || nb >= p.N) {   // warp-uniform
                    if (p.sq_partial && lane == 0) p.sq_partial[sq_tile * (BN >> 3) + q * (BN >> 5) + (c0 >> 5)] = 0.0f;
                    continue;
                }
                if (transpose) {
                    // D[m][n] -> out[n * ldc + m]: consecutive lanes write consecutive addresses
                    const int m = mw + lane;
                    if (m < p.M && q * 32 + lane < p.tile_rows) {
                        if (out_bf16) {
                            __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + obase + m;
#pragma unroll
                            for (int j = 0; j < 32; j++)
                                if (nb + j < p.N) {
                                    float v = __uint_as_float(r[j]) * p.scale;
                                    if (bias) v += __ldg(bias + nb + j);
                                    if (relu) v = fmaxf(v, 0.0f);
                                    o[(long)(nb + j) * p.ldc] = __float2bfloat16_rn(v);
                                }
                        } else {
                            float* o = reinterpret_cast<float*>(p.out) + obase + m;
#pragma unroll
                            for (int j = 0; j < 32; j++)
                                if (nb + j < p.N) {
                                    float v = __uint_as_float(r[j]) * p.scale;
                                    if (bias) v += __ldg(bias + nb + j);
                                    if (relu) v = fmaxf(v, 0.0f);
                                    o[(long)(nb + j) * p.ldc] = v;
                                }
                        }
                    }
                    continue;
                }
                // Direct path: the thread owns row mw + lane and holds its 32 columns, 64 contiguous bytes of bf16
                // or 128 of fp32 in the output: whole 32-byte sectors, written with 32-byte stores from registers.
                if (direct_ok && !use_mask && !rowmap && nb + 32 <= p.N) {
                    const int m = mw + lane;
                    float row_sq = 0.0f;
                    if (m < p.M && q * 32 + lane < p.tile_rows) {
                        float vals[32];
#pragma unroll
                        for (int j = 0; j < 32; j++) vals[j] = __uint_as_float(r[j]) * p.scale;
                        if (bias) {
#pragma unroll
                            for (int j4 = 0; j4 < 8; j4++) {   // all lanes read the same addresses: one broadcast each
                                const float4 bv = direct_bias_vec ? __ldg(reinterpret_cast<const float4*>(bias + nb) + j4)
                                                                  : make_float4(__ldg(bias + nb + 4 * j4), __ldg(bias + nb + 4 * j4 + 1),
                                                                                __ldg(bias + nb + 4 * j4 + 2), __ldg(bias + nb + 4 * j4 + 3));
                                vals[4 * j4] += bv.x; vals[4 * j4 + 1] += bv.y; vals[4 * j4 + 2] += bv.z; vals[4 * j4 + 3] += bv.w;
                            }
                        }
                        if (relu) {
#pragma unroll
                            for (int j = 0; j < 32; j++) vals[j] = fmaxf(vals[j], 0.0f);
                        }
                        if (p.sq_partial) {   // this row's share of the block's sum of squares (fixed order)
                            float sq = 0.0f;
#pragma unroll
                            for (int j = 0; j < 32; j++) sq = fmaf(vals[j], vals[j], sq);
                            row_sq = sq;
                        }
                        const long off = obase + (long)m * p.ldc + nb;
                        if (out_bf16) {
                            uint32_t o[16];
#pragma unroll
                            for (int j = 0; j < 16; j++) o[j] = pack2(vals[2 * j], vals[2 * j + 1]);
                            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + off;
                            st_global_v8(dst, &o[0]);
                            st_global_v8(dst + 16, &o[8]);
                        } else {
                            float* dst = reinterpret_cast<float*>(p.out) + off;
#pragma unroll
                            for (int j8 = 0; j8 < 4; j8++) st_global_v8(dst + 8 * j8, reinterpret_cast<const uint32_t*>(&vals[8 * j8]));
                        }
                    }
                    if (p.sq_partial) {   // rows of the block added by a butterfly: the same tree every time
                        for (int o = 16; o > 0; o >>= 1) row_sq += __shfl_xor_sync(0xffffffffu, row_sq, o);
                        if (lane == 0) p.sq_partial[sq_tile * (BN >> 3) + q * (BN >> 5) + (c0 >> 5)] = row_sq;
                    }
                    continue;
                }
                // row-major output: park the raw 32 x 32 block in shared memory (lane = row), then let every
                // 8 lanes handle one row segment of 128 contiguous bytes, so the global accesses coalesce
                {
                    uint4* w = reinterpret_cast<uint4*>(stage + lane * kEpiRowBytes);
#pragma unroll
                    for (int j = 0; j < 8; j++) w[j] = make_uint4(r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
                }
                __syncwarp();
                const int cl = (lane & 7) * 4;          // first of this lane's 4 columns inside the block
                const int n = nb + cl;
                // fast path: the whole 32 x 32 block is inside the matrix and 16-byte stores are possible;
                // straight-line code, the loads it needs (bias, mask) issued up front
                if (vec_ok && mw + 32 <= p.M && q * 32 + 32 <= p.tile_rows && nb + 32 <= p.N && (!use_mask || mask_vec)) {
                    float4 bv = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (bias) {
                        if ((reinterpret_cast<uintptr_t>(bias + n) & 15) == 0) bv = __ldg(reinterpret_cast<const float4*>(bias + n));
                        else bv = make_float4(__ldg(bias + n), __ldg(bias + n + 1), __ldg(bias + n + 2), __ldg(bias + n + 3));
                    }
                    const int r0 = lane >> 3;
                    long roff[8];
#pragma unroll
                    for (int i = 0; i < 8; i++) roff[i] = row_off(q * 32 + r0 + 4 * i) + n;
                    uint2 mk[8];
                    if (use_mask) {
#pragma unroll
                        for (int i = 0; i < 8; i++) mk[i] = __ldg(reinterpret_cast<const uint2*>(mask + roff[i]));
                    }
                    const uint8_t* sp = stage + r0 * kEpiRowBytes + cl * 4;
#pragma unroll
                    for (int i = 0; i < 8; i++) {
                        const uint4 raw = *reinterpret_cast<const uint4*>(sp + i * 4 * kEpiRowBytes);
                        float v0 = fmaf(__uint_as_float(raw.x), p.scale, bv.x), v1 = fmaf(__uint_as_float(raw.y), p.scale, bv.y);
                        float v2 = fmaf(__uint_as_float(raw.z), p.scale, bv.z), v3 = fmaf(__uint_as_float(raw.w), p.scale, bv.w);
                        if (relu) { v0 = fmaxf(v0, 0.f); v1 = fmaxf(v1, 0.f); v2 = fmaxf(v2, 0.f); v3 = fmaxf(v3, 0.f); }
                        if (use_mask) {
                            const __nv_bfloat162* mh = reinterpret_cast<const __nv_bfloat162*>(&mk[i]);
                            const float2 ma = __bfloat1622float2(mh[0]), mb = __bfloat1622float2(mh[1]);
                            if (!(ma.x > 0.f)) v0 = 0.f;
                            if (!(ma.y > 0.f)) v1 = 0.f;
                            if (!(mb.x > 0.f)) v2 = 0.f;
                            if (!(mb.y > 0.f)) v3 = 0.f;
                        }
                        const long off = obase + roff[i];
                        if (out_bf16) {
                            uint2 u;
                            u.x = pack2(v0, v1); u.y = pack2(v2, v3);
                            *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + off) = u;
                        } else {
                            *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + off) = make_float4(v0, v1, v2, v3);
                        }
                    }
                    __syncwarp();
                    continue;
                }
#pragma unroll
                for (int i = 0; i < 8; i++) {
                    const int rr = i * 4 + (lane >> 3);
                    const int m = mw + rr;
                    if (m >= p.M || q * 32 + rr >= p.tile_rows || n >= p.N) continue;
                    const uint4 raw = *reinterpret_cast<const uint4*>(stage + rr * kEpiRowBytes + cl * 4);
                    float v[4] = {__uint_as_float(raw.x) * p.scale, __uint_as_float(raw.y) * p.scale,
                                  __uint_as_float(raw.z) * p.scale, __uint_as_float(raw.w) * p.scale};
                    const int valid = min(4, p.N - n);
                    if (bias) {
#pragma unroll
                        for (int j = 0; j < 4; j++) if (j < valid) v[j] += __ldg(bias + n + j);
                    }
                    if (relu) {
#pragma unroll
                        for (int j = 0; j < 4; j++) v[j] = fmaxf(v[j], 0.0f);
                    }
                    const long off = row_off(q * 32 + rr) + n;
                    if (use_mask) {
                        if (mask_vec && valid == 4 && ((off & 3) == 0)) {
                            const uint2 mk = __ldg(reinterpret_cast<const uint2*>(mask + off));
                            const __nv_bfloat162* mh = reinterpret_cast<const __nv_bfloat162*>(&mk);
                            const float2 m0f = __bfloat1622float2(mh[0]), m1f = __bfloat1622float2(mh[1]);
                            if (!(m0f.x > 0.0f)) v[0] = 0.0f;
                            if (!(m0f.y > 0.0f)) v[1] = 0.0f;
                            if (!(m1f.x > 0.0f)) v[2] = 0.0f;
                            if (!(m1f.y > 0.0f)) v[3] = 0.0f;
                        } else {
#pragma unroll
                            for (int j = 0; j < 4; j++)
                                if (j < valid && !(__bfloat162float(mask[off + j]) > 0.0f)) v[j] = 0.0f;
                        }
                    }
                    if (out_bf16) {
                        __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(p.out) + obase + off;
                        if (vec_ok && valid == 4 && (((obase + off) & 3) == 0)) {
                            __nv_bfloat162 h0 = __floats2bfloat162_rn(v[0], v[1]), h1 = __floats2bfloat162_rn(v[2], v[3]);
                            uint2 u;
                            u.x = *reinterpret_cast<uint32_t*>(&h0); u.y = *reinterpret_cast<uint32_t*>(&h1);
                            *reinterpret_cast<uint2*>(o) = u;
                        } else {
#pragma unroll
                            for (int j = 0; j < 4; j++) if (j < valid) o[j] = __float2bfloat16_rn(v[j]);
                        }
                    } else {
                        float* o = reinterpret_cast<float*>(p.out) + obase + off;
                        if (vec_ok && valid == 4 && (((obase + off) & 3) == 0)) {
                            *reinterpret_cast<float4*>(o) = make_float4(v[0], v[1], v[2], v[3]);
                        } else {
#pragma unroll
                            for (int j = 0; j < 4; j++) if (j < valid) o[j] = v[j];
                        }
                    }
                }
                __syncwarp();   // the staging block is rewritten by the next column block
            }
            // this warp no longer reads the accumulator buffer
            tcgen05_fence_before();
            if (lane == 0) mbar_arrive(&acc_empty[ab]);
        }
    }

    // teardown
    tcgen05_fence_before();
    __syncthreads();
    if (abort_flag) {
        if (threadIdx.x == 0) {
            if (p.error_word) atomicExch(p.error_word, 1);
            // let copies that were already issued land before the shared memory goes away
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

// ------------------------------------------------------------------ split-K reduction
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const float* __restrict__ partials, float* __restrict__ out,
                                                            long count, int split_k, long split_stride,
                                                            long partial_group_stride, long out_group_stride) {
    pdl_wait();
    pdl_launch();
    const int g = blockIdx.y;
    const float* pg = partials + (long)g * partial_group_stride;
    float* og = out + (long)g * out_group_stride;
    for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < count; i += (long)gridDim.x * blockDim.x) {
        float acc = pg[i];
        for (int s = 1; s < split_k; s++) acc += pg[(long)s * split_stride + i];  // fixed order
        og[i] = acc;
    }
}
// Up to six such reductions in one launch (the conv weight and bias gradients of a step), 16 bytes per thread.
__global__ void __launch_bounds__(256) splitk_reduce_multi_kernel(const float* __restrict__ ws, float* __restrict__ out,
                                                                  ReduceSegs sg, long total4, long ws_group_stride,
                                                                  long out_group_stride, AgentMap am) {
    pdl_wait();
    pdl_launch();
    const int g = agent_slot(am, blockIdx.y);
    const float* wg = ws + (long)g * ws_group_stride;
    float* og = out + (long)g * out_group_stride;
    for (long j = blockIdx.x * (long)blockDim.x + threadIdx.x; j < total4; j += (long)gridDim.x * blockDim.x) {
        int k = 0;
        long jj = j;
        while (k + 1 < sg.n && jj >= sg.s[k].count / 4) { jj -= sg.s[k].count / 4; k++; }
        const float* src = wg + sg.s[k].ws_off + jj * 4;
        const long cnt = sg.s[k].count;
        const int split = sg.s[k].split;
        float4 t = *reinterpret_cast<const float4*>(src);
        for (int s0 = 1; s0 < split; s0 += 4) {   // fixed order; four loads in flight
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; u++)
                v[u] = s0 + u < split ? *reinterpret_cast<const float4*>(src + (long)(s0 + u) * cnt) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 4; u++)
                if (s0 + u < split) { t.x += v[u].x; t.y += v[u].y; t.z += v[u].z; t.w += v[u].w; }
        }
        *reinterpret_cast<float4*>(og + sg.s[k].out_off + jj * 4) = t;
    }
}
cudaError_t launch_splitk_reduce_multi(const float* ws, float* out, const ReduceSegs& segs, int groups,
                                       long ws_group_stride, long out_group_stride, cudaStream_t st, const AgentMap* am) {
    if (segs.n < 1 || segs.n > 6 || ((ws_group_stride | out_group_stride) & 3)) return cudaErrorInvalidValue;
    long total4 = 0;
    for (int k = 0; k < segs.n; k++) {
        if ((segs.s[k].out_off | segs.s[k].count | segs.s[k].ws_off) & 3 || segs.s[k].split < 1) return cudaErrorInvalidValue;
        total4 += segs.s[k].count / 4;
    }
    if ((reinterpret_cast<uintptr_t>(ws) | reinterpret_cast<uintptr_t>(out)) & 15) return cudaErrorInvalidValue;
    int bx = (int)((total4 + 255) / 256);
    if (bx > sm_count() * 4) bx = sm_count() * 4;
    (void)launch_pdl(splitk_reduce_multi_kernel, dim3(bx, groups), dim3(256), 0, st, ws, out, segs, total4, ws_group_stride,
                     out_group_stride, am ? *am : AgentMap{});
    return cudaGetLastError();
}

// Same fixed-order reduction followed by the forward epilogue of a dense layer: + bias[n], ReLU, bf16.
__global__ void __launch_bounds__(256) splitk_reduce_act_kernel(const float* __restrict__ partials,
                                                                __nv_bfloat16* __restrict__ out, const float* __restrict__ bias,
                                                                long bias_group_stride, int group0, long count, int N,
                                                                int split_k, long split_stride, long partial_group_stride,
                                                                long out_group_stride) {
    pdl_wait();
    pdl_launch();
    const int g = blockIdx.y;
    const float4* pg = reinterpret_cast<const float4*>(partials + (long)g * partial_group_stride);
    const float* bg = bias + (long)(group0 + g) * bias_group_stride;
    uint2* og = reinterpret_cast<uint2*>(out + (long)g * out_group_stride);
    const long n4 = count / 4, s4 = split_stride / 4;
    for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n4; i += (long)gridDim.x * blockDim.x) {
        float4 acc = pg[i];
        for (int s = 1; s < split_k; s++) {   // fixed order
            const float4 v = pg[(long)s * s4 + i];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        const int n = (int)((i * 4) % N);
        acc.x = fmaxf(acc.x + __ldg(bg + n), 0.f); acc.y = fmaxf(acc.y + __ldg(bg + n + 1), 0.f);
        acc.z = fmaxf(acc.z + __ldg(bg + n + 2), 0.f); acc.w = fmaxf(acc.w + __ldg(bg + n + 3), 0.f);
        uint2 u;
        u.x = pack2(acc.x, acc.y); u.y = pack2(acc.z, acc.w);
        og[i] = u;
    }
}
cudaError_t launch_splitk_reduce_act(const float* partials, __nv_bfloat16* out, const float* bias, long bias_group_stride,
                                     int group0, long count, int N, int split_k, long split_stride, int groups,
                                     long partial_group_stride, long out_group_stride, cudaStream_t st) {
    if ((count & 3) || (N & 3) || (split_stride & 3) || (partial_group_stride & 3) || (out_group_stride & 3))
        return cudaErrorInvalidValue;
    int bx = (int)((count / 4 + 255) / 256);
    if (bx > sm_count() * 4) bx = sm_count() * 4;
    (void)launch_pdl(splitk_reduce_act_kernel, dim3(dim3(bx, groups)), dim3(256), 0, st, partials, out, bias, bias_group_stride, group0, count, N,
                                                               split_k, split_stride, partial_group_stride, out_group_stride);
    return cudaGetLastError();
}

cudaError_t launch_splitk_reduce(const float* partials, float* out, long count, int split_k, long split_stride,
                                 int groups, long partial_group_stride, long out_group_stride, cudaStream_t st) {
    int bx = (int)((count + 255) / 256);
    if (bx > sm_count() * 4) bx = sm_count() * 4;
    (void)launch_pdl(splitk_reduce_kernel, dim3(dim3(bx, groups)), dim3(256), 0, st, partials, out, count, split_k, split_stride,
                                                           partial_group_stride, out_group_stride);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

int sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

cudaError_t gemm_init() {
    cudaError_t e;
    if (!g_encode) {   // once per process
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    // the opt-in to large dynamic shared memory is a property of the function on ONE device: once per device
    static bool attr_done[64] = {};
    int dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!attr_done[dev]) {
        if ((e = cudaFuncSetAttribute(gemm_tcgen05_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes)) != cudaSuccess)
            return e;
        attr_done[dev] = true;
    }
    return cudaSuccess;
}

bool make_tensor_map(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t groups,
                     uint64_t row_stride_bytes, uint64_t group_stride_bytes, uint32_t box_cols, uint32_t box_rows) {
    if (!g_encode) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15) || (row_stride_bytes & 15) || (group_stride_bytes & 15)) return false;
    if (groups == 0) groups = 1;
    if (group_stride_bytes == 0) group_stride_bytes = rows * row_stride_bytes;
    cuuint64_t dims[3] = {cols, rows, groups};
    cuuint64_t strides[2] = {row_stride_bytes, group_stride_bytes};
    cuuint32_t box[3] = {box_cols, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_tensor_map_f32(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t row_stride_bytes,
                         uint32_t box_cols, uint32_t box_rows) {
    if (!g_encode) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15) || (row_stride_bytes & 15) || box_cols > 256 || box_rows > 256) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {row_stride_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The same matrix seen as [rows][cols / 256][256] (cols a multiple of 256): a box {256, box_blocks, box_rows} is
// box_rows x (256 * box_blocks) floats in one copy, past the 256-element limit of a box edge.
bool make_tensor_map_f32_wide(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t row_stride_bytes,
                              uint32_t box_blocks, uint32_t box_rows) {
    if (!g_encode) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15) || (row_stride_bytes & 15) || (cols & 255) || box_blocks > 256 || box_rows > 256)
        return false;
    cuuint64_t dims[3] = {256, cols / 256, rows};
    cuuint64_t strides[2] = {1024, row_stride_bytes};
    cuuint32_t box[3] = {256, box_blocks, box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_tensor_map_nd(CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                        const uint64_t* strides_bytes, const uint32_t* box, int swizzle) {
    if (!g_encode || rank < 3 || rank > 5) return false;
    if (reinterpret_cast<uintptr_t>(base) & 15) return false;
    cuuint64_t d[5], st[4];
    cuuint32_t b[5], es[5];
    for (int i = 0; i < rank; i++) { d[i] = dims[i]; b[i] = box[i]; es[i] = 1; if (box[i] > 256) return false; }
    for (int i = 0; i + 1 < rank; i++) { st[i] = strides_bytes[i]; if (st[i] & 15) return false; }
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es,
                          CU_TENSOR_MAP_INTERLEAVE_NONE,
                          swizzle == 3 ? CU_TENSOR_MAP_SWIZZLE_NONE
                          : swizzle == 2 ? CU_TENSOR_MAP_SWIZZLE_32B : (swizzle == 1 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B),
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_operand(GemmOperand* op, const void* base, int mn_major, uint64_t mn_extent, uint64_t k_extent,
                  uint64_t groups, uint64_t ld_elems, uint64_t group_stride_elems, int tile_mn) {
    op->mn_major = mn_major;
    if (!mn_major)
        return make_tensor_map(&op->map, base, k_extent, mn_extent, groups, ld_elems * 2, group_stride_elems * 2, BK,
                               (uint32_t)tile_mn);
    return make_tensor_map(&op->map, base, mn_extent, k_extent, groups, ld_elems * 2, group_stride_elems * 2, 64, BK);
}

cudaError_t launch_gemm(const GemmOperand& A, const GemmOperand& B, const GemmArgs& args, cudaStream_t st) {
    if (args.block_n != 32 && args.block_n != 64 && args.block_n != 128 &&
        !(args.block_n == 256 && args.conv_mode == CONV_NONE))
        return cudaErrorInvalidValue;
    if (B.mn_major && args.block_n < 64 && !(args.conv_mode != CONV_NONE && args.conv_layer == 0)) return cudaErrorInvalidValue;
    if (args.split_k < 1 || args.groups < 1 || args.M < 1 || args.N < 1 || args.K < 1) return cudaErrorInvalidValue;
    if (args.sq_partial && ((args.block_n != 128 && args.block_n != 256) || args.split_k != 1 || (args.N & 31) || (args.ldc & 7) ||
                            (args.flags & (EPI_OUT_BF16 | EPI_TRANSPOSE | EPI_MASK | EPI_ROWMAP_S2)) ||
                            (reinterpret_cast<uintptr_t>(args.out) & 31) || (args.out_group_stride & 7) ||
                            args.conv_mode != CONV_NONE))
        return cudaErrorInvalidValue;
    if ((args.flags & EPI_GATE) && (!args.gate || (args.N & 31) || (args.flags & (EPI_TRANSPOSE | EPI_ROWMAP_S2))))
        return cudaErrorInvalidValue;
    GemmArgs a = args;
    if (a.conv_mode == CONV_NONE) {
        a.tile_rows = BM;
        a.k_steps = (a.K + BK - 1) / BK;
        a.stage_a_bytes = kStageA;
        a.stage_b_bytes = a.block_n * BK * 2;
    } else {
        if (a.conv_layer < 0 || a.conv_layer > 2) return cudaErrorInvalidValue;
        if (a.conv_layer == 0 && (a.conv_mode == CONV_DGRAD || a.block_n != 32)) return cudaErrorInvalidValue;
        const int P = a.conv_layer == 0 ? 100 : (a.conv_layer == 1 ? 81 : 49);
        const int row_bytes = a.conv_layer == 0 ? 64 : 128;
        if (a.conv_nb < 1 || a.tile_rows < 1 || a.tile_rows > BM || a.k_steps < 1) return cudaErrorInvalidValue;
        if (a.conv_mode != CONV_DGRAD && a.conv_nb * P > 128) return cudaErrorInvalidValue;
        if (a.box_rows < 1 || a.box_rows > 128) return cudaErrorInvalidValue;
        if (a.conv_mode == CONV_FWD || a.conv_mode == CONV_DGRAD) {
            if (a.conv_mode == CONV_FWD) {
                if (A.mn_major || B.mn_major || a.tile_rows != a.conv_nb * P || a.box_rows != a.tile_rows) return cudaErrorInvalidValue;
                a.conv_q = a.conv_layer == 2 ? 9 : 8;    // 64-element (conv1: 32-element) blocks of a patch
            } else {
                if (A.mn_major || !B.mn_major || a.block_n != 64 || a.tile_rows != a.box_rows) return cudaErrorInvalidValue;
                a.conv_q = a.conv_layer == 2 ? 9 : 4;    // kernel offsets that reach one pixel (class)
            }
            if (a.kpack < 1) a.kpack = 1;
            if (a.kpack > 8) return cudaErrorInvalidValue;
            a.k_steps = (a.conv_q + a.kpack - 1) / a.kpack;
            a.a_sub_bytes = (a.box_rows * row_bytes + 1023) / 1024 * 1024;
            // the last block's MMA reads 128 rows from its start: keep that inside the stage
            a.stage_a_bytes = (a.kpack - 1) * a.a_sub_bytes + BM * row_bytes;
            a.stage_b_bytes = a.kpack * a.block_n * row_bytes;
        } else {
            if (!A.mn_major || !B.mn_major || (a.block_n != 64 && a.conv_layer != 0) || a.kstep_rows % 16 ||
                a.kstep_rows < a.conv_nb * P || a.kstep_rows > 128 || a.tile_rows != BM)
                return cudaErrorInvalidValue;
            a.stage_a_bytes = (a.conv_layer == 0 ? 4 : 2) * a.kstep_rows * row_bytes;
            a.stage_b_bytes = a.kstep_rows * row_bytes;
        }
    }
    const int mt = (a.M + a.tile_rows - 1) / a.tile_rows, nt = (a.N + a.block_n - 1) / a.block_n;
    const long total = (long)mt * nt * a.groups * a.split_k;
    const int per_split = (a.k_steps + a.split_k - 1) / a.split_k;
    // ring depth: enough to cover a tile's reduction and keep loads of the next tile in flight
    a.stages = per_split + 1 < kStages ? per_split + 1 : kStages;
    if (a.stages < 2) a.stages = 2;
    size_t smem = (size_t)a.stages * (a.stage_a_bytes + a.stage_b_bytes) + 4 * kEpiWarpBytes + 1024;
    // two resident CTAs per SM (two producers, two MMA issuers, eight epilogue warps) beat one CTA
    // with a deeper ring: shrink the ring until two fit
    while (a.block_n < 256 && smem > (size_t)(110 * 1024) && a.stages > 2) {
        a.stages--;
        smem = (size_t)a.stages * (a.stage_a_bytes + a.stage_b_bytes) + 4 * kEpiWarpBytes + 1024;
    }
    while (smem > (size_t)kSmemBytes && a.stages > 2) {
        a.stages--;
        smem = (size_t)a.stages * (a.stage_a_bytes + a.stage_b_bytes) + 4 * kEpiWarpBytes + 1024;
    }
    if (smem > (size_t)kSmemBytes) return cudaErrorInvalidValue;
    int per_sm = (int)((220u * 1024u) / smem);
    if (per_sm > 2) per_sm = 2;   // 2 x 256 tensor-memory columns is all an SM has
    if (per_sm < 1) per_sm = 1;
    long cap = (long)sm_count() * per_sm;
    if (a.max_ctas > 0 && cap > (long)a.max_ctas * per_sm) cap = (long)a.max_ctas * per_sm;
    const int grid = (int)(total < cap ? total : cap);
    (void)launch_pdl(gemm_tcgen05_kernel, dim3(grid), dim3(192), smem, st, A.map, B.map, a, A.mn_major, B.mn_major, total, mt, nt);
    return cudaGetLastError();
}

}  // namespace gala
