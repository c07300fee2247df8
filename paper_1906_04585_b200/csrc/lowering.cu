// Helpers around the convolutions of the 84x84x4 -> 20x20x32 -> 9x9x64 -> 7x7x64 trunk (Appendix
// C.2 network): the uint8 -> bf16 frame copy that the implicit conv1 products read, and the bias
// gradients.  The convolutions themselves (forward, data and weight gradients) are implicit GEMMs
// in gemm.cu; no patch matrix is ever written.
#include "internal.h"

namespace gala {

// uint8 frames -> bf16 frames (0..255 are exact in bf16; the 1/255 scale is applied after the
// contraction).  16 bytes in, 32 bytes out per thread and step.
__global__ void __launch_bounds__(256) cast_frames_kernel(PtrBatch obs, __nv_bfloat16* __restrict__ out, long out_group_stride,
                                                          long n16) {
    pdl_wait();
    pdl_launch();
    const int g = blockIdx.y;
    const uint4* src = reinterpret_cast<const uint4*>(obs.p[g]);
    uint4* dst = reinterpret_cast<uint4*>(out + (long)g * out_group_stride);
    for (long i = blockIdx.x * (long)blockDim.x + threadIdx.x; i < n16; i += (long)gridDim.x * blockDim.x) {
        const uint4 v = __ldg(src + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[8];
#pragma unroll
        for (int q = 0; q < 4; q++) {
            __nv_bfloat162 p0 = __floats2bfloat162_rn((float)(w[q] & 255u), (float)((w[q] >> 8) & 255u));
            __nv_bfloat162 p1 = __floats2bfloat162_rn((float)((w[q] >> 16) & 255u), (float)(w[q] >> 24));
            o[2 * q] = *reinterpret_cast<uint32_t*>(&p0);
            o[2 * q + 1] = *reinterpret_cast<uint32_t*>(&p1);
        }
        dst[2 * i] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[2 * i + 1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}
cudaError_t launch_cast_frames(const PtrBatch& obs, __nv_bfloat16* out, long out_group_stride, int samples, int groups,
                               cudaStream_t st) {
    const long n16 = (long)samples * (84 * 84 * 4 / 16);
    int bx = (int)((n16 + 255) / 256);
    if (bx > sm_count() * 8) bx = sm_count() * 8;
    (void)launch_pdl(cast_frames_kernel, dim3(dim3(bx, groups)), dim3(256), 0, st, obs, out, out_group_stride, n16);
    return cudaGetLastError();
}

// Bias gradient: out[c] = sum over rows of dy[row][c].  Rows are cut into kColsumChunks fixed
// chunks (one block each).  Inside a block a thread owns 8 adjacent columns (one 16-byte load per
// row) and every (256*8/C)-th row of the chunk; the row lanes are combined in index order, and the
// block that finishes last adds the chunk sums in index order, so the result does not depend on
// scheduling.  C is a power of two, 8 <= C <= 512.
// Up to kColsumJobs tensors are reduced by one launch (blockIdx.z picks the tensor).
__global__ void __launch_bounds__(256) colsum_kernel(ColsumJobs jobs, int n_jobs, ColsumSlices sl,
                                                     float* __restrict__ out_base, long out_group_stride,
                                                     double* partial_base, unsigned* ticket_base, AgentMap am) {
    pdl_wait();
    pdl_launch();
    const int gz = blockIdx.y;            // position in the launch
    const int g = agent_slot(am, gz);     // agent whose tensors are addressed
    __shared__ float red[256 * 8];
    if ((int)blockIdx.z == n_jobs) {
        // Bias slices of a conv2 data-gradient launch: CTA b of sl.grid worked on samples
        // [total * b / grid, total * (b + 1) / grid); those whose range meets agent g's samples left 8 warp slices
        // of 32 channels each.  Thread (w, c) adds slice w of the CTAs in order, then the 8 sums are added in order.
        if (blockIdx.x != 0) return;
        const long total = (long)gridDim.y * sl.rows, lo = (long)gz * sl.rows, hi = lo + sl.rows;
        int b_lo = (int)(lo * sl.grid / total);
        while (b_lo > 0 && total * b_lo / sl.grid > lo) b_lo--;
        while (total * (b_lo + 1) / sl.grid <= lo) b_lo++;
        int b_hi = b_lo;                                   // last CTA whose range starts below hi
        while (b_hi + 1 < sl.grid && total * (b_hi + 1) / sl.grid < hi) b_hi++;
        const int w = threadIdx.x >> 5, c = threadIdx.x & 31;
        const float* src = sl.partial + ((long)g * kConvMaxGrid * 8 + w) * 32 + c;
        float s = 0.0f;
        for (int b = b_lo; b <= b_hi; b += 4) {
            float v[4];
#pragma unroll
            for (int u = 0; u < 4; u++) v[u] = b + u <= b_hi ? __ldcg(src + (long)(b + u) * 8 * 32) : 0.0f;
#pragma unroll
            for (int u = 0; u < 4; u++) s += v[u];
        }
        red[threadIdx.x] = s;
        __syncthreads();
        if (threadIdx.x < 32) {
            float t = 0.0f;
            for (int k = 0; k < 8; k++) t += red[k * 32 + threadIdx.x];
            out_base[(long)g * out_group_stride + sl.out_off + threadIdx.x] = t;
        }
        return;
    }
    const ColsumJob job = jobs.j[blockIdx.z];
    const long rows = job.rows;
    const int C = job.C;
    float* out = out_base + job.out_off;
    double* partial = partial_base + (long)blockIdx.z * kColsumChunks * 512;
    unsigned* ticket = ticket_base + blockIdx.z;
    const uint4* src = reinterpret_cast<const uint4*>(job.dy + (long)g * job.group_stride);
    const long per = (rows + kColsumChunks - 1) / kColsumChunks;
    const long lo = (long)blockIdx.x * per;
    long hi = lo + per; if (hi > rows) hi = rows;
    __shared__ bool last;
    double* part = partial + (long)g * kColsumJobs * kColsumChunks * 512 + (long)blockIdx.x * C;
    const int cchunks = C / 8;                    // 16-byte column groups per row
    const int lanes = 256 / cchunks > 0 ? 256 / cchunks : 1;   // row lanes (C <= 512 -> cchunks <= 64)
    const int cc = threadIdx.x % cchunks, rl = threadIdx.x / cchunks;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (rl < lanes) {
        // four rows a step, so that four 16-byte loads are in flight per thread; the sums keep the row order
        for (long r = lo + rl; r < hi; r += 4L * lanes) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; u++) {
                const long ru = r + (long)u * lanes;
                v[u] = ru < hi ? __ldg(src + ru * cchunks + cc) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 4; u++) {
                const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v[u]);
#pragma unroll
                for (int q = 0; q < 4; q++) {
                    const float2 f = __bfloat1622float2(h[q]);
                    acc[2 * q] += f.x; acc[2 * q + 1] += f.y;
                }
            }
        }
    }
#pragma unroll
    for (int q = 0; q < 8; q++) red[threadIdx.x * 8 + q] = acc[q];
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        const int ccq = c / 8, q = c % 8;
        float s = 0.0f;
        for (int l = 0; l < lanes; l++) s += red[(l * cchunks + ccq) * 8 + q];
        part[c] = (double)s;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        unsigned t = atomicAdd(&ticket[g * kColsumJobs], 1u);
        last = (t == kColsumChunks - 1);
    }
    __syncthreads();
    if (last) {
        __threadfence();
        const volatile double* pg = partial + (long)g * kColsumJobs * kColsumChunks * 512;
        for (int c = threadIdx.x; c < C; c += blockDim.x) {
            double s = 0.0;
            for (int k = 0; k < kColsumChunks; k++) s += pg[(long)k * C + c];
            out[(long)g * out_group_stride + c] = (float)s;
        }
        if (threadIdx.x == 0) ticket[g * kColsumJobs] = 0;
    }
}
cudaError_t launch_colsum(const ColsumJobs& jobs, int n_jobs, float* out_base, long out_group_stride, double* partial,
                          unsigned* ticket, int groups, cudaStream_t st, const ColsumSlices* slices, const AgentMap* am) {
    if (n_jobs < 1 || n_jobs > kColsumJobs) return cudaErrorInvalidValue;
    ColsumSlices sl{};
    if (slices) {
        sl = *slices;
        if (!sl.partial || sl.rows < 1 || sl.grid != conv_grid((long)groups * sl.rows, sl.grid)) return cudaErrorInvalidValue;
    }
    for (int i = 0; i < n_jobs; i++) {
        const int C = jobs.j[i].C;
        if (C > 512 || C < 8 || (C & (C - 1))) return cudaErrorInvalidValue;
    }
    (void)launch_pdl(colsum_kernel, dim3(kColsumChunks, groups, n_jobs + (slices ? 1 : 0)), dim3(256), 0, st, jobs, n_jobs, sl,
                     out_base, out_group_stride, partial, ticket, am ? *am : AgentMap{});
    return cudaGetLastError();
}

}  // namespace gala
