// Convolution lowering for the 84x84x4 -> 20x20x32 -> 9x9x64 -> 7x7x64 trunk (Appendix C.2
// network): patch matrices for the tensor-core GEMMs, their adjoint (scatter of patch gradients
// back onto the input grid), and bias gradients.  All tensors are NHWC, patch columns are
// ordered (kh, kw, cin) like the weights, so one kernel row of a patch is one contiguous run
// of k*cin elements of the input.
#include "internal.h"

namespace gala {

struct ConvGeom { int in, out, k, s, cin; };
__host__ __device__ inline ConvGeom conv_geom(int layer) {
    ConvGeom g;
    g.in = layer == 0 ? 84 : (layer == 1 ? 20 : 9);
    g.out = layer == 0 ? 20 : (layer == 1 ? 9 : 7);
    g.k = layer == 0 ? 8 : (layer == 1 ? 4 : 3);
    g.s = layer == 0 ? 4 : (layer == 1 ? 2 : 1);
    g.cin = layer == 0 ? 4 : (layer == 1 ? 32 : 64);
    return g;
}

// uint8 frames -> bf16 patch rows [sample*400 + oy*20 + ox][ky][kx][c] (256 wide).  One thread
// converts one kernel row of one patch: 32 contiguous bytes in, 64 contiguous bytes out.  Values
// 0..255 are exact in bf16; the 1/255 scale is applied after the contraction.
__global__ void __launch_bounds__(256) im2col_u8_kernel(PtrBatch obs, __nv_bfloat16* __restrict__ cols,
                                                        long cols_group_stride, int samples) {
    const int g = blockIdx.y;
    const uint8_t* src = reinterpret_cast<const uint8_t*>(obs.p[g]);
    __nv_bfloat16* dst = cols + (long)g * cols_group_stride;
    const long total = (long)samples * 400 * 8;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int ky = (int)(idx & 7);
        const long patch = idx >> 3;
        const int b = (int)(patch / 400), pp = (int)(patch % 400);
        const int oy = pp / 20, ox = pp % 20;
        const uint8_t* s = src + ((long)b * 84 * 84 + (long)(oy * 4 + ky) * 84 + ox * 4) * 4;
        const uint4 lo = __ldg(reinterpret_cast<const uint4*>(s));
        const uint4 hi = __ldg(reinterpret_cast<const uint4*>(s) + 1);
        const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
        uint4* d = reinterpret_cast<uint4*>(dst + patch * 256 + ky * 32);
#pragma unroll
        for (int q = 0; q < 4; q++) {
            uint32_t o[4];
#pragma unroll
            for (int h = 0; h < 2; h++) {
                const uint32_t v = w[q * 2 + h];
                __nv_bfloat162 p0 = __floats2bfloat162_rn((float)(v & 255u), (float)((v >> 8) & 255u));
                __nv_bfloat162 p1 = __floats2bfloat162_rn((float)((v >> 16) & 255u), (float)(v >> 24));
                o[h * 2] = *reinterpret_cast<uint32_t*>(&p0);
                o[h * 2 + 1] = *reinterpret_cast<uint32_t*>(&p1);
            }
            d[q] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}
cudaError_t launch_im2col_u8(const PtrBatch& obs, __nv_bfloat16* cols, long cols_group_stride, int samples,
                             int groups, cudaStream_t st) {
    long total = (long)samples * 400 * 8;
    int bx = (int)((total + 255) / 256);
    if (bx > 148 * 16) bx = 148 * 16;
    im2col_u8_kernel<<<dim3(bx, groups), 256, 0, st>>>(obs, cols, cols_group_stride, samples);
    return cudaGetLastError();
}

// uint8 frames -> bf16 frames (0..255 are exact in bf16; the 1/255 scale is applied after the
// contraction).  16 bytes in, 32 bytes out per thread and step.
__global__ void __launch_bounds__(256) cast_frames_kernel(PtrBatch obs, __nv_bfloat16* __restrict__ out, long out_group_stride,
                                                          long n16) {
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
    if (bx > 148 * 8) bx = 148 * 8;
    cast_frames_kernel<<<dim3(bx, groups), 256, 0, st>>>(obs, out, out_group_stride, n16);
    return cudaGetLastError();
}

// bf16 NHWC activations -> bf16 patch rows, 16 bytes per thread per step.
__global__ void __launch_bounds__(256) im2col_bf16_kernel(const __nv_bfloat16* __restrict__ act, long act_group_stride,
                                                          __nv_bfloat16* __restrict__ cols, long cols_group_stride,
                                                          int layer, int samples) {
    const ConvGeom cg = conv_geom(layer);
    const int g = blockIdx.y;
    const uint4* src = reinterpret_cast<const uint4*>(act + (long)g * act_group_stride);
    uint4* dst = reinterpret_cast<uint4*>(cols + (long)g * cols_group_stride);
    const int row_chunks = cg.k * cg.cin / 8;           // 16-byte chunks in one kernel row of a patch
    const int patch_chunks = row_chunks * cg.k;
    const int pix_chunks = cg.cin / 8;
    const int P = cg.out * cg.out;
    const long total = (long)samples * P * patch_chunks;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int c = (int)(idx % patch_chunks);
        const long patch = idx / patch_chunks;
        const int ky = c / row_chunks, cr = c % row_chunks;
        const int b = (int)(patch / P), pp = (int)(patch % P);
        const int oy = pp / cg.out, ox = pp % cg.out;
        const long s = ((long)b * cg.in * cg.in + (long)(oy * cg.s + ky) * cg.in + ox * cg.s) * pix_chunks + cr;
        dst[idx] = __ldg(src + s);
    }
}
cudaError_t launch_im2col_bf16(const __nv_bfloat16* act, long act_group_stride, __nv_bfloat16* cols,
                               long cols_group_stride, int layer, int samples, int groups, cudaStream_t st) {
    const ConvGeom cg = conv_geom(layer);
    long total = (long)samples * cg.out * cg.out * (cg.k * cg.k * cg.cin / 8);
    int bx = (int)((total + 255) / 256);
    if (bx > 148 * 16) bx = 148 * 16;
    im2col_bf16_kernel<<<dim3(bx, groups), 256, 0, st>>>(act, act_group_stride, cols, cols_group_stride, layer, samples);
    return cudaGetLastError();
}

// Adjoint of the lowering, gather form: every input pixel sums the fp32 patch-gradient entries
// that were copied from it, in a fixed order, then the ReLU derivative of that pixel's forward
// activation is applied and the result is stored in bf16.  One thread per (pixel, 8 channels).
__global__ void __launch_bounds__(256) col2im_kernel(const float* __restrict__ dcols, long dcols_group_stride,
                                                     const __nv_bfloat16* __restrict__ act_in, long act_group_stride,
                                                     __nv_bfloat16* __restrict__ dx, long dx_group_stride, int layer,
                                                     int samples) {
    const ConvGeom cg = conv_geom(layer);
    const int g = blockIdx.y;
    const float4* src = reinterpret_cast<const float4*>(dcols + (long)g * dcols_group_stride);
    const uint4* act = reinterpret_cast<const uint4*>(act_in + (long)g * act_group_stride);
    uint4* dst = reinterpret_cast<uint4*>(dx + (long)g * dx_group_stride);
    const int pix_chunks = cg.cin / 8;
    const int row_chunks = cg.k * pix_chunks;
    const int patch_chunks = row_chunks * cg.k;
    const int P = cg.out * cg.out;
    const long total = (long)samples * cg.in * cg.in * pix_chunks;
    for (long idx = blockIdx.x * (long)blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const int cc = (int)(idx % pix_chunks);
        const long pix = idx / pix_chunks;
        const int b = (int)(pix / (cg.in * cg.in)), rem = (int)(pix % (cg.in * cg.in));
        const int y = rem / cg.in, x = rem % cg.in;
        float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int ky = y % cg.s; ky < cg.k; ky += cg.s) {
            const int oy = (y - ky) / cg.s;
            if (y - ky < 0) break;
            if (oy >= cg.out) continue;
            for (int kx = x % cg.s; kx < cg.k; kx += cg.s) {
                const int ox = (x - kx) / cg.s;
                if (x - kx < 0) break;
                if (ox >= cg.out) continue;
                const long patch = (long)b * P + oy * cg.out + ox;
                const float4* v = src + (patch * patch_chunks + ky * row_chunks + kx * pix_chunks + cc) * 2;
                const float4 v0 = __ldg(v), v1 = __ldg(v + 1);
                acc[0] += v0.x; acc[1] += v0.y; acc[2] += v0.z; acc[3] += v0.w;
                acc[4] += v1.x; acc[5] += v1.y; acc[6] += v1.z; acc[7] += v1.w;
            }
        }
        const uint4 a = __ldg(act + idx);
        const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a);
        uint32_t o[4];
#pragma unroll
        for (int q = 0; q < 4; q++) {
            float2 f = __bfloat1622float2(ah[q]);
            __nv_bfloat162 r = __floats2bfloat162_rn(f.x > 0.0f ? acc[2 * q] : 0.0f, f.y > 0.0f ? acc[2 * q + 1] : 0.0f);
            o[q] = *reinterpret_cast<uint32_t*>(&r);
        }
        dst[idx] = make_uint4(o[0], o[1], o[2], o[3]);
    }
}
cudaError_t launch_col2im(const float* dcols, long dcols_group_stride, const __nv_bfloat16* act_in,
                          long act_group_stride, __nv_bfloat16* dx, long dx_group_stride, int layer, int samples,
                          int groups, cudaStream_t st) {
    const ConvGeom cg = conv_geom(layer);
    long total = (long)samples * cg.in * cg.in * (cg.cin / 8);
    int bx = (int)((total + 255) / 256);
    if (bx > 148 * 16) bx = 148 * 16;
    col2im_kernel<<<dim3(bx, groups), 256, 0, st>>>(dcols, dcols_group_stride, act_in, act_group_stride, dx,
                                                    dx_group_stride, layer, samples);
    return cudaGetLastError();
}

// Bias gradient: out[c] = sum over rows of dy[row][c].  Rows are cut into kColsumChunks fixed
// chunks (one block each).  Inside a block a thread owns 8 adjacent columns (one 16-byte load per
// row) and every (256*8/C)-th row of the chunk; the row lanes are combined in index order, and the
// block that finishes last adds the chunk sums in index order, so the result does not depend on
// scheduling.  C is a power of two, 8 <= C <= 512.
// Up to kColsumJobs tensors are reduced by one launch (blockIdx.z picks the tensor).
__global__ void __launch_bounds__(256) colsum_kernel(ColsumJobs jobs, float* __restrict__ out_base, long out_group_stride,
                                                     double* partial_base, unsigned* ticket_base) {
    const int g = blockIdx.y;
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
    __shared__ float red[256 * 8];
    __shared__ bool last;
    double* part = partial + (long)g * kColsumJobs * kColsumChunks * 512 + (long)blockIdx.x * C;
    const int cchunks = C / 8;                    // 16-byte column groups per row
    const int lanes = 256 / cchunks > 0 ? 256 / cchunks : 1;   // row lanes (C <= 512 -> cchunks <= 64)
    const int cc = threadIdx.x % cchunks, rl = threadIdx.x / cchunks;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (rl < lanes) {
        for (long r = lo + rl; r < hi; r += lanes) {
            const uint4 v = __ldg(src + r * cchunks + cc);
            const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
            for (int q = 0; q < 4; q++) {
                const float2 f = __bfloat1622float2(h[q]);
                acc[2 * q] += f.x; acc[2 * q + 1] += f.y;
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
                          unsigned* ticket, int groups, cudaStream_t st) {
    if (n_jobs < 1 || n_jobs > kColsumJobs) return cudaErrorInvalidValue;
    for (int i = 0; i < n_jobs; i++) {
        const int C = jobs.j[i].C;
        if (C > 512 || C < 8 || (C & (C - 1))) return cudaErrorInvalidValue;
    }
    colsum_kernel<<<dim3(kColsumChunks, groups, n_jobs), 256, 0, st>>>(jobs, out_base, out_group_stride, partial, ticket);
    return cudaGetLastError();
}

}  // namespace gala
