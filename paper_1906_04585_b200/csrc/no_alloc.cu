// Split-K grouped GEMM for callers that must not allocate device memory.
//
// gala_gemm_bf16 takes its scratch (split-K partial sums and an error word) from cudaMalloc and
// gives it back with cudaFree.  Both calls synchronise the whole device and can fail outright when
// another component owns the free memory -- typically a framework's caching allocator that has
// already reserved nearly all of HBM, or a serving loop with a fixed memory plan and a latency
// budget that a device-wide stall would break.  For those callers the scratch lives here, in a
// fixed array that is part of the library image: every GPU that loads the library carries it from
// load to exit, and no allocation routine of any kind is called.
#include <cstdarg>
#include <cstdio>
#include <cstring>

#include "internal.h"

using namespace gala;

namespace {

constexpr long kStaticScratchFloats = 2L * 1024 * 1024;  // 8 MiB of partial sums
constexpr int kHeaderFloats = 64;                        // first 256 bytes: error word (+ padding)
constexpr int kMaxDevices = 64;

// Inside device code this name is the array.  In host code it is only a handle for the runtime's
// symbol calls; the device address has to be asked for (once per device).
static __device__ __align__(256) float g_static_scratch[kHeaderFloats + kStaticScratchFloats];

float* g_scratch_addr[kMaxDevices] = {};

void say(char* buf, int len, const char* fmt, ...) {
    if (!buf || len <= 0) return;
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, (size_t)len, fmt, ap);
    va_end(ap);
}

}  // namespace

extern "C" int gala_gemm_bf16_static(const void* A, const void* B, float* D, int groups, int M, int N, int K,
                                     int a_mn, int b_mn, int split_k, void* stream, char* errbuf, int errbuf_len) {
    if (errbuf && errbuf_len > 0) errbuf[0] = 0;
    if (!A || !B || !D || groups < 1 || M < 1 || N < 1 || K < 1 || split_k < 1) {
        say(errbuf, errbuf_len, "gala_gemm_bf16_static: null pointer or non-positive size");
        return GALA_EINVAL;
    }
    if ((K % 8) || (a_mn && (M % 8)) || (b_mn && (N % 8))) {
        say(errbuf, errbuf_len, "gala_gemm_bf16_static: rows must be 16-byte aligned (K, and M or N when stored "
                                "[K][.], multiples of 8)");
        return GALA_EINVAL;
    }
    const long count = (long)M * N;
    const long need = split_k > 1 ? (long)groups * split_k * count : 0;
    if (need > kStaticScratchFloats) {
        say(errbuf, errbuf_len, "gala_gemm_bf16_static: groups*split_k*M*N = %ld floats of partial sums exceed the "
                                "built-in scratch of %ld floats (8 MiB); lower split_k or use gala_gemm_bf16",
            need, kStaticScratchFloats);
        return GALA_EINVAL;
    }
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        say(errbuf, errbuf_len, "gala_gemm_bf16_static: cudaGetDevice: %s", cudaGetErrorString(e));
        return GALA_ECUDA;
    }
    if (!g_scratch_addr[dev]) {  // set-up, once per device, with that device current
        float* p = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
        if (e != cudaSuccess || !p) {
            say(errbuf, errbuf_len, "gala_gemm_bf16_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
            return GALA_ECUDA;
        }
        g_scratch_addr[dev] = p;
    }
    if (gemm_init() != cudaSuccess) {   // encoder once per process, shared-memory opt-in once per device
        say(errbuf, errbuf_len, "gala_gemm_bf16_static: tensor-map encoder not available from the driver");
        return GALA_ECUDA;
    }
    float* scratch = g_scratch_addr[dev];
    int* err = reinterpret_cast<int*>(scratch);
    float* ws = scratch + kHeaderFloats;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    const int bn = N >= 512 ? 256 : b_mn ? (N > 64 ? 128 : 64) : (N > 64 ? 128 : (N > 32 ? 64 : 32));
    GemmOperand oa, ob;
    if (!make_operand(&oa, A, a_mn, M, K, groups, a_mn ? M : K, (uint64_t)M * K, 128) ||
        !make_operand(&ob, B, b_mn, N, K, groups, b_mn ? N : K, (uint64_t)N * K, bn)) {
        say(errbuf, errbuf_len, "gala_gemm_bf16_static: operand pointers must be 16-byte aligned");
        return GALA_EINVAL;
    }
    // the array keeps whatever the previous call left: the error word must start at zero; the
    // partial sums need no clearing because every split writes all of its M x N block
    if ((e = cudaMemsetAsync(err, 0, sizeof(int), st)) != cudaSuccess) {
        say(errbuf, errbuf_len, "gala_gemm_bf16_static: cudaMemsetAsync: %s", cudaGetErrorString(e));
        return GALA_ECUDA;
    }
    GemmArgs a;
    memset(&a, 0, sizeof a);
    a.M = M; a.N = N; a.K = K; a.block_n = bn; a.groups = groups; a.split_k = split_k; a.scale = 1.0f;
    a.ldc = N; a.error_word = err;
    if (split_k == 1) {
        a.out = D; a.out_group_stride = count;
        e = launch_gemm(oa, ob, a, st);
    } else {
        a.out = ws; a.out_group_stride = (long)split_k * count; a.out_split_stride = count;
        e = launch_gemm(oa, ob, a, st);
        if (e == cudaSuccess)
            e = launch_splitk_reduce(ws, D, count, split_k, count, groups, (long)split_k * count, count, st);
    }
    if (e != cudaSuccess) {
        say(errbuf, errbuf_len, "gala_gemm_bf16_static: launch failed: %s", cudaGetErrorString(e));
        return GALA_ECUDA;
    }
    // the error word comes back on the caller's stream, so that the one wait below is for this call's work only
    int w = 0;
    if ((e = cudaMemcpyAsync(&w, err, sizeof w, cudaMemcpyDeviceToHost, st)) == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess || w) {
        say(errbuf, errbuf_len, "gala_gemm_bf16_static: %s",
            e != cudaSuccess ? cudaGetErrorString(e) : "a bounded device-side wait ran out");
        return GALA_ECUDA;
    }
    return GALA_OK;
}
