// baoc_sample_stats_noalloc: one gradient observation of ONE block without any
// allocation and without a handle.
//
// Some callers may not allocate device memory at the moment they need the
// statistics: code that runs inside a framework's allocator hook or memory-
// pressure callback, a training loop that has handed every free byte to its
// caching allocator and must not trigger a cudaMalloc (which synchronises the
// device and can fail), or a host runtime that simply has no allocator to lend a
// workspace from.  The handle-based path needs a caller-provided workspace for
// its tables and per-tile partial sums; this variant keeps the partial sums in a
// fixed array that is part of the library image instead.
//
// The arithmetic is that of the per-step statistics kernel (Eq. 3 and the sums
// behind the cosine of Eq. 5); only the bookkeeping differs.
#include <cmath>
#include <cuda_runtime.h>
#include <mutex>
#include <string>

#include "baoc_device.cuh"

namespace baoc {

constexpr int kNoAllocPartials = 5;                         // doubles per tile
constexpr int64_t kNoAllocMaxTiles = BAOC_NOALLOC_MAX_NUMEL / kTile;

// Per-tile partial sums of the current call.  Every GPU that loads the library
// holds these 640 KB until the process exits; every call on a device shares them.
static __device__ __align__(256) double g_noalloc_partials[kNoAllocMaxTiles * kNoAllocPartials];

__device__ __forceinline__ float ema1(float s, float x, float one_minus_beta) { return fmaf(one_minus_beta, x - s, s); }

// One CTA per tile of kTile elements.  Reads g_t, g_{t-1} (bf16), m, v (fp32);
// writes m, v, g_{t-1}; leaves 5 partial sums in the tile's slot of the scratch:
// <g_t, g_{t-1}>, ||g_t||^2, <g_t, m_{t-1}>, ||m_{t-1}||^2, ||g_{t-1}||^2.
__global__ void __launch_bounds__(kThreads)
stats_step_single_kernel(const uint16_t* __restrict__ g, uint16_t* __restrict__ gp, float* __restrict__ m,
                         float* __restrict__ v, int64_t numel, float om, float ov, double* __restrict__ partials) {
    const int64_t base = int64_t(blockIdx.x) * kTile;
    float a_dot = 0.f, a_n2 = 0.f, a_dm = 0.f, a_m2 = 0.f, a_p2 = 0.f;
    constexpr int kSlices = kTile / (kThreads * 8);
#pragma unroll
    for (int s = 0; s < kSlices; ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        if (e + 8 <= numel) {
            float x[8], p[8];
            const uint4 wg = ld_stream_u4(g + e);
            unpack8(wg, x);
            unpack8(ld_stream_u4(gp + e), p);
            const float4 m0 = ld_stream_f4(m + e), m1 = ld_stream_f4(m + e + 4);
            const float4 v0 = ld_stream_f4(v + e), v1 = ld_stream_f4(v + e + 4);
            float mm[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
            float vv[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                a_dot = fmaf(x[j], p[j], a_dot);
                a_n2 = fmaf(x[j], x[j], a_n2);
                a_dm = fmaf(x[j], mm[j], a_dm);
                a_m2 = fmaf(mm[j], mm[j], a_m2);
                a_p2 = fmaf(p[j], p[j], a_p2);
                mm[j] = ema1(mm[j], x[j], om);
                vv[j] = ema1(vv[j], x[j] * x[j], ov);
            }
            st_stream_f4(m + e, make_float4(mm[0], mm[1], mm[2], mm[3]));
            st_stream_f4(m + e + 4, make_float4(mm[4], mm[5], mm[6], mm[7]));
            st_stream_f4(v + e, make_float4(vv[0], vv[1], vv[2], vv[3]));
            st_stream_f4(v + e + 4, make_float4(vv[4], vv[5], vv[6], vv[7]));
            st_stream_u4(gp + e, wg);
        } else if (e < numel) {
            const int cnt = int(numel - e);
            for (int j = 0; j < cnt; ++j) {
                const uint16_t gb = g[e + j];
                const float x = bf16_bits_to_float(gb), p = bf16_bits_to_float(gp[e + j]);
                const float mm = m[e + j], vv = v[e + j];
                a_dot = fmaf(x, p, a_dot); a_n2 = fmaf(x, x, a_n2);
                a_dm = fmaf(x, mm, a_dm); a_m2 = fmaf(mm, mm, a_m2); a_p2 = fmaf(p, p, a_p2);
                m[e + j] = ema1(mm, x, om);
                v[e + j] = ema1(vv, x * x, ov);
                gp[e + j] = gb;
            }
        }
    }
    double acc[kNoAllocPartials] = {double(a_dot), double(a_n2), double(a_dm), double(a_m2), double(a_p2)};
    cta_reduce_store<kNoAllocPartials>(acc, partials + size_t(blockIdx.x) * kNoAllocPartials);
}

// One CTA: add the tiles' partial sums in a fixed order and write
// out[0] = cos(g_t, g_{t-1}), out[1] = ||g_t||^2, out[2] = cos(g_t, m_{t-1}), out[3] = ||m_{t-1}||^2,
// with the cosine <a,b> / (||a|| ||b|| + eps) and a non-finite cosine counted as 0.
__global__ void __launch_bounds__(kThreads)
stats_single_combine_kernel(const double* __restrict__ partials, int ntiles, double eps, double* __restrict__ out) {
    __shared__ double s[kNoAllocPartials];
    double acc[kNoAllocPartials] = {0.0, 0.0, 0.0, 0.0, 0.0};
    for (int i = threadIdx.x; i < ntiles; i += kThreads) {
        const double* p = partials + size_t(i) * kNoAllocPartials;
#pragma unroll
        for (int k = 0; k < kNoAllocPartials; ++k) acc[k] += p[k];
    }
    cta_reduce_store<kNoAllocPartials>(acc, s);
    if (threadIdx.x == 0) {
        const double c0 = s[0] / (sqrt(s[1]) * sqrt(s[4]) + eps);
        const double c1 = s[2] / (sqrt(s[1]) * sqrt(s[3]) + eps);
        out[0] = isfinite(c0) ? c0 : 0.0;
        out[1] = s[1];
        out[2] = isfinite(c1) ? c1 : 0.0;
        out[3] = s[3];
    }
}

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_mu;
double* g_scratch_addr[kMaxDevices] = {};       // device address of g_noalloc_partials, per device
thread_local std::string g_err;

int fail_na(int code, const std::string& msg) {
    g_err = msg;
    return code;
}

}  // namespace
}  // namespace baoc

using namespace baoc;

extern "C" {

const char* baoc_noalloc_last_error(void) { return g_err.c_str(); }

int baoc_sample_stats_noalloc(const void* grad_bf16, void* gprev_bf16, float* m, float* v, int64_t numel,
                              double beta_m, double beta_v, double eps, double* out4, baoc_stream_t stream) {
    if (!grad_bf16 || !gprev_bf16 || !m || !v || !out4) return fail_na(BAOC_E_INVALID, "baoc_sample_stats_noalloc: null pointer");
    if (numel < 1) return fail_na(BAOC_E_INVALID, "baoc_sample_stats_noalloc: numel must be at least 1");
    if (numel > int64_t(BAOC_NOALLOC_MAX_NUMEL))
        return fail_na(BAOC_E_WORKSPACE, "baoc_sample_stats_noalloc: numel exceeds BAOC_NOALLOC_MAX_NUMEL (" +
                                             std::to_string(int64_t(BAOC_NOALLOC_MAX_NUMEL)) +
                                             " elements, the capacity of the built-in scratch); use the handle-based path");
    if (!(beta_m >= 0 && beta_m < 1 && beta_v >= 0 && beta_v < 1 && eps >= 0))
        return fail_na(BAOC_E_INVALID, "baoc_sample_stats_noalloc: coefficients out of range");
    const uintptr_t bits = reinterpret_cast<uintptr_t>(grad_bf16) | reinterpret_cast<uintptr_t>(gprev_bf16) |
                           reinterpret_cast<uintptr_t>(m) | reinterpret_cast<uintptr_t>(v);
    if (bits & 15u) return fail_na(BAOC_E_ALIGN, "baoc_sample_stats_noalloc: array not 16-byte aligned");
    if (reinterpret_cast<uintptr_t>(out4) & 7u) return fail_na(BAOC_E_ALIGN, "baoc_sample_stats_noalloc: out4 not 8-byte aligned");

    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_na(BAOC_E_CUDA, std::string("cudaGetDevice: ") + cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return fail_na(BAOC_E_INVALID, "baoc_sample_stats_noalloc: device index out of range");
    double* scratch = nullptr;
    {
        // Set-up, once per device, with that device current: in host code the
        // array's name is only a stand-in, so ask the runtime for its address.
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_scratch_addr[dev]) {
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_noalloc_partials);
            if (e != cudaSuccess) return fail_na(BAOC_E_CUDA, std::string("cudaGetSymbolAddress: ") + cudaGetErrorString(e));
            g_scratch_addr[dev] = static_cast<double*>(p);
        }
        scratch = g_scratch_addr[dev];
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int ntiles = int((numel + kTile - 1) / kTile);
    stats_step_single_kernel<<<unsigned(ntiles), kThreads, 0, s>>>(
        static_cast<const uint16_t*>(grad_bf16), static_cast<uint16_t*>(gprev_bf16), m, v, numel, float(1.0 - beta_m),
        float(1.0 - beta_v), scratch);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail_na(BAOC_E_CUDA, std::string("stats_step_single_kernel: ") + cudaGetErrorString(e));
    stats_single_combine_kernel<<<1, kThreads, 0, s>>>(scratch, ntiles, eps, out4);
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail_na(BAOC_E_CUDA, std::string("stats_single_combine_kernel: ") + cudaGetErrorString(e));
    return BAOC_OK;
}

}  // extern "C"
