// Device helpers shared by the statistics and step kernels: vector loads and
// stores with streaming cache hints, bf16 unpacking, deterministic CTA
// reductions, and the 8-bit block-wise absmax code arithmetic.
#pragma once

#include <cstdint>
#include <cuda_runtime.h>

#include "baoc_internal.h"
#include "baoc_check.cuh"

namespace baoc {

__device__ __forceinline__ int64_t min64(int64_t a, int64_t b) { return a < b ? a : b; }
__device__ __forceinline__ int64_t max64(int64_t a, int64_t b) { return a > b ? a : b; }

// ---- 128-bit streaming loads / stores ---------------------------------------
// Every array on this path is touched once per launch, so loads bypass L1
// allocation and stores are marked evict-first.

__device__ __forceinline__ uint4 ld_stream_u4(const void* p) {
    uint4 r;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ float4 ld_stream_f4(const void* p) {
    float4 r;
    asm volatile("ld.global.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(p));
    return r;
}
// 256-bit forms (sm_100): one request for a thread's eight fp32 values.  The address must be 32-byte aligned: true for
// every tensor of the bound workspace and state buffer at an element index that is a multiple of eight; caller-owned
// arrays promise 16 bytes only.
__device__ __forceinline__ void ld_stream_f8(const void* p, float4& a, float4& b) {
    asm volatile("ld.global.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(a.x), "=f"(a.y), "=f"(a.z), "=f"(a.w), "=f"(b.x), "=f"(b.y), "=f"(b.z), "=f"(b.w) : "l"(p));
}
__device__ __forceinline__ void ld_stream_u8(const void* p, uint32_t (&x)[8]) {
    asm volatile("ld.global.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3]), "=r"(x[4]), "=r"(x[5]), "=r"(x[6]), "=r"(x[7]) : "l"(p));
}
__device__ __forceinline__ void st_stream_f8(void* p, const float (&x)[8]) {
    asm volatile("st.global.cs.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "f"(x[0]), "f"(x[1]), "f"(x[2]), "f"(x[3]),
                 "f"(x[4]), "f"(x[5]), "f"(x[6]), "f"(x[7]) : "memory");
}
__device__ __forceinline__ uint2 ld_stream_u2(const void* p) {
    uint2 r;
    asm volatile("ld.global.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p));
    return r;
}
// A load that stays where it is written: the compiler may neither delay it to its first use nor repeat it there.  For
// values fetched well ahead of their use (a register prefetch), where sinking the load would expose its full latency.
__device__ __forceinline__ float ld_pinned_f32(const float* p) {
    float v;
    asm volatile("ld.global.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream_f4(void* p, float4 v) {
    asm volatile("st.global.cs.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void st_stream_u4(void* p, uint4 v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void st_stream_u2(void* p, uint2 v) {
    asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" ::"l"(p), "r"(v.x), "r"(v.y) : "memory");
}

// ---- asynchronous global -> shared copies (per-thread staging) ------------------
// A thread copies its own next operands into its own slot of shared memory and
// later reads that slot back itself, so the only synchronisation needed is the
// thread's own wait on its copy groups (a hardware wait, not a spin loop).
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// the same through L1 (a later copy of the neighbouring 16 bytes finds the sector there)
__device__ __forceinline__ void cp_async16_l1(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async8(uint32_t dst, const void* src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int kPending>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(kPending) : "memory"); }

// ---- bf16 ------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(uint32_t(b) << 16); }

// double -> fp32 -> bf16, round to nearest even at both roundings (non-finite values keep their upper half).
__device__ __forceinline__ uint16_t bf16_from_double(double x) {
    const float f = __double2float_rn(x);
    const uint32_t u = __float_as_uint(f);
    if ((u & 0x7f800000u) == 0x7f800000u) return uint16_t(u >> 16);
    return uint16_t((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
}

// Unpack 8 bf16 values held in a uint4 into floats.
__device__ __forceinline__ void unpack8(const uint4& w, float (&x)[8]) {
    x[0] = bf16_lo(w.x); x[1] = bf16_hi(w.x); x[2] = bf16_lo(w.y); x[3] = bf16_hi(w.y);
    x[4] = bf16_lo(w.z); x[5] = bf16_hi(w.z); x[6] = bf16_lo(w.w); x[7] = bf16_hi(w.w);
}

// Two float4 as an array of eight floats.
__device__ __forceinline__ void f4_to8(const float4& a, const float4& b, float (&x)[8]) {
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}

// A float that holds a bf16 value, widened to double without a conversion
// instruction (the conversion pipe is narrow): re-bias the exponent with
// integer arithmetic.  Zeros, subnormals, infinities and NaNs take the
// ordinary conversion.
__device__ __forceinline__ double widen_bf16_float(float x) {
    const uint32_t u = __float_as_uint(x);
    const uint32_t e = u & 0x7f800000u;
    if (e == 0u || e == 0x7f800000u) return double(x);
    const uint32_t hi = (u & 0x80000000u) | (((u & 0x7fffffffu) >> 3) + (896u << 20));
    return __hiloint2double(int(hi), 0);
}

// Small integer (|q| < 2^31) to double, exact, without a conversion instruction.
__device__ __forceinline__ double int_to_double(int q) {
    return __hiloint2double(0x43300000, int(uint32_t(q) ^ 0x80000000u)) - 4503601774854144.0;   // 2^52 + 2^31
}
// Small integer (|q| < 2^22) to float, exact.
__device__ __forceinline__ float int_to_float(int q) {
    return __int_as_float(0x4B400000 + q) - 12582912.0f;                                         // 1.5 * 2^23
}
// Round a double of magnitude < 2^31 to the nearest integer, ties to even.
__device__ __forceinline__ int round_to_int(double x) {
    return __double2loint(x + 6755399441055744.0);                                               // 1.5 * 2^52
}

// ---- deterministic CTA reduction ---------------------------------------------
// Sums K values per thread over the CTA in a fixed order (butterfly inside a
// warp, then warps in index order) and lets thread 0 store the K results.
template <int K>
__device__ __forceinline__ void cta_reduce_store(double (&val)[K], double* out) {
    __shared__ double sh[kThreads / 32][K];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        double x = val[k];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        if (lane == 0) sh[warp][k] = x;
    }
    __syncthreads();
    if (threadIdx.x < K) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) s += sh[w][threadIdx.x];
        out[threadIdx.x] = s;
    }
    __syncthreads();
}

// Sum K doubles per tile slot over the tiles of one block in a fixed order: thread
// t takes tiles t, t+T, ..., then the CTA reduces.  out[K] per block.
template <int K>
__device__ __forceinline__ void block_tiles_sum(const double* __restrict__ part, int64_t tile0, int ntiles, double* out) {
    double acc[K];
#pragma unroll
    for (int k = 0; k < K; ++k) acc[k] = 0.0;
    // (four slots requested before the first is added: the order of the additions is unchanged)
#pragma unroll 4
    for (int i = threadIdx.x; i < ntiles; i += kThreads) {
        const double* p = part + size_t(tile0 + i) * K;
#pragma unroll
        for (int k = 0; k < K; ++k) acc[k] += p[k];
    }
    cta_reduce_store<K>(acc, out);
}

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}

// ---- packed fp32 pairs ---------------------------------------------------------
// sm_100 executes add / mul / fma on two fp32 values held in one 64-bit register
// with a single instruction; each half is rounded to nearest like the scalar form.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f32x2 splat2(float x) { return pack2(x, x); }
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// max(a, b, c) in one instruction
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// ---- approximate square root and reciprocal (one instruction each, relative error 2^-23, subnormals flushed) ----
__device__ __forceinline__ float sqrt_approx(float x) {
    float r;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float rcp_approx(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
// Warp maximum of non-negative floats (their bit patterns order like unsigned integers): one reduction instruction.
__device__ __forceinline__ float warp_max_nonneg(float x) {
    return __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(x)));
}

// ---- 8-bit block-wise absmax codes -----------------------------------------------
// code = clamp(rne(L * x / a)), x ~ code * a / L, with L = 127 (signed) or 255
// (unsigned) and a the fp32 absmax of the 256-element quantisation block.  The
// scaling and rounding are done in double so that the decision agrees with a
// double-precision evaluation of the same formula.  The fast path multiplies by
// the precomputed L / a; that product is within a few ulp of (L * x) / a, so the
// two can only round to different integers when the value sits on a tie.  bf16
// gradients make exact ties common (x / a is often a ratio of small integers),
// hence a value within 1e-9 of a half-integer is redone with the division, which
// is the correctly rounded form of the definition.
__device__ __forceinline__ double code_scale(float absmax, double levels) {
    return absmax > 0.0f ? levels / double(absmax) : 0.0;
}
__device__ __forceinline__ int encode_round(double x, float absmax, double scale, double levels) {
    constexpr double kMagic = 6755399441055744.0;                 // 1.5 * 2^52: adding it rounds to an integer, ties to even
    const double q = x * scale;
    const double t = q + kMagic;
    const double d = q - (t - kMagic);                            // signed distance to the chosen integer
    if (fabs(d) > 0.5 - 1e-9) return __double2loint((levels * x) / double(absmax) + kMagic);
    return __double2loint(t);
}
__device__ __forceinline__ int encode_signed(double x, float absmax, double scale) {
    return max(-127, min(127, encode_round(x, absmax, scale, 127.0)));
}
__device__ __forceinline__ int encode_unsigned(double x, float absmax, double scale) {
    return max(0, min(255, encode_round(x, absmax, scale, 255.0)));
}

// ---- the non-linear ("dynamic") 8-bit codebook ---------------------------------------
// Magnitudes 10^-E (0.1 + 0.9 (k+1) / 2^F), k < 2^F, F = B - 1 - E, E < B, with B = 7 value bits (signed) or 8
// (unsigned), and zero; a code is the index of the nearest entry in ascending order.  In ascending order the positive
// magnitude number p >= 1 has F = floor(log2 p), E = B - 1 - F, k = p - 2^F, so a CTA builds the tables in place.
struct DynTables {
    double ts[256], ms[256];     // signed entries (255 used) and the midpoints between neighbours (254 used), padded upwards
    double tu[256], mu[256];     // unsigned entries and their 255 midpoints
};
static __constant__ double kPow10[8] = {1.0, 1e-1, 1e-2, 1e-3, 1e-4, 1e-5, 1e-6, 1e-7};
__device__ __forceinline__ double dyn_magnitude(int p, int value_bits) {
    const double* p10 = kPow10;
    const int F = 31 - __clz(p), E = value_bits - 1 - F, k = p - (1 << F);
    const double frac = __dadd_rn(0.1, __dmul_rn(__dmul_rn(0.9, double(k + 1)), 1.0 / double(1 << F)));
    return __dmul_rn(p10[E], frac);
}
__device__ __forceinline__ void dyn_build(DynTables* T) {      // all kThreads = 256 threads of the CTA
    const int i = threadIdx.x;
    T->tu[i] = i == 0 ? 0.0 : dyn_magnitude(i, 8);
    T->ts[i] = i == 127 ? 0.0 : (i < 127 ? -dyn_magnitude(127 - i, 7) : (i < 255 ? dyn_magnitude(i - 127, 7) : 2.0));
    __syncthreads();
    T->mu[i] = i < 255 ? 0.5 * (T->tu[i] + T->tu[i + 1]) : 4.0;     // the padding is above every y in [-1, 1]
    T->ms[i] = i < 254 ? 0.5 * (T->ts[i] + T->ts[i + 1]) : 4.0;
    __syncthreads();
}
// Index of the entry nearest to y: the number of midpoints below y (a tie goes to the entry of smaller magnitude).
__device__ __forceinline__ int dyn_nearest(const double* mid, double y) {
    int lo = 0;
    const bool neg = y < 0.0;
#pragma unroll
    for (int step = 128; step > 0; step >>= 1) {
        const double m = mid[lo + step - 1];
        if (neg ? y >= m : y > m) lo += step;
    }
    return lo;
}
// The same tables in fp32 (for sums that are compared at 1e-4): ts, ms, tu, mu, 256 floats each.
__device__ __forceinline__ void dyn_build_f32(float* t4) {           // all kThreads = 256 threads of the CTA
    const int i = threadIdx.x;
    const double u0 = i == 0 ? 0.0 : dyn_magnitude(i, 8), u1 = i < 255 ? dyn_magnitude(i + 1, 8) : 8.0;
    auto sgn = [](int k) { return k == 127 ? 0.0 : (k < 127 ? -dyn_magnitude(127 - k, 7) : (k < 255 ? dyn_magnitude(k - 127, 7) : 8.0)); };
    const double s0 = sgn(i), s1 = sgn(i + 1 < 256 ? i + 1 : 255);
    t4[i] = float(s0); t4[256 + i] = i < 254 ? float(0.5 * (s0 + s1)) : 4.0f;
    t4[512 + i] = float(u0); t4[768 + i] = i < 255 ? float(0.5 * (u0 + u1)) : 4.0f;
    __syncthreads();
}
__device__ __forceinline__ int dyn_nearest_f32(const float* mid, float y) {
    int lo = 0;
    const bool neg = y < 0.f;
#pragma unroll
    for (int step = 128; step > 0; step >>= 1) {
        const float m = mid[lo + step - 1];
        if (neg ? y >= m : y > m) lo += step;
    }
    return lo;
}

}  // namespace baoc
