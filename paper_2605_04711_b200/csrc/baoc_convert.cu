// State migration for an online re-configuration (Sec. 3.1, remark on re-planning; appendix study of online
// re-allocation with optimizer-state inheritance): a moment held under the old configuration is re-stored in the form
// the new configuration keeps.  Values are decoded and re-encoded in double, so the stored result is the correctly
// rounded one whatever the pair of precisions; the kernels run once per re-configuration and are not tuned.
#include "baoc_device.cuh"

namespace baoc {

// Decode element e of a stored moment.
__device__ __forceinline__ double moment_at(const MomentRef& s, int64_t e, double inv_mean_r) {
    switch (s.kind) {
        case kMomF32: {
            const double x = double(static_cast<const float*>(s.data)[e]);
            return s.divisor != 0.0 ? x / s.divisor : x;
        }
        case kMomBF16: return double(bf16_bits_to_float(static_cast<const uint16_t*>(s.data)[e]));
        case kMomI8: return (double(static_cast<const int8_t*>(s.data)[e]) * double(s.absmax[e / kQBlock])) / 127.0;
        case kMomU8: return (double(static_cast<const uint8_t*>(s.data)[e]) * double(s.absmax[e / kQBlock])) / 255.0;
        case kMomFactored: {
            const int64_t row = e / s.cols;
            const int col = int(e - row * s.cols);
            return double(s.r[row]) * double(s.c[col]) * inv_mean_r;
        }
        default: return 0.0;
    }
}

// 1 / mean(r) of a factored source, summed in a fixed order by the whole CTA (0 when the mean is 0).
__device__ __forceinline__ double inv_mean_of_rows(const MomentRef& s) {
    __shared__ double total[1];
    double local[1] = {0.0};
    for (int i = threadIdx.x; i < s.rows; i += kThreads) local[0] += double(s.r[i]);
    cta_reduce_store<1>(local, total);
    const double mean = total[0] / double(s.rows);
    return mean != 0.0 ? 1.0 / mean : 0.0;
}

__device__ __forceinline__ uint16_t bf16_from_double(double x) {
    const float f = __double2float_rn(x);
    const uint32_t u = __float_as_uint(f);
    if ((u & 0x7f800000u) == 0x7f800000u) return uint16_t(u >> 16);
    return uint16_t((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
}

// Element-wise source -> element-wise destination.  A warp owns one 256-element quantisation block per pass.
__global__ void __launch_bounds__(kThreads)
convert_moment_kernel(const MomentRef src, const MomentRef dst, int64_t numel) {
    const double inv_mean_r = src.kind == kMomFactored ? inv_mean_of_rows(src) : 0.0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t w0 = (int64_t(blockIdx.x) * (kThreads / 32) + warp) * kQBlock;
    if (w0 >= numel) return;
    double x[8];
    float amax = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int64_t e = w0 + lane * 8 + j;
        x[j] = e < numel ? moment_at(src, e, inv_mean_r) : 0.0;
        amax = fmaxf(amax, __double2float_rn(fabs(x[j])));          // rounding is monotone: max of roundings = rounding of max
    }
    const bool to_codes = dst.kind == kMomI8 || dst.kind == kMomU8;
    if (to_codes) amax = warp_max(amax);
    const double levels = dst.kind == kMomI8 ? 127.0 : 255.0;
    const double scale = code_scale(amax, levels);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int64_t e = w0 + lane * 8 + j;
        if (e >= numel) continue;
        switch (dst.kind) {
            case kMomF32: static_cast<float*>(dst.data)[e] = __double2float_rn(x[j]); break;
            case kMomBF16: static_cast<uint16_t*>(dst.data)[e] = bf16_from_double(x[j]); break;
            case kMomI8: static_cast<int8_t*>(dst.data)[e] = int8_t(encode_signed(x[j], amax, scale)); break;
            case kMomU8: static_cast<uint8_t*>(dst.data)[e] = uint8_t(encode_unsigned(x[j], amax, scale)); break;
            default: break;
        }
    }
    if (to_codes && lane == 0) dst.absmax[w0 / kQBlock] = amax;
}

// Element-wise second moment -> factored: r_i = mean over the row, c_j = mean over the column.
__global__ void __launch_bounds__(kThreads)
factor_rows_kernel(const MomentRef src, float* __restrict__ r) {
    __shared__ double total[1];
    const int64_t row = blockIdx.x;
    double local[1] = {0.0};
    for (int j = threadIdx.x; j < src.cols; j += kThreads) local[0] += moment_at(src, row * src.cols + j, 0.0);
    cta_reduce_store<1>(local, total);
    if (threadIdx.x == 0) r[row] = __double2float_rn(total[0] / double(src.cols));
}

__global__ void __launch_bounds__(kThreads)
factor_cols_kernel(const MomentRef src, float* __restrict__ c) {
    const int col = blockIdx.x * kThreads + threadIdx.x;
    if (col >= src.cols) return;
    double s = 0.0;
    for (int64_t i = 0; i < src.rows; ++i) s += moment_at(src, i * src.cols + col, 0.0);
    c[col] = __double2float_rn(s / double(src.rows));
}

// Factored -> factored (same shape): plain copies.
__global__ void copy_floats_kernel(const float* __restrict__ a, float* __restrict__ b, int64_t n) {
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < n) b[i] = a[i];
}

#define BAOC_LAUNCH_CHECK()                                   \
    do {                                                      \
        cudaError_t e_ = cudaGetLastError();                  \
        if (e_ != cudaSuccess) return int(e_);                \
    } while (0)

int launch_convert_moment(const MomentRef& src, const MomentRef& dst, int64_t numel, cudaStream_t s) {
    if (dst.kind == kMomFactored) {
        if (src.kind == kMomFactored) {
            copy_floats_kernel<<<unsigned((src.rows + 255) / 256), 256, 0, s>>>(src.r, const_cast<float*>(dst.r), src.rows);
            BAOC_LAUNCH_CHECK();
            copy_floats_kernel<<<unsigned((src.cols + 255) / 256), 256, 0, s>>>(src.c, const_cast<float*>(dst.c), src.cols);
            BAOC_LAUNCH_CHECK();
            return 0;
        }
        factor_rows_kernel<<<unsigned(src.rows), kThreads, 0, s>>>(src, const_cast<float*>(dst.r));
        BAOC_LAUNCH_CHECK();
        factor_cols_kernel<<<unsigned((src.cols + kThreads - 1) / kThreads), kThreads, 0, s>>>(src, const_cast<float*>(dst.c));
        BAOC_LAUNCH_CHECK();
        return 0;
    }
    const int64_t per_cta = int64_t(kThreads / 32) * kQBlock;
    convert_moment_kernel<<<unsigned((numel + per_cta - 1) / per_cta), kThreads, 0, s>>>(src, dst, numel);
    BAOC_LAUNCH_CHECK();
    return 0;
}

}  // namespace baoc
