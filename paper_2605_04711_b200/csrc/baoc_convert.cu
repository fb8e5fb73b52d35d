// State migration for an online re-configuration (Sec. 3.1, remark on re-planning; appendix study of online
// re-allocation with optimizer-state inheritance): a moment held under the old configuration is re-stored in the form
// the new configuration keeps.  Values are decoded and re-encoded in double, so the stored result is the correctly
// rounded one whatever the pair of precisions; the kernels run once per re-configuration and are not tuned.
#include "baoc_device.cuh"

namespace baoc {

// Entry i of a factored state's row (kRow) or column statistics, decoded from its stored form.
template <bool kRow>
__device__ __forceinline__ double factor_at(const MomentRef& s, int64_t i) {
    const void* p = kRow ? s.r : s.c;
    if (s.fbits == 32) return double(static_cast<const float*>(p)[i]);
    if (s.fbits == 16) return double(bf16_bits_to_float(static_cast<const uint16_t*>(p)[i]));
    const float* a = kRow ? s.ar : s.ac;
    return (double(static_cast<const uint8_t*>(p)[i]) * double(a[i / kQBlock])) / 255.0;
}

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
            return factor_at<true>(s, row) * factor_at<false>(s, col) * inv_mean_r;
        }
        default: return 0.0;
    }
}

// 1 / mean(r) of a factored source, summed in a fixed order by the whole CTA (0 when the mean is 0).
__device__ __forceinline__ double inv_mean_of_rows(const MomentRef& s) {
    __shared__ double total[1];
    double local[1] = {0.0};
    for (int i = threadIdx.x; i < s.rows; i += kThreads) local[0] += factor_at<true>(s, i);
    cta_reduce_store<1>(local, total);
    const double mean = total[0] / double(s.rows);
    return mean != 0.0 ? 1.0 / mean : 0.0;
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

// Factored -> factored (same shape): the statistics themselves, decoded into the destination's fp32 arrays.
__global__ void factor_copy_kernel(const MomentRef src, float* __restrict__ r, float* __restrict__ c) {
    const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < src.rows) r[i] = __double2float_rn(factor_at<true>(src, i));
    if (i < src.cols) c[i] = __double2float_rn(factor_at<false>(src, i));
}

#define BAOC_LAUNCH_CHECK()                                   \
    do {                                                      \
        cudaError_t e_ = cudaGetLastError();                  \
        if (e_ != cudaSuccess) return int(e_);                \
    } while (0)

static int launch_vector_convert(const MomentRef& src, const MomentRef& dst, int64_t numel, cudaStream_t s) {
    const int64_t per_cta = int64_t(kThreads / 32) * kQBlock;
    convert_moment_kernel<<<unsigned((numel + per_cta - 1) / per_cta), kThreads, 0, s>>>(src, dst, numel);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_convert_moment(const MomentRef& src, const MomentRef& dst, int64_t numel, cudaStream_t s) {
    if (dst.kind == kMomFactored) {
        // first the fp32 arrays of the destination (its state when it keeps fp32, else its working copies) ...
        if (src.kind == kMomFactored) {
            const int64_t n = src.rows > src.cols ? src.rows : src.cols;
            factor_copy_kernel<<<unsigned((n + 255) / 256), 256, 0, s>>>(src, dst.wr, dst.wc);
            BAOC_LAUNCH_CHECK();
        } else {
            factor_rows_kernel<<<unsigned(src.rows), kThreads, 0, s>>>(src, dst.wr);
            BAOC_LAUNCH_CHECK();
            factor_cols_kernel<<<unsigned((src.cols + kThreads - 1) / kThreads), kThreads, 0, s>>>(src, dst.wc);
            BAOC_LAUNCH_CHECK();
        }
        if (dst.fbits == 32) return 0;
        // ... then their bf16 rounding or 8-bit codes, as two plain vectors
        MomentRef from{}, to{};
        from.kind = kMomF32; to.kind = dst.fbits == 16 ? kMomBF16 : kMomU8;
        from.data = dst.wr; to.data = dst.r; to.absmax = dst.ar;
        int rc = launch_vector_convert(from, to, dst.rows, s);
        if (rc) return rc;
        from.data = dst.wc; to.data = dst.c; to.absmax = dst.ac;
        return launch_vector_convert(from, to, dst.cols, s);
    }
    return launch_vector_convert(src, dst, numel, s);
}

}  // namespace baoc
