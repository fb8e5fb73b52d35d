// Kernels of the training phase: the fused heterogeneous optimizer step
// (Definition 3.1 tuples; Algorithm 1 "Training") and the row/column reduction
// that the factored second moment (and the structure residual of Eq. 7) needs.
#include "baoc_device.cuh"

namespace baoc {

// ============================================================================
// Row/column reduction of a row-major matrix.  One CTA reduces a piece of
// 64*L rows x 512 columns: thread (ty, tx) = (tid/64, tid%64) owns columns
// 8*tx..8*tx+7 of the strip and rows ty, ty+4, ... of each 64-row group.
// Row sums go to rowpart[strip][row], column sums to colpart[chunk][col], both
// in double; a later kernel adds the pieces in a fixed order.
// kSquare: the source is a bf16 gradient and its squares are summed;
// otherwise the source is an fp32 array summed as it is.
// ============================================================================
template <bool kSquare>
__device__ __forceinline__ void load8(const void* src, const float* th, float wd, int64_t idx, int valid, bool vec,
                                      float (&x)[8]) {
    if constexpr (kSquare) {
        const uint16_t* p = static_cast<const uint16_t*>(src) + idx;
        if (vec && valid == 8) {
            unpack8(ld_stream_u4(p), x);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) x[j] = j < valid ? bf16_bits_to_float(p[j]) : 0.f;
        }
        if (th) {                                  // coupled decay: the squares are those of g + wd*theta
            float t[8];
            if (vec && valid == 8) {
                const float4 a = ld_stream_f4(th + idx), b = ld_stream_f4(th + idx + 4);
                t[0] = a.x; t[1] = a.y; t[2] = a.z; t[3] = a.w; t[4] = b.x; t[5] = b.y; t[6] = b.z; t[7] = b.w;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) t[j] = j < valid ? th[idx + j] : 0.f;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) x[j] = fmaf(wd, t[j], x[j]);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] *= x[j];
    } else {
        const float* p = static_cast<const float*>(src) + idx;
        if (vec && valid == 8) {
            const float4 a = ld_stream_f4(p), b = ld_stream_f4(p + 4);
            x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) x[j] = j < valid ? p[j] : 0.f;
        }
    }
}

template <bool kSquare>
__device__ __forceinline__ void rowcol_reduce_piece(const void* src, const float* th, float wd, int rows, int cols,
                                                    const RedGeom geo, uint32_t chunk, uint32_t strip) {
    __shared__ float sh_row[kRedRows][65];
    __shared__ float sh_col[4][kRedCols];
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
    const int col0 = int(strip) * kRedCols + tx * 8;
    const int valid = max(0, min(8, cols - col0));
    const bool vec = (cols & 7) == 0;
    const int64_t row_begin = int64_t(chunk) * kRedRows * geo.L;
    float colacc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) colacc[j] = 0.f;

    for (int l = 0; l < geo.L; ++l) {
        const int64_t r0 = row_begin + int64_t(l) * kRedRows;
        float rowacc[kRedRows / 4];
#pragma unroll
        for (int k = 0; k < kRedRows / 4; ++k) {
            const int64_t r = r0 + ty + 4 * k;
            float s = 0.f;
            if (r < rows && valid > 0) {
                float x[8];
                load8<kSquare>(src, th, wd, r * cols + col0, valid, vec, x);
#pragma unroll
                for (int j = 0; j < 8; ++j) { s += x[j]; colacc[j] += x[j]; }
            }
            rowacc[k] = s;
        }
#pragma unroll
        for (int k = 0; k < kRedRows / 4; ++k) sh_row[ty + 4 * k][tx] = rowacc[k];
        __syncthreads();
        if (threadIdx.x < kRedRows) {
            const int64_t r = r0 + threadIdx.x;
            if (r < rows) {
                double s = 0.0;
#pragma unroll 8
                for (int j = 0; j < 64; ++j) s += double(sh_row[threadIdx.x][j]);
                geo.rowpart[size_t(strip) * rows + r] = s;
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) sh_col[ty][tx * 8 + j] = colacc[j];
    __syncthreads();
    for (int c = threadIdx.x; c < kRedCols; c += kThreads) {
        const int col = int(strip) * kRedCols + c;
        if (col < cols) {
            const double s = double(sh_col[0][c]) + double(sh_col[1][c]) + double(sh_col[2][c]) + double(sh_col[3][c]);
            geo.colpart[size_t(chunk) * cols + col] = s;
        }
    }
}

// Gradient squares of the factored blocks of the step.
__global__ void __launch_bounds__(kThreads)
factored_reduce_kernel(const StepBlock* __restrict__ blocks, const RedTile* __restrict__ rtiles,
                       const void* const* __restrict__ grads, const float* const* __restrict__ params,
                       const __grid_constant__ StepParams SP) {
    const RedTile t = rtiles[blockIdx.x];
    const StepBlock* b = blocks + t.block;
    const CfgStep& P = SP.c[b->cfg];
    rowcol_reduce_piece<true>(grads[t.block], P.coupled ? params[t.block] : nullptr, P.wd, b->rows, b->cols, b->red,
                              t.chunk, t.strip);
}

// Second moments of the matrix blocks of the statistics pass.
__global__ void __launch_bounds__(kThreads)
moment_reduce_kernel(const StatBlock* __restrict__ blocks, const RedTile* __restrict__ rtiles) {
    const RedTile t = rtiles[blockIdx.x];
    const StatBlock* b = blocks + t.block;
    rowcol_reduce_piece<false>(b->v, nullptr, 0.f, b->rows, b->cols, b->red, t.chunk, t.strip);
}

// One CTA per matrix block: add the pieces into rowsum / colsum (double).
__global__ void __launch_bounds__(kThreads)
moment_reduce_combine_kernel(const StatBlock* __restrict__ blocks, const int32_t* __restrict__ ids) {
    const StatBlock* b = blocks + ids[blockIdx.x];
    const int rows = b->rows, cols = b->cols;
    for (int i = threadIdx.x; i < rows; i += kThreads) {
        double s = 0.0;
        for (int st = 0; st < b->red.strips; ++st) s += b->red.rowpart[size_t(st) * rows + i];
        b->rowsum[i] = s;
    }
    for (int j = threadIdx.x; j < cols; j += kThreads) {
        double s = 0.0;
        for (int ch = 0; ch < b->red.chunks; ++ch) s += b->red.colpart[size_t(ch) * cols + j];
        b->colsum[j] = s;
    }
}

// kCombineSlabs CTAs per factored block, each owning a slab of the rows and of
// the columns: r_i <- beta2 r_i + (1-beta2) mean_j g_ij^2, c_j likewise over rows.
// Every CTA leaves the sum of its new r_i; the CTA that takes the last ticket of
// the block adds the slab sums in index order and stores the mean of r (no CTA
// waits for another).
__global__ void __launch_bounds__(kThreads)
factored_combine_kernel(const StepBlock* __restrict__ blocks, const int32_t* __restrict__ ids,
                        const __grid_constant__ StepParams P) {
    __shared__ double total[1];
    const StepBlock* b = blocks + ids[blockIdx.x];
    const int rows = b->rows, cols = b->cols, slab = blockIdx.y;
    const double beta2 = P.c[b->cfg].beta2_d;
    float* __restrict__ r = static_cast<float*>(b->s0);
    float* __restrict__ c = static_cast<float*>(b->s1);
    const int rpc = (rows + kCombineSlabs - 1) / kCombineSlabs, cpc = (cols + kCombineSlabs - 1) / kCombineSlabs;
    double local[1] = {0.0};
    for (int i = slab * rpc + threadIdx.x; i < min(rows, (slab + 1) * rpc); i += kThreads) {
        double s = 0.0;
        for (int st = 0; st < b->red.strips; ++st) s += b->red.rowpart[size_t(st) * rows + i];
        const float rn = float(beta2 * double(r[i]) + (1.0 - beta2) * (s / double(cols)));
        r[i] = rn;
        local[0] += double(rn);
    }
    cta_reduce_store<1>(local, total);
    for (int j = slab * cpc + threadIdx.x; j < min(cols, (slab + 1) * cpc); j += kThreads) {
        double s = 0.0;
#pragma unroll 4
        for (int ch = 0; ch < b->red.chunks; ++ch) s += b->red.colpart[size_t(ch) * cols + j];
        c[j] = float(beta2 * double(c[j]) + (1.0 - beta2) * (s / double(rows)));
    }
    if (threadIdx.x == 0) {
        volatile double* part = b->mean_part;
        unsigned int* ticket = reinterpret_cast<unsigned int*>(b->mean_part + kCombineSlabs);
        part[slab] = total[0];
        __threadfence();
        if (atomicAdd(ticket, 1u) == unsigned(kCombineSlabs - 1)) {
            __threadfence();
            double s = 0.0;
            for (int k = 0; k < kCombineSlabs; ++k) s += part[k];
            b->a0[0] = float(s / double(rows));
            *ticket = 0u;                            // ready for the next step
        }
    }
}

// ============================================================================
// Fused heterogeneous step.  One CTA per tile; the tile's block selects the
// update path, so a CTA never diverges on it.  Every thread owns 8
// consecutive elements per 2048-element slice, and all loads of a tile are
// issued before the first use.
//
// The direction m / (sqrt(v / bc2) + eps) is evaluated as
// m * rcp(sqrt(v) * rsqrt(bc2) + eps) with the approximate square root and
// reciprocal (relative error 2^-23 each): the update is lr * direction, a
// small fraction of the parameter, so the parameter keeps full fp32 accuracy,
// and the moments themselves never pass through an approximation.
// ============================================================================
__device__ __forceinline__ float sqrt_approx(float x) {
    float r;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float rcp_approx(float x) {
    float r;
    asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

__device__ __forceinline__ void prologue(float& x, float& t, const CfgStep& P) {
    if (P.coupled) x = fmaf(P.wd, t, x);          // coupled decay joins the gradient
    else t = fmaf(P.decay, t, t);                 // decoupled: theta <- theta - lr*wd*theta (decay holds -lr*wd)
}

// theta <- theta - step * num / (sqrt(v / bc2) + eps)
__device__ __forceinline__ float adaptive_apply(float t, float num, float v, float step, const CfgStep& P) {
    const float denom = fmaf(sqrt_approx(v), P.rsqrt_bc2, P.eps);
    return fmaf(-step * num, rcp_approx(denom), t);
}

struct PathA32 {
    static __device__ __forceinline__ void upd(float x, float& t, float& m, float& v, const CfgStep& P) {
        prologue(x, t, P);
        m = fmaf(P.beta1, m, P.om1 * x);
        v = fmaf(P.beta2, v, P.om2 * (x * x));
        t = adaptive_apply(t, m, v, P.step_m, P);
    }
};
struct PathR {
    static __device__ __forceinline__ void upd(float x, float& t, float& v, const CfgStep& P) {
        prologue(x, t, P);
        v = fmaf(P.beta2, v, P.om2 * (x * x));
        t = adaptive_apply(t, x, v, P.step_g, P);
    }
};
struct PathS {
    static __device__ __forceinline__ void upd(float x, float& t, float& m, const CfgStep& P) {
        prologue(x, t, P);
        m = fmaf(P.beta1, m, x);
        t = fmaf(-P.step_g, m, t);
    }
};

__device__ __forceinline__ void f4_to(const float4& a, const float4& b, float (&x)[8]) {
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void st8(float* p, const float (&x)[8]) {
    st_stream_f4(p, make_float4(x[0], x[1], x[2], x[3]));
    st_stream_f4(p + 4, make_float4(x[4], x[5], x[6], x[7]));
}
// 0 * x is 0 for a finite x and NaN otherwise: one FMA per value folds a
// non-finite test of many values into one accumulator.
__device__ __forceinline__ float poison(float acc, float x) { return fmaf(x, 0.0f, acc); }

constexpr int kSlices = kTile / (kThreads * 8);
constexpr int kSlicesF = kTileF / (kThreads * 8);

// fp32 Adam / RMS / SGD-momentum: kM = has first moment, kV = has second moment.
template <bool kM, bool kV>
__device__ __forceinline__ unsigned tile_dense(const StepBlock* b, const CfgStep& P, const uint16_t* __restrict__ g,
                                               float* __restrict__ th, int64_t base) {
    const int64_t numel = b->numel;
    float* __restrict__ m = kM ? static_cast<float*>(b->s0) : nullptr;
    float* __restrict__ v = kV ? static_cast<float*>(kM ? b->s1 : b->s0) : nullptr;
    float chk = 0.f;
    uint4 wg[kSlices];
    float4 t0[kSlices], t1[kSlices], m0[kSlices], m1[kSlices], v0[kSlices], v1[kSlices];
    bool full[kSlices];
#pragma unroll
    for (int s = 0; s < kSlices; ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        full[s] = e + 8 <= numel;
        if (full[s]) {
            wg[s] = ld_stream_u4(g + e);
            t0[s] = ld_stream_f4(th + e); t1[s] = ld_stream_f4(th + e + 4);
            if (kM) { m0[s] = ld_stream_f4(m + e); m1[s] = ld_stream_f4(m + e + 4); }
            if (kV) { v0[s] = ld_stream_f4(v + e); v1[s] = ld_stream_f4(v + e + 4); }
        }
    }
#pragma unroll
    for (int s = 0; s < kSlices; ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        if (full[s]) {
            float x[8], t[8], mm[8], vv[8];
            unpack8(wg[s], x); f4_to(t0[s], t1[s], t);
            if (kM) f4_to(m0[s], m1[s], mm);
            if (kV) f4_to(v0[s], v1[s], vv);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (kM && kV) PathA32::upd(x[j], t[j], mm[j], vv[j], P);
                else if (kV) PathR::upd(x[j], t[j], vv[j], P);
                else PathS::upd(x[j], t[j], mm[j], P);
                chk = poison(chk, t[j]);
            }
            st8(th + e, t);
            if (kM) st8(m + e, mm);
            if (kV) st8(v + e, vv);
        } else if (e < numel) {
            const int cnt = int(numel - e);
            for (int j = 0; j < cnt; ++j) {
                const float x = bf16_bits_to_float(g[e + j]);
                float t = th[e + j], mm = 0.f, vv = 0.f;
                if (kM) mm = m[e + j];
                if (kV) vv = v[e + j];
                if (kM && kV) PathA32::upd(x, t, mm, vv, P);
                else if (kV) PathR::upd(x, t, vv, P);
                else PathS::upd(x, t, mm, P);
                chk = poison(chk, t);
                th[e + j] = t;
                if (kM) m[e + j] = mm;
                if (kV) v[e + j] = vv;
            }
        }
    }
    return chk != 0.f;                               // NaN compares unequal
}

// Factored second moment: v_ij = r_i c_j / mean(r) from the already updated
// row and column statistics; no per-element state.  When the row length is a
// multiple of 8 a thread's 8 elements lie in one row, so it needs one row
// statistic and two 128-bit loads of column statistics (which stay in L1/L2:
// every row of the tile re-reads them).
__device__ __forceinline__ unsigned tile_factored(const StepBlock* b, const CfgStep& P, const uint16_t* __restrict__ g,
                                                  float* __restrict__ th, int64_t base) {
    const int64_t numel = b->numel;
    const int cols = b->cols;
    const float* __restrict__ r = static_cast<const float*>(b->s0);
    const float* __restrict__ c = static_cast<const float*>(b->s1);
    const float rm = b->a0[0];
    const float inv_rm = rm > 0.f ? 1.0f / rm : 0.f;
    float chk = 0.f;
    if ((cols & 7) == 0) {
        const int64_t row0 = base / cols;
        const uint32_t col0 = uint32_t(base - row0 * cols);
        uint4 wg[kSlicesF];
        float4 t0[kSlicesF], t1[kSlicesF];
        float ri[kSlicesF];
        uint32_t cl[kSlicesF];
        bool in[kSlicesF];
#pragma unroll
        for (int s = 0; s < kSlicesF; ++s) {
            const uint32_t off = uint32_t(s) * (kThreads * 8) + threadIdx.x * 8;
            const int64_t e = base + off;
            in[s] = e < numel;                        // numel is a multiple of 8 here
            if (in[s]) {
                const uint32_t cc = col0 + off;       // < cols + kTileF
                const uint32_t q = cc / uint32_t(cols);
                const uint32_t col = cc - q * uint32_t(cols);
                wg[s] = ld_stream_u4(g + e);
                t0[s] = ld_stream_f4(th + e); t1[s] = ld_stream_f4(th + e + 4);
                cl[s] = col;
                ri[s] = __ldg(r + row0 + q);
            }
        }
#pragma unroll
        for (int s = 0; s < kSlicesF; ++s) {
            if (!in[s]) continue;
            const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
            float x[8], t[8], cj[8];
            unpack8(wg[s], x); f4_to(t0[s], t1[s], t);
            f4_to(__ldg(reinterpret_cast<const float4*>(c + cl[s])), __ldg(reinterpret_cast<const float4*>(c + cl[s] + 4)), cj);
            const float rs = ri[s] * inv_rm;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                prologue(x[j], t[j], P);
                t[j] = adaptive_apply(t[j], x[j], rs * cj[j], P.step_g, P);
                chk = poison(chk, t[j]);
            }
            st8(th + e, t);
        }
        return chk != 0.f;
    }
    // any other row length: walk the row/column position element by element
#pragma unroll 1
    for (int s = 0; s < kSlicesF; ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        if (e >= numel) continue;
        const int cnt = int(min64(8, numel - e));
        int64_t row = e / cols;
        int col = int(e - row * cols);
        float rs = __ldg(r + row) * inv_rm;
        for (int j = 0; j < cnt; ++j) {
            float x = bf16_bits_to_float(g[e + j]);
            float t = th[e + j];
            prologue(x, t, P);
            t = adaptive_apply(t, x, rs * __ldg(c + col), P.step_g, P);
            chk = poison(chk, t);
            th[e + j] = t;
            if (++col == cols) { col = 0; ++row; if (j + 1 < cnt) rs = __ldg(r + row) * inv_rm; }
        }
    }
    return chk != 0.f;
}

// ----------------------------------------------------------------------------
// Adam with block-wise absmax 8-bit states.  A warp owns one 256-element
// quantisation block per slice (8 elements per lane).
//
// The integer codes and the fp32 absmax must agree with a double-precision
// evaluation of   m' = beta1 (code a / 127) + (1 - beta1) g,  a' = fl32(max|m'|),
// code' = rne(127 m' / a')   (and likewise for v with 255 levels).  Doing all of
// it in double costs about 20 FP64 operations per element and makes the path
// FP64-bound, so the work is split:
//   * every element is evaluated in fp32 (the parameter update needs those
//     values anyway); its error against the exact value is below
//     E = 2^-21 (a_old + max|m'|) (five roundings of magnitude <= 2^-24 of terms
//     bounded by a_old and max|m'|, with head room);
//   * the new absmax is the fp32 rounding of the largest exact |m'|, and only
//     elements within 2E of the fp32 maximum can hold it, so only those are
//     recomputed in double;
//   * a code is rne(q) with q = 127 m' / a'; the fp32 q is within
//     w = 127 E / a' + 2^-14 of the exact one, so unless it lies within w of a
//     half-integer the fp32 rounding is already the exact answer; the few
//     elements that do are recomputed in double (exact ties, which bf16
//     gradients produce from a zero state, fall in here and are resolved by the
//     correctly rounded division).
// ----------------------------------------------------------------------------
struct Q8Ctx {
    double b1, b2, wd;
    float am_old, av_old;
    int coupled;
};

__device__ __forceinline__ double exact_grad(uint32_t gbits16, float theta, const Q8Ctx& q) {
    double gd = widen_bf16_float(__uint_as_float(gbits16 << 16));
    if (q.coupled) gd += q.wd * double(theta);
    return gd;
}
__device__ __forceinline__ double exact_m(int cm, double gd, const Q8Ctx& q) {
    return q.b1 * (int_to_double(cm) * double(q.am_old) * (1.0 / 127.0)) + (1.0 - q.b1) * gd;
}
__device__ __forceinline__ double exact_v(int cv, double gd, const Q8Ctx& q) {
    return q.b2 * (int_to_double(cv) * double(q.av_old) * (1.0 / 255.0)) + (1.0 - q.b2) * (gd * gd);
}

// clamp(rne(L * x / a)) by the correctly rounded division (a > 0 whenever this is reached with x != 0).
__device__ __forceinline__ int encode_exact(double x, float absmax, double levels, int lo) {
    if (!(absmax > 0.0f)) return 0;
    return max(lo, min(int(levels), round_to_int((levels * x) / double(absmax))));
}

__device__ __forceinline__ uint32_t half_of(const uint4& w, int j) {
    const uint32_t word = j < 2 ? w.x : (j < 4 ? w.y : (j < 6 ? w.z : w.w));
    return (j & 1) ? (word >> 16) : (word & 0xffffu);
}
__device__ __forceinline__ uint32_t byte_of(const uint2& w, int j) { return ((j < 4 ? w.x : w.y) >> (8 * (j & 3))) & 0xffu; }
// Lowest bytes of four words, packed in order.
__device__ __forceinline__ uint32_t pack_low_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    return __byte_perm(__byte_perm(a, b, 0x0040u), __byte_perm(c, d, 0x0040u), 0x5410u);
}
// Warp maximum of non-negative floats (their bit patterns order like unsigned integers): one reduction instruction.
__device__ __forceinline__ float warp_max_nonneg(float x) {
    return __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(x)));
}

__device__ __forceinline__ unsigned tile_int8(const StepBlock* b, const CfgStep& P, const uint16_t* __restrict__ g,
                                              float* __restrict__ th, int64_t base) {
    constexpr float kSlack = 4.76837158203125e-7f;                 // 2^-21
    constexpr float kMagic = 12582912.0f;                          // 1.5 * 2^23: adding it rounds to an integer, ties to even
    const int64_t numel = b->numel;
    int8_t* __restrict__ qm = static_cast<int8_t*>(b->s0);
    uint8_t* __restrict__ qv = static_cast<uint8_t*>(b->s1);
    float* __restrict__ am = b->a0;
    float* __restrict__ av = b->a1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float chk = 0.f;

    // one slice at a time: the path is bound by instruction issue, not by bytes in flight, and holding the
    // next slice's loads would push the whole kernel past 80 registers (three CTAs per SM)
#pragma unroll 1
    for (int s = 0; s < kSlices; ++s) {
        const int64_t w0 = base + int64_t(s) * (kThreads * 8) + int64_t(warp) * kQBlock;
        if (w0 >= numel) break;                                     // whole warp out of range (and so is the next slice)
        const int64_t e = w0 + lane * 8;
        const int cnt = int(max64(0, min64(8, numel - e)));
        const float amo = am[w0 / kQBlock], avo = av[w0 / kQBlock];
        uint4 wg;
        float4 t0, t1;
        uint2 wm, wv;
        if (cnt == 8) {
            wg = ld_stream_u4(g + e);
            t0 = ld_stream_f4(th + e); t1 = ld_stream_f4(th + e + 4);
            wm = ld_stream_u2(qm + e);
            wv = ld_stream_u2(qv + e);
        } else {                                                    // ragged end of the block: zero-fill
            const int n = cnt;
            auto gg = [&](int j) { return j < n ? uint32_t(g[e + j]) : 0u; };
            auto tt = [&](int j) { return j < n ? th[e + j] : 0.f; };
            auto mm = [&](int j) { return j < n ? uint32_t(uint8_t(qm[e + j])) : 0u; };
            auto vv = [&](int j) { return j < n ? uint32_t(qv[e + j]) : 0u; };
            wg = make_uint4(gg(0) | gg(1) << 16, gg(2) | gg(3) << 16, gg(4) | gg(5) << 16, gg(6) | gg(7) << 16);
            t0 = make_float4(tt(0), tt(1), tt(2), tt(3)); t1 = make_float4(tt(4), tt(5), tt(6), tt(7));
            wm = make_uint2(mm(0) | mm(1) << 8 | mm(2) << 16 | mm(3) << 24, mm(4) | mm(5) << 8 | mm(6) << 16 | mm(7) << 24);
            wv = make_uint2(vv(0) | vv(1) << 8 | vv(2) << 16 | vv(3) << 24, vv(4) | vv(5) << 8 | vv(6) << 16 | vv(7) << 24);
        }
        float x[8], t[8], mf[8], vf[8];
        unpack8(wg, x); f4_to(t0, t1, t);
        Q8Ctx q;
        q.b1 = P.beta1_d; q.b2 = P.beta2_d; q.wd = P.wd_d;
        q.am_old = amo; q.av_old = avo; q.coupled = P.coupled;

        // fp32 pass: effective gradient, decayed parameter, new moments, their maxima.
        // A code byte b is turned into the float 2^23 + b by placing it in the low
        // mantissa byte of 0x4B000000 (signed codes are first offset by 128).
        const float b1s = P.beta1 * (amo / 127.0f), b2s = P.beta2 * (avo / 255.0f);
        const float vbias = -8388608.0f * b2s;                      // exact: a power-of-two multiple
        const uint32_t ms[2] = {wm.x ^ 0x80808080u, wm.y ^ 0x80808080u};
        const uint32_t vs[2] = {wv.x, wv.y};
        float mx = 0.f, vx = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float fm = __uint_as_float(__byte_perm(ms[j >> 2], 0x4B000000u, 0x7440u | (j & 3))) - 8388736.0f;
            const float fv = __uint_as_float(__byte_perm(vs[j >> 2], 0x4B000000u, 0x7440u | (j & 3)));
            prologue(x[j], t[j], P);
            mf[j] = fmaf(fm, b1s, P.om1 * x[j]);
            vf[j] = fmaf(P.om2 * x[j], x[j], fmaf(fv, b2s, vbias));
            mx = fmaxf(mx, fabsf(mf[j])); vx = fmaxf(vx, vf[j]);
        }
        mx = warp_max_nonneg(mx); vx = warp_max_nonneg(vx);
        const float Em = kSlack * (amo + mx), Ev = kSlack * (avo + vx);

        // exact absmax: only elements within 2E of the fp32 maximum can hold it.
        // (theta: the coupled gradient needs the parameter before the update; prologue leaves it untouched then.)
        float am_c = 0.f, av_c = 0.f;
        const float m_thr = mx - 2.0f * Em, v_thr = vx - 2.0f * Ev;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const bool cand_m = fabsf(mf[j]) >= m_thr, cand_v = vf[j] >= v_thr;
            if (cand_m || cand_v) {
                const double gd = exact_grad(half_of(wg, j), t[j], q);
                if (cand_m) am_c = fmaxf(am_c, __double2float_rn(fabs(exact_m(int(int8_t(byte_of(wm, j))), gd, q))));
                if (cand_v) av_c = fmaxf(av_c, __double2float_rn(exact_v(int(byte_of(wv, j)), gd, q)));
            }
        }
        const float am_new = warp_max_nonneg(am_c), av_new = warp_max_nonneg(av_c);

        // codes: rne(q) = low byte of the float q + 1.5*2^23, taken from the fp32
        // value unless it is within w of a half-integer
        const float km = am_new > 0.f ? 127.0f / am_new : 0.f, kv = av_new > 0.f ? 255.0f / av_new : 0.f;
        const float hm = 0.5f - (Em * km + 6.103515625e-5f), hv = 0.5f - (Ev * kv + 6.103515625e-5f);
        uint32_t cmw[8], cvw[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float rm_ = fmaf(mf[j], km, kMagic), rv_ = fmaf(vf[j], kv, kMagic);
            const float dm = fmaf(mf[j], km, kMagic - rm_), dv = fmaf(vf[j], kv, kMagic - rv_);
            cmw[j] = __float_as_uint(rm_); cvw[j] = __float_as_uint(rv_);
            const bool slow_m = !(fabsf(dm) <= hm), slow_v = !(fabsf(dv) <= hv);
            if (slow_m || slow_v) {
                const double gd = exact_grad(half_of(wg, j), t[j], q);
                if (slow_m) cmw[j] = uint32_t(encode_exact(exact_m(int(int8_t(byte_of(wm, j))), gd, q), am_new, 127.0, -127));
                if (slow_v) cvw[j] = uint32_t(encode_exact(exact_v(int(byte_of(wv, j)), gd, q), av_new, 255.0, 0));
            }
        }
        const uint2 om = make_uint2(pack_low_bytes(cmw[0], cmw[1], cmw[2], cmw[3]), pack_low_bytes(cmw[4], cmw[5], cmw[6], cmw[7]));
        const uint2 ov = make_uint2(pack_low_bytes(cvw[0], cvw[1], cvw[2], cvw[3]), pack_low_bytes(cvw[4], cvw[5], cvw[6], cvw[7]));

        // parameter update from the un-requantised fp32 moments
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            t[j] = adaptive_apply(t[j], mf[j], vf[j], P.step_m, P);
            chk = poison(chk, t[j]);
        }

        if (cnt == 8) {
            st8(th + e, t);
            st_stream_u2(qm + e, om);
            st_stream_u2(qv + e, ov);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {                          // static indices keep t[] in registers
                if (j < cnt) {
                    th[e + j] = t[j];
                    qm[e + j] = int8_t(((j < 4 ? om.x : om.y) >> (8 * (j & 3))) & 0xffu);
                    qv[e + j] = uint8_t(((j < 4 ? ov.x : ov.y) >> (8 * (j & 3))) & 0xffu);
                }
            }
        }
        if (lane == 0) { am[w0 / kQBlock] = am_new; av[w0 / kQBlock] = av_new; }
    }
    return chk != 0.f;
}

__global__ void __launch_bounds__(kThreads, 3)
fused_step_kernel(const StepBlock* __restrict__ blocks, const Tile* __restrict__ tiles,
                  const void* const* __restrict__ grads, float* const* __restrict__ params,
                  uint32_t* __restrict__ flags, const __grid_constant__ StepParams SP) {
    const Tile t = tiles[blockIdx.x];
    const StepBlock* b = blocks + t.block;
    const CfgStep& P = SP.c[b->cfg];
    const uint16_t* g = static_cast<const uint16_t*>(grads[t.block]);
    float* th = params[t.block];
    const int64_t base = int64_t(t.piece) * (b->path == kPathF ? kTileF : kTile);
    unsigned bad = 0;
    switch (b->path) {
        case kPathA32: bad = tile_dense<true, true>(b, P, g, th, base); break;
        case kPathR: bad = tile_dense<false, true>(b, P, g, th, base); break;
        case kPathS: bad = tile_dense<true, false>(b, P, g, th, base); break;
        case kPathA8: bad = tile_int8(b, P, g, th, base); break;
        case kPathF: bad = tile_factored(b, P, g, th, base); break;
        default: break;
    }
    if (bad) atomicOr(flags + t.block, 1u);
}

// ---- launchers ------------------------------------------------------------------
#define BAOC_LAUNCH_CHECK()                                   \
    do {                                                      \
        cudaError_t e_ = cudaGetLastError();                  \
        if (e_ != cudaSuccess) return int(e_);                \
    } while (0)

int launch_moment_reduce(const StatBlock* blocks, const RedTile* rtiles, const int32_t* ids, int64_t n_red, int n_matrix,
                         cudaStream_t s) {
    if (n_red <= 0) return 0;
    moment_reduce_kernel<<<unsigned(n_red), kThreads, 0, s>>>(blocks, rtiles);
    BAOC_LAUNCH_CHECK();
    moment_reduce_combine_kernel<<<n_matrix, kThreads, 0, s>>>(blocks, ids);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_factored_reduce(const StepBlock* blocks, const RedTile* rtiles, const int32_t* ids, const void* const* grads,
                           const float* const* params, int64_t n_red, int n_factored, const StepParams& P, cudaStream_t s) {
    if (n_red <= 0) return 0;
    factored_reduce_kernel<<<unsigned(n_red), kThreads, 0, s>>>(blocks, rtiles, grads, params, P);
    BAOC_LAUNCH_CHECK();
    factored_combine_kernel<<<dim3(unsigned(n_factored), kCombineSlabs), kThreads, 0, s>>>(blocks, ids, P);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_fused_step(const StepBlock* blocks, const Tile* tiles, const void* const* grads, float* const* params,
                      uint32_t* flags, int64_t n_tiles, const StepParams& P, cudaStream_t s) {
    fused_step_kernel<<<unsigned(n_tiles), kThreads, 0, s>>>(blocks, tiles, grads, params, flags, P);
    BAOC_LAUNCH_CHECK();
    return 0;
}

}  // namespace baoc
