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
    __shared__ float sh_row[2][kRedRows][65];                      // two buffers: one barrier per 64 rows, the sums of one
    __shared__ float sh_col[4][kRedCols];                          // group overlap the loads of the next
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
        if (kSquare && vec && valid == 8 && th == nullptr) {
            // common case: all 16 row segments of this thread are requested before the first one is used
            const uint16_t* p = static_cast<const uint16_t*>(src) + col0;
            uint4 w[kRedRows / 4];
#pragma unroll
            for (int k = 0; k < kRedRows / 4; ++k) {
                const int64_t r = r0 + ty + 4 * k;
                w[k] = r < rows ? ld_stream_u4(p + r * cols) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int k = 0; k < kRedRows / 4; ++k) {
                float x[8];
                unpack8(w[k], x);
                float s = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) { x[j] *= x[j]; s += x[j]; colacc[j] += x[j]; }
                rowacc[k] = s;
            }
        } else if (!kSquare && vec && valid == 8) {
            // fp32 input (the window's second moments): the row segments are requested eight at a time
            const float* p = static_cast<const float*>(src) + col0;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float4 a[kRedRows / 8], b[kRedRows / 8];
#pragma unroll
                for (int k = 0; k < kRedRows / 8; ++k) {
                    const int64_t r = r0 + ty + 4 * (h * (kRedRows / 8) + k);
                    const bool in = r < rows;
                    a[k] = in ? ld_stream_f4(p + r * cols) : make_float4(0.f, 0.f, 0.f, 0.f);
                    b[k] = in ? ld_stream_f4(p + r * cols + 4) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int k = 0; k < kRedRows / 8; ++k) {
                    const float x[8] = {a[k].x, a[k].y, a[k].z, a[k].w, b[k].x, b[k].y, b[k].z, b[k].w};
                    float s = 0.f;
#pragma unroll
                    for (int j = 0; j < 8; ++j) { s += x[j]; colacc[j] += x[j]; }
                    rowacc[h * (kRedRows / 8) + k] = s;
                }
            }
        } else {
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
        }
        float (*buf)[65] = sh_row[l & 1];
#pragma unroll
        for (int k = 0; k < kRedRows / 4; ++k) buf[ty + 4 * k][tx] = rowacc[k];
        __syncthreads();                                            // the buffer written two groups ago is free again by now
        {   // four threads per row: 16 of the 64 per-thread sums each, then two exchanges (a fixed order)
            const int row = threadIdx.x >> 2, part = threadIdx.x & 3;
            double s = 0.0;
#pragma unroll
            for (int j = 0; j < 16; ++j) s += double(buf[row][part * 16 + j]);
            s += __shfl_xor_sync(0xffffffffu, s, 1);
            s += __shfl_xor_sync(0xffffffffu, s, 2);
            const int64_t r = r0 + row;
            if (part == 0 && r < rows) geo.rowpart[size_t(strip) * rows + r] = s;
        }
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

#ifdef BAOC_CHECKED
// A reduction CTA: its piece exists, names a block and a (chunk, strip) of that block's geometry, and the partial sums
// it will write lie inside the bound buffer.
__device__ __forceinline__ bool check_red_piece(const CheckCtx& ck, unsigned kernel, const RedTile& t, int rows, int cols,
                                                const RedGeom& geo) {
    if (int(t.chunk) >= geo.chunks || int(t.strip) >= geo.strips) return check_fail(kChkTileStart, kernel, t.chunk, geo.chunks, t.strip, geo.strips);
    const int64_t r0 = int64_t(t.chunk) * kRedRows * geo.L, nr = min64(int64_t(kRedRows) * geo.L, rows - r0);
    const int64_t c0 = int64_t(t.strip) * kRedCols, nc = min64(kRedCols, cols - c0);
    return check_range(ck, kernel, geo.rowpart + size_t(t.strip) * rows + r0, 8 * nr, 0) &&
           check_range(ck, kernel, geo.colpart + size_t(t.chunk) * cols + c0, 8 * nc, 1);
}
#endif

// Gradient squares of the factored blocks of the step.
__global__ void __launch_bounds__(kThreads, 4)
factored_reduce_kernel(const StepBlock* __restrict__ blocks, const RedTile* __restrict__ rtiles,
                       const void* const* __restrict__ grads, const float* const* __restrict__ params,
                       const __grid_constant__ StepParams SP BAOC_CHECK_PARAM) {
#ifdef BAOC_CHECKED
    {
        if (int64_t(blockIdx.x) >= ck.n_tiles) { check_fail(kChkTileIndex, kKerFactoredReduce, blockIdx.x, ck.n_tiles, 0, 0); return; }
        const RedTile ct = rtiles[blockIdx.x];
        if (ct.block >= unsigned(ck.n_blocks)) { check_fail(kChkBlockIndex, kKerFactoredReduce, ct.block, ck.n_blocks, blockIdx.x, 0); return; }
        const StepBlock* cb = blocks + ct.block;
        if (!check_red_piece(ck, kKerFactoredReduce, ct, cb->rows, cb->cols, cb->red) ||
            !check_caller_ptr(kKerFactoredReduce, grads[ct.block], 2))
            return;
    }
#endif
    const RedTile t = rtiles[blockIdx.x];
    const StepBlock* b = blocks + t.block;
    const CfgStep& P = SP.c[b->cfg];
    rowcol_reduce_piece<true>(grads[t.block], P.coupled ? params[t.block] : nullptr, P.wd, b->rows, b->cols, b->red,
                              t.chunk, t.strip);
}

// Second moments of the matrix blocks of the statistics pass.
__global__ void __launch_bounds__(kThreads)
moment_reduce_kernel(const StatBlock* __restrict__ blocks, const RedTile* __restrict__ rtiles BAOC_CHECK_PARAM) {
#ifdef BAOC_CHECKED
    {
        if (int64_t(blockIdx.x) >= ck.n_tiles) { check_fail(kChkTileIndex, kKerMomentReduce, blockIdx.x, ck.n_tiles, 0, 0); return; }
        const RedTile ct = rtiles[blockIdx.x];
        if (ct.block >= unsigned(ck.n_blocks)) { check_fail(kChkBlockIndex, kKerMomentReduce, ct.block, ck.n_blocks, blockIdx.x, 0); return; }
        const StatBlock* cb = blocks + ct.block;
        const int64_t cpad = (cb->numel + kQBlock - 1) / kQBlock * kQBlock;
        if (!check_red_piece(ck, kKerMomentReduce, ct, cb->rows, cb->cols, cb->red) ||
            !check_range(ck, kKerMomentReduce, cb->v, 4 * cpad, 2))
            return;
    }
#endif
    const RedTile t = rtiles[blockIdx.x];
    const StatBlock* b = blocks + t.block;
    rowcol_reduce_piece<false>(b->v, nullptr, 0.f, b->rows, b->cols, b->red, t.chunk, t.strip);
}

// kCombineSlabs CTAs per matrix block, each owning a slab of the rows and of the columns: add the pieces into
// rowsum / colsum (double).
__global__ void __launch_bounds__(kThreads)
moment_reduce_combine_kernel(const StatBlock* __restrict__ blocks, const int32_t* __restrict__ ids) {
    const StatBlock* b = blocks + ids[blockIdx.x];
    const int rows = b->rows, cols = b->cols, slab = blockIdx.y;
    const int rpc = (rows + kCombineSlabs - 1) / kCombineSlabs, cpc = (cols + kCombineSlabs - 1) / kCombineSlabs;
    for (int i = slab * rpc + threadIdx.x; i < min(rows, (slab + 1) * rpc); i += kThreads) {
        double s = 0.0;
        for (int st = 0; st < b->red.strips; ++st) s += b->red.rowpart[size_t(st) * rows + i];
        b->rowsum[i] = s;
    }
    for (int j = slab * cpc + threadIdx.x; j < min(cols, (slab + 1) * cpc); j += kThreads) {
        double s = 0.0;
#pragma unroll 4
        for (int ch = 0; ch < b->red.chunks; ++ch) s += b->red.colpart[size_t(ch) * cols + j];
        b->colsum[j] = s;
    }
}

// One CTA per matrix block: the block's total, the sum of its row sums in a fixed order, stored behind them.
__global__ void __launch_bounds__(kThreads)
moment_total_kernel(const StatBlock* __restrict__ blocks, const int32_t* __restrict__ ids) {
    const StatBlock* b = blocks + ids[blockIdx.x];
    double acc[1] = {0.0};
    for (int i = threadIdx.x; i < b->rows; i += kThreads) acc[0] += b->rowsum[i];
    cta_reduce_store<1>(acc, b->rowsum + b->rows);
}

// kCombineSlabs CTAs per factored block, each owning a slab of the rows and of
// the columns: r_i <- beta2 r_i + (1-beta2) mean_j g_ij^2, c_j likewise over rows.
// Every CTA leaves the sum of its new r_i; the CTA that takes the last ticket of
// the block adds the slab sums in index order and stores the mean of r (no CTA
// waits for another).
// Row (kRow) or column statistics kept as bf16 values or 8-bit codes: a warp owns one 256-element quantisation block at
// a time.  The stored value is read, the new one is written un-rounded (fp32) to the working copy the update kernel
// reads, and its rounding / its code is what is stored.  Returns the thread's share of the sum of the new values.
template <bool kRow>
__device__ __forceinline__ double combine_reduced(const StepBlock* b, double beta2, double eps1, int slab) {
    const int n = kRow ? b->rows : b->cols, other = kRow ? b->cols : b->rows;
    const int parts = kRow ? b->red.strips : b->red.chunks;
    const double* __restrict__ part = kRow ? b->red.rowpart : b->red.colpart;
    float* __restrict__ work = static_cast<float*>(kRow ? b->s0 : b->s1);
    void* stored = kRow ? b->f0 : b->f1;
    float* __restrict__ amax_io = kRow ? b->fa0 : b->fa1;
    const bool codes = b->fbits == 8;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nblk = (n + kQBlock - 1) / kQBlock;
    const int bpc = (nblk + kCombineSlabs - 1) / kCombineSlabs;
    double sum = 0.0;
    for (int q = slab * bpc + warp; q < min(nblk, (slab + 1) * bpc); q += kThreads / 32) {
        const double a_old = codes ? double(amax_io[q]) : 0.0;
        double x[8];
        float amax = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = q * kQBlock + lane * 8 + j;
            x[j] = 0.0;
            if (i < n) {
                double s = 0.0;
                for (int p = 0; p < parts; ++p) s += part[size_t(p) * n + i];
                const double old = codes ? (double(static_cast<const uint8_t*>(stored)[i]) * a_old) / 255.0
                                         : double(bf16_bits_to_float(static_cast<const uint16_t*>(stored)[i]));
                x[j] = beta2 * old + (1.0 - beta2) * (s / double(other) + eps1);
                const float xf = __double2float_rn(x[j]);
                work[i] = xf;
                sum += double(xf);
                amax = fmaxf(amax, xf);                      // x >= 0; rounding is monotone, so this is the rounded maximum
            }
        }
        if (codes) {
            __syncwarp();                                    // every lane has read the old absmax before lane 0 replaces it
            amax = warp_max(amax);
            const double scale = code_scale(amax, 255.0);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = q * kQBlock + lane * 8 + j;
                if (i < n) static_cast<uint8_t*>(stored)[i] = uint8_t(encode_unsigned(x[j], amax, scale));
            }
            if (lane == 0) amax_io[q] = amax;
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = q * kQBlock + lane * 8 + j;
                if (i < n) static_cast<uint16_t*>(stored)[i] = bf16_from_double(x[j]);
            }
        }
    }
    return sum;
}

__global__ void __launch_bounds__(kThreads)
factored_combine_kernel(const StepBlock* __restrict__ blocks, const int32_t* __restrict__ ids,
                        const __grid_constant__ StepParams P BAOC_CHECK_PARAM) {
#ifdef BAOC_CHECKED
    {
        const int cid = ids[blockIdx.x];
        if (cid < 0 || cid >= ck.n_blocks) { check_fail(kChkBlockIndex, kKerFactoredCombine, cid, ck.n_blocks, blockIdx.x, 0); return; }
        const StepBlock* cb = blocks + cid;
        if (!check_range(ck, kKerFactoredCombine, cb->s0, 4ll * cb->rows, 0) || !check_range(ck, kKerFactoredCombine, cb->s1, 4ll * cb->cols, 1) ||
            !check_range(ck, kKerFactoredCombine, cb->a0, 4, 2) ||
            !check_range(ck, kKerFactoredCombine, cb->mean_part, 8ll * (kCombineSlabs + 1), 3) ||
            !check_range(ck, kKerFactoredCombine, cb->red.rowpart, 8ll * cb->red.strips * cb->rows, 4) ||
            !check_range(ck, kKerFactoredCombine, cb->red.colpart, 8ll * cb->red.chunks * cb->cols, 5))
            return;
        if (cb->fbits != 32) {
            const int64_t eb = cb->fbits == 16 ? 2 : 1;
            if (!check_range(ck, kKerFactoredCombine, cb->f0, eb * cb->rows, 6) || !check_range(ck, kKerFactoredCombine, cb->f1, eb * cb->cols, 7)) return;
            if (cb->fbits == 8 && (!check_range(ck, kKerFactoredCombine, cb->fa0, 4ll * ((cb->rows + kQBlock - 1) / kQBlock), 8) ||
                                   !check_range(ck, kKerFactoredCombine, cb->fa1, 4ll * ((cb->cols + kQBlock - 1) / kQBlock), 9)))
                return;
        }
    }
#endif
    __shared__ double total[1];
    const StepBlock* b = blocks + ids[blockIdx.x];
    const int rows = b->rows, cols = b->cols, slab = blockIdx.y;
    const double beta2 = P.c[b->cfg].beta2_d, eps1 = P.c[b->cfg].eps1_d;   // (the mean of g^2 + eps1 is the mean of g^2, plus eps1)
    double local[1] = {0.0};
    if (b->fbits != 32) {
        local[0] = combine_reduced<true>(b, beta2, eps1, slab);
        cta_reduce_store<1>(local, total);
        combine_reduced<false>(b, beta2, eps1, slab);
    } else {
        float* __restrict__ r = static_cast<float*>(b->s0);
        float* __restrict__ c = static_cast<float*>(b->s1);
        const int rpc = (rows + kCombineSlabs - 1) / kCombineSlabs, cpc = (cols + kCombineSlabs - 1) / kCombineSlabs;
        for (int i = slab * rpc + threadIdx.x; i < min(rows, (slab + 1) * rpc); i += kThreads) {
            double s = 0.0;
            for (int st = 0; st < b->red.strips; ++st) s += b->red.rowpart[size_t(st) * rows + i];
            const float rn = float(beta2 * double(r[i]) + (1.0 - beta2) * (s / double(cols) + eps1));
            r[i] = rn;
            local[0] += double(rn);
        }
        cta_reduce_store<1>(local, total);
        for (int j = slab * cpc + threadIdx.x; j < min(cols, (slab + 1) * cpc); j += kThreads) {
            double s = 0.0;
#pragma unroll 4
            for (int ch = 0; ch < b->red.chunks; ++ch) s += b->red.colpart[size_t(ch) * cols + j];
            c[j] = float(beta2 * double(c[j]) + (1.0 - beta2) * (s / double(rows) + eps1));
        }
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
// and the moments themselves never pass through an approximation.  Both are
// the flush-to-zero forms, which are single instructions (the others wrap the
// same unit in subnormal scaling: six instructions per square root): a second
// moment below 1.2e-38 counts as 0 under the root, far below any eps in use.
// ============================================================================

__device__ __forceinline__ void prologue(float& x, float& t, const CfgStep& P) {
    if (P.coupled) x = fmaf(P.wd, t, x);          // coupled decay joins the gradient
    else t = fmaf(P.decay, t, t);                 // decoupled: theta <- theta - lr*wd*theta (decay holds -lr*wd)
}

// theta <- theta - step * num / (sqrt(v / bc2) + eps)
__device__ __forceinline__ float adaptive_apply(float t, float num, float v, float step, const CfgStep& P) {
    const float denom = fmaf(sqrt_approx(v), P.rsqrt_bc2, P.eps);
    return fmaf(-step * num, rcp_approx(denom), t);
}

__device__ __forceinline__ void f4_to(const float4& a, const float4& b, float (&x)[8]) {
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void st8(float* p, const float (&x)[8]) {
    st_stream_f4(p, make_float4(x[0], x[1], x[2], x[3]));
    st_stream_f4(p + 4, make_float4(x[4], x[5], x[6], x[7]));
}
// Eight fp32 values to a caller-owned array (parameters): one 256-bit store where the array happens to be 32-byte
// aligned (the interface promises 16), else two 128-bit ones.  wide is uniform over the CTA.
__device__ __forceinline__ void st8_param(float* p, const float (&x)[8], bool wide) {
    if (wide) st_stream_f8(p, x); else st8(p, x);
}
__device__ __forceinline__ bool aligned32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0u; }
// 0 * x is 0 for a finite x and NaN otherwise: one FMA per value folds a
// non-finite test of many values into one accumulator.
__device__ __forceinline__ float poison(float acc, float x) { return fmaf(x, 0.0f, acc); }

constexpr int kSlices = kTile / (kThreads * 8);
constexpr int kSlicesF = kTileF / (kThreads * 8);
constexpr int kSlicesQ = kTileQ / (kThreads * 8);
constexpr int kStagesQ = 3;                                          // two slices in flight while one is consumed
constexpr int kStageBytes = kThreads * 64;                           // g 16 B/thread at 0, theta 32 at 4096, m codes 8 at 12288, v codes 8 at 14336

// Dense paths: one streaming pass per element, state in fp32 or bf16.
//   kM = has a first moment / momentum buffer, kV = has a second moment, kB16 = the state is stored as bf16.
//   kM && kV: Adam;  kV only: momentum-free RMS scaling;  kM only: SGD with momentum;  neither: plain gradient step.
// With bf16 storage the parameter update uses the un-rounded fp32 moments and the stored value is the
// round-to-nearest-even bf16 of the new moment.  That rounding is a decision on a floating-point value, so it is
// taken exactly: the fp32 moment is within err of the exact one, and unless it lies within err of the midpoint
// between the two bf16 neighbours its rounding is already the exact answer; the few that do are recomputed in
// double (and rounded double -> fp32 -> bf16).
// Two floats rounded to bf16 (nearest, ties to even) and packed, `lo` in the low half: one instruction.
__device__ __forceinline__ uint32_t pack_bf16x2_rne(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

template <bool kM, bool kV, bool kB16>
struct DenseElem {
    // One element.  x: gradient, t: parameter (updated), m / v: old moments (replaced by the new fp32 ones),
    // mr / vr (kB16): the values whose bf16 rounding is to be stored: the new moments, or their exact recomputation.
    static __device__ __forceinline__ void upd(float x, float& t, float& m, float& v, float& mr, float& vr,
                                               const CfgStep& P) {
        // The fp32 moment differs from the exact one by at most 2^-24 (2 |p| + |m|) (p: the gradient term, rounded once
        // as a product and once through the rounded coefficient; m: the final FMA), plus as much again through p when
        // a coupled decay has rounded the gradient first: 2^-22 (|p| + |m|) covers the first, 2^-21 both.
        const float kErr = P.coupled ? 4.76837158203125e-7f : 2.384185791015625e-7f;
        const float x_raw = x, t_old = t, m_old = m, v_old = v;
        prologue(x, t, P);
        float pm = 0.f, pv = 0.f;
        if (kM) { pm = kV ? P.om1 * x : x; m = fmaf(P.beta1, m_old, pm); }
        if (kV) { pv = P.om2 * (x * x); v = fmaf(P.beta2, v_old, pv); }
        if (kB16) {
            auto exact_g = [&]() { return P.coupled ? double(x_raw) + P.wd_d * double(t_old) : double(x_raw); };
            if (kM) {
                const float mid = __uint_as_float((__float_as_uint(m) & 0xffff0000u) | 0x8000u);
                mr = m;
                if (fabsf(m - mid) <= kErr * (fabsf(pm) + fabsf(m)))
                    mr = __double2float_rn(P.beta1_d * double(m_old) + (kV ? 1.0 - P.beta1_d : 1.0) * exact_g());
            }
            if (kV) {
                const float mid = __uint_as_float((__float_as_uint(v) & 0xffff0000u) | 0x8000u);
                vr = v;
                if (fabsf(v - mid) <= kErr * (pv + v)) {
                    const double gd = exact_g();
                    vr = __double2float_rn(P.beta2_d * double(v_old) + (1.0 - P.beta2_d) * (gd * gd));
                }
            }
        }
        if (kM && kV) t = adaptive_apply(t, m, v, P.step_m, P);
        else if (kV) t = adaptive_apply(t, x, v, P.step_g, P);
        else if (kM) t = fmaf(-P.step_g, m, t);
        else t = fmaf(-P.step_g, x, t);
    }
};

template <bool kM, bool kV, bool kB16>
__device__ __forceinline__ unsigned tile_dense(const StepBlock* b, const CfgStep& P, const uint16_t* __restrict__ g,
                                               float* __restrict__ th, int64_t base) {
    const int64_t numel = b->numel;
    void* const mp = kM ? b->s0 : nullptr;
    void* const vp = kV ? (kM ? b->s1 : b->s0) : nullptr;
    float* __restrict__ m = static_cast<float*>(mp);
    float* __restrict__ v = static_cast<float*>(vp);
    uint16_t* __restrict__ mh = static_cast<uint16_t*>(mp);
    uint16_t* __restrict__ vh = static_cast<uint16_t*>(vp);
    float chk = 0.f;
    const bool th_wide = aligned32(th);                              // uniform over the CTA
    uint4 wg[kSlices];
    float4 t0[kSlices], t1[kSlices], m0[kSlices], m1[kSlices], v0[kSlices], v1[kSlices];
    uint4 mw[kSlices], vw[kSlices];
    bool full[kSlices];
#pragma unroll
    for (int s = 0; s < kSlices; ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        full[s] = e + 8 <= numel;
        if (full[s]) {
            wg[s] = ld_stream_u4(g + e);
            if (th_wide) ld_stream_f8(th + e, t0[s], t1[s]);
            else { t0[s] = ld_stream_f4(th + e); t1[s] = ld_stream_f4(th + e + 4); }
            if (kB16) {
                if (kM) mw[s] = ld_stream_u4(mh + e);
                if (kV) vw[s] = ld_stream_u4(vh + e);
            } else {                                                 // state tensors: 32-byte aligned at multiples of eight elements
                if (kM) ld_stream_f8(m + e, m0[s], m1[s]);
                if (kV) ld_stream_f8(v + e, v0[s], v1[s]);
            }
        }
    }
#pragma unroll
    for (int s = 0; s < kSlices; ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        if (full[s]) {
            float x[8], t[8], mm[8], vv[8];
            float mb[8], vb[8];
            unpack8(wg[s], x); f4_to(t0[s], t1[s], t);
            if (kB16) {
                if (kM) unpack8(mw[s], mm);
                if (kV) unpack8(vw[s], vv);
            } else {
                if (kM) f4_to(m0[s], m1[s], mm);
                if (kV) f4_to(v0[s], v1[s], vv);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                DenseElem<kM, kV, kB16>::upd(x[j], t[j], mm[j], vv[j], mb[j], vb[j], P);
                chk = poison(chk, t[j]);
            }
            st8_param(th + e, t, th_wide);
            if (kB16) {
                if (kM) st_stream_u4(mh + e, make_uint4(pack_bf16x2_rne(mb[0], mb[1]), pack_bf16x2_rne(mb[2], mb[3]),
                                                        pack_bf16x2_rne(mb[4], mb[5]), pack_bf16x2_rne(mb[6], mb[7])));
                if (kV) st_stream_u4(vh + e, make_uint4(pack_bf16x2_rne(vb[0], vb[1]), pack_bf16x2_rne(vb[2], vb[3]),
                                                        pack_bf16x2_rne(vb[4], vb[5]), pack_bf16x2_rne(vb[6], vb[7])));
            } else {
                if (kM) st_stream_f8(m + e, mm);
                if (kV) st_stream_f8(v + e, vv);
            }
        } else if (e < numel) {
            const int cnt = int(numel - e);
            for (int j = 0; j < cnt; ++j) {
                const float x = bf16_bits_to_float(g[e + j]);
                float t = th[e + j], mm = 0.f, vv = 0.f;
                float mb = 0.f, vb = 0.f;
                if (kM) mm = kB16 ? bf16_bits_to_float(mh[e + j]) : m[e + j];
                if (kV) vv = kB16 ? bf16_bits_to_float(vh[e + j]) : v[e + j];
                DenseElem<kM, kV, kB16>::upd(x, t, mm, vv, mb, vb, P);
                chk = poison(chk, t);
                th[e + j] = t;
                if (kB16) {
                    if (kM) mh[e + j] = uint16_t(pack_bf16x2_rne(mb, 0.f));
                    if (kV) vh[e + j] = uint16_t(pack_bf16x2_rne(vb, 0.f));
                } else {
                    if (kM) m[e + j] = mm;
                    if (kV) v[e + j] = vv;
                }
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
// kOpt: the block's tuple carries Adafactor's options: the step size and the clip factor are per-block values that the
// norms kernels have left behind the mean of r, and a decoupled decay uses that step size.
template <bool kOpt>
__device__ __forceinline__ unsigned tile_factored(const StepBlock* b, const CfgStep& P, const uint16_t* __restrict__ g,
                                                  float* __restrict__ th, int64_t base, unsigned char* stage) {
    const int64_t numel = b->numel;
    const int cols = b->cols;
    const float* __restrict__ r = static_cast<const float*>(b->s0);
    const float* __restrict__ c = static_cast<const float*>(b->s1);
    const float rm = b->a0[0];
    const float inv_rm = rm > 0.f ? 1.0f / rm : 0.f;
    float chk = 0.f;
    float step = P.step_g, decay = P.decay;
    if (kOpt) {
        const float alpha = (P.af_flags & kAfRelative) ? b->a0[2] : P.step_g;
        step = (P.af_flags & kAfClip) ? alpha * b->a0[1] : alpha;
        decay = P.decay != 0.f ? -alpha * P.wd : 0.f;            // decoupled: theta <- theta (1 - alpha wd)
    }
    auto pro = [&](float& x, float& t) {
        if (P.coupled) x = fmaf(P.wd, t, x);
        else t = fmaf(decay, t, t);
    };
    if ((cols & 7) == 0) {
        // Streaming form: each thread copies the 48 bytes of its own next eight elements (gradient, parameters)
        // into its own shared-memory slot three slices ahead with cp.async and reads them back itself: no
        // registers are held by loads in flight and no barrier is needed.
        constexpr int kStagesF = 4;
        constexpr int kStageBytesF = kThreads * 48;                   // g 16 B/thread at 0, theta 32 B/thread at 4096
        static_assert(kStagesF * kStageBytesF <= kStagesQ * kStageBytes, "the factored ring must fit the shared staging buffer");
        const int64_t row0 = base / cols;
        const uint32_t col0 = uint32_t(base - row0 * cols);
        const int left = int(min64(numel - base, kTileF));          // a multiple of 8 here
        const uint16_t* __restrict__ gt = g + base;
        float* __restrict__ tht = th + base;
        const bool th_wide = aligned32(tht);                          // uniform over the CTA
        const float* __restrict__ rt = r + row0;
        const int toff = threadIdx.x * 8;
        const uint32_t sm0 = smem_addr(stage), sg = threadIdx.x * 16, st_ = 4096 + threadIdx.x * 32;
        uint32_t fill = 0, take = 0;
        auto prefetch = [&](int s) {
            const int e = s * (kThreads * 8) + toff;
            if (s < kSlicesF && e < left) {
                const uint32_t d = sm0 + fill;
                cp_async16(d + sg, gt + e);
                cp_async16(d + st_, tht + e);
                cp_async16(d + st_ + 16, tht + e + 4);
            }
            cp_async_commit();
            fill = fill == (kStagesF - 1) * kStageBytesF ? 0u : fill + kStageBytesF;
        };
#pragma unroll
        for (int k = 0; k < kStagesF - 1; ++k) prefetch(k);
#pragma unroll 1
        for (int s = 0; s < kSlicesF; ++s) {
            prefetch(s + kStagesF - 1);
            const int e = s * (kThreads * 8) + toff;
            if (e >= left) break;                                   // later slices are out of range too
            const uint32_t cc = col0 + uint32_t(e);                 // < cols + kTileF
            const uint32_t q = cc / uint32_t(cols);
            const uint32_t col = cc - q * uint32_t(cols);
            float cj[8];
            f4_to(__ldg(reinterpret_cast<const float4*>(c + col)), __ldg(reinterpret_cast<const float4*>(c + col + 4)), cj);
            const float rs = __ldg(rt + q) * inv_rm;
            cp_async_wait<kStagesF - 1>();                          // this slice's copies have landed
            const unsigned char* mine = stage + take;
            take = take == (kStagesF - 1) * kStageBytesF ? 0u : take + kStageBytesF;
            float x[8], t[8];
            unpack8(*reinterpret_cast<const uint4*>(mine + sg), x);
            f4_to(*reinterpret_cast<const float4*>(mine + st_), *reinterpret_cast<const float4*>(mine + st_ + 16), t);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                pro(x[j], t[j]);
                t[j] = adaptive_apply(t[j], x[j], rs * cj[j], step, P);
                chk = poison(chk, t[j]);
            }
            st8_param(tht + e, t, th_wide);
        }
        cp_async_wait<0>();
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
            pro(x, t);
            t = adaptive_apply(t, x, rs * __ldg(c + col), step, P);
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
//   * every element is evaluated in fp32, two elements per instruction (the
//     parameter update needs those values anyway); its error against the exact
//     value is below E = 2^-21 (a_old + max|m'|): first-order bound
//     2^-24 (4 max|m'| + 6 a_old) from the roundings of a_old/127, beta1*that,
//     (1-beta1)*g (with a coupled, rounded g) and the final FMA;
//   * the new absmax is the fp32 rounding of the largest exact |m'|, and only
//     elements within 2E of the fp32 maximum can hold it.  Lanes that own such an
//     element are visited in a warp-uniform loop: their raw inputs are broadcast
//     and lanes 0-7 (first moment) and 8-15 (second moment) recompute the lane's
//     eight elements in double, so the recomputation never diverges;
//   * a code is rne(q) with q = 127 m' / a'; the fp32 q is within
//     w = 127 E / a' + 2^-14 of the exact one, so unless it lies within w of a
//     half-integer the fp32 rounding is already the exact answer.  Lanes with such
//     an element are visited the same way and get all eight codes from the
//     correctly rounded double division (exact ties, which bf16 gradients
//     produce from a zero state, are resolved there).
// ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pick_word(uint32_t a, uint32_t b, uint32_t c, uint32_t d, int k) {
    return (k & 2) ? ((k & 1) ? d : c) : ((k & 1) ? b : a);
}

// Raw inputs of the 8 elements of lane `src`, as seen by lane j = lane & 7 of a helper group.
struct Q8Raw {
    uint32_t gbits;      // bf16 gradient of element j
    uint32_t cm, cv;     // code bytes of element j
    float theta;         // parameter of element j before the update (coupled decay only)
};

template <bool kCoupled>
__device__ __forceinline__ Q8Raw q8_fetch(int src, int j, const uint4& wg, const uint2& wm, const uint2& wv,
                                          const float4& t0, const float4& t1) {
    const unsigned full = 0xffffffffu;
    const uint32_t gx = __shfl_sync(full, wg.x, src), gy = __shfl_sync(full, wg.y, src);
    const uint32_t gz = __shfl_sync(full, wg.z, src), gw = __shfl_sync(full, wg.w, src);
    const uint32_t mx = __shfl_sync(full, wm.x, src), my = __shfl_sync(full, wm.y, src);
    const uint32_t vx = __shfl_sync(full, wv.x, src), vy = __shfl_sync(full, wv.y, src);
    Q8Raw r;
    const uint32_t w = pick_word(gx, gy, gz, gw, j >> 1);
    r.gbits = (j & 1) ? (w >> 16) : (w & 0xffffu);
    r.cm = (((j & 4) ? my : mx) >> (8 * (j & 3))) & 0xffu;
    r.cv = (((j & 4) ? vy : vx) >> (8 * (j & 3))) & 0xffu;
    r.theta = 0.f;
    if (kCoupled) {                                                 // the select uses the asking lane's j, so it follows the shuffles
        const float x0 = __shfl_sync(full, t0.x, src), x1 = __shfl_sync(full, t0.y, src);
        const float x2 = __shfl_sync(full, t0.z, src), x3 = __shfl_sync(full, t0.w, src);
        const float x4 = __shfl_sync(full, t1.x, src), x5 = __shfl_sync(full, t1.y, src);
        const float x6 = __shfl_sync(full, t1.z, src), x7 = __shfl_sync(full, t1.w, src);
        const float a = (j & 1) ? x1 : x0, b = (j & 1) ? x3 : x2, c = (j & 1) ? x5 : x4, d = (j & 1) ? x7 : x6;
        r.theta = (j & 4) ? ((j & 2) ? d : c) : ((j & 2) ? b : a);
    }
    return r;
}

// Exact (double) new moment of one element: first moment for group 0, second for group 1.
// kUnitGain: the first moment is a momentum buffer mu m + g rather than an average beta1 m + (1 - beta1) g.
template <bool kCoupled, bool kUnitGain>
__device__ __forceinline__ double q8_exact(const Q8Raw& r, bool second, float am_old, float av_old, const CfgStep& P) {
    double gd = widen_bf16_float(__uint_as_float(r.gbits << 16));
    if (kCoupled) gd += P.wd_d * double(r.theta);
    const double beta = second ? P.beta2_d : P.beta1_d;
    const int code = second ? int(r.cv) : int(int8_t(r.cm));
    const double old = int_to_double(code) * (second ? double(av_old) * (1.0 / 255.0) : double(am_old) * (1.0 / 127.0));
    return beta * old + ((kUnitGain && !second) ? 1.0 : 1.0 - beta) * (second ? gd * gd : gd);
}

// clamp(rne(L * x / a)) by the correctly rounded division.
__device__ __forceinline__ int encode_exact(double x, float absmax, double levels, int lo) {
    if (!(absmax > 0.0f)) return 0;
    return max(lo, min(int(levels), round_to_int((levels * x) / double(absmax))));
}

// Lowest bytes of four words, packed in order.
__device__ __forceinline__ uint32_t pack_low_bytes(uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    return __byte_perm(__byte_perm(a, b, 0x0040u), __byte_perm(c, d, 0x0040u), 0x5410u);
}

// kM / kV: which moments the configuration keeps (both: Adam; kV only: RMS scaling; kM only: SGD with momentum).
template <bool kCoupled, bool kM, bool kV>
__device__ __forceinline__ unsigned tile_int8(const StepBlock* b, const CfgStep& P, const uint16_t* __restrict__ g,
                                              float* __restrict__ th, int64_t base, unsigned char* stage) {
    constexpr float kSlack = 4.76837158203125e-7f;                 // 2^-21
    constexpr float kMagic = 12582912.0f;                          // 1.5 * 2^23: adding it rounds to an integer, ties to even
    const unsigned full = 0xffffffffu;
    const int64_t numel = b->numel;
    int8_t* __restrict__ qm = static_cast<int8_t*>(b->s0);
    uint8_t* __restrict__ qv = static_cast<uint8_t*>(b->s1);
    float* __restrict__ am = b->a0;
    float* __restrict__ av = b->a1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int hj = lane & 7;                                        // element handled when helping another lane
    const bool hv_grp = (lane & 8) != 0, helper = lane < 16;       // lanes 0-7: first moment, 8-15: second moment
    f32x2 chk = pack2(0.f, 0.f);

    // Slices are prefetched two ahead through shared memory: every thread copies the 64 bytes of its own next
    // eight elements (gradient, parameters, both code words) into its own slot with cp.async and reads them back
    // itself, so no registers are held across the long arithmetic of the current slice and no barrier is needed.
    // All indexing inside the tile is 32-bit and relative to the tile's first element.
    const int left = int(min64(numel - base, kTileQ));              // elements of the block in this tile (>= 1)
    const uint16_t* __restrict__ gt = g + base;
    float* __restrict__ tht = th + base;
    const bool th_wide = aligned32(tht);                             // uniform over the CTA
    int8_t* __restrict__ qmt = qm + base;
    uint8_t* __restrict__ qvt = qv + base;
    float* __restrict__ amt = am + base / kQBlock;                   // base is a multiple of the quantisation block
    float* __restrict__ avt = av + base / kQBlock;
    const int toff = threadIdx.x * 8;                                // this thread's first element within a slice
    const uint32_t sm0 = smem_addr(stage);
    const uint32_t sg = threadIdx.x * 16, st_ = 4096 + threadIdx.x * 32, scm = 12288 + threadIdx.x * 8, scv = 14336 + threadIdx.x * 8;
    uint32_t fill = 0;                                               // byte offset of the stage the next prefetch fills
    auto prefetch = [&](int s) {
        const int e = s * (kThreads * 8) + toff;
        if (s < kSlicesQ && e + 8 <= left) {                        // ragged or absent elements are loaded directly later
            const uint32_t d = sm0 + fill;
            cp_async16(d + sg, gt + e);
            cp_async16(d + st_, tht + e);
            cp_async16(d + st_ + 16, tht + e + 4);
            if (kM) cp_async8(d + scm, qmt + e);
            if (kV) cp_async8(d + scv, qvt + e);
        }
        cp_async_commit();
        fill = fill == (kStagesQ - 1) * kStageBytes ? 0u : fill + kStageBytes;
    };
    // The old absmax values of the whole tile are fetched once, before the first wait: lane l < 8 of a warp holds the
    // first moment's absmax of the warp's quantisation block in slice l, lane 8 + l the second moment's.  (Fetched
    // slice by slice they arrived late: a plain load queues behind the copies in flight and takes longer than a slice.)
    static_assert(kSlicesQ <= 8, "one lane per slice and moment");
    float amax_old = 0.f;
    {
        const int sl = lane & 7, w = sl * (kThreads * 8) + warp * kQBlock;
        const bool second = (lane & 8) != 0;
        if (lane < 16 && sl < kSlicesQ && w < left && (second ? kV : kM))
            amax_old = ld_pinned_f32((second ? avt : amt) + w / kQBlock);
    }
#pragma unroll
    for (int k = 0; k < kStagesQ - 1; ++k) prefetch(k);
    uint32_t take = 0;                                               // byte offset of the stage the current slice sits in
#pragma unroll 1
    for (int s = 0; s < kSlicesQ; ++s) {
        const int w0 = s * (kThreads * 8) + warp * kQBlock;
        prefetch(s + kStagesQ - 1);
        const float amo = kM ? __shfl_sync(full, amax_old, s) : 0.f, avo = kV ? __shfl_sync(full, amax_old, 8 + s) : 0.f;
        cp_async_wait<kStagesQ - 1>();                              // this slice's copies have landed (the later ones may be in flight)
        if (w0 >= left) break;                                      // whole warp out of range (and so are the later slices)
        const int e = w0 + lane * 8;
        const int cnt = max(0, min(8, left - e));
        const unsigned char* mine = stage + take;
        take = take == (kStagesQ - 1) * kStageBytes ? 0u : take + kStageBytes;
        uint4 wg;
        float4 t0, t1;
        uint2 wm, wv;
        if (cnt == 8) {
            wg = *reinterpret_cast<const uint4*>(mine + sg);
            t0 = *reinterpret_cast<const float4*>(mine + st_);
            t1 = *reinterpret_cast<const float4*>(mine + st_ + 16);
            wm = kM ? *reinterpret_cast<const uint2*>(mine + scm) : make_uint2(0u, 0u);
            wv = kV ? *reinterpret_cast<const uint2*>(mine + scv) : make_uint2(0u, 0u);
        } else {                                                    // ragged end of the block: zero-fill
            const int n = cnt;
            auto gg = [&](int j) { return j < n ? uint32_t(gt[e + j]) : 0u; };
            auto tt = [&](int j) { return j < n ? tht[e + j] : 0.f; };
            auto mm = [&](int j) { return (kM && j < n) ? uint32_t(uint8_t(qmt[e + j])) : 0u; };
            auto vv = [&](int j) { return (kV && j < n) ? uint32_t(qvt[e + j]) : 0u; };
            wg = make_uint4(gg(0) | gg(1) << 16, gg(2) | gg(3) << 16, gg(4) | gg(5) << 16, gg(6) | gg(7) << 16);
            t0 = make_float4(tt(0), tt(1), tt(2), tt(3)); t1 = make_float4(tt(4), tt(5), tt(6), tt(7));
            wm = make_uint2(mm(0) | mm(1) << 8 | mm(2) << 16 | mm(3) << 24, mm(4) | mm(5) << 8 | mm(6) << 16 | mm(7) << 24);
            wv = make_uint2(vv(0) | vv(1) << 8 | vv(2) << 16 | vv(3) << 24, vv(4) | vv(5) << 8 | vv(6) << 16 | vv(7) << 24);
        }
        // t0, t1 keep the parameters before the update: the coupled exact side needs them

        // ---- fp32 pass, two elements per instruction: effective gradient, decayed parameter, new moments
        // A code byte c becomes the float 2^23 + c by placing it in the low mantissa
        // byte of 0x4B000000 (signed codes are first offset by 128).
        const float b1s = P.beta1 * (amo * (1.0f / 127.0f)), b2s = P.beta2 * (avo * (1.0f / 255.0f));
        const f32x2 B1S = splat2(b1s), B2S = splat2(b2s), VB = splat2(-8388608.0f * b2s);   // the bias is exact: a power-of-two multiple
        const f32x2 OM1 = splat2(P.om1), OM2 = splat2(P.om2), MOFF = splat2(-8388736.0f);
        const uint32_t gw[4] = {wg.x, wg.y, wg.z, wg.w};
        const uint32_t ms[2] = {wm.x ^ 0x80808080u, wm.y ^ 0x80808080u};
        const uint32_t vs[2] = {wv.x, wv.y};
        f32x2 T[4], MF[4], VF[4], XE[4];                             // XE: effective gradients, kept only when they are the numerator
        float lm = 0.f, lv = 0.f;                                   // this lane's maxima
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            f32x2 X = pack2(bf16_lo(gw[p]), bf16_hi(gw[p]));
            T[p] = p == 0 ? pack2(t0.x, t0.y) : (p == 1 ? pack2(t0.z, t0.w) : (p == 2 ? pack2(t1.x, t1.y) : pack2(t1.z, t1.w)));
            if (kCoupled) X = fma2(splat2(P.wd), T[p], X);
            else T[p] = fma2(splat2(P.decay), T[p], T[p]);
            const uint32_t mw = ms[p >> 1], vw = vs[p >> 1];
            const int k0 = (2 * p) & 3, k1 = (2 * p + 1) & 3;
            const f32x2 FM = add2(pack2(__uint_as_float(__byte_perm(mw, 0x4B000000u, 0x7440u | k0)),
                                        __uint_as_float(__byte_perm(mw, 0x4B000000u, 0x7440u | k1))), MOFF);
            const f32x2 FV = pack2(__uint_as_float(__byte_perm(vw, 0x4B000000u, 0x7440u | k0)),
                                   __uint_as_float(__byte_perm(vw, 0x4B000000u, 0x7440u | k1)));
            float a0, a1;
            if (kM) {                                               // Adam: beta1 m + (1 - beta1) g;  momentum SGD: mu m + g
                MF[p] = fma2(FM, B1S, kV ? mul2(OM1, X) : X);
                unpack2(MF[p], a0, a1);
                lm = max3(lm, fabsf(a0), fabsf(a1));
            }
            if (kV) {
                VF[p] = fma2(mul2(OM2, X), X, fma2(FV, B2S, VB));
                unpack2(VF[p], a0, a1);
                lv = max3(lv, a0, a1);
                if (!kM) XE[p] = X;
            }
        }
        const float mx = kM ? warp_max_nonneg(lm) : 0.f, vx = kV ? warp_max_nonneg(lv) : 0.f;
        const float Em = kSlack * (amo + mx), Ev = kSlack * (avo + vx);

        // ---- exact absmax
        unsigned cand_m = kM ? __ballot_sync(full, lm >= mx - 2.0f * Em) : 0u;
        unsigned cand_v = kV ? __ballot_sync(full, lv >= vx - 2.0f * Ev) : 0u;
        float am_c = 0.f, av_c = 0.f;
        while (cand_m | cand_v) {                                   // warp-uniform
            const int Lm = cand_m ? __ffs(cand_m) - 1 : -1, Lv = cand_v ? __ffs(cand_v) - 1 : -1;
            cand_m &= cand_m - 1u; cand_v &= cand_v - 1u;           // (0 & anything stays 0)
            const int src = hv_grp ? Lv : Lm;
            const Q8Raw r = q8_fetch<kCoupled>(max(src, 0), hj, wg, wm, wv, t0, t1);
            const float val = __double2float_rn(fabs(q8_exact<kCoupled, kM && !kV>(r, hv_grp, amo, avo, P)));
            if (helper && src >= 0) {
                if (hv_grp) av_c = fmaxf(av_c, val); else am_c = fmaxf(am_c, val);
            }
        }
        const float am_new = kM ? warp_max_nonneg(am_c) : 0.f, av_new = kV ? warp_max_nonneg(av_c) : 0.f;

        // ---- codes: rne(q) = low byte of the float q + 1.5*2^23
        // L / a' from the approximate reciprocal and one Newton step: within about one ulp (2^-23) of the quotient, so
        // q = m' * (L / a') is off by at most L * 2^-23 = 3.0e-5 on that account, inside the 2^-14 of the window below
        // (a subnormal a' flushes to an infinite scale; the non-finite distance then sends the lane to the exact side)
        const float rm0 = rcp_approx(am_new), rv0 = rcp_approx(av_new);
        const float km = am_new > 0.f ? 127.0f * (rm0 * fmaf(-am_new, rm0, 2.0f)) : 0.f;
        const float kv = av_new > 0.f ? 255.0f * (rv0 * fmaf(-av_new, rv0, 2.0f)) : 0.f;
        const float hm = 0.5f - (Em * km + 6.103515625e-5f), hv = 0.5f - (Ev * kv + 6.103515625e-5f);
        const f32x2 KM = splat2(km), KV = splat2(kv), MAGIC = splat2(kMagic), MINUS1 = splat2(-1.0f);
        uint32_t cmw[8], cvw[8];
        float dm = 0.f, dv = 0.f;                                   // largest distance to the chosen integer in this lane
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            float r0, r1, d0, d1;
            cmw[2 * p] = cmw[2 * p + 1] = cvw[2 * p] = cvw[2 * p + 1] = 0u;
            if (kM) {
                const f32x2 RM = fma2(MF[p], KM, MAGIC);
                const f32x2 DM = fma2(MF[p], KM, fma2(RM, MINUS1, MAGIC));
                unpack2(RM, r0, r1); unpack2(DM, d0, d1);
                cmw[2 * p] = __float_as_uint(r0); cmw[2 * p + 1] = __float_as_uint(r1);
                dm = max3(dm, fabsf(d0), fabsf(d1));
            }
            if (kV) {
                const f32x2 RV = fma2(VF[p], KV, MAGIC);
                const f32x2 DV = fma2(VF[p], KV, fma2(RV, MINUS1, MAGIC));
                unpack2(RV, r0, r1); unpack2(DV, d0, d1);
                cvw[2 * p] = __float_as_uint(r0); cvw[2 * p + 1] = __float_as_uint(r1);
                dv = max3(dv, fabsf(d0), fabsf(d1));
            }
        }
        uint2 om = make_uint2(pack_low_bytes(cmw[0], cmw[1], cmw[2], cmw[3]), pack_low_bytes(cmw[4], cmw[5], cmw[6], cmw[7]));
        uint2 ov = make_uint2(pack_low_bytes(cvw[0], cvw[1], cvw[2], cvw[3]), pack_low_bytes(cvw[4], cvw[5], cvw[6], cvw[7]));
        unsigned slow_m = kM ? __ballot_sync(full, !(dm <= hm)) : 0u, slow_v = kV ? __ballot_sync(full, !(dv <= hv)) : 0u;
        while (slow_m | slow_v) {                                   // warp-uniform, rare
            const int Lm = slow_m ? __ffs(slow_m) - 1 : -1, Lv = slow_v ? __ffs(slow_v) - 1 : -1;
            slow_m &= slow_m - 1u; slow_v &= slow_v - 1u;
            const int src = hv_grp ? Lv : Lm;
            const Q8Raw r = q8_fetch<kCoupled>(max(src, 0), hj, wg, wm, wv, t0, t1);
            const double x = q8_exact<kCoupled, kM && !kV>(r, hv_grp, amo, avo, P);
            const int code = hv_grp ? encode_exact(x, av_new, 255.0, 0) : encode_exact(x, am_new, 127.0, -127);
            const uint32_t piece = (helper && src >= 0) ? (uint32_t(code) & 0xffu) << (8 * (hj & 3)) : 0u;
            const uint32_t mlo = __reduce_or_sync(full, (!hv_grp && hj < 4) ? piece : 0u);
            const uint32_t mhi = __reduce_or_sync(full, (!hv_grp && hj >= 4) ? piece : 0u);
            const uint32_t vlo = __reduce_or_sync(full, (hv_grp && hj < 4) ? piece : 0u);
            const uint32_t vhi = __reduce_or_sync(full, (hv_grp && hj >= 4) ? piece : 0u);
            if (lane == Lm) om = make_uint2(mlo, mhi);
            if (lane == Lv) ov = make_uint2(vlo, vhi);
        }

        // ---- parameter update from the un-requantised fp32 moments
        // Adam: theta <- theta - step_m_hat * m / (sqrt(v) + eps_hat), the bias correction of v folded into both
        // constants;  RMS scaling: the same with the effective gradient and step_g_hat;  momentum SGD: theta - lr * m
        const f32x2 EPS = splat2(P.eps_hat), NSTEP = splat2(kV ? (kM ? -P.step_m_hat : -P.step_g_hat) : -P.step_g);
        float t[8];
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            if (kV) {
                float v0, v1, q0, q1;
                unpack2(VF[p], v0, v1);
                unpack2(add2(pack2(sqrt_approx(v0), sqrt_approx(v1)), EPS), q0, q1);
                T[p] = fma2(mul2(NSTEP, kM ? MF[p] : XE[p]), pack2(rcp_approx(q0), rcp_approx(q1)), T[p]);
            } else {
                T[p] = fma2(NSTEP, MF[p], T[p]);
            }
            chk = add2(chk, T[p]);                                  // a non-finite parameter makes the sum non-finite
            unpack2(T[p], t[2 * p], t[2 * p + 1]);
        }

        if (cnt == 8) {
            st8_param(tht + e, t, th_wide);
            if (kM) st_stream_u2(qmt + e, om);
            if (kV) st_stream_u2(qvt + e, ov);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {                          // static indices keep t[] in registers
                if (j < cnt) {
                    tht[e + j] = t[j];
                    if (kM) qmt[e + j] = int8_t(((j < 4 ? om.x : om.y) >> (8 * (j & 3))) & 0xffu);
                    if (kV) qvt[e + j] = uint8_t(((j < 4 ? ov.x : ov.y) >> (8 * (j & 3))) & 0xffu);
                }
            }
        }
        if (lane == 0) {
            if (kM) amt[w0 / kQBlock] = am_new;
            if (kV) avt[w0 / kQBlock] = av_new;
        }
    }
    cp_async_wait<0>();
    float c0, c1;
    unpack2(chk, c0, c1);
    return !isfinite(c0) | !isfinite(c1);
}

// ----------------------------------------------------------------------------
// Adam with 8-bit moments in the non-linear ("dynamic") codebook: the alternative
// reading of the 8-bit quantiser.  Magnitudes 10^-E (0.1 + 0.9 (k+1) / 2^F), k < 2^F,
// F = B - 1 - E, E < B, with B = 7 value bits (signed, first moments) or 8 (unsigned,
// second moments), and zero; a code is the index of the nearest entry in ascending
// order.  In ascending order the positive magnitude number p >= 1 has F = floor(log2 p),
// E = B - 1 - F, k = p - 2^F, so the tables are built in place by every CTA (into
// shared memory) and no table is stored anywhere.
// The whole update of the moments and the choice of the codes is done in double, in
// the order a plain double-precision evaluation takes, so that the stored codes and
// absmax values are that evaluation's; a step of this path is bound by fp64
// arithmetic, not by memory.  The parameter update is the fp32 one of the other paths.
// ----------------------------------------------------------------------------
__device__ __forceinline__ double warp_max_f64(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmax(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}

template <bool kCoupled>
__device__ __forceinline__ unsigned tile_int8_dyn(const StepBlock* b, const CfgStep& P, const uint16_t* __restrict__ g,
                                                  float* __restrict__ th, int64_t base, unsigned char* stage) {
    static_assert(sizeof(DynTables) <= kStagesQ * kStageBytes, "the tables must fit the shared staging buffer");
    DynTables* T = reinterpret_cast<DynTables*>(stage);
    dyn_build(T);
    const int64_t numel = b->numel;
    uint8_t* __restrict__ qm = static_cast<uint8_t*>(b->s0) + base;
    uint8_t* __restrict__ qv = static_cast<uint8_t*>(b->s1) + base;
    float* __restrict__ am = b->a0 + base / kQBlock;
    float* __restrict__ av = b->a1 + base / kQBlock;
    const uint16_t* __restrict__ gt = g + base;
    float* __restrict__ tht = th + base;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int left = int(min64(numel - base, kTileQ));
    const double om1 = 1.0 - P.beta1_d, om2 = 1.0 - P.beta2_d;
    float chk = 0.f;
#pragma unroll 1
    for (int s = 0; s < kSlicesQ; ++s) {
        const int w0 = s * (kThreads * 8) + warp * kQBlock;
        if (w0 >= left) break;                                       // whole warp out of range (and so are the later slices)
        const int e = w0 + lane * 8;
        const int cnt = max(0, min(8, left - e));
        const double amo = double(am[w0 / kQBlock]), avo = double(av[w0 / kQBlock]);
        double m[8], v[8];
        float t[8];
        double lm = 0.0, lv = 0.0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            m[j] = 0.0; v[j] = 0.0; t[j] = 0.f;
            if (j < cnt) {
                double gd = double(bf16_bits_to_float(gt[e + j]));
                t[j] = tht[e + j];
                if (kCoupled) gd += P.wd_d * double(t[j]);
                else t[j] = fmaf(P.decay, t[j], t[j]);
                m[j] = P.beta1_d * (T->ts[qm[e + j]] * amo) + om1 * gd;
                v[j] = P.beta2_d * (T->tu[qv[e + j]] * avo) + om2 * (gd * gd);
                lm = fmax(lm, fabs(m[j])); lv = fmax(lv, v[j]);
            }
        }
        const float am_new = __double2float_rn(warp_max_f64(lm)), av_new = __double2float_rn(warp_max_f64(lv));
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (j < cnt) {
                qm[e + j] = uint8_t(dyn_nearest(T->ms, am_new > 0.f ? m[j] / double(am_new) : 0.0));
                qv[e + j] = uint8_t(dyn_nearest(T->mu, av_new > 0.f ? v[j] / double(av_new) : 0.0));
                t[j] = adaptive_apply(t[j], float(m[j]), float(v[j]), P.step_m, P);
                chk = poison(chk, t[j]);
                tht[e + j] = t[j];
            }
        }
        if (lane == 0) { am[w0 / kQBlock] = am_new; av[w0 / kQBlock] = av_new; }
    }
    return chk != 0.f;
}

// ----------------------------------------------------------------------------
// Adafactor's update clipping and relative step size need two norms over a whole
// block before any of its elements is updated: RMS(u) of the update
// u = g / (sqrt(v / bc2) + eps) with the new factored second moment, and RMS(theta)
// of the parameters before the step.  One CTA per tile of such a block leaves
// {sum u^2, sum theta^2} in the block's list of tile sums; one CTA per block then
// adds them in tile order and stores the clip factor 1 / max(1, RMS(u)) and the step
// size max(1e-3, RMS(theta)) min(1e-2, 1/sqrt(t)) behind the block's mean of r.
// ----------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
factored_norms_kernel(const StepBlock* __restrict__ blocks, const Tile* __restrict__ tiles,
                      const void* const* __restrict__ grads, const float* const* __restrict__ params,
                      const __grid_constant__ StepParams SP BAOC_CHECK_PARAM) {
#ifdef BAOC_CHECKED
    {
        if (int64_t(blockIdx.x) >= ck.n_tiles) { check_fail(kChkTileIndex, kKerFactoredNorms, blockIdx.x, ck.n_tiles, 0, 0); return; }
        const Tile ct = tiles[blockIdx.x];
        if (ct.block >= unsigned(ck.n_blocks)) { check_fail(kChkBlockIndex, kKerFactoredNorms, ct.block, ck.n_blocks, blockIdx.x, 0); return; }
        const StepBlock* cb = blocks + ct.block;
        if (!check_tile(ck, kKerFactoredNorms, blockIdx.x, ct.block, int64_t(ct.piece) * kTileF, cb->numel) ||
            !check_range(ck, kKerFactoredNorms, cb->s0, 4ll * cb->rows, 0) || !check_range(ck, kKerFactoredNorms, cb->s1, 4ll * cb->cols, 1) ||
            !check_range(ck, kKerFactoredNorms, cb->a0, 12, 2) || !check_range(ck, kKerFactoredNorms, cb->norm_part + 2 * size_t(ct.piece), 16, 3) ||
            !check_caller_ptr(kKerFactoredNorms, grads[ct.block], 4) || !check_caller_ptr(kKerFactoredNorms, params[ct.block], 5))
            return;
    }
#endif
    const Tile t = tiles[blockIdx.x];
    const StepBlock* b = blocks + t.block;
    const CfgStep& P = SP.c[b->cfg];
    const uint16_t* __restrict__ g = static_cast<const uint16_t*>(grads[t.block]);
    const float* __restrict__ th = params[t.block];
    const float* __restrict__ r = static_cast<const float*>(b->s0);
    const float* __restrict__ c = static_cast<const float*>(b->s1);
    const int64_t numel = b->numel, base = int64_t(t.piece) * kTileF;
    const int cols = b->cols;
    const float rm = b->a0[0];
    const float inv_rm = rm > 0.f ? 1.0f / rm : 0.f;
    double acc[2] = {0.0, 0.0};
#pragma unroll 1
    for (int s = 0; s < kSlicesF; ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        if (e >= numel) continue;
        const int cnt = int(min64(8, numel - e));
        int64_t row = e / cols;
        int col = int(e - row * cols);
        float rs = __ldg(r + row) * inv_rm;
        float u2 = 0.f, t2 = 0.f;
        for (int j = 0; j < cnt; ++j) {
            float x = bf16_bits_to_float(g[e + j]);
            const float tt = th[e + j];
            if (P.coupled) x = fmaf(P.wd, tt, x);
            const float u = x * rcp_approx(fmaf(sqrt_approx(rs * __ldg(c + col)), P.rsqrt_bc2, P.eps));
            u2 = fmaf(u, u, u2); t2 = fmaf(tt, tt, t2);
            if (++col == cols) { col = 0; ++row; if (j + 1 < cnt) rs = __ldg(r + row) * inv_rm; }
        }
        acc[0] += double(u2); acc[1] += double(t2);
    }
    cta_reduce_store<2>(acc, b->norm_part + 2 * size_t(t.piece));
}

__global__ void __launch_bounds__(kThreads)
factored_scale_kernel(const StepBlock* __restrict__ blocks, const int32_t* __restrict__ ids, const __grid_constant__ StepParams SP) {
    __shared__ double sums[2];
    const StepBlock* b = blocks + ids[blockIdx.x];
    const CfgStep& P = SP.c[b->cfg];
    const int ntiles = int((b->numel + kTileF - 1) / kTileF);
    double acc[2] = {0.0, 0.0};
    for (int i = threadIdx.x; i < ntiles; i += kThreads) { acc[0] += b->norm_part[2 * i]; acc[1] += b->norm_part[2 * i + 1]; }
    cta_reduce_store<2>(acc, sums);
    if (threadIdx.x == 0) {
        const double n = double(b->numel);
        const double rms_u = sqrt(sums[0] / n), rms_t = sqrt(sums[1] / n);
        b->a0[1] = float(1.0 / fmax(1.0, rms_u));
        b->a0[2] = float(fmax(1e-3, rms_t) * P.rho_d);
    }
}

// Three instances of the kernel, one per family of update paths, each over its own stretch of the tile table:
//   kFamHead   the five headline paths (fp32 Adam / RMS / SGD-momentum, 8-bit Adam, factored): 80 registers, three
//              CTAs per SM, 48 KB of shared memory for the cp.async rings;
//   kFamDense  the stateless and bf16-state dense paths: no shared memory, 64 registers, four CTAs per SM (these
//              paths keep fewer bytes per thread in flight, so they want the extra CTA);
//   kFamQ8     8-bit RMS scaling and 8-bit SGD-momentum: as the headline 8-bit path; also the alternative readings
//              (Adam on the non-linear 8-bit codebook, the factored tuple with Adafactor's options).
// Compiled into one kernel, the extra paths cost the headline ones registers at the 80-register budget (about 9 % on
// the factored tiles), so a step is one launch when the assignment stays within one family and up to three otherwise.
template <int kFam>
__global__ void __launch_bounds__(kThreads, kFam == kFamDense ? 4 : 3)
fused_step_kernel(const StepBlock* __restrict__ blocks, const Tile* __restrict__ tiles,
                  const void* const* __restrict__ grads, float* const* __restrict__ params,
                  uint32_t* __restrict__ flags, const __grid_constant__ StepParams SP BAOC_CHECK_PARAM) {
#ifdef BAOC_CHECKED
    {   // validate the tile and every state range its path will touch before touching anything
        if (int64_t(blockIdx.x) >= ck.n_tiles) { check_fail(kChkTileIndex, kKerFusedStep, blockIdx.x, ck.n_tiles, 0, 0); return; }
        const Tile ct = tiles[blockIdx.x];
        if (ct.block >= unsigned(ck.n_blocks)) { check_fail(kChkBlockIndex, kKerFusedStep, ct.block, ck.n_blocks, blockIdx.x, 0); return; }
        const StepBlock* cb = blocks + ct.block;
        const int64_t te = step_tile_elems(cb->path), cbase = int64_t(ct.piece) * te, cn = min64(te, cb->numel - cbase);
        if (!check_tile(ck, kKerFusedStep, blockIdx.x, ct.block, cbase, cb->numel) ||
            !check_range(ck, kKerFusedStep, flags + ct.block, 4, 0) || cb->cfg < 0 || cb->cfg >= kMaxSlots ||
            !check_caller_ptr(kKerFusedStep, grads[ct.block], 1) || !check_caller_ptr(kKerFusedStep, params[ct.block], 2))
            return;
        const int64_t q0 = cbase / kQBlock, nq = (cbase + cn + kQBlock - 1) / kQBlock - q0;
        auto elems = [&](const void* p, int64_t bytes_per, int what) {
            return check_range(ck, kKerFusedStep, static_cast<const char*>(p) + cbase * bytes_per, cn * bytes_per, what);
        };
        auto scales = [&](const float* p, int what) { return check_range(ck, kKerFusedStep, p + q0, 4 * nq, what); };
        bool ok = true;
        switch (cb->path) {
            case kPathA32: ok = elems(cb->s0, 4, 10) && elems(cb->s1, 4, 11); break;
            case kPathA16: ok = elems(cb->s0, 2, 10) && elems(cb->s1, 2, 11); break;
            case kPathA8: case kPathA8N: ok = elems(cb->s0, 1, 10) && elems(cb->s1, 1, 11) && scales(cb->a0, 12) && scales(cb->a1, 13); break;
            case kPathR: case kPathS: ok = elems(cb->s0, 4, 10); break;
            case kPathR16: case kPathS16: ok = elems(cb->s0, 2, 10); break;
            case kPathR8: ok = elems(cb->s1, 1, 11) && scales(cb->a1, 13); break;
            case kPathS8: ok = elems(cb->s0, 1, 10) && scales(cb->a0, 12); break;
            case kPathF: case kPathFA:
                ok = check_range(ck, kKerFusedStep, cb->s0, 4ll * cb->rows, 10) && check_range(ck, kKerFusedStep, cb->s1, 4ll * cb->cols, 11) &&
                     check_range(ck, kKerFusedStep, cb->a0, 12, 12);
                break;
            default: break;
        }
        if (!ok) return;
    }
#endif
    const Tile t = tiles[blockIdx.x];
    const StepBlock* b = blocks + t.block;
    const CfgStep& P = SP.c[b->cfg];
    const uint16_t* g = static_cast<const uint16_t*>(grads[t.block]);
    float* th = params[t.block];
    const int64_t base = int64_t(t.piece) * step_tile_elems(b->path);
    unsigned bad = 0;
    if (kFam == kFamDense) {
        switch (b->path) {
            case kPathG: bad = tile_dense<false, false, false>(b, P, g, th, base); break;
            case kPathA16: bad = tile_dense<true, true, true>(b, P, g, th, base); break;
            case kPathR16: bad = tile_dense<false, true, true>(b, P, g, th, base); break;
            case kPathS16: bad = tile_dense<true, false, true>(b, P, g, th, base); break;
            default: break;
        }
    } else {
        __shared__ __align__(16) unsigned char q_stage[kStagesQ * kStageBytes];   // per-thread staging of the 8-bit and factored paths
        if (kFam == kFamHead) {
            switch (b->path) {
                case kPathA32: bad = tile_dense<true, true, false>(b, P, g, th, base); break;
                case kPathR: bad = tile_dense<false, true, false>(b, P, g, th, base); break;
                case kPathS: bad = tile_dense<true, false, false>(b, P, g, th, base); break;
                case kPathA8: bad = P.coupled ? tile_int8<true, true, true>(b, P, g, th, base, q_stage) : tile_int8<false, true, true>(b, P, g, th, base, q_stage); break;
                case kPathF: bad = tile_factored<false>(b, P, g, th, base, q_stage); break;
                default: break;
            }
        } else {
            switch (b->path) {
                case kPathR8: bad = P.coupled ? tile_int8<true, false, true>(b, P, g, th, base, q_stage) : tile_int8<false, false, true>(b, P, g, th, base, q_stage); break;
                case kPathS8: bad = P.coupled ? tile_int8<true, true, false>(b, P, g, th, base, q_stage) : tile_int8<false, true, false>(b, P, g, th, base, q_stage); break;
                case kPathA8N: bad = P.coupled ? tile_int8_dyn<true>(b, P, g, th, base, q_stage) : tile_int8_dyn<false>(b, P, g, th, base, q_stage); break;
                case kPathFA: bad = tile_factored<true>(b, P, g, th, base, q_stage); break;
                default: break;
            }
        }
    }
    if (bad) atomicOr(flags + t.block, 1u);
}

// ---- launchers ------------------------------------------------------------------
#define BAOC_LAUNCH_CHECK()                                   \
    do {                                                      \
        cudaError_t e_ = cudaGetLastError();                  \
        if (e_ != cudaSuccess) return int(e_);                \
    } while (0)

BAOC_DEFINE_CHECK_FETCH(step_check_fetch)

#ifdef BAOC_CHECKED
// The range check run on numbers that violate it; no memory but the record is touched.
__global__ void check_selftest_kernel(const CheckCtx ck) {
    if (threadIdx.x == 0) check_range(ck, kKerSelfTest, ck.hi - 16, 32, 99);
}
#endif
int launch_check_selftest(cudaStream_t s) {
#ifdef BAOC_CHECKED
    static char fake[64];                                   // a host range: only its addresses are compared, nothing dereferences them
    const CheckCtx ck{fake, fake + 64, 0, 0, 0};
    check_selftest_kernel<<<1, 32, 0, s>>>(ck);
    BAOC_LAUNCH_CHECK();
#else
    (void)s;
#endif
    return 0;
}

int launch_moment_reduce(const StatBlock* blocks, const RedTile* rtiles, const int32_t* ids, int64_t n_red, int n_matrix,
                         const CheckCtx& ck, cudaStream_t s) {
    (void)ck;
    if (n_red <= 0) return 0;
    moment_reduce_kernel<<<unsigned(n_red), kThreads, 0, s>>>(blocks, rtiles BAOC_CHECK_ARG(ck));
    BAOC_LAUNCH_CHECK();
    moment_reduce_combine_kernel<<<dim3(unsigned(n_matrix), kCombineSlabs), kThreads, 0, s>>>(blocks, ids);
    BAOC_LAUNCH_CHECK();
    moment_total_kernel<<<n_matrix, kThreads, 0, s>>>(blocks, ids);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_factored_reduce(const StepBlock* blocks, const RedTile* rtiles, const int32_t* ids, const void* const* grads,
                           const float* const* params, int64_t n_red, int n_factored, const StepParams& P, const CheckCtx& ck,
                           cudaStream_t s) {
    (void)ck;
    if (n_red <= 0) return 0;
    factored_reduce_kernel<<<unsigned(n_red), kThreads, 0, s>>>(blocks, rtiles, grads, params, P BAOC_CHECK_ARG(ck));
    BAOC_LAUNCH_CHECK();
    factored_combine_kernel<<<dim3(unsigned(n_factored), kCombineSlabs), kThreads, 0, s>>>(blocks, ids, P BAOC_CHECK_ARG(ck));
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_factored_norms(const StepBlock* blocks, const Tile* tiles, const int32_t* ids, const void* const* grads,
                          const float* const* params, int64_t n_tiles, int n, const StepParams& P, const CheckCtx& ck,
                          cudaStream_t s) {
    (void)ck;
    if (n_tiles <= 0 || n <= 0) return 0;
    factored_norms_kernel<<<unsigned(n_tiles), kThreads, 0, s>>>(blocks, tiles, grads, params, P BAOC_CHECK_ARG(ck));
    BAOC_LAUNCH_CHECK();
    factored_scale_kernel<<<n, kThreads, 0, s>>>(blocks, ids, P);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_fused_step(const StepBlock* blocks, const Tile* tiles, const void* const* grads, float* const* params,
                      uint32_t* flags, int64_t n_tiles, int family, const StepParams& P, const CheckCtx& ck, cudaStream_t s) {
    (void)ck;
    if (n_tiles <= 0) return 0;
    const unsigned grid = unsigned(n_tiles);
    if (family == kFamHead) fused_step_kernel<kFamHead><<<grid, kThreads, 0, s>>>(blocks, tiles, grads, params, flags, P BAOC_CHECK_ARG(ck));
    else if (family == kFamDense) fused_step_kernel<kFamDense><<<grid, kThreads, 0, s>>>(blocks, tiles, grads, params, flags, P BAOC_CHECK_ARG(ck));
    else fused_step_kernel<kFamQ8><<<grid, kThreads, 0, s>>>(blocks, tiles, grads, params, flags, P BAOC_CHECK_ARG(ck));
    BAOC_LAUNCH_CHECK();
    return 0;
}

}  // namespace baoc
