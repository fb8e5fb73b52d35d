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
__device__ __forceinline__ void load8(const void* src, int64_t idx, int valid, bool vec, float (&x)[8]) {
    if constexpr (kSquare) {
        const uint16_t* p = static_cast<const uint16_t*>(src) + idx;
        if (vec && valid == 8) {
            unpack8(ld_stream_u4(p), x);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) x[j] = j < valid ? bf16_bits_to_float(p[j]) : 0.f;
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
__device__ __forceinline__ void rowcol_reduce_piece(const void* src, int rows, int cols, const RedGeom geo,
                                                    uint32_t chunk, uint32_t strip) {
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
                load8<kSquare>(src, r * cols + col0, valid, vec, x);
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
                       const void* const* __restrict__ grads) {
    const RedTile t = rtiles[blockIdx.x];
    const StepBlock* b = blocks + t.block;
    rowcol_reduce_piece<true>(grads[t.block], b->rows, b->cols, b->red, t.chunk, t.strip);
}

// Second moments of the matrix blocks of the statistics pass.
__global__ void __launch_bounds__(kThreads)
moment_reduce_kernel(const StatBlock* __restrict__ blocks, const RedTile* __restrict__ rtiles) {
    const RedTile t = rtiles[blockIdx.x];
    const StatBlock* b = blocks + t.block;
    rowcol_reduce_piece<false>(b->v, b->rows, b->cols, b->red, t.chunk, t.strip);
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

// One CTA per factored block: r_i <- beta2 r_i + (1-beta2) mean_j g_ij^2,
// c_j likewise over rows, then the mean of the new r.
__global__ void __launch_bounds__(kThreads)
factored_combine_kernel(const StepBlock* __restrict__ blocks, const int32_t* __restrict__ ids,
                        const __grid_constant__ StepParams P) {
    __shared__ double total[1];
    const StepBlock* b = blocks + ids[blockIdx.x];
    const int rows = b->rows, cols = b->cols;
    const double beta2 = P.c[b->cfg].beta2_d;
    float* __restrict__ r = static_cast<float*>(b->s0);
    float* __restrict__ c = static_cast<float*>(b->s1);
    double local[1] = {0.0};
    for (int i = threadIdx.x; i < rows; i += kThreads) {
        double s = 0.0;
        for (int st = 0; st < b->red.strips; ++st) s += b->red.rowpart[size_t(st) * rows + i];
        const float rn = float(beta2 * double(r[i]) + (1.0 - beta2) * (s / double(cols)));
        r[i] = rn;
        local[0] += double(rn);
    }
    cta_reduce_store<1>(local, total);
    for (int j = threadIdx.x; j < cols; j += kThreads) {
        double s = 0.0;
        for (int ch = 0; ch < b->red.chunks; ++ch) s += b->red.colpart[size_t(ch) * cols + j];
        c[j] = float(beta2 * double(c[j]) + (1.0 - beta2) * (s / double(rows)));
    }
    __syncthreads();
    if (threadIdx.x == 0) b->a0[0] = float(total[0] / double(rows));
}

// ============================================================================
// Fused heterogeneous step.  One CTA per tile; the tile's block selects the
// update path, so a CTA never diverges on it.  Every thread owns 8
// consecutive elements per 2048-element slice.
// ============================================================================
__device__ __forceinline__ void prologue(float& x, float& t, const CfgStep& P) {
    if (P.coupled) x = fmaf(P.wd, t, x);          // coupled decay joins the gradient
    else t = fmaf(P.decay, t, t);                 // decoupled: theta <- theta - lr*wd*theta (decay holds -lr*wd)
}

__device__ __forceinline__ float adam_dir(float mhat, float v, const CfgStep& P) {
    return mhat / (sqrtf(v / P.bc2) + P.eps);
}

struct PathA32 {
    static __device__ __forceinline__ void upd(float x, float& t, float& m, float& v, const CfgStep& P) {
        prologue(x, t, P);
        m = fmaf(P.beta1, m, (1.0f - P.beta1) * x);
        v = fmaf(P.beta2, v, (1.0f - P.beta2) * (x * x));
        t = fmaf(-P.lr, adam_dir(m / P.bc1, v, P), t);
    }
};
struct PathR {
    static __device__ __forceinline__ void upd(float x, float& t, float& v, const CfgStep& P) {
        prologue(x, t, P);
        v = fmaf(P.beta2, v, (1.0f - P.beta2) * (x * x));
        t = fmaf(-P.lr, adam_dir(x, v, P), t);
    }
};
struct PathS {
    static __device__ __forceinline__ void upd(float x, float& t, float& m, const CfgStep& P) {
        prologue(x, t, P);
        m = fmaf(P.beta1, m, x);
        t = fmaf(-P.lr, m, t);
    }
};

__device__ __forceinline__ void f4_to(const float4& a, const float4& b, float (&x)[8]) {
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void st8(float* p, const float (&x)[8]) {
    st_stream_f4(p, make_float4(x[0], x[1], x[2], x[3]));
    st_stream_f4(p + 4, make_float4(x[4], x[5], x[6], x[7]));
}

constexpr int kSlices = kTile / (kThreads * 8);

// fp32 Adam / RMS / SGD-momentum: kM = has first moment, kV = has second moment.
template <bool kM, bool kV>
__device__ __forceinline__ unsigned tile_dense(const StepBlock* b, const CfgStep& P, const uint16_t* __restrict__ g,
                                               float* __restrict__ th, int64_t base) {
    const int64_t numel = b->numel;
    float* __restrict__ m = kM ? static_cast<float*>(b->s0) : nullptr;
    float* __restrict__ v = kV ? static_cast<float*>(kM ? b->s1 : b->s0) : nullptr;
    unsigned bad = 0;
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
                bad |= !isfinite(t[j]);
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
                bad |= !isfinite(t);
                th[e + j] = t;
                if (kM) m[e + j] = mm;
                if (kV) v[e + j] = vv;
            }
        }
    }
    return bad;
}

// Factored second moment: v_ij = r_i c_j / mean(r) from the already updated
// row and column statistics; no per-element state.
__device__ __forceinline__ unsigned tile_factored(const StepBlock* b, const CfgStep& P, const uint16_t* __restrict__ g,
                                                  float* __restrict__ th, int64_t base) {
    const int64_t numel = b->numel;
    const int cols = b->cols;
    const float* __restrict__ r = static_cast<const float*>(b->s0);
    const float* __restrict__ c = static_cast<const float*>(b->s1);
    const float rm = b->a0[0];
    const float inv_rm = rm > 0.f ? 1.0f / rm : 0.f;
    unsigned bad = 0;
#pragma unroll
    for (int s = 0; s < kSlices; ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        if (e >= numel) continue;
        const int cnt = int(min64(8, numel - e));
        float x[8], t[8];
        if (cnt == 8) {
            unpack8(ld_stream_u4(g + e), x);
            f4_to(ld_stream_f4(th + e), ld_stream_f4(th + e + 4), t);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                x[j] = j < cnt ? bf16_bits_to_float(g[e + j]) : 0.f;
                t[j] = j < cnt ? th[e + j] : 0.f;
            }
        }
        int64_t row = e / cols;
        int col = int(e - row * cols);
        float ri = __ldg(r + row) * inv_rm;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (j < cnt) {
                float vv = ri * __ldg(c + col);
                float xx = x[j];
                prologue(xx, t[j], P);
                t[j] = fmaf(-P.lr, adam_dir(xx, vv, P), t[j]);
                bad |= !isfinite(t[j]);
                if (++col == cols) { col = 0; ++row; if (j + 1 < cnt) ri = __ldg(r + row) * inv_rm; }
            }
        }
        if (cnt == 8) st8(th + e, t);
        else
            for (int j = 0; j < cnt; ++j) th[e + j] = t[j];
    }
    return bad;
}

// Adam with block-wise absmax 8-bit states.  A warp owns one 256-element
// quantisation block per slice.  The moments are rebuilt, updated and
// re-encoded in double so that the integer codes agree with a double-precision
// evaluation; the parameter update itself runs in fp32 like the other paths.
__device__ __forceinline__ unsigned tile_int8(const StepBlock* b, const CfgStep& P, const uint16_t* __restrict__ g,
                                              float* __restrict__ th, int64_t base) {
    const int64_t numel = b->numel;
    int8_t* __restrict__ qm = static_cast<int8_t*>(b->s0);
    uint8_t* __restrict__ qv = static_cast<uint8_t*>(b->s1);
    float* __restrict__ am = b->a0;
    float* __restrict__ av = b->a1;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const double b1 = P.beta1_d, b2 = P.beta2_d;
    const double o1 = 1.0 - b1, o2 = 1.0 - b2;
    unsigned bad = 0;
#pragma unroll
    for (int s = 0; s < kSlices; ++s) {
        const int64_t w0 = base + int64_t(s) * (kThreads * 8) + int64_t(warp) * kQBlock;
        if (w0 >= numel) continue;                              // whole warp out of range
        const int64_t e = w0 + lane * 8;
        const int cnt = int(max64(0, min64(8, numel - e)));
        const int64_t qb = w0 / kQBlock;
        float x[8], t[8];
        uint2 wm, wv;
        if (cnt == 8) {
            unpack8(ld_stream_u4(g + e), x);
            f4_to(ld_stream_f4(th + e), ld_stream_f4(th + e + 4), t);
            wm = ld_stream_u2(qm + e);
            wv = ld_stream_u2(qv + e);
        } else {
            uint32_t pm[2] = {0u, 0u}, pv[2] = {0u, 0u};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const bool in = j < cnt;
                x[j] = in ? bf16_bits_to_float(g[e + j]) : 0.f;
                t[j] = in ? th[e + j] : 0.f;
                const uint32_t cm = in ? uint32_t(uint8_t(qm[e + j])) : 0u;
                const uint32_t cv = in ? uint32_t(qv[e + j]) : 0u;
                pm[j >> 2] |= cm << (8 * (j & 3));
                pv[j >> 2] |= cv << (8 * (j & 3));
            }
            wm = make_uint2(pm[0], pm[1]);
            wv = make_uint2(pv[0], pv[1]);
        }
        const float am_old = am[qb], av_old = av[qb];
        const double sm = double(am_old) / 127.0, sv = double(av_old) / 255.0;
        const float smf = am_old / 127.0f, svf = av_old / 255.0f;
        double md[8], vd[8];
        double mx_m = 0.0, mx_v = 0.0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const uint32_t wmj = j < 4 ? wm.x : wm.y, wvj = j < 4 ? wv.x : wv.y;
            const int cm = int(int8_t((wmj >> (8 * (j & 3))) & 0xffu));
            const int cv = int((wvj >> (8 * (j & 3))) & 0xffu);
            // double side: the states and their codes
            double gd = widen_bf16_float(x[j]);
            if (P.coupled) gd += double(P.wd) * double(t[j]);
            // fp32 side: the parameter update
            float mf = int_to_float(cm) * smf, vf = int_to_float(cv) * svf;
            PathA32::upd(x[j], t[j], mf, vf, P);
            bad |= !isfinite(t[j]);
            md[j] = b1 * (int_to_double(cm) * sm) + o1 * gd;
            vd[j] = b2 * (int_to_double(cv) * sv) + o2 * (gd * gd);
            mx_m = fmax(mx_m, fabs(md[j]));
            mx_v = fmax(mx_v, vd[j]);
        }
        // rounding to fp32 is monotone, so the maximum of the rounded values is the rounded maximum
        const float am_new = warp_max(__double2float_rn(mx_m));
        const float av_new = warp_max(__double2float_rn(mx_v));
        const double km = code_scale(am_new, 127.0), kv = code_scale(av_new, 255.0);
        uint32_t om[2] = {0u, 0u}, ov[2] = {0u, 0u};
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            om[j >> 2] |= (uint32_t(encode_signed(md[j], km)) & 0xffu) << (8 * (j & 3));
            ov[j >> 2] |= uint32_t(encode_unsigned(vd[j], kv)) << (8 * (j & 3));
        }
        if (cnt == 8) {
            st8(th + e, t);
            st_stream_u2(qm + e, make_uint2(om[0], om[1]));
            st_stream_u2(qv + e, make_uint2(ov[0], ov[1]));
        } else {
            for (int j = 0; j < cnt; ++j) {
                th[e + j] = t[j];
                qm[e + j] = int8_t((om[j >> 2] >> (8 * (j & 3))) & 0xffu);
                qv[e + j] = uint8_t((ov[j >> 2] >> (8 * (j & 3))) & 0xffu);
            }
        }
        if (lane == 0) { am[qb] = am_new; av[qb] = av_new; }
    }
    return bad;
}

__global__ void __launch_bounds__(kThreads)
fused_step_kernel(const StepBlock* __restrict__ blocks, const Tile* __restrict__ tiles,
                  const void* const* __restrict__ grads, float* const* __restrict__ params,
                  uint32_t* __restrict__ flags, const __grid_constant__ StepParams SP) {
    const Tile t = tiles[blockIdx.x];
    const StepBlock* b = blocks + t.block;
    const CfgStep& P = SP.c[b->cfg];
    const uint16_t* g = static_cast<const uint16_t*>(grads[t.block]);
    float* th = params[t.block];
    const int64_t base = int64_t(t.piece) * kTile;
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
                           int64_t n_red, int n_factored, const StepParams& P, cudaStream_t s) {
    if (n_red <= 0) return 0;
    factored_reduce_kernel<<<unsigned(n_red), kThreads, 0, s>>>(blocks, rtiles, grads);
    BAOC_LAUNCH_CHECK();
    factored_combine_kernel<<<n_factored, kThreads, 0, s>>>(blocks, ids, P);
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
