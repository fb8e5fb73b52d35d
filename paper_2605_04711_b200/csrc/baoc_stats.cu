// Kernels of the sampling window (Sec. 3.3) that run at every observation: the
// streaming pass that updates the EMA moments (Eq. 3) and the sums behind the
// direction-stability cosine (Eq. 5), its combine, and the gather of a sampled
// sub-grid.  The end-of-window sweeps are in baoc_finalize.cu.
#include "baoc_device.cuh"

namespace baoc {

// ============================================================================
// Per-step pass.  One CTA per tile of kTile elements of one block; every thread
// owns 8 consecutive elements per 2048-element slice.  Reads g_t, g_{t-1}
// (bf16), m, v (fp32); writes m, v, g_{t-1}; leaves 4 partial sums per tile:
// <g_t, g_{t-1}>, ||g_t||^2, <g_t, m_{t-1}>, ||m_{t-1}||^2.
// ============================================================================
// Eq. 3 as s + (1 - beta)(x - s): only 1 - beta enters, and it is rounded to
// fp32 from its double value, so the recursion's coefficient carries no
// cancellation error (1.0f - float(0.999) is off by 1.3e-5 relative).
__device__ __forceinline__ float ema(float s, float x, float one_minus_beta) { return fmaf(one_minus_beta, x - s, s); }

__global__ void __launch_bounds__(kThreads)
stats_step_kernel(const StatBlock* __restrict__ blocks, const Tile* __restrict__ tiles,
                  const void* const* __restrict__ grads, double* __restrict__ partials, float om, float ov BAOC_CHECK_PARAM) {
#ifdef BAOC_CHECKED
    {   // validate the tile and every range of the workspace it will touch before touching anything
        if (int64_t(blockIdx.x) >= ck.n_tiles) { check_fail(kChkTileIndex, kKerStatsStep, blockIdx.x, ck.n_tiles, 0, 0); return; }
        const Tile ct = tiles[blockIdx.x];
        if (ct.block >= unsigned(ck.n_blocks)) { check_fail(kChkBlockIndex, kKerStatsStep, ct.block, ck.n_blocks, blockIdx.x, 0); return; }
        const StatBlock* cb = blocks + ct.block;
        const int64_t cbase = int64_t(ct.piece) * kTile, cn = min64(kTile, cb->numel - cbase);
        if (!check_tile(ck, kKerStatsStep, blockIdx.x, ct.block, cbase, cb->numel) ||
            !check_range(ck, kKerStatsStep, cb->m + cbase, 4 * cn, 0) || !check_range(ck, kKerStatsStep, cb->v + cbase, 4 * cn, 1) ||
            !check_range(ck, kKerStatsStep, cb->gprev + cbase, 2 * cn, 2) ||
            !check_range(ck, kKerStatsStep, partials + size_t(blockIdx.x) * kStatPartials, 8 * kStatPartials, 3) ||
            !check_caller_ptr(kKerStatsStep, grads[ct.block], 4))
            return;
    }
#endif
    const Tile t = tiles[blockIdx.x];
    const StatBlock* b = blocks + t.block;
    const int64_t numel = b->numel;
    const uint16_t* __restrict__ g = static_cast<const uint16_t*>(grads[t.block]);
    uint16_t* __restrict__ gp = b->gprev;
    float* __restrict__ m = b->m;
    float* __restrict__ v = b->v;
    const int64_t base = int64_t(t.piece) * kTile;
    constexpr int kSlices = kTile / (kThreads * 8);

    float a_dot = 0.f, a_n2 = 0.f, a_dm = 0.f, a_m2 = 0.f;

    uint4 wg[kSlices], wp[kSlices];
    float4 m0[kSlices], m1[kSlices], v0[kSlices], v1[kSlices];
    bool full[kSlices];
#pragma unroll
    for (int s = 0; s < kSlices; ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        full[s] = e + 8 <= numel;
        if (full[s]) {
            wg[s] = ld_stream_u4(g + e);
            wp[s] = ld_stream_u4(gp + e);
            ld_stream_f8(m + e, m0[s], m1[s]);                // (workspace tensors: 32-byte aligned at multiples of eight elements)
            ld_stream_f8(v + e, v0[s], v1[s]);
        }
    }
#pragma unroll
    for (int s = 0; s < kSlices; ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        if (full[s]) {
            float x[8], p[8];
            unpack8(wg[s], x); unpack8(wp[s], p);
            float mm[8] = {m0[s].x, m0[s].y, m0[s].z, m0[s].w, m1[s].x, m1[s].y, m1[s].z, m1[s].w};
            float vv[8] = {v0[s].x, v0[s].y, v0[s].z, v0[s].w, v1[s].x, v1[s].y, v1[s].z, v1[s].w};
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                a_dot = fmaf(x[j], p[j], a_dot);
                a_n2 = fmaf(x[j], x[j], a_n2);
                a_dm = fmaf(x[j], mm[j], a_dm);
                a_m2 = fmaf(mm[j], mm[j], a_m2);
                mm[j] = ema(mm[j], x[j], om);
                vv[j] = ema(vv[j], x[j] * x[j], ov);
            }
            st_stream_f8(m + e, mm);
            st_stream_f8(v + e, vv);
            st_stream_u4(gp + e, wg[s]);
        } else if (e < numel) {
            const int cnt = int(numel - e);
            for (int j = 0; j < cnt; ++j) {
                const uint16_t gb = g[e + j];
                const float x = bf16_bits_to_float(gb), p = bf16_bits_to_float(gp[e + j]);
                const float mm = m[e + j], vv = v[e + j];
                a_dot = fmaf(x, p, a_dot); a_n2 = fmaf(x, x, a_n2);
                a_dm = fmaf(x, mm, a_dm); a_m2 = fmaf(mm, mm, a_m2);
                m[e + j] = ema(mm, x, om);
                v[e + j] = ema(vv, x * x, ov);
                gp[e + j] = gb;
            }
        }
    }
    double acc[kStatPartials] = {double(a_dot), double(a_n2), double(a_dm), double(a_m2)};
    cta_reduce_store<kStatPartials>(acc, partials + size_t(blockIdx.x) * kStatPartials);
}

__device__ __forceinline__ double safe_cos(double dot, double n2a, double n2b, double eps) {
    const double c = dot / (sqrt(n2a) * sqrt(n2b) + eps);
    return isfinite(c) ? c : 0.0;          // a cosine that is not a number counts as 0
}

// Combine: one CTA per block.  acc[block] = {rho_bar, n_cos, ||g_{t-1}||^2,
// last_cos, rho_mom, n_cos_mom, -, -}.
__global__ void __launch_bounds__(kThreads)
stats_combine_kernel(const StatBlock* __restrict__ blocks, const double* __restrict__ partials,
                     double* __restrict__ acc_all, int has_prev, double beta_rho, double eps BAOC_CHECK_PARAM) {
#ifdef BAOC_CHECKED
    {
        if (int(blockIdx.x) >= ck.n_blocks) { check_fail(kChkBlockIndex, kKerStatsCombine, blockIdx.x, ck.n_blocks, 0, 0); return; }
        const StatBlock* cb = blocks + blockIdx.x;
        if (!check_range(ck, kKerStatsCombine, partials + size_t(cb->tile0) * kStatPartials, 8ll * kStatPartials * cb->ntiles, 0) ||
            !check_range(ck, kKerStatsCombine, acc_all + size_t(blockIdx.x) * kBlockAcc, 8 * kBlockAcc, 1))
            return;
    }
#endif
    __shared__ double s[kStatPartials];
    const StatBlock* b = blocks + blockIdx.x;
    block_tiles_sum<kStatPartials>(partials, b->tile0, b->ntiles, s);
    __syncthreads();
    if (threadIdx.x == 0) {
        double* acc = acc_all + size_t(blockIdx.x) * kBlockAcc;
        const double dot = s[0], n2 = s[1], dm = s[2], m2 = s[3];
        if (has_prev) {
            const double c = safe_cos(dot, n2, acc[2], eps);
            acc[3] = c;
            acc[0] = acc[1] == 0.0 ? c : beta_rho * acc[0] + (1.0 - beta_rho) * c;
            acc[1] += 1.0;
            const double cm = safe_cos(dm, n2, m2, eps);
            acc[4] = acc[5] == 0.0 ? cm : beta_rho * acc[4] + (1.0 - beta_rho) * cm;
            acc[5] += 1.0;
        }
        acc[2] = n2;
    }
}

// ============================================================================
// Coordinate sampling: gather the sub-grid rows[ridx] x cols[cidx] of every block
// into its compact sample buffer (bf16 gradients each step, fp32 parameters at
// the end of the window).  One CTA per tile of the sample; element k of the
// sample is (ridx[k / n_cols], cidx[k % n_cols]).  Padding up to the next
// quantisation block is zero-filled so that the streaming kernels may read it.
// ============================================================================
template <typename T>
__global__ void __launch_bounds__(kThreads)
sample_gather_kernel(const StatBlock* __restrict__ blocks, const Tile* __restrict__ tiles, const void* const* __restrict__ src
                     BAOC_CHECK_PARAM) {
#ifdef BAOC_CHECKED
    {
        if (int64_t(blockIdx.x) >= ck.n_tiles) { check_fail(kChkTileIndex, kKerSampleGather, blockIdx.x, ck.n_tiles, 0, 0); return; }
        const Tile ct = tiles[blockIdx.x];
        if (ct.block >= unsigned(ck.n_blocks)) { check_fail(kChkBlockIndex, kKerSampleGather, ct.block, ck.n_blocks, blockIdx.x, 0); return; }
        const StatBlock* cb = blocks + ct.block;
        const int64_t cbase = int64_t(ct.piece) * kTile;
        const int64_t cpad = (cb->numel + kQBlock - 1) / kQBlock * kQBlock, cn = min64(kTile, cpad - cbase);
        const void* dst = sizeof(T) == 2 ? static_cast<const void*>(cb->gsample + cbase) : static_cast<const void*>(cb->psample + cbase);
        if (!check_tile(ck, kKerSampleGather, blockIdx.x, ct.block, cbase, cb->numel) ||
            !check_range(ck, kKerSampleGather, dst, int64_t(sizeof(T)) * cn, 0) ||
            !check_range(ck, kKerSampleGather, cb->ridx, 8ll * cb->rows, 1) || !check_range(ck, kKerSampleGather, cb->cidx, 4ll * cb->cols, 2) ||
            !check_caller_ptr(kKerSampleGather, src[ct.block], 3))
            return;
    }
#endif
    const Tile t = tiles[blockIdx.x];
    const StatBlock* b = blocks + t.block;
    const int64_t numel = b->numel, padded = (numel + kQBlock - 1) / kQBlock * kQBlock;
    const int cols = b->cols;
    const T* __restrict__ in = static_cast<const T*>(src[t.block]);
    T* __restrict__ out = sizeof(T) == 2 ? reinterpret_cast<T*>(b->gsample) : reinterpret_cast<T*>(b->psample);
    const int64_t base = int64_t(t.piece) * kTile;
    for (int i = threadIdx.x; i < kTile; i += kThreads) {
        const int64_t k = base + i;
        if (k >= padded) break;
        T val = T(0);
        if (k < numel) {
            const int64_t r = k / cols;
            const int c = int(k - r * cols);
            val = in[b->ridx[r] * b->full_cols + b->cidx[c]];
        }
        out[k] = val;
    }
}

// ---- launchers ------------------------------------------------------------------
#define BAOC_LAUNCH_CHECK()                                   \
    do {                                                      \
        cudaError_t e_ = cudaGetLastError();                  \
        if (e_ != cudaSuccess) return int(e_);                \
    } while (0)

BAOC_DEFINE_CHECK_FETCH(stats_check_fetch)

int launch_stats_step(const StatBlock* blocks, const Tile* tiles, const void* const* grads, double* partials,
                      int64_t n_tiles, float one_minus_beta_m, float one_minus_beta_v, const CheckCtx& ck, cudaStream_t s) {
    (void)ck;
    stats_step_kernel<<<unsigned(n_tiles), kThreads, 0, s>>>(blocks, tiles, grads, partials, one_minus_beta_m,
                                                             one_minus_beta_v BAOC_CHECK_ARG(ck));
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_stats_combine(const StatBlock* blocks, const double* partials, double* acc, int n_blocks, int has_prev,
                         double beta_rho, double eps, const CheckCtx& ck, cudaStream_t s) {
    (void)ck;
    stats_combine_kernel<<<n_blocks, kThreads, 0, s>>>(blocks, partials, acc, has_prev, beta_rho, eps BAOC_CHECK_ARG(ck));
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_sample_gather(const StatBlock* blocks, const Tile* tiles, const void* const* src, int64_t n_tiles, int fp32,
                         const CheckCtx& ck, cudaStream_t s) {
    (void)ck;
    if (fp32) sample_gather_kernel<float><<<unsigned(n_tiles), kThreads, 0, s>>>(blocks, tiles, src BAOC_CHECK_ARG(ck));
    else sample_gather_kernel<uint16_t><<<unsigned(n_tiles), kThreads, 0, s>>>(blocks, tiles, src BAOC_CHECK_ARG(ck));
    BAOC_LAUNCH_CHECK();
    return 0;
}

}  // namespace baoc
