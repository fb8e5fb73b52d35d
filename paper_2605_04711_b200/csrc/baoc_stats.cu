// Kernels of the sampling window (Sec. 3.3): the per-step streaming pass that
// updates the EMA moments (Eq. 3) and the sums behind the direction-stability
// cosine (Eq. 5), its combine, and the end-of-window finalize sweeps that
// produce the sums behind Eq. 4-8.
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
                  const void* const* __restrict__ grads, double* __restrict__ partials, float om, float ov) {
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
            m0[s] = ld_stream_f4(m + e); m1[s] = ld_stream_f4(m + e + 4);
            v0[s] = ld_stream_f4(v + e); v1[s] = ld_stream_f4(v + e + 4);
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
            st_stream_f4(m + e, make_float4(mm[0], mm[1], mm[2], mm[3]));
            st_stream_f4(m + e + 4, make_float4(mm[4], mm[5], mm[6], mm[7]));
            st_stream_f4(v + e, make_float4(vv[0], vv[1], vv[2], vv[3]));
            st_stream_f4(v + e + 4, make_float4(vv[4], vv[5], vv[6], vv[7]));
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

// Sum K doubles per tile over the tiles of one block in a fixed order: thread
// t takes tiles t, t+T, ..., then the CTA reduces.  out[K] per block.
template <int K>
__device__ __forceinline__ void block_tiles_sum(const double* __restrict__ part, int64_t tile0, int ntiles, double* out) {
    double acc[K];
#pragma unroll
    for (int k = 0; k < K; ++k) acc[k] = 0.0;
    for (int i = threadIdx.x; i < ntiles; i += kThreads) {
        const double* p = part + size_t(tile0 + i) * K;
#pragma unroll
        for (int k = 0; k < K; ++k) acc[k] += p[k];
    }
    cta_reduce_store<K>(acc, out);
}

__device__ __forceinline__ double safe_cos(double dot, double n2a, double n2b, double eps) {
    const double c = dot / (sqrt(n2a) * sqrt(n2b) + eps);
    return isfinite(c) ? c : 0.0;          // a cosine that is not a number counts as 0
}

// Combine: one CTA per block.  acc[block] = {rho_bar, n_cos, ||g_{t-1}||^2,
// last_cos, rho_mom, n_cos_mom, -, -}.
__global__ void __launch_bounds__(kThreads)
stats_combine_kernel(const StatBlock* __restrict__ blocks, const double* __restrict__ partials,
                     double* __restrict__ acc_all, int has_prev, double beta_rho, double eps) {
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
// Finalize sweep 1: per tile, 14 sums over the window's moments (fp32), the
// parameters and the quantised moments.  A warp owns one 256-element
// quantisation block per slice, so the absmax is a warp reduction.
//   0 sum m^2      1 sum v        2 sum v^2       3 sum p, p = 1/(sqrt(v)+eps)
//   4 sum theta^2  5 sum u32^2    6 sum u8^2      7 sum u32*u8
//   8 sum u16^2    9 sum u32*u16  10 sum (m-m8)^2 11 sum (v-v8)^2
//   12 sum (m-m16)^2              13 sum (v-v16)^2
// with u = m/(sqrt(v)+eps_adam) from full-precision, 8-bit and bf16 moments.
// ============================================================================
__device__ __forceinline__ float round_to_bf16(float x) {
    uint32_t u = __float_as_uint(x);
    if ((u & 0x7f800000u) == 0x7f800000u) return x;
    u = (u + 0x7fffu + ((u >> 16) & 1u)) & 0xffff0000u;
    return __uint_as_float(u);
}

// p = 1 / (sqrt(v) + eps) of Eq. 6 in fp32 with correctly rounded square root and division; both finalize
// sweeps evaluate it through this one function so that they see identical values.
__device__ __forceinline__ float precond_of(float v, float eps) { return __fdiv_rn(1.0f, __fsqrt_rn(v) + eps); }

// The 8-bit and 16-bit round trips and the three directions are evaluated in fp32: the sums they feed are compared
// at 1e-4, far above fp32 rounding, and a code that lands on the other side of a rounding tie moves a cosine by
// less than 1e-8.  The directions use the approximate square root and reciprocal (2^-23).
__global__ void __launch_bounds__(kThreads)
stats_final_sums_kernel(const StatBlock* __restrict__ blocks, const Tile* __restrict__ tiles,
                        const float* const* __restrict__ params, double* __restrict__ fin, double eps, float eps_adam) {
    constexpr float kMagic = 12582912.0f;                           // 1.5 * 2^23: adding it rounds to an integer, ties to even
    const Tile t = tiles[blockIdx.x];
    const StatBlock* b = blocks + t.block;
    const int64_t numel = b->numel;
    const float* __restrict__ m = b->m;
    const float* __restrict__ v = b->v;
    const float* __restrict__ th = params[t.block];
    const int64_t base = int64_t(t.piece) * kTile;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float eps_f = float(eps);
    double acc[kFinalSums];
#pragma unroll
    for (int k = 0; k < kFinalSums; ++k) acc[k] = 0.0;

#pragma unroll
    for (int s = 0; s < kTile / (kThreads * 8); ++s) {
        const int64_t w0 = base + int64_t(s) * (kThreads * 8) + int64_t(warp) * kQBlock;
        if (w0 >= numel) continue;                                  // whole warp out of range
        const int64_t e = w0 + lane * 8;
        const int cnt = int(max64(0, min64(8, numel - e)));
        // m and v are padded with zeros to whole quantisation blocks, so the 128-bit loads are always in bounds;
        // theta is not
        float mm[8], vv[8], tt[8];
        {
            const float4 a0 = ld_stream_f4(m + e), a1 = ld_stream_f4(m + e + 4);
            const float4 b0 = ld_stream_f4(v + e), b1 = ld_stream_f4(v + e + 4);
            mm[0] = a0.x; mm[1] = a0.y; mm[2] = a0.z; mm[3] = a0.w; mm[4] = a1.x; mm[5] = a1.y; mm[6] = a1.z; mm[7] = a1.w;
            vv[0] = b0.x; vv[1] = b0.y; vv[2] = b0.z; vv[3] = b0.w; vv[4] = b1.x; vv[5] = b1.y; vv[6] = b1.z; vv[7] = b1.w;
            if (cnt == 8) {
                const float4 c0 = ld_stream_f4(th + e), c1 = ld_stream_f4(th + e + 4);
                tt[0] = c0.x; tt[1] = c0.y; tt[2] = c0.z; tt[3] = c0.w; tt[4] = c1.x; tt[5] = c1.y; tt[6] = c1.z; tt[7] = c1.w;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) tt[j] = j < cnt ? th[e + j] : 0.f;
            }
        }
        float am = 0.f, av = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) { am = fmaxf(am, fabsf(mm[j])); av = fmaxf(av, vv[j]); }
        am = warp_max_nonneg(am); av = warp_max_nonneg(av);
        const float km = am > 0.f ? 127.0f / am : 0.f, kv = av > 0.f ? 255.0f / av : 0.f;
        const float dm = am / 127.0f, dv = av / 255.0f;
        float f[kFinalSums], pj[8];
#pragma unroll
        for (int k = 0; k < kFinalSums; ++k) f[k] = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const bool in = j < cnt;                                // padding contributes zeros to every sum but p
            const float mj = mm[j], vj = vv[j];
            const float m8 = (fmaf(mj, km, kMagic) - kMagic) * dm;
            const float v8 = (fmaf(vj, kv, kMagic) - kMagic) * dv;
            const float m16 = round_to_bf16(mj), v16 = round_to_bf16(vj);
            const float sq = __fsqrt_rn(vj);                        // shared by the direction and by p (precond_of's own value)
            const float u32 = mj * rcp_approx(sq + eps_adam);
            const float u8 = m8 * rcp_approx(sqrt_approx(v8) + eps_adam);
            const float u16 = m16 * rcp_approx(sqrt_approx(v16) + eps_adam);
            pj[j] = in ? __fdiv_rn(1.0f, sq + eps_f) : 0.f;
            f[0] = fmaf(mj, mj, f[0]); f[1] += vj; f[2] = fmaf(vj, vj, f[2]);
            f[4] = fmaf(tt[j], tt[j], f[4]);
            f[5] = fmaf(u32, u32, f[5]); f[6] = fmaf(u8, u8, f[6]); f[7] = fmaf(u32, u8, f[7]);
            f[8] = fmaf(u16, u16, f[8]); f[9] = fmaf(u32, u16, f[9]);
            f[10] = fmaf(mj - m8, mj - m8, f[10]); f[11] = fmaf(vj - v8, vj - v8, f[11]);
            f[12] = fmaf(mj - m16, mj - m16, f[12]); f[13] = fmaf(vj - v16, vj - v16, f[13]);
        }
#pragma unroll
        for (int k = 0; k < kFinalSums; ++k) acc[k] += double(f[k]);
        // p is summed in pairs (p + p and p + 0 are exact in fp32) and from there in double, so that a block whose p
        // are all equal gets exactly p as its mean and a distortion of exactly 0, whatever its length
        acc[3] += (double(pj[0] + pj[1]) + double(pj[2] + pj[3])) + (double(pj[4] + pj[5]) + double(pj[6] + pj[7]));
    }
    cta_reduce_store<kFinalSums>(acc, fin + size_t(blockIdx.x) * kFinalSums);
}

// Per-block combine of sweep 1: fin_out[block][0..13] = the 14 sums.
__global__ void __launch_bounds__(kThreads)
stats_final_combine_kernel(const StatBlock* __restrict__ blocks, const double* __restrict__ fin, double* __restrict__ fin_out) {
    const StatBlock* b = blocks + blockIdx.x;
    block_tiles_sum<kFinalSums>(fin, b->tile0, b->ntiles, fin_out + size_t(blockIdx.x) * kFinOut);
}

// ============================================================================
// Finalize sweep 2: residual sums that need block-level means first.
//   0 sum ((p/pbar - 1) * theta)^2            (Eq. 6 numerator)
//   1 sum (S_ij - a_i b_j / mu)^2             (Eq. 7 numerator, matrix blocks)
// Differences of nearly equal numbers: all in double.
// ============================================================================
__global__ void __launch_bounds__(kThreads)
stats_final_resid_kernel(const StatBlock* __restrict__ blocks, const Tile* __restrict__ tiles,
                         const float* const* __restrict__ params, const double* __restrict__ fin_out,
                         double* __restrict__ fin, double eps) {
    const Tile t = tiles[blockIdx.x];
    const StatBlock* b = blocks + t.block;
    const int64_t numel = b->numel;
    const int cols = b->cols;
    const float* __restrict__ v = b->v;
    const float* __restrict__ th = params[t.block];
    const double* __restrict__ rowsum = b->rowsum;
    const double* __restrict__ colsum = b->colsum;
    const double* sums = fin_out + size_t(t.block) * kFinOut;
    const double pbar = sums[3] / double(numel);
    const double inv_pbar = pbar > 0.0 ? 1.0 / pbar : 0.0;
    const bool matrix = cols > 1;
    // a_i b_j / mu = rowsum_i * colsum_j / total
    const double total = sums[1];
    const double inv_total = (matrix && total > 0.0) ? 1.0 / total : 0.0;
    const int64_t base = int64_t(t.piece) * kTile;
    const float eps_f = float(eps);
    double acc[kResidSums] = {0.0, 0.0};
#pragma unroll
    for (int s = 0; s < kTile / (kThreads * 8); ++s) {
        const int64_t e = base + int64_t(s) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
        if (e >= numel) continue;
        const int cnt = int(min64(8, numel - e));
        float vv[8], tt[8];
        {   // v is padded to whole quantisation blocks, theta is not
            const float4 b0 = ld_stream_f4(v + e), b1 = ld_stream_f4(v + e + 4);
            vv[0] = b0.x; vv[1] = b0.y; vv[2] = b0.z; vv[3] = b0.w; vv[4] = b1.x; vv[5] = b1.y; vv[6] = b1.z; vv[7] = b1.w;
            if (cnt == 8) {
                const float4 c0 = ld_stream_f4(th + e), c1 = ld_stream_f4(th + e + 4);
                tt[0] = c0.x; tt[1] = c0.y; tt[2] = c0.z; tt[3] = c0.w; tt[4] = c1.x; tt[5] = c1.y; tt[6] = c1.z; tt[7] = c1.w;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) tt[j] = j < cnt ? th[e + j] : 0.f;
            }
        }
        int64_t r = matrix ? e / cols : 0;
        int c = matrix ? int(e - r * cols) : 0;
        double rs = matrix ? __ldg(rowsum + r) * inv_total : 0.0;
        if (cnt == 8 && (!matrix || (cols & 7) == 0)) {
            // the eight elements lie in one row (or the block is a vector): one row sum, four 16-byte loads of column sums
            double cs[8];
            if (matrix) {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const double2 w = __ldg(reinterpret_cast<const double2*>(colsum + c) + q);
                    cs[2 * q] = w.x; cs[2 * q + 1] = w.y;
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const double d = (double(precond_of(vv[j], eps_f)) * inv_pbar - 1.0) * double(tt[j]);
                acc[0] += d * d;
                if (matrix) {
                    const double diff = double(vv[j]) - rs * cs[j];
                    acc[1] += diff * diff;
                }
            }
            continue;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (j < cnt) {
                const double d = (double(precond_of(vv[j], eps_f)) * inv_pbar - 1.0) * double(tt[j]);
                acc[0] += d * d;
                if (matrix) {
                    const double diff = double(vv[j]) - rs * __ldg(colsum + c);
                    acc[1] += diff * diff;
                    if (++c == cols) { c = 0; ++r; if (j + 1 < cnt) rs = __ldg(rowsum + r) * inv_total; }
                }
            }
        }
    }
    cta_reduce_store<kResidSums>(acc, fin + size_t(blockIdx.x) * kResidSums);
}

__global__ void __launch_bounds__(kThreads)
stats_resid_combine_kernel(const StatBlock* __restrict__ blocks, const double* __restrict__ fin, double* __restrict__ fin_out) {
    const StatBlock* b = blocks + blockIdx.x;
    block_tiles_sum<kResidSums>(fin, b->tile0, b->ntiles, fin_out + size_t(blockIdx.x) * kFinOut + kFinalSums);
}

// ============================================================================
// Exact quantiles of v by radix select on the fp32 bit patterns (v >= 0, so the
// unsigned order of the patterns is the numeric order).  Four ranks per block
// (the two order statistics around each of the two quantile positions), eight
// bits per pass.  Ranks that still share a prefix share one histogram.
// ============================================================================
// Contention: the first pass looks at the sign/exponent byte, which nearly all elements of a block share, so a
// plain shared-memory histogram would serialise on one counter.  A thread therefore counts runs of equal digits
// over its 16 consecutive elements and adds a run at a time, and every histogram has 8 copies (one per lane & 7)
// that are added up at the end.
constexpr int kHistCopies = 8;
constexpr int kHistTiles = 16;        // consecutive tiles per CTA: the shared histograms are cleared and flushed once per run of tiles of one block

__global__ void __launch_bounds__(kThreads)
select_hist_kernel(const StatBlock* __restrict__ blocks, const Tile* __restrict__ tiles,
                   const RankSel* __restrict__ sel, uint32_t* __restrict__ hist, int64_t n_tiles, int shift) {
    __shared__ uint32_t sh[kRanks][kHistCopies][256];
    const uint32_t high_mask = shift >= 24 ? 0u : (0xffffffffu << (shift + 8));
    const int copy = threadIdx.x & (kHistCopies - 1);
    const int64_t first = int64_t(blockIdx.x) * kHistTiles, last = min64(first + kHistTiles, n_tiles);
    uint32_t prefix[kRanks];
    bool lead[kRanks];
    int cur_block = -1;
    // add the copies of the finished block's histograms to its global ones, and clear them
    auto flush = [&](int blk) {
        uint32_t* out = hist + size_t(blk) * kRanks * 256;
        for (int i = threadIdx.x; i < kRanks * 256; i += kThreads) {
            const int r = i >> 8, d = i & 255;
            uint32_t cnt = 0u;
#pragma unroll
            for (int c = 0; c < kHistCopies; ++c) { cnt += sh[r][c][d]; sh[r][c][d] = 0u; }
            if (cnt) atomicAdd(out + i, cnt);
        }
    };
    for (int i = threadIdx.x; i < kRanks * kHistCopies * 256; i += kThreads) (&sh[0][0][0])[i] = 0u;
    for (int64_t ti = first; ti < last; ++ti) {
        const Tile t = tiles[ti];
        if (int(t.block) != cur_block) {                            // uniform over the CTA
            __syncthreads();
            if (cur_block >= 0) { flush(cur_block); __syncthreads(); }
            cur_block = int(t.block);
#pragma unroll
            for (int r = 0; r < kRanks; ++r) {
                const RankSel s = sel[size_t(t.block) * kRanks + r];
                prefix[r] = s.prefix; lead[r] = s.leader == r;
            }
        }
        const StatBlock* b = blocks + t.block;
        const int64_t numel = b->numel;
        const uint32_t* __restrict__ v = reinterpret_cast<const uint32_t*>(b->v);
        const int64_t base = int64_t(t.piece) * kTile;
        uint32_t u[16];
        int valid[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {                              // v is padded to whole quantisation blocks: in bounds whenever e < numel
            const int64_t e = base + int64_t(h) * (kThreads * 8) + int64_t(threadIdx.x) * 8;
            valid[h] = e < numel ? int(min64(8, numel - e)) : 0;
            uint4 a = make_uint4(0u, 0u, 0u, 0u), c = a;
            if (valid[h] > 0) { a = ld_stream_u4(v + e); c = ld_stream_u4(v + e + 4); }
            u[8 * h + 0] = a.x; u[8 * h + 1] = a.y; u[8 * h + 2] = a.z; u[8 * h + 3] = a.w;
            u[8 * h + 4] = c.x; u[8 * h + 5] = c.y; u[8 * h + 6] = c.z; u[8 * h + 7] = c.w;
        }
#pragma unroll
        for (int r = 0; r < kRanks; ++r) {
            if (!lead[r]) continue;
            int cur = -1;
            uint32_t n = 0u;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                if ((k & 7) < valid[k >> 3] && ((u[k] ^ prefix[r]) & high_mask) == 0u) {
                    const int d = int((u[k] >> shift) & 255u);
                    if (d == cur) {
                        ++n;
                    } else {
                        if (n) atomicAdd(&sh[r][copy][cur], n);
                        cur = d; n = 1u;
                    }
                }
            }
            if (n) atomicAdd(&sh[r][copy][cur], n);
        }
    }
    __syncthreads();
    if (cur_block >= 0) flush(cur_block);
}

// One thread per (block, rank): pick the digit that holds the rank, extend the
// prefix, and recompute which ranks still share a prefix.  Clears the
// histograms for the next pass.
__global__ void select_pick_kernel(RankSel* __restrict__ sel, uint32_t* __restrict__ hist, int n_blocks, int shift) {
    const int blk = blockIdx.x * blockDim.x + threadIdx.x;
    if (blk >= n_blocks) return;
    RankSel s[kRanks];
    for (int r = 0; r < kRanks; ++r) s[r] = sel[size_t(blk) * kRanks + r];
    for (int r = 0; r < kRanks; ++r) {
        const uint32_t* hh = hist + (size_t(blk) * kRanks + s[r].leader) * 256;
        int64_t rem = s[r].remaining;
        int d = 0;
        for (; d < 255; ++d) {
            const int64_t c = hh[d];
            if (rem < c) break;
            rem -= c;
        }
        s[r].remaining = rem;
        s[r].prefix |= uint32_t(d) << shift;
    }
    for (int r = 0; r < kRanks; ++r) {
        int leader = r;
        for (int q = 0; q < r; ++q)
            if (s[q].prefix == s[r].prefix) { leader = q; break; }
        s[r].leader = leader;
    }
    for (int r = 0; r < kRanks; ++r) sel[size_t(blk) * kRanks + r] = s[r];
    for (int i = 0; i < kRanks * 256; ++i) hist[size_t(blk) * kRanks * 256 + i] = 0u;
}

// Start of a select: ranks floor(q (n-1)) and the next one for q = 0.1, 0.9.
__global__ void select_init_kernel(const StatBlock* __restrict__ blocks, RankSel* __restrict__ sel,
                                   uint32_t* __restrict__ hist, int n_blocks) {
    const int blk = blockIdx.x * blockDim.x + threadIdx.x;
    if (blk >= n_blocks) return;
    const int64_t n = blocks[blk].numel;
    const double qs[2] = {0.1, 0.9};
    for (int k = 0; k < 2; ++k) {
        const double pos = qs[k] * double(n - 1);
        const int64_t lo = int64_t(floor(pos));
        const int64_t hi = min64(lo + 1, n - 1);
        sel[size_t(blk) * kRanks + 2 * k] = RankSel{0u, 0, lo};
        sel[size_t(blk) * kRanks + 2 * k + 1] = RankSel{0u, 0, hi};
    }
    for (int i = 0; i < kRanks * 256; ++i) hist[size_t(blk) * kRanks * 256 + i] = 0u;
}

// End of the window: gather everything the host needs into fin_out[block]:
//   [0..13] sweep-1 sums, [14..15] sweep-2 sums, [16..19] the four order
//   statistics (as doubles), [20..27] the running window values.
__global__ void stats_gather_kernel(const RankSel* __restrict__ sel, const double* __restrict__ acc,
                                    double* __restrict__ fin_out, int n_blocks) {
    const int blk = blockIdx.x * blockDim.x + threadIdx.x;
    if (blk >= n_blocks) return;
    double* o = fin_out + size_t(blk) * kFinOut;
    for (int r = 0; r < kRanks; ++r) o[16 + r] = double(__uint_as_float(sel[size_t(blk) * kRanks + r].prefix));
    for (int k = 0; k < kBlockAcc; ++k) o[20 + k] = acc[size_t(blk) * kBlockAcc + k];
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
sample_gather_kernel(const StatBlock* __restrict__ blocks, const Tile* __restrict__ tiles, const void* const* __restrict__ src) {
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

int launch_stats_step(const StatBlock* blocks, const Tile* tiles, const void* const* grads, double* partials,
                      int64_t n_tiles, float one_minus_beta_m, float one_minus_beta_v, cudaStream_t s) {
    stats_step_kernel<<<unsigned(n_tiles), kThreads, 0, s>>>(blocks, tiles, grads, partials, one_minus_beta_m,
                                                             one_minus_beta_v);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_stats_combine(const StatBlock* blocks, const double* partials, double* acc, int n_blocks, int has_prev,
                         double beta_rho, double eps, cudaStream_t s) {
    stats_combine_kernel<<<n_blocks, kThreads, 0, s>>>(blocks, partials, acc, has_prev, beta_rho, eps);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_final_sums(const StatBlock* blocks, const Tile* tiles, const float* const* params, double* fin,
                      double* fin_out, int64_t n_tiles, int n_blocks, double eps, float eps_adam, cudaStream_t s) {
    stats_final_sums_kernel<<<unsigned(n_tiles), kThreads, 0, s>>>(blocks, tiles, params, fin, eps, eps_adam);
    BAOC_LAUNCH_CHECK();
    stats_final_combine_kernel<<<n_blocks, kThreads, 0, s>>>(blocks, fin, fin_out);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_final_resid(const StatBlock* blocks, const Tile* tiles, const float* const* params, double* fin,
                       double* fin_out, int64_t n_tiles, int n_blocks, double eps, cudaStream_t s) {
    stats_final_resid_kernel<<<unsigned(n_tiles), kThreads, 0, s>>>(blocks, tiles, params, fin_out, fin, eps);
    BAOC_LAUNCH_CHECK();
    stats_resid_combine_kernel<<<n_blocks, kThreads, 0, s>>>(blocks, fin, fin_out);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_select(const StatBlock* blocks, const Tile* tiles, RankSel* sel, uint32_t* hist, int64_t n_tiles,
                  int n_blocks, cudaStream_t s) {
    const int tb = 128, gb = (n_blocks + tb - 1) / tb;
    select_init_kernel<<<gb, tb, 0, s>>>(blocks, sel, hist, n_blocks);
    BAOC_LAUNCH_CHECK();
    for (int shift = 24; shift >= 0; shift -= 8) {
        select_hist_kernel<<<unsigned((n_tiles + kHistTiles - 1) / kHistTiles), kThreads, 0, s>>>(blocks, tiles, sel, hist, n_tiles, shift);
        BAOC_LAUNCH_CHECK();
        select_pick_kernel<<<gb, tb, 0, s>>>(sel, hist, n_blocks, shift);
        BAOC_LAUNCH_CHECK();
    }
    return 0;
}

int launch_sample_gather(const StatBlock* blocks, const Tile* tiles, const void* const* src, int64_t n_tiles, int fp32,
                         cudaStream_t s) {
    if (fp32) sample_gather_kernel<float><<<unsigned(n_tiles), kThreads, 0, s>>>(blocks, tiles, src);
    else sample_gather_kernel<uint16_t><<<unsigned(n_tiles), kThreads, 0, s>>>(blocks, tiles, src);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_gather(const RankSel* sel, const double* acc, double* fin_out, int n_blocks, cudaStream_t s) {
    const int tb = 128, gb = (n_blocks + tb - 1) / tb;
    stats_gather_kernel<<<gb, tb, 0, s>>>(sel, acc, fin_out, n_blocks);
    BAOC_LAUNCH_CHECK();
    return 0;
}

}  // namespace baoc
