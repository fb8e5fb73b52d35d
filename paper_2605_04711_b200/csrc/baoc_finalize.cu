// End-of-window finalize of the sampling window (Sec. 3.3): the sums behind the
// signal-to-noise ratio (Eq. 5), the distortion (Eq. 6), the structure residual
// (Eq. 7) and the precision cosines (Eq. 8), and the exact quantiles behind the
// anisotropy (Eq. 4).  Three sweeps over the window's moments:
//   1. final_sums_kernel         reads m, v, theta: 16 sums per block, and the histogram of the top 12 bits of the
//                                select's key (SelKey: fitted per block to a sample of v by final_pilot_kernel)
//   2. final_resid_hist_kernel   reads v by pieces (rows of a strip of columns): Eq. 7 residual (after the row/column
//                                sums), histogram of the next digit of the elements that share a rank's first digit,
//                                and the list of those elements
//   3. final_last_kernel         reads those lists (well under a percent of v): histogram of the last digit
// A CTA of the first sweep works through a run of consecutive tiles, keeps its
// partial sums and histogram on chip while the tiles belong to one block, and
// hands them over once per block (a deterministic, fixed partition of the work).
#include <cstring>
#include <type_traits>

#include "baoc_device.cuh"

namespace baoc {

// ============================================================================
// Pilot value of the preconditioner p = 1/(sqrt(v)+eps) of Eq. 6: the mean of p
// over up to 1024 evenly spaced elements of the block.  Eq. 6 needs
// sum ((p/pbar - 1) theta)^2, which a single sweep can only form from sums that
// do not involve pbar; sums of the deviations p - p0 from a pilot value close
// to pbar do that without cancellation (p0 = pbar would be exact), and for a
// block whose p are all equal p0 is exactly that value and every deviation 0.
// ============================================================================
__device__ __forceinline__ float precond_of(float v, float eps) { return rcp_approx(sqrt_approx(v) + eps); }

// ---- the key of the quantile select (see SelKey) --------------------------------
// clamp(pattern - lo, 0, wmax) in two instructions; lo >= -1, and a pattern with the sign bit set (no second moment has
// one) counts as below everything.
__device__ __forceinline__ uint32_t sel_key(uint32_t pattern, int lo, int wmax) {
    return uint32_t(min(__viaddmax_s32_relu(int(pattern), -lo, 0), wmax));
}
__device__ __forceinline__ int sel_wmax(int s) { return int((uint32_t(kSelBins) << s) - 1u); }
// lowest bit and width of the digit of pass 0, 1, 2
__device__ __forceinline__ void sel_digit(int s, int pass, int& shift, int& bits) {
    const int b2 = s < kSelBits ? s : kSelBits;
    if (pass == 0) { shift = s; bits = kSelBits; }
    else if (pass == 1) { shift = s - b2; bits = b2; }
    else { shift = 0; bits = s - b2; }
}

// Also the key of the block's select: lo one below the smallest pattern of the sample, s the smallest shift for which
// the largest pattern of the sample stays below the top of the key range.
__global__ void __launch_bounds__(kThreads)
final_pilot_kernel(const StatBlock* __restrict__ blocks, float eps, float v_scale, double* __restrict__ fin_out,
                   SelKey* __restrict__ selkey) {
    __shared__ double total[1];
    __shared__ int s_min, s_max;
    const StatBlock* b = blocks + blockIdx.x;
    const int64_t numel = b->numel;
    const int64_t n = min64(numel, 1024);
    const int64_t stride = numel / n;
    if (threadIdx.x == 0) { s_min = 0x7f800000; s_max = 0; }
    __syncthreads();
    double acc[1] = {0.0};
    int lo = 0x7f800000, hi = 0;
    for (int64_t k = threadIdx.x; k < n; k += kThreads) {
        const float x = b->v[k * stride];
        acc[0] += double(precond_of(x * v_scale, eps));          // (the key is fitted to v as stored: a positive factor keeps the order)
        const int pat = min(max(__float_as_int(x), 0), 0x7f800000);
        lo = min(lo, pat); hi = max(hi, pat);
    }
    lo = __reduce_min_sync(0xffffffffu, lo); hi = __reduce_max_sync(0xffffffffu, hi);
    if ((threadIdx.x & 31) == 0) { atomicMin(&s_min, lo); atomicMax(&s_max, hi); }
    cta_reduce_store<1>(acc, total);
    // n identical fp32 values sum exactly in double, and the correctly rounded quotient is that value again
    if (threadIdx.x == 0) {
        fin_out[size_t(blockIdx.x) * kFinOut + kFinPilot] = double(float(total[0] / double(n)));
        SelKey key;
        key.lo = s_min - 1;
        const int64_t top = int64_t(s_max) - key.lo + 2;       // the sample's largest key, and one value above it, below wmax
        key.s = 0;
        while (key.s < kSelFullS && (int64_t(kSelBins) << key.s) < top) ++key.s;
        selkey[blockIdx.x] = key;
    }
}

// ============================================================================
// Sweep 1.  Per block, 16 sums over the window's moments (fp32), the parameters
// and the quantised moments:
//   0 sum m^2      1 sum v        2 sum v^2       3 sum (p - p0)
//   4 sum theta^2  5 sum u32^2    6 sum u8^2      7 sum u32*u8
//   8 sum u16^2    9 sum u32*u16  10 sum (m-m8)^2 11 sum (v-v8)^2
//   12 sum (m-m16)^2              13 sum (v-v16)^2
//   14 sum (p - p0) theta^2       15 sum (p - p0)^2 theta^2
// with u = m/(sqrt(v)+eps_adam) from full-precision, 8-bit and bf16 moments and
// p0 the block's pilot value.  A warp owns one 256-element quantisation block per
// slice, so the absmax is a warp reduction.
//
// Everything is evaluated in fp32, two elements per instruction: the sums are
// compared at 1e-4, far above fp32 rounding, and a code that lands on the other
// side of a rounding tie moves a cosine by less than 1e-8.  Square roots and
// reciprocals are the approximate ones (2^-23).  The bf16 round trip is a
// Veltkamp split (x*(2^16+1) - (x*(2^16+1) - x) keeps the upper 8 significant
// bits, rounded to nearest), which runs on the FMA pipe instead of the narrow
// conversion pipe.  A thread keeps its partial sums in fp32 for at most
// kFinRunTiles tiles (512 elements per thread) and widens them to double for the
// reduction across the CTA.
//
// The slices are staged through shared memory by per-thread cp.async copies two
// slices ahead (96 bytes per thread and slice: m, v, theta), so loads in flight
// hold no registers during the long arithmetic of the current slice.
// ============================================================================
// One tile of the first sweep as its slices see it.
struct FsTile {
    const float* m;      // the tile's first element of m, v and theta
    const float* v;
    const float* th;
    int left;            // elements of the block from there on, at most a tile's
    int block;
    float p0;            // the block's pilot value and select key
    int key_lo, key_s;
};

constexpr int kFsStageBytes = kThreads * 96;                 // m (32 B/thread) at 0, v at 8192, theta at 16384
constexpr int kFsStages = 3;
constexpr int kFsSmemBytes = kFsStages * kFsStageBytes + kSelBins * 4 + 4096;   // the staging ring, the histogram of the first digit, the codebook

__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ float rsqrt_approx(float x) {
    float r;
    asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

// One slice of eight elements per thread (a warp: one 256-element quantisation block).  kFull: all eight elements of
// every lane of the warp lie inside the block; otherwise cnt of them do and the padding (m = v = theta = 0) is
// masked out of the one sum it would otherwise enter (p - p0).
//
// The bf16 direction costs no extra square root or reciprocal: with n = (v - v16) / v (|n| <= 2^-8),
// sqrt(v16) - sqrt(v) = -sqrt(v) n (1/2 + n/8) up to n^3, and with e that difference over (sqrt(v) + eps_adam)
// (|e| <= 2^-9), 1 / (sqrt(v16) + eps_adam) = (1 - e + e^2) / (sqrt(v) + eps_adam) up to e^3: both truncations are
// below 1e-8 of the direction, far below what a cosine compared at 1e-4 can see.
// kDyn: the 8-bit round trip goes through the non-linear codebook (dyn: its fp32 tables in shared memory) instead of the
// linear absmax codes.
// kDebias: m and v are multiplied by m_scale and v_scale first (the select's digit is taken from v as stored).
template <bool kFull, bool kDyn, bool kDebias>
__device__ __forceinline__ void fs_slice(float (&mm)[8], float (&vv)[8], const float (&tt)[8], int cnt,
                                         float p0, float eps_f, float eps_adam, f32x2 (&F)[kFinalSums], uint32_t* hist1,
                                         int key_lo, int key_s, float m_scale, float v_scale, const float* dyn) {
    // ---- first radix pass of the quantile select: the top 12 bits of the block's key (see SelKey).  The key range is
    // fitted to the block, so its second moments spread over most of the 4096 bins and a plain shared-memory histogram
    // with one atomic per element meets few collisions.
#pragma unroll
    for (int j = 0; j < 8; ++j)
        if (kFull || j < cnt)
            atomicAdd(hist1 + min(__viaddmax_s32_relu(__float_as_int(vv[j]), -key_lo, 0) >> key_s, kSelBins - 1), 1u);
    if (kDebias) {
#pragma unroll
        for (int j = 0; j < 8; ++j) { mm[j] *= m_scale; vv[j] *= v_scale; }
    }
    const f32x2 P0 = splat2(p0), MAGIC = splat2(12582912.0f), C16 = splat2(65537.0f), EA = splat2(eps_adam), EPS = splat2(eps_f),
                ONE = splat2(1.0f), MONE = splat2(-1.0f);
    // ---- absmax of the warp's quantisation block, code scales
    float am = 0.f, av = 0.f;
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        am = max3(am, fabsf(mm[2 * p]), fabsf(mm[2 * p + 1]));
        av = max3(av, vv[2 * p], vv[2 * p + 1]);
    }
    am = warp_max_nonneg(am); av = warp_max_nonneg(av);
    const float rm0 = rcp_approx(am), rv0 = rcp_approx(av);          // L / a from the reciprocal and one Newton step
    const f32x2 KM = splat2(am > 0.f ? 127.0f * (rm0 * fmaf(-am, rm0, 2.0f)) : 0.f);
    const f32x2 KV = splat2(av > 0.f ? 255.0f * (rv0 * fmaf(-av, rv0, 2.0f)) : 0.f);
    // a / L in two parts (the second one the exact remainder of the first, divided by L), so that code * a / L comes
    // out correctly rounded and the block's largest element, whose code is L, is reproduced exactly
    const float dmh = am * (1.0f / 127.0f), dvh = av * (1.0f / 255.0f);
    const f32x2 DM = splat2(dmh), DV = splat2(dvh);
    const f32x2 DML = splat2(fmaf(-127.0f, dmh, am) * (1.0f / 127.0f)), DVL = splat2(fmaf(-255.0f, dvh, av) * (1.0f / 255.0f));

#pragma unroll
    for (int p = 0; p < 4; ++p) {
        const f32x2 M = pack2(mm[2 * p], mm[2 * p + 1]), V = pack2(vv[2 * p], vv[2 * p + 1]);
        const f32x2 T = pack2(tt[2 * p], tt[2 * p + 1]);
        // 8-bit round trips: code = rne(x L / a) by the magic-number addition, value = code a / L
        f32x2 M8, V8;
        if (kDyn) {
            const float ia = am > 0.f ? rm0 : 0.f, iv = av > 0.f ? rv0 : 0.f;
            M8 = pack2(dyn[dyn_nearest_f32(dyn + 256, mm[2 * p] * ia)] * am, dyn[dyn_nearest_f32(dyn + 256, mm[2 * p + 1] * ia)] * am);
            V8 = pack2(dyn[512 + dyn_nearest_f32(dyn + 768, vv[2 * p] * iv)] * av, dyn[512 + dyn_nearest_f32(dyn + 768, vv[2 * p + 1] * iv)] * av);
        } else {
            const f32x2 QM = sub2(fma2(M, KM, MAGIC), MAGIC), QV = sub2(fma2(V, KV, MAGIC), MAGIC);
            M8 = fma2(QM, DM, mul2(QM, DML)); V8 = fma2(QV, DV, mul2(QV, DVL));
        }
        // bf16 round trips
        const f32x2 CM = mul2(M, C16), CV = mul2(V, C16);
        // (written as x*(-1) + y: a plain packed subtraction here came out as the identity, the two differences folded)
        const f32x2 M16 = fma2(fma2(M, MONE, CM), MONE, CM), V16 = fma2(fma2(V, MONE, CV), MONE, CV);
        const f32x2 E0 = sub2(M, M8), E1 = sub2(V, V8), E2 = sub2(M, M16), E3 = sub2(V, V16);
        // full-precision direction and the preconditioner: sqrt(v) = v rsqrt(v) (a v below the smallest normal number
        // counts as that number under the root: its root is far below either epsilon)
        float a0, a1, b0, b1;
        const f32x2 R = pack2(rsqrt_approx(fmaxf(vv[2 * p], 1.17549435e-38f)), rsqrt_approx(fmaxf(vv[2 * p + 1], 1.17549435e-38f)));
        const f32x2 S = mul2(V, R);
        unpack2(add2(S, EA), a0, a1);
        const f32x2 R32 = pack2(rcp_approx(a0), rcp_approx(a1));
        const f32x2 U32 = mul2(M, R32);
        unpack2(add2(S, EPS), a0, a1);
        f32x2 PD = sub2(pack2(rcp_approx(a0), rcp_approx(a1)), P0);
        if (!kFull) PD = mul2(PD, pack2(2 * p < cnt ? 1.f : 0.f, 2 * p + 1 < cnt ? 1.f : 0.f));
        // 8-bit direction: the quantised second moment is not close to v in relative terms, so its own root
        unpack2(V8, b0, b1);
        unpack2(add2(pack2(sqrt_approx(b0), sqrt_approx(b1)), EA), b0, b1);
        const f32x2 U8 = mul2(M8, pack2(rcp_approx(b0), rcp_approx(b1)));
        // bf16 direction from the series
        const f32x2 N = mul2(E3, mul2(R, R));
        const f32x2 H = mul2(N, fma2(N, splat2(0.125f), splat2(0.5f)));
        const f32x2 NE = mul2(mul2(S, H), R32);                                  // -(sqrt(v16) - sqrt(v)) / (sqrt(v) + eps_adam)
        const f32x2 U16 = mul2(M16, mul2(R32, fma2(NE, add2(NE, ONE), ONE)));
        // the sums
        F[0] = fma2(M, M, F[0]); F[1] = add2(F[1], V); F[2] = fma2(V, V, F[2]); F[3] = add2(F[3], PD);
        const f32x2 T2 = mul2(T, T), PT = mul2(PD, T2);
        F[4] = add2(F[4], T2); F[14] = add2(F[14], PT); F[15] = fma2(PD, PT, F[15]);
        F[5] = fma2(U32, U32, F[5]); F[6] = fma2(U8, U8, F[6]); F[7] = fma2(U32, U8, F[7]);
        F[8] = fma2(U16, U16, F[8]); F[9] = fma2(U32, U16, F[9]);
        F[10] = fma2(E0, E0, F[10]); F[11] = fma2(E1, E1, F[11]); F[12] = fma2(E2, E2, F[12]); F[13] = fma2(E3, E3, F[13]);
    }
}

template <bool kDyn, bool kDebias>
__global__ void __launch_bounds__(kThreads, 2)
final_sums_kernel(const StatBlock* __restrict__ blocks, const Tile* __restrict__ tiles,
                  const float* const* __restrict__ params, double* __restrict__ fin,
                  const double* __restrict__ fin_out, uint32_t* __restrict__ hist, const SelKey* __restrict__ selkey,
                  int64_t n_tiles, int tiles_per_cta, float eps_f, float eps_adam, float m_scale, float v_scale BAOC_CHECK_PARAM) {
#ifdef BAOC_CHECKED
    {   // validate every tile of this CTA's run, and the ranges of the workspace it will touch, before touching anything
        const int64_t c0 = int64_t(blockIdx.x) * tiles_per_cta, c1 = min64(c0 + tiles_per_cta, n_tiles);
        if (c0 >= ck.n_tiles || n_tiles != ck.n_tiles) { check_fail(kChkTileIndex, kKerFinalSums, c0, ck.n_tiles, n_tiles, 0); return; }
        for (int64_t ti = c0; ti < c1; ++ti) {
            const Tile ct = tiles[ti];
            if (ct.block >= unsigned(ck.n_blocks)) { check_fail(kChkBlockIndex, kKerFinalSums, ct.block, ck.n_blocks, ti, 0); return; }
            const StatBlock* cb = blocks + ct.block;
            const int64_t cbase = int64_t(ct.piece) * kTile;
            const int64_t cpad = (cb->numel + kQBlock - 1) / kQBlock * kQBlock, cn = min64(kTile, cpad - cbase);
            if (!check_tile(ck, kKerFinalSums, ti, ct.block, cbase, cb->numel) ||
                !check_range(ck, kKerFinalSums, cb->m + cbase, 4 * cn, 0) || !check_range(ck, kKerFinalSums, cb->v + cbase, 4 * cn, 1) ||
                !check_range(ck, kKerFinalSums, fin + size_t(ti) * kFinalSums, 8 * kFinalSums, 2) ||
                !check_range(ck, kKerFinalSums, hist + size_t(ct.block) * kRanks * kSelBins, 4ll * kSelBins, 3) ||
                !check_range(ck, kKerFinalSums, fin_out + size_t(ct.block) * kFinOut, 8 * kFinOut, 4) ||
                !check_caller_ptr(kKerFinalSums, params[ct.block], 5))
                return;
        }
    }
#endif
    extern __shared__ __align__(16) unsigned char dyn[];
    unsigned char* stage = dyn;
    uint32_t* hist1 = reinterpret_cast<uint32_t*>(dyn + kFsStages * kFsStageBytes);      // kSelBins counters
    float* dyn_tables = reinterpret_cast<float*>(dyn + kFsStages * kFsStageBytes + kSelBins * 4);
    if (kDyn) dyn_build_f32(dyn_tables);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t first = int64_t(blockIdx.x) * tiles_per_cta, last = min64(first + tiles_per_cta, n_tiles);
    const int nsl = int(last - first) * (kTile / (kThreads * 8));     // slices of this CTA
    const uint32_t sm0 = smem_addr(stage);
    // a thread's 32 bytes per array as two 16-byte pieces: the lanes' first pieces lie side by side, then their second
    // pieces, so that a quarter warp's 16-byte accesses cover 128 contiguous bytes (no bank conflicts)
    const uint32_t om = uint32_t(warp) * 1024u + uint32_t(lane) * 16u, ov = 8192 + om, ot = 16384 + om;
    constexpr uint32_t kHalf = 512;

    // What the slices of the CTA's tiles need from the tables, gathered once (one thread per tile follows the chain
    // tile -> block -> pointers; the slices then read it from shared memory instead of following it themselves).
    __shared__ FsTile desc[kFinRunTiles];
    if (threadIdx.x < int(last - first)) {
        const Tile t = tiles[first + threadIdx.x];
        const StatBlock* b = blocks + t.block;
        const int64_t base = int64_t(t.piece) * kTile;
        const SelKey key = selkey[t.block];
        FsTile d;
        d.m = b->m + base; d.v = b->v + base; d.th = params[t.block] + base;
        d.left = int(min64(b->numel - base, kTile));
        d.block = int(t.block);
        d.p0 = float(fin_out[size_t(t.block) * kFinOut + kFinPilot]);
        d.key_lo = key.lo; d.key_s = key.s;
        desc[threadIdx.x] = d;
    }
    for (int i = threadIdx.x; i < kSelBins; i += kThreads) hist1[i] = 0u;
    __syncthreads();

    f32x2 F[kFinalSums];
#pragma unroll
    for (int k = 0; k < kFinalSums; ++k) F[k] = pack2(0.f, 0.f);

    // hand the finished run of tiles of block blk over: its sums go to the slot of its first tile (the per-block
    // combine adds the slots of the runs' first tiles), its histogram to the block's global one
    auto flush = [&](int blk, int64_t t_begin) {
        double acc[kFinalSums];
#pragma unroll
        for (int k = 0; k < kFinalSums; ++k) {
            float lo, hi;
            unpack2(F[k], lo, hi);
            acc[k] = double(lo) + double(hi);
            F[k] = pack2(0.f, 0.f);
        }
        cta_reduce_store<kFinalSums>(acc, fin + size_t(t_begin) * kFinalSums);
        uint32_t* out = hist + size_t(blk) * kRanks * kSelBins;          // all four ranks still share one histogram
        for (int d = threadIdx.x; d < kSelBins; d += kThreads) {
            const uint32_t cnt = hist1[d];
            if (cnt) { atomicAdd(out + d, cnt); hist1[d] = 0u; }
        }
        __syncthreads();
    };

    // Each thread copies the 32 bytes per array that hold its own eight elements, as two 16-byte copies through L1:
    // the second copy finds its 32-byte sector there, so that L2 serves every sector once.
    uint32_t fill = 0, take = 0;
    const int in_slice = threadIdx.x * 8;                    // the thread's first element within a slice
    auto prefetch = [&](int k) {
        if (k < nsl) {
            const FsTile& t = desc[k >> 1];
            const int e = (k & 1) * (kThreads * 8) + in_slice;           // within the tile
            // m and v are padded with zeros to whole quantisation blocks: in bounds whenever the warp's block starts
            // inside the array; theta is not padded
            if (e - lane * 8 < t.left) {
                const uint32_t d = sm0 + fill;
                const float* pm = t.m + e;
                const float* pv = t.v + e;
                cp_async16_l1(d + om, pm); cp_async16_l1(d + om + kHalf, pm + 4);
                cp_async16_l1(d + ov, pv); cp_async16_l1(d + ov + kHalf, pv + 4);
                if (e + 8 <= t.left) {
                    const float* pt = t.th + e;
                    cp_async16_l1(d + ot, pt); cp_async16_l1(d + ot + kHalf, pt + 4);
                }
            }
        }
        cp_async_commit();
        fill = fill == (kFsStages - 1) * kFsStageBytes ? 0u : fill + kFsStageBytes;
    };
#pragma unroll
    for (int k = 0; k < kFsStages - 1; ++k) prefetch(k);

    int cur_block = -1;
    int64_t run_first = first;
    float p0 = 0.f;
    int key_lo = 0, key_s = 0;
#pragma unroll 1
    for (int k = 0; k < nsl; ++k) {
        prefetch(k + kFsStages - 1);
        cp_async_wait<kFsStages - 1>();                      // this slice's copies have landed
        const FsTile& t = desc[k >> 1];
        if (t.block != cur_block) {                          // uniform over the CTA; only at a tile boundary
            if (cur_block >= 0) flush(cur_block, run_first);
            cur_block = t.block;
            run_first = first + (k >> 1);
            p0 = t.p0; key_lo = t.key_lo; key_s = t.key_s;
        }
        const unsigned char* mine = stage + take;
        take = take == (kFsStages - 1) * kFsStageBytes ? 0u : take + kFsStageBytes;
        const int left = t.left;
        const int w0 = (k & 1) * (kThreads * 8) + warp * kQBlock;        // the warp's quantisation block, within the tile
        if (w0 >= left) continue;                            // whole warp out of range
        float mm[8], vv[8], tt[8];
        f4_to8(*reinterpret_cast<const float4*>(mine + om), *reinterpret_cast<const float4*>(mine + om + kHalf), mm);
        f4_to8(*reinterpret_cast<const float4*>(mine + ov), *reinterpret_cast<const float4*>(mine + ov + kHalf), vv);
        if (w0 + kQBlock <= left) {                          // uniform over the warp
            f4_to8(*reinterpret_cast<const float4*>(mine + ot), *reinterpret_cast<const float4*>(mine + ot + kHalf), tt);
            fs_slice<true, kDyn, kDebias>(mm, vv, tt, 8, p0, eps_f, eps_adam, F, hist1, key_lo, key_s, m_scale, v_scale, dyn_tables);
        } else {
            const int e = w0 + lane * 8;
            const int cnt = max(0, min(8, left - e));
            if (cnt == 8) {
                f4_to8(*reinterpret_cast<const float4*>(mine + ot), *reinterpret_cast<const float4*>(mine + ot + kHalf), tt);
            } else {
                const float* th = t.th;
#pragma unroll
                for (int j = 0; j < 8; ++j) tt[j] = j < cnt ? th[e + j] : 0.f;
            }
            fs_slice<false, kDyn, kDebias>(mm, vv, tt, cnt, p0, eps_f, eps_adam, F, hist1, key_lo, key_s, m_scale, v_scale, dyn_tables);
        }
    }
    cp_async_wait<0>();
    if (cur_block >= 0) flush(cur_block, run_first);
}

// Per-block combines of the sweeps.  A sweep's CTA b works through the tiles [b per, (b+1) per) of the tile table and
// leaves the sums of each run of tiles of one block in the slot of the run's first tile; the runs of a block therefore
// start at its first tile and at every multiple of `per` inside it.  Their slots are added in tile order.
template <int K>
__device__ __forceinline__ void block_runs_sum(const double* __restrict__ part, int64_t tile0, int ntiles, int per, double* out) {
    double acc[K];
#pragma unroll
    for (int k = 0; k < K; ++k) acc[k] = 0.0;
    const int64_t r0 = tile0 / per;                          // the run that holds the block's first tile
    const int nruns = int((tile0 + ntiles - 1) / per - r0) + 1;
    for (int i = threadIdx.x; i < nruns; i += kThreads) {
        const int64_t head = i == 0 ? tile0 : (r0 + i) * per;
        const double* p = part + size_t(head) * K;
#pragma unroll
        for (int k = 0; k < K; ++k) acc[k] += p[k];
    }
    cta_reduce_store<K>(acc, out);
}

__global__ void __launch_bounds__(kThreads)
final_sums_combine_kernel(const StatBlock* __restrict__ blocks, const double* __restrict__ fin, double* __restrict__ fin_out, int per) {
    const StatBlock* b = blocks + blockIdx.x;
    block_runs_sum<kFinalSums>(fin, b->tile0, b->ntiles, per, fin_out + size_t(blockIdx.x) * kFinOut);
}

__global__ void __launch_bounds__(kThreads)
final_resid_combine_kernel(const StatBlock* __restrict__ blocks, const double* __restrict__ resid_part, double* __restrict__ fin_out) {
    const StatBlock* b = blocks + blockIdx.x;
    block_tiles_sum<kResidSums>(resid_part, b->piece0, b->npieces, fin_out + size_t(blockIdx.x) * kFinOut + kFinResid);
}

// ============================================================================
// Sweeps 2 and 3: the remaining radix passes of the exact quantile select over
// the keys of v (see SelKey): four ranks per block (the two order statistics
// around each of the two quantile positions); ranks that still share a prefix
// share one histogram (the "leader" rank's).  The first pass (top 12 bits of the
// key) is part of the first sweep.
//
// Sweep 2 (final_resid_hist_kernel) reads v once more, piece by piece (SelPiece:
// a run of rows of a strip of at most 512 columns): the second pass, the next
// min(12, s) bits of the elements whose first digit is a rank's (the "survivors"),
// and in the same sweep the Eq. 7 numerator
//     sum (S_ij - a_i b_j / mu)^2 = sum (v_ij - rowsum_i colsum_j / total)^2
// of matrix blocks, in double (a difference of nearly equal numbers).  A thread
// keeps eight adjacent columns for all rows of the piece, so the column sums sit
// in registers and a row costs one row sum per thread.
// Survivors are few (the key range is fitted to the block, a bin of the first
// digit holds a fraction of a percent of it), so they are not counted where they
// are found, which would leave most lanes idle around every atomic: a thread
// copies its survivors to its warp's staging segment, and the warp counts the
// staged keys with all lanes busy (lanes holding equal keys add once) when the
// segment runs full or the piece ends.  The staged keys also go to the piece's
// survivors list in global memory.
//
// Sweep 3 (final_last_kernel) reads those lists instead of v: the third pass, the
// last s - 12 bits of the survivors whose upper bits are a rank's prefix.  A piece
// whose survivors did not fit its slots (more than one element in eight: a
// constant or nearly constant tensor) is marked, and the third pass reads v for it.
//
// The second pass counts in 16 bits, two bins per word (32 KB of histograms for a
// piece of at most 49152 elements), next to 32 KB of staging.
// ============================================================================
constexpr int kRhHistWords = kSelBins / 2;
constexpr int kRhHistBytes = kRanks * kRhHistWords * 4;
constexpr int kRhSegWords = 1024;                             // a warp's staging segment
constexpr int kRhBatch = 2;                                   // rows a thread requests before it uses the first
constexpr int kRhDrainAt = kRhSegWords - kRhBatch * 32 * 8;   // staged keys above which the segment may not hold another batch
constexpr int kRhSmemBytes = kRhHistBytes + (kThreads / 32) * kRhSegWords * 4;
static_assert(kPieceElems < 65536, "a 16-bit bin must hold a whole piece");
static_assert(kRhDrainAt >= 0, "a batch of rows must fit the staging segment");

// The distinct prefixes the ranks of a block still have (one per leader), padded with a value no key takes.
struct Leaders {
    uint32_t key[kRanks];
    int slot[kRanks];
    int n;
};
__device__ __forceinline__ Leaders leaders_of(const RankSel* __restrict__ sel, int key_shift) {
    Leaders L;
    L.n = 0;
#pragma unroll
    for (int r = 0; r < kRanks; ++r) { L.key[r] = 0xffffffffu; L.slot[r] = 0; }
#pragma unroll
    for (int r = 0; r < kRanks; ++r) {
        const RankSel s = sel[r];
        if (s.leader == r) {
#pragma unroll
            for (int k = 0; k < kRanks; ++k)
                if (k == L.n) { L.key[k] = s.prefix >> key_shift; L.slot[k] = r; }
            ++L.n;
        }
    }
    return L;
}

// Geometry of a piece for the CTA: threads across (8 columns each), rows per step.
struct PieceGeom {
    int cols;        // row length of the block (kPieceCols for a vector block)
    int width;       // columns of the piece
    int tx, ty;      // this thread's place: columns col0 + 8 tx .. + 7 of rows row0 + ty, row0 + ty + step, ...
    int step;
    int nc;          // columns of this thread that exist (0..8)
    bool vec;        // rows start 16-byte aligned: 16-byte loads
};
__device__ __forceinline__ PieceGeom piece_geom(const SelPiece& pc, const StatBlock* b) {
    PieceGeom g;
    g.cols = b->cols > 1 ? b->cols : kPieceCols;
    g.width = min(kPieceCols, g.cols - int(pc.col0));
    int across = 1, sh = 0;
    while (across * 8 < g.width) { across <<= 1; ++sh; }
    g.tx = threadIdx.x & (across - 1); g.ty = threadIdx.x >> sh;
    g.step = kThreads >> sh;
    g.nc = max(0, min(8, g.width - g.tx * 8));
    g.vec = (g.cols & 3) == 0;
    return g;
}
// The thread's eight patterns of row r (zeros where there is no element); returns how many exist.
__device__ __forceinline__ int piece_load(const uint32_t* __restrict__ v, const SelPiece& pc, const PieceGeom& g, int64_t numel,
                                          int64_t r, uint32_t (&u)[8]) {
    const int64_t e = r * g.cols + pc.col0 + g.tx * 8;
    const int n = int(max64(0, min64(g.nc, numel - e)));          // (a vector block's last row may be short)
    if (g.vec && n == 8) {
        const uint4 a = ld_stream_u4(v + e), c = ld_stream_u4(v + e + 4);
        u[0] = a.x; u[1] = a.y; u[2] = a.z; u[3] = a.w; u[4] = c.x; u[5] = c.y; u[6] = c.z; u[7] = c.w;
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) u[j] = j < n ? v[e + j] : 0u;
    }
    return n;
}

__global__ void __launch_bounds__(kThreads, 3)
final_resid_hist_kernel(const StatBlock* __restrict__ blocks, const SelPiece* __restrict__ pieces, const RankSel* __restrict__ sel,
                        const SelKey* __restrict__ selkey, double* __restrict__ resid_part, uint32_t* __restrict__ hist,
                        uint32_t* __restrict__ surv, uint32_t* __restrict__ surv_cnt, int64_t n_pieces, int with_resid BAOC_CHECK_PARAM) {
    const SelPiece pc = pieces[blockIdx.x];
#ifdef BAOC_CHECKED
    {
        if (int64_t(blockIdx.x) >= ck.n_tiles || n_pieces != ck.n_tiles) { check_fail(kChkTileIndex, kKerFinalHist, blockIdx.x, ck.n_tiles, n_pieces, 0); return; }
        if (pc.block >= unsigned(ck.n_blocks)) { check_fail(kChkBlockIndex, kKerFinalHist, pc.block, ck.n_blocks, blockIdx.x, 0); return; }
        const StatBlock* cb = blocks + pc.block;
        const int64_t ccols = cb->cols > 1 ? cb->cols : kPieceCols, crows = cb->cols > 1 ? cb->rows : (cb->numel + kPieceCols - 1) / kPieceCols;
        if (int64_t(pc.col0) >= ccols || int64_t(pc.row0) + pc.nrows > crows || pc.nrows == 0) { check_fail(kChkTileStart, kKerFinalHist, pc.col0, ccols, pc.row0 + pc.nrows, crows); return; }
        const int64_t cpad = (cb->numel + kQBlock - 1) / kQBlock * kQBlock;
        if (!check_range(ck, kKerFinalHist, cb->v, 4 * cpad, 0) ||
            !check_range(ck, kKerFinalHist, hist + size_t(pc.block) * kRanks * kSelBins, 4ll * kRanks * kSelBins, 1) ||
            !check_range(ck, kKerFinalHist, sel + size_t(pc.block) * kRanks, int64_t(sizeof(RankSel)) * kRanks, 2) ||
            !check_range(ck, kKerFinalHist, resid_part + blockIdx.x, 8, 3) ||
            !check_range(ck, kKerFinalHist, surv + pc.surv_off, 4ll * pc.slots, 6) ||
            !check_range(ck, kKerFinalHist, surv_cnt + blockIdx.x, 4, 7) ||
            (cb->cols > 1 && (!check_range(ck, kKerFinalHist, cb->rowsum, 8ll * (cb->rows + 1), 4) ||
                              !check_range(ck, kKerFinalHist, cb->colsum, 8ll * cb->cols, 5))))
            return;
    }
#endif
    extern __shared__ __align__(16) unsigned char dyn[];
    uint32_t (*sh)[kRhHistWords] = reinterpret_cast<uint32_t (*)[kRhHistWords]>(dyn);
    uint32_t* stage = reinterpret_cast<uint32_t*>(dyn + kRhHistBytes);
    __shared__ int wcnt[kThreads / 32];                       // keys a warp has staged
    __shared__ int run_cnt, run_over;                         // survivors of the piece listed so far; the piece outgrew its slots
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const StatBlock* b = blocks + pc.block;
    const SelKey key = selkey[pc.block];
    if (key.s < 0) return;                                    // uniform over the CTA: the block sits this round out
    int d_shift, d_bits;
    sel_digit(key.s, 1, d_shift, d_bits);
    const int wmax = sel_wmax(key.s);
    const bool resid = with_resid != 0 && b->cols > 1;
    if (!resid && d_bits == 0) {                              // nothing to do here (uniform)
        if (threadIdx.x == 0) { surv_cnt[blockIdx.x] = 0u; if (with_resid) resid_part[blockIdx.x] = 0.0; }
        return;
    }
    const Leaders L = leaders_of(sel + size_t(pc.block) * kRanks, key.s);
    const PieceGeom g = piece_geom(pc, b);
    const int64_t numel = b->numel;
    const uint32_t* __restrict__ v = reinterpret_cast<const uint32_t*>(b->v);
    uint32_t* seg = stage + warp * kRhSegWords;
    uint32_t* list = surv + pc.surv_off;

    if (d_bits > 0)
        for (int i = threadIdx.x; i < kRanks * kRhHistWords; i += kThreads) (&sh[0][0])[i] = 0u;
    if (threadIdx.x < kThreads / 32) wcnt[threadIdx.x] = 0;
    if (threadIdx.x == 0) { run_cnt = 0; run_over = 0; }
    // the thread's column sums, and 1 / total
    double cs[8];
    double inv_total = 0.0;
    const double* __restrict__ rowsum = b->rowsum;
    if (resid) {
        const double total = rowsum[b->rows];                 // the block's sum of v, left there by the row/column combine
        inv_total = total > 0.0 ? 1.0 / total : 0.0;
#pragma unroll
        for (int j = 0; j < 8; ++j) cs[j] = j < g.nc ? b->colsum[pc.col0 + g.tx * 8 + j] : 0.0;
    }
    __syncthreads();

    // the warp's staged keys: listed, and counted into the histograms of this pass's digit
    auto drain = [&]() {
        const int staged = wcnt[warp];                        // uniform over the warp
        if (staged == 0) return;
        int off = 0;
        if (lane == 0) {
            off = atomicAdd(&run_cnt, staged);
            if (off + staged > int(pc.slots)) run_over = 1;
        }
        off = __shfl_sync(0xffffffffu, off, 0);
        const bool fits = off + staged <= int(pc.slots);
        for (int i0 = 0; i0 < staged; i0 += 32) {
            const int i = i0 + lane;
            const bool on = i < staged;
            const unsigned act = __ballot_sync(0xffffffffu, on);
            if (on) {
                const uint32_t x = seg[i];
                if (fits) list[off + i] = x;
                const unsigned same = __match_any_sync(act, x);
                if (lane == __ffs(int(same)) - 1) {           // one lane per distinct key adds for all of them
                    const uint32_t top = x >> key.s, d = (x >> d_shift) & ((1u << d_bits) - 1u);
                    const uint32_t n = uint32_t(__popc(same)) << ((d & 1u) * 16u);
#pragma unroll
                    for (int k = 0; k < kRanks; ++k)
                        if (top == L.key[k]) atomicAdd(&sh[k][d >> 1], n);
                }
            }
        }
        __syncwarp();
        if (lane == 0) wcnt[warp] = 0;
        __syncwarp();
    };

    double acc[kResidSums] = {0.0};
    const int64_t r_end = int64_t(pc.row0) + pc.nrows;
    // Which elements survive.  A leader whose first digit is neither the lowest nor the highest bin covers the patterns
    // [lo + (digit << s), lo + ((digit + 1) << s)): one subtraction and one unsigned comparison per element and leader,
    // no key.  The two end bins also hold the clamped elements, so a block with a leader there takes the general test
    // on the key itself.
    const bool inner = L.n <= 2 && L.key[0] - 1u < uint32_t(kSelBins - 2) && (L.n < 2 || L.key[1] - 1u < uint32_t(kSelBins - 2));
    const uint32_t span = 1u << key.s;
    const uint32_t base0 = uint32_t(key.lo) + (L.key[0] << key.s);
    const uint32_t base1 = L.n > 1 ? uint32_t(key.lo) + (L.key[1] << key.s) : base0;
    // a vector block's last row may be short; every other row of a piece holds the thread's nc columns
    const int64_t short_row = (b->cols > 1 || (numel % kPieceCols) == 0) ? -1 : numel / kPieceCols;
    const uint32_t* __restrict__ vp = v + (int64_t(pc.row0) + g.ty) * g.cols + pc.col0 + g.tx * 8;
    const int64_t v_step = int64_t(g.step) * g.cols;

    // The walk over the piece's rows, compiled once per combination of what the whole CTA does or does not do
    // (kResid: Eq. 7; kKeys: this pass has a digit to find; kInner: the cheap survivor test applies), so that none of
    // it is decided again for every row.
    auto rows = [&](auto resid_tag, auto keys_tag, auto inner_tag) {
        constexpr bool kResid = decltype(resid_tag)::value, kKeys = decltype(keys_tag)::value, kInner = decltype(inner_tag)::value;
        // one row of the thread: kWide: all eight elements exist
        auto row = [&](auto wide_tag, uint32_t (&u)[8], int n, double rsum) {
            constexpr bool kWide = decltype(wide_tag)::value;
            if (kResid) {
                const double a = rsum * inv_total;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (kWide || j < n) {
                        const double d = fma(-a, cs[j], double(__uint_as_float(u[j])));
                        acc[0] = fma(d, d, acc[0]);
                    }
                }
            }
            if (!kKeys) return;
            uint32_t mask = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                bool p;
                if (kInner) {
                    p = (u[j] - base0 < span) | (u[j] - base1 < span);
                } else {
                    const uint32_t top = sel_key(u[j], key.lo, wmax) >> key.s;
                    p = (top == L.key[0]) | (top == L.key[1]) | (top == L.key[2]) | (top == L.key[3]);
                }
                if ((kWide || j < n) && p) mask |= 1u << j;
            }
            if (mask) {                                       // few threads
                int pos = atomicAdd(&wcnt[warp], __popc(mask));
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (mask & (1u << j)) seg[pos++] = sel_key(u[j], key.lo, wmax);
            }
        };
        // whole batches of full rows first (no per-row decisions), then what is left, row by row
        // (uniform over the CTA) every row of a thread is eight elements, two 16-byte loads, or the thread has no column at all
        const bool plain = g.vec && (g.width & 7) == 0 && short_row < 0;
        const bool rows32 = (g.cols & 7) == 0;                // every row of the thread starts 32-byte aligned: one 256-bit load
        const int64_t batch = int64_t(kRhBatch) * g.step;
        const int64_t r_full = plain ? int64_t(pc.row0) + (int64_t(pc.nrows) / batch) * batch : int64_t(pc.row0);
        int64_t r0 = int64_t(pc.row0);
#pragma unroll 1
        for (; r0 < r_full; r0 += batch) {                    // the same trips for every thread
            if (g.nc == 8) {
                uint32_t u[kRhBatch][8];
                double rs[kRhBatch];
#pragma unroll
                for (int k = 0; k < kRhBatch; ++k) {
                    if (rows32) {
                        ld_stream_u8(vp + k * v_step, u[k]);
                    } else {
                        const uint4 a = ld_stream_u4(vp + k * v_step), c = ld_stream_u4(vp + k * v_step + 4);
                        u[k][0] = a.x; u[k][1] = a.y; u[k][2] = a.z; u[k][3] = a.w; u[k][4] = c.x; u[k][5] = c.y; u[k][6] = c.z; u[k][7] = c.w;
                    }
                    rs[k] = kResid ? __ldg(rowsum + (r0 + g.ty + int64_t(k) * g.step)) : 0.0;
                }
#pragma unroll
                for (int k = 0; k < kRhBatch; ++k) row(std::true_type{}, u[k], 8, rs[k]);
            }
            vp += kRhBatch * v_step;
            if (kKeys) {
                __syncwarp();
                if (wcnt[warp] > kRhDrainAt) drain();         // uniform over the warp: room for the next batch
            }
        }
#pragma unroll 1
        for (; r0 < r_end; r0 += batch) {                     // the same trips for every thread
            uint32_t u[kRhBatch][8];
            int n[kRhBatch];
            double rs[kRhBatch];
#pragma unroll
            for (int k = 0; k < kRhBatch; ++k) {
                const int64_t r = r0 + g.ty + int64_t(k) * g.step;
                n[k] = 0;
                rs[k] = 0.0;
                if (r < r_end) {
                    n[k] = piece_load(v, pc, g, numel, r, u[k]);
                    if (kResid) rs[k] = __ldg(rowsum + r);
                }
            }
#pragma unroll
            for (int k = 0; k < kRhBatch; ++k) {
                if (n[k] == 8) row(std::true_type{}, u[k], 8, rs[k]);
                else if (n[k] > 0) row(std::false_type{}, u[k], n[k], rs[k]);
            }
            if (kKeys) {
                __syncwarp();
                if (wcnt[warp] > kRhDrainAt) drain();
            }
        }
    };
    const std::true_type yes{};
    const std::false_type no{};
    if (resid) {                                              // all uniform over the CTA
        if (d_bits == 0) rows(yes, no, no);
        else if (inner) rows(yes, yes, yes);
        else rows(yes, yes, no);
    } else {
        if (inner) rows(no, yes, yes);
        else rows(no, yes, no);
    }
    __syncwarp();
    drain();
    if (with_resid) cta_reduce_store<kResidSums>(acc, resid_part + blockIdx.x);
    else __syncthreads();
    if (threadIdx.x == 0) surv_cnt[blockIdx.x] = run_over ? kSurvOverflow : uint32_t(run_cnt);
    if (d_bits == 0 || (run_cnt == 0 && run_over == 0)) return;   // uniform over the CTA: nothing was counted
#pragma unroll
    for (int k = 0; k < kRanks; ++k) {
        if (k >= L.n) continue;                               // uniform over the CTA
        uint32_t* out = hist + (size_t(pc.block) * kRanks + L.slot[k]) * kSelBins;
        for (int w = threadIdx.x; w < kRhHistWords; w += kThreads) {
            const uint32_t x = sh[k][w];
            if (x) {
                if (x & 0xffffu) atomicAdd(out + 2 * w, x & 0xffffu);
                if (x >> 16) atomicAdd(out + 2 * w + 1, x >> 16);
            }
        }
    }
}

// Sweep 3: the last bits of the key (at most 7), one CTA per piece: its survivors list or, for a piece that was
// marked, its elements of v.  The histogram (256 bins of 32 bits per leader) is handed over per piece.
constexpr int kLastBins = 1 << kSel3Bits;

__global__ void __launch_bounds__(kThreads)
final_last_kernel(const StatBlock* __restrict__ blocks, const SelPiece* __restrict__ pieces, const RankSel* __restrict__ sel,
                  const SelKey* __restrict__ selkey, uint32_t* __restrict__ hist, const uint32_t* __restrict__ surv,
                  const uint32_t* __restrict__ surv_cnt, int64_t n_pieces BAOC_CHECK_PARAM) {
    __shared__ uint32_t sh[kRanks][kLastBins];
    __shared__ int counted;
    const int lane = threadIdx.x & 31;
    const SelPiece pc = pieces[blockIdx.x];
#ifdef BAOC_CHECKED
    if (int64_t(blockIdx.x) >= ck.n_tiles || n_pieces != ck.n_tiles) { check_fail(kChkTileIndex, kKerFinalLast, blockIdx.x, ck.n_tiles, n_pieces, 0); return; }
    if (pc.block >= unsigned(ck.n_blocks)) { check_fail(kChkBlockIndex, kKerFinalLast, pc.block, ck.n_blocks, blockIdx.x, 0); return; }
#endif
    const StatBlock* b = blocks + pc.block;
    const SelKey key = selkey[pc.block];
    int d_shift, d_bits;
    sel_digit(key.s, 2, d_shift, d_bits);
    if (key.s < 0 || d_bits == 0) return;                     // uniform over the CTA: not in this round, or nothing left to find
    const uint32_t cnt = surv_cnt[blockIdx.x];
    if (cnt == 0u) return;
#ifdef BAOC_CHECKED
    if (!check_range(ck, kKerFinalLast, surv_cnt + blockIdx.x, 4, 0) ||
        !check_range(ck, kKerFinalLast, surv + pc.surv_off, 4ll * pc.slots, 1) ||
        !check_range(ck, kKerFinalLast, hist + size_t(pc.block) * kRanks * kSelBins, 4ll * kRanks * kSelBins, 2) ||
        (cnt != kSurvOverflow && cnt > pc.slots && !check_fail(kChkRange, kKerFinalLast, 3, cnt, pc.slots, blockIdx.x)))
        return;
#endif
    const Leaders L = leaders_of(sel + size_t(pc.block) * kRanks, d_bits);
    for (int i = threadIdx.x; i < kRanks * kLastBins; i += kThreads) (&sh[0][0])[i] = 0u;
    if (threadIdx.x == 0) counted = 0;
    __syncthreads();

    // one lane per distinct key among the lanes `act` adds for all of them
    auto count_same = [&](unsigned act, uint32_t x) {
        const unsigned same = __match_any_sync(act, x);
        if (lane == __ffs(int(same)) - 1) {
            const uint32_t upper = x >> d_bits, d = x & ((1u << d_bits) - 1u);
#pragma unroll
            for (int k = 0; k < kRanks; ++k)
                if (upper == L.key[k]) { atomicAdd(&sh[k][d], uint32_t(__popc(same))); counted = 1; }
        }
    };

    if (cnt != kSurvOverflow) {
        const uint32_t* __restrict__ list = surv + pc.surv_off;
        for (uint32_t i0 = 0; i0 < cnt; i0 += kThreads) {     // uniform over the CTA
            const uint32_t i = i0 + threadIdx.x;
            const bool on = i < cnt;
            const unsigned act = __ballot_sync(0xffffffffu, on);
            if (on) count_same(act, list[i]);
        }
    } else {
        const PieceGeom g = piece_geom(pc, b);
        const uint32_t* __restrict__ v = reinterpret_cast<const uint32_t*>(b->v);
        const int wmax = sel_wmax(key.s);
#ifdef BAOC_CHECKED
        if (!check_range(ck, kKerFinalLast, v, 4 * ((b->numel + kQBlock - 1) / kQBlock * kQBlock), 4)) return;
#endif
        const int64_t r_end = int64_t(pc.row0) + pc.nrows;
        for (int64_t r0 = int64_t(pc.row0); r0 < r_end; r0 += g.step) {   // uniform over the CTA
            const int64_t r = r0 + g.ty;
            uint32_t u[8];
            const int n = r < r_end ? piece_load(v, pc, g, b->numel, r, u) : 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t x = sel_key(u[j], key.lo, wmax), upper = x >> d_bits;
                const bool hit = (j < n) & ((upper == L.key[0]) | (upper == L.key[1]) | (upper == L.key[2]) | (upper == L.key[3]));
                const unsigned act = __ballot_sync(0xffffffffu, hit);
                if (hit) count_same(act, x);
            }
        }
    }
    __syncthreads();
    if (!counted) return;                                     // uniform over the CTA
#pragma unroll
    for (int k = 0; k < kRanks; ++k) {
        if (k >= L.n) continue;                               // uniform over the CTA
        uint32_t* out = hist + (size_t(pc.block) * kRanks + L.slot[k]) * kSelBins;
        for (int w = threadIdx.x; w < kLastBins; w += kThreads) {
            const uint32_t x = sh[k][w];
            if (x) atomicAdd(out + w, x);
        }
    }
}

// One CTA per block: for each of the four ranks find the bin of its leader's
// histogram that holds the rank (a scan over the CTA), extend the prefix by this
// pass's digit, recompute which ranks still share a prefix, and clear the
// histograms for the next pass.
__global__ void __launch_bounds__(kThreads)
select_pick_kernel(RankSel* __restrict__ sel, uint32_t* __restrict__ hist, const SelKey* __restrict__ selkey, int pass) {
    __shared__ unsigned long long warp_tot[kThreads / 32];
    __shared__ int res_d[kRanks];
    __shared__ long long res_rem[kRanks];
    const int blk = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const SelKey key = selkey[blk];
    int shift, bits;
    sel_digit(key.s, pass, shift, bits);
    if (key.s < 0 || bits == 0) return;                       // uniform over the CTA: not in this round, or no digit left (nothing was counted)
    const int bins = pass < 2 ? kSelBins : kLastBins;
    RankSel s[kRanks];
#pragma unroll
    for (int r = 0; r < kRanks; ++r) s[r] = sel[size_t(blk) * kRanks + r];
    if (threadIdx.x < kRanks) { res_d[threadIdx.x] = bins - 1; res_rem[threadIdx.x] = 0; }
    const int per = bins / kThreads;                          // 1 or 16 bins per thread
    for (int r = 0; r < kRanks; ++r) {
        const uint32_t* hh = hist + (size_t(blk) * kRanks + s[r].leader) * kSelBins + threadIdx.x * per;
        unsigned long long local = 0ull;
        for (int i = 0; i < per; ++i) local += hh[i];
        unsigned long long incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        __syncthreads();                                      // the previous rank's readers are done with warp_tot
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        for (int w = 0; w < warp; ++w) incl += warp_tot[w];
        const unsigned long long excl = incl - local, rem = (unsigned long long)(s[r].remaining);
        if (excl <= rem && rem < incl) {                      // exactly one thread
            unsigned long long left = rem - excl;
            int d = 0;
            for (; d < per - 1; ++d) {
                const unsigned long long c = hh[d];
                if (left < c) break;
                left -= c;
            }
            res_d[r] = threadIdx.x * per + d;
            res_rem[r] = (long long)(left);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int r = 0; r < kRanks; ++r) {
            s[r].prefix |= uint32_t(res_d[r]) << shift;
            s[r].remaining = res_rem[r];
        }
        for (int r = 0; r < kRanks; ++r) {
            int leader = r;
            for (int q = 0; q < r; ++q)
                if (s[q].prefix == s[r].prefix) { leader = q; break; }
            s[r].leader = leader;
        }
        for (int r = 0; r < kRanks; ++r) sel[size_t(blk) * kRanks + r] = s[r];
    }
    uint32_t* mine = hist + size_t(blk) * kRanks * kSelBins;
    for (int i = threadIdx.x; i < kRanks * kSelBins; i += kThreads) mine[i] = 0u;
}

// Start of a select: ranks floor(q (n-1)) and the next one for q = 0.1, 0.9; all four share the empty prefix.
__global__ void select_init_kernel(const StatBlock* __restrict__ blocks, RankSel* __restrict__ sel,
                                   const SelKey* __restrict__ selkey, int n_blocks) {
    const int blk = blockIdx.x * blockDim.x + threadIdx.x;
    if (blk >= n_blocks || (selkey != nullptr && selkey[blk].s < 0)) return;
    const int64_t n = blocks[blk].numel;
    const double qs[2] = {0.1, 0.9};
    for (int k = 0; k < 2; ++k) {
        const double pos = qs[k] * double(n - 1);
        const int64_t lo = int64_t(floor(pos));
        const int64_t hi = min64(lo + 1, n - 1);
        sel[size_t(blk) * kRanks + 2 * k] = RankSel{0u, 0, lo};
        sel[size_t(blk) * kRanks + 2 * k + 1] = RankSel{0u, 0, hi};
    }
}

// End of the window: gather what the host needs into fin_out[block]:
//   [0..15] sweep-1 sums, [16..19] the four order statistics (as doubles),
//   [20..27] the running window values, [28] the Eq. 7 numerator, [29] the pilot value,
//   [30] whether an order statistic came out at an end of the key range (a clamped element: to be found again).
__global__ void stats_gather_kernel(const RankSel* __restrict__ sel, const SelKey* __restrict__ selkey,
                                    const double* __restrict__ acc, double* __restrict__ fin_out, int n_blocks) {
    const int blk = blockIdx.x * blockDim.x + threadIdx.x;
    if (blk >= n_blocks) return;
    const SelKey key = selkey[blk];
    if (key.s < 0) return;
    double* o = fin_out + size_t(blk) * kFinOut;
    const uint32_t wmax = uint32_t(sel_wmax(key.s));
    bool clamped = false;
    for (int r = 0; r < kRanks; ++r) {
        const uint32_t w = sel[size_t(blk) * kRanks + r].prefix;
        clamped |= w == 0u || w == wmax;
        o[kFinRanks + r] = double(__int_as_float(int(w) + key.lo));
    }
    o[kFinFlag] = clamped ? 1.0 : 0.0;
    for (int k = 0; k < kBlockAcc; ++k) o[kFinAcc + k] = acc[size_t(blk) * kBlockAcc + k];
}

// First pass of the select on its own (the first sweep does it for the first round): the top 12 bits of the key of
// every element of the blocks that take part.
__global__ void __launch_bounds__(kThreads)
select_first_kernel(const StatBlock* __restrict__ blocks, const Tile* __restrict__ tiles, const SelKey* __restrict__ selkey,
                    uint32_t* __restrict__ hist, int64_t n_tiles, int tiles_per_cta BAOC_CHECK_PARAM) {
    __shared__ uint32_t sh[kSelBins];
    const int64_t first = int64_t(blockIdx.x) * tiles_per_cta, last = min64(first + tiles_per_cta, n_tiles);
#ifdef BAOC_CHECKED
    {
        if (first >= ck.n_tiles || n_tiles != ck.n_tiles) { check_fail(kChkTileIndex, kKerSelectFirst, first, ck.n_tiles, n_tiles, 0); return; }
        for (int64_t ti = first; ti < last; ++ti) {
            const Tile ct = tiles[ti];
            if (ct.block >= unsigned(ck.n_blocks)) { check_fail(kChkBlockIndex, kKerSelectFirst, ct.block, ck.n_blocks, ti, 0); return; }
            const StatBlock* cb = blocks + ct.block;
            const int64_t cbase = int64_t(ct.piece) * kTile;
            const int64_t cpad = (cb->numel + kQBlock - 1) / kQBlock * kQBlock, cn = min64(kTile, cpad - cbase);
            if (!check_tile(ck, kKerSelectFirst, ti, ct.block, cbase, cb->numel) ||
                !check_range(ck, kKerSelectFirst, cb->v + cbase, 4 * cn, 0) ||
                !check_range(ck, kKerSelectFirst, hist + size_t(ct.block) * kRanks * kSelBins, 4ll * kSelBins, 1) ||
                !check_range(ck, kKerSelectFirst, selkey + ct.block, int64_t(sizeof(SelKey)), 2))
                return;
        }
    }
#endif
    for (int i = threadIdx.x; i < kSelBins; i += kThreads) sh[i] = 0u;
    __syncthreads();
#pragma unroll 1
    for (int64_t t_begin = first; t_begin < last;) {
        const Tile t = tiles[t_begin];
        const StatBlock* b = blocks + t.block;
        const int64_t t_end = min64(last, b->tile0 + b->ntiles);
        const SelKey key = selkey[t.block];
        if (key.s >= 0) {                                     // uniform over the CTA
            const uint32_t* __restrict__ v = reinterpret_cast<const uint32_t*>(b->v);
            const int64_t e0 = int64_t(t.piece) * kTile, e1 = min64(b->numel, e0 + (t_end - t_begin) * int64_t(kTile));
            const int wmax = sel_wmax(key.s);
            for (int64_t i = e0 + threadIdx.x; i < e1; i += kThreads) atomicAdd(&sh[sel_key(v[i], key.lo, wmax) >> key.s], 1u);
            __syncthreads();
            uint32_t* out = hist + size_t(t.block) * kRanks * kSelBins;          // all four ranks still share one histogram
            for (int d = threadIdx.x; d < kSelBins; d += kThreads) {
                const uint32_t c = sh[d];
                if (c) { atomicAdd(out + d, c); sh[d] = 0u; }
            }
            __syncthreads();
        }
        t_begin = t_end;
    }
}

// ---- launchers ------------------------------------------------------------------
#define BAOC_LAUNCH_CHECK()                                   \
    do {                                                      \
        cudaError_t e_ = cudaGetLastError();                  \
        if (e_ != cudaSuccess) return int(e_);                \
    } while (0)

BAOC_DEFINE_CHECK_FETCH(finalize_check_fetch)

// Tiles per CTA of a sweep: as many as `most`, fewer when the workload would then not give every SM a few CTAs.
static int run_tiles(int64_t n_tiles, int most, int ctas_per_sm = 6) {
    const int64_t want = n_tiles / (int64_t(148) * ctas_per_sm);
    return int(want < 1 ? 1 : (want > most ? most : want));
}

template <bool kDyn, bool kDebias>
static cudaError_t launch_sums_instance(unsigned grid, const StatBlock* blocks, const Tile* tiles, const float* const* params,
                                        double* fin, const double* fin_out, uint32_t* hist, const SelKey* selkey, int64_t n_tiles,
                                        int per, float eps, float eps_adam, float m_scale, float v_scale, const CheckCtx& ck,
                                        cudaStream_t s) {
    (void)ck;
    cudaError_t e = cudaFuncSetAttribute(final_sums_kernel<kDyn, kDebias>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFsSmemBytes);
    if (e != cudaSuccess) return e;
    final_sums_kernel<kDyn, kDebias><<<grid, kThreads, kFsSmemBytes, s>>>(blocks, tiles, params, fin, fin_out, hist, selkey, n_tiles,
                                                                            per, eps, eps_adam, m_scale, v_scale BAOC_CHECK_ARG(ck));
    return cudaGetLastError();
}

int launch_final_sums(const StatBlock* blocks, const Tile* tiles, const float* const* params, double* fin,
                      double* fin_out, uint32_t* hist, RankSel* sel, SelKey* selkey, int64_t n_tiles, int n_blocks, double eps,
                      float eps_adam, int quantizer8, int debias, float m_scale, float v_scale, const CheckCtx& ck, cudaStream_t s) {
    const int tb = 128, gb = (n_blocks + tb - 1) / tb;
    cudaError_t e = cudaMemsetAsync(hist, 0, size_t(n_blocks) * kRanks * kSelBins * sizeof(uint32_t), s);
    if (e != cudaSuccess) return int(e);
    select_init_kernel<<<gb, tb, 0, s>>>(blocks, sel, nullptr, n_blocks);
    BAOC_LAUNCH_CHECK();
    final_pilot_kernel<<<n_blocks, kThreads, 0, s>>>(blocks, float(eps), debias ? v_scale : 1.0f, fin_out, selkey);
    BAOC_LAUNCH_CHECK();
    const int per = run_tiles(n_tiles, kFinRunTiles, 12);     // long runs (a run's hand-over costs a tenth of eight tiles' work), but six waves of CTAs at least
    const unsigned grid = unsigned((n_tiles + per - 1) / per);
    if (quantizer8)
        e = debias ? launch_sums_instance<true, true>(grid, blocks, tiles, params, fin, fin_out, hist, selkey, n_tiles, per, float(eps), eps_adam, m_scale, v_scale, ck, s)
                   : launch_sums_instance<true, false>(grid, blocks, tiles, params, fin, fin_out, hist, selkey, n_tiles, per, float(eps), eps_adam, 1.f, 1.f, ck, s);
    else
        e = debias ? launch_sums_instance<false, true>(grid, blocks, tiles, params, fin, fin_out, hist, selkey, n_tiles, per, float(eps), eps_adam, m_scale, v_scale, ck, s)
                   : launch_sums_instance<false, false>(grid, blocks, tiles, params, fin, fin_out, hist, selkey, n_tiles, per, float(eps), eps_adam, 1.f, 1.f, ck, s);
    if (e != cudaSuccess) return int(e);
    final_sums_combine_kernel<<<n_blocks, kThreads, 0, s>>>(blocks, fin, fin_out, per);
    BAOC_LAUNCH_CHECK();
    select_pick_kernel<<<n_blocks, kThreads, 0, s>>>(sel, hist, selkey, 0);
    BAOC_LAUNCH_CHECK();
    return 0;
}

// The second and third pass of the select (with the Eq. 7 residual in the second sweep if with_resid), and the gather.
static int select_rest(const SelectArgs& a, int with_resid, const CheckCtx& ck, cudaStream_t s) {
    (void)ck;
    cudaError_t e = cudaFuncSetAttribute(final_resid_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRhSmemBytes);
    if (e != cudaSuccess) return int(e);
    const unsigned grid = unsigned(a.n_pieces);
    final_resid_hist_kernel<<<grid, kThreads, kRhSmemBytes, s>>>(a.blocks, a.pieces, a.sel, a.selkey, a.resid_part, a.hist, a.surv,
                                                                a.surv_cnt, a.n_pieces, with_resid BAOC_CHECK_ARG(ck));
    BAOC_LAUNCH_CHECK();
    if (with_resid) {
        final_resid_combine_kernel<<<a.n_blocks, kThreads, 0, s>>>(a.blocks, a.resid_part, a.fin_out);
        BAOC_LAUNCH_CHECK();
    }
    select_pick_kernel<<<a.n_blocks, kThreads, 0, s>>>(a.sel, a.hist, a.selkey, 1);
    BAOC_LAUNCH_CHECK();
    final_last_kernel<<<grid, kThreads, 0, s>>>(a.blocks, a.pieces, a.sel, a.selkey, a.hist, a.surv, a.surv_cnt, a.n_pieces BAOC_CHECK_ARG(ck));
    BAOC_LAUNCH_CHECK();
    select_pick_kernel<<<a.n_blocks, kThreads, 0, s>>>(a.sel, a.hist, a.selkey, 2);
    BAOC_LAUNCH_CHECK();
    const int tb = 128, gb = (a.n_blocks + tb - 1) / tb;
    stats_gather_kernel<<<gb, tb, 0, s>>>(a.sel, a.selkey, a.acc, a.fin_out, a.n_blocks);
    BAOC_LAUNCH_CHECK();
    return 0;
}

int launch_final_resid_select(const SelectArgs& a, const CheckCtx& ck, cudaStream_t s) { return select_rest(a, 1, ck, s); }

int launch_select_again(const SelectArgs& a, const CheckCtx& ck, cudaStream_t s) {
    const int tb = 128, gb = (a.n_blocks + tb - 1) / tb;
    select_init_kernel<<<gb, tb, 0, s>>>(a.blocks, a.sel, a.selkey, a.n_blocks);
    BAOC_LAUNCH_CHECK();
    const int per = run_tiles(a.n_tiles, kSelRunTiles);
    const unsigned grid = unsigned((a.n_tiles + per - 1) / per);
#ifdef BAOC_CHECKED
    CheckCtx ck_tiles = ck;                                   // this kernel walks tiles, the later sweeps pieces
    ck_tiles.n_tiles = a.n_tiles;
#endif
    select_first_kernel<<<grid, kThreads, 0, s>>>(a.blocks, a.tiles, a.selkey, a.hist, a.n_tiles, per BAOC_CHECK_ARG(ck_tiles));
    BAOC_LAUNCH_CHECK();
    select_pick_kernel<<<a.n_blocks, kThreads, 0, s>>>(a.sel, a.hist, a.selkey, 0);
    BAOC_LAUNCH_CHECK();
    return select_rest(a, 0, ck, s);
}

}  // namespace baoc
