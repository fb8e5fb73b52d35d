// Host side of the library: handle, cost model, normalisation and risk
// (Appendix A, Eq. 9-21), and the exact budgeted allocation (Eq. 1-2).
// Nothing in this file touches the GPU.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <limits>
#include <map>
#include <new>

#include "baoc_internal.h"

namespace baoc {

int fail(const Handle* h, int code, const std::string& msg) {
    if (h) h->err = msg;
    return code;
}

int64_t state_mem_bytes(const baoc_config_t& c, const baoc_block_t& b) {
    const int64_t d = b.numel;
    const int64_t nq = ceil_div(d, kQBlock);
    auto per_tensor = [&]() -> int64_t {
        if (c.bits == 32) return 4 * d;
        if (c.bits == 16) return 2 * d;
        return d + 4 * nq;                 // 1-byte codes + one fp32 absmax per quantisation block
    };
    int64_t total = 0;
    if (c.momentum) total += per_tensor();
    if (c.adaptive) {
        if (!c.factored) total += per_tensor();
        else {
            // row and column statistics in the tuple's precision; as 8-bit codes each vector has its own quantisation blocks
            const int64_t rc = int64_t(b.rows) + int64_t(b.cols);
            if (c.bits == 32) total += 4 * rc;
            else if (c.bits == 16) total += 2 * rc;
            else total += rc + 4 * (ceil_div(b.rows, kQBlock) + ceil_div(b.cols, kQBlock));
        }
    }
    return total;
}

// Bytes the step must move per block: bf16 gradient read, fp32 parameter read
// and write, every state read and written once.  The factored path reads the
// gradient twice (row/column pass, then the update).
double step_traffic_bytes(const baoc_config_t& c, const baoc_block_t& b) {
    double bytes = 2.0 * b.numel + 8.0 * b.numel + 2.0 * double(state_mem_bytes(c, b));
    if (c.factored) bytes += 2.0 * b.numel;
    if (c.factored && (c.af_flags & (kAfClip | kAfRelative))) bytes += 6.0 * b.numel;   // one more sweep over g and theta for the two norms
    return bytes;
}

// About 16 * refine row chunks per matrix (never finer than one group of 64 rows), and more for a tall matrix: a CTA
// walks its chunk one group after the other, so a chunk of more than eight groups (an embedding table of tens of
// thousands of rows cut into 16) would leave a few CTAs running long after the rest of the grid has finished.
RedGeom red_geometry(int32_t rows, int32_t cols, int refine) {
    RedGeom g{};
    g.rowpart = nullptr; g.colpart = nullptr; g.red0 = -1;
    const int64_t groups = ceil_div(rows, kRedRows);
    g.L = int32_t(std::max<int64_t>(1, ceil_div(groups, std::min<int64_t>(16 * int64_t(refine), groups))));
    g.L = std::min<int32_t>(g.L, 8);
    g.chunks = int32_t(ceil_div(rows, int64_t(kRedRows) * g.L));
    g.strips = int32_t(ceil_div(cols, kRedCols));
    return g;
}

// How much finer than 16 row chunks per matrix the reduction has to cut so that all the matrices together give about
// four CTAs per SM: coarse chunks move the fewest partial sums, but a few narrow matrices alone (an embedding table
// of 768 columns is two strips) would leave most of the GPU idle.
static int red_refinement(int64_t ctas_at_16_chunks) {
    constexpr int64_t kWant = 4 * 148;
    if (ctas_at_16_chunks <= 0 || ctas_at_16_chunks >= kWant) return 1;
    return int(std::min<int64_t>(64, ceil_div(kWant, ctas_at_16_chunks)));
}

static size_t take(size_t* cur, size_t bytes) {
    size_t at = *cur;
    *cur = size_t(round_up(int64_t(at + bytes), 256));
    return at;
}

// Pieces of the select's second sweep, block by block: strips of at most kPieceCols columns, cut into runs of rows of at
// most kPieceElems elements (a multiple of 16 rows: the CTA's row step at full width).  Sets piece0 / npieces of the
// blocks and returns the words of the survivors list: one slot per eight elements of a piece.
void build_sel_pieces(const Handle* h, std::vector<SelPiece>* out, std::vector<StatBlock>* blocks, uint64_t* surv_words) {
    out->clear();
    uint64_t off = 0;
    for (int i = 0; i < h->n_blocks; ++i) {
        const baoc_block_t& b = h->stat_shapes[i];
        const int64_t C = b.cols > 1 ? b.cols : kPieceCols;
        const int64_t R = b.cols > 1 ? b.rows : ceil_div(b.numel, kPieceCols);
        (*blocks)[i].piece0 = int64_t(out->size());
        for (int64_t c0 = 0; c0 < C; c0 += kPieceCols) {
            const int64_t width = std::min<int64_t>(kPieceCols, C - c0);
            const int64_t rows_per = std::max<int64_t>(16, kPieceElems / width / 16 * 16);
            for (int64_t r0 = 0; r0 < R; r0 += rows_per) {
                const int64_t nr = std::min(rows_per, R - r0);
                const uint32_t slots = uint32_t(round_up(ceil_div(nr * width, 8), 32));
                out->push_back(SelPiece{uint32_t(i), uint32_t(c0), uint32_t(r0), uint32_t(nr), off, slots, 0u});
                off += slots;
            }
        }
        (*blocks)[i].npieces = int32_t(int64_t(out->size()) - (*blocks)[i].piece0);
    }
    *surv_words = off;
}

// Statistics workspace: tables, moments, previous gradient, partial sums,
// per-block accumulators and the scratch of the finalize pass.  Pointers in
// h_stat_blocks are offsets from a null base until a workspace is bound.
void compute_stat_layout(Handle* h) {
    const int n = h->n_blocks;
    int64_t tiles = 0, red = 0, padded = 0, sum_rows = 0, sum_cols = 0, redpart = 0, n_ridx = 0, n_cidx = 0;
    h->h_stat_blocks.assign(n, StatBlock{});
    if (!h->sampled) h->stat_shapes = h->blocks;
    int64_t coarse = 0;
    for (int i = 0; i < n; ++i) {
        const baoc_block_t& b = h->stat_shapes[i];
        if (b.cols > 1) { const RedGeom g = red_geometry(b.rows, b.cols, 1); coarse += int64_t(g.chunks) * g.strips; }
    }
    const int refine = red_refinement(coarse);
    for (int i = 0; i < n; ++i) {
        const baoc_block_t& b = h->stat_shapes[i];
        StatBlock& s = h->h_stat_blocks[i];
        s.full_cols = h->blocks[i].cols;
        if (h->sampled) {
            s.ridx = reinterpret_cast<const int64_t*>(size_t(n_ridx) * 8);
            s.cidx = reinterpret_cast<const int32_t*>(size_t(n_cidx) * 4);
            s.gsample = reinterpret_cast<uint16_t*>(size_t(padded) * 2);
            s.psample = reinterpret_cast<float*>(size_t(padded) * 4);
            n_ridx += int64_t(h->s_rows[i].size()); n_cidx += int64_t(h->s_cols[i].size());
        }
        s.numel = b.numel; s.rows = b.rows; s.cols = b.cols;
        s.tile0 = tiles; s.ntiles = int32_t(ceil_div(b.numel, kTile));
        tiles += s.ntiles;
        s.m = reinterpret_cast<float*>(size_t(padded) * 4);
        s.v = reinterpret_cast<float*>(size_t(padded) * 4);
        s.gprev = reinterpret_cast<uint16_t*>(size_t(padded) * 2);
        padded += round_up(b.numel, kQBlock);
        s.red = red_geometry(b.rows, b.cols, refine);
        if (b.cols > 1) {
            s.red.red0 = int32_t(red);
            red += int64_t(s.red.chunks) * s.red.strips;
            s.rowsum = reinterpret_cast<double*>(size_t(sum_rows) * 8);
            s.colsum = reinterpret_cast<double*>(size_t(sum_cols) * 8);
            sum_rows += b.rows + 1;                                // the row sums, then their total
            sum_cols += round_up(b.cols, 2);                       // column sums start 16-byte aligned (read in pairs)
            s.red.rowpart = reinterpret_cast<double*>(size_t(redpart) * 8);
            redpart += int64_t(s.red.strips) * b.rows;
            s.red.colpart = reinterpret_cast<double*>(size_t(redpart) * 8);
            redpart += int64_t(s.red.chunks) * b.cols;
        }
    }
    h->n_stat_tiles = tiles; h->n_red_tiles = red;
    std::vector<SelPiece> pieces;
    uint64_t surv_words = 0;
    build_sel_pieces(h, &pieces, &h->h_stat_blocks, &surv_words);
    h->n_sel_pieces = int64_t(pieces.size());
    auto& L = h->sl;
    size_t cur = 0;
    L.blocks = take(&cur, sizeof(StatBlock) * n);
    L.tiles = take(&cur, sizeof(Tile) * size_t(tiles));
    L.red_tiles = take(&cur, sizeof(RedTile) * size_t(std::max<int64_t>(red, 1)));
    L.matrix_ids = take(&cur, 4 * size_t(n));
    L.grads = take(&cur, 8 * size_t(n));
    L.params = take(&cur, 8 * size_t(n));
    L.m = take(&cur, 4 * size_t(padded));
    L.v = take(&cur, 4 * size_t(padded));
    L.gprev = take(&cur, 2 * size_t(padded));
    L.partials = take(&cur, 8 * size_t(kStatPartials) * size_t(tiles));
    L.acc = take(&cur, 8 * size_t(kBlockAcc) * n);
    L.fin = take(&cur, 8 * size_t(kFinalSums) * size_t(tiles));
    L.fin_out = take(&cur, 8 * size_t(kFinOut) * n);
    L.hist = take(&cur, 4 * size_t(kSelBins) * kRanks * n);
    L.sel = take(&cur, sizeof(RankSel) * size_t(kRanks) * n);
    L.selkey = take(&cur, sizeof(SelKey) * size_t(n));
    L.pieces = take(&cur, sizeof(SelPiece) * pieces.size());
    L.resid_part = take(&cur, 8 * pieces.size());
    L.surv = take(&cur, 4 * size_t(surv_words));
    L.surv_cnt = take(&cur, 4 * pieces.size());
    L.rowsum = take(&cur, 8 * size_t(std::max<int64_t>(sum_rows, 1)));
    L.colsum = take(&cur, 8 * size_t(std::max<int64_t>(sum_cols, 1)));
    L.redpart = take(&cur, 8 * size_t(std::max<int64_t>(redpart, 1)));
    L.ridx = L.cidx = L.gsample = L.psample = L.sgrads = L.sparams = cur;
    if (h->sampled) {
        L.ridx = take(&cur, 8 * size_t(std::max<int64_t>(n_ridx, 1)));
        L.cidx = take(&cur, 4 * size_t(std::max<int64_t>(n_cidx, 1)));
        L.gsample = take(&cur, 2 * size_t(padded));
        L.psample = take(&cur, 4 * size_t(padded));
        L.sgrads = take(&cur, 8 * size_t(n));
        L.sparams = take(&cur, 8 * size_t(n));
    }
    L.total = cur;
}

void compute_copy_groups(const Handle* h, std::vector<int>* b0s, std::vector<int>* b1s) {
    b0s->clear(); b1s->clear();
    const int64_t per_group = ceil_div(h->numel, Handle::kCopyGroups);
    int b0 = 0, g = 0;
    while (b0 < h->n_blocks) {
        int b1 = b0;
        int64_t acc = 0;
        while (b1 < h->n_blocks && (acc < per_group || g == Handle::kCopyGroups - 1)) acc += h->blocks[b1++].numel;
        b0s->push_back(b0); b1s->push_back(b1);
        b0 = b1;
        ++g;
    }
}

// Optimizer-state buffer of one assignment: tables, non-finite flags, the
// scratch of the factored path and the states themselves.
int compute_step_layout(const Handle* h, const int32_t* assign, Handle::StepLayout* out, std::vector<StepBlock>* blocks,
                        std::vector<Tile>* tiles, std::vector<RedTile>* red, int64_t* state_mem, int64_t* step_bytes) {
    const int n = h->n_blocks;
    std::vector<StepBlock> sb(n);
    std::vector<Tile> tl;
    std::vector<RedTile> rt;
    size_t states = 0, redpart = 0;
    int64_t mem = 0;
    double traffic = 0;
    int64_t coarse = 0;
    for (int i = 0; i < n; ++i)
        if (assign[i] >= 0 && assign[i] < h->n_cfg && is_factored_path(path_of(h->cfgs[assign[i]]))) {
            const RedGeom g = red_geometry(h->blocks[i].rows, h->blocks[i].cols, 1);
            coarse += int64_t(g.chunks) * g.strips;
        }
    const int refine = red_refinement(coarse);
    for (int i = 0; i < n; ++i) {
        const int c = assign[i];
        if (c < 0 || c >= h->n_cfg) return fail(h, BAOC_E_INVALID, "assignment names a configuration that does not exist");
        const baoc_block_t& b = h->blocks[i];
        const Path p = path_of(h->cfgs[c]);
        if (p == kPathNone) return fail(h, BAOC_E_INVALID, "assignment names a configuration tuple the library cannot instantiate");
        if (is_factored_path(p) && b.cols <= 1) return fail(h, BAOC_E_INVALID, "the factored configuration needs a matrix block");
        StepBlock& s = sb[i];
        s = StepBlock{};
        s.numel = b.numel; s.rows = b.rows; s.cols = b.cols; s.cfg = c; s.path = p;
        s.red = red_geometry(b.rows, b.cols, refine);
        const size_t dpad = size_t(round_up(b.numel, kQBlock));
        const size_t nq = size_t(ceil_div(b.numel, kQBlock));
        auto place = [&](size_t bytes) { return reinterpret_cast<void*>(take(&states, bytes)); };
        switch (p) {
            case kPathA32: s.s0 = place(4 * dpad); s.s1 = place(4 * dpad); break;
            case kPathA8: case kPathA8N:
                s.s0 = place(dpad); s.s1 = place(dpad);
                s.a0 = static_cast<float*>(place(4 * nq)); s.a1 = static_cast<float*>(place(4 * nq));
                break;
            case kPathR: case kPathS: s.s0 = place(4 * dpad); break;
            case kPathA16: s.s0 = place(2 * dpad); s.s1 = place(2 * dpad); break;
            case kPathR16: case kPathS16: s.s0 = place(2 * dpad); break;
            case kPathR8: s.s1 = place(dpad); s.a1 = static_cast<float*>(place(4 * nq)); break;
            case kPathS8: s.s0 = place(dpad); s.a0 = static_cast<float*>(place(4 * nq)); break;
            case kPathG: break;
            case kPathF: case kPathFA: {
                s.fbits = h->cfgs[c].bits;
                s.af_flags = h->cfgs[c].af_flags;
                if (p == kPathFA) {
                    s.norm_part = reinterpret_cast<double*>(redpart);
                    redpart += 8 * 2 * size_t(ceil_div(b.numel, kTileF));
                }
                if (s.fbits == 32) { s.s0 = place(4 * size_t(b.rows)); s.s1 = place(4 * size_t(b.cols)); }
                else {
                    // the fp32 working copies live in the scratch region (offsets from its base), the stored form in the states
                    s.s0 = reinterpret_cast<void*>(take(&redpart, 4 * size_t(b.rows)));
                    s.s1 = reinterpret_cast<void*>(take(&redpart, 4 * size_t(b.cols)));
                    const size_t eb = s.fbits == 16 ? 2 : 1;
                    s.f0 = place(eb * size_t(b.rows)); s.f1 = place(eb * size_t(b.cols));
                    if (s.fbits == 8) {
                        s.fa0 = static_cast<float*>(place(4 * size_t(ceil_div(b.rows, kQBlock))));
                        s.fa1 = static_cast<float*>(place(4 * size_t(ceil_div(b.cols, kQBlock))));
                    }
                }
                s.a0 = static_cast<float*>(place(16));
                s.red.red0 = int32_t(rt.size());
                for (int ch = 0; ch < s.red.chunks; ++ch)
                    for (int st = 0; st < s.red.strips; ++st) rt.push_back(RedTile{uint32_t(i), uint32_t(ch), uint32_t(st), 0});
                s.red.rowpart = reinterpret_cast<double*>(redpart);
                redpart += 8 * size_t(s.red.strips) * b.rows;
                s.red.colpart = reinterpret_cast<double*>(redpart);
                redpart += 8 * size_t(s.red.chunks) * b.cols;
                s.mean_part = reinterpret_cast<double*>(redpart);
                redpart += 8 * size_t(kCombineSlabs + 1);
                break;
            }
            default: break;
        }
        mem += state_mem_bytes(h->cfgs[c], b);
        traffic += step_traffic_bytes(h->cfgs[c], b);
    }
    for (int p : kPathOrder)
        for (int i = 0; i < n; ++i)
            if (sb[i].path == p) {
                const int64_t nt = ceil_div(sb[i].numel, step_tile_elems(p));
                for (int64_t k = 0; k < nt; ++k) tl.push_back(Tile{uint32_t(i), uint32_t(k)});
            }
    size_t cur = 0;
    out->blocks = take(&cur, sizeof(StepBlock) * n);
    out->tiles = take(&cur, sizeof(Tile) * tl.size());
    out->tiles_by_group = take(&cur, sizeof(Tile) * tl.size());
    out->red_tiles = take(&cur, sizeof(RedTile) * std::max<size_t>(rt.size(), 1));
    out->f_ids = take(&cur, 8 * size_t(n));               // the factored blocks, then those with Adafactor's options
    out->grads = take(&cur, 8 * size_t(n));
    out->params = take(&cur, 8 * size_t(n));
    out->flags = take(&cur, 4 * size_t(n));
    out->redpart = take(&cur, std::max<size_t>(redpart, 8));
    out->states = take(&cur, std::max<size_t>(states, 8));
    out->total = cur;
    if (blocks) *blocks = sb;
    if (tiles) *tiles = tl;
    if (red) *red = rt;
    if (state_mem) *state_mem = mem;
    if (step_bytes) *step_bytes = int64_t(traffic);
    return BAOC_OK;
}

// ---- Eq. 1 ----
static double agg(const baoc_config_t& c) {
    return double(1 - c.adaptive) + double(1 - c.momentum) + double(1 - c.decoupled_wd) + double(c.factored) +
           32.0 / double(c.bits) - 1.0;
}

static double clip(double x, double lo, double hi) { return std::min(std::max(x, lo), hi); }

// ---- Eq. 10-20 ----
static void normalise(const baoc_opts_t& o, baoc_block_stats_t* s) {
    s->s_A = clip((s->A - o.a_lo) / (o.a_hi - o.a_lo), 0.0, 1.0);
    s->s_rho = clip((s->rho_bar - o.rho_lo) / (o.rho_hi - o.rho_lo), 0.0, 1.0);
    s->s_snr = clip((std::log(1.0 + s->snr) - o.snr_lo) / (o.snr_hi - o.snr_lo), 0.0, 1.0);
    s->s_M = o.use_snr ? s->s_rho * s->s_snr : s->s_rho;
    s->C_tilde = std::log(1.0 + s->C);
    s->s_F = clip(s->F, 0.0, 1.0);
    s->lQ32 = -std::log(clip(s->Q32, o.eps, 1.0) + o.eps);
    s->lQ16 = -std::log(clip(s->Q16, o.eps, 1.0) + o.eps);
    s->lQ8 = -std::log(clip(s->Q8, o.eps, 1.0) + o.eps);
}

// ---- Eq. 9 / 21 ----
static double risk_of(const baoc_opts_t& o, const baoc_block_stats_t& s, const baoc_config_t& c) {
    const double lq = c.bits == 32 ? s.lQ32 : (c.bits == 16 ? s.lQ16 : s.lQ8);
    return o.w[0] * s.s_A * double(1 - c.adaptive) + o.w[1] * s.s_M * double(1 - c.momentum) +
           o.w[2] * s.C_tilde * double(1 - c.decoupled_wd) + o.w[3] * s.s_F * double(c.factored) + o.w[4] * lq;
}

// ============================================================================
// Exact solver of Eq. 2: a multiple-choice knapsack with two capacity rows.
// Dynamic programming over the blocks in their natural order.  A state is a
// partial assignment summarised by (memory used, time used, cost); states are
// pruned by (i) capacity, (ii) a Lagrangian lower bound of both capacity rows
// with fixed integer multipliers, evaluated exactly in 128-bit arithmetic,
// against the best complete assignment known, and (iii) dominance.  States
// carry their rank in the lexicographic order of partial assignments, and a
// state only displaces another if it is cheaper, or equally cheap and
// lexicographically smaller, with no more of either resource: this keeps the
// lexicographically smallest optimal assignment alive to the end.
// ============================================================================
namespace {

using i128 = __int128;
constexpr int kLamShift = 40;       // multipliers are integers / 2^40
constexpr i128 kOne = i128(1) << kLamShift;

struct Item {
    int cfg;
    int64_t phi, mem, rt;
    i128 red;                       // phi*2^S + l1*mem + l2*rt
};

struct State {
    int64_t um, ur, cost;
    int64_t key;                    // lexicographic rank: parent rank * 64 + item index
    int32_t parent;
    int32_t item;
};

struct Solver {
    int n = 0;
    std::vector<std::vector<Item>> items;     // per block, allowed and undominated, ascending cfg
    int64_t B = 0, R = 0;
    int64_t l1 = 0, l2 = 0;                    // scaled multipliers
    int64_t state_limit = 0;
    bool limit_hit = false;
    bool use_time = true;

    std::vector<i128> suf_red;
    std::vector<int64_t> suf_mem, suf_rt;      // suffix sums of per-block minima
    std::vector<int64_t> lag_mem, lag_rt, lag_phi;   // suffix sums over the Lagrangian minimisers
    std::vector<int> lag_item;

    bool have_ub = false;
    int64_t ub = 0;                            // value of the best complete assignment known
    std::vector<int> ub_assign;                // its items (by index into items[i])

    double lagr(double a, double b, double* gm, double* gr) const {
        double tot = -a * double(B) - b * double(R), sm = 0, sr = 0;
        for (int i = 0; i < n; ++i) {
            double bv = std::numeric_limits<double>::infinity();
            const Item* bi = nullptr;
            for (const Item& it : items[i]) {
                double v = double(it.phi) + a * double(it.mem) + b * double(it.rt);
                if (v < bv) { bv = v; bi = &it; }
            }
            tot += bv; sm += double(bi->mem); sr += double(bi->rt);
        }
        if (gm) *gm = sm - double(B);
        if (gr) *gr = sr - double(R);
        return tot;
    }

    // Maximise the concave dual by alternating one-dimensional bisections on
    // the sign of the subgradient; the upper end of the last bracket is kept so
    // that the minimisers respect the row.
    void fit_multipliers() {
        double a = 0, b = 0;
        auto line = [&](bool first) {
            double gm, gr;
            double& x = first ? a : b;
            x = 0;
            lagr(a, b, &gm, &gr);
            if ((first ? gm : gr) <= 0) return;            // row slack at zero price
            double lo = 0, hi = 1;
            for (int k = 0; k < 80; ++k) {
                x = hi; lagr(a, b, &gm, &gr);
                if ((first ? gm : gr) <= 0) break;
                lo = hi; hi *= 4;
            }
            for (int k = 0; k < 70; ++k) {
                x = 0.5 * (lo + hi); lagr(a, b, &gm, &gr);
                if ((first ? gm : gr) > 0) lo = x; else hi = x;
            }
            x = hi;
        };
        for (int round = 0; round < 4; ++round) { line(true); if (use_time) line(false); }
        const double sc = std::ldexp(1.0, kLamShift);
        auto q = [&](double x) { return x <= 0 ? int64_t(0) : int64_t(std::min(std::ceil(x * sc), 9.0e18)); };
        l1 = q(a); l2 = use_time ? q(b) : 0;
    }

    void prepare() {
        suf_red.assign(n + 1, 0); suf_mem.assign(n + 1, 0); suf_rt.assign(n + 1, 0);
        lag_mem.assign(n + 1, 0); lag_rt.assign(n + 1, 0); lag_phi.assign(n + 1, 0); lag_item.assign(n, 0);
        for (int k = n - 1; k >= 0; --k) {
            const auto& v = items[k];
            i128 mr = v[0].red; int64_t mm = v[0].mem, mt = v[0].rt; int arg = 0;
            for (size_t j = 0; j < v.size(); ++j) {
                if (v[j].red < mr) { mr = v[j].red; arg = int(j); }
                mm = std::min(mm, v[j].mem); mt = std::min(mt, v[j].rt);
            }
            suf_red[k] = suf_red[k + 1] + mr; suf_mem[k] = suf_mem[k + 1] + mm; suf_rt[k] = suf_rt[k + 1] + mt;
            lag_item[k] = arg;
            lag_mem[k] = lag_mem[k + 1] + v[arg].mem; lag_rt[k] = lag_rt[k + 1] + v[arg].rt; lag_phi[k] = lag_phi[k + 1] + v[arg].phi;
        }
    }

    // lower bound (scaled by 2^S) on the cost of any completion of a state at level k
    i128 bound(int k, const State& s) const {
        return i128(s.cost) * kOne + i128(l1) * (s.um - B) + i128(l2) * (s.ur - R) + suf_red[k];
    }

    // returns false when infeasible; on success `out` holds the chosen item index per block
    bool solve(std::vector<int>* out, int64_t* value) {
        prepare();
        std::vector<std::vector<std::pair<int32_t, int32_t>>> trace(n);   // per level: (parent, item) of each survivor
        std::vector<State> cur(1, State{0, 0, 0, 0, -1, -1}), nxt;
        // completion of the root by the Lagrangian minimisers
        auto try_complete = [&](int k, const State& s, int32_t idx) {
            if (s.um + lag_mem[k] <= B && s.ur + lag_rt[k] <= R) {
                const int64_t v = s.cost + lag_phi[k];
                if (!have_ub || v < ub) { have_ub = true; ub = v; pending_level = k; pending_state = idx; }
            }
        };
        pending_level = -1; pending_state = -1;
        try_complete(0, cur[0], 0);
        std::vector<int> pending_assign;
        auto materialise = [&](int level, int32_t idx) {
            // rebuild the prefix of state idx at `level` and append the Lagrangian minimisers
            std::vector<int> a(n, 0);
            for (int k = level; k < n; ++k) a[k] = lag_item[k];
            int32_t p = idx;
            for (int k = level - 1; k >= 0; --k) { a[k] = trace[k][p].second; p = trace[k][p].first; }
            ub_assign = a;
        };
        if (pending_level == 0) { materialise(0, 0); pending_level = -1; }

        for (int k = 0; k < n; ++k) {
            nxt.clear();
            const auto& v = items[k];
            for (size_t si = 0; si < cur.size(); ++si) {
                const State& s = cur[si];
                for (size_t j = 0; j < v.size(); ++j) {
                    State t{s.um + v[j].mem, use_time ? s.ur + v[j].rt : 0, s.cost + v[j].phi, int64_t(si) * 64 + int64_t(j),
                            int32_t(si), int32_t(j)};
                    if (t.um + suf_mem[k + 1] > B || (use_time && t.ur + suf_rt[k + 1] > R)) continue;
                    if (have_ub && bound(k + 1, t) > i128(ub) * kOne) continue;
                    nxt.push_back(t);
                }
            }
            if (nxt.empty()) break;
            // dominance: sweep by memory, staircase over time of the best (cost, key)
            std::sort(nxt.begin(), nxt.end(), [](const State& a, const State& b) {
                if (a.um != b.um) return a.um < b.um;
                if (a.ur != b.ur) return a.ur < b.ur;
                if (a.cost != b.cost) return a.cost < b.cost;
                return a.key < b.key;
            });
            std::vector<State> keep;
            keep.reserve(nxt.size());
            if (!use_time) {
                bool any = false; int64_t bc = 0, bk = 0;
                for (const State& t : nxt) {
                    if (any && (bc < t.cost || (bc == t.cost && bk < t.key))) continue;
                    keep.push_back(t); any = true; bc = t.cost; bk = t.key;
                }
            } else {
                std::map<int64_t, std::pair<int64_t, int64_t>> front;      // ur -> best (cost, key) at <= ur
                for (const State& t : nxt) {
                    const std::pair<int64_t, int64_t> val(t.cost, t.key);
                    auto it = front.upper_bound(t.ur);
                    if (it != front.begin()) {
                        auto pv = std::prev(it);
                        if (pv->second < val) continue;                     // dominated
                    }
                    keep.push_back(t);
                    auto ins = front.insert_or_assign(t.ur, val).first;
                    auto nx = std::next(ins);
                    while (nx != front.end() && !(nx->second < val)) nx = front.erase(nx);
                }
            }
            if (int64_t(keep.size()) > state_limit) {
                // keep the most promising states; the answer is then feasible but not proven optimal
                limit_hit = true;
                std::nth_element(keep.begin(), keep.begin() + state_limit, keep.end(), [&](const State& a, const State& b) {
                    return bound(k + 1, a) < bound(k + 1, b);
                });
                keep.resize(size_t(state_limit));
            }
            std::sort(keep.begin(), keep.end(), [](const State& a, const State& b) { return a.key < b.key; });
            trace[k].resize(keep.size());
            for (size_t i = 0; i < keep.size(); ++i) trace[k][i] = {keep[i].parent, keep[i].item};
            cur.swap(keep);
            if (k + 1 < n) {
                pending_level = -1;
                for (size_t i = 0; i < cur.size(); ++i) try_complete(k + 1, cur[i], int32_t(i));
                if (pending_level >= 0) materialise(pending_level, pending_state);
            }
        }
        // complete states of the last level
        bool found = false; int64_t bv = 0; int32_t bi = -1;
        if (!nxt.empty() || n == 0)
            for (size_t i = 0; i < cur.size(); ++i)
                if (!found || cur[i].cost < bv) { found = true; bv = cur[i].cost; bi = int32_t(i); }   // cur is in lexicographic order
        if (found && (!have_ub || bv <= ub)) {
            std::vector<int> a(n, 0);
            int32_t p = bi;
            for (int k = n - 1; k >= 0; --k) { a[k] = trace[k][p].second; p = trace[k][p].first; }
            *out = a; *value = bv;
            return true;
        }
        if (have_ub) { *out = ub_assign; *value = ub; return true; }
        return false;
    }

    int pending_level = -1;
    int32_t pending_state = -1;
};

}  // namespace
}  // namespace baoc

using namespace baoc;

extern "C" {

void baoc_default_opts(baoc_opts_t* o) {
    if (!o) return;
    std::memset(o, 0, sizeof(*o));
    o->beta_m = 0.9; o->beta_v = 0.999; o->beta_rho = 0.9; o->eps = 1e-12;
    o->a_lo = std::log(2.0); o->a_hi = std::log(10.0);
    o->rho_lo = 0.2; o->rho_hi = 0.6; o->snr_lo = 0.0; o->snr_hi = 2.0;
    for (double& w : o->w) w = 1.0;
    o->gamma = 0.1; o->eps_adam = 1e-8; o->use_snr = 1; o->qblock = kQBlock; o->node_limit = 0;
}

int baoc_create(baoc_t** out, int n_blocks, const baoc_block_t* blocks, int n_cfg, const baoc_config_t* cfgs,
                const baoc_opts_t* opts) {
    if (!out) return BAOC_E_INVALID;
    *out = nullptr;
    if (!blocks || !cfgs || n_blocks <= 0 || n_cfg <= 0 || n_cfg > kMaxCfg) return BAOC_E_INVALID;
    baoc_opts_t o;
    if (opts) o = *opts; else baoc_default_opts(&o);
    if (o.qblock != kQBlock || o.quantizer8 < 0 || o.quantizer8 > 1 || o.debias < 0 || o.debias > 1) return BAOC_E_INVALID;
    if (!(o.beta_m >= 0 && o.beta_m < 1 && o.beta_v >= 0 && o.beta_v < 1 && o.beta_rho >= 0 && o.beta_rho < 1)) return BAOC_E_INVALID;
    if (!(o.a_hi > o.a_lo && o.rho_hi > o.rho_lo && o.snr_hi > o.snr_lo && o.eps >= 0)) return BAOC_E_INVALID;
    int64_t total = 0;
    for (int i = 0; i < n_blocks; ++i) {
        const baoc_block_t& b = blocks[i];
        if (b.numel <= 0 || b.rows <= 0 || b.cols <= 0 || int64_t(b.rows) * int64_t(b.cols) != b.numel) return BAOC_E_INVALID;
        if (ceil_div(b.numel, kTile) > int64_t(0x7fffffff)) return BAOC_E_INVALID;
        total += b.numel;
    }
    for (int c = 0; c < n_cfg; ++c) {
        const baoc_config_t& k = cfgs[c];
        if (k.adaptive > 1 || k.momentum > 1 || k.decoupled_wd > 1 || k.factored > 1) return BAOC_E_INVALID;
        if (k.quantizer > 1 || k.af_flags > 15 || k.reserved != 0) return BAOC_E_INVALID;
        if (k.bits != 8 && k.bits != 16 && k.bits != 32) return BAOC_E_INVALID;
        if (!(k.beta1 >= 0 && k.beta1 < 1 && k.beta2 >= 0 && k.beta2 < 1 && k.eps >= 0)) return BAOC_E_INVALID;
        if (!std::isfinite(k.lr) || !std::isfinite(k.weight_decay)) return BAOC_E_INVALID;
    }
    baoc_handle* h = new (std::nothrow) baoc_handle();
    if (!h) return BAOC_E_INVALID;
    h->n_blocks = n_blocks; h->n_cfg = n_cfg;
    h->blocks.assign(blocks, blocks + n_blocks);
    h->cfgs.assign(cfgs, cfgs + n_cfg);
    h->opts = o;
    h->numel = total;
    compute_stat_layout(h);
    *out = h;
    return BAOC_OK;
}

void baoc_destroy(baoc_t* h) { delete h; }

const char* baoc_last_error(const baoc_t* h) { return h ? h->err.c_str() : "null handle"; }

int baoc_set_sampling(baoc_t* h, const baoc_sample_t* samples) {
    if (!h) return BAOC_E_INVALID;
    if (h->ws_bound && h->stats_steps > 0) return fail(h, BAOC_E_STATE, "baoc_set_sampling: the window has started; set the sample before the first observation");
    if (!samples) {                                        // back to the dense sample
        h->sampled = false; h->s_rows.clear(); h->s_cols.clear();
        compute_stat_layout(h);
        h->ws_bound = false;
        return BAOC_OK;
    }
    const int n = h->n_blocks;
    std::vector<std::vector<int64_t>> rows(n);
    std::vector<std::vector<int32_t>> cols(n);
    std::vector<baoc_block_t> shapes(n);
    for (int i = 0; i < n; ++i) {
        const baoc_block_t& b = h->blocks[i];
        const baoc_sample_t& sm = samples[i];
        const bool vec = b.cols <= 1;
        if (!sm.rows || sm.n_rows < 1 || sm.n_rows > b.rows) return fail(h, BAOC_E_INVALID, "baoc_set_sampling: bad row sample");
        if (vec ? (sm.n_cols != 1) : (!sm.cols || sm.n_cols < 1 || sm.n_cols > b.cols)) return fail(h, BAOC_E_INVALID, "baoc_set_sampling: bad column sample");
        rows[i].assign(sm.rows, sm.rows + sm.n_rows);
        if (vec) cols[i].assign(1, 0); else cols[i].assign(sm.cols, sm.cols + sm.n_cols);
        for (size_t k = 0; k < rows[i].size(); ++k)
            if (rows[i][k] < 0 || rows[i][k] >= b.rows || (k && rows[i][k] <= rows[i][k - 1]))
                return fail(h, BAOC_E_INVALID, "baoc_set_sampling: row indices must be in range and strictly increasing");
        for (size_t k = 0; k < cols[i].size(); ++k)
            if (cols[i][k] < 0 || cols[i][k] >= b.cols || (k && cols[i][k] <= cols[i][k - 1]))
                return fail(h, BAOC_E_INVALID, "baoc_set_sampling: column indices must be in range and strictly increasing");
        shapes[i].rows = int32_t(rows[i].size()); shapes[i].cols = int32_t(cols[i].size());
        shapes[i].numel = int64_t(shapes[i].rows) * shapes[i].cols;
    }
    h->sampled = true; h->s_rows.swap(rows); h->s_cols.swap(cols); h->stat_shapes.swap(shapes);
    compute_stat_layout(h);
    h->ws_bound = false;                                   // the workspace has a new size and layout: bind again
    return BAOC_OK;
}

int baoc_query(const baoc_t* h, baoc_info_t* info) {
    if (!h || !info) return BAOC_E_INVALID;
    info->n_blocks = h->n_blocks; info->n_cfg = h->n_cfg; info->numel = h->numel;
    info->n_tiles = h->n_stat_tiles; info->stats_steps = h->stats_steps;
    info->state_bytes = h->configured ? h->state_mem : 0;
    info->kernel_launches = h->launches;
    info->select_retries = h->select_retries;
    {   // g_t, g_{t-1}, m, v read; m, v, g_{t-1} written, over what the statistics see (+ the gather of a sample)
        int64_t seen = 0;
        for (const baoc_block_t& b : (h->sampled ? h->stat_shapes : h->blocks)) seen += b.numel;
        info->stats_bytes_per_call = (h->sampled ? 26 : 22) * seen;
    }
    info->step_bytes_per_call = h->configured ? h->step_bytes : 0;
    return BAOC_OK;
}

int baoc_cost_model(const baoc_t* h, int64_t* mem_bytes, double* time_ratio) {
    if (!h) return BAOC_E_INVALID;
    baoc_config_t adam{}; adam.adaptive = 1; adam.momentum = 1; adam.decoupled_wd = 1; adam.bits = 32;
    for (int i = 0; i < h->n_blocks; ++i)
        for (int c = 0; c < h->n_cfg; ++c) {
            if (mem_bytes) mem_bytes[size_t(i) * h->n_cfg + c] = state_mem_bytes(h->cfgs[c], h->blocks[i]);
            if (time_ratio)
                time_ratio[size_t(i) * h->n_cfg + c] =
                    step_traffic_bytes(h->cfgs[c], h->blocks[i]) / step_traffic_bytes(adam, h->blocks[i]);
        }
    return BAOC_OK;
}

int baoc_risk_from_raw(const baoc_t* h, baoc_block_stats_t* stats, double* risk_out) {
    if (!h || !stats || !risk_out) return h ? fail(h, BAOC_E_INVALID, "baoc_risk_from_raw: null argument") : BAOC_E_INVALID;
    for (int i = 0; i < h->n_blocks; ++i) {
        normalise(h->opts, &stats[i]);
        for (int c = 0; c < h->n_cfg; ++c) risk_out[size_t(i) * h->n_cfg + c] = risk_of(h->opts, stats[i], h->cfgs[c]);
    }
    return BAOC_OK;
}

int baoc_allocate(baoc_t* h, const double* risk, const int64_t* mem_bytes, const double* time_ratio, int64_t b_mem,
                  double b_time, const uint8_t* forbid, const double* pref, int32_t* assign_out, double* objective_out) {
    if (!h) return BAOC_E_INVALID;
    if (!risk || !mem_bytes || !time_ratio || !assign_out) return fail(h, BAOC_E_INVALID, "baoc_allocate: null argument");
    if (b_mem < 0 || !(b_time >= 0)) return fail(h, BAOC_E_INVALID, "baoc_allocate: negative budget");
    const int n = h->n_blocks, K = h->n_cfg;
    const double phi_scale = std::ldexp(1.0, 30), r_scale = std::ldexp(1.0, 20);

    Solver s;
    s.n = n; s.B = b_mem;
    s.R = int64_t(std::floor(double(n) * b_time * r_scale));
    s.state_limit = h->opts.node_limit > 0 ? h->opts.node_limit : int64_t(2000000);
    s.items.resize(n);
    for (int i = 0; i < n; ++i) {
        std::vector<Item> all;
        for (int c = 0; c < K; ++c) {
            const size_t k = size_t(i) * K + c;
            if (forbid && forbid[k]) continue;
            const Path p = path_of(h->cfgs[c]);
            if (p == kPathNone) continue;
            if (is_factored_path(p) && h->blocks[i].cols <= 1) continue;
            if (!std::isfinite(risk[k]) || !std::isfinite(time_ratio[k]) || time_ratio[k] < 0 || mem_bytes[k] < 0)
                return fail(h, BAOC_E_INVALID, "baoc_allocate: non-finite or negative input");
            const double phi = (risk[k] - (pref ? pref[k] : 0.0)) + h->opts.gamma * agg(h->cfgs[c]);
            if (!(std::fabs(phi) < 1e6)) return fail(h, BAOC_E_INVALID, "baoc_allocate: objective coefficient out of range");
            Item it;
            it.cfg = c;
            it.phi = int64_t(std::nearbyint(phi * phi_scale));
            it.mem = mem_bytes[k];
            it.rt = int64_t(std::nearbyint(time_ratio[k] * r_scale));
            it.red = 0;
            all.push_back(it);
        }
        // drop pairs that can never be part of the answer
        for (size_t a = 0; a < all.size(); ++a) {
            bool dominated = false;
            for (size_t b = 0; b < all.size() && !dominated; ++b) {
                if (a == b) continue;
                const Item &x = all[a], &y = all[b];
                if (y.mem <= x.mem && y.rt <= x.rt && (y.phi < x.phi || (y.phi == x.phi && y.cfg < x.cfg))) dominated = true;
            }
            if (!dominated) s.items[i].push_back(all[a]);
        }
        if (s.items[i].empty()) return fail(h, BAOC_E_INFEASIBLE, "baoc_allocate: a block has no admissible configuration");
    }

    // a capacity row that no assignment can violate is dropped
    {
        int64_t worst = 0;
        for (const auto& v : s.items) { int64_t m = 0; for (const Item& it : v) m = std::max(m, it.rt); worst += m; }
        s.use_time = worst > s.R;
    }
    s.fit_multipliers();
    for (auto& v : s.items)
        for (Item& it : v) it.red = i128(it.phi) * kOne + i128(s.l1) * it.mem + i128(s.l2) * it.rt;
    std::vector<int> pick;
    int64_t opt = 0;
    if (!s.solve(&pick, &opt)) {
        if (s.limit_hit) return fail(h, BAOC_E_INFEASIBLE, "baoc_allocate: state limit reached before any feasible assignment");
        return fail(h, BAOC_E_INFEASIBLE, "baoc_allocate: no assignment satisfies the budgets");
    }
    for (int i = 0; i < n; ++i) assign_out[i] = s.items[i][pick[i]].cfg;
    if (objective_out) *objective_out = double(opt) / phi_scale;
    if (s.limit_hit) { h->err = "baoc_allocate: state limit reached, assignment feasible but optimality not proven"; return BAOC_W_NODE_LIMIT; }
    return BAOC_OK;
}

}  // extern "C"
