// Internal declarations shared by the host and CUDA translation units of the
// library.  Nothing here is part of the public ABI (see include/baoc.h).
#pragma once

#include <cstddef>
#include <cstdint>
#include <string>
#include <vector>

#include "baoc.h"

#ifdef __CUDACC__
#define BAOC_HD __host__ __device__
#else
#define BAOC_HD
#endif

struct CUstream_st;
typedef CUstream_st* cudaStream_t;

namespace baoc {

constexpr int kMaxCfg = 32;
constexpr int kMaxSlots = 48;         // distinct (configuration, moment start steps) combinations one step can carry
constexpr int kQBlock = 256;          // elements per 8-bit quantisation block
constexpr int kTile = 4096;           // elements per tile of the streaming kernels
constexpr int kThreads = 256;         // threads per CTA of the streaming kernels
constexpr int kStatPartials = 4;      // doubles per tile written by the per-step statistics kernel
constexpr int kFinalSums = 16;        // doubles per tile slot written by the first finalize sweep
constexpr int kResidSums = 1;         // doubles per tile slot written by the second finalize sweep
constexpr int kBlockAcc = 8;          // doubles per block of running window values
constexpr int kRanks = 4;             // order statistics per block for the two quantiles
constexpr int kFinOut = 32;           // doubles per block copied to the host at the end of the window:
constexpr int kFinRanks = 16;         //   [0..15] first-sweep sums, [16..19] the four order statistics,
constexpr int kFinAcc = 20;           //   [20..27] the running window values,
constexpr int kFinResid = 28;         //   [28] the Eq. 7 numerator,
constexpr int kFinPilot = 29;         //   [29] the pilot value of the Eq. 6 preconditioner,
constexpr int kFinFlag = 30;          //   [30] non-zero: an order statistic lies outside the key range of the select
constexpr int kSelBits = 12;          // bits of the first and (at most) of the second radix pass of the quantile select
constexpr int kSelBins = 1 << kSelBits;
constexpr int kSel3Bits = 32 - 2 * kSelBits;   // bins of the third and last pass: 2^8 (a key has at most 31 bits: 12 + 12 + 7)
constexpr int kFinRunTiles = 32;      // most tiles a CTA of the first finalize sweep works through (its partial sums stay in fp32 that long)
constexpr int kSelRunTiles = 15;      // tiles a CTA of the stand-alone first pass (a repeated select) works through
constexpr int kPieceCols = 512;       // widest piece of the select's second sweep, in columns
constexpr int kPieceElems = 49152;    // most elements of a piece (its histograms count in 16 bits)
constexpr uint32_t kSurvOverflow = 0xffffffffu;   // count of a run whose survivors did not fit: the last pass reads v instead
constexpr int kRedRows = 64;          // rows per CTA of the row/column reduction kernel
constexpr int kRedCols = 512;         // columns per CTA of the row/column reduction kernel
constexpr int kTileF = 16384;         // elements per tile of the factored path (its slices are prefetched through shared memory)
constexpr int kTileQ = 16384;         // elements per tile of the 8-bit path (its slices are prefetched through shared memory)
constexpr int kCombineSlabs = 32;     // CTAs per factored block of the row/column combine

// Update paths of the fused step.
enum Path : int32_t {
    kPathA32 = 0, kPathA8 = 1, kPathR = 2, kPathF = 3, kPathS = 4,
    kPathG = 5,          // plain gradient step (SGD / SGDW without momentum): no state
    kPathA16 = 6,        // Adam / AdamW with bf16 moments
    kPathR16 = 7,        // momentum-free RMS scaling with a bf16 second moment
    kPathS16 = 8,        // SGD with a bf16 momentum buffer
    kPathR8 = 9,         // momentum-free RMS scaling with a block-wise absmax 8-bit second moment
    kPathS8 = 10,        // SGD with a block-wise absmax 8-bit momentum buffer
    kPathA8N = 11,       // Adam / AdamW with 8-bit moments in the non-linear (dynamic) codebook
    kPathFA = 12,        // factored second moment with Adafactor's options (beta2 schedule, update clipping, relative step)
    kPathCount = 13,
    kPathNone = -1
};

// Bits of baoc_config_t::af_flags.
enum AfFlags : int32_t { kAfSchedule = 1, kAfClip = 2, kAfRelative = 4, kAfEps1 = 8 };

inline bool is_factored_path(int path) { return path == kPathF || path == kPathFA; }

inline Path path_of(const baoc_config_t& c) {
    if (c.af_flags != 0 && !c.factored) return kPathNone;               // Adafactor's options belong to the factored tuple
    if (c.quantizer != 0 && !(c.bits == 8 && c.adaptive && c.momentum && !c.factored)) return kPathNone;   // the codebook is offered for 8-bit Adam
    if (c.factored) return (c.adaptive && !c.momentum) ? (c.af_flags ? kPathFA : kPathF) : kPathNone;   // row/column statistics in fp32, bf16 or 8-bit codes
    if (c.adaptive && c.momentum) return c.bits == 32 ? kPathA32 : (c.bits == 16 ? kPathA16 : (c.quantizer ? kPathA8N : kPathA8));
    if (c.adaptive && !c.momentum) return c.bits == 32 ? kPathR : (c.bits == 16 ? kPathR16 : kPathR8);
    if (!c.adaptive && c.momentum) return c.bits == 32 ? kPathS : (c.bits == 16 ? kPathS16 : kPathS8);
    return kPathG;       // neither mechanism: stateless, whatever bit-width the tuple names
}

// Families of update paths: each has its own instance of the fused kernel and its own stretch of the tile table.
enum Family : int32_t { kFamHead = 0, kFamDense = 1, kFamQ8 = 2, kFamCount = 3 };
inline int family_of(int path) {
    switch (path) {
        case kPathG: case kPathA16: case kPathR16: case kPathS16: return kFamDense;
        case kPathR8: case kPathS8: case kPathA8N: case kPathFA: return kFamQ8;
        default: return kFamHead;
    }
}

// Elements per tile of the fused step, by update path.
BAOC_HD inline int64_t step_tile_elems(int path) {
    return (path == kPathF || path == kPathFA) ? kTileF
                                               : ((path == kPathA8 || path == kPathR8 || path == kPathS8 || path == kPathA8N) ? kTileQ : kTile);
}

// Order of the paths in the step's tile table: the families one after another (each has its own kernel instance),
// within a family in descending bytes per element, so that the light tiles fill the tail of the grid.
constexpr int kPathOrder[kPathCount] = {kPathA32, kPathR, kPathS, kPathA8, kPathF, kPathA16, kPathR16, kPathS16, kPathG,
                                        kPathR8, kPathS8, kPathA8N, kPathFA};

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }

// Checked build (-DBAOC_CHECKED, see baoc_check.cuh): what a launch may touch (the bound buffer and the sizes of the
// tables it indexes), and the record of the first violation a kernel found.  Plain data; a normal build passes the
// context to the launchers too and ignores it.
struct CheckCtx {
    const char* lo;
    const char* hi;
    long long n_tiles;
    int n_blocks;
    int pad;
};
struct CheckRecord {
    unsigned int code;       // 0: clean
    unsigned int kernel;
    long long a, b, c, d;    // the offending numbers (index and limit, or range and buffer bounds)
};

// One tile of a streaming kernel: which block, and which kTile-sized piece of it.
struct Tile {
    uint32_t block;
    uint32_t piece;
};

// Geometry of the row/column reduction of one matrix block.  The matrix is cut
// into chunks of 64*L rows and strips of kRedCols columns; one CTA reduces one
// (chunk, strip) piece and writes its row sums to rowpart[strip][row] and its
// column sums to colpart[chunk][col].
struct RedGeom {
    double* rowpart;
    double* colpart;
    int32_t red0;        // index of the block's first reduction CTA (-1: no reduction for this block)
    int32_t chunks, strips, L;
};

// Per-block record of the statistics pass (device copy lives in the workspace).
struct StatBlock {
    float* m;            // EMA first moment (Eq. 3)
    float* v;            // EMA second moment
    uint16_t* gprev;     // previous gradient, bf16 bits
    double* rowsum;      // row sums of v (matrix blocks), length rows, followed by their total
    double* colsum;      // column sums of v, length cols
    int64_t numel;
    int64_t tile0;       // index of the block's first tile
    int32_t rows, cols;
    int32_t ntiles, npieces;   // tiles of the block; pieces of the select's second sweep (see SelPiece)
    RedGeom red;
    // coordinate sampling: the statistics see the sub-grid rows[ridx] x cols[cidx] of the block (null: the whole block)
    const int64_t* ridx;
    const int32_t* cidx;
    uint16_t* gsample;   // gathered gradient of the current step, bf16 bits
    float* psample;      // gathered parameters (finalize)
    int64_t full_cols;   // row length of the whole block
    int64_t piece0;      // index of the block's first piece
};

// Per-block record of the fused step (device copy lives in the state buffer).
struct StepBlock {
    void* s0;            // A32: m   A8: codes of m   R: v   F: r (rows)   S: m
    void* s1;            // A32: v   A8: codes of v          F: c (cols)
    float* a0;           // A8: absmax of m per quantisation block;  F: [0] = mean of r
    float* a1;           // A8: absmax of v per quantisation block
    double* mean_part;   // F: kCombineSlabs partial sums of the new r, then one ticket counter (uint32)
    int64_t numel;
    int32_t rows, cols;
    int32_t cfg;         // slot of the step's parameter table: the configuration together with the steps at which the
                         // block's moments last started from zero (they set the bias corrections)
    int32_t path;
    RedGeom red;
    // Factored path with bf16 or 8-bit statistics: s0 / s1 are then fp32 working copies in the scratch region (what
    // the update kernel reads: the new, un-rounded statistics) and the state proper is stored here.
    void* f0;            // stored row statistics: bf16 values or 8-bit codes (null when the state is fp32)
    void* f1;            // stored column statistics
    float* fa0;          // 8-bit: absmax of the row statistics per quantisation block
    float* fa1;          // 8-bit: absmax of the column statistics
    int32_t fbits;       // 32, 16 or 8 (factored blocks; 0 otherwise)
    int32_t af_flags;    // Adafactor's options of the block's tuple (kPathFA)
    double* norm_part;   // kPathFA: per tile of the block {sum u^2, sum theta^2}; a0[1] = clip factor, a0[2] = step size
};

// A stored moment, for the migration kernels of a re-configuration.
enum MomentKind : int32_t { kMomNone = 0, kMomF32 = 1, kMomBF16 = 2, kMomI8 = 3, kMomU8 = 4, kMomFactored = 5 };
struct MomentRef {
    void* data;          // fp32 / bf16 values or 8-bit codes
    float* absmax;       // one fp32 per 256 codes (8-bit kinds)
    void* r;             // factored: row statistics as stored (fp32, bf16 or 8-bit codes, by fbits)
    void* c;             // factored: column statistics as stored
    float* ar;           // factored, 8-bit: absmax of r / of c per 256 codes
    float* ac;
    float* wr;           // factored destination: the fp32 arrays the update kernel reads (r, c themselves when fbits == 32)
    float* wc;
    int32_t kind;
    int32_t rows, cols;  // the block's shape
    int32_t fbits;       // factored: 32, 16 or 8
    double divisor;      // fp32 sources only: the value read is data[e] / divisor (0: no division)
};

// State of one radix select: the bits found so far and the rank still to find
// among the elements that share them.
struct RankSel {
    uint32_t prefix;
    int32_t leader;      // first rank of the block with the same prefix (its histogram is shared)
    int64_t remaining;
};

// The key the select orders a block's second moments by: w = clamp(pattern - lo, 0, (4096 << s) - 1) for the fp32 bit
// pattern of an element (v >= 0, so patterns order like values): 12 + s bits, found in passes of 12, min(12, s) and
// s - 12 bits.  lo and s come from the smallest and largest pattern of a sample of the block, so that the first digit
// already spreads the block over most of its 4096 bins; an order statistic that comes out at either end of the key
// range (an element outside the sample's range) is found again with lo = -1, s = 19, which covers every finite value.
// s < 0: the block takes no part in this round of the select.
struct SelKey {
    int32_t lo;
    int32_t s;
};
constexpr int kSelFullS = 31 - kSelBits;   // with lo = -1 the key pattern + 1 of every finite non-negative value fits

// One CTA of the select's second sweep: rows [row0, row0 + nrows) x columns [col0, col0 + min(kPieceCols, cols - col0))
// of a matrix block; a vector block counts as a matrix of kPieceCols columns (its last row may be short).  The piece's
// survivors (elements that share a rank's first digit) are listed in surv[surv_off, surv_off + slots).
struct SelPiece {
    uint32_t block;
    uint32_t col0;
    uint32_t row0;
    uint32_t nrows;
    uint64_t surv_off;
    uint32_t slots;
    uint32_t pad;
};

// One CTA of the row/column reduction: a kRedRows x kRedCols piece of a matrix block.
struct RedTile {
    uint32_t block;
    uint32_t chunk;      // row chunk
    uint32_t strip;      // column strip
    uint32_t pad;
};

// Per-configuration scalars of one step, passed to the kernel by value.
struct CfgStep {
    float beta1, beta2;
    float om1, om2;      // 1 - beta1, 1 - beta2 (rounded from double)
    float eps;
    float wd;            // weight decay coefficient
    float decay;         // -lr*wd when the decay is decoupled, else 0
    float step_m;        // lr / (1 - beta1^t): multiplies a bias-corrected first moment
    float step_g;        // lr: multiplies a raw gradient or momentum buffer
    float rsqrt_bc2;     // 1 / sqrt(1 - beta2^t)
    float step_g_hat;    // lr * sqrt(1 - beta2^t)
    float step_m_hat;    // step_m * sqrt(1 - beta2^t): with eps_hat the update is step_m_hat * m / (sqrt(v) + eps_hat)
    float eps_hat;       // eps * sqrt(1 - beta2^t)
    int32_t coupled;     // 1: add wd*theta to the gradient
    int32_t af_flags;    // Adafactor's options (factored tuple)
    double beta1_d, beta2_d;   // the coefficients widened, for the exact side of the 8-bit path (beta2_d: this step's value under the schedule)
    double wd_d;
    double eps1_d;       // added to every squared gradient of the factored reduction (0 unless the tuple asks for it)
    double rho_d;        // relative step: min(1e-2, 1 / sqrt(t))
};
struct StepParams {
    CfgStep c[kMaxSlots];
};

struct Handle {
    int n_blocks = 0, n_cfg = 0;
    std::vector<baoc_block_t> blocks;
    std::vector<baoc_config_t> cfgs;
    baoc_opts_t opts{};
    mutable std::string err;
    int64_t numel = 0;
    int64_t launches = 0;

    // statistics workspace
    char* ws = nullptr;
    size_t ws_bytes = 0;
    bool ws_bound = false;
    int64_t stats_steps = 0;
    int64_t n_stat_tiles = 0;
    int64_t n_red_tiles = 0;         // reduction CTAs over all matrix blocks
    int n_matrix = 0;                // blocks with cols > 1
    std::vector<StatBlock> h_stat_blocks;
    bool sampled = false;                                  // statistics on a sampled sub-grid of every block
    std::vector<baoc_block_t> stat_shapes;                 // what the statistics see: the blocks, or their samples
    std::vector<std::vector<int64_t>> s_rows;
    std::vector<std::vector<int32_t>> s_cols;
    std::vector<int64_t> flat_ridx;                        // staging of the uploads (must outlive the async copies)
    std::vector<int32_t> flat_cidx;
    std::vector<const void*> sample_tables;
    std::vector<const void*> last_stat_grads;
    std::vector<const void*> last_stat_params;
    std::vector<SelKey> selkey_staging;                    // keys of a repeated select (must outlive the async copy)
    int64_t n_sel_pieces = 0;                              // pieces of the select's second sweep
    int64_t select_retries = 0;                            // blocks whose select was repeated in the last baoc_risk
    struct StatLayout {
        size_t blocks, tiles, red_tiles, matrix_ids, grads, params, m, v, gprev, partials, acc, fin, fin_out, hist, sel, selkey, pieces, resid_part, surv, surv_cnt,
               rowsum, colsum, redpart, ridx, cidx, gsample, psample, sgrads, sparams, total;
    } sl{};

    // optimizer state
    char* st = nullptr;
    size_t st_bytes = 0;
    bool configured = false;
    std::vector<int32_t> assign;
    std::vector<StepBlock> h_step_blocks;
    int64_t n_step_tiles = 0;
    int64_t n_step_red_tiles = 0;
    int n_factored = 0;              // blocks on a factored path (with or without Adafactor's options)
    int n_fa = 0;                    // of those, blocks with Adafactor's options; their tiles close the tile table
    int64_t fa_tile0 = 0, n_fa_tiles = 0;
    int64_t fam_tiles[kFamCount] = {0, 0, 0};   // tiles of each path family; the tile table holds the families one after another
    // Bias corrections count the gradients a moment has seen.  A re-configuration may restart some moments, so every
    // block carries the step counts at which its first and second moment last started from zero; blocks that share a
    // configuration and both counts share a slot of the step's parameter table.
    struct Slot { int32_t cfg; int64_t t_m0, t_v0; };
    std::vector<int64_t> t_m0, t_v0;
    std::vector<Slot> slots;
    std::vector<int32_t> slot_of;
    int64_t state_mem = 0;           // StateMem of the assignment (sum of M_{i,c_i})
    int64_t step_bytes = 0;          // algorithmic bytes of one step
    std::vector<int32_t> f_id_staging;   // staging of the id lists (must outlive the asynchronous upload)
    std::vector<const void*> last_step_grads;
    std::vector<const void*> last_step_params;
    struct StepLayout {
        size_t blocks, tiles, tiles_by_group, red_tiles, f_ids, grads, params, flags, redpart, states, total;
    } tl{};
    // The end-to-end call copies the gradients in groups of whole blocks and lets each group take its statistics step
    // and its optimizer step as soon as it has landed: a second tile table holds the step's tiles group by group
    // (within a group family by family), and every group knows its stretches of the tables.
    struct GroupStep {
        int b0, b1;                      // blocks [b0, b1)
        int64_t tile0;                   // first tile of the group in the by-group table
        int64_t fam_tiles[kFamCount];    // its tiles per path family
        int64_t red0, n_red;             // its stretch of the row/column reduction table
        int32_t f0, n_f;                 // its stretch of the list of factored blocks
    };
    std::vector<GroupStep> groups;
    std::vector<Tile> group_tiles;       // staging of the by-group table (must outlive the asynchronous upload)
    // Optional schedule of the factored blocks in baoc_step: groups of whole factored blocks of at most
    // factored_group_bytes of gradient each take their row/column reduction, its combine and their update tiles back to
    // back, so that the update's second read of the gradient can come from L2 (0: one reduction and one update launch
    // for all blocks).  A group is a stretch of the reduction table, of the list of factored blocks and of the main
    // tile table (the factored tiles close the headline family's stretch, block by block).
    struct FactoredGroup { int64_t tile0, n_tiles, red0, n_red; int32_t f0, n_f; };
    int64_t factored_group_bytes = 0;
    std::vector<FactoredGroup> f_groups;
    int64_t n_factored_tiles = 0;

    // optional per-kernel timing of the step (CUDA events, owned by the CUDA translation unit)
    bool prof_on = false, prof_valid = false;
    void* prof_ev[3] = {nullptr, nullptr, nullptr};
    // host-to-device pipeline of baoc_step_from_host: an internal copy stream and one event per group of blocks
    static constexpr int kCopyGroups = 8;
    void* copy_stream = nullptr;
    void* copy_ev[kCopyGroups + 1] = {};
    void (*cuda_cleanup)(Handle*) = nullptr;
    ~Handle() { if (cuda_cleanup) cuda_cleanup(this); }
};

int fail(const Handle* h, int code, const std::string& msg);

// Reduction geometry of a rows x cols matrix (pointers left null).
RedGeom red_geometry(int32_t rows, int32_t cols, int refine);

// M_{i,c}: bytes of persistent state of one block under one configuration.
int64_t state_mem_bytes(const baoc_config_t& c, const baoc_block_t& b);
// Algorithmic HBM bytes per step of one block under one configuration.
double step_traffic_bytes(const baoc_config_t& c, const baoc_block_t& b);

void compute_stat_layout(Handle* h);
void build_sel_pieces(const Handle* h, std::vector<SelPiece>* out, std::vector<StatBlock>* blocks, uint64_t* surv_words);

// Kernel launchers (defined in the .cu files).  Each returns 0 or a cudaError_t value.
int launch_stats_step(const StatBlock* blocks, const Tile* tiles, const void* const* grads, double* partials,
                      int64_t n_tiles, float one_minus_beta_m, float one_minus_beta_v, const CheckCtx& ck, cudaStream_t s);
int launch_stats_combine(const StatBlock* blocks, const double* partials, double* acc, int n_blocks, int has_prev,
                         double beta_rho, double eps, const CheckCtx& ck, cudaStream_t s);
// First finalize sweep (with the pilot values, the start of the select and its first radix pass), then, after the
// row/column sums of the matrix blocks, the second and third sweep and the gather of the per-block results.
int launch_final_sums(const StatBlock* blocks, const Tile* tiles, const float* const* params, double* fin,
                      double* fin_out, uint32_t* hist, RankSel* sel, SelKey* selkey, int64_t n_tiles, int n_blocks, double eps,
                      float eps_adam, int quantizer8, int debias, float m_scale, float v_scale, const CheckCtx& ck, cudaStream_t s);
// The buffers of the select's second and third sweep.
struct SelectArgs {
    const StatBlock* blocks;
    const Tile* tiles;
    const SelPiece* pieces;
    RankSel* sel;
    const SelKey* selkey;
    uint32_t* hist;
    uint32_t* surv;
    uint32_t* surv_cnt;      // per piece: survivors listed, or kSurvOverflow
    double* resid_part;      // per piece: its part of the Eq. 7 numerator
    double* fin_out;
    const double* acc;
    int64_t n_tiles, n_pieces;
    int n_blocks;
};
int launch_final_resid_select(const SelectArgs& a, const CheckCtx& ck, cudaStream_t s);
// The select once more, from its first pass, for the blocks whose selkey has s >= 0 (the others keep their results).
int launch_select_again(const SelectArgs& a, const CheckCtx& ck, cudaStream_t s);
int launch_sample_gather(const StatBlock* blocks, const Tile* tiles, const void* const* src, int64_t n_tiles, int fp32,
                         const CheckCtx& ck, cudaStream_t s);
int launch_moment_reduce(const StatBlock* blocks, const RedTile* rtiles, const int32_t* ids, int64_t n_red, int n_matrix,
                         const CheckCtx& ck, cudaStream_t s);
int launch_factored_reduce(const StepBlock* blocks, const RedTile* rtiles, const int32_t* ids, const void* const* grads,
                           const float* const* params, int64_t n_red, int n_factored, const StepParams& P, const CheckCtx& ck,
                           cudaStream_t s);
int launch_fused_step(const StepBlock* blocks, const Tile* tiles, const void* const* grads, float* const* params,
                      uint32_t* flags, int64_t n_tiles, int family, const StepParams& P, const CheckCtx& ck, cudaStream_t s);
// Checked build: fetch (and clear) the violation record of each CUDA translation unit, and a self-test kernel that runs
// the range check on numbers that violate it (no memory is touched).  Each returns 0 or a cudaError_t value.
int stats_check_fetch(CheckRecord* out);
int finalize_check_fetch(CheckRecord* out);
int step_check_fetch(CheckRecord* out);
int launch_check_selftest(cudaStream_t s);
// Adafactor's options: per tile of the given blocks the sums of u^2 and theta^2, then per block the clip factor and the
// step size (ids: the blocks, n of them; tiles: their stretch of the tile table).
int launch_factored_norms(const StepBlock* blocks, const Tile* tiles, const int32_t* ids, const void* const* grads,
                          const float* const* params, int64_t n_tiles, int n, const StepParams& P, const CheckCtx& ck,
                          cudaStream_t s);
int launch_convert_moment(const MomentRef& src, const MomentRef& dst, int64_t numel, cudaStream_t s);
// Copy groups of the end-to-end call: up to Handle::kCopyGroups runs of whole blocks of about equal bytes.
void compute_copy_groups(const Handle* h, std::vector<int>* b0, std::vector<int>* b1);
int compute_step_layout(const Handle* h, const int32_t* assign, Handle::StepLayout* out,
                        std::vector<StepBlock>* blocks, std::vector<Tile>* tiles,
                        std::vector<RedTile>* red, int64_t* state_mem, int64_t* step_bytes);

}  // namespace baoc

struct baoc_handle : public baoc::Handle {};
