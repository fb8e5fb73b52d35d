/*
 * baoc.h -- C ABI of the B200 (sm_100a) library for the data-parallel hot path
 * of BAOC, the Budget-Aware Optimizer Configurator.
 *
 * The path: during a sampling window every parameter block's gradient is
 * streamed once per step to update the block's statistics (Sec. 3.3, Eq. 3-8);
 * at the end of the window the statistics are reduced to a risk matrix
 * (Eq. 9, Appendix A Eq. 10-21); a budgeted allocation picks one configuration
 * per block (Eq. 1-2); from then on one fused step updates every block under
 * its own configuration (Definition 3.1, Algorithm 1 "Training").
 *
 * Conventions
 *   - Every function returns an int status: 0 = BAOC_OK, negative = error,
 *     positive = warning (result still valid).  baoc_last_error() returns a
 *     message for the last non-zero status of a handle.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA
 *     global memory of the current device.  The library never allocates device
 *     memory: it reports sizes, the caller allocates and passes pointers, and
 *     keeps them alive while the handle uses them.
 *   - Device pointers must be 16-byte aligned (BAOC_E_ALIGN otherwise).  Block
 *     element counts are arbitrary (>= 1).
 *   - All GPU work is queued on the caller's stream (a cudaStream_t passed as
 *     baoc_stream_t; NULL is the default stream).  Only baoc_risk(),
 *     baoc_read_stats() and baoc_nonfinite() wait for the stream, because they
 *     return data to the host.
 *   - A handle is not thread-safe.  Invalid arguments are rejected on the host
 *     before anything is launched; no call can fault the device on bad input
 *     that the host can see (null pointers, bad sizes, wrong call order).
 *   - Gradients are bfloat16, parameters fp32, one contiguous array per block.
 */
#ifndef BAOC_H
#define BAOC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct baoc_handle baoc_t;
typedef void* baoc_stream_t;          /* a cudaStream_t */

enum {
    BAOC_OK = 0,
    BAOC_E_INVALID = -1,     /* null pointer, bad size, bad value */
    BAOC_E_ALIGN = -2,       /* a device pointer is not 16-byte aligned */
    BAOC_E_STATE = -3,       /* call order: e.g. step before configure */
    BAOC_E_INFEASIBLE = -4,  /* no assignment satisfies both budgets and the mask */
    BAOC_E_CUDA = -5,        /* a CUDA runtime call failed (message has the reason) */
    BAOC_E_NONFINITE = -6,   /* reserved */
    BAOC_E_WORKSPACE = -7,   /* workspace or state buffer too small */
    BAOC_W_NODE_LIMIT = 1    /* allocator hit its node limit: assignment feasible, optimality not proven */
};

/* One parameter block B_i (Sec. 3.1): numel = d_i parameters viewed as a
 * rows x cols row-major matrix.  A vector has rows = numel, cols = 1; tensors
 * of more than two dimensions are flattened to (dim0, rest). rows*cols == numel. */
typedef struct {
    int64_t numel;
    int32_t rows, cols;
} baoc_block_t;

/* A configuration tuple c = (y_a, y_m, y_d, y_f, b) of Definition 3.1 and the
 * hyper-parameters of the update rule it selects.  Tuples the library can
 * instantiate (Sec. 4.1 lists the mechanisms, each at 8/16/32-bit states):
 *   (1,1,*,0,32|16|8)  Adam / AdamW with fp32, bf16 or block-wise absmax 8-bit moments (8-bit: linear codes or the
 *                      non-linear codebook, see quantizer);
 *   (1,0,*,0,32|16|8)  momentum-free RMS scaling with an fp32, bf16 or 8-bit second moment;
 *   (1,0,*,1,32|16|8)  factored second moment (matrix blocks only), its row and column statistics kept
 *                      in fp32, in bf16 or as block-wise absmax 8-bit codes; optionally with the remaining parts
 *                      of Adafactor (see af_flags);
 *   (0,1,*,0,32|16|8)  SGD with momentum (beta1 is the momentum coefficient), fp32, bf16 or 8-bit buffer;
 *   (0,0,*,0,any)      plain gradient step (SGD / SGDW): no state, so the bit-width only enters Agg(c).
 * y_d selects decoupled (1) or coupled (0) weight decay in all of them.  With
 * bf16 or 8-bit states the parameter update uses the new moments before they are
 * rounded for storage.  Other tuples (factored with momentum or without
 * adaptive scaling) may appear in the candidate set for risk and cost queries
 * but cannot be assigned. */
typedef struct {
    uint8_t adaptive, momentum, decoupled_wd, factored, bits;
    uint8_t quantizer;   /* 8-bit Adam only: 0 = linear absmax codes, 1 = the non-linear codebook (below) */
    uint8_t af_flags;    /* factored tuple only: Adafactor's options (below), 0 = none */
    uint8_t reserved;    /* 0 */
    float lr, beta1, beta2, eps, weight_decay;
} baoc_config_t;

/* Two alternative readings that a configuration may select.
 *
 * quantizer = BAOC_Q_DYNAMIC.  The paper calls Q_b "a standard quantizer" and
 * cites block-wise 8-bit optimizers for its AdamW8 baseline (Sec. 4.1).  Their
 * data type is non-linear: an optional sign bit, a run of zero bits whose
 * length E is a decimal exponent, an indicator bit, and F remaining bits as a
 * linear fraction of the decade.  This library builds its own table from that
 * description: magnitudes 10^-E (0.1 + 0.9 (k+1) / 2^F), k = 0 .. 2^F - 1,
 * F = B - 1 - E, E = 0 .. B - 1, with B = 7 for first moments (signed: 255
 * entries with zero) and B = 8 for second moments (256 entries with zero).  A
 * code is the index of the entry nearest to x / absmax in ascending order (a
 * tie goes to the smaller magnitude); blocks of 256 elements and fp32 absmax as
 * for the linear codes.  Offered for the tuple (1,1,*,0,8); baoc_opts_t's
 * quantizer8 selects it for the precision cosine of Eq. 8.
 *
 * af_flags.  The paper names Adafactor among its mechanisms (Sec. 4.1) without
 * saying which parts of the published algorithm are meant; the factored tuple
 * by default keeps only the factored second moment.  The flags add the rest:
 *   BAOC_AF_SCHEDULE  beta2_t = 1 - t^-0.8 instead of the constant beta2, and
 *                     no bias correction of the second moment;
 *   BAOC_AF_CLIP      the update u = g / (sqrt(v) + eps) is divided by
 *                     max(1, RMS(u)) (clipping threshold 1);
 *   BAOC_AF_RELATIVE  step size max(1e-3, RMS(theta)) * min(1e-2, 1/sqrt(t))
 *                     instead of lr, with theta before the step (a decoupled
 *                     decay uses the same step size);
 *   BAOC_AF_EPS1      1e-30 is added to every squared gradient before the row
 *                     and column means.
 * Clipping and the relative step need the norms of u and theta over the whole
 * block: one more sweep over the block's gradient and parameters per step. */
enum { BAOC_Q_LINEAR = 0, BAOC_Q_DYNAMIC = 1 };
enum { BAOC_AF_SCHEDULE = 1, BAOC_AF_CLIP = 2, BAOC_AF_RELATIVE = 4, BAOC_AF_EPS1 = 8 };

/* Options of the statistics, normalisation and allocation (defaults from
 * baoc_default_opts: Eq. 3 "standard Adam values", Appendix A anchors,
 * gamma = 0.1).  qblock must be 256. */
typedef struct {
    double beta_m, beta_v;        /* Eq. 3 */
    double beta_rho;              /* Eq. 5 smoothing factor */
    double eps;                   /* Appendix A.1: 1e-12 */
    double a_lo, a_hi;            /* Eq. 11 */
    double rho_lo, rho_hi;        /* Eq. 13 */
    double snr_lo, snr_hi;        /* Eq. 15 */
    double w[5];                  /* user weights W: w_A, w_M, w_C, w_F, w_Q */
    double gamma;                 /* weight of Agg(c) in the objective */
    double eps_adam;              /* epsilon of the update direction in Eq. 8 */
    int32_t use_snr;              /* Eq. 17; 0 selects s_M = s_rho */
    int32_t qblock;               /* elements per 8-bit quantisation block */
    int64_t node_limit;           /* allocator search-node limit (0 = default) */
    int32_t quantizer8;           /* the 8-bit quantiser of Eq. 8: BAOC_Q_LINEAR (default) or BAOC_Q_DYNAMIC */
    int32_t debias;               /* 0 (default): the diagnostics of Eq. 4-8 are taken from the recursion of Eq. 3 as it
                                   * stands; 1: from the bias-corrected moments m / (1 - beta_m^T), v / (1 - beta_v^T)
                                   * after the T gradients observed (the alternative reading of the hats in Eq. 3) */
} baoc_opts_t;

/* Per-block diagnostics z_i: raw (Eq. 4-8), normalised (Eq. 10-20) and a few
 * extras that are not used by the risk. */
typedef struct {
    double A, rho_bar, snr, C, F, Q32, Q16, Q8;
    double q10, q90;              /* the two quantiles of Eq. 4 */
    double rho_mom;               /* EMA of cos(g_t, m_{t-1}) */
    double err_m8, err_v8, err_m16, err_v16;   /* ||x - Q_b(x)|| / ||x|| */
    double s_A, s_rho, s_snr, s_M, C_tilde, s_F, lQ32, lQ16, lQ8;
    double last_cos;              /* cosine of the last step */
    int64_t n_cos;                /* number of cosines averaged into rho_bar */
} baoc_block_stats_t;

typedef struct {
    int32_t n_blocks, n_cfg;
    int64_t numel;                /* sum of d_i */
    int64_t n_tiles;              /* tiles of the statistics pass */
    int64_t stats_steps;          /* gradient observations so far in this window */
    int64_t state_bytes;          /* StateMem of the configured assignment (0 before configure) */
    int64_t kernel_launches;      /* kernels this handle has launched so far */
    int64_t stats_bytes_per_call; /* algorithmic HBM bytes of one baoc_sample_stats */
    int64_t step_bytes_per_call;  /* algorithmic HBM bytes of one baoc_step under the assignment */
    int64_t select_retries;       /* blocks whose quantile select (Eq. 4) the last baoc_risk had to repeat over the
                                   * full value range because an order statistic lay outside the range of the
                                   * block's sample; 0 in the usual case */
} baoc_info_t;

/* Fill *o with the defaults.  Host only. */
void baoc_default_opts(baoc_opts_t* o);

/* Create a handle for n_blocks blocks and n_cfg candidate configurations
 * (Algorithm 1 inputs).  Copies all arrays.  opts may be NULL (defaults).
 * Host only; touches no GPU.  Errors: BAOC_E_INVALID (null, n <= 0,
 * rows*cols != numel, n_cfg > 32, bits not in {8,16,32}, qblock != 256). */
int baoc_create(baoc_t** h, int n_blocks, const baoc_block_t* blocks,
                int n_cfg, const baoc_config_t* cfgs, const baoc_opts_t* opts);

/* Free the handle (host memory only; device buffers belong to the caller). */
void baoc_destroy(baoc_t* h);

/* Message of the last error on this handle ("" if none).  Never NULL. */
const char* baoc_last_error(const baoc_t* h);

/* Fill *info.  Host only. */
int baoc_query(const baoc_t* h, baoc_info_t* info);

/* ---- sampling window (Algorithm 1 "Warmup and diagnostics") -------------- */

/* Bytes of device workspace the statistics need: the EMA moments of Eq. 3
 * (fp32), the previous gradient (bf16), per-tile partial sums, per-block
 * accumulators, tables and the scratch of the finalize pass. */
int baoc_stats_workspace_bytes(const baoc_t* h, size_t* bytes);

/* Give the handle its statistics workspace (device, >= the size above,
 * 256-byte aligned).  Queues the zero-fill of the moments and the upload of
 * the tile tables on the stream and starts a new window. */
int baoc_bind_stats_workspace(baoc_t* h, void* dev, size_t bytes, baoc_stream_t stream);

/* Coordinate sampling (Sec. 3.1: the statistics are computed on a fixed sample
 * Omega_i of each block's coordinates, |Omega_i| = ceil(s d_i), s = 0.1 % by
 * default, drawn once).  By default this library observes every coordinate
 * (s = 1).  With a sample set, block i is observed on the sub-grid
 * rows[0..n_rows) x cols[0..n_cols) of its rows x cols matrix, so that the
 * "matrix form of the sampled gradients" of Eq. 7 exists (a vector block has
 * n_cols = 1 and cols = NULL); n_rows * n_cols plays the role of |Omega_i|.
 * Indices are host arrays, in range and strictly increasing; the library copies
 * them.  The draw itself is the caller's (it is an input, like the gradients).
 * Every per-parameter quantity of the window (moments, previous gradient,
 * quantiles, Eq. 6's parameters) then lives on the sample: each observation
 * first gathers g[Omega] into the workspace, baoc_risk gathers theta[Omega].
 * Call before baoc_bind_stats_workspace (the workspace size changes; a bound
 * workspace must be bound again); samples == NULL returns to the dense sample.
 * BAOC_E_STATE once the window has observations. */
typedef struct {
    int64_t n_rows;
    int32_t n_cols;
    const int64_t* rows;
    const int32_t* cols;
} baoc_sample_t;
int baoc_set_sampling(baoc_t* h, const baoc_sample_t* samples /* [n_blocks] or NULL */);

/* One gradient observation of every block (Eq. 3 and the cosine of Eq. 5).
 * grads: host array of n_blocks device pointers to bf16 gradients (block i has
 * numel_i elements).  The sample is dense (every coordinate of every block)
 * unless baoc_set_sampling chose a sub-grid.  Queues one streaming kernel and
 * one small combine kernel (after a gather kernel when sampling); does not wait. */
int baoc_sample_stats(baoc_t* h, const void* const* grads, baoc_stream_t stream);

/* Copy the running per-block values of the window (rho_bar, last_cos, n_cos,
 * rho_mom; other fields zero) to host stats_out[n_blocks].  Waits. */
int baoc_read_stats(baoc_t* h, baoc_block_stats_t* stats_out, baoc_stream_t stream);

/* End of the window: finalize the diagnostics (Eq. 4-8) on the device, copy
 * them to the host, normalise them (Eq. 10-20) and fill the risk matrix
 * R_i(c) (Eq. 9).  params: host array of n_blocks device pointers to fp32
 * parameters (used by Eq. 6).  risk_out: host [n_blocks*n_cfg], row-major by
 * block.  stats_out: host [n_blocks] or NULL.  Waits for the stream.
 * BAOC_E_STATE if no gradient has been observed. */
int baoc_risk(baoc_t* h, const float* const* params, double* risk_out,
              baoc_block_stats_t* stats_out, baoc_stream_t stream);

/* Host-only part of baoc_risk: read the raw fields of stats[i] (A, rho_bar,
 * snr, C, F, Q32, Q16, Q8), fill their normalised fields in place and write
 * risk_out[n_blocks*n_cfg].  No GPU needed. */
int baoc_risk_from_raw(const baoc_t* h, baoc_block_stats_t* stats, double* risk_out);

/* ---- allocation (Algorithm 1 "Allocation", Eq. 1-2) ---------------------- */

/* Cost model.  mem_bytes[i*n_cfg+c] = M_{i,c}, the persistent state bytes of
 * block i under configuration c (StateMem definition, Sec. 3.1; padding
 * excluded).  time_ratio[i*n_cfg+c] = algorithmic HBM bytes per parameter of
 * c divided by those of fp32 Adam, a stand-in for the measured r_{i,c}.
 * Either output may be NULL.  Host only. */
int baoc_cost_model(const baoc_t* h, int64_t* mem_bytes, double* time_ratio);

/* Measured cost model (Sec. 3.1, "Time Budget Definition": r_{i,c} = t_{i,c} /
 * t_{i,base} from a one-step timing of updating block i with configuration c on
 * the target hardware and the same tensor shapes).  For every pair the library
 * can instantiate, the block alone is stepped `reps` times (after one warm-up)
 * under that configuration with the learning rate forced to 0, timed with CUDA
 * events on the stream; time_ratio_out[i*n_cfg+c] = t_{i,c} / t_{i,base_cfg}
 * (pairs that cannot be assigned keep the value of baoc_cost_model);
 * time_ms_out (may be NULL) gets the milliseconds, -1 for unmeasured pairs.
 * With lr = 0 the parameters come out bit-identical provided eps > 0 for the
 * adaptive tuples; the handle's own statistics and optimizer state are not
 * touched: the states of the timed steps live in scratch_dev (device, 256-byte
 * aligned, >= baoc_time_scratch_bytes).  grads / params: host arrays of
 * n_blocks device pointers as in baoc_step.  Waits for the stream many times; a
 * warm-up-time helper, not part of the training loop. */
int baoc_time_scratch_bytes(const baoc_t* h, size_t* bytes);
int baoc_measure_time_ratios(baoc_t* h, const void* const* grads, float* const* params, void* scratch_dev,
                             size_t scratch_bytes, int base_cfg, int reps, double* time_ratio_out,
                             double* time_ms_out, baoc_stream_t stream);

/* Solve Eq. 2 exactly on the host: minimise sum_i Phi_{i,c_i} with
 * Phi = (R - pref) + gamma*Agg(c) subject to sum M <= b_mem and
 * (1/N) sum r <= b_time, one configuration per block.  Arithmetic is fixed
 * point: Phi -> rne(Phi*2^30), r -> rne(r*2^20), time cap floor(N*b_time*2^20);
 * among optimal assignments the lexicographically smallest (block 0 first,
 * lower configuration index first) is returned.  forbid[i*n_cfg+c] != 0
 * excludes a pair (hard constraint); pairs the library cannot instantiate
 * (factored on a vector block, unsupported tuples) are excluded as well.
 * forbid, pref, objective_out may be NULL.  All arrays host.  Returns
 * BAOC_E_INFEASIBLE when nothing fits, BAOC_W_NODE_LIMIT when the search
 * stopped early (assignment feasible but not proven optimal). */
int baoc_allocate(baoc_t* h, const double* risk, const int64_t* mem_bytes,
                  const double* time_ratio, int64_t b_mem, double b_time,
                  const uint8_t* forbid, const double* pref,
                  int32_t* assign_out, double* objective_out);

/* ---- block partitioning (appendix on block partitioning, Algorithm 2) ----- */

/* From candidate units to blocks.  The units come in forward order (the
 * structural scan of the model is the caller's); numel[j] = n_j parameters;
 * z: row-major [n_units][k] normalised diagnostic vectors (for instance s_A,
 * s_M, C~, s_F, l_Q of baoc_block_stats_t after a window run with the units
 * as blocks); w: k non-negative weights or NULL for w_k = 1; alpha: the
 * minimum block size as a fraction of all parameters (n_min = alpha*|Theta|);
 * tau: the statistic-difference threshold, negative for the paper's choice,
 * the upper quartile of Delta(U_a,U_b) = max_k w_k |z_a,k - z_b,k| over all
 * pairs of units.  The algorithm's steps are stated loosely; this library's
 * reading: every gap between adjacent units is a candidate boundary; a group
 * of units has the size-weighted mean of their vectors; a unit or group below
 * n_min joins the adjacent group with the smaller Delta (ties: the smaller
 * neighbour, then the left one); a boundary between adjacent groups survives
 * iff their Delta exceeds tau; a formed block is cut again where the means of
 * its two sides differ most, if by more than tau and both sides reach n_min;
 * what is still below n_min is merged as before.  Blocks are runs of
 * consecutive units: block_of_unit[j] (out, [n_units]) is non-decreasing from
 * 0.  n_blocks and tau_used may be NULL.  Host only, no handle, no GPU.
 * BAOC_E_INVALID: null, n_units < 1, k outside 1..64, numel < 1, alpha outside
 * [0,1], a negative weight, a non-finite z or w, tau NaN. */
int baoc_partition(int n_units, const int64_t* numel, const double* z, int k, const double* w,
                   double alpha, double tau, int32_t* block_of_unit, int32_t* n_blocks,
                   double* tau_used);

/* ---- training (Algorithm 1 "Training") ----------------------------------- */

/* Bytes of device memory the optimizer state of this assignment needs
 * (states plus alignment padding, tables and the scratch of the factored
 * path).  assign: host [n_blocks]. */
int baoc_state_bytes(const baoc_t* h, const int32_t* assign, size_t* bytes);

/* Instantiate the optimizer O({c_i}): lay the states out in state_dev
 * (device, 256-byte aligned, >= baoc_state_bytes), queue their zero-fill and
 * the upload of the tile table.  The step counter restarts. */
int baoc_configure(baoc_t* h, const int32_t* assign, void* state_dev, size_t bytes,
                   baoc_stream_t stream);

/* Online re-configuration with optimizer-state inheritance (Sec. 3.1, remark on
 * re-planning; appendix study "online reallocation with state inheritance").
 * The paper says only that compatible states are migrated when possible; this
 * library's rule, with inherit != 0:
 *   - a first moment is kept between tuples of the same family (Adam-type
 *     averages, or momentum buffers of SGD), re-stored in the new precision;
 *   - an element-wise second moment (Adam, RMS scaling) is kept by any tuple
 *     with an element-wise second moment, and becomes its row and column means
 *     under the factored tuple; a factored one becomes r_i c_j / mean(r)
 *     element-wise;
 *   - every other moment of the new tuple starts from zero, and its bias
 *     correction restarts: it counts steps from steps_done.
 * With inherit == 0 every moment restarts.  new_assign: host [n_blocks].
 * new_state_dev: device, 256-byte aligned, >= baoc_state_bytes(new_assign), and
 * NOT overlapping the current state buffer, which is read while the new one is
 * written (the transient memory the paper's remark mentions); once the stream
 * has passed this call the old buffer may be freed.  steps_done: the number of
 * baoc_step calls made so far (the next call passes steps_done + 1).  Queues
 * the zero-fill, the table uploads and the migration kernels; does not wait.
 * BAOC_E_STATE before the first baoc_configure. */
int baoc_reconfigure(baoc_t* h, const int32_t* new_assign, void* new_state_dev, size_t bytes,
                     int64_t steps_done, int inherit, baoc_stream_t stream);

/* baoc_configure with a warm start: the moments the sampling window has built
 * (Eq. 3) become the optimizer's initial moments instead of zeros (Algorithm 1
 * hands over from "Warmup and diagnostics" to "Training" without saying what
 * the new optimizer starts from; the same appendix study shows that dropped
 * states cost quality).  The rule, per block, with T_w observations in the
 * window:
 *   - a tuple with an Adam-type first moment whose beta1 equals the window's
 *     beta_m (compared as fp32) starts from m_hat; an SGD momentum buffer with
 *     that coefficient starts from m_hat / (1 - beta_m), which is the buffer
 *     m <- beta*m + g would have built from the same gradients;
 *   - a tuple with a second moment whose beta2 equals the window's beta_v
 *     starts from v_hat (element-wise, or its row and column means when
 *     factored);
 *   - each value is stored in the tuple's precision; a moment that is started
 *     this way has seen T_w gradients, so at step t its bias correction uses
 *     the exponent t + T_w; any other moment starts from zero as in
 *     baoc_configure.
 * Needs a bound workspace with at least one observation and a dense window
 * (BAOC_E_STATE otherwise: a sampled sub-grid does not cover the block).
 * state_dev as for baoc_configure; it must not overlap the workspace.  The
 * step counter restarts: the next baoc_step passes 1.  Queues the zero-fill,
 * the table uploads and the conversion kernels; does not wait. */
int baoc_configure_from_window(baoc_t* h, const int32_t* assign, void* state_dev, size_t bytes,
                               baoc_stream_t stream);

/* One training step of every block under its configuration.  grads / params:
 * host arrays of n_blocks device pointers (bf16 / fp32).  step_t: 1-based step
 * number (bias corrections).  Queues the fused update kernel, one launch per
 * family of update paths in use (headline tuples; stateless and bf16-state
 * tuples; 8-bit single-moment tuples), preceded by the row/column reduction
 * kernels when some block is factored; does not wait. */
int baoc_step(baoc_t* h, const void* const* grads, float* const* params,
              int64_t step_t, baoc_stream_t stream);

/* Schedule of the factored blocks inside baoc_step.  The factored second moment
 * needs the row and column sums of g*g of a whole matrix before any element of
 * that matrix can be updated, so its gradient is read twice: by the reduction,
 * then by the update.  group_bytes == 0 (the default): one reduction over all
 * factored blocks, then one update launch for all blocks.  group_bytes > 0:
 * the factored blocks are taken in groups of whole blocks of at most that many
 * bytes of gradient (a larger block forms a group alone), and every group runs
 * its reduction, the combine and its update tiles back to back, so that the
 * second read can be served from L2 (which holds 126 MB on B200); the results
 * are bit-identical, the step then takes 3 launches per group.  Call before
 * baoc_configure (BAOC_E_STATE afterwards).  Definition 3.1 fixes what is
 * computed, not in which order the blocks are visited. */
int baoc_set_factored_schedule(baoc_t* h, int64_t group_bytes);

/* End-to-end convenience for callers whose gradients live in host memory:
 * copies block i's bf16 gradient from host_grads[i] (pinned memory advised) to
 * the device buffer dev_grads[i], then does baoc_sample_stats (if do_stats)
 * and baoc_step (if step_t > 0) on the same stream.  With do_stats the copy
 * runs on an internal stream in up to eight groups of whole blocks, and each
 * group takes its statistics step and its optimizer step as soon as it has
 * landed, so that all but the last group's work hides behind the transfer;
 * every block sees exactly the arithmetic of the separate calls.  Does not
 * wait. */
int baoc_step_from_host(baoc_t* h, const void* const* host_grads, void* const* dev_grads,
                        float* const* params, int do_stats, int64_t step_t,
                        baoc_stream_t stream);

/* Where a block's window or optimizer state lives, for inspection,
 * checkpointing and tests.  which: 0 = EMA first moment (fp32), 1 = EMA second
 * moment (fp32), 2 = previous gradient (bf16) of the statistics workspace;
 * 10..13 = the block's optimizer state tensors under the configured
 * assignment: Adam m, v (fp32 or bf16); 8-bit Adam codes of m (int8), codes of v
 * (uint8), absmax of m (fp32), absmax of v (fp32); RMS v; SGD m (fp32 or bf16);
 * 8-bit RMS / SGD-momentum: codes, then their absmax; factored r (rows), c
 * (cols) as fp32 or bf16, or as uint8 codes followed by the absmax of r and
 * of c (one fp32 per 256 codes); nothing for the plain gradient step.  Writes the device pointer, the element count and the element size
 * in bytes; BAOC_E_INVALID if the block has no such tensor, BAOC_E_STATE if the
 * buffer is not bound yet.  Host only. */
int baoc_view(const baoc_t* h, int block, int which, void** dev_ptr, int64_t* count, int32_t* elem_bytes);

/* Number of blocks whose last fused step saw a non-finite gradient or
 * produced a non-finite parameter; flags[n_blocks] (host, may be NULL) gets
 * one byte per block.  Waits. */
int baoc_nonfinite(baoc_t* h, uint8_t* flags, int32_t* count, baoc_stream_t stream);

/* ---- checkpoint / resume ---------------------------------------------------------
 * All per-parameter state of a handle lives in the two caller-owned device
 * buffers (statistics workspace, optimizer state); the handle itself only adds
 * the window's step count and the configured assignment.  A checkpoint is
 * therefore: the bytes of those buffers (copied by the caller, with the stream
 * idle) plus the small host blob of baoc_export.  The paper only notes that
 * re-planning needs state to be carried over (Sec. 3.1, online variant); the
 * format is this library's own.
 *
 * baoc_export: writes the blob to buf (host, capacity bytes) and its length to
 * *size; with buf == NULL only *size is written.  BAOC_E_WORKSPACE if capacity
 * is too small.  Host only.
 *
 * baoc_import: h must have been created with the same blocks and the same
 * configuration tuples (hyper-parameters may differ).  ws_dev / state_dev are
 * device buffers that already hold the checkpointed bytes, at any 256-byte
 * aligned address (the tables inside them are rebuilt for the new addresses and
 * uploaded on the stream; moments, codes and accumulators are left as they
 * are).  Either may be NULL if the checkpointed handle had none.  Afterwards
 * the handle continues exactly where the exported one stopped.
 * BAOC_E_INVALID for a foreign, truncated or mismatching blob. */
int baoc_export(const baoc_t* h, void* buf, size_t capacity, size_t* size);
int baoc_import(baoc_t* h, const void* blob, size_t size, void* ws_dev, size_t ws_bytes,
                void* state_dev, size_t state_bytes, baoc_stream_t stream);

/* Per-kernel timing of baoc_step, for benchmarks.  With profiling on, every
 * baoc_step records CUDA events on its stream around the factored row/column
 * kernels and around the fused update kernel (events are created on the first
 * enable; no device memory is involved).  baoc_profile_last waits for the last
 * step and writes ms[0] = row/column kernels (0 when no block is factored),
 * ms[1] = fused update kernel (with a grouped factored schedule the kernels
 * alternate: ms[0] = 0 and ms[1] = the whole step).  BAOC_E_STATE if profiling
 * is off or no step ran. */
int baoc_profile(baoc_t* h, int enable);
int baoc_profile_last(baoc_t* h, float* ms2);

/* ---- checked build ------------------------------------------------------------
 * The paper has no counterpart of this.  The library can be built with
 * -DBAOC_CHECKED (libbaoc_checked.so): every CTA of the streaming kernels of the
 * window and of the step then validates, before it touches memory, that its tile
 * exists, names a block of the table and starts inside it, and that every range
 * of the bound workspace or state buffer it is about to read or write lies inside
 * that buffer.  The first violation is recorded (nothing traps, the CTA returns,
 * the context stays usable).  It is the stand-in for a memory checker where none
 * can be run; caller-owned arrays are covered by guard words in the test harness.
 *
 * baoc_check_status: waits for the device, then writes the first recorded
 * violation since the last call to *out and clears the records.  enabled = 1 in
 * a checked build, 0 in a normal one (where code is always 0).  code: 0 clean,
 * 1 tile index beyond the table, 2 block index beyond the table, 3 tile start
 * outside its block, 4 a range outside the bound buffer (a = which array,
 * b = offset of the range in the buffer, c = its bytes, d = the buffer's
 * bytes), 5 null pointer; kernel: 1 statistics step, 2 its combine, 3 sample
 * gather, 4 first finalize sweep, 5 later sweeps, 6 / 7 row-column reduction of
 * the window / of the step, 8 its combine, 9 fused step, 10 the self-test, 11 the norms of the
 * factored tuple's Adafactor options.
 *
 * baoc_check_selftest: queues a one-thread kernel that runs the range check on
 * numbers that violate it (a 32-byte range that starts 16 bytes before the end
 * of a buffer; no memory is touched), so that a test can see a violation being
 * recorded and the context staying usable.  BAOC_E_STATE in a normal build. */
typedef struct {
    int32_t enabled;
    uint32_t code, kernel;
    int32_t reserved;
    int64_t a, b, c, d;
} baoc_check_t;
int baoc_check_status(baoc_check_t* out);
int baoc_check_selftest(baoc_stream_t stream);

/* ---- allocation-free variant ------------------------------------------------ */

/* Largest block baoc_sample_stats_noalloc accepts (64 Mi elements).  The
 * library image carries 5 doubles of scratch per 4096 elements of this
 * maximum: 640 KB of device memory on every GPU that loads the library, held
 * until the process exits. */
#define BAOC_NOALLOC_MAX_NUMEL 67108864

/* The paper has no counterpart of this entry point; it exists for callers that
 * cannot allocate device memory when they need a block's statistics: code
 * running inside an allocator hook or an out-of-memory callback, a trainer
 * whose caching allocator owns every free byte and must not fall through to
 * cudaMalloc (which synchronises the device and may fail), or a host runtime
 * with no allocator to lend a workspace from.  It needs no handle and no
 * workspace: the per-tile partial sums live in a fixed array inside the
 * library, and the function calls no cudaMalloc, cudaFree or other allocating
 * routine.
 *
 * One gradient observation of ONE block, with the arithmetic of
 * baoc_sample_stats (Eq. 3 and the cosine of Eq. 5):
 *   m <- beta_m m + (1-beta_m) g,  v <- beta_v v + (1-beta_v) g*g,
 *   out4[0] = cos(g, gprev)   with cos(a,b) = <a,b> / (||a|| ||b|| + eps), 0 if not finite,
 *   out4[1] = ||g||^2,  out4[2] = cos(g, m before the update),  out4[3] = ||m before the update||^2,
 *   gprev <- g.
 * grad_bf16 (in), gprev_bf16 (in/out): device, bf16[numel]; m, v (in/out):
 * device, fp32[numel]; all four 16-byte aligned and owned by the caller, who
 * zero-fills gprev, m and v before the first observation (the first cosine is
 * then 0).  out4: device, 4 doubles, written by the second of the two kernels
 * this call queues on the stream; the call does not wait.
 *
 * Errors: BAOC_E_INVALID (null pointer, numel < 1, coefficient outside [0,1)),
 * BAOC_E_ALIGN, BAOC_E_WORKSPACE when numel > BAOC_NOALLOC_MAX_NUMEL (use the
 * handle-based path for larger blocks), BAOC_E_CUDA.  baoc_noalloc_last_error()
 * returns the message of the calling thread's last failure.
 *
 * The first call on each device looks up the device address of the built-in
 * scratch (cudaGetSymbolAddress, with that device current) and keeps it; make
 * that first call before any stream capture begins.  Make it at start-up, as a
 * warm-up on a small block, while allocation is still allowed: the CUDA runtime
 * may load the library's device code lazily, so the first call is also the one
 * that places the scratch array and the two kernels on the device (it can fail
 * with BAOC_E_CUDA when memory is already exhausted); from the second call on a
 * device nothing is loaded or placed any more.  The address that is kept does
 * not survive cudaDeviceReset: a process that resets a device must not call
 * this function on it afterwards.  Every call on a device
 * shares the one scratch array, which keeps the previous call's contents:
 * nothing in it needs clearing, because each call overwrites every slot it
 * later reads, but two calls that overlap on the GPU (different streams, or
 * different host threads) race on it, so serialise them on one stream. */
int baoc_sample_stats_noalloc(const void* grad_bf16, void* gprev_bf16, float* m, float* v, int64_t numel,
                              double beta_m, double beta_v, double eps, double* out4, baoc_stream_t stream);
const char* baoc_noalloc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* BAOC_H */
