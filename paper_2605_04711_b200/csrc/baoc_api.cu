// GPU-facing entry points of the C ABI: workspace binding, the sampling-window
// calls, the end-of-window risk, optimizer instantiation and the fused step.
// Every argument is validated on the host before anything is queued.
#include <cmath>
#include <cstring>
#include <cuda_runtime.h>

#include "baoc_internal.h"

using namespace baoc;

namespace {

int cuda_fail(const Handle* h, const char* what, cudaError_t e) {
    return fail(h, BAOC_E_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}
int launch_fail(const Handle* h, const char* what, int code) {
    return fail(h, BAOC_E_CUDA, std::string(what) + ": " + cudaGetErrorString(cudaError_t(code)));
}

#define CU(call, what)                                        \
    do {                                                      \
        cudaError_t e_ = (call);                              \
        if (e_ != cudaSuccess) return cuda_fail(h, what, e_); \
    } while (0)
#define LAUNCH(call, what)                              \
    do {                                                \
        int r_ = (call);                                \
        if (r_ != 0) return launch_fail(h, what, r_);   \
    } while (0)

// Events and the copy stream a handle may own (created on first use, destroyed with the handle).
void destroy_cuda_objects(Handle* h) {
    for (void*& e : h->prof_ev) {
        if (e) cudaEventDestroy(static_cast<cudaEvent_t>(e));
        e = nullptr;
    }
    for (void*& e : h->copy_ev) {
        if (e) cudaEventDestroy(static_cast<cudaEvent_t>(e));
        e = nullptr;
    }
    if (h->copy_stream) cudaStreamDestroy(static_cast<cudaStream_t>(h->copy_stream));
    h->copy_stream = nullptr;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Check a host array of device pointers; upload it when it differs from the
// copy the device already has.
int sync_pointer_table(Handle* h, const void* const* ptrs, std::vector<const void*>* cache, void* dev_table,
                       cudaStream_t s, const char* what) {
    const int n = h->n_blocks;
    for (int i = 0; i < n; ++i) {
        if (!ptrs[i]) return fail(h, BAOC_E_INVALID, std::string(what) + ": null block pointer");
        if (!aligned16(ptrs[i])) return fail(h, BAOC_E_ALIGN, std::string(what) + ": block pointer not 16-byte aligned");
    }
    if (cache->size() == size_t(n) && std::memcmp(cache->data(), ptrs, sizeof(void*) * n) == 0) return BAOC_OK;
    cache->assign(ptrs, ptrs + n);
    CU(cudaMemcpyAsync(dev_table, cache->data(), sizeof(void*) * n, cudaMemcpyHostToDevice, s), what);
    return BAOC_OK;
}

template <typename T>
T* at(char* base, size_t off) { return reinterpret_cast<T*>(base + off); }

// What a launch over n_tiles tiles (or reduction pieces) may touch: the statistics workspace, or the state buffer.
CheckCtx ws_ctx(const Handle* h, int64_t n_tiles) { return CheckCtx{h->ws, h->ws + h->ws_bytes, (long long)n_tiles, h->n_blocks, 0}; }
CheckCtx st_ctx(const Handle* h, int64_t n_tiles) { return CheckCtx{h->st, h->st + h->st_bytes, (long long)n_tiles, h->n_blocks, 0}; }

// The streaming part of one observation for the blocks [b0, b1): their tiles are contiguous in the tile table.
int stats_step_range(Handle* h, int b0, int b1, cudaStream_t s) {
    const auto& L = h->sl;
    const int64_t t0 = h->h_stat_blocks[b0].tile0;
    const int64_t t1 = b1 < h->n_blocks ? h->h_stat_blocks[b1].tile0 : h->n_stat_tiles;
    if (t1 <= t0) return BAOC_OK;
    if (h->sampled) {
        LAUNCH(launch_sample_gather(at<StatBlock>(h->ws, L.blocks), at<Tile>(h->ws, L.tiles) + t0, at<const void*>(h->ws, L.grads),
                                    t1 - t0, 0, ws_ctx(h, t1 - t0), s), "sample_gather_kernel");
        h->launches += 1;
    }
    LAUNCH(launch_stats_step(at<StatBlock>(h->ws, L.blocks), at<Tile>(h->ws, L.tiles) + t0,
                             at<const void*>(h->ws, h->sampled ? L.sgrads : L.grads),
                             at<double>(h->ws, L.partials) + size_t(t0) * kStatPartials, t1 - t0,
                             float(1.0 - h->opts.beta_m), float(1.0 - h->opts.beta_v), ws_ctx(h, t1 - t0), s), "stats_step_kernel");
    h->launches += 1;
    return BAOC_OK;
}

int stats_combine_all(Handle* h, cudaStream_t s) {
    const auto& L = h->sl;
    LAUNCH(launch_stats_combine(at<StatBlock>(h->ws, L.blocks), at<double>(h->ws, L.partials), at<double>(h->ws, L.acc),
                                h->n_blocks, h->stats_steps > 0 ? 1 : 0, h->opts.beta_rho, h->opts.eps, ws_ctx(h, h->n_stat_tiles), s),
           "stats_combine_kernel");
    h->launches += 1;
    h->stats_steps += 1;
    return BAOC_OK;
}

int do_sample_stats(Handle* h, const void* const* grads, cudaStream_t s) {
    int rc = sync_pointer_table(h, grads, &h->last_stat_grads, h->ws + h->sl.grads, s, "baoc_sample_stats");
    if (rc) return rc;
    rc = stats_step_range(h, 0, h->n_blocks, s);
    if (rc) return rc;
    return stats_combine_all(h, s);
}

void fill_step_params(const Handle* h, int64_t t, StepParams* P) {
    std::memset(P, 0, sizeof(*P));
    for (size_t sl = 0; sl < h->slots.size(); ++sl) {
        const Handle::Slot& slot = h->slots[sl];
        const baoc_config_t& k = h->cfgs[slot.cfg];
        CfgStep& o = P->c[sl];
        const double b1 = double(k.beta1), b2 = double(k.beta2), lr = double(k.lr);
        o.beta1 = k.beta1; o.beta2 = k.beta2; o.eps = k.eps; o.wd = k.weight_decay;
        o.om1 = float(1.0 - b1); o.om2 = float(1.0 - b2);
        const bool has_wd = k.weight_decay != 0.0f;
        o.coupled = (has_wd && !k.decoupled_wd) ? 1 : 0;
        o.decay = (has_wd && k.decoupled_wd) ? -float(lr * double(k.weight_decay)) : 0.0f;
        // each moment counts the gradients it has seen since it last started from zero
        const double tm = double(std::max<int64_t>(1, t - slot.t_m0)), tv = double(std::max<int64_t>(1, t - slot.t_v0));
        double bc2 = 1.0 - std::pow(b2, tv);
        const double bc1 = 1.0 - std::pow(b1, tm);
        o.af_flags = k.factored ? int32_t(k.af_flags) : 0;
        double b2_now = b2;
        if (o.af_flags & kAfSchedule) {                    // Adafactor: beta2_t = 1 - t^-0.8, no bias correction
            b2_now = 1.0 - std::pow(tv, -0.8);
            bc2 = 1.0;
        }
        o.eps1_d = (o.af_flags & kAfEps1) ? 1e-30 : 0.0;
        o.rho_d = std::min(1e-2, 1.0 / std::sqrt(tv));
        o.step_m = float(lr / bc1);
        o.step_g = k.lr;
        o.rsqrt_bc2 = float(1.0 / std::sqrt(bc2));
        o.step_m_hat = float(lr / bc1 * std::sqrt(bc2));
        o.step_g_hat = float(lr * std::sqrt(bc2));
        o.eps_hat = float(double(k.eps) * std::sqrt(bc2));
        o.beta1_d = b1; o.beta2_d = b2_now; o.wd_d = double(k.weight_decay);
    }
}

// Group the blocks into slots by (configuration, moment start steps); writes the slot index into the block records.
int build_slots(Handle* h, const int32_t* assign, std::vector<StepBlock>* sb) {
    h->slots.clear();
    h->slot_of.assign(h->n_blocks, 0);
    for (int i = 0; i < h->n_blocks; ++i) {
        const Handle::Slot want{assign[i], h->t_m0[i], h->t_v0[i]};
        size_t k = 0;
        for (; k < h->slots.size(); ++k)
            if (h->slots[k].cfg == want.cfg && h->slots[k].t_m0 == want.t_m0 && h->slots[k].t_v0 == want.t_v0) break;
        if (k == h->slots.size()) {
            if (k == size_t(kMaxSlots)) return fail(h, BAOC_E_INVALID, "too many distinct (configuration, moment start step) combinations for one step");
            h->slots.push_back(want);
        }
        h->slot_of[i] = int32_t(k);
        (*sb)[i].cfg = int32_t(k);
    }
    return BAOC_OK;
}

// What a step does before its launches: pointer tables, the step's scalars, cleared flags.
int step_prologue(Handle* h, const void* const* grads, float* const* params, int64_t t, cudaStream_t s, StepParams* P) {
    int rc = sync_pointer_table(h, grads, &h->last_step_grads, h->st + h->tl.grads, s, "baoc_step (grads)");
    if (rc) return rc;
    rc = sync_pointer_table(h, reinterpret_cast<const void* const*>(params), &h->last_step_params, h->st + h->tl.params, s,
                            "baoc_step (params)");
    if (rc) return rc;
    fill_step_params(h, t, P);
    CU(cudaMemsetAsync(h->st + h->tl.flags, 0, 4 * size_t(h->n_blocks), s), "baoc_step (flags)");
    return BAOC_OK;
}

// The optimizer step of one copy group: its factored blocks' row/column kernels, then its tiles family by family.
int step_group(Handle* h, const Handle::GroupStep& g, const StepParams& P, cudaStream_t s) {
    const auto& L = h->tl;
    if (g.n_f > 0) {
        LAUNCH(launch_factored_reduce(at<StepBlock>(h->st, L.blocks), at<RedTile>(h->st, L.red_tiles) + g.red0,
                                      at<int32_t>(h->st, L.f_ids) + g.f0, at<const void*>(h->st, L.grads),
                                      at<const float*>(h->st, L.params), g.n_red, g.n_f, P, st_ctx(h, g.n_red), s),
               "factored_reduce_kernel");
        h->launches += 2;
    }
    int64_t first = g.tile0;
    for (int fam = 0; fam < kFamCount; ++fam) {
        if (g.fam_tiles[fam] == 0) continue;
        LAUNCH(launch_fused_step(at<StepBlock>(h->st, L.blocks), at<Tile>(h->st, L.tiles_by_group) + first,
                                 at<const void*>(h->st, L.grads), at<float*>(h->st, L.params), at<uint32_t>(h->st, L.flags),
                                 g.fam_tiles[fam], fam, P, st_ctx(h, g.fam_tiles[fam]), s),
               "fused_step_kernel");
        h->launches += 1;
        first += g.fam_tiles[fam];
    }
    return BAOC_OK;
}

// The launches of one step of every block, after the prologue: the whole tile table, one launch per path family present.
int step_launches(Handle* h, const StepParams& P, cudaStream_t s) {
    const auto& L = h->tl;
    const bool grouped = h->factored_group_bytes > 0 && h->n_factored > 0 && h->n_fa == 0;   // blocks with Adafactor's options keep the one-reduction schedule
    if (h->prof_on) CU(cudaEventRecord(static_cast<cudaEvent_t>(h->prof_ev[0]), s), "baoc_step (profile)");
    if (h->n_factored > 0 && !grouped) {
        LAUNCH(launch_factored_reduce(at<StepBlock>(h->st, L.blocks), at<RedTile>(h->st, L.red_tiles),
                                      at<int32_t>(h->st, L.f_ids), at<const void*>(h->st, L.grads),
                                      at<const float*>(h->st, L.params), h->n_step_red_tiles, h->n_factored, P,
                                      st_ctx(h, h->n_step_red_tiles), s),
               "factored_reduce_kernel");
        h->launches += 2;
        if (h->n_fa > 0) {
            LAUNCH(launch_factored_norms(at<StepBlock>(h->st, L.blocks), at<Tile>(h->st, L.tiles) + h->fa_tile0,
                                         at<int32_t>(h->st, L.f_ids) + h->n_factored, at<const void*>(h->st, L.grads),
                                         at<const float*>(h->st, L.params), h->n_fa_tiles, h->n_fa, P, st_ctx(h, h->n_fa_tiles), s),
                   "factored_norms_kernel");
            h->launches += 2;
        }
    }
    if (h->prof_on) CU(cudaEventRecord(static_cast<cudaEvent_t>(h->prof_ev[1]), s), "baoc_step (profile)");
    int64_t first = 0;
    for (int fam = 0; fam < kFamCount; ++fam) {
        if (h->fam_tiles[fam] == 0) continue;
        // grouped schedule: the headline family's launch stops before the factored tiles, which close its stretch
        const int64_t here = (grouped && fam == kFamHead) ? h->fam_tiles[fam] - h->n_factored_tiles : h->fam_tiles[fam];
        if (here > 0) {
            LAUNCH(launch_fused_step(at<StepBlock>(h->st, L.blocks), at<Tile>(h->st, L.tiles) + first, at<const void*>(h->st, L.grads),
                                     at<float*>(h->st, L.params), at<uint32_t>(h->st, L.flags), here, fam, P, st_ctx(h, here), s),
                   "fused_step_kernel");
            h->launches += 1;
        }
        if (grouped && fam == kFamHead) {
            // every group: row/column reduction, its combine, then the group's update tiles, back to back
            const int64_t f_first = first + here;
            for (const Handle::FactoredGroup& g : h->f_groups) {
                LAUNCH(launch_factored_reduce(at<StepBlock>(h->st, L.blocks), at<RedTile>(h->st, L.red_tiles) + g.red0,
                                              at<int32_t>(h->st, L.f_ids) + g.f0, at<const void*>(h->st, L.grads),
                                              at<const float*>(h->st, L.params), g.n_red, g.n_f, P, st_ctx(h, g.n_red), s),
                       "factored_reduce_kernel");
                LAUNCH(launch_fused_step(at<StepBlock>(h->st, L.blocks), at<Tile>(h->st, L.tiles) + f_first + g.tile0,
                                         at<const void*>(h->st, L.grads), at<float*>(h->st, L.params),
                                         at<uint32_t>(h->st, L.flags), g.n_tiles, kFamHead, P, st_ctx(h, g.n_tiles), s),
                       "fused_step_kernel");
                h->launches += 3;
            }
        }
        first += h->fam_tiles[fam];
    }
    if (h->prof_on) {
        CU(cudaEventRecord(static_cast<cudaEvent_t>(h->prof_ev[2]), s), "baoc_step (profile)");
        h->prof_valid = true;
    }
    return BAOC_OK;
}

int do_step(Handle* h, const void* const* grads, float* const* params, int64_t t, cudaStream_t s) {
    StepParams P;
    int rc = step_prologue(h, grads, params, t, s, &P);
    if (rc) return rc;
    return step_launches(h, P, s);
}

}  // namespace

extern "C" {

int baoc_stats_workspace_bytes(const baoc_t* h, size_t* bytes) {
    if (!h || !bytes) return BAOC_E_INVALID;
    *bytes = h->sl.total;
    return BAOC_OK;
}

static int bind_stats(baoc_t* h, void* dev, size_t bytes, baoc_stream_t stream, bool reset) {
    if (!h) return BAOC_E_INVALID;
    if (!dev) return fail(h, BAOC_E_INVALID, "baoc_bind_stats_workspace: null workspace");
    if (reinterpret_cast<uintptr_t>(dev) & 255u) return fail(h, BAOC_E_ALIGN, "baoc_bind_stats_workspace: workspace not 256-byte aligned");
    if (bytes < h->sl.total) return fail(h, BAOC_E_WORKSPACE, "baoc_bind_stats_workspace: workspace too small");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const auto& L = h->sl;
    char* ws = static_cast<char*>(dev);
    const int n = h->n_blocks;

    std::vector<StatBlock> sb = h->h_stat_blocks;
    std::vector<Tile> tiles;
    std::vector<RedTile> red;
    std::vector<int32_t> ids;
    tiles.reserve(size_t(h->n_stat_tiles));
    for (int i = 0; i < n; ++i) {
        StatBlock& b = sb[i];
        b.m = reinterpret_cast<float*>(ws + L.m + reinterpret_cast<size_t>(b.m));
        b.v = reinterpret_cast<float*>(ws + L.v + reinterpret_cast<size_t>(b.v));
        b.gprev = reinterpret_cast<uint16_t*>(ws + L.gprev + reinterpret_cast<size_t>(b.gprev));
        if (h->sampled) {
            b.ridx = reinterpret_cast<const int64_t*>(ws + L.ridx + reinterpret_cast<size_t>(b.ridx));
            b.cidx = reinterpret_cast<const int32_t*>(ws + L.cidx + reinterpret_cast<size_t>(b.cidx));
            b.gsample = reinterpret_cast<uint16_t*>(ws + L.gsample + reinterpret_cast<size_t>(b.gsample));
            b.psample = reinterpret_cast<float*>(ws + L.psample + reinterpret_cast<size_t>(b.psample));
        }
        for (int k = 0; k < b.ntiles; ++k) tiles.push_back(Tile{uint32_t(i), uint32_t(k)});
        if (b.cols > 1) {
            b.rowsum = reinterpret_cast<double*>(ws + L.rowsum + reinterpret_cast<size_t>(b.rowsum));
            b.colsum = reinterpret_cast<double*>(ws + L.colsum + reinterpret_cast<size_t>(b.colsum));
            b.red.rowpart = reinterpret_cast<double*>(ws + L.redpart + reinterpret_cast<size_t>(b.red.rowpart));
            b.red.colpart = reinterpret_cast<double*>(ws + L.redpart + reinterpret_cast<size_t>(b.red.colpart));
            for (int ch = 0; ch < b.red.chunks; ++ch)
                for (int st = 0; st < b.red.strips; ++st) red.push_back(RedTile{uint32_t(i), uint32_t(ch), uint32_t(st), 0});
            ids.push_back(i);
        }
    }
    h->n_matrix = int(ids.size());
    std::vector<SelPiece> pieces;
    uint64_t surv_words = 0;
    build_sel_pieces(h, &pieces, &sb, &surv_words);
    if (h->sampled) {
        // index lists and the tables of sample-buffer pointers (the host vectors outlive the copies: they belong to the handle)
        h->sample_tables.clear();
        std::vector<int64_t>& ri = h->flat_ridx; std::vector<int32_t>& ci = h->flat_cidx;
        ri.clear(); ci.clear();
        for (int i = 0; i < n; ++i) {
            ri.insert(ri.end(), h->s_rows[i].begin(), h->s_rows[i].end());
            ci.insert(ci.end(), h->s_cols[i].begin(), h->s_cols[i].end());
            h->sample_tables.push_back(sb[i].gsample);
        }
        for (int i = 0; i < n; ++i) h->sample_tables.push_back(sb[i].psample);
        CU(cudaMemcpyAsync(ws + L.ridx, ri.data(), 8 * ri.size(), cudaMemcpyHostToDevice, s), "upload sample rows");
        CU(cudaMemcpyAsync(ws + L.cidx, ci.data(), 4 * ci.size(), cudaMemcpyHostToDevice, s), "upload sample columns");
        CU(cudaMemcpyAsync(ws + L.sgrads, h->sample_tables.data(), 8 * size_t(n), cudaMemcpyHostToDevice, s), "upload sample gradient table");
        CU(cudaMemcpyAsync(ws + L.sparams, h->sample_tables.data() + n, 8 * size_t(n), cudaMemcpyHostToDevice, s), "upload sample parameter table");
    }
    CU(cudaMemcpyAsync(ws + L.blocks, sb.data(), sizeof(StatBlock) * n, cudaMemcpyHostToDevice, s), "upload block table");
    CU(cudaMemcpyAsync(ws + L.tiles, tiles.data(), sizeof(Tile) * tiles.size(), cudaMemcpyHostToDevice, s), "upload tile table");
    CU(cudaMemcpyAsync(ws + L.pieces, pieces.data(), sizeof(SelPiece) * pieces.size(), cudaMemcpyHostToDevice, s), "upload piece table");
    if (!red.empty())
        CU(cudaMemcpyAsync(ws + L.red_tiles, red.data(), sizeof(RedTile) * red.size(), cudaMemcpyHostToDevice, s), "upload reduction table");
    if (!ids.empty())
        CU(cudaMemcpyAsync(ws + L.matrix_ids, ids.data(), 4 * ids.size(), cudaMemcpyHostToDevice, s), "upload matrix ids");
    // moments, previous gradient and running values start at zero
    if (reset) {
        CU(cudaMemsetAsync(ws + L.m, 0, L.partials - L.m, s), "zero moments");
        CU(cudaMemsetAsync(ws + L.acc, 0, 8 * size_t(kBlockAcc) * n, s), "zero accumulators");
    }
    h->ws = ws; h->ws_bytes = bytes; h->ws_bound = true;
    if (reset) h->stats_steps = 0;
    h->last_stat_grads.clear(); h->last_stat_params.clear();
    return BAOC_OK;
}

int baoc_bind_stats_workspace(baoc_t* h, void* dev, size_t bytes, baoc_stream_t stream) {
    return bind_stats(h, dev, bytes, stream, true);
}

int baoc_sample_stats(baoc_t* h, const void* const* grads, baoc_stream_t stream) {
    if (!h) return BAOC_E_INVALID;
    if (!grads) return fail(h, BAOC_E_INVALID, "baoc_sample_stats: null gradient table");
    if (!h->ws_bound) return fail(h, BAOC_E_STATE, "baoc_sample_stats: no statistics workspace bound");
    return do_sample_stats(h, grads, static_cast<cudaStream_t>(stream));
}

int baoc_read_stats(baoc_t* h, baoc_block_stats_t* out, baoc_stream_t stream) {
    if (!h) return BAOC_E_INVALID;
    if (!out) return fail(h, BAOC_E_INVALID, "baoc_read_stats: null output");
    if (!h->ws_bound) return fail(h, BAOC_E_STATE, "baoc_read_stats: no statistics workspace bound");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<double> acc(size_t(kBlockAcc) * h->n_blocks);
    CU(cudaMemcpyAsync(acc.data(), h->ws + h->sl.acc, 8 * acc.size(), cudaMemcpyDeviceToHost, s), "baoc_read_stats");
    CU(cudaStreamSynchronize(s), "baoc_read_stats");
    for (int i = 0; i < h->n_blocks; ++i) {
        std::memset(&out[i], 0, sizeof(out[i]));
        const double* a = &acc[size_t(i) * kBlockAcc];
        out[i].rho_bar = a[0]; out[i].n_cos = int64_t(a[1]); out[i].last_cos = a[3]; out[i].rho_mom = a[4];
    }
    return BAOC_OK;
}

int baoc_risk(baoc_t* h, const float* const* params, double* risk_out, baoc_block_stats_t* stats_out, baoc_stream_t stream) {
    if (!h) return BAOC_E_INVALID;
    if (!params || !risk_out) return fail(h, BAOC_E_INVALID, "baoc_risk: null argument");
    if (!h->ws_bound) return fail(h, BAOC_E_STATE, "baoc_risk: no statistics workspace bound");
    if (h->stats_steps <= 0) return fail(h, BAOC_E_STATE, "baoc_risk: no gradient has been observed in this window");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int n = h->n_blocks;
    int rc = sync_pointer_table(h, reinterpret_cast<const void* const*>(params), &h->last_stat_params, h->ws + h->sl.params, s, "baoc_risk (params)");
    if (rc) return rc;
    const auto& L = h->sl;
    char* ws = h->ws;
    const StatBlock* blocks = at<StatBlock>(ws, L.blocks);
    const Tile* tiles = at<Tile>(ws, L.tiles);
    const float* const* dparams = at<const float*>(ws, h->sampled ? L.sparams : L.params);
    if (h->sampled) {
        LAUNCH(launch_sample_gather(blocks, tiles, at<const void*>(ws, L.params), h->n_stat_tiles, 1, ws_ctx(h, h->n_stat_tiles), s),
               "sample_gather_kernel");
        h->launches += 1;
    }
    // The alternative reading of the hats in Eq. 3: Adam's bias correction for the steps observed.  A positive factor per
    // moment: the first sweep applies it as it loads m and v; the order statistics and the Eq. 7 residual, which are
    // taken from v as stored, are scaled on the host.
    const double m_scale = h->opts.debias ? 1.0 / (1.0 - std::pow(h->opts.beta_m, double(h->stats_steps))) : 1.0;
    const double v_scale = h->opts.debias ? 1.0 / (1.0 - std::pow(h->opts.beta_v, double(h->stats_steps))) : 1.0;
    LAUNCH(launch_final_sums(blocks, tiles, dparams, at<double>(ws, L.fin), at<double>(ws, L.fin_out), at<uint32_t>(ws, L.hist),
                             at<RankSel>(ws, L.sel), at<SelKey>(ws, L.selkey), h->n_stat_tiles, n, h->opts.eps, float(h->opts.eps_adam),
                             h->opts.quantizer8, h->opts.debias, float(m_scale), float(v_scale), ws_ctx(h, h->n_stat_tiles), s),
           "final_sums_kernel");
    h->launches += 5;
    if (h->n_matrix > 0) {
        LAUNCH(launch_moment_reduce(blocks, at<RedTile>(ws, L.red_tiles), at<int32_t>(ws, L.matrix_ids), h->n_red_tiles,
                                    h->n_matrix, ws_ctx(h, h->n_red_tiles), s), "moment_reduce_kernel");
        h->launches += 3;
    }
    SelectArgs sa{blocks, tiles, at<SelPiece>(ws, L.pieces), at<RankSel>(ws, L.sel), at<SelKey>(ws, L.selkey),
                  at<uint32_t>(ws, L.hist), at<uint32_t>(ws, L.surv), at<uint32_t>(ws, L.surv_cnt), at<double>(ws, L.resid_part),
                  at<double>(ws, L.fin_out), at<double>(ws, L.acc), h->n_stat_tiles, h->n_sel_pieces, n};
    LAUNCH(launch_final_resid_select(sa, ws_ctx(h, h->n_sel_pieces), s), "final_resid_hist_kernel");
    h->launches += 6;

    std::vector<double> out(size_t(kFinOut) * n);
    CU(cudaMemcpyAsync(out.data(), ws + L.fin_out, 8 * out.size(), cudaMemcpyDeviceToHost, s), "baoc_risk (copy back)");
    CU(cudaStreamSynchronize(s), "baoc_risk (wait)");
    // The select orders each block by a key fitted to a sample of it.  A block whose order statistic came out at an end
    // of that key range holds elements outside the sample's range there: it is selected again over the full range.
    h->select_retries = 0;
    h->selkey_staging.assign(size_t(n), SelKey{0, -1});
    for (int i = 0; i < n; ++i)
        if (out[size_t(i) * kFinOut + kFinFlag] != 0.0) { h->selkey_staging[i] = SelKey{-1, kSelFullS}; ++h->select_retries; }
    if (h->select_retries > 0) {
        CU(cudaMemcpyAsync(ws + L.selkey, h->selkey_staging.data(), sizeof(SelKey) * size_t(n), cudaMemcpyHostToDevice, s),
           "baoc_risk (select keys)");
        LAUNCH(launch_select_again(sa, ws_ctx(h, h->n_sel_pieces), s), "select_first_kernel");
        h->launches += 8;
        CU(cudaMemcpyAsync(out.data(), ws + L.fin_out, 8 * out.size(), cudaMemcpyDeviceToHost, s), "baoc_risk (copy back)");
        CU(cudaStreamSynchronize(s), "baoc_risk (wait)");
    }

    std::vector<baoc_block_stats_t> tmp;
    baoc_block_stats_t* st = stats_out;
    if (!st) { tmp.resize(n); st = tmp.data(); }
    const double eps = h->opts.eps;
    auto cosine = [&](double dot, double na2, double nb2) {
        const double c = dot / (std::sqrt(na2) * std::sqrt(nb2) + eps);
        return std::isfinite(c) ? c : 0.0;
    };
    auto rel = [](double err2, double ref2) { return ref2 > 0.0 ? std::sqrt(err2) / std::sqrt(ref2) : 0.0; };
    for (int i = 0; i < n; ++i) {
        const double* o = &out[size_t(i) * kFinOut];
        const baoc_block_t& b = h->stat_shapes[i];           // the block, or its sample
        baoc_block_stats_t& z = st[i];
        std::memset(&z, 0, sizeof(z));
        // Eq. 4: quantiles by linear interpolation at position q (n - 1)
        const double qs[2] = {0.1, 0.9};
        double qv[2];
        for (int k = 0; k < 2; ++k) {
            const double pos = qs[k] * double(b.numel - 1);
            const double frac = pos - std::floor(pos);
            const double lo = o[kFinRanks + 2 * k] * v_scale, hi = o[kFinRanks + 2 * k + 1] * v_scale;   // the select ran on v as stored
            qv[k] = lo + frac * (hi - lo);
        }
        z.q10 = qv[0]; z.q90 = qv[1];
        z.A = std::log((qv[1] + eps) / (qv[0] + eps));
        z.rho_bar = o[kFinAcc]; z.n_cos = int64_t(o[kFinAcc + 1]); z.last_cos = o[kFinAcc + 3]; z.rho_mom = o[kFinAcc + 4];
        z.snr = o[0] / (o[1] + eps);                                        // Eq. 5 right
        {   // Eq. 6 from the sums of the deviations d = p - p0 from the pilot value: with delta = pbar - p0,
            // sum ((p / pbar - 1) theta)^2 = (sum d^2 theta^2 - 2 delta sum d theta^2 + delta^2 sum theta^2) / pbar^2
            const double delta = o[3] / double(b.numel), pbar = o[kFinPilot] + delta;
            const double num2 = std::max(0.0, o[15] - 2.0 * delta * o[14] + delta * delta * o[4]);
            z.C = pbar > 0.0 ? (std::sqrt(num2) / pbar) / (std::sqrt(o[4]) + eps) : 0.0;
        }
        z.F = b.cols > 1 ? (std::sqrt(o[kFinResid]) * v_scale) / (std::sqrt(o[2]) + eps) : 1.0;   // Eq. 7 (the residual sweep ran on v as stored)
        z.Q32 = cosine(o[5], o[5], o[5]);                                   // Eq. 8
        z.Q16 = cosine(o[9], o[5], o[8]);
        z.Q8 = cosine(o[7], o[5], o[6]);
        z.err_m8 = rel(o[10], o[0]); z.err_v8 = rel(o[11], o[2]);
        z.err_m16 = rel(o[12], o[0]); z.err_v16 = rel(o[13], o[2]);
    }
    return baoc_risk_from_raw(h, st, risk_out);
}

int baoc_state_bytes(const baoc_t* h, const int32_t* assign, size_t* bytes) {
    if (!h) return BAOC_E_INVALID;
    if (!assign || !bytes) return fail(h, BAOC_E_INVALID, "baoc_state_bytes: null argument");
    Handle::StepLayout L{};
    int rc = compute_step_layout(h, assign, &L, nullptr, nullptr, nullptr, nullptr, nullptr);
    if (rc) return rc;
    *bytes = L.total;
    return BAOC_OK;
}

// reset: zero the state and restart every moment's step count;  zero_only: zero the state, keep the counts the
// caller has just set (re-configuration);  neither: leave both alone (resume from a checkpoint).
static int configure_state(baoc_t* h, const int32_t* assign, void* state_dev, size_t bytes, baoc_stream_t stream, bool reset,
                           bool zero_only = false) {
    if (!h) return BAOC_E_INVALID;
    if (!assign || !state_dev) return fail(h, BAOC_E_INVALID, "baoc_configure: null argument");
    if (reinterpret_cast<uintptr_t>(state_dev) & 255u) return fail(h, BAOC_E_ALIGN, "baoc_configure: state buffer not 256-byte aligned");
    Handle::StepLayout L{};
    std::vector<StepBlock> sb;
    std::vector<Tile> tiles;
    std::vector<RedTile> red;
    int64_t mem = 0, traffic = 0;
    int rc = compute_step_layout(h, assign, &L, &sb, &tiles, &red, &mem, &traffic);
    if (rc) return rc;
    if (bytes < L.total) return fail(h, BAOC_E_WORKSPACE, "baoc_configure: state buffer too small");
    if (reset || h->t_m0.size() != size_t(h->n_blocks)) { h->t_m0.assign(h->n_blocks, 0); h->t_v0.assign(h->n_blocks, 0); }
    rc = build_slots(h, assign, &sb);
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* st = static_cast<char*>(state_dev);
    const int n = h->n_blocks;
    std::vector<int32_t> ids;
    for (int i = 0; i < n; ++i) {
        StepBlock& b = sb[i];
        auto fix = [&](void* p) { return static_cast<void*>(st + L.states + reinterpret_cast<size_t>(p)); };
        auto fix_scratch = [&](void* p) { return static_cast<void*>(st + L.redpart + reinterpret_cast<size_t>(p)); };
        if (is_factored_path(b.path) && b.fbits != 32) {
            b.s0 = fix_scratch(b.s0); b.s1 = fix_scratch(b.s1);
            b.f0 = fix(b.f0); b.f1 = fix(b.f1);
            if (b.fbits == 8) { b.fa0 = static_cast<float*>(fix(b.fa0)); b.fa1 = static_cast<float*>(fix(b.fa1)); }
        } else if (b.path == kPathA32 || b.path == kPathA8 || b.path == kPathA8N || is_factored_path(b.path) || b.path == kPathA16) { b.s0 = fix(b.s0); b.s1 = fix(b.s1); }
        else if (b.path == kPathR8) { b.s1 = fix(b.s1); b.a1 = static_cast<float*>(fix(b.a1)); }
        else if (b.path == kPathS8) { b.s0 = fix(b.s0); b.a0 = static_cast<float*>(fix(b.a0)); }
        else if (b.path != kPathG) b.s0 = fix(b.s0);
        if (b.path == kPathA8 || b.path == kPathA8N) { b.a0 = static_cast<float*>(fix(b.a0)); b.a1 = static_cast<float*>(fix(b.a1)); }
        if (b.path == kPathFA) b.norm_part = reinterpret_cast<double*>(st + L.redpart + reinterpret_cast<size_t>(b.norm_part));
        if (is_factored_path(b.path)) {
            b.a0 = static_cast<float*>(fix(b.a0));
            b.red.rowpart = reinterpret_cast<double*>(st + L.redpart + reinterpret_cast<size_t>(b.red.rowpart));
            b.red.colpart = reinterpret_cast<double*>(st + L.redpart + reinterpret_cast<size_t>(b.red.colpart));
            b.mean_part = reinterpret_cast<double*>(st + L.redpart + reinterpret_cast<size_t>(b.mean_part));
            ids.push_back(i);
        }
    }
    CU(cudaMemcpyAsync(st + L.blocks, sb.data(), sizeof(StepBlock) * n, cudaMemcpyHostToDevice, s), "upload step block table");
    CU(cudaMemcpyAsync(st + L.tiles, tiles.data(), sizeof(Tile) * tiles.size(), cudaMemcpyHostToDevice, s), "upload step tile table");
    // the same tiles group by group (copy groups of the end-to-end call), within a group family by family in path order
    std::vector<Handle::GroupStep> groups;
    h->group_tiles.clear();
    {
        std::vector<int> gb0, gb1;
        compute_copy_groups(h, &gb0, &gb1);
        int32_t f_seen = 0;
        for (size_t g = 0; g < gb0.size(); ++g) {
            Handle::GroupStep gs{};
            gs.b0 = gb0[g]; gs.b1 = gb1[g];
            gs.tile0 = int64_t(h->group_tiles.size());
            for (int p : kPathOrder)
                for (int i = gs.b0; i < gs.b1; ++i)
                    if (sb[i].path == p) {
                        const int64_t nt = ceil_div(sb[i].numel, step_tile_elems(p));
                        for (int64_t k = 0; k < nt; ++k) h->group_tiles.push_back(Tile{uint32_t(i), uint32_t(k)});
                        gs.fam_tiles[family_of(p)] += nt;
                    }
            gs.red0 = -1; gs.f0 = f_seen;
            for (int i = gs.b0; i < gs.b1; ++i)
                if (is_factored_path(sb[i].path)) {
                    if (gs.red0 < 0) gs.red0 = sb[i].red.red0;
                    gs.n_red += int64_t(sb[i].red.chunks) * sb[i].red.strips;
                    gs.n_f += 1;
                }
            if (gs.red0 < 0) gs.red0 = 0;
            f_seen += gs.n_f;
            groups.push_back(gs);
        }
    }
    CU(cudaMemcpyAsync(st + L.tiles_by_group, h->group_tiles.data(), sizeof(Tile) * h->group_tiles.size(), cudaMemcpyHostToDevice, s),
       "upload step tile table (by group)");
    if (!red.empty())
        CU(cudaMemcpyAsync(st + L.red_tiles, red.data(), sizeof(RedTile) * red.size(), cudaMemcpyHostToDevice, s), "upload step reduction table");
    // behind the factored blocks' ids: those with Adafactor's options (their tiles close the tile table)
    const size_t n_all_f = ids.size();
    int64_t fa_tiles = 0;
    for (int i = 0; i < n; ++i)
        if (sb[i].path == kPathFA) { ids.push_back(i); fa_tiles += ceil_div(sb[i].numel, kTileF); }
    h->n_fa = int(ids.size() - n_all_f);
    h->n_fa_tiles = fa_tiles;
    h->fa_tile0 = int64_t(tiles.size()) - fa_tiles;
    h->f_id_staging = ids;
    if (!ids.empty())
        CU(cudaMemcpyAsync(st + L.f_ids, h->f_id_staging.data(), 4 * ids.size(), cudaMemcpyHostToDevice, s), "upload factored ids");
    ids.resize(n_all_f);
    if (reset || zero_only) CU(cudaMemsetAsync(st + L.flags, 0, L.total - L.flags, s), "zero optimizer state");
    {   // factored blocks in index order: that is their order in the tile table, the reduction table and the id list
        h->f_groups.clear();
        h->n_factored_tiles = 0;
        Handle::FactoredGroup g{0, 0, 0, 0, 0, 0};
        int64_t bytes_in_group = 0;
        for (int i = 0; i < n; ++i) {
            if (!is_factored_path(sb[i].path)) continue;
            const int64_t gb = 2 * sb[i].numel, nt = ceil_div(sb[i].numel, kTileF), nr = int64_t(sb[i].red.chunks) * sb[i].red.strips;
            if (g.n_f > 0 && bytes_in_group + gb > h->factored_group_bytes) {
                h->f_groups.push_back(g);
                g = Handle::FactoredGroup{g.tile0 + g.n_tiles, 0, g.red0 + g.n_red, 0, g.f0 + g.n_f, 0};
                bytes_in_group = 0;
            }
            g.n_tiles += nt; g.n_red += nr; g.n_f += 1;
            bytes_in_group += gb;
            h->n_factored_tiles += nt;
        }
        if (g.n_f > 0) h->f_groups.push_back(g);
    }
    h->st = st; h->st_bytes = bytes; h->tl = L; h->configured = true;
    h->assign.assign(assign, assign + n);
    h->h_step_blocks = sb;
    h->groups = groups;
    h->n_step_tiles = int64_t(tiles.size()); h->n_step_red_tiles = int64_t(red.size());
    h->n_factored = int(ids.size());
    for (int64_t& c : h->fam_tiles) c = 0;
    for (const StepBlock& b : sb) h->fam_tiles[family_of(b.path)] += ceil_div(b.numel, step_tile_elems(b.path));
    h->state_mem = mem; h->step_bytes = traffic;
    h->last_step_grads.clear(); h->last_step_params.clear();
    return BAOC_OK;
}

int baoc_configure(baoc_t* h, const int32_t* assign, void* state_dev, size_t bytes, baoc_stream_t stream) {
    return configure_state(h, assign, state_dev, bytes, stream, true);
}

// ---- online re-configuration with state inheritance ----------------------------------
namespace {
// Which family a path's first moment belongs to (1: Adam-type average, 2: momentum buffer, 0: none).
int m_family(int path) {
    switch (path) {
        case kPathA32: case kPathA16: case kPathA8: return 1;
        case kPathS: case kPathS16: case kPathS8: return 2;
        default: return 0;
    }
}
MomentRef first_moment(const StepBlock& b) {
    MomentRef r{};
    r.rows = b.rows; r.cols = b.cols;
    switch (b.path) {
        case kPathA32: case kPathS: r.data = b.s0; r.kind = kMomF32; break;
        case kPathA16: case kPathS16: r.data = b.s0; r.kind = kMomBF16; break;
        case kPathA8: case kPathS8: r.data = b.s0; r.absmax = b.a0; r.kind = kMomI8; break;
        default: r.kind = kMomNone; break;
    }
    return r;
}
MomentRef second_moment(const StepBlock& b) {
    MomentRef r{};
    r.rows = b.rows; r.cols = b.cols;
    switch (b.path) {
        case kPathA32: r.data = b.s1; r.kind = kMomF32; break;
        case kPathA16: r.data = b.s1; r.kind = kMomBF16; break;
        case kPathA8: case kPathR8: r.data = b.s1; r.absmax = b.a1; r.kind = kMomU8; break;
        case kPathR: r.data = b.s0; r.kind = kMomF32; break;
        case kPathR16: r.data = b.s0; r.kind = kMomBF16; break;
        case kPathF: case kPathFA:
            r.kind = kMomFactored; r.fbits = b.fbits;
            r.wr = static_cast<float*>(b.s0); r.wc = static_cast<float*>(b.s1);
            if (b.fbits == 32) { r.r = b.s0; r.c = b.s1; }
            else { r.r = b.f0; r.c = b.f1; r.ar = b.fa0; r.ac = b.fa1; }
            break;
        default: r.kind = kMomNone; break;
    }
    return r;
}
}  // namespace

int baoc_reconfigure(baoc_t* h, const int32_t* new_assign, void* new_state_dev, size_t bytes, int64_t steps_done,
                     int inherit, baoc_stream_t stream) {
    if (!h) return BAOC_E_INVALID;
    if (!new_assign || !new_state_dev) return fail(h, BAOC_E_INVALID, "baoc_reconfigure: null argument");
    if (!h->configured) return fail(h, BAOC_E_STATE, "baoc_reconfigure: no assignment configured yet");
    if (steps_done < 0) return fail(h, BAOC_E_INVALID, "baoc_reconfigure: negative step count");
    {   // the new buffer must not overlap the old one: the old state is read while the new one is written
        const char* a = h->st; const char* b = static_cast<const char*>(new_state_dev);
        if (b < a + h->tl.total && a < b + bytes) return fail(h, BAOC_E_INVALID, "baoc_reconfigure: the new state buffer overlaps the current one");
    }
    const int n = h->n_blocks;
    const std::vector<StepBlock> old_blocks = h->h_step_blocks;
    const std::vector<int64_t> old_tm = h->t_m0, old_tv = h->t_v0;
    // which moments are inherited, and from there the start steps of the new moments
    std::vector<char> keep_m(n, 0), keep_v(n, 0);
    for (int i = 0; i < n; ++i) {
        if (new_assign[i] < 0 || new_assign[i] >= h->n_cfg) return fail(h, BAOC_E_INVALID, "baoc_reconfigure: assignment names a configuration that does not exist");
        const Path pn = path_of(h->cfgs[new_assign[i]]);
        const int po = old_blocks[i].path;
        keep_m[i] = inherit && m_family(pn) != 0 && m_family(pn) == m_family(po);
        keep_v[i] = inherit && second_moment(old_blocks[i]).kind != kMomNone &&
                    (pn == kPathA32 || pn == kPathA16 || pn == kPathA8 || pn == kPathR || pn == kPathR16 || pn == kPathR8 || is_factored_path(pn));
        h->t_m0[i] = keep_m[i] ? old_tm[i] : steps_done;
        h->t_v0[i] = keep_v[i] ? old_tv[i] : steps_done;
    }
    int rc = configure_state(h, new_assign, new_state_dev, bytes, stream, false, true);
    if (rc) { h->t_m0 = old_tm; h->t_v0 = old_tv; return rc; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (int i = 0; i < n; ++i) {
        const StepBlock& nb = h->h_step_blocks[i];
        if (keep_m[i]) {
            LAUNCH(launch_convert_moment(first_moment(old_blocks[i]), first_moment(nb), nb.numel, s), "convert_moment_kernel");
            h->launches += 1;
        }
        if (keep_v[i]) {
            LAUNCH(launch_convert_moment(second_moment(old_blocks[i]), second_moment(nb), nb.numel, s), "convert_moment_kernel");
            h->launches += 1;
        }
    }
    return BAOC_OK;
}

// ---- hand-over from the sampling window with its moments ------------------------------
int baoc_configure_from_window(baoc_t* h, const int32_t* assign, void* state_dev, size_t bytes, baoc_stream_t stream) {
    if (!h) return BAOC_E_INVALID;
    if (!assign || !state_dev) return fail(h, BAOC_E_INVALID, "baoc_configure_from_window: null argument");
    if (!h->ws_bound || h->stats_steps < 1) return fail(h, BAOC_E_STATE, "baoc_configure_from_window: the window holds no observation");
    if (h->sampled) return fail(h, BAOC_E_STATE, "baoc_configure_from_window: the window saw a sampled sub-grid, not every coordinate");
    {
        const char* a = h->ws; const char* b = static_cast<const char*>(state_dev);
        if (b < a + h->ws_bytes && a < b + bytes) return fail(h, BAOC_E_INVALID, "baoc_configure_from_window: the state buffer overlaps the statistics workspace");
    }
    const int n = h->n_blocks;
    const float bm = float(h->opts.beta_m), bv = float(h->opts.beta_v);
    std::vector<char> keep_m(n, 0), keep_v(n, 0);
    std::vector<int64_t> tm(n, 0), tv(n, 0);
    for (int i = 0; i < n; ++i) {
        if (assign[i] < 0 || assign[i] >= h->n_cfg) return fail(h, BAOC_E_INVALID, "baoc_configure_from_window: assignment names a configuration that does not exist");
        const baoc_config_t& c = h->cfgs[assign[i]];
        const Path p = path_of(c);
        keep_m[i] = m_family(p) != 0 && c.beta1 == bm;
        keep_v[i] = (p == kPathA32 || p == kPathA16 || p == kPathA8 || p == kPathR || p == kPathR16 || p == kPathR8 || is_factored_path(p)) &&
                    c.beta2 == bv && !(c.af_flags & kAfSchedule);
        tm[i] = keep_m[i] ? -h->stats_steps : 0;
        tv[i] = keep_v[i] ? -h->stats_steps : 0;
    }
    const std::vector<int64_t> old_tm = h->t_m0, old_tv = h->t_v0;
    h->t_m0 = tm; h->t_v0 = tv;
    int rc = configure_state(h, assign, state_dev, bytes, stream, false, true);
    if (rc) { h->t_m0 = old_tm; h->t_v0 = old_tv; return rc; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (int i = 0; i < n; ++i) {
        const StepBlock& nb = h->h_step_blocks[i];
        const StatBlock& wb = h->h_stat_blocks[i];
        MomentRef src{};
        src.rows = nb.rows; src.cols = nb.cols; src.kind = kMomF32;
        if (keep_m[i]) {
            src.data = h->ws + h->sl.m + reinterpret_cast<size_t>(wb.m);        // the handle's table holds offsets
            src.divisor = m_family(nb.path) == 2 ? 1.0 - h->opts.beta_m : 0.0;   // a momentum buffer sums what the window averaged
            LAUNCH(launch_convert_moment(src, first_moment(nb), nb.numel, s), "convert_moment_kernel");
            h->launches += 1;
        }
        if (keep_v[i]) {
            src.data = h->ws + h->sl.v + reinterpret_cast<size_t>(wb.v); src.divisor = 0.0;
            LAUNCH(launch_convert_moment(src, second_moment(nb), nb.numel, s), "convert_moment_kernel");
            h->launches += 1;
        }
    }
    return BAOC_OK;
}

// ---- one-step timing of every (block, configuration) pair ---------------------------
namespace {
size_t single_block_state_bytes(const Handle* h, int block, int cfg) {
    baoc_handle one;
    one.n_blocks = 1; one.n_cfg = h->n_cfg; one.blocks.assign(1, h->blocks[block]); one.cfgs = h->cfgs; one.opts = h->opts;
    one.numel = h->blocks[block].numel;
    Handle::StepLayout L{};
    const int32_t a = cfg;
    if (compute_step_layout(&one, &a, &L, nullptr, nullptr, nullptr, nullptr, nullptr) != BAOC_OK) return 0;
    return L.total;
}
bool assignable(const Handle* h, int block, int cfg) {
    const Path p = path_of(h->cfgs[cfg]);
    return p != kPathNone && !(is_factored_path(p) && h->blocks[block].cols <= 1);
}
}  // namespace

int baoc_time_scratch_bytes(const baoc_t* h, size_t* bytes) {
    if (!h) return BAOC_E_INVALID;
    if (!bytes) return fail(h, BAOC_E_INVALID, "baoc_time_scratch_bytes: null output");
    size_t need = 0;
    for (int i = 0; i < h->n_blocks; ++i)
        for (int c = 0; c < h->n_cfg; ++c)
            if (assignable(h, i, c)) need = std::max(need, single_block_state_bytes(h, i, c));
    *bytes = need;
    return BAOC_OK;
}

int baoc_measure_time_ratios(baoc_t* h, const void* const* grads, float* const* params, void* scratch_dev,
                             size_t scratch_bytes, int base_cfg, int reps, double* time_ratio_out,
                             double* time_ms_out, baoc_stream_t stream) {
    if (!h) return BAOC_E_INVALID;
    if (!grads || !params || !scratch_dev || !time_ratio_out) return fail(h, BAOC_E_INVALID, "baoc_measure_time_ratios: null argument");
    if (base_cfg < 0 || base_cfg >= h->n_cfg || reps < 1 || reps > 1000) return fail(h, BAOC_E_INVALID, "baoc_measure_time_ratios: bad base configuration or repetition count");
    if (reinterpret_cast<uintptr_t>(scratch_dev) & 255u) return fail(h, BAOC_E_ALIGN, "baoc_measure_time_ratios: scratch not 256-byte aligned");
    size_t need = 0;
    baoc_time_scratch_bytes(h, &need);
    if (scratch_bytes < need) return fail(h, BAOC_E_WORKSPACE, "baoc_measure_time_ratios: scratch too small");
    for (int i = 0; i < h->n_blocks; ++i) {
        if (!grads[i] || !params[i]) return fail(h, BAOC_E_INVALID, "baoc_measure_time_ratios: null block pointer");
        if (!aligned16(grads[i]) || !aligned16(params[i])) return fail(h, BAOC_E_ALIGN, "baoc_measure_time_ratios: block pointer not 16-byte aligned");
        if (!assignable(h, i, base_cfg)) return fail(h, BAOC_E_INVALID, "baoc_measure_time_ratios: the base configuration cannot be assigned to every block");
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaEvent_t e0, e1;
    CU(cudaEventCreate(&e0), "baoc_measure_time_ratios");
    if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return fail(h, BAOC_E_CUDA, "baoc_measure_time_ratios: event creation failed"); }
    const int K = h->n_cfg;
    std::vector<double> ms(size_t(h->n_blocks) * K, -1.0);
    int rc = BAOC_OK;
    for (int i = 0; i < h->n_blocks && rc == BAOC_OK; ++i) {
        // a one-block handle with every learning rate at zero: the step runs at full cost, the parameters come
        // out bit-identical (theta * (1 - 0) - 0 * direction) and only the scratch state is written
        baoc_handle one;
        one.n_blocks = 1; one.n_cfg = K; one.blocks.assign(1, h->blocks[i]); one.cfgs = h->cfgs; one.opts = h->opts;
        one.numel = h->blocks[i].numel;
        for (baoc_config_t& c : one.cfgs) {
            c.lr = 0.0f;
            // Adafactor's relative step size does not come from lr: time it as update clipping, which runs the same
            // sweep for the two norms, so that the step size stays lr = 0
            if (c.af_flags & kAfRelative) c.af_flags = uint8_t((c.af_flags & ~kAfRelative) | kAfClip);
        }
        const void* g1[1] = {grads[i]};
        float* p1[1] = {params[i]};
        for (int c = 0; c < K && rc == BAOC_OK; ++c) {
            if (!assignable(h, i, c)) continue;
            const int32_t a = c;
            rc = configure_state(&one, &a, scratch_dev, scratch_bytes, stream, true);
            if (rc == BAOC_OK) rc = do_step(&one, g1, p1, 1, s);                       // warm-up (also uploads the pointer tables)
            if (rc != BAOC_OK) break;
            cudaEventRecord(e0, s);
            for (int r = 0; r < reps && rc == BAOC_OK; ++r) rc = do_step(&one, g1, p1, 2 + r, s);
            cudaEventRecord(e1, s);
            if (rc != BAOC_OK) break;
            float t = 0.f;
            if (cudaEventSynchronize(e1) != cudaSuccess || cudaEventElapsedTime(&t, e0, e1) != cudaSuccess) { rc = BAOC_E_CUDA; one.err = "event timing failed"; break; }
            ms[size_t(i) * K + c] = double(t) / reps;
        }
        if (rc != BAOC_OK) h->err = "baoc_measure_time_ratios: " + one.err;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc != BAOC_OK) return rc;
    std::vector<double> model(size_t(h->n_blocks) * K);
    baoc_cost_model(h, nullptr, model.data());
    for (int i = 0; i < h->n_blocks; ++i) {
        const double base = ms[size_t(i) * K + base_cfg];
        for (int c = 0; c < K; ++c) {
            const size_t k = size_t(i) * K + c;
            // pairs that cannot be assigned keep the bytes model's value (the allocator masks them anyway)
            time_ratio_out[k] = (ms[k] >= 0.0 && base > 0.0) ? ms[k] / base : model[k];
            if (time_ms_out) time_ms_out[k] = ms[k];
        }
    }
    return BAOC_OK;
}

// ---- checkpoint / resume ---------------------------------------------------------
namespace {
struct BlobHeader {
    uint32_t magic, version;
    int32_t n_blocks, n_cfg;
    int64_t numel, stats_steps;
    int32_t ws_bound, configured;
    uint64_t shape_hash;
};
constexpr uint32_t kBlobMagic = 0x434f4142u;   // "BAOC"

// FNV-1a over the block shapes and the configuration tuples (not their hyper-parameters, which may change on resume)
uint64_t shape_hash(const Handle* h) {
    uint64_t x = 1469598103934665603ull;
    auto mix = [&](const void* p, size_t n) {
        const unsigned char* b = static_cast<const unsigned char*>(p);
        for (size_t i = 0; i < n; ++i) { x ^= b[i]; x *= 1099511628211ull; }
    };
    for (const baoc_block_t& b : h->blocks) { mix(&b.numel, 8); mix(&b.rows, 4); mix(&b.cols, 4); }
    for (const baoc_config_t& c : h->cfgs) mix(&c.adaptive, 7);      // the tuple, the 8-bit quantiser and Adafactor's options
    return x;
}
}  // namespace

int baoc_export(const baoc_t* h, void* buf, size_t capacity, size_t* size) {
    if (!h) return BAOC_E_INVALID;
    if (!size) return fail(h, BAOC_E_INVALID, "baoc_export: null size");
    const size_t need = sizeof(BlobHeader) + (h->configured ? (4 + 16) * size_t(h->n_blocks) : 0);
    *size = need;
    if (!buf) return BAOC_OK;
    if (capacity < need) return fail(h, BAOC_E_WORKSPACE, "baoc_export: buffer too small");
    BlobHeader hd{};
    hd.magic = kBlobMagic; hd.version = 3; hd.n_blocks = h->n_blocks; hd.n_cfg = h->n_cfg;
    hd.numel = h->numel; hd.stats_steps = h->stats_steps;
    hd.ws_bound = h->ws_bound ? 1 : 0; hd.configured = h->configured ? 1 : 0;
    hd.shape_hash = shape_hash(h);
    std::memcpy(buf, &hd, sizeof(hd));
    if (h->configured) {                                   // assignment, then the moment start steps of every block
        char* p = static_cast<char*>(buf) + sizeof(hd);
        const size_t n = size_t(h->n_blocks);
        std::memcpy(p, h->assign.data(), 4 * n);
        std::memcpy(p + 4 * n, h->t_m0.data(), 8 * n);
        std::memcpy(p + 12 * n, h->t_v0.data(), 8 * n);
    }
    return BAOC_OK;
}

int baoc_import(baoc_t* h, const void* blob, size_t size, void* ws_dev, size_t ws_bytes, void* state_dev,
                size_t state_bytes, baoc_stream_t stream) {
    if (!h) return BAOC_E_INVALID;
    if (!blob || size < sizeof(BlobHeader)) return fail(h, BAOC_E_INVALID, "baoc_import: blob missing or truncated");
    BlobHeader hd;
    std::memcpy(&hd, blob, sizeof(hd));
    if (hd.magic != kBlobMagic || hd.version != 3) return fail(h, BAOC_E_INVALID, "baoc_import: not a blob of this library version");
    if (hd.n_blocks != h->n_blocks || hd.n_cfg != h->n_cfg || hd.numel != h->numel || hd.shape_hash != shape_hash(h))
        return fail(h, BAOC_E_INVALID, "baoc_import: the blob belongs to a different block set or candidate set");
    if (hd.stats_steps < 0) return fail(h, BAOC_E_INVALID, "baoc_import: corrupt blob");
    if (hd.configured && size < sizeof(BlobHeader) + 20 * size_t(h->n_blocks)) return fail(h, BAOC_E_INVALID, "baoc_import: blob truncated");
    if (hd.ws_bound && !ws_dev) return fail(h, BAOC_E_INVALID, "baoc_import: the checkpoint had a statistics workspace; pass its copy");
    if (hd.configured && !state_dev) return fail(h, BAOC_E_INVALID, "baoc_import: the checkpoint had optimizer state; pass its copy");
    if (hd.ws_bound) {
        int rc = bind_stats(h, ws_dev, ws_bytes, stream, false);
        if (rc) return rc;
        h->stats_steps = hd.stats_steps;
    }
    if (hd.configured) {
        std::vector<int32_t> assign(h->n_blocks);
        std::memcpy(assign.data(), static_cast<const char*>(blob) + sizeof(BlobHeader), 4 * size_t(h->n_blocks));
        const char* p = static_cast<const char*>(blob) + sizeof(BlobHeader) + 4 * size_t(h->n_blocks);
        h->t_m0.resize(h->n_blocks); h->t_v0.resize(h->n_blocks);
        std::memcpy(h->t_m0.data(), p, 8 * size_t(h->n_blocks));
        std::memcpy(h->t_v0.data(), p + 8 * size_t(h->n_blocks), 8 * size_t(h->n_blocks));
        int rc = configure_state(h, assign.data(), state_dev, state_bytes, stream, false);
        if (rc) return rc;
    }
    return BAOC_OK;
}

int baoc_step(baoc_t* h, const void* const* grads, float* const* params, int64_t step_t, baoc_stream_t stream) {
    if (!h) return BAOC_E_INVALID;
    if (!grads || !params) return fail(h, BAOC_E_INVALID, "baoc_step: null pointer table");
    if (step_t < 1) return fail(h, BAOC_E_INVALID, "baoc_step: step numbers start at 1");
    if (!h->configured) return fail(h, BAOC_E_STATE, "baoc_step: no assignment configured");
    return do_step(h, grads, params, step_t, static_cast<cudaStream_t>(stream));
}

int baoc_step_from_host(baoc_t* h, const void* const* host_grads, void* const* dev_grads, float* const* params,
                        int do_stats, int64_t step_t, baoc_stream_t stream) {
    if (!h) return BAOC_E_INVALID;
    if (!host_grads || !dev_grads) return fail(h, BAOC_E_INVALID, "baoc_step_from_host: null pointer table");
    if (do_stats && !h->ws_bound) return fail(h, BAOC_E_STATE, "baoc_step_from_host: no statistics workspace bound");
    if (step_t > 0 && (!h->configured || !params)) return fail(h, BAOC_E_STATE, "baoc_step_from_host: no assignment configured");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (int i = 0; i < h->n_blocks; ++i) {
        if (!host_grads[i] || !dev_grads[i]) return fail(h, BAOC_E_INVALID, "baoc_step_from_host: null block pointer");
        if (!aligned16(dev_grads[i])) return fail(h, BAOC_E_ALIGN, "baoc_step_from_host: block pointer not 16-byte aligned");
    }
    const void* const* dg = reinterpret_cast<const void* const*>(dev_grads);
    // copy blocks [b0, b1); blocks that are contiguous on both sides travel in one copy
    auto copy_range = [&](int b0, int b1, cudaStream_t cs) -> cudaError_t {
        int i = b0;
        while (i < b1) {
            int j = i;
            size_t bytes = 2 * size_t(h->blocks[i].numel);
            while (j + 1 < b1 &&
                   static_cast<const char*>(host_grads[j + 1]) == static_cast<const char*>(host_grads[i]) + bytes &&
                   static_cast<const char*>(dev_grads[j + 1]) == static_cast<const char*>(dev_grads[i]) + bytes) {
                ++j;
                bytes += 2 * size_t(h->blocks[j].numel);
            }
            cudaError_t e = cudaMemcpyAsync(dev_grads[i], host_grads[i], bytes, cudaMemcpyHostToDevice, cs);
            if (e != cudaSuccess) return e;
            i = j + 1;
        }
        return cudaSuccess;
    };
    if (!do_stats) {
        CU(copy_range(0, h->n_blocks, s), "baoc_step_from_host (copy)");
        if (step_t > 0) return do_step(h, dg, params, step_t, s);
        return BAOC_OK;
    }
    // With statistics: the copy runs on an internal stream in up to kCopyGroups groups of whole blocks, and the
    // caller's stream observes a group as soon as it has landed, so the statistics pass hides behind the transfer.
    if (!h->copy_stream) {
        cudaStream_t cs;
        CU(cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking), "baoc_step_from_host (copy stream)");
        h->copy_stream = cs;
        for (void*& e : h->copy_ev) {
            cudaEvent_t ev;
            CU(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming), "baoc_step_from_host (event)");
            e = ev;
        }
        h->cuda_cleanup = destroy_cuda_objects;
    }
    cudaStream_t cs = static_cast<cudaStream_t>(h->copy_stream);
    int rc = sync_pointer_table(h, dg, &h->last_stat_grads, h->ws + h->sl.grads, s, "baoc_step_from_host");
    if (rc) return rc;
    // Everything that can fail on the host alone comes before the copy stream is forked from the caller's stream.
    // With an optimizer step as well, every group also takes its step as soon as its statistics are queued, so that
    // only the last group's work is left when the transfer ends.  Each block sees exactly the launches of baoc_step.
    std::vector<int> gb0, gb1;
    compute_copy_groups(h, &gb0, &gb1);
    if (gb0.size() > size_t(Handle::kCopyGroups)) return fail(h, BAOC_E_INVALID, "baoc_step_from_host: more copy groups than events");
    if (step_t > 0) {                                       // the by-group tile table was laid out for these very groups
        bool same = h->groups.size() == gb0.size();
        for (size_t g = 0; same && g < gb0.size(); ++g) same = h->groups[g].b0 == gb0[g] && h->groups[g].b1 == gb1[g];
        if (!same) return fail(h, BAOC_E_STATE, "baoc_step_from_host: the configured state was laid out for other copy groups");
    }
    StepParams P;
    if (step_t > 0) {
        rc = step_prologue(h, dg, params, step_t, s, &P);
        if (rc) return rc;
    }
    // the copies must not overtake earlier work of the caller's stream that still reads the device gradients
    CU(cudaEventRecord(static_cast<cudaEvent_t>(h->copy_ev[Handle::kCopyGroups]), s), "baoc_step_from_host");
    CU(cudaStreamWaitEvent(cs, static_cast<cudaEvent_t>(h->copy_ev[Handle::kCopyGroups]), 0), "baoc_step_from_host");
    // From here on the copy stream runs ahead of the caller's stream.  Whatever goes wrong, the caller's stream is
    // joined to the copies already queued before the call returns, so that a retry or any later work on that stream
    // cannot race with a transfer still in flight.
    auto join = [&]() {
        if (cudaEventRecord(static_cast<cudaEvent_t>(h->copy_ev[Handle::kCopyGroups]), cs) == cudaSuccess)
            cudaStreamWaitEvent(s, static_cast<cudaEvent_t>(h->copy_ev[Handle::kCopyGroups]), 0);
    };
    for (size_t g = 0; g < gb0.size(); ++g) {
        cudaError_t e = copy_range(gb0[g], gb1[g], cs);
        if (e == cudaSuccess) e = cudaEventRecord(static_cast<cudaEvent_t>(h->copy_ev[g]), cs);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s, static_cast<cudaEvent_t>(h->copy_ev[g]), 0);
        if (e != cudaSuccess) { join(); return cuda_fail(h, "baoc_step_from_host (copy)", e); }
        rc = stats_step_range(h, gb0[g], gb1[g], s);
        // blocks with Adafactor's options need their norms between the reduction and the update: with such blocks the
        // step follows the transfer as a whole instead of group by group
        if (rc == BAOC_OK && step_t > 0 && h->n_fa == 0) rc = step_group(h, h->groups[g], P, s);
        if (rc) { join(); return rc; }
    }
    if (step_t > 0 && h->n_fa > 0) {
        rc = step_launches(h, P, s);
        if (rc) return rc;
    }
    return stats_combine_all(h, s);
}



int baoc_set_factored_schedule(baoc_t* h, int64_t group_bytes) {
    if (!h) return BAOC_E_INVALID;
    if (group_bytes < 0) return fail(h, BAOC_E_INVALID, "baoc_set_factored_schedule: negative size");
    if (h->configured) return fail(h, BAOC_E_STATE, "baoc_set_factored_schedule: set the schedule before baoc_configure");
    h->factored_group_bytes = group_bytes;
    return BAOC_OK;
}

int baoc_check_status(baoc_check_t* out) {
    if (!out) return BAOC_E_INVALID;
    std::memset(out, 0, sizeof(*out));
#ifdef BAOC_CHECKED
    out->enabled = 1;
    if (cudaDeviceSynchronize() != cudaSuccess) return BAOC_E_CUDA;
    int (*const fetch[])(CheckRecord*) = {stats_check_fetch, finalize_check_fetch, step_check_fetch};
    for (auto f : fetch) {
        CheckRecord r{};
        if (f(&r) != 0) return BAOC_E_CUDA;
        if (r.code != 0 && out->code == 0) {                 // every unit is fetched and cleared; the first violation is reported
            out->code = r.code; out->kernel = r.kernel; out->a = r.a; out->b = r.b; out->c = r.c; out->d = r.d;
        }
    }
#endif
    return BAOC_OK;
}

int baoc_check_selftest(baoc_stream_t stream) {
#ifdef BAOC_CHECKED
    return launch_check_selftest(static_cast<cudaStream_t>(stream)) == 0 ? BAOC_OK : BAOC_E_CUDA;
#else
    (void)stream;
    return BAOC_E_STATE;
#endif
}

int baoc_profile(baoc_t* h, int enable) {
    if (!h) return BAOC_E_INVALID;
    if (enable && !h->prof_ev[0]) {
        for (void*& e : h->prof_ev) {
            cudaEvent_t ev;
            CU(cudaEventCreate(&ev), "baoc_profile");
            e = ev;
        }
        h->cuda_cleanup = destroy_cuda_objects;
    }
    h->prof_on = enable != 0;
    h->prof_valid = false;
    return BAOC_OK;
}

int baoc_profile_last(baoc_t* h, float* ms2) {
    if (!h) return BAOC_E_INVALID;
    if (!ms2) return fail(h, BAOC_E_INVALID, "baoc_profile_last: null output");
    if (!h->prof_on || !h->prof_valid) return fail(h, BAOC_E_STATE, "baoc_profile_last: profiling is off or no step has run");
    CU(cudaEventSynchronize(static_cast<cudaEvent_t>(h->prof_ev[2])), "baoc_profile_last");
    CU(cudaEventElapsedTime(&ms2[0], static_cast<cudaEvent_t>(h->prof_ev[0]), static_cast<cudaEvent_t>(h->prof_ev[1])), "baoc_profile_last");
    CU(cudaEventElapsedTime(&ms2[1], static_cast<cudaEvent_t>(h->prof_ev[1]), static_cast<cudaEvent_t>(h->prof_ev[2])), "baoc_profile_last");
    return BAOC_OK;
}

int baoc_view(const baoc_t* h, int block, int which, void** dev_ptr, int64_t* count, int32_t* elem_bytes) {
    if (!h) return BAOC_E_INVALID;
    if (!dev_ptr || !count || !elem_bytes || block < 0 || block >= h->n_blocks) return fail(h, BAOC_E_INVALID, "baoc_view: bad argument");
    const baoc_block_t& b = h->blocks[block];
    if (which >= 0 && which <= 2) {
        if (!h->ws_bound) return fail(h, BAOC_E_STATE, "baoc_view: no statistics workspace bound");
        const StatBlock& s = h->h_stat_blocks[block];
        const size_t off = reinterpret_cast<size_t>(which == 2 ? static_cast<void*>(s.gprev) : static_cast<void*>(which == 0 ? s.m : s.v));
        const size_t region = which == 0 ? h->sl.m : (which == 1 ? h->sl.v : h->sl.gprev);
        *dev_ptr = h->ws + region + off; *count = h->stat_shapes[block].numel; *elem_bytes = which == 2 ? 2 : 4;
        return BAOC_OK;
    }
    if (which >= 10 && which <= 13) {
        if (!h->configured) return fail(h, BAOC_E_STATE, "baoc_view: no assignment configured");
        const StepBlock& s = h->h_step_blocks[block];
        const int k = which - 10;
        const int64_t nq = ceil_div(b.numel, kQBlock);
        void* p = nullptr; int64_t n = 0; int32_t eb = 4;
        switch (s.path) {
            case kPathA32: if (k == 0) { p = s.s0; n = b.numel; } else if (k == 1) { p = s.s1; n = b.numel; } break;
            case kPathA8: case kPathA8N:
                if (k == 0) { p = s.s0; n = b.numel; eb = 1; } else if (k == 1) { p = s.s1; n = b.numel; eb = 1; }
                else if (k == 2) { p = s.a0; n = nq; } else { p = s.a1; n = nq; }
                break;
            case kPathR: case kPathS: if (k == 0) { p = s.s0; n = b.numel; } break;
            case kPathA16: if (k == 0) { p = s.s0; n = b.numel; eb = 2; } else if (k == 1) { p = s.s1; n = b.numel; eb = 2; } break;
            case kPathR16: case kPathS16: if (k == 0) { p = s.s0; n = b.numel; eb = 2; } break;
            case kPathR8: if (k == 0) { p = s.s1; n = b.numel; eb = 1; } else if (k == 1) { p = s.a1; n = nq; } break;
            case kPathS8: if (k == 0) { p = s.s0; n = b.numel; eb = 1; } else if (k == 1) { p = s.a0; n = nq; } break;
            case kPathF: case kPathFA:
                if (s.fbits == 32) { if (k == 0) { p = s.s0; n = b.rows; } else if (k == 1) { p = s.s1; n = b.cols; } }
                else {
                    const int32_t e = s.fbits == 16 ? 2 : 1;
                    if (k == 0) { p = s.f0; n = b.rows; eb = e; } else if (k == 1) { p = s.f1; n = b.cols; eb = e; }
                    else if (s.fbits == 8 && k == 2) { p = s.fa0; n = ceil_div(b.rows, kQBlock); }
                    else if (s.fbits == 8 && k == 3) { p = s.fa1; n = ceil_div(b.cols, kQBlock); }
                }
                break;
            default: break;
        }
        if (!p) return fail(h, BAOC_E_INVALID, "baoc_view: the block has no such state tensor");
        *dev_ptr = p; *count = n; *elem_bytes = eb;
        return BAOC_OK;
    }
    return fail(h, BAOC_E_INVALID, "baoc_view: unknown tensor id");
}

int baoc_nonfinite(baoc_t* h, uint8_t* flags, int32_t* count, baoc_stream_t stream) {
    if (!h) return BAOC_E_INVALID;
    if (!count) return fail(h, BAOC_E_INVALID, "baoc_nonfinite: null count");
    if (!h->configured) return fail(h, BAOC_E_STATE, "baoc_nonfinite: no assignment configured");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<uint32_t> f(h->n_blocks);
    CU(cudaMemcpyAsync(f.data(), h->st + h->tl.flags, 4 * f.size(), cudaMemcpyDeviceToHost, s), "baoc_nonfinite");
    CU(cudaStreamSynchronize(s), "baoc_nonfinite");
    int32_t c = 0;
    for (int i = 0; i < h->n_blocks; ++i) {
        if (flags) flags[i] = f[i] ? 1 : 0;
        c += f[i] ? 1 : 0;
    }
    *count = c;
    return BAOC_OK;
}

}  // extern "C"
