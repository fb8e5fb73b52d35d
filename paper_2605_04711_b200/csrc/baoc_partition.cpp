// Block partitioning (appendix on block partitioning, Algorithm 2): from candidate units in forward order, their
// parameter counts and their normalised diagnostic vectors to the final blocks.  Host only.
//
// A block is always a run of consecutive units, so the partition is kept as a sorted list of run starts.  The
// algorithm's steps are stated loosely; the reading implemented here:
//   - every gap between adjacent units is a candidate boundary;
//   - a run's diagnostic vector is the size-weighted mean of its units' vectors, accumulated in unit order as offsets
//     from the first unit's vector (identical units average to exactly that vector);
//   - Delta(a, b) = max_k w_k |z_a,k - z_b,k|; tau defaults to the upper quartile (linear interpolation at position
//     0.75 (P - 1)) of Delta over all P pairs of candidate units;
//   - minimum-size filtering: while a run is smaller than n_min = alpha |Theta| and it is not the only run, the first such
//     run joins the adjacent run with the smaller Delta to it (ties: the smaller neighbour, then the left one);
//   - block formation: the boundary between two adjacent runs of the filtered list survives iff their Delta exceeds tau;
//   - post-processing: a block made of several filtered runs is cut at the run boundary where the Delta between the means
//     of its two sides is largest, if that Delta exceeds tau and both sides reach n_min, and the halves are examined
//     again; then the minimum-size filtering runs once more.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

#include "baoc.h"

namespace {

struct Units {
    int m, k;
    const int64_t* numel;
    const double* z;
    std::vector<double> w;
    double n_min;

    int64_t size(int lo, int hi) const {
        int64_t s = 0;
        for (int j = lo; j < hi; ++j) s += numel[j];
        return s;
    }
    void mean(int lo, int hi, double* out) const {
        const double* first = z + size_t(lo) * k;
        std::vector<double> acc(k, 0.0);
        double tot = 0.0;
        for (int j = lo; j < hi; ++j) {
            const double n = double(numel[j]);
            for (int c = 0; c < k; ++c) acc[c] = acc[c] + n * (z[size_t(j) * k + c] - first[c]);
            tot += n;
        }
        for (int c = 0; c < k; ++c) out[c] = first[c] + acc[c] / tot;
    }
    double delta(const double* a, const double* b) const {
        double d = 0.0;
        for (int c = 0; c < k; ++c) d = std::max(d, w[c] * std::fabs(a[c] - b[c]));
        return d;
    }
    double delta_runs(int lo_a, int hi_a, int lo_b, int hi_b) const {
        std::vector<double> a(k), b(k);
        mean(lo_a, hi_a, a.data());
        mean(lo_b, hi_b, b.data());
        return delta(a.data(), b.data());
    }
};

// starts: sorted run starts, starts[0] == 0; run r covers [starts[r], r + 1 < n ? starts[r + 1] : m).
int run_end(const std::vector<int>& starts, size_t r, int m) { return r + 1 < starts.size() ? starts[r + 1] : m; }

void size_filter(const Units& u, std::vector<int>* starts) {
    std::vector<int>& s = *starts;
    while (s.size() > 1) {
        size_t small = s.size();
        for (size_t r = 0; r < s.size(); ++r)
            if (double(u.size(s[r], run_end(s, r, u.m))) < u.n_min) { small = r; break; }
        if (small == s.size()) return;
        const int lo = s[small], hi = run_end(s, small, u.m);
        bool take_right;
        if (small == 0) take_right = true;
        else if (small + 1 == s.size()) take_right = false;
        else {
            const double dl = u.delta_runs(lo, hi, s[small - 1], lo), dr = u.delta_runs(lo, hi, hi, run_end(s, small + 1, u.m));
            const int64_t nl = u.size(s[small - 1], lo), nr = u.size(hi, run_end(s, small + 1, u.m));
            take_right = dr < dl || (dr == dl && nr < nl);
        }
        s.erase(s.begin() + (take_right ? small + 1 : small));      // dropping a run's start joins it to its left neighbour
    }
}

// Cut the block made of the filtered runs [r0, r1) where its two sides differ most; append the starts of the pieces after the first.
void split(const Units& u, const std::vector<int>& runs, size_t r0, size_t r1, double tau, std::vector<int>* out) {
    const int lo = runs[r0], hi = run_end(runs, r1 - 1, u.m);
    double best = -1.0;
    size_t cut = 0;
    for (size_t c = r0 + 1; c < r1; ++c) {
        const int mid = runs[c];
        if (double(u.size(lo, mid)) < u.n_min || double(u.size(mid, hi)) < u.n_min) continue;
        const double d = u.delta_runs(lo, mid, mid, hi);
        if (d > best) { best = d; cut = c; }
    }
    if (cut == 0 || !(best > tau)) return;
    split(u, runs, r0, cut, tau, out);
    out->push_back(runs[cut]);
    split(u, runs, cut, r1, tau, out);
}

}  // namespace

extern "C" int baoc_partition(int n_units, const int64_t* numel, const double* z, int k, const double* w, double alpha,
                              double tau, int32_t* block_of_unit, int32_t* n_blocks, double* tau_used) {
    if (n_units < 1 || !numel || !z || k < 1 || k > 64 || !block_of_unit) return BAOC_E_INVALID;
    if (!(alpha >= 0.0 && alpha <= 1.0) || std::isnan(tau)) return BAOC_E_INVALID;
    int64_t total = 0;
    for (int j = 0; j < n_units; ++j) {
        if (numel[j] < 1) return BAOC_E_INVALID;
        total += numel[j];
    }
    for (size_t i = 0; i < size_t(n_units) * k; ++i)
        if (!std::isfinite(z[i])) return BAOC_E_INVALID;
    Units u{n_units, k, numel, z, std::vector<double>(k, 1.0), alpha * double(total)};
    if (w)
        for (int c = 0; c < k; ++c) {
            if (!(w[c] >= 0.0) || !std::isfinite(w[c])) return BAOC_E_INVALID;
            u.w[c] = w[c];
        }
    if (tau < 0.0) {
        std::vector<double> pair;
        pair.reserve(size_t(n_units) * (n_units - 1) / 2);
        for (int a = 0; a < n_units; ++a)
            for (int b = a + 1; b < n_units; ++b) pair.push_back(u.delta(z + size_t(a) * k, z + size_t(b) * k));
        tau = 0.0;
        if (!pair.empty()) {
            std::sort(pair.begin(), pair.end());
            const double pos = 0.75 * double(pair.size() - 1);
            const size_t i = size_t(std::floor(pos));
            const double frac = pos - double(i);
            tau = i + 1 < pair.size() ? pair[i] + frac * (pair[i + 1] - pair[i]) : pair[i];
        }
    }
    std::vector<int> runs(n_units);
    for (int j = 0; j < n_units; ++j) runs[j] = j;
    size_filter(u, &runs);
    // block formation, then the split of each formed block
    std::vector<int> blocks{0};
    size_t first = 0;
    for (size_t r = 0; r < runs.size(); ++r) {
        const bool last = r + 1 == runs.size();
        const bool boundary = !last && u.delta_runs(runs[r], runs[r + 1], runs[r + 1], run_end(runs, r + 1, n_units)) > tau;
        if (last || boundary) {
            split(u, runs, first, r + 1, tau, &blocks);
            if (!last) blocks.push_back(runs[r + 1]);
            first = r + 1;
        }
    }
    size_filter(u, &blocks);
    for (size_t b = 0; b < blocks.size(); ++b)
        for (int j = blocks[b]; j < run_end(blocks, b, n_units); ++j) block_of_unit[j] = int32_t(b);
    if (n_blocks) *n_blocks = int32_t(blocks.size());
    if (tau_used) *tau_used = tau;
    return BAOC_OK;
}
