// Offline side of the method on top of the kernels: the tree search that generates an ensemble of elastic
// configurations (Sec. III-B, Algorithm 1) and the pruning of mid-precision modules (Sec. III-C), driven by
// per-module tables instead of perplexity runs.  Host code; the only kernel here measures the output error
// of a layer (the stand-in for the calibration-set evaluation).
#include <algorithm>
#include <cmath>
#include <vector>

#include <cuda_bf16.h>

#include "fq_internal.cuh"

namespace {

double state_cost(const uint8_t* st, const double* cost, int M, int Lv)
{
    double c = 0.0;
    for (int m = 0; m < M; m++) c += cost[m * Lv + st[m]];
    return c;
}
uint64_t state_foot(const uint8_t* st, const uint64_t* foot, int M, int Lv)
{
    uint64_t f = 0;
    for (int m = 0; m < M; m++) f += foot[m * Lv + st[m]];
    return f;
}

__global__ void sqdiff_kernel(const __nv_bfloat16* a, const __nv_bfloat16* b, size_t n, double* out)
{
    double d2 = 0.0, b2 = 0.0;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const double x = (double)__bfloat162float(a[i]), y = (double)__bfloat162float(b[i]);
        d2 += (x - y) * (x - y);
        b2 += y * y;
    }
    for (int o = 16; o > 0; o >>= 1) {
        d2 += __shfl_xor_sync(0xffffffffu, d2, o);
        b2 += __shfl_xor_sync(0xffffffffu, b2, o);
    }
    if ((threadIdx.x & 31) == 0) { atomicAdd(out, d2); atomicAdd(out + 1, b2); }
}

// Beam search over one-way precision chains (Sec. III-B, Algorithm 1).  A beam entry is a whole chain
// (configuration after configuration, M levels each); every round extends each entry by one move, "module m goes
// down one stored precision", and keeps the `stems` best distinct extensions.
struct Move { int stem, module; double sens, cost; uint64_t foot; };
using Chain = std::vector<uint8_t>;

// The moves open to one beam entry, cut down to the `branches` whose single-module sensitivity is smallest
// (ties keep module order), each scored by the evaluation function of the configuration it leads to.
void shortlist(int stem, const uint8_t* last, const double* cost, const double* sens, const uint64_t* foot, int M, int Lv,
               int branches, std::vector<Move>& pool)
{
    std::vector<Move> open;
    for (int m = 0; m < M; m++)
        if (last[m] + 1 < Lv) open.push_back(Move{stem, m, sens[m * Lv + last[m] + 1], 0.0, 0});
    std::stable_sort(open.begin(), open.end(), [](const Move& a, const Move& b) { return a.sens < b.sens; });
    if ((int)open.size() > branches) open.resize(branches);
    Chain cfg(last, last + M);
    for (Move& mv : open) {
        cfg[mv.module]++;
        mv.cost = state_cost(cfg.data(), cost, M, Lv);
        mv.foot = state_foot(cfg.data(), foot, M, Lv);
        cfg[mv.module]--;
        pool.push_back(mv);
    }
}

// The next beam: moves in order of evaluation (then footprint, then beam and module order), each appended to a
// copy of its entry; a configuration that two entries reach is kept once.
std::vector<Chain> next_beam(const std::vector<Chain>& beam, std::vector<Move>& pool, int depth, int M, int stems)
{
    std::stable_sort(pool.begin(), pool.end(), [](const Move& a, const Move& b) {
        if (a.cost != b.cost) return a.cost < b.cost;
        return a.foot < b.foot;
    });
    std::vector<Chain> next;
    for (const Move& mv : pool) {
        if ((int)next.size() == stems) break;
        const Chain& from = beam[mv.stem];
        Chain grown(from.begin(), from.begin() + (size_t)depth * M);
        grown.insert(grown.end(), from.begin() + (size_t)(depth - 1) * M, from.begin() + (size_t)depth * M);
        grown[(size_t)depth * M + mv.module]++;
        bool seen = false;
        for (const Chain& q : next)
            if (std::equal(q.end() - M, q.end(), grown.end() - M)) { seen = true; break; }
        if (!seen) next.push_back(std::move(grown));
    }
    return next;
}

}  // namespace

extern "C" {

int fq_search_chain(const double* cost, const double* sens, const uint64_t* foot, int n_modules, int n_levels,
                    int stems, int branches, uint8_t* chain_out, int* n_states_out, double* curve_cost_out)
{
    if (!cost || !sens || !foot || !chain_out) return FQ_ERR_ARG;
    if (n_modules < 1 || n_levels < 2 || n_levels > 8 || stems < 1 || branches < 1) return FQ_ERR_ARG;
    const int M = n_modules, Lv = n_levels;
    const int n_moves = M * (Lv - 1);                       // from all-highest to all-lowest, one level of one module at a time
    std::vector<Chain> beam(1, Chain(M, 0));
    for (int depth = 1; depth <= n_moves; depth++) {
        std::vector<Move> pool;
        for (int s = 0; s < (int)beam.size(); s++)
            shortlist(s, beam[s].data() + (size_t)(depth - 1) * M, cost, sens, foot, M, Lv, branches, pool);
        beam = next_beam(beam, pool, depth, M, stems);
    }
    // the chain whose trade-off curve is best: smallest sum of the evaluation over its configurations
    int best = 0;
    double best_c = 0.0;
    for (int s = 0; s < (int)beam.size(); s++) {
        double c = 0.0;
        for (int t = 0; t <= n_moves; t++) c += state_cost(beam[s].data() + (size_t)t * M, cost, M, Lv);
        if (s == 0 || c < best_c) { best = s; best_c = c; }
    }
    std::copy(beam[best].begin(), beam[best].end(), chain_out);
    if (n_states_out) *n_states_out = n_moves + 1;
    if (curve_cost_out) *curve_cost_out = best_c;
    return FQ_OK;
}

int fq_prune_chain(const uint8_t* chain, int n_states, int n_modules, int n_levels, const uint64_t* foot, double fraction,
                   uint8_t* pruned_chain_out, uint8_t* dropped_out, uint64_t* storage_before_out, uint64_t* storage_after_out)
{
    if (!chain || !foot || !pruned_chain_out || !dropped_out) return FQ_ERR_ARG;
    if (n_states < 1 || n_modules < 1 || n_levels < 2 || n_levels > 8 || !(fraction >= 0.0 && fraction <= 1.0)) return FQ_ERR_ARG;
    const int M = n_modules, Lv = n_levels;
    struct Item { int module, level; long long uses, late; };
    std::vector<Item> items;                                 // every module of every mid-precision model
    for (int m = 0; m < M; m++)
        for (int l = 1; l + 1 < Lv; l++) {
            Item it{m, l, 0, 0};
            for (int t = 0; t < n_states; t++)
                if (chain[(size_t)t * M + m] == l) { it.uses++; it.late += t; }   // later = smaller footprint
            items.push_back(it);
        }
    // least important first: fewer configurations use it; among equals, used at larger footprints
    std::stable_sort(items.begin(), items.end(), [](const Item& a, const Item& b) {
        if (a.uses != b.uses) return a.uses < b.uses;
        return a.late < b.late;
    });
    const int n_drop = (int)std::floor(fraction * (double)items.size() + 1e-9);
    std::fill(dropped_out, dropped_out + (size_t)M * Lv, (uint8_t)0);
    for (int i = 0; i < n_drop; i++) dropped_out[items[i].module * Lv + items[i].level] = 1;
    uint64_t before = 0, after = 0;
    for (int m = 0; m < M; m++)
        for (int l = 0; l < Lv; l++) {
            before += foot[m * Lv + l];
            if (!dropped_out[m * Lv + l]) after += foot[m * Lv + l];
        }
    // a configuration that used a dropped module falls to the next stored lower precision (still one-way)
    for (int t = 0; t < n_states; t++)
        for (int m = 0; m < M; m++) {
            int l = chain[(size_t)t * M + m];
            while (dropped_out[m * Lv + l]) l++;            // n_low is never dropped
            pruned_chain_out[(size_t)t * M + m] = (uint8_t)l;
        }
    if (storage_before_out) *storage_before_out = before;
    if (storage_after_out) *storage_after_out = after;
    return FQ_OK;
}

int fq_sqdiff(const uint16_t* a_bf16_dev, const uint16_t* b_bf16_dev, size_t n, double* sums_dev, void* stream)
{
    if (!a_bf16_dev || !b_bf16_dev || !sums_dev || n == 0) return FQ_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(sums_dev, 0, 2 * sizeof(double), st) != cudaSuccess) return FQ_ERR_CUDA;
    const int blocks = (int)std::min<size_t>((n + 255) / 256, (size_t)fq::current_sm_count() * 8);
    sqdiff_kernel<<<blocks, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(a_bf16_dev),
                                          reinterpret_cast<const __nv_bfloat16*>(b_bf16_dev), n, sums_dev);
    return cudaGetLastError() == cudaSuccess ? FQ_OK : FQ_ERR_CUDA;
}

}  // extern "C"
