// Planner of the tensor-core SpMM path (batch >= 8, fp16 values).
//
// The uneven kernel matrices (Section 4.3.2 of the paper) are balanced on three levels here.  The
// matrix is cut into CTA tiles -- RG consecutive block-rows times a contiguous range of
// block-columns -- and the ranges of a row group are cut where the modelled work is equal, not
// where the column count is.  The warps of a CTA are dealt to the block-rows of its group in
// proportion to the rows' work inside the range.  And the items of a block-row (column slices of
// its blocks, so that no single item dominates) go, in block-column order, to whichever of the
// row's warps has the least work so far: at every point of the walk through the block-columns the
// warps of a row have done about the same amount of work, so they move through the shared ring of
// input tiles together.  The choice of RG and of the number S of column ranges per row group trades
// three kinds of traffic per CTA against each other: the weights (once in all), the packed inputs
// (once per row group, divided by S) and the sums that the S > 1 CTAs of a row group, one thread-block
// cluster, add up through distributed shared memory (in the fixed order of the ranges).
#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <numeric>

#include "csb_internal.hpp"

namespace csb {

static inline size_t pad_to(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Widest column slice whose rows still fit the item budget; a multiple of 16 so that slices are
// whole k-slabs of the m16n8k16 contraction.
static int slice_width(int m) { return m <= 16 ? 64 : m <= 32 ? 32 : 16; }

static size_t spmm_item_bytes(int m, int nk) {
    const int np2 = (nk + 1) / 2;
    return pad_to(sizeof(SpmmItemHeader) + pad_to((size_t)nk, 4) + (size_t)m * np2 * 4, 16);
}

// Modelled cost of an item for one warp, in instructions: a fixed part (header, row map, ring
// bookkeeping) and per 16-column slab the operand loads and the tensor instructions.
static double item_cost(int nk, int MT, int NT) { return 110.0 + (double)((nk + 15) / 16) * (14.0 + MT * (6.0 + 2.0 * NT)); }

static void emit_spmm_item(const csb_matrix* A, int64_t b, int k0, int k1, int tile, int col_base, std::vector<uint8_t>& out) {
    const int m = A->m[b], n = A->n[b], nk = k1 - k0, np2 = (nk + 1) / 2;
    const size_t base = out.size(), bytes = spmm_item_bytes(m, nk);
    out.resize(base + bytes, 0);
    uint8_t* p = out.data() + base;
    SpmmItemHeader h{};
    h.tile = (uint16_t)tile; h.nk = (uint8_t)nk; h.np2 = (uint8_t)np2; h.size16 = (uint16_t)(bytes / 16);
    const uint8_t* ri = A->row_idx.data() + A->ridx_off[b];
    uint64_t mask = 0;
    for (int r = 0; r < m; ++r) mask |= 1ull << ri[r];
    h.mask_lo = (uint32_t)mask; h.mask_hi = (uint32_t)(mask >> 32);
    std::memcpy(p, &h, sizeof h);
    const uint8_t* ci = A->col_idx.data() + A->cidx_off[b];
    for (int k = 0; k < nk; ++k) p[sizeof h + k] = (uint8_t)(col_base + ci[k0 + k]);
    uint8_t* v = p + sizeof h + pad_to((size_t)nk, 4);
    const uint8_t* src = A->val.data() + A->val_off[b] * 2;
    for (int r = 0; r < m; ++r)
        std::memcpy(v + (size_t)r * np2 * 4, src + ((size_t)r * n + k0) * 2, (size_t)nk * 2);
}

struct PlannedItem { int64_t block; int k0, k1, tile, col_base; };

int plan_spmm_host(const csb_matrix* A, int NT, int sm_count, SpmmHostPlan* out) {
    if (A->val_dtype != CSB_F16 || A->block_r > 64 || A->nbc > 60000) return 1;
    const int64_t nbr = A->nbr, nbc = A->nbc;
    const int MT = A->block_r <= 16 ? 1 : A->block_r <= 32 ? 2 : 4;
    const int nb_max = 8 * NT, n_warps = spmm_warps(NT), G = spmm_tile_blocks(A->block_c);
    const double x_bytes = (double)A->cols * spmm_pitch(NT), w_bytes = (double)A->nnz * 2.0 + 24.0 * (double)A->nblk;
    // ---- shape of the CTA tile: at most four block-rows, so that a block-row has several warps to
    // share its blocks between
    int best_RG = 1, best_S = 1;
    double best = 1e300;
    for (int RG = 4; RG >= 1; RG /= 2) {
        const int64_t groups = (nbr + RG - 1) / RG;
        int64_t S = std::max<int64_t>(1, sm_count / groups);
        S = std::min<int64_t>(std::min<int64_t>(S, nbc), 8);      // the CTAs of a row group form one cluster: at most 8
        const double ctas = (double)(groups * S);
        const double waves = std::ceil(ctas / sm_count);
        // (a cluster costs two cluster-wide barriers and the wait for its slowest CTA: as much time as about 120 KB of traffic per CTA (measured: a small GRU layer runs faster without, the 8192 x 8192 sweep with))
        static const double cluster_cost = getenv("CSB_SPMM_CLUSTER_COST") ? atof(getenv("CSB_SPMM_CLUSTER_COST")) : 120e3;
        const double per_cta = w_bytes / ctas + x_bytes / (double)S + (S > 1 ? 2.0 * RG * A->block_r * nb_max * 4.0 + cluster_cost : 0.0);
        // short ranges leave a warp only a few items to even its load out with
        const double cost = per_cta * waves * (1.0 + 6.0 * (double)S / (double)nbc);
        if (cost < best) { best = cost; best_RG = RG; best_S = (int)S; }
    }
    const int RG = best_RG, S = best_S;
    const int64_t groups = (nbr + RG - 1) / RG;
    out->RG = RG; out->S = S; out->n_groups = (int)groups; out->max_tiles = 0;
    out->ctas.clear(); out->chunks.clear(); out->bytes.clear(); out->stream_begin.clear();
    std::vector<double> cta_cost, warp_cost;
    auto cost_of_block = [&](int64_t b) {
        const int m = A->m[b], n = A->n[b];
        if (!m || !n) return 0.0;
        double c = 0.0;
        for (int k0 = 0; k0 < n; k0 += slice_width(m)) c += item_cost(std::min(n, k0 + slice_width(m)) - k0, MT, NT);
        return c;
    };
    for (int64_t g = 0; g < groups; ++g) {
        const int64_t br0 = g * RG, br1 = std::min(nbr, br0 + RG);
        const int nrows = (int)(br1 - br0);
        // ---- column ranges of equal modelled work
        std::vector<double> prefix(nbc + 1, 0.0);
        for (int64_t j = 0; j < nbc; ++j) {
            double c = 16.0 / G;                              // every tile is waited for and released by every warp
            for (int64_t bi = br0; bi < br1; ++bi) c += cost_of_block(bi * nbc + j);
            prefix[j + 1] = prefix[j] + c;
        }
        const double total = prefix[nbc];
        // range s ends at the first column where the running cost reaches s / S of the total, but every
        // range keeps at least one column (S <= nbc)
        std::vector<int64_t> cut(S + 1, 0);
        cut[S] = nbc;
        for (int s = 1; s < S; ++s) {
            int64_t j = cut[s - 1] + 1;
            while (j < nbc - (S - s) && prefix[j] < total * s / S) ++j;
            cut[s] = j;
        }
        for (int s = 0; s < S; ++s) {
            const int64_t j0 = cut[s], j1 = cut[s + 1];
            SpmmCta cta{};
            cta.group = (int32_t)g; cta.split = s; cta.tile0 = (int32_t)j0; cta.ntiles = (int32_t)((j1 - j0 + G - 1) / G);
            out->max_tiles = std::max<int>(out->max_tiles, cta.ntiles);
            cta_cost.push_back(prefix[j1] - prefix[j0]);
            // ---- warps per block-row in proportion to the rows' work (largest remainders; at least one each)
            std::vector<double> row_work(nrows, 0.0);
            for (int rr = 0; rr < nrows; ++rr)
                for (int64_t j = j0; j < j1; ++j) row_work[rr] += cost_of_block((br0 + rr) * nbc + j);
            double all = 0.0;
            for (double v : row_work) all += v;
            std::vector<int> nw(nrows, 1);
            int left = n_warps - nrows;
            std::vector<double> want(nrows, 0.0);
            for (int rr = 0; rr < nrows; ++rr) want[rr] = all > 0.0 ? row_work[rr] / all * n_warps : (double)n_warps / nrows;
            while (left > 0) {                                // the row whose warps carry the most so far gets the next one
                int pick = 0;
                double worst = -1.0;
                for (int rr = 0; rr < nrows; ++rr) { const double load = want[rr] / nw[rr]; if (load > worst) { worst = load; pick = rr; } }
                ++nw[pick];
                --left;
            }
            int wi = 0;
            for (int rr = 0; rr < nrows; ++rr) for (int k = 0; k < nw[rr]; ++k) cta.warp_row[wi++] = (uint8_t)rr;
            out->ctas.push_back(cta);
            // ---- the items of a row, in block-column order, to the least loaded of its warps
            int w0 = 0;
            for (int rr = 0; rr < nrows; ++rr) {
                std::vector<std::vector<PlannedItem>> per_warp(nw[rr]);
                std::vector<double> load(nw[rr], 0.0);
                for (int64_t j = j0; j < j1; ++j) {
                    const int64_t b = (br0 + rr) * nbc + j;
                    const int m = A->m[b], n = A->n[b];
                    if (!m || !n) continue;
                    const int ksl = slice_width(m);
                    for (int k0 = 0; k0 < n; k0 += ksl) {
                        const int k1 = std::min(n, k0 + ksl);
                        const int w = (int)(std::min_element(load.begin(), load.end()) - load.begin());
                        per_warp[w].push_back(PlannedItem{b, k0, k1, (int)((j - j0) / G), (int)((j - j0) % G) * A->block_c});
                        load[w] += item_cost(k1 - k0, MT, NT);
                    }
                }
                for (int k = 0; k < nw[rr]; ++k) {
                    out->stream_begin.push_back((uint32_t)out->chunks.size());
                    warp_cost.push_back(load[k]);
                    size_t start = 0, used = 0;           // the chunk being filled
                    bool open = false;
                    auto close = [&]() {
                        if (!open) return;
                        uint32_t hdr[4] = {(uint32_t)((used - 16) / 16), 0u, 0u, 0u};
                        std::memcpy(out->bytes.data() + start, hdr, 16);
                        out->chunks.push_back(Chunk{(uint32_t)(start / 16), (uint32_t)used});
                        open = false;
                    };
                    for (const PlannedItem& it : per_warp[k]) {
                        const size_t ib = spmm_item_bytes(A->m[it.block], it.k1 - it.k0);
                        if (open && used + ib > (size_t)kSpmmStageBytes) close();
                        if (!open) {
                            start = out->bytes.size();
                            out->bytes.resize(start + 16, 0);
                            used = 16;
                            open = true;
                        }
                        emit_spmm_item(A, it.block, it.k0, it.k1, it.tile, it.col_base, out->bytes);
                        used += ib;
                    }
                    close();
                }
                w0 += nw[rr];
            }
            (void)w0;
        }
    }
    out->stream_begin.push_back((uint32_t)out->chunks.size());
    // what a warp needs to run its ring: one descriptor to start from, and in every chunk's header the
    // sizes of the three chunks that follow it
    const size_t n_streams = out->stream_begin.size() - 1;
    out->warp_desc.assign(n_streams * 4, 0u);
    for (size_t w = 0; w < n_streams; ++w) {
        const uint32_t c0 = out->stream_begin[w], c1 = out->stream_begin[w + 1];
        auto bytes_of = [&](uint32_t c) { return c < c1 ? out->chunks[c].bytes : 0u; };
        out->warp_desc[4 * w] = c0 < c1 ? out->chunks[c0].off16 : 0u;
        out->warp_desc[4 * w + 1] = c1 - c0;
        out->warp_desc[4 * w + 2] = bytes_of(c0) | (bytes_of(c0 + 1) << 16);
        out->warp_desc[4 * w + 3] = bytes_of(c0 + 2);
        for (uint32_t c = c0; c < c1; ++c) {
            uint32_t next[3] = {bytes_of(c + 1), bytes_of(c + 2), bytes_of(c + 3)};
            std::memcpy(out->bytes.data() + (size_t)out->chunks[c].off16 * 16 + 4, next, 12);
        }
    }
    auto mean_over_max = [](const std::vector<double>& v) {
        double mx = 0.0, sum = 0.0;
        for (double c : v) { mx = std::max(mx, c); sum += c; }
        return mx > 0.0 ? sum / (double)v.size() / mx : 1.0;
    };
    out->balance = mean_over_max(cta_cost);
    out->warp_balance = mean_over_max(warp_cost);
    return CSB_OK;
}

}  // namespace csb
