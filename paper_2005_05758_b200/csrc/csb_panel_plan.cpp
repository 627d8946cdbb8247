// Host planner of the panel layout: the device form of a CSB matrix that the batch-1
// product (SpMV) streams.
//
// The paper's CSB-Engine walks the blocks of a matrix in row-major order and hides their
// uneven sizes with compile-time workload sharing (Sections 4.3.1, 5.2).  Here the output
// rows are cut into one contiguous range per CTA of a persistent grid, of about equal modelled
// cost, and a CTA gets everything that lands in its rows: of every block that has kept rows in
// the range, those rows with all the block's kept columns.  Ranges do not follow block-row
// borders (a block-row's kept rows may go to two or more CTAs), so every output row is written
// by exactly one CTA and nothing has to be joined across CTAs.  What a CTA streams is a *panel*:
//
//   meta    PanelHeader, per-warp item ranges, item descriptors, gather descriptors, per-stage
//           item counts, column indices, row indices
//   values  the kernel-matrix rows of the panel's items back to back, fetched by the CTA in
//           fixed-size stages through one shared-memory ring
//
// An item is at most 32 kept rows of one block with all its kept columns.  Its values are the
// canonical row-major kernel-matrix rows re-tiled so that a lane reads 16 bytes = 8 consecutive
// kept columns of one kept row: [octet o][row r][8], then the 4-, 2- and 1-column remainders
// as [r][4], [r][2], [r][1].  No padding inside an item; items are padded to 16 bytes.
//
// The gathered input of a block (its kept columns of x) is built once per CTA in shared
// memory, so the multiply loop reads it with vector loads.  A panel's items are laid out
// longest first and dealt to the CTA's warps in that order, each to the warp with the least
// work so far; the deal is part of the plan, so the summation order is fixed.
#include <algorithm>
#include <cstdlib>

#include "csb_internal.hpp"

namespace csb {

static inline size_t pad_to(size_t v, size_t a) { return (v + a - 1) / a * a; }
static inline int log2_ceil(int v) { int l = 0; while ((1 << l) < v) ++l; return l; }

// How many items of this height share a warp: one with more than 16 rows, two with 9..16, four
// with 8 or fewer (log2 of that number).
static inline int panel_item_logg(int mi) { return mi > 16 ? 0 : mi > 8 ? 1 : 2; }
// Loop steps of an item: its column octets divided among the lane sub-groups of its lane group.
static inline int panel_item_steps(int mi, int n) {
    const int gw = 32 >> panel_item_logg(mi), S = gw >> log2_ceil(mi);
    return ((n >> 3) + S - 1) / S;
}
// Modelled time of a bundle: a fixed part, and per member its loop steps, remainder columns and
// joining shuffles.  The shape follows the kernel's instruction counts (110 fixed, 28 per step), but
// the two weights are fitted to measured times of the 8192 x 8192 sweep: what a CTA's time follows is
// the number of its bundles far more than their length (with the instruction counts as weights the
// CTAs of one product finished between 5.1 and 8.2 us after their gather; 4x: 11.2 -> 10.35 us,
// 8x: 8.3 -> 7.65, 25x: 6.0 -> 5.75 with the fitted ones).  CSB_PANEL_COST_FIXED / _STEP override them.
static const double kPanelBundleFixed = getenv("CSB_PANEL_COST_FIXED") ? atof(getenv("CSB_PANEL_COST_FIXED")) : 55.0;
static const double kPanelStep = getenv("CSB_PANEL_COST_STEP") ? atof(getenv("CSB_PANEL_COST_STEP")) : 4.0;
static double panel_member_cost(int mi, int n) {
    const int gw = 32 >> panel_item_logg(mi), S = gw >> log2_ceil(mi);
    return kPanelStep * panel_item_steps(mi, n) + ((n & 7) ? 34.0 : 0.0) + 8.0 * log2_ceil(S);
}
// Cost of an item as seen by the row cut: its share of a bundle.
static double panel_item_cost(int mi, int n) {
    return (kPanelBundleFixed + panel_member_cost(mi, n)) / (double)(1 << panel_item_logg(mi)) + 10.0;
}

struct PanelItemSrc {
    int64_t block;
    int r0, mi;            // kept-row range [r0, r0 + mi) of the block's kept-row list
    size_t bytes;          // padded value bytes
    double cost;
    uint32_t xoff;         // the block's place in the gathered inputs
};

int plan_panels_host(const csb_matrix* A, int ctas, int warps, int stage_bytes, int max_xg_floats, int max_rows,
                     PanelHostPlan* out) {
    *out = PanelHostPlan{};
    if (A->val_dtype != CSB_F16) return 1;
    if (A->block_c > 128 || A->cols > 16384) return 1;
    if (stage_bytes < 8192 || (stage_bytes & (stage_bytes - 1))) return 1;
    const int BR = A->block_r, BC = A->block_c;

    // ---- which blocks keep a given output row (blocks without kept columns store nothing)
    std::vector<uint32_t> rb_begin(A->rows + 1, 0);
    size_t total_bytes = 0;
    for (int64_t b = 0; b < A->nblk; ++b) {
        const int m = A->m[b], n = A->n[b];
        if (m == 0 || n == 0) continue;
        const uint8_t* ri = A->row_idx.data() + A->ridx_off[b];
        for (int r = 0; r < m; ++r) ++rb_begin[(b / A->nbc) * BR + ri[r] + 1];
        total_bytes += (size_t)m * n * 2;
    }
    for (int64_t r = 0; r < A->rows; ++r) rb_begin[r + 1] += rb_begin[r];
    std::vector<uint32_t> rb(rb_begin[A->rows]);
    {
        std::vector<uint32_t> fill(rb_begin.begin(), rb_begin.end() - 1);
        for (int64_t b = 0; b < A->nblk; ++b) {
            const int m = A->m[b], n = A->n[b];
            if (m == 0 || n == 0) continue;
            const uint8_t* ri = A->row_idx.data() + A->ridx_off[b];
            for (int r = 0; r < m; ++r) rb[fill[(b / A->nbc) * BR + ri[r]]++] = (uint32_t)b;
        }
    }
    int n_ctas = (int)std::min<int64_t>(ctas, std::max<int64_t>(1, (int64_t)total_bytes / 8192));
    n_ctas = (int)std::min<int64_t>(std::min<int64_t>(n_ctas, (int64_t)kMaxPanelCtas), A->rows);

    // ---- one contiguous row range per CTA.  The cost of a range is the cost of its items, and an
    // item's fixed part is paid again by every CTA that holds rows of the block, so the cost is
    // followed row by row: rows are packed into a CTA until a limit T would be passed, and T is
    // the smallest limit (by bisection) that needs no more than n_ctas CTAs.
    std::vector<uint16_t> cnt(A->nblk, 0);                 // rows of the block in the CTA being filled
    auto block_cost = [&](int m, int n) { double c = 0.0; for (int r0 = 0; r0 < m; r0 += 32) c += panel_item_cost(std::min(32, m - r0), n); return c; };
    auto pack = [&](double T, std::vector<int64_t>* cuts, double* worst) -> int {
        int used = 1;
        double cur = 0.0;
        *worst = 0.0;
        int64_t start = 0;
        if (cuts) { cuts->assign(1, 0); }
        auto reset = [&](int64_t from, int64_t to) { for (int64_t r = from; r < to; ++r) for (uint32_t i = rb_begin[r]; i < rb_begin[r + 1]; ++i) cnt[rb[i]] = 0; };
        for (int64_t r = 0; r < A->rows; ++r) {
            double delta = 0.0;
            for (uint32_t i = rb_begin[r]; i < rb_begin[r + 1]; ++i) { const uint32_t b = rb[i]; delta += block_cost(cnt[b] + 1, A->n[b]) - block_cost(cnt[b], A->n[b]); }
            if ((cur > 0.0 && cur + delta > T) || r - start >= max_rows) {
                *worst = std::max(*worst, cur);
                reset(start, r);
                start = r; cur = 0.0; ++used;
                if (cuts) cuts->push_back(r);
                delta = 0.0;
                for (uint32_t i = rb_begin[r]; i < rb_begin[r + 1]; ++i) delta += block_cost(1, A->n[rb[i]]);
            }
            for (uint32_t i = rb_begin[r]; i < rb_begin[r + 1]; ++i) ++cnt[rb[i]];
            cur += delta;
        }
        *worst = std::max(*worst, cur);
        reset(start, A->rows);
        if (cuts) cuts->push_back(A->rows);
        return used;
    };
    std::vector<int64_t> cut;
    {
        double worst = 0.0, lo = 0.0, hi = 0.0;
        pack(1e300, nullptr, &hi);                         // everything in one CTA: an upper bound
        hi = std::max(hi, 1.0);
        for (int it = 0; it < 40 && hi - lo > 1e-3 * hi; ++it) {
            const double mid = 0.5 * (lo + hi);
            if (pack(mid, nullptr, &worst) <= n_ctas) hi = mid; else lo = mid;
        }
        n_ctas = pack(hi, &cut, &worst);
        if (n_ctas > (int)kMaxPanelCtas) return 1;        // only when max_rows forces more ranges than the grid has
    }

    out->warps = warps;
    out->stage_bytes = stage_bytes;
    out->cta.resize(n_ctas);
    double max_cta_cost = 0.0, max_warp_cost = 0.0, sum_cta_cost = 0.0;
    for (int c = 0; c < n_ctas; ++c) {
        const int64_t R0 = cut[c], R1 = cut[c + 1];
        if (R1 - R0 > max_rows) return 1;
        std::vector<PanelItemSrc> items;
        std::vector<PanelItem> desc;
        std::vector<PanelGather> gath;
        std::vector<uint8_t> cidx, ridx, values;
        for (int64_t bi = R0 / BR; bi < A->nbr && bi * BR < R1; ++bi) {
            const int lo = (int)std::max<int64_t>(0, R0 - bi * BR), hi = (int)std::min<int64_t>(BR, R1 - bi * BR);   // in-block rows [lo, hi)
            for (int64_t bj = 0; bj < A->nbc; ++bj) {
                const int64_t b = bi * A->nbc + bj;
                const int m = A->m[b], n = A->n[b];
                if (m == 0 || n == 0) continue;
                const uint8_t* ri = A->row_idx.data() + A->ridx_off[b];
                const int ra = (int)(std::lower_bound(ri, ri + m, lo) - ri), rb = (int)(std::lower_bound(ri, ri + m, hi) - ri);
                if (ra == rb) continue;
                PanelGather g{};
                g.xbase = (uint16_t)(bj * BC); g.n = (uint16_t)n; g.xoff = (uint32_t)cidx.size();
                gath.push_back(g);
                const uint8_t* ci = A->col_idx.data() + A->cidx_off[b];
                cidx.insert(cidx.end(), ci, ci + n);
                while (cidx.size() & 3) cidx.push_back(0);
                for (int r0 = ra; r0 < rb; r0 += 32) {
                    PanelItemSrc it{};
                    it.block = b; it.r0 = r0; it.mi = std::min(32, rb - r0);
                    it.bytes = pad_to((size_t)it.mi * n * 2, 16);
                    it.cost = panel_item_cost(it.mi, n);
                    it.xoff = g.xoff;
                    items.push_back(it);
                }
            }
        }
        if (items.size() > 0x3fff) return 1;
        // ---- bundles: items of 16 or fewer rows go through a warp two at a time, of 8 or fewer
        // four at a time (each on its own group of lanes), so the fixed work per item is shared.
        // Members of a bundle are picked with about the same number of loop steps.
        struct Bundle { std::vector<uint32_t> members; int logg; double cost; size_t bytes; };
        std::vector<Bundle> bundles;
        for (int logg = 0; logg <= 2; ++logg) {
            std::vector<uint32_t> cls;
            for (uint32_t i = 0; i < items.size(); ++i) if (panel_item_logg(items[i].mi) == logg) cls.push_back(i);
            std::stable_sort(cls.begin(), cls.end(), [&](uint32_t x, uint32_t y) {
                return panel_item_steps(items[x].mi, A->n[items[x].block]) > panel_item_steps(items[y].mi, A->n[items[y].block]); });
            for (size_t k = 0; k < cls.size(); k += (size_t)1 << logg) {
                Bundle bu{};
                bu.logg = logg;
                double worst = 0.0;
                for (size_t j = k; j < std::min(cls.size(), k + ((size_t)1 << logg)); ++j) {
                    bu.members.push_back(cls[j]);
                    bu.bytes += items[cls[j]].bytes;
                    worst = std::max(worst, panel_member_cost(items[cls[j]].mi, A->n[items[cls[j]].block]));
                }
                bu.cost = kPanelBundleFixed + worst + 10.0 * (double)bu.members.size();
                bundles.push_back(std::move(bu));
            }
        }
        // longest first, then packed into stages (first fit), so that no bundle straddles a stage
        std::stable_sort(bundles.begin(), bundles.end(), [](const Bundle& x, const Bundle& y) { return x.cost > y.cost; });
        std::vector<std::vector<uint32_t>> stage_of;          // bundles of every stage, in placement order
        std::vector<size_t> fill;
        for (uint32_t k = 0; k < bundles.size(); ++k) {
            if (bundles[k].bytes > (size_t)stage_bytes) return 1;
            size_t st = 0;
            while (st < fill.size() && fill[st] + bundles[k].bytes > (size_t)stage_bytes) ++st;
            if (st == fill.size()) { fill.push_back(0); stage_of.emplace_back(); }
            fill[st] += bundles[k].bytes;
            stage_of[st].push_back(k);
        }
        const size_t n_stages = fill.size();
        std::vector<uint16_t> expect(n_stages, 0);
        // emit the values stage by stage and deal the bundles, in stream order, to the least loaded warp
        std::vector<double> load(warps, 0.0);
        std::vector<std::vector<uint32_t>> per_warp(warps);
        desc.assign(items.size(), PanelItem{});
        for (size_t st = 0; st < n_stages; ++st) {
            values.resize(st * (size_t)stage_bytes, 0);         // the previous stage is padded to its end
            expect[st] = (uint16_t)stage_of[st].size();
            for (uint32_t k : stage_of[st]) {
                const int w = (int)(std::min_element(load.begin(), load.end()) - load.begin());
                per_warp[w].push_back(k);
                load[w] += bundles[k].cost;
                for (uint32_t i : bundles[k].members) {
                    const PanelItemSrc& it = items[i];
                    const int64_t b = it.block, bi = b / A->nbc;
                    const int n = A->n[b];
                    const uint8_t* ri = A->row_idx.data() + A->ridx_off[b];
                    PanelItem& d = desc[i];
                    d.off16 = (uint32_t)(values.size() / 16);
                    d.xoff4 = (uint16_t)(it.xoff / 4);
                    d.zoff = (int16_t)(bi * BR - R0);
                    d.roff = (uint16_t)ridx.size();
                    d.m = (uint8_t)it.mi; d.logp = (uint8_t)log2_ceil(it.mi);
                    d.n = (uint16_t)n; d.pad = 0;
                    ridx.insert(ridx.end(), ri + it.r0, ri + it.r0 + it.mi);
                    // values: [octet][row][8], then [row][4], [row][2], [row][1]
                    const uint8_t* v = A->val.data() + (A->val_off[b] + (uint64_t)it.r0 * n) * 2;
                    const size_t base = values.size();
                    values.resize(base + it.bytes, 0);
                    uint8_t* p = values.data() + base;
                    const int noct = n >> 3;
                    for (int o = 0; o < noct; ++o)
                        for (int r = 0; r < it.mi; ++r, p += 16) std::memcpy(p, v + ((size_t)r * n + 8 * o) * 2, 16);
                    int kk = noct * 8;
                    for (int w2 = 4; w2 >= 1; w2 >>= 1)
                        if (n & w2) {
                            for (int r = 0; r < it.mi; ++r, p += 2 * w2) std::memcpy(p, v + ((size_t)r * n + kk) * 2, 2 * w2);
                            kk += w2;
                        }
                }
            }
        }
        if (cidx.size() > (size_t)max_xg_floats || cidx.size() / 4 > 0xffff || ridx.size() > 0xffff || values.size() / 16 > 0xffffffffull)
            return 1;                                            // beyond the kernel's limits: the caller keeps the other path
        double cta_cost = 0.0;
        for (int w = 0; w < warps; ++w) { cta_cost += load[w]; max_warp_cost = std::max(max_warp_cost, load[w]); }
        sum_cta_cost += cta_cost;
        max_cta_cost = std::max(max_cta_cost, cta_cost);
        // descriptors in the order the warps take them: a bundle's members side by side, missing
        // members as empty descriptors (no rows, no columns) that point at the bundle's stage
        std::vector<PanelItem> table;
        std::vector<uint16_t> wlist, wbegin(warps + 1, 0);
        for (int w = 0; w < warps; ++w) {
            wbegin[w] = (uint16_t)wlist.size();
            for (uint32_t k : per_warp[w]) {
                const Bundle& bu = bundles[k];
                if (table.size() > 0x3fff - 4) return 1;
                wlist.push_back((uint16_t)(table.size() | ((size_t)bu.logg << 14)));
                for (int g = 0; g < (1 << bu.logg); ++g) {
                    if (g < (int)bu.members.size()) { table.push_back(desc[bu.members[g]]); continue; }
                    PanelItem e{};
                    e.off16 = desc[bu.members[0]].off16;
                    e.logp = (uint8_t)(5 - bu.logg);
                    table.push_back(e);
                }
            }
        }
        wbegin[warps] = (uint16_t)wlist.size();
        if (wlist.size() > 0xffff) return 1;

        // ---- emit the panel
        PanelHeader h{};
        h.n_items = (uint32_t)table.size(); h.n_bundles = (uint32_t)wlist.size(); h.n_gather = (uint32_t)gath.size(); h.n_xg = (uint32_t)cidx.size();
        h.n_stages = (uint32_t)n_stages; h.value_bytes = (uint32_t)values.size(); h.ridx_bytes = (uint32_t)ridx.size();
        h.row0 = (uint32_t)R0; h.n_rows = (uint32_t)(R1 - R0);
        size_t off = sizeof(PanelHeader);
        h.warp_off = (uint32_t)off; off = pad_to(off + (size_t)(warps + 1) * 2, 16);
        h.list_off = (uint32_t)off; off = pad_to(off + wlist.size() * 2, 16);
        h.items_off = (uint32_t)off; off += (size_t)h.n_items * sizeof(PanelItem);
        h.gather_off = (uint32_t)off; off = pad_to(off + gath.size() * sizeof(PanelGather), 16);
        h.expect_off = (uint32_t)off; off = pad_to(off + n_stages * 2, 16);
        h.cidx_off = (uint32_t)off; off = pad_to(off + cidx.size(), 16);
        h.ridx_off = (uint32_t)off; off = pad_to(off + ridx.size(), 128);
        const size_t meta_bytes = off;
        const size_t base = pad_to(out->bytes.size(), 128);
        out->bytes.resize(base + meta_bytes + pad_to(values.size(), 128), 0);
        uint8_t* p = out->bytes.data() + base;
        std::memcpy(p, &h, sizeof h);
        std::memcpy(p + h.warp_off, wbegin.data(), wbegin.size() * 2);
        if (!wlist.empty()) std::memcpy(p + h.list_off, wlist.data(), wlist.size() * 2);
        if (!table.empty()) std::memcpy(p + h.items_off, table.data(), table.size() * sizeof(PanelItem));
        if (!gath.empty()) std::memcpy(p + h.gather_off, gath.data(), gath.size() * sizeof(PanelGather));
        if (n_stages) std::memcpy(p + h.expect_off, expect.data(), n_stages * 2);
        if (!cidx.empty()) std::memcpy(p + h.cidx_off, cidx.data(), cidx.size());
        if (!ridx.empty()) std::memcpy(p + h.ridx_off, ridx.data(), ridx.size());
        if (!values.empty()) std::memcpy(p + meta_bytes, values.data(), values.size());
        PanelCta& ct = out->cta[c];
        ct.off16 = (uint32_t)(base / 16); ct.meta_bytes = (uint32_t)meta_bytes; ct.value_bytes = (uint32_t)values.size();
        ct.n_rows = (uint32_t)(R1 - R0);
        out->max_meta = std::max(out->max_meta, meta_bytes);
        out->max_xg = std::max(out->max_xg, cidx.size());
        out->max_rows = std::max<size_t>(out->max_rows, (size_t)(R1 - R0));
    }
    if (out->bytes.size() / 16 > 0xffffffffull) return 1;
    out->balance = max_cta_cost > 0.0 ? (sum_cta_cost / n_ctas) / max_cta_cost : 1.0;
    out->warp_balance = max_warp_cost > 0.0 ? (sum_cta_cost / ((double)n_ctas * warps)) / max_warp_cost : 1.0;
    return CSB_OK;
}

}  // namespace csb
