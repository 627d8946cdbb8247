// Block -> warp schedules for the two kernels (host side, run once per matrix / stack).
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>

#include "csb_internal.hpp"

namespace csb {

static int env_gw() {
    const char* v = getenv("CSB_GROUP_WIDTH");
    const int g = v && *v ? atoi(v) : 0;
    return (g == 8 || g == 16 || g == 32) ? g : 0;
}

// Schedule for the bare product: walk the blocks in row-major order, give every warp of
// the persistent grid one contiguous, equal-cost run of items, and mark the end of each
// block-row inside a warp with how its accumulators leave the warp: straight to y when the
// warp owns the whole block-row, else as a partial sum in its own slot.
int plan_product_host(const csb_matrix* A, int ctas, int warps_per_cta, int64_t useful_warps, int stage_bytes,
                      ProductHostPlan* out) {
    int n_warps = (int)std::min<int64_t>((int64_t)ctas * warps_per_cta, std::max<int64_t>(1, useful_warps));
    const int rpw = rows_per_word(A->val_dtype);
    std::vector<int> rl;
    rl.reserve(A->nblk);
    for (int64_t b = 0; b < A->nblk; ++b)
        if (A->m[b] && A->n[b]) rl.push_back((A->m[b] + rpw - 1) / rpw);
    const int gw = env_gw() ? env_gw() : pick_group_width(rl);
    out->stream.group_width = gw;
    const int value_budget = item_value_budget(stage_bytes, gw);
    std::vector<ItemSpec> items;
    std::vector<int64_t> item_row;                      // block-row of each item; -1 items are placeholders
    std::vector<char> placeholder;
    for (int64_t bi = 0; bi < A->nbr; ++bi) {
        const size_t before = items.size();
        for (int64_t bj = 0; bj < A->nbc; ++bj) {
            const int64_t b = bi * A->nbc + bj;
            ItemSpec proto{};
            proto.xbase = (uint32_t)(bj * A->block_c);
            slice_block(A, b, 0, A->m[b], 0, A->n[b], gw * rpw, value_budget, proto, &items);
        }
        const bool empty = items.size() == before;
        if (empty) items.push_back(ItemSpec{});         // nothing kept: the block-row still owes zeros to y
        item_row.resize(items.size(), bi);
        placeholder.resize(items.size(), empty ? 1 : 0);
    }
    std::vector<double> cost(items.size());
    double total = 0;
    for (size_t i = 0; i < items.size(); ++i) { cost[i] = placeholder[i] ? 4.0 : (double)item_steps(A, items[i], gw); total += cost[i]; }

    // Row-owned mode: with about as many block-rows as CTAs (or more), a block-row belongs to ONE
    // CTA, whose warps share its items and add their sums up in shared memory behind a CTA
    // barrier: no partial sums in global memory, no fences, no arrival counters.  Only a
    // block-row so heavy that it alone would set the run time is divided into pieces for several
    // CTAs; each piece leaves its CTA as one partial sum, and the CTA that arrives last adds them.
    const char* ro_env = getenv("CSB_ROW_OWNED");
    const bool row_owned = ro_env && *ro_env ? atoi(ro_env) != 0 : (A->nbr * 5 >= (int64_t)ctas * 4 && n_warps >= ctas);
    if (row_owned) {
        const int G = 32 / gw;
        const int n_ctas = ctas;
        // warps per CTA: enough lane groups for the items of a typical block-row, no more
        const double items_per_row = (double)items.size() / (double)A->nbr;
        const int wpc = std::max(1, std::min(warps_per_cta, (int)(items_per_row / G / 2.0 + 0.999)));
        // Costs in the time of one CTA (its items spread over wpc * G lane groups): a piece also
        // costs a barrier and a reduction, a divided block-row the round trips of the exchange.
        const double kFlush = 16.0, kExchange = 70.0;
        const char* split_env = getenv("CSB_ROW_SPLIT");
        const bool may_split = !(split_env && *split_env && atoi(split_env) == 0);
        const double bins = (double)wpc * G;
        std::vector<size_t> row_begin(A->nbr + 1, items.size());
        std::vector<double> row_cost(A->nbr, 0.0);
        for (size_t i = items.size(); i-- > 0;) { row_cost[item_row[i]] += cost[i] / bins; row_begin[item_row[i]] = i; }
        struct Piece { int64_t row; int k, of; double cost; };
        auto make_pieces = [&](double T, std::vector<Piece>* out_pieces) {
            out_pieces->clear();
            for (int64_t bi = 0; bi < A->nbr; ++bi) {
                int p = 1;
                const double room = T - kFlush - kExchange;
                if (may_split && row_cost[bi] + kFlush > T && room > 0) p = (int)std::ceil(row_cost[bi] / room);
                const int n_items = (int)(row_begin[bi + 1] - row_begin[bi]);
                p = std::max(1, std::min(p, std::min(n_items, 64)));
                for (int k = 0; k < p; ++k)
                    out_pieces->push_back({bi, k, p, row_cost[bi] / p + kFlush + (p > 1 ? kExchange : 0.0)});
            }
        };
        auto pack = [&](const std::vector<Piece>& pcs, std::vector<int>* where) {
            // heaviest piece first onto the least loaded CTA; returns the largest load
            std::vector<size_t> order(pcs.size());
            for (size_t i = 0; i < order.size(); ++i) order[i] = i;
            std::stable_sort(order.begin(), order.end(), [&](size_t x, size_t y) { return pcs[x].cost > pcs[y].cost; });
            std::vector<double> load(n_ctas, 0.0);
            where->assign(pcs.size(), 0);
            for (size_t i : order) {
                const int c = (int)(std::min_element(load.begin(), load.end()) - load.begin());
                (*where)[i] = c;
                load[c] += pcs[i].cost;
            }
            return *std::max_element(load.begin(), load.end());
        };
        // the target time T decides which block-rows are divided; try a ladder of targets between
        // the even share and the heaviest block-row and keep the best packing
        double sum_cost = 0, max_cost = 0;
        for (double c : row_cost) { sum_cost += c + kFlush; max_cost = std::max(max_cost, c + kFlush); }
        const double lo = std::max(sum_cost / n_ctas, 1.0);
        std::vector<Piece> pieces, best_pieces;
        std::vector<int> where, best_where;
        double best = -1, undivided = 0;
        for (int step = 0; step <= 24; ++step) {
            // step 0 divides nothing; a division has to pay for itself with some margin
            const double T = max_cost <= lo ? max_cost : lo * std::pow(max_cost / lo, (24 - step) / 24.0);
            make_pieces(T, &pieces);
            const double mk = pack(pieces, &where);
            if (step == 0) undivided = mk;
            if (getenv("CSB_PLAN_DEBUG")) fprintf(stderr, "T=%.1f pieces=%zu makespan=%.1f lo=%.1f max=%.1f\n", T, pieces.size(), mk, lo, max_cost);
            if (best < 0 || (mk < best && mk < 0.95 * undivided)) { best = mk; best_pieces = pieces; best_where = where; }
            if (max_cost <= lo) break;
        }
        // slots of the divided block-rows
        out->part_base.assign(A->nbr, 0);
        out->part_count.assign(A->nbr, 0);
        uint32_t slots = 0;
        for (const Piece& pc : best_pieces)
            if (pc.of > 1 && pc.k == 0) { out->part_base[pc.row] = slots; out->part_count[pc.row] = (uint32_t)pc.of; slots += (uint32_t)pc.of; }
        out->n_slots = slots;
        // per CTA: its pieces, divided ones first (their partner may be waiting), then by row
        std::vector<std::vector<size_t>> cta_pieces(n_ctas);
        int n_used = 1;                                          // the packing fills CTAs from the front
        for (size_t i = 0; i < best_pieces.size(); ++i) { cta_pieces[best_where[i]].push_back(i); n_used = std::max(n_used, best_where[i] + 1); }
        std::vector<std::vector<Segment>> per_warp((size_t)n_used * wpc);
        std::vector<double> cta_load(n_ctas, 0.0);
        for (int c = 0; c < n_used; ++c) {
            std::stable_sort(cta_pieces[c].begin(), cta_pieces[c].end(), [&](size_t x, size_t y) {
                return (best_pieces[x].of > 1) > (best_pieces[y].of > 1);
            });
            for (size_t pi : cta_pieces[c]) {
                const Piece& pc = best_pieces[pi];
                cta_load[c] += pc.cost;
                const int64_t bi = pc.row;
                // the piece's items: a contiguous range of the block-row, cut by cost
                std::vector<size_t> idx;
                {
                    double cum = 0;
                    const double tot = row_cost[bi] * bins;
                    for (size_t i = row_begin[bi]; i < row_begin[bi + 1]; ++i) {
                        const int k = tot > 0 ? std::min(pc.of - 1, (int)((cum + 0.5 * cost[i]) / tot * pc.of)) : 0;
                        if (k == pc.k && !placeholder[i]) idx.push_back(i);
                        cum += cost[i];
                    }
                }
                const uint32_t tail = pc.of > 1 ? (kFlushCta | kFlushCtaPartial | ((out->part_base[bi] + (uint32_t)pc.k) << kSlotShift))
                                                : (uint32_t)kFlushCta;
                std::stable_sort(idx.begin(), idx.end(), [&](size_t x, size_t y) { return cost[x] > cost[y]; });
                std::vector<double> load((size_t)wpc * G, 0.0);
                for (int w = 0; w < wpc; ++w) {
                    per_warp[(size_t)c * wpc + w].emplace_back();
                    Segment& sg = per_warp[(size_t)c * wpc + w].back();
                    sg.zbase = (uint32_t)(bi * A->block_r);
                    sg.tail = tail;
                }
                for (size_t i : idx) {
                    const int bin = (int)(std::min_element(load.begin(), load.end()) - load.begin());
                    per_warp[(size_t)c * wpc + bin / G].back().items.push_back(items[i]);
                    load[bin] += cost[i];
                }
            }
        }
        out->row_owned = 1; out->ctas = n_used; out->warps_per_cta = wpc;
        build_stream(A, per_warp, stage_bytes, &out->stream);
        double mx = 0, sum = 0;
        for (double l : cta_load) { mx = std::max(mx, l); sum += l; }
        out->balance = mx > 0 ? sum / n_ctas / mx : 1.0;         // idle CTAs count against the balance
        return CSB_OK;
    }

    std::vector<std::vector<Segment>> per_warp(n_warps);
    const double target = total / n_warps;
    double cum = 0;
    for (size_t i = 0; i < items.size(); ++i) {
        int w = (int)((cum + 0.5 * cost[i]) / target);
        w = std::min(std::max(w, 0), n_warps - 1);
        std::vector<Segment>& segs = per_warp[w];
        const uint32_t zb = (uint32_t)(item_row[i] * A->block_r);
        if (segs.empty() || segs.back().zbase != zb) { segs.emplace_back(); segs.back().zbase = zb; }
        if (!placeholder[i]) segs.back().items.push_back(items[i]);
        cum += cost[i];
    }
    // contributors per block-row, in warp order
    out->part_base.assign(A->nbr, 0);
    out->part_count.assign(A->nbr, 0);
    std::vector<uint32_t> contributors(A->nbr, 0);
    for (auto& segs : per_warp)
        for (auto& sg : segs) contributors[sg.zbase / A->block_r]++;
    uint32_t slots = 0;
    for (int64_t bi = 0; bi < A->nbr; ++bi)
        if (contributors[bi] > 1) { out->part_base[bi] = slots; out->part_count[bi] = contributors[bi]; slots += contributors[bi]; }
    out->n_slots = slots;
    std::vector<uint32_t> next_slot(out->part_base);
    for (auto& segs : per_warp)
        for (auto& sg : segs) {
            const int64_t bi = sg.zbase / A->block_r;
            sg.tail = contributors[bi] > 1 ? (kFlushPartial | (next_slot[bi]++ << kSlotShift)) : (uint32_t)kFlushDirect;
        }
    build_stream(A, per_warp, stage_bytes, &out->stream);
    double mx = 0, sum = 0;
    for (double c : out->stream.warp_cost) { mx = std::max(mx, c); sum += c; }
    out->balance = mx > 0 ? sum / n_warps / mx : 1.0;
    return CSB_OK;
}

// Schedule for the recurrent time loop.  Every CTA owns a tile of hidden units of one layer
// together with ALL gate rows of those units (rows u, H+u, 2H+u, ...), so the gate arithmetic
// needs no data from other CTAs and one grid-wide barrier per step is enough.  CTAs are shared
// out between the layers in proportion to their stored weights (the layers run as a
// wavefront: layer l works on step t while layer l+1 works on step t-1); unit tiles and the
// warps inside a CTA are cut by cost, not by count.
int plan_rnn_host(int gates, int n_layers, const csb_matrix* const* Wm, const int* in_size, int H, int n_ctas,
                  int warps, int stage_bytes, RnnHostPlan* out) {
    out->warps = warps;
    out->max_U = 0;
    // every layer gets enough CTAs for its tiles to stay under the unit limit; the rest are
    // shared out by stored weights
    const int floor_ctas = std::min(H, (H + 47) / 48);
    std::vector<int> ncta(n_layers, floor_ctas);
    {
        if (floor_ctas * n_layers > n_ctas) {
            set_error("%d layers of hidden size %d need %d CTAs, %d available", n_layers, H, floor_ctas * n_layers, n_ctas);
            return CSB_ERR_UNSUPPORTED;
        }
        double tot = 0;
        for (int l = 0; l < n_layers; ++l) tot += (double)Wm[l]->nnz + 1.0;
        const int spare = n_ctas - floor_ctas * n_layers;
        for (int l = 0; l < n_layers; ++l)
            ncta[l] = std::min(H, floor_ctas + (int)((double)spare * ((double)Wm[l]->nnz + 1.0) / tot));
    }
    // unit tiles per layer: contiguous, about equal stored weights
    std::vector<std::vector<int>> cuts(n_layers);
    for (int l = 0; l < n_layers; ++l) {
        const csb_matrix* A = Wm[l];
        std::vector<double> rowcost(A->rows, 0.0);
        for (int64_t b = 0; b < A->nblk; ++b) {
            const int64_t bi = b / A->nbc;
            const uint8_t* ri = A->row_idx.data() + A->ridx_off[b];
            for (int r = 0; r < A->m[b]; ++r) rowcost[bi * A->block_r + ri[r]] += A->n[b] + 2.0;
        }
        std::vector<double> ucost(H, 8.0);
        for (int g = 0; g < gates; ++g)
            for (int u = 0; u < H; ++u) ucost[u] += rowcost[(int64_t)g * H + u];
        double tot = 0;
        for (double c : ucost) tot += c;
        std::vector<int>& cut = cuts[l];
        // A tile that straddles two block-rows gets twice the items of one that does not, and the
        // fixed cost per item is what dominates small items.  So when the gates' block-rows line
        // up with the units (H a multiple of the block height) and there are at least as many
        // CTAs as block-rows, every block-row is cut into the same number of tiles, by cost, and
        // no tile straddles.  Otherwise: contiguous tiles of about equal cost.
        const int BR = A->block_r, nbr_g = (H + BR - 1) / BR;
        const int per_row = ncta[l] / nbr_g;
        if (H % BR == 0 && per_row >= 1 && BR / per_row <= kMaxTileUnits && per_row <= BR) {
            cut.assign(1, 0);
            for (int bi = 0; bi < nbr_g; ++bi) {
                double rtot = 0, cum = 0;
                for (int u = bi * BR; u < (bi + 1) * BR; ++u) rtot += ucost[u];
                int t = 1;
                for (int u = bi * BR; u < (bi + 1) * BR && t < per_row; ++u) {
                    cum += ucost[u];
                    const int left_units = (bi + 1) * BR - (u + 1), left_tiles = per_row - t;
                    const bool full = u + 1 - cut.back() >= kMaxTileUnits;
                    if (cum >= rtot * t / per_row || left_units <= left_tiles || full) { cut.push_back(u + 1); ++t; }
                }
                cut.push_back((bi + 1) * BR);
            }
            ncta[l] = (int)cut.size() - 1;
        } else {
            cut.assign(ncta[l] + 1, H);
            cut[0] = 0;
            double cum = 0;
            int t = 1;
            for (int u = 0; u < H && t < ncta[l]; ++u) {
                cum += ucost[u];
                const int left_units = H - (u + 1), left_tiles = ncta[l] - t;
                const bool full = u + 1 - cut[t - 1] >= kMaxTileUnits;
                if (cum >= tot * t / ncta[l] || left_units <= left_tiles || full) cut[t++] = u + 1;
            }
        }
        for (int c = 0; c < ncta[l]; ++c) {
            const int U = cut[c + 1] - cut[c];
            if (U > kMaxTileUnits) {
                set_error("hidden size %d over %d CTAs gives tiles of %d units (limit %d)", H, ncta[l], U, (int)kMaxTileUnits);
                return CSB_ERR_UNSUPPORTED;
            }
            out->max_U = std::max(out->max_U, U);
        }
    }
    // items of one CTA (layer l, units [u0, u1)) for a given lane-group width
    auto tile_items = [&](int l, int u0, int u1, int gw, std::vector<ItemSpec>* items, std::vector<int>* rl) {
        const csb_matrix* A = Wm[l];
        const int I = in_size[l], U = u1 - u0, rpw = rows_per_word(A->val_dtype);
        const int max_rows = gw * rpw, value_budget = item_value_budget(stage_bytes, gw);
        for (int g = 0; g < gates; ++g) {
            const int64_t row0 = (int64_t)g * H + u0, row1 = (int64_t)g * H + u1;
            for (int64_t bi = row0 / A->block_r; bi <= (row1 - 1) / A->block_r; ++bi) {
                const int lo = (int)std::max<int64_t>(0, row0 - bi * A->block_r);
                const int hi = (int)std::min<int64_t>(A->block_r, row1 - bi * A->block_r);
                for (int64_t bj = 0; bj < A->nbc; ++bj) {
                    const int64_t b = bi * A->nbc + bj;
                    const uint8_t* ri = A->row_idx.data() + A->ridx_off[b];
                    const uint8_t* ci = A->col_idx.data() + A->cidx_off[b];
                    const int m = A->m[b], n = A->n[b];
                    const int r0 = (int)(std::lower_bound(ri, ri + m, lo) - ri);
                    const int r1 = (int)(std::lower_bound(ri, ri + m, hi) - ri);
                    if (rl) { if (r1 > r0 && n) rl->push_back((r1 - r0 + rpw - 1) / rpw); continue; }
                    const int64_t split_col = (int64_t)I - bj * A->block_c;      // first recurrent column, block-local
                    const int ks = split_col <= 0 ? 0 : split_col >= A->block_c ? n
                                   : (int)(std::lower_bound(ci, ci + n, (int)split_col) - ci);
                    ItemSpec proto{};
                    proto.ridx_bias = (int)(row0 - bi * A->block_r);
                    proto.xbase = (uint32_t)(bj * A->block_c);
                    proto.zbase = (uint32_t)(g * U);
                    slice_block(A, b, r0, r1, 0, ks, max_rows, value_budget, proto, items);
                    proto.xbase = (uint32_t)(bj * A->block_c - I);                 // may wrap; col_idx brings it back
                    proto.flags = kItemRecurrent;
                    if (gates == 3 && g == 2) proto.zbase = (uint32_t)(3 * U);     // GRU candidate gate, hidden part
                    slice_block(A, b, r0, r1, ks, n, max_rows, value_budget, proto, items);
                }
            }
        }
    };
    // lane-group width from the row counts the tiles actually see
    std::vector<int> rl;
    for (int l = 0; l < n_layers; ++l)
        for (int c = 0; c < ncta[l]; c += std::max(1, ncta[l] / 8)) tile_items(l, cuts[l][c], cuts[l][c + 1], 32, nullptr, &rl);
    const int gw = env_gw() ? env_gw() : pick_group_width(rl);
    out->stream.group_width = gw;
    double cost_sum = 0, cost_max = 0;
    for (int l = 0; l < n_layers; ++l) {
        const csb_matrix* A = Wm[l];
        for (int c = 0; c < ncta[l]; ++c) {
            const int u0 = cuts[l][c], u1 = cuts[l][c + 1];
            std::vector<ItemSpec> items;
            tile_items(l, u0, u1, gw, &items, nullptr);
            // warps of this CTA: items dealt longest first to the least loaded warp (any warp may
            // take any item: accumulators are private and added in a fixed order afterwards).
            // Input-column items and recurrent-column items are dealt separately and laid out as
            // two segments per warp, input first: the kernel walks them at different times.
            std::vector<std::vector<Segment>> per_warp(warps, std::vector<Segment>(2));
            for (int w = 0; w < warps; ++w) per_warp[w][1].zbase = 1;       // chunk tag: 0 input, 1 recurrent
            double total = 0;
            std::vector<double> cost(items.size());
            for (size_t i = 0; i < items.size(); ++i) { cost[i] = (double)item_steps(A, items[i], gw); total += cost[i]; }
            for (int part = 0; part < 2; ++part) {
                std::vector<size_t> order;
                for (size_t i = 0; i < items.size(); ++i)
                    if (((items[i].flags & kItemRecurrent) != 0) == (part == 1)) order.push_back(i);
                std::stable_sort(order.begin(), order.end(), [&](size_t x, size_t y) { return cost[x] > cost[y]; });
                // bins are lane groups (G per warp): equal item counts per group matter as much as
                // equal cost, because the groups of a warp advance in lock-step rounds
                const int G = 32 / gw;
                std::vector<double> load((size_t)warps * G, 0.0);
                for (size_t i : order) {
                    const int bin = (int)(std::min_element(load.begin(), load.end()) - load.begin());
                    per_warp[bin / G][part].items.push_back(items[i]);
                    load[bin] += cost[i];
                }
            }
            const size_t first_chunk = out->stream.chunks.size();
            RnnCtaDesc d{l, u0, u1 - u0, (uint32_t)out->stream.n_warps};
            build_stream(A, per_warp, stage_bytes, &out->stream);
            out->ctas.push_back(d);
            // how many chunks of each warp carry the input tag
            for (int w = 0; w < warps; ++w) {
                uint32_t n_in = 0;
                const uint32_t cb = out->stream.warp_chunk_begin[d.warp0 + w], ce = out->stream.warp_chunk_begin[d.warp0 + w + 1];
                for (uint32_t c = cb; c < ce; ++c) {
                    ChunkHeader h;
                    std::memcpy(&h, out->stream.bytes.data() + (size_t)out->stream.chunks[c].off16 * 16, sizeof h);
                    if (h.zbase == 0) ++n_in;
                }
                out->warp_in_chunks.push_back(n_in);
            }
            (void)first_chunk;
            cost_sum += total;
            cost_max = std::max(cost_max, total);
        }
    }
    out->max_warp_bytes = 0;
    for (int w = 0; w < out->stream.n_warps; ++w) {
        size_t bytes = 0;
        for (uint32_t c = out->stream.warp_chunk_begin[w]; c < out->stream.warp_chunk_begin[w + 1]; ++c) bytes += out->stream.chunks[c].bytes;
        out->max_warp_bytes = std::max(out->max_warp_bytes, bytes);
    }
    out->balance = cost_max > 0 ? cost_sum / out->ctas.size() / cost_max : 1.0;
    return CSB_OK;
}

}  // namespace csb
