// One-shot planning: repack the canonical CSB arrays into the private device
// stream format and build the block -> warp schedule.
//
// The paper balances uneven kernel-matrix sizes at compile time (Section 5.2,
// Algorithm 2) for its PE-group torus.  Here the same need is met by cutting the
// row-major sequence of blocks into one contiguous, equal-cost segment per warp
// of a persistent grid; large blocks are sliced so no single item dominates.
#include <algorithm>
#include <cstdio>

#include "csb_internal.hpp"

namespace csb {

static inline size_t pad_to(size_t v, size_t a) { return (v + a - 1) / a * a; }

size_t item_bytes(const csb_matrix* A, const ItemSpec& it) {
    const int nk = it.k1 - it.k0, mr = it.r1 - it.r0;
    const int rpw = rows_per_word(A->val_dtype);
    const int RL = (mr + rpw - 1) / rpw;
    return pad_to(sizeof(ItemHeader) + pad_to((size_t)nk + mr, 4) + (size_t)nk * RL * 4, kItemAlign);
}

void emit_item(const csb_matrix* A, const ItemSpec& it, std::vector<uint8_t>& out) {
    const int nk = it.k1 - it.k0, mr = it.r1 - it.r0;
    const int vs = val_size(A->val_dtype), rpw = rows_per_word(A->val_dtype);
    const int RL = (mr + rpw - 1) / rpw;
    const size_t base = out.size();
    out.resize(base + item_bytes(A, it), 0);
    uint8_t* p = out.data() + base;
    ItemHeader h{(uint16_t)nk, (uint16_t)mr, it.xbase, it.zbase, it.tail};
    std::memcpy(p, &h, sizeof h);
    p += sizeof h;
    if (it.block >= 0) {
        const uint8_t* ci = A->col_idx.data() + A->cidx_off[it.block];
        const uint8_t* ri = A->row_idx.data() + A->ridx_off[it.block];
        for (int k = 0; k < nk; ++k) p[k] = ci[it.k0 + k];
        for (int r = 0; r < mr; ++r) p[nk + r] = (uint8_t)(ri[it.r0 + r] - it.ridx_bias);
        p += pad_to((size_t)nk + mr, 4);
        const int n = A->n[it.block];
        const uint8_t* v = A->val.data() + A->val_off[it.block] * vs;
        for (int k = 0; k < nk; ++k)
            for (int w = 0; w < RL; ++w)
                for (int q = 0; q < rpw; ++q) {
                    const int r = it.r0 + w * rpw + q;
                    if (r < it.r1) std::memcpy(p + (((size_t)k * RL + w) * rpw + q) * vs,
                                               v + ((size_t)r * n + it.k0 + k) * vs, vs);
                }
    }
}

void build_stream(const csb_matrix* A, const std::vector<std::vector<ItemSpec>>& per_warp,
                  int stage_bytes, StreamPlan* out) {
    // appends: a stream may hold the warps of several matrices (stacked layers)
    if (!out->warp_chunk_begin.empty()) out->warp_chunk_begin.pop_back();
    for (size_t w = 0; w < per_warp.size(); ++w) {
        out->warp_chunk_begin.push_back((uint32_t)out->chunks.size());
        size_t chunk_start = out->bytes.size();
        double cost = 0;
        for (const ItemSpec& it : per_warp[w]) {
            const size_t ib = item_bytes(A, it);
            if (out->bytes.size() - chunk_start + ib > (size_t)stage_bytes && out->bytes.size() > chunk_start) {
                out->chunks.push_back({(uint32_t)(chunk_start / 16), (uint32_t)(out->bytes.size() - chunk_start)});
                chunk_start = out->bytes.size();
            }
            emit_item(A, it, out->bytes);
            cost += (double)ib + 48.0;
        }
        if (out->bytes.size() > chunk_start)
            out->chunks.push_back({(uint32_t)(chunk_start / 16), (uint32_t)(out->bytes.size() - chunk_start)});
        out->warp_cost.push_back(cost);
    }
    out->warp_chunk_begin.push_back((uint32_t)out->chunks.size());
    out->n_warps = (int)out->warp_cost.size();
}

// Split one block (restricted to kept rows [r0, r1)) into items that respect the
// per-item row and column limits and a byte budget.
void slice_block(const csb_matrix* A, int64_t b, int r0, int r1, int k0, int k1, int value_budget,
                 ItemSpec proto, std::vector<ItemSpec>* out) {
    const int rpw = rows_per_word(A->val_dtype), maxr = max_item_rows(A->val_dtype);
    if (r1 <= r0 || k1 <= k0) return;
    const int nrs = (r1 - r0 + maxr - 1) / maxr;
    for (int s = 0; s < nrs; ++s) {
        const int ra = r0 + (int)((int64_t)(r1 - r0) * s / nrs), rb = r0 + (int)((int64_t)(r1 - r0) * (s + 1) / nrs);
        const int RL = (rb - ra + rpw - 1) / rpw;
        int kmax = std::min<int>(kMaxNk, std::max(1, value_budget / (RL * 4)));
        const int nks = (k1 - k0 + kmax - 1) / kmax;
        for (int q = 0; q < nks; ++q) {
            ItemSpec it = proto;
            it.block = b; it.r0 = ra; it.r1 = rb;
            it.k0 = k0 + (int)((int64_t)(k1 - k0) * q / nks);
            it.k1 = k0 + (int)((int64_t)(k1 - k0) * (q + 1) / nks);
            out->push_back(it);
        }
    }
}

// Schedule for the bare product: walk the blocks in row-major order, give every warp of
// the persistent grid one contiguous, equal-cost run of items, and tag the last item a
// warp holds of each block-row with how its accumulators leave the warp: straight to y
// when the warp owns the whole block-row, else as a partial sum in its own slot.
int plan_product_host(const csb_matrix* A, int n_warps, int stage_bytes, ProductHostPlan* out) {
    const int value_budget = std::max(256, std::min(2048, stage_bytes - 16 - 2 * kMaxNk - 64));
    std::vector<ItemSpec> items;
    std::vector<int64_t> item_row;                      // block-row of each item
    for (int64_t bi = 0; bi < A->nbr; ++bi) {
        const size_t before = items.size();
        for (int64_t bj = 0; bj < A->nbc; ++bj) {
            const int64_t b = bi * A->nbc + bj;
            ItemSpec proto{};
            proto.xbase = (uint32_t)(bj * A->block_c);
            proto.zbase = (uint32_t)(bi * A->block_r);
            slice_block(A, b, 0, A->m[b], 0, A->n[b], value_budget, proto, &items);
        }
        if (items.size() == before) {                   // nothing kept: still owes zeros to y
            ItemSpec e{};
            e.block = -1;
            e.zbase = (uint32_t)(bi * A->block_r);
            items.push_back(e);
        }
        item_row.resize(items.size(), bi);
    }
    std::vector<double> cost(items.size());
    double total = 0;
    for (size_t i = 0; i < items.size(); ++i) { cost[i] = (double)item_bytes(A, items[i]) + 48.0; total += cost[i]; }
    std::vector<std::vector<ItemSpec>> per_warp(n_warps);
    std::vector<std::vector<int64_t>> rows_of(n_warps);
    const double target = total / n_warps;
    double cum = 0;
    for (size_t i = 0; i < items.size(); ++i) {
        int w = (int)((cum + 0.5 * cost[i]) / target);
        w = std::min(std::max(w, 0), n_warps - 1);
        per_warp[w].push_back(items[i]);
        rows_of[w].push_back(item_row[i]);
        cum += cost[i];
    }
    // contributors per block-row, in warp order
    out->part_base.assign(A->nbr, 0);
    out->part_count.assign(A->nbr, 0);
    std::vector<uint32_t> contributors(A->nbr, 0);
    for (int w = 0; w < n_warps; ++w)
        for (size_t i = 0; i < rows_of[w].size(); ++i)
            if (i + 1 == rows_of[w].size() || rows_of[w][i + 1] != rows_of[w][i]) contributors[rows_of[w][i]]++;
    uint32_t slots = 0;
    for (int64_t bi = 0; bi < A->nbr; ++bi)
        if (contributors[bi] > 1) { out->part_base[bi] = slots; out->part_count[bi] = contributors[bi]; slots += contributors[bi]; }
    out->n_slots = slots;
    std::vector<uint32_t> next_slot(out->part_base);
    for (int w = 0; w < n_warps; ++w)
        for (size_t i = 0; i < rows_of[w].size(); ++i)
            if (i + 1 == rows_of[w].size() || rows_of[w][i + 1] != rows_of[w][i]) {
                const int64_t bi = rows_of[w][i];
                per_warp[w][i].tail = contributors[bi] > 1 ? (kFlushPartial | (next_slot[bi]++ << kSlotShift))
                                                           : (uint32_t)kFlushDirect;
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
    // CTAs per layer
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
    const int value_budget = std::max(256, std::min(2048, stage_bytes - 16 - 2 * kMaxNk - 64));
    double cost_sum = 0, cost_max = 0;
    for (int l = 0; l < n_layers; ++l) {
        const csb_matrix* A = Wm[l];
        const int I = in_size[l];
        // cost of every matrix row = stored weights in it
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
        // contiguous unit tiles of about equal cost
        std::vector<int> cut(ncta[l] + 1, H);
        cut[0] = 0;
        {
            double cum = 0;
            int t = 1;
            for (int u = 0; u < H && t < ncta[l]; ++u) {
                cum += ucost[u];
                const int left_units = H - (u + 1), left_tiles = ncta[l] - t;
                const bool full = u + 1 - cut[t - 1] >= kMaxTileUnits;
                if (cum >= tot * t / ncta[l] || left_units <= left_tiles || full) { cut[t++] = u + 1; }
            }
        }
        for (int c = 0; c < ncta[l]; ++c) {
            const int u0 = cut[c], u1 = cut[c + 1];
            const int U = u1 - u0;
            if (U > kMaxTileUnits) {
                set_error("hidden size %d over %d CTAs gives tiles of %d units (limit %d)", H, ncta[l], U, kMaxTileUnits);
                return CSB_ERR_UNSUPPORTED;
            }
            out->max_U = std::max(out->max_U, U);
            std::vector<ItemSpec> items;
            for (int g = 0; g < gates && U > 0; ++g) {
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
                        const int64_t split_col = (int64_t)I - bj * A->block_c;      // first recurrent column, block-local
                        const int ks = split_col <= 0 ? 0 : split_col >= A->block_c ? n
                                       : (int)(std::lower_bound(ci, ci + n, (int)split_col) - ci);
                        ItemSpec proto{};
                        proto.ridx_bias = (int)(row0 - bi * A->block_r);
                        proto.xbase = (uint32_t)(bj * A->block_c);
                        proto.zbase = (uint32_t)(g * U);
                        slice_block(A, b, r0, r1, 0, ks, value_budget, proto, &items);
                        proto.xbase = (uint32_t)(bj * A->block_c - I);                 // may wrap; col_idx brings it back
                        proto.tail = kSrcRecurrent;
                        if (gates == 3 && g == 2) proto.zbase = (uint32_t)(3 * U);     // GRU candidate gate, hidden part
                        slice_block(A, b, r0, r1, ks, n, value_budget, proto, &items);
                    }
                }
            }
            // warps of this CTA: contiguous runs of about equal cost
            std::vector<std::vector<ItemSpec>> per_warp(warps);
            double total = 0;
            std::vector<double> cost(items.size());
            for (size_t i = 0; i < items.size(); ++i) { cost[i] = (double)item_bytes(A, items[i]) + 48.0; total += cost[i]; }
            double cum = 0;
            for (size_t i = 0; i < items.size(); ++i) {
                int w = total > 0 ? (int)((cum + 0.5 * cost[i]) / (total / warps)) : 0;
                per_warp[std::min(std::max(w, 0), warps - 1)].push_back(items[i]);
                cum += cost[i];
            }
            RnnCtaDesc d{l, u0, U, (uint32_t)out->stream.n_warps};
            build_stream(A, per_warp, stage_bytes, &out->stream);
            out->ctas.push_back(d);
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
