// Planner of the tensor-core SpMM path (batch >= 8, fp16 values): its own stream layout, in
// which every kernel matrix is cut into 16 x 8 tiles (kept rows x kept columns, zero padded)
// stored in the register order of mma.sync.m16n8k8's A operand, so that one 8-byte load per lane
// fetches a lane's share of a tile.  Scheduling is row-owned: a CTA owns whole block-rows, its
// warps share the items and their private sums are joined in shared memory behind a CTA barrier.
#include <algorithm>
#include <numeric>

#include "csb_internal.hpp"

namespace csb {

static inline size_t pad_to(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct MmaItem {
    int64_t block;
    int r0, r1, k0, k1;
    uint32_t xbase;
};

static size_t mma_item_bytes(const MmaItem& it) {
    const int nk = it.k1 - it.k0, mr = it.r1 - it.r0;
    const int RT = (mr + 15) / 16, KT = (nk + 7) / 8;
    return pad_to(sizeof(MmaItemHeader) + pad_to((size_t)nk, 4) + pad_to((size_t)mr, 4), 16) + (size_t)RT * KT * 256;
}

static uint16_t half_bits(const csb_matrix* A, int64_t block, int r, int k) {
    uint16_t h;
    std::memcpy(&h, A->val.data() + (A->val_off[block] + (size_t)r * A->n[block] + k) * 2, 2);
    return h;
}

static void emit_mma_item(const csb_matrix* A, const MmaItem& it, std::vector<uint8_t>& out) {
    const int nk = it.k1 - it.k0, mr = it.r1 - it.r0;
    const int RT = (mr + 15) / 16, KT = (nk + 7) / 8;
    const size_t base = out.size();
    out.resize(base + mma_item_bytes(it), 0);
    uint8_t* p = out.data() + base;
    MmaItemHeader h{};
    h.nk = (uint8_t)nk; h.mr = (uint8_t)mr; h.RT = (uint8_t)RT; h.KT = (uint8_t)KT; h.xbase = it.xbase;
    std::memcpy(p, &h, sizeof h);
    uint8_t* q = p + sizeof h;
    const uint8_t* ci = A->col_idx.data() + A->cidx_off[it.block];
    const uint8_t* ri = A->row_idx.data() + A->ridx_off[it.block];
    for (int k = 0; k < nk; ++k) q[k] = ci[it.k0 + k];
    q += pad_to((size_t)nk, 4);
    for (int r = 0; r < mr; ++r) q[r] = ri[it.r0 + r];
    uint8_t* tiles = p + pad_to(sizeof(MmaItemHeader) + pad_to((size_t)nk, 4) + pad_to((size_t)mr, 4), 16);
    // tile (rt, kt), lane l = 4*g + t holds a0 = {W[g][2t], W[g][2t+1]}, a1 = {W[g+8][2t], W[g+8][2t+1]}
    for (int rt = 0; rt < RT; ++rt)
        for (int kt = 0; kt < KT; ++kt) {
            uint8_t* tile = tiles + ((size_t)rt * KT + kt) * 256;
            for (int l = 0; l < 32; ++l) {
                const int g = l / 4, t = l % 4;
                for (int half = 0; half < 2; ++half)
                    for (int e = 0; e < 2; ++e) {
                        const int r = rt * 16 + g + 8 * half, k = kt * 8 + 2 * t + e;
                        const uint16_t v = (r < mr && k < nk) ? half_bits(A, it.block, it.r0 + r, it.k0 + k) : (uint16_t)0;
                        std::memcpy(tile + l * 8 + half * 4 + e * 2, &v, 2);
                    }
            }
        }
}

int plan_mma_host(const csb_matrix* A, int ctas, int warps_per_cta, int stage_bytes, MmaHostPlan* out) {
    const int tile_budget = std::max(1, (stage_bytes - 16 - 16 - 128) / 256);     // tiles per item
    // items per block-row
    std::vector<std::vector<MmaItem>> row_items(A->nbr);
    std::vector<double> row_cost(A->nbr, 0.0);
    auto cost_of = [](const MmaItem& it) { return (double)(((it.r1 - it.r0 + 15) / 16) * ((it.k1 - it.k0 + 7) / 8)) + 6.0; };
    for (int64_t bi = 0; bi < A->nbr; ++bi)
        for (int64_t bj = 0; bj < A->nbc; ++bj) {
            const int64_t b = bi * A->nbc + bj;
            const int m = A->m[b], n = A->n[b];
            if (!m || !n) continue;
            const int nrs = (m + 63) / 64;
            for (int s = 0; s < nrs; ++s) {
                const int ra = (int)((int64_t)m * s / nrs), rb = (int)((int64_t)m * (s + 1) / nrs);
                const int RT = (rb - ra + 15) / 16;
                const int kmax = std::min<int>(kMmaMaxNk, std::max(8, tile_budget / RT * 8));
                const int nks = (n + kmax - 1) / kmax;
                for (int q = 0; q < nks; ++q) {
                    MmaItem it{b, ra, rb, (int)((int64_t)n * q / nks), (int)((int64_t)n * (q + 1) / nks), (uint32_t)(bj * A->block_c)};
                    // column slices start on multiples of 8 where possible, so no tile is split
                    row_items[bi].push_back(it);
                    row_cost[bi] += cost_of(it);
                }
            }
        }
    const int n_ctas = (int)std::min<int64_t>(ctas, A->nbr);
    std::vector<int64_t> order(A->nbr);
    std::iota(order.begin(), order.end(), (int64_t)0);
    std::stable_sort(order.begin(), order.end(), [&](int64_t x, int64_t y) { return row_cost[x] > row_cost[y]; });
    std::vector<double> cta_load(n_ctas, 0.0);
    std::vector<std::vector<int64_t>> cta_rows(n_ctas);
    for (int64_t bi : order) {
        const int c = (int)(std::min_element(cta_load.begin(), cta_load.end()) - cta_load.begin());
        cta_rows[c].push_back(bi);
        cta_load[c] += row_cost[bi] / warps_per_cta + 20.0;
    }
    out->ctas = n_ctas; out->warps_per_cta = warps_per_cta;
    out->warp_chunk_begin.clear();
    for (int c = 0; c < n_ctas; ++c) {
        // per warp, per block-row: a list of items (dealt longest first)
        std::vector<std::vector<std::vector<MmaItem>>> per_warp(warps_per_cta, std::vector<std::vector<MmaItem>>(cta_rows[c].size()));
        for (size_t ri = 0; ri < cta_rows[c].size(); ++ri) {
            std::vector<MmaItem> items = row_items[cta_rows[c][ri]];
            std::stable_sort(items.begin(), items.end(), [&](const MmaItem& x, const MmaItem& y) { return cost_of(x) > cost_of(y); });
            std::vector<double> load(warps_per_cta, 0.0);
            for (const MmaItem& it : items) {
                const int w = (int)(std::min_element(load.begin(), load.end()) - load.begin());
                per_warp[w][ri].push_back(it);
                load[w] += cost_of(it);
            }
        }
        for (int w = 0; w < warps_per_cta; ++w) {
            out->warp_chunk_begin.push_back((uint32_t)out->chunks.size());
            for (size_t ri = 0; ri < cta_rows[c].size(); ++ri) {
                const uint32_t zbase = (uint32_t)(cta_rows[c][ri] * A->block_r);
                const std::vector<MmaItem>& items = per_warp[w][ri];
                size_t i = 0;
                do {
                    // one chunk: header + as many items as fit a ring stage
                    const size_t start = out->bytes.size();
                    out->bytes.resize(start + sizeof(ChunkHeader), 0);
                    size_t bytes = sizeof(ChunkHeader);
                    while (i < items.size() && (bytes + mma_item_bytes(items[i]) <= (size_t)stage_bytes || bytes == sizeof(ChunkHeader))) {
                        bytes += mma_item_bytes(items[i]);
                        emit_mma_item(A, items[i], out->bytes);
                        ++i;
                    }
                    const bool last = i >= items.size();
                    ChunkHeader h{};
                    h.sub16[0] = (uint16_t)((out->bytes.size() - start - sizeof(ChunkHeader)) / 16);
                    h.zbase = zbase; h.tail = last ? (uint32_t)kFlushCta : (uint32_t)kFlushNone;
                    std::memcpy(out->bytes.data() + start, &h, sizeof h);
                    out->chunks.push_back({(uint32_t)(start / 16) | ((h.tail & 3u) << 30), (uint32_t)(out->bytes.size() - start)});
                    out->max_chunk_bytes = std::max<size_t>(out->max_chunk_bytes, out->bytes.size() - start);
                } while (i < items.size());
            }
        }
    }
    out->warp_chunk_begin.push_back((uint32_t)out->chunks.size());
    double mx = 0, sum = 0;
    for (double l : cta_load) { mx = std::max(mx, l); sum += l; }
    out->balance = mx > 0 ? sum / ctas / mx : 1.0;
    return CSB_OK;
}

}  // namespace csb
