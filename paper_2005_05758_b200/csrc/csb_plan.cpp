// One-shot planning: repack the canonical CSB arrays into the private device
// stream format and build the block -> warp schedule.
//
// The paper balances uneven kernel-matrix sizes at compile time (Section 5.2,
// Algorithm 2) for its PE-group torus.  Here the same need is met on three levels:
// the row-major sequence of blocks is cut into one contiguous, equal-cost run per
// warp of a persistent grid; large blocks are sliced so no single item dominates;
// and inside a warp the items of a chunk are dealt to the lane groups longest
// first, so the groups that run in lock-step carry about the same number of steps.
#include <algorithm>
#include <cstdio>
#include <numeric>

#include "csb_internal.hpp"

namespace csb {

static inline size_t pad_to(size_t v, size_t a) { return (v + a - 1) / a * a; }

static inline int row_words(const csb_matrix* A, int mr) {
    const int rpw = rows_per_word(A->val_dtype);
    return (mr + rpw - 1) / rpw;
}

static inline size_t item_values_offset(int nk, int mr) {
    return pad_to(sizeof(ItemHeader) + pad_to((size_t)nk, 4) + pad_to((size_t)mr, 4), kItemAlign);
}

size_t item_bytes(const csb_matrix* A, const ItemSpec& it) {
    const int nk = it.k1 - it.k0, mr = it.r1 - it.r0;
    return pad_to(item_values_offset(nk, mr) + (size_t)nk * row_words(A, mr) * 4, kItemAlign);
}

// Lock-step cost of an item for a lane group of width gw (unit: about nine instructions), from
// instruction counts of the kernel: a fixed part for header decode, gather, fold and scatter, and
// the multiply loop's iterations over quad-columns and tail columns.
enum { kItemFixedSteps = 27 };
int item_steps(const csb_matrix* A, const ItemSpec& it, int gw) {
    // about 9 instructions per unit: ~150 fixed, ~22 per quad-column iteration, ~9 per tail-column
    // iteration, ~10 per fold round
    const int nk = it.k1 - it.k0, RL = std::max(1, row_words(A, it.r1 - it.r0));
    const int S = std::max(1, gw / RL);
    int fold = 0;
    while ((1 << fold) < S) ++fold;
    const int quad_iters = ((nk >> 2) + S - 1) / S, tail_iters = ((nk & 3) + S - 1) / S;
    return (150 + 22 * quad_iters + 9 * tail_iters + 10 * fold + 4) / 9;
}

void emit_item(const csb_matrix* A, const ItemSpec& it, int gw, std::vector<uint8_t>& out) {
    const int nk = it.k1 - it.k0, mr = it.r1 - it.r0;
    const int vs = val_size(A->val_dtype), rpw = rows_per_word(A->val_dtype);
    const int RL = row_words(A, mr);
    const size_t base = out.size();
    out.resize(base + item_bytes(A, it), 0);
    uint8_t* p = out.data() + base;
    ItemHeader h{};
    h.nk = (uint8_t)nk; h.mr = (uint8_t)mr; h.RL = (uint8_t)RL; h.S = (uint8_t)(gw / std::max(RL, 1));
    h.xbase = it.xbase; h.zbase = (uint16_t)it.zbase; h.magic = (uint16_t)((1024 + RL - 1) / std::max(RL, 1));
    h.size16 = (uint16_t)(item_bytes(A, it) / 16); h.flags = (uint8_t)it.flags; h.voff16 = (uint8_t)(item_values_offset(nk, mr) / 16);
    std::memcpy(p, &h, sizeof h);
    const uint8_t* ci = A->col_idx.data() + A->cidx_off[it.block];
    const uint8_t* ri = A->row_idx.data() + A->ridx_off[it.block];
    const int n = A->n[it.block];
    const uint8_t* v = A->val.data() + A->val_off[it.block] * vs;
    uint8_t* idx = p + sizeof h;
    for (int k = 0; k < nk; ++k) idx[k] = ci[it.k0 + k];
    idx += pad_to((size_t)nk, 4);
    for (int r = 0; r < mr; ++r) idx[r] = (uint8_t)(ri[it.r0 + r] - it.ridx_bias);
    p += item_values_offset(nk, mr);
    // word (k, w) = kept rows w*rpw .. of kept column k.  Columns 4q..4q+3 are interleaved into
    // quad-words [q][w][4]; the nk % 4 columns left over follow as [k][w].
    const int nquad = nk / 4;
    auto word_at = [&](int k, int w) -> uint8_t* {
        if (k < nquad * 4) return p + ((((size_t)(k / 4) * RL + w) * 4) + (k % 4)) * 4;
        return p + ((size_t)nquad * RL * 4 + (size_t)(k - nquad * 4) * RL + w) * 4;
    };
    for (int k = 0; k < nk; ++k)
        for (int w = 0; w < RL; ++w)
            for (int q = 0; q < rpw; ++q) {
                const int r = it.r0 + w * rpw + q;
                if (r < it.r1) std::memcpy(word_at(k, w) + q * vs, v + ((size_t)r * n + it.k0 + k) * vs, vs);
            }
}

// Largest value payload of one item so that a chunk can hold one item per lane group.
int item_value_budget(int stage_bytes, int gw) {
    const int G = 32 / gw;
    return std::max(128, (stage_bytes - 16) / G - 16 - 2 * kMaxNk - 32);
}

// The narrowest lane group that still fits four out of five items without row slicing.
int pick_group_width(const std::vector<int>& item_row_words) {
    if (item_row_words.empty()) return 8;
    std::vector<int> v(item_row_words);
    const size_t q = std::min(v.size() - 1, v.size() * 4 / 5);
    std::nth_element(v.begin(), v.begin() + q, v.end());
    return v[q] <= 8 ? 8 : v[q] <= 16 ? 16 : 32;
}

// Close one chunk: deal its items to the lane groups, longest first onto the least loaded
// group, and lay the sub-streams out behind the chunk header.
static void emit_chunk(const csb_matrix* A, const std::vector<ItemSpec>& items, uint32_t zbase, uint32_t tail, int gw,
                       StreamPlan* out, double* cost) {
    const int G = 32 / gw;
    std::vector<size_t> order(items.size());
    std::iota(order.begin(), order.end(), 0);
    std::vector<int> steps(items.size());
    for (size_t i = 0; i < items.size(); ++i) steps[i] = item_steps(A, items[i], gw);
    std::stable_sort(order.begin(), order.end(), [&](size_t a, size_t b) { return steps[a] > steps[b]; });
    std::vector<std::vector<size_t>> sub(G);
    std::vector<long> load(G, 0);
    for (size_t i : order) {
        const int g = (int)(std::min_element(load.begin(), load.end()) - load.begin());
        sub[g].push_back(i);
        load[g] += steps[i];
    }
    const size_t start = out->bytes.size();
    out->bytes.resize(start + sizeof(ChunkHeader), 0);
    ChunkHeader h{};
    h.zbase = zbase; h.tail = tail;
    for (int g = 0; g < G; ++g) {
        const size_t s0 = out->bytes.size();
        for (size_t i : sub[g]) emit_item(A, items[i], gw, out->bytes);
        h.sub16[g] = (uint16_t)((out->bytes.size() - s0) / 16);
    }
    std::memcpy(out->bytes.data() + start, &h, sizeof h);
    // the flush kind rides in the top two bits of the offset, so the kernel knows it without the chunk
    out->chunks.push_back({(uint32_t)(start / 16) | ((tail & 3u) << 30), (uint32_t)(out->bytes.size() - start)});
    *cost += (double)*std::max_element(load.begin(), load.end()) + 4.0;
}

void build_stream(const csb_matrix* A, const std::vector<std::vector<Segment>>& per_warp, int stage_bytes,
                  StreamPlan* out) {
    // appends: a stream may hold the warps of several matrices (stacked layers)
    const int gw = out->group_width;
    if (!out->warp_chunk_begin.empty()) out->warp_chunk_begin.pop_back();
    for (const std::vector<Segment>& segs : per_warp) {
        out->warp_chunk_begin.push_back((uint32_t)out->chunks.size());
        double cost = 0;
        for (const Segment& sg : segs) {
            std::vector<ItemSpec> cur;
            size_t bytes = sizeof(ChunkHeader);
            for (const ItemSpec& it : sg.items) {
                const size_t ib = item_bytes(A, it);
                if (bytes + ib > (size_t)stage_bytes && !cur.empty()) {
                    emit_chunk(A, cur, sg.zbase, kFlushNone, gw, out, &cost);
                    cur.clear();
                    bytes = sizeof(ChunkHeader);
                }
                cur.push_back(it);
                bytes += ib;
            }
            if (!cur.empty() || sg.tail != kFlushNone) emit_chunk(A, cur, sg.zbase, sg.tail, gw, out, &cost);
        }
        out->warp_cost.push_back(cost);
    }
    out->warp_chunk_begin.push_back((uint32_t)out->chunks.size());
    out->n_warps = (int)out->warp_cost.size();
}

// Split one block (restricted to kept rows [r0, r1) and kept columns [k0, k1)) into items
// that respect the per-item row and column limits and a byte budget.
void slice_block(const csb_matrix* A, int64_t b, int r0, int r1, int k0, int k1, int max_rows, int value_budget,
                 ItemSpec proto, std::vector<ItemSpec>* out) {
    if (r1 <= r0 || k1 <= k0) return;
    const int nrs = (r1 - r0 + max_rows - 1) / max_rows;
    for (int s = 0; s < nrs; ++s) {
        const int ra = r0 + (int)((int64_t)(r1 - r0) * s / nrs), rb = r0 + (int)((int64_t)(r1 - r0) * (s + 1) / nrs);
        const int RL = row_words(A, rb - ra);
        const int kmax = std::min<int>(kMaxNk, std::max(1, value_budget / (RL * 4)));
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

}  // namespace csb
