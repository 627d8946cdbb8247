// Internal declarations shared by the host-side pieces of libcsb (encoder,
// planner, launch glue).  Nothing here is part of the public C ABI.
#pragma once

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/csb.h"

namespace csb {

// ---- error plumbing -------------------------------------------------------
void set_error(const char* fmt, ...);   // formats into the thread-local detail string
void clear_error();

// ---- device stream format -------------------------------------------------
// The private device layout is a byte stream per warp, cut into chunks that one
// bulk copy moves into shared memory.  A warp is split into G = 32 / GW lane
// groups of GW lanes (GW is fixed per stream); every group works through its own
// list of items, so G items are in flight per warp.
//
//   chunk  = ChunkHeader (16 B), then the G sub-streams back to back
//   sub-stream g = the items of lane group g, each aligned to 16 B
//   item   = ItemHeader (16 B)
//            col_idx[nk]  uint8   gather indices, relative to xbase     (padded to 4 B)
//            row_idx[mr]  uint8   scatter indices, relative to zbase    (padded to 16 B from the item's start)
//            values: a word is the kept rows of one kept column that one lane owns
//                      f16: two consecutive kept rows (half2), RL = ceil(mr/2) words per column
//                      f32: one kept row, RL = mr
//                    (padding rows inside the last word are zero); columns 4q..4q+3 are
//                    interleaved into 16-byte quad-words [q][w][4], the nk % 4 columns left
//                    over follow as plain words [k][w]                  (item padded to 16 B)
//
// The indices sit at fixed places behind the header, so a lane can ask for them (and for the
// next item's header) before it has looked at anything else of the item.
//
// An item is one block of the CSB matrix or a slice of it (a range of its kept
// rows and of its kept columns).  Column-major kernel matrices let one lane own
// the same output rows for the whole item, so a product needs no cross-lane
// reduction except across the S = GW / RL lane sub-groups that split the columns.
struct ItemHeader {
    uint8_t nk;        // kept columns in this item (<= kMaxNk)
    uint8_t mr;        // kept rows in this item (<= GW * rows per word)
    uint8_t RL;        // row words per column
    uint8_t S;         // column sub-groups, GW / RL
    uint32_t xbase;    // first column of the block in the gathered vector
    uint16_t zbase;    // first accumulator slot of the block's rows
    uint16_t magic;    // ceil(1024 / RL): lane / RL == (lane * magic) >> 10 for lane < 32
    uint16_t size16;   // size of the item in 16-byte units
    uint8_t flags;     // bit 0: columns index the recurrent (h) vector
    uint8_t voff16;    // where the values start, in 16-byte units from the item's start
};
static_assert(sizeof(ItemHeader) == 16, "header is one 16-byte word");

struct ChunkHeader {
    uint16_t sub16[4]; // size of each lane group's sub-stream in 16-byte units
    uint32_t zbase;    // product: first matrix row of the block-row this chunk belongs to
    uint32_t tail;     // bits 0..1 flush kind, bit 2 with kFlushCta: the CTA holds a piece only, bits 3.. partial-sum slot
};
static_assert(sizeof(ChunkHeader) == 16, "header is one 16-byte word");

enum : uint32_t { kFlushNone = 0, kFlushDirect = 1, kFlushPartial = 2, kFlushCta = 3, kFlushCtaPartial = 4, kSlotShift = 3 };
enum : uint16_t { kItemRecurrent = 1 };
enum { kMaxNk = 64, kItemAlign = 16 };

struct Chunk {
    uint32_t off16;    // offset of the chunk in the stream, in 16-byte units; top two bits: flush kind
    uint32_t bytes;    // multiple of 16, <= stage_bytes
};

// Host image of one planned stream (before upload).
struct StreamPlan {
    std::vector<uint8_t> bytes;            // all chunks back to back
    std::vector<Chunk> chunks;
    std::vector<uint32_t> warp_chunk_begin; // [n_warps + 1]
    std::vector<double> warp_cost;
    int n_warps = 0;
    int group_width = 32;                  // GW
};

// Planned product (SpMV / SpMM) on the device.
struct ProductPlan {
    int ctas = 0, warps = 0, stage_bytes = 0, stages = 0, group_width = 32;
    int row_owned = 0;                     // CTA-run schedule (block-rows reduced per CTA): launch shape is fixed
    int x_in_smem = 0;
    size_t smem_bytes = 0;
    uint8_t* d_stream = nullptr;
    Chunk* d_chunks = nullptr;
    void* d_warp_desc = nullptr;           // uint4 per warp: first chunk, end chunk, first chunk's off16 and bytes
    // partial block-row sums: slots [part_base[bi], part_base[bi] + part_count[bi]) belong to block-row bi
    uint32_t* d_part_base = nullptr;
    uint32_t* d_part_count = nullptr;
    uint32_t* d_arrivals = nullptr;        // [nbr], zero between launches
    float* d_partials = nullptr;           // [n_slots * block_r * max_batch_tile]
    uint32_t n_slots = 0;
    int n_warps = 0;                       // warps the stream was cut for
    uint32_t* h_status = nullptr;          // mapped host word the kernels raise on a bounded-wait expiry
    uint32_t* d_status = nullptr;
    int64_t stream_bytes = 0;
    double balance = 1.0;
};

struct Planner;                            // csb_plan.cpp
struct RnnPlan;                            // csb_rnn.cu
struct MmaPlan;                            // tensor-core SpMM plan (below)
struct PanelPlan;                          // panel layout of the batch-1 product (below)
struct FixedPlan;                          // fixed-point product (csb_fixed.cu)

}  // namespace csb

// The opaque handle of the C ABI.
struct csb_matrix {
    int64_t rows = 0, cols = 0;
    int block_r = 0, block_c = 0;
    int64_t nbr = 0, nbc = 0, nblk = 0, nnz = 0;
    int val_dtype = CSB_F16;
    int q_frac_bits = 0;                   // CSB_Q16: fraction bits of the stored values
    int device = -1;
    csb_plan_opts opts{};
    // canonical arrays (Section 3.1.1 + offsets)
    std::vector<uint16_t> m, n;
    std::vector<uint8_t> row_idx, col_idx;
    std::vector<uint64_t> val_off;
    std::vector<uint32_t> ridx_off, cidx_off;
    std::vector<uint8_t> val;              // nnz * (2 | 4) bytes
    // device side
    csb::ProductPlan product;
    mutable csb::MmaPlan* mma = nullptr;   // tensor-core SpMM plan, built lazily
    mutable std::mutex mma_mu;
    csb::PanelPlan* panel = nullptr;       // panel layout for batch 1 (fp16 values), or NULL
    csb::FixedPlan* fixed = nullptr;       // device copy of the canonical arrays (CSB_Q16 handles)
    int sm_count = 0;
    size_t smem_optin = 0;
    uint64_t uid = 0;                      // identity for the recurrent-plan cache
};

namespace csb {

inline int val_size(int dt) { return dt == CSB_F32 ? 4 : 2; }
inline int rows_per_word(int dt) { return dt == CSB_F16 ? 2 : 1; }
inline int max_item_rows(int dt) { return dt == CSB_F16 ? 64 : 32; }

// csb_encode.cpp
int encode_host(const float* dense, int64_t rows, int64_t cols, int64_t ld, int br, int bc,
                const uint8_t* row_keep, const uint8_t* col_keep, int val_dtype, csb_matrix* A);
int validate_host(const csb_matrix* A);

// csb_plan.cpp -- one item source: (block, row subset, column range)
struct ItemSpec {
    int64_t block;       // canonical block id
    int r0, r1;          // range [r0, r1) into the block's kept-row list
    int k0, k1;          // range [k0, k1) into the block's kept-column list
    uint32_t xbase, zbase;
    int ridx_bias;       // subtracted from the in-block row index before it is stored
    uint16_t flags;
};
// A run of items of one warp that ends in one action (flush of a block-row, or nothing).
struct Segment {
    std::vector<ItemSpec> items;
    uint32_t zbase = 0, tail = 0;
};
size_t item_bytes(const csb_matrix* A, const ItemSpec& it);
int item_steps(const csb_matrix* A, const ItemSpec& it, int gw);
void emit_item(const csb_matrix* A, const ItemSpec& it, int gw, std::vector<uint8_t>& out);
// Cut per-warp segment lists into chunks and append them to the stream.
void build_stream(const csb_matrix* A, const std::vector<std::vector<Segment>>& per_warp, int stage_bytes,
                  StreamPlan* out);
void slice_block(const csb_matrix* A, int64_t b, int r0, int r1, int k0, int k1, int max_rows, int value_budget,
                 ItemSpec proto, std::vector<ItemSpec>* out);
int item_value_budget(int stage_bytes, int gw);
int pick_group_width(const std::vector<int>& item_row_words);
struct ProductHostPlan {
    StreamPlan stream;
    std::vector<uint32_t> part_base, part_count;   // per block-row
    uint32_t n_slots = 0;
    double balance = 1.0;
    int row_owned = 0, ctas = 0, warps_per_cta = 0;   // row-owned mode fixes the launch shape
};
int plan_product_host(const csb_matrix* A, int ctas, int warps_per_cta, int64_t useful_warps, int stage_bytes,
                      ProductHostPlan* out);

// Recurrent time loop: one descriptor per CTA.
struct RnnCtaDesc {
    int32_t layer, u0, U;      // hidden units [u0, u0 + U) of `layer`
    uint32_t warp0;            // first of this CTA's warps in the stream's warp table
};
enum { kMaxTileUnits = 64, kMaxLayers = 8 };
struct RnnHostPlan {
    StreamPlan stream;                 // stream.group_width is chosen by the planner
    std::vector<RnnCtaDesc> ctas;
    std::vector<uint32_t> warp_in_chunks;   // per warp: chunks of input-column items (laid out first)
    int warps = 0, max_U = 0;
    size_t max_warp_bytes = 0;
    double balance = 1.0;
};
int plan_rnn_host(int gates, int n_layers, const csb_matrix* const* Wm, const int* in_size, int H, int n_ctas,
                  int warps, int stage_bytes, RnnHostPlan* out);

// ---- tensor-core SpMM path (csb_spmm_plan.cpp, csb_spmm_mma.cu) ----
// The matrix is cut into CTA tiles: a group of RG consecutive block-rows times a contiguous range of
// block-columns.  The warps of a CTA (16, or 32 for batches of up to 8) are dealt to the block-rows of its group in proportion to
// their work; a warp keeps the block_r x batch outputs of its block-row in registers for the whole
// range, and the blocks of a block-row go, in block-column order, to whichever of its warps has the
// least work so far.  A warp's weights come through its own ring of bulk copies as items; the batch
// of inputs comes through one ring of block-column tiles shared by the CTA.  An item is a column
// slice (<= 64 kept columns) of one block:
//   SpmmItemHeader (16 B), col_idx[nk] (column indices inside the input tile, padded to 4 B), then the kernel
//   matrix rows of the slice, row-major, each padded to an even number of halves (np2 words).
// Items travel in chunks of at most kSpmmStageBytes; the chunks of a warp lie back to back, and a
// chunk's 16-byte header holds the size of its items (16-byte units) and the byte sizes of the next
// three chunks of the warp, so that a warp refills its ring without looking anything up in global memory.
struct SpmmItemHeader {
    uint16_t tile;            // input tile (spmm_tile_blocks block-columns), counted from the CTA's first one
    uint8_t nk;               // kept columns in this item, 1..64
    uint8_t np2;              // 32-bit words per stored row, ceil(nk / 2)
    uint32_t mask_lo, mask_hi;   // bit r: in-block row r is kept in this block
    uint16_t size16;          // size of the item in 16-byte units
    uint16_t pad;
};
static_assert(sizeof(SpmmItemHeader) == 16, "header is one 16-byte word");
enum { kSpmmStageBytes = 2304, kSpmmMaxWarps = 32 };
struct SpmmCta {
    int32_t group, split, tile0, ntiles;     // row group, which column range of it, its first block-column, its input tiles
    uint8_t warp_row[kSpmmMaxWarps];         // which block-row of the group each warp works for (ascending)
};
static_assert(sizeof(SpmmCta) == 48, "three 16-byte words");
// Warps per CTA: the 16 accumulator registers of one 8-column batch tile leave room for 32 warps per
// SM, which halves the chain of dependent work a warp has to get through; wider tiles allow 16.
inline int spmm_warps(int NT) { return NT == 1 ? 32 : 16; }
// Batch classes: how many 8-column batch tiles a warp carries.  A pass covers 8 * NT <= 32 batch columns.
inline int spmm_nt(int batch) { return batch <= 8 ? 1 : batch <= 16 ? 2 : 4; }
inline int spmm_class_index(int batch) { return batch <= 8 ? 0 : batch <= 16 ? 1 : 2; }
inline int spmm_pitch(int NT) { return NT * 32 + 16; }   // bytes of one packed input column: hi parts, lo parts, 16 spare
// An input tile of the shared ring spans this many block-columns (at most 256 matrix columns, so that a
// column index inside a tile is one byte): fewer, larger tiles mean fewer hand-overs between the warps.
inline int spmm_tile_blocks(int block_c) { return block_c >= 256 ? 1 : std::min(4, 256 / block_c); }
struct SpmmHostPlan {
    std::vector<uint8_t> bytes;               // all chunks back to back
    std::vector<Chunk> chunks;
    std::vector<uint32_t> stream_begin;       // [n_ctas * warps + 1] first chunk of every warp's weight stream
    std::vector<uint32_t> warp_desc;          // four words per warp: first chunk's offset (16-byte units), chunk count,
                                              // bytes of chunks 0 and 1 (16 bits each), bytes of chunk 2
    std::vector<SpmmCta> ctas;
    int RG = 1, S = 1, n_groups = 0, max_tiles = 0;
    double balance = 1.0, warp_balance = 1.0; // mean / max of the modelled cost over CTAs, and over warps
};
// Plans for `sm_count` SMs; returns CSB_OK, or 1 when the path does not suit the matrix.
int plan_spmm_host(const csb_matrix* A, int NT, int sm_count, SpmmHostPlan* out);
struct MmaPlan {                           // device side, one per batch class, built on first use
    struct PerClass {
        bool built = false, unusable = false;
        int RG = 1, S = 1, n_ctas = 0, n_groups = 0, x_depth = 0, w_stages = 0;
        size_t smem_bytes = 0;
        uint8_t* d_stream = nullptr; uint32_t* d_warp_desc = nullptr; SpmmCta* d_ctas = nullptr;
        void* d_xp = nullptr;
        int64_t stream_bytes = 0;
        double balance = 1.0, warp_balance = 1.0;
    } cls[3];
};
int launch_spmm_mma(const csb_matrix* A, const float* X, int64_t ldx, int batch, float* Y, int64_t ldy, void* stream,
                    const uint8_t* packed = nullptr);
bool spmm_mma_applicable(const csb_matrix* A, int batch);
// The time loop of a recurrent stack inside the batched product kernel (csb_spmm_mma.cu): everything on the device.
struct RnnTileLoop {
    int L, B, H, gates; int64_t T;
    const csb_matrix* const* W; const float* const* bias; const int* in_size;
    const float* x; float* y;              // [T, B, I0]; [T, B, H] or null
    uint8_t* const* xp;                    // per layer: packed inputs of its product, initialised for step 0
    float* z; float* c; float* hs;         // pre-activations [rows of the product, gates * H]; c [L, B, H] (LSTM); h [L, B, H]
    unsigned int* gbar;                    // one word for the grid barrier
    int pitch, cap;
};
int launch_rnn_tile_loop(const RnnTileLoop& R, void* stream);
void free_mma(csb_matrix* A);

// ---- panel layout of the batch-1 product (csb_panel_plan.cpp, csb_panel.cu) ----
enum { kMaxPanelCtas = 192 };
struct PanelItem {          // one item: up to 32 kept rows of a block, all its kept columns
    uint32_t off16;         // where its values start in the panel's value stream, 16-byte units
    uint16_t xoff4;         // the block's gathered inputs, in units of four floats
    int16_t zoff;           // block-row's first row minus the panel's first row (may be negative)
    uint16_t roff;          // the item's row indices (in-block, one byte each) inside the panel's index bytes
    uint8_t m;              // kept rows in the item, 1..32
    uint8_t logp;           // log2 of the lane stride P, the smallest power of two >= m
    uint16_t n;             // kept columns, 1..block_c
    uint16_t pad;
};
static_assert(sizeof(PanelItem) == 16, "descriptor is one 16-byte word");
struct PanelGather {        // one block whose kept inputs the CTA gathers
    uint16_t xbase;         // first column of the block
    uint16_t n;             // kept columns
    uint32_t xoff;          // where its indices (bytes) and its gathered inputs (floats) start; multiple of 4
};
static_assert(sizeof(PanelGather) == 8, "two per 16-byte word");
struct PanelHeader {        // start of a panel's meta part; offsets are from the panel's start
    uint32_t n_items, n_gather, n_xg, n_stages;
    uint32_t value_bytes, ridx_bytes, row0, n_rows;
    uint32_t warp_off, items_off, gather_off, expect_off;
    uint32_t cidx_off, ridx_off, list_off, n_bundles;
};
static_assert(sizeof(PanelHeader) == 64, "header is four 16-byte words");
struct PanelCta { uint32_t off16, meta_bytes, value_bytes, n_rows; };
struct PanelHostPlan {
    std::vector<uint8_t> bytes;            // all panels, each aligned to 128 bytes
    std::vector<PanelCta> cta;
    int warps = 0, stage_bytes = 0;
    size_t max_meta = 0, max_xg = 0, max_rows = 0;
    double balance = 1.0, warp_balance = 1.0;
};
// Returns CSB_OK, or 1 when the matrix does not suit the panel path (the caller keeps the other one).
int plan_panels_host(const csb_matrix* A, int ctas, int warps, int stage_bytes, int max_xg_floats, int max_rows,
                     PanelHostPlan* out);
struct PanelPlan {                         // device side
    bool built = false;
    int ctas = 0, warps = 0, stage_bytes = 0, log2_ring = 0, max_rows = 0, max_xg = 0, max_meta = 0;
    size_t smem_bytes = 0;
    uint8_t* d_panels = nullptr;
    std::vector<PanelCta> cta;
    int64_t stream_bytes = 0;
    double balance = 1.0, warp_balance = 1.0;
};
int plan_panels(csb_matrix* A);            // after plan_product; leaves A->panel NULL when the path does not apply
void free_panels(csb_matrix* A);
int launch_panels(const csb_matrix* A, const float* x, float* y, void* stream);

// csb_product.cu
int plan_product(csb_matrix* A);           // plans, uploads, fills A->product
void free_product(csb_matrix* A);
int launch_product(const csb_matrix* A, const float* X, int64_t ldx, int batch, float* Y, int64_t ldy,
                   void* stream);

// csb_api.cpp
// Y[b, :] = A . X[b, :] through whichever kernel serves the batch size (what csb_spmm does after its argument checks).
int product_any(const csb_matrix* A, const float* X, int64_t ldx, int batch, float* Y, int64_t ldy, void* stream);
// A new handle (same device, planned) holding block-rows [bi0, bi1) of A; the caller frees it with csb_free.
int slice_block_rows(const csb_matrix* A, int64_t bi0, int64_t bi1, csb_matrix** out);

// csb_fixed.cu -- 16-bit fixed-point product straight from the canonical arrays
int plan_fixed(csb_matrix* A);
void free_fixed(csb_matrix* A);
int launch_fixed(const csb_matrix* A, const int16_t* Xq, int64_t ldx, int batch, int64_t* acc, int64_t ldy, void* stream);

// csb_cells.cu
void drop_cell_plans(const csb_matrix* A); // forget cached plans of the cell variants that use A

// csb_rnn.cu
void drop_rnn_plans(const csb_matrix* A);  // forget cached time-loop plans that use A

// csb_rnn_step.cu -- batch >= 16 (>= 8 for big layers): one timestep at a time, products on tensor cores
bool rnn_stepwise_wanted(int gates, int L, const csb_matrix* const* W, int B);
int rnn_forward_stepwise(int gates, int L, const csb_matrix* const* W, const float* const* bias, const float* x, int64_t T, int B, int H,
                         const int* in_size, const float* h0, const float* c0, float* y, float* hT, float* cT, unsigned flags,
                         void* stream);            // 1: a layer's tensor-core plan does not fit, nothing visible was written
void drop_step_plans(const csb_matrix* A);

}  // namespace csb
