// The C ABI of libcsb: argument checks, error strings, handle lifetime.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <new>

#include "csb_internal.hpp"

namespace csb {

static thread_local char g_err[512] = "";

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
}
void clear_error() { g_err[0] = 0; }

static std::atomic<uint64_t> g_uid{1};

int product_any(const csb_matrix* A, const float* X, int64_t ldx, int batch, float* Y, int64_t ldy, void* stream) {
    if (spmm_mma_applicable(A, batch)) {
        const int rc = launch_spmm_mma(A, X, ldx, batch, Y, ldy, stream);
        if (rc != 1) return rc;                       // 1: the tensor-core plan does not fit this matrix
    }
    if (batch == 1 && A->panel && A->panel->built) return launch_panels(A, X, Y, stream);
    return launch_product(A, X, ldx, batch, Y, ldy, stream);
}

int slice_block_rows(const csb_matrix* A, int64_t bi0, int64_t bi1, csb_matrix** out) {
    *out = nullptr;
    if (bi0 < 0 || bi1 > A->nbr || bi0 >= bi1) { set_error("block-row range [%lld, %lld) of %lld", (long long)bi0, (long long)bi1, (long long)A->nbr); return CSB_ERR_INVALID_ARG; }
    csb_matrix* S = new (std::nothrow) csb_matrix();
    if (!S) { set_error("out of host memory"); return CSB_ERR_ALLOC; }
    int rc = CSB_OK;
    try {
        S->rows = std::min<int64_t>(A->rows, bi1 * A->block_r) - bi0 * A->block_r; S->cols = A->cols;
        S->block_r = A->block_r; S->block_c = A->block_c; S->nbr = bi1 - bi0; S->nbc = A->nbc; S->nblk = S->nbr * S->nbc;
        S->val_dtype = A->val_dtype; S->device = A->device; S->opts = A->opts; S->uid = g_uid.fetch_add(1);
        const int64_t b0 = bi0 * A->nbc, b1 = bi1 * A->nbc;
        const int vs = val_size(A->val_dtype);
        S->m.assign(A->m.begin() + b0, A->m.begin() + b1);
        S->n.assign(A->n.begin() + b0, A->n.begin() + b1);
        S->row_idx.assign(A->row_idx.begin() + A->ridx_off[b0], A->row_idx.begin() + A->ridx_off[b1]);
        S->col_idx.assign(A->col_idx.begin() + A->cidx_off[b0], A->col_idx.begin() + A->cidx_off[b1]);
        S->val.assign(A->val.begin() + A->val_off[b0] * vs, A->val.begin() + A->val_off[b1] * vs);
        S->val_off.resize(S->nblk + 1); S->ridx_off.resize(S->nblk + 1); S->cidx_off.resize(S->nblk + 1);
        for (int64_t b = 0; b <= S->nblk; ++b) {
            S->val_off[b] = A->val_off[b0 + b] - A->val_off[b0];
            S->ridx_off[b] = A->ridx_off[b0 + b] - A->ridx_off[b0];
            S->cidx_off[b] = A->cidx_off[b0 + b] - A->cidx_off[b0];
        }
        S->nnz = (int64_t)S->val_off[S->nblk];
        rc = validate_host(S);
        if (rc == CSB_OK && S->device >= 0) { rc = plan_product(S); if (rc == CSB_OK) rc = plan_panels(S); }
    } catch (const std::bad_alloc&) { set_error("out of host memory while slicing"); rc = CSB_ERR_ALLOC; }
    if (rc != CSB_OK) { csb_free(S); return rc; }
    *out = S;
    return CSB_OK;
}

}  // namespace csb

using namespace csb;

extern "C" {

const char* csb_strerror(int status) {
    switch (status) {
        case CSB_OK: return "ok";
        case CSB_ERR_INVALID_ARG: return "invalid argument";
        case CSB_ERR_SHAPE: return "shape mismatch";
        case CSB_ERR_DTYPE: return "unknown value type";
        case CSB_ERR_ALLOC: return "allocation failed";
        case CSB_ERR_CUDA: return "CUDA runtime error";
        case CSB_ERR_LAUNCH: return "grid cannot be launched co-resident";
        case CSB_ERR_TIMEOUT: return "bounded device-side wait expired";
        case CSB_ERR_UNSUPPORTED: return "unsupported";
        default: return "unknown status";
    }
}

const char* csb_last_error(void) { return g_err; }

static int encode_common(const float* dense, int64_t rows, int64_t cols, int64_t ld, int block_r, int block_c,
                         const uint8_t* row_keep, const uint8_t* col_keep, int val_dtype, int frac_bits, int device,
                         const csb_plan_opts* opts, csb_matrix_t** out) {
    clear_error();
    if (!out) { set_error("out is NULL"); return CSB_ERR_INVALID_ARG; }
    *out = nullptr;
    if (!dense || !row_keep || !col_keep) { set_error("dense / row_keep / col_keep is NULL"); return CSB_ERR_INVALID_ARG; }
    if (rows <= 0 || cols <= 0 || ld < cols) { set_error("rows=%lld cols=%lld ld=%lld", (long long)rows, (long long)cols, (long long)ld); return CSB_ERR_INVALID_ARG; }
    if (rows > 0x7fffffff || cols > 0x7fffffff) { set_error("dimensions above 2^31-1 are not supported"); return CSB_ERR_UNSUPPORTED; }
    if (block_r < 1 || block_r > 256 || block_c < 1 || block_c > 256) { set_error("block sizes must be 1..256, got %dx%d", block_r, block_c); return CSB_ERR_INVALID_ARG; }
    if (val_dtype != CSB_F32 && val_dtype != CSB_F16 && val_dtype != CSB_Q16) { set_error("val_dtype %d", val_dtype); return CSB_ERR_DTYPE; }
    if (val_dtype == CSB_Q16 && (block_r > 128 || block_c > 128 || frac_bits < 0 || frac_bits > 30)) {
        set_error("fixed point: blocks up to 128x128 and 0..30 fraction bits, got %dx%d and %d", block_r, block_c, frac_bits);
        return CSB_ERR_INVALID_ARG;
    }
    if (device < -1) { set_error("device %d", device); return CSB_ERR_INVALID_ARG; }
    if (opts && (opts->ctas < 0 || opts->warps_per_cta < 0 || opts->warps_per_cta > 16 || opts->stages < 0 || opts->stages > 8 ||
                 (opts->stage_bytes != 0 && (opts->stage_bytes < 1024 || opts->stage_bytes > 16384)))) {
        set_error("csb_plan_opts out of range: ctas %d (>= 0), warps_per_cta %d (0..16), stage_bytes %d (0 or 1024..16384), stages %d (0..8)",
                  opts->ctas, opts->warps_per_cta, opts->stage_bytes, opts->stages);
        return CSB_ERR_INVALID_ARG;
    }
    csb_matrix* A = new (std::nothrow) csb_matrix();
    if (!A) { set_error("out of host memory"); return CSB_ERR_ALLOC; }
    A->device = device;
    A->uid = g_uid.fetch_add(1);
    A->q_frac_bits = frac_bits;
    if (opts) A->opts = *opts;
    int rc = encode_host(dense, rows, cols, ld, block_r, block_c, row_keep, col_keep, val_dtype, A);
    if (rc == CSB_OK) rc = validate_host(A);
    if (rc == CSB_OK && device >= 0) {
        try {
            if (val_dtype == CSB_Q16) rc = plan_fixed(A);
            else { rc = plan_product(A); if (rc == CSB_OK) rc = plan_panels(A); }
        }
        catch (const std::bad_alloc&) { set_error("out of host memory while planning"); rc = CSB_ERR_ALLOC; }
    }
    if (rc != CSB_OK) { csb_free(A); return rc; }
    *out = A;
    return CSB_OK;
}

int csb_encode(const float* dense, int64_t rows, int64_t cols, int64_t ld, int block_r, int block_c,
               const uint8_t* row_keep, const uint8_t* col_keep, int val_dtype, int device,
               const csb_plan_opts* opts, csb_matrix_t** out) {
    if (val_dtype == CSB_Q16) { clear_error(); set_error("fixed-point handles are made by csb_encode_q16 (it takes the fraction bits)"); return CSB_ERR_DTYPE; }
    return encode_common(dense, rows, cols, ld, block_r, block_c, row_keep, col_keep, val_dtype, 0, device, opts, out);
}

int csb_encode_q16(const float* dense, int64_t rows, int64_t cols, int64_t ld, int block_r, int block_c,
                   const uint8_t* row_keep, const uint8_t* col_keep, int frac_bits, int device, csb_matrix_t** out) {
    return encode_common(dense, rows, cols, ld, block_r, block_c, row_keep, col_keep, CSB_Q16, frac_bits, device, nullptr, out);
}

int csb_spmm_q16(const csb_matrix_t* A, const int16_t* Xq, int64_t ldx, int batch, int64_t* acc, int64_t ldy, void* stream) {
    clear_error();
    if (!A) { set_error("A is NULL"); return CSB_ERR_INVALID_ARG; }
    if (A->val_dtype != CSB_Q16) { set_error("the handle does not hold fixed-point values (make it with csb_encode_q16)"); return CSB_ERR_UNSUPPORTED; }
    if (batch < 0) { set_error("batch %d", batch); return CSB_ERR_INVALID_ARG; }
    if (batch == 0) return CSB_OK;
    if (!Xq || !acc) { set_error("Xq or acc is NULL"); return CSB_ERR_INVALID_ARG; }
    if (ldx < A->cols || ldy < A->rows) { set_error("ldx=%lld < cols or ldy=%lld < rows", (long long)ldx, (long long)ldy); return CSB_ERR_SHAPE; }
    if (A->device < 0 || !A->fixed) { set_error("matrix was encoded host-only (device = -1)"); return CSB_ERR_UNSUPPORTED; }
    return launch_fixed(A, Xq, ldx, batch, acc, ldy, stream);
}

int csb_view(const csb_matrix_t* A, csb_view_t* v) {
    clear_error();
    if (!A || !v) { set_error("NULL argument"); return CSB_ERR_INVALID_ARG; }
    v->rows = A->rows; v->cols = A->cols; v->block_r = A->block_r; v->block_c = A->block_c;
    v->nbr = A->nbr; v->nbc = A->nbc; v->nblk = A->nblk; v->nnz = A->nnz; v->val_dtype = A->val_dtype;
    v->m = A->m.data(); v->n = A->n.data(); v->row_idx = A->row_idx.data(); v->col_idx = A->col_idx.data();
    v->val_off = A->val_off.data(); v->ridx_off = A->ridx_off.data(); v->cidx_off = A->cidx_off.data();
    v->val = A->val.data();
    return CSB_OK;
}

int csb_info(const csb_matrix_t* A, csb_info_t* o) {
    clear_error();
    if (!A || !o) { set_error("NULL argument"); return CSB_ERR_INVALID_ARG; }
    const int64_t idx = (int64_t)A->ridx_off[A->nblk] + (int64_t)A->cidx_off[A->nblk];
    o->nnz = A->nnz;
    o->pruning_rate = A->nnz ? (double)A->rows * (double)A->cols / (double)A->nnz : 0.0;
    o->nio = A->nnz ? (double)idx / (double)A->nnz : 0.0;
    o->algorithmic_bytes = A->nnz * val_size(A->val_dtype) + idx + 6 * A->nblk;
    o->device_stream_bytes = A->product.stream_bytes;
    o->plan_ctas = A->product.ctas;
    o->plan_warps = A->product.warps;
    o->balance = A->product.balance;
    o->panel_stream_bytes = 0; o->panel_ctas = 0; o->panel_warps = 0; o->panel_balance = 0.0;
    if (A->panel && A->panel->built) {
        o->panel_stream_bytes = A->panel->stream_bytes; o->panel_ctas = A->panel->ctas;
        o->panel_warps = A->panel->warps; o->panel_balance = A->panel->balance;
    }
    return CSB_OK;
}

int csb_plan_dump(const csb_matrix_t* A, int ctas, int warps_per_cta, int stage_bytes, int64_t* info_out,
                  uint8_t* stream_out, int64_t stream_cap, uint32_t* chunks_out, int64_t chunks_cap,
                  uint32_t* warp_begin_out, int64_t warp_cap) {
    clear_error();
    if (!A || !info_out || ctas < 1 || warps_per_cta < 1 || warps_per_cta > 16 || stage_bytes < 1024 || (stage_bytes & 15)) {
        set_error("csb_plan_dump: bad argument");
        return CSB_ERR_INVALID_ARG;
    }
    ProductHostPlan H;
    int rc;
    try { rc = plan_product_host(A, ctas, warps_per_cta, (int64_t)ctas * warps_per_cta, stage_bytes, &H); }
    catch (const std::bad_alloc&) { set_error("out of host memory while planning"); return CSB_ERR_ALLOC; }
    if (rc != CSB_OK) return rc;
    const StreamPlan& S = H.stream;
    info_out[0] = S.n_warps; info_out[1] = (int64_t)S.chunks.size(); info_out[2] = (int64_t)S.bytes.size();
    info_out[3] = S.group_width; info_out[4] = H.row_owned; info_out[5] = H.row_owned ? H.ctas : ctas;
    info_out[6] = H.row_owned ? H.warps_per_cta : warps_per_cta; info_out[7] = H.n_slots;
    if (stream_out) {
        if (stream_cap < (int64_t)S.bytes.size()) { set_error("stream buffer too small"); return CSB_ERR_INVALID_ARG; }
        std::memcpy(stream_out, S.bytes.data(), S.bytes.size());
    }
    if (chunks_out) {
        if (chunks_cap < (int64_t)S.chunks.size()) { set_error("chunk buffer too small"); return CSB_ERR_INVALID_ARG; }
        for (size_t i = 0; i < S.chunks.size(); ++i) { chunks_out[2 * i] = S.chunks[i].off16; chunks_out[2 * i + 1] = S.chunks[i].bytes; }
    }
    if (warp_begin_out) {
        if (warp_cap < (int64_t)S.warp_chunk_begin.size()) { set_error("warp table too small"); return CSB_ERR_INVALID_ARG; }
        for (size_t i = 0; i < S.warp_chunk_begin.size(); ++i) warp_begin_out[i] = S.warp_chunk_begin[i];
    }
    return CSB_OK;
}

int csb_panel_dump(const csb_matrix_t* A, int ctas, int warps_per_cta, int stage_bytes, int64_t* info_out,
                   uint8_t* panels_out, int64_t panels_cap, uint32_t* cta_out, int64_t cta_cap) {
    clear_error();
    if (!A || !info_out || ctas < 1 || warps_per_cta < 1 || warps_per_cta > 32) { set_error("csb_panel_dump: bad argument"); return CSB_ERR_INVALID_ARG; }
    PanelHostPlan H;
    int rc;
    try { rc = plan_panels_host(A, ctas, warps_per_cta, stage_bytes, 16384, 8192 / warps_per_cta, &H); }
    catch (const std::bad_alloc&) { set_error("out of host memory while planning"); return CSB_ERR_ALLOC; }
    if (rc == 1) { set_error("the panel layout does not apply to this matrix (fp16 values, block_c <= 128, cols <= 16384, power-of-two stage >= 8192)"); return CSB_ERR_UNSUPPORTED; }
    if (rc != CSB_OK) return rc;
    info_out[0] = (int64_t)H.cta.size(); info_out[1] = (int64_t)H.bytes.size(); info_out[2] = 0;
    info_out[3] = (int64_t)H.max_meta; info_out[4] = (int64_t)H.max_xg; info_out[5] = (int64_t)H.max_rows;
    info_out[6] = (int64_t)(H.balance * 1e6); info_out[7] = (int64_t)(H.warp_balance * 1e6);
    if (panels_out) {
        if (panels_cap < (int64_t)H.bytes.size()) { set_error("panel buffer too small"); return CSB_ERR_INVALID_ARG; }
        std::memcpy(panels_out, H.bytes.data(), H.bytes.size());
    }
    if (cta_out) {
        if (cta_cap < (int64_t)H.cta.size()) { set_error("CTA table too small"); return CSB_ERR_INVALID_ARG; }
        for (size_t c = 0; c < H.cta.size(); ++c) {
            cta_out[4 * c] = H.cta[c].off16; cta_out[4 * c + 1] = H.cta[c].meta_bytes;
            cta_out[4 * c + 2] = H.cta[c].value_bytes; cta_out[4 * c + 3] = H.cta[c].n_rows;
        }
    }
    return CSB_OK;
}

void csb_free(csb_matrix_t* A) {
    if (!A) return;
    drop_cell_plans(A);
    drop_rnn_plans(A);
    free_fixed(A);
    free_mma(A);
    free_panels(A);
    free_product(A);
    delete A;
}

int csb_spmm(const csb_matrix_t* A, const float* X, int64_t ldx, int batch, float* Y, int64_t ldy, void* stream) {
    clear_error();
    if (!A) { set_error("A is NULL"); return CSB_ERR_INVALID_ARG; }
    if (batch < 0) { set_error("batch %d", batch); return CSB_ERR_INVALID_ARG; }
    if (batch == 0) return CSB_OK;
    if (!X || !Y) { set_error("X or Y is NULL"); return CSB_ERR_INVALID_ARG; }
    if (ldx < A->cols || ldy < A->rows) { set_error("ldx=%lld < cols or ldy=%lld < rows", (long long)ldx, (long long)ldy); return CSB_ERR_SHAPE; }
    if (A->device < 0) { set_error("matrix was encoded host-only (device = -1)"); return CSB_ERR_UNSUPPORTED; }
    if (A->val_dtype == CSB_Q16) { set_error("fixed-point handles serve csb_spmm_q16 only"); return CSB_ERR_UNSUPPORTED; }
    return product_any(A, X, ldx, batch, Y, ldy, stream);
}

int csb_spmv(const csb_matrix_t* A, const float* x, float* y, void* stream) {
    if (!A) { clear_error(); set_error("A is NULL"); return CSB_ERR_INVALID_ARG; }
    return csb_spmm(A, x, A->cols, 1, y, A->rows, stream);
}

}  // extern "C"
