// Host-side CSB encoder and validator (Section 3.1.1 of the paper).
//
// From a dense weight and per-block row / column keep masks it writes the five
// arrays of the format -- kernel-matrix sizes m{}, n{}, kept-line indices
// RowIdx{}, ColIdx{} and the concatenated kernel matrices Val{} -- plus the
// prefix-sum offsets that random access needs and the paper's sequential
// hardware does without.
#include <cmath>
#include <cstdio>
#include <new>

#include "csb_internal.hpp"

namespace csb {

// binary32 -> binary16, round to nearest, ties to even; overflow gives infinity,
// values below half the smallest subnormal give (signed) zero, NaN stays NaN.
static uint16_t f32_to_f16_rne(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    const uint32_t sign = (u >> 16) & 0x8000u;
    const uint32_t absu = u & 0x7fffffffu;
    if (absu >= 0x7f800000u)                      // inf / NaN
        return (uint16_t)(sign | 0x7c00u | (absu > 0x7f800000u ? 0x0200u | ((absu >> 13) & 0x3ffu) : 0u));
    if (absu >= 0x477ff000u)                      // >= 65520: rounds to infinity
        return (uint16_t)(sign | 0x7c00u);
    if (absu < 0x38800000u) {                     // below 2^-14: subnormal half or zero
        if (absu < 0x33000000u) return (uint16_t)sign;          // < 2^-25
        const int e = (int)(absu >> 23);                        // biased exponent, 102..112
        const uint32_t mant = (absu & 0x7fffffu) | 0x800000u;   // 24-bit significand
        const int shift = 126 - e;                              // 14..24: result = mant >> shift
        uint32_t q = mant >> shift;
        const uint32_t rem = mant & ((1u << shift) - 1u);
        const uint32_t half = 1u << (shift - 1);
        if (rem > half || (rem == half && (q & 1u))) ++q;
        return (uint16_t)(sign | q);
    }
    uint32_t q = (absu - 0x38000000u) >> 13;      // rebias exponent 127 -> 15, keep 10 mantissa bits
    const uint32_t rem = absu & 0x1fffu;
    if (rem > 0x1000u || (rem == 0x1000u && (q & 1u))) ++q;     // carry may bump the exponent: correct
    return (uint16_t)(sign | q);
}

// binary32 -> 16-bit fixed point with `frac_bits` fraction bits: the nearest integer to w * 2^frac_bits,
// halves to the even one, saturated to the int16 range; NaN becomes 0.  (The scaling by a power of
// two is exact in double precision, nearbyint rounds to nearest-even in the default rounding mode.)
static int16_t f32_to_q16(float w, int frac_bits) {
    if (w != w) return 0;
    const double q = std::nearbyint(std::ldexp((double)w, frac_bits));
    return (int16_t)(q < -32768.0 ? -32768.0 : q > 32767.0 ? 32767.0 : q);
}

int encode_host(const float* dense, int64_t rows, int64_t cols, int64_t ld, int br, int bc,
                const uint8_t* row_keep, const uint8_t* col_keep, int val_dtype, csb_matrix* A) {
    A->rows = rows; A->cols = cols; A->block_r = br; A->block_c = bc; A->val_dtype = val_dtype;
    A->nbr = (rows + br - 1) / br;
    A->nbc = (cols + bc - 1) / bc;
    A->nblk = A->nbr * A->nbc;
    const int vs = val_size(val_dtype);
    try {
        A->m.assign(A->nblk, 0); A->n.assign(A->nblk, 0);
        A->val_off.assign(A->nblk + 1, 0); A->ridx_off.assign(A->nblk + 1, 0); A->cidx_off.assign(A->nblk + 1, 0);
        // pass 1: counts and offsets
        uint64_t vo = 0, ro = 0, co = 0;
        for (int64_t bi = 0; bi < A->nbr; ++bi) {
            const int rlim = (int)std::min<int64_t>(br, rows - bi * br);
            for (int64_t bj = 0; bj < A->nbc; ++bj) {
                const int64_t b = bi * A->nbc + bj;
                const int clim = (int)std::min<int64_t>(bc, cols - bj * bc);
                int m = 0, n = 0;
                for (int i = 0; i < rlim; ++i) m += row_keep[b * br + i] != 0;
                for (int j = 0; j < clim; ++j) n += col_keep[b * bc + j] != 0;
                A->m[b] = (uint16_t)m; A->n[b] = (uint16_t)n;
                A->val_off[b] = vo; A->ridx_off[b] = (uint32_t)ro; A->cidx_off[b] = (uint32_t)co;
                vo += (uint64_t)m * n; ro += m; co += n;
                if (ro > 0xffffffffull || co > 0xffffffffull) {
                    set_error("index lists exceed 2^32 entries");
                    return CSB_ERR_UNSUPPORTED;
                }
            }
        }
        A->val_off[A->nblk] = vo; A->ridx_off[A->nblk] = (uint32_t)ro; A->cidx_off[A->nblk] = (uint32_t)co;
        A->nnz = (int64_t)vo;
        A->row_idx.resize(ro); A->col_idx.resize(co); A->val.resize(vo * vs);
        // pass 2: indices and values
        for (int64_t bi = 0; bi < A->nbr; ++bi) {
            const int rlim = (int)std::min<int64_t>(br, rows - bi * br);
            for (int64_t bj = 0; bj < A->nbc; ++bj) {
                const int64_t b = bi * A->nbc + bj;
                const int clim = (int)std::min<int64_t>(bc, cols - bj * bc);
                uint8_t* ri = A->row_idx.data() + A->ridx_off[b];
                uint8_t* ci = A->col_idx.data() + A->cidx_off[b];
                int m = 0, n = 0;
                for (int i = 0; i < rlim; ++i) if (row_keep[b * br + i]) ri[m++] = (uint8_t)i;
                for (int j = 0; j < clim; ++j) if (col_keep[b * bc + j]) ci[n++] = (uint8_t)j;
                uint8_t* v = A->val.data() + A->val_off[b] * vs;
                for (int r = 0; r < m; ++r) {
                    const float* src = dense + (bi * br + ri[r]) * ld + bj * bc;
                    for (int k = 0; k < n; ++k) {
                        const float w = src[ci[k]];
                        if (vs == 4) std::memcpy(v, &w, 4);
                        else if (val_dtype == CSB_Q16) { const int16_t q = f32_to_q16(w, A->q_frac_bits); std::memcpy(v, &q, 2); }
                        else { const uint16_t h = f32_to_f16_rne(w); std::memcpy(v, &h, 2); }
                        v += vs;
                    }
                }
            }
        }
    } catch (const std::bad_alloc&) {
        set_error("out of host memory while encoding %lld x %lld", (long long)rows, (long long)cols);
        return CSB_ERR_ALLOC;
    }
    return CSB_OK;
}

// Structural self-check of the canonical arrays: offsets are the prefix sums of
// the counts, index lists ascend and stay inside the (possibly short) block.
int validate_host(const csb_matrix* A) {
    uint64_t vo = 0, ro = 0, co = 0;
    for (int64_t b = 0; b < A->nblk; ++b) {
        const int64_t bi = b / A->nbc, bj = b % A->nbc;
        const int rlim = (int)std::min<int64_t>(A->block_r, A->rows - bi * A->block_r);
        const int clim = (int)std::min<int64_t>(A->block_c, A->cols - bj * A->block_c);
        if (A->val_off[b] != vo || A->ridx_off[b] != ro || A->cidx_off[b] != co) {
            set_error("offsets of block %lld are not prefix sums", (long long)b);
            return CSB_ERR_INVALID_ARG;
        }
        const int m = A->m[b], n = A->n[b];
        if (m > rlim || n > clim) { set_error("block %lld keeps more lines than it has", (long long)b); return CSB_ERR_INVALID_ARG; }
        for (int r = 0; r < m; ++r) {
            const int v = A->row_idx[ro + r];
            if (v >= rlim || (r && v <= A->row_idx[ro + r - 1])) { set_error("row indices of block %lld", (long long)b); return CSB_ERR_INVALID_ARG; }
        }
        for (int k = 0; k < n; ++k) {
            const int v = A->col_idx[co + k];
            if (v >= clim || (k && v <= A->col_idx[co + k - 1])) { set_error("column indices of block %lld", (long long)b); return CSB_ERR_INVALID_ARG; }
        }
        vo += (uint64_t)m * n; ro += m; co += n;
    }
    if ((int64_t)vo != A->nnz || A->val.size() != vo * val_size(A->val_dtype)) {
        set_error("value array length does not match sum of m*n");
        return CSB_ERR_INVALID_ARG;
    }
    return CSB_OK;
}

}  // namespace csb
