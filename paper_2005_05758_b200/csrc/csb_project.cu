// Projection of a dense weight onto the CSB pattern: the RowPrune / ColumnPrune step of the
// paper's Algorithm 1 (Section 3.2), which turns any dense matrix and a target pruning rate into
// the per-block row and column keep masks that csb_encode takes.
//
// RowPrune works on every block-column on its own: the squared l2-norm of each row segment (the
// part of a matrix row inside the block-column) is taken and the weakest fraction p of the
// segments is pruned; ColumnPrune then does the same with the column segments of every block-row
// of the result.  p = 1 - sqrt(1 - PR), so about PR of the weights are gone after both.
//
// Four kernels, all on one stream: segment norms of the rows (one pass over the matrix, fp64
// sums), selection per block-column, segment norms of the columns (a second pass, skipping the
// pruned row segments), selection per block-row.  A selection is a radix select in shared memory
// (eight 8-bit passes over the ordered bit patterns of the norms) for the value of the last
// pruned segment, and a second short one over the indices of the segments that tie with it:
// among equal norms the higher index goes first.
#include <algorithm>

#include "csb_internal.hpp"

namespace csb {

#define CSB_CUDA(call)                                                                     \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            set_error("%s failed: %s", #call, cudaGetErrorString(e_));                     \
            return e_ == cudaErrorMemoryAllocation ? CSB_ERR_ALLOC : CSB_ERR_CUDA;         \
        }                                                                                  \
    } while (0)

constexpr int kSelectThreads = 1024;
constexpr int64_t kMaxSelect = 20480;          // segments per selection: their norms sit in shared memory

// Squared norms of the row segments: rn[bj * R + r] = sum over the block-column's columns of W[r, c]^2.
// One CTA per row; its warps take the block-columns in turn and read them with coalesced loads.
__global__ void csb_row_segment_norms_kernel(const float* __restrict__ W, long long ld, int R, int C, int BC, int nbc,
                                             double* __restrict__ rn) {
    const int r = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    const float* row = W + (size_t)r * ld;
    for (int bj = warp; bj < nbc; bj += nw) {
        const int c0 = bj * BC, c1 = min(C, c0 + BC);
        double s = 0.0;
        for (int c = c0 + lane; c < c1; c += 32) { const double v = (double)__ldg(row + c); s += v * v; }
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0) rn[(size_t)bj * R + r] = s;
    }
}

// Squared norms of the column segments after RowPrune: cn[bi * C + c] = sum over the block-row's
// rows whose segment survived in c's block of W[r, c]^2.  One thread per column.
__global__ void csb_col_segment_norms_kernel(const float* __restrict__ W, long long ld, int R, int C, int BR, int BC, int nbc,
                                             const uint8_t* __restrict__ row_keep, double* __restrict__ cn) {
    const int bi = blockIdx.y, c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    const int r0 = bi * BR, r1 = min(R, r0 + BR);
    const uint8_t* rk = row_keep + ((size_t)bi * nbc + c / BC) * BR;
    double s = 0.0;
    for (int r = r0; r < r1; ++r)
        if (rk[r - r0]) { const double v = (double)__ldg(W + (size_t)r * ld + c); s += v * v; }
    cn[(size_t)bi * C + c] = s;
}

// k-th smallest (1-based) of the keys that pass `pred`, by 8-bit radix passes from the top;
// returns the key and, through rank_in_equals, how many of the keys equal to it are among the k
// smallest.  All threads of the CTA call it; hist is 256 counters, sel two words of shared memory.
template <typename Key, int BYTES, typename Get, typename Pred>
__device__ Key radix_select(int n, unsigned int k, Get get, Pred pred, unsigned int* hist, unsigned long long* sel,
                            unsigned int* rank_in_equals) {
    Key prefix = 0, mask = 0;
    for (int shift = 8 * (BYTES - 1); shift >= 0; shift -= 8) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0u;
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            if (!pred(i)) continue;
            const Key key = get(i);
            if ((key & mask) == prefix) atomicAdd(&hist[(unsigned int)((key >> shift) & (Key)255)], 1u);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned int cum = 0, b = 0;
            for (; b < 255u; ++b) { if (cum + hist[b] >= k) break; cum += hist[b]; }
            sel[0] = b; sel[1] = k - cum;
        }
        __syncthreads();
        prefix |= (Key)sel[0] << shift;
        mask |= (Key)255 << shift;
        k = (unsigned int)sel[1];
        __syncthreads();
    }
    *rank_in_equals = k;
    return prefix;
}

// One CTA per group (a block-column's row segments, or a block-row's column segments): prune the
// k weakest of its n segments and write the keep flags where csb_encode expects them.
//   rows == 1: group g is block-column g, segment s is matrix row s   -> row_keep[((s / B) * nbc + g) * B + s % B]
//   rows == 0: group g is block-row g, segment s is matrix column s   -> col_keep[(g * nbc + s / B) * B + s % B]
__global__ void __launch_bounds__(kSelectThreads, 1) csb_select_prune_kernel(const double* __restrict__ norms, int n, unsigned int k,
                                                                             int rows, int B, int nbc, uint8_t* __restrict__ keep) {
    extern __shared__ __align__(16) unsigned char sm[];
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(sm);
    unsigned int* hist = reinterpret_cast<unsigned int*>(keys + n);
    unsigned long long* sel = reinterpret_cast<unsigned long long*>(hist + 256);
    const int g = blockIdx.x;
    // sums of squares are >= +0, so the bit patterns order like the values
    for (int i = threadIdx.x; i < n; i += blockDim.x) keys[i] = (unsigned long long)__double_as_longlong(norms[(size_t)g * n + i]);
    __syncthreads();
    unsigned long long v = ~0ull;
    unsigned int idx_cut = 0xffffffffu;             // among the segments that tie with v, those with index >= idx_cut go
    if (k > 0) {
        unsigned int need = 0;
        v = radix_select<unsigned long long, 8>(n, k, [&](int i) { return keys[i]; }, [&](int) { return true; }, hist, sel, &need);
        // the `need` highest indices among the ties: the need-th smallest of the inverted indices
        unsigned int dummy = 0;
        const unsigned int inv = radix_select<unsigned int, 4>(n, need, [&](int i) { return 0xffffffffu - (unsigned int)i; },
                                                               [&](int i) { return keys[i] == v; }, hist, sel, &dummy);
        idx_cut = 0xffffffffu - inv;
    }
    for (int s = threadIdx.x; s < n; s += blockDim.x) {
        const bool gone = k > 0 && (keys[s] < v || (keys[s] == v && (unsigned int)s >= idx_cut));
        const size_t at = rows ? ((size_t)(s / B) * nbc + g) * B + s % B : ((size_t)g * nbc + s / B) * B + s % B;
        keep[at] = gone ? 0 : 1;
    }
}

static unsigned int pruned_count(double p, int64_t n) {
    const double v = p * (double)n + 0.5;
    return (unsigned int)std::min<double>((double)n, v < 0 ? 0.0 : std::floor(v));
}

int project_device(const float* W, int64_t R, int64_t C, int64_t ld, int BR, int BC, double PR, uint8_t* row_keep,
                   uint8_t* col_keep, void* workspace, int64_t workspace_bytes, void* stream) {
    const int64_t nbr = (R + BR - 1) / BR, nbc = (C + BC - 1) / BC;
    const int64_t need = (nbc * R + nbr * C) * 8;
    if (workspace_bytes < need) { set_error("workspace of %lld bytes, %lld needed", (long long)workspace_bytes, (long long)need); return CSB_ERR_INVALID_ARG; }
    if (R > kMaxSelect || C > kMaxSelect) { set_error("rows and columns above %lld are not supported by the selection kernel", (long long)kMaxSelect); return CSB_ERR_UNSUPPORTED; }
    cudaStream_t st = (cudaStream_t)stream;
    double* rn = reinterpret_cast<double*>(workspace);
    double* cn = rn + nbc * R;
    const double p = 1.0 - std::sqrt(1.0 - PR);
    static bool configured = false;
    if (!configured) {
        CSB_CUDA(cudaFuncSetAttribute(csb_select_prune_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kMaxSelect * 8 + 2048)));
        configured = true;
    }
    // flags of in-block lines beyond the matrix edge stay zero
    CSB_CUDA(cudaMemsetAsync(row_keep, 0, (size_t)(nbr * nbc * BR), st));
    CSB_CUDA(cudaMemsetAsync(col_keep, 0, (size_t)(nbr * nbc * BC), st));
    csb_row_segment_norms_kernel<<<(unsigned)R, 256, 0, st>>>(W, ld, (int)R, (int)C, BC, (int)nbc, rn);
    csb_select_prune_kernel<<<(unsigned)nbc, kSelectThreads, (size_t)R * 8 + 1024 + 16, st>>>(rn, (int)R, pruned_count(p, R), 1, BR, (int)nbc, row_keep);
    csb_col_segment_norms_kernel<<<dim3((unsigned)((C + 255) / 256), (unsigned)nbr), 256, 0, st>>>(W, ld, (int)R, (int)C, BR, BC, (int)nbc, row_keep, cn);
    csb_select_prune_kernel<<<(unsigned)nbr, kSelectThreads, (size_t)C * 8 + 1024 + 16, st>>>(cn, (int)C, pruned_count(p, C), 0, BC, (int)nbc, col_keep);
    CSB_CUDA(cudaGetLastError());
    return CSB_OK;
}

}  // namespace csb

extern "C" {

int64_t csb_project_workspace_bytes(int64_t rows, int64_t cols, int block_r, int block_c) {
    if (rows <= 0 || cols <= 0 || block_r < 1 || block_c < 1) return 0;
    const int64_t nbr = (rows + block_r - 1) / block_r, nbc = (cols + block_c - 1) / block_c;
    return (nbc * rows + nbr * cols) * 8;
}

int csb_project(const float* dense, int64_t rows, int64_t cols, int64_t ld, int block_r, int block_c, double prune_fraction,
                uint8_t* row_keep, uint8_t* col_keep, void* workspace, int64_t workspace_bytes, void* stream) {
    csb::clear_error();
    if (!dense || !row_keep || !col_keep || !workspace) { csb::set_error("dense, row_keep, col_keep or workspace is NULL"); return CSB_ERR_INVALID_ARG; }
    if (rows <= 0 || cols <= 0 || ld < cols) { csb::set_error("rows=%lld cols=%lld ld=%lld", (long long)rows, (long long)cols, (long long)ld); return CSB_ERR_INVALID_ARG; }
    if (block_r < 1 || block_r > 256 || block_c < 1 || block_c > 256) { csb::set_error("block sizes must be 1..256, got %dx%d", block_r, block_c); return CSB_ERR_INVALID_ARG; }
    if (!(prune_fraction >= 0.0 && prune_fraction <= 1.0)) { csb::set_error("prune_fraction %g is outside [0, 1]", prune_fraction); return CSB_ERR_INVALID_ARG; }
    return csb::project_device(dense, rows, cols, ld, block_r, block_c, prune_fraction, row_keep, col_keep, workspace, workspace_bytes, stream);
}

}  // extern "C"
