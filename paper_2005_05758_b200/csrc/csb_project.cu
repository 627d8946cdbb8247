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
// One thread per segment, consecutive threads on consecutive segments of a row: a warp reads one
// contiguous stretch of the row, every thread its own BC floats with 16-byte loads (many loads in
// flight per thread, every sector used whole).  `vec` says that rows and segments are 16-byte aligned.
__global__ void csb_row_segment_norms_kernel(const float* __restrict__ W, long long ld, int R, int C, int BC, int nbc, int vec,
                                             double* __restrict__ rn) {
    const long long seg = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (seg >= (long long)R * nbc) return;
    const int r = (int)(seg / nbc), bj = (int)(seg % nbc);
    const int c0 = bj * BC, c1 = min(C, c0 + BC);
    const float* p = W + (size_t)r * ld + c0;
    double s = 0.0;
    int c = c0;
    if (vec) {
        for (; c + 16 <= c1; c += 16, p += 16) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p + 4));
            const float4 d = __ldg(reinterpret_cast<const float4*>(p + 8)), e = __ldg(reinterpret_cast<const float4*>(p + 12));
            s += (double)a.x * a.x; s += (double)a.y * a.y; s += (double)a.z * a.z; s += (double)a.w * a.w;
            s += (double)b.x * b.x; s += (double)b.y * b.y; s += (double)b.z * b.z; s += (double)b.w * b.w;
            s += (double)d.x * d.x; s += (double)d.y * d.y; s += (double)d.z * d.z; s += (double)d.w * d.w;
            s += (double)e.x * e.x; s += (double)e.y * e.y; s += (double)e.z * e.z; s += (double)e.w * e.w;
        }
        for (; c + 4 <= c1; c += 4, p += 4) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(p));
            s += (double)a.x * a.x; s += (double)a.y * a.y; s += (double)a.z * a.z; s += (double)a.w * a.w;
        }
    }
    for (; c < c1; ++c, ++p) { const double v = (double)__ldg(p); s += v * v; }
    rn[(size_t)bj * R + r] = s;
}

// Squared norms of the column segments after RowPrune: cn[bi * C + c] = sum over the block-row's
// rows whose segment survived in c's block of W[r, c]^2.  A thread takes VEC (1 or 4) neighbouring
// columns of one block, so that they share the block's row flags; pruned row segments are not read.
template <int VEC>
__global__ void csb_col_segment_norms_kernel(const float* __restrict__ W, long long ld, int R, int C, int BR, int BC, int nbc,
                                             const uint8_t* __restrict__ row_keep, double* __restrict__ cn) {
    const int bi = blockIdx.y, c = (blockIdx.x * blockDim.x + threadIdx.x) * VEC;
    if (c >= C) return;
    const int r0 = bi * BR, r1 = min(R, r0 + BR);
    const uint8_t* rk = row_keep + ((size_t)bi * nbc + c / BC) * BR;
    double s[VEC];
#pragma unroll
    for (int q = 0; q < VEC; ++q) s[q] = 0.0;
    int r = r0;
    for (; r + 8 <= r1; r += 8) {                         // eight rows' loads go out together
        float v[8][VEC];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const bool kept = rk[r - r0 + j] != 0;
            if (VEC == 4) {
                const float4 t = kept ? __ldg(reinterpret_cast<const float4*>(W + (size_t)(r + j) * ld + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
                v[j][0] = t.x; v[j][VEC > 1 ? 1 : 0] = t.y; v[j][VEC > 2 ? 2 : 0] = t.z; v[j][VEC > 3 ? 3 : 0] = t.w;
            } else {
                v[j][0] = kept ? __ldg(W + (size_t)(r + j) * ld + c) : 0.f;
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int q = 0; q < VEC; ++q) s[q] += (double)v[j][q] * v[j][q];
    }
    for (; r < r1; ++r)
        if (rk[r - r0]) {
#pragma unroll
            for (int q = 0; q < VEC; ++q) { const double t = (double)__ldg(W + (size_t)r * ld + c + q); s[q] += t * t; }
        }
#pragma unroll
    for (int q = 0; q < VEC; ++q) cn[(size_t)bi * C + c + q] = s[q];
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
        // norms of one group are of similar size, so in the top passes nearly all keys fall into one
        // bucket: lanes of a warp that hit the same bucket add once, together
        for (int i0 = 0; i0 < n; i0 += blockDim.x) {
            const int i = i0 + threadIdx.x;
            unsigned int bucket = 0xffffffffu;
            if (i < n && pred(i)) {
                const Key key = get(i);
                if ((key & mask) == prefix) bucket = (unsigned int)((key >> shift) & (Key)255);
            }
            if (shift >= 8 * (BYTES - 2)) {
                // the top two digits: one add per bucket and warp
                const unsigned int peers = __match_any_sync(0xffffffffu, bucket);
                if (bucket != 0xffffffffu && (threadIdx.x & 31) == (unsigned)(__ffs(peers) - 1)) atomicAdd(&hist[bucket], (unsigned int)__popc(peers));
            } else if (bucket != 0xffffffffu) {
                atomicAdd(&hist[bucket], 1u);               // few keys are still in the running and they spread out
            }
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // warp 0 finds the bucket where the running count reaches k: eight buckets per lane
            const unsigned int lane = threadIdx.x;
            unsigned int mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) mine += hist[lane * 8 + j];
            unsigned int incl = mine;
            for (int off = 1; off < 32; off <<= 1) { const unsigned int o = __shfl_up_sync(0xffffffffu, incl, off); if (lane >= (unsigned)off) incl += o; }
            const unsigned int before = incl - mine;
            const unsigned int hit = __ballot_sync(0xffffffffu, incl >= k);
            if (lane == (unsigned)(__ffs(hit) - 1)) {
                unsigned int cum = before, b = lane * 8;
                for (int j = 0; j < 7; ++j, ++b) { if (cum + hist[b] >= k) break; cum += hist[b]; }
                sel[0] = b; sel[1] = k - cum;
            }
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
        // how many segments tie with v, and the lowest index among them (block-wide, through two words)
        if (threadIdx.x == 0) { sel[0] = 0ull; sel[1] = ~0ull; }
        __syncthreads();
        {
            unsigned int cnt = 0, lowest = 0xffffffffu;
            for (int i = threadIdx.x; i < n; i += blockDim.x)
                if (keys[i] == v) { ++cnt; lowest = min(lowest, (unsigned int)i); }
            if (cnt) { atomicAdd(&sel[0], (unsigned long long)cnt); atomicMin(&sel[1], (unsigned long long)lowest); }
        }
        __syncthreads();
        const unsigned int ties = (unsigned int)sel[0], lowest_tie = (unsigned int)sel[1];
        __syncthreads();
        if (need >= ties) idx_cut = lowest_tie;            // all of them go (the usual case: a single one)
        else {
            // the `need` highest indices among the ties: the need-th smallest of the inverted indices
            unsigned int dummy = 0;
            const unsigned int inv = radix_select<unsigned int, 4>(n, need, [&](int i) { return 0xffffffffu - (unsigned int)i; },
                                                                   [&](int i) { return keys[i] == v; }, hist, sel, &dummy);
            idx_cut = 0xffffffffu - inv;
        }
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
    // the selection kernel's shared memory is opted in per device (setting it twice is harmless)
    int dev = 0;
    CSB_CUDA(cudaGetDevice(&dev));
    static bool configured[64] = {};
    if (dev >= 64 || !configured[dev]) {
        CSB_CUDA(cudaFuncSetAttribute(csb_select_prune_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(kMaxSelect * 8 + 2048)));
        if (dev < 64) configured[dev] = true;
    }
    // flags of in-block lines beyond the matrix edge stay zero
    CSB_CUDA(cudaMemsetAsync(row_keep, 0, (size_t)(nbr * nbc * BR), st));
    CSB_CUDA(cudaMemsetAsync(col_keep, 0, (size_t)(nbr * nbc * BC), st));
    const int vec = (reinterpret_cast<uintptr_t>(W) & 15) == 0 && ld % 4 == 0 && BC % 4 == 0;
    csb_row_segment_norms_kernel<<<(unsigned)((R * nbc + 255) / 256), 256, 0, st>>>(W, ld, (int)R, (int)C, BC, (int)nbc, vec, rn);
    csb_select_prune_kernel<<<(unsigned)nbc, kSelectThreads, (size_t)R * 8 + 1024 + 16, st>>>(rn, (int)R, pruned_count(p, R), 1, BR, (int)nbc, row_keep);
    if (vec && C % 4 == 0)
        csb_col_segment_norms_kernel<4><<<dim3((unsigned)((C / 4 + 127) / 128), (unsigned)nbr), 128, 0, st>>>(W, ld, (int)R, (int)C, BR, BC, (int)nbc, row_keep, cn);
    else
        csb_col_segment_norms_kernel<1><<<dim3((unsigned)((C + 255) / 256), (unsigned)nbr), 256, 0, st>>>(W, ld, (int)R, (int)C, BR, BC, (int)nbc, row_keep, cn);
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
