// 16-bit fixed-point CSB product (the arithmetic of the paper's processing elements: Section 6.2.2,
// weights quantised to 16-bit fixed point; Section 6.3.1, 16-bit fixed-point multipliers).
//
// acc[b, r] = sum over the kept cross-points of row r of w_q * x_q[b, .], all in integers: a
// 16 x 16-bit product fits 31 bits and the sums are kept in 64 bits, which cannot overflow, so the
// result is exact and does not depend on the order of summation.  That is what lets this kernel
// add through atomics in shared memory without giving up bit-reproducibility.
//
// The kernel reads the canonical arrays of Section 3.1.1 as they are (m{}, n{}, RowIdx{}, ColIdx{},
// Val{} and the offsets), uploaded once.  A CTA works for one block-row and a range of its
// block-columns (enough ranges to fill the GPU several times over: what a warp does per block is a
// chain of dependent loads); its warps take the blocks of the range in turn, and the CTAs of a
// block-row add their sums into the output with 64-bit integer atomics.  For a block, the lanes first
// fetch the inputs behind the kept columns through ColIdx (lane g holds columns g, g + 32, ...); then
// every lane owns one kept row of the kernel matrix (32 rows at a time) and walks it column by column:
// its own weight times the column's input, handed round by a shuffle, into a 64-bit sum (one
// multiply-add with a wide result per weight, no reduction across lanes); the sum is added into the
// block-row's accumulators through RowIdx.
#include <algorithm>

#include "csb_internal.hpp"
#include "csb_device.cuh"

namespace csb {

#define CSB_CUDA(call)                                                                     \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            set_error("%s failed: %s", #call, cudaGetErrorString(e_));                     \
            return e_ == cudaErrorMemoryAllocation ? CSB_ERR_ALLOC : CSB_ERR_CUDA;         \
        }                                                                                  \
    } while (0)

struct FixedPlan {
    uint16_t* d_m = nullptr; uint16_t* d_n = nullptr;
    uint8_t* d_ridx = nullptr; uint8_t* d_cidx = nullptr;
    unsigned long long* d_val_off = nullptr; uint32_t* d_ridx_off = nullptr; uint32_t* d_cidx_off = nullptr;
    int16_t* d_val = nullptr;
};

struct FixedArgs {
    const uint16_t* m; const uint16_t* n;
    const uint8_t* ridx; const uint8_t* cidx;
    const unsigned long long* val_off; const uint32_t* ridx_off; const uint32_t* cidx_off;
    const int16_t* val;
    const int16_t* Xq; long long ldx;
    long long* acc; long long ldy;
    int rows, cols, block_r, block_c, nbc, nb, cols_per_cta;   // cols_per_cta: block-columns per CTA
};

constexpr int kFixedWarps = 8, kFixedMaxBlock = 128;

template <int BT>
__global__ void __launch_bounds__(kFixedWarps * 32) csb_q16_kernel(const FixedArgs a) {
    __shared__ unsigned long long s_acc[kFixedMaxBlock * BT];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bi = blockIdx.x;
    for (int i = threadIdx.x; i < a.block_r * BT; i += blockDim.x) s_acc[i] = 0ull;
    __syncthreads();
    const int bj_end = min(a.nbc, (int)(blockIdx.y + 1) * a.cols_per_cta);
    for (int bj = blockIdx.y * a.cols_per_cta + warp; bj < bj_end; bj += kFixedWarps) {
        const long long b = (long long)bi * a.nbc + bj;
        const int m = a.m[b], n = a.n[b];
        if (!m || !n) continue;
        const uint8_t* ci = a.cidx + a.cidx_off[b];
        const uint8_t* ri = a.ridx + a.ridx_off[b];
        const int16_t* v = a.val + a.val_off[b];
        // the inputs behind kept columns lane, lane + 32, ... (up to 4 of them: blocks are at most 128 wide)
        int xk[4][BT];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = lane + 32 * j;
            const long long col = (long long)bj * a.block_c + (k < n ? (int)ci[k] : 0);
#pragma unroll
            for (int bt = 0; bt < BT; ++bt) xk[j][bt] = (k < n && bt < a.nb) ? (int)a.Xq[(long long)bt * a.ldx + col] : 0;
        }
        for (int r0 = 0; r0 < m; r0 += 32) {
            const int r = r0 + lane;
            const bool live = r < m;
            const int16_t* row = v + (long long)(live ? r : 0) * n;
            long long sum[BT];
#pragma unroll
            for (int bt = 0; bt < BT; ++bt) sum[bt] = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int kn = min(32, n - 32 * j);                 // warp-uniform
#pragma unroll 4
                for (int kk = 0; kk < kn; ++kk) {
                    const long long w = (long long)row[32 * j + kk];
#pragma unroll
                    for (int bt = 0; bt < BT; ++bt)
                        sum[bt] += w * (long long)__shfl_sync(0xffffffffu, xk[j][bt], kk);   // 16 x 16 bits: exact
                }
            }
            if (live) {
                const int out = (int)ri[r] * BT;
#pragma unroll
                for (int bt = 0; bt < BT; ++bt)
                    if (sum[bt]) atomicAdd(&s_acc[out + bt], (unsigned long long)sum[bt]);
            }
        }
    }
    __syncthreads();
    const int nrows = min(a.block_r, a.rows - bi * a.block_r);
    for (int i = threadIdx.x; i < nrows * a.nb; i += blockDim.x) {
        const int bt = i / nrows, r = i - bt * nrows;
        const unsigned long long v = s_acc[r * BT + bt];
        if (gridDim.y == 1) a.acc[(long long)bt * a.ldy + (long long)bi * a.block_r + r] = (long long)v;
        else if (v) atomicAdd(reinterpret_cast<unsigned long long*>(a.acc + (long long)bt * a.ldy + (long long)bi * a.block_r + r), v);
    }
}

template <typename V>
static int upload_arr(const V* h, size_t n, V** d) {
    CSB_CUDA(cudaMalloc((void**)d, std::max<size_t>(n, 1) * sizeof(V)));
    if (n) CSB_CUDA(cudaMemcpy(*d, h, n * sizeof(V), cudaMemcpyHostToDevice));
    return CSB_OK;
}

int plan_fixed(csb_matrix* A) {
    int prev = 0;
    CSB_CUDA(cudaGetDevice(&prev));
    CSB_CUDA(cudaSetDevice(A->device));
    struct Restore { int prev; ~Restore() { cudaSetDevice(prev); } } restore{prev};
    cudaDeviceProp prop{};
    CSB_CUDA(cudaGetDeviceProperties(&prop, A->device));
    if (prop.major < 10) { set_error("device %d is sm_%d%d; this library is built for sm_100a", A->device, prop.major, prop.minor); return CSB_ERR_UNSUPPORTED; }
    A->sm_count = prop.multiProcessorCount;
    A->smem_optin = prop.sharedMemPerBlockOptin;
    FixedPlan* P = new (std::nothrow) FixedPlan();
    if (!P) { set_error("out of host memory"); return CSB_ERR_ALLOC; }
    A->fixed = P;
    int rc;
    if ((rc = upload_arr(A->m.data(), A->m.size(), &P->d_m)) != CSB_OK) return rc;
    if ((rc = upload_arr(A->n.data(), A->n.size(), &P->d_n)) != CSB_OK) return rc;
    if ((rc = upload_arr(A->row_idx.data(), A->row_idx.size(), &P->d_ridx)) != CSB_OK) return rc;
    if ((rc = upload_arr(A->col_idx.data(), A->col_idx.size(), &P->d_cidx)) != CSB_OK) return rc;
    if ((rc = upload_arr((const unsigned long long*)A->val_off.data(), A->val_off.size(), &P->d_val_off)) != CSB_OK) return rc;
    if ((rc = upload_arr(A->ridx_off.data(), A->ridx_off.size(), &P->d_ridx_off)) != CSB_OK) return rc;
    if ((rc = upload_arr(A->cidx_off.data(), A->cidx_off.size(), &P->d_cidx_off)) != CSB_OK) return rc;
    if ((rc = upload_arr((const int16_t*)A->val.data(), A->val.size() / 2, &P->d_val)) != CSB_OK) return rc;
    CSB_CUDA(cudaDeviceSynchronize());
    return CSB_OK;
}

void free_fixed(csb_matrix* A) {
    if (!A->fixed) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(A->device);
    FixedPlan* P = A->fixed;
    cudaFree(P->d_m); cudaFree(P->d_n); cudaFree(P->d_ridx); cudaFree(P->d_cidx); cudaFree(P->d_val_off); cudaFree(P->d_ridx_off);
    cudaFree(P->d_cidx_off); cudaFree(P->d_val);
    cudaSetDevice(prev);
    delete P;
    A->fixed = nullptr;
}

int launch_fixed(const csb_matrix* A, const int16_t* Xq, int64_t ldx, int batch, int64_t* acc, int64_t ldy, void* stream) {
    int prev = 0;
    CSB_CUDA(cudaGetDevice(&prev));
    if (prev != A->device) CSB_CUDA(cudaSetDevice(A->device));
    struct Restore { int prev, cur; ~Restore() { if (prev != cur) cudaSetDevice(prev); } } restore{prev, A->device};
    const FixedPlan& P = *A->fixed;
    FixedArgs a{};
    a.m = P.d_m; a.n = P.d_n; a.ridx = P.d_ridx; a.cidx = P.d_cidx; a.val_off = P.d_val_off; a.ridx_off = P.d_ridx_off;
    a.cidx_off = P.d_cidx_off; a.val = P.d_val; a.ldx = ldx; a.ldy = ldy;
    a.rows = (int)A->rows; a.cols = (int)A->cols; a.block_r = A->block_r; a.block_c = A->block_c; a.nbc = (int)A->nbc;
    cudaStream_t st = (cudaStream_t)stream;
    // ranges of block-columns per block-row: about eight CTAs per SM in all, at least one block per warp
    const int64_t want = std::max<int64_t>(1, (int64_t)8 * A->sm_count / std::max<int64_t>(A->nbr, 1));
    const int splits = (int)std::max<int64_t>(1, std::min<int64_t>(want, (A->nbc + kFixedWarps - 1) / kFixedWarps));
    a.cols_per_cta = (int)((A->nbc + splits - 1) / splits);
    const dim3 grid((unsigned)A->nbr, (unsigned)((A->nbc + a.cols_per_cta - 1) / a.cols_per_cta));
    if (grid.y > 1)                                       // the CTAs of a block-row add into the output: it starts from zero
        CSB_CUDA(cudaMemset2DAsync(acc, (size_t)ldy * 8, 0, (size_t)A->rows * 8, (size_t)batch, st));
    for (int b0 = 0; b0 < batch;) {
        const int left = batch - b0;
        a.Xq = Xq + (int64_t)b0 * ldx; a.acc = (long long*)acc + (int64_t)b0 * ldy;
        if (left >= 2) { a.nb = std::min(4, left); csb_q16_kernel<4><<<grid, kFixedWarps * 32, 0, st>>>(a); }
        else { a.nb = 1; csb_q16_kernel<1><<<grid, kFixedWarps * 32, 0, st>>>(a); }
        CSB_CUDA(cudaGetLastError());
        b0 += a.nb;
    }
    return CSB_OK;
}

}  // namespace csb
