// Tensor-core CSB-SpMM (batch >= 8, fp16 values, fp32 accumulation).
//
// With a batch of vectors the product of a block's kernel matrix (m kept rows x n kept columns)
// with the gathered inputs (n x batch) is a small dense contraction, the one place on this path
// where tensor cores apply.  Every kernel matrix is stored as 16 x 8 tiles in the register order of
// mma.sync.m16n8k8's A operand; the gathered inputs sit in shared memory as [column][batch] rows
// of fp16 and reach the B operand through ldmatrix.trans.  fp32 inputs are split into two fp16
// halves (x = hi + lo) and multiplied separately, so no input precision is lost; products are
// accumulated in fp32.  One launch handles a slab of up to 32 batch columns.
//
// The bulk-copy ring, the row-owned schedule (a CTA owns whole block-rows, a CTA barrier ends each
// one, warps' private sums are added in a fixed order) and the bounded waits are those of the
// CUDA-core product kernel.
#include <algorithm>
#include <cstdio>
#include <mutex>

#include "csb_internal.hpp"
#include "csb_device.cuh"

namespace csb {

constexpr int kSlab = 32;                    // batch columns per launch
constexpr int kXRowBytes = 80;               // one gathered column: 32 halves + 16 bytes so ldmatrix rows miss each other's banks
constexpr int kZStride = 34;                 // floats per output row in a warp's private sums (32 + 2: spreads banks)
constexpr uint32_t kOffMaskM = 0x3fffffffu;
constexpr int kXBuf = 2 * kMmaMaxNk * kXRowBytes;   // one gather buffer: hi rows, then lo rows

struct MmaArgs {
    const uint8_t* stream;
    const Chunk* chunks;
    const uint4* warp_desc;
    const __half* xp;          // [cols][64]: 32 hi halves, 32 lo halves of the slab
    float* Y;                  // slab's first batch row
    long long ldy;
    uint32_t* status;
    int n_warps, nb, rows, block_r, stage_bytes, stages;
};

struct MmaSmem {
    size_t ring, bars, zs, xs, total;
    __host__ __device__ MmaSmem(int W, int stages, int stage_bytes, int block_r) {
        ring = 0;
        bars = ring + (size_t)W * stages * stage_bytes;
        zs = (bars + (size_t)W * stages * 8 + 15) & ~(size_t)15;
        xs = (zs + (size_t)W * block_r * kZStride * 4 + 15) & ~(size_t)15;
        total = xs + (size_t)W * 2 * 2 * kMmaMaxNk * kXRowBytes;       // two buffers x (hi, lo) x rows
    }
};

// Pack a slab of X: fp32 [batch][cols] -> fp16 hi / lo [cols][64] (batch columns past nb are zero).
__global__ void csb_pack_x_kernel(const float* __restrict__ X, long long ldx, int nb, int cols, __half* __restrict__ xp) {
    pdl_launch_dependents();
    pdl_wait();                                    // X may come from the kernel in front; xp may still be read by it
    const int col = blockIdx.x * (blockDim.x / kSlab) + threadIdx.x / kSlab, b = threadIdx.x % kSlab;
    if (col >= cols) return;
    const float x = b < nb ? X[(long long)b * ldx + col] : 0.f;
    const __half hi = __float2half_rn(x);
    const __half lo = __float2half_rn(x - __half2float(hi));
    xp[(size_t)col * 64 + b] = hi;
    xp[(size_t)col * 64 + kSlab + b] = lo;
}

__device__ __forceinline__ void mma_m16n8k8(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* row_ptr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(row_ptr)));
}

template <int NT>
__global__ void __launch_bounds__(256, 1) csb_spmm_mma_kernel(const MmaArgs a) {
    pdl_launch_dependents();
    extern __shared__ __align__(128) uint8_t smem[];
    const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const MmaSmem L(W, a.stages, a.stage_bytes, a.block_r);
    uint8_t* ring = smem + L.ring + (size_t)warp * a.stages * a.stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.bars) + warp * a.stages;
    float* zs_all = reinterpret_cast<float*>(smem + L.zs);
    float* zs = zs_all + (size_t)warp * a.block_r * kZStride;
    uint8_t* xs_base = smem + L.xs + (size_t)warp * 2 * kXBuf;
    const int g = lane >> 2, t = lane & 3;

    const int gw = blockIdx.x * W + warp;
    uint4 wd = make_uint4(0u, 0u, 0u, 0u);
    if (gw < a.n_warps) wd = __ldg(a.warp_desc + gw);
    const uint32_t c0 = wd.x, c1 = wd.y;
    if (lane == 0) {
        for (int s = 0; s < a.stages; ++s) mbar_init(&bars[s], 1);
        mbar_fence_init();
        if (c0 < c1) {
            mbar_expect_tx(&bars[0], wd.w);
            bulk_g2s(ring, a.stream + (size_t)(wd.z & kOffMaskM) * 16, wd.w, &bars[0]);
        }
        for (int s = 1; s < a.stages && c0 + s < c1; ++s) {
            const Chunk ch = a.chunks[c0 + s];
            mbar_expect_tx(&bars[s], ch.bytes);
            bulk_g2s(ring + (size_t)s * a.stage_bytes, a.stream + (size_t)(ch.off16 & kOffMaskM) * 16, ch.bytes, &bars[s]);
        }
    }
    for (int i = lane; i < a.block_r * kZStride; i += 32) zs[i] = 0.f;
    __syncwarp();
    // everything so far touched only the planned stream (written once, at plan time) and shared
    // memory; the packed inputs and Y belong to the work in front on the stream
    pdl_wait();

    bool dead = false, reported = false;
    Chunk cur = Chunk{wd.z, wd.w};
    for (uint32_t c = c0; c < c1; ++c) {
        const int s = (int)((c - c0) % (uint32_t)a.stages);
        const uint32_t parity = ((c - c0) / (uint32_t)a.stages) & 1u;
        const uint32_t flush = cur.off16 >> 30;
        const Chunk nxt = (c + 1 < c1) ? a.chunks[c + 1] : Chunk{0, 0};
        const Chunk refill = (c + a.stages < c1) ? a.chunks[c + a.stages] : Chunk{0, 0};
        if (!dead) dead = __any_sync(0xffffffffu, !mbar_wait_bounded(&bars[s], parity));
        if (dead && !reported) {
            reported = true;
            if (lane == 0) {
                *(volatile uint32_t*)a.status = (uint32_t)kDevCopyTimeout;
                for (uint32_t j = c; j < c1 && j < c + (uint32_t)a.stages; ++j)
                    mbar_wait_bounded(&bars[(j - c0) % (uint32_t)a.stages], ((j - c0) / (uint32_t)a.stages) & 1u);
            }
        }
        if (dead) {                                   // keep the CTA's barriers company, touch no data
            if (flush == kFlushCta) { __syncthreads(); __syncthreads(); }
            cur = nxt;
            continue;
        }
        const uint8_t* p = ring + (size_t)s * a.stage_bytes;
        const uint4 chh = *reinterpret_cast<const uint4*>(p);
        const uint8_t* end = p + 16 + 16 * (chh.x & 0xffffu);
        p += 16;
        // Gather of one item into buffer `buf`, asynchronously: each kept column is 128 contiguous
        // bytes of the packed slab (64 hi, 64 lo); eight lanes move one column, four columns per pass;
        // rows past nk up to the tile edge are zeroed.
        auto gather_async = [&](const uint8_t* item, int buf) {
            const uint4 hh = *reinterpret_cast<const uint4*>(item);
            const int nk_ = (int)(hh.x & 0xffu), kpad_ = (int)(hh.x >> 24) * 8;
            const uint8_t* cidx_ = item + 16;
            uint8_t* hi = xs_base + buf * kXBuf;
            const int piece = lane & 7;                           // 16-byte piece: 0..3 hi, 4..7 lo
            for (int k = lane >> 3; k < kpad_; k += 4) {
                uint8_t* dst = hi + (piece < 4 ? 0 : kMmaMaxNk * kXRowBytes) + k * kXRowBytes + (piece & 3) * 16;
                if (k < nk_) {
                    const void* src = reinterpret_cast<const uint4*>(a.xp + (size_t)(hh.y + cidx_[k]) * 64) + piece;
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
                } else {
                    *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        auto item_size = [](const uint8_t* item) {
            const uint4 hh = *reinterpret_cast<const uint4*>(item);
            const int nk_ = (int)(hh.x & 0xffu), mr_ = (int)((hh.x >> 8) & 0xffu), RT_ = (int)((hh.x >> 16) & 0xffu), KT_ = (int)(hh.x >> 24);
            return ((16 + ((nk_ + 3) & ~3) + ((mr_ + 3) & ~3) + 15) & ~15) + RT_ * KT_ * 256;
        };
        int buf = 0;
        if (p < end) gather_async(p, 0);
        while (p < end) {
            const uint4 h = *reinterpret_cast<const uint4*>(p);
            const int nk = (int)(h.x & 0xffu), mr = (int)((h.x >> 8) & 0xffu), RT = (int)((h.x >> 16) & 0xffu), KT = (int)(h.x >> 24);
            const uint8_t* cidx = p + 16;
            const uint8_t* ridx = cidx + ((nk + 3) & ~3);
            const uint8_t* tiles = p + ((16 + ((nk + 3) & ~3) + ((mr + 3) & ~3) + 15) & ~15);
            p += item_size(p);
            // the next item's inputs are fetched while this one is multiplied
            if (p < end) {
                gather_async(p, buf ^ 1);
                asm volatile("cp.async.wait_group 1;" ::: "memory");
            } else {
                asm volatile("cp.async.wait_group 0;" ::: "memory");
            }
            __syncwarp();
            const uint8_t* xs_hi = xs_base + buf * kXBuf;
            const uint8_t* xs_lo = xs_hi + kMmaMaxNk * kXRowBytes;
            buf ^= 1;
            // ---- multiply: D[16 kept rows x 8 batch] += A[16 x 8 kept columns] . B[8 x 8], four batch tiles
            for (int rt = 0; rt < RT; ++rt) {
                float acc[NT][4];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
                const uint2* at = reinterpret_cast<const uint2*>(tiles + (size_t)rt * KT * 256) + lane;
                for (int kt = 0; kt < KT; ++kt) {
                    const uint2 af = at[kt * 32];
                    // lane l hands ldmatrix the address of row (l % 8) of matrix (l / 8) = batch tile
                    const int off = (kt * 8 + (lane & 7)) * kXRowBytes + (lane >> 3) * 16;
                    uint32_t bh[4], bl[4];
                    ldmatrix_x4_trans(bh, xs_hi + off);
                    ldmatrix_x4_trans(bl, xs_lo + off);
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {          // batch tiles past NT hold zero columns: skipped
                        mma_m16n8k8(acc[nt], af.x, af.y, bh[nt]);
                        mma_m16n8k8(acc[nt], af.x, af.y, bl[nt]);
                    }
                }
                // ---- scatter-add through the row indices: this lane holds rows g, g + 8 of the tile,
                // batch columns 2t, 2t + 1 of every batch tile
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int r = rt * 16 + g + 8 * half;
                    if (r < mr) {
                        float* z = zs + (int)ridx[r] * kZStride + 2 * t;
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            float2 cur2 = *reinterpret_cast<float2*>(z + nt * 8);
                            cur2.x += acc[nt][2 * half]; cur2.y += acc[nt][2 * half + 1];
                            *reinterpret_cast<float2*>(z + nt * 8) = cur2;
                        }
                    }
                }
            }
            __syncwarp();
        }
        if (flush == kFlushCta) {
            __syncthreads();
            // the CTA owns this block-row: add the warps' private sums in warp order and store y
            const int zbase = (int)chh.z;
            const int nrows = min(a.block_r, a.rows - zbase);
            for (int idx = threadIdx.x; idx < nrows * a.nb; idx += blockDim.x) {
                const int b = idx / nrows, r = idx % nrows;
                float sum = 0.f;
                for (int w = 0; w < W; ++w) sum += zs_all[((size_t)w * a.block_r + r) * kZStride + b];
                a.Y[(long long)b * a.ldy + zbase + r] = sum;
            }
            __syncthreads();
            for (int i = lane; i < a.block_r * kZStride; i += 32) zs[i] = 0.f;
            __syncwarp();
        }
        if (lane == 0 && refill.bytes) {
            mbar_expect_tx(&bars[s], refill.bytes);
            bulk_g2s(ring + (size_t)s * a.stage_bytes, a.stream + (size_t)(refill.off16 & kOffMaskM) * 16, refill.bytes, &bars[s]);
        }
        cur = nxt;
    }
}


#define CSB_CUDA(call)                                                                     \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            set_error("%s failed: %s", #call, cudaGetErrorString(e_));                     \
            return e_ == cudaErrorMemoryAllocation ? CSB_ERR_ALLOC : CSB_ERR_CUDA;         \
        }                                                                                  \
    } while (0)

bool spmm_mma_applicable(const csb_matrix* A, int batch) {
    if (getenv("CSB_NO_MMA") && atoi(getenv("CSB_NO_MMA"))) return false;
    return batch >= 8 && A->val_dtype == CSB_F16 && A->block_r <= 64 && A->device >= 0 && !(A->mma && A->mma->unusable);
}

template <typename V>
static int upload_v(const std::vector<V>& h, V** d) {
    const size_t bytes = std::max<size_t>(h.size(), 1) * sizeof(V);
    CSB_CUDA(cudaMalloc((void**)d, bytes));
    if (!h.empty()) CSB_CUDA(cudaMemcpy(*d, h.data(), h.size() * sizeof(V), cudaMemcpyHostToDevice));
    return CSB_OK;
}

static int build_mma_plan(const csb_matrix* A, MmaPlan* P) {
    P->warps = 8; P->stage_bytes = 4096; P->stages = 2;
    const int ctas = A->opts.ctas > 0 ? A->opts.ctas : A->sm_count;
    const MmaSmem L(P->warps, P->stages, P->stage_bytes, A->block_r);
    if (L.total > A->smem_optin) { P->unusable = true; return CSB_OK; }
    MmaHostPlan H;
    int rc = plan_mma_host(A, ctas, P->warps, P->stage_bytes, &H);
    if (rc != CSB_OK) return rc;
    if (H.max_chunk_bytes > (size_t)P->stage_bytes) { P->unusable = true; return CSB_OK; }
    P->ctas = H.ctas; P->n_warps = H.ctas * H.warps_per_cta; P->balance = H.balance;
    P->stream_bytes = (int64_t)H.bytes.size();
    std::vector<uint4> wdesc(P->n_warps);
    for (int w = 0; w < P->n_warps; ++w) {
        const uint32_t c0 = H.warp_chunk_begin[w], c1 = H.warp_chunk_begin[w + 1];
        wdesc[w] = make_uint4(c0, c1, c0 < c1 ? H.chunks[c0].off16 : 0u, c0 < c1 ? H.chunks[c0].bytes : 0u);
    }
    if ((rc = upload_v(H.bytes, &P->d_stream)) != CSB_OK) return rc;
    if ((rc = upload_v(H.chunks, &P->d_chunks)) != CSB_OK) return rc;
    if ((rc = upload_v(wdesc, (uint4**)&P->d_warp_desc)) != CSB_OK) return rc;
    P->xp_bytes = (size_t)A->cols * 64 * sizeof(__half);
    CSB_CUDA(cudaMalloc(&P->d_xp, P->xp_bytes));
    CSB_CUDA(cudaFuncSetAttribute(csb_spmm_mma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total));
    CSB_CUDA(cudaFuncSetAttribute(csb_spmm_mma_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total));
    CSB_CUDA(cudaFuncSetAttribute(csb_spmm_mma_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total));
    CSB_CUDA(cudaDeviceSynchronize());
    P->built = true;
    return CSB_OK;
}

void free_mma(csb_matrix* A) {
    if (!A->mma) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(A->device);
    cudaFree(A->mma->d_stream); cudaFree(A->mma->d_chunks); cudaFree(A->mma->d_warp_desc); cudaFree(A->mma->d_xp);
    cudaSetDevice(prev);
    delete A->mma;
    A->mma = nullptr;
}

// Returns CSB_OK after launching, or kMmaNotUsed (1) when the caller should use the CUDA-core path.
int launch_spmm_mma(const csb_matrix* A, const float* X, int64_t ldx, int batch, float* Y, int64_t ldy, void* stream) {
    const ProductPlan& PP = A->product;
    if (PP.h_status && *PP.h_status != 0) { set_error("an earlier product on this handle gave up waiting on the device (code %u)", *PP.h_status); return CSB_ERR_TIMEOUT; }
    int prev = 0;
    CSB_CUDA(cudaGetDevice(&prev));
    if (prev != A->device) CSB_CUDA(cudaSetDevice(A->device));
    struct Restore { int prev, cur; ~Restore() { if (prev != cur) cudaSetDevice(prev); } } restore{prev, A->device};
    {
        std::lock_guard<std::mutex> lk(A->mma_mu);
        if (!A->mma) {
            A->mma = new (std::nothrow) MmaPlan();
            if (!A->mma) { set_error("out of host memory"); return CSB_ERR_ALLOC; }
            int rc;
            try { rc = build_mma_plan(A, A->mma); }
            catch (const std::bad_alloc&) { set_error("out of host memory while planning the batched product"); rc = CSB_ERR_ALLOC; }
            if (rc != CSB_OK) { A->mma->unusable = true; return rc; }
        }
    }
    const MmaPlan& P = *A->mma;
    if (P.unusable || !P.built) return 1;
    cudaStream_t st = (cudaStream_t)stream;
    const MmaSmem L(P.warps, P.stages, P.stage_bytes, A->block_r);
    MmaArgs a{};
    a.stream = P.d_stream; a.chunks = P.d_chunks; a.warp_desc = (const uint4*)P.d_warp_desc; a.xp = (const __half*)P.d_xp;
    a.ldy = ldy; a.status = PP.d_status; a.n_warps = P.n_warps; a.rows = (int)A->rows; a.block_r = A->block_r;
    a.stage_bytes = P.stage_bytes; a.stages = P.stages;
    for (int b0 = 0; b0 < batch; b0 += kSlab) {
        a.nb = std::min(kSlab, batch - b0);
        a.Y = Y + (int64_t)b0 * ldy;
        // both kernels order themselves behind the work in front (pdl_wait at their top), so they may
        // be launched with programmatic stream serialization: their scheduling overlaps its tail
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg{};
        cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = 1;
        cfg.gridDim = dim3((unsigned)((A->cols + 7) / 8)); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0;
        CSB_CUDA(cudaLaunchKernelEx(&cfg, csb_pack_x_kernel, X + (int64_t)b0 * ldx, (long long)ldx, a.nb, (int)A->cols, (__half*)P.d_xp));
        cfg.gridDim = dim3((unsigned)P.ctas); cfg.blockDim = dim3((unsigned)P.warps * 32u); cfg.dynamicSmemBytes = L.total;
        if (a.nb <= 8) CSB_CUDA(cudaLaunchKernelEx(&cfg, csb_spmm_mma_kernel<1>, a));
        else if (a.nb <= 16) CSB_CUDA(cudaLaunchKernelEx(&cfg, csb_spmm_mma_kernel<2>, a));
        else CSB_CUDA(cudaLaunchKernelEx(&cfg, csb_spmm_mma_kernel<4>, a));
        CSB_CUDA(cudaGetLastError());
    }
    return CSB_OK;
}

}  // namespace csb
