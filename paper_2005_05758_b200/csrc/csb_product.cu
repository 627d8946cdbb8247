// CSB sparse product kernel (SpMV and the CUDA-core batched form) and its launch glue.
//
// What the paper's CSB-Engine does per block (Section 4.3.1) -- read the kept inputs
// through ColIdx, multiply by the kernel matrix, accumulate into the outputs through
// RowIdx, sum along the block-row -- is done here by independent warps of a persistent
// grid.  Every warp owns one contiguous run of the planned item stream and pulls it
// through its own shared-memory ring with bulk asynchronous copies, so global memory is
// read once, in large aligned pieces, while the irregular indexing happens on chip.
#include <algorithm>
#include <cstdio>
#include <mutex>

#include "csb_internal.hpp"
#include "csb_device.cuh"

namespace csb {

struct ProductArgs {
    const uint8_t* stream;
    const Chunk* chunks;
    const uint4* warp_desc;    // per warp: first chunk, end chunk, first chunk's off16 and bytes
    const uint32_t* part_base;
    const uint32_t* part_count;
    uint32_t* arrivals;
    float* partials;
    const float* X;
    float* Y;
    long long ldx, ldy;
    uint32_t* status;
    int n_warps, nb, rows, cols, block_r, stage_bytes, stages, x_in_smem;
};


constexpr uint32_t kOffMask = 0x3fffffffu;   // Chunk::off16 without the flush kind in its top two bits

__host__ __device__ inline size_t align16(size_t v) { return (v + 15) & ~(size_t)15; }

// Shared-memory carve-up, identical on host and device.
struct ProductSmem {
    size_t ring, bars, xbar, flag, zs, xg, xs, total;
    int zs_stride;                                     // floats per lane group
    __host__ __device__ ProductSmem(int W, int G, int stages, int stage_bytes, int block_r, int BT, int cols_in_smem) {
        zs_stride = block_r * BT + group_pad(32 / G);
        ring = 0;
        bars = ring + (size_t)W * stages * stage_bytes;
        xbar = bars + (size_t)W * stages * 8;
        flag = xbar + 8;                               // one word: did this CTA arrive last at a divided block-row
        zs = align16(flag + 8);
        xg = align16(zs + (size_t)W * G * zs_stride * 4);
        xs = align16(xg + (size_t)W * G * xg_stride(32 / G, BT) * 4);
        total = align16(xs + (size_t)cols_in_smem * 4);
    }
};

// End of a block-row inside a warp: add the lane groups' private sums in group order, then
// either store to y (the warp owned the whole block-row) or park the sums in the warp's slot;
// the warp that arrives last adds all slots of that block-row in slot order and writes y.
template <int BT, int G>
__device__ __forceinline__ void flush_block_row(const ProductArgs& a, float* zs, int zs_stride, uint32_t zbase, uint32_t tail,
                                                int lane) {
    const int nrows = min(a.block_r, a.rows - (int)zbase);
    const bool direct = (tail & 3u) == kFlushDirect;
    float* dst = a.partials + (size_t)(tail >> kSlotShift) * a.block_r * BT;
    for (int i = lane; i < nrows * BT; i += 32) {
        float v = zs[i];
        zs[i] = 0.f;
#pragma unroll
        for (int g = 1; g < G; ++g) { v += zs[g * zs_stride + i]; zs[g * zs_stride + i] = 0.f; }
        if (direct) {
            const int r = i / BT, bt = i % BT;
            if (bt < a.nb) a.Y[(long long)bt * a.ldy + zbase + r] = v;
        } else {
            __stcg(dst + i, v);
        }
    }
    if (direct) return;
    const uint32_t bi = zbase / (uint32_t)a.block_r;
    __threadfence();
    __syncwarp();
    int last = 0;
    if (lane == 0) last = (atomicAdd(&a.arrivals[bi], 1u) == a.part_count[bi] - 1u);
    last = __shfl_sync(0xffffffffu, last, 0);
    if (!last) return;
    __threadfence();
    const uint32_t pb = a.part_base[bi], pc = a.part_count[bi];
    const size_t pstride = (size_t)a.block_r * BT;
    for (int i = lane; i < nrows * BT; i += 32) {
        // eight loads in flight; the grouping is fixed, so the sum is reproducible
        const float* src = a.partials + (size_t)pb * pstride + i;
        float s[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (uint32_t q = 0; q < pc; q += 8) {
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = (q + j < pc) ? __ldcg(src + (size_t)(q + j) * pstride) : 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] += v[j];
        }
        const float sum = ((s[0] + s[1]) + (s[2] + s[3])) + ((s[4] + s[5]) + (s[6] + s[7]));
        const int r = i / BT, bt = i % BT;
        if (bt < a.nb) a.Y[(long long)bt * a.ldy + zbase + r] = sum;
    }
    if (lane == 0) a.arrivals[bi] = 0u;                // ready for the next launch
}

// End of a block-row that one CTA owns (all its warps are past the barrier): add the private
// sums of every warp and lane group in a fixed order and store y.  `parts` adjacent lanes share
// one output, each adds every parts-th copy, a fixed xor-tree joins them.
// When the CTA holds only a piece of the block-row (`partial` points at its slot), the sums go
// there instead, each thread fencing what it wrote.
template <int BT>
__device__ __forceinline__ void cta_flush_block_row(const ProductArgs& a, const float* zs_all, int zs_stride, int copies,
                                                    uint32_t zbase, float* partial) {
    const int nrows = min(a.block_r, a.rows - (int)zbase);
    const int NZ = nrows * BT;
    int parts = 1;
    while (parts < 32 && parts * 2 * NZ <= (int)blockDim.x && parts * 2 <= copies) parts *= 2;
    const int span = (NZ * parts + 31) & ~31;
    for (int idx = threadIdx.x; idx < span; idx += blockDim.x) {
        const int e = idx / parts, pt = idx % parts;
        float sum = 0.f;
        if (e < NZ) {
            const float* src = zs_all + e;
            for (int c = pt; c < copies; c += 8 * parts) {
                float v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) v[j] = (c + j * parts < copies) ? src[(c + j * parts) * zs_stride] : 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) sum += v[j];
            }
        }
        for (int off = parts >> 1; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
        if (e < NZ && pt == 0) {
            const int r = e / BT, bt = e % BT;
            if (partial) { __stcg(partial + e, sum); __threadfence(); }
            else if (bt < a.nb) a.Y[(long long)bt * a.ldy + zbase + r] = sum;
        }
    }
}

// The CTA that arrived last at a divided block-row adds the pieces in slot order and stores y.
template <int BT>
__device__ __forceinline__ void cta_join_block_row(const ProductArgs& a, uint32_t zbase) {
    const int nrows = min(a.block_r, a.rows - (int)zbase);
    const uint32_t bi = zbase / (uint32_t)a.block_r;
    const uint32_t pb = a.part_base[bi], pc = a.part_count[bi];
    const size_t pstride = (size_t)a.block_r * BT;
    for (int e = threadIdx.x; e < nrows * BT; e += blockDim.x) {
        const float* src = a.partials + (size_t)pb * pstride + e;
        float sum = 0.f;
        for (uint32_t q = 0; q < pc; q += 4) {
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = (q + j < pc) ? __ldcg(src + (size_t)(q + j) * pstride) : 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) sum += v[j];
        }
        const int r = e / BT, bt = e % BT;
        if (bt < a.nb) a.Y[(long long)bt * a.ldy + zbase + r] = sum;
    }
    if (threadIdx.x == 0) a.arrivals[bi] = 0u;         // ready for the next launch
}

template <typename T, int BT, int GW>
__global__ void __launch_bounds__(512, 1) csb_product_kernel(const ProductArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int G = 32 / GW;
    const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const ProductSmem L(W, G, a.stages, a.stage_bytes, a.block_r, BT, a.x_in_smem ? a.cols : 0);
    uint8_t* ring = smem + L.ring + (size_t)warp * a.stages * a.stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L.bars) + warp * a.stages;
    float* zs = reinterpret_cast<float*>(smem + L.zs) + warp * G * L.zs_stride;
    float* xg = reinterpret_cast<float*>(smem + L.xg) + warp * G * xg_stride(GW, BT);
    const float* xs = reinterpret_cast<const float*>(smem + L.xs);

    const int gw = blockIdx.x * W + warp;
    // One 16-byte descriptor per warp (first chunk index, end chunk index, first chunk's place
    // and size) starts the pipeline with a single round trip; the loads of x are issued before
    // anything waits on it.
    uint4 wd = make_uint4(0u, 0u, 0u, 0u);
    if (gw < a.n_warps) wd = __ldg(a.warp_desc + gw);
    const uint32_t c0 = wd.x, c1 = wd.y;
    // x comes in with one bulk copy per CTA when its address and size allow (16-byte multiples)
    bool x_dead = false;
    uint64_t* xbar = reinterpret_cast<uint64_t*>(smem + L.xbar);
    const bool x_bulk = a.x_in_smem && (reinterpret_cast<uintptr_t>(a.X) & 15) == 0 && (a.cols & 3) == 0;
    if (x_bulk && threadIdx.x == 0) {
        mbar_init(xbar, 1);
        mbar_fence_init();
        mbar_expect_tx(xbar, (uint32_t)a.cols * 4u);
        for (uint32_t off = 0; off < (uint32_t)a.cols * 4u; off += 16384u)
            bulk_g2s(smem + L.xs + off, reinterpret_cast<const uint8_t*>(a.X) + off, min(16384u, (uint32_t)a.cols * 4u - off), xbar);
    }
    if (lane == 0) {
        for (int s = 0; s < a.stages; ++s) mbar_init(&bars[s], 1);
        mbar_fence_init();
        if (c0 < c1) {
            mbar_expect_tx(&bars[0], wd.w);
            bulk_g2s(ring, a.stream + (size_t)(wd.z & kOffMask) * 16, wd.w, &bars[0]);
        }
        for (int s = 1; s < a.stages && c0 + s < c1; ++s) {
            const Chunk ch = a.chunks[c0 + s];
            mbar_expect_tx(&bars[s], ch.bytes);
            bulk_g2s(ring + (size_t)s * a.stage_bytes, a.stream + (size_t)(ch.off16 & kOffMask) * 16, ch.bytes, &bars[s]);
        }
    }
    for (int i = lane; i < G * L.zs_stride; i += 32) zs[i] = 0.f;
    if (a.x_in_smem) {
        if (!x_bulk) {
            float* xw = reinterpret_cast<float*>(smem + L.xs);
            for (int i = threadIdx.x; i < a.cols; i += blockDim.x) xw[i] = __ldg(a.X + i);
        }
        __syncthreads();                              // x staged by loads, or xbar initialised
        if (x_bulk && !mbar_wait_bounded(xbar, 0)) x_dead = true;     // reported and drained below
    } else {
        __syncwarp();
    }

    bool dead = x_dead;
    bool reported = false;
    Chunk cur = Chunk{wd.z, wd.w};
    for (uint32_t c = c0; c < c1; ++c) {
        const int s = (int)((c - c0) % (uint32_t)a.stages);
        const uint32_t parity = ((c - c0) / (uint32_t)a.stages) & 1u;
        const uint32_t flush = cur.off16 >> 30;                       // known without the chunk itself
        const Chunk nxt = (c + 1 < c1) ? a.chunks[c + 1] : Chunk{0, 0};
        const Chunk refill = (c + a.stages < c1) ? a.chunks[c + a.stages] : Chunk{0, 0};
        if (!dead) dead = __any_sync(0xffffffffu, !mbar_wait_bounded(&bars[s], parity));
        if (dead && !reported) {
            // report, then give the copies still in flight a bounded chance to land.  A warp of
            // a row-owned CTA keeps going through its chunk list without touching any data: the
            // other warps of the CTA expect it at every block-row's barrier.
            reported = true;
            if (lane == 0) {
                *(volatile uint32_t*)a.status = (uint32_t)kDevCopyTimeout;
                for (uint32_t j = c; j < c1 && j < c + (uint32_t)a.stages; ++j)
                    mbar_wait_bounded(&bars[(j - c0) % (uint32_t)a.stages], ((j - c0) / (uint32_t)a.stages) & 1u);
            }
        }
        if (dead) {
            if (flush == kFlushCta) { __syncthreads(); __syncthreads(); __syncthreads(); }
            cur = nxt;
            continue;
        }
        const uint8_t* p = ring + (size_t)s * a.stage_bytes;
        const uint4 ch = *reinterpret_cast<const uint4*>(p);
        walk_chunk<T, BT, GW>(p, ch, lane, xg, zs, L.zs_stride,
                              [&](uint32_t xbase, uint32_t c4, uint32_t, int left, float* dst) {
            if (BT == 1) {
                // index 0 of the block is always a valid column, so padding indices may be read
                float4 v;
                if (a.x_in_smem) {
                    v.x = xs[xbase + (c4 & 0xffu)]; v.y = xs[xbase + ((c4 >> 8) & 0xffu)];
                    v.z = xs[xbase + ((c4 >> 16) & 0xffu)]; v.w = xs[xbase + (c4 >> 24)];
                } else {
                    v.x = __ldg(a.X + xbase + (c4 & 0xffu)); v.y = __ldg(a.X + xbase + ((c4 >> 8) & 0xffu));
                    v.z = __ldg(a.X + xbase + ((c4 >> 16) & 0xffu)); v.w = __ldg(a.X + xbase + (c4 >> 24));
                }
                *reinterpret_cast<float4*>(dst) = v;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float* src = a.X + xbase + ((c4 >> (8 * j)) & 0xffu);
#pragma unroll
                    for (int bt = 0; bt < BT; ++bt) dst[j * BT + bt] = bt < a.nb ? __ldg(src + (long long)bt * a.ldx) : 0.f;
                }
            }
        }
        );
        if (flush == kFlushCta) {
            // the CTA owns this block-row: every warp is here with its last chunk of it
            // (three barriers whether the block-row is whole or a piece, so that a warp that gave
            // up on its copies can keep step without reading the chunk)
            volatile uint32_t* s_last = reinterpret_cast<volatile uint32_t*>(smem + L.flag);
            const bool piece = (ch.w & kFlushCtaPartial) != 0;
            __syncthreads();
            cta_flush_block_row<BT>(a, reinterpret_cast<const float*>(smem + L.zs), L.zs_stride, W * G, ch.z,
                                    piece ? a.partials + (size_t)(ch.w >> kSlotShift) * a.block_r * BT : nullptr);
            __syncthreads();
            for (int i = lane; i < G * L.zs_stride; i += 32) zs[i] = 0.f;
            if (piece && threadIdx.x == 0) {
                const uint32_t bi = ch.z / (uint32_t)a.block_r;
                __threadfence();
                *s_last = (atomicAdd(&a.arrivals[bi], 1u) == a.part_count[bi] - 1u) ? 1u : 0u;
            }
            __syncthreads();
            if (piece && *s_last) {
                __threadfence();
                cta_join_block_row<BT>(a, ch.z);
            }
            __syncwarp();
        } else if (flush != kFlushNone) {
            flush_block_row<BT, G>(a, zs, L.zs_stride, ch.z, ch.w, lane);
            __syncwarp();
        }
        if (lane == 0 && refill.bytes) {
            mbar_expect_tx(&bars[s], refill.bytes);
            bulk_g2s(ring + (size_t)s * a.stage_bytes, a.stream + (size_t)(refill.off16 & kOffMask) * 16, refill.bytes, &bars[s]);
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

template <typename V>
static int upload(const std::vector<V>& h, V** d) {
    *d = nullptr;
    const size_t bytes = std::max<size_t>(h.size(), 1) * sizeof(V);
    CSB_CUDA(cudaMalloc((void**)d, bytes));
    if (!h.empty()) CSB_CUDA(cudaMemcpy(*d, h.data(), h.size() * sizeof(V), cudaMemcpyHostToDevice));
    return CSB_OK;
}

static const int kBatchTiles[] = {8, 4, 1};
enum { kMaxBatchTile = 8, kTileDoesNotFit = 1 };


// Largest warp count per CTA whose carve-up fits the opt-in shared memory.
static int fit_warps(const csb_matrix* A, int want, int BT, int cols_in_smem, size_t* smem) {
    const ProductPlan& P = A->product;
    for (int W = want; W >= 1; --W) {
        const ProductSmem L(W, 32 / P.group_width, P.stages, P.stage_bytes, A->block_r, BT, cols_in_smem);
        if (L.total <= A->smem_optin) { *smem = L.total; return W; }
    }
    return 0;
}

int plan_product(csb_matrix* A) {
    ProductPlan& P = A->product;
    int dev_prev = 0;
    CSB_CUDA(cudaGetDevice(&dev_prev));
    CSB_CUDA(cudaSetDevice(A->device));
    cudaDeviceProp prop{};
    CSB_CUDA(cudaGetDeviceProperties(&prop, A->device));
    if (prop.major < 10) { set_error("device %d is sm_%d%d; this library is built for sm_100a", A->device, prop.major, prop.minor); return CSB_ERR_UNSUPPORTED; }
    A->sm_count = prop.multiProcessorCount;
    A->smem_optin = prop.sharedMemPerBlockOptin;
    const int ctas = A->opts.ctas > 0 ? A->opts.ctas : A->sm_count;
    const int wpc = std::min(16, A->opts.warps_per_cta > 0 ? A->opts.warps_per_cta : 16);
    P.stage_bytes = ((A->opts.stage_bytes > 0 ? A->opts.stage_bytes : 4096) + 15) & ~15;
    P.stage_bytes = std::max(P.stage_bytes, 1024);
    P.stages = std::min(8, std::max(1, A->opts.stages > 0 ? A->opts.stages : 2));
    // small matrices: no more warps than there is work for (about 2 KB of stream each)
    const int64_t approx = A->nnz * val_size(A->val_dtype) + (int64_t)A->ridx_off[A->nblk] + A->cidx_off[A->nblk] + 16 * A->nblk;
    const int64_t useful = std::max<int64_t>(1, approx / 2048);
    // A row-owned plan fixes the CTA shape (its warps meet at CTA barriers), so that shape must fit
    // shared memory at the narrowest batch tile; if the rings asked for do not, plan for fewer warps.
    ProductHostPlan H;
    int rc = CSB_OK;
    for (int w_try = wpc;; w_try /= 2) {
        H = ProductHostPlan();
        rc = plan_product_host(A, ctas, w_try, useful, P.stage_bytes, &H);
        if (rc != CSB_OK) return rc;
        P.row_owned = H.row_owned;
        P.group_width = H.stream.group_width;
        P.warps = H.row_owned ? H.warps_per_cta : 1;
        size_t smem = 0;
        if (fit_warps(A, P.warps, 1, 0, &smem) == P.warps) break;
        if (w_try <= 1 || !H.row_owned) {
            set_error("a shared-memory ring of %d stages of %d bytes per warp does not fit one CTA (%zu bytes available)", P.stages,
                      P.stage_bytes, A->smem_optin);
            return CSB_ERR_INVALID_ARG;
        }
    }
    const int n_warps = H.stream.n_warps;
    if (H.row_owned) { P.warps = H.warps_per_cta; P.ctas = H.ctas; }
    else { P.warps = std::max(1, (n_warps + ctas - 1) / ctas); P.ctas = (n_warps + P.warps - 1) / P.warps; }
    P.n_slots = H.n_slots;
    P.balance = H.balance;
    P.stream_bytes = (int64_t)H.stream.bytes.size();
    P.n_warps = n_warps;
    if ((rc = upload(H.stream.bytes, &P.d_stream)) != CSB_OK) return rc;
    if ((rc = upload(H.stream.chunks, &P.d_chunks)) != CSB_OK) return rc;
    std::vector<uint4> wdesc(n_warps);
    for (int w = 0; w < n_warps; ++w) {
        const uint32_t c0 = H.stream.warp_chunk_begin[w], c1 = H.stream.warp_chunk_begin[w + 1];
        wdesc[w] = make_uint4(c0, c1, c0 < c1 ? H.stream.chunks[c0].off16 : 0u, c0 < c1 ? H.stream.chunks[c0].bytes : 0u);   // off16 keeps its flush bits
    }
    if ((rc = upload(wdesc, (uint4**)&P.d_warp_desc)) != CSB_OK) return rc;
    if ((rc = upload(H.part_base, &P.d_part_base)) != CSB_OK) return rc;
    if ((rc = upload(H.part_count, &P.d_part_count)) != CSB_OK) return rc;
    CSB_CUDA(cudaMalloc((void**)&P.d_arrivals, std::max<size_t>(A->nbr, 1) * 4));
    CSB_CUDA(cudaMemset(P.d_arrivals, 0, std::max<size_t>(A->nbr, 1) * 4));
    CSB_CUDA(cudaMalloc((void**)&P.d_partials, std::max<size_t>((size_t)P.n_slots * A->block_r * kMaxBatchTile, 1) * 4));
    CSB_CUDA(cudaHostAlloc((void**)&P.h_status, 4, cudaHostAllocMapped));
    *P.h_status = 0;
    CSB_CUDA(cudaHostGetDevicePointer((void**)&P.d_status, P.h_status, 0));
    CSB_CUDA(cudaDeviceSynchronize());
    CSB_CUDA(cudaSetDevice(dev_prev));
    return CSB_OK;
}

void free_product(csb_matrix* A) {
    ProductPlan& P = A->product;
    if (A->device < 0) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(A->device);
    cudaFree(P.d_stream); cudaFree(P.d_chunks); cudaFree(P.d_warp_desc); cudaFree(P.d_part_base);
    cudaFree(P.d_part_count); cudaFree(P.d_arrivals); cudaFree(P.d_partials);
    if (P.h_status) cudaFreeHost(P.h_status);
    P = ProductPlan{};
    cudaSetDevice(prev);
}

template <typename T, int BT, int GW>
static int launch_tile(const csb_matrix* A, ProductArgs a, cudaStream_t st) {
    const ProductPlan& P = A->product;
    size_t smem = 0;
    int cols_in_smem = 0;
    if (BT == 1 && (size_t)A->cols * 4 <= 64 * 1024) {
        size_t s2 = 0;
        if (fit_warps(A, P.warps, 1, (int)A->cols, &s2) == P.warps) cols_in_smem = (int)A->cols;
    }
    const int W = fit_warps(A, P.warps, BT, cols_in_smem, &smem);
    if (W == 0) { set_error("a single warp's shared-memory ring does not fit (%d stages of %d bytes)", P.stages, P.stage_bytes); return CSB_ERR_LAUNCH; }
    if (P.row_owned && W != P.warps) return kTileDoesNotFit;      // the CTA shape is part of the plan: caller narrows the batch tile
    a.x_in_smem = cols_in_smem > 0;
    const int ctas = (P.n_warps + W - 1) / W;
    static bool configured[64] = {};                   // per device; setting it twice is harmless
    if (A->device >= 64 || !configured[A->device]) {
        CSB_CUDA(cudaFuncSetAttribute(csb_product_kernel<T, BT, GW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)A->smem_optin));
        if (A->device < 64) configured[A->device] = true;
    }
    csb_product_kernel<T, BT, GW><<<ctas, W * 32, smem, st>>>(a);
    CSB_CUDA(cudaGetLastError());
    return CSB_OK;
}

template <typename T, int BT>
static int dispatch_gw(const csb_matrix* A, const ProductArgs& a, cudaStream_t st) {
    switch (A->product.group_width) {
        case 8: return launch_tile<T, BT, 8>(A, a, st);
        case 16: return launch_tile<T, BT, 16>(A, a, st);
        default: return launch_tile<T, BT, 32>(A, a, st);
    }
}

static int dispatch_tile(const csb_matrix* A, const ProductArgs& a, cudaStream_t st, int bt) {
    const bool h = A->val_dtype == CSB_F16;
    if (bt == 8) return h ? dispatch_gw<__half, 8>(A, a, st) : dispatch_gw<float, 8>(A, a, st);
    if (bt == 4) return h ? dispatch_gw<__half, 4>(A, a, st) : dispatch_gw<float, 4>(A, a, st);
    return h ? dispatch_gw<__half, 1>(A, a, st) : dispatch_gw<float, 1>(A, a, st);
}


int launch_product(const csb_matrix* A, const float* X, int64_t ldx, int batch, float* Y, int64_t ldy, void* stream) {
    const ProductPlan& P = A->product;
    if (P.h_status && *P.h_status != 0) { set_error("an earlier product on this handle gave up waiting on the device (code %u)", *P.h_status); return CSB_ERR_TIMEOUT; }
    int prev = 0;
    CSB_CUDA(cudaGetDevice(&prev));
    if (prev != A->device) CSB_CUDA(cudaSetDevice(A->device));
    ProductArgs a{};
    a.stream = P.d_stream; a.chunks = P.d_chunks; a.warp_desc = (const uint4*)P.d_warp_desc;
    a.part_base = P.d_part_base; a.part_count = P.d_part_count; a.arrivals = P.d_arrivals; a.partials = P.d_partials;
    a.ldx = ldx; a.ldy = ldy; a.status = P.d_status; a.n_warps = P.n_warps;
    a.rows = (int)A->rows; a.cols = (int)A->cols; a.block_r = A->block_r; a.stage_bytes = P.stage_bytes; a.stages = P.stages;
    cudaStream_t st = (cudaStream_t)stream;
    int rc = CSB_OK;
    int widest = kMaxBatchTile;                        // narrowed when a tile's shared memory does not fit the planned CTA
    for (int b0 = 0; b0 < batch && rc == CSB_OK;) {
        int bt = 1;
        for (int cand : kBatchTiles) if (cand <= widest && (batch - b0 >= cand || cand == 1)) { bt = cand; break; }
        if (batch - b0 > 1 && bt == 1 && widest >= 4) bt = 4;          // 2 or 3 left: one padded tile of 4
        a.X = X + (int64_t)b0 * ldx; a.Y = Y + (int64_t)b0 * ldy; a.nb = std::min(bt, batch - b0);
        rc = dispatch_tile(A, a, st, bt);
        if (rc == kTileDoesNotFit) {
            if (bt == 1) { set_error("the planned CTA of %d warps does not fit shared memory even for one batch column", P.warps); rc = CSB_ERR_LAUNCH; break; }
            widest = bt == 8 ? 4 : 1; rc = CSB_OK; continue;
        }
        b0 += a.nb;
    }
    if (prev != A->device) cudaSetDevice(prev);
    return rc;
}


// ---------------------------------------------------------------------------------------
// SpMV whose scratch is built into the library image (see csb_spmv_static_scratch in csb.h).
//
// The block-row reduction of the product kernel needs scratch in global memory: one slot of
// partial sums per (warp, block-row) pair that shares a block-row, and one arrival counter per
// block-row.  csb_spmv keeps that scratch in buffers cudaMalloc'ed with the handle.  Here it
// sits in one fixed array that every GPU loading the library carries until the process exits.
// ---------------------------------------------------------------------------------------
constexpr size_t kStaticArrivalBytes = 64u << 10;                 // 16384 block-rows
constexpr size_t kStaticPartialBytes = (4u << 20) - kStaticArrivalBytes;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticArrivalBytes + kStaticPartialBytes];

// In host code the array's name stands for the symbol, not for an address on the device; the
// address is asked for once per device, with that device current.
static unsigned char* g_static_scratch_addr[64] = {};
static std::mutex g_static_scratch_mu;

static int static_scratch_address(int device, unsigned char** out) {
    if (device < 0 || device >= 64) { set_error("device ordinal %d is outside 0..63", device); return CSB_ERR_UNSUPPORTED; }
    std::lock_guard<std::mutex> lk(g_static_scratch_mu);
    if (!g_static_scratch_addr[device]) {
        void* p = nullptr;
        CSB_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));      // the caller made `device` current
        g_static_scratch_addr[device] = (unsigned char*)p;
    }
    *out = g_static_scratch_addr[device];
    return CSB_OK;
}

int launch_spmv_static_scratch(const csb_matrix* A, const float* x, float* y, void* stream) {
    const ProductPlan& P = A->product;
    if (P.h_status && *P.h_status != 0) { set_error("an earlier product on this handle gave up waiting on the device (code %u)", *P.h_status); return CSB_ERR_TIMEOUT; }
    const size_t need_arrivals = (size_t)A->nbr * 4, need_partials = (size_t)P.n_slots * A->block_r * 4;
    if (need_arrivals > kStaticArrivalBytes || need_partials > kStaticPartialBytes) {
        set_error("matrix needs %zu bytes of arrival counters and %zu bytes of partial sums; the built-in scratch holds %zu and %zu "
                  "(use csb_spmv, whose scratch is sized per handle)", need_arrivals, need_partials, kStaticArrivalBytes, kStaticPartialBytes);
        return CSB_ERR_UNSUPPORTED;
    }
    int prev = 0;
    CSB_CUDA(cudaGetDevice(&prev));
    if (prev != A->device) CSB_CUDA(cudaSetDevice(A->device));
    struct Restore { int prev, cur; ~Restore() { if (prev != cur) cudaSetDevice(prev); } } restore{prev, A->device};
    unsigned char* scratch = nullptr;
    int rc = static_scratch_address(A->device, &scratch);
    if (rc != CSB_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // The array keeps whatever the last call left.  The counters must start at zero; the partial
    // sums need no clearing, every slot that is read is written first in the same launch.
    CSB_CUDA(cudaMemsetAsync(scratch, 0, need_arrivals, st));
    ProductArgs a{};
    a.stream = P.d_stream; a.chunks = P.d_chunks; a.warp_desc = (const uint4*)P.d_warp_desc;
    a.part_base = P.d_part_base; a.part_count = P.d_part_count;
    a.arrivals = reinterpret_cast<uint32_t*>(scratch);
    a.partials = reinterpret_cast<float*>(scratch + kStaticArrivalBytes);
    a.ldx = A->cols; a.ldy = A->rows; a.status = P.d_status; a.n_warps = P.n_warps;
    a.rows = (int)A->rows; a.cols = (int)A->cols; a.block_r = A->block_r; a.stage_bytes = P.stage_bytes; a.stages = P.stages;
    a.X = x; a.Y = y; a.nb = 1;
    rc = dispatch_tile(A, a, st, 1);
    if (rc == kTileDoesNotFit) { set_error("the planned CTA of %d warps does not fit shared memory", P.warps); rc = CSB_ERR_LAUNCH; }
    return rc;
}

}  // namespace csb

extern "C" int csb_spmv_static_scratch(const csb_matrix_t* A, const float* x, float* y, void* stream) {
    csb::clear_error();
    if (!A || !x || !y) { csb::set_error("A, x or y is NULL"); return CSB_ERR_INVALID_ARG; }
    if (A->device < 0) { csb::set_error("matrix was encoded host-only (device = -1)"); return CSB_ERR_UNSUPPORTED; }
    if (A->val_dtype == CSB_Q16) { csb::set_error("fixed-point handles serve csb_spmm_q16 only"); return CSB_ERR_UNSUPPORTED; }
    return csb::launch_spmv_static_scratch(A, x, y, stream);
}
