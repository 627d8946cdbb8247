// Tensor-core CSB-SpMM (batch >= 8, fp16 values, fp32 accumulation).
//
// With a batch of vectors the product of a block's kernel matrix (m kept rows x n kept columns)
// with the gathered inputs (n x batch) of Section 4.3.1 is a small dense contraction, the one place
// on this path where tensor cores apply.  How it is laid out here:
//
//   * A warp works for one block-row over a range of block-columns and keeps that block-row's
//     outputs, all block_r rows x up to 32 batch columns, in the accumulator registers of
//     mma.sync.m16n8k16 for the whole range (several warps share a block-row's blocks; their sums
//     meet once, at the end).  The kernel matrix is the A operand with its kept rows put back at their
//     RowIdx positions: a lane finds the stored row behind an output row with a population count
//     on the block's 64-bit row mask and loads its fragment straight from the compact row-major
//     values (rows that are not kept give zero registers).  So nothing is scattered and nothing is
//     read-modify-written per block; the row indices never leave the registers.
//   * The inputs are packed once per call into binary16 pairs x = hi + lo (no input precision is
//     lost as long as |x| < 65504), one row of batch values per matrix column, and reach shared
//     memory as whole block-column tiles through a ring that all warps of the CTA share, so a tile
//     is fetched from L2 once per CTA and not once per block.  A tile spans up to four block-columns
//     (256 matrix columns), so that the warps hand tiles over a few times per CTA only.  The gather through ColIdx is done by
//     the operand load itself: every lane hands ldmatrix.trans the address of the tile row of one
//     kept column.  hi and lo are multiplied separately into the same accumulators.
//   * The weights of a warp come through its own ring of bulk copies, so warps with light and heavy
//     blocks do not wait for each other; they only meet at the input tiles, which a warp releases
//     in order whether it used them or not, the last warp to release a slot refilling it.
//   * A CTA covers RG block-rows x a range of block-columns (the planner's cut).  When a row group
//     is divided between S CTAs these are launched as one thread-block cluster and add their sums
//     through distributed shared memory, every CTA for a share of the rows and in the order of the
//     ranges, so results are bit-reproducible and no scratch in global memory is needed.
//   * More than 32 batch columns are served in passes of 32 (the weights of the later passes come
//     from L2).
#include <algorithm>
#include <cstdio>
#include <mutex>

#include "csb_internal.hpp"
#include "csb_device.cuh"
#include "csb_gates.cuh"

namespace csb {

constexpr uint32_t kOffMaskM = 0x3fffffffu;
constexpr uint32_t kNoRow = 0xffffffffu;
constexpr size_t kLoopTileBytes = 32 * 33 * 4;  // the time loop's transposition tile of the gate arithmetic
constexpr size_t kSpmmStaticSmem = 256;       // the kernel's statically allocated shared memory (CTA descriptor, row table), rounded up

struct SpmmArgs {
    const uint8_t* stream;
    const uint4* warp_desc;    // per warp: first chunk's offset, chunk count, sizes of its first three chunks
    const SpmmCta* ctas;
    const uint8_t* xp;         // packed inputs: one row of `pitch` bytes per matrix column
    float* Y;
    long long ldy;
    uint32_t* status;
    int nb, rows, cols, block_r, block_c, tile_cols, RG, S, x_depth, w_stages, pitch, tile_bytes;   // tile_cols: matrix columns per input tile
    int q_rows;                // rows of the largest row group the shared-memory carve-up must hold (RG * block_r of one product)
#ifdef CSB_SPMM_CLOCKS
    long long* clocks;         // instrumented build only: [CTA][warp][16] cycles per phase
#endif
};

// The recurrent time loop around the product (batches of 8 and more, up to 32 product rows): one
// cooperative launch runs all steps of all layers.  Per layer and step: the product pass of that
// layer's matrix over its packed inputs into Z, a grid barrier, the gate arithmetic (tiles of 32 hidden
// units dealt to the CTAs; h_t goes straight into the packed inputs of the next products), a grid barrier.
struct SpmmLoopLayer {
    const uint8_t* stream; const uint4* warp_desc; const SpmmCta* ctas;
    const uint8_t* xp;         // packed inputs of this layer's product, rows 0 .. in_size + H - 1
    const float* bias; float* c; float* hs;
    uint8_t* xp_self;          // = xp + in_size * pitch: where h_t of this layer goes
    uint8_t* xp_next;          // the input rows of the layer above, or null
    int rows, cols, n_ctas, RG;
};
struct SpmmLoop {
    SpmmLoopLayer layer[kMaxLayers];
    float* Z; long long ldz;   // pre-activations of the layer being worked on: [product rows][gates * H]
    const float* x;            // [T, B, I0]
    float* y;                  // [T, B, H] or null
    uint8_t* xp0;              // packed inputs of layer 0 (x_{t+1} is packed into its first I0 rows)
    unsigned int* gbar;        // grid barrier counter, zero at launch
    unsigned long long barrier_ns;
    int T, L, B, H, I0, gates, cap;
};

#ifdef CSB_SPMM_CLOCKS
#define SPMM_LAP(i) do { const long long n_ = clock64(); sprof[i] += n_ - st_; st_ = n_; } while (0)
#else
#define SPMM_LAP(i) do { } while (0)
#endif

// Shared-memory carve-up, identical on host and device.  The small fixed part comes first; the two
// rings follow and are reused for the warps' partial sums once the main loop is over.
// Floats per row of a warp's sums in shared memory: the fragments go in with 8-byte stores and a row
// comes out with 16-byte loads, both without bank conflicts at this pitch.
__host__ __device__ constexpr int spmm_sum_pitch(int NT) { return NT == 1 ? 8 : 8 * NT + 8; }
__host__ __device__ constexpr size_t spmm_q_bytes(int NT, int group_rows) { return (size_t)8 * NT * (group_rows + 1) * 4; }

struct SpmmSmem {
    size_t wfull, xfull, wcnt, xcnt, dead, zero, extra, rings, wring, xring, qsums, total;
    // q_bytes: room for the CTA's own sums of its row group; extra_bytes: a region outside the rings (the time
    // loop's tile of the gate arithmetic, which runs while the next pass's first weights are on their way)
    __host__ __device__ SpmmSmem(int n_warps, int w_stages, int x_depth, int tile_bytes, int pitch, int MT, int NT, size_t q_bytes,
                                 size_t extra_bytes = 0) {
        const int n_streams = n_warps;
        wfull = 0;
        xfull = wfull + (size_t)n_streams * w_stages * 8;
        wcnt = xfull + (size_t)x_depth * 8;
        xcnt = wcnt + (size_t)n_streams * w_stages * 4;
        dead = xcnt + (size_t)x_depth * 4;
        zero = (dead + 4 + 127) & ~(size_t)127;
        extra = (zero + (size_t)pitch + 127) & ~(size_t)127;
        rings = (extra + extra_bytes + 127) & ~(size_t)127;
        wring = rings;
        xring = wring + (size_t)n_streams * w_stages * kSpmmStageBytes;
        const size_t ring_end = xring + (size_t)x_depth * tile_bytes;
        qsums = (rings + (size_t)n_warps * MT * 16 * spmm_sum_pitch(NT) * 4 + 127) & ~(size_t)127;
        const size_t sums_end = qsums + q_bytes;
        total = ring_end > sums_end ? ring_end : sums_end;
    }
};

// Pack X: fp32 [batch][cols] -> per column one row of binary16 values: the hi parts of the 8 * NT batch
// columns, then the lo parts (x = hi + lo); batch columns past nb are zero.
__global__ void csb_pack_x_kernel(const float* __restrict__ X, long long ldx, int nb, int cols, uint8_t* __restrict__ xp, int pitch, int NT) {
    pdl_launch_dependents();
    pdl_wait();                                    // X may come from the kernel in front; xp may still be read by it
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5, c0 = blockIdx.x * 32;
    const int cap = 8 * NT;
    for (int b = ty; b < cap; b += 8) tile[b][tx] = (b < nb && c0 + tx < cols) ? X[(long long)b * ldx + c0 + tx] : 0.f;
    __syncthreads();
    for (int idx = threadIdx.x; idx < 32 * cap; idx += blockDim.x) {
        const int c = idx / cap, b = idx % cap;
        if (c0 + c >= cols) break;
        const float x = tile[b][c];
        const __half hi = __float2half_rn(x);
        const __half lo = __float2half_rn(x - __half2float(hi));
        __half* row = reinterpret_cast<__half*>(xp + (size_t)(c0 + c) * pitch);
        row[b] = hi;
        row[cap + b] = lo;
    }
}

__device__ __forceinline__ void mma_m16n8k16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ uint32_t atom_add_acq_rel_shared(uint32_t* p, uint32_t v) {
    uint32_t old;
    asm volatile("atom.acq_rel.cta.shared.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(smem_u32(p)), "r"(v) : "memory");
    return old;
}

// Thread-block cluster: barrier over all threads of all CTAs of the cluster (release / acquire), this
// CTA's rank, the address of a shared-memory location in another CTA of the cluster, and a load from it.
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cluster_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
// n / d for 0 <= n < 2^23 through the reciprocal inv = 1 / d (a handful of instructions where the
// integer division is a few dozen; the epilogue divides several times per output)
__device__ __forceinline__ int div_small(int n, int d, float inv) {
    int q = __float2int_rz(__int2float_rn(n) * inv);
    if (q * d > n) --q;
    else if ((q + 1) * d <= n) ++q;
    return q;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

__device__ __forceinline__ unsigned int ld_acquire_gpu_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// One product pass (LOOP = false: the whole kernel), or the time loop of a recurrent stack around it.
template <int MT, int NT, bool LOOP>
__device__ __forceinline__ void spmm_tile_body(SpmmArgs a, const SpmmLoop* lp) {
    constexpr int kSpmmWarps = NT == 1 ? 32 : 16;
    if (!LOOP) pdl_launch_dependents();
    extern __shared__ __align__(128) uint8_t smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const SpmmSmem L(kSpmmWarps, a.w_stages, a.x_depth, a.tile_bytes, a.pitch, MT, NT, spmm_q_bytes(NT, a.q_rows), LOOP ? kLoopTileBytes : 0);
    uint64_t* wfull = reinterpret_cast<uint64_t*>(smem + L.wfull) + warp * a.w_stages;
    uint64_t* xfull = reinterpret_cast<uint64_t*>(smem + L.xfull);
    uint32_t* xcnt = reinterpret_cast<uint32_t*>(smem + L.xcnt);
    volatile uint32_t* s_dead = reinterpret_cast<volatile uint32_t*>(smem + L.dead);
    uint8_t* wring = smem + L.wring + (size_t)warp * a.w_stages * kSpmmStageBytes;
    uint8_t* xring = smem + L.xring;
    const uint32_t zero_addr = smem_u32(smem + L.zero);

#ifdef CSB_SPMM_CLOCKS
    long long sprof[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
    long long st_ = clock64();
#endif
    // the CTA's descriptor goes to shared memory, one word per thread
    __shared__ __align__(16) SpmmCta s_me;
    __shared__ int s_first[5];                     // first warp of every block-row of the group (the warps of a row are neighbours)
    if (threadIdx.x == 0) {
        for (int i = 0; i < kSpmmWarps * a.w_stages; ++i) mbar_init(reinterpret_cast<uint64_t*>(smem + L.wfull) + i, 1);
        for (int i = 0; i < a.x_depth; ++i) { mbar_init(&xfull[i], 1); xcnt[i] = 0u; }
        *s_dead = 0u;
        mbar_fence_init();
    }
    for (int i = threadIdx.x; i < (a.pitch + 16) / 4; i += blockDim.x) reinterpret_cast<uint32_t*>(smem + L.zero)[i] = 0u;
    // ring positions: they run on from pass to pass of the time loop (every use of a slot is one phase of its barrier)
    int xs = 0, s = 0;                             // slot of the input ring the warp is at; stage of its weight ring
    uint32_t xpar = 0u, parity = 0u;               // and the parities of their current uses
    unsigned int gbar_round = 0;                   // grid barriers passed (time loop)
    // time loop: what the next pass starts with is fetched while this one ends
    bool primed = false;
    uint4 wd_next = make_uint4(0u, 0u, 0u, 0u);
    uint32_t me_word_next = 0u, issue_off_next = 0u;
    // The first chunks of a warp's weight stream go out, into the stages in ring order from where the warp
    // stands; returns where the next chunk to be fetched starts.  (A warp's chunks lie back to back.)
    auto first_weights = [&](const uint8_t* stream, const uint4& d) -> uint32_t {
        const uint32_t first[3] = {d.z & 0xffffu, d.z >> 16, d.w};
        uint32_t off = d.x;
        // (time loop: the rings were last touched by ordinary loads and stores, the sums of the pass in front,
        // which a CTA barrier separates from these copies)
        int si = s;
        for (int k = 0; k < a.w_stages && k < (int)d.y; ++k) {
            if (lane == 0) {
                mbar_expect_tx(&wfull[si], first[k]);
                bulk_g2s(wring + (size_t)si * kSpmmStageBytes, stream + (size_t)off * 16, first[k], &wfull[si]);
            }
            off += first[k] >> 4;
            if (++si == a.w_stages) si = 0;
        }
        return off;
    };
    const int n_pass = LOOP ? lp->T * lp->L : 1;
    for (int pass = 0; pass < n_pass; ++pass) {
    const int layer = LOOP ? pass % lp->L : 0, step = LOOP ? pass / lp->L : 0;
    bool pass_dead = false;
    if (LOOP) {
        const SpmmLoopLayer& ly = lp->layer[layer];
        a.stream = ly.stream; a.warp_desc = ly.warp_desc; a.ctas = ly.ctas; a.xp = ly.xp;
        a.rows = ly.rows; a.cols = ly.cols; a.RG = ly.RG; a.Y = lp->Z; a.ldy = lp->ldz;
    }
    if (!LOOP || (int)blockIdx.x < lp->layer[layer].n_ctas) {
    // (time loop: descriptors and first weights of this pass were fetched during the pass in front, where there was one)
    const bool was_primed = LOOP && primed;
    primed = false;
    if (threadIdx.x < sizeof(SpmmCta) / 4)
        reinterpret_cast<uint32_t*>(&s_me)[threadIdx.x] = was_primed ? me_word_next : reinterpret_cast<const uint32_t*>(a.ctas + blockIdx.x)[threadIdx.x];
    const uint4 wd = was_primed ? wd_next : __ldg(a.warp_desc + (size_t)blockIdx.x * kSpmmWarps + warp);
    const uint32_t n_chunks = wd.y;
    __syncthreads();
    const SpmmCta* me = &s_me;
    const int ntiles = me->ntiles, tile0 = me->tile0;
    auto tile_bytes_of = [&](int tl) { return (uint32_t)min(a.tile_cols, a.cols - (tile0 * a.block_c + tl * a.tile_cols)) * (uint32_t)a.pitch; };
    auto tile_src = [&](int tl) { return a.xp + (size_t)(tile0 * a.block_c + tl * a.tile_cols) * a.pitch; };
    // the weights were written at plan time: their first copies go out before the work in front is waited for
    // (a warp's chunks lie back to back; issue_off is where the next one to be fetched starts)
    uint32_t issue_off = was_primed ? issue_off_next : first_weights(a.stream, wd);
    if (threadIdx.x == 0) {
        int rr = 0;
        s_first[0] = 0;
        for (int w = 0; w < kSpmmWarps; ++w)
            while (rr < (int)me->warp_row[w]) s_first[++rr] = w;
        while (rr < 4) s_first[++rr] = kSpmmWarps;
    }
    if (!LOOP) pdl_wait();                         // the packed inputs and Y belong to the work in front on the stream
    // (time loop: the packed inputs were written with ordinary stores by other CTAs, before the grid barrier;
    // every lane that may issue a copy of them orders that behind its view of the barrier, once per pass)
    if (LOOP && lane == 0) fence_proxy_async_all();
    // One lane fetches a tile with one bulk copy.  (No proxy fence in front of a refill: the slot's
    // readers have their data in registers by the time they release it, and the release orders them
    // before this copy is issued.)
    auto fetch_tile = [&](int slot, int tl) {
        if (lane == 0) {
            mbar_expect_tx(&xfull[slot], tile_bytes_of(tl));
            bulk_g2s(xring + (size_t)slot * a.tile_bytes, tile_src(tl), tile_bytes_of(tl), &xfull[slot]);
        }
    };
    if (warp < a.x_depth && warp < ntiles) fetch_tile((xs + warp) % a.x_depth, warp);     // the first tiles, one warp each
    SPMM_LAP(0);                                   // set-up, first copies out, the work in front waited for
    // A wait gives up after a second, or as soon as any warp of the CTA has given up.
    auto wait_bar = [&](uint64_t* bar, uint32_t parity) -> bool {
        bool ok = mbar_try_wait(bar, parity);
        if (!ok) {
            unsigned long long t0 = 0;                // the clock is a slow read: only every 256 failed polls
            unsigned int spins = 0;
            for (;;) {
                if (mbar_try_wait_parked(bar, parity, 4000u)) { ok = true; break; }
                if ((++spins & 255u) == 0) {
                    if (*s_dead) break;
                    const unsigned long long now = global_ns();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > kCopyWaitNs) { *s_dead = 1u; *(volatile uint32_t*)a.status = (uint32_t)kDevCopyTimeout; break; }
                }
            }
        }
        return __all_sync(0xffffffffu, ok);          // the whole warp goes on, or none of it
    };
    // The tile this warp is at (tcur) sits in slot xs of the input ring, in the use of that slot with
    // parity xpar; both move along with tcur, so nothing is divided.
    int tcur = 0;
    auto wait_x = [&]() -> bool { return wait_bar(&xfull[xs], xpar); };
    // This warp is done with tile tcur; the last warp of the CTA to say so refills the slot.
    auto release_x = [&]() {
        __syncwarp();
        uint32_t last = 0u;
        // A plain (relaxed) add: the loads this warp made from the slot have all returned (the tensor
        // instructions that used them have been issued), and a fence here would also wait for the
        // weight copies this lane has in flight from HBM.
        if (lane == 0) {
            last = atomicAdd(&xcnt[xs], 1u) == (uint32_t)kSpmmWarps - 1u;
            if (last) *reinterpret_cast<volatile uint32_t*>(&xcnt[xs]) = 0u;
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last && tcur + a.x_depth < ntiles) fetch_tile(xs, tcur + a.x_depth);
        ++tcur;
        if (++xs == a.x_depth) { xs = 0; xpar ^= 1u; }
    };

    float acc[MT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;

    const uint32_t x_lane_off = (uint32_t)(lane >> 4) * 16u;                 // this lane's 16 bytes inside a tile row
    const int kr_lane = ((lane >> 3) & 1) * 8 + (lane & 7);                  // its k row inside a 16-column slab
    bool alive = true;
    for (uint32_t c = 0; c < n_chunks && alive; ++c) {
        SPMM_LAP(4);
        if (!wait_bar(&wfull[s], parity)) { alive = false; break; }
        SPMM_LAP(1);                               // waiting for weights
        const uint8_t* p = wring + (size_t)s * kSpmmStageBytes;
        const uint4 chh = *reinterpret_cast<const uint4*>(p);              // items' size, sizes of the next three chunks
        const uint8_t* end = p + 16 + 16 * (size_t)chh.x;
        const uint32_t refill_bytes = a.w_stages == 3 ? chh.w : chh.z;     // the chunk w_stages further on
        p += 16;
        while (p < end) {
            const uint4 h = *reinterpret_cast<const uint4*>(p);
            const int tile = (int)(h.x & 0xffffu), nk = (int)((h.x >> 16) & 0xffu), np2 = (int)(h.x >> 24);
            const uint32_t mask_lo = h.y, mask_hi = h.z;
            const uint8_t* cidx = p + 16;
            const uint32_t vals = smem_u32(cidx + ((nk + 3) & ~3));
            p += 16 * (size_t)(h.w & 0xffffu);
            // tiles this warp has no block in are passed in order
            SPMM_LAP(4);
            while (tcur < tile && alive) {
                if (!wait_x()) { alive = false; break; }
                release_x();
            }
            if (!alive || !wait_x()) { alive = false; break; }
            SPMM_LAP(2);                           // passing tiles and waiting for this item's tile
            const uint32_t xtile = smem_u32(xring + (size_t)xs * a.tile_bytes);
            // address of this lane's words in the stored row behind each of its output rows (rows that are
            // not kept have none).  Lane l works out where in-block rows l and l + 32 are stored (a
            // population count on the row mask) and the lanes fetch what they need by shuffle.
            uint32_t rowaddr[MT][2];
            {
                const uint32_t below = (1u << lane) - 1u;
                const uint32_t e_lo = ((mask_lo >> lane) & 1u) ? (uint32_t)__popc(mask_lo & below) : 0xffffu;
                const uint32_t e_hi = ((mask_hi >> lane) & 1u) ? (uint32_t)(__popc(mask_lo) + __popc(mask_hi & below)) : 0xffffu;
                const uint32_t mine = e_lo | (e_hi << 16);
#pragma unroll
                for (int q = 0; q < (MT < 2 ? MT : 2); ++q)
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        const uint32_t v = __shfl_sync(0xffffffffu, mine, 16 * q + g + 8 * hh);
                        const uint32_t lo = v & 0xffffu, hi = v >> 16;
                        rowaddr[q][hh] = lo != 0xffffu ? vals + (lo * (uint32_t)np2 + (uint32_t)t) * 4u : kNoRow;
                        if (MT > 2) rowaddr[(q + 2) % MT][hh] = hi != 0xffffu ? vals + (hi * (uint32_t)np2 + (uint32_t)t) * 4u : kNoRow;
                    }
            }
            for (int kb = 0; kb < nk; kb += 16) {
                // ---- B operand: the gathered inputs, 16 kept columns x this warp's batch columns
                const int kr = kb + kr_lane;
                const uint32_t rowp = (kr < nk ? xtile + (uint32_t)cidx[kr] * (uint32_t)a.pitch : zero_addr) + x_lane_off;
                uint32_t bh[NT][2], bl[NT][2];
                if (NT == 1) {
                    uint32_t r4[4];
                    ldmatrix_x4_trans(r4, rowp);                       // (hi, k 0-7), (hi, k 8-15), (lo, k 0-7), (lo, k 8-15)
                    bh[0][0] = r4[0]; bh[0][1] = r4[1]; bl[0][0] = r4[2]; bl[0][1] = r4[3];
                } else {
#pragma unroll
                    for (int q = 0; q < NT / 2; ++q) {
                        uint32_t r4[4];
                        ldmatrix_x4_trans(r4, rowp + 32u * q);         // batch tiles 2q, 2q + 1 of the hi part
                        bh[2 * q][0] = r4[0]; bh[2 * q][1] = r4[1]; bh[(2 * q + 1) % NT][0] = r4[2]; bh[(2 * q + 1) % NT][1] = r4[3];
                        ldmatrix_x4_trans(r4, rowp + 16u * NT + 32u * q);   // the same of the lo part
                        bl[2 * q][0] = r4[0]; bl[2 * q][1] = r4[1]; bl[(2 * q + 1) % NT][0] = r4[2]; bl[(2 * q + 1) % NT][1] = r4[3];
                    }
                }
                // ---- A operand: the kernel matrix with its rows at their RowIdx positions.  Words past the
                // end of a stored row (last slab of a slice that is not a multiple of 16 wide) are zero.
                const uint32_t koff = (uint32_t)kb * 2u;                             // bytes into a stored row
                const bool v0 = (uint32_t)(kb >> 1) + (uint32_t)t < (uint32_t)np2, v1 = (uint32_t)(kb >> 1) + (uint32_t)t + 4u < (uint32_t)np2;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    uint32_t af[4];
                    af[0] = (rowaddr[mt][0] != kNoRow && v0) ? lds_u32(rowaddr[mt][0] + koff) : 0u;
                    af[1] = (rowaddr[mt][1] != kNoRow && v0) ? lds_u32(rowaddr[mt][1] + koff) : 0u;
                    af[2] = (rowaddr[mt][0] != kNoRow && v1) ? lds_u32(rowaddr[mt][0] + koff + 16u) : 0u;
                    af[3] = (rowaddr[mt][1] != kNoRow && v1) ? lds_u32(rowaddr[mt][1] + koff + 16u) : 0u;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        mma_m16n8k16(acc[mt][nt], af, bh[nt][0], bh[nt][1]);
                        mma_m16n8k16(acc[mt][nt], af, bl[nt][0], bl[nt][1]);
                    }
                }
            }
            SPMM_LAP(3);                           // row map, operand loads, tensor instructions
        }
        if (!alive) break;
        // this warp is done with the stage and refills it
        __syncwarp();
        if (refill_bytes) {
            if (lane == 0) {
                mbar_expect_tx(&wfull[s], refill_bytes);
                bulk_g2s(wring + (size_t)s * kSpmmStageBytes, a.stream + (size_t)issue_off * 16, refill_bytes, &wfull[s]);
            }
            issue_off += refill_bytes >> 4;
        }
        if (++s == a.w_stages) { s = 0; parity ^= 1u; }
    }
    SPMM_LAP(4);                                   // ring bookkeeping
    while (tcur < ntiles && alive) {
        if (!wait_x()) { alive = false; break; }
        release_x();
    }
    SPMM_LAP(5);                                   // the tiles behind this warp's last item
    if (LOOP && pass + 1 < n_pass) {
        // descriptors of this CTA in the next pass: asked for now, used once the sums below are done
        const SpmmLoopLayer& nx = lp->layer[(pass + 1) % lp->L];
        if ((int)blockIdx.x < nx.n_ctas) {
            wd_next = __ldg(nx.warp_desc + (size_t)blockIdx.x * kSpmmWarps + warp);
            if (threadIdx.x < sizeof(SpmmCta) / 4) me_word_next = __ldg(reinterpret_cast<const uint32_t*>(nx.ctas + blockIdx.x) + threadIdx.x);
            primed = true;
        }
    }
    __syncthreads();
    SPMM_LAP(6);                                   // waiting for the other warps of the CTA
    const bool dead = *s_dead != 0u;
    if (dead) {
        // a wait gave up (the status word says so): give copies that may still be in flight a bounded
        // time to land before the CTA's shared memory goes away, and write nothing
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        if (!LOOP && a.S == 1) return;             // (a CTA of a cluster still has to keep the cluster's barriers company)
        pass_dead = true;
    }

    // ---- the warps' sums meet in shared memory (the rings are no longer in use)
    constexpr int kP = spmm_sum_pitch(NT);
    float* P = reinterpret_cast<float*>(smem + L.rings);           // [warp][row of the block][kP]
    {
        float* Pw = P + (size_t)warp * MT * 16 * kP;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float* q = Pw + (16 * mt + g) * kP + 8 * nt + 2 * t;
                *reinterpret_cast<float2*>(q) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
                *reinterpret_cast<float2*>(q + 8 * kP) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
            }
    }
    __syncthreads();
    SPMM_LAP(7);                                   // accumulators to shared memory
    const int group_rows = a.RG * a.block_r, row0 = me->group * group_rows;
    const int nrows = min(group_rows, a.rows - row0);
    // this CTA's sums over its range: [batch column][row of the group], one float of padding per column
    // (written four columns at a time without bank conflicts, read by the cluster in runs of consecutive rows)
    float* part = reinterpret_cast<float*>(smem + L.qsums);
    const int kQ = group_rows + 1;
    {
        // one thread per row and four batch columns; the warps of a block-row are added in warp order
        constexpr int kQuads = 2 * NT;
        const int total = dead ? 0 : nrows * kQuads;
        const float inv_br = 1.f / (float)a.block_r;
        // (four of a thread's outputs at a time, so that their loads are in flight together)
        for (int i0 = threadIdx.x; i0 < total; i0 += 4 * blockDim.x) {
            const float* src[4];
            int cnt[4], rl[4], q4[4], cmax = 0;
            float4 sum[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = min(i0 + j * (int)blockDim.x, total - 1);
                rl[j] = i / kQuads; q4[j] = i % kQuads;
                const int rr = div_small(rl[j], a.block_r, inv_br), rin = rl[j] - rr * a.block_r;
                const int w0 = s_first[rr];
                cnt[j] = s_first[rr + 1] - w0;
                cmax = max(cmax, cnt[j]);
                src[j] = P + ((size_t)w0 * MT * 16 + rin) * kP + 4 * q4[j];
                sum[j] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            for (int k = 0; k < cmax; ++k) {
                float4 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) v[j] = k < cnt[j] ? *reinterpret_cast<const float4*>(src[j] + (size_t)k * MT * 16 * kP) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int j = 0; j < 4; ++j) { sum[j].x += v[j].x; sum[j].y += v[j].y; sum[j].z += v[j].z; sum[j].w += v[j].w; }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (i0 + j * (int)blockDim.x < total) {
                    float* dst = part + 4 * q4[j] * kQ + rl[j];
                    dst[0] = sum[j].x; dst[kQ] = sum[j].y; dst[2 * kQ] = sum[j].z; dst[3 * kQ] = sum[j].w;
                }
        }
    }
    __syncthreads();
    SPMM_LAP(8);                                   // sums over the warps of a block-row
    // The S CTAs of a row group form a thread-block cluster.  Once all of them have their sums in shared
    // memory, every CTA adds up the S ranges, in range order, for its share of the group's rows, reading
    // the other CTAs' sums through distributed shared memory; nobody leaves before everybody has read.
    // (The CTA barriers in front keep each warp together for the aligned cluster barrier.)
    if (a.S > 1) cluster_barrier();
    SPMM_LAP(9);                                   // waiting for the cluster's other CTAs
    {
        const uint32_t rank = a.S > 1 ? cluster_rank() : 0u;
        const int share = (nrows + a.S - 1) / a.S, r_lo = min(nrows, (int)rank * share), r_n = min(nrows, r_lo + share) - r_lo;
        const uint32_t q_local = smem_u32(part);
        uint32_t q_of[8];
#pragma unroll
        for (int s2 = 0; s2 < 8; ++s2) q_of[s2] = a.S > 1 && s2 < a.S ? map_to_cluster_cta(q_local, (uint32_t)s2) : q_local;
        // a warp takes batch columns, its lanes consecutive rows: stores of 128 contiguous bytes
        // (two batch columns x two runs of rows per lane at a time: up to 32 remote loads in flight)
        for (int b0 = warp; b0 < (dead ? 0 : a.nb); b0 += 2 * kSpmmWarps)
            for (int r0 = lane; r0 < r_n; r0 += 64) {
                float v[4][8];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int b = b0 + (j >> 1) * kSpmmWarps, r = r0 + (j & 1) * 32;
                    const bool live = b < a.nb && r < r_n;
                    const uint32_t off = (uint32_t)(b * kQ + r_lo + r) * 4u;
#pragma unroll
                    for (int s2 = 0; s2 < 8; ++s2) {
                        if (a.S > 1) v[j][s2] = live && s2 < a.S ? ld_cluster_f32(q_of[s2] + off) : 0.f;
                        else v[j][s2] = live && s2 == 0 ? part[b * kQ + r_lo + r] : 0.f;
                    }
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int b = b0 + (j >> 1) * kSpmmWarps, r = r0 + (j & 1) * 32;
                    float sum = v[j][0];
#pragma unroll
                    for (int s2 = 1; s2 < 8; ++s2) sum += v[j][s2];
                    if (b < a.nb && r < r_n) a.Y[(long long)b * a.ldy + row0 + r_lo + r] = sum;
                }
            }
    }
    SPMM_LAP(10);                                  // sums over the ranges, store
    if (a.S > 1) {
        __syncthreads();
        cluster_barrier();
    }
    SPMM_LAP(11);                                  // until every CTA of the cluster has read
    // (time loop) the rings are free again: the next pass's first weights go out and land while the gates are done
    if (LOOP) {
        __syncthreads();                           // every thread is done reading the sums that lie where the rings are
        if (primed && !pass_dead) issue_off_next = first_weights(lp->layer[(pass + 1) % lp->L].stream, wd_next);
        else primed = false;
    }
    }                                              // (CTAs beyond this layer's plan sit the pass out)
    if (LOOP) {
        // ---- every CTA's part of Z is written: gate arithmetic of (layer, step), then on to the next pass.
        // A CTA that gave up does not come here; the others then run into the bound of the barrier.
        if (pass_dead) break;
        auto grid_sync = [&]() -> bool {
            __syncthreads();
            ++gbar_round;
            if (threadIdx.x == 0) {
                __threadfence();
                atomicAdd(lp->gbar, 1u);
                const unsigned int target = gbar_round * gridDim.x;
                unsigned long long t0 = 0;
                unsigned int spins = 0;
                while (ld_acquire_gpu_u32(lp->gbar) < target) {
                    if ((++spins & 63u) == 0) {
                        const unsigned long long now = global_ns();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > lp->barrier_ns) { *s_dead = 1u; *(volatile uint32_t*)a.status = (uint32_t)kDevBarrierTimeout; break; }
                    }
                }
            }
            __syncthreads();
            return *s_dead == 0u;
        };
        SPMM_LAP(15);                              // (time loop) next pass's first weights out
        if (!grid_sync()) break;
        SPMM_LAP(12);                              // (time loop) grid barrier behind the product pass
        {
            const SpmmLoopLayer& ly = lp->layer[layer];
            float (*tile)[33] = reinterpret_cast<float (*)[33]>(smem + L.extra);
            const int B = lp->B, H = lp->H, h_tiles = (H + 31) / 32;
            const bool pack_x = layer == 0 && step + 1 < lp->T;
            const int n_tiles = h_tiles + (pack_x ? (lp->I0 + 31) / 32 : 0);
            float* y_t = (layer == lp->L - 1 && lp->y) ? lp->y + (size_t)step * B * H : nullptr;
            for (int tl = blockIdx.x; tl < n_tiles; tl += gridDim.x) {
                if (tl < h_tiles) {
                    if (lp->gates == 4) lstm_gates_tile(tile, lp->Z, ly.bias, ly.c, ly.hs, ly.xp_self, ly.xp_next, y_t, a.pitch, lp->cap, B, H, tl * 32);
                    else gru_gates_tile(tile, lp->Z, ly.bias, ly.hs, ly.xp_self, ly.xp_next, y_t, a.pitch, lp->cap, B, H, tl * 32);
                } else {
                    pack_columns(tile, lp->x + (size_t)(step + 1) * B * lp->I0, (long long)lp->I0, B, lp->I0, (tl - h_tiles) * 32, lp->xp0,
                                 a.pitch, lp->cap, 0);
                }
                __syncthreads();                   // the tile is free again
            }
        }
        SPMM_LAP(13);                              // (time loop) gate arithmetic
        if (pass + 1 < n_pass && !grid_sync()) break;
        SPMM_LAP(14);                              // (time loop) grid barrier behind the gates
    }
    }                                              // passes
#ifdef CSB_SPMM_CLOCKS
    if (lane == 0) for (int i = 0; i < 16; ++i) a.clocks[((size_t)blockIdx.x * kSpmmWarps + warp) * 16 + i] = sprof[i];
#endif
}

template <int MT, int NT>
__global__ void __launch_bounds__((NT == 1 ? 32 : 16) * 32, 1) csb_spmm_tile_kernel(const SpmmArgs a) {
    spmm_tile_body<MT, NT, false>(a, nullptr);
}

// The recurrent time loop (see SpmmLoop): launched cooperatively, so that the bounded grid barriers can be passed.
template <int MT, int NT>
__global__ void __launch_bounds__((NT == 1 ? 32 : 16) * 32, 1) csb_rnn_tile_kernel(const SpmmArgs a, const __grid_constant__ SpmmLoop lp) {
    spmm_tile_body<MT, NT, true>(a, &lp);
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
    if (!(batch >= 8 && A->val_dtype == CSB_F16 && A->block_r <= 64 && A->device >= 0)) return false;
    return !(A->mma && A->mma->cls[spmm_class_index(batch)].unusable);
}

template <typename V>
static int upload_v(const std::vector<V>& h, V** d) {
    const size_t bytes = std::max<size_t>(h.size(), 1) * sizeof(V);
    CSB_CUDA(cudaMalloc((void**)d, bytes));
    if (!h.empty()) CSB_CUDA(cudaMemcpy(*d, h.data(), h.size() * sizeof(V), cudaMemcpyHostToDevice));
    return CSB_OK;
}

static int mt_of(const csb_matrix* A) { return A->block_r <= 16 ? 1 : A->block_r <= 32 ? 2 : 4; }

template <int MT, int NT>
static cudaError_t set_smem_attr(size_t bytes) {
    return cudaFuncSetAttribute(csb_spmm_tile_kernel<MT, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}
template <int MT, int NT>
static cudaError_t max_clusters(int* n, const cudaLaunchConfig_t* cfg) {
    return cudaOccupancyMaxActiveClusters(n, csb_spmm_tile_kernel<MT, NT>, cfg);
}
template <int MT, int NT>
static cudaError_t launch_tile_kernel(const cudaLaunchConfig_t* cfg, const SpmmArgs& a) {
    return cudaLaunchKernelEx(cfg, csb_spmm_tile_kernel<MT, NT>, a);
}
#define CSB_SPMM_DISPATCH(fn, MT, NT, ...)                                                                        \
    ((MT) == 1 ? ((NT) == 1 ? fn<1, 1>(__VA_ARGS__) : (NT) == 2 ? fn<1, 2>(__VA_ARGS__) : fn<1, 4>(__VA_ARGS__))  \
     : (MT) == 2 ? ((NT) == 1 ? fn<2, 1>(__VA_ARGS__) : (NT) == 2 ? fn<2, 2>(__VA_ARGS__) : fn<2, 4>(__VA_ARGS__)) \
                 : ((NT) == 1 ? fn<4, 1>(__VA_ARGS__) : (NT) == 2 ? fn<4, 2>(__VA_ARGS__) : fn<4, 4>(__VA_ARGS__)))

static int build_spmm_plan(const csb_matrix* A, int ci, MmaPlan::PerClass* P) {
    const int NT = 1 << ci;
    SpmmHostPlan H;
    const int sms = A->opts.ctas > 0 ? A->opts.ctas : A->sm_count;
    int rc = plan_spmm_host(A, NT, sms, &H);
    if (rc == 1) { P->unusable = true; return CSB_OK; }
    if (rc != CSB_OK) return rc;
    const int MT = mt_of(A), pitch = spmm_pitch(NT);
    const int tile_bytes = (spmm_tile_blocks(A->block_c) * A->block_c * pitch + 127) & ~127;
    // rings: as many weight stages (3, else 2) and input tiles (up to 8, at least 2) as shared memory holds
    int w_stages = 0, x_depth = 0;
    size_t smem = 0;
    for (int ws = 3; ws >= 2 && !x_depth; --ws)
        for (int xd = std::min(8, std::max(2, H.max_tiles)); xd >= 2; --xd) {
            const SpmmSmem L(spmm_warps(NT), ws, xd, tile_bytes, pitch, MT, NT, spmm_q_bytes(NT, H.RG * A->block_r));
            if (L.total + kSpmmStaticSmem <= A->smem_optin) { w_stages = ws; x_depth = xd; smem = L.total; break; }
        }
    if (!x_depth) { P->unusable = true; return CSB_OK; }
    P->RG = H.RG; P->S = H.S; P->n_ctas = (int)H.ctas.size(); P->n_groups = H.n_groups;
    P->w_stages = w_stages; P->x_depth = x_depth; P->smem_bytes = smem; P->balance = H.balance; P->warp_balance = H.warp_balance;
    P->stream_bytes = (int64_t)H.bytes.size();
    if ((rc = upload_v(H.bytes, &P->d_stream)) != CSB_OK) return rc;
    if ((rc = upload_v(H.warp_desc, &P->d_warp_desc)) != CSB_OK) return rc;
    if ((rc = upload_v(H.ctas, &P->d_ctas)) != CSB_OK) return rc;
    const size_t xp_bytes = (size_t)A->nbc * A->block_c * pitch;          // whole tiles, so that a tile copy never runs past the end
    CSB_CUDA(cudaMalloc(&P->d_xp, xp_bytes));
    CSB_CUDA(cudaMemset(P->d_xp, 0, xp_bytes));
    // (the limit belongs to the kernel, not to this plan: other matrices launch the same instantiation with other sizes)
    CSB_CUDA(CSB_SPMM_DISPATCH(set_smem_attr, MT, NT, A->smem_optin - kSpmmStaticSmem));
    if (H.S > 1) {
        // the S CTAs of a row group are launched as one cluster: make sure such a cluster can be resident
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)H.S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3((unsigned)H.ctas.size()); cfg.blockDim = dim3((unsigned)spmm_warps(NT) * 32u); cfg.dynamicSmemBytes = smem;
        cfg.attrs = attr; cfg.numAttrs = 1;
        int clusters = 0;
        CSB_CUDA(CSB_SPMM_DISPATCH(max_clusters, MT, NT, &clusters, &cfg));
        if (clusters < 1) { P->unusable = true; return CSB_OK; }
    }
    CSB_CUDA(cudaDeviceSynchronize());
    P->built = true;
    return CSB_OK;
}

void free_mma(csb_matrix* A) {
    if (!A->mma) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(A->device);
    for (auto& c : A->mma->cls) {
        cudaFree(c.d_stream); cudaFree(c.d_warp_desc); cudaFree(c.d_ctas);
        cudaFree(c.d_xp);
    }
    cudaSetDevice(prev);
    delete A->mma;
    A->mma = nullptr;
}

#ifdef CSB_SPMM_CLOCKS
static long long* g_spmm_clocks = nullptr;
static int g_spmm_clock_warps = 0;
extern "C" int csb_debug_spmm_clocks(long long* host_out, int max_warps) {
    cudaMemcpy(host_out, g_spmm_clocks, (size_t)std::min(max_warps, g_spmm_clock_warps) * 16 * 8, cudaMemcpyDeviceToHost);
    return g_spmm_clock_warps;
}
#endif

// The plan of A for batch class ci, built on first use (the device of A is current).  CSB_OK, an error, or 1 = the
// tensor-core layout does not serve this matrix.
static int ensure_spmm_plan(const csb_matrix* A, int ci) {
    std::lock_guard<std::mutex> lk(A->mma_mu);
    if (!A->mma) {
        A->mma = new (std::nothrow) MmaPlan();
        if (!A->mma) { set_error("out of host memory"); return CSB_ERR_ALLOC; }
    }
    MmaPlan::PerClass& C = A->mma->cls[ci];
    if (!C.built && !C.unusable) {
        int rc;
        try { rc = build_spmm_plan(A, ci, &C); }
        catch (const std::bad_alloc&) { set_error("out of host memory while planning the batched product"); rc = CSB_ERR_ALLOC; }
        if (rc != CSB_OK) { C.unusable = true; return rc; }
    }
    return (C.unusable || !C.built) ? 1 : CSB_OK;
}

// Returns CSB_OK after launching, or 1 when the caller should use the CUDA-core path.
// With `packed` (and X == nullptr) the inputs are taken from a buffer the caller has filled in the
// packed layout of the batch's class (one row of spmm_pitch(NT) bytes per matrix column: the hi parts of
// 8 * NT batch slots, then the lo parts); a single pass, so at most 32 batch columns.
int launch_spmm_mma(const csb_matrix* A, const float* X, int64_t ldx, int batch, float* Y, int64_t ldy, void* stream, const uint8_t* packed) {
    if (packed && batch > 32) { set_error("pre-packed inputs serve at most 32 batch columns"); return CSB_ERR_INVALID_ARG; }
    const ProductPlan& PP = A->product;
    if (PP.h_status && *PP.h_status != 0) { set_error("an earlier product on this handle gave up waiting on the device (code %u)", *PP.h_status); return CSB_ERR_TIMEOUT; }
    int prev = 0;
    CSB_CUDA(cudaGetDevice(&prev));
    if (prev != A->device) CSB_CUDA(cudaSetDevice(A->device));
    struct Restore { int prev, cur; ~Restore() { if (prev != cur) cudaSetDevice(prev); } } restore{prev, A->device};
    const int ci = spmm_class_index(batch);
    {
        const int rc = ensure_spmm_plan(A, ci);
        if (rc != CSB_OK) return rc;
    }
    const MmaPlan::PerClass& P = A->mma->cls[ci];
    const int NT = 1 << ci, MT = mt_of(A), cap = 8 * NT;
    cudaStream_t st = (cudaStream_t)stream;
    SpmmArgs a{};
    a.stream = P.d_stream; a.warp_desc = (const uint4*)P.d_warp_desc; a.ctas = P.d_ctas;
    a.xp = packed ? packed : (const uint8_t*)P.d_xp; a.ldy = ldy; a.status = PP.d_status;
    a.rows = (int)A->rows; a.cols = (int)A->cols; a.block_r = A->block_r; a.block_c = A->block_c;
    a.RG = P.RG; a.S = P.S; a.x_depth = P.x_depth; a.w_stages = P.w_stages; a.q_rows = P.RG * A->block_r;
    a.tile_cols = spmm_tile_blocks(A->block_c) * A->block_c;
    a.pitch = spmm_pitch(NT); a.tile_bytes = (a.tile_cols * a.pitch + 127) & ~127;
#ifdef CSB_SPMM_CLOCKS
    if (!g_spmm_clocks) cudaMalloc((void**)&g_spmm_clocks, (size_t)1 << 24);
    a.clocks = g_spmm_clocks;
    g_spmm_clock_warps = P.n_ctas * spmm_warps(NT);
#endif
    for (int b0 = 0; b0 < batch; b0 += cap) {
        a.nb = std::min(cap, batch - b0);
        a.Y = Y + (int64_t)b0 * ldy;
        // both kernels order themselves behind the work in front (pdl_wait), so they may be launched
        // with programmatic stream serialization: their scheduling overlaps its tail
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;             // the CTAs that share a row group
        attr[1].val.clusterDim.x = (unsigned)P.S; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
        cudaLaunchConfig_t cfg{};
        cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = 1;
        cfg.gridDim = dim3((unsigned)((A->cols + 31) / 32)); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0;
        if (!packed)
            CSB_CUDA(cudaLaunchKernelEx(&cfg, csb_pack_x_kernel, X + (int64_t)b0 * ldx, (long long)ldx, a.nb, (int)A->cols, (uint8_t*)P.d_xp,
                                        a.pitch, NT));
        cfg.gridDim = dim3((unsigned)P.n_ctas); cfg.blockDim = dim3((unsigned)spmm_warps(NT) * 32u); cfg.dynamicSmemBytes = P.smem_bytes;
        cfg.numAttrs = P.S > 1 ? 2 : 1;
        CSB_CUDA(CSB_SPMM_DISPATCH(launch_tile_kernel, MT, NT, &cfg, a));
        CSB_CUDA(cudaGetLastError());
    }
    return CSB_OK;
}

template <int MT, int NT>
static cudaError_t set_loop_smem_attr(size_t bytes) {
    return cudaFuncSetAttribute(csb_rnn_tile_kernel<MT, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}
template <int MT, int NT>
static cudaError_t max_loop_clusters(int* n, const cudaLaunchConfig_t* cfg) {
    return cudaOccupancyMaxActiveClusters(n, csb_rnn_tile_kernel<MT, NT>, cfg);
}
template <int MT, int NT>
static cudaError_t launch_loop_kernel(const cudaLaunchConfig_t* cfg, const SpmmArgs& a, const SpmmLoop& lp) {
    return cudaLaunchKernelEx(cfg, csb_rnn_tile_kernel<MT, NT>, a, lp);
}

// The whole sequence of a recurrent stack in one cooperative launch of the product kernel's time loop.
// Returns CSB_OK after launching, an error, or 1 when the loop does not serve this stack (layers whose
// plans differ in block shape or cluster size, a plan that does not fit, a grid that cannot be
// co-resident): the caller then issues the steps as separate launches.  The device of W[0] is current.
int launch_rnn_tile_loop(const RnnTileLoop& R, void* stream) {
    const csb_matrix* A0 = R.W[0];
    const int vrows = R.gates == 3 ? 2 * R.B : R.B;
    if (vrows > 32 || R.L > kMaxLayers) return 1;
    const int ci = spmm_class_index(vrows), NT = 1 << ci, MT = mt_of(A0);
    SpmmArgs a{};
    SpmmLoop lp{};
    int S = 0, n_ctas = 0, w_stages = 3, x_depth = 8, q_rows = 0;
    for (int l = 0; l < R.L; ++l) {
        const csb_matrix* A = R.W[l];
        if (A->block_r != A0->block_r || A->block_c != A0->block_c || A->device != A0->device) return 1;
        const int rc = ensure_spmm_plan(A, ci);
        if (rc != CSB_OK) return rc;
        if (A->product.h_status && *A->product.h_status != 0) { set_error("an earlier product on a layer's handle gave up waiting on the device"); return CSB_ERR_TIMEOUT; }
        const MmaPlan::PerClass& P = A->mma->cls[ci];
        if (l == 0) S = P.S;
        if (P.S != S) return 1;                              // one cluster shape per launch
        n_ctas = std::max(n_ctas, P.n_ctas);
        w_stages = std::min(w_stages, P.w_stages); x_depth = std::min(x_depth, P.x_depth);
        q_rows = std::max(q_rows, P.RG * A->block_r);
        SpmmLoopLayer& ly = lp.layer[l];
        ly.stream = P.d_stream; ly.warp_desc = (const uint4*)P.d_warp_desc; ly.ctas = P.d_ctas; ly.xp = R.xp[l];
        ly.bias = R.bias ? R.bias[l] : nullptr;
        ly.c = R.c ? R.c + (size_t)l * R.B * R.H : nullptr;
        ly.hs = R.hs + (size_t)l * R.B * R.H;
        ly.xp_self = R.xp[l] + (size_t)R.in_size[l] * R.pitch;
        ly.xp_next = l + 1 < R.L ? R.xp[l + 1] : nullptr;
        ly.rows = (int)A->rows; ly.cols = (int)A->cols; ly.n_ctas = P.n_ctas; ly.RG = P.RG;
    }
    a.status = A0->product.d_status;
    a.nb = vrows; a.block_r = A0->block_r; a.block_c = A0->block_c; a.S = S; a.x_depth = x_depth; a.w_stages = w_stages; a.q_rows = q_rows;
    a.tile_cols = spmm_tile_blocks(A0->block_c) * A0->block_c;
    a.pitch = spmm_pitch(NT); a.tile_bytes = (a.tile_cols * a.pitch + 127) & ~127;
    if (a.pitch != R.pitch) { set_error("packed inputs of another batch class"); return CSB_ERR_INVALID_ARG; }
    // the loop's own tile may cost the input ring a slot
    while (x_depth > 2 && SpmmSmem(spmm_warps(NT), w_stages, x_depth, a.tile_bytes, a.pitch, MT, NT, spmm_q_bytes(NT, q_rows), kLoopTileBytes).total +
                                  kSpmmStaticSmem > A0->smem_optin)
        --x_depth;
    a.x_depth = x_depth;
    const SpmmSmem Lay(spmm_warps(NT), w_stages, x_depth, a.tile_bytes, a.pitch, MT, NT, spmm_q_bytes(NT, q_rows), kLoopTileBytes);
    if (Lay.total + kSpmmStaticSmem > A0->smem_optin) return 1;
#ifdef CSB_SPMM_CLOCKS
    if (!g_spmm_clocks) cudaMalloc((void**)&g_spmm_clocks, (size_t)1 << 24);
    a.clocks = g_spmm_clocks;
    g_spmm_clock_warps = n_ctas * spmm_warps(NT);
#endif
    lp.Z = R.z; lp.ldz = (long long)R.gates * R.H; lp.x = R.x; lp.y = R.y; lp.xp0 = R.xp[0]; lp.gbar = R.gbar;
    lp.barrier_ns = 2000000000ull;
    lp.T = (int)R.T; lp.L = R.L; lp.B = R.B; lp.H = R.H; lp.I0 = R.in_size[0]; lp.gates = R.gates; lp.cap = R.cap;
    cudaStream_t st = (cudaStream_t)stream;
    CSB_CUDA(CSB_SPMM_DISPATCH(set_loop_smem_attr, MT, NT, A0->smem_optin - kSpmmStaticSmem));
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)S; attr[1].val.clusterDim.y = 1; attr[1].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg{};
    cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = S > 1 ? 2 : 1;
    cfg.gridDim = dim3((unsigned)n_ctas); cfg.blockDim = dim3((unsigned)spmm_warps(NT) * 32u); cfg.dynamicSmemBytes = Lay.total;
    // every CTA must be resident at once, or the grid barrier cannot be passed
    int fit = 0;
    if (S > 1) {
        int clusters = 0;
        if (CSB_SPMM_DISPATCH(max_loop_clusters, MT, NT, &clusters, &cfg) != cudaSuccess) { cudaGetLastError(); return 1; }
        fit = clusters * S;
    } else {
        fit = A0->sm_count;                                  // one CTA of this size per SM
    }
    if (n_ctas > fit) return 1;
    if ((unsigned long long)2 * (unsigned long long)R.T * R.L * n_ctas >= (1ull << 32)) return 1;   // the barrier counts arrivals in 32 bits
    CSB_CUDA(cudaMemsetAsync(R.gbar, 0, 4, st));
    // a launch that is refused (a grid that cannot be co-resident after all) is no error: the caller issues the steps
    if (CSB_SPMM_DISPATCH(launch_loop_kernel, MT, NT, &cfg, a, lp) != cudaSuccess) { cudaGetLastError(); return 1; }
    return CSB_OK;
}

}  // namespace csb

// Inspection / testing aid: the plan of the batched product, made on the host only.
extern "C" int csb_spmm_plan_dump(const csb_matrix_t* A, int batch, int sm_count, int64_t* info_out, uint8_t* stream_out, int64_t stream_cap,
                                  uint32_t* chunks_out, int64_t chunks_cap, uint32_t* stream_begin_out, int64_t begin_cap, int32_t* cta_out,
                                  int64_t cta_cap) {
    using namespace csb;
    clear_error();
    if (!A || !info_out || batch < 1 || sm_count < 1) { set_error("csb_spmm_plan_dump: bad argument"); return CSB_ERR_INVALID_ARG; }
    SpmmHostPlan H;
    int rc;
    try { rc = plan_spmm_host(A, spmm_nt(batch), sm_count, &H); }
    catch (const std::bad_alloc&) { set_error("out of host memory while planning"); return CSB_ERR_ALLOC; }
    if (rc == 1) { set_error("the tensor-core layout does not apply to this matrix (fp16 values, block_r <= 64)"); return CSB_ERR_UNSUPPORTED; }
    if (rc != CSB_OK) return rc;
    info_out[0] = (int64_t)H.ctas.size(); info_out[1] = (int64_t)H.chunks.size(); info_out[2] = (int64_t)H.bytes.size();
    info_out[3] = H.RG; info_out[4] = spmm_nt(batch) | (spmm_warps(spmm_nt(batch)) << 8) | (spmm_tile_blocks(A->block_c) << 16); info_out[5] = H.S; info_out[6] = (int64_t)(H.warp_balance * 1e6);
    info_out[7] = (int64_t)(H.balance * 1e6);
    if (stream_out) {
        if (stream_cap < (int64_t)H.bytes.size()) { set_error("stream buffer too small"); return CSB_ERR_INVALID_ARG; }
        std::memcpy(stream_out, H.bytes.data(), H.bytes.size());
    }
    if (chunks_out) {
        if (chunks_cap < (int64_t)H.chunks.size()) { set_error("chunk buffer too small"); return CSB_ERR_INVALID_ARG; }
        for (size_t i = 0; i < H.chunks.size(); ++i) { chunks_out[2 * i] = H.chunks[i].off16; chunks_out[2 * i + 1] = H.chunks[i].bytes; }
    }
    if (stream_begin_out) {
        if (begin_cap < (int64_t)H.stream_begin.size()) { set_error("stream table too small"); return CSB_ERR_INVALID_ARG; }
        for (size_t i = 0; i < H.stream_begin.size(); ++i) stream_begin_out[i] = H.stream_begin[i];
    }
    if (cta_out) {
        if (cta_cap < (int64_t)H.ctas.size()) { set_error("CTA table too small"); return CSB_ERR_INVALID_ARG; }
        std::memcpy(cta_out, H.ctas.data(), H.ctas.size() * sizeof(SpmmCta));
    }
    return CSB_OK;
}
