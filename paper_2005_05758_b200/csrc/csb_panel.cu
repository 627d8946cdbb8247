// Batch-1 CSB product (SpMV) over the panel layout, fp16 values with fp32 accumulation.
//
// The work of the paper's CSB-Engine (Section 4.3.1: read the kept inputs through ColIdx,
// multiply by the kernel matrix, accumulate into the outputs through RowIdx, sum along the
// block-row) is arranged so that the irregular parts happen once per CTA and the inner loop is
// a plain stream:
//
//   * a CTA owns a contiguous range of output rows and with it one panel: of every block with
//     kept rows in the range, those rows.  Every output is written by exactly one CTA, so
//     nothing is joined across CTAs and there are no atomics on y;
//   * one bulk copy brings in the panel's bookkeeping, one brings in x, and the kept inputs of
//     all of the panel's blocks are gathered once into shared memory;
//   * the panel's values flow through one shared-memory ring in fixed-size stages.  Whoever
//     finishes the last item of a stage refills its slot, so there is no producer thread and
//     nobody waits for a slower neighbour;
//   * a warp takes one bundle at a time: one item (up to 32 kept rows of a block) on all its
//     lanes, or two items of at most 16 rows / four of at most 8 rows side by side on lane
//     groups of 16 / 8, so that the fixed work per item is shared.  A lane owns one kept row
//     and reads 16 bytes = 8 kept columns per step; lanes left over in a group split the
//     columns 2-, 4-, ... ways and a few shuffles join them.  Products are accumulated with
//     packed fp32 multiply-adds;
//   * every warp adds into its own copy of the CTA's output rows; at the end the CTA adds the
//     copies in warp order and stores y.  The deal of items to warps is part of the plan, so
//     the result does not depend on timing.
#include <algorithm>
#include <cstdlib>

#include "csb_internal.hpp"
#include "csb_device.cuh"

namespace csb {

struct PanelArgs {
    const uint8_t* panels;
    const float* x;
    float* y;
    uint32_t* status;
    int rows, cols;
    int log2_stage, log2_slots;        // ring = 2^log2_slots stages of 2^log2_stage bytes
    int max_rows;                      // accumulators per warp
    int max_xg, max_meta;
    uint4 cta[kMaxPanelCtas];          // PanelCta per CTA
#ifdef CSB_PANEL_CLOCKS
    unsigned long long* clocks;        // instrumented build only: [CTA][8] wall-clock stamps in ns
#endif
};

#ifdef CSB_PANEL_CLOCKS
#define PANEL_STAMP(i) do { if (threadIdx.x == 0) a.clocks[(size_t)blockIdx.x * 8 + (i)] = global_ns(); } while (0)
#else
#define PANEL_STAMP(i) do { } while (0)
#endif

__host__ __device__ inline size_t panel_align(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Shared-memory carve-up, identical on host and device.
struct PanelSmem {
    size_t ring, xs, xg, zs, meta, bars, done, issued, dead, total;
    __host__ __device__ PanelSmem(int W, int log2_stage, int log2_slots, int cols, int max_xg, int max_rows, int max_meta) {
        const int slots = 1 << log2_slots;
        ring = 0;
        xs = (size_t)slots << log2_stage;
        xg = panel_align(xs + (size_t)cols * 4, 16);
        zs = panel_align(xg + (size_t)max_xg * 4, 16);
        meta = panel_align(zs + (size_t)W * max_rows * 4, 128);
        bars = panel_align(meta + (size_t)max_meta, 16);
        done = bars + (size_t)(slots + 2) * 8;
        issued = done + (size_t)slots * 4;
        dead = issued + (size_t)slots * 4;
        total = panel_align(dead + 4, 16);
    }
};

__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;"
        : "=l"(d)
        : "l"(*reinterpret_cast<unsigned long long*>(&a)), "l"(*reinterpret_cast<unsigned long long*>(&b)),
          "l"(*reinterpret_cast<unsigned long long*>(&c)));
    return *reinterpret_cast<float2*>(&d);
}
__device__ __forceinline__ float2 h2f2(uint32_t w) { return __half22float2(*reinterpret_cast<const __half2*>(&w)); }

// Blocks until the grids this one depends on (the work in front of it on the stream) have
// completed and their writes are visible; returns at once for an ordinary launch.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Wait for a phase; gives up after the wall-clock bound or as soon as another warp of the CTA
// has given up.
__device__ __forceinline__ bool panel_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* dead) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0;                     // the clock is a slow read: looked at every 256 failed polls only
    unsigned int spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 255u) == 0) {
            if (*dead) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kCopyWaitNs) return false;
        }
    }
}

// Wait until stage `st` of the value stream has landed in its ring slot.  The barrier of a slot
// is tested by phase parity, which can only tell apart two neighbouring phases: a warp that runs
// ahead and asks for the slot's next use while the copy of the current one is still in flight
// would be answered by the wrong phase.  So the warp first waits until the copy it needs has
// been issued (the slot's issue count, written by whoever refills it); from then on the barrier
// is either in that phase or just past it, and the parity test is exact.
__device__ __forceinline__ bool panel_wait_stage(uint64_t* full, volatile uint32_t* issued, uint32_t st, int log2_slots,
                                                 volatile uint32_t* dead) {
    const uint32_t slot = st & ((1u << log2_slots) - 1u), use = st >> log2_slots;
    if (use > 0u && issued[slot] <= use) {
        unsigned long long t0 = 0;
        unsigned int spins = 0;
        while (issued[slot] <= use) {
            if ((++spins & 255u) == 0) {
                if (*dead) return false;
                const unsigned long long now = global_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > kCopyWaitNs) return false;
            }
        }
    }
    return panel_wait(&full[slot], use & 1u, dead);
}

__global__ void __launch_bounds__(1024, 1) csb_panel_kernel(const __grid_constant__ PanelArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const PanelSmem L(W, a.log2_stage, a.log2_slots, a.cols, a.max_xg, a.max_rows, a.max_meta);
    const uint4 ct = a.cta[blockIdx.x];
    const uint8_t* panel = a.panels + (size_t)ct.x * 16;
    const uint32_t meta_bytes = ct.y, value_bytes = ct.z;
    const uint8_t* values = panel + meta_bytes;
    const uint32_t slots = 1u << a.log2_slots, SB = 1u << a.log2_stage;
    const uint32_t ring_mask = (SB << a.log2_slots) - 1u;
    const uint32_t n_stages = (value_bytes + SB - 1u) >> a.log2_stage;
    uint8_t* ring = smem + L.ring;
    float* xs = reinterpret_cast<float*>(smem + L.xs);
    float* xg = reinterpret_cast<float*>(smem + L.xg);
    float* zs_all = reinterpret_cast<float*>(smem + L.zs);
    const uint8_t* meta = smem + L.meta;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + L.bars);
    uint64_t* metabar = full + slots;
    uint64_t* xbar = full + slots + 1;
    uint32_t* done = reinterpret_cast<uint32_t*>(smem + L.done);
    volatile uint32_t* issued = reinterpret_cast<volatile uint32_t*>(smem + L.issued);
    volatile uint32_t* s_dead = reinterpret_cast<volatile uint32_t*>(smem + L.dead);

    const bool x_bulk = (reinterpret_cast<uintptr_t>(a.x) & 15) == 0 && (a.cols & 3) == 0;
    // Launched with programmatic stream serialization, this grid may start while the kernel in
    // front of it on the stream is still draining: whatever comes next may be scheduled as early
    // as the hardware likes, and this grid touches x and y only behind grid_dependency_wait().
    // The panels are written once at plan time, so their copies go out before that wait.
    asm volatile("griddepcontrol.launch_dependents;");
    PANEL_STAMP(0);
    // the first copies go out from separate lanes of warp 0, each with the barrier it set up itself:
    // lane s < slots takes stage s, the next two lanes take the bookkeeping and x
    if (warp == 0 && (uint32_t)lane < slots + 2u) {
        const uint32_t s = (uint32_t)lane;
        mbar_init(&full[s], 1);
        if (s < slots) { done[s] = 0u; issued[s] = 0u; }
        if (s == slots) *s_dead = 0u;
        mbar_fence_init();
        // the bookkeeping first, then x (the gather of the inputs, which everything else waits for, needs
        // both; x may still be being written by the kernel in front), then the values
        if (s == slots) {
            mbar_expect_tx(metabar, meta_bytes);
            bulk_g2s(smem + L.meta, panel, meta_bytes, metabar);
        }
        if (s == slots + 1u && x_bulk) {
            grid_dependency_wait();
            const uint32_t xb = (uint32_t)a.cols * 4u;
            mbar_expect_tx(xbar, xb);
            for (uint32_t off = 0; off < xb; off += 16384u)
                bulk_g2s(smem + L.xs + off, reinterpret_cast<const uint8_t*>(a.x) + off, min(16384u, xb - off), xbar);
        }
        __syncwarp(slots + 2u >= 32u ? 0xffffffffu : (1u << (slots + 2u)) - 1u);
        if (s < slots && s < n_stages) {
            const uint32_t bytes = min(SB, value_bytes - (s << a.log2_stage));
            issued[s] = 1u;
            mbar_expect_tx(&full[s], bytes);
            bulk_g2s(ring + ((size_t)s << a.log2_stage), values + ((size_t)s << a.log2_stage), bytes, &full[s]);
        }
    }
    for (int i = threadIdx.x; i < W * a.max_rows; i += blockDim.x) zs_all[i] = 0.f;
    if (!x_bulk) {
        grid_dependency_wait();
        for (int i = threadIdx.x; i < a.cols; i += blockDim.x) xs[i] = __ldg(a.x + i);
    }
    __syncthreads();                                       // barriers initialised, counters and sums cleared
    PANEL_STAMP(1);

    bool gave_up = !panel_wait(metabar, 0, s_dead);
    if (!gave_up && x_bulk) gave_up = !panel_wait(xbar, 0, s_dead);
    if (gave_up) *s_dead = 1u;
    gave_up = __syncthreads_or(gave_up) != 0;

    const PanelHeader* H = reinterpret_cast<const PanelHeader*>(meta);
    PANEL_STAMP(2);
    if (!gave_up) {
        // ---- gather the kept inputs of every block of the panel, once: four blocks per warp and
        // round, eight lanes per block, a lane resolves four column indices at a time (indices and
        // gathered inputs of a block are padded to four; padding indices are zero, i.e. the block's
        // first column, which exists)
        {
            const uint2* gath = reinterpret_cast<const uint2*>(meta + H->gather_off);
            const uint8_t* cidx = meta + H->cidx_off;
            const int n_gather = (int)H->n_gather;
            for (int g0 = warp * 4; g0 < n_gather; g0 += W * 4) {
                const int g = g0 + (lane >> 3);
                const uint2 gd = g < n_gather ? gath[g] : make_uint2(0u, 0u);
                const uint32_t xbase = gd.x & 0xffffu, n = gd.x >> 16, xoff = gd.y;
                for (uint32_t k = (uint32_t)(lane & 7) * 4u; k < n; k += 32u) {
                    const uint32_t c4 = *reinterpret_cast<const uint32_t*>(cidx + xoff + k);
                    float4 v;
                    v.x = xs[xbase + (c4 & 0xffu)]; v.y = xs[xbase + ((c4 >> 8) & 0xffu)];
                    v.z = xs[xbase + ((c4 >> 16) & 0xffu)]; v.w = xs[xbase + (c4 >> 24)];
                    *reinterpret_cast<float4*>(xg + xoff + k) = v;
                }
            }
        }
        __syncthreads();
        PANEL_STAMP(3);

        // ---- this warp's bundles: one item on all 32 lanes, or two / four small ones side by side
        const uint16_t* wb = reinterpret_cast<const uint16_t*>(meta + H->warp_off);
        const uint16_t* wlist = reinterpret_cast<const uint16_t*>(meta + H->list_off);
        const uint4* items = reinterpret_cast<const uint4*>(meta + H->items_off);
        const uint16_t* expect = reinterpret_cast<const uint16_t*>(meta + H->expect_off);
        const uint8_t* ridx = meta + H->ridx_off;
        const float4* xg4 = reinterpret_cast<const float4*>(xg);
        float* zs = zs_all + (size_t)warp * a.max_rows;
        const uint32_t i_end = wb[warp + 1];
        uint32_t idx = wb[warp];
        uint32_t e = idx < i_end ? wlist[idx] : 0u;
        for (; idx < i_end; ++idx) {
            const int logg = (int)(e >> 14);
            const int gl = lane & ((32 >> logg) - 1), grp = lane >> (5 - logg);
            const uint4 d = items[(e & 0x3fffu) + grp];
            if (idx + 1 < i_end) e = wlist[idx + 1];          // on its way while this bundle is worked on
            const uint32_t off = d.x << 4;
            const uint32_t xoff4 = d.y & 0xffffu, roff = d.z & 0xffffu;
            const int zoff = (int)(int16_t)(d.y >> 16);
            const int m = (int)((d.z >> 16) & 0xffu), logp = (int)(d.z >> 24), n = (int)(d.w & 0xffffu);
            const int my_row = zoff + (int)ridx[roff + (gl < m ? gl : 0)];
            const uint32_t st = off >> a.log2_stage;          // the same for every member of the bundle
            if (__any_sync(0xffffffffu, !panel_wait_stage(full, issued, st, a.log2_slots, s_dead))) { *s_dead = 1u; break; }

            const int r = gl & ((1 << logp) - 1), sub = gl >> logp, S = 32 >> (logg + logp);
            const int noct = n >> 3;
            float2 a0 = make_float2(0.f, 0.f), a1 = make_float2(0.f, 0.f);
            float2 b0 = make_float2(0.f, 0.f), b1 = make_float2(0.f, 0.f);
            {
                uint32_t q = off + ((uint32_t)(sub * m + r) << 4);
                const uint32_t qstep = (uint32_t)(S * m) << 4;
                const float4* xq = xg4 + xoff4 + 2 * sub;
                int o = sub;
                for (; o + S < noct; o += 2 * S) {          // two octets per round, loads first
                    const uint4 w = *reinterpret_cast<const uint4*>(ring + (q & ring_mask));
                    const uint4 v = *reinterpret_cast<const uint4*>(ring + ((q + qstep) & ring_mask));
                    const float4 x0 = xq[0], x1 = xq[1], x2 = xq[2 * S], x3 = xq[2 * S + 1];
                    a0 = ffma2(h2f2(w.x), make_float2(x0.x, x0.y), a0);
                    a1 = ffma2(h2f2(w.y), make_float2(x0.z, x0.w), a1);
                    b0 = ffma2(h2f2(v.x), make_float2(x2.x, x2.y), b0);
                    b1 = ffma2(h2f2(v.y), make_float2(x2.z, x2.w), b1);
                    a0 = ffma2(h2f2(w.z), make_float2(x1.x, x1.y), a0);
                    a1 = ffma2(h2f2(w.w), make_float2(x1.z, x1.w), a1);
                    b0 = ffma2(h2f2(v.z), make_float2(x3.x, x3.y), b0);
                    b1 = ffma2(h2f2(v.w), make_float2(x3.z, x3.w), b1);
                    q += 2 * qstep;
                    xq += 4 * S;
                }
                if (o < noct) {
                    const uint4 w = *reinterpret_cast<const uint4*>(ring + (q & ring_mask));
                    const float4 x0 = xq[0], x1 = xq[1];
                    a0 = ffma2(h2f2(w.x), make_float2(x0.x, x0.y), a0);
                    a1 = ffma2(h2f2(w.y), make_float2(x0.z, x0.w), a1);
                    a0 = ffma2(h2f2(w.z), make_float2(x1.x, x1.y), a0);
                    a1 = ffma2(h2f2(w.w), make_float2(x1.z, x1.w), a1);
                }
            }
            float acc = 0.f;
            if ((n & 7) && gl < m) {
                // the last n % 8 columns: [row][4], [row][2], [row][1] behind the octets
                uint32_t tb = off + ((uint32_t)(noct * m) << 4);
                const float* xt = xg + 4 * xoff4 + 8 * noct;
                if (n & 4) {
                    const uint2 w = *reinterpret_cast<const uint2*>(ring + ((tb + 8u * gl) & ring_mask));
                    const float4 x0 = *reinterpret_cast<const float4*>(xt);
                    b0 = ffma2(h2f2(w.x), make_float2(x0.x, x0.y), b0);
                    b1 = ffma2(h2f2(w.y), make_float2(x0.z, x0.w), b1);
                    tb += 8u * m; xt += 4;
                }
                if (n & 2) {
                    const uint32_t w = *reinterpret_cast<const uint32_t*>(ring + ((tb + 4u * gl) & ring_mask));
                    const float2 x0 = *reinterpret_cast<const float2*>(xt);
                    a0 = ffma2(h2f2(w), x0, a0);
                    tb += 4u * m; xt += 2;
                }
                if (n & 1) {
                    const __half w = *reinterpret_cast<const __half*>(ring + ((tb + 2u * gl) & ring_mask));
                    acc = __half2float(w) * xt[0];
                }
            }
            acc += ((a0.x + a1.x) + (b0.x + b1.x)) + ((a0.y + a1.y) + (b0.y + b1.y));
            // join the lanes that split the columns of a row (fixed tree inside the lane group)
            if (logg == 0) {
                for (int o = 16; o >= (1 << logp); o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                if (lane < m) zs[my_row] += acc;
            } else {
                const int pmin = (int)__reduce_min_sync(0xffffffffu, 1u << logp);
                for (int o = 16 >> logg; o >= pmin; o >>= 1) {
                    const float t = __shfl_xor_sync(0xffffffffu, acc, o);
                    if (o >= (1 << logp)) acc += t;
                }
                // members of a bundle may add into the same output: one lane group at a time
                for (int g = 0; g < (1 << logg); ++g) {
                    if (grp == g && gl < m) zs[my_row] += acc;
                    __syncwarp();
                }
            }
            __syncwarp();
            // ---- the bundle is done with its stage; the last one out refills the slot
            if (lane == 0) {
                __threadfence_block();
                const uint32_t slot = st & (slots - 1u);
                if (atomicAdd(&done[slot], 1u) + 1u == (uint32_t)expect[st]) {
                    *reinterpret_cast<volatile uint32_t*>(&done[slot]) = 0u;
                    const uint32_t nx = st + slots;
                    if (nx < n_stages) {
                        __threadfence_block();
                        fence_proxy_async_all();
                        const uint32_t bytes = min(SB, value_bytes - (nx << a.log2_stage));
                        issued[slot] = issued[slot] + 1u;
                        mbar_expect_tx(&full[slot], bytes);
                        bulk_g2s(ring + ((size_t)slot << a.log2_stage), values + ((size_t)nx << a.log2_stage), bytes, &full[slot]);
                    }
                }
            }
        }
    }
#ifdef CSB_PANEL_CLOCKS
    if (lane == 0 && warp == 0) a.clocks[(size_t)blockIdx.x * 8 + 6] = global_ns();   // warp 0 out of its items
#endif
    __syncthreads();
    PANEL_STAMP(4);
    if (*s_dead) {
        // report, give the copies still in flight a bounded chance to land, and leave
        if (threadIdx.x == 0) {
            *(volatile uint32_t*)a.status = (uint32_t)kDevCopyTimeout;
            mbar_wait_bounded(metabar, 0);
            if (x_bulk) mbar_wait_bounded(xbar, 0);
            for (uint32_t s = 0; s < slots; ++s)
                if (issued[s]) mbar_wait_bounded(&full[s], (issued[s] - 1u) & 1u);
        }
        return;
    }

    // ---- add the warps' copies in warp order and store the CTA's rows
    const int n_rows = (int)H->n_rows, row0 = (int)H->row0;
    for (int t = threadIdx.x; t < n_rows; t += blockDim.x) {
        float v = 0.f;
        for (int w = 0; w < W; ++w) v += zs_all[(size_t)w * a.max_rows + t];
        a.y[row0 + t] = v;
    }
    PANEL_STAMP(5);
    PANEL_STAMP(7);
}

#define CSB_CUDA(call)                                                                     \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            set_error("%s failed: %s", #call, cudaGetErrorString(e_));                     \
            return e_ == cudaErrorMemoryAllocation ? CSB_ERR_ALLOC : CSB_ERR_CUDA;         \
        }                                                                                  \
    } while (0)

static int env_int(const char* name, int dflt) {
    const char* v = getenv(name);
    return v && *v ? atoi(v) : dflt;
}
static int log2_floor(int v) { int l = 0; while ((2 << l) <= v) ++l; return l; }

int plan_panels(csb_matrix* A) {
    if (A->val_dtype != CSB_F16 || env_int("CSB_NO_PANEL", 0)) return CSB_OK;
    const int warps = std::min(32, std::max(1, env_int("CSB_PANEL_WARPS", 32)));
    int stage = env_int("CSB_PANEL_STAGE", 16384);
    stage = 1 << std::min(15, std::max(13, log2_floor(stage)));
    const int ctas = std::min<int>(kMaxPanelCtas, A->opts.ctas > 0 ? A->opts.ctas : A->sm_count);
    PanelHostPlan H;
    const int hrc = plan_panels_host(A, ctas, warps, stage, 16384, 8192 / warps, &H);
    if (hrc == 1) return CSB_OK;
    if (hrc != CSB_OK) return hrc;
    PanelPlan* P = new PanelPlan();
    P->ctas = (int)H.cta.size(); P->warps = warps; P->stage_bytes = stage;
    P->max_xg = (int)H.max_xg; P->max_meta = (int)H.max_meta; P->max_rows = (int)std::max<size_t>(H.max_rows, 1);
    const int want_ring = std::min(17, std::max(log2_floor(stage) + 1, env_int("CSB_PANEL_RING_LOG2", 17)));
    P->log2_ring = 0;
    for (int lr = want_ring; lr > log2_floor(stage); --lr) {
        const PanelSmem L(warps, log2_floor(stage), lr - log2_floor(stage), (int)A->cols, P->max_xg, P->max_rows, P->max_meta);
        if (L.total <= A->smem_optin) { P->log2_ring = lr; P->smem_bytes = L.total; break; }
    }
    if (!P->log2_ring) { delete P; return CSB_OK; }        // does not fit: the other path serves this matrix
    int prev = 0;
    CSB_CUDA(cudaGetDevice(&prev));
    CSB_CUDA(cudaSetDevice(A->device));
    A->panel = P;                                          // from here on csb_free releases what was allocated
    P->cta = H.cta;
    P->stream_bytes = (int64_t)H.bytes.size();
    P->balance = H.balance; P->warp_balance = H.warp_balance;
    CSB_CUDA(cudaMalloc((void**)&P->d_panels, std::max<size_t>(H.bytes.size(), 16)));
    CSB_CUDA(cudaMemcpy(P->d_panels, H.bytes.data(), H.bytes.size(), cudaMemcpyHostToDevice));
    CSB_CUDA(cudaFuncSetAttribute(csb_panel_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)A->smem_optin));
    CSB_CUDA(cudaDeviceSynchronize());
    CSB_CUDA(cudaSetDevice(prev));
    P->built = true;
    return CSB_OK;
}

void free_panels(csb_matrix* A) {
    PanelPlan* P = A->panel;
    if (!P) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(A->device);
    cudaFree(P->d_panels);
    cudaSetDevice(prev);
    delete P;
    A->panel = nullptr;
}

#ifdef CSB_PANEL_CLOCKS
static unsigned long long* g_panel_clocks = nullptr;
extern "C" int csb_debug_panel_clocks(unsigned long long* host_out, int ctas) {
    return (int)cudaMemcpy(host_out, g_panel_clocks, (size_t)ctas * 8 * 8, cudaMemcpyDeviceToHost);
}
#endif

int launch_panels(const csb_matrix* A, const float* x, float* y, void* stream) {
    const PanelPlan& P = *A->panel;
    const ProductPlan& Q = A->product;
    if (Q.h_status && *Q.h_status != 0) { set_error("an earlier product on this handle gave up waiting on the device (code %u)", *Q.h_status); return CSB_ERR_TIMEOUT; }
    int prev = 0;
    CSB_CUDA(cudaGetDevice(&prev));
    if (prev != A->device) CSB_CUDA(cudaSetDevice(A->device));
    PanelArgs a{};
    a.panels = P.d_panels; a.x = x; a.y = y; a.status = Q.d_status;
    a.rows = (int)A->rows; a.cols = (int)A->cols;
    a.log2_stage = log2_floor(P.stage_bytes); a.log2_slots = P.log2_ring - a.log2_stage;
    a.max_rows = P.max_rows; a.max_xg = P.max_xg; a.max_meta = P.max_meta;
    for (int c = 0; c < P.ctas; ++c) a.cta[c] = make_uint4(P.cta[c].off16, P.cta[c].meta_bytes, P.cta[c].value_bytes, P.cta[c].n_rows);
#ifdef CSB_PANEL_CLOCKS
    static unsigned long long* d_clocks = nullptr;
    if (!d_clocks) cudaMalloc((void**)&d_clocks, (size_t)kMaxPanelCtas * 8 * 8);
    a.clocks = d_clocks;
    g_panel_clocks = d_clocks;
#endif
    // Programmatic stream serialization lets this grid's start-up (barriers, first copies of the
    // panels) overlap the end of the kernel in front of it; the kernel orders itself behind that
    // kernel before it touches x or y.  CSB_PANEL_PDL=0 asks for an ordinary launch.
    const int use_pdl = env_int("CSB_PANEL_PDL", 1);      // read at every launch, so a caller can compare both kinds
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)P.ctas); cfg.blockDim = dim3((unsigned)P.warps * 32u);
    cfg.dynamicSmemBytes = P.smem_bytes; cfg.stream = (cudaStream_t)stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = use_pdl ? 1u : 0u;
    cudaError_t e = cudaLaunchKernelEx(&cfg, csb_panel_kernel, a);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (prev != A->device) cudaSetDevice(prev);
    if (e != cudaSuccess) { set_error("panel kernel launch failed: %s", cudaGetErrorString(e)); return CSB_ERR_CUDA; }
    return CSB_OK;
}

}  // namespace csb
