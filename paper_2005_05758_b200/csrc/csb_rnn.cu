// Persistent LSTM / GRU time-loop kernel and its launch glue.
//
// One cooperative launch runs the whole sequence (Section 2.1 of the paper: per step one
// CSB product with [u_t ; h_{t-1}] followed by the element-wise gate arithmetic, the c / h
// "context link" feeding the next step).  A CTA owns a tile of hidden units with all gate
// rows of those units; its compressed weights stay in shared memory for the whole sequence
// when they fit (otherwise they are re-streamed from L2 through the same bulk-copy ring as
// the bare product).  Only h_t crosses CTAs, through global memory.  At batch 1 every h value
// is published together with the number of its step in one 8-byte store and readers spin
// (bounded) on the step number, so CTAs and stacked layers run as a dataflow pipeline without a
// grid barrier.  At larger batches one bounded grid barrier per step orders the exchange and
// stacked layers run as a wavefront: in tick k layer l does step k - 2 l.
#include <algorithm>
#include <list>
#include <memory>
#include <mutex>

#include "csb_internal.hpp"
#include "csb_device.cuh"

namespace csb {

struct RnnArgs {
    const uint8_t* stream;
    const Chunk* chunks;
    const uint32_t* warp_chunk_begin;
    const uint32_t* warp_in_chunks;   // per warp: how many of its chunks hold input-column items (they come first)
    const RnnCtaDesc* ctas;
    const float* x;            // [T, B, I0]
    float* y;                  // [T, B, H] or null
    float* hbuf;               // [L][4][B][H]: h of step t lives in slot t & 3 (h0 in slot 3)
    float* cstate;             // [L][B][H], in: c0, out: cT
    const float* bias[kMaxLayers];
    int in_size[kMaxLayers];
    unsigned int* barrier;     // zero at launch
    uint32_t* status;
    unsigned long long barrier_ns;
    unsigned int barrier_extra;   // test hook: arrivals that never come
    int T, B, H, L, gates, stage_bytes, stages, resident, max_warp_bytes, max_U, max_C;
    int v_tile;                // batched: [u_t ; h_{t-1}] of the current batch tile is staged in shared memory, [bt][column]
    int v_bulk;                // batch 1: [u_t ; h_{t-1}] may come in by bulk copy (16-byte aligned pieces)
    // batch 1, flagged exchange of h (below): every h value travels with the number of its step
    uint2* hll;                // [L][4][H] pairs (bits of h, step + 2), zero at launch; null = grid-barrier time loop
    unsigned int* progress;    // [L] CTAs-times-steps whose input has been read, zero at launch
    int layer_ctas[kMaxLayers];
#ifdef CSB_PHASE_CLOCKS
    long long* clocks;         // [n_ctas][8] cycles summed over ticks: stage, walk, reduce, gates, barrier / wait for h, sums only, slot guard
#endif
};

#ifdef CSB_PHASE_CLOCKS
#define RNN_LAP(i) do { if (threadIdx.x == 0) { const long long n_ = clock64(); rprof[i] += n_ - rt; rt = n_; } } while (0)
#else
#define RNN_LAP(i) do { } while (0)
#endif

struct RnnSmem {
    size_t weights, bars, zs, xg, v, cs, zsum, vbar, flag, total;
    int zs_stride;
    __host__ __device__ RnnSmem(int W, int G, int stages, int stage_bytes, int resident, int max_warp_bytes, int max_U, int BT,
                                int B, int max_C, int v_tile) {
        zs_stride = 4 * max_U * BT + group_pad(32 / G);   // floats per lane group
        weights = 0;
        const size_t per_warp = resident ? (size_t)max_warp_bytes : (size_t)stages * stage_bytes;
        bars = weights + (size_t)W * per_warp;
        zs = (bars + (size_t)W * (resident ? 1 : stages) * 8 + 15) & ~(size_t)15;
        xg = (zs + (size_t)W * G * zs_stride * 4 + 15) & ~(size_t)15;
        v = (xg + (size_t)W * G * xg_stride(32 / G, BT) * 4 + 15) & ~(size_t)15;
        cs = (v + (BT == 1 ? (size_t)max_C * 4 : (v_tile ? (size_t)max_C * BT * 4 : 0)) + 15) & ~(size_t)15;
        zsum = (cs + (size_t)max_U * B * 4 + 15) & ~(size_t)15;
        vbar = (zsum + (size_t)4 * max_U * BT * 4 + 15) & ~(size_t)15;
        flag = vbar + 16;                              // two mbarriers: input half, recurrent half
        total = flag + 16;
    }
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Grid barrier in two halves, so that work that does not need the other CTAs' results can sit
// between them.  arrive: every thread's stores are ordered before one release-increment.
// wait: one thread polls until `target` arrivals are visible; the wait is bounded in wall-clock
// time, on expiry the status word is raised and every thread gets `false`.
__device__ __forceinline__ void grid_arrive(const RnnArgs& a) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(a.barrier, 1u);
    }
}
__device__ __forceinline__ bool grid_wait(const RnnArgs& a, unsigned int target, volatile int* s_flag) {
    if (threadIdx.x == 0) {
        bool ok = true;
        unsigned long long t0 = 0;
        unsigned int spins = 0;
        while (ld_acquire_u32(a.barrier) < target) {
            if ((++spins & 63u) == 0) {
                const unsigned long long now = global_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > a.barrier_ns) { ok = false; break; }
            }
        }
        if (!ok) *(volatile uint32_t*)a.status = (uint32_t)kDevBarrierTimeout;
        *s_flag = ok ? 1 : 0;
    }
    __syncthreads();
    return *s_flag != 0;
}

__device__ __forceinline__ float sigmoidf_acc(float a) { return 1.f / (1.f + expf(-a)); }

// Flagged exchange of h at batch 1.  A value and the number of the step it belongs to are written
// with ONE aligned 8-byte store and read with one 8-byte load, so a reader that sees the step
// number it is waiting for also holds the value: no fence, no counter, no second trip to memory.
__device__ __forceinline__ void st_flagged(uint2* p, float v, uint32_t tag) {
    asm volatile("st.volatile.global.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(__float_as_uint(v)), "r"(tag) : "memory");
}
__device__ __forceinline__ uint2 ld_flagged(const uint2* p) {
    uint2 v;
    asm volatile("ld.volatile.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned int ld_relaxed_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Time loop.  Tick k: layer l works on step t = k - lag*l (lag = 2 above the first layer).  Inside
// a tick a CTA
//   1. waits for the previous tick's barrier (h_{t-1} of its own layer is then visible),
//   2. stages h_{t-1}, walks the items that multiply it (the input half of the product was done
//      before the wait), adds up the accumulators, does the gate arithmetic, writes h_t,
//   3. arrives at this tick's barrier,
//   4. and, while the others arrive, stages u_{t+1} and walks the input-half items of the NEXT
//      step (batch 1 only).  With lag 2 the layer below produced u_{t+1} a full tick ago, so that
//      needs nothing from the barrier it has just arrived at.
// h of step s of a layer lives in slot s & 3 of a four-slot ring in global memory.
// Most warps a CTA of the time loop may have; the register budget of the kernel follows from it.
#ifndef CSB_RNN_MAX_WARPS
#define CSB_RNN_MAX_WARPS 16
#endif
constexpr int kRnnMaxWarps = CSB_RNN_MAX_WARPS;

template <typename T, int BT, int GW, bool RES>
__global__ void __launch_bounds__(kRnnMaxWarps * 32, 1) csb_rnn_kernel(const RnnArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    constexpr int G = 32 / GW;
    const int W = blockDim.x >> 5, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const RnnSmem S(W, G, a.stages, a.stage_bytes, RES, a.max_warp_bytes, a.max_U, BT, a.B, a.max_C, a.v_tile);
    const RnnCtaDesc me = a.ctas[blockIdx.x];
    const int layer = me.layer, U = me.U, u0 = me.u0, H = a.H, B = a.B;
    const int I = a.in_size[layer];
    const size_t per_warp = RES ? (size_t)a.max_warp_bytes : (size_t)a.stages * a.stage_bytes;
    uint8_t* wbuf = smem + S.weights + warp * per_warp;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S.bars) + warp * (RES ? 1 : a.stages);
    float* zs_all = reinterpret_cast<float*>(smem + S.zs);
    float* zs = zs_all + warp * G * S.zs_stride;
    float* xg = reinterpret_cast<float*>(smem + S.xg) + warp * G * xg_stride(GW, BT);
    float* vs = reinterpret_cast<float*>(smem + S.v);
    float* cs = reinterpret_cast<float*>(smem + S.cs);
    volatile int* s_flag = reinterpret_cast<volatile int*>(smem + S.flag);
    float* zsum = reinterpret_cast<float*>(smem + S.zsum);
    uint64_t* vbar = reinterpret_cast<uint64_t*>(smem + S.vbar);       // [0] input half, [1] recurrent half
    uint32_t v_uses[2] = {0, 0};

    const uint32_t c0 = a.warp_chunk_begin[me.warp0 + warp], c1 = a.warp_chunk_begin[me.warp0 + warp + 1];
    const uint32_t nchunks = c1 - c0;
    const uint32_t n_in = a.warp_in_chunks[me.warp0 + warp];        // chunks of the input half come first
    const uint8_t* wsrc = a.stream + (size_t)(nchunks ? a.chunks[c0].off16 : 0) * 16;
    uint32_t wbytes = 0, rec_off = 0;
    bool alive = true;

    // ---- weights: load once (resident) or prime the ring (streaming) ----
    // streaming: every step walks the ring once per batch tile; chunk sequence numbers keep counting
    unsigned long long n_done = 0;
    const unsigned long long n_total = (unsigned long long)a.T * ((B + BT - 1) / BT) * nchunks;
    if (RES) {
        for (uint32_t c = c0; c < c1; ++c) {                               // chunks of a warp are contiguous
            if (c - c0 == n_in) rec_off = wbytes;
            wbytes += a.chunks[c].bytes;
        }
        if (n_in == nchunks) rec_off = wbytes;
        if (lane == 0) {
            mbar_init(&bars[0], 1);
            mbar_fence_init();
            if (wbytes) {
                mbar_expect_tx(&bars[0], wbytes);
                for (uint32_t off = 0; off < wbytes; off += 16384u)
                    bulk_g2s(wbuf + off, wsrc + off, min(16384u, wbytes - off), &bars[0]);
            }
        }
        __syncwarp();
        if (wbytes && !mbar_wait_bounded(&bars[0], 0)) alive = false;
    } else {
        if (lane == 0) {
            for (int s = 0; s < a.stages; ++s) mbar_init(&bars[s], 1);
            mbar_fence_init();
            for (unsigned long long n_issued = 0; n_issued < (unsigned long long)a.stages && n_issued < n_total; ++n_issued) {
                const Chunk ch = a.chunks[c0 + (uint32_t)(n_issued % nchunks)];
                const int s = (int)(n_issued % (unsigned)a.stages);
                mbar_expect_tx(&bars[s], ch.bytes);
                bulk_g2s(wbuf + (size_t)s * a.stage_bytes, a.stream + (size_t)ch.off16 * 16, ch.bytes, &bars[s]);
            }
        }
        __syncwarp();
    }
    // cell state of this tile
    for (int i = threadIdx.x; i < U * B; i += blockDim.x) {
        const int b = i / U, u = i % U;
        cs[b * a.max_U + u] = a.gates == 4 ? a.cstate[((size_t)layer * B + b) * H + u0 + u] : 0.f;
    }
    if (threadIdx.x == 0) {
        *s_flag = 1;
        mbar_init(&vbar[0], 1);
        mbar_init(&vbar[1], 1);
        mbar_fence_init();
    }
    __syncthreads();

    const float* bias = a.bias[layer];
    const int lag = a.L > 1 ? 2 : 1;
    const int n_ticks = a.T + lag * (a.L - 1);
    const size_t slot_sz = (size_t)B * H;
    auto h_slot = [&](int l, int step) { return a.hbuf + ((size_t)l * 4 + (step & 3)) * slot_sz; };
    auto input_of = [&](int step) -> const float* { return layer == 0 ? a.x + (size_t)step * B * I : h_slot(layer - 1, step); };
    const int in_ld = layer == 0 ? I : H;
#ifdef CSB_PHASE_CLOCKS
    long long rprof[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    long long rt = clock64();
#endif

    // One half of [u ; h] into shared memory (batch 1; half 0 = input, 1 = recurrent).  With bulk
    // copies the issue and the wait are separate, so a copy can be in flight while other work
    // runs; without them stage_wait does the loads.
    auto stage_issue = [&](int half, float* dst, const float* src, int n) {
        if (a.v_bulk && threadIdx.x == 0) {
            fence_proxy_async_all();          // src may have been written with ordinary stores by other CTAs
            mbar_expect_tx(&vbar[half], (uint32_t)n * 4u);
            bulk_g2s(dst, src, (uint32_t)n * 4u, &vbar[half]);
        }
    };
    auto stage_wait = [&](int half, float* dst, const float* src, int n) {
        if (a.v_bulk) {
            if (!mbar_wait_bounded(&vbar[half], v_uses[half] & 1u)) alive = false;
            ++v_uses[half];
        } else {
#pragma unroll 4
            for (int i = threadIdx.x; i < n; i += blockDim.x) dst[i] = __ldcg(src + i);
            __syncthreads();
        }
    };
    // walk this warp's chunks of one half (part 0: input columns, part 1: recurrent columns)
    auto walk_part = [&](int part, const float* in_src, const float* rec_src, int b0, int nb) {
        auto gather = [&](uint32_t xbase, uint32_t c4, uint32_t flags, int left, float* dst) {
            const bool rec = (flags & kItemRecurrent) != 0;
            if (BT == 1) {
                // padding indices are zero; xbase (+ I for the recurrent part) is the block's first
                // column, which exists, so they may be read.  (32-bit sum: for a block that
                // straddles the x | h boundary xbase is "negative".)
                const uint32_t base = xbase + (rec ? (uint32_t)I : 0u);
                float4 v;
                v.x = vs[base + (c4 & 0xffu)]; v.y = vs[base + ((c4 >> 8) & 0xffu)];
                v.z = vs[base + ((c4 >> 16) & 0xffu)]; v.w = vs[base + (c4 >> 24)];
                *reinterpret_cast<float4*>(dst) = v;
            } else {
                if (a.v_tile) {
                    // staged tile: row bt holds [u ; h] of batch column b0 + bt (zeros past nb); padding
                    // indices are zero and land on the block's first column, which exists
                    const uint32_t base = xbase + (rec ? (uint32_t)I : 0u);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t c = base + ((c4 >> (8 * j)) & 0xffu);
#pragma unroll
                        for (int bt = 0; bt < BT; ++bt) dst[j * BT + bt] = vs[(uint32_t)bt * (uint32_t)a.max_C + c];
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t col = xbase + ((c4 >> (8 * j)) & 0xffu);
#pragma unroll
                        for (int bt = 0; bt < BT; ++bt)
                            dst[j * BT + bt] = (j < left && bt < nb)
                                ? (rec ? __ldcg(rec_src + (size_t)(b0 + bt) * H + col) : __ldcg(in_src + (size_t)(b0 + bt) * in_ld + col))
                                : 0.f;
                    }
                }
            }
        };
        if (!alive) return;
        if (RES) {
            const uint8_t* p = wbuf + (part ? rec_off : 0u);
            const uint8_t* end = wbuf + (part ? wbytes : rec_off);
            while (p < end) {
                const uint4 ch = *reinterpret_cast<const uint4*>(p);
                walk_chunk<T, BT, GW>(p, ch, lane, xg, zs, S.zs_stride, gather);
                p += chunk_bytes(ch);
            }
        } else {
            const uint32_t cnt = part ? nchunks - n_in : n_in;
            for (uint32_t c = 0; c < cnt; ++c) {
                const int s = (int)(n_done % (unsigned)a.stages);
                const uint32_t parity = (uint32_t)((n_done / (unsigned)a.stages) & 1u);
                if (!mbar_wait_bounded(&bars[s], parity)) alive = false;
                alive = !__any_sync(0xffffffffu, !alive);
                if (!alive) {
                    if (lane == 0)        // bounded drain of the copies still in flight
                        for (unsigned long long n = n_done + 1; n < n_done + a.stages && n < n_total; ++n)
                            mbar_wait_bounded(&bars[n % (unsigned)a.stages], (uint32_t)((n / (unsigned)a.stages) & 1u));
                    return;
                }
                const uint8_t* p = wbuf + (size_t)s * a.stage_bytes;
                const uint4 ch = *reinterpret_cast<const uint4*>(p);
                walk_chunk<T, BT, GW>(p, ch, lane, xg, zs, S.zs_stride, gather);
                __syncwarp();
                ++n_done;
                if (lane == 0 && n_done + a.stages - 1 < n_total) {
                    const unsigned long long n = n_done + a.stages - 1;
                    const Chunk nx = a.chunks[c0 + (uint32_t)(n % nchunks)];
                    mbar_expect_tx(&bars[s], nx.bytes);
                    bulk_g2s(wbuf + (size_t)s * a.stage_bytes, a.stream + (size_t)nx.off16 * 16, nx.bytes, &bars[s]);
                }
            }
        }
    };
    auto zero_zs = [&]() {
        for (int i = lane; i < G * S.zs_stride; i += 32) zs[i] = 0.f;
        __syncwarp();
    };


    // ------------------------------------------------------------------------------------------
    // Batch 1 with the flagged exchange: no grid barrier.  Every CTA runs through its own steps;
    // what it needs from others (h_{t-1} of its layer, h_t of the layer below) it reads as
    // (value, step) pairs and spins on the step number, what it produces it publishes the same
    // way.  h of step s sits in slot s & 3; before a CTA overwrites a slot it makes sure the layer
    // above has read the step that is four back (a per-layer count of "CTA has read its input of
    // step s", looked at one tick late, so it is off the critical path).  Every spin is bounded.
    if (BT == 1 && a.hll != nullptr) {
        uint2* ll_self = a.hll + (size_t)layer * 4 * H;
        const uint2* ll_below = layer > 0 ? a.hll + (size_t)(layer - 1) * 4 * H : nullptr;
        const uint32_t never = a.barrier_extra ? 0x40000000u : 0u;     // test hook: wait for a step that never comes
        // read n flagged values of step `step` into shared memory; false = gave up (CTA-uniform after the barrier)
        auto stage_flagged = [&](float* dst, const uint2* src, int n, int step) {
            const uint32_t want = (uint32_t)(step + 2) + never;
            for (int i0 = threadIdx.x; i0 < n; i0 += 4 * blockDim.x) {
                uint2 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) { const int i = i0 + j * blockDim.x; v[j] = i < n ? ld_flagged(src + i) : make_uint2(0u, want); }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int i = i0 + j * blockDim.x;
                    if (i >= n) continue;
                    unsigned long long t0 = 0;
                    unsigned int spins = 0;
                    while (v[j].y != want) {
                        if (*s_flag == 0) break;
                        if ((++spins & 63u) == 0) {
                            const unsigned long long now = global_ns();
                            if (t0 == 0) t0 = now;
                            else if (now - t0 > a.barrier_ns) { *(volatile uint32_t*)a.status = (uint32_t)kDevBarrierTimeout; *s_flag = 0; break; }
                        }
                        v[j] = ld_flagged(src + i);
                    }
                    dst[i] = __uint_as_float(v[j].x);
                }
            }
        };
        // h0 of this tile becomes "step -1" of the exchange
        for (int u = threadIdx.x; u < U; u += blockDim.x)
            st_flagged(ll_self + (size_t)3 * H + u0 + u, __ldcg(h_slot(layer, -1) + u0 + u), 1u);
        unsigned int above_seen = 0;
        // the sums after the walk: `parts` adjacent lanes share one accumulator entry, each adds every
        // parts-th copy in order, a fixed xor-tree joins them; the lane that holds the total applies
        // bias and the gate's activation.  One entry per thread, the same in every step.
        const int NZ = 4 * U, NC = W * G;
        int lp = 0;
        while (lp < 5 && (2 << lp) * NZ <= (int)blockDim.x) ++lp;
        const int parts = 1 << lp;
        const int my_e = (int)threadIdx.x >> lp, my_pt = (int)threadIdx.x & (parts - 1);
        const bool one_entry = NZ * parts <= (int)blockDim.x;
        const bool sum_active = (int)threadIdx.x < ((NZ * parts + 31) & ~31);
        const int my_g = my_e / U, my_u = my_e % U;
        const float my_bias = (bias && my_e < NZ) ? __ldg(bias + my_g * H + u0 + my_u) : 0.f;
        for (int t = 0; t < a.T; ++t) {
            // ---- input half: x_t, or h_t of the layer below
            if (layer == 0) {
                if (t == 0) stage_issue(0, vs, a.x, I);                // later steps: issued a step ahead, below
                stage_wait(0, vs, a.x + (size_t)t * I, I);
                if (a.v_bulk) __syncthreads();
            } else { stage_flagged(vs, ll_below + (size_t)(t & 3) * H, I, t); __syncthreads(); }
            RNN_LAP(0);
            if (*s_flag == 0 || !__syncthreads_and(alive)) break;
            if (layer > 0 && threadIdx.x == 0) atomicAdd(a.progress + layer, 1u);      // this CTA has read its input of step t
            // the count of the layer above is asked for now and used at the end of the step
            unsigned int above_now = above_seen;
            const bool need_above = layer + 1 < a.L && t >= 4;
            if (need_above && threadIdx.x == 0) above_now = ld_relaxed_u32(a.progress + layer + 1);
            zero_zs();
            walk_part(0, nullptr, nullptr, 0, 1);
            // ---- recurrent half: h_{t-1} of this layer from every CTA of the layer
            RNN_LAP(1);
            stage_flagged(vs + I, ll_self + (size_t)((t - 1) & 3) * H, H, t - 1);
            __syncthreads();
            if (*s_flag == 0) break;
            RNN_LAP(4);
            // every warp is past the input half of vs: the next step's x may come in (bulk copy only;
            // without it stage_wait loads at the top of the step)
            if (layer == 0 && t + 1 < a.T) stage_issue(0, vs, a.x + (size_t)(t + 1) * I, I);
            walk_part(1, nullptr, nullptr, 0, 1);
            __syncthreads();
            RNN_LAP(1);
            // ---- add the accumulator copies, bias and activations (the thread's entry, its share of
            // the copies and its bias were worked out before the loop)
            if (!one_entry) {
                // more entries than threads (few warps, wide tile): every thread takes several
                for (int e = threadIdx.x; e < NZ; e += blockDim.x) {
                    float sum = 0.f;
                    for (int c = 0; c < NC; ++c) sum += zs_all[e + c * S.zs_stride];
                    const int g = e / U, u = e % U;
                    float z = sum + (bias ? __ldg(bias + g * H + u0 + u) : 0.f);
                    if (a.gates == 4) z = g == 2 ? tanhf(z) : sigmoidf_acc(z);
                    else if (g < 2) z = sigmoidf_acc(z);
                    zsum[e] = z;
                }
            } else if (sum_active) {
                float sum = 0.f;
                if (my_e < NZ) {
                    const float* src = zs_all + my_e;
                    for (int c = my_pt; c < NC; c += 8 * parts) {       // eight loads in flight, added in order
                        float v[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) v[j] = (c + j * parts < NC) ? src[(c + j * parts) * S.zs_stride] : 0.f;
#pragma unroll
                        for (int j = 0; j < 8; ++j) sum += v[j];
                    }
                }
                for (int off = parts >> 1; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
                RNN_LAP(7);
                if (my_e < NZ && my_pt == 0) {
                    float z = sum + my_bias;
                    if (a.gates == 4) z = my_g == 2 ? tanhf(z) : sigmoidf_acc(z);
                    else if (my_g < 2) z = sigmoidf_acc(z);
                    zsum[my_e] = z;
                }
            }
            RNN_LAP(5);
            // slot t & 3 still holds step t - 4: every CTA of the layer above must have read it, i.e.
            // each of its n CTAs must have counted at least t - 3 reads.  Only the sum of the counts is
            // kept.  CTAs of one layer are never more than two steps apart (a CTA cannot finish step
            // s + 1 before all of them have published, hence read the input of, step s), so if one CTA
            // stood at t - 4 the others would stand at t - 2 at most and the sum at n (t - 2) - 2 at
            // most: a sum of n (t - 2) - 1 rules that out.  The layer above reaches n (t - 2) without
            // anything newer than step t - 3 from this layer, so the wait ends.
            if (need_above && threadIdx.x == 0) {
                const unsigned int need = (unsigned int)(t - 2) * (unsigned int)a.layer_ctas[layer + 1] - 1u;
                unsigned long long t0 = 0;
                unsigned int spins = 0;
                while (above_now < need) {
                    if ((++spins & 63u) == 0) {
                        const unsigned long long now = global_ns();
                        if (t0 == 0) t0 = now;
                        else if (now - t0 > a.barrier_ns) { *(volatile uint32_t*)a.status = (uint32_t)kDevBarrierTimeout; *s_flag = 0; break; }
                    }
                    above_now = ld_relaxed_u32(a.progress + layer + 1);
                }
                above_seen = above_now;
            }
            RNN_LAP(6);
            __syncthreads();
            if (*s_flag == 0) break;
            RNN_LAP(2);
            // ---- gates, state, publish
            float* h_dst = h_slot(layer, t);
            for (int u = threadIdx.x; u < U; u += blockDim.x) {
                float z[4];
#pragma unroll
                for (int g = 0; g < 4; ++g) z[g] = zsum[g * U + u];
                float h;
                if (a.gates == 4) {
                    const float c = z[1] * cs[u] + z[0] * z[2];
                    cs[u] = c;
                    h = z[3] * tanhf(c);
                    if (t == a.T - 1) a.cstate[(size_t)layer * H + u0 + u] = c;
                } else {
                    const float n = tanhf(z[2] + z[0] * z[3]);
                    const float hp = vs[I + u0 + u];                   // h_{t-1}, staged above
                    h = (1.f - z[1]) * n + z[1] * hp;
                }
                st_flagged(ll_self + (size_t)(t & 3) * H + u0 + u, h, (uint32_t)(t + 2));
                h_dst[u0 + u] = h;
                if (layer == a.L - 1 && a.y) a.y[(size_t)t * H + u0 + u] = h;
            }
            __syncthreads();
            RNN_LAP(3);
        }
#ifdef CSB_PHASE_CLOCKS
        if (threadIdx.x == 0) for (int i = 0; i < 8; ++i) a.clocks[(size_t)blockIdx.x * 8 + i] = rprof[i];
#endif
        if (!alive && lane == 0) *(volatile uint32_t*)a.status = (uint32_t)kDevCopyTimeout;
        return;
    }

    bool pre_done = false;        // the input half of the coming step is already in the accumulators
    bool in_flight = false;       // the copy of the coming step's input half has been issued
    for (int tick = 0; tick < n_ticks; ++tick) {
        const int t = tick - lag * layer;
        const bool active = t >= 0 && t < a.T;
        const bool pre_next = BT == 1 && t + 1 >= 0 && t + 1 < a.T && tick + 1 < n_ticks;
        if (tick > 0 && !grid_wait(a, (unsigned)tick * (gridDim.x + a.barrier_extra), s_flag)) break;
        RNN_LAP(4);
        if (active) {
            const float* in_src = input_of(t);
            const float* rec_src = h_slot(layer, t - 1);
            float* h_dst = h_slot(layer, t);
            for (int b0 = 0; b0 < B; b0 += BT) {
                const int nb = min(BT, B - b0);
                if (BT == 1) stage_issue(1, vs + I, rec_src, H);
                if (BT > 1 && a.v_tile) {
                    // this batch tile's [u ; h], one row per batch column (the previous tile's readers
                    // left at the barrier that ends the gate arithmetic)
                    const int C = I + H;
                    for (int bt = 0; bt < BT; ++bt) {
                        const float* ui = in_src + (size_t)(b0 + bt) * in_ld;
                        const float* hi = rec_src + (size_t)(b0 + bt) * H;
                        float* row = vs + (size_t)bt * a.max_C;
                        for (int i = threadIdx.x; i < C; i += blockDim.x)
                            row[i] = bt < nb ? __ldcg(i < I ? ui + i : hi + (i - I)) : 0.f;
                    }
                    __syncthreads();
                }
                if (!pre_done) {
                    if (BT == 1) { stage_issue(0, vs, in_src, I); stage_wait(0, vs, in_src, I); }
                    zero_zs();
                    walk_part(0, in_src, rec_src, b0, nb);
                    if (BT == 1) __syncthreads();          // every warp is done with the input half of vs
                }
                // the next step's input half is on its way while this step's recurrent half is walked
                if (pre_next) { stage_issue(0, vs, input_of(t + 1), I); in_flight = true; }
                if (BT == 1) stage_wait(1, vs + I, rec_src, H);
                RNN_LAP(0);
                walk_part(1, in_src, rec_src, b0, nb);
                __syncthreads();
                RNN_LAP(1);
                // ---- gate arithmetic for this batch tile ----
                // add the W*G private accumulator copies: `parts` adjacent lanes share one entry,
                // each adds every parts-th copy in order, then a fixed xor-tree joins them
                {
                    const int NZ = 4 * U * BT, NC = W * G;
                    int parts = 1;
                    while (parts < 32 && parts * 2 * NZ <= (int)blockDim.x) parts *= 2;
                    const int span = (NZ * parts + 31) & ~31;
                    for (int idx = threadIdx.x; idx < span; idx += blockDim.x) {
                        const int e = idx / parts, pt = idx % parts;
                        float sum = 0.f;
                        if (e < NZ) {
                            const float* src = zs_all + e;
                            for (int c = pt; c < NC; c += 8 * parts) {       // eight loads in flight, added in order
                                float v[8];
#pragma unroll
                                for (int j = 0; j < 8; ++j) v[j] = (c + j * parts < NC) ? src[(c + j * parts) * S.zs_stride] : 0.f;
#pragma unroll
                                for (int j = 0; j < 8; ++j) sum += v[j];
                            }
                        }
                        for (int off = parts >> 1; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
                        // the lane that holds the total applies bias and the gate's own activation
                        // right away, so the activations of one unit run in parallel
                        if (e < NZ && pt == 0) {
                            const int g = e / (U * BT), u = (e / BT) % U;
                            float z = sum + (bias ? __ldg(bias + g * H + u0 + u) : 0.f);
                            if (a.gates == 4) z = g == 2 ? tanhf(z) : sigmoidf_acc(z);      // i, f, o: logistic; g: tanh
                            else if (g < 2) z = sigmoidf_acc(z);                            // r, z; the candidate's two parts stay raw
                            zsum[e] = z;
                        }
                    }
                }
                __syncthreads();
                RNN_LAP(2);
                for (int i = threadIdx.x; i < U * nb; i += blockDim.x) {
                    const int bt = i / U, u = i % U, b = b0 + bt;
                    float z[4];
#pragma unroll
                    for (int g = 0; g < 4; ++g) z[g] = zsum[(g * U + u) * BT + bt];
                    float h;
                    if (a.gates == 4) {
                        const float c = z[1] * cs[b * a.max_U + u] + z[0] * z[2];
                        cs[b * a.max_U + u] = c;
                        h = z[3] * tanhf(c);
                        if (t == a.T - 1) a.cstate[((size_t)layer * B + b) * H + u0 + u] = c;
                    } else {
                        // slots: r, z, candidate input part (+ b_in), candidate hidden part (+ b_hn)
                        const float n = tanhf(z[2] + z[0] * z[3]);
                        const float hp = __ldcg(rec_src + (size_t)b * H + u0 + u);
                        h = (1.f - z[1]) * n + z[1] * hp;
                    }
                    h_dst[(size_t)b * H + u0 + u] = h;
                    if (layer == a.L - 1 && a.y) a.y[((size_t)t * B + b) * H + u0 + u] = h;
                }
                __syncthreads();
                pre_done = false;
                RNN_LAP(3);
            }
        }
        if (tick + 1 < n_ticks) grid_arrive(a);
        // the input half of the next step, while the other CTAs arrive
        if (pre_next) {
            if (!in_flight) stage_issue(0, vs, input_of(t + 1), I);
            stage_wait(0, vs, input_of(t + 1), I);
            in_flight = false;
            zero_zs();
            walk_part(0, nullptr, nullptr, 0, 1);
            pre_done = true;
        }
        RNN_LAP(1);
    }
    if (!alive && lane == 0) *(volatile uint32_t*)a.status = (uint32_t)kDevCopyTimeout;
#ifdef CSB_PHASE_CLOCKS
    if (threadIdx.x == 0) for (int i = 0; i < 8; ++i) a.clocks[(size_t)blockIdx.x * 8 + i] = rprof[i];
#endif
}


#define CSB_CUDA(call)                                                                     \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            set_error("%s failed: %s", #call, cudaGetErrorString(e_));                     \
            return e_ == cudaErrorMemoryAllocation ? CSB_ERR_ALLOC : CSB_ERR_CUDA;         \
        }                                                                                  \
    } while (0)

// Everything one (cell, layer stack, batch) combination needs on the device; built on first
// use and kept until one of its matrices is freed.
struct RnnPlan {
    int gates = 0, L = 0, B = 0, H = 0, device = 0, val_dtype = 0;
    std::vector<uint64_t> uids;
    int in_size[kMaxLayers] = {};
    int n_ctas = 0, warps = 0, BT = 1, GW = 32, v_tile = 0, resident = 0, stages = 0, stage_bytes = 0, max_warp_bytes = 0, max_U = 0, max_C = 0;
    size_t smem = 0;
    double balance = 1.0;
    int64_t stream_bytes = 0;
    uint8_t* d_stream = nullptr; Chunk* d_chunks = nullptr; uint32_t* d_wcb = nullptr; uint32_t* d_win = nullptr; RnnCtaDesc* d_ctas = nullptr;
    float* d_hbuf = nullptr; float* d_cstate = nullptr; unsigned int* d_barrier = nullptr;
    uint2* d_hll = nullptr; unsigned int* d_progress = nullptr;      // flagged exchange of h (batch 1)
    int layer_ctas[kMaxLayers] = {};
    uint32_t* h_status = nullptr; uint32_t* d_status = nullptr;
    float* d_stage = nullptr; size_t stage_cap = 0;      // host-I/O staging: x, y, states
    ~RnnPlan() {
        cudaFree(d_stream); cudaFree(d_chunks); cudaFree(d_wcb); cudaFree(d_win); cudaFree(d_ctas); cudaFree(d_hbuf);
        cudaFree(d_cstate); cudaFree(d_barrier); cudaFree(d_stage); cudaFree(d_hll); cudaFree(d_progress);
        if (h_status) cudaFreeHost(h_status);
    }
};

static std::mutex g_rnn_mu;
static std::list<std::unique_ptr<RnnPlan>> g_rnn_plans;
static unsigned long long g_barrier_ns = 2000ull * 1000ull * 1000ull;
static unsigned int g_barrier_extra = 0;

void drop_rnn_plans(const csb_matrix* A) {
    drop_step_plans(A);
    std::lock_guard<std::mutex> lk(g_rnn_mu);
    int prev = 0;
    cudaGetDevice(&prev);
    for (auto it = g_rnn_plans.begin(); it != g_rnn_plans.end();) {
        if (std::find((*it)->uids.begin(), (*it)->uids.end(), A->uid) != (*it)->uids.end()) {
            cudaSetDevice((*it)->device);
            it = g_rnn_plans.erase(it);
        } else ++it;
    }
    cudaSetDevice(prev);
}

template <typename V>
static int upload_vec(const std::vector<V>& h, V** d) {
    const size_t bytes = std::max<size_t>(h.size(), 1) * sizeof(V);
    CSB_CUDA(cudaMalloc((void**)d, bytes));
    if (!h.empty()) CSB_CUDA(cudaMemcpy(*d, h.data(), h.size() * sizeof(V), cudaMemcpyHostToDevice));
    return CSB_OK;
}

static int env_int(const char* name, int dflt) {
    const char* v = getenv(name);
    return v && *v ? atoi(v) : dflt;
}

static int build_rnn_plan(int gates, int L, const csb_matrix* const* W, int B, int H, const int* in_size, RnnPlan* P) {
    const csb_matrix* A0 = W[0];
    P->gates = gates; P->L = L; P->B = B; P->H = H; P->device = A0->device; P->val_dtype = A0->val_dtype;
    for (int l = 0; l < L; ++l) { P->uids.push_back(W[l]->uid); P->in_size[l] = in_size[l]; P->max_C = std::max(P->max_C, in_size[l] + H); }
    P->BT = B == 1 ? 1 : (B <= 4 ? 4 : 8);
    P->warps = std::min(kRnnMaxWarps, std::max(1, env_int("CSB_RNN_WARPS", 16)));
    P->stage_bytes = 3072; P->stages = 3;
    int64_t approx = 0;
    for (int l = 0; l < L; ++l) approx += W[l]->nnz * val_size(W[l]->val_dtype) + 32 * W[l]->nblk;
    int want = (int)std::min<int64_t>(A0->sm_count, std::max<int64_t>(L, approx / (24 * 1024)));
    want = std::max(want, L * ((H + 47) / 48));        // tiles are cut by cost; leave room under the 64-unit limit
    if (P->BT > 1) want = A0->sm_count;               // batched: small unit tiles keep the per-group accumulators small
    // batch 1 with the flagged exchange: more CTAs cost nothing at a barrier any more, and shorter
    // item lists per warp shorten the walk (measured: cfg 3 5.8 -> 4.1 us per step on all SMs)
    if (P->BT == 1 && !env_int("CSB_RNN_NO_FLAGGED", 0)) want = A0->sm_count;
    want = env_int("CSB_RNN_CTAS", want);
    want = std::min(std::max(want, L), A0->sm_count);
    // fewer warps per CTA shrink the per-warp accumulators and rings until the carve-up fits
    RnnHostPlan Hp;
    int rc = CSB_OK;
    const int first = P->warps;
    bool fits = false;
    // candidates, best first: with the batched input tile staged in shared memory when it fits beside
    // at least 8 warps; each with one chunk per warp (weights resident) before ring-sized chunks
    struct Cand { int warps, v_tile; };
    std::vector<Cand> cands;
    for (int vt : {1, 0})
        for (int wt : {first, 12, 8}) if (wt <= first && (vt == 0 || P->BT > 1)) cands.push_back({wt, vt});
    for (int wt : {6, 4, 2, 1}) if (wt <= first) { if (P->BT > 1) cands.push_back({wt, 1}); cands.push_back({wt, 0}); }
    for (const Cand& cd : cands) {
        const int wtry = cd.warps;
        for (int pass = 0; pass < 2 && !fits; ++pass) {
            if (pass == 0 && env_int("CSB_RNN_STREAM", 0)) continue;
            const int chunk_bytes = pass == 0 ? (256 << 10) : P->stage_bytes;
            Hp = RnnHostPlan();
            rc = plan_rnn_host(gates, L, W, in_size, H, want, wtry, chunk_bytes, &Hp);
            if (rc != CSB_OK) return rc;
            P->warps = wtry;
            P->v_tile = cd.v_tile;
            P->max_U = Hp.max_U; P->max_warp_bytes = (int)Hp.max_warp_bytes; P->GW = Hp.stream.group_width;
            const int G = 32 / P->GW;
            const RnnSmem sm(wtry, G, P->stages, P->stage_bytes, pass == 0, P->max_warp_bytes, P->max_U, P->BT, B, P->max_C, cd.v_tile);
            if (sm.total <= A0->smem_optin) { P->resident = pass == 0; P->smem = sm.total; fits = true; }
        }
        if (fits) break;
    }
    if (!fits) { set_error("time-loop kernel does not fit the %zu bytes of shared memory per CTA", A0->smem_optin); return CSB_ERR_LAUNCH; }
    P->n_ctas = (int)Hp.ctas.size();
    P->balance = Hp.balance;
    P->stream_bytes = (int64_t)Hp.stream.bytes.size();
    if ((rc = upload_vec(Hp.stream.bytes, &P->d_stream)) != CSB_OK) return rc;
    if ((rc = upload_vec(Hp.stream.chunks, &P->d_chunks)) != CSB_OK) return rc;
    if ((rc = upload_vec(Hp.stream.warp_chunk_begin, &P->d_wcb)) != CSB_OK) return rc;
    if ((rc = upload_vec(Hp.warp_in_chunks, &P->d_win)) != CSB_OK) return rc;
    if ((rc = upload_vec(Hp.ctas, &P->d_ctas)) != CSB_OK) return rc;
    CSB_CUDA(cudaMalloc((void**)&P->d_hbuf, (size_t)L * 4 * B * H * 4));
    CSB_CUDA(cudaMalloc((void**)&P->d_cstate, (size_t)L * B * H * 4));
    CSB_CUDA(cudaMalloc((void**)&P->d_barrier, 4));
    for (const RnnCtaDesc& cd : Hp.ctas) ++P->layer_ctas[cd.layer];
    if (P->BT == 1) {
        CSB_CUDA(cudaMalloc((void**)&P->d_hll, (size_t)L * 4 * H * sizeof(uint2)));
        CSB_CUDA(cudaMalloc((void**)&P->d_progress, (size_t)kMaxLayers * 4));
    }
    CSB_CUDA(cudaHostAlloc((void**)&P->h_status, 4, cudaHostAllocMapped));
    *P->h_status = 0;
    CSB_CUDA(cudaHostGetDevicePointer((void**)&P->d_status, P->h_status, 0));
    return CSB_OK;
}

template <typename T, int BT, int GW, bool RES>
static int launch_rnn(const RnnPlan* P, RnnArgs& a, cudaStream_t st) {
    CSB_CUDA(cudaFuncSetAttribute(csb_rnn_kernel<T, BT, GW, RES>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)P->smem));
    int occ = 0;
    CSB_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, csb_rnn_kernel<T, BT, GW, RES>, P->warps * 32, P->smem));
    int sms = 0;
    CSB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, P->device));
    if (occ < 1 || P->n_ctas > occ * sms) {
        set_error("grid of %d CTAs cannot be co-resident (%d per SM x %d SMs)", P->n_ctas, occ, sms);
        return CSB_ERR_LAUNCH;
    }
    void* params[] = {(void*)&a};
    const cudaError_t e = cudaLaunchCooperativeKernel((const void*)csb_rnn_kernel<T, BT, GW, RES>, dim3(P->n_ctas), dim3(P->warps * 32),
                                                      params, P->smem, st);
    if (e == cudaErrorCooperativeLaunchTooLarge) { set_error("cooperative launch too large"); return CSB_ERR_LAUNCH; }
    CSB_CUDA(e);
    return CSB_OK;
}

template <typename T, int BT>
static int dispatch_rnn_gw(const RnnPlan* P, RnnArgs& a, cudaStream_t st) {
    switch (P->GW) {
        case 8: return P->resident ? launch_rnn<T, BT, 8, true>(P, a, st) : launch_rnn<T, BT, 8, false>(P, a, st);
        case 16: return P->resident ? launch_rnn<T, BT, 16, true>(P, a, st) : launch_rnn<T, BT, 16, false>(P, a, st);
        default: return P->resident ? launch_rnn<T, BT, 32, true>(P, a, st) : launch_rnn<T, BT, 32, false>(P, a, st);
    }
}

#ifdef CSB_PHASE_CLOCKS
static long long* g_rnn_clocks = nullptr;
static int g_rnn_clock_ctas = 0;
extern "C" int csb_debug_rnn_clocks(long long* host_out, int max_ctas) {
    cudaMemcpy(host_out, g_rnn_clocks, (size_t)std::min(max_ctas, g_rnn_clock_ctas) * 8 * 8, cudaMemcpyDeviceToHost);
    return g_rnn_clock_ctas;
}
#endif

static int rnn_forward(int gates, int L, const csb_matrix_t* const* W, const float* const* bias, const float* x, int64_t T,
                       int B, const float* h0, const float* c0, float* y, float* hT, float* cT, unsigned flags, void* stream) {
    clear_error();
    if (L < 1 || L > kMaxLayers || !W) { set_error("n_layers %d (1..%d) or W is NULL", L, (int)kMaxLayers); return CSB_ERR_INVALID_ARG; }
    if (T < 0 || B < 0 || T > 0x7fffffff) { set_error("T=%lld B=%d", (long long)T, B); return CSB_ERR_INVALID_ARG; }
    for (int l = 0; l < L; ++l) if (!W[l]) { set_error("W[%d] is NULL", l); return CSB_ERR_INVALID_ARG; }
    if (W[0]->rows % gates) { set_error("W[0] has %lld rows, not a multiple of %d gates", (long long)W[0]->rows, gates); return CSB_ERR_SHAPE; }
    const int H = (int)(W[0]->rows / gates);
    int in_size[kMaxLayers];
    for (int l = 0; l < L; ++l) {
        in_size[l] = (int)(W[l]->cols - H);
        if (W[l]->rows != (int64_t)gates * H || in_size[l] <= 0 || (l > 0 && in_size[l] != H)) {
            set_error("layer %d: weight is %lld x %lld, expected %d x (%s + %d)", l, (long long)W[l]->rows, (long long)W[l]->cols,
                      gates * H, l ? "H" : "I", H);
            return CSB_ERR_SHAPE;
        }
        if (W[l]->device < 0) { set_error("layer %d was encoded host-only", l); return CSB_ERR_UNSUPPORTED; }
        if (W[l]->val_dtype == CSB_Q16) { set_error("layer %d holds fixed-point values: those serve csb_spmm_q16 only", l); return CSB_ERR_UNSUPPORTED; }
        if (W[l]->device != W[0]->device || W[l]->val_dtype != W[0]->val_dtype) {
            set_error("layers must share device and value type");
            return CSB_ERR_UNSUPPORTED;
        }
    }
    if (T == 0 || B == 0) return CSB_OK;
    if (!x) { set_error("x is NULL"); return CSB_ERR_INVALID_ARG; }
    const int I0 = in_size[0];
    int prev = 0;
    CSB_CUDA(cudaGetDevice(&prev));
    CSB_CUDA(cudaSetDevice(W[0]->device));
    struct Restore { int d; ~Restore() { cudaSetDevice(d); } } restore{prev};

    // larger batches with fp16 values: step by step, the products on tensor cores
    if (rnn_stepwise_wanted(gates, L, W, B)) {
        const int rc = rnn_forward_stepwise(gates, L, W, bias, x, T, B, H, in_size, h0, c0, y, hT, cT, flags, stream);
        if (rc != 1) return rc;
    }

    RnnPlan* P = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_rnn_mu);
        for (auto& p : g_rnn_plans) {
            if (p->gates != gates || p->L != L || p->B != B) continue;
            bool same = true;
            for (int l = 0; l < L; ++l) same = same && p->uids[l] == W[l]->uid;
            if (same) { P = p.get(); break; }
        }
        if (!P) {
            std::unique_ptr<RnnPlan> np(new RnnPlan());
            int rc = CSB_OK;
            try { rc = build_rnn_plan(gates, L, W, B, H, in_size, np.get()); }
            catch (const std::bad_alloc&) { set_error("out of host memory while planning the time loop"); rc = CSB_ERR_ALLOC; }
            if (rc != CSB_OK) return rc;
            CSB_CUDA(cudaDeviceSynchronize());
            P = np.get();
            g_rnn_plans.push_back(std::move(np));
        }
    }
    cudaStream_t st = (cudaStream_t)stream;
    const bool host_io = (flags & CSB_FLAG_HOST_IO) != 0;
    const size_t nx = (size_t)T * B * I0, ny = (size_t)T * B * H, ns = (size_t)L * B * H;
    const float* dx = x;
    float* dy = y;
    if (host_io) {
        const size_t need = nx + (y ? ny : 0);
        if (need > P->stage_cap) {
            CSB_CUDA(cudaStreamSynchronize(st));
            cudaFree(P->d_stage); P->d_stage = nullptr; P->stage_cap = 0;
            CSB_CUDA(cudaMalloc((void**)&P->d_stage, need * 4));
            P->stage_cap = need;
        }
        CSB_CUDA(cudaMemcpyAsync(P->d_stage, x, nx * 4, cudaMemcpyHostToDevice, st));
        dx = P->d_stage;
        dy = y ? P->d_stage + nx : nullptr;
    }
    const cudaMemcpyKind in_kind = host_io ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice;
    const cudaMemcpyKind out_kind = host_io ? cudaMemcpyDeviceToHost : cudaMemcpyDeviceToDevice;
    const size_t row = (size_t)B * H * 4;
    // h0 goes to slot 3 of every layer's four-slot ring (the slot of "step -1"), c0 to the cell-state buffer
    if (h0) CSB_CUDA(cudaMemcpy2DAsync(P->d_hbuf + 3 * (size_t)B * H, 4 * row, h0, row, row, L, in_kind, st));
    else CSB_CUDA(cudaMemsetAsync(P->d_hbuf, 0, 4 * row * L, st));
    if (gates == 4) {
        if (c0) CSB_CUDA(cudaMemcpyAsync(P->d_cstate, c0, ns * 4, in_kind, st));
        else CSB_CUDA(cudaMemsetAsync(P->d_cstate, 0, ns * 4, st));
    }
    CSB_CUDA(cudaMemsetAsync(P->d_barrier, 0, 4, st));
    *P->h_status = 0;

    RnnArgs a{};
    a.stream = P->d_stream; a.chunks = P->d_chunks; a.warp_chunk_begin = P->d_wcb; a.warp_in_chunks = P->d_win; a.ctas = P->d_ctas;
    a.x = dx; a.y = dy; a.hbuf = P->d_hbuf; a.cstate = P->d_cstate;
    for (int l = 0; l < L; ++l) { a.bias[l] = bias ? bias[l] : nullptr; a.in_size[l] = in_size[l]; }
    a.barrier = P->d_barrier; a.status = P->d_status; a.barrier_ns = g_barrier_ns; a.barrier_extra = g_barrier_extra;
    a.T = (int)T; a.B = B; a.H = H; a.L = L; a.gates = gates; a.stage_bytes = P->stage_bytes; a.stages = P->stages;
    a.v_tile = env_int("CSB_RNN_NO_VTILE", 0) ? 0 : P->v_tile;
    a.v_bulk = 0;
    if (P->BT == 1 && H % 4 == 0 && (reinterpret_cast<uintptr_t>(dx) & 15) == 0) {
        a.v_bulk = 1;
        for (int l = 0; l < L; ++l) if (in_size[l] % 4) a.v_bulk = 0;
    }
    if (env_int("CSB_RNN_NO_VBULK", 0)) a.v_bulk = 0;
    a.hll = nullptr; a.progress = P->d_progress;
    for (int l = 0; l < L; ++l) a.layer_ctas[l] = P->layer_ctas[l];
    if (P->BT == 1 && P->d_hll && !env_int("CSB_RNN_NO_FLAGGED", 0)) {
        // every pair starts as "no step" and the read counts at zero
        CSB_CUDA(cudaMemsetAsync(P->d_hll, 0, (size_t)L * 4 * H * sizeof(uint2), st));
        CSB_CUDA(cudaMemsetAsync(P->d_progress, 0, (size_t)kMaxLayers * 4, st));
        a.hll = P->d_hll;
    }
    a.resident = P->resident; a.max_warp_bytes = P->max_warp_bytes; a.max_U = P->max_U; a.max_C = P->max_C;
#ifdef CSB_PHASE_CLOCKS
    static long long* d_rclocks = nullptr;
    if (!d_rclocks) cudaMalloc((void**)&d_rclocks, 1 << 16);
    a.clocks = d_rclocks;
    g_rnn_clocks = d_rclocks;
    g_rnn_clock_ctas = P->n_ctas;
#endif
    int rc;
    const bool half = P->val_dtype == CSB_F16;
    if (P->BT == 1) rc = half ? dispatch_rnn_gw<__half, 1>(P, a, st) : dispatch_rnn_gw<float, 1>(P, a, st);
    else if (P->BT == 4) rc = half ? dispatch_rnn_gw<__half, 4>(P, a, st) : dispatch_rnn_gw<float, 4>(P, a, st);
    else rc = half ? dispatch_rnn_gw<__half, 8>(P, a, st) : dispatch_rnn_gw<float, 8>(P, a, st);
    if (rc != CSB_OK) return rc;
    const int last_slot = (int)((T - 1) & 3);
    if (hT) CSB_CUDA(cudaMemcpy2DAsync(hT, row, P->d_hbuf + (size_t)last_slot * B * H, 4 * row, row, L, out_kind, st));
    if (cT && gates == 4) CSB_CUDA(cudaMemcpyAsync(cT, P->d_cstate, ns * 4, out_kind, st));
    if (host_io && y) CSB_CUDA(cudaMemcpyAsync(y, dy, ny * 4, cudaMemcpyDeviceToHost, st));
    if (host_io || !(flags & CSB_FLAG_ASYNC)) {
        CSB_CUDA(cudaStreamSynchronize(st));
        if (*P->h_status != 0) {
            set_error("the time-loop kernel gave up a bounded wait (code %u: %s)", *P->h_status,
                      *P->h_status == kDevBarrierTimeout ? "grid barrier" : "bulk copy");
            return CSB_ERR_TIMEOUT;
        }
    }
    return CSB_OK;
}

void set_barrier_test_hook(unsigned int extra, unsigned long long ns) {
    g_barrier_extra = extra;
    g_barrier_ns = ns ? ns : 2000ull * 1000ull * 1000ull;
}

}  // namespace csb

extern "C" {

int csb_lstm_forward(int n_layers, const csb_matrix_t* const* W, const float* const* bias, const float* x, int64_t T, int B,
                     const float* h0, const float* c0, float* y, float* hT, float* cT, unsigned flags, void* stream) {
    return csb::rnn_forward(4, n_layers, W, bias, x, T, B, h0, c0, y, hT, cT, flags, stream);
}

int csb_gru_forward(int n_layers, const csb_matrix_t* const* W, const float* const* bias, const float* x, int64_t T, int B,
                    const float* h0, float* y, float* hT, unsigned flags, void* stream) {
    return csb::rnn_forward(3, n_layers, W, bias, x, T, B, h0, nullptr, y, hT, nullptr, flags, stream);
}

void csb_test_barrier_hook(unsigned int extra_arrivals, unsigned long long limit_ns) {
    csb::set_barrier_test_hook(extra_arrivals, limit_ns);
}

}  // extern "C"
