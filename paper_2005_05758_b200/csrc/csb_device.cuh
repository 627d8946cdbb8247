// Device-side building blocks shared by the product kernel and the recurrent
// time-loop kernel: bulk-copy / mbarrier wrappers and the per-item arithmetic.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace csb {

enum : uint32_t { kDevOk = 0, kDevCopyTimeout = 1, kDevBarrierTimeout = 2 };
constexpr unsigned long long kCopyWaitNs = 1000ull * 1000ull * 1000ull;   // give up on a bulk copy after 1 s

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// The same test, but a thread that finds the phase unfinished may be parked by the hardware for up
// to `ns` nanoseconds (it wakes when the phase completes): waiting warps then leave the issue slots
// to the warps that still have work.
__device__ __forceinline__ bool mbar_try_wait_parked(uint64_t* bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
// Wait for a phase with a wall-clock bound; false = gave up.  The clock (a slow read) is looked at
// only every 256 failed polls, so a wait that ends within microseconds never touches it.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0 = 0;
    unsigned int spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 255u) == 0) {
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kCopyWaitNs) return false;
        }
    }
}
// One bulk asynchronous copy global -> shared; completion is counted in bytes on `bar`.
// Both addresses and the size are multiples of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Orders this thread's earlier generic-proxy view of memory before the asynchronous (bulk copy)
// accesses it issues next.
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Programmatic dependent launch.  A kernel launched with programmatic stream serialization may be
// scheduled while the kernel in front of it on the stream is still draining; pdl_wait() blocks until
// that kernel has completed and its writes are visible (at once for an ordinary launch), and
// pdl_launch_dependents() tells the hardware that whatever comes next may be scheduled.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename T> struct WordTraits;
template <> struct WordTraits<__half> {
    static constexpr int kRows = 2;
    __device__ static __forceinline__ void unpack(uint32_t w, float (&v)[2]) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
        v[0] = f.x; v[1] = f.y;
    }
};
template <> struct WordTraits<float> {
    static constexpr int kRows = 1;
    __device__ static __forceinline__ void unpack(uint32_t w, float (&v)[1]) { v[0] = __uint_as_float(w); }
};

// Per-group buffers are spaced so that the lane groups of a warp, which run in lock-step and
// tend to touch the same index at the same time, fall into different shared-memory banks.
__host__ __device__ constexpr int group_pad(int gw) { return gw == 32 ? 0 : gw; }
__host__ __device__ constexpr int xg_stride(int gw, int bt) { return kMaxNk * bt + group_pad(gw); }


template <int N> struct Log2;
template <> struct Log2<8> { static constexpr int v = 3; };
template <> struct Log2<16> { static constexpr int v = 4; };
template <> struct Log2<32> { static constexpr int v = 5; };

// Size in bytes of a chunk, from its header (sum of the sub-stream sizes plus the header).
__device__ __forceinline__ uint32_t chunk_bytes(const uint4& ch) {
    return 16u + 16u * ((ch.x & 0xffffu) + (ch.x >> 16) + (ch.y & 0xffffu) + (ch.y >> 16));
}

// Work through one chunk held in shared memory.  The warp is cut into G = 32 / GW lane groups;
// group g walks sub-stream g, so G items are in flight and share every instruction.
//
// Lane mapping inside a group, per item: a word is kRows consecutive kept rows of one kept
// column, RL words per column.  Columns are taken four at a time: a quad-word holds the words
// of one row pair for columns 4q .. 4q+3 (16 bytes), quad-column q has RL quad-words, and the
// nk % 4 columns left over follow as plain words, column-major.  The group is cut into
// S = GW / RL sub-groups; sub-group kg takes quad-columns kg, kg + S, ... (and tail columns
// kg, kg + S, ...); lane rl of a sub-group owns row word rl, i.e. the same output rows for the
// whole item.  The A = S * RL active lanes read quad-words s*A .. s*A + A-1 in step s:
// consecutive 16-byte pieces, conflict-free.
//
// Per item: gather the kept inputs through the column indices (gather4(xbase, c4, flags, left,
// dst) resolves four packed indices, `left` of them real, and writes dst[j * BT + bt]) into xg, multiply, fold the sub-groups, and add into
// zs[(zbase + row_idx) * BT + bt] of this group's private accumulators.
//   xg_w: per warp, G * xg_stride(GW, BT) floats;  zs_w: per warp, G * zs_stride floats.
template <typename T, int BT, int GW, typename Gather>
__device__ __forceinline__ void walk_chunk(const uint8_t* chunk, const uint4& ch, int lane, float* __restrict__ xg_w,
                                           float* __restrict__ zs_w, int zs_stride, Gather gather4) {
    constexpr int R = WordTraits<T>::kRows;
    const int g = lane / GW, gl = lane % GW;
    const uint32_t sz[4] = {ch.x & 0xffffu, ch.x >> 16, ch.y & 0xffffu, ch.y >> 16};
    uint32_t before = 0, mine = 0;
#pragma unroll
    for (int j = 0; j < 32 / GW; ++j) {
        if (j < g) before += sz[j];
        if (j == g) mine = sz[j];
    }
    const uint8_t* p = chunk + 16 + 16 * before;
    const uint8_t* end = p + 16 * mine;
    float* xg = xg_w + g * xg_stride(GW, BT);
    float* zs = zs_w + g * zs_stride;
    // The header and the column indices of an item are fetched one item ahead: both sit at fixed
    // places, so the loads go out together with the rest of the previous item's loads.  A lane
    // whose four indices lie past nk reads whatever follows (still inside the CTA's shared
    // memory) and never uses it.
    uint4 h = make_uint4(0u, 0u, 0u, 0u);
    uint32_t c4 = 0u;
    if (p < end) {
        h = *reinterpret_cast<const uint4*>(p);
        c4 = *reinterpret_cast<const uint32_t*>(p + 16 + 4 * gl);
    }
    while (__any_sync(0xffffffffu, p < end)) {
        // ---- header: a finished group holds zeros, which turns every step below into a no-op
        const int nk = (int)(h.x & 0xffu), mr = (int)((h.x >> 8) & 0xffu), RL = (int)((h.x >> 16) & 0xffu), S = (int)(h.x >> 24);
        const uint32_t xbase = h.y, zbase = h.z & 0xffffu, magic = h.z >> 16, flags = (h.w >> 16) & 0xffu;
        const uint8_t* item = p;
        p += 16u * (h.w & 0xffffu);
        const uint4* quads = reinterpret_cast<const uint4*>(item + 16u * (h.w >> 24));
        const int nq = (nk >> 2) * RL;                                    // quad-words (4 words each)
        const uint32_t* tailw = reinterpret_cast<const uint32_t*>(quads + nq);
        const uint8_t* ridx = item + 16 + ((nk + 3) & ~3);
        // everything that does not depend on other loads goes out now: the next item's header and
        // indices, this lane's row indices
        uint4 hn = make_uint4(0u, 0u, 0u, 0u);
        uint32_t c4n = 0u;
        if (p < end) {
            hn = *reinterpret_cast<const uint4*>(p);
            c4n = *reinterpret_cast<const uint32_t*>(p + 16 + 4 * gl);
        }
        uint32_t rr = 0u;                                                 // this lane's R row indices, one byte each
        if (gl < RL) rr = (R == 2) ? (uint32_t)*reinterpret_cast<const uint16_t*>(ridx + 2 * gl) : (uint32_t)ridx[gl];

        // ---- gather: each lane resolves four column indices at a time; indices past nk are
        // padding zeros, gather4 decides whether they may be dereferenced
        if (gl * 4 < nk) gather4(xbase, c4, flags, nk - gl * 4, xg + gl * 4 * BT);
        if (GW * 4 < kMaxNk)
            for (int k4 = (gl + GW) * 4; k4 < nk; k4 += 4 * GW)
                gather4(xbase, *reinterpret_cast<const uint32_t*>(item + 16 + k4), flags, nk - k4, xg + k4 * BT);
        __syncwarp();

        // ---- multiply: lane gl reads words gl, gl + A, ... and walks columns kg, kg + S, ...
        const int kg = (int)(((uint32_t)gl * magic) >> 10);
        const int A = S * RL;
        float acc[R][BT];
#pragma unroll
        for (int q = 0; q < R; ++q)
#pragma unroll
            for (int bt = 0; bt < BT; ++bt) acc[q][bt] = 0.f;
        if (gl < A) {
            // four columns at a time: lane gl reads quad-words gl, gl + A, ... (16 bytes each,
            // consecutive lanes consecutive quad-words) and the four inputs of those columns
            const uint4* qp = quads + gl;
            const uint4* qend = quads + nq;
            const float* xp = xg + 4 * kg * BT;
            const int xs = 4 * S * BT;
#pragma unroll 1
            for (; qp < qend; qp += A, xp += xs) {
                const uint4 w = *qp;
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
                float xv[4][BT];
                if (BT == 1) {
                    const float4 x4 = *reinterpret_cast<const float4*>(xp);
                    xv[0][0] = x4.x; xv[1][0] = x4.y; xv[2][0] = x4.z; xv[3][0] = x4.w;
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int bt = 0; bt < BT; ++bt) xv[j][bt] = xp[j * BT + bt];
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float v[R];
                    WordTraits<T>::unpack(ww[j], v);
#pragma unroll
                    for (int bt = 0; bt < BT; ++bt)
#pragma unroll
                        for (int q = 0; q < R; ++q) acc[q][bt] = fmaf(v[q], xv[j][bt], acc[q][bt]);
                }
            }
            // the last nk % 4 columns, one word per column and lane
            const uint32_t* vp = tailw + gl;
            const uint32_t* vend = tailw + (nk & 3) * RL;
            const float* xt = xg + ((nk & ~3) + kg) * BT;
            for (; vp < vend; vp += A, xt += S * BT) {
                float v[R];
                WordTraits<T>::unpack(*vp, v);
#pragma unroll
                for (int bt = 0; bt < BT; ++bt) {
                    const float x1 = xt[bt];
#pragma unroll
                    for (int q = 0; q < R; ++q) acc[q][bt] = fmaf(v[q], x1, acc[q][bt]);
                }
            }
        }

        // ---- fold the sub-groups onto sub-group 0: a tree over kg (S need not be a power of
        // two); the number of rounds is the same for the whole warp
        const int smax = (int)__reduce_max_sync(0xffffffffu, (unsigned)S);
        for (int r = 0; (1 << r) < smax; ++r) {
            const int off = RL << r;
            const bool take = off < A && gl + off < A;
#pragma unroll
            for (int q = 0; q < R; ++q)
#pragma unroll
                for (int bt = 0; bt < BT; ++bt) {
                    const float o = __shfl_down_sync(0xffffffffu, acc[q][bt], off < GW ? off : 0, GW);
                    if (take) acc[q][bt] += o;
                }
        }

        // ---- scatter-add through the row indices (distinct within an item: loads first, stores last)
        if (gl < RL) {
            const int r0 = gl * R;
            float* zr[R];
            float cur[R][BT];
#pragma unroll
            for (int q = 0; q < R; ++q) {
                const int ri = (r0 + q < mr) ? (int)((rr >> (8 * q)) & 0xffu) : (int)(rr & 0xffu);
                zr[q] = zs + ((int)zbase + ri) * BT;
#pragma unroll
                for (int bt = 0; bt < BT; ++bt) cur[q][bt] = zr[q][bt];
            }
#pragma unroll
            for (int q = 0; q < R; ++q)
                if (r0 + q < mr) {
#pragma unroll
                    for (int bt = 0; bt < BT; ++bt) zr[q][bt] = cur[q][bt] + acc[q][bt];
                }
        }
        h = hn;
        c4 = c4n;
        __syncwarp();
    }
}

}  // namespace csb
