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
// Wait for a phase with a wall-clock bound; false = gave up.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > kCopyWaitNs) return false;
    }
}
// One bulk asynchronous copy global -> shared; completion is counted in bytes on `bar`.
// Both addresses and the size are multiples of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

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
// column; the kernel matrix is stored column-major in words, RL words per column.  The group is
// cut into S = GW / RL sub-groups; sub-group kg takes columns kg, kg + S, ...; lane rl of a
// sub-group owns word rl of each column, i.e. the same output rows for the whole item.  The
// A = S * RL active lanes read words s*A .. s*A + A-1 in step s: consecutive, conflict-free.
//
// Per item: gather the kept inputs through the column indices (gather(col, flags, bt) returns
// input `col` of batch column bt) into xg, multiply, fold the sub-groups, and add into
// zs[(zbase + row_idx) * BT + bt] of this group's private accumulators.
//   xg_w: per warp, G * kMaxNk * BT floats;  zs_w: per warp, G * zs_stride floats.
template <typename T, int BT, int GW, typename Gather>
__device__ __forceinline__ void walk_chunk(const uint8_t* chunk, const uint4& ch, int lane, float* __restrict__ xg_w,
                                           float* __restrict__ zs_w, int zs_stride, Gather gather) {
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
    float* xg = xg_w + g * (kMaxNk * BT);
    float* zs = zs_w + g * zs_stride;
    while (__any_sync(0xffffffffu, p < end)) {
        int nk = 0, mr = 0, RL = 1, S = 1;
        uint32_t xbase = 0, zbase = 0, magic = 1024, flags = 0;
        if (p < end) {
            const uint4 h = *reinterpret_cast<const uint4*>(p);
            nk = (int)(h.x & 0xffu); mr = (int)((h.x >> 8) & 0xffu); RL = (int)((h.x >> 16) & 0xffu); S = (int)(h.x >> 24);
            xbase = h.y; zbase = h.z; magic = h.w & 0xffffu; flags = h.w >> 16;
        }
        const uint8_t* cidx = p + 16;
        const uint8_t* ridx = cidx + nk;
        const int idx_bytes = (nk + mr + 3) & ~3;
        const uint32_t* vals = reinterpret_cast<const uint32_t*>(p + 16 + idx_bytes);
        const int nwords = nk * RL;
        if (p < end) p += (16 + idx_bytes + nwords * 4 + 15) & ~15;

        for (int k = gl; k < nk; k += GW) {
            const uint32_t col = xbase + cidx[k];
#pragma unroll
            for (int bt = 0; bt < BT; ++bt) xg[k * BT + bt] = gather(col, flags, bt);
        }
        __syncwarp();
        const int kg = (int)(((uint32_t)gl * magic) >> 10);
        const int A = S * RL;
        float acc[R][BT];
#pragma unroll
        for (int q = 0; q < R; ++q)
#pragma unroll
            for (int bt = 0; bt < BT; ++bt) acc[q][bt] = 0.f;
        if (gl < A) {
            int k = kg;
#pragma unroll 4
            for (int w = gl; w < nwords; w += A, k += S) {
                float v[R];
                WordTraits<T>::unpack(vals[w], v);
#pragma unroll
                for (int bt = 0; bt < BT; ++bt) {
                    const float xv = xg[k * BT + bt];
#pragma unroll
                    for (int q = 0; q < R; ++q) acc[q][bt] = fmaf(v[q], xv, acc[q][bt]);
                }
            }
        }
        // fold the sub-groups onto sub-group 0: a tree over kg (S need not be a power of two)
#pragma unroll
        for (int r = 0; r < Log2<GW>::v; ++r) {
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
        if (gl < RL) {
#pragma unroll
            for (int q = 0; q < R; ++q) {
                const int r = gl * R + q;
                if (r < mr) {
                    float* z = zs + ((int)zbase + (int)ridx[r]) * BT;
#pragma unroll
                    for (int bt = 0; bt < BT; ++bt) z[bt] += acc[q][bt];
                }
            }
        }
        __syncwarp();
    }
}

}  // namespace csb
