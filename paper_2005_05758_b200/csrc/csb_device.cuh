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

// Lane mapping of one item.  A word is kRows consecutive kept rows of one kept column; the
// kernel matrix is stored column-major in words, RL words per column.  The warp is cut into
// S = 32 / RL lane groups; group kg takes columns kg, kg + S, ...; inside a group lane rl owns
// word rl of each column, i.e. the same output rows for the whole item.  A = S * RL lanes are
// active and in step s they read words s*A .. s*A + A-1: consecutive, conflict-free.
struct LaneMap {
    int RL, S, A, kg;
};
template <int kRows>
__device__ __forceinline__ LaneMap lane_map(int mr, int lane) {
    LaneMap m;
    m.RL = (mr + kRows - 1) / kRows;
    m.S = 32 / m.RL;
    m.A = m.S * m.RL;
    m.kg = lane / m.RL;
    return m;
}

// acc[q][bt] += sum over this lane's columns of value(row word, q) * xg[k][bt].
template <typename T, int BT>
__device__ __forceinline__ void item_mac(const uint32_t* __restrict__ vals, int nk, const LaneMap& lm, int lane,
                                         const float* __restrict__ xg, float (&acc)[WordTraits<T>::kRows][BT]) {
    constexpr int R = WordTraits<T>::kRows;
    if (lane < lm.A) {
        const int nwords = nk * lm.RL;
        int k = lm.kg;
#pragma unroll 4
        for (int w = lane; w < nwords; w += lm.A, k += lm.S) {
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
    // fold the lane groups onto group 0 (a tree over groups; S need not be a power of two)
    for (int off = lm.RL; off < lm.A; off <<= 1) {
#pragma unroll
        for (int q = 0; q < R; ++q)
#pragma unroll
            for (int bt = 0; bt < BT; ++bt) {
                const float o = __shfl_down_sync(0xffffffffu, acc[q][bt], off);
                if (lane + off < lm.A) acc[q][bt] += o;
            }
    }
}

// Walk the items stored in [p, end) (shared memory).  For each item: gather the kept inputs
// through the column indices (gather(col, tail, bt) returns input `col` of batch column bt),
// multiply by the kernel matrix, add into zs[(zbase_local + row_idx) * BT + bt], then let
// after(zbase, tail) act (flush of a finished block-row, or nothing).  zs_base(zbase) maps an
// item's zbase to the index its rows are relative to inside zs.
template <typename T, int BT, typename Gather, typename ZsBase, typename After>
__device__ __forceinline__ void walk_items(const uint8_t* p, const uint8_t* end, int lane, float* __restrict__ xg,
                                           float* __restrict__ zs, Gather gather, ZsBase zs_base, After after) {
    constexpr int R = WordTraits<T>::kRows;
    while (p < end) {
        const uint4 h = *reinterpret_cast<const uint4*>(p);
        const int nk = (int)(h.x & 0xffffu), mr = (int)(h.x >> 16);
        const uint32_t xbase = h.y, zbase = h.z, tail = h.w;
        const uint8_t* cidx = p + 16;
        const uint8_t* ridx = cidx + nk;
        const int idx_bytes = (nk + mr + 3) & ~3;
        const uint32_t* vals = reinterpret_cast<const uint32_t*>(p + 16 + idx_bytes);
        const int RLw = (mr + R - 1) / R;
        p += (16 + idx_bytes + nk * RLw * 4 + 15) & ~15;
        if (nk > 0 && mr > 0) {
            for (int k = lane; k < nk; k += 32) {
                const uint32_t col = xbase + cidx[k];
#pragma unroll
                for (int bt = 0; bt < BT; ++bt) xg[k * BT + bt] = gather(col, tail, bt);
            }
            __syncwarp();
            const LaneMap lm = lane_map<R>(mr, lane);
            float acc[R][BT];
#pragma unroll
            for (int q = 0; q < R; ++q)
#pragma unroll
                for (int bt = 0; bt < BT; ++bt) acc[q][bt] = 0.f;
            item_mac<T, BT>(vals, nk, lm, lane, xg, acc);
            if (lane < lm.RL) {
                float* zrow = zs + zs_base(zbase) * BT;
#pragma unroll
                for (int q = 0; q < R; ++q) {
                    const int r = lane * R + q;
                    if (r < mr) {
                        float* z = zrow + (int)ridx[r] * BT;
#pragma unroll
                        for (int bt = 0; bt < BT; ++bt) z[bt] += acc[q][bt];
                    }
                }
            }
            __syncwarp();
        }
        after(zbase, tail);
    }
}

}  // namespace csb
