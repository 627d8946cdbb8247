// Gate arithmetic of one LSTM / GRU layer and step for a tile of 32 hidden units x the whole batch
// (Section 2.1), with h_t written straight into the packed binary16 (hi, lo) input rows that the
// batched product kernel reads.  Device functions shared by the per-step gate kernels and by the
// time loop that keeps the batched product and the gates in one kernel.
//
// Packed layout: one row of `pitch` bytes per matrix column; x = hi + lo, hi at halves [slot], lo at
// [cap + slot], slot = the product row (batch column; for the GRU, whose product has 2B rows,
// slots 0 .. B-1 carry the input part and B .. 2B-1 the recurrent part).
#pragma once
#include <cuda_fp16.h>

#include <cstdint>

namespace csb {

__device__ __forceinline__ float gate_logistic(float a) { return 1.f / (1.f + expf(-a)); }

// tile[b][c], 32 columns x nb batch values, into slots slot0 .. slot0 + nb - 1 of the packed rows of
// those columns (and of a second set of rows, when given).  Consecutive threads take consecutive batch
// values of a column, so that a row's stores are contiguous.  All threads of the CTA call this.
__device__ __forceinline__ void pack_tile(const float (*tile)[33], int ncols, int nb, uint8_t* rows, int pitch, int cap, int slot0,
                                          uint8_t* rows2, int slot2) {
    for (int idx = threadIdx.x; idx < 32 * nb; idx += blockDim.x) {
        const int c = idx / nb, b = idx - c * nb;
        if (c >= ncols) break;
        const float x = tile[b][c];
        const __half hi = __float2half_rn(x);
        const __half lo = __float2half_rn(x - __half2float(hi));
        __half* r = reinterpret_cast<__half*>(rows + (size_t)c * pitch);
        r[slot0 + b] = hi;
        r[cap + slot0 + b] = lo;
        if (rows2) {
            __half* r2 = reinterpret_cast<__half*>(rows2 + (size_t)c * pitch);
            r2[slot2 + b] = hi;
            r2[cap + slot2 + b] = lo;
        }
    }
}

// Columns c0 .. c0 + 31 of src [nb, ncols] (row stride ld) into slots slot0 .. of the packed rows c0 .. of xp.
__device__ __forceinline__ void pack_columns(float (*tile)[33], const float* __restrict__ src, long long ld, int nb, int ncols, int c0,
                                             uint8_t* __restrict__ xp, int pitch, int cap, int slot0) {
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5, nw = blockDim.x >> 5;
    for (int b = ty; b < nb; b += nw) tile[b][tx] = c0 + tx < ncols ? __ldcg(src + (long long)b * ld + c0 + tx) : 0.f;
    __syncthreads();
    pack_tile(tile, min(32, ncols - c0), nb, xp + (size_t)c0 * pitch, pitch, cap, slot0, nullptr, 0);
}

// LSTM, hidden units j0 .. j0 + 31:  c_t = s(z_f) c_{t-1} + s(z_i) tanh(z_g),  h_t = s(z_o) tanh(c_t);
// rows of Z [B, 4H] stacked i, f, g, o.  h_t goes, packed, to rows j of xp_self (this layer's recurrent
// columns) and of xp_next (the input columns of the layer above, or null), as fp32 to hs[b, j] and y_t[b, j].
__device__ __forceinline__ void lstm_gates_tile(float (*tile)[33], const float* __restrict__ Z, const float* __restrict__ bias,
                                                float* __restrict__ c, float* __restrict__ hs, uint8_t* __restrict__ xp_self,
                                                uint8_t* __restrict__ xp_next, float* __restrict__ y_t, int pitch, int cap, int B, int H,
                                                int j0) {
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5, nw = blockDim.x >> 5, j = j0 + tx;
    for (int b = ty; b < B; b += nw) {
        float h = 0.f;
        if (j < H) {
            const float* z = Z + (size_t)b * 4 * H;
            float zi = __ldcg(z + j), zf = __ldcg(z + H + j), zg = __ldcg(z + 2 * H + j), zo = __ldcg(z + 3 * H + j);
            if (bias) { zi += bias[j]; zf += bias[H + j]; zg += bias[2 * H + j]; zo += bias[3 * H + j]; }
            const size_t e = (size_t)b * H + j;
            const float cn = gate_logistic(zf) * __ldcg(c + e) + gate_logistic(zi) * tanhf(zg);
            h = gate_logistic(zo) * tanhf(cn);
            c[e] = cn;
            hs[e] = h;
            if (y_t) y_t[e] = h;
        }
        tile[b][tx] = h;
    }
    __syncthreads();
    pack_tile(tile, min(32, H - j0), B, xp_self + (size_t)j0 * pitch, pitch, cap, 0, xp_next ? xp_next + (size_t)j0 * pitch : nullptr, 0);
}

// GRU (reset gate applied after the recurrent product), hidden units j0 .. j0 + 31:
//   r = s(zx_r + zh_r + b_r),  u = s(zx_z + zh_z + b_z),  n = tanh(zx_n + b_in + r (zh_n + b_hn)),
//   h_t = (1 - u) n + u h_{t-1};  zx = row b, zh = row B + b of Z [2B, 3H]; bias = b_r, b_z, b_in, b_hn.
__device__ __forceinline__ void gru_gates_tile(float (*tile)[33], const float* __restrict__ Z, const float* __restrict__ bias,
                                               float* __restrict__ hs, uint8_t* __restrict__ xp_self, uint8_t* __restrict__ xp_next,
                                               float* __restrict__ y_t, int pitch, int cap, int B, int H, int j0) {
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5, nw = blockDim.x >> 5, j = j0 + tx;
    for (int b = ty; b < B; b += nw) {
        float h = 0.f;
        if (j < H) {
            const float* zx = Z + (size_t)b * 3 * H;
            const float* zh = Z + (size_t)(B + b) * 3 * H;
            float ar = __ldcg(zx + j) + __ldcg(zh + j), au = __ldcg(zx + H + j) + __ldcg(zh + H + j);
            float nx = __ldcg(zx + 2 * H + j), nh = __ldcg(zh + 2 * H + j);
            if (bias) { ar += bias[j]; au += bias[H + j]; nx += bias[2 * H + j]; nh += bias[3 * H + j]; }
            const float r = gate_logistic(ar), u = gate_logistic(au);
            const float cand = tanhf(nx + r * nh);
            const size_t e = (size_t)b * H + j;
            h = (1.f - u) * cand + u * __ldcg(hs + e);
            hs[e] = h;
            if (y_t) y_t[e] = h;
        }
        tile[b][tx] = h;
    }
    __syncthreads();
    pack_tile(tile, min(32, H - j0), B, xp_self + (size_t)j0 * pitch, pitch, cap, B, xp_next ? xp_next + (size_t)j0 * pitch : nullptr, 0);
}

}  // namespace csb
