// LSTM and GRU layers at larger batch, one timestep at a time on tensor cores.
//
// With a batch of 16 or more the per-step product of Section 2.1, W . [u_t ; h_{t-1}] for all
// batch columns at once, is a dense contraction per block (kernel matrix times gathered inputs),
// which the batched product kernel runs on tensor cores.  The persistent time-loop kernel keeps
// that product on CUDA cores, so for these batches a step is issued as separate launches instead:
// the batched product (pack + tensor-core kernel) of every layer, then one small kernel with the
// gate arithmetic, which also routes h_t to where the next products read it.  The products of a
// layer read one buffer V_l = [u_t ; h_{t-1}] of shape [B, I_l + H]; the gate kernel of layer l
// writes h_t into the right part of V_l (for step t + 1) and into the left part of V_{l+1} (the
// layer above, same step) or into y, and the gate kernel of layer 0 also moves x_{t+1} in.
//
// Up to 32 product rows (LSTM: batch <= 32, GRU: batch <= 16) the fp32 buffers V_l do not exist at all:
// the gate arithmetic writes h_t, and that of layer 0 also x_{t+1}, straight into the packed binary16
// (hi, lo) input rows that the product kernel reads, transposed through shared memory so that the
// stores of a row are contiguous; a step is then two launches per layer (product, gates).  With
// CSB_RNN_STEP_LOOP=1, and where the layers' plans allow it, the whole sequence is instead ONE
// cooperative launch of the product kernel's time loop (product pass, grid barrier, gates, grid barrier
// per layer and step: csb_spmm_mma.cu).
//
// GRU (reset gate applied after the recurrent product) needs the input part and the recurrent part
// of the candidate's pre-activation apart.  One product still does: V_l has 2B rows, row b holds
// [u_t ; 0] and row B + b holds [0 ; h_{t-1}], so row b of the product is W_x u and row B + b is W_h h.
#include <algorithm>
#include <list>
#include <memory>
#include <mutex>

#include "csb_internal.hpp"
#include "csb_device.cuh"
#include "csb_gates.cuh"

namespace csb {

#define CSB_CUDA(call)                                                                     \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            set_error("%s failed: %s", #call, cudaGetErrorString(e_));                     \
            return e_ == cudaErrorMemoryAllocation ? CSB_ERR_ALLOC : CSB_ERR_CUDA;         \
        }                                                                                  \
    } while (0)

struct StepPlan {
    std::vector<uint64_t> uids;
    int L = 0, B = 0, H = 0, gates = 0, device = -1;
    int in_size[kMaxLayers] = {};
    float* d_v[kMaxLayers] = {};       // [B, in_size[l] + H] per layer (GRU: [2B, ...], input rows then recurrent rows)
    float* d_z = nullptr;              // [B, 4H] (GRU: [2B, 3H]) pre-activations of the layer being worked on
    float* d_c = nullptr;              // [L, B, H] cell state
    float* d_stage = nullptr;          // host-I/O staging of x and y
    size_t stage_cap = 0;
    // packed path (at most 32 product rows): per layer the packed inputs of its product, one row of
    // `pitch` bytes per column of W_l, and the fp32 h of every layer
    uint8_t* d_xp[kMaxLayers] = {};
    float* d_h = nullptr;              // [L, B, H]
    unsigned int* d_gbar = nullptr;    // grid-barrier word of the one-launch time loop
    int pitch = 0, cap = 0;
    ~StepPlan() {
        for (float* p : d_v) cudaFree(p);
        for (uint8_t* p : d_xp) cudaFree(p);
        cudaFree(d_z); cudaFree(d_c); cudaFree(d_stage); cudaFree(d_h); cudaFree(d_gbar);
    }
};
static std::mutex g_step_mu;
static std::list<std::unique_ptr<StepPlan>> g_step_plans;

void drop_step_plans(const csb_matrix* A) {
    std::lock_guard<std::mutex> lk(g_step_mu);
    int prev = 0;
    cudaGetDevice(&prev);
    for (auto it = g_step_plans.begin(); it != g_step_plans.end();) {
        if (std::find((*it)->uids.begin(), (*it)->uids.end(), A->uid) != (*it)->uids.end()) {
            cudaSetDevice((*it)->device);
            it = g_step_plans.erase(it);
        } else ++it;
    }
    cudaSetDevice(prev);
}

__device__ __forceinline__ float logistic(float a) { return 1.f / (1.f + expf(-a)); }

// Gate arithmetic of one LSTM layer and step for the whole batch (Section 2.1):
//   c_t = s(z_f) c_{t-1} + s(z_i) tanh(z_g),  h_t = s(z_o) tanh(c_t),  rows of z stacked i, f, g, o.
// h_t goes to v_self[b, off_self + j] (this layer's next product), to v_next[b, j] (the layer
// above) when there is one, and to y_t[b, j] when asked.  With x_next the kernel also copies the
// next step's input rows into v0[b, 0 .. I).
__global__ void csb_lstm_gates_kernel(const float* __restrict__ Z, const float* __restrict__ bias, float* __restrict__ c,
                                      float* __restrict__ v_self, int ld_self, int off_self, float* __restrict__ v_next,
                                      int ld_next, float* __restrict__ y_t, const float* __restrict__ x_next, int I,
                                      float* __restrict__ v0, int ld0, int B, int H) {
    pdl_launch_dependents();
    pdl_wait();                                    // Z comes from the product in front
    const int n = B * H;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int b = e / H, j = e - b * H;
        const float* z = Z + (size_t)b * 4 * H;
        float zi = z[j], zf = z[H + j], zg = z[2 * H + j], zo = z[3 * H + j];
        if (bias) { zi += bias[j]; zf += bias[H + j]; zg += bias[2 * H + j]; zo += bias[3 * H + j]; }
        const float cn = logistic(zf) * c[e] + logistic(zi) * tanhf(zg);
        const float h = logistic(zo) * tanhf(cn);
        c[e] = cn;
        v_self[(size_t)b * ld_self + off_self + j] = h;
        if (v_next) v_next[(size_t)b * ld_next + j] = h;
        if (y_t) y_t[e] = h;
    }
    if (x_next) {
        const int nx = B * I;
        for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < nx; e += gridDim.x * blockDim.x) {
            const int b = e / I, i = e - b * I;
            v0[(size_t)b * ld0 + i] = x_next[e];
        }
    }
}

// Gate arithmetic of one GRU layer and step (reset after the recurrent product):
//   r = s(zx_r + zh_r + b_r),  u = s(zx_z + zh_z + b_z),  n = tanh(zx_n + b_in + r (zh_n + b_hn)),
//   h_t = (1 - u) n + u h_{t-1};  zx = row b, zh = row B + b of Z [2B, 3H]; bias = b_r, b_z, b_in, b_hn.
// h_t goes to the recurrent rows of v_self (row B + b, columns off_self ..), to the input rows of
// v_next (row b) when there is a layer above, and to y_t; x_next as for the LSTM kernel.
__global__ void csb_gru_gates_kernel(const float* __restrict__ Z, const float* __restrict__ bias, float* __restrict__ v_self,
                                     int ld_self, int off_self, float* __restrict__ v_next, int ld_next, float* __restrict__ y_t,
                                     const float* __restrict__ x_next, int I, float* __restrict__ v0, int ld0, int B, int H) {
    pdl_launch_dependents();
    pdl_wait();                                    // Z comes from the product in front
    const int n = B * H;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int b = e / H, j = e - b * H;
        const float* zx = Z + (size_t)b * 3 * H;
        const float* zh = Z + (size_t)(B + b) * 3 * H;
        float ar = zx[j] + zh[j], au = zx[H + j] + zh[H + j], nx = zx[2 * H + j], nh = zh[2 * H + j];
        if (bias) { ar += bias[j]; au += bias[H + j]; nx += bias[2 * H + j]; nh += bias[3 * H + j]; }
        const float r = logistic(ar), u = logistic(au);
        const float cand = tanhf(nx + r * nh);
        float* hp = v_self + (size_t)(B + b) * ld_self + off_self + j;
        const float h = (1.f - u) * cand + u * *hp;
        *hp = h;
        if (v_next) v_next[(size_t)b * ld_next + j] = h;
        if (y_t) y_t[e] = h;
    }
    if (x_next) {
        const int nx = B * I;
        for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < nx; e += gridDim.x * blockDim.x) {
            const int b = e / I, i = e - b * I;
            v0[(size_t)b * ld0 + i] = x_next[e];
        }
    }
}

// ---- the packed path (device functions in csb_gates.cuh) ----------------------------------------------
// src [nb, ncols] (row stride ld) -> slots slot0 .. of the packed rows 0 .. ncols - 1 of xp; 32 columns per block.
__global__ void csb_pack_rows_kernel(const float* __restrict__ src, long long ld, int nb, int ncols, uint8_t* __restrict__ xp, int pitch,
                                     int cap, int slot0) {
    __shared__ float tile[32][33];
    pack_columns(tile, src, ld, nb, ncols, (int)blockIdx.x * 32, xp, pitch, cap, slot0);
}

// Blocks 0 .. h_blocks - 1: the LSTM gates of 32 hidden units x the batch each; blocks from h_blocks on
// pack x_next [B, I] (the next step's input of layer 0) into rows of xp0.
__global__ void csb_lstm_gates_pack_kernel(const float* __restrict__ Z, const float* __restrict__ bias, float* __restrict__ c,
                                           float* __restrict__ hs, uint8_t* __restrict__ xp_self, uint8_t* __restrict__ xp_next,
                                           float* __restrict__ y_t, const float* __restrict__ x_next, int I, uint8_t* __restrict__ xp0,
                                           int pitch, int cap, int B, int H, int h_blocks) {
    pdl_launch_dependents();
    pdl_wait();                                    // Z comes from the product in front, which also still reads xp0
    __shared__ float tile[32][33];
    if ((int)blockIdx.x < h_blocks) lstm_gates_tile(tile, Z, bias, c, hs, xp_self, xp_next, y_t, pitch, cap, B, H, (int)blockIdx.x * 32);
    else pack_columns(tile, x_next, (long long)I, B, I, ((int)blockIdx.x - h_blocks) * 32, xp0, pitch, cap, 0);
}

// The same for the GRU (its product has 2B rows: the zeros of the unused slots are written once, before the first step).
__global__ void csb_gru_gates_pack_kernel(const float* __restrict__ Z, const float* __restrict__ bias, float* __restrict__ hs,
                                          uint8_t* __restrict__ xp_self, uint8_t* __restrict__ xp_next, float* __restrict__ y_t,
                                          const float* __restrict__ x_next, int I, uint8_t* __restrict__ xp0, int pitch, int cap, int B,
                                          int H, int h_blocks) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float tile[32][33];
    if ((int)blockIdx.x < h_blocks) gru_gates_tile(tile, Z, bias, hs, xp_self, xp_next, y_t, pitch, cap, B, H, (int)blockIdx.x * 32);
    else pack_columns(tile, x_next, (long long)I, B, I, ((int)blockIdx.x - h_blocks) * 32, xp0, pitch, cap, 0);
}

static int env_flag(const char* name) {
    const char* v = getenv(name);
    return v && *v ? atoi(v) : 0;
}

bool rnn_stepwise_wanted(int gates, int L, const csb_matrix* const* W, int B) {
    if (env_flag("CSB_RNN_NO_STEPWISE")) return false;
    // from batch 16 always; from batch 8 when the layers are big enough for three launches per layer
    // and step to pay (measured: 591 k weights 24 -> 17 us per step, 25 k weights 9 -> 13)
    int64_t nnz = 0;
    for (int l = 0; l < L; ++l) nnz += W[l]->nnz;
    if (!(B >= 16 || (B >= 8 && nnz >= 100000))) return false;
    for (int l = 0; l < L; ++l)
        if (!spmm_mma_applicable(W[l], gates == 3 ? 2 * B : B)) return false;
    return true;
}

// Returns CSB_OK, an error, or 1 when the tensor-core plan of a layer does not fit (nothing the
// caller can see has been written then; the caller runs the persistent kernel instead).
int rnn_forward_stepwise(int gates, int L, const csb_matrix* const* W, const float* const* bias, const float* x, int64_t T, int B, int H,
                         const int* in_size, const float* h0, const float* c0, float* y, float* hT, float* cT, unsigned flags,
                         void* stream) {
    StepPlan* P = nullptr;
    {
        std::lock_guard<std::mutex> lk(g_step_mu);
        for (auto& p : g_step_plans) {
            if (p->L != L || p->B != B || p->gates != gates) continue;
            bool same = true;
            for (int l = 0; l < L; ++l) same = same && p->uids[l] == W[l]->uid;
            if (same) { P = p.get(); break; }
        }
        if (!P) {
            std::unique_ptr<StepPlan> np(new StepPlan());
            np->L = L; np->B = B; np->H = H; np->gates = gates; np->device = W[0]->device;
            const int rows_v = (gates == 3 ? 2 : 1) * B;
            const bool packed_path = rows_v <= 32 && !env_flag("CSB_RNN_STEP_UNPACKED");
            if (packed_path) { np->pitch = spmm_pitch(spmm_nt(rows_v)); np->cap = 8 * spmm_nt(rows_v); }
            for (int l = 0; l < L; ++l) {
                np->uids.push_back(W[l]->uid);
                np->in_size[l] = in_size[l];
                if (packed_path) CSB_CUDA(cudaMalloc((void**)&np->d_xp[l], (size_t)(in_size[l] + H) * np->pitch));
                else CSB_CUDA(cudaMalloc((void**)&np->d_v[l], (size_t)rows_v * (in_size[l] + H) * 4));
            }
            if (packed_path) {
                CSB_CUDA(cudaMalloc((void**)&np->d_h, (size_t)L * B * H * 4));
                CSB_CUDA(cudaMalloc((void**)&np->d_gbar, 4));
            }
            CSB_CUDA(cudaMalloc((void**)&np->d_z, (size_t)(gates == 3 ? 2 : 1) * B * gates * H * 4));
            if (gates == 4) CSB_CUDA(cudaMalloc((void**)&np->d_c, (size_t)L * B * H * 4));
            P = np.get();
            g_step_plans.push_back(std::move(np));
        }
    }
    cudaStream_t st = (cudaStream_t)stream;
    const bool host_io = (flags & CSB_FLAG_HOST_IO) != 0;
    const int I0 = in_size[0];
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
    const size_t hrow = (size_t)H * 4;
    const bool gru = gates == 3;
    const int vrows = gru ? 2 * B : B;                  // rows of V_l and of the product
    if (P->pitch) {
        // ---- packed path: the gate kernels feed the products' packed inputs directly
        const int pitch = P->pitch, cap = P->cap;
        if (h0) CSB_CUDA(cudaMemcpyAsync(P->d_h, h0, ns * 4, in_kind, st));
        else CSB_CUDA(cudaMemsetAsync(P->d_h, 0, ns * 4, st));
        for (int l = 0; l < L; ++l) {
            CSB_CUDA(cudaMemsetAsync(P->d_xp[l], 0, (size_t)(in_size[l] + H) * pitch, st));
            if (h0)
                csb_pack_rows_kernel<<<(H + 31) / 32, 256, 0, st>>>(P->d_h + (size_t)l * B * H, (long long)H, B, H,
                                                                   P->d_xp[l] + (size_t)in_size[l] * pitch, pitch, cap, gru ? B : 0);
        }
        csb_pack_rows_kernel<<<(I0 + 31) / 32, 256, 0, st>>>(dx, (long long)I0, B, I0, P->d_xp[0], pitch, cap, 0);
        CSB_CUDA(cudaGetLastError());
        if (!gru) {
            if (c0) CSB_CUDA(cudaMemcpyAsync(P->d_c, c0, ns * 4, in_kind, st));
            else CSB_CUDA(cudaMemsetAsync(P->d_c, 0, ns * 4, st));
        }
        // On request (CSB_RNN_STEP_LOOP=1) the whole sequence in one launch of the product kernel's time loop,
        // where that serves the stack.  Not the default: measured, two grid barriers per layer and step cost
        // as much as the two launch hand-overs they replace (47.6 against 48-51 us per step on a two-layer
        // 2048-unit LSTM at batch 32, 14.0 against 11.4 on a 1024-unit GRU at batch 8).
        bool looped = false;
        if (env_flag("CSB_RNN_STEP_LOOP") && T < (1 << 24)) {
            RnnTileLoop R{};
            R.L = L; R.B = B; R.H = H; R.gates = gates; R.T = T; R.W = W; R.bias = bias; R.in_size = in_size;
            R.x = dx; R.y = dy; R.xp = P->d_xp; R.z = P->d_z; R.c = gru ? nullptr : P->d_c; R.hs = P->d_h; R.gbar = P->d_gbar;
            R.pitch = pitch; R.cap = cap;
            const int rc = launch_rnn_tile_loop(R, stream);
            if (rc == CSB_OK) looped = true;
            else if (rc != 1) return rc;
        }
        const int h_blocks = (H + 31) / 32, x_blocks = (I0 + 31) / 32;
        for (int64_t t = 0; t < T && !looped; ++t) {
            for (int l = 0; l < L; ++l) {
                const int rc = launch_spmm_mma(W[l], nullptr, 0, vrows, P->d_z, (int64_t)gates * H, stream, P->d_xp[l]);
                if (rc != CSB_OK) {
                    if (rc == 1 && t > 0) { set_error("the tensor-core plan of layer %d became unusable in mid-sequence", l); return CSB_ERR_CUDA; }
                    return rc;
                }
                const bool top = l == L - 1;
                const float* x_next = (l == 0 && t + 1 < T) ? dx + (size_t)(t + 1) * B * I0 : nullptr;
                cudaLaunchAttribute attr[1];
                attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
                attr[0].val.programmaticStreamSerializationAllowed = 1;
                cudaLaunchConfig_t cfg{};
                cfg.gridDim = dim3((unsigned)(h_blocks + (x_next ? x_blocks : 0))); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0;
                cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = 1;
                const float* bl = bias ? bias[l] : nullptr;
                float* hs = P->d_h + (size_t)l * B * H;
                uint8_t* xp_self = P->d_xp[l] + (size_t)in_size[l] * pitch;
                uint8_t* xp_next = top ? nullptr : P->d_xp[l + 1];
                float* yt = (top && dy) ? dy + (size_t)t * B * H : nullptr;
                if (gru)
                    CSB_CUDA(cudaLaunchKernelEx(&cfg, csb_gru_gates_pack_kernel, (const float*)P->d_z, bl, hs, xp_self, xp_next, yt, x_next, I0,
                                                P->d_xp[0], pitch, cap, B, H, h_blocks));
                else
                    CSB_CUDA(cudaLaunchKernelEx(&cfg, csb_lstm_gates_pack_kernel, (const float*)P->d_z, bl, P->d_c + (size_t)l * B * H, hs, xp_self,
                                                xp_next, yt, x_next, I0, P->d_xp[0], pitch, cap, B, H, h_blocks));
                CSB_CUDA(cudaGetLastError());
            }
        }
        if (hT) CSB_CUDA(cudaMemcpyAsync(hT, P->d_h, ns * 4, out_kind, st));
        if (cT && !gru) CSB_CUDA(cudaMemcpyAsync(cT, P->d_c, ns * 4, out_kind, st));
        if (host_io && y) CSB_CUDA(cudaMemcpyAsync(y, dy, ny * 4, cudaMemcpyDeviceToHost, st));
        if (host_io || !(flags & CSB_FLAG_ASYNC)) {
            CSB_CUDA(cudaStreamSynchronize(st));
            for (int l = 0; l < L; ++l)
                if (W[l]->product.h_status && *W[l]->product.h_status != 0) {
                    set_error("a product kernel of layer %d gave up a bounded wait (code %u)", l, *W[l]->product.h_status);
                    return CSB_ERR_TIMEOUT;
                }
        }
        return CSB_OK;
    }
    // V_l = [u_0 ; h_{-1}]: h0 (or zeros) on the right, x_0 on the left of layer 0.  GRU: the
    // recurrent rows (B ..) carry h and zeros on the left, the input rows zeros on the right.
    for (int l = 0; l < L; ++l) {
        const int ld = in_size[l] + H;
        float* hpart = P->d_v[l] + (gru ? (size_t)B * ld : 0) + in_size[l];
        if (gru) CSB_CUDA(cudaMemsetAsync(P->d_v[l], 0, (size_t)vrows * ld * 4, st));
        if (h0) CSB_CUDA(cudaMemcpy2DAsync(hpart, (size_t)ld * 4, h0 + (size_t)l * B * H, hrow, hrow, B, in_kind, st));
        else if (!gru) CSB_CUDA(cudaMemset2DAsync(hpart, (size_t)ld * 4, 0, hrow, B, st));
    }
    CSB_CUDA(cudaMemcpy2DAsync(P->d_v[0], (size_t)(I0 + H) * 4, dx, (size_t)I0 * 4, (size_t)I0 * 4, B, cudaMemcpyDeviceToDevice, st));
    if (!gru) {
        if (c0) CSB_CUDA(cudaMemcpyAsync(P->d_c, c0, ns * 4, in_kind, st));
        else CSB_CUDA(cudaMemsetAsync(P->d_c, 0, ns * 4, st));
    }

    const int threads = 256;
    const int blocks = std::max(1, std::min(1024, (B * std::max(H, I0) + threads - 1) / threads));
    for (int64_t t = 0; t < T; ++t) {
        for (int l = 0; l < L; ++l) {
            const int ld = in_size[l] + H;
            const int rc = launch_spmm_mma(W[l], P->d_v[l], ld, vrows, P->d_z, (int64_t)gates * H, stream);
            if (rc != CSB_OK) {
                // in step 0 only scratch has been written so far (y is written behind the top layer's product)
                if (rc == 1 && t > 0) { set_error("the tensor-core plan of layer %d became unusable in mid-sequence", l); return CSB_ERR_CUDA; }
                return rc;
            }
            const bool top = l == L - 1;
            const float* x_next = (l == 0 && t + 1 < T) ? dx + (size_t)(t + 1) * B * I0 : nullptr;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)blocks); cfg.blockDim = dim3((unsigned)threads); cfg.dynamicSmemBytes = 0;
            cfg.stream = st; cfg.attrs = attr; cfg.numAttrs = 1;
            const float* bl = bias ? bias[l] : nullptr;
            float* vn = top ? nullptr : P->d_v[l + 1];
            const int ldn = top ? 0 : in_size[l + 1] + H;
            float* yt = (top && dy) ? dy + (size_t)t * B * H : nullptr;
            if (gru)
                CSB_CUDA(cudaLaunchKernelEx(&cfg, csb_gru_gates_kernel, (const float*)P->d_z, bl, P->d_v[l], ld, in_size[l], vn, ldn, yt,
                                            x_next, I0, P->d_v[0], I0 + H, B, H));
            else
                CSB_CUDA(cudaLaunchKernelEx(&cfg, csb_lstm_gates_kernel, (const float*)P->d_z, bl, P->d_c + (size_t)l * B * H, P->d_v[l], ld,
                                            in_size[l], vn, ldn, yt, x_next, I0, P->d_v[0], I0 + H, B, H));
            CSB_CUDA(cudaGetLastError());
        }
    }
    if (hT)
        for (int l = 0; l < L; ++l)
            CSB_CUDA(cudaMemcpy2DAsync(hT + (size_t)l * B * H, hrow, P->d_v[l] + (gru ? (size_t)B * (in_size[l] + H) : 0) + in_size[l],
                                       (size_t)(in_size[l] + H) * 4, hrow, B, out_kind, st));
    if (cT && !gru) CSB_CUDA(cudaMemcpyAsync(cT, P->d_c, ns * 4, out_kind, st));
    if (host_io && y) CSB_CUDA(cudaMemcpyAsync(y, dy, ny * 4, cudaMemcpyDeviceToHost, st));
    if (host_io || !(flags & CSB_FLAG_ASYNC)) {
        CSB_CUDA(cudaStreamSynchronize(st));
        for (int l = 0; l < L; ++l)
            if (W[l]->product.h_status && *W[l]->product.h_status != 0) {
                set_error("a product kernel of layer %d gave up a bounded wait (code %u)", l, *W[l]->product.h_status);
                return CSB_ERR_TIMEOUT;
            }
    }
    return CSB_OK;
}

}  // namespace csb
