// Cell variants of the paper's Table 1 -- LSTM with a recurrent projection (LSTMP, models SR1),
// light GRU (Li-GRU, model SR3) -- and the GRU with its reset gate in front of the recurrent product
// (the form the GRU reference of Section 2.1 gives), one timestep at a time.
//
// These cells put a second CSB product (LSTMP: the projection; reset-before GRU: the candidate's
// product with [u ; r * h]) or a different element-wise part (Li-GRU) behind the product of the
// plain cells.  A step of a layer is issued as launches on the caller's stream: the CSB products
// through the same kernels as csb_spmv / csb_spmm (whatever serves the batch size), and one small
// kernel per element-wise part, which also routes the new state to where the next products read it.
// The products of layer l read one buffer V_l = [u_t ; s_{t-1}] of shape [B, I_l + S] (s: the
// recurrent state, S its width); states are written straight into the V buffers, so nothing is
// concatenated or copied per step except the next input frame.
#include <algorithm>
#include <list>
#include <memory>
#include <mutex>

#include "csb_internal.hpp"
#include "csb_device.cuh"

namespace csb {

#define CSB_CUDA(call)                                                                     \
    do {                                                                                   \
        cudaError_t e_ = (call);                                                           \
        if (e_ != cudaSuccess) {                                                           \
            set_error("%s failed: %s", #call, cudaGetErrorString(e_));                     \
            return e_ == cudaErrorMemoryAllocation ? CSB_ERR_ALLOC : CSB_ERR_CUDA;         \
        }                                                                                  \
    } while (0)

enum CellKind { kCellLstmp = 0, kCellLigru = 1, kCellGruRb = 2 };

struct CellPlan {
    int kind = 0, L = 0, B = 0, H = 0, S = 0, device = -1;
    std::vector<uint64_t> uids;            // W (and Wp) of every layer
    int in_size[kMaxLayers] = {};
    float* d_v[kMaxLayers] = {};           // [B, in_size[l] + S]
    float* d_v2 = nullptr;                 // reset-before GRU: [B, max(in_size) + H] = [u ; r * h] of the layer being worked on
    float* d_z = nullptr;                  // pre-activations of the layer being worked on, [B, G * H]
    float* d_z2 = nullptr;                 // reset-before GRU: the candidate's pre-activation, [B, H]
    float* d_m = nullptr;                  // LSTMP: o * tanh(c), [B, H]
    float* d_c = nullptr;                  // LSTMP: [L, B, H]
    float* d_stage = nullptr;              // host-I/O staging of x and y
    size_t stage_cap = 0;
    std::vector<csb_matrix*> rz, nn;       // reset-before GRU: rows r, z and rows n of every layer as matrices of their own
    ~CellPlan() {
        for (float* p : d_v) cudaFree(p);
        cudaFree(d_v2); cudaFree(d_z); cudaFree(d_z2); cudaFree(d_m); cudaFree(d_c); cudaFree(d_stage);
        for (csb_matrix* a : rz) csb_free(a);
        for (csb_matrix* a : nn) csb_free(a);
    }
};
static std::recursive_mutex g_cell_mu;      // (a plan that fails half-built frees its row slices, which looks for plans again)
static std::list<std::unique_ptr<CellPlan>> g_cell_plans;

void drop_cell_plans(const csb_matrix* A) {
    std::list<std::unique_ptr<CellPlan>> doomed;   // destroyed outside the lock: their slices are freed through csb_free, which comes back here
    {
        std::lock_guard<std::recursive_mutex> lk(g_cell_mu);
        for (auto it = g_cell_plans.begin(); it != g_cell_plans.end();) {
            if (std::find((*it)->uids.begin(), (*it)->uids.end(), A->uid) != (*it)->uids.end()) {
                doomed.push_back(std::move(*it));
                it = g_cell_plans.erase(it);
            } else ++it;
        }
    }
    int prev = 0;
    cudaGetDevice(&prev);
    for (auto& p : doomed) { cudaSetDevice(p->device); p.reset(); }
    cudaSetDevice(prev);
}

__device__ __forceinline__ float logistic_acc(float a) { return 1.f / (1.f + expf(-a)); }

// What every element-wise kernel does with a new state value s of unit j, batch column b: it goes to
// the recurrent part of this layer's V, to the input part of the next layer's V (when there is one)
// and to the output sequence (top layer).
struct Route {
    float* v_self; int ld_self, off_self;
    float* v_next; int ld_next;
    float* y_t;                            // [B, S] of this step, or null
    const float* x_next; int I0;           // next input frame [B, I0] to be put into v0 (layer 0 only), or null
    float* v0; int ld0;
};
__device__ __forceinline__ void route_state(const Route& r, int b, int j, int S, float s) {
    r.v_self[(size_t)b * r.ld_self + r.off_self + j] = s;
    if (r.v_next) r.v_next[(size_t)b * r.ld_next + j] = s;
    if (r.y_t) r.y_t[(size_t)b * S + j] = s;
}
__device__ __forceinline__ void route_input(const Route& r, int B) {
    if (!r.x_next) return;
    const int n = B * r.I0;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int b = e / r.I0, i = e - b * r.I0;
        r.v0[(size_t)b * r.ld0 + i] = r.x_next[e];
    }
}

// LSTMP, first half of a step: c_t = s(z_f) c_{t-1} + s(z_i) tanh(z_g), m_t = s(z_o) tanh(c_t); rows of z stacked i, f, g, o.
__global__ void csb_lstmp_gates_kernel(const float* __restrict__ Z, const float* __restrict__ bias, float* __restrict__ c, float* __restrict__ m,
                                       int B, int H) {
    const int n = B * H;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int b = e / H, j = e - b * H;
        const float* z = Z + (size_t)b * 4 * H;
        float zi = z[j], zf = z[H + j], zg = z[2 * H + j], zo = z[3 * H + j];
        if (bias) { zi += bias[j]; zf += bias[H + j]; zg += bias[2 * H + j]; zo += bias[3 * H + j]; }
        const float cn = logistic_acc(zf) * c[e] + logistic_acc(zi) * tanhf(zg);
        c[e] = cn;
        m[e] = logistic_acc(zo) * tanhf(cn);
    }
}
// LSTMP, second half: the projected state r_t = W_p m_t was written by the product into V_l's recurrent
// part; it is passed on to the layer above / the output, and the next frame moves in.
__global__ void csb_route_kernel(Route r, int B, int S) {
    const int n = B * S;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int b = e / S, j = e - b * S;
        const float s = r.v_self[(size_t)b * r.ld_self + r.off_self + j];
        if (r.v_next) r.v_next[(size_t)b * r.ld_next + j] = s;
        if (r.y_t) r.y_t[e] = s;
    }
    route_input(r, B);
}
// Li-GRU: z = s(a_z + b_z), cand = max(a_c + b_c, 0), h_t = z h_{t-1} + (1 - z) cand; rows of a stacked z, c.
__global__ void csb_ligru_gates_kernel(const float* __restrict__ Z, const float* __restrict__ bias, Route r, int B, int H) {
    const int n = B * H;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int b = e / H, j = e - b * H;
        const float* a = Z + (size_t)b * 2 * H;
        float az = a[j], ac = a[H + j];
        if (bias) { az += bias[j]; ac += bias[H + j]; }
        const float z = logistic_acc(az), cand = fmaxf(ac, 0.f);
        const float hp = r.v_self[(size_t)b * r.ld_self + r.off_self + j];
        route_state(r, b, j, H, z * hp + (1.f - z) * cand);
    }
    route_input(r, B);
}
// Reset-before GRU, first half: r = s(a_r + b_r), z = s(a_z + b_z); z stays in Z (over a_z), and
// V2 = [u_t ; r * h_{t-1}] is laid out for the candidate's product.
__global__ void csb_gru_rb_gate1_kernel(float* __restrict__ Z, const float* __restrict__ bias, const float* __restrict__ v, int ld, int I,
                                        float* __restrict__ v2, int B, int H) {
    const int n = B * H;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int b = e / H, j = e - b * H;
        float* a = Z + (size_t)b * 2 * H;
        float ar = a[j], az = a[H + j];
        if (bias) { ar += bias[j]; az += bias[H + j]; }
        a[H + j] = logistic_acc(az);
        v2[(size_t)b * ld + I + j] = logistic_acc(ar) * v[(size_t)b * ld + I + j];
    }
    const int nu = B * I;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < nu; e += gridDim.x * blockDim.x) {
        const int b = e / I, i = e - b * I;
        v2[(size_t)b * ld + i] = v[(size_t)b * ld + i];
    }
}
// Reset-before GRU, second half: n = tanh(a_n + b_n), h_t = (1 - z) n + z h_{t-1}.
__global__ void csb_gru_rb_gate2_kernel(const float* __restrict__ Z2, const float* __restrict__ Z, const float* __restrict__ bias, Route r, int B,
                                        int H) {
    const int n = B * H;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < n; e += gridDim.x * blockDim.x) {
        const int b = e / H, j = e - b * H;
        const float cand = tanhf(Z2[e] + (bias ? bias[2 * H + j] : 0.f));
        const float z = Z[(size_t)b * 2 * H + H + j];
        const float hp = r.v_self[(size_t)b * r.ld_self + r.off_self + j];
        route_state(r, b, j, H, (1.f - z) * cand + z * hp);
    }
    route_input(r, B);
}

static int cell_forward(int kind, int L, const csb_matrix_t* const* W, const csb_matrix_t* const* Wp, const float* const* bias, const float* x,
                        int64_t T, int B, const float* h0, const float* c0, float* y, float* hT, float* cT, unsigned flags, void* stream) {
    clear_error();
    if (L < 1 || L > kMaxLayers || !W || (kind == kCellLstmp && !Wp)) { set_error("n_layers %d (1..%d), W or Wp is NULL", L, (int)kMaxLayers); return CSB_ERR_INVALID_ARG; }
    if (T < 0 || B < 0) { set_error("T=%lld B=%d", (long long)T, B); return CSB_ERR_INVALID_ARG; }
    for (int l = 0; l < L; ++l)
        if (!W[l] || (kind == kCellLstmp && !Wp[l])) { set_error("matrix of layer %d is NULL", l); return CSB_ERR_INVALID_ARG; }
    const int G = kind == kCellLstmp ? 4 : kind == kCellLigru ? 2 : 3;
    if (W[0]->rows % G) { set_error("layer 0 has %lld rows, not a multiple of %d", (long long)W[0]->rows, G); return CSB_ERR_SHAPE; }
    const int H = (int)(W[0]->rows / G);
    const int S = kind == kCellLstmp ? (int)Wp[0]->rows : H;
    int in_size[kMaxLayers];
    for (int l = 0; l < L; ++l) {
        in_size[l] = (int)W[l]->cols - S;
        if (W[l]->rows != (int64_t)G * H || in_size[l] < 1 || (l > 0 && in_size[l] != S) || W[l]->device != W[0]->device || W[l]->device < 0) {
            set_error("layer %d: matrix is %lld x %lld on device %d; expected %d x (input + %d), input = %d above the first layer, all on one device",
                      l, (long long)W[l]->rows, (long long)W[l]->cols, W[l]->device, G * H, S, S);
            return CSB_ERR_SHAPE;
        }
        if (W[l]->val_dtype == CSB_Q16 || (kind == kCellLstmp && Wp[l]->val_dtype == CSB_Q16)) {
            set_error("layer %d holds fixed-point values: those serve csb_spmm_q16 only", l);
            return CSB_ERR_UNSUPPORTED;
        }
        if (kind == kCellLstmp && (Wp[l]->rows != S || Wp[l]->cols != H || Wp[l]->device != W[0]->device)) {
            set_error("layer %d: projection is %lld x %lld; expected %d x %d on the same device", l, (long long)Wp[l]->rows, (long long)Wp[l]->cols, S, H);
            return CSB_ERR_SHAPE;
        }
        if (kind == kCellGruRb && (2 * H) % W[l]->block_r) {
            set_error("layer %d: the reset-before GRU runs its gate rows and its candidate rows as two products, so 2 * hidden (%d) must be a multiple of block_r (%d)",
                      l, 2 * H, W[l]->block_r);
            return CSB_ERR_UNSUPPORTED;
        }
    }
    if (T == 0 || B == 0) return CSB_OK;
    if (!x) { set_error("x is NULL"); return CSB_ERR_INVALID_ARG; }
    int prev = 0;
    CSB_CUDA(cudaGetDevice(&prev));
    if (prev != W[0]->device) CSB_CUDA(cudaSetDevice(W[0]->device));
    struct Restore { int prev, cur; ~Restore() { if (prev != cur) cudaSetDevice(prev); } } restore{prev, W[0]->device};

    CellPlan* P = nullptr;
    {
        std::lock_guard<std::recursive_mutex> lk(g_cell_mu);
        for (auto& p : g_cell_plans) {
            if (p->kind != kind || p->L != L || p->B != B) continue;
            bool same = true;
            for (int l = 0; l < L; ++l) same = same && p->uids[l] == W[l]->uid && (kind != kCellLstmp || p->uids[L + l] == Wp[l]->uid);
            if (same) { P = p.get(); break; }
        }
        if (!P) {
            std::unique_ptr<CellPlan> np(new CellPlan());
            np->kind = kind; np->L = L; np->B = B; np->H = H; np->S = S; np->device = W[0]->device;
            for (int l = 0; l < L; ++l) np->uids.push_back(W[l]->uid);
            if (kind == kCellLstmp) for (int l = 0; l < L; ++l) np->uids.push_back(Wp[l]->uid);
            int max_in = 0;
            for (int l = 0; l < L; ++l) {
                np->in_size[l] = in_size[l];
                max_in = std::max(max_in, in_size[l]);
                CSB_CUDA(cudaMalloc((void**)&np->d_v[l], (size_t)B * (in_size[l] + S) * 4));
            }
            CSB_CUDA(cudaMalloc((void**)&np->d_z, (size_t)B * G * H * 4));
            if (kind == kCellLstmp) {
                CSB_CUDA(cudaMalloc((void**)&np->d_m, (size_t)B * H * 4));
                CSB_CUDA(cudaMalloc((void**)&np->d_c, (size_t)L * B * H * 4));
            }
            if (kind == kCellGruRb) {
                CSB_CUDA(cudaMalloc((void**)&np->d_v2, (size_t)B * (max_in + H) * 4));
                CSB_CUDA(cudaMalloc((void**)&np->d_z2, (size_t)B * H * 4));
                for (int l = 0; l < L; ++l) {
                    csb_matrix* a = nullptr;
                    const int64_t cut = (int64_t)2 * H / W[l]->block_r;
                    int rc = slice_block_rows(W[l], 0, cut, &a);
                    if (rc != CSB_OK) return rc;
                    np->rz.push_back(a);
                    rc = slice_block_rows(W[l], cut, W[l]->nbr, &a);
                    if (rc != CSB_OK) return rc;
                    np->nn.push_back(a);
                }
            }
            P = np.get();
            g_cell_plans.push_back(std::move(np));
        }
    }
    cudaStream_t st = (cudaStream_t)stream;
    const bool host_io = (flags & CSB_FLAG_HOST_IO) != 0;
    const int I0 = in_size[0];
    const size_t nx = (size_t)T * B * I0, ny = (size_t)T * B * S, nh = (size_t)L * B * S, nc = (size_t)L * B * H;
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
    const size_t srow = (size_t)S * 4;
    // V_l = [u_0 ; s_{-1}]: the initial state (or zeros) on the right, x_0 on the left of layer 0
    for (int l = 0; l < L; ++l) {
        const int ld = in_size[l] + S;
        float* spart = P->d_v[l] + in_size[l];
        if (h0) CSB_CUDA(cudaMemcpy2DAsync(spart, (size_t)ld * 4, h0 + (size_t)l * B * S, srow, srow, B, in_kind, st));
        else CSB_CUDA(cudaMemset2DAsync(spart, (size_t)ld * 4, 0, srow, B, st));
    }
    CSB_CUDA(cudaMemcpy2DAsync(P->d_v[0], (size_t)(I0 + S) * 4, dx, (size_t)I0 * 4, (size_t)I0 * 4, B, cudaMemcpyDeviceToDevice, st));
    if (kind == kCellLstmp) {
        if (c0) CSB_CUDA(cudaMemcpyAsync(P->d_c, c0, nc * 4, in_kind, st));
        else CSB_CUDA(cudaMemsetAsync(P->d_c, 0, nc * 4, st));
    }
    const int threads = 256;
    const int blocks = std::max(1, std::min(1024, (B * std::max(std::max(H, S), I0) + threads - 1) / threads));
    for (int64_t t = 0; t < T; ++t) {
        for (int l = 0; l < L; ++l) {
            const int ld = in_size[l] + S;
            const bool top = l == L - 1;
            const float* bl = bias ? bias[l] : nullptr;
            Route r{};
            r.v_self = P->d_v[l]; r.ld_self = ld; r.off_self = in_size[l];
            r.v_next = top ? nullptr : P->d_v[l + 1]; r.ld_next = top ? 0 : in_size[l + 1] + S;
            r.y_t = (top && dy) ? dy + (size_t)t * B * S : nullptr;
            r.x_next = (l == 0 && t + 1 < T) ? dx + (size_t)(t + 1) * B * I0 : nullptr; r.I0 = I0;
            r.v0 = P->d_v[0]; r.ld0 = I0 + S;
            int rc;
            if (kind == kCellLstmp) {
                if ((rc = product_any(W[l], P->d_v[l], ld, B, P->d_z, (int64_t)4 * H, stream)) != CSB_OK) return rc;
                csb_lstmp_gates_kernel<<<blocks, threads, 0, st>>>(P->d_z, bl, P->d_c + (size_t)l * B * H, P->d_m, B, H);
                if ((rc = product_any(Wp[l], P->d_m, H, B, P->d_v[l] + in_size[l], ld, stream)) != CSB_OK) return rc;
                csb_route_kernel<<<blocks, threads, 0, st>>>(r, B, S);
            } else if (kind == kCellLigru) {
                if ((rc = product_any(W[l], P->d_v[l], ld, B, P->d_z, (int64_t)2 * H, stream)) != CSB_OK) return rc;
                csb_ligru_gates_kernel<<<blocks, threads, 0, st>>>(P->d_z, bl, r, B, H);
            } else {
                if ((rc = product_any(P->rz[l], P->d_v[l], ld, B, P->d_z, (int64_t)2 * H, stream)) != CSB_OK) return rc;
                csb_gru_rb_gate1_kernel<<<blocks, threads, 0, st>>>(P->d_z, bl, P->d_v[l], ld, in_size[l], P->d_v2, B, H);
                if ((rc = product_any(P->nn[l], P->d_v2, ld, B, P->d_z2, (int64_t)H, stream)) != CSB_OK) return rc;
                csb_gru_rb_gate2_kernel<<<blocks, threads, 0, st>>>(P->d_z2, P->d_z, bl, r, B, H);
            }
            CSB_CUDA(cudaGetLastError());
        }
    }
    if (hT)
        for (int l = 0; l < L; ++l)
            CSB_CUDA(cudaMemcpy2DAsync(hT + (size_t)l * B * S, srow, P->d_v[l] + in_size[l], (size_t)(in_size[l] + S) * 4, srow, B, out_kind, st));
    if (cT && kind == kCellLstmp) CSB_CUDA(cudaMemcpyAsync(cT, P->d_c, nc * 4, out_kind, st));
    if (host_io && y) CSB_CUDA(cudaMemcpyAsync(y, dy, ny * 4, cudaMemcpyDeviceToHost, st));
    (void)nh;
    if (host_io || !(flags & CSB_FLAG_ASYNC)) {
        CSB_CUDA(cudaStreamSynchronize(st));
        auto gave_up = [&](const csb_matrix* a) { return a->product.h_status && *a->product.h_status != 0; };
        for (int l = 0; l < L; ++l)
            if (gave_up(W[l]) || (kind == kCellLstmp && gave_up(Wp[l])) || (kind == kCellGruRb && (gave_up(P->rz[l]) || gave_up(P->nn[l])))) {
                set_error("a product kernel of layer %d gave up a bounded wait", l);
                return CSB_ERR_TIMEOUT;
            }
    }
    return CSB_OK;
}

}  // namespace csb

extern "C" {

int csb_lstmp_forward(int n_layers, const csb_matrix_t* const* W, const csb_matrix_t* const* Wp, const float* const* bias, const float* x, int64_t T,
                      int B, const float* h0, const float* c0, float* y, float* hT, float* cT, unsigned flags, void* stream) {
    return csb::cell_forward(csb::kCellLstmp, n_layers, W, Wp, bias, x, T, B, h0, c0, y, hT, cT, flags, stream);
}

int csb_ligru_forward(int n_layers, const csb_matrix_t* const* W, const float* const* bias, const float* x, int64_t T, int B, const float* h0,
                      float* y, float* hT, unsigned flags, void* stream) {
    return csb::cell_forward(csb::kCellLigru, n_layers, W, nullptr, bias, x, T, B, h0, nullptr, y, hT, nullptr, flags, stream);
}

int csb_gru_reset_before_forward(int n_layers, const csb_matrix_t* const* W, const float* const* bias, const float* x, int64_t T, int B,
                                 const float* h0, float* y, float* hT, unsigned flags, void* stream) {
    return csb::cell_forward(csb::kCellGruRb, n_layers, W, nullptr, bias, x, T, B, h0, nullptr, y, hT, nullptr, flags, stream);
}

}  // extern "C"
