/*
 * libcsb -- compressed-structured-block (CSB) sparse products and the fused
 * LSTM / GRU time loop on one NVIDIA B200 (sm_100a).
 *
 * The operations follow "CSB-RNN" (arXiv 2005.05758):
 *   - the CSB matrix and its storage format: Section 3.1.1;
 *   - the CSB matrix-vector product (the CSB-Engine's job): Sections 4.2, 4.3.1;
 *   - the recurrent cell around it (products, sigmoid, tanh, element-wise
 *     product and sum, the c/h context link): Section 2.1.
 *
 * Conventions for every entry point
 *   - Returns CSB_OK (0) or a negative csb_status; no C++ exception crosses the
 *     boundary.  csb_last_error() gives a thread-local detail string.
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA
 *     global memory on the device the matrix was encoded for.  All buffers are
 *     owned by the caller and are neither retained nor freed by the library;
 *     handles (csb_matrix_t) are owned by the library until csb_free().
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Product calls only enqueue work; the recurrent calls additionally wait
 *     for their status word unless CSB_FLAG_ASYNC is given.
 *   - Matrix shape R x C: rows are output neurons, columns input neurons;
 *     blocks are block_r x block_c (1..256 each), block b = bi * nbc + bj in
 *     row-major block order; a short last block is allowed.
 *   - There is no CPU fallback: a call that needs the GPU fails with
 *     CSB_ERR_CUDA / CSB_ERR_UNSUPPORTED when no sm_100 device is present.
 */
#ifndef CSB_H_
#define CSB_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum csb_status {
    CSB_OK = 0,
    CSB_ERR_INVALID_ARG = -1,  /* null pointer, negative size, bad enum            */
    CSB_ERR_SHAPE = -2,        /* shapes of the arguments do not fit each other    */
    CSB_ERR_DTYPE = -3,        /* unknown value type                               */
    CSB_ERR_ALLOC = -4,        /* host or device allocation failed                 */
    CSB_ERR_CUDA = -5,         /* a CUDA runtime call failed (see csb_last_error)  */
    CSB_ERR_LAUNCH = -6,       /* the persistent grid cannot be co-resident        */
    CSB_ERR_TIMEOUT = -7,      /* a bounded device-side wait expired               */
    CSB_ERR_UNSUPPORTED = -8   /* valid request this build does not implement      */
} csb_status;

enum { CSB_F32 = 0, CSB_F16 = 1,            /* storage type of the packed values */
       CSB_Q16 = 2 };                       /* 16-bit fixed point; handles made by csb_encode_q16 only */
enum { CSB_FLAG_ASYNC = 1u,                 /* recurrent calls: do not wait for the status word */
       CSB_FLAG_HOST_IO = 2u };             /* recurrent calls: sequence and state pointers are host memory */

typedef struct csb_matrix csb_matrix_t;     /* opaque: canonical arrays + device layout + schedule */

/* Tuning knobs of the one-shot planning step of the CUDA-core product kernel; zero means
 * "library default".  Values outside the stated ranges make csb_encode fail with
 * CSB_ERR_INVALID_ARG; so does a ring (warps x stages x stage_bytes) that cannot fit one CTA's
 * shared memory even after the planner has reduced the warps per CTA. */
typedef struct csb_plan_opts {
    int ctas;            /* persistent grid size, >= 0 (default: SM count)                        */
    int warps_per_cta;   /* warps per CTA, 0..16 (default 16)                                     */
    int stage_bytes;     /* bytes per shared-memory ring stage of one warp, 1024..16384, rounded  */
                         /* up to a multiple of 16 (default 4096)                                 */
    int stages;          /* ring depth per warp, 1..8 (default 2)                                 */
} csb_plan_opts;

/* The canonical CSB arrays of Section 3.1.1 (n{}, m{}, RowIdx{}, ColIdx{}, Val{}) plus
 * the offsets the paper leaves out.  All pointers are host memory borrowed from the
 * handle and stay valid until csb_free(). */
typedef struct csb_view {
    int64_t rows, cols;
    int32_t block_r, block_c;
    int64_t nbr, nbc, nblk, nnz;
    int32_t val_dtype;           /* CSB_F32 | CSB_F16 | CSB_Q16 (int16 values)         */
    const uint16_t* m;           /* [nblk] kept rows per block                         */
    const uint16_t* n;           /* [nblk] kept columns per block                      */
    const uint8_t* row_idx;      /* in-block indices, 0-based, ascending, concatenated */
    const uint8_t* col_idx;
    const uint64_t* val_off;     /* [nblk+1] exclusive prefix sum of m*n               */
    const uint32_t* ridx_off;    /* [nblk+1] exclusive prefix sum of m                 */
    const uint32_t* cidx_off;    /* [nblk+1] exclusive prefix sum of n                 */
    const void* val;             /* [nnz] kernel matrices, row-major inside a block    */
} csb_view_t;

/* Figures derived at encode / plan time. */
typedef struct csb_info {
    int64_t nnz;                 /* stored weights, sum of m_b * n_b                        */
    double pruning_rate;         /* rows * cols / nnz (Section 1)                           */
    double nio;                  /* normalized index overhead, sum(m+n) / nnz (Sec. 6.2.1)  */
    int64_t algorithmic_bytes;   /* values + index lists + 6-byte block headers             */
    int64_t device_stream_bytes; /* bytes of the private device layout actually streamed    */
    int32_t plan_ctas, plan_warps;
    double balance;              /* mean / max of the per-warp scheduled cost (1 = perfect) */
    /* the panel layout that csb_spmv streams for fp16 matrices (all zero when it does not apply) */
    int64_t panel_stream_bytes;  /* bytes of all panels (bookkeeping + values)              */
    int32_t panel_ctas, panel_warps;
    double panel_balance;        /* mean / max of the per-CTA modelled cost                 */
} csb_info_t;

/*
 * csb_encode -- build the CSB storage format (Section 3.1.1) from a dense weight and
 * per-block keep masks, and plan its execution on `device`.
 *   dense     host, float32, rows x cols, row stride ld (>= cols) elements.
 *   row_keep  host, [nblk * block_r] bytes; byte b*block_r + i != 0 keeps in-block row i of
 *             block b.  col_keep likewise, [nblk * block_c].  Bytes that fall beyond the
 *             matrix edge in a short last block are ignored.
 *   val_dtype CSB_F32 keeps the bit patterns; CSB_F16 rounds to binary16, nearest-even.
 *   device    CUDA device ordinal, or -1 for the host-side arrays only (csb_view works,
 *             products fail with CSB_ERR_UNSUPPORTED).
 *   opts      may be NULL.
 * A block with no kept row or no kept column stores no values but still lists the other
 * side's indices.  On success *out owns copies of everything; the inputs may be released.
 * Errors: INVALID_ARG (null, sizes <= 0, ld < cols, blocks outside 1..256), DTYPE, ALLOC, CUDA.
 */
int csb_encode(const float* dense, int64_t rows, int64_t cols, int64_t ld, int block_r, int block_c,
               const uint8_t* row_keep, const uint8_t* col_keep, int val_dtype, int device,
               const csb_plan_opts* opts, csb_matrix_t** out);

/*
 * csb_project -- project a dense weight onto the CSB pattern: the RowPrune / ColumnPrune step of
 * Algorithm 1 (Section 3.2), which gives the keep masks csb_encode takes.  RowPrune: in every
 * block-column on its own, the squared l2-norm of each row segment (the part of a matrix row inside
 * the block-column) is taken and the weakest segments are pruned; ColumnPrune: the same with the
 * column segments of every block-row of the result (pruned row segments count as zeros).  Each
 * prunes the fraction p = 1 - sqrt(1 - prune_fraction), so about prune_fraction of the weights are
 * gone after both (prune_fraction = 0.75 is the paper's "4x").  Where the paper is silent: the
 * number pruned per block-column is floor(p * rows + 0.5) (per block-row floor(p * cols + 0.5));
 * among equal norms the higher index is pruned first; norms are summed in fp64.
 *   dense       device, float32, rows x cols, row stride ld (>= cols) elements; not modified.
 *   row_keep    device, [nblk * block_r] bytes, written: 1 = kept, in csb_encode's layout (flags of
 *               in-block lines beyond the matrix edge are 0).  col_keep likewise, [nblk * block_c].
 *   workspace   device, csb_project_workspace_bytes(...) bytes of scratch, caller-owned.
 * Asynchronous on `stream`; all pointers on the current device.  The pruned matrix itself is
 * dense with the masked entries zeroed; csb_encode applies the masks.
 * Errors: INVALID_ARG (null, sizes, blocks outside 1..256, fraction outside [0, 1], workspace
 * too small), UNSUPPORTED (rows or cols above 20480), CUDA.
 */
int64_t csb_project_workspace_bytes(int64_t rows, int64_t cols, int block_r, int block_c);
int csb_project(const float* dense, int64_t rows, int64_t cols, int64_t ld, int block_r, int block_c, double prune_fraction,
                uint8_t* row_keep, uint8_t* col_keep, void* workspace, int64_t workspace_bytes, void* stream);

/* Borrow the canonical arrays (host memory, valid until csb_free). */
int csb_view(const csb_matrix_t* A, csb_view_t* out);

/* Encoder / planner statistics. */
int csb_info(const csb_matrix_t* A, csb_info_t* out);

/* Release a handle and everything planned from it (NULL is a no-op).  Must not run while
 * work using the handle is still in flight. */
void csb_free(csb_matrix_t* A);

/*
 * csb_spmv -- y = A . x, the CSB matrix-vector product (Sections 4.2, 4.3.1): per block the kept
 * inputs are read through ColIdx, multiplied by the kernel matrix and accumulated into the
 * outputs through RowIdx; blocks of a block-row accumulate into the same outputs.
 *   x  device, float32 [cols];  y  device, float32 [rows], overwritten (rows kept in no block
 *   become exactly 0).  fp32 accumulation, fixed summation order (bit-reproducible).
 * Asynchronous on `stream`.  Calls on the same handle must not overlap on the GPU: they share
 * the handle's scratch for partial block-row sums.
 * Matrices with fp16 values (block_c <= 128, cols <= 16384) run the panel kernel: every CTA owns
 * a range of output rows, so it needs no scratch.  That kernel is launched with programmatic
 * stream serialization: its start-up overlaps the end of the work in front of it on `stream`,
 * and it waits for that work before it reads x or writes y (CSB_PANEL_PDL=0 in the environment,
 * looked up at every call, asks for an ordinary launch; CSB_NO_PANEL=1 at encode time for the other
 * kernel).
 */
int csb_spmv(const csb_matrix_t* A, const float* x, float* y, void* stream);

/*
 * csb_spmm -- Y[b, :] = A . X[b, :] for b < batch: the CSB matrix-vector product of Sections 4.2 and
 * 4.3.1 (gather through ColIdx, kernel matrix, accumulate through RowIdx) with a batch of vectors.
 *   X  device, float32, batch rows of `cols` values, row stride ldx >= cols;
 *   Y  device, float32, batch rows of `rows` values, row stride ldy >= rows, overwritten.
 * batch = 0 is a no-op.  Same ordering / overlap rules as csb_spmv; results are bit-reproducible.
 * With batch >= 8, fp16 values and block_r <= 64 the product runs on tensor cores (the kernel
 * matrix times the gathered inputs is then a dense contraction), 32 batch columns per pass: the
 * inputs are split into two binary16 halves (x = hi + lo, so no input precision is lost as long
 * as |x| < 65504; larger or non-finite inputs give inf / NaN) and multiplied with
 * mma.sync.m16n8k16, fp32 accumulation, a block-row's outputs staying in registers across its
 * blocks.  The first such call on a handle for a batch size class (<= 8, <= 16, more)
 * builds a device layout for that class and a staging buffer for the packed inputs (allocates and
 * synchronises the device once; make it outside of any stream capture).  The two kernels of this path are launched
 * with programmatic stream serialization and wait, first thing, for the work in front of them on
 * `stream`.  Other cases use the CUDA-core kernel in batch tiles of 8 / 4 / 1.
 */
int csb_spmm(const csb_matrix_t* A, const float* X, int64_t ldx, int batch, float* Y, int64_t ldy,
             void* stream);

/*
 * csb_spmv_static_scratch -- y = A . x like csb_spmv, for callers that must not allocate device
 * memory.  (The paper has no counterpart; this is a packaging variant of the same kernel.)
 *
 * Who needs it: code that runs after an application has frozen its device-memory budget, or from
 * a thread or callback in which cudaMalloc / cudaFree are off limits because they synchronise the
 * whole device and may fail late -- an inference server's request loop, a real-time control loop,
 * a plug-in that is handed a fixed arena.  The product kernel needs scratch in global memory
 * (partial sums of block-rows shared by several warps, and their arrival counters).  csb_spmv
 * takes it from buffers allocated together with the handle; this variant takes it from one fixed
 * 4 MiB array that is part of the library image, so it calls no allocator at all (neither CUDA's
 * nor any library's).  Every GPU that loads the library holds those 4 MiB until the process ends.
 *
 *   A, x, y, stream   as for csb_spmv (device pointers, fp32, y overwritten, asynchronous).
 * Limits: at most 16384 block-rows (64 KiB of counters) and 4 MiB - 64 KiB of partial sums,
 * i.e. (number of shared warp/block-row pairs) * block_r * 4 bytes; a matrix beyond either limit
 * is refused with CSB_ERR_UNSUPPORTED and a message that names both sizes (csb_spmv still works).
 * Set-up: the first call on each device looks up the array's device address (once, cached); make
 * that first call outside of any stream capture.  Every call clears the counters it is going to
 * use on `stream` before the kernel; the partial sums are not cleared because each slot is
 * written before it is read.  The array is shared by ALL handles and keeps the last call's
 * contents: two calls of this function that overlap on the GPU (different streams, or different
 * host threads without ordering between their streams) race on it and give wrong results.  Calls
 * queued on one stream are safe.  Results equal those of csb_spmv's stream kernel bit for bit
 * (csb_spmv itself may run the panel kernel, whose summation order differs).
 * Errors: INVALID_ARG (null), UNSUPPORTED (host-only handle, limits, device ordinal > 63),
 * TIMEOUT (an earlier product on the handle gave up a bounded wait), CUDA.
 */
int csb_spmv_static_scratch(const csb_matrix_t* A, const float* x, float* y, void* stream);

/*
 * csb_lstm_forward -- a stack of LSTM layers over a whole sequence in one persistent kernel
 * (Section 2.1; one CSB product per layer and step, gate arithmetic fused behind it).
 *   W[l]     CSB matrix [4*H, I_l + H], I_0 = I, I_l = H above; stacked gate rows i, f, g, o;
 *            columns [0, I_l) multiply the layer input, the rest multiply h_{t-1}.
 *   bias[l]  device float32 [4*H], or NULL (bias may itself be NULL = no bias anywhere).
 *   x        float32 [T, B, I];  h0, c0  float32 [L, B, H] or NULL (zeros);
 *   y        float32 [T, B, H] top layer's h_t, or NULL;  hT, cT  float32 [L, B, H] or NULL.
 *   Per layer and step:  z = W.[u_t ; h_{t-1}] + b;  c_t = s(z_f)*c_{t-1} + s(z_i)*tanh(z_g);
 *   h_t = s(z_o)*tanh(c_t), with s the logistic function and u_t the layer's input.
 *   flags    CSB_FLAG_ASYNC: return without waiting (the status word is then not checked).
 *            CSB_FLAG_HOST_IO: x, h0, c0, y, hT, cT are HOST pointers; the call copies them
 *            through device staging buffers on `stream` and waits for the result.
 * The first call for a given (W..., B) builds and caches the time-loop schedule and its
 * device state (allocates, synchronises); later calls reuse it.  T = 0 or B = 0 is a no-op.
 * That cached state (the ring of h slots, the barrier and status words, staging buffers) is one
 * per (W..., B), not one per stream: two recurrent calls on the same matrices and batch size must
 * not overlap on the GPU.  Calls queued on one stream are safe; calls on different streams need an
 * event (or a synchronisation) between them, and then give identical bits.  The handles
 * themselves are immutable and may be used from any stream.
 * With B >= 16 (B >= 8 when the layers hold 100000 weights or more), fp16 values and block_r <= 64
 * the sequence is not run by the persistent kernel
 * but step by step: per layer and step the batched product on tensor cores (as csb_spmm, same
 * input-range rule) and one kernel with the gate arithmetic; same results within rounding, same
 * arguments and flags (CSB_RNN_NO_STEPWISE=1 in the environment keeps the persistent kernel).
 * Errors: SHAPE (rows != 4H, cols != I_l + H, layers disagree), LAUNCH (grid cannot be
 * co-resident; nothing was launched), TIMEOUT (the bounded grid barrier gave up; outputs are
 * undefined, the context stays usable), CUDA.
 */
int csb_lstm_forward(int n_layers, const csb_matrix_t* const* W, const float* const* bias,
                     const float* x, int64_t T, int B, const float* h0, const float* c0,
                     float* y, float* hT, float* cT, unsigned flags, void* stream);

/*
 * csb_gru_forward -- a stack of GRU layers over a whole sequence (the GRU cell of Section 2.1: one
 * CSB product per layer and step, gate arithmetic fused behind it); arguments, flags, caching and
 * the no-overlap rule as for csb_lstm_forward.  W[l] is [3*H, I_l + H], rows r, z, n; bias[l] is
 * device float32 [4*H] = b_r, b_z, b_in, b_hn.  The reset gate acts after the recurrent product:
 *   r = s(zx_r + zh_r + b_r);  z = s(zx_z + zh_z + b_z);
 *   n = tanh(zx_n + b_in + r * (zh_n + b_hn));  h_t = (1 - z) * n + z * h_{t-1},
 * where zx / zh are the parts of the product over the input / hidden columns.
 * At the same batch sizes as for the LSTM (fp16 values, block_r <= 64) the sequence runs step by
 * step: one tensor-core product per layer and step over 2B rows (row b holds [u_t ; 0], row
 * B + b holds [0 ; h_{t-1}], which keeps zx and zh apart) and one gate kernel.
 */
int csb_gru_forward(int n_layers, const csb_matrix_t* const* W, const float* const* bias,
                    const float* x, int64_t T, int B, const float* h0, float* y, float* hT,
                    unsigned flags, void* stream);

/*
 * 16-bit fixed-point CSB product: the arithmetic of the paper's own processing elements (weights
 * quantised to 16-bit fixed point, Section 6.2.2; 16-bit fixed-point multipliers, Section 6.3.1).
 * The paper fixes neither the place of the binary point, the rounding nor the accumulator width;
 * here a value v with f fraction bits is the integer clamp(rint(v * 2^f), -32768, 32767) (halves
 * to even, NaN -> 0), f is the caller's choice per matrix and per input, and the product returns
 * the exact integer accumulators (64 bits, cannot overflow), so the real result is
 * acc * 2^-(f_w + f_x) and does not depend on the order of summation.
 *
 * csb_encode_q16 -- as csb_encode, the values stored as int16 with `frac_bits` fraction bits
 * (0..30; csb_view then gives val_dtype = CSB_Q16 and int16 values).  block_r and block_c at
 * most 128.  Such a handle serves csb_spmm_q16 only: the floating-point products and the
 * recurrent calls refuse it with CSB_ERR_UNSUPPORTED.
 *
 * csb_spmm_q16 -- acc[b, :] = A_q . x_q[b, :] in integers.
 *   Xq   device, int16, batch rows of `cols` fixed-point inputs, row stride ldx >= cols;
 *   acc  device, int64, batch rows of `rows` accumulators, row stride ldy >= rows, overwritten
 *        (rows kept in no block become 0).  batch = 0 is a no-op; asynchronous on `stream`.
 * Errors: INVALID_ARG, SHAPE, UNSUPPORTED (handle is not CSB_Q16, host-only handle), CUDA.
 */
int csb_encode_q16(const float* dense, int64_t rows, int64_t cols, int64_t ld, int block_r, int block_c,
                   const uint8_t* row_keep, const uint8_t* col_keep, int frac_bits, int device, csb_matrix_t** out);
int csb_spmm_q16(const csb_matrix_t* A, const int16_t* Xq, int64_t ldx, int batch, int64_t* acc, int64_t ldy, void* stream);

/*
 * Cell variants of the paper's benchmark models (Table 1) and of the GRU reference of Section 2.1.
 * They run one timestep at a time: per layer and step the CSB products go through the kernels of
 * csb_spmv / csb_spmm (whichever serves the batch size) and small kernels do the element-wise
 * part.  Arguments, flags (CSB_FLAG_ASYNC, CSB_FLAG_HOST_IO), caching of per-(matrices, B) device
 * state on the first call and the no-overlap rule are those of csb_lstm_forward; T = 0 or B = 0
 * is a no-op; errors are INVALID_ARG, SHAPE, UNSUPPORTED, ALLOC, CUDA, TIMEOUT as there.
 *
 * csb_lstmp_forward -- LSTM with a recurrent projection (LSTMP, Table 1: the SR1 layers, whose sizes
 * fit a projection to 512 units and no peephole weights).
 *   W[l]   CSB matrix [4*H, I_l + P], rows i, f, g, o; the last P columns multiply the projected state;
 *          I_l = P above the first layer.   Wp[l]  CSB matrix [P, H], the projection (no bias).
 *   bias[l] device float32 [4*H] or NULL;  x [T, B, I];  h0 [L, B, P], c0 [L, B, H] or NULL (zeros);
 *   y [T, B, P] (top layer's projected state) or NULL;  hT [L, B, P], cT [L, B, H] or NULL.
 *   z = W.[u_t ; r_{t-1}] + b;  c_t = s(z_f) c_{t-1} + s(z_i) tanh(z_g);  m_t = s(z_o) tanh(c_t);  r_t = Wp.m_t.
 *
 * csb_ligru_forward -- light GRU (Li-GRU, Table 1: model SR3): no reset gate, rectified candidate.  The
 * batch normalisation of the cell's feed-forward products is, at inference, a per-unit scale (folded
 * into the weight rows by the caller) and shift (the bias here).
 *   W[l]   CSB matrix [2*H, I_l + H], rows z (update gate), c (candidate);  bias[l] [2*H] or NULL.
 *   a = W.[u_t ; h_{t-1}] + b;  z = s(a_z);  h_t = z h_{t-1} + (1 - z) max(a_c, 0).
 *
 * csb_gru_reset_before_forward -- GRU whose reset gate acts BEFORE the candidate's recurrent product
 * (two dependent products per step, where csb_gru_forward needs one).
 *   W[l]   CSB matrix [3*H, I_l + H], rows r, z, n;  bias[l] [3*H] = b_r, b_z, b_n or NULL.
 *   [a_r ; a_z] = W[0:2H].[u_t ; h_{t-1}];  r = s(a_r + b_r);  z = s(a_z + b_z);
 *   n = tanh(W[2H:3H].[u_t ; r * h_{t-1}] + b_n);  h_t = (1 - z) n + z h_{t-1}.
 *   The two row ranges run as products of their own, so 2*H must be a multiple of block_r (else UNSUPPORTED).
 */
int csb_lstmp_forward(int n_layers, const csb_matrix_t* const* W, const csb_matrix_t* const* Wp, const float* const* bias,
                      const float* x, int64_t T, int B, const float* h0, const float* c0, float* y, float* hT, float* cT,
                      unsigned flags, void* stream);
int csb_ligru_forward(int n_layers, const csb_matrix_t* const* W, const float* const* bias, const float* x, int64_t T, int B,
                      const float* h0, float* y, float* hT, unsigned flags, void* stream);
int csb_gru_reset_before_forward(int n_layers, const csb_matrix_t* const* W, const float* const* bias, const float* x, int64_t T,
                                 int B, const float* h0, float* y, float* hT, unsigned flags, void* stream);

/*
 * csb_test_barrier_hook -- testing aid for the give-up path of the time loop's waits on other
 * CTAs (the paper has no counterpart).  Makes every later recurrent call expect `extra_arrivals`
 * arrivals at its grid barrier that never come (at batch 1, where CTAs exchange h as flagged
 * values instead: wait for a step number that never comes) and bounds each such wait to
 * `limit_ns` nanoseconds, so the kernel returns with CSB_ERR_TIMEOUT instead of completing; (0, 0) restores normal operation
 * (no extra arrivals, 2 s bound).  Process-wide; not for production use.
 */
void csb_test_barrier_hook(unsigned int extra_arrivals, unsigned long long limit_ns);

/*
 * csb_plan_dump -- inspection / testing aid (the paper has no counterpart): plan the bare product
 * for a persistent grid of `ctas` x `warps_per_cta` warps and ring stages of `stage_bytes` bytes,
 * on the host only (works for handles encoded with device = -1), and copy the planned device
 * stream out so that its layout and schedule can be checked without a GPU.
 *   info_out        host, int64[8]: warps, chunks, stream bytes, lane-group width, row-owned flag,
 *                   CTAs, warps per CTA, partial-sum slots.  Always written.
 *   stream_out      host, `stream_cap` bytes, or NULL;  chunks_out  host, uint32 pairs
 *                   (offset in 16-byte units with the flush kind in the top two bits, bytes),
 *                   `chunks_cap` pairs, or NULL;  warp_begin_out  host, uint32[`warp_cap`], first
 *                   chunk of every warp plus one end entry, or NULL.
 * A buffer that is too small is an error (CSB_ERR_INVALID_ARG); call once with NULL buffers to
 * learn the sizes.
 */
int csb_plan_dump(const csb_matrix_t* A, int ctas, int warps_per_cta, int stage_bytes, int64_t* info_out,
                  uint8_t* stream_out, int64_t stream_cap, uint32_t* chunks_out, int64_t chunks_cap,
                  uint32_t* warp_begin_out, int64_t warp_cap);

/*
 * csb_panel_dump -- inspection / testing aid (the paper has no counterpart): plan the panel layout
 * that csb_spmv streams for fp16 matrices (one panel per CTA, which owns a contiguous range of
 * output rows: bookkeeping, then the re-tiled kernel-matrix rows), on the host only, and copy it
 * out so that layout and schedule can be checked without a GPU.
 *   info_out    host, int64[8]: CTAs, bytes of all panels, 0, largest bookkeeping part, largest
 *               gathered-input count, most output rows per CTA, and the CTA-level and warp-level
 *               balance (mean / max of the modelled cost) times 1e6.
 *   panels_out  host, `panels_cap` bytes, or NULL;  cta_out  host, four uint32 per CTA (offset of
 *               the panel in 16-byte units, bytes of bookkeeping, bytes of values, output rows),
 *               `cta_cap` entries, or NULL.
 * Errors: UNSUPPORTED when the layout does not apply (fp32 values, block_c > 128, cols > 16384,
 * stage_bytes not a power of two >= 8192, or a panel beyond the kernel's limits), INVALID_ARG for
 * a buffer that is too small; call once with NULL buffers to learn the sizes.
 */
int csb_panel_dump(const csb_matrix_t* A, int ctas, int warps_per_cta, int stage_bytes, int64_t* info_out,
                   uint8_t* panels_out, int64_t panels_cap, uint32_t* cta_out, int64_t cta_cap);

/*
 * csb_spmm_plan_dump -- inspection / testing aid (the paper has no counterpart): plan the
 * tensor-core layout of the batched product for a pass of `batch` columns (the class of batch sizes
 * <= 8, <= 16 or more) and `sm_count` SMs on the host only and copy it out, so that the layout and
 * the block -> CTA -> warp schedule can be checked without a GPU.  A CTA covers RG consecutive
 * block-rows times a range of block-columns and has W warps (32 for up to 8 batch columns, else
 * 16), each working for one block-row of the group; S CTAs share a row group.  Weight stream
 * cta * W + w belongs to warp w.
 *   info_out          host, int64[8]: CTAs, chunks, stream bytes, RG, 8-column batch tiles per warp
 *                     + 256 * W + 65536 * G (an input tile spans G block-columns), S, and the
 *                     warp-level and CTA-level balance (mean / max of the modelled cost) times 1e6.
 *   stream_out        host, `stream_cap` bytes, or NULL;  chunks_out  host, uint32 pairs (offset in
 *                     16-byte units, bytes), or NULL;  stream_begin_out  host, uint32 first chunk of
 *                     every weight stream plus one end entry, or NULL;  cta_out  host, 48 bytes per
 *                     CTA (int32 row group, range number, first block-column, input tiles, then
 *                     32 bytes: the block-row of the group each warp works for), `cta_cap` CTAs, or NULL.
 * A chunk is 16 bytes (first word: size of what follows in 16-byte units) followed by items; an
 * item is 16 bytes (u16 input tile counted from the CTA's first, u8 kept columns nk, u8 words
 * per stored row, u64 mask of the kept in-block rows, u16 size in 16-byte units), nk column indices
 * inside the input tile (block-column inside the tile times block_c plus the in-block index)
 * padded to 4 bytes, and the kept rows of the column slice, row-major, each padded to an even
 * number of halves.
 * Errors: UNSUPPORTED when the layout does not apply (fp32 values, block_r > 64), INVALID_ARG for a
 * buffer that is too small; call once with NULL buffers to learn the sizes.
 */
int csb_spmm_plan_dump(const csb_matrix_t* A, int batch, int sm_count, int64_t* info_out, uint8_t* stream_out, int64_t stream_cap,
                       uint32_t* chunks_out, int64_t chunks_cap, uint32_t* stream_begin_out, int64_t begin_cap, int32_t* cta_out,
                       int64_t cta_cap);

/* Short text for a status code; never NULL. */
const char* csb_strerror(int status);

/* Detail of the calling thread's most recent failure ("" if none); valid until that thread's
 * next library call. */
const char* csb_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* CSB_H_ */
