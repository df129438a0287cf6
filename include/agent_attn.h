/*
 * agent_attn.h - C ABI of the Agent Attention forward pass for NVIDIA B200 (sm_100a).
 *
 * The library evaluates, per (batch, head) pair ("slab") of N = grid_h * grid_w tokens laid
 * out row-major on a 2-D grid (token t = y * grid_w + x), the module of Eq. 6 of
 * "Agent Attention: On the Integration of Softmax and Linear Attention":
 *
 *     A   = Pooling(Q)                                   (n agents, text under Eq. 6)
 *     V_A = softmax(scale1 * A K^T + B1) V               (agent aggregation, Eq. 3 / Eq. 5)
 *     O   = softmax(scale2 * Q A^T + B2) V_A + DWC(V)    (agent broadcast,  Eq. 3 / Eq. 5 / Eq. 6)
 *
 * with scale = 1/sqrt(d) by default (Sec. 3.2), dense additive agent biases B1 [n x N] and
 * B2 [N x n] per head (Eq. 5; not multiplied by the scale), and DWC a depthwise 3x3
 * cross-correlation over the token grid with zero padding and no additive bias (Eq. 6, k = 3
 * in Eq. 7).
 *
 * General rules
 *  - Every pointer named "device" must be device memory of the handle's GPU, 16-byte aligned,
 *    dense with the stated shape (last index fastest).  The caller owns all buffers; the
 *    library allocates no device memory in any call below except agent_attn_create (one small
 *    status word).  Nothing may alias `out`.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  All device
 *    work is enqueued on it; calls return without synchronising unless stated otherwise.
 *  - Every int-returning function returns an aa_status.  On failure nothing was launched (or,
 *    for AA_ERR_CUDA, the launch failed) and agent_attn_last_error() describes the reason.
 *    No call throws, aborts or traps.
 *  - Results are bit-identical from run to run for the same inputs, handle configuration and
 *    device.
 */
#ifndef AGENT_ATTN_H_
#define AGENT_ATTN_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct agent_attn_handle agent_attn_handle;   /* opaque; host memory owned by the library */

typedef enum { AA_F32 = 0, AA_BF16 = 1, AA_F16 = 2 } aa_dtype;

typedef enum {
    AA_OK = 0,
    AA_ERR_INVALID_ARG = 1,   /* null pointer, bad shape, misaligned pointer, aliasing */
    AA_ERR_UNSUPPORTED = 2,   /* head_dim > 128, n_agents > 256, unknown dtype, ... */
    AA_ERR_WORKSPACE   = 3,   /* workspace (or staging) buffer too small */
    AA_ERR_CUDA        = 4,   /* a CUDA runtime call failed (no usable GPU included) */
    AA_ERR_TIMEOUT     = 5    /* a bounded device-side wait gave up (see query_status) */
} aa_status;

typedef enum {
    AA_PATH_AUTO = 0,         /* tensor-core kernels for bf16/f16: three streaming kernels for long token grids
                                 with few agents (n <= 64, d = 64, N >= 1024), one persistent task-queue kernel
                                 for short ones, tensor-memory kernels for n > 64; fp32 FMA kernels for f32 */
    AA_PATH_SIMT = 1,         /* fp32 FMA kernels for every dtype (slow; for cross-checks) */
    AA_PATH_UNFUSED = 2,      /* like AUTO, but always one kernel per step (pool, aggregate, broadcast) */
    AA_PATH_QUEUE = 3         /* like AUTO, but without the streaming kernels: the task-queue kernel wherever it
                                 applies (n <= 64, d = 64, W <= 64), whatever the number of tokens */
} aa_path;

typedef struct {
    int   batch;              /* B: batch entries per call                                  */
    int   heads;              /* h: heads per batch entry; slab index = b * heads + head    */
    int   head_dim;           /* d: 8..128, head_dim * sizeof(element) a multiple of 16     */
    int   max_tokens;         /* largest N = grid_h * grid_w any call will use              */
    int   max_agents;         /* largest n any call will use (<= 256)                       */
    int   dtype;              /* aa_dtype: element type of Q, K, V, A, B1, B2, Wd and out   */
    float scale1;             /* logit scale of the aggregation; 0 selects 1/sqrt(d)        */
    float scale2;             /* logit scale of the broadcast;   0 selects 1/sqrt(d)        */
    int   device;             /* CUDA device ordinal                                        */
    int   path;               /* aa_path                                                    */
} agent_attn_config;

/* Dense agent biases of Eq. 5, already composed (App. B); either member may be NULL. */
typedef struct {
    const void* b1;           /* device [heads][n][N]: added to scale1 * A K^T              */
    const void* b2;           /* device [heads][N][n]: added to scale2 * Q A^T              */
} agent_attn_bias;

/* Creates a handle for one configuration.  Makes cfg->device current for the duration of the
 * call, allocates one 4-byte device status word, and keeps only host-side plan data.
 * Errors: AA_ERR_INVALID_ARG (null, non-positive sizes), AA_ERR_UNSUPPORTED (limits above),
 * AA_ERR_CUDA (no such device, or the device is not compute capability 10.x). */
int agent_attn_create(agent_attn_handle** out, const agent_attn_config* cfg);

/* Frees the handle and its status word.  NULL is accepted. */
int agent_attn_destroy(agent_attn_handle* h);

/* Text of the most recent failure on this handle ("" if none); valid until the next call on
 * the handle.  NULL handle returns a static string. */
const char* agent_attn_last_error(const agent_attn_handle* h);

/* Bytes of device workspace that agent_attn_forward / agent_attn_aggregate need for this
 * grid and agent count (holds A, V_A, the per-split online-softmax partials (max, sum, acc),
 * one arrival counter per slab and, for the streaming kernels, scaled copies of the agents, the
 * biases clamped to finite values and re-laid for the tensor core, and the depthwise filter as
 * diagonal operand slices).  Returns 0 on invalid arguments.  Its contents need no initialisation
 * and carry nothing from call to call; it may be reused by any number of calls that do not
 * overlap on the GPU.  After agent_attn_forward the pooled agents A ([B][heads][n][d], element
 * type) sit at offset 0 and the agent features V_A (same shape) at the next multiple of 256 bytes:
 * callers may read them (the tests do). */
size_t agent_attn_workspace_bytes(const agent_attn_handle* h, int grid_h, int grid_w, int n_agents);

/* The whole module, Eq. 6.
 *   Q, K, V     device [B][heads][N][d]
 *   A           device [B][heads][n][d] agent tokens, or NULL: A = average pooling of Q over the
 *               grid to a p x p agent grid with n = p * p (window of cell (ay, ax): rows
 *               floor(ay*H/p) .. ceil((ay+1)*H/p) - 1, columns likewise); then n_agents must be a
 *               perfect square with p <= min(grid_h, grid_w)
 *   bias        NULL, or biases of Eq. 5 (members may be NULL individually)
 *   dwc_weight  device [heads][d][3][3] or NULL (no DWC term).  tap (u, v) multiplies
 *               V[y + u - 1][x + v - 1]; taps outside the grid contribute zero
 *   out         device [B][heads][N][d]
 *   workspace   device, >= agent_attn_workspace_bytes(...)
 * Errors: AA_ERR_INVALID_ARG, AA_ERR_UNSUPPORTED (N > max_tokens, n > max_agents),
 * AA_ERR_WORKSPACE, AA_ERR_CUDA.  Performs no host synchronisation and no allocation. */
int agent_attn_forward(agent_attn_handle* h,
                       const void* Q, const void* K, const void* V, const void* A,
                       int grid_h, int grid_w, int n_agents,
                       const agent_attn_bias* bias, const void* dwc_weight,
                       void* out, void* workspace, size_t workspace_bytes, void* stream);

/* The whole module, Eq. 6, on token-major tensors with explicit strides (Eq. 1 computes Q, K and V with one
 * projection per token: its output, kept as [B][N][heads][d] or interleaved as [B][N][3][heads][d], is read
 * in place, and O can be written as [B][N][heads][d] for the projection that follows).
 *   Q, K, V      device; element (b, head, token, c) of each at
 *                base + b * in_strides[0] + head * in_strides[1] + token * in_strides[2] + c
 *   in_strides   host, 3 values in ELEMENTS: batch, head, token stride shared by Q, K and V (the d channels of
 *                a token are contiguous); each a multiple of 16 bytes, token stride >= head_dim
 *   out          device; element (b, head, token, c) at base + b * out_strides[0] + head * out_strides[1]
 *                + token * out_strides[2] + c
 *   everything else as in agent_attn_forward (A, biases and the filter are dense).
 * Dense strides {heads*N*d, N*d, d} make this call identical to agent_attn_forward.  Other strides run on the
 * fused and the tensor-memory kernels only: AA_ERR_UNSUPPORTED for fp32, head_dim > 64 (or != 64 with
 * n_agents <= 64), caller-supplied A with n_agents <= 64, n_agents > 64 not a multiple of 8, N not a multiple
 * of 8 with a bias, and handles created with a path other than AA_PATH_AUTO.  Other errors as in
 * agent_attn_forward.  No host synchronisation, no allocation. */
int agent_attn_forward_strided(agent_attn_handle* h,
                               const void* Q, const void* K, const void* V, const void* A,
                               const long long in_strides[3],
                               int grid_h, int grid_w, int n_agents,
                               const agent_attn_bias* bias, const void* dwc_weight,
                               void* out, const long long out_strides[3],
                               void* workspace, size_t workspace_bytes, void* stream);

/* Gradient buffers of agent_attn_backward, all fp32 device memory owned by the caller and overwritten
 * by the call (no accumulation into their previous contents). */
typedef struct {
    void* dq;                 /* [B][heads][N][d], required                                  */
    void* dk;                 /* [B][heads][N][d], required                                  */
    void* dv;                 /* [B][heads][N][d], required                                  */
    void* db1;                /* [heads][n][N], or NULL: gradient of bias b1, summed over B  */
    void* db2;                /* [heads][N][n], or NULL: gradient of bias b2, summed over B  */
    void* dwd;                /* [heads][d][3][3], or NULL: gradient of the depthwise filter */
} agent_attn_grads;

/* Bytes of device workspace agent_attn_backward needs (fp32 copies of A, V_A, dV_A, dA, the row
 * statistics of the aggregation softmax and its per-block partial states).  0 on invalid arguments
 * or an unsupported shape. */
size_t agent_attn_backward_workspace_bytes(const agent_attn_handle* h, int grid_h, int grid_w, int n_agents);

/* Gradients of Eq. 6 with pooled agents (A = Pooling(Q), so dQ includes the path through the agents):
 * given d_out = dL/dO, writes dL/dQ, dL/dK, dL/dV and, where requested, dL/dB1, dL/dB2 (Eq. 5) and the
 * gradient of the depthwise filter.  The forward quantities are recomputed from Q, K and V; nothing
 * has to be saved by the forward call.
 *   Q, K, V, d_out   device [B][heads][N][d] in the handle's element type
 *   bias, dwc_weight as in agent_attn_forward (the same values the forward pass used)
 *   grads            host struct of fp32 device buffers (see agent_attn_grads)
 *   workspace        device, >= agent_attn_backward_workspace_bytes(...)
 * n_agents must be a perfect square p*p with p <= min(grid_h, grid_w), and n_agents * head_dim <= 16384.
 * Arithmetic: handles created with AA_PATH_AUTO run the three attention stages on the tensor cores for 16-bit
 * element types with n_agents <= 64 and head_dim == 64 (A, the probabilities and the logit gradients are
 * rounded to the element type before they enter a product, as in the forward pass; V_A, dV_A and the
 * probabilities that form V_A are carried as two 16-bit terms); every other shape, fp32 inputs, and handles
 * created with AA_PATH_SIMT or AA_PATH_UNFUSED compute in fp32 on CUDA cores throughout.  Sums over tokens
 * and over the batch are accumulated with floating-point atomics, so the low-order bits of the results may
 * differ from run to run (the one exception to the reproducibility rule above).
 * Errors: AA_ERR_INVALID_ARG (null, misaligned or aliasing buffers, n not a square, dwd without a
 * filter), AA_ERR_UNSUPPORTED (shape limits), AA_ERR_WORKSPACE, AA_ERR_CUDA.  No host synchronisation,
 * no allocation. */
int agent_attn_backward(agent_attn_handle* h,
                        const void* Q, const void* K, const void* V, const void* d_out,
                        int grid_h, int grid_w, int n_agents,
                        const agent_attn_bias* bias, const void* dwc_weight,
                        const agent_attn_grads* grads,
                        void* workspace, size_t workspace_bytes, void* stream);

/* Step 1 alone: agent tokens by pooling (text under Eq. 6).  Q device [B][heads][N][d] ->
 * A_out device [B][heads][n][d], n = pool_h * pool_w, windows as described above. */
int agent_attn_pool(agent_attn_handle* h, const void* Q, int grid_h, int grid_w,
                    int pool_h, int pool_w, void* A_out, void* stream);

/* Step 2 alone: agent aggregation V_A = softmax(scale1 * A K^T + B1) V (Eq. 3, Eq. 5).
 * A device [B][heads][n][d]; K, V device [B][heads][N][d]; b1 device [heads][n][N] or NULL;
 * VA_out device [B][heads][n][d].  The N keys of a slab are split over thread blocks; the
 * workspace (>= agent_attn_workspace_bytes for any grid with grid_h * grid_w = n_tokens)
 * receives their partial (max, sum, acc) states, which the last block to finish merges in a
 * fixed order. */
int agent_attn_aggregate(agent_attn_handle* h, const void* A, const void* K, const void* V,
                         const void* b1, int n_tokens, int n_agents, void* VA_out,
                         void* workspace, size_t workspace_bytes, void* stream);

/* Step 3 alone: agent broadcast plus the DWC term, O = softmax(scale2 * Q A^T + B2) V_A + DWC(V)
 * (Eq. 3, Eq. 5, Eq. 6).  Q, V device [B][heads][N][d]; A, VA device [B][heads][n][d];
 * b2 device [heads][N][n] or NULL; dwc_weight device [heads][d][3][3] or NULL (V is then
 * unused and may be NULL). */
int agent_attn_broadcast(agent_attn_handle* h, const void* Q, const void* A, const void* VA,
                         const void* V, const void* b2, const void* dwc_weight,
                         int grid_h, int grid_w, int n_agents, void* out, void* stream);

/* Dense agent bias from its three components (App. B): out = (B'_c + B'_r + B'_b).reshape(n, N).
 *   col   device [heads][n][grid_w]            column bias, repeated over the grid rows, or NULL
 *   row   device [heads][n][grid_h]            row bias, repeated over the grid columns, or NULL
 *   blk   device [heads][n][block_h][block_w]  block bias, resized to grid_h x grid_w by bilinear
 *         interpolation with half-pixel centres and edge clamping (the paper says "repeating or
 *         interpolating"; this is the reading taken), or NULL
 *   transpose == 0: out device [heads][n][N] (the layout of b1);  != 0: [heads][N][n] (that of b2)
 * At least one component must be given.  The result is what agent_attn_forward takes as a bias. */
int agent_attn_compose_bias(agent_attn_handle* h, const void* col, const void* row, const void* blk,
                            int block_h, int block_w, int grid_h, int grid_w, int n_agents,
                            int transpose, void* out, void* stream);

/* Bytes of device staging memory that agent_attn_forward_host needs (room for Q, K, V, A, B1,
 * B2, Wd, out and the workspace, each 256-byte aligned).  0 on invalid arguments. */
size_t agent_attn_staging_bytes(const agent_attn_handle* h, int grid_h, int grid_w, int n_agents);

/* Eq. 6 on HOST buffers: same arguments as agent_attn_forward, but Q, K, V, A, the bias
 * members, dwc_weight and out are host pointers (pinned memory makes the copies asynchronous).
 * `staging` is device memory of >= agent_attn_staging_bytes(...) owned by the caller.
 * Enqueues host-to-device copies of every input, the forward pass and the device-to-host copy
 * of out on `stream`; the caller synchronises the stream before reading `out`. */
int agent_attn_forward_host(agent_attn_handle* h,
                            const void* Q, const void* K, const void* V, const void* A,
                            int grid_h, int grid_w, int n_agents,
                            const agent_attn_bias* bias, const void* dwc_weight,
                            void* out, void* staging, size_t staging_bytes, void* stream);

/* Synchronises `stream`, then returns the device-side status word: AA_OK, or AA_ERR_TIMEOUT if
 * a kernel's bounded wait expired since the last query (the word is cleared). */
int agent_attn_query_status(agent_attn_handle* h, void* stream);

/* Number of kernels the most recent successful call on this handle enqueued. */
int agent_attn_last_launch_count(const agent_attn_handle* h);

/* Test hook (no counterpart in the paper): how many times a block of the task-queue kernel polls another block's
 * counter before its wait gives up; 0xffffffff restores the built-in limit.  With 0 the first unsatisfied poll
 * expires: the kernel records AA_ERR_TIMEOUT in the status word and carries on with whatever the workspace holds
 * (a wrong result, every access still inside the caller's buffers; no copy is left in flight, since the mbarrier
 * waits keep their own limit).  Affects AA_PATH_QUEUE handles and the shapes AA_PATH_AUTO gives to that kernel. */
int agent_attn_test_set_poll_limit(agent_attn_handle* h, unsigned polls);

/* Measurement hook (no counterpart in the paper): which of the three streaming kernels agent_attn_forward
 * launches on the shapes it gives to them: bit 0 = prep (pooling, prepared operands), bit 1 = aggregation,
 * bit 2 = broadcast + depthwise term; 7 (the default) = the whole path.  A later stage launched alone reads what
 * an earlier full call left in the workspace, so each kernel can be timed by itself between CUDA events. */
int agent_attn_test_set_stage_mask(agent_attn_handle* h, unsigned mask);

/* Agent aggregation without any caller- or library-side allocation (the paper has no counterpart
 * of this call; it computes exactly what agent_attn_aggregate computes).
 *
 * Who it is for: code that must not, or cannot, call cudaMalloc at the point where it needs the
 * aggregation - for example a plugin running inside a host application that owns the memory pool,
 * a real-time loop with a fixed memory budget, or a caller that only holds its input and output
 * buffers and has nowhere to put a workspace.  agent_attn_aggregate needs a caller-provided
 * workspace for the per-split partial softmax states; this variant keeps them in a fixed array
 * inside the library image instead (agent_attn_static_scratch_bytes() = 32 MiB, resident on every
 * GPU that loads the library until the process exits).
 *
 * Arguments as agent_attn_aggregate, minus the workspace.  Shapes whose partial states do not fit
 * the fixed array are rejected with AA_ERR_WORKSPACE and a message that states both sizes.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress) and
 * caches it; make that first call outside any stream capture.  The call performs no cudaMalloc,
 * cudaFree or other allocating routine.  All calls (all handles, all streams) share the one
 * array: the arrival counters are cleared on `stream` at the start of each call and the partial
 * states are fully rewritten, so nothing is carried over from the previous call, but two calls
 * that overlap on the GPU (different streams, or different threads without ordering) race on it
 * and must be serialised by the caller. */
int agent_attn_aggregate_static(agent_attn_handle* h, const void* A, const void* K, const void* V,
                                const void* b1, int n_tokens, int n_agents, void* VA_out,
                                void* stream);

/* Size in bytes of the fixed scratch array used by agent_attn_aggregate_static. */
size_t agent_attn_static_scratch_bytes(void);

#ifdef __cplusplus
}
#endif
#endif  /* AGENT_ATTN_H_ */
