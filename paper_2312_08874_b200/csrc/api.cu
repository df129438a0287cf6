// C ABI of the agent-attention library: argument checks, workspace carving and kernel launches.
// Every step of the path runs in the CUDA kernels of this directory; there is no CPU fallback.
#include "../../include/agent_attn.h"
#include "kernels.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

using namespace aa;

struct agent_attn_handle {
    agent_attn_config cfg;
    float scale1, scale2;
    int sm_count;
    int elem_bytes;
    int* d_status;          // one device word: the kernels' bounded waits (mbarriers, flags) report here
    int launches;
    int fused_key[3];       // (grid_h, grid_w, n_agents) that fused_plan was made for
    FusedPlan fused_plan;
    int stream_key[4];      // (grid_h, grid_w, n_agents, pooled) that stream_plan was made for
    StreamPlan stream_plan;
    StreamArgs stream_args; // last call of the streaming path: its tensor maps are reused while the pointers repeat
    bool stream_args_valid;
    unsigned poll_limit;    // flag-poll limit of the task-queue kernel (test hook; 0xffffffff = the kernel's own)
    unsigned stage_mask;    // which of the three streaming kernels a forward call launches (measurement hook; 7 = all)
    char err[512];
};

namespace {

const char* kNullHandleMsg = "agent_attn: null handle";

int fail(agent_attn_handle* h, int code, const char* fmt, ...) {
    if (h) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(h->err, sizeof(h->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// AA_PATH_QUEUE differs from AA_PATH_AUTO only in skipping the streaming kernels.
bool auto_like(const agent_attn_handle* h) { return h->cfg.path == AA_PATH_AUTO || h->cfg.path == AA_PATH_QUEUE; }

bool use_simt(const agent_attn_handle* h) {
    return h->cfg.dtype == AA_F32 || h->cfg.path == AA_PATH_SIMT;
}

// Large agent counts go to the tensor-memory kernel (the shape rule does not depend on the bias, so
// that the workspace size is the same with and without one).
bool use_umma(const agent_attn_handle* h, int n_tokens, int n_agents) {
    return !use_simt(h) && auto_like(h) &&
           aggregate_umma_eligible(h->cfg.dtype, n_agents, n_tokens, h->cfg.head_dim, true);
}

AggPlan plan_for(const agent_attn_handle* h, int n_tokens, int n_agents) {
    const int slabs = h->cfg.batch * h->cfg.heads;
    if (use_umma(h, n_tokens, n_agents))
        return plan_aggregate_umma(slabs, n_agents, n_tokens, h->cfg.head_dim, h->sm_count);
    return use_simt(h) ? plan_aggregate_simt(slabs, n_agents, n_tokens, h->cfg.head_dim, h->sm_count)
                       : plan_aggregate_mma(slabs, n_agents, n_tokens, h->cfg.head_dim, h->sm_count);
}

// Plan of the streaming path for a call shape (cached in the handle); ok = false where it does not apply.
const StreamPlan& stream_plan_for(agent_attn_handle* h, int grid_h, int grid_w, int n_agents, bool pooled) {
    if (h->stream_key[0] != grid_h || h->stream_key[1] != grid_w || h->stream_key[2] != n_agents ||
        h->stream_key[3] != (pooled ? 1 : 2)) {
        h->stream_plan = (h->cfg.path == AA_PATH_AUTO && h->cfg.dtype != AA_F32)
                             ? plan_stream(h->cfg.dtype, h->cfg.batch * h->cfg.heads, grid_h, grid_w, h->cfg.head_dim,
                                           n_agents, pooled, h->sm_count)
                             : StreamPlan{};
        h->stream_key[0] = grid_h; h->stream_key[1] = grid_w; h->stream_key[2] = n_agents;
        h->stream_key[3] = pooled ? 1 : 2;
        h->stream_args_valid = false;
    }
    return h->stream_plan;
}

// Workspace layout: [A | V_A | partials | tickets | streaming path: scaled agents, prepared biases], each region
// 256-byte aligned.
struct WsLayout {
    size_t a_off, va_off, part_off, ticket_off, extra_off, total;
};
WsLayout ws_layout(const agent_attn_handle* h, int n_tokens, int n_agents, int grid_h = 0, int grid_w = 0) {
    const size_t slabs = (size_t)h->cfg.batch * h->cfg.heads;
    const AggPlan pl = plan_for(h, n_tokens, n_agents);
    const size_t av = align_up(slabs * n_agents * h->cfg.head_dim * h->elem_bytes, 256);
    WsLayout w;
    w.a_off = 0;
    w.va_off = av;
    w.part_off = 2 * av;
    // sized for either launch plan (per-step kernels or the fused kernel)
    size_t part_floats = slabs * pl.parts * partial_floats(pl.rows_pad, pl.dpad);
    if (grid_h > 0 && auto_like(h)) {
        const size_t fused_floats = slabs * (size_t)fused_parts_per_slab(h->cfg.dtype, grid_h, grid_w, h->cfg.head_dim, n_agents) *
                                    partial_floats(64, h->cfg.head_dim);
        if (part_floats < fused_floats) part_floats = fused_floats;
    }
    size_t extra = 0;
    if (grid_h > 0) {
        // the larger of the plans for pooled and for caller-supplied agents (the size must not depend on A)
        for (int pooled = 0; pooled < 2; ++pooled) {
            const StreamPlan sp = (h->cfg.path == AA_PATH_AUTO && h->cfg.dtype != AA_F32)
                                      ? plan_stream(h->cfg.dtype, (int)slabs, grid_h, grid_w, h->cfg.head_dim, n_agents, pooled != 0, h->sm_count)
                                      : StreamPlan{};
            if (!sp.ok) continue;
            const size_t sf = slabs * (size_t)sp.splits * partial_floats(64, 64);
            if (part_floats < sf) part_floats = sf;
            extra = stream_extra_bytes((int)slabs, h->cfg.heads, n_tokens, n_agents);
        }
    }
    w.ticket_off = w.part_off + align_up(part_floats * sizeof(float), 256);
    w.extra_off = w.ticket_off + align_up(fused_counter_words((int)slabs) * sizeof(unsigned), 256);
    w.total = w.extra_off + extra;
    return w;
}

int check_shape(agent_attn_handle* h, int n_tokens, int n_agents) {
    if (n_tokens <= 0 || n_agents <= 0)
        return fail(h, AA_ERR_INVALID_ARG, "token and agent counts must be positive (N=%d, n=%d)", n_tokens, n_agents);
    if (n_tokens > h->cfg.max_tokens)
        return fail(h, AA_ERR_UNSUPPORTED, "N=%d exceeds the handle's max_tokens=%d", n_tokens, h->cfg.max_tokens);
    if (n_agents > h->cfg.max_agents)
        return fail(h, AA_ERR_UNSUPPORTED, "n=%d exceeds the handle's max_agents=%d", n_agents, h->cfg.max_agents);
    return AA_OK;
}

int isqrt_exact(int n) {
    int p = (int)std::lround(std::sqrt((double)n));
    return (p * p == n) ? p : -1;
}

// Layouts of the token-major tensors of a call: Q, K and V share `in`, O has `out`.
struct CallLayout {
    TokLayout in, out;
    bool strided;
};
CallLayout dense_call(const agent_attn_handle* h, int n_tokens) {
    CallLayout l;
    l.in = l.out = dense_layout(h->cfg.heads, n_tokens, h->cfg.head_dim);
    l.strided = false;
    return l;
}

int do_pool(agent_attn_handle* h, const void* Q, int gh, int gw, int ph, int pw, void* A, cudaStream_t st,
            const CallLayout* cl = nullptr) {
    PoolArgs pa;
    pa.q = Q; pa.a = A;
    pa.slabs = h->cfg.batch * h->cfg.heads;
    pa.H = gh; pa.W = gw; pa.d = h->cfg.head_dim; pa.ph = ph; pa.pw = pw;
    pa.heads = h->cfg.heads;
    pa.lq = cl ? cl->in : dense_layout(h->cfg.heads, (long long)gh * gw, h->cfg.head_dim);
    cudaError_t e = launch_pool(h->cfg.dtype, pa, st);
    if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "pool launch failed: %s", cudaGetErrorString(e));
    h->launches++;
    return AA_OK;
}

int do_aggregate(agent_attn_handle* h, const void* A, const void* K, const void* V, const void* b1,
                 int N, int n, void* VA, float* partials, unsigned* tickets, cudaStream_t st,
                 const CallLayout* cl = nullptr) {
    if (cl && cl->strided && !use_umma(h, N, n))
        return fail(h, AA_ERR_UNSUPPORTED, "strided K and V need the fused or the tensor-memory kernels (16-bit, d <= 64, n <= 256)");
    const AggPlan pl = plan_for(h, N, n);
    cudaError_t e = cudaMemsetAsync(tickets, 0, (size_t)h->cfg.batch * h->cfg.heads * sizeof(unsigned), st);
    if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "ticket reset failed: %s", cudaGetErrorString(e));
    AttnArgs a;
    memset(&a, 0, sizeof(a));
    a.qm = A; a.km = K; a.vm = V; a.bias = b1; a.out = VA;
    a.partials = partials; a.tickets = tickets;
    a.slabs = h->cfg.batch * h->cfg.heads; a.heads = h->cfg.heads;
    a.rows = n; a.cols = N; a.d = h->cfg.head_dim;
    a.scale = h->scale1; a.splits = pl.splits;
    a.status = h->d_status;
    a.lin = cl ? cl->in : dense_layout(h->cfg.heads, N, h->cfg.head_dim);
    a.lout = a.lin;
    a.strided = cl && cl->strided;
    e = use_umma(h, N, n) ? launch_aggregate_umma(h->cfg.dtype, a, pl, st)
        : use_simt(h)     ? launch_aggregate_simt(h->cfg.dtype, a, pl, st)
                          : launch_aggregate_mma(h->cfg.dtype, a, pl, st);
    if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "aggregation launch failed: %s", cudaGetErrorString(e));
    h->launches += use_umma(h, N, n) ? 2 : 1;      // the tensor-memory path merges in a second kernel
    return AA_OK;
}

int do_broadcast(agent_attn_handle* h, const void* Q, const void* A, const void* VA, const void* V,
                 const void* b2, const void* wd, int gh, int gw, int n, void* out, cudaStream_t st,
                 const CallLayout* cl = nullptr) {
    AttnArgs a;
    memset(&a, 0, sizeof(a));
    a.qm = Q; a.km = A; a.vm = VA; a.bias = b2; a.out = out;
    a.slabs = h->cfg.batch * h->cfg.heads; a.heads = h->cfg.heads;
    a.rows = gh * gw; a.cols = n; a.d = h->cfg.head_dim;
    a.scale = h->scale2; a.splits = 1;
    a.dwc_v = wd ? V : nullptr; a.dwc_w = wd; a.H = gh; a.W = gw;
    a.status = h->d_status;
    a.lin = cl ? cl->in : dense_layout(h->cfg.heads, (long long)gh * gw, h->cfg.head_dim);
    a.lout = cl ? cl->out : a.lin;
    a.strided = cl && cl->strided;
    const bool umma = !use_simt(h) && auto_like(h) &&
                      broadcast_umma_eligible(h->cfg.dtype, n, gh * gw, h->cfg.head_dim);
    if (a.strided && !umma)
        return fail(h, AA_ERR_UNSUPPORTED, "strided Q, V and out need the fused or the tensor-memory kernels (16-bit, d <= 64, n a multiple of 8 up to 256)");
    cudaError_t e = umma          ? launch_broadcast_umma(h->cfg.dtype, a, h->sm_count, st)
                    : use_simt(h) ? launch_broadcast_simt(h->cfg.dtype, a, st)
                                  : launch_broadcast_mma(h->cfg.dtype, a, st);
    if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "broadcast launch failed: %s", cudaGetErrorString(e));
    h->launches++;
    return AA_OK;
}

// Device guard: the handle's device is current inside every call and restored on exit.
struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; prev = -1; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" {

int agent_attn_create(agent_attn_handle** out, const agent_attn_config* cfg) {
    if (!out || !cfg) return AA_ERR_INVALID_ARG;
    *out = nullptr;
    if (cfg->batch <= 0 || cfg->heads <= 0 || cfg->head_dim <= 0 || cfg->max_tokens <= 0 ||
        cfg->max_agents <= 0 || cfg->scale1 < 0.f || cfg->scale2 < 0.f)
        return AA_ERR_INVALID_ARG;
    if (cfg->dtype != AA_F32 && cfg->dtype != AA_BF16 && cfg->dtype != AA_F16) return AA_ERR_UNSUPPORTED;
    if (cfg->path != AA_PATH_AUTO && cfg->path != AA_PATH_SIMT && cfg->path != AA_PATH_UNFUSED && cfg->path != AA_PATH_QUEUE)
        return AA_ERR_UNSUPPORTED;
    const int es = cfg->dtype == AA_F32 ? 4 : 2;
    if (cfg->head_dim > 128 || cfg->head_dim < 8 || (cfg->head_dim * es) % 16 != 0) return AA_ERR_UNSUPPORTED;
    if (cfg->max_agents > 256) return AA_ERR_UNSUPPORTED;
    if ((long long)cfg->batch * cfg->heads > 65535) return AA_ERR_UNSUPPORTED;

    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || cfg->device < 0 || cfg->device >= count) {
        cudaGetLastError();
        return AA_ERR_CUDA;
    }
    DeviceGuard guard(cfg->device);
    if (!guard.ok) return AA_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, cfg->device) != cudaSuccess) return AA_ERR_CUDA;
    if (prop.major != 10) return AA_ERR_CUDA;       // the kernels are built for sm_100a only

    agent_attn_handle* h = new (std::nothrow) agent_attn_handle;
    if (!h) return AA_ERR_INVALID_ARG;
    memset(h, 0, sizeof(*h));
    h->cfg = *cfg;
    h->elem_bytes = es;
    h->sm_count = prop.multiProcessorCount;
    const float def = 1.0f / std::sqrt((float)cfg->head_dim);
    h->scale1 = cfg->scale1 > 0.f ? cfg->scale1 : def;
    h->scale2 = cfg->scale2 > 0.f ? cfg->scale2 : def;
    h->poll_limit = 0xffffffffu;
    h->stage_mask = 7u;
    if (cudaMalloc(&h->d_status, sizeof(int)) != cudaSuccess || cudaMemset(h->d_status, 0, sizeof(int)) != cudaSuccess) {
        delete h;
        return AA_ERR_CUDA;
    }
    *out = h;
    return AA_OK;
}

int agent_attn_destroy(agent_attn_handle* h) {
    if (!h) return AA_OK;
    {
        DeviceGuard guard(h->cfg.device);
        if (h->d_status) cudaFree(h->d_status);
    }
    delete h;
    return AA_OK;
}

const char* agent_attn_last_error(const agent_attn_handle* h) { return h ? h->err : kNullHandleMsg; }

int agent_attn_last_launch_count(const agent_attn_handle* h) { return h ? h->launches : 0; }

int agent_attn_test_set_stage_mask(agent_attn_handle* h, unsigned mask) {
    if (!h || (mask & 7u) == 0u) return AA_ERR_INVALID_ARG;
    h->stage_mask = mask & 7u;
    return AA_OK;
}

int agent_attn_test_set_poll_limit(agent_attn_handle* h, unsigned polls) {
    if (!h) return AA_ERR_INVALID_ARG;
    h->poll_limit = polls;
    return AA_OK;
}

size_t agent_attn_workspace_bytes(const agent_attn_handle* h, int grid_h, int grid_w, int n_agents) {
    if (!h || grid_h <= 0 || grid_w <= 0 || n_agents <= 0) return 0;
    if ((long long)grid_h * grid_w > h->cfg.max_tokens || n_agents > h->cfg.max_agents) return 0;
    return ws_layout(h, grid_h * grid_w, n_agents, grid_h, grid_w).total;
}

int agent_attn_pool(agent_attn_handle* h, const void* Q, int grid_h, int grid_w, int pool_h, int pool_w,
                    void* A_out, void* stream) {
    if (!h) return AA_ERR_INVALID_ARG;
    h->err[0] = 0;
    if (!Q || !A_out) return fail(h, AA_ERR_INVALID_ARG, "null pointer");
    if (grid_h <= 0 || grid_w <= 0 || pool_h <= 0 || pool_w <= 0 || pool_h > grid_h || pool_w > grid_w)
        return fail(h, AA_ERR_INVALID_ARG, "pool grid %dx%d does not fit token grid %dx%d", pool_h, pool_w, grid_h, grid_w);
    if (int rc = check_shape(h, grid_h * grid_w, pool_h * pool_w)) return rc;
    if (misaligned(Q) || misaligned(A_out)) return fail(h, AA_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return fail(h, AA_ERR_CUDA, "cannot select device %d", h->cfg.device);
    h->launches = 0;
    return do_pool(h, Q, grid_h, grid_w, pool_h, pool_w, A_out, (cudaStream_t)stream);
}

int agent_attn_aggregate(agent_attn_handle* h, const void* A, const void* K, const void* V, const void* b1,
                         int n_tokens, int n_agents, void* VA_out, void* workspace, size_t workspace_bytes,
                         void* stream) {
    if (!h) return AA_ERR_INVALID_ARG;
    h->err[0] = 0;
    if (!A || !K || !V || !VA_out || !workspace) return fail(h, AA_ERR_INVALID_ARG, "null pointer");
    if (int rc = check_shape(h, n_tokens, n_agents)) return rc;
    if (misaligned(A) || misaligned(K) || misaligned(V) || misaligned(VA_out) || misaligned(workspace) ||
        (b1 && misaligned(b1)))
        return fail(h, AA_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    const WsLayout w = ws_layout(h, n_tokens, n_agents);
    if (workspace_bytes < w.total)
        return fail(h, AA_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, w.total);
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return fail(h, AA_ERR_CUDA, "cannot select device %d", h->cfg.device);
    h->launches = 0;
    char* ws = static_cast<char*>(workspace);
    return do_aggregate(h, A, K, V, b1, n_tokens, n_agents, VA_out, reinterpret_cast<float*>(ws + w.part_off),
                        reinterpret_cast<unsigned*>(ws + w.ticket_off), (cudaStream_t)stream);
}

int agent_attn_broadcast(agent_attn_handle* h, const void* Q, const void* A, const void* VA, const void* V,
                         const void* b2, const void* dwc_weight, int grid_h, int grid_w, int n_agents,
                         void* out, void* stream) {
    if (!h) return AA_ERR_INVALID_ARG;
    h->err[0] = 0;
    if (!Q || !A || !VA || !out || (dwc_weight && !V)) return fail(h, AA_ERR_INVALID_ARG, "null pointer");
    if (grid_h <= 0 || grid_w <= 0) return fail(h, AA_ERR_INVALID_ARG, "grid must be positive");
    if (int rc = check_shape(h, grid_h * grid_w, n_agents)) return rc;
    if (misaligned(Q) || misaligned(A) || misaligned(VA) || misaligned(out) || (V && misaligned(V)) ||
        (b2 && misaligned(b2)) || (dwc_weight && misaligned(dwc_weight)))
        return fail(h, AA_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    if (out == Q || out == V || out == A || out == VA) return fail(h, AA_ERR_INVALID_ARG, "out must not alias an input");
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return fail(h, AA_ERR_CUDA, "cannot select device %d", h->cfg.device);
    h->launches = 0;
    return do_broadcast(h, Q, A, VA, V, b2, dwc_weight, grid_h, grid_w, n_agents, out, (cudaStream_t)stream);
}

static int forward_impl(agent_attn_handle* h, const void* Q, const void* K, const void* V, const void* A,
                        int grid_h, int grid_w, int n_agents, const agent_attn_bias* bias, const void* dwc_weight,
                        void* out, void* workspace, size_t workspace_bytes, void* stream, const CallLayout* clp) {
    if (!h) return AA_ERR_INVALID_ARG;
    h->err[0] = 0;
    if (!Q || !K || !V || !out || !workspace) return fail(h, AA_ERR_INVALID_ARG, "null pointer");
    if (grid_h <= 0 || grid_w <= 0) return fail(h, AA_ERR_INVALID_ARG, "grid must be positive");
    if ((long long)grid_h * grid_w > 0x7fffffffLL) return fail(h, AA_ERR_INVALID_ARG, "grid too large");
    const int N = grid_h * grid_w;
    if (int rc = check_shape(h, N, n_agents)) return rc;
    int p = 0;
    if (!A) {
        p = isqrt_exact(n_agents);
        if (p < 0 || p > grid_h || p > grid_w)
            return fail(h, AA_ERR_INVALID_ARG,
                        "pooled agents need n = p*p with p <= min(grid_h, grid_w); got n=%d on %dx%d",
                        n_agents, grid_h, grid_w);
    }
    const void* b1 = bias ? bias->b1 : nullptr;
    const void* b2 = bias ? bias->b2 : nullptr;
    if (misaligned(Q) || misaligned(K) || misaligned(V) || misaligned(out) || misaligned(workspace) ||
        (A && misaligned(A)) || (b1 && misaligned(b1)) || (b2 && misaligned(b2)) ||
        (dwc_weight && misaligned(dwc_weight)))
        return fail(h, AA_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    if (out == Q || out == K || out == V) return fail(h, AA_ERR_INVALID_ARG, "out must not alias an input");
    const WsLayout w = ws_layout(h, N, n_agents, grid_h, grid_w);
    if (workspace_bytes < w.total)
        return fail(h, AA_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, w.total);
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return fail(h, AA_ERR_CUDA, "cannot select device %d", h->cfg.device);
    h->launches = 0;
    cudaStream_t st = (cudaStream_t)stream;
    char* ws = static_cast<char*>(workspace);
    const CallLayout cl = clp ? *clp : dense_call(h, N);
    if (h->cfg.path == AA_PATH_AUTO && h->cfg.dtype != AA_F32 && !cl.strided) {
        // long token grids with few agents: three streaming kernels, phase by phase over the batch
        const StreamPlan& sp = stream_plan_for(h, grid_h, grid_w, n_agents, A == nullptr);
        if (sp.ok) {
            const int slabs = h->cfg.batch * h->cfg.heads;
            StreamArgs sa;
            memset(&sa, 0, sizeof(sa));
            sa.q = Q; sa.k = K; sa.v = V; sa.a_user = A; sa.b1 = b1; sa.b2 = b2; sa.dwc_w = dwc_weight; sa.out = out;
            sa.a_ws = ws + w.a_off; sa.va_ws = ws + w.va_off;
            const size_t av = align_up((size_t)slabs * n_agents * 64 * 2, 256);
            sa.a1s = ws + w.extra_off; sa.a2s = ws + w.extra_off + av;
            sa.b1c = ws + w.extra_off + 2 * av;
            sa.b2p = ws + w.extra_off + 2 * av + align_up((size_t)h->cfg.heads * N * 64 * 2, 256);
            sa.wt = ws + w.extra_off + 2 * av + 2 * align_up((size_t)h->cfg.heads * N * 64 * 2, 256);
            sa.partials = reinterpret_cast<float*>(ws + w.part_off);
            sa.tickets = reinterpret_cast<unsigned*>(ws + w.ticket_off);
            sa.status = h->d_status;
            sa.slabs = slabs; sa.heads = h->cfg.heads; sa.H = grid_h; sa.W = grid_w; sa.n = n_agents; sa.p = p;
            sa.scale1 = h->scale1; sa.scale2 = h->scale2; sa.sm_count = h->sm_count; sa.plan = sp;
            // the tensor maps depend on the pointers and the shape only: reuse them while both repeat
            const size_t key_bytes = offsetof(StreamArgs, tm_k);
            if (h->stream_args_valid && memcmp(&sa, &h->stream_args, key_bytes) == 0) {
                sa = h->stream_args;
            } else {
                if (!stream_make_maps(&sa)) return fail(h, AA_ERR_CUDA, "tensor map encoding failed");
                h->stream_args = sa;
                h->stream_args_valid = true;
            }
            cudaError_t e = cudaSuccess;
            h->launches = 0;
            if (e == cudaSuccess && (h->stage_mask & 1u)) { e = launch_stream_prep(h->cfg.dtype, sa, st); h->launches++; }
            if (e == cudaSuccess && (h->stage_mask & 2u)) { e = launch_stream_aggregate(h->cfg.dtype, sa, st); h->launches++; }
            if (e == cudaSuccess && (h->stage_mask & 4u)) { e = launch_stream_broadcast(h->cfg.dtype, sa, st); h->launches++; }
            if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "streaming launch failed: %s", cudaGetErrorString(e));
            return AA_OK;
        }
    }
    if (!A && auto_like(h) && h->cfg.dtype != AA_F32) {
        // one persistent kernel for the whole module where the shape allows it
        if (h->fused_key[0] != grid_h || h->fused_key[1] != grid_w || h->fused_key[2] != n_agents) {
            h->fused_plan = plan_fused(h->cfg.dtype, h->cfg.batch * h->cfg.heads, grid_h, grid_w, h->cfg.head_dim,
                                       n_agents, h->sm_count);
            h->fused_key[0] = grid_h; h->fused_key[1] = grid_w; h->fused_key[2] = n_agents;
        }
        if (h->fused_plan.ok) {
            const int slabs = h->cfg.batch * h->cfg.heads;
            unsigned* counters = reinterpret_cast<unsigned*>(ws + w.ticket_off);
            cudaError_t e = cudaMemsetAsync(counters, 0, fused_counter_words(slabs) * sizeof(unsigned), st);
            if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "counter reset failed: %s", cudaGetErrorString(e));
            FusedArgs fa;
            memset(&fa, 0, sizeof(fa));
            fa.q = Q; fa.k = K; fa.v = V; fa.b1 = b1; fa.b2 = b2; fa.dwc_w = dwc_weight; fa.out = out;
            fa.a_ws = ws + w.a_off; fa.va_ws = ws + w.va_off;
            fa.partials = reinterpret_cast<float*>(ws + w.part_off);
            fa.counters = counters; fa.status = h->d_status;
            fa.poll_limit = h->poll_limit == 0xffffffffu ? (1u << 20) : h->poll_limit;
            fa.slabs = slabs; fa.heads = h->cfg.heads; fa.H = grid_h; fa.W = grid_w; fa.d = h->cfg.head_dim;
            fa.n = n_agents; fa.p = p; fa.scale1 = h->scale1; fa.scale2 = h->scale2; fa.plan = h->fused_plan;
            fa.lin = cl.in; fa.lout = cl.out;
            if (!fused_make_maps(&fa)) return fail(h, AA_ERR_CUDA, "tensor map encoding failed");
            e = launch_fused(h->cfg.dtype, fa, st);
            if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "fused launch failed: %s", cudaGetErrorString(e));
            h->launches = 1;
            return AA_OK;
        }
    }
    // strided tensors are read in place only by the task-queue and the tensor-memory kernels: decide before anything
    // is launched
    if (cl.strided && !(use_umma(h, N, n_agents) && !use_simt(h) && auto_like(h) &&
                        broadcast_umma_eligible(h->cfg.dtype, n_agents, N, h->cfg.head_dim)))
        return fail(h, AA_ERR_UNSUPPORTED,
                    "strided tensors need the task-queue kernel (16-bit, d = 64, n <= 64, pooled agents, W <= 64) or the "
                    "tensor-memory kernels (16-bit, d <= 64, n a multiple of 8 in 72..256)");
    const void* agents = A;
    if (!A) {
        if (int rc = do_pool(h, Q, grid_h, grid_w, p, p, ws + w.a_off, st, &cl)) return rc;
        agents = ws + w.a_off;
    }
    void* va = ws + w.va_off;
    if (int rc = do_aggregate(h, agents, K, V, b1, N, n_agents, va, reinterpret_cast<float*>(ws + w.part_off),
                              reinterpret_cast<unsigned*>(ws + w.ticket_off), st, &cl))
        return rc;
    return do_broadcast(h, Q, agents, va, V, b2, dwc_weight, grid_h, grid_w, n_agents, out, st, &cl);
}

int agent_attn_forward(agent_attn_handle* h, const void* Q, const void* K, const void* V, const void* A,
                       int grid_h, int grid_w, int n_agents, const agent_attn_bias* bias, const void* dwc_weight,
                       void* out, void* workspace, size_t workspace_bytes, void* stream) {
    return forward_impl(h, Q, K, V, A, grid_h, grid_w, n_agents, bias, dwc_weight, out, workspace, workspace_bytes,
                        stream, nullptr);
}

int agent_attn_forward_strided(agent_attn_handle* h, const void* Q, const void* K, const void* V, const void* A,
                               const long long in_strides[3], int grid_h, int grid_w, int n_agents,
                               const agent_attn_bias* bias, const void* dwc_weight, void* out,
                               const long long out_strides[3], void* workspace, size_t workspace_bytes, void* stream) {
    if (!h) return AA_ERR_INVALID_ARG;
    h->err[0] = 0;
    if (!in_strides || !out_strides) return fail(h, AA_ERR_INVALID_ARG, "null stride array");
    if (grid_h <= 0 || grid_w <= 0) return fail(h, AA_ERR_INVALID_ARG, "grid must be positive");
    const long long N = (long long)grid_h * grid_w, d = h->cfg.head_dim;
    CallLayout cl;
    cl.in.sb = in_strides[0]; cl.in.sh = in_strides[1]; cl.in.st = in_strides[2];
    cl.out.sb = out_strides[0]; cl.out.sh = out_strides[1]; cl.out.st = out_strides[2];
    for (const TokLayout* l : {&cl.in, &cl.out}) {
        if (l->sb <= 0 || l->sh <= 0 || l->st < d)
            return fail(h, AA_ERR_INVALID_ARG, "strides must be positive and the token stride at least head_dim");
        if ((l->sb * h->elem_bytes) % 16 || (l->sh * h->elem_bytes) % 16 || (l->st * h->elem_bytes) % 16)
            return fail(h, AA_ERR_INVALID_ARG, "strides must be multiples of 16 bytes");
    }
    const TokLayout dl = dense_layout(h->cfg.heads, N, (int)d);
    auto same = [](const TokLayout& a, const TokLayout& b) { return a.sb == b.sb && a.sh == b.sh && a.st == b.st; };
    cl.strided = !(same(cl.in, dl) && same(cl.out, dl));
    return forward_impl(h, Q, K, V, A, grid_h, grid_w, n_agents, bias, dwc_weight, out, workspace, workspace_bytes,
                        stream, &cl);
}

int agent_attn_compose_bias(agent_attn_handle* h, const void* col, const void* row, const void* blk, int block_h,
                            int block_w, int grid_h, int grid_w, int n_agents, int transpose, void* out,
                            void* stream) {
    if (!h) return AA_ERR_INVALID_ARG;
    h->err[0] = 0;
    if (!out || (!col && !row && !blk)) return fail(h, AA_ERR_INVALID_ARG, "null pointer");
    if (grid_h <= 0 || grid_w <= 0) return fail(h, AA_ERR_INVALID_ARG, "grid must be positive");
    if (blk && (block_h <= 0 || block_w <= 0)) return fail(h, AA_ERR_INVALID_ARG, "block bias needs a positive size");
    if (int rc = check_shape(h, grid_h * grid_w, n_agents)) return rc;
    if (misaligned(out) || (col && misaligned(col)) || (row && misaligned(row)) || (blk && misaligned(blk)))
        return fail(h, AA_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return fail(h, AA_ERR_CUDA, "cannot select device %d", h->cfg.device);
    ComposeArgs a;
    a.col = col; a.row = row; a.blk = blk; a.out = out;
    a.heads = h->cfg.heads; a.n = n_agents; a.h = grid_h; a.w = grid_w;
    a.h0 = blk ? block_h : 1; a.w0 = blk ? block_w : 1; a.transpose = transpose ? 1 : 0;
    cudaError_t e = launch_compose_bias(h->cfg.dtype, a, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "bias composition launch failed: %s", cudaGetErrorString(e));
    h->launches = 1;
    return AA_OK;
}

size_t agent_attn_staging_bytes(const agent_attn_handle* h, int grid_h, int grid_w, int n_agents) {
    const size_t ws = agent_attn_workspace_bytes(h, grid_h, grid_w, n_agents);
    if (!ws) return 0;
    const size_t es = h->elem_bytes, slabs = (size_t)h->cfg.batch * h->cfg.heads;
    const size_t N = (size_t)grid_h * grid_w, d = h->cfg.head_dim, n = n_agents, heads = h->cfg.heads;
    const size_t qkv = align_up(slabs * N * d * es, 256);
    return 4 * qkv + align_up(slabs * n * d * es, 256) + 2 * align_up(heads * n * N * es, 256) +
           align_up(heads * d * 9 * es, 256) + align_up(ws, 256);
}

int agent_attn_forward_host(agent_attn_handle* h, const void* Q, const void* K, const void* V, const void* A,
                            int grid_h, int grid_w, int n_agents, const agent_attn_bias* bias,
                            const void* dwc_weight, void* out, void* staging, size_t staging_bytes, void* stream) {
    if (!h) return AA_ERR_INVALID_ARG;
    h->err[0] = 0;
    if (!Q || !K || !V || !out || !staging) return fail(h, AA_ERR_INVALID_ARG, "null pointer");
    const size_t need = agent_attn_staging_bytes(h, grid_h, grid_w, n_agents);
    if (!need) return fail(h, AA_ERR_INVALID_ARG, "bad grid or agent count for this handle");
    if (staging_bytes < need) return fail(h, AA_ERR_WORKSPACE, "staging has %zu bytes, %zu needed", staging_bytes, need);
    if (misaligned(staging)) return fail(h, AA_ERR_INVALID_ARG, "staging must be 16-byte aligned");
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return fail(h, AA_ERR_CUDA, "cannot select device %d", h->cfg.device);
    cudaStream_t st = (cudaStream_t)stream;
    const size_t es = h->elem_bytes, slabs = (size_t)h->cfg.batch * h->cfg.heads;
    const size_t N = (size_t)grid_h * grid_w, d = h->cfg.head_dim, n = n_agents, heads = h->cfg.heads;
    const size_t qkv_b = slabs * N * d * es, a_b = slabs * n * d * es, bias_b = heads * n * N * es, w_b = heads * d * 9 * es;
    char* s = static_cast<char*>(staging);
    char* dQ = s;                       s += align_up(qkv_b, 256);
    char* dK = s;                       s += align_up(qkv_b, 256);
    char* dV = s;                       s += align_up(qkv_b, 256);
    char* dO = s;                       s += align_up(qkv_b, 256);
    char* dA = s;                       s += align_up(a_b, 256);
    char* dB1 = s;                      s += align_up(bias_b, 256);
    char* dB2 = s;                      s += align_up(bias_b, 256);
    char* dW = s;                       s += align_up(w_b, 256);
    char* dWs = s;
    const size_t ws_bytes = agent_attn_workspace_bytes(h, grid_h, grid_w, n_agents);
    struct Cp { void* dst; const void* src; size_t bytes; } cps[] = {
        {dQ, Q, qkv_b}, {dK, K, qkv_b}, {dV, V, qkv_b}, {dA, A, a_b},
        {dB1, bias ? bias->b1 : nullptr, bias_b}, {dB2, bias ? bias->b2 : nullptr, bias_b}, {dW, dwc_weight, w_b}};
    for (const Cp& c : cps) {
        if (!c.src) continue;
        cudaError_t e = cudaMemcpyAsync(c.dst, c.src, c.bytes, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "host-to-device copy failed: %s", cudaGetErrorString(e));
    }
    agent_attn_bias db;
    db.b1 = (bias && bias->b1) ? dB1 : nullptr;
    db.b2 = (bias && bias->b2) ? dB2 : nullptr;
    int rc = agent_attn_forward(h, dQ, dK, dV, A ? dA : nullptr, grid_h, grid_w, n_agents, bias ? &db : nullptr,
                                dwc_weight ? dW : nullptr, dO, dWs, ws_bytes, stream);
    if (rc) return rc;
    cudaError_t e = cudaMemcpyAsync(out, dO, qkv_b, cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "device-to-host copy failed: %s", cudaGetErrorString(e));
    return AA_OK;
}

int agent_attn_query_status(agent_attn_handle* h, void* stream) {
    if (!h) return AA_ERR_INVALID_ARG;
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return fail(h, AA_ERR_CUDA, "cannot select device %d", h->cfg.device);
    cudaStream_t st = (cudaStream_t)stream;
    int word = 0;
    cudaError_t e = cudaStreamSynchronize(st);
    if (e == cudaSuccess) e = cudaMemcpy(&word, h->d_status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "status query failed: %s", cudaGetErrorString(e));
    if (word != 0) {
        cudaMemset(h->d_status, 0, sizeof(int));
        return fail(h, AA_ERR_TIMEOUT, "a device-side bounded wait expired (code %d)", word);
    }
    return AA_OK;
}

// Workspace of the backward pass: [A | V_A | dV_A | dA | lse | dot | window table | partial (max, sum)], fp32, each
// region 256-byte aligned (V_A, dV_A and dA are cleared with one memset, so their regions have one size).
namespace {
struct BwdLayout {
    size_t a, va, dva, da, lse, dot, tab, part, total;
};
bool bwd_layout(const agent_attn_handle* h, int N, int n, BwdPlan* pl, BwdLayout* w) {
    const int slabs = h->cfg.batch * h->cfg.heads;
    if (!plan_backward(slabs, n, N, h->cfg.head_dim, h->sm_count, pl)) return false;
    const size_t snd = align_up((size_t)slabs * n * h->cfg.head_dim * sizeof(float), 256);
    const size_t sn = align_up((size_t)slabs * n * sizeof(float), 256);
    w->a = 0; w->va = snd; w->dva = 2 * snd; w->da = 3 * snd;
    w->lse = 4 * snd; w->dot = w->lse + sn; w->tab = w->dot + sn;
    w->part = w->tab + align_up((size_t)N * 48, 256);
    size_t part_floats = (size_t)slabs * pl->chunks * n * 2;
    if (backward_mma_eligible(h->cfg.dtype, n, h->cfg.head_dim)) {      // partials of the tensor-core stage 1
        const size_t mma_floats = backward_mma_part_floats(slabs, plan_backward_mma(slabs, N, h->sm_count));
        if (part_floats < mma_floats) part_floats = mma_floats;
    }
    w->total = w->part + align_up(part_floats * sizeof(float), 256);
    return true;
}
}  // namespace

size_t agent_attn_backward_workspace_bytes(const agent_attn_handle* h, int grid_h, int grid_w, int n_agents) {
    if (!h || grid_h <= 0 || grid_w <= 0 || n_agents <= 0) return 0;
    if ((long long)grid_h * grid_w > h->cfg.max_tokens || n_agents > h->cfg.max_agents) return 0;
    BwdPlan pl;
    BwdLayout w;
    return bwd_layout(h, grid_h * grid_w, n_agents, &pl, &w) ? w.total : 0;
}

int agent_attn_backward(agent_attn_handle* h, const void* Q, const void* K, const void* V, const void* d_out,
                        int grid_h, int grid_w, int n_agents, const agent_attn_bias* bias, const void* dwc_weight,
                        const agent_attn_grads* grads, void* workspace, size_t workspace_bytes, void* stream) {
    if (!h) return AA_ERR_INVALID_ARG;
    h->err[0] = 0;
    if (!Q || !K || !V || !d_out || !grads || !workspace) return fail(h, AA_ERR_INVALID_ARG, "null pointer");
    if (!grads->dq || !grads->dk || !grads->dv) return fail(h, AA_ERR_INVALID_ARG, "dq, dk and dv are required");
    if (grads->dwd && !dwc_weight) return fail(h, AA_ERR_INVALID_ARG, "dwd requested without a depthwise filter");
    if (grid_h <= 0 || grid_w <= 0) return fail(h, AA_ERR_INVALID_ARG, "grid must be positive");
    if ((long long)grid_h * grid_w > 0x7fffffffLL) return fail(h, AA_ERR_INVALID_ARG, "grid too large");
    const int N = grid_h * grid_w;
    if (int rc = check_shape(h, N, n_agents)) return rc;
    const int p = isqrt_exact(n_agents);
    if (p < 0 || p > grid_h || p > grid_w)
        return fail(h, AA_ERR_INVALID_ARG, "pooled agents need n = p*p with p <= min(grid_h, grid_w); got n=%d on %dx%d",
                    n_agents, grid_h, grid_w);
    const void* b1 = bias ? bias->b1 : nullptr;
    const void* b2 = bias ? bias->b2 : nullptr;
    const void* ptrs[] = {Q, K, V, d_out, workspace, grads->dq, grads->dk, grads->dv, grads->db1, grads->db2,
                          grads->dwd, b1, b2, dwc_weight};
    for (const void* q : ptrs)
        if (q && misaligned(q)) return fail(h, AA_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    const void* outs[] = {grads->dq, grads->dk, grads->dv, grads->db1, grads->db2, grads->dwd};
    const void* ins[] = {Q, K, V, d_out, b1, b2, dwc_weight};
    for (size_t i = 0; i < 6; ++i) {
        if (!outs[i]) continue;
        for (const void* q : ins)
            if (outs[i] == q) return fail(h, AA_ERR_INVALID_ARG, "a gradient buffer aliases an input");
        for (size_t j = 0; j < i; ++j)
            if (outs[i] == outs[j]) return fail(h, AA_ERR_INVALID_ARG, "two gradient buffers alias");
    }
    BwdCall c;
    memset(&c, 0, sizeof(c));
    BwdLayout w;
    if (!bwd_layout(h, N, n_agents, &c.plan, &w))
        return fail(h, AA_ERR_UNSUPPORTED, "backward needs n * head_dim <= 16384 (n=%d, d=%d)", n_agents, h->cfg.head_dim);
    if (workspace_bytes < w.total)
        return fail(h, AA_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, w.total);
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return fail(h, AA_ERR_CUDA, "cannot select device %d", h->cfg.device);
    h->launches = 0;
    char* ws = static_cast<char*>(workspace);
    c.q = Q; c.k = K; c.v = V; c.d_out = d_out; c.b1 = b1; c.b2 = b2; c.wd = dwc_weight;
    c.dq = static_cast<float*>(grads->dq); c.dk = static_cast<float*>(grads->dk); c.dv = static_cast<float*>(grads->dv);
    c.db1 = static_cast<float*>(grads->db1); c.db2 = static_cast<float*>(grads->db2);
    c.dwd = static_cast<float*>(grads->dwd);
    c.ws_a = reinterpret_cast<float*>(ws + w.a); c.ws_va = reinterpret_cast<float*>(ws + w.va);
    c.ws_dva = reinterpret_cast<float*>(ws + w.dva); c.ws_da = reinterpret_cast<float*>(ws + w.da);
    c.ws_lse = reinterpret_cast<float*>(ws + w.lse); c.ws_dot = reinterpret_cast<float*>(ws + w.dot);
    c.ws_part = reinterpret_cast<float*>(ws + w.part);
    c.ws_tab = reinterpret_cast<int4*>(ws + w.tab);
    c.clear_bytes = w.lse - w.va;
    c.slabs = h->cfg.batch * h->cfg.heads; c.heads = h->cfg.heads; c.H = grid_h; c.W = grid_w;
    c.d = h->cfg.head_dim; c.n = n_agents; c.p = p; c.sm_count = h->sm_count;
    c.scale1 = h->scale1; c.scale2 = h->scale2;
    c.dtype = h->cfg.dtype;
    c.use_mma = auto_like(h) && backward_mma_eligible(h->cfg.dtype, n_agents, h->cfg.head_dim);
    if (c.use_mma) c.plan_mma = plan_backward_mma(c.slabs, N, h->sm_count);
    cudaError_t e = launch_backward(h->cfg.dtype, c, (cudaStream_t)stream);
    if (e != cudaSuccess) return fail(h, AA_ERR_CUDA, "backward launch failed: %s", cudaGetErrorString(e));
    h->launches = backward_launch_count(c.use_mma != 0);
    return AA_OK;
}

}  // extern "C"

// --------------------------------------------------------------------------------------------
// Aggregation for callers that cannot allocate device memory.
//
// The split partials and arrival counters of the aggregation live in this fixed array, which is
// part of the library image: every GPU that loads the library holds it until the process exits.
// In host code `g_static_scratch` is only a stand-in symbol, not a device address; the address a
// kernel may use is obtained once per device with cudaGetSymbolAddress (device current) below.
#define AA_STATIC_SCRATCH_BYTES (32u * 1024u * 1024u)
static __device__ __align__(256) unsigned char g_static_scratch[AA_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
void* g_static_ptr[kMaxDevices] = {nullptr};

// Device address of the static scratch on the current device (looked up on first use).
cudaError_t static_scratch_address(int device, void** out) {
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    if (!g_static_ptr[device]) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_static_ptr[device] = ptr;
    }
    *out = g_static_ptr[device];
    return cudaSuccess;
}
}  // namespace

extern "C" size_t agent_attn_static_scratch_bytes(void) { return AA_STATIC_SCRATCH_BYTES; }

extern "C" int agent_attn_aggregate_static(agent_attn_handle* h, const void* A, const void* K, const void* V,
                                           const void* b1, int n_tokens, int n_agents, void* VA_out,
                                           void* stream) {
    if (!h) return AA_ERR_INVALID_ARG;
    h->err[0] = 0;
    if (!A || !K || !V || !VA_out) return fail(h, AA_ERR_INVALID_ARG, "null pointer");
    if (int rc = check_shape(h, n_tokens, n_agents)) return rc;
    if (misaligned(A) || misaligned(K) || misaligned(V) || misaligned(VA_out) || (b1 && misaligned(b1)))
        return fail(h, AA_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    // scratch layout: [partials | arrival counters], each 256-byte aligned
    const size_t slabs = (size_t)h->cfg.batch * h->cfg.heads;
    const AggPlan pl = plan_for(h, n_tokens, n_agents);
    const size_t part_bytes = align_up(slabs * pl.parts * partial_floats(pl.rows_pad, pl.dpad) * sizeof(float), 256);
    const size_t need = part_bytes + align_up(slabs * sizeof(unsigned), 256);
    if (need > AA_STATIC_SCRATCH_BYTES)
        return fail(h, AA_ERR_WORKSPACE,
                    "this shape needs %zu bytes of scratch but the built-in scratch holds %u bytes; "
                    "use agent_attn_aggregate with a caller-provided workspace",
                    need, (unsigned)AA_STATIC_SCRATCH_BYTES);
    DeviceGuard guard(h->cfg.device);
    if (!guard.ok) return fail(h, AA_ERR_CUDA, "cannot select device %d", h->cfg.device);
    void* base = nullptr;
    cudaError_t e = static_scratch_address(h->cfg.device, &base);
    if (e != cudaSuccess)
        return fail(h, AA_ERR_CUDA, "cannot resolve the built-in scratch on device %d: %s", h->cfg.device,
                    cudaGetErrorString(e));
    h->launches = 0;
    char* s = static_cast<char*>(base);
    // do_aggregate clears the arrival counters on the stream before the kernel; the partials are
    // fully rewritten by every call, so nothing else of the previous call's contents is read.
    return do_aggregate(h, A, K, V, b1, n_tokens, n_agents, VA_out, reinterpret_cast<float*>(s),
                        reinterpret_cast<unsigned*>(s + part_bytes), (cudaStream_t)stream);
}
