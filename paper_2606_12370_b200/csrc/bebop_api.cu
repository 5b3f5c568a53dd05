// extern "C" entry points: host-side validation, workspace planning, dispatch.
// No allocation, no synchronisation; everything is enqueued on the caller's stream.
#include "../../include/bebop.h"
#include "bebop_kernels.h"

using namespace bebop;

namespace {

// Test hook: route bebop_verify through the general (split-row) path even where the fused
// kernel applies, so that both paths are covered by the parity tests.
int g_last_kernel = 0;   // what the last call ran: 1 general kernels, 2 pipelined kernel, 3 fused kernel
int g_path = 0;   // 0: the faster of the fused and the pipelined kernel where they apply, else the general kernels;
                  // 1: general kernels only; 2: never the fused kernel; 3: the fused kernel wherever it applies

int g_expire_wait = 0;   // test hook: which device-side wait the next call lets give up at once
float g_draw_kappa = -1.f;   // test hook: factor of the fast draw's error bound (negative: the built-in value)

// Built-in scratch of bebop_tv_static: one array per device the module is loaded on.  Nothing in it
// has to start at zero (every partial is written before it is read).
static __device__ __align__(256) unsigned char g_tv_scratch[BEBOP_TV_STATIC_SCRATCH_BYTES];
constexpr int kMaxDevices = 64;
// device address of g_tv_scratch, looked up once per device.  A plain host cache: two threads that make a device's
// first call at the same time both look the address up and store the same value.
void* g_tv_scratch_ptr[kMaxDevices] = {nullptr};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Compute capability of the current device, cached per device ordinal.
bebop_status_t check_arch() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return BEBOP_ERR_CUDA;
    if (dev >= 0 && dev < 64 && cached[dev]) return cached[dev] == 10 ? BEBOP_OK : BEBOP_ERR_ARCH;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return BEBOP_ERR_CUDA;
    if (dev >= 0 && dev < 64) cached[dev] = major;
    return major == 10 ? BEBOP_OK : BEBOP_ERR_ARCH;
}

bebop_status_t check_shape(int B, int K, int V, bebop_dtype_t dt) {
    if (dt != BEBOP_F32 && dt != BEBOP_BF16) return BEBOP_ERR_DTYPE;
    if (B <= 0 || K <= 0 || V <= 0 || K > BEBOP_MAX_K) return BEBOP_ERR_SHAPE;
    if ((int64_t)V > (int64_t)1 << 30) return BEBOP_ERR_SHAPE;
    return BEBOP_OK;
}

bebop_status_t check_rows(const void* base, int64_t ld, int V, bebop_dtype_t dt) {
    if (!base) return BEBOP_ERR_NULL;
    if (ld < V) return BEBOP_ERR_SHAPE;
    const int64_t es = dt == BEBOP_F32 ? 4 : 2;
    if (!aligned16(base) || (ld * es) % 16 != 0) return BEBOP_ERR_ALIGN;
    return BEBOP_OK;
}

RowArgs row_args(const void* target, int64_t ld_t, const void* draft, int64_t ld_d,
                 int64_t t_seq_rows, int64_t d_seq_rows, const int32_t* draft_len,
                 const float* temperature, float temperature_all, int B, int K, int V,
                 bebop_dtype_t dt, const Plan& p) {
    RowArgs a;
    const int64_t es = dt == BEBOP_F32 ? 4 : 2;
    a.target = static_cast<const char*>(target);
    a.draft = static_cast<const char*>(draft);
    a.t_row_bytes = ld_t * es;
    a.d_row_bytes = ld_d * es;
    a.t_seq_rows = t_seq_rows;
    a.d_seq_rows = d_seq_rows;
    a.draft_len = draft_len;
    a.temperature = temperature;
    a.temperature_all = temperature_all;
    a.B = B; a.K = K; a.V = V; a.dt = (int)dt; a.nvec = p.nvec; a.nsplit = p.nsplit;
    return a;
}

}  // namespace

namespace bebop {
int take_expire_wait() { const int w = g_expire_wait; g_expire_wait = 0; return w; }
float draw_kappa() { return g_draw_kappa >= 0.f ? g_draw_kappa : 4.0f; }
}  // namespace bebop

extern "C" {

size_t bebop_workspace_bytes(int B, int K, int V, bebop_dtype_t dt) {
    if (check_shape(B, K, V, dt) != BEBOP_OK) return 0;
    return make_plan(B, K, V, (int)dt).total;
}

bebop_status_t bebop_verify(const void* target_logits, int64_t ld_target, const void* draft_logits,
                            int64_t ld_draft, const int32_t* draft_tokens, const int32_t* draft_len,
                            const float* temperature, float temperature_all, const float* u_accept,
                            const float* u_final, int B, int K, int V, bebop_dtype_t dt,
                            int32_t* accept_len, int32_t* out_tokens, float* tv, float* p_draft,
                            float* q_draft, int32_t* row_status, void* workspace,
                            size_t workspace_bytes, void* cuda_stream) {
    bebop_status_t s = check_shape(B, K, V, dt);
    if (s != BEBOP_OK) return s;
    if (!draft_tokens || !u_accept || !u_final || !accept_len || !out_tokens || !workspace)
        return BEBOP_ERR_NULL;
    if ((s = check_rows(target_logits, ld_target, V, dt)) != BEBOP_OK) return s;
    if ((s = check_rows(draft_logits, ld_draft, V, dt)) != BEBOP_OK) return s;
    if (!temperature && !(temperature_all > 0.f && temperature_all < INFINITY)) return BEBOP_ERR_TEMPERATURE;
    const Plan p = make_plan(B, K, V, (int)dt);
    if (workspace_bytes < p.total) return BEBOP_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return BEBOP_ERR_ALIGN;
    if ((s = check_arch()) != BEBOP_OK) return s;
    RowArgs a = row_args(target_logits, ld_target, draft_logits, ld_draft, K + 1, K, draft_len,
                         temperature, temperature_all, B, K, V, dt, p);
    VerifyOut o{accept_len, out_tokens, tv, p_draft, q_draft, row_status};
    char* ws = static_cast<char*>(workspace);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaSuccess;
    bool launched = false;
    g_last_kernel = 1;
    if ((g_path == 3 || (g_path == 0 && fuse_preferred(a, false))) && fuse_supported(a)) {
        e = fuse_verify(a, p, draft_tokens, u_accept, u_final, o, ws, stream, &launched);
        if (launched) g_last_kernel = 3;
    }
    if (e == cudaSuccess && !launched && g_path != 1 && pipe_supported(a)) {
        e = pipe_verify(a, p, draft_tokens, u_accept, u_final, o, ws, stream, &launched);
        if (launched) g_last_kernel = 2;
    }
    if (e == cudaSuccess && !launched) e = general_verify(a, p, draft_tokens, u_accept, u_final, o, ws, stream);
    return e == cudaSuccess ? BEBOP_OK : BEBOP_ERR_CUDA;
}

bebop_status_t bebop_tv(const void* target_logits, int64_t ld_target, const void* draft_logits,
                        int64_t ld_draft, const float* temperature, float temperature_all, int N, int V,
                        bebop_dtype_t dt, float* tv, float* s_aux, int32_t* row_status, void* workspace,
                        size_t workspace_bytes, void* cuda_stream) {
    bebop_status_t s = check_shape(N, 1, V, dt);
    if (s != BEBOP_OK) return s;
    if (!tv || !workspace) return BEBOP_ERR_NULL;
    if ((s = check_rows(target_logits, ld_target, V, dt)) != BEBOP_OK) return s;
    if ((s = check_rows(draft_logits, ld_draft, V, dt)) != BEBOP_OK) return s;
    if (!temperature && !(temperature_all > 0.f && temperature_all < INFINITY)) return BEBOP_ERR_TEMPERATURE;
    const Plan p = make_plan(N, 1, V, (int)dt);
    if (workspace_bytes < p.total) return BEBOP_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return BEBOP_ERR_ALIGN;
    if ((s = check_arch()) != BEBOP_OK) return s;
    RowArgs a = row_args(target_logits, ld_target, draft_logits, ld_draft, 1, 1, nullptr, temperature,
                         temperature_all, N, 1, V, dt, p);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaSuccess;
    bool launched = false;
    VerifyOut o{nullptr, nullptr, tv, nullptr, nullptr, row_status};
    g_last_kernel = 1;
    if ((g_path == 3 || (g_path == 0 && fuse_preferred(a, true))) && fuse_supported(a)) {
        e = fuse_verify(a, p, nullptr, nullptr, nullptr, o, static_cast<char*>(workspace), stream, &launched, true, s_aux);
        if (launched) g_last_kernel = 3;
    }
    if (e == cudaSuccess && !launched && g_path != 1 && pipe_supported(a)) {
        // the pipelined kernel with row pairs in place of sequences: first sweep, second sweep, no draw
        e = pipe_verify(a, p, nullptr, nullptr, nullptr, o, static_cast<char*>(workspace), stream, &launched, true, s_aux);
        if (launched) g_last_kernel = 2;
    }
    if (e == cudaSuccess && !launched)
        e = general_tv(a, p, tv, s_aux, row_status, static_cast<char*>(workspace), stream);
    return e == cudaSuccess ? BEBOP_OK : BEBOP_ERR_CUDA;
}

bebop_status_t bebop_greedy_verify(const void* target_logits, int64_t ld_target,
                                   const int32_t* draft_tokens, const int32_t* draft_len, int B, int K,
                                   int V, bebop_dtype_t dt, int32_t* accept_len, int32_t* out_tokens,
                                   int32_t* row_status, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream) {
    bebop_status_t s = check_shape(B, K, V, dt);
    if (s != BEBOP_OK) return s;
    if (!draft_tokens || !accept_len || !out_tokens || !workspace) return BEBOP_ERR_NULL;
    if ((s = check_rows(target_logits, ld_target, V, dt)) != BEBOP_OK) return s;
    const Plan p = make_plan(B, K, V, (int)dt);
    if (workspace_bytes < p.total) return BEBOP_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return BEBOP_ERR_ALIGN;
    if ((s = check_arch()) != BEBOP_OK) return s;
    RowArgs a = row_args(target_logits, ld_target, nullptr, 0, K + 1, K, draft_len, nullptr, 1.f, B, K,
                         V, dt, p);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = cudaSuccess;
    bool launched = false;
    g_last_kernel = 1;
    if (g_path != 1 && pipe_supported(a)) {
        e = pipe_greedy(a, p, draft_tokens, accept_len, out_tokens, row_status, static_cast<char*>(workspace), stream, &launched);
        if (launched) g_last_kernel = 2;
    }
    if (e == cudaSuccess && !launched)
        e = general_greedy(a, p, draft_tokens, accept_len, out_tokens, row_status, static_cast<char*>(workspace), stream);
    return e == cudaSuccess ? BEBOP_OK : BEBOP_ERR_CUDA;
}

bebop_status_t bebop_tv_static(const void* target_logits, int64_t ld_target, const void* draft_logits,
                               int64_t ld_draft, const float* temperature, float temperature_all, int N,
                               int V, bebop_dtype_t dt, float* tv, float* s_aux, int32_t* row_status,
                               void* cuda_stream) {
    bebop_status_t s = check_shape(N, 1, V, dt);
    if (s != BEBOP_OK) return s;
    if (!tv) return BEBOP_ERR_NULL;
    if ((s = check_rows(target_logits, ld_target, V, dt)) != BEBOP_OK) return s;
    if ((s = check_rows(draft_logits, ld_draft, V, dt)) != BEBOP_OK) return s;
    if (!temperature && !(temperature_all > 0.f && temperature_all < INFINITY)) return BEBOP_ERR_TEMPERATURE;
    // the two partial arrays of the TV sweep, packed from the start of the built-in scratch
    Plan p = make_plan(N, 1, V, (int)dt);
    const size_t stats_bytes = align256(sizeof(float) * 2 * (size_t)N * 2 * p.nsplit);
    const size_t zpart_bytes = align256(sizeof(float) * 2 * (size_t)N * p.nsplit);
    if (stats_bytes + zpart_bytes > BEBOP_TV_STATIC_SCRATCH_BYTES) return BEBOP_ERR_STATIC_SCRATCH;
    p.off_stats = 0;
    p.off_zpart = stats_bytes;
    if ((s = check_arch()) != BEBOP_OK) return s;
    // set-up, once per device: the device address of the scratch array
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BEBOP_ERR_CUDA;
    if (!g_tv_scratch_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_tv_scratch) != cudaSuccess || !ptr) { cudaGetLastError(); return BEBOP_ERR_CUDA; }
        g_tv_scratch_ptr[dev] = ptr;
    }
    RowArgs a = row_args(target_logits, ld_target, draft_logits, ld_draft, 1, 1, nullptr, temperature,
                         temperature_all, N, 1, V, dt, p);
    cudaError_t e = general_tv(a, p, tv, s_aux, row_status, static_cast<char*>(g_tv_scratch_ptr[dev]),
                               static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? BEBOP_OK : BEBOP_ERR_CUDA;
}

void bebop_debug_force_general_path(int on) { g_path = on; }

int bebop_debug_last_kernel(void) { return g_last_kernel; }

void bebop_debug_expire_wait(int which) { g_expire_wait = which; }

void bebop_debug_set_draw_kappa(float kappa) { g_draw_kappa = kappa; }

void bebop_debug_set_timing_events(void* start, void* stop) { pipe_set_events(static_cast<cudaEvent_t>(start), static_cast<cudaEvent_t>(stop)); }

size_t bebop_debug_fallback_offset(int B, int K, int V, bebop_dtype_t dt) {
    if (check_shape(B, K, V, dt) != BEBOP_OK) return 0;
    return make_plan(B, K, V, (int)dt).off_pipe + kFbCountOffset;
}

const char* bebop_status_string(bebop_status_t status) {
    switch (status) {
        case BEBOP_OK: return "ok";
        case BEBOP_ERR_NULL: return "a required pointer is NULL";
        case BEBOP_ERR_SHAPE: return "bad shape: need B, K, V > 0, K <= 32, ld >= V";
        case BEBOP_ERR_DTYPE: return "unknown dtype";
        case BEBOP_ERR_ALIGN: return "logit rows must be 16-byte aligned, workspace 256-byte aligned";
        case BEBOP_ERR_WORKSPACE: return "workspace smaller than bebop_workspace_bytes()";
        case BEBOP_ERR_TEMPERATURE: return "temperature_all must be finite and > 0";
        case BEBOP_ERR_ARCH: return "device is not sm_100";
        case BEBOP_ERR_CUDA: return "CUDA launch error";
        case BEBOP_ERR_STATIC_SCRATCH:
            return "shape needs more than the built-in scratch of bebop_tv_static: use bebop_tv with a workspace";
    }
    return "unknown status";
}

}  // extern "C"
