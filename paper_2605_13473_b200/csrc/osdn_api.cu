// C ABI of the OSDN library: argument validation, workspace carving, launch plans.
// No device memory is allocated here and no state survives a call (apart from a
// thread-local launch counter used for benchmark accounting).
#include <cmath>
#include <cstring>
#include <mutex>
#include <vector>

#include "osdn_common.cuh"

namespace osdn {
int tc_forward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
               bool save, cudaStream_t st);
int tc_backward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                cudaStream_t st);
bool tc_supported(const osdn_params& p);
bool tc_backward_supported(const osdn_params& p);
int launch_wait_timeout_selftest(int* status, long long limit_cycles, int code, cudaStream_t st);
}  // namespace osdn

using namespace osdn;

namespace {

thread_local int g_last_launches = 0;

// ---- optional stage timing ------------------------------------------------------------------
constexpr int MAX_MARKS = 2048;
struct StageTimer {
    bool enabled = false;
    int count = 0;
    cudaEvent_t ev[MAX_MARKS] = {};
    const char* name[MAX_MARKS] = {};   // nullptr marks the end of a kernel sequence
    int created = 0;
};
StageTimer g_timer;

void timer_push(cudaStream_t st, const char* name)
{
    if (!g_timer.enabled || g_timer.count >= MAX_MARKS) return;
    const int i = g_timer.count;
    if (i >= g_timer.created) {
        if (cudaEventCreate(&g_timer.ev[i]) != cudaSuccess) return;
        g_timer.created = i + 1;
    }
    if (cudaEventRecord(g_timer.ev[i], st) != cudaSuccess) return;
    g_timer.name[i] = name;
    g_timer.count = i + 1;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int validate(const osdn_params* p)
{
    if (!p) return OSDN_INVALID_ARG;
    if (p->io_dtype != OSDN_FP32 && p->io_dtype != OSDN_BF16) return OSDN_INVALID_ARG;
    if (p->apf_mode < 0 || p->apf_mode > 3) return OSDN_INVALID_ARG;
    if (p->B <= 0 || p->H <= 0) return OSDN_INVALID_ARG;
    if (p->T <= 0) return OSDN_UNSUPPORTED_SHAPE;
    if (p->chunk != CH) return OSDN_UNSUPPORTED_SHAPE;
    if ((p->K != 64 && p->K != 128) || (p->V != 64 && p->V != 128)) return OSDN_UNSUPPORTED_SHAPE;
    if (p->nseq < 0) return OSDN_INVALID_ARG;
    if (p->nseq > 0 && (p->B != 1 || !p->cu_seqlens)) return OSDN_INVALID_ARG;
    if (!(p->d_min <= p->d_max) || !(p->eps > 0.f) || !std::isfinite(p->eta)) return OSDN_INVALID_ARG;
    const double tokens = (double)p->B * p->T;
    if (tokens * p->H * (p->K > p->V ? p->K : p->V) > 2.0e10) return OSDN_UNSUPPORTED_SHAPE;
    if (tokens > 1.0e9) return OSDN_UNSUPPORTED_SHAPE;
    return OSDN_OK;
}

Hyper make_hyper(const osdn_params& p)
{
    Hyper h;
    h.eta = p.eta; h.d_min = p.d_min; h.d_max = p.d_max; h.eps = p.eps;
    h.scale = p.scale > 0.f ? p.scale : 1.0f / std::sqrt((float)p.K);
    h.beta_aware = p.beta_aware ? 1 : 0; h.apf_mode = p.apf_mode; h.clamp = p.clamp ? 1 : 0;
    return h;
}

// The tensor-core kernels serve bf16 I/O.  A forward that saves residuals and the backward that
// consumes them must use the same kernel family, so both follow tc_backward_supported.
bool use_tc(const osdn_params& p, bool with_residuals)
{
    if (p.io_dtype != OSDN_BF16 || (p.flags & OSDN_FLAG_FORCE_SIMT) || !tc_supported(p)) return false;
    return with_residuals ? tc_backward_supported(p) : true;
}

int run_forward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                bool save, cudaStream_t st)
{
    int n0 = launch_build_table(p, L, ws, st);
    if (n0 < 0) return -1;
    int n1 = use_tc(p, save) ? tc_forward(p, hy, L, ws, a, save, st) : simt_forward(p, hy, L, ws, a, save, st);
    if (n1 < 0) return -1;
    return n0 + n1;
}

}  // namespace

namespace osdn {
void stage_mark(cudaStream_t st, const char* name) { timer_push(st, name); }
void stage_end(cudaStream_t st) { timer_push(st, nullptr); }
}  // namespace osdn

extern "C" {

void osdn_stage_timing_enable(int on)
{
    g_timer.enabled = on != 0;
    g_timer.count = 0;
}

int osdn_stage_timing_read(int index, const char** name, float* ms)
{
    if (index < 0 || index + 1 >= g_timer.count || !g_timer.name[index]) {
        if (name) *name = nullptr;
        if (ms) *ms = 0.f;
        return g_timer.count;
    }
    float t = 0.f;
    if (cudaEventElapsedTime(&t, g_timer.ev[index], g_timer.ev[index + 1]) != cudaSuccess) t = -1.f;
    if (name) *name = g_timer.name[index];
    if (ms) *ms = t;
    return g_timer.count;
}

size_t osdn_workspace_bytes(const osdn_params* p, int need_bwd)
{
    if (validate(p) != OSDN_OK) return 0;
    return make_layout(*p, need_bwd != 0).total;
}

int osdn_fwd(const osdn_params* p, const void* q, const void* k, const void* v, const float* beta,
             const float* gate, const float* apf_log_ret, const float* init_state, const float* precond_in,
             void* out, float* final_state, float* precond_out, void* workspace, size_t workspace_bytes,
             void* cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != OSDN_OK) return rc;
    if (!q || !k || !v || !beta || !gate || !out || !workspace) return OSDN_INVALID_ARG;
    if (p->apf_mode >= OSDN_APF_SEPARATE && !apf_log_ret) return OSDN_INVALID_ARG;
    const void* ptrs[] = {q, k, v, beta, gate, apf_log_ret, init_state, precond_in, out, final_state,
                          precond_out};
    for (const void* x : ptrs)
        if (x && !aligned16(x)) return OSDN_MISALIGNED;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return OSDN_MISALIGNED;
    const bool save = (p->flags & OSDN_FLAG_SAVE_RESIDUALS) != 0;
    const WsLayout L = make_layout(*p, save);
    if (workspace_bytes < L.total) return OSDN_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(static_cast<char*>(workspace) + L.status, 0, 256, st) != cudaSuccess)
        return OSDN_CUDA_ERROR;
    Pointers a{};
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.gate = gate; a.log_ret = apf_log_ret;
    a.init_state = init_state; a.precond_in = precond_in; a.out = out; a.final_state = final_state;
    a.precond_out = precond_out;
    const int n = run_forward(*p, make_hyper(*p), L, workspace, a, save, st);
    if (n < 0) return OSDN_CUDA_ERROR;
    g_last_launches = n;
    return OSDN_OK;
}

int osdn_bwd(const osdn_params* p, const void* q, const void* k, const void* v, const float* beta,
             const float* gate, const float* apf_log_ret, const float* init_state, const float* precond_in,
             const void* dout, const float* dfinal_state, const float* dprecond_out, void* dq, void* dk,
             void* dv, float* dbeta, float* dgate, float* dapf_log_ret, float* dinit_state,
             float* dprecond_in, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != OSDN_OK) return rc;
    if (!q || !k || !v || !beta || !gate || !dout || !dq || !dk || !dv || !dbeta || !dgate || !workspace)
        return OSDN_INVALID_ARG;
    if (p->apf_mode >= OSDN_APF_SEPARATE && (!apf_log_ret || !dapf_log_ret)) return OSDN_INVALID_ARG;
    const void* ptrs[] = {q, k, v, beta, gate, apf_log_ret, init_state, precond_in, dout, dfinal_state,
                          dprecond_out, dq, dk, dv, dbeta, dgate, dapf_log_ret, dinit_state, dprecond_in};
    for (const void* x : ptrs)
        if (x && !aligned16(x)) return OSDN_MISALIGNED;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return OSDN_MISALIGNED;
    const WsLayout L = make_layout(*p, true);
    if (workspace_bytes < L.total) return OSDN_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Hyper hy = make_hyper(*p);
    Pointers a{};
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.gate = gate; a.log_ret = apf_log_ret;
    a.init_state = init_state; a.precond_in = precond_in;
    a.dout = dout; a.dfinal_state = dfinal_state; a.dprecond_out = dprecond_out;
    a.dq = dq; a.dk = dk; a.dv = dv; a.dbeta = dbeta; a.dgate = dgate; a.dlog_ret = dapf_log_ret;
    a.dinit_state = dinit_state; a.dprecond_in = dprecond_in;
    int total = 0;
    if (!(p->flags & OSDN_FLAG_RESIDUALS_VALID)) {
        // Recompute the forward residuals; the forward output itself lands in scratch.
        if (cudaMemsetAsync(static_cast<char*>(workspace) + L.status, 0, 256, st) != cudaSuccess)
            return OSDN_CUDA_ERROR;
        Pointers f = a;
        f.out = static_cast<char*>(workspace) + L.out_scratch;
        f.final_state = nullptr;
        f.precond_out = nullptr;
        const int n = run_forward(*p, hy, L, workspace, f, true, st);
        if (n < 0) return OSDN_CUDA_ERROR;
        total += n;
    }
    const int n = use_tc(*p, true) ? tc_backward(*p, hy, L, workspace, a, st) : simt_backward(*p, hy, L, workspace, a, st);
    if (n < 0) return OSDN_CUDA_ERROR;
    g_last_launches = total + n;
    return OSDN_OK;
}

size_t osdn_kda_workspace_bytes(const osdn_params* p, int need_bwd)
{
    if (validate(p) != OSDN_OK || p->apf_mode == OSDN_APF_ALIAS_GATE) return 0;
    const WsLayout L = make_layout(*p, need_bwd != 0);
    return align_up(L.total, 256) + kda_extra_bytes(*p, L, need_bwd != 0);
}

int osdn_kda_fwd(const osdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                 const float* gate_k, const float* apf_log_ret, const float* init_state, const float* precond_in,
                 void* out, float* final_state, float* precond_out, void* workspace, size_t workspace_bytes,
                 void* cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != OSDN_OK) return rc;
    if (p->apf_mode == OSDN_APF_ALIAS_GATE) return OSDN_INVALID_ARG;   // the retention is separate from a channel gate
    if (!q || !k || !v || !beta || !gate_k || !out || !workspace) return OSDN_INVALID_ARG;
    if (p->apf_mode >= OSDN_APF_SEPARATE && !apf_log_ret) return OSDN_INVALID_ARG;
    const void* ptrs[] = {q, k, v, beta, gate_k, apf_log_ret, init_state, precond_in, out, final_state, precond_out};
    for (const void* x : ptrs)
        if (x && !aligned16(x)) return OSDN_MISALIGNED;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return OSDN_MISALIGNED;
    const bool save = (p->flags & OSDN_FLAG_SAVE_RESIDUALS) != 0;
    const WsLayout L = make_layout(*p, save);
    if (workspace_bytes < align_up(L.total, 256) + kda_extra_bytes(*p, L, save)) return OSDN_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(static_cast<char*>(workspace) + L.status, 0, 256, st) != cudaSuccess) return OSDN_CUDA_ERROR;
    Pointers a{};
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.gate = gate_k; a.log_ret = apf_log_ret;
    a.init_state = init_state; a.precond_in = precond_in; a.out = out; a.final_state = final_state;
    a.precond_out = precond_out;
    const int n = kda_forward(*p, make_hyper(*p), L, workspace, a, save, st);
    if (n < 0) return OSDN_CUDA_ERROR;
    g_last_launches = n;
    return OSDN_OK;
}

int osdn_kda_bwd(const osdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                 const float* gate_k, const float* apf_log_ret, const float* init_state, const float* precond_in,
                 const void* dout, const float* dfinal_state, const float* dprecond_out, void* dq, void* dk,
                 void* dv, float* dbeta, float* dgate_k, float* dapf_log_ret, float* dinit_state,
                 float* dprecond_in, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != OSDN_OK) return rc;
    if (p->apf_mode == OSDN_APF_ALIAS_GATE) return OSDN_INVALID_ARG;
    if (!q || !k || !v || !beta || !gate_k || !dout || !dq || !dk || !dv || !dbeta || !dgate_k || !workspace)
        return OSDN_INVALID_ARG;
    if (p->apf_mode >= OSDN_APF_SEPARATE && (!apf_log_ret || !dapf_log_ret)) return OSDN_INVALID_ARG;
    const void* ptrs[] = {q, k, v, beta, gate_k, apf_log_ret, init_state, precond_in, dout, dfinal_state,
                          dprecond_out, dq, dk, dv, dbeta, dgate_k, dapf_log_ret, dinit_state, dprecond_in};
    for (const void* x : ptrs)
        if (x && !aligned16(x)) return OSDN_MISALIGNED;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return OSDN_MISALIGNED;
    const WsLayout L = make_layout(*p, true);
    if (workspace_bytes < align_up(L.total, 256) + kda_extra_bytes(*p, L, true)) return OSDN_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const Hyper hy = make_hyper(*p);
    Pointers a{};
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.gate = gate_k; a.log_ret = apf_log_ret;
    a.init_state = init_state; a.precond_in = precond_in;
    a.dout = dout; a.dfinal_state = dfinal_state; a.dprecond_out = dprecond_out;
    a.dq = dq; a.dk = dk; a.dv = dv; a.dbeta = dbeta; a.dgate = dgate_k; a.dlog_ret = dapf_log_ret;
    a.dinit_state = dinit_state; a.dprecond_in = dprecond_in;
    int total = 0;
    if (!(p->flags & OSDN_FLAG_RESIDUALS_VALID)) {
        if (cudaMemsetAsync(static_cast<char*>(workspace) + L.status, 0, 256, st) != cudaSuccess) return OSDN_CUDA_ERROR;
        Pointers f = a;
        f.out = static_cast<char*>(workspace) + L.out_scratch;
        f.final_state = nullptr;
        f.precond_out = nullptr;
        const int n = kda_forward(*p, hy, L, workspace, f, true, st);
        if (n < 0) return OSDN_CUDA_ERROR;
        total += n;
    }
    const int n = kda_backward(*p, hy, L, workspace, a, st);
    if (n < 0) return OSDN_CUDA_ERROR;
    g_last_launches = total + n;
    return OSDN_OK;
}

int osdn_precond_update(const osdn_params* p, const void* k, const float* beta, const float* gate_or_log_ret,
                        const float* precond_in, void* k_tilde_out, float* precond_out, void* cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != OSDN_OK) return rc;
    if (!k || !beta || !precond_out) return OSDN_INVALID_ARG;
    if (p->apf_mode != OSDN_APF_NONE && !gate_or_log_ret) return OSDN_INVALID_ARG;
    const void* ptrs[] = {k, beta, gate_or_log_ret, precond_in, k_tilde_out, precond_out};
    for (const void* x : ptrs)
        if (x && !aligned16(x)) return OSDN_MISALIGNED;
    const int n = phase1_update(*p, make_hyper(*p), k, beta, gate_or_log_ret, precond_in, k_tilde_out,
                                      precond_out, nullptr, nullptr, static_cast<cudaStream_t>(cuda_stream));
    if (n < 0) return OSDN_CUDA_ERROR;
    g_last_launches = n;
    return OSDN_OK;
}

int osdn_residual_ratio(const osdn_params* p, const void* k, const float* beta, const float* gate_or_log_ret,
                        const float* precond_in, float* ratio_out, float* log_ratio_sum, float* precond_out,
                        void* cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != OSDN_OK) return rc;
    if (!k || !beta || (!ratio_out && !log_ratio_sum)) return OSDN_INVALID_ARG;
    if (p->apf_mode != OSDN_APF_NONE && !gate_or_log_ret) return OSDN_INVALID_ARG;
    const void* ptrs[] = {k, beta, gate_or_log_ret, precond_in, ratio_out, log_ratio_sum, precond_out};
    for (const void* x : ptrs)
        if (x && !aligned16(x)) return OSDN_MISALIGNED;
    const int n = phase1_update(*p, make_hyper(*p), k, beta, gate_or_log_ret, precond_in, nullptr, precond_out,
                                ratio_out, log_ratio_sum, static_cast<cudaStream_t>(cuda_stream));
    if (n < 0) return OSDN_CUDA_ERROR;
    g_last_launches = n;
    return OSDN_OK;
}

int osdn_decode_step(const osdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                     const float* gate, const float* apf_log_ret, float* state, float* precond, void* out,
                     void* cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != OSDN_OK) return rc;
    if (p->nseq != 0) return OSDN_INVALID_ARG;   // a dense [B, T, H, *] block of new tokens
    if (!q || !k || !v || !beta || !gate || !state || !precond || !out) return OSDN_INVALID_ARG;
    if (p->apf_mode >= OSDN_APF_SEPARATE && !apf_log_ret) return OSDN_INVALID_ARG;
    const void* ptrs[] = {q, k, v, beta, gate, apf_log_ret, state, precond, out};
    for (const void* x : ptrs)
        if (x && !aligned16(x)) return OSDN_MISALIGNED;
    const int n = decode_step(*p, make_hyper(*p), q, k, v, beta, gate, apf_log_ret, state, precond, out,
                              static_cast<cudaStream_t>(cuda_stream));
    if (n < 0) return OSDN_CUDA_ERROR;
    g_last_launches = n;
    return OSDN_OK;
}

// ---- host-buffer convenience --------------------------------------------------------------
namespace {
struct Staging {
    size_t q, k, v, beta, gate, out, dout, dq, dk, dv, dbeta, dgate, ws, total, ws_bytes;
};
Staging make_staging(const osdn_params& p, bool bwd)
{
    Staging s{};
    const size_t Ttot = p.nseq > 0 ? (size_t)p.T : (size_t)p.B * p.T;
    const size_t es = p.io_dtype == OSDN_BF16 ? 2 : 4;
    size_t off = 0;
    auto take = [&](size_t b) { size_t o = off; off = align_up(off + b, 256); return o; };
    s.q = take(Ttot * p.H * p.K * es); s.k = take(Ttot * p.H * p.K * es); s.v = take(Ttot * p.H * p.V * es);
    s.beta = take(Ttot * p.H * 4); s.gate = take(Ttot * p.H * 4); s.out = take(Ttot * p.H * p.V * es);
    if (bwd) {
        s.dout = take(Ttot * p.H * p.V * es); s.dq = take(Ttot * p.H * p.K * es);
        s.dk = take(Ttot * p.H * p.K * es); s.dv = take(Ttot * p.H * p.V * es);
        s.dbeta = take(Ttot * p.H * 4); s.dgate = take(Ttot * p.H * 4);
    }
    s.ws_bytes = make_layout(p, bwd).total;
    s.ws = take(s.ws_bytes);
    s.total = off;
    return s;
}
}  // namespace

size_t osdn_host_staging_bytes(const osdn_params* p, int with_bwd)
{
    if (validate(p) != OSDN_OK) return 0;
    return make_staging(*p, with_bwd != 0).total;
}

namespace {
// Copy streams and events of the pipelined host step, created once per device.
struct HostPipe {
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
    std::vector<cudaEvent_t> arrived, computed;
};
std::mutex g_pipe_mutex;
HostPipe* host_pipe(int nseq)
{
    static HostPipe pipes[64];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe& hp = pipes[dev];
    if (!hp.in) {
        if (cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&hp.fork, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&hp.join, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    }
    while ((int)hp.arrived.size() < nseq) {
        cudaEvent_t e1, e2;
        if (cudaEventCreateWithFlags(&e1, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        if (cudaEventCreateWithFlags(&e2, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        hp.arrived.push_back(e1);
        hp.computed.push_back(e2);
    }
    return &hp;
}
}  // namespace

int osdn_step_host(const osdn_params* p, const void* q_host, const void* k_host, const void* v_host,
                   const float* beta_host, const float* gate_host, const void* dout_host, void* out_host,
                   void* dq_host, void* dk_host, void* dv_host, float* dbeta_host, float* dgate_host,
                   void* staging, size_t staging_bytes, void* cuda_stream)
{
    int rc = validate(p);
    if (rc != OSDN_OK) return rc;
    const bool bwd = dout_host != nullptr;
    if (!q_host || !k_host || !v_host || !beta_host || !gate_host || !out_host || !staging) return OSDN_INVALID_ARG;
    if (bwd && (!dq_host || !dk_host || !dv_host || !dbeta_host || !dgate_host)) return OSDN_INVALID_ARG;
    if (p->apf_mode >= OSDN_APF_SEPARATE) return OSDN_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(staging) & 255u) return OSDN_MISALIGNED;
    const Staging s = make_staging(*p, bwd);
    if (staging_bytes < s.total) return OSDN_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    char* d = static_cast<char*>(staging);
    const size_t es = p->io_dtype == OSDN_BF16 ? 2 : 4;
    // A dense batch is cut into its sequences (they are independent problems): while one sequence is
    // computed the next one's inputs arrive and the previous one's results leave, on two copy streams
    // that fork from and join `cuda_stream`.  Packed batches and single sequences go in one piece.
    const int pieces = (p->nseq == 0 && p->B > 1) ? p->B : 1;
    const size_t Tp = p->nseq > 0 ? (size_t)p->T : (size_t)(p->B / pieces) * p->T;   // tokens per piece
    const size_t nk = Tp * p->H * p->K * es, nv = Tp * p->H * p->V * es, ns = Tp * p->H * 4;
    HostPipe* hp = pieces > 1 ? host_pipe(pieces) : nullptr;
    if (pieces > 1 && !hp) return OSDN_CUDA_ERROR;
    cudaStream_t sin = hp ? hp->in : st, sout = hp ? hp->out : st;
    bool ok = true;
    auto cpy = [&](void* dst, const void* src, size_t n, cudaMemcpyKind kind, cudaStream_t on) {
        ok = ok && cudaMemcpyAsync(dst, src, n, kind, on) == cudaSuccess;
    };
    auto hoff = [](const void* base, size_t off) { return static_cast<const char*>(base) + off; };
    auto hoffw = [](void* base, size_t off) { return static_cast<char*>(base) + off; };
    if (hp) {
        ok = ok && cudaEventRecord(hp->fork, st) == cudaSuccess;
        ok = ok && cudaStreamWaitEvent(sin, hp->fork, 0) == cudaSuccess;
        ok = ok && cudaStreamWaitEvent(sout, hp->fork, 0) == cudaSuccess;
    }
    for (int b = 0; b < pieces; ++b) {
        cpy(d + s.q + b * nk, hoff(q_host, b * nk), nk, cudaMemcpyHostToDevice, sin);
        cpy(d + s.k + b * nk, hoff(k_host, b * nk), nk, cudaMemcpyHostToDevice, sin);
        cpy(d + s.v + b * nv, hoff(v_host, b * nv), nv, cudaMemcpyHostToDevice, sin);
        cpy(d + s.beta + b * ns, hoff(beta_host, b * ns), ns, cudaMemcpyHostToDevice, sin);
        cpy(d + s.gate + b * ns, hoff(gate_host, b * ns), ns, cudaMemcpyHostToDevice, sin);
        if (bwd) cpy(d + s.dout + b * nv, hoff(dout_host, b * nv), nv, cudaMemcpyHostToDevice, sin);
        if (hp) ok = ok && cudaEventRecord(hp->arrived[b], sin) == cudaSuccess;
    }
    if (!ok) return OSDN_CUDA_ERROR;
    osdn_params pp = *p;
    if (pieces > 1) pp.B = 1;
    int launches = 0;
    for (int b = 0; b < pieces; ++b) {
        if (hp && cudaStreamWaitEvent(st, hp->arrived[b], 0) != cudaSuccess) return OSDN_CUDA_ERROR;
        pp.flags = (p->flags & OSDN_FLAG_FORCE_SIMT) | (bwd ? OSDN_FLAG_SAVE_RESIDUALS : 0);
        rc = osdn_fwd(&pp, d + s.q + b * nk, d + s.k + b * nk, d + s.v + b * nv,
                      reinterpret_cast<float*>(d + s.beta + b * ns), reinterpret_cast<float*>(d + s.gate + b * ns),
                      nullptr, nullptr, nullptr, d + s.out + b * nv, nullptr, nullptr, d + s.ws, s.ws_bytes,
                      cuda_stream);
        if (rc != OSDN_OK) return rc;
        launches += g_last_launches;
        if (bwd) {
            pp.flags |= OSDN_FLAG_RESIDUALS_VALID;
            rc = osdn_bwd(&pp, d + s.q + b * nk, d + s.k + b * nk, d + s.v + b * nv,
                          reinterpret_cast<float*>(d + s.beta + b * ns),
                          reinterpret_cast<float*>(d + s.gate + b * ns), nullptr, nullptr, nullptr,
                          d + s.dout + b * nv, nullptr, nullptr, d + s.dq + b * nk, d + s.dk + b * nk,
                          d + s.dv + b * nv, reinterpret_cast<float*>(d + s.dbeta + b * ns),
                          reinterpret_cast<float*>(d + s.dgate + b * ns), nullptr, nullptr, nullptr, d + s.ws,
                          s.ws_bytes, cuda_stream);
            if (rc != OSDN_OK) return rc;
            launches += g_last_launches;
        }
        if (hp) {
            ok = ok && cudaEventRecord(hp->computed[b], st) == cudaSuccess;
            ok = ok && cudaStreamWaitEvent(sout, hp->computed[b], 0) == cudaSuccess;
        }
        cpy(hoffw(out_host, b * nv), d + s.out + b * nv, nv, cudaMemcpyDeviceToHost, sout);
        if (bwd) {
            cpy(hoffw(dq_host, b * nk), d + s.dq + b * nk, nk, cudaMemcpyDeviceToHost, sout);
            cpy(hoffw(dk_host, b * nk), d + s.dk + b * nk, nk, cudaMemcpyDeviceToHost, sout);
            cpy(hoffw(dv_host, b * nv), d + s.dv + b * nv, nv, cudaMemcpyDeviceToHost, sout);
            cpy(hoffw(dbeta_host, b * ns), d + s.dbeta + b * ns, ns, cudaMemcpyDeviceToHost, sout);
            cpy(hoffw(dgate_host, b * ns), d + s.dgate + b * ns, ns, cudaMemcpyDeviceToHost, sout);
        }
    }
    if (hp) {   // everything the copy streams did is ordered before what follows on the caller's stream
        ok = ok && cudaEventRecord(hp->join, sout) == cudaSuccess;
        ok = ok && cudaStreamWaitEvent(st, hp->join, 0) == cudaSuccess;
        ok = ok && cudaEventRecord(hp->join, sin) == cudaSuccess;
        ok = ok && cudaStreamWaitEvent(st, hp->join, 0) == cudaSuccess;
    }
    g_last_launches = launches;
    return ok ? OSDN_OK : OSDN_CUDA_ERROR;
}

// ---- forward without a caller workspace ----------------------------------------------------
// Scratch for osdn_fwd_static.  In host code the name below is only a handle for the symbol, not a
// device address: the address is looked up once per device with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[OSDN_STATIC_SCRATCH_BYTES];

namespace {
constexpr int MAX_DEVICES = 64;
std::mutex g_static_mutex;
void* g_static_ptr[MAX_DEVICES] = {};

// Device address of g_static_scratch on the current device (looked up on first use).  The stream a
// caller passes must belong to the device that is current at the call.
void* static_scratch_address()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return nullptr;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) return nullptr;
        g_static_ptr[dev] = ptr;
    }
    return g_static_ptr[dev];
}
}  // namespace

int osdn_fwd_static(const osdn_params* p, const void* q, const void* k, const void* v, const float* beta,
                    const float* gate, const float* apf_log_ret, const float* init_state, const float* precond_in,
                    void* out, float* final_state, float* precond_out, void* cuda_stream)
{
    g_last_launches = 0;
    int rc = validate(p);
    if (rc != OSDN_OK) return rc;
    if (!q || !k || !v || !beta || !gate || !out) return OSDN_INVALID_ARG;
    if (p->apf_mode >= OSDN_APF_SEPARATE && !apf_log_ret) return OSDN_INVALID_ARG;
    const void* ptrs[] = {q, k, v, beta, gate, apf_log_ret, init_state, precond_in, out, final_state,
                          precond_out};
    for (const void* x : ptrs)
        if (x && !aligned16(x)) return OSDN_MISALIGNED;
    osdn_params pp = *p;
    pp.flags = p->flags & OSDN_FLAG_FORCE_SIMT;
    const WsLayout L = make_layout(pp, false);
    if (L.total > (size_t)OSDN_STATIC_SCRATCH_BYTES) return OSDN_STATIC_SCRATCH_TOO_SMALL;
    void* scratch = static_scratch_address();
    if (!scratch) return OSDN_CUDA_ERROR;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // the device status word is the only part that must start at zero
    if (cudaMemsetAsync(static_cast<char*>(scratch) + L.status, 0, 256, st) != cudaSuccess) return OSDN_CUDA_ERROR;
    Pointers a{};
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.gate = gate; a.log_ret = apf_log_ret;
    a.init_state = init_state; a.precond_in = precond_in; a.out = out; a.final_state = final_state;
    a.precond_out = precond_out;
    const int n = run_forward(pp, make_hyper(pp), L, scratch, a, false, st);
    if (n < 0) return OSDN_CUDA_ERROR;
    g_last_launches = n;
    return OSDN_OK;
}

int osdn_read_static_status(int32_t* status_host)
{
    if (!status_host) return OSDN_INVALID_ARG;
    void* scratch = static_scratch_address();
    if (!scratch) return OSDN_CUDA_ERROR;
    return cudaMemcpy(status_host, scratch, sizeof(int32_t), cudaMemcpyDeviceToHost) == cudaSuccess
               ? OSDN_OK : OSDN_CUDA_ERROR;
}

int osdn_selftest_wait_timeout(void* workspace, uint32_t limit_us, void* cuda_stream)
{
    if (!workspace || limit_us == 0 || limit_us > 100000u) return OSDN_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return OSDN_MISALIGNED;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemsetAsync(workspace, 0, 256, st) != cudaSuccess) return OSDN_CUDA_ERROR;
    // about 2000 clock cycles per microsecond at the chip's highest clock: the limit is an upper bound
    const long long cycles = 2000ll * (long long)limit_us;
    const int n = launch_wait_timeout_selftest(static_cast<int*>(workspace), cycles, OSDN_DEVICE_SELFTEST_TIMEOUT, st);
    g_last_launches = n > 0 ? n : 0;
    return n > 0 ? OSDN_OK : OSDN_CUDA_ERROR;
}

int osdn_workspace_region(const osdn_params* p, int need_bwd, const char* name, size_t* offset, size_t* bytes)
{
    if (validate(p) != OSDN_OK || !name || !offset || !bytes || !need_bwd) return OSDN_INVALID_ARG;
    const WsLayout L = make_layout(*p, true);
    const size_t Ttot = p->nseq > 0 ? (size_t)p->T : (size_t)p->B * p->T;
    if (!std::strcmp(name, "p1_skip")) {
        *offset = L.p1skip;
        *bytes = 4 * (size_t)L.NTmax * p->H * 2;
        return OSDN_OK;
    }
    if (!std::strcmp(name, "p1_mask")) {
        *offset = L.pmask;
        *bytes = 4 * Ttot * p->H * 32;
        return OSDN_OK;
    }
    return OSDN_INVALID_ARG;
}

int osdn_read_device_status(const void* workspace, int32_t* status_host)
{
    if (!workspace || !status_host) return OSDN_INVALID_ARG;
    return cudaMemcpy(status_host, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost) == cudaSuccess
               ? OSDN_OK : OSDN_CUDA_ERROR;
}

const char* osdn_status_string(int status)
{
    switch (status) {
        case OSDN_OK: return "ok";
        case OSDN_INVALID_ARG: return "invalid argument";
        case OSDN_UNSUPPORTED_SHAPE: return "unsupported shape";
        case OSDN_MISALIGNED: return "pointer not sufficiently aligned";
        case OSDN_WORKSPACE_TOO_SMALL: return "workspace too small";
        case OSDN_CUDA_ERROR: return "CUDA error";
        case OSDN_STATIC_SCRATCH_TOO_SMALL:
            return "problem too large for the built-in scratch of osdn_fwd_static (use osdn_fwd with a workspace)";
        default: return "unknown status";
    }
}

int osdn_last_launch_count(void) { return g_last_launches; }

}  // extern "C"
