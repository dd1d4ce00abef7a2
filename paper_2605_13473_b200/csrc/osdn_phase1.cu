// Phase 1 of the layer: the online preconditioner sweep (Algorithm 1 with APF and the box
// projection) and its reverse sweep (Section 3.5), on CUDA cores in fp32.
//
// The sweep is a length-L sequential chain per (sequence, head).  Two observations keep it off
// the critical path without changing what is computed:
//
//  * Everything of a step that does not depend on d (k^2, its sum, the retention) is evaluated for
//    all tokens in parallel first (phase1_spec).
//  * Once every coordinate of d sits on the lower face of the box, the step for token t maps
//    d_min*1 to d_min*1 again iff every pre-projection value rho_t d_min + c_t k_t^2 is below d_min,
//    a condition that involves token t alone.  phase1_spec evaluates exactly that step for every
//    token ("flag" bit) with the same arithmetic as the sequential kernel.  The sequential kernel
//    (phase1_seq) then only walks tokens where d is not on the face or the flag is clear; flagged
//    tokens entered on the face are skipped (their write key d_min*k was already emitted, their
//    projection mask is all zero).  On the benchmark distributions with the retention aliased to
//    the gate this removes almost every token from the chain; on inputs where d really moves it
//    degenerates to the plain sequential scan.
//
// For the backward pass the forward records, per processed token, d_t and the projection mask,
// and per chunk which tokens were skipped.  A skipped token has an all-zero mask, so the reverse
// recurrence restarts there: lambda_t = k_t (.) dL/dktil_t, dk_t = dk_read_t + d_min dL/dktil_t.
#include "osdn_common.cuh"

namespace osdn {

namespace {

__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// One step of the recurrence on the warp-distributed vector d (lane owns coordinates lane + 32 r).
//   c = eta b (1 - b <d, kap>) / n ;  x = rho d + c kap ;  d <- clip(x)
// n_signed: max(sum kap, eps), negated when the floor eps is active.  pass[r]: ballot of the
// coordinates whose projection passes gradient; all_low: every x strictly below d_min.
template <int R>
__device__ __forceinline__ void p1_step(float (&d)[R], const float (&kap)[R], float n, float b, float rho,
                                        const Hyper& hy, unsigned (&pass)[R], bool& all_low, float& c_out,
                                        float& al_out)
{
    float al = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) al = fmaf(d[r], kap[r], al);
    al = warp_sum(al);
    const float c = hy.eta * b * (1.0f - b * al) / n;
    bool low = true;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        float x = fmaf(c, kap[r], rho * d[r]);
        bool p = true;
        if (hy.clamp) {
            p = (x >= hy.d_min) && (x <= hy.d_max);
            low = low && (x < hy.d_min);
            x = fminf(fmaxf(x, hy.d_min), hy.d_max);
        } else {
            low = false;
        }
        pass[r] = __ballot_sync(0xffffffffu, p);
        d[r] = x;
    }
    all_low = __all_sync(0xffffffffu, low);
    c_out = c;
    al_out = al;
}

template <typename T, int R>
__device__ __forceinline__ float load_key(const T* kp, size_t th, int lane, float (&kk)[R], float (&kap)[R])
{
    float sumk = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        kk[r] = ldf(kp + th * (32 * R) + lane + 32 * r);
        kap[r] = kk[r] * kk[r];
        sumk += kap[r];
    }
    return warp_sum(sumk);
}

// ---------------------------------------------------------------------------------------------
// plain streaming sweep (the stand-alone preconditioner update; no workspace)
// ---------------------------------------------------------------------------------------------
struct P1Args {
    int S, H, T_dense;
    const int* cu;
    const void* k;
    const float *beta, *retsrc, *d0;
    void* ktil;
    float* d_final;
    Hyper hy;
};

template <typename TI, typename TO, int K>
__global__ void __launch_bounds__(128) phase1_stream_kernel(P1Args a)
{
    constexpr int R = K / 32;
    const int lane = threadIdx.x & 31;
    const int chain = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (chain >= a.S * a.H) return;
    const int s = chain / a.H, h = chain % a.H;
    const int t0 = a.cu ? a.cu[s] : s * a.T_dense;
    const int len = a.cu ? max(a.cu[s + 1] - a.cu[s], 0) : a.T_dense;
    const TI* kp = static_cast<const TI*>(a.k);
    TO* kt = static_cast<TO*>(a.ktil);
    float d[R];
#pragma unroll
    for (int r = 0; r < R; ++r) d[r] = a.d0 ? a.d0[((size_t)s * a.H + h) * K + lane + 32 * r] : 1.0f;
    const Hyper hy = a.hy;
    for (int i = 0; i < len; ++i) {
        const size_t th = (size_t)(t0 + i) * a.H + h;
        float kk[R], kap[R];
        const float sumk = load_key<TI, R>(kp, th, lane, kk, kap);
        if (kt) {
#pragma unroll
            for (int r = 0; r < R; ++r) stf(kt + th * K + lane + 32 * r, d[r] * kk[r]);
        }
        const float n = fmaxf(sumk, hy.eps);
        const float b = hy.beta_aware ? a.beta[th] : 1.0f;
        const float rho = hy.apf_mode == 0 ? 1.0f : expf(a.retsrc[th]);
        unsigned pass[R];
        bool low;
        float c, al;
        p1_step<R>(d, kap, n, b, rho, hy, pass, low, c, al);
    }
#pragma unroll
    for (int r = 0; r < R; ++r) a.d_final[((size_t)s * a.H + h) * K + lane + 32 * r] = d[r];
}

// ---------------------------------------------------------------------------------------------
// forward: parallel speculative pass, then the sequential pass over what is left
// ---------------------------------------------------------------------------------------------
struct P1Fwd {
    int S, H, NT;
    Table tab;
    const void* k;
    const float *beta, *retsrc, *d0;
    void* ktil;          // [T,H,K] float or bf16
    float* d_final;      // nullable
    P1Regions r;
    int save;
    Hyper hy;
};

// one warp per (chunk, head, 32-token half)
template <typename TI, typename TO, int K>
__global__ void __launch_bounds__(128) phase1_spec_kernel(P1Fwd a)
{
    constexpr int R = K / 32;
    const int lane = threadIdx.x & 31;
    const long w = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long tile = w >> 1;
    const int half = (int)(w & 1);
    if (tile >= (long)a.NT * a.H) return;
    const int c = (int)(tile / a.H), h = (int)(tile % a.H);
    const int len = a.tab.chunk_len[c], tok0 = a.tab.chunk_tok0[c];
    const TI* kp = static_cast<const TI*>(a.k);
    TO* kt = static_cast<TO*>(a.ktil);
    const Hyper hy = a.hy;
    unsigned word = 0;
    for (int j = 0; j < 32; ++j) {
        const int i = half * 32 + j;
        if (i >= len) break;
        const size_t th = (size_t)(tok0 + i) * a.H + h;
        float kk[R], kap[R];
        const float sumk = load_key<TI, R>(kp, th, lane, kk, kap);
        const float n = fmaxf(sumk, hy.eps);
        const float rho = hy.apf_mode == 0 ? 1.0f : expf(a.retsrc[th]);
        if (lane == 0) {
            a.r.n[th] = sumk > hy.eps ? n : -n;
            a.r.rho[th] = rho;
        }
        if (hy.clamp) {
            const float b = hy.beta_aware ? a.beta[th] : 1.0f;
            float d[R];
#pragma unroll
            for (int r = 0; r < R; ++r) d[r] = hy.d_min;
            unsigned pass[R];
            bool low;
            float cc, al;
            p1_step<R>(d, kap, n, b, rho, hy, pass, low, cc, al);
            if (low) {
                word |= 1u << j;
#pragma unroll
                for (int r = 0; r < R; ++r) stf(kt + th * K + lane + 32 * r, hy.d_min * kk[r]);
            }
        }
    }
    if (lane == 0) a.r.flags[tile * 2 + half] = word;
}

template <int R> __device__ __forceinline__ bool on_lower_face(const float (&d)[R], const Hyper& hy)
{
    bool f = hy.clamp != 0;
#pragma unroll
    for (int r = 0; r < R; ++r) f = f && (d[r] == hy.d_min);
    return __all_sync(0xffffffffu, f);
}

// one warp per chain
template <typename TI, typename TO, int K>
__global__ void __launch_bounds__(128) phase1_seq_kernel(P1Fwd a)
{
    constexpr int R = K / 32;
    const int lane = threadIdx.x & 31;
    const int chain = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (chain >= a.S * a.H) return;
    const int s = chain / a.H, h = chain % a.H, H = a.H;
    const TI* kp = static_cast<const TI*>(a.k);
    TO* kt = static_cast<TO*>(a.ktil);
    const Hyper hy = a.hy;
    float d[R];
#pragma unroll
    for (int r = 0; r < R; ++r) d[r] = a.d0 ? a.d0[((size_t)s * H + h) * K + lane + 32 * r] : 1.0f;
    bool face = on_lower_face<R>(d, hy);
    const int c0 = a.tab.seq_chunk0[s], c1 = a.tab.seq_chunk0[s + 1];
    for (int c = c0; c < c1; ++c) {
        const int tok0 = a.tab.chunk_tok0[c], len = a.tab.chunk_len[c];
        const size_t tile = (size_t)c * H + h;
        const unsigned long long bits =
            (unsigned long long)a.r.flags[tile * 2] | ((unsigned long long)a.r.flags[tile * 2 + 1] << 32);
        const unsigned long long valid = len >= 64 ? ~0ull : ((1ull << len) - 1ull);
        if (a.save) {
#pragma unroll
            for (int r = 0; r < R; ++r) a.r.dbound[tile * K + lane + 32 * r] = d[r];
        }
        unsigned long long skipped = 0ull;
        if (face && (bits & valid) == valid) {
            skipped = valid;
        } else {
            for (int i = 0; i < len; ++i) {
                if (face && ((bits >> i) & 1ull)) {
                    skipped |= 1ull << i;
                    continue;
                }
                const size_t th = (size_t)(tok0 + i) * H + h;
                float kk[R], kap[R];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    kk[r] = ldf(kp + th * K + lane + 32 * r);
                    kap[r] = kk[r] * kk[r];
                }
                const float n = fabsf(a.r.n[th]);
                const float rho = a.r.rho[th];
                const float b = hy.beta_aware ? a.beta[th] : 1.0f;
#pragma unroll
                for (int r = 0; r < R; ++r) stf(kt + th * K + lane + 32 * r, d[r] * kk[r]);
                if (a.save) {
#pragma unroll
                    for (int r = 0; r < R; ++r) a.r.dtraj[th * K + lane + 32 * r] = d[r];
                }
                unsigned pass[R];
                bool low;
                float cc, al;
                p1_step<R>(d, kap, n, b, rho, hy, pass, low, cc, al);
                if (a.save && lane < R) {
                    unsigned wv = 0;
#pragma unroll
                    for (int r = 0; r < R; ++r) wv = lane == r ? pass[r] : wv;
                    a.r.pmask[th * R + lane] = wv;
                }
                face = on_lower_face<R>(d, hy);
            }
        }
        if (a.save && lane == 0) {
            a.r.skipw[tile * 2] = (unsigned)(skipped & 0xffffffffull);
            a.r.skipw[tile * 2 + 1] = (unsigned)(skipped >> 32);
        }
    }
    if (a.d_final) {
#pragma unroll
        for (int r = 0; r < R; ++r) a.d_final[((size_t)s * H + h) * K + lane + 32 * r] = d[r];
    }
}

// ---------------------------------------------------------------------------------------------
// backward
// ---------------------------------------------------------------------------------------------
struct P1Bwd {
    int S, H, NT;
    Table tab;
    const void* k;
    const float *beta, *dktil, *dkread, *dprecond_out;
    void* dk;
    float *dbeta, *dgate, *dlog_ret, *dprecond_in;
    P1Regions r;
    Hyper hy;
};

// skipped tokens: dk = dk_read + d_min dL/dktil (one warp per (chunk, head, 32-token half))
template <typename T, int K>
__global__ void __launch_bounds__(128) phase1_bwd_bulk_kernel(P1Bwd a)
{
    constexpr int R = K / 32;
    const int lane = threadIdx.x & 31;
    const long w = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long tile = w >> 1;
    const int half = (int)(w & 1);
    if (tile >= (long)a.NT * a.H) return;
    const int c = (int)(tile / a.H), h = (int)(tile % a.H);
    const int len = a.tab.chunk_len[c], tok0 = a.tab.chunk_tok0[c];
    const unsigned word = a.r.skipw[tile * 2 + half];
    T* dkp = static_cast<T*>(a.dk);
    for (int j = 0; j < 32; ++j) {
        const int i = half * 32 + j;
        if (i >= len) break;
        if (!((word >> j) & 1u)) continue;
        const size_t th = (size_t)(tok0 + i) * a.H + h;
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const size_t e = th * K + lane + 32 * r;
            stf(dkp + e, a.dkread[e] + a.hy.d_min * a.dktil[e]);
        }
    }
}

// processed tokens, in reverse; one warp per chain
template <typename T, int K>
__global__ void __launch_bounds__(128) phase1_bwd_seq_kernel(P1Bwd a)
{
    constexpr int R = K / 32;
    const int lane = threadIdx.x & 31;
    const int chain = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (chain >= a.S * a.H) return;
    const int s = chain / a.H, h = chain % a.H, H = a.H;
    const Hyper hy = a.hy;
    const T* kp = static_cast<const T*>(a.k);
    T* dkp = static_cast<T*>(a.dk);
    float lam[R];
#pragma unroll
    for (int r = 0; r < R; ++r)
        lam[r] = a.dprecond_out ? a.dprecond_out[((size_t)s * H + h) * K + lane + 32 * r] : 0.f;
    bool lam_valid = true;     // lam holds dL/dd_{t+1} for the token about to be processed
    long src = -1;             // otherwise it is k (.) dktil of this (skipped) token
    const int c0 = a.tab.seq_chunk0[s], c1 = a.tab.seq_chunk0[s + 1];
    for (int c = c1 - 1; c >= c0; --c) {
        const int tok0 = a.tab.chunk_tok0[c], len = a.tab.chunk_len[c];
        const size_t tile = (size_t)c * H + h;
        const unsigned long long sk =
            (unsigned long long)a.r.skipw[tile * 2] | ((unsigned long long)a.r.skipw[tile * 2 + 1] << 32);
        const unsigned long long valid = len >= 64 ? ~0ull : ((1ull << len) - 1ull);
        if ((sk & valid) == valid) {
            lam_valid = false;
            src = tok0;
            continue;
        }
        for (int i = len - 1; i >= 0; --i) {
            if ((sk >> i) & 1ull) {
                lam_valid = false;
                src = tok0 + i;
                continue;
            }
            if (!lam_valid) {
                const size_t ts = (size_t)src * H + h;
#pragma unroll
                for (int r = 0; r < R; ++r)
                    lam[r] = ldf(kp + ts * K + lane + 32 * r) * a.dktil[ts * K + lane + 32 * r];
                lam_valid = true;
            }
            const size_t th = (size_t)(tok0 + i) * H + h;
            float kk[R], kap[R], dt[R], dkt[R], drho = 0.f, dc = 0.f, al = 0.f;
            unsigned mw = lane < R ? a.r.pmask[th * R + lane] : 0u;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const size_t e = th * K + lane + 32 * r;
                kk[r] = ldf(kp + e);
                kap[r] = kk[r] * kk[r];
                dt[r] = a.r.dtraj[e];
                dkt[r] = a.dktil[e];
                const unsigned wr = __shfl_sync(0xffffffffu, mw, r);
                if (!((wr >> lane) & 1u)) lam[r] = 0.f;
                drho = fmaf(lam[r], dt[r], drho);
                dc = fmaf(lam[r], kap[r], dc);
                al = fmaf(dt[r], kap[r], al);
            }
            drho = warp_sum(drho);
            dc = warp_sum(dc);
            al = warp_sum(al);
            const float ns = a.r.n[th], n = fabsf(ns), rho = a.r.rho[th];
            const float b = hy.beta_aware ? a.beta[th] : 1.0f;
            const float cc = hy.eta * b * (1.0f - b * al) / n;
            const float da = -hy.eta * b * b / n * dc;
            const float db = hy.eta * (1.0f - 2.0f * b * al) / n * dc;
            const float dn = ns > 0.f ? -cc / n * dc : 0.f;
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const size_t e = th * K + lane + 32 * r;
                const float dkap = cc * lam[r] + da * dt[r] + dn;
                stf(dkp + e, a.dkread[e] + dt[r] * dkt[r] + 2.0f * kk[r] * dkap);
                lam[r] = rho * lam[r] + da * kap[r] + kk[r] * dkt[r];
            }
            if (lane == 0) {
                if (hy.beta_aware) a.dbeta[th] += db;
                if (hy.apf_mode == 1) a.dgate[th] += rho * drho;
                if (hy.apf_mode == 2 && a.dlog_ret) a.dlog_ret[th] = rho * drho;
            }
        }
    }
    if (a.dprecond_in) {
        if (!lam_valid) {
            const size_t ts = (size_t)src * H + h;
#pragma unroll
            for (int r = 0; r < R; ++r)
                lam[r] = ldf(kp + ts * K + lane + 32 * r) * a.dktil[ts * K + lane + 32 * r];
        }
#pragma unroll
        for (int r = 0; r < R; ++r) a.dprecond_in[((size_t)s * H + h) * K + lane + 32 * r] = lam[r];
    }
}

template <typename TI, typename TO, int K>
int fwd_launch(const P1Fwd& a, cudaStream_t st)
{
    const long warps = (long)a.NT * a.H * 2;
    stage_mark(st, "phase1_spec");
    phase1_spec_kernel<TI, TO, K><<<(unsigned)((warps + 3) / 4), 128, 0, st>>>(a);
    stage_mark(st, "phase1_seq");
    phase1_seq_kernel<TI, TO, K><<<(a.S * a.H + 3) / 4, 128, 0, st>>>(a);
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

template <typename T, int K>
int bwd_launch(const P1Bwd& a, bool bulk, cudaStream_t st)
{
    int n = 0;
    if (bulk) {
        const long warps = (long)a.NT * a.H * 2;
        stage_mark(st, "phase1_bwd_bulk");
        phase1_bwd_bulk_kernel<T, K><<<(unsigned)((warps + 3) / 4), 128, 0, st>>>(a);
        ++n;
    }
    stage_mark(st, "phase1_bwd_seq");
    phase1_bwd_seq_kernel<T, K><<<(a.S * a.H + 3) / 4, 128, 0, st>>>(a);
    ++n;
    return cudaGetLastError() == cudaSuccess ? n : -1;
}

}  // namespace

int phase1_forward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                   void* ktil, bool ktil_bf16, bool save, cudaStream_t st)
{
    P1Fwd f{};
    f.S = L.S; f.H = p.H; f.NT = L.NTmax; f.tab = carve_table(ws, L);
    f.k = a.k; f.beta = a.beta; f.retsrc = p.apf_mode == 2 ? a.log_ret : a.gate; f.d0 = a.precond_in;
    f.ktil = ktil; f.d_final = a.precond_out; f.r = carve_p1(ws, L); f.save = save ? 1 : 0; f.hy = hy;
    if (p.io_dtype == OSDN_FP32) {
        if (ktil_bf16) return -1;
        return p.K == 64 ? fwd_launch<float, float, 64>(f, st) : fwd_launch<float, float, 128>(f, st);
    }
    if (ktil_bf16)
        return p.K == 64 ? fwd_launch<__nv_bfloat16, __nv_bfloat16, 64>(f, st)
                         : fwd_launch<__nv_bfloat16, __nv_bfloat16, 128>(f, st);
    return p.K == 64 ? fwd_launch<__nv_bfloat16, float, 64>(f, st) : fwd_launch<__nv_bfloat16, float, 128>(f, st);
}

int phase1_backward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                    const float* dktil, const float* dkread, bool bulk, cudaStream_t st)
{
    P1Bwd b{};
    b.S = L.S; b.H = p.H; b.NT = L.NTmax; b.tab = carve_table(ws, L);
    b.k = a.k; b.beta = a.beta; b.dktil = dktil; b.dkread = dkread; b.dprecond_out = a.dprecond_out;
    b.dk = a.dk; b.dbeta = a.dbeta; b.dgate = a.dgate; b.dlog_ret = a.dlog_ret; b.dprecond_in = a.dprecond_in;
    b.r = carve_p1(ws, L); b.hy = hy;
    if (p.io_dtype == OSDN_FP32)
        return p.K == 64 ? bwd_launch<float, 64>(b, bulk, st) : bwd_launch<float, 128>(b, bulk, st);
    return p.K == 64 ? bwd_launch<__nv_bfloat16, 64>(b, bulk, st) : bwd_launch<__nv_bfloat16, 128>(b, bulk, st);
}

int phase1_update(const osdn_params& p, const Hyper& hy, const void* k, const float* beta, const float* retsrc,
                  const float* precond_in, void* ktil_out, float* precond_out, cudaStream_t st)
{
    P1Args pa{};
    pa.S = p.nseq > 0 ? p.nseq : p.B;
    pa.H = p.H; pa.T_dense = p.T; pa.cu = p.nseq > 0 ? p.cu_seqlens : nullptr;
    pa.k = k; pa.beta = beta; pa.retsrc = retsrc; pa.d0 = precond_in; pa.ktil = ktil_out;
    pa.d_final = precond_out; pa.hy = hy;
    const int chains = pa.S * pa.H;
    const unsigned grid = (chains + 3) / 4;
    stage_mark(st, "phase1_stream");
    if (p.io_dtype == OSDN_FP32) {
        if (p.K == 64) phase1_stream_kernel<float, float, 64><<<grid, 128, 0, st>>>(pa);
        else phase1_stream_kernel<float, float, 128><<<grid, 128, 0, st>>>(pa);
    } else {
        if (p.K == 64) phase1_stream_kernel<__nv_bfloat16, __nv_bfloat16, 64><<<grid, 128, 0, st>>>(pa);
        else phase1_stream_kernel<__nv_bfloat16, __nv_bfloat16, 128><<<grid, 128, 0, st>>>(pa);
    }
    stage_end(st);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace osdn
