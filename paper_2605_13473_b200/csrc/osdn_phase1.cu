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
//    a condition that involves token t alone.  phase1_spec evaluates that step for every token
//    ("flag" bit), eight lanes per token; from the face the step has a closed form.  The sequential kernel
//    (phase1_seq) then only walks tokens where d is not on the face or the flag is clear; flagged
//    tokens entered on the face are skipped (their write key d_min*k was already emitted, their
//    projection mask is all zero).  On the benchmark distributions with the retention aliased to
//    the gate this removes almost every token from the chain; on inputs where d really moves it
//    degenerates to the plain sequential scan.
//
// The sequential kernels run one warp per chain, so only the warp's own look-ahead hides memory
// latency: rows are fetched a few tokens ahead into a shared-memory ring with cp.async, whose
// completion is counted per committed group, first in first out (rows prefetched into registers
// are held back by the few counters a warp has for outstanding loads).
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

// One step of the recurrence on the warp-distributed vector d (lane l owns coordinates R l + r).
//   c = eta b (1 - b <d, kap>) / n ;  x = rho d + c kap ;  d <- clip(x)
// rho is given per owned coordinate (all equal unless the retention is a vector).
// n_signed: max(sum kap, eps), negated when the floor eps is active.  pass[r]: ballot of the
// coordinates whose projection passes gradient; all_low: every x strictly below d_min.
template <int R>
__device__ __forceinline__ void p1_step(float (&d)[R], const float (&kap)[R], float n, float b,
                                        const float (&rho)[R], const Hyper& hy, unsigned (&pass)[R], bool& all_low, float& c_out,
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
        float x = fmaf(c, kap[r], rho[r] * d[r]);
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

// Lane l of the warp owns the R = K / 32 consecutive coordinates R l .. R l + R - 1, so that a
// row of K values is one vector access per lane.
template <int R> __device__ __forceinline__ void load_row(const float* p, int lane, float (&x)[R])
{
    if constexpr (R == 4) {
        const float4 v = *reinterpret_cast<const float4*>(p + 4 * lane);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    } else {
        const float2 v = *reinterpret_cast<const float2*>(p + 2 * lane);
        x[0] = v.x; x[1] = v.y;
    }
}
template <int R> __device__ __forceinline__ void load_row(const __nv_bfloat16* p, int lane, float (&x)[R])
{
    if constexpr (R == 4) {
        const uint2 v = *reinterpret_cast<const uint2*>(p + 4 * lane);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v.y));
        x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
    } else {
        const uint32_t v = *reinterpret_cast<const uint32_t*>(p + 2 * lane);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v));
        x[0] = a.x; x[1] = a.y;
    }
}
template <int R> __device__ __forceinline__ void store_row(float* p, int lane, const float (&x)[R])
{
    if constexpr (R == 4) *reinterpret_cast<float4*>(p + 4 * lane) = make_float4(x[0], x[1], x[2], x[3]);
    else *reinterpret_cast<float2*>(p + 2 * lane) = make_float2(x[0], x[1]);
}
template <int R> __device__ __forceinline__ void store_row(__nv_bfloat16* p, int lane, const float (&x)[R])
{
    if constexpr (R == 4) {
        __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]), b = __floats2bfloat162_rn(x[2], x[3]);
        uint2 v;
        v.x = *reinterpret_cast<uint32_t*>(&a);
        v.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>(p + 4 * lane) = v;
    } else {
        __nv_bfloat162 a = __floats2bfloat162_rn(x[0], x[1]);
        *reinterpret_cast<uint32_t*>(p + 2 * lane) = *reinterpret_cast<uint32_t*>(&a);
    }
}

// A row as it sits in memory: loading it does not wait for the data (a conversion right after the
// load would stall the warp until the load returns, which defeats fetching rows ahead of their use).
template <typename T, int R> struct RawRow;
template <> struct RawRow<float, 4> { float4 v; };
template <> struct RawRow<float, 2> { float2 v; };
template <> struct RawRow<__nv_bfloat16, 4> { uint2 v; };
template <> struct RawRow<__nv_bfloat16, 2> { uint32_t v; };
template <int R> __device__ __forceinline__ void load_raw(const float* p, int lane, RawRow<float, R>& x)
{
    if constexpr (R == 4) x.v = *reinterpret_cast<const float4*>(p + 4 * lane);
    else x.v = *reinterpret_cast<const float2*>(p + 2 * lane);
}
template <int R> __device__ __forceinline__ void load_raw(const __nv_bfloat16* p, int lane, RawRow<__nv_bfloat16, R>& x)
{
    if constexpr (R == 4) x.v = *reinterpret_cast<const uint2*>(p + 4 * lane);
    else x.v = *reinterpret_cast<const uint32_t*>(p + 2 * lane);
}
template <int R> __device__ __forceinline__ void unpack(const RawRow<float, R>& x, float (&y)[R])
{
    if constexpr (R == 4) { y[0] = x.v.x; y[1] = x.v.y; y[2] = x.v.z; y[3] = x.v.w; }
    else { y[0] = x.v.x; y[1] = x.v.y; }
}
template <int R> __device__ __forceinline__ void unpack(const RawRow<__nv_bfloat16, R>& x, float (&y)[R])
{
    if constexpr (R == 4) {
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x.v.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x.v.y));
        y[0] = a.x; y[1] = a.y; y[2] = b.x; y[3] = b.y;
    } else {
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x.v));
        y[0] = a.x; y[1] = a.y;
    }
}

// Asynchronous copies into a shared-memory ring: completion is counted per committed group (first in,
// first out), so a row fetched PF tokens ahead can be waited for without waiting for the more recent
// ones.  Rows fetched into registers cannot do that: the hardware tracks outstanding loads with a
// handful of counters per warp, and a counter shared with a load issued one token ago holds back the
// use of a row issued eight tokens ago (measured: about 300 cycles per token).
template <int BYTES> __device__ __forceinline__ void cp_async(void* smem, const void* gmem)
{
    static_assert(BYTES == 4 || BYTES == 8 || BYTES == 16, "cp.async copies 4, 8 or 16 bytes");
    asm volatile("cp.async.ca.shared.global [%0], [%1], %2;" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem),
                 "n"(BYTES)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int R> __device__ __forceinline__ float square_sum(const float (&kk)[R], float (&kap)[R])
{
    float sumk = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) {
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
    float* ratio;      // nullable: residual ratio q_t per token-head
    float* log_sum;    // nullable: sum_t log q_t per chain
    Hyper hy;
};

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
    int* status;         // device status word (bounded waits of the pipelined stretches report here)
};

// Eight consecutive values of a row as floats (one 16-byte load for bf16, two for fp32).
__device__ __forceinline__ void load8(const float* p, float (&x)[8])
{
    const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&x)[8])
{
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float2 f = __bfloat1622float2(h[q]);
        x[2 * q] = f.x;
        x[2 * q + 1] = f.y;
    }
}
__device__ __forceinline__ void store8(float* p, const float (&x)[8])
{
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
    *reinterpret_cast<float4*>(p + 4) = make_float4(x[4], x[5], x[6], x[7]);
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&x)[8])
{
    uint4 v;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
    for (int q = 0; q < 4; ++q) h[q] = __floats2bfloat162_rn(x[2 * q], x[2 * q + 1]);
    *reinterpret_cast<uint4*>(p) = v;
}

// One warp per (chunk, head, 32-token half), eight lanes per token (four tokens at a time): a row is
// read in full 128-byte lines and the sums need three shuffle rounds.  The step is taken from
// d = d_min 1: then <d, k^2> = d_min sum k^2, and since x_r = rho d_min + c k_r^2 is monotone in k_r^2
// for a fixed c, "every x_r below d_min" is decided by the largest (c >= 0) or smallest (c < 0) k_r^2.
// With a vector retention (VEC) rho differs per coordinate and every x_r is formed.
template <typename TI, typename TO, int K, bool VEC>
__global__ void __launch_bounds__(128) phase1_spec_kernel(P1Fwd a)
{
    constexpr int NV = K / 64;   // 8-value vectors per lane
    const int lane = threadIdx.x & 31;
    const int grp = lane >> 3, l8 = lane & 7;
    const long w = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const long tile = w >> 1;
    const int half = (int)(w & 1);
    if (tile >= (long)a.NT * a.H) return;
    const int c = (int)(tile / a.H), h = (int)(tile % a.H);
    const int len = a.tab.chunk_len(c), tok0 = a.tab.chunk_tok0(c);
    const Hyper hy = a.hy;
    const TI* kbase = static_cast<const TI*>(a.k);
    TO* tbase = static_cast<TO*>(a.ktil);
    unsigned word = 0;
#pragma unroll 2
    for (int it = 0; it < 8; ++it) {
        const int i = half * 32 + it * 4 + grp;
        const bool in = i < len;
        const size_t th = (size_t)(tok0 + (in ? i : 0)) * a.H + h;
        float x[NV][8];
#pragma unroll
        for (int v = 0; v < NV; ++v) load8(kbase + th * K + v * 64 + l8 * 8, x[v]);
        const float ret = (!VEC && in && hy.apf_mode != 0) ? a.retsrc[th] : 0.f;
        const float b = (in && hy.beta_aware) ? a.beta[th] : 1.0f;
        float sumk = 0.f, kmax = 0.f, kmin = 3.0e38f;
#pragma unroll
        for (int v = 0; v < NV; ++v)
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float kap = x[v][e] * x[v][e];
                sumk += kap;
                kmax = fmaxf(kmax, kap);
                kmin = fminf(kmin, kap);
            }
#pragma unroll
        for (int o = 4; o > 0; o >>= 1) {
            sumk += __shfl_xor_sync(0xffffffffu, sumk, o);
            kmax = fmaxf(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
            kmin = fminf(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
        }
        const float n = fmaxf(sumk, hy.eps);
        const float rho = hy.apf_mode == 0 ? 1.0f : expf(ret);
        bool low = false;
        if (hy.clamp) {
            const float al = hy.d_min * sumk;
            const float cc = hy.eta * b * (1.0f - b * al) / n;
            if constexpr (VEC) {
                bool below = true;
#pragma unroll
                for (int v = 0; v < NV; ++v) {
                    float lr[8];
                    load8(a.retsrc + th * K + v * 64 + l8 * 8, lr);
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        below = below && fmaf(cc, x[v][e] * x[v][e], expf(lr[e]) * hy.d_min) < hy.d_min;
                }
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) below = __shfl_xor_sync(0xffffffffu, (int)below, o) && below;
                low = in && below;
            } else {
                const float xtop = fmaf(cc, cc >= 0.f ? kmax : kmin, rho * hy.d_min);
                low = in && xtop < hy.d_min;
            }
        }
        if (in && l8 == 0) {
            a.r.n[th] = sumk > hy.eps ? 1.0f / n : -1.0f / n;   // reciprocal of the normaliser, signed
            a.r.rho[th] = rho;
        }
        if (low) {   // the write key of a token entered on the face: d_min k
#pragma unroll
            for (int v = 0; v < NV; ++v) {
#pragma unroll
                for (int e = 0; e < 8; ++e) x[v][e] *= hy.d_min;
                store8(tbase + th * K + v * 64 + l8 * 8, x[v]);
            }
        }
        const unsigned bal = __ballot_sync(0xffffffffu, low);
        word |= ((bal & 1u) | ((bal >> 7) & 2u) | ((bal >> 14) & 4u) | ((bal >> 21) & 8u)) << (it * 4);
    }
    if (lane == 0) a.r.flags[tile * 2 + half] = word;
}

__device__ __forceinline__ void prefetch_l2(const void* p)
{
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}
// Warms L2 (and the address translation) for a row of `bytes` bytes that starts on a 128-byte line.
__device__ __forceinline__ void prefetch_row(const void* p, int bytes)
{
    for (int o = 0; o < bytes; o += 128) prefetch_l2(static_cast<const char*>(p) + o);
}

template <int R> __device__ __forceinline__ bool on_lower_face(const float (&d)[R], const Hyper& hy)
{
    bool f = hy.clamp != 0;
#pragma unroll
    for (int r = 0; r < R; ++r) f = f && (d[r] == hy.d_min);
    return __all_sync(0xffffffffu, f);
}

// ---------------------------------------------------------------------------------------------
// Pipelined stretches of the sequential pass.  Where nearly every token is processed (a preconditioner
// that really moves), the walk of a chain is bound by the instructions one warp issues per token, most
// of which do not depend on d: fetching and squaring the key, the step's scalars, forming and storing
// the write key, the records for the backward.  For such a stretch three warps share the chain:
//   pre   fetches a block of PB tokens and leaves k, k^2 and the scalars (e, a2, rho) in shared memory;
//   core  carries d through the block: <d, k^2>, the step, the projection; leaves d_t and the mask;
//   post  forms ktil_t = d_t (.) k_t and writes ktil, d_t and the mask words to global memory.
// Blocks go round a ring of PN buffers; the roles meet at mbarriers (full: pre -> core and post,
// done: core -> post, free: post -> pre).  Every token of a stretch is processed (none is skipped: for a
// flagged token entered on the face the step returns to the face by construction, so the values are
// the ones the skipping walk leaves), which keeps the core free of any bookkeeping.
// ---------------------------------------------------------------------------------------------
constexpr int PB = 16, PN = 3;
constexpr int P1_ERR_PIPE = 131;
constexpr long long P1_WAIT_LIMIT = 4000000000ll;   // about two seconds

__device__ __forceinline__ void p1_mbar_init(uint64_t* b, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void p1_mbar_arrive(uint64_t* b)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"((uint32_t)__cvta_generic_to_shared(b)) : "memory");
}
// Bounded: gives up after P1_WAIT_LIMIT cycles, records the error and returns false.
__device__ __forceinline__ bool p1_mbar_wait(uint64_t* b, uint32_t parity, int* status)
{
    const uint32_t addr = (uint32_t)__cvta_generic_to_shared(b);
    const long long t0 = clock64();
    while (true) {
        uint32_t ok;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(ok)
                     : "r"(addr), "r"(parity)
                     : "memory");
        if (ok) return true;
        if (clock64() - t0 > P1_WAIT_LIMIT) {
            if (status) atomicCAS(status, 0, P1_ERR_PIPE);
            return false;
        }
    }
}

template <typename TI, int K, bool VEC> struct PipeBuf {
    static constexpr int R = K / 32;
    float kap[PB][K];                       // k^2
    RawRow<TI, R> kraw[PB][32];             // k as it sits in memory
    float x[PB][K];                         // the step's value before the projection (d_{t+1} = clip(x_t)), by the core
    float d0[K];                            // d on entry to the block, by the core
    float rhov[VEC ? PB : 1][VEC ? K : 1];  // vector retention: exp(l_t) per coordinate
    float4 scal[PB];                        // e = eta b / n, a2 = e b, rho, fixed-point scale -> <d_t, k^2>
};

// What the post role derives from the core's x: d_t of every token (the clipped x of the token before it,
// the block's entry value for the first) and the projection's pass bits.  The core then carries nothing
// but the recurrence itself.
template <int R> __device__ __forceinline__ void clip_row(const float (&x)[R], const Hyper& hy, float (&d)[R], unsigned& bits)
{
    bits = 0;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        // inside the box (faces included) exactly when clamping leaves the value alone
        d[r] = hy.clamp ? fminf(fmaxf(x[r], hy.d_min), hy.d_max) : x[r];
        bits |= d[r] == x[r] ? (1u << r) : 0u;
    }
}
constexpr int RING_MAX = 6;   // the deeper of the two rings
struct PipeBars {
    uint64_t full[RING_MAX], done[RING_MAX], free_[RING_MAX];
};

// The core's work on one block: carries d through n tokens; reads kap, the scalars (and the retention
// vector), leaves d_t, the mask bits and <d_t, k^2> (in scal.w).
template <typename TI, int K, bool VEC>
__device__ __forceinline__ void pipe_core_block(PipeBuf<TI, K, VEC>& B, int n, float (&d)[K / 32], const Hyper& hy, int lane)
{
    constexpr int R = K / 32;
    store_row<R>(B.d0, lane, d);
    auto token = [&](int j) {
        const float4 sc = B.scal[j];
        float kap[R], rho[R];
        load_row<R>(B.kap[j], lane, kap);
        if constexpr (VEC) load_row<R>(B.rhov[VEC ? j : 0], lane, rho);
        else {
#pragma unroll
            for (int r = 0; r < R; ++r) rho[r] = sc.z;
        }
        float al0 = d[0] * kap[0], al1 = d[1] * kap[1];   // two short chains instead of one long one
#pragma unroll
        for (int r = 2; r < R; r += 2) {
            al0 = fmaf(d[r], kap[r], al0);
            al1 = fmaf(d[r + 1], kap[r + 1], al1);
        }
        float al;
        if (hy.clamp) {
            // With the projection on, 0 <= <d, k^2> <= d_max sum k^2: the lanes' partial sums are added as
            // fixed-point integers with one warp-wide instruction instead of five shuffle-add rounds.
            // sc.w = 2^26 / (d_max sum k^2) (from the pre role): the total stays below 2^27, a lane's
            // rounding is 2^-27 of the bound, 32 of them 2^-22 of it.
            const unsigned q = __float2uint_rn((al0 + al1) * sc.w);
            al = __uint2float_rn(__reduce_add_sync(0xffffffffu, q)) * __frcp_rn(sc.w);
        } else {
            al = warp_sum(al0 + al1);
        }
        const float cc = fmaf(-sc.y, al, sc.x);
        float x[R];
#pragma unroll
        for (int r = 0; r < R; ++r) x[r] = fmaf(cc, kap[r], rho[r] * d[r]);
        store_row<R>(B.x[j], lane, x);
#pragma unroll
        for (int r = 0; r < R; ++r) d[r] = hy.clamp ? fminf(fmaxf(x[r], hy.d_min), hy.d_max) : x[r];
        if (lane == 0) B.scal[j].w = al;
    };
    if (n == PB) {   // partly unrolled: the shared-memory reads of later tokens are issued under the shuffles of earlier ones
#pragma unroll 4
        for (int j = 0; j < PB; ++j) token(j);
    } else {
        for (int j = 0; j < n; ++j) token(j);
    }
}

// tokens [t_a, t_b) of the chain (packed token indices), all three roles; d: the core's registers
template <typename TI, typename TO, int K, bool VEC>
__device__ __forceinline__ bool pipe_stretch(const P1Fwd& a, int h, int t_a, int t_b, float (&d)[K / 32],
                                             PipeBuf<TI, K, VEC>* buf, PipeBars& bars, uint32_t& round0, int role, int lane)
{
    constexpr int R = K / 32;
    const int H = a.H;
    const Hyper hy = a.hy;
    const int nblk = (t_b - t_a + PB - 1) / PB;
    const TI* kp = static_cast<const TI*>(a.k);
    bool ok = true;
    // block b uses buffer b % PN; its barriers complete once per use: parity of the use count
    const uint32_t base = round0;   // uses of the ring before this stretch (a multiple of PN blocks is not required)
    if (role == 1) {
        // ------------------------------------------------------------------ pre
        for (int b = 0; b < nblk && ok; ++b) {
            const uint32_t use = base + b;
            const int bi = use % PN;
            if (use >= PN) ok = p1_mbar_wait(&bars.free_[bi], ((use / PN) - 1) & 1, a.status);
            if (!ok) break;
            PipeBuf<TI, K, VEC>& B = buf[bi];
            const int t0 = t_a + b * PB, n = min(PB, t_b - t0);
            RawRow<TI, R> raw[PB];
#pragma unroll
            for (int j = 0; j < PB; ++j) {
                const size_t th = (size_t)(t0 + min(j, n - 1)) * H + h;
                load_raw<R>(kp + th * K, lane, raw[j]);
            }
            if (lane < n) {
                const size_t th = (size_t)(t0 + lane) * H + h;
                const float rn = fabsf(a.r.n[th]), bb = hy.beta_aware ? a.beta[th] : 1.0f;
                const float e = hy.eta * bb * rn;
                // .w: the fixed-point scale of the core's sum, 2^26 / (d_max max(sum k^2, eps)); the core
                // replaces it by <d_t, k^2>
                B.scal[lane] = make_float4(e, e * bb, a.r.rho[th], 67108864.0f * rn / hy.d_max);
            }
#pragma unroll
            for (int j = 0; j < PB; ++j) {
                float kk[R], kap[R];
                unpack<R>(raw[j], kk);
#pragma unroll
                for (int r = 0; r < R; ++r) kap[r] = kk[r] * kk[r];
                store_row<R>(B.kap[j], lane, kap);
                B.kraw[j][lane] = raw[j];
            }
            if constexpr (VEC) {
                for (int j = 0; j < n; ++j) {
                    const size_t th = (size_t)(t0 + j) * H + h;
                    float lr[R];
                    load_row<R>(a.retsrc + th * K, lane, lr);
#pragma unroll
                    for (int r = 0; r < R; ++r) lr[r] = expf(lr[r]);
                    store_row<R>(B.rhov[VEC ? j : 0], lane, lr);
                }
            }
            __syncwarp();
            if (lane == 0) p1_mbar_arrive(&bars.full[bi]);
        }
    } else if (role == 0) {
        // ------------------------------------------------------------------ core
        for (int b = 0; b < nblk && ok; ++b) {
            const uint32_t use = base + b;
            const int bi = use % PN;
            ok = p1_mbar_wait(&bars.full[bi], (use / PN) & 1, a.status);
            if (!ok) break;
            const int n = min(PB, t_b - (t_a + b * PB));
            pipe_core_block<TI, K, VEC>(buf[bi], n, d, hy, lane);
            __syncwarp();
            if (lane == 0) p1_mbar_arrive(&bars.done[bi]);
        }
    } else {
        // ------------------------------------------------------------------ post
        TO* kt = static_cast<TO*>(a.ktil);
        for (int b = 0; b < nblk && ok; ++b) {
            const uint32_t use = base + b;
            const int bi = use % PN;
            ok = p1_mbar_wait(&bars.done[bi], (use / PN) & 1, a.status);
            if (!ok) break;
            const PipeBuf<TI, K, VEC>& B = buf[bi];
            const int t0 = t_a + b * PB, n = min(PB, t_b - t0);
            float dd[R];   // d_t of the token in hand
            load_row<R>(B.d0, lane, dd);
            auto token = [&](int j) {
                const size_t th = (size_t)(t0 + j) * H + h;
                float kk[R], wk[R], xx[R];
                unpack<R>(B.kraw[j][lane], kk);
#pragma unroll
                for (int r = 0; r < R; ++r) wk[r] = dd[r] * kk[r];
                store_row<R>(kt + th * K, lane, wk);
                if (a.save) store_row<R>(a.r.dtraj + th * K, lane, dd);
                load_row<R>(B.x[j], lane, xx);
                unsigned bits;
                clip_row<R>(xx, hy, dd, bits);   // the next token's d, this token's pass bits
                if (a.save) a.r.pmask[th * 32 + lane] = bits;
            };
            if (a.save && lane < n) a.r.al[(size_t)(t0 + lane) * H + h] = B.scal[lane].w;   // lane j: token j
            if (n == PB) {
#pragma unroll 4
                for (int j = 0; j < PB; ++j) token(j);
            } else {
                for (int j = 0; j < n; ++j) token(j);
            }
            __syncwarp();
            if (lane == 0) p1_mbar_arrive(&bars.free_[bi]);
        }
    }
    round0 = base + nblk;
    return ok;
}

// The stand-alone sweep processes every token: the whole sequence is one pipelined stretch (see the
// forward's stretches below the parallel pass).  pre also forms the normaliser here (there is no parallel
// pass before this kernel); post forms the write keys and the residual ratios.
template <typename TI, typename TO, int K, bool VEC>
__global__ void __launch_bounds__(96) phase1_stream_kernel(P1Args a)
{
    constexpr int R = K / 32;
    extern __shared__ __align__(16) uint8_t p1_dyn[];   // PipeBuf[PN], then the write strengths beta[PN][PB]
    PipeBuf<TI, K, VEC>* buf = reinterpret_cast<PipeBuf<TI, K, VEC>*>(p1_dyn);
    float(*sbeta)[PB] = reinterpret_cast<float(*)[PB]>(p1_dyn + PN * sizeof(PipeBuf<TI, K, VEC>));
    __shared__ PipeBars bars;
    const int lane = threadIdx.x & 31, role = threadIdx.x >> 5;   // 0 core, 1 pre, 2 post
    const int chain = blockIdx.x;
    const int s = chain / a.H, h = chain % a.H, H = a.H;
    // packed batch: T_dense is the packed token count; a malformed offset pair is clamped into it
    const int t0 = a.cu ? min(max(a.cu[s], 0), a.T_dense) : s * a.T_dense;
    const int len = a.cu ? min(max(a.cu[s + 1], t0), a.T_dense) - t0 : a.T_dense;
    const TI* kp = static_cast<const TI*>(a.k);
    const Hyper hy = a.hy;
    if (threadIdx.x == 0) {
        for (int i = 0; i < PN; ++i) {
            p1_mbar_init(&bars.full[i], 1);
            p1_mbar_init(&bars.done[i], 1);
            p1_mbar_init(&bars.free_[i], 1);
        }
    }
    __syncthreads();
    const int nblk = (len + PB - 1) / PB;
    const bool scalar_ret = !VEC && hy.apf_mode != 0;
    bool ok = true;
    if (role == 1) {
        for (int b = 0; b < nblk && ok; ++b) {
            const int bi = b % PN;
            if (b >= PN) ok = p1_mbar_wait(&bars.free_[bi], ((b / PN) - 1) & 1, nullptr);
            if (!ok) break;
            PipeBuf<TI, K, VEC>& B = buf[bi];
            const int tb0 = t0 + b * PB, n = min(PB, len - b * PB);
            RawRow<TI, R> raw[PB];
#pragma unroll
            for (int j = 0; j < PB; ++j) load_raw<R>(kp + ((size_t)(tb0 + min(j, n - 1)) * H + h) * K, lane, raw[j]);
            float beta = 0.f, ret = 0.f;
            if (lane < n) {
                const size_t th = (size_t)(tb0 + lane) * H + h;
                beta = a.beta[th];
                if (scalar_ret) ret = a.retsrc[th];
            }
            float sums[PB];
#pragma unroll
            for (int j = 0; j < PB; ++j) {
                float kk[R], kap[R];
                unpack<R>(raw[j], kk);
                sums[j] = 0.f;
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    kap[r] = kk[r] * kk[r];
                    sums[j] += kap[r];
                }
                store_row<R>(B.kap[j], lane, kap);
                B.kraw[j][lane] = raw[j];
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)   // the sixteen sums together: their shuffle rounds overlap
#pragma unroll
                for (int j = 0; j < PB; ++j) sums[j] += __shfl_xor_sync(0xffffffffu, sums[j], o);
            float mine = 0.f;
#pragma unroll
            for (int j = 0; j < PB; ++j) mine = lane == j ? sums[j] : mine;
            if (lane < n) {
                const float nn = fmaxf(mine, hy.eps), bb = hy.beta_aware ? beta : 1.0f;
                const float e = hy.eta * bb / nn;
                B.scal[lane] = make_float4(e, e * bb, scalar_ret ? expf(ret) : 1.0f, 67108864.0f / (nn * hy.d_max));
                sbeta[bi][lane] = beta;
            }
            if constexpr (VEC) {
                for (int j = 0; j < n; ++j) {
                    float lr[R];
                    load_row<R>(a.retsrc + ((size_t)(tb0 + j) * H + h) * K, lane, lr);
#pragma unroll
                    for (int r = 0; r < R; ++r) lr[r] = expf(lr[r]);
                    store_row<R>(B.rhov[VEC ? j : 0], lane, lr);
                }
            }
            __syncwarp();
            if (lane == 0) p1_mbar_arrive(&bars.full[bi]);
        }
    } else if (role == 0) {
        float d[R];
        if (a.d0) load_row<R>(a.d0 + ((size_t)s * H + h) * K, lane, d);
        else {
#pragma unroll
            for (int r = 0; r < R; ++r) d[r] = 1.0f;
        }
        for (int b = 0; b < nblk && ok; ++b) {
            const int bi = b % PN;
            ok = p1_mbar_wait(&bars.full[bi], (b / PN) & 1, nullptr);
            if (!ok) break;
            pipe_core_block<TI, K, VEC>(buf[bi], min(PB, len - b * PB), d, hy, lane);
            __syncwarp();
            if (lane == 0) p1_mbar_arrive(&bars.done[bi]);
        }
        if (a.d_final && ok) store_row<R>(a.d_final + ((size_t)s * H + h) * K, lane, d);
    } else {
        TO* kt = static_cast<TO*>(a.ktil);
        float lsum = 0.f;
        for (int b = 0; b < nblk && ok; ++b) {
            const int bi = b % PN;
            ok = p1_mbar_wait(&bars.done[bi], (b / PN) & 1, nullptr);
            if (!ok) break;
            const PipeBuf<TI, K, VEC>& B = buf[bi];
            const int tb0 = t0 + b * PB, n = min(PB, len - b * PB);
            if (kt) {
                float dd[R];
                load_row<R>(B.d0, lane, dd);
                for (int j = 0; j < n; ++j) {
                    float kk[R], wk[R], xx[R];
                    unpack<R>(B.kraw[j][lane], kk);
#pragma unroll
                    for (int r = 0; r < R; ++r) wk[r] = dd[r] * kk[r];
                    store_row<R>(kt + ((size_t)(tb0 + j) * H + h) * K, lane, wk);
                    load_row<R>(B.x[j], lane, xx);
                    unsigned bits;
                    clip_row<R>(xx, hy, dd, bits);
                }
            }
            if (a.ratio || a.log_sum) {
                // residual ratio of the write of a token (token-local theorem): the loss |S k - v|^2 after the
                // write over the loss before it is (1 - beta <d_t, k^2>)^2, with the write strength beta itself
                // (whether or not the step of d is beta-aware) and the d the write key was formed with
                float lq = 0.f;
                if (lane < n) {
                    const float fac = 1.0f - sbeta[bi][lane] * B.scal[lane].w;
                    const float qt = fac * fac;
                    if (a.ratio) a.ratio[(size_t)(tb0 + lane) * H + h] = qt;
                    lq = logf(fmaxf(qt, 1.17549435e-38f));
                }
                lsum += warp_sum(lq);
            }
            __syncwarp();
            if (lane == 0) p1_mbar_arrive(&bars.free_[bi]);
        }
        if (a.log_sum && lane == 0) a.log_sum[(size_t)s * H + h] = lsum;
    }
}

// one warp per chain.  Flag words are fetched for 32 chunks at a time (one chunk per lane); the
// rows of the tokens that are really processed are prefetched a few tokens ahead.
// A chunk of which at least PIPE_TRIGGER tokens had to be processed starts a pipelined stretch of up to
// PIPE_CHUNKS chunks; stretches follow one another while d stays off the lower face.
constexpr int PIPE_TRIGGER = 32, PIPE_CHUNKS = 8;

template <typename TI, typename TO, int K, bool VEC>
__global__ void __launch_bounds__(96) phase1_seq_kernel(P1Fwd a)
{
    constexpr int R = K / 32;
    // prefetch distance in tokens: short, because the long runs go through the pipelined stretches and a
    // run's start waits for whatever the run before it still had in flight (8 -> 4: osdn_1p3b 452 -> 401 us)
    constexpr int PF = 4;
    struct RingSlot {
        RawRow<TI, R> k[32];
        RawRow<float, R> lr[VEC ? 32 : 1];
        float n[32], rho[32], beta[32];
    };
    extern __shared__ __align__(16) uint8_t p1_dyn[];   // PipeBuf[PN]
    PipeBuf<TI, K, VEC>* pbuf = reinterpret_cast<PipeBuf<TI, K, VEC>*>(p1_dyn);
    __shared__ __align__(16) RingSlot ring[PF];
    __shared__ PipeBars bars;
    __shared__ int cmd[2];   // token range of the next pipelined stretch; empty: the chain is finished
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chain = blockIdx.x;
    const int s = chain / a.H, h = chain % a.H, H = a.H;
    if (threadIdx.x == 0) {
        for (int i = 0; i < PN; ++i) {
            p1_mbar_init(&bars.full[i], 1);
            p1_mbar_init(&bars.done[i], 1);
            p1_mbar_init(&bars.free_[i], 1);
        }
    }
    __syncthreads();
    uint32_t pipe_uses = 0;   // blocks that have gone through the ring so far (the same in all three warps)
    if (warp != 0) {
        // helper warps (1: pre, 2: post) serve the stretches warp 0 announces
        float none[R];
        while (true) {
            asm volatile("bar.sync 1, 96;" ::: "memory");
            const int t_a = cmd[0], t_b = cmd[1];
            if (t_b <= t_a) break;
            pipe_stretch<TI, TO, K, VEC>(a, h, t_a, t_b, none, pbuf, bars, pipe_uses, warp, lane);
            asm volatile("bar.sync 2, 96;" ::: "memory");
        }
        return;
    }
    bool pipe_next = false;
    const TI* kp = static_cast<const TI*>(a.k);
    TO* kt = static_cast<TO*>(a.ktil);
    const Hyper hy = a.hy;
    float d[R];
    if (a.d0) load_row<R>(a.d0 + ((size_t)s * H + h) * K, lane, d);
    else {
#pragma unroll
        for (int r = 0; r < R; ++r) d[r] = 1.0f;
    }
    bool face = on_lower_face<R>(d, hy);
    const int c0 = a.tab.seq_chunk0(s), c1 = a.tab.seq_chunk0(s + 1);
    const int seq_t0 = a.tab.seq_tok0(s), seq_len = a.tab.seq_len(s);
    for (int cbase = c0; cbase < c1; cbase += 32) {
        unsigned w0 = 0, w1 = 0;
        if (cbase + lane < c1) {
            const size_t tl = (size_t)(cbase + lane) * H + h;
            w0 = a.r.flags[tl * 2];
            w1 = a.r.flags[tl * 2 + 1];
            // Sparse work: unflagged tokens are processed for certain; warm L2 with their rows now.
            const int cl = cbase + lane;
            const int lenl = min(CH, seq_len - (cl - c0) * CH);
            unsigned long long m = ~((unsigned long long)w0 | ((unsigned long long)w1 << 32)) &
                                   (lenl >= 64 ? ~0ull : ((1ull << lenl) - 1ull));
            if (__popcll(m) <= 16) {
                while (m) {
                    const int t = __ffsll((long long)m) - 1;
                    m &= m - 1;
                    const size_t th = (size_t)(seq_t0 + (cl - c0) * CH + t) * H + h;
                    prefetch_row(kp + th * K, K * (int)sizeof(TI));
                    if constexpr (VEC) prefetch_row(a.retsrc + th * K, K * 4);
                    prefetch_l2(a.r.n + th);
                    prefetch_l2(a.r.rho + th);
                    prefetch_l2(a.beta + th);
                }
            }
        }
        const int cend = min(cbase + 32, c1);
        // chunks of this group whose every token is flagged (lane = chunk)
        unsigned allflag;
        {
            const int cl = cbase + lane;
            const int lenl = cl < c1 ? min(CH, seq_len - (cl - c0) * CH) : 0;
            const unsigned long long bl = (unsigned long long)w0 | ((unsigned long long)w1 << 32);
            const unsigned long long vl = lenl >= 64 ? ~0ull : ((1ull << lenl) - 1ull);
            allflag = __ballot_sync(0xffffffffu, cl < c1 && (bl & vl) == vl);
            // The first chunk of a sequence that enters off the face with at least PIPE_TRIGGER tokens that
            // are processed for certain (unflagged) starts pipelined right away.
            if (cbase == c0 && !face) {
                const int sure = __shfl_sync(0xffffffffu, __popcll(~bl & vl), 0);
                pipe_next = sure >= PIPE_TRIGGER;
            }
        }
        for (int c = cbase; c < cend; ++c) {
            if (pipe_next) {
                // a pipelined stretch: every token of the next chunks (of this group) is processed
                const int np = min(PIPE_CHUNKS, cend - c);
                const int nrel = c - c0;
                const int t_a = seq_t0 + nrel * CH, t_b = seq_t0 + min(seq_len, (nrel + np) * CH);
                if (lane == 0) {
                    cmd[0] = t_a;
                    cmd[1] = t_b;
                }
                cp_async_wait<0>();   // nothing of the token-by-token walk is still on its way
                asm volatile("bar.sync 1, 96;" ::: "memory");
                const bool okp = pipe_stretch<TI, TO, K, VEC>(a, h, t_a, t_b, d, pbuf, bars, pipe_uses, 0, lane);
                asm volatile("bar.sync 2, 96;" ::: "memory");
                if (a.save && lane < np) {
                    const size_t tl = (size_t)(c + lane) * H + h;
                    a.r.skipw[tl * 2] = 0u;
                    a.r.skipw[tl * 2 + 1] = 0u;
                }
                face = on_lower_face<R>(d, hy);
                pipe_next = okp && !face;
                c += np - 1;
                continue;
            }
            if (face) {
                // a run of fully flagged chunks entered on the face is skipped in one go
                const unsigned rest = ~allflag >> (c - cbase);
                const int run = min(rest ? __ffs((int)rest) - 1 : 32, cend - c);
                if (run > 0) {
                    if (a.save && lane < run) {
                        const int cl = c + lane;
                        const int lenl = min(CH, seq_len - (cl - c0) * CH);
                        const unsigned long long vl = lenl >= 64 ? ~0ull : ((1ull << lenl) - 1ull);
                        const size_t tl = (size_t)cl * H + h;
                        a.r.skipw[tl * 2] = (unsigned)(vl & 0xffffffffull);
                        a.r.skipw[tl * 2 + 1] = (unsigned)(vl >> 32);
                    }
                    c += run - 1;
                    continue;
                }
            }
            const int nrel = c - c0;
            const int tok0 = seq_t0 + nrel * CH, len = min(CH, seq_len - nrel * CH);
            const size_t tile = (size_t)c * H + h;
            const unsigned long long bits = (unsigned long long)__shfl_sync(0xffffffffu, w0, c - cbase) |
                                            ((unsigned long long)__shfl_sync(0xffffffffu, w1, c - cbase) << 32);
            const unsigned long long valid = len >= 64 ? ~0ull : ((1ull << len) - 1ull);
            unsigned long long skipped = 0ull;
            int processed = 0;
            if (face && (bits & valid) == valid) {
                skipped = valid;
            } else {
                // ring of prefetched rows and scalars in shared memory (every lane copies and later reads
                // its own bytes, the three scalars included, so no lane waits for another)
                auto fetch = [&](int i, int slot) {
                    const int ii = min(i, len - 1);
                    const size_t th = (size_t)(tok0 + ii) * H + h;
                    RingSlot& rs = ring[slot];
                    cp_async<R * (int)sizeof(TI)>(&rs.k[lane], kp + th * K + R * lane);
                    if constexpr (VEC) cp_async<R * 4>(&rs.lr[VEC ? lane : 0], a.retsrc + th * K + R * lane);
                    cp_async<4>(&rs.n[lane], a.r.n + th);
                    cp_async<4>(&rs.rho[lane], a.r.rho + th);
                    cp_async<4>(&rs.beta[lane], a.beta + th);
                    cp_async_commit();
                };
                int i = 0;
                while (i < len) {
                    if (face) {
                        // jump over the flagged tokens that follow while d stays on the face
                        const unsigned long long rest = (~bits & valid) >> i;
                        const int run = rest ? __ffsll((long long)rest) - 1 : len - i;
                        if (run > 0) {
                            skipped |= (run >= 64 ? ~0ull : ((1ull << run) - 1ull)) << i;
                            i += run;
                            continue;
                        }
                    }
                    // process tokens i, i+1, ... until d is back on the face (or the chunk ends)
                    cp_async_wait<0>();   // nothing of an earlier run is still on its way into the ring
#pragma unroll
                    for (int u = 0; u < PF; ++u) fetch(i + u, u);
                    bool stop = false;
                    while (i < len && !stop) {
#pragma unroll
                        for (int u = 0; u < PF; ++u) {
                            if (i < len && !stop) {
                                cp_async_wait<PF - 1>();   // the oldest group, this token's, has landed
                                const RingSlot& rs = ring[u];
                                float kk[R];
                                unpack<R>(rs.k[lane], kk);
                                const float rn = fabsf(rs.n[lane]), b = hy.beta_aware ? rs.beta[lane] : 1.0f;
                                // c = e - a2 <d, k^2>: e and a2 do not depend on d (1 / n comes from the
                                // parallel pass), so nothing but one multiply-add follows the warp sum
                                const float e = hy.eta * b * rn, a2 = e * b;
                                float rho[R];
                                if constexpr (VEC) {
                                    float lr[R];
                                    unpack<R>(rs.lr[VEC ? lane : 0], lr);
#pragma unroll
                                    for (int r = 0; r < R; ++r) rho[r] = expf(lr[r]);
                                } else {
                                    const float r1 = rs.rho[lane];
#pragma unroll
                                    for (int r = 0; r < R; ++r) rho[r] = r1;
                                }
                                fetch(i + PF, u);
                                const size_t th = (size_t)(tok0 + i) * H + h;
                                float kap[R], wk[R], rd[R], al = 0.f;
#pragma unroll
                                for (int r = 0; r < R; ++r) {
                                    kap[r] = kk[r] * kk[r];
                                    wk[r] = d[r] * kk[r];
                                    rd[r] = rho[r] * d[r];
                                    al = fmaf(d[r], kap[r], al);
                                }
                                al = warp_sum(al);
                                store_row<R>(kt + th * K, lane, wk);
                                if (a.save) store_row<R>(a.r.dtraj + th * K, lane, d);
                                const float cc = fmaf(-a2, al, e);
                                unsigned mybits = 0;         // bit r: the projection passes gradient for coordinate R lane + r
                                bool at_min = hy.clamp != 0;
#pragma unroll
                                for (int r = 0; r < R; ++r) {
                                    float x = fmaf(cc, kap[r], rd[r]);
                                    bool pz = true;
                                    if (hy.clamp) {
                                        pz = (x >= hy.d_min) && (x <= hy.d_max);
                                        x = fminf(fmaxf(x, hy.d_min), hy.d_max);
                                    }
                                    mybits |= pz ? (1u << r) : 0u;
                                    at_min = at_min && (x == hy.d_min);
                                    d[r] = x;
                                }
                                if (a.save) {
                                    a.r.pmask[th * 32 + lane] = mybits;
                                    if (lane == 0) a.r.al[th] = al;
                                }
                                face = __all_sync(0xffffffffu, at_min);
                                ++i;
                                ++processed;
                                // back on the face with a flagged token next: leave the run
                                stop = face && i < len && ((bits >> i) & 1ull);
                            }
                        }
                    }
                }
            }
            if (a.save && lane == 0) {
                a.r.skipw[tile * 2] = (unsigned)(skipped & 0xffffffffull);
                a.r.skipw[tile * 2 + 1] = (unsigned)(skipped >> 32);
            }
            pipe_next = processed >= PIPE_TRIGGER && !face;
        }
    }
    if (a.d_final) store_row<R>(a.d_final + ((size_t)s * H + h) * K, lane, d);
    cp_async_wait<0>();   // rows fetched past the last processed token are not used, but must have landed
    if (lane == 0) {      // release the helper warps
        cmd[0] = 0;
        cmd[1] = 0;
    }
    asm volatile("bar.sync 1, 96;" ::: "memory");
}

// ---------------------------------------------------------------------------------------------
// backward
// ---------------------------------------------------------------------------------------------
struct P1Bwd {
    int S, H, NT;
    Table tab;
    const void* k;
    const float *beta, *dktil, *dkread, *dprecond_out;
    const float* log_ret;   // [T,H,K], vector retention only
    void* dk;
    float *dbeta, *dgate, *dlog_ret, *dprecond_in;
    P1Regions r;
    Hyper hy;
    int* status;
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
    const int len = a.tab.chunk_len(c), tok0 = a.tab.chunk_tok0(c);
    const unsigned word = a.r.skipw[tile * 2 + half];
    T* dkp = static_cast<T*>(a.dk);
    for (int j = 0; j < 32; ++j) {
        const int i = half * 32 + j;
        if (i >= len) break;
        if (!((word >> j) & 1u)) continue;
        const size_t th = (size_t)(tok0 + i) * a.H + h;
        float x[R], y[R];
        load_row<R>(a.dkread + th * K, lane, x);
        load_row<R>(a.dktil + th * K, lane, y);
#pragma unroll
        for (int r = 0; r < R; ++r) x[r] = fmaf(a.hy.d_min, y[r], x[r]);
        store_row<R>(dkp + th * K, lane, x);
    }
}

// ---------------------------------------------------------------------------------------------
// Pipelined stretches of the reverse pass, the mirror image of the forward ones: over chunks in which
// every token was processed, lambda = dL/dd flows without a restart, and of a token's work only
//     lambda <- mask (.) lambda ;  dc = <lambda, k^2> ;  lambda <- rho lambda - a2 dc k^2 + k (.) dL/dktil
// depends on lambda.  Three warps share the chain:
//   pre   fetches a block of QB tokens (k, d_t, dL/dktil, dk_read, mask, scalars) and recomputes the
//         step's own scalars (<d_t, k^2>, c, the factors of the beta and normaliser gradients);
//   core  carries lambda through the block (top token first) and leaves the masked lambda and dc;
//   post  forms dk, the retention and beta gradients from those and writes them out.
// ---------------------------------------------------------------------------------------------
// Five buffers: the pre role holds two (one landing, one being finished), core and post one each, one spare.
constexpr int QB = 8, QN = 5;
static_assert(QN <= RING_MAX && PN <= RING_MAX, "barrier arrays");

template <typename T, int K, bool VEC> struct RevBuf {
    static constexpr int R = K / 32;
    RawRow<T, R> kraw[QB][32];
    float dt[QB][K], dkt[QB][K], dkr[QB][K];
    float lam[QB][K];                       // lambda on entry to the token (before the mask), written by the core
    // what the core reads, prepared by the pre role so that nothing but the recurrence is left to the core:
    float kap[QB][K], mkap[QB][K];          // k^2, and k^2 where the projection passed (else 0)
    float rm[QB][K];                        // retention where the projection passed (else 0)
    float w[QB][K];                         // k (.) dL/dktil
    float rv[VEC ? QB : 1][VEC ? K : 1];    // vector retention: exp(l_t)
    unsigned mask[QB][32];
    float4 sc0[QB];                         // a2, rho, cc, g1
    float4 sc1[QB];                         // g2, dc (written by the core), -, -
    float raw[4][QB];                       // n (signed), rho, beta, <d_t, k^2> as they sit in memory
};

// tokens [t_lo, t_hi) of the chain in reverse, all three roles; lam: the core's registers
template <typename T, int K, bool VEC>
__device__ __forceinline__ bool rev_stretch(const P1Bwd& a, int h, int t_lo, int t_hi, float (&lam)[K / 32],
                                            RevBuf<T, K, VEC>* buf, PipeBars& bars, uint32_t& round0, int role, int lane)
{
    constexpr int R = K / 32;
    const int H = a.H;
    const Hyper hy = a.hy;
    const int nblk = (t_hi - t_lo + QB - 1) / QB;
    const T* kp = static_cast<const T*>(a.k);
    bool ok = true;
    const uint32_t base = round0;
    // block b: tokens t_hi - 1 - (b QB + j), j = 0 .. n - 1 (slot j of the buffer)
    if (role == 1) {
        // Rows go straight into the buffer with cp.async (nothing of them is converted here), one committed
        // group per block and one block ahead: while block b is on its way, block b - 1 is finished (the
        // step's own scalars formed from the raw ones, the retention vector exponentiated) and handed over.
        auto finish = [&](int b) {
            const uint32_t use = base + b;
            const int bi = use % QN;
            RevBuf<T, K, VEC>& B = buf[bi];
            const int ttop = t_hi - 1 - b * QB, n = min(QB, ttop - t_lo + 1);
            if (lane < n) {
                const float ns = B.raw[0][lane], rho = B.raw[1][lane], alv = B.raw[3][lane];
                const float bb = hy.beta_aware ? B.raw[2][lane] : 1.0f;
                const float rn = fabsf(ns);
                const float e = hy.eta * bb * rn, a2 = e * bb;
                const float cc = fmaf(-a2, alv, e);
                const float g1 = hy.eta * (1.0f - 2.0f * bb * alv) * rn;
                const float g2 = ns > 0.f ? -cc * rn : 0.f;
                B.sc0[lane] = make_float4(a2, rho, cc, g1);
                B.sc1[lane].x = g2;
            }
            if constexpr (VEC) {
                for (int j = 0; j < n; ++j) {
                    float lr[R];
                    load_row<R>(B.rv[VEC ? j : 0], lane, lr);
#pragma unroll
                    for (int r = 0; r < R; ++r) lr[r] = expf(lr[r]);
                    store_row<R>(B.rv[VEC ? j : 0], lane, lr);
                }
            }
#pragma unroll 4
            for (int j = 0; j < QB; ++j) {   // (slots beyond n repeat the last token: harmless)
                float kk[R], dkt[R], kap[R], mkap[R], rm[R], w[R], rv[R];
                unpack<R>(B.kraw[j][lane], kk);
                load_row<R>(B.dkt[j], lane, dkt);
                const unsigned mw = B.mask[j][lane];
                if constexpr (VEC) load_row<R>(B.rv[VEC ? j : 0], lane, rv);
                else {
                    const float rho = B.raw[1][min(j, n - 1)];
#pragma unroll
                    for (int r = 0; r < R; ++r) rv[r] = rho;
                }
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const bool pass = (mw >> r) & 1u;
                    kap[r] = kk[r] * kk[r];
                    mkap[r] = pass ? kap[r] : 0.f;
                    rm[r] = pass ? rv[r] : 0.f;
                    w[r] = kk[r] * dkt[r];
                }
                store_row<R>(B.kap[j], lane, kap);
                store_row<R>(B.mkap[j], lane, mkap);
                store_row<R>(B.rm[j], lane, rm);
                store_row<R>(B.w[j], lane, w);
            }
            __syncwarp();
            if (lane == 0) p1_mbar_arrive(&bars.full[bi]);
        };
        for (int b = 0; b < nblk && ok; ++b) {
            const uint32_t use = base + b;
            const int bi = use % QN;
            if (use >= QN) ok = p1_mbar_wait(&bars.free_[bi], ((use / QN) - 1) & 1, a.status);
            if (!ok) break;
            RevBuf<T, K, VEC>& B = buf[bi];
            const int ttop = t_hi - 1 - b * QB, n = min(QB, ttop - t_lo + 1);
#pragma unroll
            for (int j = 0; j < QB; ++j) {
                const size_t th = (size_t)(ttop - min(j, n - 1)) * H + h;
                cp_async<R * (int)sizeof(T)>(&B.kraw[j][lane], kp + th * K + R * lane);
                cp_async<R * 4>(&B.dt[j][R * lane], a.r.dtraj + th * K + R * lane);
                cp_async<R * 4>(&B.dkt[j][R * lane], a.dktil + th * K + R * lane);
                cp_async<R * 4>(&B.dkr[j][R * lane], a.dkread + th * K + R * lane);
                cp_async<4>(&B.mask[j][lane], a.r.pmask + th * 32 + lane);
                if constexpr (VEC) cp_async<R * 4>(&B.rv[VEC ? j : 0][R * lane], a.log_ret + th * K + R * lane);
            }
            if (lane < n) {
                const size_t th = (size_t)(ttop - lane) * H + h;
                cp_async<4>(&B.raw[0][lane], a.r.n + th);
                cp_async<4>(&B.raw[1][lane], a.r.rho + th);
                cp_async<4>(&B.raw[2][lane], a.beta + th);
                cp_async<4>(&B.raw[3][lane], a.r.al + th);
            }
            cp_async_commit();
            if (b > 0) {
                cp_async_wait<1>();   // block b - 1 has landed
                __syncwarp();
                finish(b - 1);
            }
        }
        cp_async_wait<0>();
        __syncwarp();
        if (ok && nblk > 0) finish(nblk - 1);
    } else if (role == 0) {
        for (int b = 0; b < nblk && ok; ++b) {
            const uint32_t use = base + b;
            const int bi = use % QN;
            ok = p1_mbar_wait(&bars.full[bi], (use / QN) & 1, a.status);
            if (!ok) break;
            RevBuf<T, K, VEC>& B = buf[bi];
            const int ttop = t_hi - 1 - b * QB, n = min(QB, ttop - t_lo + 1);
            auto token = [&](int j) {
                const float a2 = B.sc0[j].x;
                float kap[R], mkap[R], rm[R], w[R];
                load_row<R>(B.mkap[j], lane, mkap);
                load_row<R>(B.kap[j], lane, kap);
                load_row<R>(B.rm[j], lane, rm);
                load_row<R>(B.w[j], lane, w);
                float dc0 = lam[0] * mkap[0], dc1 = lam[1] * mkap[1];
#pragma unroll
                for (int r = 2; r < R; r += 2) {
                    dc0 = fmaf(lam[r], mkap[r], dc0);
                    dc1 = fmaf(lam[r + 1], mkap[r + 1], dc1);
                }
                store_row<R>(B.lam[j], lane, lam);
                const float dc = warp_sum(dc0 + dc1);
                const float da = -a2 * dc;
#pragma unroll
                for (int r = 0; r < R; ++r) lam[r] = fmaf(rm[r], lam[r], fmaf(da, kap[r], w[r]));
                if (lane == 0) B.sc1[j].y = dc;
            };
            if (n == QB) {
#pragma unroll
                for (int j = 0; j < QB; ++j) token(j);
            } else {
                for (int j = 0; j < n; ++j) token(j);
            }
            __syncwarp();
            if (lane == 0) p1_mbar_arrive(&bars.done[bi]);
        }
    } else {
        T* dkp = static_cast<T*>(a.dk);
        for (int b = 0; b < nblk && ok; ++b) {
            const uint32_t use = base + b;
            const int bi = use % QN;
            ok = p1_mbar_wait(&bars.done[bi], (use / QN) & 1, a.status);
            if (!ok) break;
            const RevBuf<T, K, VEC>& B = buf[bi];
            const int ttop = t_hi - 1 - b * QB, n = min(QB, ttop - t_lo + 1);
            // <lambda, d_t> of the block's tokens first, all slots at once: the shuffle rounds of the eight
            // sums overlap instead of following one another
            float drv[QB];
#pragma unroll
            for (int j = 0; j < QB; ++j) {
                float dt[R], lm[R];
                load_row<R>(B.dt[j], lane, dt);
                load_row<R>(B.lam[j], lane, lm);
                const unsigned mw = B.mask[j][lane];
                drv[j] = 0.f;
#pragma unroll
                for (int r = 0; r < R; ++r) drv[j] = fmaf((mw >> r) & 1u ? lm[r] : 0.f, dt[r], drv[j]);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int j = 0; j < QB; ++j) drv[j] += __shfl_xor_sync(0xffffffffu, drv[j], o);
            // the per-token scalars (beta and retention gradients): lane j takes token j
            {
                float mine = 0.f;
#pragma unroll
                for (int j = 0; j < QB; ++j) mine = lane == j ? drv[j] : mine;
                if (lane < n) {
                    const size_t th = (size_t)(ttop - lane) * H + h;
                    const float4 s0 = B.sc0[lane];
                    const float dc = B.sc1[lane].y;
                    if (hy.beta_aware) atomicAdd(&a.dbeta[th], s0.w * dc);
                    if (hy.apf_mode == 1) atomicAdd(&a.dgate[th], s0.y * mine);
                    if (hy.apf_mode == 2 && a.dlog_ret) a.dlog_ret[th] = s0.y * mine;
                }
            }
            auto token = [&](int j) {
                const size_t th = (size_t)(ttop - j) * H + h;
                const float4 s0 = B.sc0[j], s1 = B.sc1[j];
                const float a2 = s0.x, cc = s0.z, g2 = s1.x, dc = s1.y;
                float kk[R], dt[R], dkt[R], dkr[R], lm[R];
                unpack<R>(B.kraw[j][lane], kk);
                load_row<R>(B.dt[j], lane, dt);
                load_row<R>(B.dkt[j], lane, dkt);
                load_row<R>(B.dkr[j], lane, dkr);
                load_row<R>(B.lam[j], lane, lm);
                {
                    const unsigned mw = B.mask[j][lane];
#pragma unroll
                    for (int r = 0; r < R; ++r) lm[r] = (mw >> r) & 1u ? lm[r] : 0.f;
                }
                const float da = -a2 * dc, dn = g2 * dc;
                if constexpr (VEC) {
                    if (a.dlog_ret) {
                        float rv[R], dl[R];
                        load_row<R>(B.rv[VEC ? j : 0], lane, rv);
#pragma unroll
                        for (int r = 0; r < R; ++r) dl[r] = rv[r] * lm[r] * dt[r];
                        store_row<R>(a.dlog_ret + th * K, lane, dl);
                    }
                }
                float out[R];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const float dkap = cc * lm[r] + da * dt[r] + dn;
                    out[r] = dkr[r] + dt[r] * dkt[r] + 2.0f * kk[r] * dkap;
                }
                store_row<R>(dkp + th * K, lane, out);
            };
            if (n == QB) {   // unrolled without a branch between the tokens: their reads and products interleave
#pragma unroll
                for (int j = 0; j < QB; ++j) token(j);
            } else {
                for (int j = 0; j < n; ++j) token(j);
            }
            __syncwarp();
            if (lane == 0) p1_mbar_arrive(&bars.free_[bi]);
        }
    }
    round0 = base + nblk;
    return ok;
}

// processed tokens, in reverse; one chain per CTA: warp 0 walks the chain, warps 1 and 2 serve its
// pipelined stretches.  Skip words are fetched for 32 chunks at a time.

template <typename T, int K, bool VEC>
__global__ void __launch_bounds__(96) phase1_bwd_seq_kernel(P1Bwd a)
{
    constexpr int R = K / 32;
    constexpr int PF = 4;   // prefetch distance in processed tokens
    // ring of prefetched rows and scalars (cp.async; every lane copies and later reads its own bytes)
    struct BSlot {
        RawRow<T, R> k[32], sk_k[32];
        RawRow<float, R> dt[32], dkt[32], dkr[32], sk_t[32], lr[VEC ? 32 : 1];
        unsigned m[32];
        float n[32], rho[32], beta[32], al[32];
    };
    extern __shared__ __align__(16) uint8_t p1_dyn[];   // RevBuf[QN]
    RevBuf<T, K, VEC>* rbuf = reinterpret_cast<RevBuf<T, K, VEC>*>(p1_dyn);
    __shared__ __align__(16) BSlot ring[PF];
    __shared__ PipeBars bars;
    __shared__ int cmd[2];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chain = blockIdx.x;
    const int s = chain / a.H, h = chain % a.H, H = a.H;
    const Hyper hy = a.hy;
    const T* kp = static_cast<const T*>(a.k);
    T* dkp = static_cast<T*>(a.dk);
    if (threadIdx.x == 0) {
        for (int i = 0; i < QN; ++i) {
            p1_mbar_init(&bars.full[i], 1);
            p1_mbar_init(&bars.done[i], 1);
            p1_mbar_init(&bars.free_[i], 1);
        }
    }
    __syncthreads();
    uint32_t pipe_uses = 0;
    if (warp != 0) {
        float none[R];
        while (true) {
            asm volatile("bar.sync 1, 96;" ::: "memory");
            const int t_lo = cmd[0], t_hi = cmd[1];
            if (t_hi <= t_lo) break;
            rev_stretch<T, K, VEC>(a, h, t_lo, t_hi, none, rbuf, bars, pipe_uses, warp, lane);
            asm volatile("bar.sync 2, 96;" ::: "memory");
        }
        return;
    }
    float lam[R];
    if (a.dprecond_out) load_row<R>(a.dprecond_out + ((size_t)s * H + h) * K, lane, lam);
    else {
#pragma unroll
        for (int r = 0; r < R; ++r) lam[r] = 0.f;
    }
    bool lam_valid = true;     // lam holds dL/dd_{t+1} for the token about to be processed
    long src = -1;             // otherwise it is k (.) dktil of this (skipped) token
    auto restart = [&](long tsrc) {
        const size_t ts = (size_t)tsrc * H + h;
        float kk[R], dk[R];
        load_row<R>(kp + ts * K, lane, kk);
        load_row<R>(a.dktil + ts * K, lane, dk);
#pragma unroll
        for (int r = 0; r < R; ++r) lam[r] = kk[r] * dk[r];
    };
    const int c0 = a.tab.seq_chunk0(s), c1 = a.tab.seq_chunk0(s + 1);
    const int seq_t0 = a.tab.seq_tok0(s), seq_len = a.tab.seq_len(s);
    for (int ctop = c1; ctop > c0; ctop -= 32) {
        // lane j holds the words of chunk ctop - 1 - j
        unsigned w0 = 0, w1 = 0;
        if (ctop - 1 - lane >= c0) {
            const size_t tl = (size_t)(ctop - 1 - lane) * H + h;
            w0 = a.r.skipw[tl * 2];
            w1 = a.r.skipw[tl * 2 + 1];
            // Sparse work (a few processed tokens per chunk): each lane warms L2 with the rows its
            // chunk's tokens will need, long before the sequential walk gets there.  These rows sit in
            // large arrays that were last touched several kernels ago; a cold access costs microseconds.
            const int cl = ctop - 1 - lane;
            const int lenl = min(CH, seq_len - (cl - c0) * CH);
            unsigned long long m = ~((unsigned long long)w0 | ((unsigned long long)w1 << 32)) &
                                   (lenl >= 64 ? ~0ull : ((1ull << lenl) - 1ull));
            if (__popcll(m) <= 16) {
                while (m) {
                    const int t = __ffsll((long long)m) - 1;
                    m &= m - 1;
                    const size_t th = (size_t)(seq_t0 + (cl - c0) * CH + t) * H + h;
                    prefetch_row(kp + th * K, K * (int)sizeof(T));
                    prefetch_row(a.r.dtraj + th * K, K * 4);
                    prefetch_row(a.dktil + th * K, K * 4);
                    prefetch_row(a.dkread + th * K, K * 4);
                    if constexpr (VEC) prefetch_row(a.log_ret + th * K, K * 4);
                    prefetch_l2(a.r.pmask + th * 32);
                    prefetch_l2(a.r.n + th);
                    prefetch_l2(a.r.rho + th);
                    prefetch_l2(a.beta + th);
                    if (t + 1 < lenl) {   // rows a restart above this token would read
                        prefetch_row(kp + (th + H) * K, K * (int)sizeof(T));
                        prefetch_row(a.dktil + (th + H) * K, K * 4);
                    }
                }
            }
        }
        const int cbot = max(ctop - 32, c0);
        for (int c = ctop - 1; c >= cbot; --c) {
            const int nrel = c - c0;
            const int tok0 = seq_t0 + nrel * CH, len = min(CH, seq_len - nrel * CH);
            const unsigned long long sk = (unsigned long long)__shfl_sync(0xffffffffu, w0, ctop - 1 - c) |
                                          ((unsigned long long)__shfl_sync(0xffffffffu, w1, ctop - 1 - c) << 32);
            const unsigned long long valid = len >= 64 ? ~0ull : ((1ull << len) - 1ull);
            if ((sk & valid) == valid) {
                lam_valid = false;
                src = tok0;
                continue;
            }
            if ((sk & valid) == 0ull) {
                // every token of the chunk was processed: a pipelined stretch over this chunk and the ones
                // below it of which the same holds (within this group of skip words, at most PIPE_CHUNKS)
                int np = 1;
                while (np < PIPE_CHUNKS && c - np >= cbot) {
                    const int cc2 = c - np;
                    const unsigned long long s2 = (unsigned long long)__shfl_sync(0xffffffffu, w0, ctop - 1 - cc2) |
                                                  ((unsigned long long)__shfl_sync(0xffffffffu, w1, ctop - 1 - cc2) << 32);
                    if (s2 != 0ull) break;   // chunks below the top one of a sequence are full
                    ++np;
                }
                const int t_hi = tok0 + len, t_lo = seq_t0 + (nrel - (np - 1)) * CH;
                if (!lam_valid) restart(src);
                if (lane == 0) {
                    cmd[0] = t_lo;
                    cmd[1] = t_hi;
                }
                cp_async_wait<0>();
                asm volatile("bar.sync 1, 96;" ::: "memory");
                rev_stretch<T, K, VEC>(a, h, t_lo, t_hi, lam, rbuf, bars, pipe_uses, 0, lane);
                asm volatile("bar.sync 2, 96;" ::: "memory");
                lam_valid = true;
                c -= np - 1;
                continue;
            }
            // The tokens to process are known up front (the clear bits of the skip word), so the rows of
            // the next PF of them are always in flight, across runs of skipped tokens.  Where the
            // recurrence restarts before a token (its upper neighbour was skipped), the two rows the
            // restart needs travel with that token's rows.
            const unsigned long long todo = ~sk & valid;
            const bool valid_in = lam_valid;
            const long src_in = src;
            auto pop_top = [](unsigned long long& m) {
                const int t = 63 - __clzll((long long)m);
                m &= ~(1ull << t);
                return t;
            };
            // one committed group per ring slot use (an empty one when nothing is left to fetch), so
            // that "all but the PF - 1 most recent groups" is always the slot about to be read
            auto fetch = [&](int i, int slot) {
                const size_t th = (size_t)(tok0 + i) * H + h;
                BSlot& rs = ring[slot];
                cp_async<R * (int)sizeof(T)>(&rs.k[lane], kp + th * K + R * lane);
                cp_async<R * 4>(&rs.dt[lane], a.r.dtraj + th * K + R * lane);
                cp_async<R * 4>(&rs.dkt[lane], a.dktil + th * K + R * lane);
                cp_async<R * 4>(&rs.dkr[lane], a.dkread + th * K + R * lane);
                if constexpr (VEC) cp_async<R * 4>(&rs.lr[VEC ? lane : 0], a.log_ret + th * K + R * lane);
                cp_async<4>(&rs.m[lane], a.r.pmask + th * 32 + lane);
                cp_async<4>(&rs.n[lane], a.r.n + th);
                cp_async<4>(&rs.rho[lane], a.r.rho + th);
                cp_async<4>(&rs.beta[lane], a.beta + th);
                cp_async<4>(&rs.al[lane], a.r.al + th);
                const bool top = i == len - 1;
                const bool need = top ? !valid_in : (((sk >> (i + 1)) & 1ull) != 0ull);
                if (need) {   // lambda restarts at the lowest token of the skipped run above
                    const size_t ts = (size_t)(top ? src_in : (long)(tok0 + i + 1)) * H + h;
                    cp_async<R * (int)sizeof(T)>(&rs.sk_k[lane], kp + ts * K + R * lane);
                    cp_async<R * 4>(&rs.sk_t[lane], a.dktil + ts * K + R * lane);
                }
                cp_async_commit();
                return need;
            };
            bool needr[PF];
            unsigned long long pfm = todo, rem = todo;
            cp_async_wait<0>();
#pragma unroll
            for (int u = 0; u < PF; ++u) {
                needr[u] = false;
                if (pfm) needr[u] = fetch(pop_top(pfm), u);
                else cp_async_commit();
            }
            while (rem) {
#pragma unroll
                for (int u = 0; u < PF; ++u) {
                    if (rem) {
                        const int i = pop_top(rem);
                        cp_async_wait<PF - 1>();
                        const BSlot& rs = ring[u];
                        float kk[R], kap[R], dt[R], dkt[R], dkr[R], drho = 0.f, dc = 0.f, al = 0.f;
                        unpack<R>(rs.k[lane], kk);
                        unpack<R>(rs.dt[lane], dt);
                        unpack<R>(rs.dkt[lane], dkt);
                        unpack<R>(rs.dkr[lane], dkr);
                        if (needr[u]) {
                            float rk[R], rt[R];
                            unpack<R>(rs.sk_k[lane], rk);
                            unpack<R>(rs.sk_t[lane], rt);
#pragma unroll
                            for (int r = 0; r < R; ++r) lam[r] = rk[r] * rt[r];
                        }
                        const unsigned mw = rs.m[lane];
                        const float ns = rs.n[lane], rn = fabsf(ns), rho = rs.rho[lane];
                        const float b = hy.beta_aware ? rs.beta[lane] : 1.0f;
                        float rv[R];
                        if constexpr (VEC) {
                            float lr[R];
                            unpack<R>(rs.lr[VEC ? lane : 0], lr);
#pragma unroll
                            for (int r = 0; r < R; ++r) rv[r] = expf(lr[r]);
                        } else {
#pragma unroll
                            for (int r = 0; r < R; ++r) rv[r] = rho;
                        }
                        if (pfm) needr[u] = fetch(pop_top(pfm), u);
                        else cp_async_commit();
                        const size_t th = (size_t)(tok0 + i) * H + h;
                        // what does not depend on lambda first: the step's own scalars (<d_t, k^2> was
                        // recorded by the forward pass)
#pragma unroll
                        for (int r = 0; r < R; ++r) kap[r] = kk[r] * kk[r];
                        al = rs.al[lane];
                        const float e = hy.eta * b * rn, a2 = e * b;
                        const float cc = fmaf(-a2, al, e);
                        const float g1 = hy.eta * (1.0f - 2.0f * b * al) * rn;
                        const float g2 = ns > 0.f ? -cc * rn : 0.f;
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            if (!((mw >> r) & 1u)) lam[r] = 0.f;
                            drho = fmaf(lam[r], dt[r], drho);
                            dc = fmaf(lam[r], kap[r], dc);
                        }
                        dc = warp_sum(dc);
                        drho = warp_sum(drho);
                        const float da = -a2 * dc, dbt = g1 * dc, dn = g2 * dc;
                        float out[R];
                        if constexpr (VEC) {   // one gradient per coordinate: r_i lambda_i d_i
                            if (a.dlog_ret) {
                                float dl[R];
#pragma unroll
                                for (int r = 0; r < R; ++r) dl[r] = rv[r] * lam[r] * dt[r];
                                store_row<R>(a.dlog_ret + th * K, lane, dl);
                            }
                        }
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            const float dkap = cc * lam[r] + da * dt[r] + dn;
                            out[r] = dkr[r] + dt[r] * dkt[r] + 2.0f * kk[r] * dkap;
                            lam[r] = rv[r] * lam[r] + da * kap[r] + kk[r] * dkt[r];
                        }
                        store_row<R>(dkp + th * K, lane, out);
                        if (lane == 0) {
                            // added on top of what the chunk-local backward wrote; as reductions
                            // without a return value, so that the sweep does not wait for memory
                            if (hy.beta_aware) atomicAdd(&a.dbeta[th], dbt);
                            if (hy.apf_mode == 1) atomicAdd(&a.dgate[th], rho * drho);
                            if (hy.apf_mode == 2 && a.dlog_ret) a.dlog_ret[th] = rho * drho;
                        }
                    }
                }
            }
            // state handed to the chunk below: lambda is live iff the chunk's first token was processed
            lam_valid = (todo & 1ull) != 0ull;
            if (!lam_valid) src = tok0;
        }
    }
    if (a.dprecond_in) {
        if (!lam_valid) restart(src);
        store_row<R>(a.dprecond_in + ((size_t)s * H + h) * K, lane, lam);
    }
    cp_async_wait<0>();
    if (lane == 0) {   // release the helper warps
        cmd[0] = 0;
        cmd[1] = 0;
    }
    asm volatile("bar.sync 1, 96;" ::: "memory");
}

template <typename TI, typename TO, int K>
int fwd_launch(const P1Fwd& a, cudaStream_t st)
{
    const long warps = (long)a.NT * a.H * 2;
    const unsigned gspec = (unsigned)((warps + 3) / 4), gseq = (unsigned)((a.S * a.H + 3) / 4);
    stage_mark(st, "phase1_spec");
    if (a.hy.apf_mode == 3) phase1_spec_kernel<TI, TO, K, true><<<gspec, 128, 0, st>>>(a);
    else phase1_spec_kernel<TI, TO, K, false><<<gspec, 128, 0, st>>>(a);
    stage_mark(st, "phase1_seq");
    const unsigned chains = (unsigned)(a.S * a.H);
    auto launch_seq = [&](auto kernel, size_t smem) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        kernel<<<chains, 96, smem, st>>>(a);
        return true;
    };
    const bool okl = a.hy.apf_mode == 3 ? launch_seq(phase1_seq_kernel<TI, TO, K, true>, PN * sizeof(PipeBuf<TI, K, true>))
                                        : launch_seq(phase1_seq_kernel<TI, TO, K, false>, PN * sizeof(PipeBuf<TI, K, false>));
    if (!okl) return -1;
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
    const unsigned chains = (unsigned)(a.S * a.H);
    auto launch_seq = [&](auto kernel, size_t smem) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        kernel<<<chains, 96, smem, st>>>(a);
        return true;
    };
    if (!(a.hy.apf_mode == 3 ? launch_seq(phase1_bwd_seq_kernel<T, K, true>, QN * sizeof(RevBuf<T, K, true>))
                             : launch_seq(phase1_bwd_seq_kernel<T, K, false>, QN * sizeof(RevBuf<T, K, false>))))
        return -1;
    ++n;
    return cudaGetLastError() == cudaSuccess ? n : -1;
}

}  // namespace

int phase1_forward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                   void* ktil, bool ktil_bf16, bool save, cudaStream_t st)
{
    P1Fwd f{};
    f.S = L.S; f.H = p.H; f.NT = L.NTmax; f.tab = carve_table(ws, L);
    f.k = a.k; f.beta = a.beta; f.retsrc = p.apf_mode >= 2 ? a.log_ret : a.gate; f.d0 = a.precond_in;
    f.ktil = ktil; f.d_final = a.precond_out; f.r = carve_p1(ws, L); f.save = save ? 1 : 0; f.hy = hy;
    f.status = reinterpret_cast<int*>(static_cast<char*>(ws) + L.status);
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
    b.r = carve_p1(ws, L); b.hy = hy; b.log_ret = a.log_ret;
    b.status = reinterpret_cast<int*>(static_cast<char*>(ws) + L.status);
    // retention gradients are written for processed tokens only; a skipped token (projection mask all
    // zero) has none
    if (p.apf_mode >= 2 && a.dlog_ret) {
        const size_t Ttot = p.nseq > 0 ? (size_t)p.T : (size_t)p.B * p.T;
        const size_t nb = Ttot * p.H * (p.apf_mode == 3 ? (size_t)p.K : 1) * sizeof(float);
        if (cudaMemsetAsync(a.dlog_ret, 0, nb, st) != cudaSuccess) return -1;
    }
    if (p.io_dtype == OSDN_FP32)
        return p.K == 64 ? bwd_launch<float, 64>(b, bulk, st) : bwd_launch<float, 128>(b, bulk, st);
    return p.K == 64 ? bwd_launch<__nv_bfloat16, 64>(b, bulk, st) : bwd_launch<__nv_bfloat16, 128>(b, bulk, st);
}

int phase1_update(const osdn_params& p, const Hyper& hy, const void* k, const float* beta, const float* retsrc,
                  const float* precond_in, void* ktil_out, float* precond_out, float* ratio_out,
                  float* log_sum_out, cudaStream_t st)
{
    P1Args pa{};
    pa.S = p.nseq > 0 ? p.nseq : p.B;
    pa.H = p.H; pa.T_dense = p.T; pa.cu = p.nseq > 0 ? p.cu_seqlens : nullptr;
    pa.k = k; pa.beta = beta; pa.retsrc = retsrc; pa.d0 = precond_in; pa.ktil = ktil_out;
    pa.d_final = precond_out; pa.ratio = ratio_out; pa.log_sum = log_sum_out; pa.hy = hy;
    const unsigned chains = (unsigned)(pa.S * pa.H);
    stage_mark(st, "phase1_stream");
    const bool vec = hy.apf_mode == 3;
    auto launch = [&](auto kernel, size_t buf_bytes) {
        const size_t smem = PN * buf_bytes + PN * PB * sizeof(float);
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        kernel<<<chains, 96, smem, st>>>(pa);
        return true;
    };
    bool ok;
    if (p.io_dtype == OSDN_FP32) {
        if (p.K == 64)
            ok = vec ? launch(phase1_stream_kernel<float, float, 64, true>, sizeof(PipeBuf<float, 64, true>))
                     : launch(phase1_stream_kernel<float, float, 64, false>, sizeof(PipeBuf<float, 64, false>));
        else
            ok = vec ? launch(phase1_stream_kernel<float, float, 128, true>, sizeof(PipeBuf<float, 128, true>))
                     : launch(phase1_stream_kernel<float, float, 128, false>, sizeof(PipeBuf<float, 128, false>));
    } else {
        using B16 = __nv_bfloat16;
        if (p.K == 64)
            ok = vec ? launch(phase1_stream_kernel<B16, B16, 64, true>, sizeof(PipeBuf<B16, 64, true>))
                     : launch(phase1_stream_kernel<B16, B16, 64, false>, sizeof(PipeBuf<B16, 64, false>));
        else
            ok = vec ? launch(phase1_stream_kernel<B16, B16, 128, true>, sizeof(PipeBuf<B16, 128, true>))
                     : launch(phase1_stream_kernel<B16, B16, 128, false>, sizeof(PipeBuf<B16, 128, false>));
    }
    if (!ok) return -1;
    stage_end(st);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace osdn
