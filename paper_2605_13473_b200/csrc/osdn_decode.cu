// Recurrent (decode) step of the layer: the gate, the preconditioner update and the rank-1
// delta-rule write for a few tokens in one launch, on a state and a preconditioner that live in the
// caller's cache (the paper's "Single-token recurrence kernel for OSGDN", for q_len <= 64).
//
//   alpha_t = exp(g_t)
//   ktil_t  = d_t (.) k_t                               (write key from the PRE-update d)
//   d_{t+1} = clip(rho_t d_t + c_t k_t^2)                c_t = eta b_t (1 - b_t <d_t, k_t^2>) / max(|k_t|^2, eps)
//             (rho_t a scalar, or one retention per coordinate in the vector-retention mode)
//   S_t     = alpha_t S_{t-1} + beta_t (v_t - alpha_t S_{t-1} k_t) ktil_t^T ,   o_t = scale S_t q_t
//
// exactly the recurrence the chunk path evaluates chunk by chunk, so that a prefill with osdn_fwd
// followed by osdn_decode_step continues the same sequence.
//
// The work is bound by reading and writing the state once (V x K fp32 per chain).  Rows of S are
// independent, so a chain is cut into V / 16 slices of 16 rows, one CTA each (4 warps x 4 rows); every
// CTA repeats the tiny preconditioner update for its own use and slice 0 stores it.  The slices of a
// chain form one thread-block cluster: the preconditioner is updated in place, so slice 0 may only
// store the advanced vector once every slice of the chain has read the old one; a cluster barrier
// (arrive after the read, wait before the store) gives exactly that order within the one launch,
// however many waves the grid takes.  Lane l of a warp owns the R = K / 32 consecutive columns
// R l .. R l + R - 1 of its rows (one vector access per row), the rows stay in registers over all
// tokens of the call.
#include "osdn_common.cuh"

namespace osdn {

namespace {

constexpr int DEC_RW = 4;        // rows per warp
constexpr int DEC_WARPS = 4;     // warps per CTA
constexpr int DEC_VB = DEC_RW * DEC_WARPS;

struct DecArgs {
    int B, L, H;
    const void *q, *k, *v;
    const float *beta, *gate, *log_ret;
    float *state, *precond;
    void* out;
    Hyper hy;
};

__device__ __forceinline__ float dec_warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

template <int R> __device__ __forceinline__ void dec_load(const float* p, int lane, float (&x)[R])
{
    if constexpr (R == 4) {
        const float4 t = *reinterpret_cast<const float4*>(p + 4 * lane);
        x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
    } else {
        const float2 t = *reinterpret_cast<const float2*>(p + 2 * lane);
        x[0] = t.x; x[1] = t.y;
    }
}
template <int R> __device__ __forceinline__ void dec_load(const __nv_bfloat16* p, int lane, float (&x)[R])
{
    if constexpr (R == 4) {
        const uint2 t = *reinterpret_cast<const uint2*>(p + 4 * lane);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&t.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&t.y));
        x[0] = a.x; x[1] = a.y; x[2] = b.x; x[3] = b.y;
    } else {
        const uint32_t t = *reinterpret_cast<const uint32_t*>(p + 2 * lane);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&t));
        x[0] = a.x; x[1] = a.y;
    }
}
template <int R> __device__ __forceinline__ void dec_store(float* p, int lane, const float (&x)[R])
{
    if constexpr (R == 4) *reinterpret_cast<float4*>(p + 4 * lane) = make_float4(x[0], x[1], x[2], x[3]);
    else *reinterpret_cast<float2*>(p + 2 * lane) = make_float2(x[0], x[1]);
}

// VEC: vector retention (one log-retention per coordinate, log_ret [B,T,H,K]).
template <typename T, int K, int V, bool VEC>
__global__ void __launch_bounds__(DEC_WARPS * 32) decode_kernel(DecArgs a)
{
    constexpr int R = K / 32;
    constexpr int SLICES = V / DEC_VB;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chain = blockIdx.x / SLICES, slice = blockIdx.x % SLICES;
    const int b = chain / a.H, h = chain % a.H;
    const int v0 = slice * DEC_VB + warp * DEC_RW;
    const Hyper hy = a.hy;
    const T* qp = static_cast<const T*>(a.q);
    const T* kp = static_cast<const T*>(a.k);
    const T* vp = static_cast<const T*>(a.v);
    T* op = static_cast<T*>(a.out);

    float S[DEC_RW][R], d[R];
    float* srow = a.state + ((size_t)chain * V + v0) * K;
    dec_load<R>(a.precond + (size_t)chain * K, lane, d);
#pragma unroll
    for (int r = 0; r < DEC_RW; ++r) dec_load<R>(srow + (size_t)r * K, lane, S[r]);
    // This slice has read the chain's preconditioner: the arrival takes the loaded values as an operand, so
    // it cannot issue before they have come back, and a load that has returned cannot see a later store.
    // (A releasing arrival would also wait for the state rows, which are still in flight here.)
    {
        float seen = d[0];
#pragma unroll
        for (int j = 1; j < R; ++j) seen += d[j];
        asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::"f"(seen) : "memory");
    }

    // inputs of a token, fetched one token ahead
    float kk[R], qq[R], vv[DEC_RW], bt, gt, lr, lrv[VEC ? R : 1];
    auto fetch = [&](int t) {
        const size_t th = ((size_t)b * a.L + t) * a.H + h;
        dec_load<R>(kp + th * K, lane, kk);
        dec_load<R>(qp + th * K, lane, qq);
#pragma unroll
        for (int r = 0; r < DEC_RW; ++r) vv[r] = ldf(vp + th * V + v0 + r);
        bt = a.beta[th];
        gt = a.gate[th];
        lr = hy.apf_mode == 2 ? a.log_ret[th] : 0.f;
        if constexpr (VEC) dec_load<R>(a.log_ret + th * K, lane, lrv);   // one log-retention per coordinate
    };
    fetch(0);
    for (int t = 0; t < a.L; ++t) {
        float k1[R], q1[R], v1[DEC_RW];
#pragma unroll
        for (int j = 0; j < R; ++j) { k1[j] = kk[j]; q1[j] = qq[j]; }
#pragma unroll
        for (int r = 0; r < DEC_RW; ++r) v1[r] = vv[r];
        const float beta = bt, alpha = expf(gt);
        const float rho1 = hy.apf_mode == 0 ? 1.0f : (hy.apf_mode == 1 ? alpha : expf(lr));
        float rho[R];
#pragma unroll
        for (int j = 0; j < R; ++j) {
            if constexpr (VEC) rho[j] = expf(lrv[j]);
            else rho[j] = rho1;
        }
        if (t + 1 < a.L) fetch(t + 1);

        // preconditioner step
        float kap[R], ktil[R], sumk = 0.f, al = 0.f;
#pragma unroll
        for (int j = 0; j < R; ++j) {
            kap[j] = k1[j] * k1[j];
            sumk += kap[j];
            al = fmaf(d[j], kap[j], al);
            ktil[j] = d[j] * k1[j];
        }
        sumk = dec_warp_sum(sumk);
        al = dec_warp_sum(al);
        const float n = fmaxf(sumk, hy.eps);
        const float bb = hy.beta_aware ? beta : 1.0f;
        const float c = hy.eta * bb * (1.0f - bb * al) / n;
#pragma unroll
        for (int j = 0; j < R; ++j) {
            float x = fmaf(c, kap[j], rho[j] * d[j]);
            if (hy.clamp) x = fminf(fmaxf(x, hy.d_min), hy.d_max);
            d[j] = x;
        }

        // rank-1 write and read-out, row by row (the four reductions of a step are independent)
        float dot[DEC_RW], o[DEC_RW];
#pragma unroll
        for (int r = 0; r < DEC_RW; ++r) {
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < R; ++j) s = fmaf(S[r][j], k1[j], s);
            dot[r] = s;
        }
#pragma unroll
        for (int r = 0; r < DEC_RW; ++r) dot[r] = dec_warp_sum(dot[r]);
#pragma unroll
        for (int r = 0; r < DEC_RW; ++r) {
            const float rv = beta * (v1[r] - alpha * dot[r]);
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < R; ++j) {
                S[r][j] = fmaf(alpha, S[r][j], rv * ktil[j]);
                s = fmaf(S[r][j], q1[j], s);
            }
            o[r] = s;
        }
#pragma unroll
        for (int r = 0; r < DEC_RW; ++r) o[r] = dec_warp_sum(o[r]);
        if (lane < DEC_RW) {
            float mine = o[0];
#pragma unroll
            for (int r = 1; r < DEC_RW; ++r) mine = lane == r ? o[r] : mine;
            const size_t th = ((size_t)b * a.L + t) * a.H + h;
            stf(op + th * V + v0 + lane, hy.scale * mine);
        }
    }
#pragma unroll
    for (int r = 0; r < DEC_RW; ++r) dec_store<R>(srow + (size_t)r * K, lane, S[r]);
    // every slice of the chain has read the old preconditioner before slice 0 overwrites it
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (slice == 0 && warp == 0) dec_store<R>(a.precond + (size_t)chain * K, lane, d);
}

// One cluster per chain: its V / 16 slices (8 or 4 CTAs, within the portable cluster size).
template <typename T, int K, int V, bool VEC> bool launch_one(unsigned chains, const DecArgs& a, cudaStream_t st)
{
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(chains * (unsigned)(V / DEC_VB));
    cfg.blockDim = dim3(DEC_WARPS * 32);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = V / DEC_VB;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, decode_kernel<T, K, V, VEC>, a) == cudaSuccess;
}

template <typename T> int launch_typed(const osdn_params& p, const DecArgs& a, cudaStream_t st)
{
    const unsigned chains = (unsigned)p.B * (unsigned)p.H;
    bool ok;
    if (a.hy.apf_mode == 3) {
        if (p.K == 128 && p.V == 128) ok = launch_one<T, 128, 128, true>(chains, a, st);
        else if (p.K == 128 && p.V == 64) ok = launch_one<T, 128, 64, true>(chains, a, st);
        else if (p.K == 64 && p.V == 128) ok = launch_one<T, 64, 128, true>(chains, a, st);
        else ok = launch_one<T, 64, 64, true>(chains, a, st);
    } else {
        if (p.K == 128 && p.V == 128) ok = launch_one<T, 128, 128, false>(chains, a, st);
        else if (p.K == 128 && p.V == 64) ok = launch_one<T, 128, 64, false>(chains, a, st);
        else if (p.K == 64 && p.V == 128) ok = launch_one<T, 64, 128, false>(chains, a, st);
        else ok = launch_one<T, 64, 64, false>(chains, a, st);
    }
    return ok && cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace

int decode_step(const osdn_params& p, const Hyper& hy, const void* q, const void* k, const void* v,
                const float* beta, const float* gate, const float* log_ret, float* state, float* precond,
                void* out, cudaStream_t st)
{
    DecArgs a{};
    a.B = p.B; a.L = p.T; a.H = p.H;
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.gate = gate; a.log_ret = log_ret;
    a.state = state; a.precond = precond; a.out = out; a.hy = hy;
    stage_mark(st, "decode_step");
    const int n = p.io_dtype == OSDN_FP32 ? launch_typed<float>(p, a, st) : launch_typed<__nv_bfloat16>(p, a, st);
    stage_end(st);
    return n;
}

}  // namespace osdn
