// Online-scaled delta rule with a channel gate (the OSKDA backbone extension: Kimi Delta Attention with
// Online Scaling).  The scalar gate exp(g_t) of the layer becomes one gate per key channel,
//     Sbar = S_{t-1} Diag(alpha_t),  u = v_t - Sbar k_t,  S_t = Sbar + beta_t u ktil_t^T,  o_t = scale S_t q_t,
// with the state kept V x K as everywhere in this library (the paper's K x V state is its transpose).
// Phase 1 (preconditioner, write keys, their adjoint) is the layer's own and is reused unchanged; this
// file holds phase 2 and its adjoint as token-recurrent CUDA-core kernels in fp32: the rows of S do not
// interact in the forward, so a warp owns a few rows (a lane holds K / 32 columns of each) and walks the
// sequence; the dot products along a row are warp reductions.  The backward walks the chunks in reverse:
// from the row checkpoint the forward left at a chunk's start it first leaves a checkpoint at every
// stretch of SUB tokens, then replays stretch by stretch, keeping the rows before every token, and takes
// the adjoint steps; the sums over rows (dq, dk, d ktil, d gate, d beta) are formed per warp, then per CTA
// in shared memory, and added to global fp32 accumulators.
#include "osdn_common.cuh"

namespace osdn {
namespace {

constexpr int KF_WARPS = 8, KF_RW = 4;   // forward: warps per CTA, state rows per warp
constexpr int KB_WARPS = 16, KB_RW = 2;   // backward: warps per CTA, state rows per warp
// The backward keeps the rows before the tokens of a SUB-token stretch only (the history then stays in L2): a
// chunk is walked once to leave a row checkpoint at every stretch start, then stretch by stretch in reverse.
constexpr int SUB = 16, NSUB = CH / SUB, HROWS = SUB + NSUB;   // history rows per state row: a stretch, then the checkpoints

template <int R> struct Vec {
    float x[R];
};

template <int R> __device__ __forceinline__ Vec<R> load_vec(const float* p)
{
    Vec<R> r;
    if constexpr (R == 4) {
        const float4 f = *reinterpret_cast<const float4*>(p);
        r.x[0] = f.x; r.x[1] = f.y; r.x[2] = f.z; r.x[3] = f.w;
    } else {
        const float2 f = *reinterpret_cast<const float2*>(p);
        r.x[0] = f.x; r.x[1] = f.y;
    }
    return r;
}
template <int R> __device__ __forceinline__ Vec<R> load_vec(const __nv_bfloat16* p)
{
    Vec<R> r;
    if constexpr (R == 4) {
        const uint2 w = *reinterpret_cast<const uint2*>(p);
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w.x));
        const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w.y));
        r.x[0] = a.x; r.x[1] = a.y; r.x[2] = b.x; r.x[3] = b.y;
    } else {
        const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
        r.x[0] = a.x; r.x[1] = a.y;
    }
    return r;
}
template <int R> __device__ __forceinline__ void store_vec(float* p, const Vec<R>& v)
{
    if constexpr (R == 4) *reinterpret_cast<float4*>(p) = make_float4(v.x[0], v.x[1], v.x[2], v.x[3]);
    else *reinterpret_cast<float2*>(p) = make_float2(v.x[0], v.x[1]);
}

__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

struct KdaArgs {
    int H, V;
    Table tab;
    const void *q, *k, *v;
    const float *beta, *gate;     // gate: [T,H,K] channel log-gates
    const float* ktil;            // [T,H,K] write keys of phase 1
    const float* init_state;      // nullable
    void* out;
    float* final_state;           // nullable
    float* ckpt;                  // nullable: [chunk, H, V, K] rows at every chunk start
    float scale;
    // backward
    const void* dout;
    const float* dfinal_state;    // nullable
    void* dv;
    float *dq_acc, *dkread, *dktil, *dgate, *dbeta;   // zeroed accumulators
    float* dinit_state;           // nullable
    float* hist;                  // [chain, V, HROWS, K] rows before every token of the stretch in progress, then
                                  // the stretch checkpoints of the chunk in progress
};

// What a row needs of one token.
template <int R> struct Tok {
    Vec<R> k, kt, g;
    float v, beta;
};

template <typename T, int R>
__device__ __forceinline__ Tok<R> load_tok(const KdaArgs& a, size_t th, int K, int row, int lane)
{
    Tok<R> t;
    t.k = load_vec<R>(static_cast<const T*>(a.k) + th * K + R * lane);
    t.kt = load_vec<R>(a.ktil + th * K + R * lane);
    t.g = load_vec<R>(a.gate + th * K + R * lane);
    t.v = ldf(static_cast<const T*>(a.v) + th * a.V + row);
    t.beta = a.beta[th];
    return t;
}

// One forward step of a row: S <- S Diag(alpha) + beta u ktil^T; returns u, leaves Sbar in `sbar`.
template <int R> __device__ __forceinline__ float row_step(Vec<R>& S, const Tok<R>& t, Vec<R>* sbar)
{
    float acc = 0.f;
#pragma unroll
    for (int x = 0; x < R; ++x) {
        S.x[x] *= __expf(t.g.x[x]);
        acc = fmaf(S.x[x], t.k.x[x], acc);
    }
    if (sbar) *sbar = S;
    const float u = t.v - warp_sum(acc);
    const float bu = t.beta * u;
#pragma unroll
    for (int x = 0; x < R; ++x) S.x[x] = fmaf(bu, t.kt.x[x], S.x[x]);
    return u;
}

// A block of KTB tokens of one chain in shared memory, filled with cp.async by the whole CTA: every row-warp
// of the CTA needs the same k, ktil, gate and q of a token, so they are fetched once per CTA instead of once
// per warp (which made the forward bound by L2 bandwidth: 1.5 KB per token and warp).
constexpr int KTB = 8;
template <typename T, int K> struct TokBlock {
    T k[KTB][K];
    T q[KTB][K];
    float kt[KTB][K];
    float g[KTB][K];
};

__device__ __forceinline__ void cp_async16(void* dst, const void* src)
{
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit_group() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// tokens [t, t + n) of the chain, n <= KTB; th0: token-head index of token t
template <typename T, int K>
__device__ __forceinline__ void fill_block(TokBlock<T, K>& blk, const KdaArgs& a, size_t th0, int H, int n, int tid, int nthreads)
{
    constexpr int PT = K * sizeof(T) / 16, PF = K * 4 / 16;   // 16-byte pieces per row
    constexpr int PER = 2 * PT + 2 * PF;
    for (int p = tid; p < n * PER; p += nthreads) {
        const int j = p / PER, r = p - j * PER;
        const size_t row = (th0 + (size_t)j * H) * K;
        if (r < PT) cp_async16(reinterpret_cast<char*>(blk.k[j]) + r * 16, reinterpret_cast<const char*>(static_cast<const T*>(a.k) + row) + r * 16);
        else if (r < 2 * PT) cp_async16(reinterpret_cast<char*>(blk.q[j]) + (r - PT) * 16, reinterpret_cast<const char*>(static_cast<const T*>(a.q) + row) + (r - PT) * 16);
        else if (r < 2 * PT + PF) cp_async16(reinterpret_cast<char*>(blk.kt[j]) + (r - 2 * PT) * 16, reinterpret_cast<const char*>(a.ktil + row) + (r - 2 * PT) * 16);
        else cp_async16(reinterpret_cast<char*>(blk.g[j]) + (r - 2 * PT - PF) * 16, reinterpret_cast<const char*>(a.gate + row) + (r - 2 * PT - PF) * 16);
    }
}

template <typename T, int K, int R>
__device__ __forceinline__ Tok<R> tok_from_block(const TokBlock<T, K>& blk, int j, int lane, float v, float beta)
{
    Tok<R> t;
    t.k = load_vec<R>(blk.k[j] + R * lane);
    t.kt = load_vec<R>(blk.kt[j] + R * lane);
    t.g = load_vec<R>(blk.g[j] + R * lane);
    t.v = v;
    t.beta = beta;
    return t;
}

// Forward: a warp owns KF_RW rows of S.  The token's k, ktil, gate and q are read once per warp and serve
// all its rows, the channel gates are exponentiated once, and the rows' reductions run side by side (their
// shuffle rounds overlap): per row and token about 45 instructions instead of 100.
template <typename T, int K>
__global__ void __launch_bounds__(KF_WARPS * 32) kda_fwd_kernel(KdaArgs a)
{
    constexpr int R = K / 32;
    static_assert(KTB * KF_RW == 32, "one lane per (token of the block, row of the warp) for the v scalars");
    __shared__ __align__(16) TokBlock<T, K> blk[2];
    const int H = a.H, V = a.V;
    const int chain = blockIdx.y, s = chain / H, h = chain - s * H;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row0 = (blockIdx.x * KF_WARPS + warp) * KF_RW;
    const int t0 = a.tab.seq_tok0(s), len = a.tab.seq_len(s), c0 = a.tab.seq_chunk0(s);
    const size_t srow = (((size_t)s * H + h) * V + row0) * K + R * lane;
    Vec<R> S[KF_RW];
#pragma unroll
    for (int r = 0; r < KF_RW; ++r) {
        if (a.init_state) S[r] = load_vec<R>(a.init_state + srow + (size_t)r * K);
        else
#pragma unroll
            for (int x = 0; x < R; ++x) S[r].x[x] = 0.f;
    }
    const int nblk = (len + KTB - 1) / KTB;
    // scalars of a block, one block ahead: lane j * KF_RW + r holds v of token j for row r; lane j < KTB also beta
    auto scalars = [&](int bi, float& vv, float& bb) {
        vv = 0.f;
        bb = 0.f;
        const int j = lane / KF_RW, r = lane % KF_RW, t = bi * KTB + j;
        if (bi < nblk && t < len) vv = ldf(static_cast<const T*>(a.v) + ((size_t)(t0 + t) * H + h) * V + row0 + r);
        if (bi < nblk && lane < KTB && bi * KTB + lane < len) bb = a.beta[(size_t)(t0 + bi * KTB + lane) * H + h];
    };
    if (nblk > 0) fill_block<T, K>(blk[0], a, (size_t)t0 * H + h, H, min(KTB, len), tid, KF_WARPS * 32);
    cp_async_commit_group();
    float sv, sb;
    scalars(0, sv, sb);
    for (int bi = 0; bi < nblk; ++bi) {
        const int tb0 = bi * KTB, n = min(KTB, len - tb0);
        if (bi + 1 < nblk)
            fill_block<T, K>(blk[(bi + 1) & 1], a, (size_t)(t0 + tb0 + KTB) * H + h, H, min(KTB, len - tb0 - KTB), tid, KF_WARPS * 32);
        cp_async_commit_group();
        float sv_next, sb_next;
        scalars(bi + 1, sv_next, sb_next);
        cp_async_wait_group<1>();
        __syncthreads();   // the block has landed for every warp
        const TokBlock<T, K>& B = blk[bi & 1];
        for (int j = 0; j < n; ++j) {
            const int t = tb0 + j;
            const size_t th = (size_t)(t0 + t) * H + h;
            if (a.ckpt && (t % CH) == 0) {
#pragma unroll
                for (int r = 0; r < KF_RW; ++r)
                    store_vec<R>(a.ckpt + (((size_t)(c0 + t / CH) * H + h) * V + row0 + r) * K + R * lane, S[r]);
            }
            const Vec<R> kk = load_vec<R>(B.k[j] + R * lane), kt = load_vec<R>(B.kt[j] + R * lane);
            const Vec<R> gg = load_vec<R>(B.g[j] + R * lane), qc = load_vec<R>(B.q[j] + R * lane);
            const float beta = __shfl_sync(0xffffffffu, sb, j);
            float al[R], acc[KF_RW];
#pragma unroll
            for (int x = 0; x < R; ++x) al[x] = __expf(gg.x[x]);
#pragma unroll
            for (int r = 0; r < KF_RW; ++r) {
                acc[r] = 0.f;
#pragma unroll
                for (int x = 0; x < R; ++x) {
                    S[r].x[x] *= al[x];
                    acc[r] = fmaf(S[r].x[x], kk.x[x], acc[r]);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int r = 0; r < KF_RW; ++r) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], o);
            float out[KF_RW];
#pragma unroll
            for (int r = 0; r < KF_RW; ++r) {
                const float bu = beta * (__shfl_sync(0xffffffffu, sv, j * KF_RW + r) - acc[r]);
                out[r] = 0.f;
#pragma unroll
                for (int x = 0; x < R; ++x) {
                    S[r].x[x] = fmaf(bu, kt.x[x], S[r].x[x]);
                    out[r] = fmaf(S[r].x[x], qc.x[x], out[r]);
                }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1)
#pragma unroll
                for (int r = 0; r < KF_RW; ++r) out[r] += __shfl_xor_sync(0xffffffffu, out[r], o);
            float mine = out[0];
#pragma unroll
            for (int r = 1; r < KF_RW; ++r) mine = lane == r ? out[r] : mine;
            if (lane < KF_RW) stf(static_cast<T*>(a.out) + th * V + row0 + lane, a.scale * mine);
        }
        sv = sv_next;
        sb = sb_next;
        __syncthreads();   // everybody is done with the block before it is refilled
    }
#pragma unroll
    for (int r = 0; r < KF_RW; ++r)
        if (a.final_state) store_vec<R>(a.final_state + srow + (size_t)r * K, S[r]);
}

// Backward: a warp owns KB_RW state rows, KB_WARPS warps per CTA.  The token operands (k, q, ktil, gates) of
// a block of KTB tokens are staged once per CTA in shared memory, one block ahead, for the replay (forward
// order) as for the adjoint steps (reverse order); the rows' per-token scalars (v, dout; beta) travel in
// registers, one block at a time; the rows before a token come from the history one token ahead of their
// use.  The rows' contributions to dq, dk, d ktil and d gate are added up inside the warp first.
template <typename T, int K>
__global__ void __launch_bounds__(KB_WARPS * 32, 2) kda_bwd_kernel(KdaArgs a)
{
    constexpr int R = K / 32;
    constexpr int NT = KB_WARPS * 32, RW = KB_RW;
    static_assert(2 * KTB * RW <= 32, "one lane per (kind, token of the block, row of the warp)");
    extern __shared__ __align__(16) uint8_t kda_dyn[];
    float* red = reinterpret_cast<float*>(kda_dyn);   // [2][KB_WARPS][4][K]: per-warp terms of dq, dk, d ktil, d gate
    TokBlock<T, K>* blk = reinterpret_cast<TokBlock<T, K>*>(kda_dyn + (size_t)2 * KB_WARPS * 4 * K * sizeof(float));
    __shared__ float red_beta[2][KB_WARPS];
    const int H = a.H, V = a.V;
    const int chain = blockIdx.y, s = chain / H, h = chain - s * H;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row0 = (blockIdx.x * KB_WARPS + warp) * RW;
    const int t0 = a.tab.seq_tok0(s), len = a.tab.seq_len(s), c0 = a.tab.seq_chunk0(s);
    const int nchunks = (len + CH - 1) / CH;
    const size_t srow = (((size_t)s * H + h) * V + row0) * K + R * lane;
    float* hist = a.hist + ((size_t)chain * V + row0) * HROWS * K + R * lane;   // row r of the warp: + r HROWS K
    Vec<R> Shat[RW];
#pragma unroll
    for (int r = 0; r < RW; ++r) {
        if (a.dfinal_state) Shat[r] = load_vec<R>(a.dfinal_state + srow + (size_t)r * K);
        else
#pragma unroll
            for (int x = 0; x < R; ++x) Shat[r].x[x] = 0.f;
    }
    int it = 0;
    for (int n = nchunks - 1; n >= 0; --n) {
        const int clen = min(CH, len - n * CH), nb = (clen + KTB - 1) / KTB;
        const int tc0 = t0 + n * CH;                       // first token of the chunk
        // lane (kind, j, r) = kind KTB RW + j RW + r: kind 0 the row's v of token j of block b, kind 1 its dout
        auto scalars = [&](int b, float& sv, float& sbeta) {
            sv = 0.f;
            sbeta = 0.f;
            const int kind = lane / (KTB * RW), j = (lane / RW) % KTB, r = lane % RW, t = b * KTB + j;
            if (b >= 0 && b < nb && t < clen && kind < 2) {
                const size_t th = (size_t)(tc0 + t) * H + h;
                sv = ldf(static_cast<const T*>(kind == 0 ? a.v : a.dout) + th * V + row0 + r);
            }
            if (b >= 0 && b < nb && lane < KTB && b * KTB + lane < clen) sbeta = a.beta[(size_t)(tc0 + b * KTB + lane) * H + h];
        };
        auto fill = [&](int b, int slot) {
            if (b >= 0 && b < nb)
                fill_block<T, K>(blk[slot], a, (size_t)(tc0 + b * KTB) * H + h, H, min(KTB, clen - b * KTB), tid, NT);
            cp_async_commit_group();
        };
        // forward steps of the warp's rows over one staged block (optionally keeping the rows before each token)
        auto forward_block = [&](const TokBlock<T, K>& B, int nt, float sv, float sbeta, Vec<R> (&S)[RW], int hist_at) {
            for (int j = 0; j < nt; ++j) {
                const float beta = __shfl_sync(0xffffffffu, sbeta, j);
#pragma unroll
                for (int r = 0; r < RW; ++r) {
                    if (hist_at >= 0) store_vec<R>(hist + ((size_t)r * HROWS + hist_at + j) * K, S[r]);
                    const Tok<R> tk = tok_from_block<T, K, R>(B, j, lane, __shfl_sync(0xffffffffu, sv, j * RW + r), beta);
                    row_step<R>(S[r], tk, nullptr);
                }
            }
        };
        // ---- once through the chunk: a row checkpoint at the start of every stretch of SUB tokens
        {
            Vec<R> S[RW];
#pragma unroll
            for (int r = 0; r < RW; ++r) S[r] = load_vec<R>(a.ckpt + (((size_t)(c0 + n) * H + h) * V + row0 + r) * K + R * lane);
            fill(0, 0);
            float sv, sbeta;
            scalars(0, sv, sbeta);
            for (int b = 0; b < nb; ++b) {
                fill(b + 1, (b + 1) & 1);
                float sv_next, sbeta_next;
                scalars(b + 1, sv_next, sbeta_next);
                cp_async_wait_group<1>();
                __syncthreads();
                if ((b * KTB) % SUB == 0) {
#pragma unroll
                    for (int r = 0; r < RW; ++r) store_vec<R>(hist + ((size_t)r * HROWS + SUB + b * KTB / SUB) * K, S[r]);
                }
                forward_block(blk[b & 1], min(KTB, clen - b * KTB), sv, sbeta, S, -1);
                sv = sv_next;
                sbeta = sbeta_next;
                __syncthreads();
            }
        }
        for (int sb = (clen - 1) / SUB; sb >= 0; --sb) {
            const int b_lo = sb * (SUB / KTB), b_hi = min(nb, (sb + 1) * (SUB / KTB));   // token blocks of the stretch
            const int s_tok0 = sb * SUB, s_len = min(SUB, clen - s_tok0);
            // ---- replay the stretch from its checkpoint, keeping the rows before every token
            {
                Vec<R> S[RW];
#pragma unroll
                for (int r = 0; r < RW; ++r) S[r] = load_vec<R>(hist + ((size_t)r * HROWS + SUB + sb) * K);
                fill(b_lo, 0);
                float sv, sbeta;
                scalars(b_lo, sv, sbeta);
                for (int b = b_lo, step = 0; b < b_hi; ++b, ++step) {
                    if (b + 1 < b_hi) fill(b + 1, (step + 1) & 1);
                    else cp_async_commit_group();
                    float sv_next, sbeta_next;
                    scalars(b + 1 < b_hi ? b + 1 : -1, sv_next, sbeta_next);
                    cp_async_wait_group<1>();
                    __syncthreads();
                    forward_block(blk[step & 1], min(KTB, clen - b * KTB), sv, sbeta, S, b * KTB - s_tok0);
                    sv = sv_next;
                    sbeta = sbeta_next;
                    __syncthreads();
                }
            }
            // ---- adjoint steps of the stretch, last token first
            fill(b_hi - 1, 0);
            float sv, sbeta;
            scalars(b_hi - 1, sv, sbeta);
            Vec<R> Sprev[RW];
#pragma unroll
            for (int r = 0; r < RW; ++r) Sprev[r] = load_vec<R>(hist + ((size_t)r * HROWS + s_len - 1) * K);
            for (int b = b_hi - 1, step = 0; b >= b_lo; --b, ++step) {
                if (b - 1 >= b_lo) fill(b - 1, (step + 1) & 1);
                else cp_async_commit_group();
                float sv_next, sbeta_next;
                scalars(b - 1 >= b_lo ? b - 1 : -1, sv_next, sbeta_next);
                cp_async_wait_group<1>();
                __syncthreads();
                const TokBlock<T, K>& B = blk[step & 1];
                const int nt = min(KTB, clen - b * KTB);
                for (int j = nt - 1; j >= 0; --j, ++it) {
                    const int jj = b * KTB + j;
                    const size_t th = (size_t)(tc0 + jj) * H + h;
                    const float beta = __shfl_sync(0xffffffffu, sbeta, j);
                    const Vec<R> q = load_vec<R>(B.q[j] + R * lane);
                    Vec<R> pq, pk, pkt, pg;   // the warp's rows added up: dq, dk (read key), d ktil, d gate
#pragma unroll
                    for (int x = 0; x < R; ++x) pq.x[x] = pk.x[x] = pkt.x[x] = pg.x[x] = 0.f;
                    float pbeta = 0.f, myv = 0.f;
#pragma unroll
                    for (int r = 0; r < RW; ++r) {
                        const Tok<R> tk = tok_from_block<T, K, R>(B, j, lane, __shfl_sync(0xffffffffu, sv, j * RW + r), beta);
                        const float sdo = a.scale * __shfl_sync(0xffffffffu, sv, KTB * RW + j * RW + r);
                        Vec<R> St = Sprev[r], Sbar;
                        if (jj > s_tok0) Sprev[r] = load_vec<R>(hist + ((size_t)r * HROWS + jj - 1 - s_tok0) * K);   // the next step's row
                        const float u = row_step<R>(St, tk, &Sbar);
                        // o_t = scale S_t q_t
                        float w = 0.f;
#pragma unroll
                        for (int x = 0; x < R; ++x) {
                            pq.x[x] = fmaf(sdo, St.x[x], pq.x[x]);
                            Shat[r].x[x] = fmaf(sdo, q.x[x], Shat[r].x[x]);
                            w = fmaf(Shat[r].x[x], tk.kt.x[x], w);
                        }
                        // S_t = Sbar + beta u ktil^T
                        w = warp_sum(w);
                        const float du = beta * w, bu = beta * u;
                        pbeta = fmaf(u, w, pbeta);
                        // u = v - Sbar k ; Sbar = S_{t-1} Diag(alpha)
#pragma unroll
                        for (int x = 0; x < R; ++x) {
                            pkt.x[x] = fmaf(bu, Shat[r].x[x], pkt.x[x]);
                            pk.x[x] = fmaf(-Sbar.x[x], du, pk.x[x]);
                            const float dsb = fmaf(-du, tk.k.x[x], Shat[r].x[x]);
                            pg.x[x] = fmaf(dsb, Sbar.x[x], pg.x[x]);
                            Shat[r].x[x] = __expf(tk.g.x[x]) * dsb;
                        }
                        myv = lane == r ? du : myv;
                    }
                    float* buf = red + ((size_t)(it & 1) * KB_WARPS + warp) * 4 * K + R * lane;
                    store_vec<R>(buf, pq);
                    store_vec<R>(buf + K, pk);
                    store_vec<R>(buf + 2 * K, pkt);
                    store_vec<R>(buf + 3 * K, pg);
                    if (lane == 0) red_beta[it & 1][warp] = pbeta;
                    if (lane < RW) stf(static_cast<T*>(a.dv) + th * V + row0 + lane, myv);
                    __syncthreads();
                    // sums over the CTA's warps; the buffers alternate, so one barrier per token is enough
                    for (int o = tid; o < 4 * K; o += NT) {
                        const float* src = red + (size_t)(it & 1) * KB_WARPS * 4 * K + o;
                        float sum = 0.f;
#pragma unroll 8
                        for (int w2 = 0; w2 < KB_WARPS; ++w2) sum += src[(size_t)w2 * 4 * K];
                        const int m = o / K, i = o - m * K;
                        float* dst = m == 0 ? a.dq_acc : m == 1 ? a.dkread : m == 2 ? a.dktil : a.dgate;
                        atomicAdd(dst + th * K + i, sum);
                    }
                    if (tid == NT - 1) {
                        float sum = 0.f;
                        for (int w2 = 0; w2 < KB_WARPS; ++w2) sum += red_beta[it & 1][w2];
                        atomicAdd(a.dbeta + th, sum);
                    }
                }
                sv = sv_next;
                sbeta = sbeta_next;
                __syncthreads();   // everybody is done with the block before it is refilled
            }
        }
        cp_async_wait_group<0>();
    }
#pragma unroll
    for (int r = 0; r < RW; ++r)
        if (a.dinit_state) store_vec<R>(a.dinit_state + srow + (size_t)r * K, Shat[r]);
}

template <typename T> __global__ void cast_rows_kernel(const float* src, T* dst, size_t n)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) stf(dst + i, src[i]);
}

}  // namespace

size_t kda_extra_bytes(const osdn_params& p, const WsLayout& L, bool need_bwd)
{
    if (!need_bwd) return 0;
    const size_t Ttot = p.nseq > 0 ? (size_t)p.T : (size_t)p.B * p.T;
    const size_t hist = align_up((size_t)L.S * p.H * p.V * HROWS * p.K * 4, 256);
    const size_t dq = align_up(Ttot * p.H * p.K * 4, 256);
    return hist + dq;
}

namespace {
KdaArgs base_args(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a)
{
    char* w = static_cast<char*>(ws);
    KdaArgs k{};
    k.H = p.H; k.V = p.V; k.tab = carve_table(ws, L);
    k.q = a.q; k.k = a.k; k.v = a.v; k.beta = a.beta; k.gate = a.gate;
    k.ktil = reinterpret_cast<const float*>(w + L.ktil);
    k.init_state = a.init_state; k.scale = hy.scale;
    k.ckpt = reinterpret_cast<float*>(w + L.Sn);
    return k;
}
}  // namespace

int kda_forward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a, bool save,
                cudaStream_t st)
{
    int launches = launch_build_table(p, L, ws, st);
    if (launches < 0) return -1;
    char* w = static_cast<char*>(ws);
    const int n1 = phase1_forward(p, hy, L, ws, a, w + L.ktil, false, save, st);
    if (n1 < 0) return -1;
    launches += n1;
    KdaArgs k = base_args(p, hy, L, ws, a);
    k.out = a.out; k.final_state = a.final_state;
    if (!save) k.ckpt = nullptr;
    const dim3 grid(p.V / (KF_WARPS * KF_RW), L.S * p.H);
    stage_mark(st, "kda_fwd");
    if (p.io_dtype == OSDN_FP32) {
        if (p.K == 64) kda_fwd_kernel<float, 64><<<grid, KF_WARPS * 32, 0, st>>>(k);
        else kda_fwd_kernel<float, 128><<<grid, KF_WARPS * 32, 0, st>>>(k);
    } else {
        if (p.K == 64) kda_fwd_kernel<__nv_bfloat16, 64><<<grid, KF_WARPS * 32, 0, st>>>(k);
        else kda_fwd_kernel<__nv_bfloat16, 128><<<grid, KF_WARPS * 32, 0, st>>>(k);
    }
    stage_end(st);
    return cudaGetLastError() == cudaSuccess ? launches + 1 : -1;
}

int kda_backward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                 cudaStream_t st)
{
    char* w = static_cast<char*>(ws);
    const size_t Ttot = p.nseq > 0 ? (size_t)p.T : (size_t)p.B * p.T;
    const size_t nK = Ttot * p.H * p.K;
    KdaArgs k = base_args(p, hy, L, ws, a);
    k.dout = a.dout; k.dfinal_state = a.dfinal_state; k.dv = a.dv; k.dinit_state = a.dinit_state;
    k.hist = reinterpret_cast<float*>(w + align_up(L.total, 256));
    k.dq_acc = reinterpret_cast<float*>(w + align_up(L.total, 256) +
                                        align_up((size_t)L.S * p.H * p.V * HROWS * p.K * 4, 256));
    k.dkread = reinterpret_cast<float*>(w + L.dkread);
    k.dktil = reinterpret_cast<float*>(w + L.dktil);
    k.dgate = a.dgate; k.dbeta = a.dbeta;
    if (cudaMemsetAsync(k.dq_acc, 0, nK * 4, st) != cudaSuccess || cudaMemsetAsync(k.dkread, 0, nK * 4, st) != cudaSuccess ||
        cudaMemsetAsync(k.dktil, 0, nK * 4, st) != cudaSuccess || cudaMemsetAsync(k.dgate, 0, nK * 4, st) != cudaSuccess ||
        cudaMemsetAsync(k.dbeta, 0, Ttot * p.H * 4, st) != cudaSuccess)
        return -1;
    const dim3 grid(p.V / (KB_WARPS * KB_RW), L.S * p.H);
    const size_t es = p.io_dtype == OSDN_BF16 ? 2 : 4;
    // the row sums' double buffer, then two token blocks (k, q in the I/O type; ktil, gates fp32)
    const size_t smem = (size_t)2 * KB_WARPS * 4 * p.K * sizeof(float) + 2 * (size_t)KTB * p.K * (2 * es + 8);
    stage_mark(st, "kda_bwd");
    auto launch = [&](auto kernel) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return false;
        kernel<<<grid, KB_WARPS * 32, smem, st>>>(k);
        return true;
    };
    bool ok;
    if (p.io_dtype == OSDN_FP32) ok = p.K == 64 ? launch(kda_bwd_kernel<float, 64>) : launch(kda_bwd_kernel<float, 128>);
    else ok = p.K == 64 ? launch(kda_bwd_kernel<__nv_bfloat16, 64>) : launch(kda_bwd_kernel<__nv_bfloat16, 128>);
    if (!ok) return -1;
    stage_mark(st, "kda_cast_dq");
    const unsigned blocks = (unsigned)((nK + 255) / 256);
    if (p.io_dtype == OSDN_FP32) cast_rows_kernel<float><<<blocks, 256, 0, st>>>(k.dq_acc, static_cast<float*>(a.dq), nK);
    else cast_rows_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(k.dq_acc, static_cast<__nv_bfloat16*>(a.dq), nK);
    // phase-1 adjoint: dk = dk(read key) + d_t (.) d ktil + preconditioner terms; adds its share to d beta
    const int n1 = phase1_backward(p, hy, L, ws, a, k.dktil, k.dkread, true, st);
    if (n1 < 0) return -1;
    stage_end(st);
    return cudaGetLastError() == cudaSuccess ? 2 + n1 : -1;
}

}  // namespace osdn
