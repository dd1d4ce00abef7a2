// CUDA-core (fp32 FMA) kernels of the OSDN layer.
//
// This family is the fp32 mode of the library (fp32 I/O needs better than TF32 accuracy)
// and the reference-quality path for bf16 I/O when OSDN_FLAG_FORCE_SIMT is set.  Every
// step of the chunkwise algorithm runs here in fp32:
//
//   phase1_fwd      Algorithm 1 with APF and the box projection, one warp per chain
//   chunk_local_fwd decay-ratio Gram A, UT inverse T, W = T diag(beta gamma) K,
//                   U = T diag(beta) V, local scores P           (gated chunk form)
//   chain_fwd       dU = U - W S^T ; O = scale[(gamma Q) S^T + P dU] ;
//                   S <- gamma_C S + dU^T (rho Ktil)              (state recurrence)
//   chain_bwd       reverse state chain: ddU, dS
//   chunk_local_bwd all chunk-local gradients (through P, W, U, T, A and the gate prefix)
//   phase1_bwd      reverse sweep over the projected affine recurrence (Section 3.5)
//
// Notation follows the paper: G_i in-chunk inclusive prefix of the log gate,
// gamma_i = exp(G_i), Gamma_ij = exp(G_i - G_j), rho_i = exp(G_C - G_i).
#include "osdn_common.cuh"

namespace osdn {

namespace {

constexpr int NTH = 256;

// ---------------------------------------------------------------------------------------
// chunk table
// ---------------------------------------------------------------------------------------
// One CTA.  Chunk counts per sequence are scanned 256 sequences at a time; every chunk then finds
// its sequence by bisection over the chunk offsets (kept in shared memory while they fit).
constexpr int TBL_THREADS = 256, TBL_SMEM_SEQ = 2048;

// The offsets live on the device, so the host cannot check them: a sequence is clamped into the packed
// token range [0, T_total] (every later access stays inside the user tensors whatever cu_seqlens
// holds), and a violated contract (cu[0] != 0, a decreasing pair, cu[S] != T_total) is reported through
// the device status word.
__device__ __forceinline__ void clamped_sequence(const int* __restrict__ cu, int s, int T_total, int& t0, int& len, bool& bad)
{
    const int a = cu[s], b = cu[s + 1];
    bad = b < a || a < 0 || b > T_total;
    t0 = min(max(a, 0), T_total);
    len = min(max(b, t0), T_total) - t0;
}

__global__ void __launch_bounds__(TBL_THREADS)
build_table_kernel(int S, int T_dense, const int* __restrict__ cu, int NTmax, Table t, int* status)
{
    __shared__ int s_c0[TBL_SMEM_SEQ + 1];
    __shared__ int s_scan[TBL_THREADS];
    __shared__ int s_carry;
    const int tid = threadIdx.x;
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int base = 0; base < S; base += TBL_THREADS) {
        const int s = base + tid;
        int t0 = 0, len = 0;
        if (s < S) {
            if (cu) {   // packed batch: T_dense is the packed token count
                bool bad;
                clamped_sequence(cu, s, T_dense, t0, len, bad);
                if (s == 0 && cu[0] != 0) bad = true;
                if (s == S - 1 && cu[S] != T_dense) bad = true;
                if (bad && status) atomicCAS(status, 0, OSDN_DEVICE_BAD_CU_SEQLENS);
            } else {
                t0 = s * T_dense;
                len = T_dense;
            }
        }
        const int nc = (len + CH - 1) / CH;
        s_scan[tid] = nc;
        __syncthreads();
        for (int o = 1; o < TBL_THREADS; o <<= 1) {   // inclusive scan
            const int v = tid >= o ? s_scan[tid - o] : 0;
            __syncthreads();
            s_scan[tid] += v;
            __syncthreads();
        }
        const int carry = s_carry;
        if (s < S) {
            const int c = min(carry + s_scan[tid] - nc, NTmax);
            t.seq_tok0_[s] = t0;
            t.seq_len_[s] = len;
            t.seq_chunk0_[s] = c;
            if (s <= TBL_SMEM_SEQ) s_c0[s] = c;
        }
        __syncthreads();
        if (tid == TBL_THREADS - 1) s_carry = carry + s_scan[tid];
        __syncthreads();
    }
    const int total = min(s_carry, NTmax);
    if (tid == 0) {
        t.seq_chunk0_[S] = total;
        if (S <= TBL_SMEM_SEQ) s_c0[S] = total;
    }
    __syncthreads();
    const bool in_smem = S <= TBL_SMEM_SEQ;
    for (int j = tid; j < NTmax; j += TBL_THREADS) {
        if (j >= total) {
            t.chunk_tok0_[j] = 0;
            t.chunk_len_[j] = 0;
            t.chunk_seq_[j] = 0;
            continue;
        }
        int lo = 0, hi = S - 1;   // last sequence whose first chunk is <= j (empty sequences share an offset)
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            const int c = in_smem ? s_c0[mid] : t.seq_chunk0_[mid];
            if (c <= j) lo = mid;
            else hi = mid - 1;
        }
        const int s = lo;
        const int c0 = in_smem ? s_c0[s] : t.seq_chunk0_[s];
        int t0 = s * T_dense, len = T_dense;
        if (cu) {
            bool bad;
            clamped_sequence(cu, s, T_dense, t0, len, bad);
        }
        const int rem = len - (j - c0) * CH;
        t.chunk_tok0_[j] = t0 + (j - c0) * CH;
        t.chunk_len_[j] = rem < CH ? rem : CH;
        t.chunk_seq_[j] = s;
    }
    // The chunks sorted by the step at which their chain needs them when every chain is to END at the same
    // time: chunk n of a sequence of nc chunks has the key longest - nc + n, so a short sequence starts
    // late and the longest ones are served first (a counting sort; the order among chunks of equal key
    // is whatever the atomics give).  pos_: [0] longest sequence in chunks, [2 + key] number of chunks
    // with that key, then its running offset, [2 + NTmax + 1 + key] fill counter.
    int* cnt = t.pos_ + 2;
    int* fill = t.pos_ + 3 + NTmax;
    for (int j = tid; j <= NTmax; j += TBL_THREADS) {
        cnt[j] = 0;
        if (j < NTmax) fill[j] = 0;
    }
    if (tid == 0) t.pos_[0] = 0;
    __syncthreads();
    for (int s = tid; s < S; s += TBL_THREADS) atomicMax(&t.pos_[0], t.seq_chunk0_[s + 1] - t.seq_chunk0_[s]);
    __syncthreads();
    const int maxn = t.pos_[0];
    auto key_of = [&](int j) {
        const int s = t.chunk_seq_[j];
        const int c0 = in_smem ? s_c0[s] : t.seq_chunk0_[s], c1 = in_smem ? s_c0[s + 1] : t.seq_chunk0_[s + 1];
        return maxn - (c1 - c0) + (j - c0);
    };
    for (int j = tid; j < total; j += TBL_THREADS) atomicAdd(&cnt[key_of(j)], 1);
    __syncthreads();
    if (tid == 0) s_carry = 0;
    __syncthreads();
    for (int base = 0; base < maxn; base += TBL_THREADS) {   // exclusive scan of the counts, in place
        const int n = base + tid;
        const int v = n < maxn ? cnt[n] : 0;
        s_scan[tid] = v;
        __syncthreads();
        for (int o = 1; o < TBL_THREADS; o <<= 1) {
            const int u = tid >= o ? s_scan[tid - o] : 0;
            __syncthreads();
            s_scan[tid] += u;
            __syncthreads();
        }
        const int carry = s_carry;
        if (n < maxn) cnt[n] = carry + s_scan[tid] - v;
        __syncthreads();
        if (tid == TBL_THREADS - 1) s_carry = carry + s_scan[tid];
        __syncthreads();
    }
    for (int j = tid; j < total; j += TBL_THREADS) {
        const int n = key_of(j);
        t.order_[cnt[n] + atomicAdd(&fill[n], 1)] = j;
    }
    for (int s = tid; s < S; s += TBL_THREADS) {
        const int nc = t.seq_chunk0_[s + 1] - t.seq_chunk0_[s];
        t.seq_first_[s] = nc > 0 ? cnt[maxn - nc] : 0;
    }
}

__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// ---------------------------------------------------------------------------------------
// CTA-wide small matrix product with operand access through functors:
//   acc(m, n) = sum_{k < K1} a1(m,k) b1(k,n) + sum_{k < K2} a2(m,k) b2(k,n);  epi(m, n, acc)
// Thread tiles are TM x TN; columns of a tile are strided by N/TN so that neighbouring
// threads touch neighbouring columns.
// ---------------------------------------------------------------------------------------
template <int M, int N, int TM, int TN, class A1, class B1, class A2, class B2, class E>
__device__ __forceinline__ void cta_mm2(int K1, A1 a1, B1 b1, int K2, A2 a2, B2 b2, E epi)
{
    constexpr int TN_CNT = N / TN, TM_CNT = M / TM;
    for (int tile = threadIdx.x; tile < TN_CNT * TM_CNT; tile += NTH) {
        const int tn = tile % TN_CNT, tm = tile / TN_CNT;
        float acc[TM][TN];
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;
        for (int k = 0; k < K1; ++k) {
            float av[TM], bv[TN];
#pragma unroll
            for (int i = 0; i < TM; ++i) av[i] = a1(tm * TM + i, k);
#pragma unroll
            for (int j = 0; j < TN; ++j) bv[j] = b1(k, tn + j * TN_CNT);
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        for (int k = 0; k < K2; ++k) {
            float av[TM], bv[TN];
#pragma unroll
            for (int i = 0; i < TM; ++i) av[i] = a2(tm * TM + i, k);
#pragma unroll
            for (int j = 0; j < TN; ++j) bv[j] = b2(k, tn + j * TN_CNT);
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < TN; ++j) epi(tm * TM + i, tn + j * TN_CNT, acc[i][j]);
    }
}

struct ZeroOp {
    __device__ __forceinline__ float operator()(int, int) const { return 0.f; }
};

template <int M, int N, int TM, int TN, class A1, class B1, class E>
__device__ __forceinline__ void cta_mm(int K1, A1 a1, B1 b1, E epi)
{
    cta_mm2<M, N, TM, TN>(K1, a1, b1, 0, ZeroOp(), ZeroOp(), epi);
}

// In-chunk gate prefix and the factors derived from it (thread 0 does the 64-term prefix).
struct GateVecs {
    float G[CH], gam[CH], rho[CH], beta[CH];
    float gC;
};

__device__ __forceinline__ void load_gates(GateVecs& gv, const float* __restrict__ gate,
                                           const float* __restrict__ beta, int tok0, int len, int H, int h)
{
    if (threadIdx.x < CH) {
        const int i = threadIdx.x;
        gv.G[i] = i < len ? gate[(size_t)(tok0 + i) * H + h] : 0.f;
        gv.beta[i] = i < len ? beta[(size_t)(tok0 + i) * H + h] : 0.f;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float acc = 0.f;
        for (int i = 0; i < CH; ++i) { acc += gv.G[i]; gv.G[i] = acc; }
        gv.gC = expf(acc);
    }
    __syncthreads();
    if (threadIdx.x < CH) {
        const int i = threadIdx.x;
        gv.gam[i] = expf(gv.G[i]);
        gv.rho[i] = expf(gv.G[CH - 1] - gv.G[i]);
    }
    __syncthreads();
}

// Load a [64 x D] token tile (rows beyond len are zero) from a packed [T,H,D] tensor.
template <typename T, int D>
__device__ __forceinline__ void load_tile(float* dst, int ld, const T* __restrict__ src, int tok0, int len,
                                          int H, int h)
{
    for (int e = threadIdx.x; e < CH * D; e += NTH) {
        const int i = e / D, c = e % D;
        dst[i * ld + c] = i < len ? ldf(src + ((size_t)(tok0 + i) * H + h) * D + c) : 0.f;
    }
}

// ---------------------------------------------------------------------------------------
// chunk-local forward: A, T = (I + A)^-1, W, U, P
// ---------------------------------------------------------------------------------------
struct ChunkArgs {
    int H;
    Table tab;
    const void *q, *k, *v;
    const float *beta, *gate;
    const float* ktil;
    float *Tm, *P, *W, *U;
    // backward extras
    const void* dout;
    const float *Sn, *dSn, *dU, *ddU;
    float *scr, *dktil, *dkread;
    void *dq, *dv;
    float *dbeta, *dgate;
    Hyper hy;
};

template <typename T, int K, int V>
__global__ void __launch_bounds__(NTH) chunk_local_fwd_kernel(ChunkArgs a)
{
    extern __shared__ float sm[];
    constexpr int LD = K + 1, LC = CH + 1;
    float* sK = sm;
    float* sKt = sK + CH * LD;
    float* sQ = sKt + CH * LD;
    float* sT = sQ + CH * LD;
    float* sA = sT + CH * LC;
    __shared__ GateVecs gv;

    const int c = blockIdx.x, h = blockIdx.y, H = a.H;
    const int len = a.tab.chunk_len(c);
    if (len == 0) return;
    const int tok0 = a.tab.chunk_tok0(c);
    const size_t tile = (size_t)c * H + h;

    load_tile<T, K>(sK, LD, static_cast<const T*>(a.k), tok0, len, H, h);
    load_tile<float, K>(sKt, LD, a.ktil, tok0, len, H, h);
    load_tile<T, K>(sQ, LD, static_cast<const T*>(a.q), tok0, len, H, h);
    load_gates(gv, a.gate, a.beta, tok0, len, H, h);

    // A_ij = 1[j<i] beta_i Gamma_ij <k_i, ktil_j>
    cta_mm<CH, CH, 4, 4>(
        K, [&](int m, int k) { return sK[m * LD + k]; }, [&](int k, int n) { return sKt[n * LD + k]; },
        [&](int i, int j, float acc) {
            sA[i * LC + j] = j < i ? gv.beta[i] * expf(gv.G[i] - gv.G[j]) * acc : 0.f;
        });
    // P_ij = 1[j<=i] Gamma_ij <q_i, ktil_j>
    float* Pg = a.P + tile * CH * CH;
    cta_mm<CH, CH, 4, 4>(
        K, [&](int m, int k) { return sQ[m * LD + k]; }, [&](int k, int n) { return sKt[n * LD + k]; },
        [&](int i, int j, float acc) { Pg[i * CH + j] = j <= i ? expf(gv.G[i] - gv.G[j]) * acc : 0.f; });
    __syncthreads();

    // T = (I + A)^-1 by forward substitution; column `col` of T solves (I + A) x = e_col.
    // Four lanes share a column and split the inner sum.
    {
        const int col = threadIdx.x >> 2, part = threadIdx.x & 3;
        for (int i = 0; i < CH; ++i) {
            float sum = 0.f;   // empty for i <= col; the shuffles stay outside any divergent branch
            for (int j = col + part; j < i; j += 4) sum = fmaf(sA[i * LC + j], sT[j * LC + col], sum);
            sum += __shfl_xor_sync(0xffffffffu, sum, 1);
            sum += __shfl_xor_sync(0xffffffffu, sum, 2);
            const float x = i < col ? 0.f : (i == col ? 1.f : -sum);
            if (part == 0) sT[i * LC + col] = x;
            __syncwarp();
        }
    }
    __syncthreads();
    float* Tg = a.Tm + tile * CH * CH;
    for (int e = threadIdx.x; e < CH * CH; e += NTH) Tg[e] = sT[(e / CH) * LC + (e % CH)];

    // W = T diag(beta gamma) K ; U = T diag(beta) V
    float* Wg = a.W + tile * CH * K;
    cta_mm<CH, K, 4, K / 16>(
        CH, [&](int m, int j) { return sT[m * LC + j] * gv.beta[j] * gv.gam[j]; },
        [&](int j, int n) { return sK[j * LD + n]; }, [&](int m, int n, float acc) { Wg[m * K + n] = acc; });
    float* Ug = a.U + tile * CH * V;
    const T* vp = static_cast<const T*>(a.v);
    cta_mm<CH, V, 4, V / 16>(
        CH, [&](int m, int j) { return sT[m * LC + j] * gv.beta[j]; },
        [&](int j, int n) { return j < len ? ldf(vp + ((size_t)(tok0 + j) * H + h) * V + n) : 0.f; },
        [&](int m, int n, float acc) { Ug[m * V + n] = acc; });
}

// ---------------------------------------------------------------------------------------
// state chain, forward.  One CTA per (chain, slice of VS state rows).
// ---------------------------------------------------------------------------------------
struct ChainArgs {
    int S, H;
    Table tab;
    const void* q;
    const float *gate, *beta, *ktil, *W, *U, *P, *init_state;
    void* out;
    float *final_state, *Sn, *dU;
    int save;
    // backward
    const void* dout;
    const float* dfinal_state;
    float *ddU, *dSn, *dinit_state;
    Hyper hy;
};

template <typename T, int K, int V, int VS>
__global__ void __launch_bounds__(NTH) chain_fwd_kernel(ChainArgs a)
{
    extern __shared__ float sm[];
    constexpr int LD = K + 1, LC = CH + 1, LV = VS + 1;
    float* sS = sm;                 // [VS][LD]
    float* sW = sS + VS * LD;       // [64][LD]
    float* sKt = sW + CH * LD;
    float* sQ = sKt + CH * LD;
    float* sP = sQ + CH * LD;       // [64][LC]
    float* sU = sP + CH * LC;       // [64][LV]  U slice, then dU
    float* sO = sU + CH * LV;       // [64][LV]
    __shared__ GateVecs gv;

    const int chain = blockIdx.x, H = a.H;
    const int s = chain / H, h = chain % H;
    const int v0 = blockIdx.y * VS;
    const int c0 = a.tab.seq_chunk0(s), c1 = a.tab.seq_chunk0(s + 1);
    const float scale = a.hy.scale;

    for (int e = threadIdx.x; e < VS * K; e += NTH) {
        const int r = e / K, k = e % K;
        sS[r * LD + k] = a.init_state ? a.init_state[(((size_t)s * H + h) * V + v0 + r) * K + k] : 0.f;
    }
    T* outp = static_cast<T*>(a.out);
    for (int c = c0; c < c1; ++c) {
        const int tok0 = a.tab.chunk_tok0(c), len = a.tab.chunk_len(c);
        const size_t tile = (size_t)c * H + h;
        __syncthreads();
        for (int e = threadIdx.x; e < CH * K; e += NTH) sW[(e / K) * LD + e % K] = a.W[tile * CH * K + e];
        load_tile<float, K>(sKt, LD, a.ktil, tok0, len, H, h);
        load_tile<T, K>(sQ, LD, static_cast<const T*>(a.q), tok0, len, H, h);
        for (int e = threadIdx.x; e < CH * CH; e += NTH) sP[(e / CH) * LC + e % CH] = a.P[tile * CH * CH + e];
        for (int e = threadIdx.x; e < CH * VS; e += NTH)
            sU[(e / VS) * LV + e % VS] = a.U[tile * CH * V + (size_t)(e / VS) * V + v0 + e % VS];
        if (a.save)
            for (int e = threadIdx.x; e < VS * K; e += NTH)
                a.Sn[(tile * V + v0 + e / K) * K + e % K] = sS[(e / K) * LD + e % K];
        load_gates(gv, a.gate, a.beta, tok0, len, H, h);

        // dU = U - W S^T
        cta_mm<CH, VS, 2, VS / 8>(
            K, [&](int m, int k) { return sW[m * LD + k]; }, [&](int k, int n) { return sS[n * LD + k]; },
            [&](int m, int n, float acc) { sU[m * LV + n] -= acc; });
        __syncthreads();
        if (a.save)
            for (int e = threadIdx.x; e < CH * VS; e += NTH)
                a.dU[tile * CH * V + (size_t)(e / VS) * V + v0 + e % VS] = sU[(e / VS) * LV + e % VS];
        // O = scale [ (gamma Q) S^T + P dU ]
        cta_mm2<CH, VS, 2, VS / 8>(
            K, [&](int m, int k) { return gv.gam[m] * sQ[m * LD + k]; },
            [&](int k, int n) { return sS[n * LD + k]; }, CH, [&](int m, int j) { return sP[m * LC + j]; },
            [&](int j, int n) { return sU[j * LV + n]; },
            [&](int m, int n, float acc) { sO[m * LV + n] = scale * acc; });
        __syncthreads();
        for (int e = threadIdx.x; e < CH * VS; e += NTH) {
            const int i = e / VS, n = e % VS;
            if (i < len) stf(outp + ((size_t)(tok0 + i) * H + h) * V + v0 + n, sO[i * LV + n]);
        }
        // S <- gamma_C S + dU^T (rho Ktil)
        cta_mm<VS, K, 2, K / 16>(
            CH, [&](int m, int i) { return sU[i * LV + m]; },
            [&](int i, int n) { return gv.rho[i] * sKt[i * LD + n]; },
            [&](int m, int n, float acc) { sS[m * LD + n] = gv.gC * sS[m * LD + n] + acc; });
    }
    __syncthreads();
    if (a.final_state)
        for (int e = threadIdx.x; e < VS * K; e += NTH)
            a.final_state[(((size_t)s * H + h) * V + v0 + e / K) * K + e % K] = sS[(e / K) * LD + e % K];
}

// ---------------------------------------------------------------------------------------
// state chain, backward (reverse over chunks)
//   ddU = scale P^T dO + (rho Ktil) dS^T ;  dS <- gamma_C dS + scale dO^T (gamma Q) - ddU^T W
// ---------------------------------------------------------------------------------------
template <typename T, int K, int V, int VS>
__global__ void __launch_bounds__(NTH) chain_bwd_kernel(ChainArgs a)
{
    extern __shared__ float sm[];
    constexpr int LD = K + 1, LC = CH + 1, LV = VS + 1;
    float* sdS = sm;                // [VS][LD]
    float* sW = sdS + VS * LD;
    float* sKt = sW + CH * LD;
    float* sQ = sKt + CH * LD;
    float* sP = sQ + CH * LD;       // [64][LC]
    float* sdO = sP + CH * LC;      // [64][LV]
    float* sddU = sdO + CH * LV;    // [64][LV]
    __shared__ GateVecs gv;

    const int chain = blockIdx.x, H = a.H;
    const int s = chain / H, h = chain % H;
    const int v0 = blockIdx.y * VS;
    const int c0 = a.tab.seq_chunk0(s), c1 = a.tab.seq_chunk0(s + 1);
    const float scale = a.hy.scale;

    for (int e = threadIdx.x; e < VS * K; e += NTH) {
        const int r = e / K, k = e % K;
        sdS[r * LD + k] = a.dfinal_state ? a.dfinal_state[(((size_t)s * H + h) * V + v0 + r) * K + k] : 0.f;
    }
    const T* dop = static_cast<const T*>(a.dout);
    for (int c = c1 - 1; c >= c0; --c) {
        const int tok0 = a.tab.chunk_tok0(c), len = a.tab.chunk_len(c);
        const size_t tile = (size_t)c * H + h;
        __syncthreads();
        for (int e = threadIdx.x; e < CH * K; e += NTH) sW[(e / K) * LD + e % K] = a.W[tile * CH * K + e];
        load_tile<float, K>(sKt, LD, a.ktil, tok0, len, H, h);
        load_tile<T, K>(sQ, LD, static_cast<const T*>(a.q), tok0, len, H, h);
        for (int e = threadIdx.x; e < CH * CH; e += NTH) sP[(e / CH) * LC + e % CH] = a.P[tile * CH * CH + e];
        for (int e = threadIdx.x; e < CH * VS; e += NTH) {
            const int i = e / VS, n = e % VS;
            sdO[i * LV + n] = i < len ? ldf(dop + ((size_t)(tok0 + i) * H + h) * V + v0 + n) : 0.f;
        }
        for (int e = threadIdx.x; e < VS * K; e += NTH)
            a.dSn[(tile * V + v0 + e / K) * K + e % K] = sdS[(e / K) * LD + e % K];
        load_gates(gv, a.gate, a.beta, tok0, len, H, h);

        cta_mm2<CH, VS, 2, VS / 8>(
            CH, [&](int i, int j) { return scale * sP[j * LC + i]; }, [&](int j, int n) { return sdO[j * LV + n]; },
            K, [&](int i, int k) { return gv.rho[i] * sKt[i * LD + k]; },
            [&](int k, int n) { return sdS[n * LD + k]; },
            [&](int i, int n, float acc) { sddU[i * LV + n] = acc; });
        __syncthreads();
        for (int e = threadIdx.x; e < CH * VS; e += NTH)
            a.ddU[tile * CH * V + (size_t)(e / VS) * V + v0 + e % VS] = sddU[(e / VS) * LV + e % VS];
        cta_mm2<VS, K, 2, K / 16>(
            CH, [&](int m, int i) { return scale * sdO[i * LV + m]; },
            [&](int i, int n) { return gv.gam[i] * sQ[i * LD + n]; }, CH,
            [&](int m, int i) { return -sddU[i * LV + m]; }, [&](int i, int n) { return sW[i * LD + n]; },
            [&](int m, int n, float acc) { sdS[m * LD + n] = gv.gC * sdS[m * LD + n] + acc; });
    }
    __syncthreads();
    if (a.dinit_state)
        for (int e = threadIdx.x; e < VS * K; e += NTH)
            a.dinit_state[(((size_t)s * H + h) * V + v0 + e / K) * K + e % K] = sdS[(e / K) * LD + e % K];
}

// ---------------------------------------------------------------------------------------
// chunk-local backward: gradients through P, the state-advance factors, W, U, T, A, gates
// ---------------------------------------------------------------------------------------
template <typename T, int K, int V>
__global__ void __launch_bounds__(NTH) chunk_local_bwd_kernel(ChunkArgs a)
{
    extern __shared__ float sm[];
    constexpr int LD = K + 1, LC = CH + 1;
    constexpr int D = K > V ? K : V;
    float* sK = sm;
    float* sKt = sK + CH * LD;
    float* sQ = sKt + CH * LD;
    float* sT = sQ + CH * LD;       // [64][LC]
    float* sX = sT + CH * LC;       // dT, later dA * beta_i * Gamma_ij
    float* sY = sX + CH * LC;       // scratch
    float* sDP = sY + CH * LC;      // dP * Gamma
    __shared__ GateVecs gv;
    __shared__ float sdG[CH], sdB[CH], sR[CH], sRed[NTH / 32];

    const int c = blockIdx.x, h = blockIdx.y, H = a.H;
    const int len = a.tab.chunk_len(c);
    if (len == 0) return;
    const int tok0 = a.tab.chunk_tok0(c);
    const size_t tile = (size_t)c * H + h;
    const float scale = a.hy.scale;

    const T* vp = static_cast<const T*>(a.v);
    const T* dop = static_cast<const T*>(a.dout);
    const float* Sg = a.Sn + tile * V * K;
    const float* dSg = a.dSn + tile * V * K;
    const float* dUg = a.dU + tile * CH * V;
    const float* ddUg = a.ddU + tile * CH * V;
    const float* Pg = a.P + tile * CH * CH;
    float* scr = a.scr + tile * 5 * CH * D;
    float* gdQ = scr;                 // gamma_i * dQg
    float* gdKt = scr + CH * D;       // rho_j * dKtr
    float* gdW = scr + 2 * CH * D;
    float* gdK = scr + 3 * CH * D;    // beta gamma dKb
    auto vld = [&](int j, int n) { return j < len ? ldf(vp + ((size_t)(tok0 + j) * H + h) * V + n) : 0.f; };
    auto dold = [&](int i, int n) { return i < len ? ldf(dop + ((size_t)(tok0 + i) * H + h) * V + n) : 0.f; };

    load_tile<T, K>(sK, LD, static_cast<const T*>(a.k), tok0, len, H, h);
    load_tile<float, K>(sKt, LD, a.ktil, tok0, len, H, h);
    load_tile<T, K>(sQ, LD, static_cast<const T*>(a.q), tok0, len, H, h);
    for (int e = threadIdx.x; e < CH * CH; e += NTH) sT[(e / CH) * LC + e % CH] = a.Tm[tile * CH * CH + e];
    if (threadIdx.x < CH) { sdG[threadIdx.x] = 0.f; sdB[threadIdx.x] = 0.f; sR[threadIdx.x] = 0.f; }
    load_gates(gv, a.gate, a.beta, tok0, len, H, h);

    // <dS, S>_F (for the gradient of the chunk-level decay gamma_C)
    {
        float part = 0.f;
        for (int e = threadIdx.x; e < V * K; e += NTH) part = fmaf(Sg[e], dSg[e], part);
        part = warp_sum(part);
        if ((threadIdx.x & 31) == 0) sRed[threadIdx.x >> 5] = part;
    }

    // (1) dP = 1[j<=i] scale dO dU^T ;  sDP = dP * Gamma ;  sY = dP * P
    cta_mm<CH, CH, 4, 4>(
        V, [&](int i, int n) { return scale * dold(i, n); }, [&](int n, int j) { return dUg[j * V + n]; },
        [&](int i, int j, float acc) {
            const float dp = j <= i ? acc : 0.f;
            sDP[i * LC + j] = dp * expf(fminf(gv.G[i] - gv.G[j], 0.f));
            sY[i * LC + j] = dp * Pg[i * CH + j];
        });
    __syncthreads();
    if (threadIdx.x < CH) {
        const int i = threadIdx.x;
        float r = 0.f, cs = 0.f;
        for (int j = 0; j < CH; ++j) { r += sY[i * LC + j]; cs += sY[j * LC + i]; }
        sdG[i] += r - cs;   // only this thread touches sdG[i] here
    }
    __syncthreads();

    // (2) gamma_i * dQg = gamma_i scale dO S ; dq = that + (dP Gamma) Ktil
    cta_mm<CH, K, 4, K / 16>(
        V, [&](int i, int n) { return scale * gv.gam[i] * dold(i, n); }, [&](int n, int k) { return Sg[n * K + k]; },
        [&](int i, int k, float acc) {
            gdQ[i * K + k] = acc;
            atomicAdd(&sdG[i], acc * sQ[i * LD + k]);
        });
    T* dqp = static_cast<T*>(a.dq);
    cta_mm<CH, K, 4, K / 16>(
        CH, [&](int i, int j) { return sDP[i * LC + j]; }, [&](int j, int k) { return sKt[j * LD + k]; },
        [&](int i, int k, float acc) {
            if (i < len) stf(dqp + ((size_t)(tok0 + i) * H + h) * K + k, gdQ[i * K + k] + acc);
        });

    // (3) rho_j * dKtr = rho_j dU dS ; r_j = <rho_j dKtr_j, ktil_j>
    cta_mm<CH, K, 4, K / 16>(
        V, [&](int j, int n) { return gv.rho[j] * dUg[j * V + n]; }, [&](int n, int k) { return dSg[n * K + k]; },
        [&](int j, int k, float acc) {
            gdKt[j * K + k] = acc;
            atomicAdd(&sR[j], acc * sKt[j * LD + k]);
        });

    // (4) dW = -ddU S
    cta_mm<CH, K, 4, K / 16>(
        V, [&](int i, int n) { return -ddUg[i * V + n]; }, [&](int n, int k) { return Sg[n * K + k]; },
        [&](int i, int k, float acc) { gdW[i * K + k] = acc; });
    __syncthreads();
    //     dT = dW Kb^T + ddU Vb^T
    cta_mm2<CH, CH, 4, 4>(
        K, [&](int i, int k) { return gdW[i * K + k]; },
        [&](int k, int j) { return gv.beta[j] * gv.gam[j] * sK[j * LD + k]; }, V,
        [&](int i, int n) { return ddUg[i * V + n]; }, [&](int n, int j) { return gv.beta[j] * vld(j, n); },
        [&](int i, int j, float acc) { sX[i * LC + j] = acc; });

    // (5) dKb = T^T dW ; dVb = T^T ddU
    cta_mm<CH, K, 4, K / 16>(
        CH, [&](int j, int i) { return sT[i * LC + j]; }, [&](int i, int k) { return gdW[i * K + k]; },
        [&](int j, int k, float acc) {
            const float gk = gv.gam[j] * sK[j * LD + k];
            gdK[j * K + k] = gv.beta[j] * gv.gam[j] * acc;
            atomicAdd(&sdB[j], acc * gk);
            atomicAdd(&sdG[j], acc * gv.beta[j] * gk);
        });
    T* dvp = static_cast<T*>(a.dv);
    cta_mm<CH, V, 4, V / 16>(
        CH, [&](int j, int i) { return sT[i * LC + j]; }, [&](int i, int n) { return ddUg[i * V + n]; },
        [&](int j, int n, float acc) {
            if (j < len) stf(dvp + ((size_t)(tok0 + j) * H + h) * V + n, gv.beta[j] * acc);
            atomicAdd(&sdB[j], acc * vld(j, n));
        });
    __syncthreads();

    // (6) dA = -strictLower(T^T dT T^T)
    cta_mm<CH, CH, 4, 4>(
        CH, [&](int x, int i) { return sT[i * LC + x]; }, [&](int i, int y) { return sX[i * LC + y]; },
        [&](int x, int y, float acc) { sY[x * LC + y] = acc; });
    __syncthreads();
    cta_mm<CH, CH, 4, 4>(
        CH, [&](int x, int z) { return sY[x * LC + z]; }, [&](int z, int y) { return sT[y * LC + z]; },
        [&](int x, int y, float acc) { sX[x * LC + y] = y < x ? -acc : 0.f; });
    __syncthreads();
    //     raw Gram once more: dbeta_i += dA_ij Gamma_ij <k_i,ktil_j>; dG from dA (.) A; sX <- dA beta_i Gamma_ij
    cta_mm<CH, CH, 4, 4>(
        K, [&](int i, int k) { return sK[i * LD + k]; }, [&](int k, int j) { return sKt[j * LD + k]; },
        [&](int i, int j, float raw) {
            const float da = sX[i * LC + j];
            const float gm = j < i ? expf(gv.G[i] - gv.G[j]) : 0.f;
            const float t = da * gm * raw;
            if (j < i) {
                atomicAdd(&sdB[i], t);
                atomicAdd(&sdG[i], t * gv.beta[i]);
                atomicAdd(&sdG[j], -t * gv.beta[i]);
            }
            sX[i * LC + j] = da * gv.beta[i] * gm;
        });
    __syncthreads();

    // (7) dk (read side) and dktil
    float* dkr = a.dkread;
    cta_mm<CH, K, 4, K / 16>(
        CH, [&](int i, int j) { return sX[i * LC + j]; }, [&](int j, int k) { return sKt[j * LD + k]; },
        [&](int i, int k, float acc) {
            if (i < len) dkr[((size_t)(tok0 + i) * H + h) * K + k] = gdK[i * K + k] + acc;
        });
    float* dkt = a.dktil;
    cta_mm2<CH, K, 4, K / 16>(
        CH, [&](int j, int i) { return sDP[i * LC + j]; }, [&](int i, int k) { return sQ[i * LD + k]; }, CH,
        [&](int j, int i) { return sX[i * LC + j]; }, [&](int i, int k) { return sK[i * LD + k]; },
        [&](int j, int k, float acc) {
            if (j < len) dkt[((size_t)(tok0 + j) * H + h) * K + k] = gdKt[j * K + k] + acc;
        });
    __syncthreads();

    // (8) gate gradients: reverse in-chunk prefix of dG; phase-2 part of dbeta
    if (threadIdx.x == 0) {
        float tot = 0.f;
        for (int w = 0; w < NTH / 32; ++w) tot += sRed[w];
        float rsum = 0.f;
        for (int j = 0; j < CH; ++j) { rsum += sR[j]; sdG[j] -= sR[j]; }
        sdG[CH - 1] += rsum + gv.gC * tot;
        float acc = 0.f;
        for (int i = CH - 1; i >= 0; --i) { acc += sdG[i]; sdG[i] = acc; }
    }
    __syncthreads();
    if (threadIdx.x < len) {
        const size_t th = (size_t)(tok0 + threadIdx.x) * H + h;
        a.dgate[th] = sdG[threadIdx.x];
        a.dbeta[th] = sdB[threadIdx.x];
    }
}

template <typename F> bool set_smem(F* kernel, size_t bytes)
{
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess;
}

constexpr int VSL = 32;  // state rows per chain CTA

template <typename T, int K, int V>
int fwd_impl(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
             bool save, cudaStream_t st)
{
    char* w = static_cast<char*>(ws);
    Table tab = carve_table(ws, L);
    int launches = 0;
    const int S = L.S, H = p.H;
    {
        const int n1 = phase1_forward(p, hy, L, ws, a, w + L.ktil, false, save, st);
        if (n1 < 0) return -1;
        launches += n1;
    }
    {
        ChunkArgs ca{};
        ca.H = H; ca.tab = tab; ca.q = a.q; ca.k = a.k; ca.v = a.v; ca.beta = a.beta; ca.gate = a.gate;
        ca.ktil = reinterpret_cast<float*>(w + L.ktil);
        ca.Tm = reinterpret_cast<float*>(w + L.Tm); ca.P = reinterpret_cast<float*>(w + L.P);
        ca.W = reinterpret_cast<float*>(w + L.W); ca.U = reinterpret_cast<float*>(w + L.U);
        ca.hy = hy;
        const size_t smem = sizeof(float) * (3 * CH * (K + 1) + 2 * CH * (CH + 1));
        if (!set_smem(chunk_local_fwd_kernel<T, K, V>, smem)) return -1;
        stage_mark(st, "simt_chunk_local_fwd");
        chunk_local_fwd_kernel<T, K, V><<<dim3(L.NTmax, H), NTH, smem, st>>>(ca);
        ++launches;
    }
    {
        ChainArgs ch{};
        ch.S = S; ch.H = H; ch.tab = tab; ch.q = a.q; ch.gate = a.gate; ch.beta = a.beta;
        ch.ktil = reinterpret_cast<float*>(w + L.ktil);
        ch.W = reinterpret_cast<float*>(w + L.W); ch.U = reinterpret_cast<float*>(w + L.U);
        ch.P = reinterpret_cast<float*>(w + L.P);
        ch.init_state = a.init_state; ch.out = a.out; ch.final_state = a.final_state;
        ch.Sn = reinterpret_cast<float*>(w + L.Sn); ch.dU = reinterpret_cast<float*>(w + L.dU);
        ch.save = save ? 1 : 0; ch.hy = hy;
        const size_t smem = sizeof(float) * (VSL * (K + 1) + 3 * CH * (K + 1) + CH * (CH + 1) + 2 * CH * (VSL + 1));
        if (!set_smem(chain_fwd_kernel<T, K, V, VSL>, smem)) return -1;
        stage_mark(st, "simt_chain_fwd");
        chain_fwd_kernel<T, K, V, VSL><<<dim3(S * H, V / VSL), NTH, smem, st>>>(ch);
        ++launches;
    }
    stage_end(st);
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

template <typename T, int K, int V>
int bwd_impl(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
             cudaStream_t st)
{
    char* w = static_cast<char*>(ws);
    Table tab = carve_table(ws, L);
    int launches = 0;
    const int S = L.S, H = p.H;
    auto F = [&](size_t off) { return reinterpret_cast<float*>(w + off); };
    {
        ChainArgs ch{};
        ch.S = S; ch.H = H; ch.tab = tab; ch.q = a.q; ch.gate = a.gate; ch.beta = a.beta;
        ch.ktil = F(L.ktil); ch.W = F(L.W); ch.P = F(L.P);
        ch.dout = a.dout; ch.dfinal_state = a.dfinal_state; ch.ddU = F(L.ddU); ch.dSn = F(L.dSn);
        ch.dinit_state = a.dinit_state; ch.hy = hy;
        const size_t smem = sizeof(float) * (VSL * (K + 1) + 3 * CH * (K + 1) + CH * (CH + 1) + 2 * CH * (VSL + 1));
        if (!set_smem(chain_bwd_kernel<T, K, V, VSL>, smem)) return -1;
        stage_mark(st, "simt_chain_bwd");
        chain_bwd_kernel<T, K, V, VSL><<<dim3(S * H, V / VSL), NTH, smem, st>>>(ch);
        ++launches;
    }
    {
        ChunkArgs ca{};
        ca.H = H; ca.tab = tab; ca.q = a.q; ca.k = a.k; ca.v = a.v; ca.beta = a.beta; ca.gate = a.gate;
        ca.ktil = F(L.ktil); ca.Tm = F(L.Tm); ca.P = F(L.P); ca.W = F(L.W); ca.U = F(L.U);
        ca.dout = a.dout; ca.Sn = F(L.Sn); ca.dSn = F(L.dSn); ca.dU = F(L.dU); ca.ddU = F(L.ddU);
        ca.scr = F(L.scr); ca.dktil = F(L.dktil); ca.dkread = F(L.dkread);
        ca.dq = a.dq; ca.dv = a.dv; ca.dbeta = a.dbeta; ca.dgate = a.dgate; ca.hy = hy;
        const size_t smem = sizeof(float) * (3 * CH * (K + 1) + 4 * CH * (CH + 1));
        if (!set_smem(chunk_local_bwd_kernel<T, K, V>, smem)) return -1;
        stage_mark(st, "simt_chunk_local_bwd");
        chunk_local_bwd_kernel<T, K, V><<<dim3(L.NTmax, H), NTH, smem, st>>>(ca);
        ++launches;
    }
    {
        const int n1 = phase1_backward(p, hy, L, ws, a, F(L.dktil), F(L.dkread), true, st);
        if (n1 < 0) return -1;
        launches += n1;
    }
    stage_end(st);
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace

int launch_build_table(const osdn_params& p, const WsLayout& L, void* ws, cudaStream_t st)
{
    Table tab = carve_table(ws, L);
    if (L.dense_T) return 0;   // dense batch: the table is arithmetic, nothing to build
    stage_mark(st, "build_table");
    build_table_kernel<<<1, TBL_THREADS, 0, st>>>(L.S, p.T, p.cu_seqlens, L.NTmax, tab,
                                                  reinterpret_cast<int*>(static_cast<char*>(ws) + L.status));
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

#define OSDN_DISPATCH(FN, ...)                                                              \
    do {                                                                                    \
        if (p.io_dtype == OSDN_FP32) {                                                      \
            if (p.K == 64 && p.V == 64) return FN<float, 64, 64>(__VA_ARGS__);              \
            if (p.K == 128 && p.V == 128) return FN<float, 128, 128>(__VA_ARGS__);          \
            if (p.K == 64 && p.V == 128) return FN<float, 64, 128>(__VA_ARGS__);            \
            if (p.K == 128 && p.V == 64) return FN<float, 128, 64>(__VA_ARGS__);            \
        } else {                                                                            \
            if (p.K == 64 && p.V == 64) return FN<__nv_bfloat16, 64, 64>(__VA_ARGS__);      \
            if (p.K == 128 && p.V == 128) return FN<__nv_bfloat16, 128, 128>(__VA_ARGS__);  \
            if (p.K == 64 && p.V == 128) return FN<__nv_bfloat16, 64, 128>(__VA_ARGS__);    \
            if (p.K == 128 && p.V == 64) return FN<__nv_bfloat16, 128, 64>(__VA_ARGS__);    \
        }                                                                                   \
        return -1;                                                                          \
    } while (0)

int simt_forward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                 bool save, cudaStream_t st)
{
    OSDN_DISPATCH(fwd_impl, p, hy, L, ws, a, save, st);
}

int simt_backward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                  cudaStream_t st)
{
    OSDN_DISPATCH(bwd_impl, p, hy, L, ws, a, st);
}

}  // namespace osdn
