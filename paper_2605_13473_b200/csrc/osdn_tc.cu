// tcgen05 / TMA kernels of the OSDN layer for bf16 I/O, K = V = 128, chunk = 64 (sm_100a).
//
// Data flow of the forward pass (gated chunk form; G_i in-chunk gate prefix, gamma = exp(G),
// Gamma_ij = exp(G_i - G_j), rho_i = exp(G_C - G_i)):
//
//   phase1_fwd (CUDA cores)      ktil = d (.) k in bf16, preconditioner at chunk starts
//   tc_chunk_fwd  per (chunk, head), parallel:
//        [K;Q] Ktil^T  -> A = strictLower(beta_i Gamma_ij <k_i,ktil_j>),  P' = scale * Lower(Gamma_ij <q_i,ktil_j>)
//        T = (I + A)^-1 (fp32 forward substitution), Tb = T diag(beta), Tbg = T diag(beta gamma)
//        W^T = K^T Tbg^T                               (tensor memory: lane = feature, column = token)
//   tc_chain_fwd  per chain, sequential over chunks, state S (V x K, fp32) resident in tensor memory:
//        dU^T = V^T Tb^T - S W^T ;  O1^T = S Q^T
//        O2^T = dU^T P'^T ;         S <- gamma_C S + (rho dU)^T Ktil
//        O^T  = scale gamma_i O1^T + O2^T
//
// Work tiles that travel between kernels are stored in HBM as ready-made images of the
// 128-byte-swizzled shared-memory layout (see umma.cuh), so that the consumer fetches them with a
// plain bulk copy; user tensors (q, k, ktil, v, dout) are fetched with TMA tensor maps.
#include <algorithm>

#include <cuda.h>
#include <cudaTypedefs.h>

#include "osdn_common.cuh"
#include <type_traits>

#include "umma.cuh"

namespace osdn {

using namespace umma;


namespace {

constexpr int KD = 128;  // K = V = 128 on this path
constexpr uint32_t BOX = 8192;   // one [64 rows x 128 B] box

// device status codes of bounded waits
enum { ERR_QUEUE = 121, ERR_READY = 122, ERR_TMA = 101, ERR_MMA1 = 102, ERR_MMA2 = 103, ERR_CHAIN_TMA = 111, ERR_CHAIN_MMA1 = 112, ERR_CHAIN_MMA2 = 113 };

constexpr uint32_t REC_BYTES = 49152;   // stride of the Tb | W^T | P' | Qg record of a tile

struct TcLayout {
    size_t ktil, WT, Tb, Tm, P, Qg, Sn, dUT, ready, ddUT, dSn, dktil, dkread, queue, total;
};

TcLayout make_tc_layout(const osdn_params& p, const WsLayout& L, bool need_bwd)
{
    TcLayout t{};
    const size_t Ttot = p.nseq > 0 ? (size_t)p.T : (size_t)p.B * p.T;
    const size_t H = p.H, NT = L.NTmax;
    size_t off = L.ktil;
    auto take = [&](size_t b) { size_t o = off; off = align_up(off + b, 1024); return o; };
    off = align_up(off, 1024);
    t.ktil = take(Ttot * H * KD * 2);
    // One record per (chunk, head) tile, Tb | W^T | P' | Qg, so that either chain kernel fetches the
    // tiles it needs (the first three forward, the last three backward) with a single bulk copy.
    const size_t rec = take(NT * H * (size_t)REC_BYTES);
    t.Tb = rec;
    t.WT = rec + 8192;
    t.P = rec + 24576;
    t.Qg = rec + 32768;
    t.Tm = take(NT * H * 8192);
    t.Sn = take(NT * H * 32768);
    t.dUT = take(NT * H * 16384);
    t.ready = take(sizeof(int) * (64 + NT * H));   // ticket counter, then one flag per tile
    if (need_bwd) {
        t.ddUT = take(NT * H * 16384);
        t.dSn = take(NT * H * 32768);
        t.dktil = take(Ttot * H * KD * 4);
        t.dkread = take(Ttot * H * KD * 4);
        t.queue = take(sizeof(int) * (64 + NT * H));
    }
    t.total = off;
    return t;
}

// ---------------------------------------------------------------------------------------------
// tensor maps
// ---------------------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled get_encoder()
{
    static PFN_cuTensorMapEncodeTiled fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(ptr);
    }
    return fn;
}

// Map over a packed [rows, H * 128] bf16 tensor; boxes of 64 rows x 64 columns, 128-byte swizzle,
// out-of-range rows read as zero.
bool make_token_map(CUtensorMap* m, const void* base, size_t rows, int H)
{
    PFN_cuTensorMapEncodeTiled enc = get_encoder();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)H * KD, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)H * KD * 2};
    cuuint32_t box[2] = {64, 64};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Map over the same kind of tensor for storing dense [64 tokens x 128 features] tiles (no swizzle).
bool make_store_map(CUtensorMap* m, void* base, size_t rows, int H)
{
    PFN_cuTensorMapEncodeTiled enc = get_encoder();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)H * KD, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)H * KD * 2};
    cuuint32_t box[2] = {KD, 64};
    cuuint32_t estr[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
}

__device__ __forceinline__ uint8_t* align1024(uint8_t* p)
{
    return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

// Zero rows [len, 64) of a box (tail chunks only).
__device__ __forceinline__ void zero_tail_rows(uint8_t* box, int len, int tid, int nthreads)
{
    const int rows = CH - len;
    for (int e = tid; e < rows * 8; e += nthreads)
        *reinterpret_cast<uint4*>(box + (len + e / 8) * 128 + (e % 8) * 16) = make_uint4(0, 0, 0, 0);
}

// ---------------------------------------------------------------------------------------------
// fp32 scratch rows of the chunk-local backward: odd stride, one row per lane without bank conflicts
// ---------------------------------------------------------------------------------------------
constexpr int LC = CH + 1;

// fp32 value as a TF32 operand (round to nearest)
__device__ __forceinline__ uint32_t to_tf32(float x)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}

// Warp-level 16x8x8 TF32 MMA (fp32 accumulate).  The 16 x 16 blocks of the triangular solve are
// below the smallest tcgen05 tile (M = 64), so they use the warp-level tensor path.
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2])
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// ---------------------------------------------------------------------------------------------
// T = (I + A)^-1 for a 64 x 64 strictly lower triangular A, in place (fp32, shared memory, row
// stride LCF), by 16 x 16 blocks: the four diagonal blocks by forward substitution with a column
// per thread in registers, then block row by block row,
//     T_bc = -T_bb sum_{m=c}^{b-1} A_bm T_mc            (c < b),
// where row b of A is still untouched and the rows above already hold T.  The inner sums are
// parked in the upper triangle (block (c, b)), so on return only entries with j <= i are meaningful.
// Called by all threads of the CTA (at least 96); ends with a barrier.
// ---------------------------------------------------------------------------------------------
constexpr int LCF = CH + 4;   // stride = 4 mod 32 words: conflict-free 16-byte row stores and A fragments

// acc (16 x 16, two 16 x 8 fragments) += A (16 x 16) * B (16 x 16), fp32 in shared memory with row
// stride LD, as one TF32 product per fragment: T leaves this kernel as a bf16 operand image (8 bits of
// mantissa), TF32 operands keep 11.  (Splitting every operand into a high and a low part, three
// products per fragment, was measured: 6 us more per launch on the 340M training shape and no
// change of the parity errors beyond their third digit.)  One warp.
template <int LD>
__device__ __forceinline__ void block16_mma_ld(float (&acc)[2][4], const float* A, const float* B, int lane)
{
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int kt = 0; kt < 2; ++kt) {
        const uint32_t a4[4] = {to_tf32(A[g * LD + 8 * kt + t]), to_tf32(A[(g + 8) * LD + 8 * kt + t]),
                                to_tf32(A[g * LD + 8 * kt + t + 4]), to_tf32(A[(g + 8) * LD + 8 * kt + t + 4])};
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            const uint32_t b2[2] = {to_tf32(B[(8 * kt + t) * LD + 8 * nt + g]), to_tf32(B[(8 * kt + t + 4) * LD + 8 * nt + g])};
            mma_tf32(acc[nt], a4, b2);
        }
    }
}

// store a 16 x 16 accumulator (optionally negated) to shared memory
template <int LD>
__device__ __forceinline__ void block16_store_ld(float* C, const float (&acc)[2][4], float sign, int lane)
{
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
        *reinterpret_cast<float2*>(C + g * LD + 8 * nt + 2 * t) = make_float2(sign * acc[nt][0], sign * acc[nt][1]);
        *reinterpret_cast<float2*>(C + (g + 8) * LD + 8 * nt + 2 * t) = make_float2(sign * acc[nt][2], sign * acc[nt][3]);
    }
}

template <typename Sync> __device__ __forceinline__ void ut_inverse_64_inplace(float* sA, int tid, Sync sync)
{
    const int warp = tid >> 5, lane = tid & 31;
    {
        float x[16];
        const int b = (tid >> 4) & 3, col = tid & 15;
        float* Ab = sA + (16 * b) * LCF + 16 * b;
        if (tid < CH) {
#pragma unroll
            for (int i = 0; i < 16; ++i) x[i] = i == col ? 1.f : 0.f;
#pragma unroll
            for (int j = 0; j < 15; ++j) {
#pragma unroll
                for (int i = j + 1; i < 16; ++i) x[i] = fmaf(-Ab[i * LCF + j], x[j], x[i]);
            }
        }
        sync();   // every column has read the block before anyone overwrites it
        if (tid < CH) {
#pragma unroll
            for (int i = 0; i < 16; ++i) Ab[i * LCF + col] = x[i];
        }
    }
    sync();
    for (int b = 1; b < 4; ++b) {
        // warp c < b: X = sum_m A_bm T_mc, parked in block (c, b); then T_bc = -T_bb X
        float acc2[2][4] = {};
        if (warp < b) {
            const int c = warp;
            float acc[2][4] = {};
            for (int m = c; m < b; ++m)
                block16_mma_ld<LCF>(acc, sA + (16 * b) * LCF + 16 * m, sA + (16 * m) * LCF + 16 * c, lane);
            float* X = sA + (16 * c) * LCF + 16 * b;
            block16_store_ld<LCF>(X, acc, 1.f, lane);
            __syncwarp();
            block16_mma_ld<LCF>(acc2, sA + (16 * b) * LCF + 16 * b, X, lane);
        }
        sync();   // row b of A has been read by every warp that needs it
        if (warp < b) block16_store_ld<LCF>(sA + (16 * b) * LCF + 16 * warp, acc2, -1.f, lane);
        sync();
    }
}

// ---------------------------------------------------------------------------------------------
// chunk-local forward
// ---------------------------------------------------------------------------------------------
struct TcChunkArgs {
    int H;
    int* ready;   // merged forward launch: per (chunk, head) tile, set to 1 once the tile's images are in global memory
    Table tab;
    const float *beta, *gate;
    float scale;
    uint8_t *WT, *Tb, *Tm, *P, *Qg;
    int save;
    int* status;
};

// 8 warps = 4 lane quadrants x 2 column halves; 50 KB of shared memory and 128 tensor-memory columns,
// so that four CTAs share an SM and hide each other's waits.
constexpr int CL_THREADS = 256;
constexpr size_t CL_SMEM = 32768 + CH * LCF * 4 + 1024;

// Small per-group state of the chunk-local forward that lives in shared memory.
struct ClGroupShared {
    uint64_t bar_tma, bar_mma1, bar_mma2;
    int ticket;
    int pad;
    float sG[CH], sBeta[CH];
};

// One (chunk, head) tile by a group of CL_THREADS threads (local index `tid`) that synchronise on hardware
// barrier `bar_id`; `sm`: CL_SMEM - 1024 bytes, 1024-byte aligned; `tb`: 128 tensor-memory columns;
// `ph`: parity of the group's three barriers (they complete once per tile).
__device__ __forceinline__ void chunk_fwd_tile(const CUtensorMap& tmK, const CUtensorMap& tmQ, const CUtensorMap& tmKt,
                                               const TcChunkArgs& a, int c, int h, uint8_t* sm, ClGroupShared& gs,
                                               uint32_t tb, int tid, int bar_id, uint32_t ph, int* publish)
{
    auto sync = [&]() { named_sync(bar_id, CL_THREADS); };
    uint64_t& bar_tma = gs.bar_tma;
    uint64_t& bar_mma1 = gs.bar_mma1;
    uint64_t& bar_mma2 = gs.bar_mma2;
    float* sG = gs.sG;
    float* sBeta = gs.sBeta;
    uint8_t* sKQ = sm;                 // per k-half h: [K rows 0-63 | Q rows 64-127], 16 KB each
    uint8_t* sKt = sKQ + 32768;        // per k-half: 8 KB
    // A, then T (fp32, in place) take over the space of Ktil once the first product has consumed it;
    // the T diag(beta gamma) operand image takes over the first Q box once Qg has been written.
    float* sA = reinterpret_cast<float*>(sKt);
    uint8_t* sTb = sKQ + BOX;          // K-major [i][j]
    const int H = a.H;
    const int len = a.tab.chunk_len(c);
    if (len == 0) return;
    const int tok0 = a.tab.chunk_tok0(c);
    const size_t tile = (size_t)c * H + h;
    const int warp = tid >> 5, lane = tid & 31;
    const int quad = warp & 3, half = warp >> 2;

    if (tid == 0) {
        mbar_expect_tx(&bar_tma, 6 * BOX);
        for (int hf = 0; hf < 2; ++hf) {
            tma_load_2d(sKQ + hf * 16384, &tmK, h * KD + hf * 64, tok0, &bar_tma);
            tma_load_2d(sKQ + hf * 16384 + BOX, &tmQ, h * KD + hf * 64, tok0, &bar_tma);
            tma_load_2d(sKt + hf * BOX, &tmKt, h * KD + hf * 64, tok0, &bar_tma);
        }
    }
    if (warp == 2) {   // per-token scalars and the in-chunk gate prefix G_i
        const bool in0 = lane < len, in1 = lane + 32 < len;
        float sa = in0 ? a.gate[(size_t)(tok0 + lane) * H + h] : 0.f;
        float sb = in1 ? a.gate[(size_t)(tok0 + lane + 32) * H + h] : 0.f;
        sBeta[lane] = in0 ? a.beta[(size_t)(tok0 + lane) * H + h] : 0.f;
        sBeta[lane + 32] = in1 ? a.beta[(size_t)(tok0 + lane + 32) * H + h] : 0.f;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float ua = __shfl_up_sync(0xffffffffu, sa, o), ub = __shfl_up_sync(0xffffffffu, sb, o);
            if (lane >= o) { sa += ua; sb += ub; }
        }
        sb += __shfl_sync(0xffffffffu, sa, 31);
        sG[lane] = sa;
        sG[lane + 32] = sb;
    }
    // The group's previous tile is published here, behind a barrier that is needed anyway: the barrier
    // orders every thread's stores before thread 0, whose fence (cumulative) then orders them before the flag.
    tc_fence_before();
    sync();
    tc_fence_after();
    if (publish && tid == 0) {
        __threadfence();
        st_release_gpu(publish, 1);
    }

    bool ok = mbar_wait(&bar_tma, ph, a.status, ERR_TMA);
    if (len < CH) {
        for (int hf = 0; hf < 2; ++hf) {
            zero_tail_rows(sKQ + hf * 16384, len, tid, CL_THREADS);
            zero_tail_rows(sKQ + hf * 16384 + BOX, len, tid, CL_THREADS);
            zero_tail_rows(sKt + hf * BOX, len, tid, CL_THREADS);
        }
        fence_proxy_async();
        sync();
    }

    // ---- D1[128 x 64] = [K;Q] Ktil^T ---------------------------------------------------------
    if (tid == 0 && ok) {
        const uint32_t idesc = make_idesc(128, 64);
        for (int s = 0; s < 8; ++s) {
            const uint64_t da = desc_advance(desc_kmajor(sKQ + (s >> 2) * 16384), 32 * (s & 3));
            const uint64_t db = desc_advance(desc_kmajor(sKt + (s >> 2) * BOX), 32 * (s & 3));
            mma_ss(tb, da, db, idesc, s > 0);
        }
        mma_commit(&bar_mma1);
    }
    // gated, scaled queries for both state chains, while the product runs: Qg = scale gamma_i Q
    // (same image layout as Q)
    for (int e = tid; e < 2 * CH * 8; e += CL_THREADS) {
        const int hf = e >> 9, i = (e >> 3) & 63, ch = e & 7;
        const uint32_t off = sw128_chunk(i, ch);
        const uint4 w = *reinterpret_cast<const uint4*>(sKQ + hf * 16384 + BOX + off);
        const float f = a.scale * __expf(sG[i]);
        const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&w);
        uint32_t o[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const float2 v = __bfloat1622float2(p2[x]);
            o[x] = pack_bf16(v.x * f, v.y * f);
        }
        *reinterpret_cast<uint4*>(a.Qg + tile * REC_BYTES + hf * BOX + off) = make_uint4(o[0], o[1], o[2], o[3]);
    }
    ok = ok && mbar_wait(&bar_mma1, ph, a.status, ERR_MMA1);
    tc_fence_after();
    if (ok) {
        const int L = quad * 32 + lane;
        const uint32_t taddr = tb + ((uint32_t)(quad * 32) << 16) + half * 32;
        if (L < CH) {   // A_ij = beta_i Gamma_ij <k_i, ktil_j>, j < i
            const int i = L;
            const float bi = sBeta[i], Gi = sG[i];
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                const int j0 = half * 32 + cb * 16;
                float av[16];
                if (j0 <= (quad & 1) * 32 + 31) {   // warp-uniform: some row of this warp reaches the block
                    uint32_t r[16];
                    tmem_ld16(taddr + cb * 16, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int x = 0; x < 16; ++x) {
                        const int j = j0 + x;
                        av[x] = j < i ? bi * __expf(Gi - sG[j]) * __uint_as_float(r[x]) : 0.f;
                    }
                } else {
#pragma unroll
                    for (int x = 0; x < 16; ++x) av[x] = 0.f;
                }
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
                    *reinterpret_cast<float4*>(sA + i * LCF + j0 + q4 * 4) =
                        make_float4(av[q4 * 4 + 0], av[q4 * 4 + 1], av[q4 * 4 + 2], av[q4 * 4 + 3]);
            }
        } else {        // P'_ij = scale Gamma_ij <q_i, ktil_j>, j <= i
            const int i = L - CH;
            const float Gi = sG[i];
            uint8_t* Pg = a.P + tile * REC_BYTES;
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                const int j0 = half * 32 + cb * 16;
                float pv[16];
                if (j0 <= (quad & 1) * 32 + 31) {   // warp-uniform
                    uint32_t r[16];
                    tmem_ld16(taddr + cb * 16, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int x = 0; x < 16; ++x) {
                        const int j = j0 + x;
                        pv[x] = j <= i ? a.scale * __expf(Gi - sG[j]) * __uint_as_float(r[x]) : 0.f;
                    }
                } else {
#pragma unroll
                    for (int x = 0; x < 16; ++x) pv[x] = 0.f;
                }
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {
                    uint4 w;
                    w.x = pack_bf16(pv[c2 * 8 + 0], pv[c2 * 8 + 1]);
                    w.y = pack_bf16(pv[c2 * 8 + 2], pv[c2 * 8 + 3]);
                    w.z = pack_bf16(pv[c2 * 8 + 4], pv[c2 * 8 + 5]);
                    w.w = pack_bf16(pv[c2 * 8 + 6], pv[c2 * 8 + 7]);
                    *reinterpret_cast<uint4*>(Pg + sw128_chunk(i, (j0 >> 3) + c2)) = w;
                }
            }
        }
    }
    sync();

    // ---- T = (I + A)^-1, blocked, in place ---------------------------------------------------------
    ut_inverse_64_inplace(sA, tid, sync);

    // ---- operand images: Tbg (shared), Tb and T (HBM) -----------------------------------------
    for (int e = tid; e < CH * 8; e += CL_THREADS) {
        const int i = e >> 3, ch = e & 7;
        const float4 t0 = *reinterpret_cast<const float4*>(sA + i * LCF + ch * 8);
        const float4 t1 = *reinterpret_cast<const float4*>(sA + i * LCF + ch * 8 + 4);
        const float tv[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
        float t[8], tb8[8], tbg[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const int j = ch * 8 + x;
            t[x] = j <= i ? tv[x] : 0.f;   // above the diagonal the array holds scratch
            tb8[x] = t[x] * sBeta[j];
            tbg[x] = tb8[x] * __expf(sG[j]);
        }
        const uint32_t off = sw128_chunk(i, ch);
        *reinterpret_cast<uint4*>(sTb + off) = make_uint4(pack_bf16(tbg[0], tbg[1]), pack_bf16(tbg[2], tbg[3]),
                                                         pack_bf16(tbg[4], tbg[5]), pack_bf16(tbg[6], tbg[7]));
        *reinterpret_cast<uint4*>(a.Tb + tile * REC_BYTES + off) =
            make_uint4(pack_bf16(tb8[0], tb8[1]), pack_bf16(tb8[2], tb8[3]), pack_bf16(tb8[4], tb8[5]),
                       pack_bf16(tb8[6], tb8[7]));
        if (a.save)
            *reinterpret_cast<uint4*>(a.Tm + tile * 8192 + off) =
                make_uint4(pack_bf16(t[0], t[1]), pack_bf16(t[2], t[3]), pack_bf16(t[4], t[5]), pack_bf16(t[6], t[7]));
    }
    fence_proxy_async();
    tc_fence_before();
    sync();

    // ---- D2[128 x 64] = K^T Tbg^T  (W^T) -----------------------------------------------------
    if (tid == 0 && ok) {
        tc_fence_after();
        const uint32_t idesc = make_idesc(128, 64, IDESC_A_MN);
        const uint64_t da0 = desc_mnmajor(sKQ, 16384);
        const uint64_t db0 = desc_kmajor(sTb);
        for (int s = 0; s < 4; ++s) mma_ss(tb + 64, desc_advance(da0, 2048 * s), desc_advance(db0, 32 * s), idesc, s > 0);
        mma_commit(&bar_mma2);
    }
    ok = ok && mbar_wait(&bar_mma2, ph, a.status, ERR_MMA2);
    tc_fence_after();
    if (ok) {
        const int k = quad * 32 + lane;
        const uint32_t taddr = tb + ((uint32_t)(quad * 32) << 16) + 64 + half * 32;
        uint8_t* Wg = a.WT + tile * REC_BYTES;
        uint32_t r[2][16];
        tmem_ld16(taddr, r[0]);
        tmem_ld16(taddr + 16, r[1]);
        tmem_ld_wait();
#pragma unroll
        for (int cb = 0; cb < 2; ++cb)
#pragma unroll
            for (int c2 = 0; c2 < 2; ++c2) {
                uint4 w;
                w.x = pack_bf16(__uint_as_float(r[cb][c2 * 8 + 0]), __uint_as_float(r[cb][c2 * 8 + 1]));
                w.y = pack_bf16(__uint_as_float(r[cb][c2 * 8 + 2]), __uint_as_float(r[cb][c2 * 8 + 3]));
                w.z = pack_bf16(__uint_as_float(r[cb][c2 * 8 + 4]), __uint_as_float(r[cb][c2 * 8 + 5]));
                w.w = pack_bf16(__uint_as_float(r[cb][c2 * 8 + 6]), __uint_as_float(r[cb][c2 * 8 + 7]));
                *reinterpret_cast<uint4*>(Wg + sw128_chunk(k, half * 4 + cb * 2 + c2)) = w;
            }
    }
    tc_fence_before();
    sync();
}

// Stand-alone launch: one tile per CTA, four CTAs per SM.
__global__ void __launch_bounds__(CL_THREADS, 4)
tc_chunk_fwd_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
                    const __grid_constant__ CUtensorMap tmKt, TcChunkArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ ClGroupShared gs;
    __shared__ uint32_t tmem_base;
    const int tid = threadIdx.x;
    if (a.tab.chunk_len(blockIdx.x) == 0) return;
    if (tid == 0) {
        mbar_init(&gs.bar_tma, 1);
        mbar_init(&gs.bar_mma1, 1);
        mbar_init(&gs.bar_mma2, 1);
        fence_mbar_init();
    }
    if ((tid >> 5) == 1) tmem_alloc(&tmem_base, 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    chunk_fwd_tile(tmK, tmQ, tmKt, a, blockIdx.x, blockIdx.y, align1024(smem_raw), gs, tmem_base, tid, 1, 0u, nullptr);
    __syncthreads();
    if ((tid >> 5) == 1) tmem_dealloc(tmem_base, 128);
}

// ---------------------------------------------------------------------------------------------
// state chain, forward
// ---------------------------------------------------------------------------------------------
struct TcChainArgs {
    int H;
    Table tab;
    const float *gate, *init_state;
    __nv_bfloat16* out;
    float* final_state;
    const uint8_t *WT, *Tb, *P;
    uint8_t *Sn, *dUT;
    float scale;
    int save;
    int* status;
    const int* ready;   // nullable: per (chunk, head) tile, nonzero once the chunk-local pass has written it
};

constexpr uint32_t STAGE_BYTES = 8192 + 16384 + 8192 + 3 * 16384;   // Tb, WT, P, Qg, V, Ktil = 81920
constexpr uint32_t ST_TB = 0, ST_WT = 8192, ST_P = 24576, ST_QG = 32768, ST_V = 49152, ST_KT = 65536;
constexpr size_t CF_SMEM = 2 * STAGE_BYTES + 32768 + 2 * 16384 + 1024;

// In-chunk gate prefix by one warp: lane l holds g_l and g_{l+32}.  Writes gamma_i = exp(G_i),
// rho_i = exp(G_C - G_i) and gamma_C into the given slot.
__device__ __forceinline__ void warp_gate_vectors(float ga, float gb, int lane, float* gam, float* rho, float* gC)
{
    float sa = ga, sb = gb;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float ua = __shfl_up_sync(0xffffffffu, sa, o), ub = __shfl_up_sync(0xffffffffu, sb, o);
        if (lane >= o) { sa += ua; sb += ub; }
    }
    const float ta = __shfl_sync(0xffffffffu, sa, 31);
    sb += ta;
    const float tot = __shfl_sync(0xffffffffu, sb, 31);
    if (gam) { gam[lane] = __expf(sa); gam[lane + 32] = __expf(sb); }
    rho[lane] = __expf(tot - sa);
    rho[lane + 32] = __expf(tot - sb);
    if (lane == 0) *gC = __expf(tot);
}

// Warp roles of the forward chain: 16 state warps (4 lane quadrants x 4 column groups), 4 output warps
// (one per lane quadrant), one warp that issues the tensor-core work, one warp that issues the loads
// and prepares the gate vectors.  The roles run decoupled and meet only at mbarriers:
//   full[st]    loads of a chunk have landed (and its gate vectors are written)      producer -> all
//   empty[st]   every product reading the stage has finished                         tensor core -> producer
//   s_ready     S is in shared memory as a bf16 operand, the accumulator is decayed  state warps -> issuer
//   du_done     dU^T accumulator complete                                            tensor core -> state warps
//   du_ready    dU^T operands are in shared memory                                   state warps -> issuer
//   s_done      the state update of the chunk is complete                            tensor core -> state warps
//   o_done[st]  both output accumulators of the chunk are complete                   tensor core -> output warps
//   o_free[st]  the output accumulators have been read                               output warps -> issuer
// The state warps carry the recurrence and never store to global memory inside the loop: a warp's
// tensor-memory load does not return while its earlier global stores are outstanding, which would
// put the latency of the output stores on the chunk-to-chunk path.
constexpr int CFW_EPI_WARPS = 16, CFW_OUT_WARPS = 4;
constexpr int CFW_OUT_WARP0 = 16, CFW_MMA_WARP = 20, CFW_TMA_WARP = 21;
constexpr int CFW_THREADS = 22 * 32;

// One chain by the first CFW_THREADS threads of the CTA (all threads of the CTA must call: the function
// synchronises the CTA).  `sm`: CF_SMEM - 1024 bytes, 1024-byte aligned; `tb`: 512 tensor-memory columns.
// With `a.ready` set, the loads of a chunk wait until the chunk-local pass has published it.
__device__ __forceinline__ void chain_fwd_role(const CUtensorMap& tmV, const CUtensorMap& tmKt, const TcChainArgs& a,
                                               int chain, uint8_t* sm, uint32_t tb)
{
    uint8_t* sStage = sm;                       // 2 stages
    uint8_t* sS = sm + 2 * STAGE_BYTES;         // S as bf16, K-major: 2 k-halves x [128 rows x 128 B]
    uint8_t* sDU1 = sS + 32768;                 // dU^T, K-major [v][i]
    uint8_t* sDU2 = sDU1 + 16384;               // (rho dU)^T
    __shared__ uint64_t bar_full[2], bar_empty[2], bar_s_ready, bar_du_done, bar_du_ready, bar_s_done;
    __shared__ uint64_t bar_o_done[2], bar_o_free[2];
    __shared__ float sRho[2][CH], sGC[2];              // slot = chunk % 2

    const int H = a.H;
    const int s = chain / H, h = chain % H;
    const int c0 = a.tab.seq_chunk0(s), c1 = a.tab.seq_chunk0(s + 1);
    const int seq_t0 = a.tab.seq_tok0(s), seq_len = a.tab.seq_len(s);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int quad = warp & 3, colq = (warp >> 2) & 3;
    const int v = quad * 32 + lane;             // state row owned by a state-warp thread
    float* fin = a.final_state ? a.final_state + (((size_t)s * H + h) * KD + v) * KD + colq * 32 : nullptr;
    const float* ini = a.init_state ? a.init_state + (((size_t)s * H + h) * KD + v) * KD + colq * 32 : nullptr;
    if (c1 <= c0) {   // empty sequence: the state passes through
        if (fin && warp < CFW_EPI_WARPS)
            for (int x = 0; x < 32; ++x) fin[x] = ini ? ini[x] : 0.f;
        return;
    }
    uint64_t* const all_bars[] = {&bar_full[0], &bar_full[1], &bar_empty[0], &bar_empty[1], &bar_s_ready, &bar_du_done,
                                  &bar_du_ready, &bar_s_done, &bar_o_done[0], &bar_o_done[1], &bar_o_free[0],
                                  &bar_o_free[1]};
    const int nchunks = c1 - c0;
    auto chunk_tok0 = [&](int n) { return seq_t0 + n * CH; };
    auto chunk_len = [&](int n) { return min(CH, seq_len - n * CH); };

    if (tid == 0) {
        mbar_init(&bar_full[0], 2);
        mbar_init(&bar_full[1], 2);
        mbar_init(&bar_empty[0], 1);
        mbar_init(&bar_empty[1], 1);
        mbar_init(&bar_s_ready, CFW_EPI_WARPS);
        mbar_init(&bar_du_done, 1);
        mbar_init(&bar_du_ready, CFW_EPI_WARPS);
        mbar_init(&bar_s_done, 1);
        mbar_init(&bar_o_done[0], 1);
        mbar_init(&bar_o_done[1], 1);
        mbar_init(&bar_o_free[0], CFW_OUT_WARPS);
        mbar_init(&bar_o_free[1], CFW_OUT_WARPS);
        fence_mbar_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tS = tb, tDU = tb + 128, tO = tb + 192;   // O^T: two buffers of 64 columns

    if (warp >= CFW_THREADS / 32) {
        // not part of the chain
    } else if (warp == CFW_TMA_WARP) {
        // ------------------------------------------------------------------ producer
        // A stage is complete when its copies have landed (transaction count, first arrival) and the
        // gate vectors of the chunk are written (second arrival).  The gates are read a chunk ahead.
        bool ok = true;
        auto load_gates = [&](int n, float& ga, float& gb) {
            const int tok0 = chunk_tok0(n), len = chunk_len(n);
            ga = lane < len ? a.gate[(size_t)(tok0 + lane) * H + h] : 0.f;
            gb = lane + 32 < len ? a.gate[(size_t)(tok0 + lane + 32) * H + h] : 0.f;
        };
        float ga, gb;
        load_gates(0, ga, gb);
        for (int n = 0; n < nchunks && ok; ++n) {
            const int st = n & 1, gs = n & 1;
            const int tok0 = chunk_tok0(n);
            float ga_next = 0.f, gb_next = 0.f;
            if (n + 1 < nchunks) load_gates(n + 1, ga_next, gb_next);
            // The record's flag is looked at before the stage is waited for: its round trip to memory then
            // runs while the products of the chunk before last still read the stage.
            if (a.ready) {   // the chunk-local pass runs beside the chains: wait until the record is written
                const int* flag = a.ready + (size_t)(c0 + n) * H + h;
                const long long t0 = clock64();
                bool seen = false;
                while (!(seen = ld_acquire_gpu(flag) != 0)) {
                    if (clock64() - t0 > WAIT_LIMIT_CYCLES) break;
                    __nanosleep(64);
                }
                if (!seen) {
                    if (lane == 0) atomicCAS(a.status, 0, ERR_READY);
                    ok = false;
                    break;
                }
                fence_proxy_async_all();
            }
            if (n >= 2) ok = mbar_wait(&bar_empty[st], ((n >> 1) - 1) & 1, a.status, ERR_CHAIN_TMA);
            if (!ok) break;
            if (lane == 0) {
                const size_t tile = (size_t)(c0 + n) * H + h;
                uint8_t* d = sStage + st * STAGE_BYTES;
                mbar_expect_tx(&bar_full[st], STAGE_BYTES);
                bulk_load(d + ST_TB, a.Tb + tile * REC_BYTES, REC_BYTES, &bar_full[st]);   // Tb, W^T, P', Qg
                for (int hf = 0; hf < 2; ++hf) tma_load_2d(d + ST_V + hf * BOX, &tmV, h * KD + hf * 64, tok0, &bar_full[st]);
                for (int hf = 0; hf < 2; ++hf) tma_load_2d(d + ST_KT + hf * BOX, &tmKt, h * KD + hf * 64, tok0, &bar_full[st]);
            }
            __syncwarp();
            warp_gate_vectors(ga, gb, lane, nullptr, sRho[gs], &sGC[gs]);
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_full[st]);
            ga = ga_next;
            gb = gb_next;
        }
    } else if (warp == CFW_MMA_WARP) {
        // ------------------------------------------------------------------ tensor-core issuer
        bool ok = true;
        bool ut_issued = false;   // V^T Tb^T of the coming chunk is already in the dU^T accumulator
        auto issue_ut = [&](uint8_t* d) {   // dU^T = V^T Tb^T
            const uint32_t idesc = make_idesc(128, 64, IDESC_A_MN);
            const uint64_t da0 = desc_mnmajor(d + ST_V, BOX), db0 = desc_kmajor(d + ST_TB);
            for (int k = 0; k < 4; ++k)
                mma_ss(tDU, desc_advance(da0, 2048 * k), desc_advance(db0, 32 * k), idesc, k > 0);
        };
        for (int n = 0; n < nchunks && ok; ++n) {
            const int st = n & 1;
            const size_t tile = (size_t)(c0 + n) * H + h;
            uint8_t* d = sStage + st * STAGE_BYTES;
            if (!ut_issued) ok = mbar_wait(&bar_full[st], (n >> 1) & 1, a.status, ERR_CHAIN_TMA);
            ok = ok && mbar_wait(&bar_s_ready, n & 1, a.status, ERR_CHAIN_MMA1);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) {
                bulk_wait_read();   // saved images of the previous chunk have left shared memory
                if (a.save) {
                    bulk_store(a.Sn + tile * 32768, sS, 32768);
                    bulk_commit();
                }
                if (!ut_issued) issue_ut(d);
                {   // dU^T -= S W^T
                    const uint32_t idesc = make_idesc(128, 64, IDESC_A_NEG | IDESC_B_MN);
                    const uint64_t db0 = desc_mnmajor(d + ST_WT, 0);
                    for (int k = 0; k < 8; ++k)
                        mma_ss(tDU, desc_advance(desc_kmajor(sS + (k >> 2) * 16384), 32 * (k & 3)),
                               desc_advance(db0, 2048 * k), idesc, 1);
                }
                mma_commit(&bar_du_done);
            }
            __syncwarp();
            // the output accumulators of chunk n - 2 (same buffers) have been read
            if (n >= 2) ok = mbar_wait(&bar_o_free[st], ((n >> 1) - 1) & 1, a.status, ERR_CHAIN_MMA2);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) {   // O^T = S Qg^T
                const uint32_t idesc = make_idesc(128, 64);
                for (int k = 0; k < 8; ++k)
                    mma_ss(tO + st * 64, desc_advance(desc_kmajor(sS + (k >> 2) * 16384), 32 * (k & 3)),
                           desc_advance(desc_kmajor(d + ST_QG + (k >> 2) * BOX), 32 * (k & 3)), idesc, k > 0);
            }
            __syncwarp();
            ok = mbar_wait(&bar_du_ready, n & 1, a.status, ERR_CHAIN_MMA2);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) {
                // The image of S sent off at the start of this chunk must have left shared memory before
                // the state update is released: its completion lets the state warps overwrite that image.
                bulk_wait_read();
                if (a.save) {
                    bulk_store(a.dUT + tile * 16384, sDU1, 16384);
                    bulk_commit();
                }
                {   // S += (rho dU)^T Ktil
                    const uint32_t idesc = make_idesc(128, 128, IDESC_B_MN);
                    const uint64_t da0 = desc_kmajor(sDU2), db0 = desc_mnmajor(d + ST_KT, BOX);
                    for (int k = 0; k < 4; ++k)
                        mma_ss(tS, desc_advance(da0, 32 * k), desc_advance(db0, 2048 * k), idesc, 1);
                }
                mma_commit(&bar_s_done);
                {   // O^T += dU^T P'^T
                    const uint32_t idesc = make_idesc(128, 64);
                    const uint64_t da0 = desc_kmajor(sDU1), db0 = desc_kmajor(d + ST_P);
                    for (int k = 0; k < 4; ++k)
                        mma_ss(tO + st * 64, desc_advance(da0, 32 * k), desc_advance(db0, 32 * k), idesc, 1);
                }
                mma_commit(&bar_o_done[st]);
                mma_commit(&bar_empty[st]);
            }
            __syncwarp();
            // The part of the next chunk's dU^T that does not depend on the state goes in now, while the
            // state warps convert S (full chunks only: a ragged chunk has its tail rows cleared first).
            ut_issued = false;
            if (n + 1 < nchunks && chunk_len(n + 1) == CH) {
                ok = mbar_wait(&bar_full[st ^ 1], ((n + 1) >> 1) & 1, a.status, ERR_CHAIN_TMA);
                if (!ok) break;
                if (lane == 0) issue_ut(sStage + (st ^ 1) * STAGE_BYTES);
                __syncwarp();
                ut_issued = true;
            }
        }
        if (lane == 0) bulk_wait_all();
    } else if (warp >= CFW_OUT_WARP0) {
        // ------------------------------------------------------------------ output warps
        // o_i = (S Qg^T + dU^T P'^T)_i is complete in the accumulator: lane = feature, 16 token columns
        // per load.  Results leave as 16-byte stores: three shuffle rounds turn "lane = feature, 16
        // tokens" into "lane = 8 consecutive features of 2 tokens" (lane bit 0 picks the token half,
        // bits 1-2 the token pair inside it, bits 3-4 the feature octet).
        const int ow = warp - CFW_OUT_WARP0;   // == lane quadrant
        const uint32_t lane_addr = (uint32_t)(ow * 32) << 16;
        const bool b0 = lane & 1, b1 = lane & 2, b2 = lane & 4;
        const int tsub = (b0 ? 8 : 0) + ((lane >> 1) & 3) * 2;
        bool ok = true;
        for (int n = 0; n < nchunks && ok; ++n) {
            const int st = n & 1;
            const int tok0 = chunk_tok0(n), len = chunk_len(n);
            // Warm L2 with the operands of chunk n + 2 (the stage copies can only run one chunk ahead).
            if (lane == 0 && n + 2 < nchunks) {
                const int t2 = chunk_tok0(n + 2);
                if (ow == 0 && !a.ready) bulk_prefetch(a.Tb + ((size_t)(c0 + n + 2) * H + h) * REC_BYTES, REC_BYTES);
                if (ow == 1)
                    for (int hf = 0; hf < 2; ++hf) tma_prefetch_2d(&tmV, h * KD + hf * 64, t2);
                if (ow == 2)
                    for (int hf = 0; hf < 2; ++hf) tma_prefetch_2d(&tmKt, h * KD + hf * 64, t2);
            }
            ok = mbar_wait(&bar_o_done[st], (n >> 1) & 1, a.status, ERR_CHAIN_MMA2);
            if (!ok) break;
            tc_fence_after();
            __nv_bfloat16* op = a.out + ((size_t)tok0 * H + h) * KD + ow * 32 + (lane >> 3) * 8;
#pragma unroll
            for (int cg = 0; cg < 4; ++cg) {
                uint32_t ra[16];
                tmem_ld16(tO + st * 64 + lane_addr + cg * 16, ra);
                tmem_ld_wait();
                if (cg == 3) {   // everything is in registers: the buffer may be overwritten
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bar_o_free[st]);
                }
                uint32_t w[8];    // feature pair (lane >> 1), token (b0 ? 8 : 0) + i
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float lo = __uint_as_float(ra[i]), hi = __uint_as_float(ra[i + 8]);
                    const float recv = __shfl_xor_sync(0xffffffffu, b0 ? lo : hi, 1);
                    w[i] = b0 ? pack_bf16(recv, hi) : pack_bf16(lo, recv);
                }
                uint32_t wa[2][2][2];   // [token-pair bit 1][token parity][feature pair 0 / 1]
#pragma unroll
                for (int th = 0; th < 2; ++th)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const uint32_t w0 = w[(th * 2 + 0) * 2 + e], w1 = w[(th * 2 + 1) * 2 + e];
                        const uint32_t keep = b1 ? w1 : w0;
                        const uint32_t recv = __shfl_xor_sync(0xffffffffu, b1 ? w0 : w1, 2);
                        wa[th][e][0] = b1 ? recv : keep;
                        wa[th][e][1] = b1 ? keep : recv;
                    }
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    uint32_t q4[4];
#pragma unroll
                    for (int sp = 0; sp < 2; ++sp) {
                        const uint32_t keep = b2 ? wa[1][e][sp] : wa[0][e][sp];
                        const uint32_t recv = __shfl_xor_sync(0xffffffffu, b2 ? wa[0][e][sp] : wa[1][e][sp], 4);
                        q4[sp] = b2 ? recv : keep;
                        q4[2 + sp] = b2 ? keep : recv;
                    }
                    const int i = cg * 16 + tsub + e;
                    if (i < len)
                        *reinterpret_cast<uint4*>(op + (size_t)i * H * KD) = make_uint4(q4[0], q4[1], q4[2], q4[3]);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ state warps
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const int etid = tid;   // 0 .. 511
        // initial state into tensor memory
        for (int cb = 0; cb < 2; ++cb) {
            uint32_t r[16];
#pragma unroll
            for (int x4 = 0; x4 < 4; ++x4) {
                const float4 f4 = ini ? *reinterpret_cast<const float4*>(ini + cb * 16 + x4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
                r[x4 * 4 + 0] = __float_as_uint(f4.x);
                r[x4 * 4 + 1] = __float_as_uint(f4.y);
                r[x4 * 4 + 2] = __float_as_uint(f4.z);
                r[x4 * 4 + 3] = __float_as_uint(f4.w);
            }
            tmem_st16(tS + lane_addr + colq * 32 + cb * 16, r);
        }
        tmem_st_wait();

        bool ok = true;
        for (int n = 0; n < nchunks && ok; ++n) {
            const int st = n & 1, gs = n & 1;
            const int len = chunk_len(n);
            uint8_t* d = sStage + st * STAGE_BYTES;
            ok = mbar_wait(&bar_full[st], (n >> 1) & 1, a.status, ERR_CHAIN_TMA);   // gate vectors, tail rows
            if (n > 0) ok = ok && mbar_wait(&bar_s_done, (n - 1) & 1, a.status, ERR_CHAIN_MMA2);
            if (!ok) break;
            tc_fence_after();
            // ---- E0: S -> bf16 operand (what the next products wait for), then decay the accumulator
            uint32_t rr[2][16];
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) tmem_ld16(tS + lane_addr + colq * 32 + cb * 16, rr[cb]);
            tmem_ld_wait();
#pragma unroll
            for (int cb = 0; cb < 2; ++cb) {
                const uint32_t* r = rr[cb];
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {
                    uint4 w;
                    w.x = pack_bf16(__uint_as_float(r[c2 * 8 + 0]), __uint_as_float(r[c2 * 8 + 1]));
                    w.y = pack_bf16(__uint_as_float(r[c2 * 8 + 2]), __uint_as_float(r[c2 * 8 + 3]));
                    w.z = pack_bf16(__uint_as_float(r[c2 * 8 + 4]), __uint_as_float(r[c2 * 8 + 5]));
                    w.w = pack_bf16(__uint_as_float(r[c2 * 8 + 6]), __uint_as_float(r[c2 * 8 + 7]));
                    *reinterpret_cast<uint4*>(sS + (colq >> 1) * 16384 + sw128_chunk(v, (colq & 1) * 4 + cb * 2 + c2)) = w;
                }
            }
            if (len < CH) {
                for (int hf = 0; hf < 2; ++hf) {
                    zero_tail_rows(d + ST_V + hf * BOX, len, etid, CFW_EPI_WARPS * 32);
                    zero_tail_rows(d + ST_KT + hf * BOX, len, etid, CFW_EPI_WARPS * 32);
                }
            }
            fence_proxy_async();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_s_ready);
            {   // gamma_C S back into the accumulator: only the state update (after du_ready) reads it
                const float gC = sGC[gs];
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
#pragma unroll
                    for (int x = 0; x < 16; ++x) rr[cb][x] = __float_as_uint(__uint_as_float(rr[cb][x]) * gC);
                    tmem_st16(tS + lane_addr + colq * 32 + cb * 16, rr[cb]);
                }
            }

            // ---- E1: dU^T -> bf16 operands
            float rho[16];
#pragma unroll
            for (int x = 0; x < 16; ++x) rho[x] = sRho[gs][colq * 16 + x];
            ok = mbar_wait(&bar_du_done, n & 1, a.status, ERR_CHAIN_MMA1);
            if (!ok) break;
            tc_fence_after();
            {
                uint32_t r[16];
                tmem_ld16(tDU + lane_addr + colq * 16, r);
                tmem_ld_wait();
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {
                    float f[8], g[8];
#pragma unroll
                    for (int x = 0; x < 8; ++x) {
                        f[x] = __uint_as_float(r[c2 * 8 + x]);
                        g[x] = f[x] * rho[c2 * 8 + x];
                    }
                    const uint32_t off = sw128_chunk(v, colq * 2 + c2);
                    *reinterpret_cast<uint4*>(sDU2 + off) = make_uint4(pack_bf16(g[0], g[1]), pack_bf16(g[2], g[3]),
                                                                      pack_bf16(g[4], g[5]), pack_bf16(g[6], g[7]));
                    *reinterpret_cast<uint4*>(sDU1 + off) = make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]),
                                                                      pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
                }
            }
            tmem_st_wait();   // the decayed accumulator is in place
            fence_proxy_async();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_du_ready);
        }
        if (ok) ok = mbar_wait(&bar_s_done, (nchunks - 1) & 1, a.status, ERR_CHAIN_MMA2);
        tc_fence_after();
        if (ok && fin) {
            for (int cb = 0; cb < 2; ++cb) {
                uint32_t r[16];
                tmem_ld16(tS + lane_addr + colq * 32 + cb * 16, r);
                tmem_ld_wait();
#pragma unroll
                for (int x4 = 0; x4 < 4; ++x4)
                    *reinterpret_cast<float4*>(fin + cb * 16 + x4 * 4) =
                        make_float4(__uint_as_float(r[x4 * 4 + 0]), __uint_as_float(r[x4 * 4 + 1]),
                                    __uint_as_float(r[x4 * 4 + 2]), __uint_as_float(r[x4 * 4 + 3]));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (tid == 0)
        for (uint64_t* b : all_bars) mbar_inval(b);
    __syncthreads();
}

// Stand-alone launch: one chain per CTA.
__global__ void __launch_bounds__(CFW_THREADS, 1)
tc_chain_fwd_kernel(const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmKt, TcChainArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t tmem_base;
    if (threadIdx.x < 32) tmem_alloc(&tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    chain_fwd_role(tmV, tmKt, a, blockIdx.x, align1024(smem_raw), tmem_base);
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(tmem_base, 512);
}

// ---------------------------------------------------------------------------------------------
// Forward of phase 2 in one launch.  Every CTA starts as three groups that take (chunk, head) tiles of
// the chunk-local pass from a ticket counter, chunk position by chunk position across the chains, and
// publish each finished tile with a flag.  Once `switch_at` tickets are out, the first `nchains` CTAs
// turn into the state chains, whose loads wait for those flags; the other CTAs keep producing, and a CTA
// whose chain is finished joins them again.  No worker ever waits, so the chains always make progress.
// ---------------------------------------------------------------------------------------------
constexpr float FWD_STEP_OVER_TILE_F = 0.65f;   // cost of a chain step in units of the time one SM needs for a tile
struct FwdSched {
    int* tickets;     // zero at launch
    int ntickets;     // number of (chunk, head) tiles
    int nchains;
    int nchunks;      // dense batch: chunk positions per chain (sequences of equal length)
    int switch_at;
    const int* order; // packed batch: the chunks sorted by position inside their sequence (else null); then
                      // ntickets and switch_at are worked out on the device from the chunk table
    const int* longest;   // packed batch: chunks of the longest sequence
    int nseq, feeders;
};

// Packed batches: the realised number of tiles and the longest chain are only known on the device.
__device__ __forceinline__ void fwd_sched_resolve(FwdSched& sc, const Table& tab, int H)
{
    if (!sc.order) return;
    sc.ntickets = tab.seq_chunk0(sc.nseq) * H;
    const float fed = (float)sc.feeders * (float)(*sc.longest) * FWD_STEP_OVER_TILE_F;
    sc.switch_at = max(0, sc.ntickets - (int)fed);
}
// Worker groups per CTA: four (1024 threads, 64 registers: the chain role loses about a tenth of its speed)
// when the chunk-local tiles are the larger part of the work, three (768 threads, 80 registers) when the
// longest chain is.
constexpr uint32_t FWD_GROUP_SMEM = (uint32_t)CL_SMEM - 1024;
static_assert(4 * FWD_GROUP_SMEM + 4 * sizeof(ClGroupShared) <= CF_SMEM - 1024, "worker groups fit");
static_assert(3 * CL_THREADS >= CFW_THREADS, "the chain fits into the CTA");

template <int FWD_GROUPS>
__device__ __forceinline__ void chunk_fwd_workers(const CUtensorMap& tmK, const CUtensorMap& tmQ,
                                                  const CUtensorMap& tmKt, const TcChunkArgs& cl, const FwdSched& sc,
                                                  int limit, uint8_t* sm, uint32_t tb)
{
    const int tid = threadIdx.x, g = tid / CL_THREADS, ltid = tid % CL_THREADS;
    ClGroupShared& gs = reinterpret_cast<ClGroupShared*>(sm + FWD_GROUPS * FWD_GROUP_SMEM)[g];
    auto gsync = [&]() { named_sync(1 + g, CL_THREADS); };
    if (ltid == 0) {
        mbar_init(&gs.bar_tma, 1);
        mbar_init(&gs.bar_mma1, 1);
        mbar_init(&gs.bar_mma2, 1);
        fence_mbar_init();
    }
    gsync();
    // The group's leader draws tickets one tile ahead, so the round trip of the atomic is hidden by the
    // tile in progress.  A ticket that has been drawn is always worked off before the group stops.
    auto draw = [&]() {
        int t = -1;
        if (*reinterpret_cast<volatile int*>(sc.tickets) < limit) {
            t = atomicAdd(sc.tickets, 1);
            if (t >= sc.ntickets) t = -1;
        }
        return t;
    };
    uint32_t ph = 0;
    int* publish = nullptr;   // flag of the tile the group finished last
    int next = ltid == 0 ? draw() : -1;
    while (true) {
        if (ltid == 0) gs.ticket = next;
        gsync();
        const int t = gs.ticket;
        if (t < 0) break;
        if (ltid == 0) next = draw();
        int c, h;
        if (sc.order) {   // packed batch: position-major order from the sorted list, heads innermost
            const int j = t / cl.H;
            h = t - j * cl.H;
            c = sc.order[j];
        } else {
            const int n = t / sc.nchains, chain = t - n * sc.nchains;
            const int s = chain / cl.H;
            h = chain - s * cl.H;
            c = s * sc.nchunks + n;
        }
        chunk_fwd_tile(tmK, tmQ, tmKt, cl, c, h, sm + g * FWD_GROUP_SMEM, gs, tb + g * 128, ltid, 1 + g, ph, publish);
        publish = cl.ready + (size_t)c * cl.H + h;
        ph ^= 1;
    }
    if (publish) {
        gsync();
        if (ltid == 0) {
            __threadfence();
            st_release_gpu(publish, 1);
        }
    }
    gsync();
    if (ltid == 0) {
        mbar_inval(&gs.bar_tma);
        mbar_inval(&gs.bar_mma1);
        mbar_inval(&gs.bar_mma2);
    }
    __syncthreads();
}

template <int FWD_GROUPS>
__global__ void __launch_bounds__(FWD_GROUPS * CL_THREADS, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmQ,
              const __grid_constant__ CUtensorMap tmKt, const __grid_constant__ CUtensorMap tmV, TcChunkArgs cl,
              TcChainArgs ch, FwdSched sched)
{
    FwdSched sc = sched;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = align1024(smem_raw);
    __shared__ uint32_t tmem_base;
    if (threadIdx.x < 32) tmem_alloc(&tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base;
    fwd_sched_resolve(sc, cl.tab, cl.H);
    const bool chain_cta = (int)blockIdx.x < sc.nchains;
    // packed batch: a chain starts when the tickets reach its own first tile (short sequences start late)
    if (chain_cta && sc.order) sc.switch_at = max(sc.switch_at, cl.tab.seq_first_[blockIdx.x / cl.H] * cl.H);
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {   // one copy of the worker code: it has to stay in the instruction cache
        chunk_fwd_workers<FWD_GROUPS>(tmK, tmQ, tmKt, cl, sc, chain_cta && pass == 0 ? sc.switch_at : sc.ntickets, sm, tb);
        if (!chain_cta || pass == 1) break;
        chain_fwd_role(tmV, tmKt, ch, blockIdx.x, sm, tb);
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) tmem_dealloc(tb, 512);
}

// ---------------------------------------------------------------------------------------------
// state chain, backward (reverse over chunks); dS (V x K, fp32) resident in tensor memory
//   ddU^T = dO^T P' + rho_i (dS Ktil^T) ;   dS <- gamma_C dS + dO^T Qg - ddU^T W
// ---------------------------------------------------------------------------------------------
struct TcChainBwdArgs {
    int H;
    Table tab;
    const float *gate, *dfinal_state;
    float* dinit_state;
    const uint8_t *WT, *P, *Qg;
    uint8_t *dSn, *ddUT;
    int* status;
};

constexpr uint32_t BS_DO = 0, BS_KT = 16384, BS_WT = 32768, BS_P = 49152, BS_QG = 57344;
constexpr uint32_t BSTAGE_BYTES = 73728;
constexpr size_t CB_SMEM = 2 * BSTAGE_BYTES + 32768 + 16384 + 1024;

// Warp roles as in the forward chain: 16 state warps (4 lane quadrants x 4 column groups), one warp
// issuing the tensor-core work, one producer warp.  Barriers:
//   full[st]   copies of a chunk have landed and its gate vectors are written          producer -> all
//   empty[st]  every product reading the stage has finished                           tensor core -> producer
//   s_ready    dS is in shared memory as a bf16 operand, the accumulator is decayed    state warps -> issuer
//   a_done     both parts of ddU^T are complete                                        tensor core -> state warps
//   a_ready    ddU^T is in shared memory as a bf16 operand                             state warps -> issuer
//   s_done     the cotangent update of the chunk is complete                           tensor core -> state warps
constexpr int CBK_EPI_WARPS = 16, CBK_MMA_WARP = 16, CBK_TMA_WARP = 17;
constexpr int CBK_THREADS = 18 * 32;

// Queue of (chunk, head) tiles between the backward chains (producers) and the chunk-local backward
// (consumers) inside one kernel: slot i holds tile + 1 once the i-th finished tile has been published
// (0 = not yet); consumers draw tickets from `head`.  The whole array is cleared before the launch.
struct TileQueue {
    int* slots;
    unsigned *head, *tail;
    // Publishes `count` tiles first, first + stride, ... (one fence and one counter update for all).
    __device__ __forceinline__ void push(int first, int stride, int count) const
    {
        if (count <= 0) return;
        fence_proxy_async_all();   // the tiles' images were written through the async proxy
        __threadfence();
        const unsigned slot = atomicAdd(tail, (unsigned)count);
        for (int i = 0; i < count; ++i) *reinterpret_cast<volatile int*>(slots + slot + i) = first + i * stride + 1;
    }
};

// One chain (sequence, head) of the backward state recurrence, by all CBK_THREADS threads of the CTA.
// `tb`: 256 free tensor-memory columns.  Every (chunk, head) tile whose cotangent images have reached
// global memory is appended to the tile queue `tq`, in the order the chains produce them.
__device__ __forceinline__ void chain_bwd_role(const CUtensorMap& tmDO, const CUtensorMap& tmKt, const TcChainBwdArgs& a,
                                               int chain, uint8_t* sm, uint32_t tb, const TileQueue& tq)
{
    uint8_t* sStage = sm;
    uint8_t* sdS = sm + 2 * BSTAGE_BYTES;       // dS as bf16, K-major, 2 k-halves x [128 x 128 B]
    uint8_t* sddU = sdS + 32768;                // ddU^T, K-major [v][i]
    __shared__ uint64_t bar_full[2], bar_empty[2], bar_s_ready, bar_a_done, bar_a_ready, bar_s_done;
    __shared__ float sRho[2][CH], sGC[2];

    const int H = a.H;
    const int s = chain / H, h = chain % H;
    const int c0 = a.tab.seq_chunk0(s), c1 = a.tab.seq_chunk0(s + 1);
    const int seq_t0 = a.tab.seq_tok0(s), seq_len = a.tab.seq_len(s);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int quad = warp & 3, colq = (warp >> 2) & 3;
    const int v = quad * 32 + lane;
    float* dini = a.dinit_state ? a.dinit_state + (((size_t)s * H + h) * KD + v) * KD + colq * 32 : nullptr;
    const float* dfin = a.dfinal_state ? a.dfinal_state + (((size_t)s * H + h) * KD + v) * KD + colq * 32 : nullptr;
    if (c1 <= c0) {
        if (dini && warp < CBK_EPI_WARPS)
            for (int x = 0; x < 32; ++x) dini[x] = dfin ? dfin[x] : 0.f;
        return;
    }
    const int nchunks = c1 - c0;
    // step n of the reverse walk handles chunk c1 - 1 - n of the sequence
    auto chunk_rel = [&](int n) { return nchunks - 1 - n; };
    auto chunk_tok0 = [&](int n) { return seq_t0 + chunk_rel(n) * CH; };
    auto chunk_len = [&](int n) { return min(CH, seq_len - chunk_rel(n) * CH); };
    auto chunk_tile = [&](int n) { return (size_t)(c0 + chunk_rel(n)) * H + h; };

    if (tid == 0) {
        mbar_init(&bar_full[0], 2);
        mbar_init(&bar_full[1], 2);
        mbar_init(&bar_empty[0], 1);
        mbar_init(&bar_empty[1], 1);
        mbar_init(&bar_s_ready, CBK_EPI_WARPS);
        mbar_init(&bar_a_done, 1);
        mbar_init(&bar_a_ready, CBK_EPI_WARPS);
        mbar_init(&bar_s_done, 1);
        fence_mbar_init();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tS = tb, tA1 = tb + 128, tA2 = tb + 192;

    if (warp == CBK_TMA_WARP) {
        // ------------------------------------------------------------------ producer
        bool ok = true;
        auto load_gates = [&](int n, float& ga, float& gb) {
            const int tok0 = chunk_tok0(n), len = chunk_len(n);
            ga = lane < len ? a.gate[(size_t)(tok0 + lane) * H + h] : 0.f;
            gb = lane + 32 < len ? a.gate[(size_t)(tok0 + lane + 32) * H + h] : 0.f;
        };
        float ga, gb;
        load_gates(0, ga, gb);
        for (int n = 0; n < nchunks && ok; ++n) {
            const int st = n & 1;
            float ga_next = 0.f, gb_next = 0.f;
            if (n + 1 < nchunks) load_gates(n + 1, ga_next, gb_next);
            if (n >= 2) ok = mbar_wait(&bar_empty[st], ((n >> 1) - 1) & 1, a.status, ERR_CHAIN_TMA);
            if (!ok) break;
            if (lane == 0) {
                const int tok0 = chunk_tok0(n);
                uint8_t* d = sStage + st * BSTAGE_BYTES;
                mbar_expect_tx(&bar_full[st], BSTAGE_BYTES);
                bulk_load(d + BS_WT, a.WT + chunk_tile(n) * REC_BYTES, 40960, &bar_full[st]);   // W^T, P', Qg
                for (int hf = 0; hf < 2; ++hf) tma_load_2d(d + BS_DO + hf * BOX, &tmDO, h * KD + hf * 64, tok0, &bar_full[st]);
                for (int hf = 0; hf < 2; ++hf) tma_load_2d(d + BS_KT + hf * BOX, &tmKt, h * KD + hf * 64, tok0, &bar_full[st]);
            }
            __syncwarp();
            warp_gate_vectors(ga, gb, lane, nullptr, sRho[st], &sGC[st]);
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&bar_full[st]);
                // warm L2 two chunks ahead: the stage copies can only run one chunk ahead
                if (n + 2 < nchunks) {
                    const int t2 = chunk_tok0(n + 2);
                    bulk_prefetch(a.WT + chunk_tile(n + 2) * REC_BYTES, 40960);
                    for (int hf = 0; hf < 2; ++hf) {
                        tma_prefetch_2d(&tmDO, h * KD + hf * 64, t2);
                        tma_prefetch_2d(&tmKt, h * KD + hf * 64, t2);
                    }
                }
            }
            ga = ga_next;
            gb = gb_next;
        }
    } else if (warp == CBK_MMA_WARP) {
        // ------------------------------------------------------------------ tensor-core issuer
        bool ok = true;
        bool a1_issued = false;   // dO^T P' of the coming chunk is already in its accumulator
        int next_pub = 1, interval = 1, published = 0;   // publication of finished tiles (lane 0)
        auto issue_a1 = [&](uint8_t* d) {   // acc1 = dO^T P'
            const uint32_t idesc = make_idesc(128, 64, IDESC_A_MN | IDESC_B_MN);
            const uint64_t da0 = desc_mnmajor(d + BS_DO, BOX), db0 = desc_mnmajor(d + BS_P, 0);
            for (int k = 0; k < 4; ++k)
                mma_ss(tA1, desc_advance(da0, 2048 * k), desc_advance(db0, 2048 * k), idesc, k > 0);
        };
        for (int n = 0; n < nchunks && ok; ++n) {
            const int st = n & 1;
            const size_t tile = chunk_tile(n);
            uint8_t* d = sStage + st * BSTAGE_BYTES;
            if (!a1_issued) ok = mbar_wait(&bar_full[st], (n >> 1) & 1, a.status, ERR_CHAIN_TMA);
            ok = ok && mbar_wait(&bar_s_ready, n & 1, a.status, ERR_CHAIN_MMA1);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) {
                bulk_wait_read();   // the ddU^T image of the previous chunk has left shared memory
                bulk_store(a.dSn + tile * 32768, sdS, 32768);   // cotangent at the end of this chunk
                bulk_commit();
                if (!a1_issued) issue_a1(d);
                {   // acc2 = dS Ktil^T
                    const uint32_t idesc = make_idesc(128, 64);
                    for (int k = 0; k < 8; ++k)
                        mma_ss(tA2, desc_advance(desc_kmajor(sdS + (k >> 2) * 16384), 32 * (k & 3)),
                               desc_advance(desc_kmajor(d + BS_KT + (k >> 2) * BOX), 32 * (k & 3)), idesc, k > 0);
                }
                mma_commit(&bar_a_done);
                {   // dS += dO^T Qg (the accumulator has been decayed before s_ready)
                    const uint32_t idesc = make_idesc(128, 128, IDESC_A_MN | IDESC_B_MN);
                    const uint64_t da0 = desc_mnmajor(d + BS_DO, BOX), db0 = desc_mnmajor(d + BS_QG, BOX);
                    for (int k = 0; k < 4; ++k)
                        mma_ss(tS, desc_advance(da0, 2048 * k), desc_advance(db0, 2048 * k), idesc, 1);
                }
            }
            __syncwarp();
            ok = mbar_wait(&bar_a_ready, n & 1, a.status, ERR_CHAIN_MMA2);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) {
                // The dS image sent off above must have left shared memory before the update is
                // released: its completion lets the state warps overwrite that image.
                bulk_wait_read();
                bulk_store(a.ddUT + tile * 16384, sddU, 16384);
                bulk_commit();
                {   // dS -= ddU^T W
                    const uint32_t idesc = make_idesc(128, 128, IDESC_A_NEG);
                    const uint64_t da0 = desc_kmajor(sddU), db0 = desc_kmajor(d + BS_WT);
                    for (int k = 0; k < 4; ++k)
                        mma_ss(tS, desc_advance(da0, 32 * k), desc_advance(db0, 32 * k), idesc, 1);
                }
                mma_commit(&bar_s_done);
                mma_commit(&bar_empty[st]);
            }
            __syncwarp();
            // the state-independent part of the next chunk's ddU^T, while the state warps convert dS
            a1_issued = false;
            if (n + 1 < nchunks && chunk_len(n + 1) == CH) {
                ok = mbar_wait(&bar_full[st ^ 1], ((n + 1) >> 1) & 1, a.status, ERR_CHAIN_TMA);
                if (!ok) break;
                if (lane == 0) issue_a1(sStage + (st ^ 1) * BSTAGE_BYTES);
                __syncwarp();
                a1_issued = true;
            }
            // Finished tiles go to the chunk-local workers in batches: a publication costs the issuing
            // thread a fence and a round trip to memory, and the workers consume far more slowly than the
            // chains produce, so the batches grow (1, 2, 4, ... up to 16 steps).  Only tiles whose two
            // bulk groups were committed at least a whole step ago are included: waiting for this
            // chunk's own stores would put their round trip on the chunk-to-chunk path.
            if (lane == 0 && n >= next_pub) {
                bulk_wait_all_but<2>();
                tq.push((int)chunk_tile(n - 1), H, n - published);   // steps published .. n - 1 (tile ids rise by H per step back)
                published = n;
                interval = min(2 * interval, 16);
                next_pub = n + interval;
            }
            __syncwarp();
        }
        if (lane == 0) {
            bulk_wait_all();
            if (ok) tq.push((int)chunk_tile(nchunks - 1), H, nchunks - published);
        }
    } else {
        // ------------------------------------------------------------------ state warps
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        for (int cb = 0; cb < 2; ++cb) {
            uint32_t r[16];
#pragma unroll
            for (int x4 = 0; x4 < 4; ++x4) {
                const float4 f4 = dfin ? *reinterpret_cast<const float4*>(dfin + cb * 16 + x4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
                r[x4 * 4 + 0] = __float_as_uint(f4.x);
                r[x4 * 4 + 1] = __float_as_uint(f4.y);
                r[x4 * 4 + 2] = __float_as_uint(f4.z);
                r[x4 * 4 + 3] = __float_as_uint(f4.w);
            }
            tmem_st16(tS + lane_addr + colq * 32 + cb * 16, r);
        }
        tmem_st_wait();

        bool ok = true;
        for (int n = 0; n < nchunks && ok; ++n) {
            const int st = n & 1;
            const int len = chunk_len(n);
            uint8_t* d = sStage + st * BSTAGE_BYTES;
            ok = mbar_wait(&bar_full[st], (n >> 1) & 1, a.status, ERR_CHAIN_TMA);   // gate vectors, tail rows
            if (n > 0) ok = ok && mbar_wait(&bar_s_done, (n - 1) & 1, a.status, ERR_CHAIN_MMA2);
            if (!ok) break;
            tc_fence_after();
            // ---- E0: dS (cotangent at the chunk end) -> bf16 operand; decay the accumulator
            {
                const float gC = sGC[st];
                uint32_t rr[2][16];
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) tmem_ld16(tS + lane_addr + colq * 32 + cb * 16, rr[cb]);
                tmem_ld_wait();
#pragma unroll
                for (int cb = 0; cb < 2; ++cb) {
                    uint32_t* r = rr[cb];
#pragma unroll
                    for (int c2 = 0; c2 < 2; ++c2) {
                        uint4 w;
                        w.x = pack_bf16(__uint_as_float(r[c2 * 8 + 0]), __uint_as_float(r[c2 * 8 + 1]));
                        w.y = pack_bf16(__uint_as_float(r[c2 * 8 + 2]), __uint_as_float(r[c2 * 8 + 3]));
                        w.z = pack_bf16(__uint_as_float(r[c2 * 8 + 4]), __uint_as_float(r[c2 * 8 + 5]));
                        w.w = pack_bf16(__uint_as_float(r[c2 * 8 + 6]), __uint_as_float(r[c2 * 8 + 7]));
                        *reinterpret_cast<uint4*>(sdS + (colq >> 1) * 16384 + sw128_chunk(v, (colq & 1) * 4 + cb * 2 + c2)) = w;
                    }
#pragma unroll
                    for (int x = 0; x < 16; ++x) r[x] = __float_as_uint(__uint_as_float(r[x]) * gC);
                    tmem_st16(tS + lane_addr + colq * 32 + cb * 16, r);
                }
                tmem_st_wait();
            }
            if (len < CH) {
                for (int hf = 0; hf < 2; ++hf) {
                    zero_tail_rows(d + BS_DO + hf * BOX, len, tid, CBK_EPI_WARPS * 32);
                    zero_tail_rows(d + BS_KT + hf * BOX, len, tid, CBK_EPI_WARPS * 32);
                }
            }
            fence_proxy_async();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_s_ready);

            // ---- E1: ddU^T = acc1 + rho_i acc2 -> bf16 operand
            float rho[16];
#pragma unroll
            for (int x = 0; x < 16; ++x) rho[x] = sRho[st][colq * 16 + x];
            ok = mbar_wait(&bar_a_done, n & 1, a.status, ERR_CHAIN_MMA1);
            if (!ok) break;
            tc_fence_after();
            {
                uint32_t r1[16], r2[16];
                tmem_ld16(tA1 + lane_addr + colq * 16, r1);
                tmem_ld16(tA2 + lane_addr + colq * 16, r2);
                tmem_ld_wait();
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {
                    float f[8];
#pragma unroll
                    for (int x = 0; x < 8; ++x)
                        f[x] = __uint_as_float(r1[c2 * 8 + x]) + rho[c2 * 8 + x] * __uint_as_float(r2[c2 * 8 + x]);
                    *reinterpret_cast<uint4*>(sddU + sw128_chunk(v, colq * 2 + c2)) =
                        make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
                }
            }
            fence_proxy_async();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_a_ready);
        }
        if (ok) ok = mbar_wait(&bar_s_done, (nchunks - 1) & 1, a.status, ERR_CHAIN_MMA2);
        tc_fence_after();
        if (ok && dini) {
            for (int cb = 0; cb < 2; ++cb) {
                uint32_t r[16];
                tmem_ld16(tS + lane_addr + colq * 32 + cb * 16, r);
                tmem_ld_wait();
#pragma unroll
                for (int x4 = 0; x4 < 4; ++x4)
                    *reinterpret_cast<float4*>(dini + cb * 16 + x4 * 4) =
                        make_float4(__uint_as_float(r[x4 * 4 + 0]), __uint_as_float(r[x4 * 4 + 1]),
                                    __uint_as_float(r[x4 * 4 + 2]), __uint_as_float(r[x4 * 4 + 3]));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {   // the barrier words are initialised again for the CTA's next chain
        mbar_inval(&bar_full[0]); mbar_inval(&bar_full[1]); mbar_inval(&bar_empty[0]); mbar_inval(&bar_empty[1]);
        mbar_inval(&bar_s_ready); mbar_inval(&bar_a_done); mbar_inval(&bar_a_ready); mbar_inval(&bar_s_done);
    }
    __syncthreads();
    tc_fence_after();
}

// ---------------------------------------------------------------------------------------------
// chunk-local backward.  Feature-major ("transposed") accumulators: lane = feature, column = token.
//   phase A : dP' = dO dU^T ; dQ1^T = S^T dO^T ; dKtr^T = dS^T dU ; dW^T = -S^T ddU
//             (reads only what the chain kernels and the caller wrote: issued a tile ahead)
//   phase B : dT = (dW K^T) beta gamma + (ddU V^T) beta ; dKb^T = dW^T T ; dVb^T = ddU^T T ;
//             dq2^T = Ktil^T M1^T ; dktil^T = Q^T M1            (M1 = scale Gamma (.) lower(dP'))
//             dbeta_j += sum_i T_ij (gamma_j dW K^T + ddU V^T)_ij
//   phase C : Y = T^T dT ; rawkk = K Ktil^T
//   phase D : Z = Y T^T, dA = -strictLower(Z), M2 = dA beta_i Gamma_ij, dbeta_i += sum_j dA_ij Gamma_ij rawkk_ij
//   phase E : dktil^T += K^T M2 ; dkr^T = Ktil^T M2^T
//   final   : dq = scale gamma dQ1 + dq2 ; dktil += rho dKtr ; dk_read = dkr + beta gamma dKb ;
//             dv = beta dVb ; dgate from the products of the gradients with their inputs
// ---------------------------------------------------------------------------------------------
struct TcChunkBwdArgs {
    int H, ntiles, nseq;
    Table tab;
    const float *beta, *gate;
    float scale, d_min;
    const uint8_t *Tm, *Sn, *dSn, *dUT, *ddUT;
    const unsigned* skipw;
    __nv_bfloat16 *dq, *dk, *dv;
    float *dbeta, *dgate, *dktil, *dkread;
    int* status;
};

constexpr int CBW_THREADS = 512;   // 16 warps = 4 lane quadrants x 4 column groups
constexpr uint32_t R_Q = 0, R_K = 16384, R_KT = 32768, R_V = 49152, R_DO = 65536, R_DU = 81920, R_DDU = 98304,
                   R_T = 114688, R_S = 122880, R_DS = 155648, R_RAW = 188416;
constexpr uint32_t R_DWT = R_DO;                 // dW^T image replaces dO after phase A
// M1, dT, Y and M2 are live one after the other (each is written once the product that read its
// predecessor has finished), so they share one 8 KB image behind the fp32 scratch.
constexpr uint32_t R_IMG = R_RAW + 24576;
// Output staging ([token][feature] tiles over dead space): dq over V (dead after phase B; dq is complete
// then and is formed while phase C runs), dv over Q (dead once dq is formed; dv is formed while phase E
// runs), dk after the last product in a region of its own; the fp32 copies of dk_read and dL/dktil,
// needed only when some token's preconditioner step was really taken, over T, S and dS.  When every token of a full chunk was
// skipped, the space of dO, dU, ddU, T, S and dS is therefore never reused inside a tile and the next
// tile's copies of them start as soon as the last product reading the current ones has finished.
constexpr uint32_t ST_DQ = R_V, ST_DV = R_Q, ST_DK = R_RAW, ST_DKR = 114688, ST_DKT = 147456;
constexpr int CBW_STORE_TID = 256;   // the thread that sends the output tiles off (and owns their bulk group)
constexpr int CBW_QUEUE_TID = 480;   // the thread that talks to the tile queue (a warp that issues no products)
static_assert(ST_DKT + 32768 <= R_RAW, "fp32 staging tiles must fit below the fp32 scratch");
constexpr size_t CBW_SMEM = R_RAW + 32768 + 1024;

// The chunk-local backward of the tiles drawn from the queue, by the first CBW_THREADS threads of the CTA
// (their barrier is hardware barrier 1).  `tb`: 512 tensor-memory columns.
__device__ __forceinline__ void chunk_bwd_role(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmKt,
                                               const CUtensorMap& tmV, const CUtensorMap& tmDO, const CUtensorMap& tmDQ,
                                               const CUtensorMap& tmDK, const CUtensorMap& tmDV, const TcChunkBwdArgs& a,
                                               uint8_t* sm, uint32_t tb, const TileQueue& tq)
{
    // bar_ct: dO and the tiles written by the chain kernels (everything phase A reads);
    // bar_tok: q, k, ktil, v
    __shared__ uint64_t bar_ct, bar_tok, bar_mma[5];
    __shared__ int sNext[4];   // next tile of this CTA: {tile, head, first token, length}; tile -1: not published yet, -2: none left
    // per-token sums of a tile (two buffers: the sums of a tile are finished while the next tile's phase B runs)
    __shared__ __align__(16) float sdBv[2][CH], sdGv[2][CH], sRedv[2][CBW_THREADS / 32];
    // in-chunk gate prefix G_i, gamma_i = exp(G_i), rho_i = exp(G_C - G_i): two buffers, the next tile's
    // vectors are formed during this tile's last stretch
    __shared__ __align__(16) float sGv[2][3][CH];
    // per-token gate and beta and the two skip words of a tile, copied asynchronously one tile ahead
    // (two buffers; values fetched into registers that early would be spilled, and the spill would wait
    // for the load)
    __shared__ __align__(16) float sScal[2][2][CH];
    __shared__ unsigned sSkipW[2][2];
    __shared__ float sRsumv[2];
    __shared__ __align__(16) float sFirstKt[KD];

    const int H = a.H;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int quad = warp & 3, colq = warp >> 2;   // lane quadrant, column group (16 columns each)
    const int f = quad * 32 + lane;                 // feature (k or v) owned in 128-lane accumulators
    // 64-row accumulators keep their rows in lanes 0-15 of each quadrant: thread t reads row
    // quad * 16 + (t & 15), eight columns (threads 16-31 the second eight of the warp's sixteen)
    const int row64 = quad * 16 + (lane & 15);
    const int jb = colq * 16 + (lane >> 4) * 8;     // first of the eight columns
    const uint32_t addr64 = ((uint32_t)(quad * 32) << 16) + colq * 16;

    if (tid == 0) {
        mbar_init(&bar_ct, 1);
        mbar_init(&bar_tok, 1);
        // the independent products of a phase are issued by different warps (the issue rate of one
        // thread, not the tensor pipe, limits these small shapes); each issuer commits for itself
        const uint32_t issuers[5] = {4, 6, 2, 1, 2};
        for (int i = 0; i < 5; ++i) mbar_init(&bar_mma[i], issuers[i]);
        fence_mbar_init();
    }
    tc_fence_before();
    named_sync(1, CBW_THREADS);
    tc_fence_after();
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;

    // tensor memory columns
    const uint32_t cDP = 64, cDQ1 = 128, cDKTR = 192, cDW = 256;                       // phase A
    const uint32_t cDTA = 320, cDTB = 384, cDKB = 256, cDVB = 64, cDQ2 = 0, cDKT = 448;   // phase B
    const uint32_t cY = 320, cRAW = 384, cZ = 320, cDKR = 384;                          // phases C, D, E

    // persistent: one CTA per SM walks over the (chunk, head) tiles.  The operands of the next tile
    // are requested as soon as the shared-memory regions they land in are dead, its per-token scalars
    // are fetched into registers one tile ahead, and its first products (phase A, which reads only what
    // the chain kernels and the caller wrote) are issued while the current tile's sums and stores
    // are still being formed.
    // Tiles come from the queue the chains fill, in the order they were finished: thread 0 draws a ticket,
    // looks the slot up (waiting, within a bound, only where nothing else is left to do) and leaves the
    // tile's coordinates in shared memory for the others.
    const int total = a.tab.seq_chunk0(a.nseq) * H;   // realised (chunk, head) tiles
    auto resolve = [&](int v) {   // queue thread only: v = slot value (tile + 1) or 0 (not published)
        if (!v) { sNext[0] = -1; return; }
        const int t = v - 1, c = t / H;
        sNext[0] = t;
        sNext[1] = t - c * H;
        sNext[2] = a.tab.chunk_tok0(c);
        sNext[3] = a.tab.chunk_len(c);
        fence_proxy_async_all();   // the tile's images are read through the async proxy
    };
    auto lookup_blocking = [&](unsigned ticket) {   // queue thread only
        if (ticket >= (unsigned)total) { sNext[0] = -2; return; }
        int v = ld_acquire_gpu(tq.slots + ticket);
        if (!v) {
            const long long t0 = clock64();
            while (!(v = ld_acquire_gpu(tq.slots + ticket))) {
                if (clock64() - t0 > WAIT_LIMIT_CYCLES || *reinterpret_cast<volatile int*>(a.status) != 0) break;
                __nanosleep(64);
            }
            if (!v) atomicCAS(a.status, 0, ERR_QUEUE);
        }
        if (!v) { sNext[0] = -2; return; }
        resolve(v);
    };
    // The copies of a tile arrive on one phase of each barrier; the transaction count is announced with
    // the first group that is issued, whichever that is.
    constexpr uint32_t CT_TX = 2 * BOX + 16384 + 16384 + 8192 + 32768 + 32768, TOK_TX = 8 * BOX;
    auto load_kkt = [&](int hh, int t0) {
        for (int hf = 0; hf < 2; ++hf) {
            tma_load_2d(sm + R_K + hf * BOX, &tmK, hh * KD + hf * 64, t0, &bar_tok);
            tma_load_2d(sm + R_KT + hf * BOX, &tmKt, hh * KD + hf * 64, t0, &bar_tok);
        }
    };
    auto load_qv = [&](int hh, int t0) {
        for (int hf = 0; hf < 2; ++hf) {
            tma_load_2d(sm + R_Q + hf * BOX, &tmQ, hh * KD + hf * 64, t0, &bar_tok);
            tma_load_2d(sm + R_V + hf * BOX, &tmV, hh * KD + hf * 64, t0, &bar_tok);
        }
    };
    auto load_dout = [&](int hh, int t0) {
        for (int hf = 0; hf < 2; ++hf) tma_load_2d(sm + R_DO + hf * BOX, &tmDO, hh * KD + hf * 64, t0, &bar_ct);
    };
    auto load_du_ds_s = [&](int t) {
        bulk_load(sm + R_DU, a.dUT + (size_t)t * 16384, 16384, &bar_ct);
        bulk_load(sm + R_DS, a.dSn + (size_t)t * 32768, 32768, &bar_ct);
        bulk_load(sm + R_S, a.Sn + (size_t)t * 32768, 32768, &bar_ct);
    };
    auto load_ddu = [&](int t) { bulk_load(sm + R_DDU, a.ddUT + (size_t)t * 16384, 16384, &bar_ct); };
    auto load_t = [&](int t) { bulk_load(sm + R_T, a.Tm + (size_t)t * 8192, 8192, &bar_ct); };
    auto fetch_scalars = [&](int t, int hh, int t0, int ln, int buf) {   // tokens beyond the chunk read as zero
        if (tid < CH) {
            const bool in = tid < ln;
            const size_t th = (size_t)(t0 + (in ? tid : 0)) * H + hh;
            cp_async4_zfill(&sScal[buf][0][tid], a.gate + th, in);
            cp_async4_zfill(&sScal[buf][1][tid], a.beta + th, in);
        } else if (tid < CH + 2) {
            cp_async4_zfill(&sSkipW[buf][tid - CH], a.skipw + (size_t)t * 2 + (tid - CH), true);
        }
        cp_async_commit();
    };
    // phase A: dP' = dO dU^T ; dQ1^T = S^T dO^T ; dKtr^T = dS^T dU ; dW^T = -S^T ddU  (warps 0-3, one each)
    auto issue_phase_a = [&](bool go) {
        if (lane == 0 && warp < 4 && go) {
            tc_fence_after();
            if (warp == 0) {   // dP'[i][j] = sum_v dO[i][v] dU[j][v]                               (M = 64)
                const uint64_t db0 = desc_mnmajor(sm + R_DU, 0);
                for (int k = 0; k < 8; ++k)
                    mma_ss(tb + cDP, desc_advance(desc_kmajor(sm + R_DO + (k >> 2) * BOX), 32 * (k & 3)),
                           desc_advance(db0, 2048 * k), make_idesc(64, 64, IDESC_B_MN), k > 0);
            }
            if (warp == 1) {   // dQ1^T[k][i] = sum_v S[v][k] dO[i][v]
                const uint64_t da0 = desc_mnmajor(sm + R_S, 16384);
                for (int k = 0; k < 8; ++k)
                    mma_ss(tb + cDQ1, desc_advance(da0, 2048 * k),
                           desc_advance(desc_kmajor(sm + R_DO + (k >> 2) * BOX), 32 * (k & 3)),
                           make_idesc(128, 64, IDESC_A_MN), k > 0);
            }
            if (warp == 2) {   // dKtr^T[k][j] = sum_v dS[v][k] dU[j][v]
                const uint64_t da0 = desc_mnmajor(sm + R_DS, 16384), db0 = desc_mnmajor(sm + R_DU, 0);
                for (int k = 0; k < 8; ++k)
                    mma_ss(tb + cDKTR, desc_advance(da0, 2048 * k), desc_advance(db0, 2048 * k),
                           make_idesc(128, 64, IDESC_A_MN | IDESC_B_MN), k > 0);
            }
            if (warp == 3) {   // dW^T[k][i] = -sum_v S[v][k] ddU[i][v]
                const uint64_t da0 = desc_mnmajor(sm + R_S, 16384), db0 = desc_mnmajor(sm + R_DDU, 0);
                for (int k = 0; k < 8; ++k)
                    mma_ss(tb + cDW, desc_advance(da0, 2048 * k), desc_advance(db0, 2048 * k),
                           make_idesc(128, 64, IDESC_A_MN | IDESC_B_MN | IDESC_A_NEG), k > 0);
            }
            mma_commit(&bar_mma[0]);
        }
    };
    auto gate_vectors = [&](int buf) {   // one warp; lane: tokens l and l + 32
        float sa = sScal[buf][0][lane], sb = sScal[buf][0][lane + 32];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float ua = __shfl_up_sync(0xffffffffu, sa, o), ub = __shfl_up_sync(0xffffffffu, sb, o);
            if (lane >= o) { sa += ua; sb += ub; }
        }
        sb += __shfl_sync(0xffffffffu, sa, 31);
        const float tot = __shfl_sync(0xffffffffu, sb, 31);
        sGv[buf][0][lane] = sa;
        sGv[buf][0][lane + 32] = sb;
        sGv[buf][1][lane] = __expf(sa);
        sGv[buf][1][lane + 32] = __expf(sb);
        sGv[buf][2][lane] = __expf(tot - sa);
        sGv[buf][2][lane + 32] = __expf(tot - sb);
    };
    // The per-token sums of a tile (gate and beta gradients) are finished one tile later, while the tensor
    // core works on the next tile's phase B: the partial terms stay in registers until then.
    float gv[16];       // per column: gate contribution of this thread's feature
    float rsum = 0.f;
    bool pend = false;  // the previous tile's sums are still to be finished
    int p_tok0 = 0, p_h = 0, p_len = 0;
    auto reduce_sums = [&](int buf) {   // all warps: 32 features of each warp, 16 columns at once
#pragma unroll
        for (int step = 0; step < 4; ++step) {   // a lane keeps one half of its columns, hands the other half over
            const int off = 16 >> step, n = 8 >> step;
            const bool upper = (lane & off) != 0;
#pragma unroll
            for (int i = 0; i < n; ++i) {
                const float gs = upper ? gv[i] : gv[i + n], gk = upper ? gv[i + n] : gv[i];
                gv[i] = gk + __shfl_xor_sync(0xffffffffu, gs, off);
            }
        }
        gv[0] += __shfl_xor_sync(0xffffffffu, gv[0], 1);   // the two lanes that ended up with the same column
        if ((lane & 1) == 0) atomicAdd(&sdGv[buf][colq * 16 + (lane >> 1)], gv[0]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) rsum += __shfl_xor_sync(0xffffffffu, rsum, o);
        if (lane == 0) atomicAdd(&sRsumv[buf], rsum);
    };
    // one warp: dgate_j is the suffix sum of the per-token terms (the in-chunk prefix G_i collects every
    // g_j with j <= i); the chunk-level term goes to the last token
    auto finish_sums = [&](int buf, int t0, int hh, int ln) {
        float s0 = sdGv[buf][lane], s1 = sdGv[buf][lane + 32];
        float gl = sScal[buf][0][lane] + sScal[buf][0][lane + 32], tot = lane < CBW_THREADS / 32 ? sRedv[buf][lane] : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            gl += __shfl_xor_sync(0xffffffffu, gl, o);
            tot += __shfl_xor_sync(0xffffffffu, tot, o);
        }
        if (lane == 31) s1 += sRsumv[buf] + __expf(gl) * tot;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float u0 = __shfl_down_sync(0xffffffffu, s0, o), u1 = __shfl_down_sync(0xffffffffu, s1, o);
            if (lane + o < 32) { s0 += u0; s1 += u1; }
        }
        s0 += __shfl_sync(0xffffffffu, s1, 0);
        if (lane < ln) {
            const size_t th = (size_t)(t0 + lane) * H + hh;
            a.dgate[th] = s0;
            a.dbeta[th] = sdBv[buf][lane];
        }
        if (lane + 32 < ln) {
            const size_t th = (size_t)(t0 + lane + 32) * H + hh;
            a.dgate[th] = s1;
            a.dbeta[th] = sdBv[buf][lane + 32];
        }
    };
    uint32_t ph = 0;   // barrier phase parity: number of tiles processed so far, mod 2
    // queue thread: the ticket of the next tile is drawn a tile ahead and its slot is read at the top of
    // the tile, long before the value is looked at, so that neither round trip to memory is waited for
    unsigned ticket_next = 0, ticket_after = 0;
    int slot_next = 0;
    if (tid == CBW_QUEUE_TID) {
        lookup_blocking(atomicAdd(tq.head, 1u));
        ticket_next = atomicAdd(tq.head, 1u);
    }
    named_sync(1, CBW_THREADS);
    int tile_l = sNext[0], h = sNext[1], tok0 = sNext[2], len = sNext[3];
    bool a_issued = false;   // phase A of the current tile was issued at the end of the previous one
    if (tile_l >= 0) {
        if (tid == 0) {
            mbar_expect_tx(&bar_ct, CT_TX);
            load_dout(h, tok0);
            load_du_ds_s(tile_l);
            load_ddu(tile_l);
            load_t(tile_l);
            mbar_expect_tx(&bar_tok, TOK_TX);
            load_kkt(h, tok0);
            load_qv(h, tok0);
        }
        fetch_scalars(tile_l, h, tok0, len, 0);
    }
    while (tile_l >= 0) {
    const float* sg = sScal[ph][0];      // log-gates of the chunk's tokens
    const float* sBeta = sScal[ph][1];
    float* sdB = sdBv[ph];
    float* sdG = sdGv[ph];
    float* sRed = sRedv[ph];
    const float* sG = sGv[ph][0];
    const float* sGam = sGv[ph][1];
    const float* sRho = sGv[ph][2];
    if (tid < CH) {
        sdB[tid] = 0.f;
        sdG[tid] = 0.f;
    }
    if (tid == 0) sRsumv[ph] = 0.f;
    cp_async_wait_all();
    named_sync(1, CBW_THREADS);
    // the next tile's slot and the ticket of the tile after it (both values are used much later)
    if (tid == CBW_QUEUE_TID) {
        ticket_after = atomicAdd(tq.head, 1u);
        slot_next = ticket_next < (unsigned)total ? ld_acquire_gpu(tq.slots + ticket_next) : 0;
    }
    const unsigned long long sk = (unsigned long long)sSkipW[ph][0] | ((unsigned long long)sSkipW[ph][1] << 32);
    // Full chunks leave through TMA tile stores (dq, dv always; dk when every token's preconditioner
    // step was skipped); ragged or mixed chunks are copied row by row.  In the all-skipped case the
    // space of dO and of each chain tile is not reused by the output staging, so the next tile's copy of
    // it starts as soon as the last product reading it has finished ("early"), and when that tile is a
    // full chunk its phase A is issued before this tile's sums are formed ("a_early").
    const bool full = len == CH;
    const bool dk_tile = full && sk == ~0ull;
    if (warp == 0) gate_vectors((int)ph);
    bool ok = mbar_wait(&bar_ct, ph, a.status, ERR_TMA);
    if (len < CH) {   // a ragged chunk never had its phase A issued ahead
        for (int hf = 0; hf < 2; ++hf) zero_tail_rows(sm + R_DO + hf * BOX, len, tid, CBW_THREADS);
        fence_proxy_async();
    }
    tc_fence_before();
    named_sync(1, CBW_THREADS);

    // ---- phase A -------------------------------------------------------------------------------
    if (!a_issued) issue_phase_a(ok);
    ok = ok && mbar_wait(&bar_mma[0], ph, a.status, ERR_MMA1);
    tc_fence_after();
    // epilogue A
    float gam8[8];   // Gamma_ij = exp(G_i - G_j) for this thread's row and columns, j <= i (else 0)
    {
        // dP' -> M1 = scale Gamma (.) lower(dP')
        const int i = row64;
        const float Gi = sG[i];
        {
            uint32_t r2[8];
            tmem_ld_half8(tb + cDP + addr64, r2);
            float m1[8];
#pragma unroll
            for (int x = 0; x < 8; ++x) gam8[x] = jb + x <= i ? __expf(Gi - sG[jb + x]) : 0.f;
            tmem_ld_wait();
#pragma unroll
            for (int x = 0; x < 8; ++x) m1[x] = a.scale * gam8[x] * __uint_as_float(r2[x]);
            *reinterpret_cast<uint4*>(sm + R_IMG + sw128_chunk(i, jb >> 3)) =
                make_uint4(pack_bf16(m1[0], m1[1]), pack_bf16(m1[2], m1[3]), pack_bf16(m1[4], m1[5]), pack_bf16(m1[6], m1[7]));
        }
        // dW^T -> bf16 image [rows k][cols i]
        {
            uint32_t r[16];
            tmem_ld16(tb + cDW + lane_addr + colq * 16, r);
            tmem_ld_wait();
#pragma unroll
            for (int c2 = 0; c2 < 2; ++c2)
                *reinterpret_cast<uint4*>(sm + R_DWT + sw128_chunk(f, colq * 2 + c2)) = make_uint4(
                    pack_bf16(__uint_as_float(r[c2 * 8 + 0]), __uint_as_float(r[c2 * 8 + 1])),
                    pack_bf16(__uint_as_float(r[c2 * 8 + 2]), __uint_as_float(r[c2 * 8 + 3])),
                    pack_bf16(__uint_as_float(r[c2 * 8 + 4]), __uint_as_float(r[c2 * 8 + 5])),
                    pack_bf16(__uint_as_float(r[c2 * 8 + 6]), __uint_as_float(r[c2 * 8 + 7])));
        }
    }
    ok = ok && mbar_wait(&bar_tok, ph, a.status, ERR_TMA);   // q, k, ktil, v have landed
    if (len < CH) {
        for (int hf = 0; hf < 2; ++hf) {
            zero_tail_rows(sm + R_Q + hf * BOX, len, tid, CBW_THREADS);
            zero_tail_rows(sm + R_K + hf * BOX, len, tid, CBW_THREADS);
            zero_tail_rows(sm + R_KT + hf * BOX, len, tid, CBW_THREADS);
            zero_tail_rows(sm + R_V + hf * BOX, len, tid, CBW_THREADS);
        }
    }
    fence_proxy_async();
    tc_fence_before();
    named_sync(1, CBW_THREADS);

    // ---- phase B -------------------------------------------------------------------------------
    if (lane == 0 && warp < 6 && ok) {
        tc_fence_after();
        if (warp == 0) {   // dT_a[i][j] = sum_k dW[i][k] K[j][k]                               (M = 64)
            const uint64_t da0 = desc_mnmajor(sm + R_DWT, 0);
            for (int k = 0; k < 8; ++k)
                mma_ss(tb + cDTA, desc_advance(da0, 2048 * k),
                       desc_advance(desc_kmajor(sm + R_K + (k >> 2) * BOX), 32 * (k & 3)),
                       make_idesc(64, 64, IDESC_A_MN), k > 0);
        }
        if (warp == 1) {   // dT_b[i][j] = sum_v ddU[i][v] V[j][v]                              (M = 64)
            const uint64_t da0 = desc_mnmajor(sm + R_DDU, 0);
            for (int k = 0; k < 8; ++k)
                mma_ss(tb + cDTB, desc_advance(da0, 2048 * k),
                       desc_advance(desc_kmajor(sm + R_V + (k >> 2) * BOX), 32 * (k & 3)),
                       make_idesc(64, 64, IDESC_A_MN), k > 0);
        }
        if (warp == 2 || warp == 3) {   // dKb^T[k][j] = sum_i dW^T[k][i] T[i][j] ;  dVb^T[v][j] = sum_i ddU^T[v][i] T[i][j]
            const uint64_t db0 = desc_mnmajor(sm + R_T, 0);
            const uint64_t da0 = desc_kmajor(sm + R_DWT), da1 = desc_kmajor(sm + R_DDU);
            if (warp == 2)
                for (int k = 0; k < 4; ++k)
                    mma_ss(tb + cDKB, desc_advance(da0, 32 * k), desc_advance(db0, 2048 * k),
                           make_idesc(128, 64, IDESC_B_MN), k > 0);
            else
                for (int k = 0; k < 4; ++k)
                    mma_ss(tb + cDVB, desc_advance(da1, 32 * k), desc_advance(db0, 2048 * k),
                           make_idesc(128, 64, IDESC_B_MN), k > 0);
        }
        if (warp == 4 || warp == 5) {   // dq2^T[k][i] = sum_j Ktil[j][k] M1[i][j] ;  dktil^T[k][j] = sum_i Q[i][k] M1[i][j]
            const uint64_t da0 = desc_mnmajor(sm + R_KT, BOX), da1 = desc_mnmajor(sm + R_Q, BOX);
            const uint64_t dbk = desc_kmajor(sm + R_IMG), dbm = desc_mnmajor(sm + R_IMG, 0);
            if (warp == 4)
                for (int k = 0; k < 4; ++k)
                    mma_ss(tb + cDQ2, desc_advance(da0, 2048 * k), desc_advance(dbk, 32 * k),
                           make_idesc(128, 64, IDESC_A_MN), k > 0);
            else
                for (int k = 0; k < 4; ++k)
                    mma_ss(tb + cDKT, desc_advance(da1, 2048 * k), desc_advance(dbm, 2048 * k),
                           make_idesc(128, 64, IDESC_A_MN | IDESC_B_MN), k > 0);
        }
        mma_commit(&bar_mma[1]);
    }
    if (pend) reduce_sums((int)(ph ^ 1u));   // the previous tile's per-token sums
    // <dS, S>_F while the tensor core works on phase B (both images share the same layout)
    {
        float p4[4] = {0.f, 0.f, 0.f, 0.f};   // independent partial sums: no chain of dependent multiply-adds
#pragma unroll
        for (int it = 0; it < 2048 / CBW_THREADS; ++it) {
            const int e = tid + it * CBW_THREADS;
            const uint4 x = *reinterpret_cast<const uint4*>(sm + R_S + e * 16);
            const uint4 y = *reinterpret_cast<const uint4*>(sm + R_DS + e * 16);
            const __nv_bfloat162* px = reinterpret_cast<const __nv_bfloat162*>(&x);
            const __nv_bfloat162* py = reinterpret_cast<const __nv_bfloat162*>(&y);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float2 fx = __bfloat1622float2(px[q]), fy = __bfloat1622float2(py[q]);
                p4[q] = fmaf(fx.x, fy.x, p4[q]);
                p4[q] = fmaf(fx.y, fy.y, p4[q]);
            }
        }
        float part = (p4[0] + p4[1]) + (p4[2] + p4[3]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
        if (lane == 0) sRed[warp] = part;
    }
    named_sync(1, CBW_THREADS);   // every thread is done reading S / dS: phase A has finished, dU, dS and S are dead
    if (pend && warp == 1) finish_sums((int)(ph ^ 1u), p_tok0, p_h, p_len);
    // the next tile, if the chains have published it already (asked again at the end of this tile if not);
    // the queue thread works this out while everybody waits for phase B, the others read it after the next barrier
    if (tid == CBW_QUEUE_TID) {
        if (ticket_next >= (unsigned)total) sNext[0] = -2;
        else resolve(slot_next);
        if (dk_tile && sNext[0] >= 0 && ok) {
            mbar_expect_tx(&bar_ct, CT_TX);
            load_du_ds_s(sNext[0]);
        }
    }
    ok = ok && mbar_wait(&bar_mma[1], ph, a.status, ERR_MMA2);
    tc_fence_after();
    {   // dT = dT_a beta_j gamma_j + dT_b beta_j  -> bf16 image [rows i][cols j];
        // dbeta_j += sum_i T_ij (gamma_j dT_a + dT_b)_ij: beta enters W = T diag(beta gamma) K and
        // U = T diag(beta) V column by column
        const int i = row64;
        uint32_t r1[8], r2[8];
        tmem_ld_half8(tb + cDTA + addr64, r1);
        tmem_ld_half8(tb + cDTB + addr64, r2);
        const uint4 tw = *reinterpret_cast<const uint4*>(sm + R_T + sw128_chunk(i, jb >> 3));
        const float4 ba = *reinterpret_cast<const float4*>(&sBeta[jb]), bb = *reinterpret_cast<const float4*>(&sBeta[jb + 4]);
        const float4 ga = *reinterpret_cast<const float4*>(&sGam[jb]), gb = *reinterpret_cast<const float4*>(&sGam[jb + 4]);
        const float bj[8] = {ba.x, ba.y, ba.z, ba.w, bb.x, bb.y, bb.z, bb.w};
        const float gj[8] = {ga.x, ga.y, ga.z, ga.w, gb.x, gb.y, gb.z, gb.w};
        float tij[8];
        {
            const __nv_bfloat162* p0 = reinterpret_cast<const __nv_bfloat162*>(&tw);
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const float2 u0 = __bfloat1622float2(p0[x]);
                tij[2 * x] = u0.x;
                tij[2 * x + 1] = u0.y;
            }
        }
        tmem_ld_wait();
        float t[8], cs[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const float u = gj[x] * __uint_as_float(r1[x]) + __uint_as_float(r2[x]);
            t[x] = bj[x] * u;
            cs[x] = tij[x] * u;
        }
        *reinterpret_cast<uint4*>(sm + R_IMG + sw128_chunk(i, jb >> 3)) =
            make_uint4(pack_bf16(t[0], t[1]), pack_bf16(t[2], t[3]), pack_bf16(t[4], t[5]), pack_bf16(t[6], t[7]));
        // column sums over the 16 rows of a half warp: in each of three steps a lane keeps one half of its
        // columns and hands the other half to its partner; a last exchange joins the two lanes that end
        // up with the same column
#pragma unroll
        for (int step = 0; step < 3; ++step) {
            const int off = 8 >> step, n = 4 >> step;
            const bool upper = (lane & off) != 0;
#pragma unroll
            for (int x = 0; x < n; ++x) {
                const float send = upper ? cs[x] : cs[x + n], keep = upper ? cs[x + n] : cs[x];
                cs[x] = keep + __shfl_xor_sync(0xffffffffu, send, off);
            }
        }
        cs[0] += __shfl_xor_sync(0xffffffffu, cs[0], 1);
        if ((lane & 1) == 0) atomicAdd(&sdB[jb + ((lane & 15) >> 1)], cs[0]);
    }
    fence_proxy_async();
    tc_fence_before();
    named_sync(1, CBW_THREADS);

    int tile_next = sNext[0], h_next = sNext[1], tok0_next = sNext[2], len_next = sNext[3];
    const bool next_known = tile_next >= 0;
    if (next_known) fetch_scalars(tile_next, h_next, tok0_next, len_next, (int)(ph ^ 1u));
    const bool early = dk_tile && next_known;
    const bool a_early = early && len_next == CH;

    // ---- phase C: Y[a][b] = sum_i T[i][a] dT[i][b] ; rawkk[i][j] = <k_i, ktil_j> -------------------
    if (lane == 0 && warp < 2 && ok) {
        tc_fence_after();
        if (warp == 0) {
            const uint64_t da0 = desc_mnmajor(sm + R_T, 0), db0 = desc_mnmajor(sm + R_IMG, 0);
            for (int k = 0; k < 4; ++k)
                mma_ss(tb + cY, desc_advance(da0, 2048 * k), desc_advance(db0, 2048 * k),
                       make_idesc(64, 64, IDESC_A_MN | IDESC_B_MN), k > 0);
        } else {
            for (int k = 0; k < 8; ++k)   // (M = 64)
                mma_ss(tb + cRAW, desc_advance(desc_kmajor(sm + R_K + (k >> 2) * BOX), 32 * (k & 3)),
                       desc_advance(desc_kmajor(sm + R_KT + (k >> 2) * BOX), 32 * (k & 3)), make_idesc(64, 64), k > 0);
        }
        mma_commit(&bar_mma[2]);
        if (early && warp == 0) {   // phase B has finished: ddU and the dW^T image (in the space of dO) are dead
            load_ddu(tile_next);
            load_dout(h_next, tok0_next);
        }
    }
    // dq = scale gamma dQ1 + dq2 (both complete since phase B) while the tensor core works on phase C
    // (lane = feature f, columns = tokens; four token columns at a time)
    const uint32_t boxf = (uint32_t)(f >> 6) * BOX;
    const uint32_t fc = f & 63;
    {
        __nv_bfloat16* stq = reinterpret_cast<__nv_bfloat16*>(sm + ST_DQ);
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
            const int j0 = colq * 16 + cb * 4;
            uint32_t rq1[4], rq2[4];
            tmem_ld4(tb + cDQ1 + lane_addr + j0, rq1);
            tmem_ld4(tb + cDQ2 + lane_addr + j0, rq2);
            float qv[4];
            const float4 g4 = *reinterpret_cast<const float4*>(&sGam[j0]);
            const float gj[4] = {g4.x, g4.y, g4.z, g4.w};
#pragma unroll
            for (int x = 0; x < 4; ++x)
                qv[x] = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sm + R_Q + boxf + sw128_elem(j0 + x, fc)));
            tmem_ld_wait();
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const float dq = a.scale * gj[x] * __uint_as_float(rq1[x]) + __uint_as_float(rq2[x]);
                gv[cb * 4 + x] = dq * qv[x];
                stq[(j0 + x) * KD + f] = __float2bfloat16_rn(dq);
            }
        }
    }
    ok = ok && mbar_wait(&bar_mma[2], ph, a.status, ERR_MMA2);
    tc_fence_after();
    float rawg[8];   // Gamma_ij <k_i, ktil_j>, j < i (kept in registers for the beta gradient of phase D)
    {
        const int i = row64;
        uint32_t r[8], r1[8];
        tmem_ld_half8(tb + cY + addr64, r);
        tmem_ld_half8(tb + cRAW + addr64, r1);
        tmem_ld_wait();
#pragma unroll
        for (int x = 0; x < 8; ++x) rawg[x] = jb + x < i ? gam8[x] * __uint_as_float(r1[x]) : 0.f;
        *reinterpret_cast<uint4*>(sm + R_IMG + sw128_chunk(i, jb >> 3)) = make_uint4(
            pack_bf16(__uint_as_float(r[0]), __uint_as_float(r[1])), pack_bf16(__uint_as_float(r[2]), __uint_as_float(r[3])),
            pack_bf16(__uint_as_float(r[4]), __uint_as_float(r[5])), pack_bf16(__uint_as_float(r[6]), __uint_as_float(r[7])));
    }
    fence_proxy_async();
    tc_fence_before();
    named_sync(1, CBW_THREADS);

    if (tid == CBW_STORE_TID && ok && full) {   // the dq tile is staged (fenced before the barrier above)
        tma_store_2d(&tmDQ, h * KD, tok0, sm + ST_DQ);
        bulk_commit();
    }
    // ---- phase D: Z[a][b] = sum_c Y[a][c] T[b][c] ; dA = -strictLower(Z) --------------------------
    if (tid == 0 && ok) {
        tc_fence_after();
        const uint64_t da0 = desc_kmajor(sm + R_IMG), db0 = desc_kmajor(sm + R_T);
        for (int k = 0; k < 4; ++k)
            mma_ss(tb + cZ, desc_advance(da0, 32 * k), desc_advance(db0, 32 * k), make_idesc(64, 64), k > 0);
        mma_commit(&bar_mma[3]);
    }
    ok = ok && mbar_wait(&bar_mma[3], ph, a.status, ERR_MMA2);
    tc_fence_after();
    {
        const int i = row64;
        const float bi = sBeta[i];
        float db = 0.f;
        uint32_t r[8];
        tmem_ld_half8(tb + cZ + addr64, r);
        tmem_ld_wait();
        float m2[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            const float da = jb + x < i ? -__uint_as_float(r[x]) : 0.f;
            db = fmaf(da, rawg[x], db);
            m2[x] = da * bi * gam8[x];
        }
        *reinterpret_cast<uint4*>(sm + R_IMG + sw128_chunk(i, jb >> 3)) =
            make_uint4(pack_bf16(m2[0], m2[1]), pack_bf16(m2[2], m2[3]), pack_bf16(m2[4], m2[5]), pack_bf16(m2[6], m2[7]));
        db += __shfl_xor_sync(0xffffffffu, db, 16);   // the two halves of a row's sixteen columns
        if (lane < 16) atomicAdd(&sdB[i], db);
    }
    fence_proxy_async();
    tc_fence_before();
    named_sync(1, CBW_THREADS);

    // ---- phase E: dktil^T += K^T M2 ; dkr^T = Ktil^T M2^T -----------------------------------------
    if (lane == 0 && warp < 2 && ok) {
        tc_fence_after();
        const uint64_t da0 = desc_mnmajor(sm + R_K, BOX), da1 = desc_mnmajor(sm + R_KT, BOX);
        const uint64_t dbm = desc_mnmajor(sm + R_IMG, 0), dbk = desc_kmajor(sm + R_IMG);
        if (warp == 0)
            for (int k = 0; k < 4; ++k)
                mma_ss(tb + cDKT, desc_advance(da0, 2048 * k), desc_advance(dbm, 2048 * k),
                       make_idesc(128, 64, IDESC_A_MN | IDESC_B_MN), 1);
        else
            for (int k = 0; k < 4; ++k)
                mma_ss(tb + cDKR, desc_advance(da1, 2048 * k), desc_advance(dbk, 32 * k),
                       make_idesc(128, 64, IDESC_A_MN), k > 0);
        mma_commit(&bar_mma[4]);
        if (early && warp == 0) load_t(tile_next);   // phase D has finished: T is dead
    }
    // dv = beta dVb (complete since phase B) while the tensor core works on phase E; staged over Q (every
    // read of q ended before the barrier that followed phase C)
    {
        __nv_bfloat16* stv = reinterpret_cast<__nv_bfloat16*>(sm + ST_DV);
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
            const int j0 = colq * 16 + cb * 4;
            uint32_t rvb[4];
            tmem_ld4(tb + cDVB + lane_addr + j0, rvb);
            const float4 b4 = *reinterpret_cast<const float4*>(&sBeta[j0]);
            const float bj[4] = {b4.x, b4.y, b4.z, b4.w};
            tmem_ld_wait();
#pragma unroll
            for (int x = 0; x < 4; ++x) stv[(j0 + x) * KD + f] = __float2bfloat16_rn(bj[x] * __uint_as_float(rvb[x]));
        }
    }
    ok = ok && mbar_wait(&bar_mma[4], ph, a.status, ERR_MMA2);
    tc_fence_after();

    // ---- final epilogue (lane = feature f, columns = tokens): dk --------------------------------------
    rsum = 0.f;
    if (ok) {
        // Results are staged in shared memory as [token][feature] tiles (the operand tiles of the
        // finished products are dead by now) and written out with 16-byte stores afterwards.
        __nv_bfloat16* stk = reinterpret_cast<__nv_bfloat16*>(sm + ST_DK);
        float* stkr = reinterpret_cast<float*>(sm + ST_DKR);
        float* stkt = reinterpret_cast<float*>(sm + ST_DKT);
        // four token columns at a time: few enough live registers for the whole loop to stay in them
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
            const int j0 = colq * 16 + cb * 4;
            uint32_t rkt[4], rdk[4], rkb[4], rkr[4];
            tmem_ld4(tb + cDKTR + lane_addr + j0, rkt);
            tmem_ld4(tb + cDKT + lane_addr + j0, rdk);
            tmem_ld4(tb + cDKB + lane_addr + j0, rkb);
            tmem_ld4(tb + cDKR + lane_addr + j0, rkr);
            float kv[4], ktv[4];
            const float4 b4 = *reinterpret_cast<const float4*>(&sBeta[j0]);
            const float4 g4 = *reinterpret_cast<const float4*>(&sGam[j0]);
            const float4 r4 = *reinterpret_cast<const float4*>(&sRho[j0]);
            const float bj[4] = {b4.x, b4.y, b4.z, b4.w}, gj[4] = {g4.x, g4.y, g4.z, g4.w};
            const float rj[4] = {r4.x, r4.y, r4.z, r4.w};
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const uint32_t eo = boxf + sw128_elem(j0 + x, fc);
                kv[x] = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sm + R_K + eo));
                ktv[x] = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sm + R_KT + eo));
            }
            tmem_ld_wait();
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int j = j0 + x;
                const float dktr = rj[x] * __uint_as_float(rkt[x]);
                const float dkt = dktr + __uint_as_float(rdk[x]);
                const float dkb = __uint_as_float(rkb[x]);
                const float dkr = bj[x] * gj[x] * dkb + __uint_as_float(rkr[x]);
                gv[cb * 4 + x] += dkr * kv[x] - dkt * ktv[x];
                rsum = fmaf(dktr, ktv[x], rsum);
                stk[j * KD + f] = __float2bfloat16_rn(dkr + a.d_min * dkt);
                if (!dk_tile) {   // fp32 copies feed the preconditioner's reverse pass only
                    stkr[j * KD + f] = dkr;
                    stkt[j * KD + f] = dkt;
                } else if (j == 0) {
                    sFirstKt[f] = dkt;   // a reverse pass may restart at the first token
                }
            }
        }
    }
    fence_proxy_async();
    tc_fence_before();
    ok = named_sync_and(1, CBW_THREADS, ok);   // block-uniform from here on; staging complete, q, k, ktil dead, accumulators read
    if (tid == CBW_STORE_TID && early) {   // the next tile's k, ktil (q, v follow once the dv, dq tiles have left their space)
        mbar_expect_tx(&bar_tok, TOK_TX);
        load_kkt(h_next, tok0_next);
    }
    if (tid == CBW_STORE_TID && ok && full) {   // the tiles leave while the per-token sums below are formed
        tma_store_2d(&tmDV, h * KD, tok0, sm + ST_DV);
        if (dk_tile) tma_store_2d(&tmDK, h * KD, tok0, sm + ST_DK);
        bulk_commit();
    }
    if (a_early) {
        // phase A of the next tile: everything it reads was requested before this tile's phase C ended
        bool okn = true;
        if (warp < 4 && ok) okn = mbar_wait(&bar_ct, ph ^ 1u, a.status, ERR_TMA);
        issue_phase_a(ok && okn);
    }
    if (ok) {
        if (!full) {
            for (int e = tid; e < len * 16; e += CBW_THREADS) {
                const int j = e >> 4, ch = e & 15;
                const size_t g = ((size_t)(tok0 + j) * H + h) * KD + ch * 8;
                *reinterpret_cast<uint4*>(a.dq + g) = *reinterpret_cast<const uint4*>(sm + ST_DQ + j * 256 + ch * 16);
                *reinterpret_cast<uint4*>(a.dv + g) = *reinterpret_cast<const uint4*>(sm + ST_DV + j * 256 + ch * 16);
            }
        }
        if (!dk_tile) {
            for (int e = tid; e < len * 16; e += CBW_THREADS) {
                const int j = e >> 4, ch = e & 15;
                const size_t g = ((size_t)(tok0 + j) * H + h) * KD + ch * 8;
                if ((sk >> j) & 1ull)
                    *reinterpret_cast<uint4*>(a.dk + g) =
                        *reinterpret_cast<const uint4*>(sm + ST_DK + j * 256 + ch * 16);
            }
        }
        if (dk_tile) {
            // only the first token's dL/dktil is needed (a reverse pass may restart there)
            for (int e = tid; e < 32; e += CBW_THREADS) {
                const size_t g = ((size_t)tok0 * H + h) * KD + e * 4;
                *reinterpret_cast<uint4*>(a.dktil + g) = *reinterpret_cast<const uint4*>(&sFirstKt[e * 4]);
            }
        } else {
            for (int e = tid; e < len * 32; e += CBW_THREADS) {
                const int j = e >> 5, ch = e & 31;
                const size_t g = ((size_t)(tok0 + j) * H + h) * KD + ch * 4;
                const bool skipped = (sk >> j) & 1ull;
                if (!skipped)
                    *reinterpret_cast<uint4*>(a.dkread + g) =
                        *reinterpret_cast<const uint4*>(sm + ST_DKR + j * 512 + ch * 16);
                if (!skipped || j == 0 || !((sk >> (j - 1)) & 1ull))
                    *reinterpret_cast<uint4*>(a.dktil + g) =
                        *reinterpret_cast<const uint4*>(sm + ST_DKT + j * 512 + ch * 16);
            }
        }
        if (full && tid == CBW_STORE_TID) {
            bulk_wait_read();   // the staging tiles may be overwritten by the next tile
            if (early) load_qv(h_next, tok0_next);
        }
    }
    if (tile_next == -1 && tid == CBW_QUEUE_TID) lookup_blocking(ticket_next);   // not published when this tile began: wait for it now
    named_sync(1, CBW_THREADS);   // every copy-out read of the staging tiles is done
    if (!next_known) {
        tile_next = sNext[0]; h_next = sNext[1]; tok0_next = sNext[2]; len_next = sNext[3];
        if (tile_next >= 0) fetch_scalars(tile_next, h_next, tok0_next, len_next, (int)(ph ^ 1u));
    }
    if (tid == 0 && tile_next >= 0) {
        if (!early) {
            mbar_expect_tx(&bar_ct, CT_TX);
            load_dout(h_next, tok0_next);
            load_du_ds_s(tile_next);
            load_ddu(tile_next);
            load_t(tile_next);
            mbar_expect_tx(&bar_tok, TOK_TX);
            load_kkt(h_next, tok0_next);
            load_qv(h_next, tok0_next);
        }
    }
    a_issued = a_early && ok;
    pend = ok;
    p_tok0 = tok0;
    p_h = h;
    p_len = len;
    ph ^= 1u;
    ticket_next = ticket_after;
    tile_l = tile_next;
    h = h_next;
    tok0 = tok0_next;
    len = len_next;
    }   // tile loop
    if (pend) {   // the last tile's sums
        reduce_sums((int)(ph ^ 1u));
        named_sync(1, CBW_THREADS);
        if (warp == 1) finish_sums((int)(ph ^ 1u), p_tok0, p_h, p_len);
    }
    if (tid == CBW_STORE_TID) bulk_wait_all();
    tc_fence_before();
    named_sync(1, CBW_THREADS);
}

// Backward of the layer's second phase in one launch.  CTA b first walks the chains b, b + grid, ...
// (reverse state recurrence), each of which publishes its finished tiles; then every CTA processes
// chunk-local tiles from the queue until none is left.  CTAs beyond the number of chains start on the
// queue at once, so the SMs the chains leave idle work on the tiles the chains have already finished.
// Nothing in a chain waits for a consumer, and a consumer waits (within a bound) only for tiles whose
// chain is running or has run: lower block indices are dispatched first.
__global__ void __launch_bounds__(CBK_THREADS, 1)
tc_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
              const __grid_constant__ CUtensorMap tmKt, const __grid_constant__ CUtensorMap tmV,
              const __grid_constant__ CUtensorMap tmDO, const __grid_constant__ CUtensorMap tmDQ,
              const __grid_constant__ CUtensorMap tmDK, const __grid_constant__ CUtensorMap tmDV,
              TcChainBwdArgs ca, TcChunkBwdArgs cb, TileQueue tq, int nchains)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* sm = align1024(smem_raw);
    __shared__ uint32_t tmem_base;
    const int warp = threadIdx.x >> 5;
    if (warp == 0) tmem_alloc(&tmem_base, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_base;
    for (int chain = (int)blockIdx.x; chain < nchains; chain += (int)gridDim.x)
        chain_bwd_role(tmDO, tmKt, ca, chain, sm, tb, tq);
    if (threadIdx.x < CBW_THREADS) chunk_bwd_role(tmQ, tmK, tmKt, tmV, tmDO, tmDQ, tmDK, tmDV, cb, sm, tb, tq);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tb, 512);
}

// Exercises the bounded wait by itself: one warp waits on a barrier that nothing ever arrives on.  The
// wait gives up after `limit_cycles`, records `code` in the status word and the kernel returns.
__global__ void wait_timeout_selftest_kernel(int* status, long long limit_cycles, int code)
{
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    mbar_wait(&bar, 0, status, code, limit_cycles);
}

int num_sms()
{
    static int n = 0;
    if (!n) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

template <typename F> bool set_smem(F* kernel, size_t bytes)
{
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) == cudaSuccess;
}

}  // namespace

// Merged forward launch: SMs that must be left over to feed the chains, and the cost of one chain step in
// units of the time one SM needs for a tile of the chunk-local pass (measured: 0.6 to 0.75 are equally good).
constexpr int FWD_MIN_FEEDERS = 32;
constexpr double FWD_STEP_OVER_TILE = FWD_STEP_OVER_TILE_F;

int launch_wait_timeout_selftest(int* status, long long limit_cycles, int code, cudaStream_t st)
{
    wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(status, limit_cycles, code);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

bool tc_supported(const osdn_params& p)
{
    return p.io_dtype == OSDN_BF16 && p.K == KD && p.V == KD && get_encoder() != nullptr;
}

int tc_forward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a, bool save,
               cudaStream_t st)
{
    char* w = static_cast<char*>(ws);
    const TcLayout t = make_tc_layout(p, L, save);
    if (t.total > L.total) return -1;
    Table tab = carve_table(ws, L);
    const int S = L.S, H = p.H;
    const size_t Ttot = p.nseq > 0 ? (size_t)p.T : (size_t)p.B * p.T;
    int* status = reinterpret_cast<int*>(w + L.status);
    int launches = 0;

    // phase 1 on CUDA cores: bf16 write keys, chunk-start preconditioners
    const int n1 = phase1_forward(p, hy, L, ws, a, w + t.ktil, true, save, st);
    if (n1 < 0) return -1;
    launches += n1;

    CUtensorMap tmK, tmQ, tmKt, tmV;
    if (!make_token_map(&tmK, a.k, Ttot, H) || !make_token_map(&tmQ, a.q, Ttot, H) ||
        !make_token_map(&tmKt, w + t.ktil, Ttot, H) || !make_token_map(&tmV, a.v, Ttot, H))
        return -1;
    TcChunkArgs ca{};
    ca.H = H; ca.tab = tab; ca.beta = a.beta; ca.gate = a.gate; ca.scale = hy.scale;
    ca.WT = reinterpret_cast<uint8_t*>(w + t.WT); ca.Tb = reinterpret_cast<uint8_t*>(w + t.Tb);
    ca.Tm = reinterpret_cast<uint8_t*>(w + t.Tm); ca.P = reinterpret_cast<uint8_t*>(w + t.P);
    ca.Qg = reinterpret_cast<uint8_t*>(w + t.Qg); ca.save = save ? 1 : 0; ca.status = status;
    TcChainArgs ch{};
    ch.H = H; ch.tab = tab; ch.gate = a.gate; ch.init_state = a.init_state;
    ch.out = static_cast<__nv_bfloat16*>(a.out); ch.final_state = a.final_state;
    ch.WT = reinterpret_cast<uint8_t*>(w + t.WT); ch.Tb = reinterpret_cast<uint8_t*>(w + t.Tb);
    ch.P = reinterpret_cast<uint8_t*>(w + t.P); ch.Sn = reinterpret_cast<uint8_t*>(w + t.Sn);
    ch.dUT = reinterpret_cast<uint8_t*>(w + t.dUT); ch.scale = hy.scale; ch.save = save ? 1 : 0;
    ch.status = status;
    // One launch for both passes when the batch is dense (equal chunk counts give the tile order the
    // chains want) and enough SMs are left over to feed the chains.
    const int grid = num_sms(), nchains = S * H;
    const int nchunks = p.nseq > 0 ? 0 : (p.T + CH - 1) / CH;
    if (nchains + FWD_MIN_FEEDERS <= grid) {
        const size_t rbytes = sizeof(int) * (64 + (size_t)L.NTmax * H);
        if (cudaMemsetAsync(w + t.ready, 0, rbytes, st) != cudaSuccess) return -1;
        FwdSched sc{};
        sc.tickets = reinterpret_cast<int*>(w + t.ready);
        sc.nchains = nchains;
        sc.nchunks = nchunks;
        sc.ntickets = nchunks * nchains;
        sc.nseq = S;
        sc.feeders = grid - nchains;
        // The chains start once the feeders alone can keep up with them to the end: a chain step costs
        // about FWD_STEP_OVER_TILE of the time one SM needs for a tile.
        const double fed = (double)(grid - nchains) * nchunks * FWD_STEP_OVER_TILE;
        sc.switch_at = (int)std::max(0.0, (double)sc.ntickets - fed);
        if (p.nseq > 0) {   // both are worked out on the device from the chunk table
            sc.order = tab.order_;
            sc.longest = tab.pos_;
        }
        ca.ready = sc.tickets + 64;
        ch.ready = sc.tickets + 64;
        // Three worker groups when the longest chain outweighs the tiles (packed batches: their longest
        // sequence is not known here, and a long tail is what packing produces), four otherwise.
        const bool chain_bound = p.nseq > 0 || (double)nchunks * 2.3 > 1.5 * (double)sc.ntickets * 5.5 / grid;
        stage_mark(st, "tc_fwd");
        if (chain_bound) {
            if (!set_smem(tc_fwd_kernel<3>, CF_SMEM)) return -1;
            tc_fwd_kernel<3><<<grid, 3 * CL_THREADS, CF_SMEM, st>>>(tmK, tmQ, tmKt, tmV, ca, ch, sc);
        } else {
            if (!set_smem(tc_fwd_kernel<4>, CF_SMEM)) return -1;
            tc_fwd_kernel<4><<<grid, 4 * CL_THREADS, CF_SMEM, st>>>(tmK, tmQ, tmKt, tmV, ca, ch, sc);
        }
        ++launches;
    } else {
        if (!set_smem(tc_chunk_fwd_kernel, CL_SMEM)) return -1;
        stage_mark(st, "tc_chunk_fwd");
        tc_chunk_fwd_kernel<<<dim3(L.NTmax, H), CL_THREADS, CL_SMEM, st>>>(tmK, tmQ, tmKt, ca);
        ++launches;
        if (!set_smem(tc_chain_fwd_kernel, CF_SMEM)) return -1;
        stage_mark(st, "tc_chain_fwd");
        tc_chain_fwd_kernel<<<S * H, CFW_THREADS, CF_SMEM, st>>>(tmV, tmKt, ch);
        ++launches;
    }
    stage_end(st);
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

bool tc_backward_supported(const osdn_params& p) { return tc_supported(p); }

int tc_backward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                cudaStream_t st)
{
    char* w = static_cast<char*>(ws);
    const TcLayout t = make_tc_layout(p, L, true);
    if (t.total > L.total) return -1;
    Table tab = carve_table(ws, L);
    const int S = L.S, H = p.H;
    const size_t Ttot = p.nseq > 0 ? (size_t)p.T : (size_t)p.B * p.T;
    int* status = reinterpret_cast<int*>(w + L.status);
    int launches = 0;
    auto U8 = [&](size_t off) { return reinterpret_cast<uint8_t*>(w + off); };
    CUtensorMap tmK, tmQ, tmKt, tmV, tmDO;
    if (!make_token_map(&tmK, a.k, Ttot, H) || !make_token_map(&tmQ, a.q, Ttot, H) ||
        !make_token_map(&tmKt, w + t.ktil, Ttot, H) || !make_token_map(&tmV, a.v, Ttot, H) ||
        !make_token_map(&tmDO, a.dout, Ttot, H))
        return -1;
    {
        TcChainBwdArgs ch{};
        ch.H = H; ch.tab = tab; ch.gate = a.gate; ch.dfinal_state = a.dfinal_state; ch.dinit_state = a.dinit_state;
        ch.WT = U8(t.WT); ch.P = U8(t.P); ch.Qg = U8(t.Qg); ch.dSn = U8(t.dSn); ch.ddUT = U8(t.ddUT);
        ch.status = status;
        TcChunkBwdArgs cb{};
        cb.H = H; cb.ntiles = L.NTmax * H; cb.nseq = S; cb.tab = tab; cb.beta = a.beta; cb.gate = a.gate; cb.scale = hy.scale; cb.d_min = hy.d_min;
        cb.Tm = U8(t.Tm); cb.Sn = U8(t.Sn); cb.dSn = U8(t.dSn); cb.dUT = U8(t.dUT); cb.ddUT = U8(t.ddUT);
        cb.skipw = carve_p1(ws, L).skipw;
        cb.dq = static_cast<__nv_bfloat16*>(a.dq); cb.dk = static_cast<__nv_bfloat16*>(a.dk);
        cb.dv = static_cast<__nv_bfloat16*>(a.dv); cb.dbeta = a.dbeta; cb.dgate = a.dgate;
        cb.dktil = reinterpret_cast<float*>(w + t.dktil); cb.dkread = reinterpret_cast<float*>(w + t.dkread);
        cb.status = status;
        CUtensorMap tmDQ, tmDK, tmDV;
        if (!make_store_map(&tmDQ, a.dq, Ttot, H) || !make_store_map(&tmDK, a.dk, Ttot, H) ||
            !make_store_map(&tmDV, a.dv, Ttot, H))
            return -1;
        // tile queue between the chains and the chunk-local workers: two counters, then one slot per tile
        const size_t qbytes = sizeof(int) * (64 + (size_t)L.NTmax * H);
        if (cudaMemsetAsync(w + t.queue, 0, qbytes, st) != cudaSuccess) return -1;
        TileQueue tq{};
        tq.head = reinterpret_cast<unsigned*>(w + t.queue);
        tq.tail = tq.head + 32;
        tq.slots = reinterpret_cast<int*>(w + t.queue) + 64;
        const size_t smem = std::max(CB_SMEM, CBW_SMEM);
        if (!set_smem(tc_bwd_kernel, smem)) return -1;
        stage_mark(st, "tc_bwd");
        tc_bwd_kernel<<<num_sms(), CBK_THREADS, smem, st>>>(tmQ, tmK, tmKt, tmV, tmDO, tmDQ, tmDK, tmDV, ch, cb, tq, S * H);
        ++launches;
    }
    const int n1 = phase1_backward(p, hy, L, ws, a, reinterpret_cast<float*>(w + t.dktil),
                                   reinterpret_cast<float*>(w + t.dkread), false, st);
    if (n1 < 0) return -1;
    launches += n1;
    stage_end(st);
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace osdn

