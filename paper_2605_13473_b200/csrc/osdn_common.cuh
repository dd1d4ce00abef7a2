// Shared declarations of the OSDN CUDA library: workspace layout, chunk table, launch
// arguments.  Device-side helpers for the two kernel families (CUDA-core fp32 kernels and
// tcgen05 bf16 kernels) live in their own files.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/osdn.h"

namespace osdn {

constexpr int CH = 64;  // chunk length (tokens)

// Scalar settings broadcast to every kernel.
struct Hyper {
    float eta, d_min, d_max, eps, scale;
    int beta_aware, apf_mode, clamp;
};

// Sequence / chunk table built on the device from cu_seqlens (or from B, T for dense input).
// Chunks never straddle sequences; chunk_len < 64 marks a ragged tail; entries beyond the
// realised chunk count have chunk_len == 0.
// Chunk table.  For a dense batch (every sequence T tokens long) the entries are pure arithmetic and
// nothing is read; for a packed batch they were written by build_table_kernel from cu_seqlens.
struct Table {
    int* seq_tok0_;    // [S]    first packed token of the sequence
    int* seq_len_;     // [S]
    int* seq_chunk0_;  // [S+1]  first chunk of the sequence; [S] = number of chunks
    int* chunk_tok0_;  // [NTmax]
    int* chunk_len_;   // [NTmax]
    int* chunk_seq_;   // [NTmax]
    int* order_;       // [NTmax]  packed batches: the chunks sorted by the step at which their chain needs them
                       //          when all chains are to end together (see build_table_kernel)
    int* pos_;         // [2 NTmax + 4] scratch of the sort; pos_[0] = chunks of the longest sequence
    int* seq_first_;   // [S]      rank of the sequence's first chunk in order_
    int dense_T;       // > 0: dense batch with sequences of this length
    int dense_nc;      //      and this many chunks per sequence
    __device__ __forceinline__ int seq_tok0(int s) const { return dense_T ? s * dense_T : seq_tok0_[s]; }
    __device__ __forceinline__ int seq_len(int s) const { return dense_T ? dense_T : seq_len_[s]; }
    __device__ __forceinline__ int seq_chunk0(int s) const { return dense_T ? s * dense_nc : seq_chunk0_[s]; }
    __device__ __forceinline__ int chunk_tok0(int c) const
    {
        return dense_T ? (c / dense_nc) * dense_T + (c % dense_nc) * CH : chunk_tok0_[c];
    }
    __device__ __forceinline__ int chunk_len(int c) const
    {
        if (!dense_T) return chunk_len_[c];
        const int rem = dense_T - (c % dense_nc) * CH;
        return rem < CH ? rem : CH;
    }
    __device__ __forceinline__ int chunk_seq(int c) const { return dense_T ? c / dense_nc : chunk_seq_[c]; }
};

// Byte offsets of every region inside the caller's workspace.
struct WsLayout {
    size_t status;      // int32 device status word (+ padding)
    size_t table;       // ints, see carve_table
    // phase 1 (shared by both kernel families)
    size_t p1n;         // [T,H]          f32   1 / max(|k|^2, eps), negated where the floor is active
    size_t p1rho;       // [T,H]          f32   retention of the preconditioner
    size_t p1al;        // [T,H]          f32   <d_t, k_t^2> of processed tokens                (save only)
    size_t p1flags;     // [NT,H,2]       u32   per token: the step maps d_min*1 to d_min*1, mask all zero
    size_t p1skip;      // [NT,H,2]       u32   tokens the sequential pass skipped           (save only)
    size_t pmask;       // [T,H,32]       u32   projection pass masks of processed tokens: word of lane l,
                        //                      bit r = coordinate (K/32) l + r passes gradient    (save only)
    size_t dtraj;       // [T,H,K]        f32   d_t of processed tokens                      (save only)
    size_t ktil;        // [T,H,K]        f32   write keys
    size_t Tm;          // [NT,H,64,64]   f32   UT inverse
    size_t P;           // [NT,H,64,64]   f32   masked, decayed q.ktil scores
    size_t W;           // [NT,H,64,K]    f32
    size_t U;           // [NT,H,64,V]    f32
    size_t dU;          // [NT,H,64,V]    f32   chunk update (new values)
    size_t Sn;          // [NT,H,V,K]     f32   state at chunk start
    // backward only
    size_t ddU;         // [NT,H,64,V]    f32
    size_t dSn;         // [NT,H,V,K]     f32   state cotangent at chunk end
    size_t dktil;       // [T,H,K]        f32
    size_t dkread;      // [T,H,K]        f32
    size_t scr;         // [NT,H,5,64,max(K,V)] f32 scratch of the chunk-local backward
    size_t out_scratch; // [T,H,V]        f32   forward output when the backward recomputes the forward
    size_t total;
    int S, NTmax;
    int dense_T;        // > 0 for a dense batch (see Table)
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline WsLayout make_layout(const osdn_params& p, bool need_bwd)
{
    WsLayout L{};
    const int S = p.nseq > 0 ? p.nseq : p.B;
    const size_t Ttot = (size_t)(p.nseq > 0 ? p.T : (size_t)p.B * p.T);
    const int NTmax = p.nseq > 0 ? (int)(Ttot / CH) + S : p.B * ((p.T + CH - 1) / CH);
    L.S = S;
    L.NTmax = NTmax;
    L.dense_T = p.nseq > 0 ? 0 : p.T;
    const size_t H = p.H, K = p.K, V = p.V, NT = NTmax;
    const size_t D = K > V ? K : V;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    L.status = take(256);
    L.table = take(sizeof(int) * (4 * (size_t)S + 1 + 6 * NT + 4));
    L.p1n = take(4 * Ttot * H);
    L.p1rho = take(4 * Ttot * H);
    L.p1flags = take(4 * NT * H * 2);
    if (need_bwd) {
        L.p1skip = take(4 * NT * H * 2);
        L.p1al = take(4 * Ttot * H);
        L.pmask = take(4 * Ttot * H * 32);
        L.dtraj = take(4 * Ttot * H * K);
    }
    L.ktil = take(4 * Ttot * H * K);
    L.Tm = take(4 * NT * H * CH * CH);
    L.P = take(4 * NT * H * CH * CH);
    L.W = take(4 * NT * H * CH * K);
    L.U = take(4 * NT * H * CH * V);
    L.dU = take(4 * NT * H * CH * V);
    L.Sn = take(4 * NT * H * V * K);
    if (need_bwd) {
        L.ddU = take(4 * NT * H * CH * V);
        L.dSn = take(4 * NT * H * V * K);
        L.dktil = take(4 * Ttot * H * K);
        L.dkread = take(4 * Ttot * H * K);
        L.scr = take(4 * NT * H * 5 * CH * D);
        L.out_scratch = take(4 * Ttot * H * V);
    }
    L.total = off;
    return L;
}

inline Table carve_table(void* ws, const WsLayout& L)
{
    int* base = reinterpret_cast<int*>(static_cast<char*>(ws) + L.table);
    Table t;
    t.seq_tok0_ = base;
    t.seq_len_ = base + L.S;
    t.seq_chunk0_ = base + 2 * L.S;
    t.chunk_tok0_ = base + 3 * L.S + 1;
    t.chunk_len_ = t.chunk_tok0_ + L.NTmax;
    t.chunk_seq_ = t.chunk_len_ + L.NTmax;
    t.order_ = t.chunk_seq_ + L.NTmax;
    t.pos_ = t.order_ + L.NTmax;
    t.seq_first_ = t.pos_ + 2 * L.NTmax + 4;
    t.dense_T = L.dense_T;
    t.dense_nc = L.dense_T ? (L.dense_T + CH - 1) / CH : 0;
    return t;
}

struct P1Regions {
    float *n, *rho, *dtraj, *al;
    unsigned *flags, *skipw, *pmask;
};

inline P1Regions carve_p1(void* ws, const WsLayout& L)
{
    char* w = static_cast<char*>(ws);
    P1Regions r;
    r.n = reinterpret_cast<float*>(w + L.p1n);
    r.rho = reinterpret_cast<float*>(w + L.p1rho);
    r.al = reinterpret_cast<float*>(w + L.p1al);
    r.flags = reinterpret_cast<unsigned*>(w + L.p1flags);
    r.skipw = reinterpret_cast<unsigned*>(w + L.p1skip);
    r.pmask = reinterpret_cast<unsigned*>(w + L.pmask);
    r.dtraj = reinterpret_cast<float*>(w + L.dtraj);
    return r;
}

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p)
{
    return __bfloat162float(*p);
}
template <typename T> __device__ __forceinline__ void stf(T* p, float x);
template <> __device__ __forceinline__ void stf<float>(float* p, float x) { *p = x; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float x)
{
    *p = __float2bfloat16_rn(x);
}

// Everything a forward / backward launch sequence needs.
struct Pointers {
    const void *q, *k, *v;
    const float *beta, *gate, *log_ret, *init_state, *precond_in;
    void* out;
    float *final_state, *precond_out;
    // backward
    const void* dout;
    const float *dfinal_state, *dprecond_out;
    void *dq, *dk, *dv;
    float *dbeta, *dgate, *dlog_ret, *dinit_state, *dprecond_in;
};

// CUDA-core fp32 kernels (osdn_simt.cu).  Return the number of launches, or -1 on a launch error.
int simt_forward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws,
                 const Pointers& a, bool save, cudaStream_t st);
int simt_backward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws,
                  const Pointers& a, cudaStream_t st);
// Phase 1 (osdn_phase1.cu).  ktil: packed [T,H,K] write keys, fp32 or bf16.  `save` records what
// the backward needs.  `bulk`: also finalise dk of skipped tokens (the tensor-core chunk kernel does
// that itself).
int phase1_forward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                   void* ktil, bool ktil_bf16, bool save, cudaStream_t st);
int phase1_backward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                    const float* dktil, const float* dkread, bool bulk, cudaStream_t st);
int phase1_update(const osdn_params& p, const Hyper& hy, const void* k, const float* beta, const float* retsrc,
                  const float* precond_in, void* ktil_out, float* precond_out, float* ratio_out,
                  float* log_sum_out, cudaStream_t st);

// Recurrent step over p.T tokens per sequence on cached state and preconditioner (both updated in
// place); one launch.
int decode_step(const osdn_params& p, const Hyper& hy, const void* q, const void* k, const void* v,
                const float* beta, const float* gate, const float* log_ret, float* state, float* precond,
                void* out, cudaStream_t st);
int launch_build_table(const osdn_params& p, const WsLayout& L, void* ws, cudaStream_t st);
// Channel-gate variant of the layer (osdn_kda.cu): a.gate is [T,H,K].  The backward needs
// kda_extra_bytes of workspace behind the common layout.
size_t kda_extra_bytes(const osdn_params& p, const WsLayout& L, bool need_bwd);
int kda_forward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a, bool save,
                cudaStream_t st);
int kda_backward(const osdn_params& p, const Hyper& hy, const WsLayout& L, void* ws, const Pointers& a,
                 cudaStream_t st);

// Optional per-kernel timing (off by default): when enabled through osdn_stage_timing_enable, every
// launch site records a CUDA event on the launching stream before its kernel; stage_end closes the
// last one.  Durations are read back with osdn_stage_timing_read after a synchronise.
void stage_mark(cudaStream_t st, const char* name);
void stage_end(cudaStream_t st);

}  // namespace osdn
