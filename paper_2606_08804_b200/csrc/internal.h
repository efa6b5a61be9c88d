// Internal declarations shared by the translation units of libqdelta.so.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/qdelta.h"

namespace qd {

constexpr int kChunk = 64;        // chunk length C of the chunkwise form
constexpr int kSliceSimt = 32;    // d_v columns one CTA of the SIMT state chains owns

// Byte offsets of the sections of the caller-provided workspace.  Every section starts on a
// 256-byte boundary.  "io" sections are stored in the call's dtype.
struct WsLayout {
    size_t status;   // u32 status word (+ padding)
    size_t g;        // fp32 [BH*T]        in-chunk cumulative log-decay g_r = sum_{i<=r} log alpha_i
    size_t P;        // io   [BH*T*C]      Gamma o (Q K^T), causal incl. diagonal, row = token
    size_t W;        // io   [BH*T*dk]     W<- = T diag(gamma) X
    size_t U;        // io   [BH*T*dv]     U~  = T V
    size_t fwd_end;
    // backward only
    size_t hs;       // fp32 [BH*N*dk*dv]  state at the entry of every chunk
    size_t D;        // io   [BH*T*dv]     Delta = U~ - W<- h   (row r = delta_r of the recurrence)
    size_t dhs;      // fp32 [BH*N*dk*dv]  gradient w.r.t. the state at the EXIT of every chunk
    size_t dD;       // io   [BH*T*dv]     gradient w.r.t. Delta
    size_t kdhd;     // fp32 [S][BH*T]     per d_v-slice partial of <(K-> dh)_r, Delta_r>
    size_t dhh;      // fp32 [S][BH*N]     per d_v-slice partial of <dh, h>_F
    size_t scratch;  // fp32 per-CTA scratch of the SIMT chunk backward
    size_t rqk;      // fp32 [2][BH*T]     QD_NORM_QK: 1/|q_t|, then 1/|k_t|
    size_t bwd_end;
    int nslices;
    int bwd_ctas;
};

WsLayout ws_layout(const qd_shape& s);
// QD_OK, or the error code every entry point reports for this shape (host-side validation only).
int check_shape(const qd_shape* s);

// Workspace of the tensor-core path (bf16, d_k = d_v = 128).  Sections start on 1024-byte boundaries.
struct TcLayout {
    size_t status;   // u32 status word
    size_t g;        // fp32 [BH*T]
    size_t Qg;       // bf16 [BH*T][dk]        diag(gamma) Q
    size_t P;        // bf16 [BH*T][C]         Gamma o (Q K^T), causal incl. diagonal
    size_t Wt;       // bf16 [BH*N][dk][C]     (T diag(gamma) X)^T per chunk
    size_t Ut;       // bf16 [BH*N][dv][C]     (T V)^T per chunk
    size_t rqk;      // fp32 [2][BH*T]         QD_NORM_QK: 1/|q_t|, then 1/|k_t|
    size_t fwd_end;
    // kept for / produced by the backward
    size_t Mt;       // bf16 [BH*N][C][C]      ((I+A)^-1)^T per chunk: [column][row]
    size_t hsT;      // bf16 [BH*N][dv][dk]    h^T at the entry of every chunk
    size_t Dt;       // bf16 [BH*N][dv][C]     Delta^T per chunk
    size_t dhsT;     // bf16 [BH*N][dv][dk]    (dL/dh)^T at the exit of every chunk
    size_t dDt;      // bf16 [BH*N][dv][C]     (dL/dDelta)^T per chunk
    size_t bwd_end;
};
TcLayout tc_layout(const qd_shape& s);
bool tc_supported(const qd_shape& s);
// Rows per sequence in the tensor-core workspace: T rounded up to a whole number of chunk PAIRS (the preparation kernel
// takes two chunks at a time).  The rows past T behave as tokens with beta = 0, alpha = 1, q = k = v = 0, which leave the
// recurrence of Section 3.3.1 untouched; TMA supplies the zeros and drops the stores.
inline int simt_padded_T(const qd_shape& s) { return (s.T + kChunk - 1) / kChunk * kChunk; }   // fp32 path: whole chunks
inline int tc_padded_T(const qd_shape& s) { return (s.T + 2 * kChunk - 1) / (2 * kChunk) * (2 * kChunk); }

// cudaFuncAttributeMaxDynamicSharedMemorySize for `kernel`: set when first needed on a device, and again only if a
// later call needs more.
cudaError_t set_max_smem_once(const void* kernel, size_t bytes);

// Launch with the programmatic-stream-serialization attribute: the kernel may begin before the previous kernel of the
// stream has finished and orders itself with grid_dep_wait() (see sm100.cuh).
template <class... KArgs, class... Args>
cudaError_t launch_overlapped(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

struct ChunkArgs {
    qd_shape s;
    const void *q, *k, *v, *beta, *alpha, *lam;
    const float* h0;
    void* o;
    float* hT;
    // backward
    const void* dO;
    const float* dhT;
    void *dq, *dk, *dv;
    float *dbeta, *dalpha, *dlam, *dh0;
    char* ws;
    WsLayout L;
    TcLayout TL;
    bool save;       // forward: keep hs and D
    bool logits;     // beta, alpha, lambda hold pre-activation logits: the kernels apply the sigmoid (QD_COEF_LOGITS)
    bool norm;       // q and k are L2-normalised per token and head inside the kernels (QD_NORM_QK)
    bool own_predecessor;   // backward: the kernel enqueued before the reverse chain is this library's forward chain
    cudaStream_t stream;
};

// SIMT fp32-arithmetic path (any supported dtype for storage)
cudaError_t simt_prep(const ChunkArgs& a);        // g, P, W<-, U~
cudaError_t simt_chain_fwd(const ChunkArgs& a);   // Delta, O, state chain (+ hs, D when a.save)
cudaError_t simt_chain_bwd(const ChunkArgs& a);   // dDelta, dhs, dh0, scalar partials
cudaError_t simt_chunk_bwd(const ChunkArgs& a);   // dq, dk, dv, dbeta, dalpha, dlambda

// tcgen05 path
cudaError_t tc_prep(const ChunkArgs& a);
cudaError_t tc_chain_fwd(const ChunkArgs& a);
cudaError_t tc_chain_bwd(const ChunkArgs& a);
cudaError_t tc_chunk_bwd(const ChunkArgs& a);

cudaError_t decode_step(int BH, int dk, int dv, int dtype, const void* q, const void* k, const void* v,
                        const void* beta, const void* alpha, const void* lam, float* state, void* o,
                        cudaStream_t stream);

cudaError_t decode_steps(int B, int S, int H, int dk, int dv, int dtype, const void* q, const void* k, const void* v,
                         const void* beta, const void* alpha, const void* lam, void* state, void* o,
                         bool logits, bool norm, bool state_bf16, cudaStream_t stream);

// ---- in-kernel L2 normalisation of q and k (QD_NORM_QK) ------------------------------------------------
// x^ = x / sqrt(sum x^2 + kNormEps), per token and head.  Its backward: dx = r (dx^ - x^ <x^, dx^>), r = 1/sqrt(sum x^2 + eps).
constexpr float kNormEps = 1e-6f;

// ---- gates given as logits (QD_COEF_LOGITS) ---------------------------------------------------------
// The coefficients of the rule are sigmoid gates (Appendix B gives lambda = sigmoid(W h + b); beta and alpha
// likewise lie in (0,1)).  With the flag the kernels take the pre-activation z and form the gate themselves, in fp32.
__device__ __forceinline__ float gate(float z, bool logits) { return logits ? 1.f / (1.f + expf(-z)) : z; }
// log of the forget gate: log(alpha), or log sigmoid(z) = min(z,0) - log1p(exp(-|z|)) without forming 1 - tiny
__device__ __forceinline__ float log_gate(float z, bool logits) {
    return logits ? fminf(z, 0.f) - log1pf(expf(-fabsf(z))) : logf(z);
}

// ---- storage-dtype helpers -------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float ld(const T* p, size_t i);
template <> __device__ __forceinline__ float ld<float>(const float* p, size_t i) { return p[i]; }
template <> __device__ __forceinline__ float ld<__nv_bfloat16>(const __nv_bfloat16* p, size_t i) {
    return __bfloat162float(p[i]);
}
template <typename T> __device__ __forceinline__ void st(T* p, size_t i, float x);
template <> __device__ __forceinline__ void st<float>(float* p, size_t i, float x) { p[i] = x; }
template <> __device__ __forceinline__ void st<__nv_bfloat16>(__nv_bfloat16* p, size_t i, float x) {
    p[i] = __float2bfloat16_rn(x);
}

}  // namespace qd
