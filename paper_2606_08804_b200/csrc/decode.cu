// Single-token recurrent step (Section 3.3.1, final update rule and read-out), in place:
//   x = k + lambda q ;  p = alpha h^T x ;  delta = beta (v - p) ;  h <- alpha h + k delta^T ;
//   o = h_new^T q = alpha h^T q + (k.q) delta .
// The step is bound by HBM traffic: the fp32 state is read once and written once.  A CTA owns
// DVS columns of one state (columns evolve independently); every thread keeps its part of the
// slice in registers between the read and the write, all loads are issued before the first use.
#include "internal.h"

namespace qd {
namespace {

template <typename IO, int DK, int DVS, int NT>
__global__ void __launch_bounds__(NT) k_decode(int dv, const IO* __restrict__ q, const IO* __restrict__ k,
                                               const IO* __restrict__ v, const IO* __restrict__ beta,
                                               const IO* __restrict__ alpha, const IO* __restrict__ lam,
                                               float* __restrict__ state, IO* __restrict__ o) {
    constexpr int C4 = DVS / 4;          // threads across one row of the slice
    constexpr int RP = NT / C4;          // rows per pass
    constexpr int NP = DK / RP;          // passes (float4 registers per thread)
    static_assert(NT % C4 == 0 && DK % RP == 0, "bad decode tiling");
    __shared__ float sx[DK], sq[DK], sk[DK];
    __shared__ float redx[RP][DVS], redq[RP][DVS];
    __shared__ float sdelta[DVS];
    __shared__ float skq[NT / 32];
    const int nsl = dv / DVS, bh = blockIdx.x / nsl, j0 = (blockIdx.x % nsl) * DVS, tid = threadIdx.x;
    const int c4 = tid % C4, rg = tid / C4;

    // issue all state loads first
    float4* base = reinterpret_cast<float4*>(state + (size_t)bh * DK * dv + j0) + c4;
    const int rstride = dv / 4;
    float4 h[NP];
#pragma unroll
    for (int pz = 0; pz < NP; ++pz) h[pz] = __ldcs(base + (size_t)(pz * RP + rg) * rstride);

    const float be = ld(beta, bh);
    const float al = alpha ? ld(alpha, bh) : 1.f;
    const float la = lam ? ld(lam, bh) : 0.f;
    float kq = 0.f;
    for (int i = tid; i < DK; i += NT) {
        const float qi = ld(q, (size_t)bh * DK + i), ki = ld(k, (size_t)bh * DK + i);
        sq[i] = qi; sk[i] = ki; sx[i] = fmaf(la, qi, ki);
        kq = fmaf(ki, qi, kq);
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) kq += __shfl_xor_sync(0xffffffffu, kq, s);
    if ((tid & 31) == 0) skq[tid >> 5] = kq;
    __syncthreads();

    float4 ax = make_float4(0.f, 0.f, 0.f, 0.f), aq = ax;
#pragma unroll
    for (int pz = 0; pz < NP; ++pz) {
        const float xi = sx[pz * RP + rg], qi = sq[pz * RP + rg];
        ax.x = fmaf(h[pz].x, xi, ax.x); ax.y = fmaf(h[pz].y, xi, ax.y);
        ax.z = fmaf(h[pz].z, xi, ax.z); ax.w = fmaf(h[pz].w, xi, ax.w);
        aq.x = fmaf(h[pz].x, qi, aq.x); aq.y = fmaf(h[pz].y, qi, aq.y);
        aq.z = fmaf(h[pz].z, qi, aq.z); aq.w = fmaf(h[pz].w, qi, aq.w);
    }
    *reinterpret_cast<float4*>(&redx[rg][c4 * 4]) = ax;
    *reinterpret_cast<float4*>(&redq[rg][c4 * 4]) = aq;
    __syncthreads();
    if (tid < DVS) {
        float rx = 0.f, rq = 0.f, kqt = 0.f;
#pragma unroll
        for (int r = 0; r < RP; ++r) { rx += redx[r][tid]; rq += redq[r][tid]; }
#pragma unroll
        for (int w = 0; w < NT / 32; ++w) kqt += skq[w];
        const float dl = be * (ld(v, (size_t)bh * dv + j0 + tid) - al * rx);
        sdelta[tid] = dl;
        st(o, (size_t)bh * dv + j0 + tid, fmaf(al, rq, kqt * dl));
    }
    __syncthreads();
    const float4 dl = *reinterpret_cast<const float4*>(&sdelta[c4 * 4]);
#pragma unroll
    for (int pz = 0; pz < NP; ++pz) {
        const float ki = sk[pz * RP + rg];
        float4 r;
        r.x = fmaf(al, h[pz].x, ki * dl.x); r.y = fmaf(al, h[pz].y, ki * dl.y);
        r.z = fmaf(al, h[pz].z, ki * dl.z); r.w = fmaf(al, h[pz].w, ki * dl.w);
        __stcs(base + (size_t)(pz * RP + rg) * rstride, r);
    }
}

// Several tokens per call (multi-token / speculative decoding): S consecutive tokens of every sequence go through the
// same recurrence, one after the other, while the state slice stays in registers -- one read and one write of the state
// for S tokens instead of S of each.  Token tensors are token-major [B, S, H, d] like those of the chunkwise calls.  The
// arithmetic of one token is exactly that of k_decode, in the same order, so S tokens here give bit-identical results to
// S single-token calls.
// SB16 (QD_STATE_BF16): the state is STORED in bf16 (half the bytes of the step); it is widened to fp32 when read, all S
// tokens of the call are applied in fp32, and it is rounded to bf16 once, when written back.
template <typename IO, int DK, int DVS, int NT, bool LOGITS, bool NORM, bool SB16>      // flags, compile-time
__global__ void __launch_bounds__(NT) k_decode_multi(int S, int H, int dv, const IO* __restrict__ q, const IO* __restrict__ k,
                                                     const IO* __restrict__ v, const IO* __restrict__ beta,
                                                     const IO* __restrict__ alpha, const IO* __restrict__ lam,
                                                     void* __restrict__ state_, IO* __restrict__ o) {
    constexpr int C4 = DVS / 4, RP = NT / C4, NP = DK / RP;
    static_assert(NT % C4 == 0 && DK % RP == 0, "bad decode tiling");
    __shared__ float sx[DK], sq[DK], sk[DK];
    __shared__ float redx[RP][DVS], redq[RP][DVS];
    __shared__ float sdelta[DVS];
    __shared__ float skq[NT / 32], snq[NT / 32], snk[NT / 32];
    const int nsl = dv / DVS, bh = blockIdx.x / nsl, j0 = (blockIdx.x % nsl) * DVS, tid = threadIdx.x;
    const int b = bh / H, hh = bh % H;
    const int c4 = tid % C4, rg = tid / C4;

    // four consecutive d_v columns per thread and row: 16 bytes of an fp32 state, 8 bytes of a bf16 state
    float4* base = reinterpret_cast<float4*>(static_cast<float*>(state_) + (size_t)bh * DK * dv + j0) + c4;
    uint2* base16 = reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(state_) + (size_t)bh * DK * dv + j0) + c4;
    const int rstride = dv / 4;
    float4 h[NP];
#pragma unroll
    for (int pz = 0; pz < NP; ++pz) {
        if (SB16) {
            const uint2 u = __ldcs(base16 + (size_t)(pz * RP + rg) * rstride);
            const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.x));
            const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.y));
            h[pz] = make_float4(lo.x, lo.y, hi.x, hi.y);
        } else {
            h[pz] = __ldcs(base + (size_t)(pz * RP + rg) * rstride);
        }
    }

    for (int s = 0; s < S; ++s) {
        const size_t row = ((size_t)b * S + s) * H + hh;        // token row of this head in the [B, S, H] view
        const float be = gate(ld(beta, row), LOGITS);
        const float al = alpha ? gate(ld(alpha, row), LOGITS) : 1.f;
        const float la = lam ? gate(ld(lam, row), LOGITS) : 0.f;
        float kq = 0.f;
        if (NORM) {
            // q^ = q / sqrt(|q|^2 + eps), k^ likewise: three block-wide sums, then the token's arrays are rescaled
            float ssq = 0.f, ssk = 0.f;
            for (int i = tid; i < DK; i += NT) {
                const float qi = ld(q, row * DK + i), ki = ld(k, row * DK + i);
                sq[i] = qi; sk[i] = ki;
                ssq = fmaf(qi, qi, ssq); ssk = fmaf(ki, ki, ssk); kq = fmaf(ki, qi, kq);
            }
#pragma unroll
            for (int w = 16; w > 0; w >>= 1) {
                kq += __shfl_xor_sync(0xffffffffu, kq, w);
                ssq += __shfl_xor_sync(0xffffffffu, ssq, w);
                ssk += __shfl_xor_sync(0xffffffffu, ssk, w);
            }
            if ((tid & 31) == 0) { skq[tid >> 5] = kq; snq[tid >> 5] = ssq; snk[tid >> 5] = ssk; }
            __syncthreads();
            float tq = 0.f, tk = 0.f, tkq = 0.f;
#pragma unroll
            for (int w = 0; w < NT / 32; ++w) { tq += snq[w]; tk += snk[w]; tkq += skq[w]; }
            const float rq = 1.f / sqrtf(tq + kNormEps), rk = 1.f / sqrtf(tk + kNormEps);
            __syncthreads();
            for (int i = tid; i < DK; i += NT) {
                const float qi = sq[i] * rq, ki = sk[i] * rk;
                sq[i] = qi; sk[i] = ki; sx[i] = fmaf(la, qi, ki);
            }
            if (tid == 0) { skq[0] = tkq * rq * rk; for (int w = 1; w < NT / 32; ++w) skq[w] = 0.f; }
        } else {
            for (int i = tid; i < DK; i += NT) {
                const float qi = ld(q, row * DK + i), ki = ld(k, row * DK + i);
                sq[i] = qi; sk[i] = ki; sx[i] = fmaf(la, qi, ki);
                kq = fmaf(ki, qi, kq);
            }
#pragma unroll
            for (int w = 16; w > 0; w >>= 1) kq += __shfl_xor_sync(0xffffffffu, kq, w);
            if ((tid & 31) == 0) skq[tid >> 5] = kq;
        }
        __syncthreads();

        float4 ax = make_float4(0.f, 0.f, 0.f, 0.f), aq = ax;
#pragma unroll
        for (int pz = 0; pz < NP; ++pz) {
            const float xi = sx[pz * RP + rg], qi = sq[pz * RP + rg];
            ax.x = fmaf(h[pz].x, xi, ax.x); ax.y = fmaf(h[pz].y, xi, ax.y);
            ax.z = fmaf(h[pz].z, xi, ax.z); ax.w = fmaf(h[pz].w, xi, ax.w);
            aq.x = fmaf(h[pz].x, qi, aq.x); aq.y = fmaf(h[pz].y, qi, aq.y);
            aq.z = fmaf(h[pz].z, qi, aq.z); aq.w = fmaf(h[pz].w, qi, aq.w);
        }
        *reinterpret_cast<float4*>(&redx[rg][c4 * 4]) = ax;
        *reinterpret_cast<float4*>(&redq[rg][c4 * 4]) = aq;
        __syncthreads();
        if (tid < DVS) {
            float rx = 0.f, rq = 0.f, kqt = 0.f;
#pragma unroll
            for (int r = 0; r < RP; ++r) { rx += redx[r][tid]; rq += redq[r][tid]; }
#pragma unroll
            for (int w = 0; w < NT / 32; ++w) kqt += skq[w];
            const float dl = be * (ld(v, row * dv + j0 + tid) - al * rx);
            sdelta[tid] = dl;
            st(o, row * dv + j0 + tid, fmaf(al, rq, kqt * dl));
        }
        __syncthreads();
        const float4 dl = *reinterpret_cast<const float4*>(&sdelta[c4 * 4]);
#pragma unroll
        for (int pz = 0; pz < NP; ++pz) {
            const float ki = sk[pz * RP + rg];
            h[pz].x = fmaf(al, h[pz].x, ki * dl.x); h[pz].y = fmaf(al, h[pz].y, ki * dl.y);
            h[pz].z = fmaf(al, h[pz].z, ki * dl.z); h[pz].w = fmaf(al, h[pz].w, ki * dl.w);
        }
        __syncthreads();                 // the token's shared arrays are rewritten by the next one
    }
#pragma unroll
    for (int pz = 0; pz < NP; ++pz) {
        if (SB16) {
            const __nv_bfloat162 lo = __floats2bfloat162_rn(h[pz].x, h[pz].y), hi = __floats2bfloat162_rn(h[pz].z, h[pz].w);
            uint2 u;
            u.x = *reinterpret_cast<const unsigned*>(&lo);
            u.y = *reinterpret_cast<const unsigned*>(&hi);
            __stcs(base16 + (size_t)(pz * RP + rg) * rstride, u);
        } else {
            __stcs(base + (size_t)(pz * RP + rg) * rstride, h[pz]);
        }
    }
}

template <typename IO, int DK>
cudaError_t launch_multi(int B, int S, int H, int dv, const void* q, const void* k, const void* v, const void* beta,
                         const void* alpha, const void* lam, void* state, void* o, bool logits, bool norm, bool sb16,
                         cudaStream_t stream) {
    constexpr int DVS = 64, NT = 128;
    dim3 grid((unsigned)(dv / DVS) * (unsigned)(B * H));
    auto kern = logits ? (norm ? k_decode_multi<IO, DK, DVS, NT, true, true, false> : k_decode_multi<IO, DK, DVS, NT, true, false, false>)
                       : (norm ? k_decode_multi<IO, DK, DVS, NT, false, true, false> : k_decode_multi<IO, DK, DVS, NT, false, false, false>);
    if (sb16)
        kern = logits ? (norm ? k_decode_multi<IO, DK, DVS, NT, true, true, true> : k_decode_multi<IO, DK, DVS, NT, true, false, true>)
                      : (norm ? k_decode_multi<IO, DK, DVS, NT, false, true, true> : k_decode_multi<IO, DK, DVS, NT, false, false, true>);
    kern<<<grid, NT, 0, stream>>>(S, H, dv, (const IO*)q, (const IO*)k, (const IO*)v, (const IO*)beta, (const IO*)alpha,
                                  (const IO*)lam, state, (IO*)o);
    return cudaGetLastError();
}

template <typename IO, int DK>
cudaError_t launch(int BH, int dv, const void* q, const void* k, const void* v, const void* beta,
                   const void* alpha, const void* lam, float* state, void* o, cudaStream_t stream) {
    constexpr int DVS = 64, NT = 128;
    dim3 grid((unsigned)(dv / DVS) * (unsigned)BH);
    k_decode<IO, DK, DVS, NT><<<grid, NT, 0, stream>>>(dv, (const IO*)q, (const IO*)k, (const IO*)v,
                                                       (const IO*)beta, (const IO*)alpha, (const IO*)lam,
                                                       state, (IO*)o);
    return cudaGetLastError();
}

}  // namespace

cudaError_t decode_step(int BH, int dk, int dv, int dtype, const void* q, const void* k, const void* v,
                        const void* beta, const void* alpha, const void* lam, float* state, void* o,
                        cudaStream_t stream) {
    if (dtype == QD_BF16) {
        if (dk == 128) return launch<__nv_bfloat16, 128>(BH, dv, q, k, v, beta, alpha, lam, state, o, stream);
        return launch<__nv_bfloat16, 64>(BH, dv, q, k, v, beta, alpha, lam, state, o, stream);
    }
    if (dk == 128) return launch<float, 128>(BH, dv, q, k, v, beta, alpha, lam, state, o, stream);
    return launch<float, 64>(BH, dv, q, k, v, beta, alpha, lam, state, o, stream);
}

cudaError_t decode_steps(int B, int S, int H, int dk, int dv, int dtype, const void* q, const void* k, const void* v,
                         const void* beta, const void* alpha, const void* lam, void* state, void* o,
                         bool logits, bool norm, bool sb16, cudaStream_t stream) {
    if (dtype == QD_BF16) {
        if (dk == 128) return launch_multi<__nv_bfloat16, 128>(B, S, H, dv, q, k, v, beta, alpha, lam, state, o, logits, norm, sb16, stream);
        return launch_multi<__nv_bfloat16, 64>(B, S, H, dv, q, k, v, beta, alpha, lam, state, o, logits, norm, sb16, stream);
    }
    if (dk == 128) return launch_multi<float, 128>(B, S, H, dv, q, k, v, beta, alpha, lam, state, o, logits, norm, sb16, stream);
    return launch_multi<float, 64>(B, S, H, dv, q, k, v, beta, alpha, lam, state, o, logits, norm, sb16, stream);
}

}  // namespace qd
