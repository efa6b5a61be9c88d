// Chunkwise Q-Delta forward and backward in plain fp32 FMA arithmetic (no tensor cores).
//
// This is the path for fp32 storage (1e-4 parity needs full fp32 products) and for shapes the
// tensor-core kernels do not cover.  It follows the chunk equations of Section 3.3.2:
//   g_r = sum_{i<=r} log alpha_i,  gamma_r = e^{g_r},  Gamma_ri = e^{g_r-g_i} (r >= i)
//   X = K + diag(lambda) Q
//   A = strictLower(diag(beta)(Gamma o X K^T)),  M = (I+A)^-1,  T = M diag(beta)     (UT transform)
//   U~ = T V,  W<- = T diag(gamma) X                                                  (extended WY)
//   Delta = U~ - W<- h;  O = diag(gamma) Q h + (Gamma o Q K^T o causal) Delta
//   h <- gamma_C h + (diag(gamma_C/gamma) K)^T Delta                                  (chunk-level update)
// and, for the backward, the exact gradient of those equations (the paper prints none).
// Every decay factor is formed as exp of a non-positive difference of cumulative logs; no
// quotient of cumulative products is ever taken.
#include "internal.h"

namespace qd {
namespace {

constexpr int C = kChunk;
constexpr int LD = C + 1;          // padded leading dimension of C x C matrices in shared memory
constexpr int DS = kSliceSimt;
constexpr int NT = 256;

struct Ptrs {
    int B, T, Tp, H, dk, dv, N;      // the workspace holds Tp = 64 N >= T rows per sequence; rows past T are tokens with
                                     // beta = 0, alpha = 1, q = k = v = dO = 0 (exact no-ops of the recurrence)
    const void *q, *k, *v, *beta, *alpha, *lam, *dO;
    const float *h0, *dhT;
    void *o, *dq, *dk_, *dv_;
    float *hT, *dbeta, *dalpha, *dlam, *dh0;
    float* g;
    void *P, *W, *U, *D, *dD;
    float *hs, *dhs, *kdhd, *dhh, *scratch;
    int nslices, save;
    int logits;                      // beta, alpha, lambda are logits of sigmoid gates
    float* rqk;                      // non-null (QD_NORM_QK): q and k are L2-normalised in here; [0, BH*Tp) 1/|q_t|, then 1/|k_t|
};

// Register-tiled product: every thread owns TM x TN outputs of an M x N result with inner
// extent K; a(m,k), b(k,n) fetch operands (from anywhere), epi(m,n,acc) consumes results.
template <int TM, int TN, class FA, class FB, class FE>
__device__ __forceinline__ void mm(int M, int N, int K, FA a, FB b, FE epi) {
    const int tn = N / TN, tiles = (M / TM) * tn;
    for (int id = threadIdx.x; id < tiles; id += blockDim.x) {
        const int m0 = (id / tn) * TM, n0 = (id % tn) * TN;
        float acc[TM][TN];
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;
        for (int kk = 0; kk < K; ++kk) {
            float av[TM], bv[TN];
#pragma unroll
            for (int i = 0; i < TM; ++i) av[i] = a(m0 + i, kk);
#pragma unroll
            for (int j = 0; j < TN; ++j) bv[j] = b(kk, n0 + j);
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
            for (int j = 0; j < TN; ++j) epi(m0 + i, n0 + j, acc[i][j]);
    }
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// 1/|q_r| and 1/|k_r| of one chunk into shared memory: computed from the rows (and kept in the workspace) by the
// preparation kernel, read back from the workspace by the others.  Without normalisation both are 1.
template <typename IO, bool COMPUTE>
__device__ __forceinline__ void load_norms(const Ptrs& p, size_t row0, size_t wrow0, int live, float* srq, float* srk) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (!p.rqk) {
        if (threadIdx.x < C) { srq[threadIdx.x] = 1.f; srk[threadIdx.x] = 1.f; }
    } else if (COMPUTE) {
        const size_t nrows = (size_t)p.B * p.H * p.Tp;
        for (int r = warp; r < C; r += NT / 32) {
            float sq = 0.f, sk = 0.f;
            if (r < live)
                for (int d = lane; d < p.dk; d += 32) {
                    const float qv = ld((const IO*)p.q, (row0 + (size_t)r * p.H) * p.dk + d);
                    const float kv = ld((const IO*)p.k, (row0 + (size_t)r * p.H) * p.dk + d);
                    sq = fmaf(qv, qv, sq); sk = fmaf(kv, kv, sk);
                }
            sq = warp_sum(sq); sk = warp_sum(sk);
            if (lane == 0) {
                const float rq = 1.f / sqrtf(sq + kNormEps), rk = 1.f / sqrtf(sk + kNormEps);
                srq[r] = rq; srk[r] = rk;
                p.rqk[wrow0 + r] = rq; p.rqk[nrows + wrow0 + r] = rk;
            }
        }
    } else if (threadIdx.x < C) {
        const size_t nrows = (size_t)p.B * p.H * p.Tp;
        srq[threadIdx.x] = p.rqk[wrow0 + threadIdx.x];
        srk[threadIdx.x] = p.rqk[nrows + wrow0 + threadIdx.x];
    }
    __syncthreads();
}

// Coefficients of one chunk into shared memory: beta, lambda, alpha, g (cumulative log alpha).
template <typename IO>
__device__ __forceinline__ void load_coeffs(const Ptrs& p, size_t row0, int live, float* sbeta, float* slam,
                                            float* salpha, float* sg) {
    const int t = threadIdx.x;
    if (t < C) {
        const size_t r = row0 + (size_t)t * p.H;
        sbeta[t] = t < live ? gate(ld((const IO*)p.beta, r), p.logits) : 0.f;
        slam[t] = (t < live && p.lam) ? gate(ld((const IO*)p.lam, r), p.logits) : 0.f;
        salpha[t] = (t < live && p.alpha) ? log_gate(ld((const IO*)p.alpha, r), p.logits) : 0.f;     // log alpha
    }
    __syncthreads();
    if (t == 0) {
        float acc = 0.f;
        for (int r = 0; r < C; ++r) { acc += salpha[r]; sg[r] = acc; }
    }
    __syncthreads();
}

// M = (I + A)^-1 for unit lower-triangular I + A (A strictly lower), by forward substitution:
// thread j solves column j.  sA and sM are C x C with leading dimension LD.
__device__ __forceinline__ void invert_unit_lower(const float* sA, float* sM) {
    const int j = threadIdx.x;
    if (j < C) {
        for (int r = 0; r < j; ++r) sM[r * LD + j] = 0.f;
        sM[j * LD + j] = 1.f;
        for (int r = j + 1; r < C; ++r) {
            float acc = 0.f;
            for (int i = j; i < r; ++i) acc = fmaf(sA[r * LD + i], sM[i * LD + j], acc);
            sM[r * LD + j] = -acc;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// K1: per chunk-head, state-independent part: g, P, W<-, U~.
template <typename IO>
__global__ void __launch_bounds__(NT) k_prep(Ptrs p) {
    __shared__ float sA[C * LD], sM[C * LD];
    __shared__ float sbeta[C], slam[C], salpha[C], sg[C], srq[C], srk[C];
    const int ch = blockIdx.x, n = ch % p.N, bh = ch / p.N, b = bh / p.H, hh = bh % p.H;
    const int dk = p.dk, dv = p.dv, H = p.H;
    const size_t row0 = ((size_t)b * p.T + (size_t)n * C) * H + hh;   // token row of local r: row0 + r*H
    const size_t wrow0 = (size_t)bh * p.Tp + (size_t)n * C;           // workspace row of local r: wrow0 + r
    const int live = min(C, p.T - n * C);                              // tokens of this chunk inside the sequence
    const IO *q = (const IO*)p.q, *k = (const IO*)p.k, *v = (const IO*)p.v;
    load_coeffs<IO>(p, row0, live, sbeta, slam, salpha, sg);
    if (threadIdx.x < C) p.g[wrow0 + threadIdx.x] = sg[threadIdx.x];
    load_norms<IO, true>(p, row0, wrow0, live, srq, srk);

    auto Qf = [&](int r, int d) { return r < live ? srq[r] * ld(q, (row0 + (size_t)r * H) * dk + d) : 0.f; };
    auto Kf = [&](int r, int d) { return r < live ? srk[r] * ld(k, (row0 + (size_t)r * H) * dk + d) : 0.f; };
    auto Xf = [&](int r, int d) { return fmaf(slam[r], Qf(r, d), Kf(r, d)); };
    // A = strictLower(beta_r Gamma_ri (x_r . k_i))
    mm<4, 4>(C, C, dk, Xf, [&](int d, int i) { return Kf(i, d); },
             [&](int r, int i, float acc) {
                 sA[r * LD + i] = (i < r) ? sbeta[r] * expf(sg[r] - sg[i]) * acc : 0.f;
             });
    // P = Gamma o (Q K^T), causal including the diagonal
    mm<4, 4>(C, C, dk, Qf, [&](int d, int i) { return Kf(i, d); },
             [&](int r, int i, float acc) {
                 st((IO*)p.P, (wrow0 + r) * C + i, (i <= r) ? expf(sg[r] - sg[i]) * acc : 0.f);
             });
    __syncthreads();
    invert_unit_lower(sA, sM);
    __syncthreads();
    auto Tf = [&](int r, int i) { return sM[r * LD + i] * sbeta[i]; };
    mm<4, 4>(C, dv, C, Tf, [&](int i, int j) { return i < live ? ld(v, (row0 + (size_t)i * H) * dv + j) : 0.f; },
             [&](int r, int j, float acc) { st((IO*)p.U, (wrow0 + r) * dv + j, acc); });
    mm<4, 4>(C, dk, C, Tf, [&](int i, int d) { return expf(sg[i]) * Xf(i, d); },
             [&](int r, int d, float acc) { st((IO*)p.W, (wrow0 + r) * dk + d, acc); });
}

// ---------------------------------------------------------------------------------------------
// K2: forward state chain.  One CTA per (sequence, 32-column slice of d_v); columns of the state
// evolve independently, the chunks of a sequence are walked in order.
template <typename IO>
__global__ void __launch_bounds__(NT) k_chain_fwd(Ptrs p) {
    extern __shared__ float sm[];
    const int dk = p.dk, dv = p.dv, H = p.H;
    float* sh = sm;                 // [dk][DS]  state slice
    float* sD = sh + dk * DS;       // [C][DS]   Delta slice
    float* sO = sD + C * DS;        // [C][DS]
    float* sg = sO + C * DS;        // [C]
    float *srq = sg + C, *srk = srq + C;
    const int nsl = dv / DS, j0 = (blockIdx.x % nsl) * DS, bh = blockIdx.x / nsl, b = bh / H, hh = bh % H;
    const IO *q = (const IO*)p.q, *k = (const IO*)p.k;
    for (int e = threadIdx.x; e < dk * DS; e += NT) {
        const int i = e / DS, j = e % DS;
        sh[e] = p.h0 ? p.h0[((size_t)bh * dk + i) * dv + j0 + j] : 0.f;
    }
    for (int n = 0; n < p.N; ++n) {
        const size_t row0 = ((size_t)b * p.T + (size_t)n * C) * H + hh;
        const size_t wrow0 = (size_t)bh * p.Tp + (size_t)n * C;
        const int live = min(C, p.T - n * C);
        if (threadIdx.x < C) sg[threadIdx.x] = p.g[wrow0 + threadIdx.x];
        load_norms<IO, false>(p, row0, wrow0, live, srq, srk);
        if (p.save) {
            float* dst = p.hs + ((size_t)bh * p.N + n) * dk * dv;
            for (int e = threadIdx.x; e < dk * DS; e += NT) dst[(size_t)(e / DS) * dv + j0 + e % DS] = sh[e];
        }
        auto hf = [&](int i, int j) { return sh[i * DS + j]; };
        // Delta = U~ - W<- h
        mm<2, 4>(C, DS, dk, [&](int r, int i) { return ld((const IO*)p.W, (wrow0 + r) * dk + i); }, hf,
                 [&](int r, int j, float acc) {
                     const float d = ld((const IO*)p.U, (wrow0 + r) * dv + j0 + j) - acc;
                     sD[r * DS + j] = d;
                     if (p.save) st((IO*)p.D, (wrow0 + r) * dv + j0 + j, d);
                 });
        // inter-chunk part of the output: diag(gamma) Q h
        mm<2, 4>(C, DS, dk, [&](int r, int i) { return r < live ? srq[r] * ld(q, (row0 + (size_t)r * H) * dk + i) : 0.f; }, hf,
                 [&](int r, int j, float acc) { sO[r * DS + j] = expf(sg[r]) * acc; });
        __syncthreads();
        // intra-chunk part: P Delta
        mm<2, 4>(C, DS, C, [&](int r, int s) { return ld((const IO*)p.P, (wrow0 + r) * C + s); },
                 [&](int s, int j) { return sD[s * DS + j]; },
                 [&](int r, int j, float acc) {
                     if (r < live) st((IO*)p.o, (row0 + (size_t)r * H) * dv + j0 + j, sO[r * DS + j] + acc);
                 });
        // h <- gamma_C h + K->^T Delta
        const float gC = sg[C - 1];
        mm<4, 4>(dk, DS, C,
                 [&](int i, int r) { return r < live ? srk[r] * ld(k, (row0 + (size_t)r * H) * dk + i) * expf(gC - sg[r]) : 0.f; },
                 [&](int r, int j) { return sD[r * DS + j]; },
                 [&](int i, int j, float acc) { sh[i * DS + j] = fmaf(expf(gC), sh[i * DS + j], acc); });
        __syncthreads();
    }
    if (p.hT)
        for (int e = threadIdx.x; e < dk * DS; e += NT)
            p.hT[((size_t)bh * dk + e / DS) * dv + j0 + e % DS] = sh[e];
}

// ---------------------------------------------------------------------------------------------
// K3: reverse state chain.  Carries dh (gradient w.r.t. the chunk's exit state) backwards:
//   dDelta = P^T dO + K-> dh ;   dh_in = gamma_C dh + (diag(gamma) Q)^T dO - W<-^T dDelta
// and leaves per chunk: dh (exit), dDelta, and two scalar partial sums the decay gradient needs.
template <typename IO>
__global__ void __launch_bounds__(NT) k_chain_bwd(Ptrs p) {
    extern __shared__ float sm[];
    __shared__ float sred[NT / 32];
    const int dk = p.dk, dv = p.dv, H = p.H;
    float* sdh = sm;                 // [dk][DS]
    float* sdD = sdh + dk * DS;      // [C][DS]
    float* sKD = sdD + C * DS;       // [C][DS]  (K-> dh) o Delta
    float* sg = sKD + C * DS;        // [C]
    float *srq = sg + C, *srk = srq + C;
    const int nsl = dv / DS, sl = blockIdx.x % nsl, j0 = sl * DS, bh = blockIdx.x / nsl, b = bh / H, hh = bh % H;
    const IO *q = (const IO*)p.q, *k = (const IO*)p.k, *dO = (const IO*)p.dO;
    const size_t BHT = (size_t)p.B * H * p.Tp, BHN = (size_t)p.B * H * p.N;
    for (int e = threadIdx.x; e < dk * DS; e += NT)
        sdh[e] = p.dhT ? p.dhT[((size_t)bh * dk + e / DS) * dv + j0 + e % DS] : 0.f;
    for (int n = p.N - 1; n >= 0; --n) {
        const size_t row0 = ((size_t)b * p.T + (size_t)n * C) * H + hh;
        const size_t wrow0 = (size_t)bh * p.Tp + (size_t)n * C;
        const int live = min(C, p.T - n * C);
        if (threadIdx.x < C) sg[threadIdx.x] = p.g[wrow0 + threadIdx.x];
        load_norms<IO, false>(p, row0, wrow0, live, srq, srk);
        // keep dh of this chunk's exit state; partial <dh, h_entry>_F over this slice
        {
            float* dst = p.dhs + ((size_t)bh * p.N + n) * dk * dv;
            const float* hsrc = p.hs + ((size_t)bh * p.N + n) * dk * dv;
            float part = 0.f;
            for (int e = threadIdx.x; e < dk * DS; e += NT) {
                const size_t off = (size_t)(e / DS) * dv + j0 + e % DS;
                dst[off] = sdh[e];
                part = fmaf(sdh[e], hsrc[off], part);
            }
            part = warp_sum(part);
            if ((threadIdx.x & 31) == 0) sred[threadIdx.x >> 5] = part;
            __syncthreads();
            if (threadIdx.x == 0) {
                float tot = 0.f;
                for (int w = 0; w < NT / 32; ++w) tot += sred[w];
                p.dhh[(size_t)sl * BHN + (size_t)bh * p.N + n] = tot;
            }
        }
        const float gC = sg[C - 1];
        // K-> dh
        mm<2, 4>(C, DS, dk,
                 [&](int s, int i) { return s < live ? srk[s] * ld(k, (row0 + (size_t)s * H) * dk + i) * expf(gC - sg[s]) : 0.f; },
                 [&](int i, int j) { return sdh[i * DS + j]; },
                 [&](int s, int j, float acc) {
                     sdD[s * DS + j] = acc;
                     sKD[s * DS + j] = acc * ld((const IO*)p.D, (wrow0 + s) * dv + j0 + j);
                 });
        __syncthreads();
        // + P^T dO   (same thread owns the same (s,j) as above: tile shapes are identical)
        mm<2, 4>(C, DS, C, [&](int s, int r) { return ld((const IO*)p.P, (wrow0 + r) * C + s); },
                 [&](int r, int j) { return r < live ? ld(dO, (row0 + (size_t)r * H) * dv + j0 + j) : 0.f; },
                 [&](int s, int j, float acc) {
                     const float d = sdD[s * DS + j] + acc;
                     sdD[s * DS + j] = d;
                     st((IO*)p.dD, (wrow0 + s) * dv + j0 + j, d);
                 });
        // row sums of (K-> dh) o Delta over this slice
        for (int s = threadIdx.x >> 5; s < C; s += NT / 32) {
            const float x = warp_sum(sKD[s * DS + (threadIdx.x & 31)]);
            if ((threadIdx.x & 31) == 0) p.kdhd[(size_t)sl * BHT + wrow0 + s] = x;
        }
        __syncthreads();
        // dh_in = gamma_C dh + (diag(gamma) Q)^T dO - W<-^T dDelta    (one product over 2C terms)
        mm<4, 4>(dk, DS, 2 * C,
                 [&](int i, int kk) {
                     return kk < C ? (kk < live ? srq[kk] * ld(q, (row0 + (size_t)kk * H) * dk + i) * expf(sg[kk]) : 0.f)
                                   : -ld((const IO*)p.W, (wrow0 + kk - C) * dk + i);
                 },
                 [&](int kk, int j) {
                     return kk < C ? (kk < live ? ld(dO, (row0 + (size_t)kk * H) * dv + j0 + j) : 0.f) : sdD[(kk - C) * DS + j];
                 },
                 [&](int i, int j, float acc) { sdh[i * DS + j] = fmaf(expf(gC), sdh[i * DS + j], acc); });
        __syncthreads();
    }
    if (p.dh0)
        for (int e = threadIdx.x; e < dk * DS; e += NT)
            p.dh0[((size_t)bh * dk + e / DS) * dv + j0 + e % DS] = sdh[e];
}

// ---------------------------------------------------------------------------------------------
// K4: chunk-parallel part of the backward: dq, dk, dv, dbeta, dlambda, dalpha.
template <typename IO>
__global__ void __launch_bounds__(NT) k_chunk_bwd(Ptrs p, int nchunks) {
    extern __shared__ float sm[];
    float* m0 = sm;                  // X K^T          -> dA o Gamma o XK
    float* m1 = m0 + C * LD;         // M              -> dP o P
    float* m2 = m1 + C * LD;         // A -> dT -> dM -> dA -> dXK
    float* m3 = m2 + C * LD;         // dP             -> dP o Gamma
    float* m4 = m3 + C * LD;         // dM M^T         -> dA o A
    float* sbeta = m4 + C * LD;
    float* slam = sbeta + C;
    float* salpha = slam + C;
    float* sg = salpha + C;
    float* sgam = sg + C;
    float* segc = sgam + C;
    float* sdbeta = segc + C;
    float* st1 = sdbeta + C;         // rowsum(dQ1 o Q)
    float* st2 = st1 + C;            // rowsum(dXg o gamma X)
    float* sdlam = st2 + C;
    float* sdg = sdlam + C;
    float *srq = sdg + C, *srk = srq + C;
    const int dk = p.dk, dv = p.dv, H = p.H;
    const IO *q = (const IO*)p.q, *k = (const IO*)p.k, *v = (const IO*)p.v, *dO = (const IO*)p.dO;
    float* sc = p.scratch + (size_t)blockIdx.x * 6 * C * dk;
    float *dW = sc, *dXg = sc + C * dk, *dX = sc + 2 * C * dk, *dQ1 = sc + 3 * C * dk;
    float *dKh = sc + 4 * C * dk, *dQh = sc + 5 * C * dk;      // QD_NORM_QK: gradients w.r.t. the normalised rows
    const size_t BHT = (size_t)p.B * H * p.Tp, BHN = (size_t)p.B * H * p.N;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int ch = blockIdx.x; ch < nchunks; ch += gridDim.x) {
        const int n = ch % p.N, bh = ch / p.N, b = bh / H, hh = bh % H;
        const size_t row0 = ((size_t)b * p.T + (size_t)n * C) * H + hh;
        const size_t wrow0 = (size_t)bh * p.Tp + (size_t)n * C;
        const int live = min(C, p.T - n * C);
        const float* hs = p.hs + ((size_t)bh * p.N + n) * dk * dv;
        const float* dhs = p.dhs + ((size_t)bh * p.N + n) * dk * dv;
        auto Qf = [&](int r, int d) { return r < live ? srq[r] * ld(q, (row0 + (size_t)r * H) * dk + d) : 0.f; };
        auto Kf = [&](int r, int d) { return r < live ? srk[r] * ld(k, (row0 + (size_t)r * H) * dk + d) : 0.f; };
        auto Vf = [&](int r, int j) { return r < live ? ld(v, (row0 + (size_t)r * H) * dv + j) : 0.f; };
        auto dOf = [&](int r, int j) { return r < live ? ld(dO, (row0 + (size_t)r * H) * dv + j) : 0.f; };
        auto Xf = [&](int r, int d) { return fmaf(slam[r], Qf(r, d), Kf(r, d)); };
        auto Df = [&](int r, int j) { return ld((const IO*)p.D, (wrow0 + r) * dv + j); };
        auto dDf = [&](int r, int j) { return ld((const IO*)p.dD, (wrow0 + r) * dv + j); };

        // S0 coefficients
        if (tid < C) {
            const size_t r = row0 + (size_t)tid * H;
            sbeta[tid] = tid < live ? gate(ld((const IO*)p.beta, r), p.logits) : 0.f;
            slam[tid] = (tid < live && p.lam) ? gate(ld((const IO*)p.lam, r), p.logits) : 0.f;
            salpha[tid] = (tid < live && p.alpha) ? gate(ld((const IO*)p.alpha, r), p.logits) : 1.f;
            sg[tid] = p.g[wrow0 + tid];
        }
        load_norms<IO, false>(p, row0, wrow0, live, srq, srk);
        if (tid < C) { sgam[tid] = expf(sg[tid]); segc[tid] = expf(sg[C - 1] - sg[tid]); }
        // S1 Gram X K^T, and A
        mm<4, 4>(C, C, dk, Xf, [&](int d, int i) { return Kf(i, d); },
                 [&](int r, int i, float acc) {
                     m0[r * LD + i] = acc;
                     m2[r * LD + i] = (i < r) ? sbeta[r] * expf(sg[r] - sg[i]) * acc : 0.f;
                 });
        __syncthreads();
        // S2 M = (I+A)^-1
        invert_unit_lower(m2, m1);
        // S3 products that need the saved states
        mm<4, 4>(C, C, dv, dOf, [&](int j, int s) { return Df(s, j); },
                 [&](int r, int s, float acc) { m3[r * LD + s] = (s <= r) ? acc : 0.f; });       // dP
        mm<4, 4>(C, dk, dv, dDf, [&](int j, int i) { return hs[(size_t)i * dv + j]; },
                 [&](int r, int i, float acc) { dW[r * dk + i] = -acc; });                        // dW<-
        mm<4, 4>(C, dk, dv, dOf, [&](int j, int d) { return hs[(size_t)d * dv + j]; },
                 [&](int r, int d, float acc) { dQ1[r * dk + d] = sgam[r] * acc; });              // diag(gamma) dO h^T
        __syncthreads();
        // S4 dT = dDelta V^T + dW<- (gamma X)^T
        mm<4, 4>(C, C, dv + dk,
                 [&](int r, int kk) { return kk < dv ? dDf(r, kk) : dW[r * dk + kk - dv]; },
                 [&](int kk, int s) { return kk < dv ? Vf(s, kk) : sgam[s] * Xf(s, kk - dv); },
                 [&](int r, int s, float acc) { m2[r * LD + s] = acc; });
        __syncthreads();
        // S5 dV = T^T dDelta, dXg = T^T dW<-, dbeta = colsum(dT o M)
        auto TTf = [&](int s, int r) { return m1[r * LD + s] * sbeta[s]; };
        mm<4, 4>(C, dv, C, TTf, [&](int r, int j) { return dDf(r, j); },
                 [&](int s, int j, float acc) { if (s < live) st((IO*)p.dv_, (row0 + (size_t)s * H) * dv + j, acc); });
        mm<4, 4>(C, dk, C, TTf, [&](int r, int i) { return dW[r * dk + i]; },
                 [&](int s, int i, float acc) { dXg[s * dk + i] = acc; });
        if (tid < C) {
            float acc = 0.f;
            for (int r = 0; r < C; ++r) acc = fmaf(m2[r * LD + tid], m1[r * LD + tid], acc);
            sdbeta[tid] = acc;
        }
        __syncthreads();
        // S6 dM = dT diag(beta)
        for (int e = tid; e < C * C; e += NT) m2[(e / C) * LD + e % C] *= sbeta[e % C];
        __syncthreads();
        // S7 dA = -strictLower(M^T dM M^T)
        mm<4, 4>(C, C, C, [&](int r, int u) { return m2[r * LD + u]; }, [&](int u, int s) { return m1[s * LD + u]; },
                 [&](int r, int s, float acc) { m4[r * LD + s] = acc; });
        __syncthreads();
        mm<4, 4>(C, C, C, [&](int r, int u) { return m1[u * LD + r]; }, [&](int u, int s) { return m4[u * LD + s]; },
                 [&](int r, int s, float acc) { m2[r * LD + s] = (s < r) ? -acc : 0.f; });
        __syncthreads();
        // S8 element-wise: split dA into its three uses; dP into dP o P and dP o Gamma
        for (int e = tid; e < C * C; e += NT) {
            const int r = e / C, s = e % C, o = r * LD + s;
            const float Gm = (s <= r) ? expf(sg[r] - sg[s]) : 0.f;
            const float da = m2[o], xk = m0[o];
            m4[o] = da * sbeta[r] * Gm * xk;                    // dA o A
            m0[o] = da * Gm * xk;                               // -> dbeta
            m2[o] = da * sbeta[r] * Gm;                         // dXK
            const float dp = m3[o];
            m1[o] = dp * ld((const IO*)p.P, (wrow0 + r) * C + s);   // dP o P
            m3[o] = dp * Gm;                                        // dP o Gamma
        }
        __syncthreads();
        // S9 dX = diag(gamma) dXg + dXK K ; row/column sums
        mm<4, 4>(C, dk, C, [&](int r, int i) { return m2[r * LD + i]; }, Kf,
                 [&](int r, int d, float acc) { dX[r * dk + d] = fmaf(sgam[r], dXg[r * dk + d], acc); });
        if (tid < C) {
            float rb = 0.f, rA = 0.f, cA = 0.f, rP = 0.f, cP = 0.f;
            for (int s = 0; s < C; ++s) {
                rb += m0[tid * LD + s];
                rA += m4[tid * LD + s]; cA += m4[s * LD + tid];
                rP += m1[tid * LD + s]; cP += m1[s * LD + tid];
            }
            sdbeta[tid] += rb;
            sdg[tid] = rP - cP + rA - cA;
        }
        __syncthreads();
        // S10 dK, dQ, and the row reductions that need full rows
        mm<4, 4>(C, dk, 2 * C + dv,
                 [&](int i, int kk) {
                     return kk < C ? m2[kk * LD + i] : (kk < 2 * C ? m3[(kk - C) * LD + i] : segc[i] * Df(i, kk - 2 * C));
                 },
                 [&](int kk, int d) {
                     return kk < C ? Xf(kk, d) : (kk < 2 * C ? Qf(kk - C, d) : dhs[(size_t)d * dv + kk - 2 * C]);
                 },
                 [&](int i, int d, float acc) {
                     if (p.rqk) dKh[i * dk + d] = acc + dX[i * dk + d];
                     else if (i < live) st((IO*)p.dk_, (row0 + (size_t)i * H) * dk + d, acc + dX[i * dk + d]);
                 });
        mm<4, 4>(C, dk, C, [&](int r, int s) { return m3[r * LD + s]; }, Kf,
                 [&](int r, int d, float acc) {
                     const float val = acc + dQ1[r * dk + d] + slam[r] * dX[r * dk + d];
                     if (p.rqk) dQh[r * dk + d] = val;
                     else if (r < live) st((IO*)p.dq, (row0 + (size_t)r * H) * dk + d, val);
                 });
        for (int r = warp; r < C; r += NT / 32) {
            float a1 = 0.f, a2 = 0.f, a3 = 0.f;
            for (int d = lane; d < dk; d += 32) {
                const float qv = Qf(r, d), xv = fmaf(slam[r], qv, Kf(r, d));
                a1 = fmaf(dQ1[r * dk + d], qv, a1);
                a2 = fmaf(dXg[r * dk + d], sgam[r] * xv, a2);
                a3 = fmaf(dX[r * dk + d], qv, a3);
            }
            a1 = warp_sum(a1); a2 = warp_sum(a2); a3 = warp_sum(a3);
            if (lane == 0) { st1[r] = a1; st2[r] = a2; sdlam[r] = a3; }
        }
        __syncthreads();
        if (p.rqk) {
            // through the normalisation: dx = r (dx^ - x^ <x^, dx^>), one warp per row
            for (int r = warp; r < live; r += NT / 32) {
                float cq = 0.f, ck = 0.f;
                for (int d = lane; d < dk; d += 32) {
                    cq = fmaf(dQh[r * dk + d], Qf(r, d), cq);
                    ck = fmaf(dKh[r * dk + d], Kf(r, d), ck);
                }
                cq = warp_sum(cq); ck = warp_sum(ck);
                for (int d = lane; d < dk; d += 32) {
                    st((IO*)p.dq, (row0 + (size_t)r * H) * dk + d, srq[r] * (dQh[r * dk + d] - Qf(r, d) * cq));
                    st((IO*)p.dk_, (row0 + (size_t)r * H) * dk + d, srk[r] * (dKh[r * dk + d] - Kf(r, d) * ck));
                }
            }
        }
        // S11 decay gradient: dg, reverse in-chunk cumulative sum, d alpha = d log alpha / alpha
        if (tid < C) {
            float kd = 0.f;
            for (int s = 0; s < p.nslices; ++s) kd += p.kdhd[(size_t)s * BHT + wrow0 + tid];
            sdg[tid] += st1[tid] + st2[tid] - kd;
            st1[tid] = kd;
        }
        __syncthreads();
        if (tid == 0) {
            float dhh = 0.f, kdt = 0.f;
            for (int s = 0; s < p.nslices; ++s) dhh += p.dhh[(size_t)s * BHN + (size_t)bh * p.N + n];
            for (int r = 0; r < C; ++r) kdt += st1[r];
            sdg[C - 1] += sgam[C - 1] * dhh + kdt;
            float acc = 0.f;
            for (int r = C - 1; r >= 0; --r) { acc += sdg[r]; sdg[r] = acc; }
        }
        __syncthreads();
        if (tid < live) {
            const size_t r = row0 + (size_t)tid * H;
            // with logit inputs the gradients are taken w.r.t. the logits: sigmoid' = s (1 - s), (log sigmoid)' = 1 - s
            const float be = sbeta[tid], la = slam[tid], al = salpha[tid];
            p.dbeta[r] = p.logits ? sdbeta[tid] * be * (1.f - be) : sdbeta[tid];
            if (p.dlam) p.dlam[r] = p.logits ? sdlam[tid] * la * (1.f - la) : sdlam[tid];
            if (p.dalpha) p.dalpha[r] = p.logits ? sdg[tid] * (1.f - al) : sdg[tid] / al;
        }
        __syncthreads();
    }
}

Ptrs make_ptrs(const ChunkArgs& a) {
    Ptrs p{};
    p.B = a.s.B; p.T = a.s.T; p.Tp = simt_padded_T(a.s); p.H = a.s.H; p.dk = a.s.dk; p.dv = a.s.dv; p.N = p.Tp / kChunk;
    p.q = a.q; p.k = a.k; p.v = a.v; p.beta = a.beta; p.alpha = a.alpha; p.lam = a.lam; p.dO = a.dO;
    p.h0 = a.h0; p.dhT = a.dhT; p.o = a.o; p.dq = a.dq; p.dk_ = a.dk; p.dv_ = a.dv;
    p.hT = a.hT; p.dbeta = a.dbeta; p.dalpha = a.dalpha; p.dlam = a.dlam; p.dh0 = a.dh0;
    p.g = (float*)(a.ws + a.L.g);
    p.P = a.ws + a.L.P; p.W = a.ws + a.L.W; p.U = a.ws + a.L.U;
    p.D = a.ws + a.L.D; p.dD = a.ws + a.L.dD;
    p.hs = (float*)(a.ws + a.L.hs); p.dhs = (float*)(a.ws + a.L.dhs);
    p.kdhd = (float*)(a.ws + a.L.kdhd); p.dhh = (float*)(a.ws + a.L.dhh);
    p.scratch = (float*)(a.ws + a.L.scratch);
    p.nslices = a.L.nslices; p.save = a.save ? 1 : 0; p.logits = a.logits ? 1 : 0;
    p.rqk = a.norm ? (float*)(a.ws + a.L.rqk) : nullptr;
    return p;
}

template <class K>
cudaError_t set_smem(K kern, size_t bytes) { return set_max_smem_once(reinterpret_cast<const void*>(kern), bytes); }

}  // namespace

cudaError_t simt_prep(const ChunkArgs& a) {
    Ptrs p = make_ptrs(a);
    const int grid = a.s.B * a.s.H * p.N;
    if (a.s.dtype == QD_BF16) k_prep<__nv_bfloat16><<<grid, NT, 0, a.stream>>>(p);
    else k_prep<float><<<grid, NT, 0, a.stream>>>(p);
    return cudaGetLastError();
}

cudaError_t simt_chain_fwd(const ChunkArgs& a) {
    Ptrs p = make_ptrs(a);
    const size_t smem = sizeof(float) * ((size_t)a.s.dk * DS + 2 * C * DS + 3 * C);
    dim3 grid((unsigned)(a.s.dv / DS) * (unsigned)(a.s.B * a.s.H));
    cudaError_t e;
    if (a.s.dtype == QD_BF16) {
        if ((e = set_smem(k_chain_fwd<__nv_bfloat16>, smem)) != cudaSuccess) return e;
        k_chain_fwd<__nv_bfloat16><<<grid, NT, smem, a.stream>>>(p);
    } else {
        if ((e = set_smem(k_chain_fwd<float>, smem)) != cudaSuccess) return e;
        k_chain_fwd<float><<<grid, NT, smem, a.stream>>>(p);
    }
    return cudaGetLastError();
}

cudaError_t simt_chain_bwd(const ChunkArgs& a) {
    Ptrs p = make_ptrs(a);
    const size_t smem = sizeof(float) * ((size_t)a.s.dk * DS + 2 * C * DS + 3 * C);
    dim3 grid((unsigned)(a.s.dv / DS) * (unsigned)(a.s.B * a.s.H));
    cudaError_t e;
    if (a.s.dtype == QD_BF16) {
        if ((e = set_smem(k_chain_bwd<__nv_bfloat16>, smem)) != cudaSuccess) return e;
        k_chain_bwd<__nv_bfloat16><<<grid, NT, smem, a.stream>>>(p);
    } else {
        if ((e = set_smem(k_chain_bwd<float>, smem)) != cudaSuccess) return e;
        k_chain_bwd<float><<<grid, NT, smem, a.stream>>>(p);
    }
    return cudaGetLastError();
}

cudaError_t simt_chunk_bwd(const ChunkArgs& a) {
    Ptrs p = make_ptrs(a);
    const int nchunks = a.s.B * a.s.H * p.N;
    const int grid = nchunks < a.L.bwd_ctas ? nchunks : a.L.bwd_ctas;
    const size_t smem = sizeof(float) * (5 * C * LD + 13 * C);
    cudaError_t e;
    if (a.s.dtype == QD_BF16) {
        if ((e = set_smem(k_chunk_bwd<__nv_bfloat16>, smem)) != cudaSuccess) return e;
        k_chunk_bwd<__nv_bfloat16><<<grid, NT, smem, a.stream>>>(p, nchunks);
    } else {
        if ((e = set_smem(k_chunk_bwd<float>, smem)) != cudaSuccess) return e;
        k_chunk_bwd<float><<<grid, NT, smem, a.stream>>>(p, nchunks);
    }
    return cudaGetLastError();
}

}  // namespace qd
