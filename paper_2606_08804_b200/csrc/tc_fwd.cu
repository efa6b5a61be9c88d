// Tensor-core (tcgen05 / TMEM / TMA) chunkwise forward for bf16, d_k = d_v = 128, chunk 64.
//
// Two kernels, following Section 3.3.2:
//   k_tc_prep       one CTA per PAIR of chunks (128 tokens): g, X = K + diag(lambda) Q, the Gram
//                   blocks X K^T and Q K^T, the UT-transform inverse, and the WY factors.  It leaves,
//                   per chunk, in bf16:  Qg = diag(gamma) Q  [token][dk],
//                   P = Gamma o (Q K^T) causal incl. diagonal [token][64],
//                   Wt = (T diag(gamma) X)^T  [dk][64 tokens],   Ut = (T V)^T  [dv][64 tokens].
//   k_tc_chain_fwd  one CTA per (batch, head): walks the chunks in order with the fp32 state in
//                   registers (thread j owns row j of h^T, i.e. column j of h), everything
//                   transposed so that d_v = 128 is the MMA M dimension:
//                     Delta^T = Ut - h^T Wt            O^T = h^T Qg^T + Delta^T P^T
//                     h^T <- gamma_C h^T + (Delta diag(gamma_C/gamma))^T K
// All waits are bounded; on expiry the CTA records QD_ERR_TIMEOUT in the workspace status word,
// releases its tensor memory and returns.
#include "internal.h"
#include "sm100.cuh"

namespace qd {
namespace {
using namespace sm100;
typedef __nv_bfloat16 bf16;

constexpr int C = kChunk;      // 64
constexpr int D = 128;         // d_k = d_v

__device__ __forceinline__ void load8(const unsigned char* p, float* f) {
    const uint4 u = *reinterpret_cast<const uint4*>(p);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const float2 t = __bfloat1622float2(h[i]); f[2 * i] = t.x; f[2 * i + 1] = t.y; }
}
__device__ __forceinline__ uint4 pack8(const float* f) {
    uint4 u;
    u.x = pack_bf16(f[0], f[1]); u.y = pack_bf16(f[2], f[3]); u.z = pack_bf16(f[4], f[5]); u.w = pack_bf16(f[6], f[7]);
    return u;
}

// =================================================================================================
struct PrepParams {
    float* rqk;                // non-null: L2-normalise q and k here; [0, BH*Tp) <- 1/|q_t|, [BH*Tp, 2 BH*Tp) <- 1/|k_t|
    int T, Tp, H, N, BH;       // T tokens per sequence; the workspace holds Tp = 64 N >= T rows per sequence (N even)
    const bf16 *beta, *alpha, *lam;
    float* g;
    bf16 *Qg, *P;
    bf16* Mt;                  // optional: ((I+A)^-1)^T per chunk, [column i][row r]; kept for the backward
    unsigned* status;
};

// 96 KB: Q (later X, in place) | K (later A in fp32, then the T tiles) | V; at the end the first and the
// last 32 KB stage U~^T and W~^T for their TMA stores.  Two CTAs fit on one SM.
constexpr int kPrepSmem = 3 * 32768 + 1024;
constexpr int kPrepThreads = 256;

// One CTA prepares a pair of chunks (128 tokens) of one head.  Thread roles change by phase:
//   scan / coefficients   thread t < 128 owns token t
//   row-wise elementwise  16 threads per 256-byte row (coalesced), 16 rows per pass
//   Gram epilogue         thread (row = t & 127, half = t >> 7) owns 32 columns of its TMEM lane
//   triangular inverse    lane quad (t >> 2, t < 128) owns columns j0 + 16 k (j0 < 16) of one chunk, quad lane t & 3 the 8-row blocks t & 3 and (t & 3) + 4
//   final epilogue        thread (d = t & 127, which = t >> 7) owns one row of U~^T resp. W~^T
// NORM (QD_NORM_QK): L2-normalise the rows of Q and K first.  LOGITS (QD_COEF_LOGITS): the coefficients are logits of
// sigmoid gates.  Compile-time, because even the untaken sigmoid / log-sigmoid code on the path of the scan, which
// every later phase of the CTA waits for, cost the kernel 8 %.
template <bool NORM, bool LOGITS>
__global__ void __launch_bounds__(kPrepThreads, 2) k_tc_prep(const __grid_constant__ CUtensorMap mapQ,
                                                             const __grid_constant__ CUtensorMap mapK,
                                                             const __grid_constant__ CUtensorMap mapV,
                                                             const __grid_constant__ CUtensorMap mapUt,
                                                             const __grid_constant__ CUtensorMap mapWt, PrepParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char *sQ = smem, *sK = smem + 32768, *sV = smem + 65536;
    // lambda absent (the gated delta rule, Eq. 3): X = K, so nothing is built, both Gram products start at once, and
    // the scratch that otherwise overwrites K overwrites Q instead
    const bool has_lam = p.lam != nullptr;
    unsigned char* sX = has_lam ? sQ : sK;                      // X overwrites Q once Q K^T has been formed
    unsigned char* sScr = has_lam ? sK : sQ;                    // dead once both Grams are read (and diag(gamma)Q is written)
    float* sA = reinterpret_cast<float*>(sScr);                 // A^T [2][column i][row r]
    unsigned char* sT = sScr;                                   // [2] T_c, [2] T_c diag(gamma): 8 KB each, alias A
    __shared__ uint64_t bar_load, bar_mma;
    __shared__ uint32_t tmem_slot;
    __shared__ float sg[128], sbeta[128], slam[128], swsum[4];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // CTAs are numbered pair-major, last pair first: the forward chain, which starts with chunk 0 of every sequence,
    // then finds the tiles written last (and K, read last) still in L2
    const int pairs = p.N / 2, pr = pairs - 1 - (int)blockIdx.x / p.BH, bh = (int)blockIdx.x % p.BH;
    const int b = bh / p.H, hh = bh % p.H;
    const int t0 = pr * 128;                                         // first token of the pair
    const size_t wtok0 = (size_t)bh * p.Tp + (size_t)t0;             // first row in the workspace's [BH*Tp] view

    if (tid == 0) {
        mbar_init(&bar_load, 1);
        mbar_init(&bar_mma, 1);
        mbar_init_fence();
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = tmem_slot;

    grid_dep_launch();                // the kernel after this one may set itself up while the last CTAs of this one run
    if (tid == 0) {
        mbar_expect_tx(&bar_load, 3 * 32768);
        for (int blk = 0; blk < 2; ++blk) {          // rows at t >= T arrive as zeros
            tma_load_3d(sQ + blk * 16384, &mapQ, hh * D + blk * 64, t0, b, &bar_load);
            tma_load_3d(sK + blk * 16384, &mapK, hh * D + blk * 64, t0, b, &bar_load);
            tma_load_3d(sV + blk * 16384, &mapV, hh * D + blk * 64, t0, b, &bar_load);
        }
    }
    // coefficients of token tid; in-chunk cumulative log-decay by a two-warp scan per chunk
    if (tid < 128) {
        // a token past the end of the sequence is an exact no-op of the recurrence: beta = 0, alpha = 1 (and q = k = v = 0)
        const bool live = t0 + tid < p.T;
        const size_t crow = ((size_t)b * p.T + t0 + tid) * p.H + hh;
        sbeta[tid] = live ? gate(__bfloat162float(p.beta[crow]), LOGITS) : 0.f;
        slam[tid] = (live && p.lam) ? gate(__bfloat162float(p.lam[crow]), LOGITS) : 0.f;
        float g = (live && p.alpha) ? log_gate(__bfloat162float(p.alpha[crow]), LOGITS) : 0.f;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xffffffffu, g, o);
            if (lane >= o) g += t;
        }
        if (lane == 31) swsum[warp] = g;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (warp & 1) g += swsum[warp - 1];
        sg[tid] = g;
        p.g[wtok0 + tid] = g;
    }

    bool fail = !mbar_wait(&bar_load, 0);
    if (__syncthreads_or(fail)) {
        if (tid == 0) *p.status = QD_ERR_TIMEOUT;
        mbar_wait(&bar_load, 0);           // loads may still be in flight: one more bounded chance
        __syncthreads();
        if (warp == 0) tmem_dealloc(tbase, 256);
        return;
    }
    // row-wise work: 16 lanes cover one 256-byte row (chunk `ch` of 16 bytes each), 16 rows per pass
    const int ch = tid & 15, rsub = tid >> 4;
    const uint32_t coff = (ch >> 3) * 16384;
    if (NORM) {
        // q^ = q / sqrt(|q|^2 + eps), k^ likewise, in place: everything below (and every later kernel, through
        // diag(gamma) Q^ and the 1/|k| written here) works on the normalised rows
        const size_t nrows = (size_t)p.BH * p.Tp;
#pragma unroll 2
        for (int it = 0; it < 8; ++it) {
            const int row = it * 16 + rsub;
            const uint32_t off = coff + sw128_chunk(row, ch & 7);
            float qv[8], kv[8], sq = 0.f, sk = 0.f;
            load8(sQ + off, qv);
            load8(sK + off, kv);
#pragma unroll
            for (int e = 0; e < 8; ++e) { sq = fmaf(qv[e], qv[e], sq); sk = fmaf(kv[e], kv[e], sk); }
#pragma unroll
            for (int o = 1; o < 16; o <<= 1) {
                sq += __shfl_xor_sync(0xffffffffu, sq, o);
                sk += __shfl_xor_sync(0xffffffffu, sk, o);
            }
            const float rq = rsqrtf(sq + kNormEps), rk = rsqrtf(sk + kNormEps);
#pragma unroll
            for (int e = 0; e < 8; ++e) { qv[e] *= rq; kv[e] *= rk; }
            sts128(sQ + off, pack8(qv));
            sts128(sK + off, pack8(kv));
            if (ch == 0) { p.rqk[wtok0 + row] = rq; p.rqk[nrows + wtok0 + row] = rk; }
        }
        fence_proxy_async();
        __syncthreads();
    }
    if (tid == 0) {
        tc_fence_after();
        // G2 = Q K^T -> columns [128,256);  without lambda also G1 = K K^T -> columns [0,128)
        umma_product<false, false>(tbase + 128, smem_u32(sQ), 16384, smem_u32(sK), 16384, 128, 128, false);
        if (!has_lam) umma_product<false, false>(tbase, smem_u32(sK), 16384, smem_u32(sK), 16384, 128, 128, false);
        umma_commit(&bar_mma);
    }
    // meanwhile: Qg = gamma Q to the workspace, a warp writes two full rows per store
    {
        bf16* qg = p.Qg + wtok0 * D + ch * 8;
#pragma unroll 4
        for (int it = 0; it < 8; ++it) {
            const int row = it * 16 + rsub;
            const float gr = __expf(sg[row]);
            float qv[8];
            load8(sQ + coff + sw128_chunk(row, ch & 7), qv);
#pragma unroll
            for (int e = 0; e < 8; ++e) qv[e] *= gr;
            *reinterpret_cast<uint4*>(qg + (size_t)row * D) = pack8(qv);
        }
    }
    fail = !mbar_wait(&bar_mma, 0);
    if (__syncthreads_or(fail)) {
        if (tid == 0) *p.status = QD_ERR_TIMEOUT;
        if (warp == 0) tmem_dealloc(tbase, 256);
        return;
    }
    if (has_lam) {
        // X = K + lambda Q, in place over Q (K-major swizzled layout)
#pragma unroll 4
        for (int it = 0; it < 8; ++it) {
            const int row = it * 16 + rsub;
            const uint32_t off = coff + sw128_chunk(row, ch & 7);
            const float lm = slam[row];
            float qv[8], kv[8];
            load8(sQ + off, qv);
            load8(sK + off, kv);
#pragma unroll
            for (int e = 0; e < 8; ++e) kv[e] = fmaf(lm, qv[e], kv[e]);
            sts128(sX + off, pack8(kv));
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            // G1 = X K^T -> columns [0,128)
            umma_product<false, false>(tbase, smem_u32(sX), 16384, smem_u32(sK), 16384, 128, 128, false);
            umma_commit(&bar_mma);
        }
        fail = !mbar_wait(&bar_mma, 1);
        if (__syncthreads_or(fail)) {
            if (tid == 0) *p.status = QD_ERR_TIMEOUT;
            if (warp == 0) tmem_dealloc(tbase, 256);
            return;
        }
    }
    tc_fence_after();
    // A = strictLower(beta_r Gamma_ri (x_r . k_i)) -> shared fp32, transposed;  P = Gamma_ri (q_r . k_i), i <= r -> workspace
    {
        const int row = tid & 127, half = tid >> 7, c = row >> 6, r = row & 63;
        const float g = sg[row], beta = sbeta[row];
        const float* gc = sg + c * C;
        float* Ac = sA + c * C * C;
        float v1[32], v2[32];
        tmem_ld32(tmem_addr(tbase, (warp & 3) * 32, c * C + half * 32), v1);
        tmem_ld32(tmem_addr(tbase, (warp & 3) * 32, 128 + c * C + half * 32), v2);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const int col = half * 32 + i;
            const float dec = (col <= r) ? __expf(g - gc[col]) : 0.f;
            v1[i] = (col < r) ? beta * dec * v1[i] : 0.f;
            v2[i] = dec * v2[i];
        }
        // A^T: entry (column i, row r) at i*64 + r, so that 8 consecutive rows of one column are contiguous
#pragma unroll
        for (int i = 0; i < 32; ++i) Ac[(half * 32 + i) * C + r] = v1[i];
        bf16* prow = p.P + (wtok0 + row) * C + half * 32;
#pragma unroll
        for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(prow + i * 8) = pack8(v2 + i * 8);
    }
    tc_fence_before();
    __syncthreads();
    // M_c = (I + A_c)^-1 by right-looking substitution, columns in registers.  A lane quad of the first four warps
    // owns four columns of one chunk, j0 + 16 k with j0 < 16 (the same loads of A serve all four); lane `ql` of the
    // quad owns the 8-row blocks ql and ql + 4.  Once m[i] is final its owner hands it to the other three lanes and
    // every later row gets its update m[r] -= A[r][i] m[i]; rows <= i of a block see A = 0 exactly, so whole blocks
    // are updated.  Column j0 + 16 k is zero above row 16 k and joins at step 16 k; blocks 0..3 are final after step
    // 30.  The loads of A are warp-wide broadcasts, and shared-memory wavefronts are what bounds this phase: hence
    // four columns per load (32 FMAs for two 16-byte loads).
    const int qd4 = tid >> 2, ql = tid & 3, ic = (qd4 >> 4) & 1, j0 = qd4 & 15;
    float m[2][4][8];
    if (tid < 128) {
        const float* Ac = sA + ic * C * C + ql * 8;
#pragma unroll
        for (int sb = 0; sb < 2; ++sb)
#pragma unroll
            for (int k = 0; k < 4; ++k)
#pragma unroll
                for (int e = 0; e < 8; ++e) m[sb][k][e] = ((ql + 4 * sb) * 8 + e == j0 + 16 * k) ? 1.f : 0.f;
#pragma unroll
        for (int i = 0; i < C - 1; ++i) {
            const int bi = i >> 3;                              // block of the pivot row; its owner is quad lane bi & 3
            const int src = (lane & ~3) | (bi & 3);
            float mi[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                mi[k] = (i >= 16 * k) ? __shfl_sync(0xffffffffu, m[bi >> 2][k][i & 7], src) : 0.f;
#pragma unroll
            for (int sb = (i < 31 ? 0 : 1); sb < 2; ++sb) {
                const float4 a0 = *reinterpret_cast<const float4*>(Ac + i * C + sb * 32);
                const float4 a1 = *reinterpret_cast<const float4*>(Ac + i * C + sb * 32 + 4);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (i >= 16 * k) {
                        float* mm = m[sb][k];
                        mm[0] = fmaf(-a0.x, mi[k], mm[0]); mm[1] = fmaf(-a0.y, mi[k], mm[1]);
                        mm[2] = fmaf(-a0.z, mi[k], mm[2]); mm[3] = fmaf(-a0.w, mi[k], mm[3]);
                        mm[4] = fmaf(-a1.x, mi[k], mm[4]); mm[5] = fmaf(-a1.y, mi[k], mm[5]);
                        mm[6] = fmaf(-a1.z, mi[k], mm[6]); mm[7] = fmaf(-a1.w, mi[k], mm[7]);
                    }
                }
            }
        }
    }
    __syncthreads();
    // T_c = M_c diag(beta), T_c diag(gamma): line j of the MN-major tiles holds column j over the rows
    if (tid < 128) {
        unsigned char* t0 = sT + ic * 8192;
        unsigned char* t1 = sT + 16384 + ic * 8192;
        bf16* mt = p.Mt ? p.Mt + ((size_t)bh * p.N + 2 * pr + ic) * C * C : nullptr;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int j = j0 + 16 * k;
            const float beta = sbeta[ic * C + j], bg = beta * __expf(sg[ic * C + j]);
#pragma unroll
            for (int sb = 0; sb < 2; ++sb) {
                const int kb = ql + 4 * sb;
                float a[8], bq[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) { a[e] = m[sb][k][e] * beta; bq[e] = m[sb][k][e] * bg; }
                sts128(t0 + sw128_chunk(j, kb), pack8(a));
                sts128(t1 + sw128_chunk(j, kb), pack8(bq));
                if (mt) *reinterpret_cast<uint4*>(mt + (size_t)j * C + kb * 8) = pack8(m[sb][k]);
            }
        }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
        tc_fence_after();
        for (int cc = 0; cc < 2; ++cc) {
            // Ut_c = V_c^T T_c^T  -> columns [cc*64, +64);   Wt_c = X_c^T (T_c diag(gamma))^T -> 128 + ...
            umma_product<true, true>(tbase + cc * C, smem_u32(sV) + cc * C * 128, 16384,
                                     smem_u32(sT) + cc * 8192, 8192, C, C, false);
            umma_product<true, true>(tbase + 128 + cc * C, smem_u32(sX) + cc * C * 128, 16384,
                                     smem_u32(sT) + 16384 + cc * 8192, 8192, C, C, false);
        }
        umma_commit(&bar_mma);
    }
    fail = !mbar_wait(&bar_mma, has_lam ? 0 : 1);          // third phase of the barrier with lambda, second without
    if (__syncthreads_or(fail)) {
        if (tid == 0) *p.status = QD_ERR_TIMEOUT;
        if (warp == 0) tmem_dealloc(tbase, 256);
        return;
    }
    tc_fence_after();
    // row d = tid & 127 of U~^T (threads < 128) resp. W~^T (the others), both chunks: staged as swizzled
    // [128][64] tiles over the dead Q/X and V regions, then written by TMA
    {
        const int d = tid & 127, which = tid >> 7;
        unsigned char* stage = which ? sV : sQ;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
            float v[32];
            tmem_ld32(tmem_addr(tbase, (warp & 3) * 32, which * 128 + q4 * 32), v);
            tmem_ld_wait();
            unsigned char* tile = stage + (q4 >> 1) * 16384;
#pragma unroll
            for (int i = 0; i < 4; ++i) sts128(tile + sw128_chunk(d, (q4 & 1) * 4 + i), pack8(v + i * 8));
        }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
        const int y = (int)(((size_t)bh * p.N + 2 * pr) * D);
        tma_store_2d(&mapUt, sQ, 0, y);
        tma_store_2d(&mapUt, sQ + 16384, 0, y + D);
        tma_store_2d(&mapWt, sV, 0, y);
        tma_store_2d(&mapWt, sV + 16384, 0, y + D);
        tma_store_commit();
        tma_store_wait_read();             // the staging tiles must outlive the reads; the writes complete with the grid
    }
    if (warp == 0) {
        __syncwarp();
        tmem_dealloc(tbase, 256);
    }
}

// =================================================================================================
struct ChainParams {
    int Tp, H, N;              // Tp = 64 N rows per sequence in the workspace
    const float* g;
    const float* h0;
    float* hT;
    int save;                  // also store, per chunk, the bf16 entry state (mapHs) and Delta^T (mapDt)
    int scaled;                // 0: no forget gate and no key normalisation: every per-token factor on Delta is 1
    const float* rk;           // non-null (QD_NORM_QK): 1/|k_t| per workspace row; the keys are read un-normalised and
                               // the factor is folded into the per-token scale of Delta
    unsigned* status;
};

constexpr int kStage = 73728;                                   // Wt 16K | Ut 16K | Qg 16K | K 16K | P 8K
constexpr int kChainSmem = 2 * kStage + 65536 + 16384 + 1024;   // + h^T 32K, Delta^T 16K, scaled Delta^T 16K, O 16K
constexpr int kChainCompute = 512;                 // 16 epilogue warps: 4 warpgroups split the accumulator columns
constexpr int kChainThreads = kChainCompute + 64;  // + 1 MMA-issue warp, 1 TMA warp
constexpr int kMmaWarp = kChainCompute / 32;
constexpr int kNb = kChainCompute + 32;            // participants of a named barrier: the epilogue threads and one waiting warp

// named barriers: compute threads arrive, the MMA and/or TMA warp wait
constexpr int kBarH = 1, kBarD = 2, kBarO = 3, kBarHt = 4, kBarDt = 5;   // ..t: the same event, awaited by the TMA warp
__device__ __forceinline__ void nb_arrive(int id, int count) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void nb_sync(int id, int count) {
    __syncwarp();                                   // the lanes of a warp reach the barrier together
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// Forward state chain.  The only true dependency per chunk is
//   h ready -> Delta-accumulator = h^T Wt -> Delta^T -> H-accumulator = (scaled Delta^T) K -> h update;
// the output products (h^T Qg^T + Delta^T P^T, double-buffered accumulator), the output epilogue and
// every TMA copy run in its shadow on their own warps.
// Compute warpgroup w owns tokens [32w, 32w+32) of the 64-column accumulators and d_k columns
// [64w, 64w+64) of the state; thread l of a warpgroup owns TMEM lane l = d_v index.
__global__ void __launch_bounds__(kChainThreads) k_tc_chain_fwd(const __grid_constant__ CUtensorMap mapWt,
                                                                const __grid_constant__ CUtensorMap mapUt,
                                                                const __grid_constant__ CUtensorMap mapQg,
                                                                const __grid_constant__ CUtensorMap mapK,
                                                                const __grid_constant__ CUtensorMap mapP,
                                                                const __grid_constant__ CUtensorMap mapHs,
                                                                const __grid_constant__ CUtensorMap mapDt,
                                                                const __grid_constant__ CUtensorMap mapO,
                                                                ChainParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* sH = smem + 2 * kStage;          // h^T as A operand: K-major, 2 blocks of [128 lines][64]
    unsigned char* sD = sH + 32768;                 // Delta^T: K-major [128 lines (dv)][64 tokens]
    unsigned char* sDs = sD + 16384;                // Delta^T scaled by gamma_C/gamma_r per token
    unsigned char* sO = sDs + 16384;                // output tile [64 tokens][128 dv], 2 blocks of [64 lines][64]
    __shared__ uint64_t bar_load[2], bar_a, bar_b, bar_o, bar_e;
    __shared__ uint32_t tmem_slot;
    __shared__ volatile int s_abort;
    // per chunk parity: gamma_C / gamma_t for the 64 tokens, then gamma_C; written by the TMA warp one chunk
    // ahead and published with its arrival on bar_a, so no epilogue thread waits for a global load
    __shared__ __align__(16) float sG[2][68];

    const int tid = threadIdx.x, warp = tid >> 5, wg = tid >> 7, l = tid & 127, wq = warp & 3;
    const int bh = blockIdx.x, b = bh / p.H, hh = bh % p.H;

    if (tid == 0) {
        mbar_init(&bar_load[0], 1); mbar_init(&bar_load[1], 1);
        mbar_init(&bar_a, 2); mbar_init(&bar_b, 2); mbar_init(&bar_o, 2); mbar_init(&bar_e, 1);
        mbar_init_fence();
        s_abort = 0;
    }
    if (tid < 32) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = tmem_slot;
    const uint32_t tD = tbase, tH = tbase + 128, tO0 = tbase + 256;      // O-accumulators: tO0 + 64 * (n & 1)
    const uint32_t lane_base = (uint32_t)wq * 32;

    // bounded wait; once any wait has expired every later wait returns at once (the kernel drains)
    auto wait = [&](uint64_t* bar, uint32_t parity) {
        if (s_abort) return;
        if (!mbar_wait(bar, parity)) { s_abort = 1; *p.status = QD_ERR_TIMEOUT; }
    };
    const float* gseq = p.g + (size_t)bh * p.Tp;

    if (warp < kMmaWarp) {
        // ---------------------------------- compute warps ----------------------------------
        float h[32];      // h^T[j = l][32 wg .. 32 wg + 31], fp32
        if (p.h0) {
            const float* src = p.h0 + (size_t)bh * D * D + (size_t)(32 * wg) * D + l;
#pragma unroll
            for (int i = 0; i < 32; ++i) h[i] = src[(size_t)i * D];
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) h[i] = 0.f;
        }
        grid_dep_wait();                  // the loads of h0 (an input) are in flight; everything below depends on the prep kernel
        grid_dep_launch();
        // my 32 columns of the operand tile: 64-column block wg >> 1, 16-byte chunks 4 (wg & 1) ..
        unsigned char* myH = sH + (wg >> 1) * 16384;
        const int hc0 = (wg & 1) * 4;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) sts128(myH + sw128_chunk(l, hc0 + ch), pack8(h + ch * 8));
        // byte offsets of my (fixed) column inside a staging line, for the 8 possible (token & 7)
        uint32_t xoff[8];
#pragma unroll
        for (int e = 0; e < 8; ++e)
            xoff[e] = (uint32_t)e * 128u + (((((uint32_t)l & 63u) >> 3) ^ (uint32_t)e) << 4) + ((uint32_t)l & 7u) * 2u;
        fence_proxy_async();
        nb_arrive(kBarH, kNb); nb_arrive(kBarHt, kNb);

        auto o_stage = [&](int m) {
            // output of chunk m: O^T row j = l, my 16 tokens -> staging tile (token-major); stored by the TMA warp
            unsigned char* stg = sO + (l >> 6) * 8192 + (wg * 16) * 128;
            float v[16];
            tmem_ld16(tmem_addr(tO0 + 64 * (m & 1), lane_base, wg * 16), v);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) sts16(stg + (i >> 3) * 1024 + xoff[i & 7], __float2bfloat16_rn(v[i]));
            tc_fence_before();
            fence_proxy_async();
            nb_arrive(kBarO, kNb);
        };

        for (int n = 0; n < p.N; ++n) {
            const unsigned char* st = smem + (n & 1) * kStage;
            wait(&bar_load[n & 1], (n >> 1) & 1);
            wait(&bar_a, n & 1);
            tc_fence_after();
            // decay ratios of my 16 tokens
            float sc[16];
            {
                const float4* gp = reinterpret_cast<const float4*>(&sG[n & 1][wg * 16]);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float4 t = gp[q];
                    sc[q * 4] = t.x; sc[q * 4 + 1] = t.y; sc[q * 4 + 2] = t.z; sc[q * 4 + 3] = t.w;
                }
            }
            const float gamC = sG[n & 1][64];
            // Delta^T = Ut - acc, my 16 tokens; two bf16 copies (plain, and scaled by gamma_C/gamma_r) as A operands
            {
                const unsigned char* ut = st + 16384;
                float v[16];
                tmem_ld16(tmem_addr(tD, lane_base, wg * 16), v);
                tmem_ld_wait();
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    float u[8], d1[8];
                    const uint32_t off = sw128_chunk(l, wg * 2 + cc);
                    load8(ut + off, u);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        u[e] -= v[cc * 8 + e];
                        d1[e] = u[e] * sc[cc * 8 + e];
                    }
                    sts128(sD + off, pack8(u));
                    if (p.scaled) sts128(sDs + off, pack8(d1));         // all factors 1: the scaled copy is Delta itself
                }
            }
            tc_fence_before();
            fence_proxy_async();
            nb_arrive(kBarD, kNb); nb_arrive(kBarDt, kNb);
            // in the shadow of the H product: output epilogue of the previous chunk
            if (n > 0) { wait(&bar_o, (n - 1) & 1); tc_fence_after(); o_stage(n - 1); }
            // h^T <- gamma_C h^T + acc (my 32 d_k columns), refresh the bf16 operand copy
            wait(&bar_b, n & 1);
            tc_fence_after();
            {
                float v[32];
                tmem_ld32(tmem_addr(tH, lane_base, wg * 32), v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) h[i] = fmaf(gamC, h[i], v[i]);
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) sts128(myH + sw128_chunk(l, hc0 + cc), pack8(h + cc * 8));
            }
            tc_fence_before();
            fence_proxy_async();
            nb_arrive(kBarH, kNb); nb_arrive(kBarHt, kNb);
        }
        wait(&bar_o, (p.N - 1) & 1);
        tc_fence_after();
        o_stage(p.N - 1);
        if (p.hT && !s_abort) {
            float* dst = p.hT + (size_t)bh * D * D + (size_t)(32 * wg) * D + l;
#pragma unroll
            for (int i = 0; i < 32; ++i) dst[(size_t)i * D] = h[i];
        }
    } else if (warp == kMmaWarp) {
        // ---------------------------------- MMA-issue warp ----------------------------------
        const bool lead = (tid & 31) == 0;
        grid_dep_wait();
        grid_dep_launch();
        const uint32_t aH = smem_u32(sH), aD = smem_u32(sD), aDs = p.scaled ? smem_u32(sDs) : smem_u32(sD);
        for (int n = 0; n < p.N; ++n) {
            const uint32_t st = smem_u32(smem + (n & 1) * kStage);
            const uint32_t tO = tO0 + 64 * (n & 1);
            if (lead) wait(&bar_load[n & 1], (n >> 1) & 1);
            nb_sync(kBarH, kNb);                          // h^T operand of chunk n is in place
            if (lead) {
                tc_fence_after();
                // Delta-accumulator = h^T Wt (B: MN-major, lines = d_k)
                umma_product<false, true>(tD, aH, 16384, st, 8192, C, D, false);
                umma_commit(&bar_a);
                // O-accumulator = h^T Qg^T (B: K-major); it reads the state tile, so the commit behind the
                // H product below (which releases that tile) must cover it
                umma_product<false, false>(tO, aH, 16384, st + 32768, 8192, C, D, false);
            }
            nb_sync(kBarD, kNb);                          // Delta^T operands of chunk n are in place
            if (lead) {
                tc_fence_after();
                // H-accumulator = scaled Delta^T K (B: MN-major, lines = tokens)
                umma_product<false, true>(tH, aDs, 16384, st + 49152, 8192, D, C, false);
                umma_commit(&bar_b);
                // O-accumulator += Delta^T P^T (B: K-major [r][s])
                umma_product<false, false>(tO, aD, 16384, st + 65536, 8192, C, C, true);
                umma_commit(&bar_o);
                umma_commit(&bar_e);
            }
        }
        nb_sync(kBarH, kNb);                              // final arrival of the compute warps
    } else {
        // ---------------------------------- TMA warp ----------------------------------
        const bool lead = (tid & 31) == 0;
        grid_dep_wait();                  // the tiles and the log-decays read below are written by the prep kernel
        grid_dep_launch();
        auto issue_load = [&](int n) {
            unsigned char* st = smem + (n & 1) * kStage;
            uint64_t* bar = &bar_load[n & 1];
            mbar_expect_tx(bar, kStage);
            const int yc = (int)(((size_t)bh * p.N + n) * D);
            const int yt = (int)((size_t)bh * p.Tp + (size_t)n * C);
            tma_load_2d(st, &mapWt, 0, yc, bar);
            tma_load_2d(st + 16384, &mapUt, 0, yc, bar);
            tma_load_2d(st + 32768, &mapQg, 0, yt, bar);
            tma_load_2d(st + 32768 + 8192, &mapQg, 64, yt, bar);
            tma_load_3d(st + 49152, &mapK, hh * D, n * C, b, bar);
            tma_load_3d(st + 49152 + 8192, &mapK, hh * D + 64, n * C, b, bar);
            tma_load_2d(st + 65536, &mapP, 0, yt, bar);
        };
        if (lead) { issue_load(0); if (p.N > 1) issue_load(1); }
        const int ln = tid & 31;
        float g0 = gseq[ln], g1 = gseq[32 + ln], gc = gseq[C - 1];     // cumulative log-decays of chunk 0
        const float* rkseq = p.rk ? p.rk + (size_t)bh * p.Tp : nullptr;
        float r0 = rkseq ? rkseq[ln] : 1.f, r1 = rkseq ? rkseq[32 + ln] : 1.f;
        for (int n = 0; n < p.N; ++n) {
            sG[n & 1][ln] = __expf(gc - g0) * r0;
            sG[n & 1][32 + ln] = __expf(gc - g1) * r1;
            if (ln == 0) sG[n & 1][64] = __expf(gc);
            __syncwarp();
            if (n + 1 < p.N) {                                  // in flight while this chunk is processed
                const float* gn = gseq + (size_t)(n + 1) * C;
                g0 = gn[ln]; g1 = gn[32 + ln]; gc = gn[C - 1];
                if (rkseq) { r0 = rkseq[(size_t)(n + 1) * C + ln]; r1 = rkseq[(size_t)(n + 1) * C + 32 + ln]; }
            }
            if (lead) {
                // every store issued so far (Delta^T of chunk n-1, output of chunk n-2) has read its tile:
                // the Delta^T tiles may be rewritten (chunk n), the output staging tile too (chunk n-1)
                tma_store_wait_read_n<0>();
                mbar_arrive(&bar_a);
                if (n > 0) mbar_arrive(&bar_o);
            }
            nb_sync(kBarHt, kNb);                          // h^T operand of chunk n is in place
            if (lead && p.save) {
                // entry state of chunk n, bf16, exactly the operand tile: rows = d_v index, cols = d_k index
                const int yh = (int)(((size_t)bh * p.N + n) * D);
                tma_store_2d(&mapHs, sH, 0, yh);
                tma_store_2d(&mapHs, sH + 16384, 64, yh);
            }
            if (lead) tma_store_commit();                 // group: entry state of chunk n
            nb_sync(kBarDt, kNb);                          // Delta^T of chunk n is in place
            if (lead) {
                if (p.save) tma_store_2d(&mapDt, sD, 0, (int)(((size_t)bh * p.N + n) * D));
                tma_store_commit();                       // group: Delta^T of chunk n
                tma_store_wait_read_n<1>();               // the entry-state tile has been read: it may be rewritten
                mbar_arrive(&bar_b);
            }
            if (n > 0) {
                nb_sync(kBarO, kNb);                      // output tile of chunk n-1 staged
                if (lead) {
                    tma_store_3d(&mapO, sO, hh * D, (n - 1) * C, b);      // rows past the end of the sequence are skipped
                    tma_store_3d(&mapO, sO + 8192, hh * D + 64, (n - 1) * C, b);
                    tma_store_commit();                   // group: output of chunk n-1
                }
            }
            if (lead) {
                wait(&bar_e, n & 1);                      // every product of chunk n has finished: refill its stage
                if (n + 2 < p.N && !s_abort) issue_load(n + 2);
            }
        }
        nb_sync(kBarHt, kNb);                              // final arrival of the compute warps
        if (lead) { tma_store_wait_read_n<0>(); mbar_arrive(&bar_o); }
        nb_sync(kBarO, kNb);                              // output tile of the last chunk staged
        if (lead) {
            tma_store_3d(&mapO, sO, hh * D, (p.N - 1) * C, b);
            tma_store_3d(&mapO, sO + 8192, hh * D + 64, (p.N - 1) * C, b);
            tma_store_commit();
            tma_store_wait_all();
            if (s_abort) { mbar_wait(&bar_load[0], 0); mbar_wait(&bar_load[1], 0); }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (tid < 32) tmem_dealloc(tbase, 512);
}

template <class K>
cudaError_t set_smem(K kern, size_t bytes) { return set_max_smem_once(reinterpret_cast<const void*>(kern), bytes); }

}  // namespace

bool tc_supported(const qd_shape& s) {
    return s.dtype == QD_BF16 && s.dk == 128 && s.dv == 128 && s.chunk == kChunk &&
           (long long)s.B * s.H * tc_padded_T(s) * 128 < 0x7fffffffLL * 64;
}

TcLayout tc_layout(const qd_shape& s) {
    TcLayout L{};
    const size_t BH = (size_t)s.B * s.H, T = (size_t)tc_padded_T(s);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = (off + bytes + 1023) & ~(size_t)1023; return o; };
    L.status = take(256);
    L.g = take(BH * T * 4);
    L.Qg = take(BH * T * s.dk * 2);
    L.P = take(BH * T * kChunk * 2);
    L.Wt = take(BH * T * s.dk * 2);
    L.Ut = take(BH * T * s.dv * 2);
    L.rqk = take(2 * BH * T * 4);
    L.fwd_end = off;
    const size_t N = T / kChunk;
    L.Mt = take(BH * T * kChunk * 2);
    L.hsT = take(BH * N * s.dk * s.dv * 2);
    L.Dt = take(BH * T * s.dv * 2);
    L.dhsT = take(BH * N * s.dk * s.dv * 2);
    L.dDt = take(BH * T * s.dv * 2);
    L.bwd_end = off;
    return L;
}

cudaError_t tc_prep(const ChunkArgs& a) {
    const qd_shape& s = a.s;
    CUtensorMap mQ, mK, mV, mUt, mWt;
    const int Tp = tc_padded_T(s);
    const uint64_t trows = (uint64_t)s.B * s.H * (Tp / kChunk) * D;          // rows of the [chunk][d][64] tiles
    if (!make_tmap_tokens(&mQ, a.q, s.B, s.T, s.H, D, 128) || !make_tmap_tokens(&mK, a.k, s.B, s.T, s.H, D, 128) ||
        !make_tmap_tokens(&mV, a.v, s.B, s.T, s.H, D, 128) ||
        !make_tmap_bf16_2d(&mUt, a.ws + a.TL.Ut, 64, trows, 128, 128) ||
        !make_tmap_bf16_2d(&mWt, a.ws + a.TL.Wt, 64, trows, 128, 128))
        return cudaErrorInvalidValue;
    PrepParams p{};
    p.T = s.T; p.Tp = Tp; p.H = s.H; p.N = Tp / kChunk; p.BH = s.B * s.H;
    p.rqk = a.norm ? (float*)(a.ws + a.TL.rqk) : nullptr;
    p.beta = (const bf16*)a.beta; p.alpha = (const bf16*)a.alpha; p.lam = (const bf16*)a.lam;
    p.g = (float*)(a.ws + a.TL.g);
    p.Qg = (bf16*)(a.ws + a.TL.Qg); p.P = (bf16*)(a.ws + a.TL.P);
    p.Mt = a.save ? (bf16*)(a.ws + a.TL.Mt) : nullptr;
    p.status = (unsigned*)(a.ws + a.TL.status);
    auto kern = a.norm ? (a.logits ? k_tc_prep<true, true> : k_tc_prep<true, false>)
                       : (a.logits ? k_tc_prep<false, true> : k_tc_prep<false, false>);
    cudaError_t e = set_smem(kern, kPrepSmem);
    if (e != cudaSuccess) return e;
    const int grid = s.B * s.H * (p.N / 2);
    kern<<<grid, kPrepThreads, kPrepSmem, a.stream>>>(mQ, mK, mV, mUt, mWt, p);
    return cudaGetLastError();
}

cudaError_t tc_chain_fwd(const ChunkArgs& a) {
    const qd_shape& s = a.s;
    const int Tp = tc_padded_T(s);
    const uint64_t BH = (uint64_t)s.B * s.H, N = Tp / kChunk;
    CUtensorMap mWt, mUt, mQg, mK, mP, mHs, mDt, mO;
    if (!make_tmap_bf16_2d(&mHs, a.ws + a.TL.hsT, D, BH * N * D, D * 2, 128) ||
        !make_tmap_bf16_2d(&mDt, a.ws + a.TL.Dt, 64, BH * N * D, 128, 128) ||
        !make_tmap_tokens(&mO, a.o, s.B, s.T, s.H, D, 64) ||
        !make_tmap_bf16_2d(&mWt, a.ws + a.TL.Wt, 64, BH * N * D, 128, 128) ||
        !make_tmap_bf16_2d(&mUt, a.ws + a.TL.Ut, 64, BH * N * D, 128, 128) ||
        !make_tmap_bf16_2d(&mQg, a.ws + a.TL.Qg, D, BH * Tp, D * 2, 64) ||
        !make_tmap_tokens(&mK, a.k, s.B, s.T, s.H, D, 64) ||
        !make_tmap_bf16_2d(&mP, a.ws + a.TL.P, 64, BH * Tp, 128, 64))
        return cudaErrorInvalidValue;
    ChainParams p{};
    p.Tp = Tp; p.H = s.H; p.N = (int)N;
    p.g = (const float*)(a.ws + a.TL.g);
    p.h0 = a.h0; p.hT = a.hT;
    p.save = a.save ? 1 : 0;
    p.scaled = (a.alpha || a.norm) ? 1 : 0;
    p.rk = a.norm ? (const float*)(a.ws + a.TL.rqk) + BH * Tp : nullptr;
    p.status = (unsigned*)(a.ws + a.TL.status);
    cudaError_t e = set_smem(k_tc_chain_fwd, kChainSmem);
    if (e != cudaSuccess) return e;
    return launch_overlapped(k_tc_chain_fwd, dim3((unsigned)BH), dim3(kChainThreads), kChainSmem, a.stream,
                             mWt, mUt, mQg, mK, mP, mHs, mDt, mO, p);
}

}  // namespace qd
