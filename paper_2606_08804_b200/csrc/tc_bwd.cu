// Tensor-core (tcgen05 / TMEM / TMA) chunkwise backward for bf16, d_k = d_v = 128, chunk 64.
//
// The paper prints no backward pass; these kernels evaluate the exact gradient of the chunk
// equations of Section 3.3.2 (see the forward kernels for the notation):
//   k_tc_chain_bwd  one CTA per (batch, head), chunks in REVERSE order, dh^T (fp32) in registers:
//                     dDelta^T = dO^T P + diag-scaled (dh^T K^T)          (scale gamma_C/gamma_s per token s)
//                     dh^T <- gamma_C dh^T + dO^T Qg - dDelta^T W<-
//                   leaves per chunk dDelta^T and the bf16 dh^T at the chunk's exit.
//   k_tc_chunk_bwd  one CTA per chunk: every remaining product (dP, dT, dA = -M^T dM M^T, dX, ...),
//                   d_k/d_v-shaped results transposed (d index on the 128 TMEM lanes), 64 x 64-shaped
//                   ones in natural orientation on lanes 0..63; row dot-products that run across lanes
//                   use a warp-shuffle column reduction.
// All waits are bounded (see tc_fwd.cu).
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

// One halving step of a column sum across the lanes of a warp: lanes whose `off` bit is set keep the upper half
// of the N values, the others the lower half; each adds what its partner sends.
template <int N>
__device__ __forceinline__ void fold(float* v, int lane, int off) {
    const bool up = (lane & off) != 0;
#pragma unroll
    for (int k = 0; k < N / 2; ++k) {
        const float keep = up ? v[N / 2 + k] : v[k];
        const float send = up ? v[k] : v[N / 2 + k];
        v[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
}

// =================================================================================================
struct ChainBwdParams {
    int Tp, H, N;              // Tp = 64 N rows per sequence in the workspace
    int dhT_early;             // the kernel before this one in the stream is the library's own: dhT is older than it
    const float* rk;           // non-null (QD_NORM_QK): 1/|k_t| per workspace row, folded into the per-token scale
    const float* g;
    const float* dhT;
    float* dh0;
    unsigned* status;
};

constexpr int kStage = 73728;                           // Wt 16K | dO 16K | Qg 16K | K 16K | P 8K
constexpr int kChainSmem = 2 * kStage + 32768 + 16384 + 1024;
constexpr int kChainCompute = 512;                 // 16 epilogue warps: 4 warpgroups split the accumulator columns
constexpr int kChainThreads = kChainCompute + 64;  // + 1 MMA-issue warp, 1 TMA warp
constexpr int kMmaWarp = kChainCompute / 32;
constexpr int kNb = kChainCompute + 32;            // participants of a named barrier: the epilogue threads and one waiting warp

// named barriers: compute threads arrive, the MMA and TMA warps wait
constexpr int kBarH = 1, kBarD = 2, kBarHt = 4, kBarDt = 5;   // ..t: the same event, awaited by the TMA warp
__device__ __forceinline__ void nb_arrive(int id, int count) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void nb_sync(int id, int count) {
    __syncwarp();                                   // the lanes of a warp reach the barrier together
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// Reverse state chain.  Per chunk the dependency is
//   dh ready -> A2 = dh^T K^T -> dDelta^T -> H-accumulator -= dDelta^T W<- -> dh update;
// A1 = dO^T P and the dO^T Qg part of the H-accumulator do not depend on dh; every TMA copy is
// issued by its own warp.
// Compute warpgroup w owns tokens [32w, 32w+32) of the 64-column accumulators and d_k columns
// [64w, 64w+64) of dh^T; thread l of a warpgroup owns TMEM lane l = d_v index.
__global__ void __launch_bounds__(kChainThreads) k_tc_chain_bwd(const __grid_constant__ CUtensorMap mapWt,
                                                                const __grid_constant__ CUtensorMap mapdO,
                                                                const __grid_constant__ CUtensorMap mapQg,
                                                                const __grid_constant__ CUtensorMap mapK,
                                                                const __grid_constant__ CUtensorMap mapP,
                                                                const __grid_constant__ CUtensorMap mapdHs,
                                                                const __grid_constant__ CUtensorMap mapdDt,
                                                                ChainBwdParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* sdH = smem + 2 * kStage;         // dh^T as A operand: K-major, 2 blocks of [128 lines][64]
    unsigned char* sdD = sdH + 32768;               // dDelta^T: K-major [128 lines (dv)][64 tokens]
    __shared__ uint64_t bar_load[2], bar_a, bar_b, bar_e;
    __shared__ uint32_t tmem_slot;
    __shared__ volatile int s_abort;
    // per iteration parity: gamma_C / gamma_t for the 64 tokens, then gamma_C; written by the TMA warp one chunk
    // ahead and published with its arrival on bar_a
    __shared__ __align__(16) float sG[2][68];

    const int tid = threadIdx.x, warp = tid >> 5, wg = tid >> 7, l = tid & 127, wq = warp & 3;
    const int bh = blockIdx.x, b = bh / p.H, hh = bh % p.H;

    if (tid == 0) {
        mbar_init(&bar_load[0], 1); mbar_init(&bar_load[1], 1);
        mbar_init(&bar_a, 2); mbar_init(&bar_b, 2); mbar_init(&bar_e, 1);
        mbar_init_fence();
        s_abort = 0;
    }
    if (tid < 32) { tmem_alloc(&tmem_slot, 256); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = tmem_slot;
    const uint32_t tA1 = tbase, tA2 = tbase + 64, tH = tbase + 128;
    const uint32_t lane_base = (uint32_t)wq * 32;

    // bounded wait; once any wait has expired every later wait returns at once (the kernel drains)
    auto wait = [&](uint64_t* bar, uint32_t parity) {
        if (s_abort) return;
        if (!mbar_wait(bar, parity)) { s_abort = 1; *p.status = QD_ERR_TIMEOUT; }
    };
    const float* gseq = p.g + (size_t)bh * p.Tp;

    if (warp < kMmaWarp) {
        // ---------------------------------- compute warps ----------------------------------
        float dh[32];     // dh^T[j = l][32 wg .. 32 wg + 31]
        // dhT is an input of the call.  When the kernel before this one is the library's own forward chain, dhT is older
        // than that kernel and may be read while it drains; otherwise the predecessor may be the very kernel that wrote
        // dhT, whose writes are only guaranteed visible after the wait.
        if (!p.dhT_early) grid_dep_wait();
        if (p.dhT) {
            const float* src = p.dhT + (size_t)bh * D * D + (size_t)(32 * wg) * D + l;
#pragma unroll
            for (int i = 0; i < 32; ++i) dh[i] = src[(size_t)i * D];
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) dh[i] = 0.f;
        }
        if (p.dhT_early) grid_dep_wait();  // the loads of dhT are in flight; everything below depends on earlier kernels
        grid_dep_launch();
        // my 32 columns of the operand tile: 64-column block wg >> 1, 16-byte chunks 4 (wg & 1) ..
        unsigned char* myH = sdH + (wg >> 1) * 16384;
        const int hc0 = (wg & 1) * 4;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) sts128(myH + sw128_chunk(l, hc0 + ch), pack8(dh + ch * 8));
        fence_proxy_async();
        nb_arrive(kBarH, kNb); nb_arrive(kBarHt, kNb);

        for (int it = 0; it < p.N; ++it) {
            wait(&bar_a, it & 1);
            tc_fence_after();
            float sc[16];
            {
                const float4* gp = reinterpret_cast<const float4*>(&sG[it & 1][wg * 16]);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float4 t = gp[q];
                    sc[q * 4] = t.x; sc[q * 4 + 1] = t.y; sc[q * 4 + 2] = t.z; sc[q * 4 + 3] = t.w;
                }
            }
            const float gamC = sG[it & 1][64];
            // dDelta^T = A1 + gamma_C/gamma_s A2, my 16 tokens
            {
                float a1[16], a2[16];
                tmem_ld16(tmem_addr(tA1, lane_base, wg * 16), a1);
                tmem_ld16(tmem_addr(tA2, lane_base, wg * 16), a2);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 16; ++i) a1[i] = fmaf(sc[i], a2[i], a1[i]);
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) sts128(sdD + sw128_chunk(l, wg * 2 + cc), pack8(a1 + cc * 8));
            }
            tc_fence_before();
            fence_proxy_async();
            nb_arrive(kBarD, kNb); nb_arrive(kBarDt, kNb);
            wait(&bar_b, it & 1);
            tc_fence_after();
            {
                float v[32];
                tmem_ld32(tmem_addr(tH, lane_base, wg * 32), v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) dh[i] = fmaf(gamC, dh[i], v[i]);
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) sts128(myH + sw128_chunk(l, hc0 + cc), pack8(dh + cc * 8));
            }
            tc_fence_before();
            fence_proxy_async();
            nb_arrive(kBarH, kNb); nb_arrive(kBarHt, kNb);
        }
        if (p.dh0 && !s_abort) {
            float* dst = p.dh0 + (size_t)bh * D * D + (size_t)(32 * wg) * D + l;
#pragma unroll
            for (int i = 0; i < 32; ++i) dst[(size_t)i * D] = dh[i];
        }
    } else if (warp == kMmaWarp) {
        // ---------------------------------- MMA-issue warp ----------------------------------
        const bool lead = (tid & 31) == 0;
        grid_dep_wait();
        grid_dep_launch();
        const uint32_t adH = smem_u32(sdH), adD = smem_u32(sdD);
        for (int it = 0; it < p.N; ++it) {
            const uint32_t st = smem_u32(smem + (it & 1) * kStage);
            if (lead) wait(&bar_load[it & 1], (it >> 1) & 1);
            nb_sync(kBarH, kNb);                          // dh^T operand (exit state of this chunk) is in place
            if (lead) {
                tc_fence_after();
                const uint32_t sdO = st + 16384;
                // A2 = dh^T K^T (A, B K-major) -- the critical product;  A1 = dO^T P (A, B MN-major: lines = token r)
                umma_product<false, false>(tA2, adH, 16384, st + 49152, 8192, C, D, false);
                umma_product<true, true>(tA1, sdO, 8192, st + 65536, 8192, C, C, false);
                umma_commit(&bar_a);
                // H-accumulator = dO^T Qg (B MN-major: lines = token r, two blocks of d_k)
                umma_product<true, true>(tH, sdO, 8192, st + 32768, 8192, D, C, false);
            }
            nb_sync(kBarD, kNb);                          // dDelta^T operand is in place
            if (lead) {
                tc_fence_after();
                // H-accumulator -= dDelta^T W<-   (A negated; B K-major: lines = d_k index, contraction over tokens)
                umma_product<false, false>(tH, adD, 16384, st, 16384, D, C, true, true);
                umma_commit(&bar_b);
                umma_commit(&bar_e);
            }
        }
        nb_sync(kBarH, kNb);                              // final arrival of the compute warps
    } else {
        // ---------------------------------- TMA warp ----------------------------------
        const bool lead = (tid & 31) == 0;
        grid_dep_wait();
        grid_dep_launch();
        // iteration `it` processes chunk n = N-1-it
        auto issue_load = [&](int it) {
            const int n = p.N - 1 - it;
            unsigned char* st = smem + (it & 1) * kStage;
            uint64_t* bar = &bar_load[it & 1];
            mbar_expect_tx(bar, kStage);
            const int yc = (int)(((size_t)bh * p.N + n) * D);
            const int yt = (int)((size_t)bh * p.Tp + (size_t)n * C);
            tma_load_2d(st, &mapWt, 0, yc, bar);
            tma_load_3d(st + 16384, &mapdO, hh * D, n * C, b, bar);          // rows past the end of the sequence: zeros
            tma_load_3d(st + 16384 + 8192, &mapdO, hh * D + 64, n * C, b, bar);
            tma_load_2d(st + 32768, &mapQg, 0, yt, bar);
            tma_load_2d(st + 32768 + 8192, &mapQg, 64, yt, bar);
            tma_load_3d(st + 49152, &mapK, hh * D, n * C, b, bar);
            tma_load_3d(st + 49152 + 8192, &mapK, hh * D + 64, n * C, b, bar);
            tma_load_2d(st + 65536, &mapP, 0, yt, bar);
        };
        if (lead) { issue_load(0); if (p.N > 1) issue_load(1); }
        const int ln = tid & 31;
        const float* gl = gseq + (size_t)(p.N - 1) * C;               // cumulative log-decays of the last chunk
        float g0 = gl[ln], g1 = gl[32 + ln], gc = gl[C - 1];
        const float* rkseq = p.rk ? p.rk + (size_t)bh * p.Tp : nullptr;
        float r0 = rkseq ? rkseq[(size_t)(p.N - 1) * C + ln] : 1.f, r1 = rkseq ? rkseq[(size_t)(p.N - 1) * C + 32 + ln] : 1.f;
        for (int it = 0; it < p.N; ++it) {
            const int n = p.N - 1 - it;
            sG[it & 1][ln] = __expf(gc - g0) * r0;
            sG[it & 1][32 + ln] = __expf(gc - g1) * r1;
            if (ln == 0) sG[it & 1][64] = __expf(gc);
            __syncwarp();
            if (n > 0) {                                      // in flight while this chunk is processed
                const float* gn = gseq + (size_t)(n - 1) * C;
                g0 = gn[ln]; g1 = gn[32 + ln]; gc = gn[C - 1];
                if (rkseq) { r0 = rkseq[(size_t)(n - 1) * C + ln]; r1 = rkseq[(size_t)(n - 1) * C + 32 + ln]; }
            }
            if (lead) {
                tma_store_wait_read_n<0>();               // dDelta^T tile of the previous chunk has been read
                mbar_arrive(&bar_a);
            }
            nb_sync(kBarHt, kNb);                          // dh^T operand (exit state of chunk n) is in place
            if (lead) {
                // gradient w.r.t. the exit state of chunk n, bf16, as the operand tile (rows = d_v, cols = d_k)
                const int yh = (int)(((size_t)bh * p.N + n) * D);
                tma_store_2d(&mapdHs, sdH, 0, yh);
                tma_store_2d(&mapdHs, sdH + 16384, 64, yh);
                tma_store_commit();
            }
            nb_sync(kBarDt, kNb);                          // dDelta^T of chunk n is in place
            if (lead) {
                tma_store_2d(&mapdDt, sdD, 0, (int)(((size_t)bh * p.N + n) * D));
                tma_store_commit();
                tma_store_wait_read_n<1>();               // the dh^T tile has been read: it may be rewritten
                mbar_arrive(&bar_b);
                wait(&bar_e, it & 1);                     // every product of this chunk has finished: refill its stage
                if (it + 2 < p.N && !s_abort) issue_load(it + 2);
            }
        }
        nb_sync(kBarHt, kNb);                              // final arrival of the compute warps
        if (lead) {
            tma_store_wait_all();
            if (s_abort) { mbar_wait(&bar_load[0], 0); mbar_wait(&bar_load[1], 0); }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (tid < 32) tmem_dealloc(tbase, 256);
}

// =================================================================================================
struct ChunkBwdParams {
    int logits;                // beta, alpha, lambda are logits of sigmoid gates; their gradients are taken w.r.t. the logits
    const float* rqk;          // QD_NORM_QK: 1/|q_t| per workspace row, then (BH*Tp further) 1/|k_t|
    int group;                 // GROUPED instances: sequences per group of work items
    int T, Tp, H, N, BH, total;   // T tokens per sequence, Tp = 64 N rows per sequence in the workspace; total = BH*N chunks
    const bf16 *beta, *alpha, *lam;
    const float* g;
    float *dbeta, *dalpha, *dlam;
    unsigned* status;
};

// shared-memory map of k_tc_chunk_bwd (bytes from the 1024-aligned base)
constexpr int oQ = 0, oK = 16384, oV = 32768, odO = 49152, oX = 65536, oMt = 81920, oP = 90112, oDt = 98304,
              odDt = 114688, oH = 131072, odH = 163840;                            // TMA-loaded tiles (X is built)
constexpr int kBwdEarlyBytes = 2 * 16384 + 2 * 8192;
// tiles built later reuse regions whose contents are dead by then
constexpr int odPG = oV, odTb = oV + 8192, odW = 196608, oN = oH, odXK = oH + 8192, oPP = oH + 16384,
              oAA = odH + 1024, oStDv = odDt, oStDk = oDt, oStDq = odDt;
constexpr int kBwdSmem = 196608 + 16384 + 1024;      // + the dW<-^T tile, written while dO is still an operand
constexpr int LDAA = C + 1;
constexpr int kNWG = 4;                       // warpgroups; each owns 64/kNWG columns of every 64-column accumulator
constexpr int kCW = C / kNWG, kG8 = kCW / 8;    // columns per warpgroup, groups of 8 columns
constexpr int kBwdCompute = 128 * kNWG;                 // epilogue threads
constexpr int kBwdThreads = kBwdCompute + 32;            // + one warp that issues every TMA copy and every MMA
// named barriers of k_tc_chunk_bwd: 1 = the epilogue threads among themselves; the others are raised by the
// epilogue threads (bar.arrive) when an operand tile is complete and awaited by the issuing warp (bar.sync)
constexpr int kNbC = 1, kNbX = 2, kNbDW = 3, kNbDTb = 4, kNbN = 5, kNbDXK = 6, kNbOut = 7, kNbDV = 8, kNbScr = 9;

// Column sums across the 32 lanes of a warp for 8 columns: returns, in every lane, the warp-wide sum of
// column col8_of_lane(lane) (four lanes hold each column).
__device__ __forceinline__ float col_reduce8(float* v, int lane) {
    fold<8>(v, lane, 16); fold<4>(v, lane, 8); fold<2>(v, lane, 4);
    float x = v[0];
    x += __shfl_xor_sync(0xffffffffu, x, 2);
    x += __shfl_xor_sync(0xffffffffu, x, 1);
    return x;
}
__device__ __forceinline__ int col8_of_lane(int lane) { return ((lane & 16) ? 4 : 0) + ((lane & 8) ? 2 : 0) + ((lane & 4) ? 1 : 0); }
// 8 TMEM columns of this thread's lane (no wait)
__device__ __forceinline__ void ld8(uint32_t taddr, float* v) { tmem_ld8(taddr, v); }

// Two warpgroups: warpgroup w (threads 128w..128w+127) owns TMEM columns [32w, 32w+32) of every
// 64-column accumulator; inside a warpgroup thread l owns TMEM lane l.
// HAS_LAM = false: lambda is absent and d lambda is not asked for (the gated delta rule, Eq. 3): X = K, nothing is built,
// no column sum for d lambda.  HAS_ALPHA = false: alpha is absent and d alpha is not asked for (no forget gate; with
// HAS_LAM = false too this is DeltaNet, Eq. 2): every decay factor is 1 and none of the sums that only feed d alpha is
// taken.  The <true, true> instances serve every other case (an absent input then reads as lambda = 0, alpha = 1).
// NORM (QD_NORM_QK): the Q and K tiles arrive un-normalised and are normalised in place with the factors the forward
// left in the workspace; dq and dk are taken through the normalisation, dx = r (dx^ - x^ <x^, dx^>), which needs the
// row sums <x^, dx^> before anything can be stored: the last epilogue then runs twice, once for the sums and once
// for the stores.
template <bool HAS_LAM, bool HAS_ALPHA, bool NORM, bool GROUPED>
__global__ void __launch_bounds__(kBwdThreads) k_tc_chunk_bwd(const __grid_constant__ CUtensorMap mapQ,
                                                              const __grid_constant__ CUtensorMap mapK,
                                                              const __grid_constant__ CUtensorMap mapV,
                                                              const __grid_constant__ CUtensorMap mapdO,
                                                              const __grid_constant__ CUtensorMap mapMt,
                                                              const __grid_constant__ CUtensorMap mapP,
                                                              const __grid_constant__ CUtensorMap mapDt,
                                                              const __grid_constant__ CUtensorMap mapdDt,
                                                              const __grid_constant__ CUtensorMap mapHs,
                                                              const __grid_constant__ CUtensorMap mapdHs,
                                                              const __grid_constant__ CUtensorMap mapdQ,
                                                              const __grid_constant__ CUtensorMap mapdK,
                                                              const __grid_constant__ CUtensorMap mapdV,
                                                              ChunkBwdParams p) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar_load, bar_late, bm_a, bm_b, bm_c, bm_2, bm_3, bm_4, bm_5;
    __shared__ uint32_t tmem_slot;
    __shared__ volatile int s_abort, s_latch;
    __shared__ float sbeta[C], slam[C], salpha[C], sg[C], sgam[C];
    __shared__ float4 scf[C];         // per token: {gamma beta, gamma_C / gamma, gamma, lambda}, one load in the last epilogue
    __shared__ float sred[3][4][C];   // per-warp column sums: [0] <(K-> dh)_r, Delta_r>, [1] d lambda, [2] rowsum(dQ1 o Q)
    __shared__ float2 srn[C];          // NORM: {1/|k_t|, 1/|q_t|}
    __shared__ __align__(16) float srow[6][kNWG][C];   // per-row partial sums over each warpgroup's columns: rPP, d beta, t2, rAA; [4], [5]: d beta and
                                         // rAA of the column groups that the upper lanes take
    __shared__ float sdg[C], skd[C], swp[kBwdCompute / 32], scol[2][kBwdCompute / 64][C];

    const int tid = threadIdx.x, wg = tid >> 7, l = tid & 127, lane = tid & 31, wq = (tid >> 5) & 3;
    const int c0 = wg * kCW;                                      // my columns of a 64-column accumulator

    if (tid == 0) {
        mbar_init(&bar_load, 1);
        mbar_init(&bar_late, 1);
        mbar_init(&bm_a, 1); mbar_init(&bm_b, 1); mbar_init(&bm_c, 1); mbar_init(&bm_2, 1); mbar_init(&bm_3, 1); mbar_init(&bm_4, 1);
        mbar_init(&bm_5, 2);              // the products' completion and "the dv staging tile has been read"
        mbar_init_fence();
        s_abort = 0;
        s_latch = 0;
    }
    if (tid < 32) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_slot;
    const uint32_t T0 = tb, T1 = tb + 64, T2 = tb + 128, T3 = tb + 192, T4 = tb + 256, T5 = tb + 320, T6 = tb + 384,
                   T7 = tb + 448;
    const uint32_t lane_base = (uint32_t)wq * 32;
    auto my = [&](uint32_t t) { return tmem_addr(t, lane_base, (uint32_t)c0); };

    // The tiles of a chunk arrive in two groups.  "early": V, dO, M^T, P -- their regions are dead once the
    // last products of the previous chunk have finished; "late": Q, Delta^T, dDelta^T, h^T, dh^T -- regions
    // that the previous chunk uses up to its end (staging tiles of the stores, scratch of the reductions).
    // Work item `ch` is chunk n_ of sequence bh_.  GROUPED = false: sequence-major numbering.  GROUPED = true: items are
    // numbered in groups of p.group sequences, chunk-major inside a group, so that at any time the CTAs of the grid work
    // on a few chunk indices of p.group sequences instead of on ~148 consecutive chunks of one long sequence.  Measured,
    // sequence-major against groups of 32: 0.330 / 0.316 ms on 32 sequences of 128 chunks, 0.347 / 0.320 on 16 of 256,
    // 1.47 / 1.18 on 32 of 512, no gain on 128 sequences of 32 chunks; all sequences at a time (chunk-major) was the
    // slowest there.  Compile-time, because the kernel's code generation is at a knife's edge: the grouped arithmetic
    // compiled into the sequence-major path cost it 3.5 %, as a non-inlined function 14 %.
    auto item = [&](int ch, int& n_, int& bh_) {
        if (GROUPED) {
            const int per = p.group * p.N, grp = ch / per, r = ch - grp * per;
            const int g0 = grp * p.group, gs = min(p.group, p.BH - g0);       // the last group may be smaller
            n_ = r / gs;
            bh_ = g0 + r - n_ * gs;
        } else {
            bh_ = ch / p.N;
            n_ = ch - bh_ * p.N;
        }
    };
    auto issue_early = [&](int ch) {
        int n_, bh_; item(ch, n_, bh_);
        const int b_ = bh_ / p.H, hh_ = bh_ % p.H;
        const int yt = (int)((size_t)bh_ * p.Tp + (size_t)n_ * C);
        mbar_expect_tx(&bar_load, kBwdEarlyBytes);
        for (int blk = 0; blk < 2; ++blk) {       // token rows past the end of the sequence arrive as zeros
            tma_load_3d(sm + oV + blk * 8192, &mapV, hh_ * D + blk * 64, n_ * C, b_, &bar_load);
            tma_load_3d(sm + odO + blk * 8192, &mapdO, hh_ * D + blk * 64, n_ * C, b_, &bar_load);
        }
        tma_load_2d(sm + oMt, &mapMt, 0, yt, &bar_load);
        tma_load_2d(sm + oP, &mapP, 0, yt, &bar_load);
    };
    // The late group goes in three batches as its regions fall free: part 0 = Q, K (after the last epilogue),
    // part 1 = h^T, dh^T (after the last products and the column sums have read the scratch that aliases them), part 2 = Delta^T,
    // dDelta^T (after the stores have read the staging tiles).  Only the last batch arrives on the barrier.
    auto issue_late = [&](int ch, int part) {
        int n_, bh_; item(ch, n_, bh_);
        const int b_ = bh_ / p.H, hh_ = bh_ % p.H;
        const int yc = (int)(((size_t)bh_ * p.N + n_) * D);
        if (part == 0) {
            mbar_expect_tx_only(&bar_late, 2 * 16384);
            for (int blk = 0; blk < 2; ++blk) {
                tma_load_3d(sm + oQ + blk * 8192, &mapQ, hh_ * D + blk * 64, n_ * C, b_, &bar_late);
                tma_load_3d(sm + oK + blk * 8192, &mapK, hh_ * D + blk * 64, n_ * C, b_, &bar_late);
            }
        } else if (part == 1) {
            mbar_expect_tx_only(&bar_late, 2 * 32768);
            for (int blk = 0; blk < 2; ++blk) {
                tma_load_2d(sm + oH + blk * 16384, &mapHs, blk * 64, yc, &bar_late);
                tma_load_2d(sm + odH + blk * 16384, &mapdHs, blk * 64, yc, &bar_late);
            }
        } else {
            mbar_expect_tx(&bar_late, 2 * 16384);
            tma_load_2d(sm + oDt, &mapDt, 0, yc, &bar_late);
            tma_load_2d(sm + odDt, &mapdDt, 0, yc, &bar_late);
        }
    };
    // the late group of a chunk into L2 only, issued a chunk time before its load: the load, which can only be
    // issued at the very end of the previous chunk and is waited for at once, then finds the tiles in L2
    auto prefetch_late = [&](int ch) {
        int n_, bh_; item(ch, n_, bh_);
        const int b_ = bh_ / p.H, hh_ = bh_ % p.H;
        const int yc = (int)(((size_t)bh_ * p.N + n_) * D);
        for (int blk = 0; blk < 2; ++blk) {
            tma_prefetch_3d(&mapQ, hh_ * D + blk * 64, n_ * C, b_);
            tma_prefetch_3d(&mapK, hh_ * D + blk * 64, n_ * C, b_);
            tma_prefetch_2d(&mapHs, blk * 64, yc);
            tma_prefetch_2d(&mapdHs, blk * 64, yc);
        }
        tma_prefetch_2d(&mapDt, 0, yc);
        tma_prefetch_2d(&mapdDt, 0, yc);
    };
    // coefficients of token tid (< C) of a chunk, fetched one chunk ahead into registers
    float cf_beta = 0.f, cf_lam = 0.f, cf_alpha = 1.f, cf_g = 0.f, cf_rq = 1.f, cf_rk = 1.f;
    auto fetch_coef = [&](int ch) {
        if (tid < C) {
            int n_, bh_; item(ch, n_, bh_);
            const int b_ = bh_ / p.H, hh_ = bh_ % p.H;
            const bool live = n_ * C + tid < p.T;             // tokens past the end of the sequence: beta = 0, alpha = 1
            const size_t cr = ((size_t)b_ * p.T + (size_t)n_ * C + tid) * p.H + hh_;
            cf_beta = live ? gate(__bfloat162float(p.beta[cr]), p.logits) : 0.f;
            cf_lam = (live && p.lam) ? gate(__bfloat162float(p.lam[cr]), p.logits) : 0.f;
            cf_alpha = (live && p.alpha) ? gate(__bfloat162float(p.alpha[cr]), p.logits) : 1.f;
            cf_g = p.g[(size_t)bh_ * p.Tp + (size_t)n_ * C + tid];
            if (NORM) {
                cf_rq = p.rqk[(size_t)bh_ * p.Tp + (size_t)n_ * C + tid];
                cf_rk = p.rqk[(size_t)p.BH * p.Tp + (size_t)bh_ * p.Tp + (size_t)n_ * C + tid];
            }
        }
    };
    // bounded wait; once any wait has expired every later wait returns at once and the kernel drains: all
    // threads still pass every barrier, results are garbage, the status word says so
    auto wait = [&](uint64_t* bar, uint32_t parity) {
        if (s_abort) return;
        if (!mbar_wait(bar, parity)) { s_abort = 1; *p.status = QD_ERR_TIMEOUT; }
    };
    const uint32_t aQ = smem_u32(sm + oQ), aK = smem_u32(sm + oK), aV = smem_u32(sm + oV), adO = smem_u32(sm + odO),
                   aX = smem_u32(sm + oX), aMt = smem_u32(sm + oMt), aDt = smem_u32(sm + oDt),
                   adDt = smem_u32(sm + odDt), aH = smem_u32(sm + oH), adH = smem_u32(sm + odH);
    const uint32_t adPG = smem_u32(sm + odPG), adTb = smem_u32(sm + odTb), adW = smem_u32(sm + odW),
                   aN = smem_u32(sm + oN), adXK = smem_u32(sm + odXK);
    constexpr bool has_lam = HAS_LAM, has_alpha = HAS_ALPHA, want_dl = HAS_LAM, want_da = HAS_ALPHA;
    const uint32_t aXe = has_lam ? aX : aK;

    if (tid >= kBwdCompute) {
        // =============================== issuing warp: TMA copies and MMAs ===============================
        const bool lead = lane == 0;
        if (lead && (int)blockIdx.x < p.total) {
            // first chunk: everything that the reverse chain (the kernel before this one) does not write is fetched
            // before waiting for it -- inputs, and tiles of kernels that had finished before the reverse chain began
            const int ch = blockIdx.x;
            int n_, bh_; item(ch, n_, bh_);
            const int yc = (int)(((size_t)bh_ * p.N + n_) * D);
            issue_early(ch);
            issue_late(ch, 0);
            mbar_expect_tx_only(&bar_late, 32768 + 16384);
            for (int blk = 0; blk < 2; ++blk) tma_load_2d(sm + oH + blk * 16384, &mapHs, blk * 64, yc, &bar_late);
            tma_load_2d(sm + oDt, &mapDt, 0, yc, &bar_late);
            grid_dep_wait();
            mbar_expect_tx(&bar_late, 32768 + 16384);
            for (int blk = 0; blk < 2; ++blk) tma_load_2d(sm + odH + blk * 16384, &mapdHs, blk * 64, yc, &bar_late);
            tma_load_2d(sm + odDt, &mapdDt, 0, yc, &bar_late);
        }
        grid_dep_wait();
        for (int ch_id = blockIdx.x, it = 0; ch_id < p.total; ch_id += gridDim.x, ++it) {
            int n, bh; item(ch_id, n, bh);
            const int b = bh / p.H, hh = bh % p.H;
            const int next_id = ch_id + gridDim.x;
            const uint32_t ph = it & 1;
            if (s_latch) break;
            if (lead) {
                wait(&bar_load, ph);
                wait(&bar_late, ph);
                tc_fence_after();
                umma_product<true, true>(T3, aH, 16384, adDt, 8192, C, D, false, true);     // -h dDelta^T      [i][r] = dW<-^T
                umma_commit(&bm_a);
                umma_product<false, false>(T6, adDt, 16384, aMt, 8192, C, C, false);        // dDelta^T M       [j][s]
                umma_product<false, true>(T2, aV, 8192, adDt, 8192, C, D, false);           // V dDelta^T       [s][r]
                umma_commit(&bm_b);                 // from here on no product reads V or dDelta^T any more
                umma_product<false, true>(T1, adO - 8192, 8192, aDt, 8192, C, D, false);    // dO Delta^T [r][s], rows r on lanes 64 + r
                umma_product<true, false>(T4, aH, 16384, adO, 8192, C, D, false);           // h dO^T           [i][r]
                umma_commit(&bm_c);                 // from here on no product reads dO or h any more
                if (next_id < p.total) prefetch_late(next_id);
            }
            nb_sync(kNbX, kBwdThreads);                                  // X has been built
            nb_sync(kNbDW, kBwdThreads);                                 // the dW<-^T tile is complete
            if (lead) {
                tc_fence_after();
                // the product that the dependent chain waits for goes first, the two that are needed late after it
                umma_product<false, true>(T3, aXe, 8192, adW, 8192, C, D, false);           // X dW<-^T         [s][r]
                umma_commit(&bm_2);
                umma_product<true, true>(T5, adH, 16384, aDt, 8192, C, D, false);           // dh Delta^T       [i][s]
                umma_product<false, false>(T0, aXe, 8192, aK, 8192, C, D, false);           // X K^T            [r][i]
                umma_product<false, false>(T7, aXe - 8192, 8192, aK, 8192, C, D, false);    // once more, rows r on lanes 64 + r
            }
            nb_sync(kNbDV, kBwdThreads);                                 // the dv staging tile is complete, T6 has been read
            if (lead) {
                tma_store_3d(&mapdV, sm + oStDv, hh * D, n * C, b);          // rows past the end of the sequence are skipped
                tma_store_3d(&mapdV, sm + oStDv + 8192, hh * D + 64, n * C, b);
                tma_store_commit();
                tc_fence_after();
                umma_product<false, false>(T6, adW, 16384, aMt, 8192, C, C, false);         // dW<-^T M         [i][s]
            }
            nb_sync(kNbDTb, kBwdThreads);
            if (lead) {
                tc_fence_after();
                umma_product<true, true>(T3, adTb, 8192, aMt, 8192, C, C, false);           // N~ = dT diag(beta) M^T   [r][u]
                umma_commit(&bm_3);
            }
            nb_sync(kNbN, kBwdThreads);
            if (lead) {
                tc_fence_after();
                umma_product<false, true>(T2, aMt, 8192, aN, 8192, C, C, false, true);      // dA = -M^T N~     [r][s]
                umma_product<false, true>(T3, aMt - 8192, 8192, aN, 8192, C, C, false, true);   // once more, rows r on lanes 64 + r
                umma_commit(&bm_4);
            }
            nb_sync(kNbDXK, kBwdThreads);
            if (lead) {
                tc_fence_after();
                umma_product<true, false>(T7, aK, 8192, adXK, 8192, C, C, false);           // (dXK K)^T        [i][r]
                umma_product<true, true>(T1, aXe, 8192, adXK, 8192, C, C, false);           // (dXK^T X)^T      [i][s]
                umma_product<true, true>(T1, aQ, 8192, adPG, 8192, C, C, true);             // + (dPG^T Q)^T
                umma_product<true, false>(T2, aK, 8192, adPG, 8192, C, C, false);           // (dPG K)^T        [i][r]
                umma_commit(&bm_5);
                tma_store_wait_read();                                   // the dv staging tile may be reused now
                mbar_arrive(&bm_5);
                wait(&bm_5, ph);
                // V, dO, M^T, P of this chunk are dead: fetch the next chunk's
                if (next_id < p.total && !s_abort) issue_early(next_id);
            }
            nb_sync(kNbScr, kBwdThreads);                                // the column sums have read the scratch over h^T, dh^T
            if (lead) {
                fence_proxy_async();
                if (next_id < p.total && !s_abort) issue_late(next_id, 1);
            }
            nb_sync(kNbOut, kBwdThreads);                                // the dk and dq staging tiles are complete
            if (lead) {
                tma_store_3d(&mapdK, sm + oStDk, hh * D, n * C, b);
                tma_store_3d(&mapdK, sm + oStDk + 8192, hh * D + 64, n * C, b);
                tma_store_3d(&mapdQ, sm + oStDq, hh * D, n * C, b);
                tma_store_3d(&mapdQ, sm + oStDq + 8192, hh * D + 64, n * C, b);
                tma_store_commit();
                fence_proxy_async();                                     // the epilogue's reads of Q precede the copy into its region
                if (next_id < p.total && !s_abort) issue_late(next_id, 0);
            }
            // s_latch is read by everyone right after the barrier and not written again before the next one;
            // an expiry that this read misses is seen one chunk later (waits return at once meanwhile)
            if (lead) s_latch = s_abort;
            __syncthreads();                                             // every read of this chunk's tiles and scratch is done
            if (lead) {
                tma_store_wait_read();                                   // the staging tiles have been read by the stores
                fence_proxy_async();
                if (next_id < p.total && !s_abort) issue_late(next_id, 2);
            }
        }
        if (lead) tma_store_wait_all();
    } else {
    // ======================================== epilogue threads ========================================
    auto csync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(kNbC), "r"(kBwdCompute) : "memory"); };   // warps arrive converged
    if ((int)blockIdx.x < p.total) fetch_coef(blockIdx.x);
    grid_dep_wait();                    // coefficients and log-decays are older than the reverse chain; the results below are not

    for (int ch_id = blockIdx.x, it = 0; ch_id < p.total; ch_id += gridDim.x, ++it) {
    int n, bh; item(ch_id, n, bh);
    const int b = bh / p.H, hh = bh % p.H;
    const size_t row0 = (size_t)b * p.T + (size_t)n * C;          // token row in the [B*T] view
    const int live = min(C, p.T - n * C);                          // tokens of this chunk inside the sequence (may be <= 0)
    const int next_id = ch_id + gridDim.x;
    const uint32_t ph = it & 1;
    if (s_latch) break;
    if (tid < C) {
        sbeta[tid] = cf_beta;
        slam[tid] = cf_lam;
        salpha[tid] = cf_alpha;
        sg[tid] = cf_g;
        sgam[tid] = __expf(cf_g);
        if (NORM) srn[tid] = make_float2(cf_rk, cf_rq);
    }
    csync();
    if (tid < C) {
        const float ec = __expf(sg[C - 1] - sg[tid]);
        scf[tid] = make_float4(sgam[tid] * sbeta[tid], ec, sgam[tid], slam[tid]);
    }
    wait(&bar_load, ph);
    wait(&bar_late, ph);
    // ---- X = K + lambda Q (the products that do not read X are already running); partial <dh,h>_F -------
    if (has_lam || NORM) {
        constexpr int kPer = 16 / (kBwdCompute / 64);     // 16-byte chunks of a row per thread
        const int r = tid & 63, part = tid >> 6;
        const float lm = slam[r];
        const float rq = NORM ? srn[r].y : 1.f, rk = NORM ? srn[r].x : 1.f;
#pragma unroll
        for (int cc = 0; cc < kPer; ++cc) {
            const int ci = part * kPer + cc;              // chunk 0..15 of the row: block ci>>3, chunk ci&7
            const uint32_t off = (ci >> 3) * 8192 + sw128_chunk(r, ci & 7);
            float qv[8], kv[8];
            load8(sm + oQ + off, qv);
            load8(sm + oK + off, kv);
            if (NORM) {                                   // q^ and k^ in place: no product has read Q or K yet
#pragma unroll
                for (int e = 0; e < 8; ++e) { qv[e] *= rq; kv[e] *= rk; }
                sts128(sm + oQ + off, pack8(qv));
                sts128(sm + oK + off, pack8(kv));
            }
            if (has_lam) {
#pragma unroll
                for (int e = 0; e < 8; ++e) kv[e] = fmaf(lm, qv[e], kv[e]);
                sts128(sm + oX + off, pack8(kv));
            }
        }
    }
    fence_proxy_async();
    tc_fence_before();                                    // also orders the previous chunk's TMEM reads before the new products
    nb_arrive(kNbX, kBwdThreads);
    float dhh_part = 0.f;
    if (want_da)
#pragma unroll
    for (int cc = 0; cc < 16 / kNWG; ++cc) {
        const int ci = wg * (16 / kNWG) + cc;                // chunk 0..15 of line l
        const uint32_t off = (ci >> 3) * 16384 + sw128_chunk(l, ci & 7);
        float a[8], c8[8];
        load8(sm + oH + off, a);
        load8(sm + odH + off, c8);
#pragma unroll
        for (int e = 0; e < 8; ++e) dhh_part = fmaf(a[e], c8[e], dhh_part);
    }
    // ---- dW<-^T = -h dDelta^T: row i = l as an operand tile (region of its own: dO is still being read) -----
    wait(&bm_a, ph);
    tc_fence_after();
#pragma unroll
    for (int g8 = 0; g8 < kG8; ++g8) {
        float dw[8];
        ld8(my(T3) + g8 * 8, dw);
        tmem_ld_wait();
        sts128(sm + odW + sw128_chunk(l, wg * kG8 + g8), pack8(dw));
    }
    fence_proxy_async();
    tc_fence_before();
    nb_arrive(kNbDW, kBwdThreads);
    wait(&bm_b, ph);
    tc_fence_after();
    float* sPP = reinterpret_cast<float*>(sm + oPP);
    {
        // my columns in groups of 8 (one 16-byte bf16 chunk each)
        unsigned char* stg = sm + oStDv + (l >> 6) * 8192;
#pragma unroll
        for (int g8 = 0; g8 < kG8; ++g8) {
            const int cb = c0 + g8 * 8;
            float dvv[8];
            ld8(my(T6) + g8 * 8, dvv);
            tmem_ld_wait();
            // dV^T row j = l scaled by beta_s into the staging tile
#pragma unroll
            for (int e = 0; e < 8; ++e)
                sts16(stg + sw128_off(cb + e, l & 63), __float2bfloat16_rn(sbeta[cb + e] * dvv[e]));
        }
    }
    fence_proxy_async();
    tc_fence_before();
    nb_arrive(kNbDV, kBwdThreads);
    float* sAA = reinterpret_cast<float*>(sm + oAA);
    // One group of 8 columns of the dA epilogue for row r; tA = dA, tX = X K^T, both with row r on this thread's lane.
    auto dA_group = [&](uint32_t tA, uint32_t tX, int g8, int r, float& db, float& rAA) {
        const float gr = sg[r], br = sbeta[r];
        const int cb = c0 + g8 * 8;
        float da[8], xk[8];
        ld8(my(tA) + g8 * 8, da);
        ld8(my(tX) + g8 * 8, xk);
        tmem_ld_wait();
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int s = cb + e;
            const bool on = s < r;
            const float gm = on ? (has_alpha ? __expf(gr - sg[s]) : 1.f) : 0.f;
            const float d = on ? da[e] : 0.f;
            const float dgx = d * gm * xk[e];
            db += dgx;
            const float aa = br * dgx;
            rAA += aa;
            if (want_da) sts32(&sAA[r * LDAA + s], aa);
            da[e] = d * br * gm;                               // dXK
        }
        sts128(sm + odXK + sw128_chunk(r, wg * kG8 + g8), pack8(da));
    };
    static_assert(kG8 == 2, "the dA epilogue gives one column group to each half of a warpgroup");
    // From here to the column sums the two halves of every warpgroup go separate ways.  Lanes 64..127 (whose rows
    // of the 64-row accumulators are padding) take dP, whose product was issued with its rows on their lanes; lanes
    // 0..63 walk the dependent chain dT -> N~ -> dA -> dXK.  Both raise every barrier of the chain exactly once.
    if (l >= C) {
        nb_arrive(kNbDTb, kBwdThreads);
        nb_arrive(kNbN, kBwdThreads);
        wait(&bm_c, ph);                  // dP's product; its scratch lies over h^T, which that group has read
        tc_fence_after();
        // dP row r = l - 64: causal mask, dP o P (row and column sums), dP o Gamma as an operand tile
        const int r = l - C;
        const float gr = sg[r];
        float rPP = 0.f;
#pragma unroll
        for (int g8 = 0; g8 < kG8; ++g8) {
            const int cb = c0 + g8 * 8, ck = wg * kG8 + g8;
            float v[8], pv[8], pg[8];
            ld8(my(T1) + g8 * 8, v);
            tmem_ld_wait();
            load8(sm + oP + sw128_chunk(r, ck), pv);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int s = cb + e;
                const float dp = (s <= r) ? v[e] : 0.f;
                const float pp = dp * pv[e];
                rPP += pp;
                if (want_da) sts32(&sPP[r * C + ((s + r) & (C - 1))], pp);   // rotated rows: 64 x 64 floats fit the h^T half exactly
                pg[e] = (s <= r) ? (has_alpha ? dp * __expf(gr - sg[s]) : dp) : 0.f;
            }
            sts128(sm + odPG + sw128_chunk(r, ck), pack8(pg));
        }
        srow[0][wg][r] = rPP;
        // second column group of the dA epilogue, from the copies of dA and X K^T whose rows lie on these lanes
        wait(&bm_4, ph);
        tc_fence_after();
        float db = 0.f, rAA = 0.f;
        dA_group(T3, T7, 1, r, db, rAA);
        srow[4][wg][r] = db;
        srow[5][wg][r] = rAA;
    } else {
    wait(&bm_2, ph);
    tc_fence_after();
    if (l < C) {
        // dT^T row s = l, my 32 values of r;  M[r][s] = line s of Mt
        const int s = l;
        const float gs = sgam[s], bs = sbeta[s];
        float mb = 0.f, db = 0.f;
#pragma unroll
        for (int g8 = 0; g8 < kG8; ++g8) {
            const int ck = wg * kG8 + g8;
            float a[8], bq[8], m[8], tb8[8];
            ld8(my(T2) + g8 * 8, a);
            ld8(my(T3) + g8 * 8, bq);
            tmem_ld_wait();
            load8(sm + oMt + sw128_chunk(s, ck), m);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const float dt = fmaf(gs, bq[e], a[e]);
                db = fmaf(dt, m[e], db);
                mb = fmaf(m[e], bq[e], mb);
                tb8[e] = bs * dt;
            }
            sts128(sm + odTb + sw128_chunk(s, ck), pack8(tb8));
        }
        srow[1][wg][s] = db;
        srow[2][wg][s] = gs * bs * mb;
    }
    fence_proxy_async();
    tc_fence_before();
    nb_arrive(kNbDTb, kBwdThreads);
    // ---- N~ = dT diag(beta) M^T, copied out as an operand tile --------------------------------------
    wait(&bm_3, ph);
    tc_fence_after();
    if (l < C) {
#pragma unroll
        for (int g8 = 0; g8 < kG8; ++g8) {
            float v[8];
            ld8(my(T3) + g8 * 8, v);
            tmem_ld_wait();
            sts128(sm + oN + sw128_chunk(l, wg * kG8 + g8), pack8(v));
        }
    }
    fence_proxy_async();
    tc_fence_before();
    nb_arrive(kNbN, kBwdThreads);
    // ---- dA = -M^T N~ -----------------------------------------------------------------------------
    wait(&bm_4, ph);
    tc_fence_after();
    {
        const int r = l;
        float rAA = 0.f, db = 0.f;
        dA_group(T2, T0, 0, r, db, rAA);
        srow[1][wg][r] += db;
        srow[3][wg][r] = rAA;
    }
    }  // lanes 0..63: the dependent chain
    fence_proxy_async();
    tc_fence_before();
    nb_arrive(kNbDXK, kBwdThreads);
    // ---- the last products; meanwhile the column sums of dA o A and dP o P (kBwdCompute/64 threads per column)
    // and the coefficients of the next chunk -------------------------------------------------------------------
    csync();
    if (want_da) {
        const float* sAAc = reinterpret_cast<const float*>(sm + oAA);
        const int r = tid & 63, part = tid >> 6;
        float cA = 0.f, cP = 0.f;
        constexpr int kRows = C / (kBwdCompute / 64);
#pragma unroll
        for (int k = 0; k < kRows; ++k) {
            cA += sAAc[(part * kRows + k) * LDAA + r];
            cP += sPP[(part * kRows + k) * C + ((r + part * kRows + k) & (C - 1))];
        }
        scol[0][part][r] = cA;
        scol[1][part][r] = cP;
    }
    nb_arrive(kNbScr, kBwdThreads);      // the scratch tiles over h^T and dh^T are dead from here on
    if (want_da) {
        dhh_part += __shfl_xor_sync(0xffffffffu, dhh_part, 16);
        dhh_part += __shfl_xor_sync(0xffffffffu, dhh_part, 8);
        dhh_part += __shfl_xor_sync(0xffffffffu, dhh_part, 4);
        dhh_part += __shfl_xor_sync(0xffffffffu, dhh_part, 2);
        dhh_part += __shfl_xor_sync(0xffffffffu, dhh_part, 1);
        if (lane == 0) swp[tid >> 5] = dhh_part;
    }
    csync();
    // everything of the decay gradient that does not wait for the last epilogue
    float dg_pre = 0.f;
    if (tid < C) {
        const int r = tid;
        float cAA = 0.f, cPP = 0.f;
#pragma unroll
        for (int w4 = 0; w4 < kBwdCompute / 64; ++w4) { cAA += scol[0][w4][r]; cPP += scol[1][w4][r]; }
        float rPP = 0.f, t2 = 0.f, rAA = 0.f, dbt = 0.f;
#pragma unroll
        for (int w4 = 0; w4 < kNWG; ++w4) {
            rPP += srow[0][w4][r]; dbt += srow[1][w4][r] + srow[4][w4][r]; t2 += srow[2][w4][r]; rAA += srow[3][w4][r] + srow[5][w4][r];
        }
        dg_pre = rPP - cPP + t2 + rAA - cAA;
        // with logit inputs: d/dz of sigmoid(z) is sigmoid(z) (1 - sigmoid(z))
        if (r < live) p.dbeta[(row0 + r) * p.H + hh] = p.logits ? dbt * sbeta[r] * (1.f - sbeta[r]) : dbt;
    }
    if (next_id < p.total) fetch_coef(next_id);
    wait(&bm_5, ph);
    tc_fence_after();
    // The last epilogue: thread = d_k index i, its 16 tokens in groups of 8: dk and dq, transposed, into their staging
    // tiles, and the column sums (over i, i.e. across the lanes) that d lambda and the decay gradient need.
    {
        const int i = l;
        unsigned char* stk = sm + oStDk + (i >> 6) * 8192;
        unsigned char* stq = sm + oStDq + (i >> 6) * 8192;
        const unsigned char* qcol = sm + oQ + (i >> 6) * 8192;
        const unsigned char* kcol = sm + oK + (i >> 6) * 8192;
#pragma unroll
        for (int g8 = 0; g8 < kG8; ++g8) {
            const int cb = c0 + g8 * 8;
            float dx[8], v[8], w[8], u[8], z[8], y[8];
            ld8(my(T6) + g8 * 8, dx);
            ld8(my(T7) + g8 * 8, v);
            ld8(my(T1) + g8 * 8, w);
            ld8(my(T5) + g8 * 8, u);
            ld8(my(T4) + g8 * 8, z);
            ld8(my(T2) + g8 * 8, y);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int t = cb + e;
                const float4 cf = scf[t];
                const float dxe = fmaf(cf.x, dx[e], v[e]);                                  // dX^T[i][t]
                const float kh = cf.y * u[e];                                               // (K-> ^T applied to dh Delta^T)[i][t]
                sts16(stk + sw128_off(t, i & 63), __float2bfloat16_rn(w[e] + kh + dxe));    // d k  (d k^ with NORM)
                // <(K-> dh)_t, Delta_t> = gamma_C/gamma_t sum_i K[t][i] (dh Delta^T)[i][t], all of it in fp32
                u[e] = kh * __bfloat162float(*reinterpret_cast<const bf16*>(kcol + sw128_off(t, i & 63)));
                const float q1 = cf.z * z[e];
                sts16(stq + sw128_off(t, i & 63), __float2bfloat16_rn(q1 + y[e] + cf.w * dxe));   // d q  (d q^ with NORM)
                const float qv = __bfloat162float(*reinterpret_cast<const bf16*>(qcol + sw128_off(t, i & 63)));
                z[e] = q1 * qv;
                dx[e] = dxe * qv;
            }
            // column sums over the d_k index (across the lanes): d lambda, and the two that only the decay gradient needs
            if (want_dl) {
                const float dls = col_reduce8(dx, lane);
                if ((lane & 3) == 0) sred[1][wq][cb + col8_of_lane(lane)] = dls;
            }
            if (want_da) {
                const float t1s = col_reduce8(z, lane), kds = col_reduce8(u, lane);
                if ((lane & 3) == 0) {
                    const int col = cb + col8_of_lane(lane);
                    sred[0][wq][col] = kds;
                    sred[2][wq][col] = t1s;
                }
            }
        }
    }
    if (NORM) {
        // Through the normalisation: dx = r (dx^ - x^ <x^, dx^>).  The staged tiles hold dk^ and dq^ token-major, like the
        // K^ and Q^ tiles, so both steps are row-wise passes with 16-byte accesses: thread (row r, part) takes two
        // 16-byte chunks of its row; first the partial row dot products (eight parts per row, summed through scratch
        // over the dead row sums), then the corrected rows.
        float (*part_k)[C] = reinterpret_cast<float (*)[C]>(&srow[0][0][0]);     // [8][C]
        float (*part_q)[C] = reinterpret_cast<float (*)[C]>(&srow[2][0][0]);     // [8][C]
        constexpr int kPer = 16 / (kBwdCompute / 64);
        static_assert(kBwdCompute / 64 == 8 && kNWG == 4, "scratch of the row dot products: 8 parts of 64 rows, twice");
        const int r = tid & 63, part = tid >> 6;
        csync();                             // the staged tiles are complete; the row sums have been consumed
        float ck = 0.f, cq = 0.f;
#pragma unroll
        for (int cc = 0; cc < kPer; ++cc) {
            const int ci = part * kPer + cc;
            const uint32_t off = (ci >> 3) * 8192 + sw128_chunk(r, ci & 7);
            float a8[8], x8[8];
            load8(sm + oStDk + off, a8);
            load8(sm + oK + off, x8);
#pragma unroll
            for (int e = 0; e < 8; ++e) ck = fmaf(a8[e], x8[e], ck);
            load8(sm + oStDq + off, a8);
            load8(sm + oQ + off, x8);
#pragma unroll
            for (int e = 0; e < 8; ++e) cq = fmaf(a8[e], x8[e], cq);
        }
        part_k[part][r] = ck;
        part_q[part][r] = cq;
        csync();
        ck = 0.f; cq = 0.f;
#pragma unroll
        for (int pp = 0; pp < 8; ++pp) { ck += part_k[pp][r]; cq += part_q[pp][r]; }
        const float2 rn = srn[r];            // {1/|k|, 1/|q|}
#pragma unroll
        for (int cc = 0; cc < kPer; ++cc) {
            const int ci = part * kPer + cc;
            const uint32_t off = (ci >> 3) * 8192 + sw128_chunk(r, ci & 7);
            float a8[8], x8[8];
            load8(sm + oStDk + off, a8);
            load8(sm + oK + off, x8);
#pragma unroll
            for (int e = 0; e < 8; ++e) a8[e] = rn.x * fmaf(-ck, x8[e], a8[e]);
            sts128(sm + oStDk + off, pack8(a8));
            load8(sm + oStDq + off, a8);
            load8(sm + oQ + off, x8);
#pragma unroll
            for (int e = 0; e < 8; ++e) a8[e] = rn.y * fmaf(-cq, x8[e], a8[e]);
            sts128(sm + oStDq + off, pack8(a8));
        }
    }
    fence_proxy_async();
    tc_fence_before();
    nb_arrive(kNbOut, kBwdThreads);
    csync();
    // ---- decay gradient ----------------------------------------------------------------------------
    if (tid < C && (want_dl || want_da)) {
        const int r = tid;
        float kd = 0.f, dl = 0.f, t1 = 0.f;
#pragma unroll
        for (int w4 = 0; w4 < 4; ++w4) { kd += sred[0][w4][r]; dl += sred[1][w4][r]; t1 += sred[2][w4][r]; }
        sdg[r] = t1 + dg_pre - kd;
        skd[r] = kd;                            // summed below into dg of the last token
        if (want_dl && r < live) p.dlam[(row0 + r) * p.H + hh] = p.logits ? dl * slam[r] * (1.f - slam[r]) : dl;
    }
    csync();
    if (tid < 32 && want_da) {
        // warp 0: lane owns tokens 2*lane, 2*lane+1; d log alpha_i = sum_{r >= i} dg_r (suffix sums)
        const float a = sdg[2 * lane];
        float b2 = sdg[2 * lane + 1];
        float kds = skd[2 * lane] + skd[2 * lane + 1];
        float dhh = lane < kBwdCompute / 32 ? swp[lane] : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            kds += __shfl_xor_sync(0xffffffffu, kds, o);
            dhh += __shfl_xor_sync(0xffffffffu, dhh, o);
        }
        if (lane == 31) b2 += sgam[C - 1] * dhh + kds;
        float sfx = a + b2;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_down_sync(0xffffffffu, sfx, o);
            if (lane + o < 32) sfx += t;
        }
        if (p.dalpha) {
            // d log alpha -> d alpha = d log alpha / alpha;  with logit inputs d/dz log sigmoid(z) = 1 - sigmoid(z)
            const float a0 = salpha[2 * lane], a1 = salpha[2 * lane + 1];
            if (2 * lane < live) p.dalpha[(row0 + 2 * lane) * p.H + hh] = p.logits ? sfx * (1.f - a0) : sfx / a0;
            if (2 * lane + 1 < live) p.dalpha[(row0 + 2 * lane + 1) * p.H + hh] = p.logits ? (sfx - a) * (1.f - a1) : (sfx - a) / a1;
        }
    }
    __syncthreads();                     // every read of this chunk's tiles and scratch is done
    }  // chunk loop
    }  // epilogue threads
    tc_fence_before();
    __syncthreads();
    if (tid == kBwdCompute && s_abort) { mbar_wait(&bar_load, 0); mbar_wait(&bar_late, 0); }   // one more bounded chance for copies in flight
    if (tid < 32) tmem_dealloc(tb, 512);
}

template <class K>
cudaError_t set_smem(K kern, size_t bytes) { return set_max_smem_once(reinterpret_cast<const void*>(kern), bytes); }

}  // namespace

cudaError_t tc_chain_bwd(const ChunkArgs& a) {
    const qd_shape& s = a.s;
    const int Tp = tc_padded_T(s);
    const uint64_t BH = (uint64_t)s.B * s.H, N = Tp / kChunk;
    CUtensorMap mWt, mdO, mQg, mK, mP, mdHs, mdDt;
    if (!make_tmap_bf16_2d(&mWt, a.ws + a.TL.Wt, 64, BH * N * D, 128, 128) ||
        !make_tmap_tokens(&mdO, a.dO, s.B, s.T, s.H, D, 64) ||
        !make_tmap_bf16_2d(&mQg, a.ws + a.TL.Qg, D, BH * Tp, D * 2, 64) ||
        !make_tmap_tokens(&mK, a.k, s.B, s.T, s.H, D, 64) ||
        !make_tmap_bf16_2d(&mP, a.ws + a.TL.P, 64, BH * Tp, 128, 64) ||
        !make_tmap_bf16_2d(&mdHs, a.ws + a.TL.dhsT, D, BH * N * D, D * 2, 128) ||
        !make_tmap_bf16_2d(&mdDt, a.ws + a.TL.dDt, 64, BH * N * D, 128, 128))
        return cudaErrorInvalidValue;
    ChainBwdParams p{};
    p.Tp = Tp; p.H = s.H; p.N = (int)N;
    p.dhT_early = a.own_predecessor ? 1 : 0;
    p.rk = a.norm ? (const float*)(a.ws + a.TL.rqk) + BH * Tp : nullptr;
    p.g = (const float*)(a.ws + a.TL.g);
    p.dhT = a.dhT; p.dh0 = a.dh0;
    p.status = (unsigned*)(a.ws + a.TL.status);
    cudaError_t e = set_smem(k_tc_chain_bwd, kChainSmem);
    if (e != cudaSuccess) return e;
    return launch_overlapped(k_tc_chain_bwd, dim3((unsigned)BH), dim3(kChainThreads), kChainSmem, a.stream,
                             mWt, mdO, mQg, mK, mP, mdHs, mdDt, p);
}

cudaError_t tc_chunk_bwd(const ChunkArgs& a) {
    const qd_shape& s = a.s;
    const int Tp = tc_padded_T(s);
    const uint64_t BH = (uint64_t)s.B * s.H, N = Tp / kChunk;
    CUtensorMap mQ, mK, mV, mdO, mMt, mP, mDt, mdDt, mHs, mdHs, mdQ, mdK, mdV;
    if (!make_tmap_tokens(&mdQ, a.dq, s.B, s.T, s.H, D, 64) ||
        !make_tmap_tokens(&mdK, a.dk, s.B, s.T, s.H, D, 64) ||
        !make_tmap_tokens(&mdV, a.dv, s.B, s.T, s.H, D, 64) ||
        !make_tmap_tokens(&mQ, a.q, s.B, s.T, s.H, D, 64) ||
        !make_tmap_tokens(&mK, a.k, s.B, s.T, s.H, D, 64) ||
        !make_tmap_tokens(&mV, a.v, s.B, s.T, s.H, D, 64) ||
        !make_tmap_tokens(&mdO, a.dO, s.B, s.T, s.H, D, 64) ||
        !make_tmap_bf16_2d(&mMt, a.ws + a.TL.Mt, 64, BH * Tp, 128, 64) ||
        !make_tmap_bf16_2d(&mP, a.ws + a.TL.P, 64, BH * Tp, 128, 64) ||
        !make_tmap_bf16_2d(&mDt, a.ws + a.TL.Dt, 64, BH * N * D, 128, 128) ||
        !make_tmap_bf16_2d(&mdDt, a.ws + a.TL.dDt, 64, BH * N * D, 128, 128) ||
        !make_tmap_bf16_2d(&mHs, a.ws + a.TL.hsT, D, BH * N * D, D * 2, 128) ||
        !make_tmap_bf16_2d(&mdHs, a.ws + a.TL.dhsT, D, BH * N * D, D * 2, 128))
        return cudaErrorInvalidValue;
    ChunkBwdParams p{};
    p.T = s.T; p.Tp = Tp; p.H = s.H; p.N = (int)N; p.BH = (int)BH; p.total = (int)(BH * N);
    p.beta = (const bf16*)a.beta; p.alpha = (const bf16*)a.alpha; p.lam = (const bf16*)a.lam;
    p.g = (const float*)(a.ws + a.TL.g);
    p.dbeta = a.dbeta; p.dalpha = a.dalpha; p.dlam = a.dlam;
    p.logits = a.logits ? 1 : 0;
    p.rqk = a.norm ? (const float*)(a.ws + a.TL.rqk) : nullptr;
    p.status = (unsigned*)(a.ws + a.TL.status);
    // the instance without lambda / without the forget gate needs the input AND its gradient to be absent
    const bool lam = a.lam || a.dlam, alpha = a.alpha || a.dalpha;
    const bool grouped = N >= 64;         // long sequences: work items in groups of 32 sequences (see the kernel)
    p.group = 32;
    using Kern = decltype(&k_tc_chunk_bwd<true, true, false, false>);
    static const Kern table[16] = {
        k_tc_chunk_bwd<false, false, false, false>, k_tc_chunk_bwd<false, false, false, true>,
        k_tc_chunk_bwd<false, false, true, false>,  k_tc_chunk_bwd<false, false, true, true>,
        k_tc_chunk_bwd<false, true, false, false>,  k_tc_chunk_bwd<false, true, false, true>,
        k_tc_chunk_bwd<false, true, true, false>,   k_tc_chunk_bwd<false, true, true, true>,
        k_tc_chunk_bwd<true, false, false, false>,  k_tc_chunk_bwd<true, false, false, true>,
        k_tc_chunk_bwd<true, false, true, false>,   k_tc_chunk_bwd<true, false, true, true>,
        k_tc_chunk_bwd<true, true, false, false>,   k_tc_chunk_bwd<true, true, false, true>,
        k_tc_chunk_bwd<true, true, true, false>,    k_tc_chunk_bwd<true, true, true, true>,
    };
    const Kern kern = table[(lam ? 8 : 0) + (alpha ? 4 : 0) + (a.norm ? 2 : 0) + (grouped ? 1 : 0)];
    cudaError_t e = set_smem(kern, kBwdSmem);
    if (e != cudaSuccess) return e;
    // persistent: one CTA per SM walks the work items with stride gridDim.x
    int dev = 0, sms = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    const unsigned grid = (unsigned)std::min<uint64_t>(BH * N, (uint64_t)sms);
    return launch_overlapped(kern, dim3(grid), dim3(kBwdThreads), kBwdSmem, a.stream, mQ, mK, mV, mdO, mMt, mP,
                             mDt, mdDt, mHs, mdHs, mdQ, mdK, mdV, p);
}

}  // namespace qd
