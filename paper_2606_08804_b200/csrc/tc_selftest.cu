// Unit checks of the sm_100a primitives.
//  * one CTA computes D[128 x N] = Aop * Bop^T over a contraction of K with tcgen05.mma from
//    128-byte-swizzled shared-memory tiles, in each of the four operand-major combinations the kernels
//    use, with tiles filled either by TMA or by threads;
//  * one CTA waits, with a short limit, on an mbarrier that nothing ever arrives on: the path every kernel
//    takes when a bounded wait runs out (record QD_ERR_TIMEOUT, release tensor memory, return).
#include "internal.h"
#include "sm100.cuh"

namespace qd {

namespace {
using namespace sm100;

struct SelfArgs {
    const __nv_bfloat16 *A, *B;
    float* D;
    int N, K, a_mn, b_mn, by_threads;
    int RA, CA, RB, CB;
    unsigned* status;
};

__global__ void __launch_bounds__(128) k_selftest(const __grid_constant__ CUtensorMap mapA,
                                                  const __grid_constant__ CUtensorMap mapB, SelfArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    unsigned char* sA = smem;               // up to 2 blocks of [128][64] bf16
    unsigned char* sB = smem + 32768;
    __shared__ uint64_t bar_load, bar_mma;
    __shared__ uint32_t tmem_slot;
    __shared__ int failed;
    const int tid = threadIdx.x, warp = tid >> 5;
    const uint32_t ncols = a.by_threads == 2 ? 256u : (a.N < 32 ? 32u : (uint32_t)a.N);
    if (tid == 0) {
        mbar_init(&bar_load, 1);
        mbar_init(&bar_mma, 1);
        mbar_init_fence();
        failed = 0;
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, ncols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = tmem_slot;
    const uint32_t a_blk = (uint32_t)a.RA * 128u, b_blk = (uint32_t)a.RB * 128u;

    if (a.by_threads == 2) {
        // A (row-major [128][K]) goes to tensor memory: thread = row, bf16 pairs packed per 32-bit column,
        // columns [N, N + K/2); B to shared memory by threads
        for (int c8 = 0; c8 < a.K / 16; ++c8) {
            uint32_t r[8];
            for (int j = 0; j < 8; ++j) {
                const __nv_bfloat16 lo = a.A[(size_t)tid * a.K + c8 * 16 + 2 * j], hi = a.A[(size_t)tid * a.K + c8 * 16 + 2 * j + 1];
                r[j] = (uint32_t)(*(const unsigned short*)&lo) | ((uint32_t)(*(const unsigned short*)&hi) << 16);
            }
            tmem_st8(tmem_addr(tbase, warp * 32, a.N + c8 * 8), r);
        }
        tmem_st_wait();
        for (int e = tid; e < a.RB * a.CB; e += 128) {
            const int r = e / a.CB, c = e % a.CB;
            *(__nv_bfloat16*)(sB + (c >> 6) * b_blk + sw128_off(r, c & 63)) = a.B[e];
        }
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
    } else if (a.by_threads) {
        for (int e = tid; e < a.RA * a.CA; e += 128) {
            const int r = e / a.CA, c = e % a.CA;
            *(__nv_bfloat16*)(sA + (c >> 6) * a_blk + sw128_off(r, c & 63)) = a.A[e];
        }
        for (int e = tid; e < a.RB * a.CB; e += 128) {
            const int r = e / a.CB, c = e % a.CB;
            *(__nv_bfloat16*)(sB + (c >> 6) * b_blk + sw128_off(r, c & 63)) = a.B[e];
        }
        fence_proxy_async();
        __syncthreads();
    } else {
        if (tid == 0) {
            mbar_expect_tx(&bar_load, (uint32_t)(a.RA * a.CA + a.RB * a.CB) * 2u);
            for (int cb = 0; cb < a.CA / 64; ++cb) tma_load_2d(sA + cb * a_blk, &mapA, cb * 64, 0, &bar_load);
            for (int cb = 0; cb < a.CB / 64; ++cb) tma_load_2d(sB + cb * b_blk, &mapB, cb * 64, 0, &bar_load);
        }
        if (!mbar_wait(&bar_load, 0)) failed = 1;
        __syncthreads();
    }
    if (!failed) {
        if (tid == 0) {
            tc_fence_after();
            const uint32_t sa = smem_u32(sA), sb = smem_u32(sB);
            if (a.by_threads == 2) {
                if (a.b_mn) umma_product_ts<true>(tbase, tbase + a.N, sb, b_blk, a.N, a.K, false);
                else umma_product_ts<false>(tbase, tbase + a.N, sb, b_blk, a.N, a.K, false);
            } else if (a.a_mn && a.b_mn) umma_product<true, true>(tbase, sa, a_blk, sb, b_blk, a.N, a.K, false);
            else if (a.a_mn) umma_product<true, false>(tbase, sa, a_blk, sb, b_blk, a.N, a.K, false);
            else if (a.b_mn) umma_product<false, true>(tbase, sa, a_blk, sb, b_blk, a.N, a.K, false);
            else umma_product<false, false>(tbase, sa, a_blk, sb, b_blk, a.N, a.K, false);
            umma_commit(&bar_mma);
        }
        if (!mbar_wait(&bar_mma, 0)) failed = 1;
    }
    __syncthreads();
    if (!failed) {
        tc_fence_after();
        for (int c0 = 0; c0 < a.N; c0 += 32) {
            float v[32];
            tmem_ld32(tmem_addr(tbase, warp * 32, c0), v);
            tmem_ld_wait();
            for (int j = 0; j < 32; ++j) a.D[(size_t)tid * a.N + c0 + j] = v[j];
        }
    } else if (tid == 0) {
        *a.status = QD_ERR_TIMEOUT;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tbase, ncols);
}

}  // namespace
}  // namespace qd

// Not part of the public header: a hardware self-check used by the GPU tests.
// A, B: device bf16 matrices (see k_selftest); D: device fp32 [128][N]; status: device u32.
extern "C" int qdelta_selftest_umma(const void* A, const void* B, float* D, int N, int K, int a_mn, int b_mn,
                                    int by_threads, unsigned* status, qd_stream stream) {
    using namespace qd;
    if (!A || !B || !D || !status) return QD_ERR_INVALID_ARG;
    if ((N != 64 && N != 128) || (K != 64 && K != 128)) return QD_ERR_UNSUPPORTED;
    SelfArgs a{};
    a.A = (const __nv_bfloat16*)A; a.B = (const __nv_bfloat16*)B; a.D = D;
    a.N = N; a.K = K; a.a_mn = a_mn; a.b_mn = b_mn; a.by_threads = by_threads; a.status = status;
    a.RA = a_mn ? K : 128; a.CA = a_mn ? 128 : K;
    a.RB = b_mn ? K : N;   a.CB = b_mn ? N : K;
    CUtensorMap mA, mB;
    if (!make_tmap_bf16_2d(&mA, A, a.CA, a.RA, (uint64_t)a.CA * 2, a.RA)) return QD_ERR_CUDA;
    if (!make_tmap_bf16_2d(&mB, B, a.CB, a.RB, (uint64_t)a.CB * 2, a.RB)) return QD_ERR_CUDA;
    const size_t smem = 65536 + 1024;
    if (set_max_smem_once(reinterpret_cast<const void*>(k_selftest), smem) != cudaSuccess) return QD_ERR_CUDA;
    k_selftest<<<1, 128, smem, (cudaStream_t)stream>>>(mA, mB, a);
    return cudaGetLastError() == cudaSuccess ? QD_OK : QD_ERR_CUDA;
}

namespace qd {
namespace {
using namespace sm100;

// Every thread waits on a barrier that is never completed.  out[0] <- QD_ERR_TIMEOUT when the wait gave up (QD_OK if it
// did not, which would be a bug), out[1] <- nanoseconds thread 0 spent in the wait.
__global__ void __launch_bounds__(128) k_selftest_timeout(unsigned* out, unsigned limit_ns) {
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int expired;
    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) {
        mbar_init(&bar, 1);
        mbar_init_fence();
        expired = 0;
    }
    if (warp == 0) { tmem_alloc(&tmem_slot, 32); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tbase = tmem_slot;
    const uint32_t t0 = global_timer_lo();
    if (!mbar_wait(&bar, 0, limit_ns)) expired = 1;
    const uint32_t t1 = global_timer_lo();
    __syncthreads();
    if (tid == 0) {
        out[0] = expired ? (unsigned)QD_ERR_TIMEOUT : (unsigned)QD_OK;
        out[1] = t1 - t0;
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tbase, 32);
}

}  // namespace
}  // namespace qd

// Not part of the public header: used by the GPU tests.  out: device pointer to two 32-bit words.
extern "C" int qdelta_selftest_timeout(unsigned* out, unsigned limit_ns, qd_stream stream) {
    if (!out || limit_ns == 0 || limit_ns > 100u * 1000u * 1000u) return QD_ERR_INVALID_ARG;   // at most 0.1 s
    qd::k_selftest_timeout<<<1, 128, 0, (cudaStream_t)stream>>>(out, limit_ns);
    return cudaGetLastError() == cudaSuccess ? QD_OK : QD_ERR_CUDA;
}
