// Unit check of the sm_100a primitives: one CTA computes D[128 x N] = Aop * Bop^T over a
// contraction of K with tcgen05.mma from 128-byte-swizzled shared-memory tiles, in each of the four
// operand-major combinations the kernels use, with tiles filled either by TMA or by threads.
// Also hosts the tensor-map encoder.
#include "internal.h"
#include "sm100.cuh"

#include <cudaTypedefs.h>

namespace qd {

bool make_tmap_bf16_2d(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes,
                       uint32_t box_rows) {
    static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || !fn)
            return false;
        encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    }
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {pitch_bytes};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

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
    if (cudaFuncSetAttribute(k_selftest, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return QD_ERR_CUDA;
    k_selftest<<<1, 128, smem, (cudaStream_t)stream>>>(mA, mB, a);
    return cudaGetLastError() == cudaSuccess ? QD_OK : QD_ERR_CUDA;
}

// ---- MMA issue-rate probe (timing only; operands are zeros) ------------------------------------------
namespace qd {
namespace {
using namespace sm100;

// `nthr` issuing threads (lane 0 of warps 0..nthr-1), each issuing `reps` products D[128 x N] += A B^T (K = 128,
// 8 instructions, descriptors precomputed, fully unrolled) into its own accumulator.
template <int N, bool TS>
__global__ void __launch_bounds__(128) k_mma_rate(int nthr, int reps, long long* out) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5;
    for (int i = tid; i < (32768 + 65536) / 16; i += 128) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) { mbar_init(&bar, (uint32_t)nthr); mbar_init_fence(); }
    if (warp == 0) { tmem_alloc(&tmem_slot, 512); tmem_relinquish(); }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tb = tmem_slot;
    if ((tid & 31) == 0 && warp < nthr) {
        const uint32_t sa = smem_u32(smem), sb = smem_u32(smem + 32768);
        constexpr uint32_t idesc = make_idesc(128, N, false, false);
        const uint64_t a0 = desc_kmajor(sa), b0 = desc_kmajor(sb);
        constexpr uint32_t b_blk = (uint32_t)N * 128u;
        const uint32_t tA = tb + 448;
        const uint32_t d = tb + (uint32_t)warp * (N > 64 ? 64u : (uint32_t)N);   // accumulators may overlap for N = 256: timing only
        uint64_t ad[8], bd[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            ad[k] = a0 + (((uint32_t)(k >> 2) * 16384u + (uint32_t)(k & 3) * 32u) >> 4);
            bd[k] = b0 + (((uint32_t)(k >> 2) * b_blk + (uint32_t)(k & 3) * 32u) >> 4);
        }
        const long long t0 = clock64();
#pragma unroll 1
        for (int r = 0; r < reps; ++r) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (TS) umma_ts(d, tA + k * 8, bd[k], idesc, true);
                else umma_ss(d, ad[k], bd[k], idesc, true);
            }
        }
        const long long t1 = clock64();
        umma_commit(&bar);
        mbar_wait(&bar, 0);
        const long long t2 = clock64();
        if (warp == 0) { out[0] = t1 - t0; out[1] = t2 - t0; }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tb, 512);
}

}  // namespace
}  // namespace qd

// Timing probe, not part of the public header.  out[0] = cycles thread 0 needed to issue, out[1] = cycles until
// every issuing thread's products have completed.
extern "C" int qdelta_selftest_mma_rate(int N, int nthr, int ts, int reps, long long* out, qd_stream stream) {
    using namespace qd;
    if (!out || nthr < 1 || nthr > 4 || (N != 64 && N != 128 && N != 256)) return QD_ERR_INVALID_ARG;
    const size_t smem = 32768 + 65536 + 1024;
    auto launch = [&](auto kern) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return (int)QD_ERR_CUDA;
        kern<<<1, 128, smem, (cudaStream_t)stream>>>(nthr, reps, out);
        return cudaGetLastError() == cudaSuccess ? (int)QD_OK : (int)QD_ERR_CUDA;
    };
    if (N == 64) return ts ? launch(k_mma_rate<64, true>) : launch(k_mma_rate<64, false>);
    if (N == 128) return ts ? launch(k_mma_rate<128, true>) : launch(k_mma_rate<128, false>);
    return ts ? launch(k_mma_rate<256, true>) : launch(k_mma_rate<256, false>);
}
