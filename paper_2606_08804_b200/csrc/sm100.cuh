// Device primitives for sm_100a: mbarrier with BOUNDED waits, TMA bulk-tensor copies, tcgen05
// (tensor memory allocation, UMMA issue/commit, TMEM loads) and the shared-memory / instruction
// descriptors of the 128-byte-swizzled operand layouts used by the kernels of this library.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace qd {
namespace sm100 {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---- mbarrier ----------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// raises the transaction count of the current phase without arriving (for copies issued in several batches:
// the last batch arrives with mbar_expect_tx)
__device__ __forceinline__ void mbar_expect_tx_only(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up about `limit_ns` nanoseconds of the global timer after its first unsuccessful poll.  Returns
// false on expiry; the caller records the failure and leaves.  One second is several hundred times the longest kernel
// of this library and far inside any host-side watchdog.  The low 32 bits of the timer wrap every 4.29 s, so differences
// below that are exact.  How often a waiting thread polls matters: polls are shared-memory traffic that competes with
// the operand reads of the MMAs.  Measured on the chunk-backward kernel: a tight polling loop 0.347 ms, the timer read
// every 64 polls 0.303 ms, the timer read after every poll (this loop) 0.289 ms; suspend-time hints on try_wait
// (0.5 - 50 us) 0.292 ms and slower state chains.
__device__ __forceinline__ uint32_t global_timer_lo() {
    uint32_t t;
    asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t));
    return t;
}
constexpr uint32_t kWaitLimitNs = 1000u * 1000u * 1000u;
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t limit_ns = kWaitLimitNs) {
    uint32_t t0 = 0;
#pragma unroll 1
    for (uint32_t polls = 0;; ++polls) {
        if (mbar_try_wait(bar, parity)) return true;
        const uint32_t now = global_timer_lo();          // also paces the polls
        if (polls == 0) t0 = now;
        else if (now - t0 > limit_ns) return false;
    }
}

// ---- programmatic dependent launch ------------------------------------------------------------------------------
// A kernel launched with cudaLaunchAttributeProgrammaticStreamSerialization may begin while the kernel before it in
// the stream is still running.  grid_dep_wait() returns once that kernel has completed and its writes are visible
// (at once if the launch had no such relation); everything before it may only touch data that is older than the
// preceding kernel.  grid_dep_launch() lets the kernel after this one begin; the kernels here call it right after
// their own wait, so a kernel that has begun can rely on everything up to its predecessor's predecessor.
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- fences ------------------------------------------------------------------------------------
// generic-proxy writes to shared memory -> visible to the async proxy (TMA, UMMA operand reads)
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// ---- TMA ---------------------------------------------------------------------------------------
// 2-D tiled load, no multicast.  x (innermost, elements) must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
// 3-D tiled copies of the token-major tensors [B][T][H*D]: x = column (elements, a multiple of 8), t = token,
// b = batch index.  Rows at t >= T are outside the tensor: a load fills them with zeros, a store skips them --
// which is how a sequence length that is not a multiple of the chunk is handled (t is never negative).
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* map, int x, int t, int b, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(t), "r"(b)
        : "memory");
}
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, const void* smem_src, int x, int t, int b) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(map), "r"(smem_u32(smem_src)), "r"(x), "r"(t), "r"(b)
                 : "memory");
}
__device__ __forceinline__ void tma_prefetch_3d(const CUtensorMap* map, int x, int t, int b) {
    asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(map), "r"(x), "r"(t), "r"(b) : "memory");
}
// Prefetch of a tile into L2 (no shared-memory destination, no completion to wait for).
__device__ __forceinline__ void tma_prefetch_2d(const CUtensorMap* map, int x, int y) {
    asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global.tile [%0, {%1, %2}];" ::"l"(map), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* smem_src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// wait until at most N of this thread's most recent bulk groups still have to read their source
template <int N>
__device__ __forceinline__ void tma_store_wait_read_n() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---- tensor memory -----------------------------------------------------------------------------
// One full warp allocates `ncols` (power of two >= 32) TMEM columns; the base address lands in *slot.
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 32 lanes x 32 columns of 32-bit: thread i of the warp receives lane (base lane + i), columns c..c+31.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
    uint32_t* r = reinterpret_cast<uint32_t*>(v);
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}
// store 8 consecutive 32-bit columns of this thread's lane
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// address of (lane, column) relative to an allocation base
__device__ __forceinline__ uint32_t tmem_addr(uint32_t base, uint32_t lane, uint32_t col) {
    return base + (lane << 16) + col;
}

// ---- UMMA descriptors --------------------------------------------------------------------------
// Shared-memory operand tiles use the 128-byte swizzle: a tile is a stack of 128-byte lines
// (64 bf16), eight lines form a 1024-byte atom, and inside a line the 16-byte chunk index is
// XOR-ed with (line index mod 8).  This is what a TMA load with a 64-element inner box and
// SWIZZLE_128B writes, provided the tile starts on a 1024-byte boundary.
//
//  K-major operand  (contraction index contiguous): line = one MN row, 64 K-elements per line;
//      more K lives in further "column blocks" (whole tiles of [rows][64]).  SBO = 1024 bytes
//      between 8-row groups, LBO unused.  Advancing K by 16 elements = +32 bytes of start address.
//  MN-major operand (M or N index contiguous): line = one K index, 64 MN-elements per line;
//      SBO = 1024 bytes between groups of 8 K indices, LBO = bytes between blocks of 64 MN
//      elements.  Advancing K by 16 = +2048 bytes of start address.
constexpr uint64_t kDescSw128 = (uint64_t)2 << 61;
constexpr uint64_t kDescVersion = (uint64_t)1 << 46;
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr) {
    return kDescSw128 | kDescVersion | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 16) | (uint64_t)((saddr & 0x3FFFF) >> 4);
}
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr, uint32_t lbo_bytes) {
    return kDescSw128 | kDescVersion | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16) |
           (uint64_t)((saddr & 0x3FFFF) >> 4);
}
// instruction descriptor: bf16 x bf16 -> fp32, dense
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, bool a_mn, bool b_mn, bool a_neg = false) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((a_neg ? 1u : 0u) << 13) | ((a_mn ? 1u : 0u) << 15) |
           ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]; issued by ONE thread.
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// arrive on an mbarrier once all UMMAs issued so far by this thread have completed
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// One whole product D[128 x N] (+)= A * B with contraction extent K (multiple of 16), operands in
// the swizzled layouts above.  a_blk / b_blk: bytes between 64-element blocks of the operand
// (K-major: between K column blocks; MN-major: between MN blocks, i.e. the LBO).
template <bool A_MN, bool B_MN>
__device__ __forceinline__ void umma_product(uint32_t d_tmem, uint32_t a_saddr, uint32_t a_blk, uint32_t b_saddr,
                                             uint32_t b_blk, int N, int K, bool accumulate, bool a_neg = false) {
    const uint32_t idesc = make_idesc(128, N, A_MN, B_MN, a_neg);
    // base descriptors once; a K step only moves the 14-bit start-address field (units of 16 bytes)
    const uint64_t a0 = A_MN ? desc_mnmajor(a_saddr, a_blk) : desc_kmajor(a_saddr);
    const uint64_t b0 = B_MN ? desc_mnmajor(b_saddr, b_blk) : desc_kmajor(b_saddr);
#pragma unroll
    for (int k = 0; k < K; k += 16) {
        const uint32_t ao = A_MN ? (uint32_t)k * 128u : (uint32_t)(k >> 6) * a_blk + (uint32_t)(k & 63) * 2u;
        const uint32_t bo = B_MN ? (uint32_t)k * 128u : (uint32_t)(k >> 6) * b_blk + (uint32_t)(k & 63) * 2u;
        umma_ss(d_tmem, a0 + (uint64_t)(ao >> 4), b0 + (uint64_t)(bo >> 4), idesc, accumulate || k > 0);
    }
}

// D[tmem] (+)= A[tmem] * B[smem]: the A operand (M = 128 rows on the 128 lanes, bf16 pairs packed two per
// 32-bit column: column c of lane m holds A[m][2c], A[m][2c+1]) is read from tensor memory.
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
template <bool B_MN>
__device__ __forceinline__ void umma_product_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_saddr, uint32_t b_blk, int N,
                                                int K, bool accumulate, bool a_neg = false) {
    const uint32_t idesc = make_idesc(128, N, false, B_MN, a_neg);
    const uint64_t b0 = B_MN ? desc_mnmajor(b_saddr, b_blk) : desc_kmajor(b_saddr);
#pragma unroll
    for (int k = 0; k < K; k += 16) {
        const uint32_t bo = B_MN ? (uint32_t)k * 128u : (uint32_t)(k >> 6) * b_blk + (uint32_t)(k & 63) * 2u;
        umma_ts(d_tmem, a_tmem + (uint32_t)(k >> 1), b0 + (uint64_t)(bo >> 4), idesc, accumulate || k > 0);
    }
}

// Byte offset of element (line, e) inside a swizzled [lines][64] bf16 tile (e in 0..63).
__device__ __forceinline__ uint32_t sw128_off(uint32_t line, uint32_t e) {
    return line * 128u + ((((e >> 3) ^ line) & 7u) << 4) + ((e & 7u) << 1);
}
// Byte offset of 16-byte chunk c (0..7) of a line.
__device__ __forceinline__ uint32_t sw128_chunk(uint32_t line, uint32_t c) { return line * 128u + (((c ^ line) & 7u) << 4); }

// Shared-memory stores issued as volatile asm WITHOUT a memory clobber: the compiler keeps their
// order among themselves and relative to barriers, but is free to hoist ordinary shared-memory
// loads above them (it cannot otherwise prove that a tile store does not alias a coefficient
// array, and serialises every load behind the preceding store).  Only use for data that the
// storing thread does not read back before the next barrier.
__device__ __forceinline__ void sts128(void* p, uint4 v) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(smem_u32(p)), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w));
}
__device__ __forceinline__ void sts16(void* p, __nv_bfloat16 v) {
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(smem_u32(p)), "h"(*reinterpret_cast<unsigned short*>(&v)));
}
__device__ __forceinline__ void sts32(void* p, float v) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(smem_u32(p)), "f"(v));
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&t);
}

}  // namespace sm100

// ---- host side: tensor maps (tmap.cu) ---------------------------------------------------------------
// 2-D bf16 tensor [rows][cols] with row pitch `pitch_bytes`, boxes of [box_rows][64] elements,
// 128-byte swizzle.  Returns false if the driver entry point is missing or the encode fails.
bool make_tmap_bf16_2d(CUtensorMap* map, const void* base, uint64_t cols, uint64_t rows, uint64_t pitch_bytes,
                       uint32_t box_rows);
// 3-D map of a token-major bf16 tensor [B][T][H*D] (q, k, v, o, dO and the gradients), boxes of
// [1][box_rows][64]; coordinates (column, token, batch).
bool make_tmap_tokens(CUtensorMap* map, const void* base, int B, int T, int H, int D, uint32_t box_rows);

}  // namespace qd
