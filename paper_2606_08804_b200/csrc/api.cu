// C-ABI entry points: argument validation, workspace carving, kernel sequencing.
#include "internal.h"

#include <vector>

namespace qd {

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

WsLayout ws_layout(const qd_shape& s) {
    WsLayout L{};
    const size_t BH = (size_t)s.B * s.H, T = (size_t)simt_padded_T(s), N = T / kChunk;
    const size_t io = s.dtype == QD_BF16 ? 2 : 4;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align256(off + bytes); return o; };
    L.status = take(256);
    L.g = take(BH * T * 4);
    L.P = take(BH * T * kChunk * io);
    L.W = take(BH * T * s.dk * io);
    L.U = take(BH * T * s.dv * io);
    L.rqk = take(2 * BH * T * 4);
    L.fwd_end = off;
    L.nslices = s.dv / kSliceSimt;
    L.bwd_ctas = 296;
    L.hs = take(BH * N * s.dk * s.dv * 4);
    L.D = take(BH * T * s.dv * io);
    L.dhs = take(BH * N * s.dk * s.dv * 4);
    L.dD = take(BH * T * s.dv * io);
    L.kdhd = take((size_t)L.nslices * BH * T * 4);
    L.dhh = take((size_t)L.nslices * BH * N * 4);
    L.scratch = take((size_t)L.bwd_ctas * 6 * kChunk * s.dk * 4);
    L.bwd_end = off;
    return L;
}

int check_shape(const qd_shape* s) {
    if (!s) return QD_ERR_INVALID_ARG;
    if (s->B <= 0 || s->T <= 0 || s->H <= 0 || s->dk <= 0 || s->dv <= 0 || s->chunk <= 0) return QD_ERR_INVALID_ARG;
    if (s->dtype != QD_F32 && s->dtype != QD_BF16) return QD_ERR_UNSUPPORTED;
    if (s->chunk != kChunk) return QD_ERR_UNSUPPORTED;
    if ((s->dk != 64 && s->dk != 128) || (s->dv != 64 && s->dv != 128)) return QD_ERR_UNSUPPORTED;
    if ((long long)s->B * s->H * ((s->T + 127) / 128 * 2) > 0x7fffffffLL / 4) return QD_ERR_UNSUPPORTED;
    return QD_OK;
}

static bool misaligned(const void* p) { return ((uintptr_t)p & 15) != 0; }

// ---- optional per-stage timing with CUDA events on the launching stream ------------------------
enum Stage { ST_PREP = 0, ST_CHAIN_FWD, ST_CHAIN_BWD, ST_CHUNK_BWD, ST_DECODE, ST_COUNT };
static const char* kStageNames[ST_COUNT] = {"prep", "chain_fwd", "chain_bwd", "chunk_bwd", "decode"};
struct Pending { cudaEvent_t a, b; int stage; };
static bool g_profile = false;
static std::vector<Pending> g_pending;
static std::vector<cudaEvent_t> g_pool;
static double g_ms[ST_COUNT];
static long long g_launches[ST_COUNT];

static cudaEvent_t get_event() {
    cudaEvent_t e = nullptr;
    if (!g_pool.empty()) { e = g_pool.back(); g_pool.pop_back(); return e; }
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    return e;
}

// Brackets one kernel launch with two events when profiling is on.
struct StageTimer {
    cudaEvent_t a = nullptr, b = nullptr;
    int stage; cudaStream_t s;
    StageTimer(int stage_, cudaStream_t s_) : stage(stage_), s(s_) {
        if (!g_profile) return;
        a = get_event(); b = get_event();
        if (a && b) cudaEventRecord(a, s);
    }
    ~StageTimer() {
        if (!g_profile || !a || !b) return;
        cudaEventRecord(b, s);
        g_pending.push_back({a, b, stage});
    }
};

template <class F> static cudaError_t timed(int stage, cudaStream_t s, F f) {
    StageTimer t(stage, s);
    return f();
}

}  // namespace qd

using namespace qd;

extern "C" {

size_t qdelta_chunk_workspace_bytes(const qd_shape* shape, int for_backward) {
    if (check_shape(shape) != QD_OK) return 0;
    // the tensor-core path and the fp32 path lay the workspace out differently; a shape takes exactly one of them
    if (tc_supported(*shape)) {
        TcLayout TL = tc_layout(*shape);
        return for_backward ? TL.bwd_end : TL.fwd_end;
    }
    WsLayout L = ws_layout(*shape);
    return for_backward ? L.bwd_end : L.fwd_end;
}

int qdelta_chunk_path(const qd_shape* shape) {
    if (check_shape(shape) != QD_OK) return -1;
    return tc_supported(*shape) ? 1 : 0;
}

int qdelta_chunk_fwd(const qd_shape* shape, const void* q, const void* k, const void* v, const void* beta,
                     const void* alpha, const void* lambda, const float* h0, void* o, float* hT,
                     void* workspace, size_t workspace_bytes, unsigned flags, qd_stream stream) {
    int rc = check_shape(shape);
    if (rc != QD_OK) return rc;
    if (!q || !k || !v || !beta || !o) return QD_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k, v, h0, o, hT, workspace};
    for (const void* p : ptrs)
        if (p && misaligned(p)) return QD_ERR_INVALID_ARG;
    const void* coef[] = {beta, alpha, lambda};
    for (const void* p : coef)
        if (p && ((uintptr_t)p & (shape->dtype == QD_BF16 ? 1 : 3))) return QD_ERR_INVALID_ARG;
    if (flags & ~(unsigned)(QD_FWD_SAVE_FOR_BWD | QD_COEF_LOGITS | QD_NORM_QK)) return QD_ERR_INVALID_ARG;
    ChunkArgs a{};
    a.s = *shape;
    a.L = ws_layout(*shape);
    a.save = (flags & QD_FWD_SAVE_FOR_BWD) != 0;
    a.logits = (flags & QD_COEF_LOGITS) != 0;
    a.norm = (flags & QD_NORM_QK) != 0;
    if (!workspace || workspace_bytes < qdelta_chunk_workspace_bytes(shape, a.save ? 1 : 0)) return QD_ERR_WORKSPACE;
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.alpha = alpha; a.lam = lambda; a.h0 = h0; a.o = o; a.hT = hT;
    a.ws = (char*)workspace;
    a.stream = (cudaStream_t)stream;
    if (cudaMemsetAsync(a.ws + a.L.status, 0, 256, a.stream) != cudaSuccess) return QD_ERR_CUDA;   // offset 0 in both layouts
    if (tc_supported(*shape)) {
        a.TL = tc_layout(*shape);
        if (timed(ST_PREP, a.stream, [&] { return tc_prep(a); }) != cudaSuccess) return QD_ERR_CUDA;
        if (timed(ST_CHAIN_FWD, a.stream, [&] { return tc_chain_fwd(a); }) != cudaSuccess) return QD_ERR_CUDA;
        return QD_OK;
    }
    if (timed(ST_PREP, a.stream, [&] { return simt_prep(a); }) != cudaSuccess) return QD_ERR_CUDA;
    if (timed(ST_CHAIN_FWD, a.stream, [&] { return simt_chain_fwd(a); }) != cudaSuccess) return QD_ERR_CUDA;
    return QD_OK;
}

int qdelta_chunk_bwd(const qd_shape* shape, const void* q, const void* k, const void* v, const void* beta,
                     const void* alpha, const void* lambda, const float* h0, const void* dO, const float* dhT,
                     void* dq, void* dk, void* dv, float* dbeta, float* dalpha, float* dlambda, float* dh0,
                     void* workspace, size_t workspace_bytes, unsigned flags, qd_stream stream) {
    int rc = check_shape(shape);
    if (rc != QD_OK) return rc;
    if (!q || !k || !v || !beta || !dO || !dq || !dk || !dv || !dbeta) return QD_ERR_INVALID_ARG;
    if ((alpha && !dalpha) || (lambda && !dlambda)) return QD_ERR_INVALID_ARG;
    const void* ptrs[] = {q, k, v, h0, dO, dhT, dq, dk, dv, dh0, workspace};
    for (const void* p : ptrs)
        if (p && misaligned(p)) return QD_ERR_INVALID_ARG;
    const void* coef[] = {beta, alpha, lambda};
    for (const void* p : coef)
        if (p && ((uintptr_t)p & (shape->dtype == QD_BF16 ? 1 : 3))) return QD_ERR_INVALID_ARG;
    const void* gcoef[] = {dbeta, dalpha, dlambda};
    for (const void* p : gcoef)
        if (p && ((uintptr_t)p & 3)) return QD_ERR_INVALID_ARG;
    if (flags & ~(unsigned)(QD_BWD_REUSE_FWD | QD_COEF_LOGITS | QD_NORM_QK)) return QD_ERR_INVALID_ARG;
    ChunkArgs a{};
    a.s = *shape;
    a.L = ws_layout(*shape);
    a.save = true;
    a.logits = (flags & QD_COEF_LOGITS) != 0;
    a.norm = (flags & QD_NORM_QK) != 0;
    if (!workspace || workspace_bytes < qdelta_chunk_workspace_bytes(shape, 1)) return QD_ERR_WORKSPACE;
    a.q = q; a.k = k; a.v = v; a.beta = beta; a.alpha = alpha; a.lam = lambda; a.h0 = h0;
    a.dO = dO; a.dhT = dhT; a.dq = dq; a.dk = dk; a.dv = dv;
    a.dbeta = dbeta; a.dalpha = dalpha; a.dlam = dlambda; a.dh0 = dh0;
    a.ws = (char*)workspace;
    a.stream = (cudaStream_t)stream;
    if (tc_supported(*shape)) {
        a.TL = tc_layout(*shape);
        if (!(flags & QD_BWD_REUSE_FWD)) {
            // recompute what a saving forward leaves behind; its o goes to the dDelta section, which
            // the reverse chain overwrites afterwards
            if (cudaMemsetAsync(a.ws + a.TL.status, 0, 256, a.stream) != cudaSuccess) return QD_ERR_CUDA;
            a.o = a.ws + a.TL.dDt;
            a.hT = nullptr;
            if (timed(ST_PREP, a.stream, [&] { return tc_prep(a); }) != cudaSuccess) return QD_ERR_CUDA;
            if (timed(ST_CHAIN_FWD, a.stream, [&] { return tc_chain_fwd(a); }) != cudaSuccess) return QD_ERR_CUDA;
            a.own_predecessor = true;      // the reverse chain follows this library's forward chain in the stream
        }
        if (timed(ST_CHAIN_BWD, a.stream, [&] { return tc_chain_bwd(a); }) != cudaSuccess) return QD_ERR_CUDA;
        if (timed(ST_CHUNK_BWD, a.stream, [&] { return tc_chunk_bwd(a); }) != cudaSuccess) return QD_ERR_CUDA;
        return QD_OK;
    }
    if (!(flags & QD_BWD_REUSE_FWD)) {
        // recompute the forward intermediates (outputs of the forward itself are not rewritten:
        // o goes to the dD section, which the reverse chain overwrites afterwards)
        if (cudaMemsetAsync(a.ws + a.L.status, 0, 256, a.stream) != cudaSuccess) return QD_ERR_CUDA;
        a.o = a.ws + a.L.dD;
        a.hT = nullptr;
        if (timed(ST_PREP, a.stream, [&] { return simt_prep(a); }) != cudaSuccess) return QD_ERR_CUDA;
        if (timed(ST_CHAIN_FWD, a.stream, [&] { return simt_chain_fwd(a); }) != cudaSuccess) return QD_ERR_CUDA;
    }
    if (timed(ST_CHAIN_BWD, a.stream, [&] { return simt_chain_bwd(a); }) != cudaSuccess) return QD_ERR_CUDA;
    if (timed(ST_CHUNK_BWD, a.stream, [&] { return simt_chunk_bwd(a); }) != cudaSuccess) return QD_ERR_CUDA;
    return QD_OK;
}

int qdelta_recurrent_step(int B, int H, int dk, int dv, int dtype, const void* q, const void* k, const void* v,
                          const void* beta, const void* alpha, const void* lambda, float* state, void* o,
                          qd_stream stream) {
    if (B <= 0 || H <= 0) return QD_ERR_INVALID_ARG;
    if (dtype != QD_F32 && dtype != QD_BF16) return QD_ERR_UNSUPPORTED;
    if ((dk != 64 && dk != 128) || (dv != 64 && dv != 128)) return QD_ERR_UNSUPPORTED;
    if (!q || !k || !v || !beta || !state || !o) return QD_ERR_INVALID_ARG;
    if ((long long)B * H > 0x3fffffffLL) return QD_ERR_UNSUPPORTED;
    const void* ptrs[] = {q, k, v, state};
    for (const void* p : ptrs)
        if (p && misaligned(p)) return QD_ERR_INVALID_ARG;
    const void* coef[] = {beta, alpha, lambda, o};
    for (const void* p : coef)
        if (p && ((uintptr_t)p & (dtype == QD_BF16 ? 1 : 3))) return QD_ERR_INVALID_ARG;
    if (timed(ST_DECODE, (cudaStream_t)stream, [&] {
            return decode_step(B * H, dk, dv, dtype, q, k, v, beta, alpha, lambda, state, o, (cudaStream_t)stream);
        }) != cudaSuccess)
        return QD_ERR_CUDA;
    return QD_OK;
}

int qdelta_recurrent_steps(int B, int S, int H, int dk, int dv, int dtype, const void* q, const void* k, const void* v,
                           const void* beta, const void* alpha, const void* lambda, void* state, void* o,
                           unsigned flags, qd_stream stream) {
    if (B <= 0 || H <= 0 || S <= 0) return QD_ERR_INVALID_ARG;
    if (flags & ~(unsigned)(QD_COEF_LOGITS | QD_NORM_QK | QD_STATE_BF16)) return QD_ERR_INVALID_ARG;
    if (dtype != QD_F32 && dtype != QD_BF16) return QD_ERR_UNSUPPORTED;
    if ((dk != 64 && dk != 128) || (dv != 64 && dv != 128)) return QD_ERR_UNSUPPORTED;
    if (!q || !k || !v || !beta || !state || !o) return QD_ERR_INVALID_ARG;
    if ((long long)B * H > 0x3fffffffLL || (long long)B * S * H > 0x7fffffffLL / 128) return QD_ERR_UNSUPPORTED;
    const void* ptrs[] = {q, k, v, state};
    for (const void* p : ptrs)
        if (p && misaligned(p)) return QD_ERR_INVALID_ARG;
    const void* coef[] = {beta, alpha, lambda, o};
    for (const void* p : coef)
        if (p && ((uintptr_t)p & (dtype == QD_BF16 ? 1 : 3))) return QD_ERR_INVALID_ARG;
    if (timed(ST_DECODE, (cudaStream_t)stream, [&] {
            return decode_steps(B, S, H, dk, dv, dtype, q, k, v, beta, alpha, lambda, state, o,
                                (flags & QD_COEF_LOGITS) != 0, (flags & QD_NORM_QK) != 0, (flags & QD_STATE_BF16) != 0,
                                (cudaStream_t)stream);
        }) != cudaSuccess)
        return QD_ERR_CUDA;
    return QD_OK;
}

int qdelta_workspace_status(const void* workspace, int* status_out, qd_stream stream) {
    if (!workspace || !status_out) return QD_ERR_INVALID_ARG;
    unsigned w = 0;
    if (cudaMemcpyAsync(&w, workspace, 4, cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess) return QD_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return QD_ERR_CUDA;
    *status_out = (int)w;
    return QD_OK;
}

int qdelta_profile_enable(int on) {
    g_profile = on != 0;
    return QD_OK;
}

int qdelta_profile_stage_count(void) { return ST_COUNT; }

const char* qdelta_profile_stage_name(int stage) {
    return (stage >= 0 && stage < ST_COUNT) ? kStageNames[stage] : "";
}

int qdelta_profile_read(int stage, double* total_ms, long long* launches, int reset) {
    if (stage < 0 || stage >= ST_COUNT || !total_ms || !launches) return QD_ERR_INVALID_ARG;
    for (const Pending& p : g_pending) {
        float ms = 0.f;
        if (cudaEventSynchronize(p.b) != cudaSuccess || cudaEventElapsedTime(&ms, p.a, p.b) != cudaSuccess)
            return QD_ERR_CUDA;
        g_ms[p.stage] += ms;
        g_launches[p.stage] += 1;
        g_pool.push_back(p.a);
        g_pool.push_back(p.b);
    }
    g_pending.clear();
    *total_ms = g_ms[stage];
    *launches = g_launches[stage];
    if (reset) { g_ms[stage] = 0.0; g_launches[stage] = 0; }
    return QD_OK;
}

const char* qdelta_status_string(int status) {
    switch (status) {
        case QD_OK: return "QD_OK";
        case QD_ERR_INVALID_ARG: return "QD_ERR_INVALID_ARG";
        case QD_ERR_UNSUPPORTED: return "QD_ERR_UNSUPPORTED";
        case QD_ERR_WORKSPACE: return "QD_ERR_WORKSPACE";
        case QD_ERR_CUDA: return "QD_ERR_CUDA";
        case QD_ERR_TIMEOUT: return "QD_ERR_TIMEOUT";
        case QD_ERR_STATIC_SCRATCH: return "QD_ERR_STATIC_SCRATCH (shape needs more than the built-in scratch array)";
        default: return "QD_ERR_UNKNOWN";
    }
}

}  // extern "C"
